"""Helpers for the GPU parity tests (all calls go through the C-ABI binding)."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")


def require_gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_33762_b200 import build
    build.build()


def make_ctx(shape, gpu_blocks, host_blocks, pool, **kw):
    from paper_2609_33762_b200 import eakv
    return eakv.Context(num_layers=shape.num_layers, kv_heads=shape.kv_heads,
                        head_dim=shape.head_dim, block_size=shape.block_size,
                        elem_bytes=shape.elem_bytes, gpu_blocks=gpu_blocks,
                        host_blocks=host_blocks, kv_base=[t.data_ptr() for t in pool], **kw)


def hash_ctx(block_size, **kw):
    """A context whose only purpose is hashing (tiny pool and tier)."""
    from eakv_workloads import KVShape
    shape = KVShape(1, 1, 8, block_size)
    pool = [torch.zeros((1, shape.piece_bytes // 2), dtype=torch.int16, device="cuda")
            for _ in range(2)]
    ctx = make_ctx(shape, 1, 1, pool, **kw)
    ctx._keep = pool
    return ctx


def gpu_keys(ctx, tokens, parent=None, offset_tokens=0):
    """Run eakv_hash_blocks on a token list; returns Python ints."""
    tokens = np.asarray(tokens, dtype=np.int32)
    pad = np.zeros(offset_tokens, dtype=np.int32)
    dev = torch.from_numpy(np.concatenate([pad, tokens])).cuda()
    nblk = len(tokens) // ctx.block_size
    out = torch.full((max(nblk, 1) + 1,), -1, dtype=torch.int64, device="cuda")
    parent = ctx.eakv_hash_seed() if parent is None else parent
    got = ctx.eakv_hash_blocks(dev.data_ptr() + 4 * offset_tokens, len(tokens), parent,
                               out.data_ptr())
    torch.cuda.synchronize()
    assert got == nblk
    res = out.cpu().numpy()
    assert res[nblk] == -1          # nothing written past the last key
    return [int(x) for x in res[:nblk].view(np.uint64)]
