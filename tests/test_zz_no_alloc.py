"""The allocation-free entry point eakv_hash_blocks_static against the CPU oracle and against
eakv_hash_blocks.  It exists for callers that cannot request device memory (for instance code
running inside a serving process whose engine already owns the GPU's memory): its scratch is
a fixed array inside the library that all calls share, so every case here makes two calls in a
row with different inputs and checks both, bit for bit.  The file sorts last on purpose: a run
that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest

from gpu_util import hash_ctx, require_gpu, torch
from oracle import hash as ohash

pytestmark = pytest.mark.gpu


def keys_via_context(ctx, dev_tokens, n, parent):
    out = torch.zeros(max(n // ctx.block_size, 1), dtype=torch.int64, device="cuda")
    got = ctx.eakv_hash_blocks(dev_tokens.data_ptr(), n, parent, out.data_ptr())
    torch.cuda.synchronize()
    return out.cpu().numpy()[:got].view(np.uint64).copy()


def keys_via_static(eakv, dev_tokens, n, b, base, parent):
    out = torch.full((max(n // b, 1) + 1,), -1, dtype=torch.int64, device="cuda")
    got = eakv.eakv_hash_blocks_static(dev_tokens.data_ptr(), n, b, base, parent, out.data_ptr())
    torch.cuda.synchronize()
    res = out.cpu().numpy()
    assert res[got] == -1                       # nothing written past the last key
    return res[:got].view(np.uint64).copy()


# block sizes that reach every kernel behind the entry point: 16/32/64 (compile-time staged
# kernels), 12 (staged kernel with a run-time block size), 10 and 66 (one thread per block,
# scalar loads), 128 and 1024 (a group of threads per block, power table read on the device)
@pytest.mark.parametrize("b", [16, 32, 64, 12, 10, 66, 128, 1024])
def test_static_scratch_variant_equals_the_oracle_twice_in_a_row(b):
    require_gpu()
    from paper_2609_33762_b200 import eakv
    rng = np.random.default_rng(99 + b)
    ctx = hash_ctx(b)
    base, seed = ctx.eakv_hash_base(), ctx.eakv_hash_seed()
    assert (base, seed) == (ohash.HASH_BASE, ohash.HASH_SEED)
    # two calls back to back: the second is shorter and starts from another parent, so
    # anything left over from the first (partials, counter, power table) would show
    for n, parent in ((b * 3000 + 7, seed), (b * 37 + 1, 12345)):
        tok_np = rng.integers(0, 151936, size=n, dtype=np.int32)
        toks = torch.from_numpy(tok_np).cuda()
        want = np.array(ohash.hash_blocks(tok_np.tolist(), b, parent, base), dtype=np.uint64)
        got = keys_via_static(eakv, toks, n, b, base, parent)
        assert len(got) == n // b and np.array_equal(got, want), (b, n)
        assert np.array_equal(keys_via_context(ctx, toks, n, parent), want)
    ctx.close()
    eakv.eakv_hash_blocks_static_status()        # no self-check tripped


def test_static_variant_rebuilds_its_power_table_for_another_base():
    require_gpu()
    from paper_2609_33762_b200 import eakv
    rng = np.random.default_rng(7)
    for b, base in ((16, 987654321), (256, 3), (16, 0)):
        tok_np = rng.integers(0, 151936, size=b * 300, dtype=np.int32)
        toks = torch.from_numpy(tok_np).cuda()
        want = np.array(ohash.hash_blocks(tok_np.tolist(), b, 7, base or ohash.HASH_BASE), dtype=np.uint64)
        assert np.array_equal(keys_via_static(eakv, toks, b * 300, b, base, 7), want)
    eakv.eakv_hash_blocks_static_status()


def test_static_variant_rejects_what_its_scratch_cannot_hold():
    require_gpu()
    from paper_2609_33762_b200 import eakv
    b = 4
    n = (eakv.STATIC_MAX_BLOCKS + 1) * b
    tok_np = np.random.default_rng(3).integers(0, 151936, size=n, dtype=np.int32)
    toks = torch.from_numpy(tok_np).cuda()
    out = torch.zeros(eakv.STATIC_MAX_BLOCKS + 1, dtype=torch.int64, device="cuda")
    with pytest.raises(eakv.EakvError) as ei:
        eakv.eakv_hash_blocks_static(toks.data_ptr(), n, b, 0, 1, out.data_ptr())
    assert ei.value.code == eakv.E_CAPACITY
    # exactly the maximum is accepted (and right); too-large block sizes and null buffers are refused
    assert eakv.eakv_hash_blocks_static(toks.data_ptr(), n - b, b, 0, 1, out.data_ptr()) == eakv.STATIC_MAX_BLOCKS
    torch.cuda.synchronize()
    want = np.array(ohash.hash_blocks(tok_np[:n - b].tolist(), b, 1), dtype=np.uint64)
    assert np.array_equal(out.cpu().numpy()[:-1].view(np.uint64), want)
    for args in ((toks.data_ptr(), 64, 8192, 0, 1, out.data_ptr()), (0, 64, 16, 0, 1, out.data_ptr())):
        with pytest.raises(eakv.EakvError) as ei:
            eakv.eakv_hash_blocks_static(*args)
        assert ei.value.code == eakv.E_INVAL
    eakv.eakv_hash_blocks_static_status()
