"""Parity at the benchmark's full size and launch configuration: 4,096 blocks of 1.5 MiB per
call over a 65,536-block (96 GiB) paged pool, uniform-random block ids, default copy path,
tier in HBM and in pinned host memory.  The oracle computes sampled outputs one by one; the
rest is covered by a device-side property (every stored slot equals its source block)."""
import numpy as np
import pytest

from eakv_workloads import SHAPES, counter_words_at_torch, counter_words_numpy, counter_words_torch
from oracle import hash as ohash
from oracle import storeload as osl

from gpu_util import require_gpu, torch

pytestmark = pytest.mark.gpu

M = 4096
POOL = 65536
SALT = 1000


@pytest.fixture(scope="module")
def pool():
    require_gpu()
    from paper_2609_33762_b200.harness import PagedPool
    shape = SHAPES["qwen3_30b_a3b"]
    free, _ = torch.cuda.mem_get_info()
    nb = POOL
    need = (nb + 3 * M) * shape.block_bytes + (8 << 30)
    if free < need:
        nb = int((free - (8 << 30)) // shape.block_bytes) - 3 * M
        if nb < 4 * M:
            pytest.skip("not enough free device memory for the full-size case")
    W = shape.piece_bytes // 2

    def fill(q, t):
        step = 4096
        for b0 in range(0, nb, step):
            b1 = min(nb, b0 + step)
            t[b0:b1] = counter_words_torch(SALT + q, b0 * W, (b1 - b0) * W, t.device).view(b1 - b0, W)

    p = PagedPool(shape, nb, "cuda:0", fill=fill)
    torch.cuda.synchronize()
    return p


def expected_block(shape, blk, q):
    W = shape.piece_bytes // 2
    return counter_words_numpy(SALT + q, blk * W, W).view(np.uint8)


def oracle_slots_for_sample(shape, table, slots, sample):
    """Run the oracle's store on a compact pool holding just the sampled blocks."""
    Q, P = shape.pieces_per_block, shape.piece_bytes
    mini_pool = [np.stack([expected_block(shape, int(table[j]), q) for j in sample]) for q in range(Q)]
    mini_tier = np.zeros((len(sample), Q, P), dtype=np.uint8)
    osl.store(mini_pool, mini_tier, list(range(len(sample))), [1] * len(sample), list(range(len(sample))))
    return mini_tier          # mini_tier[i] is what slot slots[sample[i]] must hold


@pytest.mark.parametrize("where", ["hbm", "host_staged", "host_zero_copy"])
def test_full_size_store_load(pool, where):
    from paper_2609_33762_b200 import eakv
    shape = pool.shape
    nb = pool.gpu_blocks
    rng = np.random.default_rng(17)
    perm = rng.permutation(nb)
    table = perm[:M].astype(np.int32)                 # sources of the store
    dest = perm[M:2 * M].astype(np.int32)             # fresh blocks for the load
    slots = rng.permutation(M).astype(np.int32)
    Q, W = shape.pieces_per_block, shape.piece_bytes // 2
    kw = dict(tier_location=eakv.TIER_PINNED_HOST)
    tier_t = None
    if where == "hbm":
        tier_t = torch.zeros((M, Q, W), dtype=torch.int16, device="cuda")
        kw = dict(tier_location=eakv.TIER_DEVICE, tier_memory=tier_t.data_ptr())
    elif where == "host_zero_copy":
        kw["link_strategy"] = eakv.LINK_ZERO_COPY
    else:
        kw["min_staged_run_bytes"] = -1               # random slots, yet through the staging path
    ctx = eakv.Context(num_layers=shape.num_layers, kv_heads=shape.kv_heads, head_dim=shape.head_dim,
                       block_size=shape.block_size, gpu_blocks=nb, host_blocks=M,
                       kv_base=pool.kv_base, **kw)
    ctx.eakv_store(table, None, slots)
    ctx.eakv_sync()
    sample = sorted(set(np.linspace(0, M - 1, 24).astype(int).tolist() + [0, 1, M - 2, M - 1]))
    want = oracle_slots_for_sample(shape, table, slots, sample)
    if tier_t is not None:
        got = tier_t[torch.as_tensor(slots[sample].astype(np.int64), device="cuda")].cpu().numpy().view(np.uint8)
    else:
        got = ctx.tier_host_view()[slots[sample]]
    assert np.array_equal(got.reshape(want.shape), want)
    if tier_t is not None:                            # property over every slot, on the device
        idx_s = torch.as_tensor(slots.astype(np.int64), device="cuda")
        idx_b = torch.as_tensor(table.astype(np.int64), device="cuda")
        for q in (0, Q // 2, Q - 1):
            assert torch.equal(tier_t[idx_s, q], pool.pieces[q][idx_b])
    # load into fresh blocks: sampled destinations equal the oracle's bytes of the source block
    ctx.eakv_load(slots, dest)
    ctx.eakv_sync()
    for j in sample[::3]:
        for q in (0, Q - 1):
            got_blk = pool.pieces[q][int(dest[j])].cpu().numpy().view(np.uint8)
            assert np.array_equal(got_blk, expected_block(shape, int(table[j]), q))
    idx_d = torch.as_tensor(dest.astype(np.int64), device="cuda")
    idx_b = torch.as_tensor(table.astype(np.int64), device="cuda")
    for q in (1, Q - 2):
        assert torch.equal(pool.pieces[q][idx_d], pool.pieces[q][idx_b])
    ctx.close()
    # restore the overwritten destination blocks so the next variant sees the seeded pool
    ids = torch.as_tensor(dest.astype(np.int64), device="cuda")
    col = torch.arange(W, dtype=torch.int64, device="cuda").reshape(1, -1)
    for q, t in enumerate(pool.pieces):
        for j in range(0, M, 1024):
            start = ids[j:j + 1024].reshape(-1, 1) * W + col
            t[ids[j:j + 1024]] = counter_words_at_torch(SALT + q, start)


def test_full_size_hash_64k_prompt_and_batch():
    require_gpu()
    from gpu_util import hash_ctx
    rng = np.random.default_rng(18)
    ctx = hash_ctx(16, hash_scratch_blocks=1 << 17)
    n = 65536
    toks = rng.integers(0, 151936, size=n, dtype=np.int32)
    dev = torch.from_numpy(toks).cuda()
    out = torch.zeros(n // 16, dtype=torch.int64, device="cuda")
    ctx.eakv_hash_blocks(dev.data_ptr(), n, ctx.eakv_hash_seed(), out.data_ptr())
    torch.cuda.synchronize()
    assert [int(x) for x in out.cpu().numpy().view(np.uint64)] == ohash.hash_blocks(toks.tolist(), 16)
    # a batch of 24 prompts of that length: sampled prompts checked in full
    P = 24
    big = rng.integers(0, 151936, size=P * n, dtype=np.int32)
    dev = torch.from_numpy(big).cuda()
    out = torch.zeros(P * n // 16, dtype=torch.int64, device="cuda")
    offsets = np.arange(P + 1, dtype=np.int64) * n
    boff = ctx.eakv_hash_blocks_batched(dev.data_ptr(), offsets, None, out.data_ptr())
    torch.cuda.synchronize()
    res = out.cpu().numpy().view(np.uint64)
    for i in (0, 11, 23):
        assert [int(x) for x in res[boff[i]:boff[i + 1]]] == ohash.hash_blocks(big[i * n:(i + 1) * n].tolist(), 16)
    ctx.close()
