"""GPU parity: eakv_hash_blocks / eakv_hash_blocks_batched against oracle.hash, bit-exact."""
import numpy as np
import pytest

from oracle import hash as oh

from gpu_util import gpu_keys, hash_ctx, require_gpu, torch

pytestmark = pytest.mark.gpu
P = (1 << 61) - 1


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


@pytest.mark.parametrize("b", [16, 32, 4, 12, 10, 1, 1024, 256])
def test_lengths_and_block_sizes(b):
    rng = np.random.default_rng(b)
    ctx = hash_ctx(b)
    lengths = [0, 1, b - 1, b, b + 1, 31, 32, 33, 1023, 1024, 1025, 4095, 4096, 4097,
               5 * 4096 + 3 * b + 1, 131072]
    for n in lengths:
        if n < 0:
            continue
        toks = rng.integers(0, 151936, size=n, dtype=np.int32)
        assert gpu_keys(ctx, toks) == oh.hash_blocks(toks.tolist(), b), (b, n)
    ctx.close()


def test_extreme_token_ids_and_parents():
    ctx = hash_ctx(16)
    hi = np.full(16 * 40 + 5, 2**31 - 1, dtype=np.int32)
    zero = np.zeros(16 * 40, dtype=np.int32)
    for toks in (hi, zero):
        for parent in (0, 1, P - 1, oh.HASH_SEED):
            assert gpu_keys(ctx, toks, parent) == oh.hash_blocks(toks.tolist(), 16, parent)
    # parents at or above p are reduced first
    toks = np.arange(64, dtype=np.int32)
    assert gpu_keys(ctx, toks, P + 5) == oh.hash_blocks(toks.tolist(), 16, 5)
    ctx.close()


def test_canonical_zero_key():
    # pick the parent so that the first block's key is exactly 0 (never p)
    b = 4
    ctx = hash_ctx(b)
    B = oh.HASH_BASE
    toks = [7, 0, 151935, 3, 9, 9, 9, 9]
    c = 0
    for t in toks[:b]:
        c = (c * B + t + 1) % P
    parent = (-c * pow(pow(B, b, P), P - 2, P)) % P
    keys = gpu_keys(ctx, toks, parent)
    assert keys[0] == 0
    assert keys == oh.hash_blocks(toks, b, parent)
    ctx.close()


def test_resume_and_unaligned_pointers():
    b = 16
    ctx = hash_ctx(b)
    rng = np.random.default_rng(3)
    toks = rng.integers(0, 151936, size=b * 300 + 7, dtype=np.int32)
    full = oh.hash_blocks(toks.tolist(), b)
    assert gpu_keys(ctx, toks) == full
    for j in (1, 2, 255, 256, 257, 299):
        assert gpu_keys(ctx, toks[j * b:], parent=full[j - 1]) == full[j:]
    # token pointer only 4-byte aligned: scalar load path
    for off in (1, 2, 3):
        assert gpu_keys(ctx, toks, offset_tokens=off) == full
    ctx.close()


def test_scratch_smaller_than_prompt_chains_launches():
    b = 16
    ctx = hash_ctx(b, hash_scratch_blocks=300)
    rng = np.random.default_rng(4)
    toks = rng.integers(0, 151936, size=b * 1000 + 3, dtype=np.int32)
    assert gpu_keys(ctx, toks) == oh.hash_blocks(toks.tolist(), b)
    ctx.close()


@pytest.mark.parametrize("b", [16, 32, 10])
def test_batched_ragged(b):
    ctx = hash_ctx(b)
    rng = np.random.default_rng(5 + b)
    lens = [0, 1, b - 1, b, 3 * b + 1, 4096, 4096 + b, 9000, 0, 70000, b * 256, 5]
    if b % 4 == 0:
        lens = [x - x % 4 if i % 2 == 0 else x for i, x in enumerate(lens)]   # some aligned starts
    offsets = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    toks = rng.integers(0, 151936, size=int(offsets[-1]), dtype=np.int32)
    parents = [int(x) for x in rng.integers(0, P, size=len(lens), dtype=np.uint64)]
    dev = torch.from_numpy(toks).cuda()
    total = sum(x // b for x in lens)
    for par in (None, parents):
        out = torch.full((total + 1,), -1, dtype=torch.int64, device="cuda")
        boff = ctx.eakv_hash_blocks_batched(dev.data_ptr(), offsets, par, out.data_ptr())
        torch.cuda.synchronize()
        res = out.cpu().numpy()
        assert res[total] == -1
        assert boff.tolist() == np.concatenate([[0], np.cumsum([x // b for x in lens])]).tolist()
        for i, n in enumerate(lens):
            p = oh.HASH_SEED if par is None else par[i]
            expect = oh.hash_blocks(toks[offsets[i]:offsets[i + 1]].tolist(), b, p)
            got = [int(x) for x in res[boff[i]:boff[i + 1]].view(np.uint64)]
            assert got == expect, (b, i, n)
    ctx.close()


def test_batched_many_prompts_back_to_back():
    # ticket counters must return to zero after every launch
    b = 16
    ctx = hash_ctx(b)
    rng = np.random.default_rng(6)
    lens = rng.integers(0, 3000, size=200)
    offsets = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    toks = rng.integers(0, 151936, size=int(offsets[-1]), dtype=np.int32)
    dev = torch.from_numpy(toks).cuda()
    total = int(sum(x // b for x in lens))
    expect = []
    for i in range(len(lens)):
        expect += oh.hash_blocks(toks[offsets[i]:offsets[i + 1]].tolist(), b)
    for _ in range(3):
        out = torch.zeros(total, dtype=torch.int64, device="cuda")
        ctx.eakv_hash_blocks_batched(dev.data_ptr(), offsets, None, out.data_ptr())
        torch.cuda.synchronize()
        assert [int(x) for x in out.cpu().numpy().view(np.uint64)] == expect
    ctx.close()


def test_modular_multiply_edge_operands():
    """With block size 1 the first key is parent * B + x, so base and parent choose the
    multiplier's operands directly: (p-1)^2, (p-1)*1, 2^60 * 2 == 1, 0 * x, 1 * 1."""
    for base in (P - 1, 1 << 60, 1, 2, P - 2):
        ctx = hash_ctx(1, hash_base=base, hash_seed=1)
        assert ctx.eakv_hash_base() == base
        for parent in (P - 1, 0, 1, 2, 1 << 60, P - 2):
            for toks in ([0], [2**31 - 1], [5, 0, 151935, 7]):
                assert gpu_keys(ctx, toks, parent) == oh.hash_blocks(toks, 1, parent, base), (base, parent)
        ctx.close()
    # by hand: (p-1)*(p-1) + 1 == 2 and 2^60*2 + 1 == 2 (mod p)
    ctx = hash_ctx(1, hash_base=P - 1, hash_seed=1)
    assert gpu_keys(ctx, [0], P - 1) == [2]
    ctx.close()
    ctx = hash_ctx(1, hash_base=1 << 60, hash_seed=1)
    assert gpu_keys(ctx, [0], 2) == [2]
    ctx.close()
    # the same operands through the block scan of a multi-block prompt (A = B^b)
    for b, base in ((16, P - 1), (4, 1 << 60)):
        ctx = hash_ctx(b, hash_base=base, hash_seed=1)
        toks = np.full(b * 600 + 3, 2**31 - 1, dtype=np.int32)
        assert gpu_keys(ctx, toks, P - 1) == oh.hash_blocks(toks.tolist(), b, P - 1, base)
        ctx.close()


def test_custom_base_and_seed():
    ctx = hash_ctx(16, hash_base=1234567891011, hash_seed=42)
    assert ctx.eakv_hash_base() == 1234567891011 and ctx.eakv_hash_seed() == 42
    toks = np.arange(100, dtype=np.int32)
    assert gpu_keys(ctx, toks) == oh.hash_blocks(toks.tolist(), 16, 42, 1234567891011)
    ctx.close()


def test_batched_capacity_errors_and_empty_batches():
    from paper_2609_33762_b200 import eakv
    ctx = hash_ctx(16, hash_scratch_blocks=64, max_call_blocks=8)
    toks = torch.zeros(16 * 100, dtype=torch.int32, device="cuda")
    out = torch.zeros(100, dtype=torch.int64, device="cuda")
    with pytest.raises(eakv.EakvError) as ei:           # 100 blocks > 64 blocks of scratch
        ctx.eakv_hash_blocks_batched(toks.data_ptr(), [0, 1600], None, out.data_ptr())
    assert ei.value.code == eakv.E_CAPACITY
    with pytest.raises(eakv.EakvError) as ei:           # 9 prompts > 8
        ctx.eakv_hash_blocks_batched(toks.data_ptr(), list(range(0, 160, 16)), None, out.data_ptr())
    assert ei.value.code == eakv.E_CAPACITY
    with pytest.raises(eakv.EakvError) as ei:           # offsets must not decrease
        ctx.eakv_hash_blocks_batched(toks.data_ptr(), [0, 64, 32], None, out.data_ptr())
    assert ei.value.code == eakv.E_INVAL
    assert ctx.eakv_hash_blocks_batched(toks.data_ptr(), [0], None, out.data_ptr()).tolist() == [0]
    assert ctx.eakv_hash_blocks_batched(toks.data_ptr(), [0, 5, 9], None, out.data_ptr()).tolist() == [0, 0, 0]
    # the single-prompt call still works afterwards, chained over the small scratch
    t = np.arange(1600, dtype=np.int32)
    assert gpu_keys(ctx, t) == oh.hash_blocks(t.tolist(), 16)
    ctx.close()


@pytest.mark.parametrize("b", [16, 32, 64])
def test_large_batch_two_launch_path(b):
    """Batches of many prompts take the two-launch form (token phase, then one scan CTA per prompt):
    ragged lengths, empty prompts, parents, a prompt longer than one scan pass, three calls in a row."""
    ctx = hash_ctx(b, hash_scratch_blocks=1 << 18)
    rng = np.random.default_rng(60 + b)
    lens = [int(x) for x in rng.integers(0, 9000, size=420)]
    lens[3], lens[17], lens[100], lens[200] = 0, b - 1, 70000, 64 * 2048 + 5 * b + 3   # > 2,048 runs of 64 tokens
    lens = [x - x % 4 for x in lens]                       # every prompt starts 16-byte aligned
    offsets = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    toks = rng.integers(0, 151936, size=int(offsets[-1]), dtype=np.int32)
    parents = [int(x) for x in rng.integers(0, P, size=len(lens), dtype=np.uint64)]
    dev = torch.from_numpy(toks).cuda()
    total = sum(x // b for x in lens)
    expect = {}
    for par in (None, parents):
        for i, n in enumerate(lens):
            p0 = oh.HASH_SEED if par is None else par[i]
            expect[(par is None, i)] = oh.hash_blocks(toks[offsets[i]:offsets[i + 1]].tolist(), b, p0)
    for rep in range(3):
        par = None if rep != 1 else parents
        out = torch.full((total + 1,), -1, dtype=torch.int64, device="cuda")
        before = ctx.eakv_get_stats()["kernel_launches"]
        boff = ctx.eakv_hash_blocks_batched(dev.data_ptr(), offsets, par, out.data_ptr())
        ctx.eakv_sync()
        assert ctx.eakv_get_stats()["kernel_launches"] - before == 3      # arguments, token phase, scan
        res = out.cpu().numpy()
        assert res[total] == -1
        for i in range(len(lens)):
            got = [int(x) for x in res[boff[i]:boff[i + 1]].view(np.uint64)]
            assert got == expect[(par is None, i)], (b, rep, i, lens[i])
    ctx.close()


def test_hash_self_check_reports_range_and_recovers():
    """The hash kernels check every tile against the number of keys the call may write; told a
    narrower number than the call needs they skip the tiles beyond it and eakv_sync reports
    EAKV_E_RANGE once.  Nothing outside the buffers is touched, and the next call is exact again."""
    from paper_2609_33762_b200 import eakv
    rng = np.random.default_rng(12)
    for b, nblk in ((16, 3000), (128, 700), (10, 900)):
        ctx = hash_ctx(b)
        toks = rng.integers(0, 151936, size=nblk * b, dtype=np.int32)
        ctx.eakv_selfcheck_limits(hash_blocks=200)
        dev = torch.from_numpy(toks).cuda()
        out = torch.full((nblk + 1,), -1, dtype=torch.int64, device="cuda")
        ctx.eakv_hash_blocks(dev.data_ptr(), len(toks), ctx.eakv_hash_seed(), out.data_ptr())
        with pytest.raises(eakv.EakvError) as ei:
            ctx.eakv_sync()
        assert ei.value.code == eakv.E_RANGE
        assert int(out[nblk].item()) == -1
        ctx.eakv_sync()
        ctx.eakv_selfcheck_limits()
        assert gpu_keys(ctx, toks) == oh.hash_blocks(toks.tolist(), b)
        ctx.close()


def test_ordinary_host_memory_is_refused_not_dereferenced():
    """A token or key pointer into ordinary (pageable) host memory would cost the CUDA context if a
    kernel read it: the calls ask the runtime what the address is and return EAKV_E_INVAL without
    launching.  Pinned host memory and device memory go through, with the oracle's keys."""
    from paper_2609_33762_b200 import eakv
    b = 16
    ctx = hash_ctx(b)
    toks = np.random.default_rng(13).integers(0, 151936, size=40 * b, dtype=np.int32)
    want = oh.hash_blocks(toks.tolist(), b)
    out = torch.zeros(40, dtype=torch.int64, device="cuda")
    pageable_out = np.zeros(40, dtype=np.uint64)
    dev = torch.from_numpy(toks).cuda()
    for tok_ptr, out_ptr in ((toks.ctypes.data, out.data_ptr()), (dev.data_ptr(), pageable_out.ctypes.data)):
        with pytest.raises(eakv.EakvError) as ei:
            ctx.eakv_hash_blocks(tok_ptr, len(toks), ctx.eakv_hash_seed(), out_ptr)
        assert ei.value.code == eakv.E_INVAL
    with pytest.raises(eakv.EakvError) as ei:
        ctx.eakv_turn_begin(toks.ctypes.data, len(toks), None, 0, 0)
    assert ei.value.code == eakv.E_INVAL
    ctx.eakv_sync()                                           # nothing was launched, nothing is wrong
    pinned = torch.from_numpy(toks).pin_memory()
    pinned_out = torch.zeros(40, dtype=torch.int64).pin_memory()
    ctx.eakv_hash_blocks(pinned.data_ptr(), len(toks), ctx.eakv_hash_seed(), pinned_out.data_ptr())
    ctx.eakv_sync()
    torch.cuda.synchronize()
    assert [int(x) for x in pinned_out.numpy().view(np.uint64)] == [int(k) for k in want]
    assert gpu_keys(ctx, toks) == want
    ctx.close()
