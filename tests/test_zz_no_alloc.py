"""The allocation-free entry point eakv_hash_blocks_static must return the same keys as
eakv_hash_blocks.  It exists for callers that cannot request device memory (for instance
code running inside a serving process whose engine already owns the GPU's memory): its
scratch is a fixed array inside the library that all calls share, so this test makes two
calls in a row with different inputs and checks both, bit for bit.  The file sorts last on
purpose: a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest

from gpu_util import hash_ctx, require_gpu, torch

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


def test_static_scratch_variant_matches_context_variant_twice_in_a_row():
    require_gpu()
    from paper_2609_33762_b200 import eakv
    rng = np.random.default_rng(99)
    for b in (16, 32, 10):
        ctx = hash_ctx(b)
        base, seed = ctx.eakv_hash_base(), ctx.eakv_hash_seed()
        # two calls back to back: the second is shorter and starts from another parent, so
        # anything left over from the first (partials, counter, power table) would show
        for n, parent in ((b * 5000 + 7, seed), (b * 37 + 1, 12345)):
            toks = torch.from_numpy(rng.integers(0, 151936, size=n, dtype=np.int32)).cuda()
            want = keys_via_context(ctx, toks, n, parent)
            got = keys_via_static(eakv, toks, n, b, base, parent)
            assert len(got) == n // b and np.array_equal(got, want), (b, n)
        ctx.close()
    # another base between calls: the power table is rebuilt per call
    ctx = hash_ctx(16, hash_base=987654321)
    toks = torch.from_numpy(rng.integers(0, 151936, size=16 * 300, dtype=np.int32)).cuda()
    want = keys_via_context(ctx, toks, 16 * 300, 7)
    assert np.array_equal(keys_via_static(eakv, toks, 16 * 300, 16, 987654321, 7), want)
    ctx.close()


def test_static_variant_rejects_what_its_scratch_cannot_hold():
    require_gpu()
    from paper_2609_33762_b200 import eakv
    b = 4
    n = (eakv.STATIC_MAX_BLOCKS + 1) * b
    toks = torch.zeros(n, dtype=torch.int32, device="cuda")
    out = torch.zeros(eakv.STATIC_MAX_BLOCKS + 1, dtype=torch.int64, device="cuda")
    with pytest.raises(eakv.EakvError) as ei:
        eakv.eakv_hash_blocks_static(toks.data_ptr(), n, b, 0, 1, out.data_ptr())
    assert ei.value.code == eakv.E_CAPACITY
    # exactly the maximum is accepted; too-large block sizes and null buffers are refused
    assert eakv.eakv_hash_blocks_static(toks.data_ptr(), n - b, b, 0, 1, out.data_ptr()) == eakv.STATIC_MAX_BLOCKS
    torch.cuda.synchronize()
    for args in ((toks.data_ptr(), 64, 8192, 0, 1, out.data_ptr()), (0, 64, 16, 0, 1, out.data_ptr())):
        with pytest.raises(eakv.EakvError) as ei:
            eakv.eakv_hash_blocks_static(*args)
        assert ei.value.code == eakv.E_INVAL
