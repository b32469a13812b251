"""Pins for the trace oracle's two-granularity mode (host chunks of R engine blocks: Section 5.1
and Appendix A give 1,024-token host chunks over 16-token blocks; Section 3.2 keys a chunk by
its entire prefix; Appendix C counts restoration "after chunk and block alignment").

None of these compares the oracle with the CUDA library.  They use what the definition fixes:
  * re-blocking: a chunk's key is the prefix hash at its last token, so a host tier of chunks of
    R blocks of b tokens must behave exactly like a one-granularity tier of blocks of b*R tokens;
  * a hand-computed prompt of 2 chunks + 3 blocks + a partial block;
  * the bytes every resident chunk slot and every keyed GPU block must hold.
"""
import numpy as np
import pytest

from eakv_workloads import CONFIGS, SHAPES, KVShape, key_words_numpy, make_trace
from oracle import hash as ohash
from oracle.tier import FILTER_CONDITIONED, FILTER_FIXED, WRITE_ALL
from oracle.trace import TraceOracle

HOST_FIELDS = ("hit", "admit", "slot", "evicted", "new_chunks", "save", "pressure")


def scaled_c2_trace():
    """Config 2's generator at a size the Python oracle finishes in a second: 6 agents x 8 turns,
    prompts of 1k-6k tokens with tool-gap interleave (so requests of different agents alternate
    and the tier evicts)."""
    import dataclasses
    cfg = dataclasses.replace(CONFIGS["c2"], first_prompt=1024, append_median=400.0, context_cap=6000)
    return make_trace(cfg, agents=6, turns=8)


@pytest.mark.parametrize("policy", [WRITE_ALL, FILTER_FIXED, FILTER_CONDITIONED])
@pytest.mark.parametrize("R", [2, 4, 8])
def test_chunks_of_R_blocks_equal_one_granularity_with_R_times_larger_blocks(R, policy):
    trace = scaled_c2_trace()
    b = 16
    kappa = 1024 // (b * R) + 2                  # first prompts pass the filter, refills do not
    fine = KVShape(2, 1, 8, b)
    coarse = KVShape(2, 1, 8, b * R)
    K = 6000 // (b * R) + 24                     # chunks: the longest prompt fits, the pool's contexts do not
    kw = dict(policy=policy, kappa_blocks=kappa, window_ms=20_000, len_window=16)
    a = TraceOracle(fine, 4096, K, chunk_blocks=R, **kw)
    c = TraceOracle(coarse, 4096, K, chunk_blocks=1, **kw)
    a.run(trace)
    c.run(trace)
    assert len(a.records) == len(c.records) == len(trace.requests)
    for ra, rc in zip(a.records, c.records):
        # the coarse run's block keys ARE the chunk keys of the fine run
        assert ra["keys"][R - 1::R] == rc["keys"]
        assert ra["H"] == rc["H"] * R
        assert ra["H"] % R == 0 and ra["H"] <= len(ra["keys"])
        for f in HOST_FIELDS:
            assert ra[f] == rc[f], f
        # stored blocks: R per admitted chunk; the restore run ends at a chunk boundary
        assert ra["stored"] == R * sum(rc["admit"])
    assert a.host.stats == c.host.stats
    assert list(a.host.order.items()) == list(c.host.order.items())
    if policy != WRITE_ALL:
        assert a.host.stats["declined_requests"] > 0        # the filter really engaged
    assert a.host.stats["evicted"] > 0 and a.host.stats["hits"] > 0


def test_hand_case_two_chunks_three_blocks_and_a_partial_tail():
    """R = 4, b = 16: a prompt of 2*64 + 3*16 + 5 = 181 tokens has 11 full blocks and 2 full
    chunks.  Only the 2 chunks are looked up and stored: 8 blocks, into block slots 4s .. 4s+3
    of chunk slots 0 and 1; blocks 8-10 and the tail never reach the host tier."""
    R, b = 4, 16
    sh = SHAPES["tiny"]
    rng = np.random.default_rng(5)
    toks = rng.integers(0, 151936, size=181, dtype=np.int32)
    o = TraceOracle(sh, 64, 8, payload=key_words_numpy, chunk_blocks=R)
    rec = o.turn(toks, agent=0, now_ms=0)
    keys = ohash.hash_blocks(toks.tolist(), b)
    assert len(keys) == 11 and rec["keys"] == keys
    # chunk keys: prefix hash after token 63 and after token 127 (the chunk's LAST block's key)
    want_chunk_keys = [ohash.hash_blocks(toks[:64].tolist(), 64)[0], ohash.hash_blocks(toks[:128].tolist(), 64)[1]]
    assert want_chunk_keys == [keys[3], keys[7]]
    assert list(o.host.order.keys()) == want_chunk_keys
    assert rec["hit"] == [0, 0] and rec["admit"] == [1, 1] and rec["slot"] == [0, 1]
    assert rec["new_chunks"] == 2 and rec["H"] == 0 and rec["G"] == 0
    assert rec["stored"] == 8 and rec["loaded"] == 0 and rec["filled"] == 11
    assert rec["fresh_tokens"] == 181
    W = sh.piece_bytes // 2
    for q in range(sh.pieces_per_block):
        words = key_words_numpy(keys, q, W)
        for j in range(8):                       # block j of the prompt sits in block slot j
            assert (o.tier[j, q].view(np.uint16) == words[j]).all()
        assert not o.tier[8:].any()              # nothing else was written: blocks 8-10 stay out

    # the same prompt again with 80 more tokens: 16 full blocks = 4 chunks; H = 2 chunks = 8
    # blocks although 11 blocks are GPU-resident; u = 4 - 2 = 2 chunks
    toks2 = np.concatenate([toks, rng.integers(0, 151936, size=80, dtype=np.int32)])
    rec2 = o.turn(toks2, agent=0, now_ms=1)
    assert rec2["G"] == 11 and rec2["H"] == 8 and rec2["new_chunks"] == 2
    assert rec2["hit"] == [1, 1, 0, 0] and rec2["admit"] == [0, 0, 1, 1] and rec2["slot"] == [0, 1, 2, 3]
    assert rec2["loaded"] == 0 and rec2["stored"] == 8           # G >= H: nothing to restore
    assert rec2["fresh_tokens"] == 261 - 11 * 16

    # a GPU tier too small to keep the prompt: the third turn restores [G, H) = [0, 16)
    o3 = TraceOracle(sh, 17, 8, payload=key_words_numpy, chunk_blocks=R)
    o3.turn(toks2, 0, 0)
    other = rng.integers(0, 151936, size=16 * 16, dtype=np.int32)
    o3.turn(other, 1, 1)                          # evicts agent 0's blocks from the 17-block GPU tier
    rec3 = o3.turn(toks2, 0, 2)
    assert rec3["G"] == 0 and rec3["H"] == 16 and rec3["loaded"] == 16 and rec3["filled"] == 0
    keys2 = ohash.hash_blocks(toks2.tolist(), b)
    for q in (0, sh.pieces_per_block - 1):
        words = key_words_numpy(keys2, q, W)
        for j, blk in enumerate(rec3["gpu_block"]):
            assert (o3.pool[q][blk].view(np.uint16) == words[j]).all(), (q, j)


def test_write_threshold_counts_chunks_not_blocks():
    """Fixed admission (p = 1) with kappa = 2: a prompt needing u = 2 new chunks is saved, one
    needing u = 3 is declined.  Counted in blocks both would exceed kappa (8 and 12 blocks)."""
    R, b = 4, 16
    sh = SHAPES["tiny"]
    rng = np.random.default_rng(6)
    o = TraceOracle(sh, 64, 16, policy=FILTER_FIXED, kappa_blocks=2, chunk_blocks=R)
    r = o.turn(rng.integers(0, 1000, size=2 * 64 + 40, dtype=np.int32), 0, 0)
    assert r["new_chunks"] == 2 and r["save"] and r["admit"] == [1, 1]
    r = o.turn(rng.integers(0, 1000, size=3 * 64 + 40, dtype=np.int32), 1, 1)
    assert r["new_chunks"] == 3 and not r["save"] and r["admit"] == [0, 0, 0] and r["stored"] == 0


@pytest.mark.parametrize("R", [2, 4])
def test_config0_every_resident_chunk_slot_and_gpu_block_holds_its_payload(R):
    """Whole trace with bytes: after the run, chunk slot s holds the payload of that chunk's R
    blocks at block slots s*R .. s*R+R-1, and every keyed GPU block (restored ones included)
    holds its own payload."""
    tr = make_trace("c0")
    sh = SHAPES["tiny"]
    o = TraceOracle(sh, 128, 1024 // R, payload=key_words_numpy, chunk_blocks=R)
    recs = o.run(tr)
    assert o.totals["loaded_blocks"] > 0 and o.totals["stored_blocks"] > 0
    blocks_of = {}                                # chunk key -> its R block keys
    for r in recs:
        k = r["keys"]
        for c in range(len(k) // R):
            blocks_of[k[c * R + R - 1]] = k[c * R: c * R + R]
    W = sh.piece_bytes // 2
    assert len(o.host.order) > 0
    for q in (0, 3, sh.pieces_per_block - 1):
        for ck, s in o.host.order.items():
            words = key_words_numpy(blocks_of[ck], q, W)
            for i in range(R):
                assert (o.tier[s * R + i, q].view(np.uint16) == words[i]).all(), (ck, s, i)
        gkeys = list(o.gpu.order.keys())
        words = key_words_numpy(gkeys, q, W)
        for r_, k in enumerate(gkeys):
            assert (o.pool[q][o.gpu.order[k]].view(np.uint16) == words[r_]).all()
    for r in recs:
        assert r["H"] % R == 0 and r["loaded"] == max(0, r["H"] - r["G"])
