"""Pins for oracle.storeload and oracle.trace: byte-exact round trips, untouched guards,
and the capacity model agreeing exactly with the simulated tier (Mattson) on config 0."""
import numpy as np

from eakv_workloads import SHAPES, key_words_numpy, make_trace
from oracle import stackdist as sd
from oracle import storeload as sl
from oracle.trace import GpuTier, TraceOracle


def make_pool(rng, q, nb, p):
    return [rng.integers(0, 256, size=(nb, p), dtype=np.uint8) for _ in range(q)]


def test_roundtrip_and_guards():
    rng = np.random.default_rng(0)
    Q, NB, KH, P = 6, 20, 12, 64
    pool = make_pool(rng, Q, NB, P)
    orig = [a.copy() for a in pool]
    tier = np.full((KH, Q, P), 0xAB, dtype=np.uint8)
    table = [7, 3, 19, 0]
    admit = [1, 0, 1, 1]
    slots = [5, 9, 0, 11]
    sl.store(pool, tier, table, admit, slots)
    for j, (blk, a, s) in enumerate(zip(table, admit, slots)):
        for q in range(Q):
            if a:
                assert (tier[s, q] == orig[q][blk]).all()
            else:
                assert (tier[s, q] == 0xAB).all()       # masked entry untouched
    untouched = [s for s in range(KH) if s not in (5, 0, 11)]
    assert (tier[untouched] == 0xAB).all()
    assert all((a == b).all() for a, b in zip(pool, orig))   # store never writes the pool
    # load into fresh blocks reproduces the bytes; other blocks keep their content
    dst = [1, 2, 4]
    sl.load(pool, tier, [5, 0, 11], dst)
    for (s, d, src) in zip([5, 0, 11], dst, [7, 19, 0]):
        for q in range(Q):
            assert (pool[q][d] == orig[q][src]).all()
    for q in range(Q):
        others = [i for i in range(NB) if i not in dst]
        assert (pool[q][others] == orig[q][others]).all()


def test_bytes_are_opaque():
    # NaN payloads, negative zero and infinities survive a round trip bit for bit
    words = np.array([0x7FC1, 0xFFFF, 0x8000, 0x7F80, 0xFF80, 0x0001], dtype=np.uint16)
    pool = [np.zeros((2, 12), dtype=np.uint8)]
    pool[0][0] = words.view(np.uint8)
    tier = np.zeros((1, 1, 12), dtype=np.uint8)
    sl.store(pool, tier, [0], [1], [0])
    sl.load(pool, tier, [0], [1])
    assert (pool[0][1].view(np.uint16) == words).all()


def test_empty_calls():
    pool = [np.ones((2, 8), dtype=np.uint8)]
    tier = np.zeros((2, 1, 8), dtype=np.uint8)
    sl.store(pool, tier, [], [], [])
    sl.load(pool, tier, [], [])
    assert tier.sum() == 0


def test_gpu_tier_lru_and_tail():
    g = GpuTier(4)
    res, ids, tail = g.step(["a", "b", "c"], True)
    assert res == [0, 0, 0] and ids == [0, 1, 2] and tail == 3
    g.release(tail)
    res, ids, tail = g.step(["a", "d", "e"], False)   # d takes the released block, e evicts b
    assert res == [1, 0, 0] and ids == [0, 3, 1] and tail == -1
    assert "b" not in g and "c" in g


def test_c0_trace_oracle_consistency():
    """Write-all run of config 0 (and its large-tier sibling): the stack-distance model
    predicts the simulated host hits exactly, loaded bytes equal the payload function,
    and totals add up."""
    tr = make_trace("c0")
    sh = SHAPES["tiny"]
    for KH in (256, 1024):
        o = TraceOracle(sh, 128, KH, payload=key_words_numpy)
        recs = o.run(tr)
        pred = sd.predict_trace([r["keys"] for r in recs], [r["n_tokens"] for r in recs],
                                [r["G"] for r in recs], KH, sh.block_size)
        assert pred["host_cover"] == [r["H"] for r in recs]
        assert pred["hit_flags"] == [bool(h) for r in recs for h in r["hit"]]
        assert pred["restored_blocks"] == o.totals["loaded_blocks"]
        assert pred["computed_tokens"] == o.totals["fresh_tokens"]
        assert o.totals["stored_blocks"] == o.host.stats["admitted"]
        # every key-indexed GPU block and every host slot holds exactly its payload
        W = sh.piece_bytes // 2
        for index, store, getter in ((o.gpu.order, "pool", lambda q, i: o.pool[q][i]),
                                     (o.host.order, "tier", lambda q, i: o.tier[i, q])):
            keys = list(index.keys())
            for q in (0, sh.pieces_per_block - 1):
                words = key_words_numpy(keys, q, W)
                for r, k in enumerate(keys):
                    assert (getter(q, index[k]).view(np.uint16) == words[r]).all(), store
    # larger tier: hits are monotone per reference (inclusion) and restores happen
    a = TraceOracle(sh, 128, 256); a.run(tr)
    b = TraceOracle(sh, 128, 1024); b.run(tr)
    for ra, rb in zip(a.records, b.records):
        assert all((not x) or y for x, y in zip(ra["hit"], rb["hit"]))
    assert b.totals["loaded_blocks"] > a.totals["loaded_blocks"] > 0
