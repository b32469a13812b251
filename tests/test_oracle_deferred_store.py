"""Pins for the trace oracle's deferred host writes (``TraceOracle.begin(defer_store=True)`` /
``store``): requests whose KV is written to the host tier only after other requests have been
looked up.  What is fixed from outside the oracle:

  * the bookkeeping is still the reference model's: a deferred run and a run that writes at the
    lookup list the same units in the same order with the same slots;
  * no reader ever sees bytes that are not its key's: at every step each listed unit whose write
    is not pending holds exactly its blocks' payload, and every restored GPU block holds the
    payload of the key it was restored for (checked against the payload function itself);
  * a hand-computed case (tier of 8 units, two requests of 6): the second lookup evicts four
    units of the first before they were written; the first request then writes only the two it
    still owns;
  * store directly after begin is the non-deferred turn, record by record and byte by byte.
"""
import numpy as np
import pytest

from eakv_workloads import KVShape, key_words_numpy
from oracle.trace import TraceOracle

from deferred_util import drive, operations

SHAPE = KVShape(1, 1, 8, 4)          # one layer, block of 4 tokens: 2 pieces of 64 bytes


def block_payload(shape, key):
    W = shape.piece_bytes // 2
    return [key_words_numpy(np.asarray([key], dtype=np.uint64), q, W)[0].view(np.uint8)
            for q in range(shape.pieces_per_block)]


def check_readable_bytes(o, unit_blocks):
    """Every listed unit that is not pending holds its blocks' payload; pending ones are listed."""
    R = o.R
    for k in o.pending:
        assert k in o.host.order
    for ukey, slot in o.host.order.items():
        if ukey in o.pending:
            continue
        for i, bkey in enumerate(unit_blocks[ukey]):
            want = block_payload(o.shape, bkey)
            for q in range(o.shape.pieces_per_block):
                assert np.array_equal(o.tier[slot * R + i, q], want[q]), (ukey, slot, i, q)


def test_hand_case_evicted_before_written():
    o = TraceOracle(SHAPE, 64, 8, payload=key_words_numpy)
    t1 = list(range(100, 124))                 # 6 blocks
    t2 = list(range(200, 224))
    r1 = o.begin(1, t1, 0, 0, defer_store=True)
    assert r1["slot"] == [0, 1, 2, 3, 4, 5] and r1["admit"] == [1] * 6
    r2 = o.begin(2, t2, 1, 1, defer_store=True)
    # two free slots, then the four least recent units of request 1 go, unwritten
    assert r2["slot"] == [6, 7, 0, 1, 2, 3]
    assert [k for k, _ in r2["evicted"]] == r1["keys"][:4]
    assert set(o.pending) == set(r1["keys"][4:]) | set(r2["keys"])
    assert o.store(2) == 6
    assert o.store(1) == 2                      # only the two units it still owns
    assert not o.pending
    for key, slot in list(zip(r2["keys"], r2["slot"])) + list(zip(r1["keys"][4:], [4, 5])):
        for q, want in enumerate(block_payload(SHAPE, key)):
            assert np.array_equal(o.tier[slot, q], want)


def test_pending_units_are_not_restorable_and_not_written_twice():
    o = TraceOracle(SHAPE, 64, 16, payload=key_words_numpy)
    t = list(range(300, 316))                   # 4 blocks
    r1 = o.begin(1, t, 0, 0, defer_store=True)
    r2 = o.begin(2, t + [7, 7, 7, 7], 1, 1, defer_store=True)
    assert r2["hit"][:4] == [1] * 4 and r2["admit"] == [0, 0, 0, 0, 1]     # listed: no second write
    assert (r2["G"], r2["H"]) == (4, 0)                                        # shared on the GPU; nothing restorable on the host yet
    assert o.store(1) == 4 and o.store(2) == 1
    o.finish(1)
    o.finish(2)


@pytest.mark.parametrize("R", [1, 2])
@pytest.mark.parametrize("seed", [1, 2, 3])
def test_random_interleavings_never_expose_unwritten_bytes(seed, R):
    b = SHAPE.block_size
    kh = 40 // R
    o = TraceOracle(SHAPE, 48, kh, payload=key_words_numpy, chunk_blocks=R)
    ref = TraceOracle(SHAPE, 48, kh, chunk_blocks=R)       # writes at the lookup: bookkeeping only
    unit_blocks = {}
    stats = dict(skipped=0, begins=0)

    def on_begin(rid, agent, tokens, now):
        rec = o.begin(rid, tokens, agent, now, defer_store=True)
        want = ref.begin(rid, tokens, agent, now)
        assert (rec is None) == (want is None)
        if rec is None:
            return False
        stats["begins"] += 1
        keys = rec["keys"]
        for c in range(len(keys) // R):
            unit_blocks[keys[c * R + R - 1]] = keys[c * R:(c + 1) * R]
        # the reference model's bookkeeping, untouched by the deferral
        for f in ("hit", "admit", "slot", "evicted", "gpu_block", "gpu_resident", "G"):
            assert rec[f] == want[f], f
        assert rec["H"] <= want["H"]
        # what was restored is the payload of the keys it was restored for
        for j in range(rec["G"], rec["G"] + rec["loaded"]):
            for q, w in enumerate(block_payload(SHAPE, keys[j])):
                assert np.array_equal(o.pool[q][rec["gpu_block"][j]], w)
        check_readable_bytes(o, unit_blocks)
        return True

    def on_store(rid):
        admitted = sum(o.open[rid]["admit_b"])
        stats["skipped"] += admitted - o.store(rid)
        check_readable_bytes(o, unit_blocks)

    def on_finish(rid):
        o.finish(rid)
        ref.finish(rid)

    drive(operations(seed, 400, b, 30 * b, max_open=4), on_begin, on_store, on_finish)
    assert list(o.host.order.items()) == list(ref.host.order.items())
    assert not o.pending and not o.open
    assert stats["begins"] > 100 and stats["skipped"] > 0       # the case under test did occur


def test_store_right_after_begin_is_the_plain_turn():
    b = SHAPE.block_size
    a = TraceOracle(SHAPE, 48, 36, payload=key_words_numpy)
    c = TraceOracle(SHAPE, 48, 36, payload=key_words_numpy)

    def on_begin(rid, agent, tokens, now):
        ra = a.begin(rid, tokens, agent, now, defer_store=True)
        rc = c.begin(rid, tokens, agent, now)
        assert (ra is None) == (rc is None)
        if ra is None:
            return False
        assert a.store(rid) == ra["stored"]
        assert ra == rc
        return True

    drive(operations(9, 300, b, 30 * b, max_open=3), on_begin, lambda rid: None,
          lambda rid: (a.finish(rid), c.finish(rid)))
    assert np.array_equal(a.tier, c.tier)
    for q in range(SHAPE.pieces_per_block):
        assert np.array_equal(a.pool[q], c.pool[q])
