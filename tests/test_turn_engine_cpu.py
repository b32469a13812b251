"""The two-call turn engine (eakv_turn_begin / eakv_turn_end / eakv_turn_abort) as pure
bookkeeping on the CPU: a control-plane-only context runs it when the caller supplies every
key.  Checked against the trace oracle per request, and for what a refused, failed or aborted
turn must leave behind: no key may stay listed whose bytes were never written."""
from dataclasses import replace

import numpy as np
import pytest

from eakv_workloads import CONFIGS, SHAPES, make_trace
from oracle import hash as ohash
from oracle.trace import TraceOracle


@pytest.fixture(scope="module")
def eakv():
    from paper_2609_33762_b200 import build, eakv as m
    build.build()
    return m


def cp_ctx(eakv, block_size, gpu_blocks, host_blocks, **kw):
    return eakv.Context(num_layers=1, kv_heads=1, head_dim=8, block_size=block_size,
                        gpu_blocks=gpu_blocks, host_blocks=host_blocks, kv_base=None,
                        control_plane_only=True, **kw)


def keys_of(tokens, b):
    return np.asarray(ohash.hash_blocks(np.asarray(tokens).tolist(), b), dtype=np.uint64)


def compare_view(v, w, R=1):
    assert [int(k) for k in v["keys"]] == w["keys"]
    assert (v["gpu_prefix_blocks"], v["host_prefix_blocks"], v["new_chunks"], bool(v["pressure"]), bool(v["save"])) == \
           (w["G"], w["H"], w["new_chunks"], w["pressure"], w["save"])
    for f in ("hit", "admit", "slot"):
        assert v[f].tolist() == w[f], f
    assert list(zip(v["evicted_keys"].tolist(), v["evicted_slots"].tolist())) == w["evicted"]
    assert v["gpu_resident"].tolist() == w["gpu_resident"] and v["gpu_block"].tolist() == w["gpu_block"]
    assert v["restore_hi"] - v["restore_lo"] == w["loaded"]
    assert v["n_stored_blocks"] == w["stored"] and v["fresh_tokens"] == w["fresh_tokens"]
    assert v["n_fill"] == w["filled"]


@pytest.mark.parametrize("R,policy", [(1, 0), (1, 2), (4, 0), (4, 1), (2, 2)])
def test_turn_engine_bookkeeping_equals_oracle(eakv, R, policy):
    cfg = replace(CONFIGS["c2"], shape="tiny", agents=6, turns=14, first_prompt=500,
                  append_median=200.0, context_cap=3500, tool_gap_mean_ms=15_000.0)
    shape = SHAPES["tiny"]
    b = shape.block_size
    trace = make_trace(cfg, seed=41)
    kw = dict(policy=policy, kappa_blocks=max(1, 8 // R), window_ms=60_000, len_window=32)
    kh = 700 // R
    oracle = TraceOracle(shape, 256, kh, chunk_blocks=R, **kw)
    ctx = cp_ctx(eakv, b, 256, kh, chunk_blocks=R, **kw)
    for req in trace.requests:
        toks = trace.prompt(req)
        w = oracle.turn(toks, req.agent, req.time_ms)
        v = ctx.eakv_turn_begin(0, len(toks), keys_of(toks, b), req.agent, req.time_ms)
        compare_view(v, w, R)
        ctx.eakv_turn_end()
    st = ctx.eakv_get_stats()
    for f in ("requests", "references", "hits", "admitted", "declined", "evicted"):
        assert st[f] == oracle.host.stats[f], f
    if policy != 1:                              # the fixed filter declines nearly everything
        assert oracle.totals["loaded_blocks"] > 0
    ctx.close()


def test_turn_without_all_keys_needs_a_device(eakv):
    ctx = cp_ctx(eakv, 4, 16, 16)
    with pytest.raises(eakv.EakvError) as ei:
        ctx.eakv_turn_begin(0, 16, np.asarray([1, 2], dtype=np.uint64), 0, 0)     # 4 blocks, 2 keys
    assert ei.value.code == eakv.E_INVAL
    with pytest.raises(eakv.EakvError):
        ctx.eakv_turn_end()                      # no turn was opened
    ctx.close()


def test_prompt_larger_than_the_gpu_tier_is_refused_before_anything_changes(eakv):
    """A prompt with more blocks than the GPU tier hands out: EAKV_E_CAPACITY, and neither tier
    has changed, in particular the host index does not list keys whose slots were never written."""
    b = 4
    ctx = cp_ctx(eakv, b, 8, 64)                              # K_G = 8 blocks, K_H = 64
    small = np.arange(1, 7, dtype=np.uint64)                  # 6 blocks: fits
    v = ctx.eakv_turn_begin(0, 6 * b, small, 0, 0)
    assert v["n_stored_blocks"] == 6
    ctx.eakv_turn_end()
    before = ctx.eakv_get_stats()
    big = np.arange(100, 112, dtype=np.uint64)                # 12 blocks > K_G
    with pytest.raises(eakv.EakvError) as ei:
        ctx.eakv_turn_begin(0, 12 * b, big, 1, 1)
    assert ei.value.code == eakv.E_CAPACITY
    G, H, _, _ = ctx.eakv_match(big)
    assert (G, H) == (0, 0)
    assert ctx.eakv_get_stats() == before
    # exactly K_G blocks with a partial tail does not fit either (the tail needs a ninth block)
    eight = np.arange(200, 208, dtype=np.uint64)
    with pytest.raises(eakv.EakvError) as ei:
        ctx.eakv_turn_begin(0, 8 * b + 1, eight, 1, 2)
    assert ei.value.code == eakv.E_CAPACITY and ctx.eakv_match(eight)[:2] == (0, 0)
    # more units than the host tier
    ctx2 = cp_ctx(eakv, b, 64, 4)
    with pytest.raises(eakv.EakvError) as ei:
        ctx2.eakv_turn_begin(0, 6 * b, small, 0, 0)
    assert ei.value.code == eakv.E_CAPACITY and ctx2.eakv_match(small)[:2] == (0, 0)
    # the first context still serves what it stored, and the next turn opens normally
    assert ctx.eakv_match(small)[:2] == (6, 6)
    v = ctx.eakv_turn_begin(0, 6 * b, small, 0, 3)
    assert v["hit"].tolist() == [1] * 6
    ctx.eakv_turn_end()
    ctx.close(); ctx2.close()


def test_aborted_turn_takes_back_what_it_never_produced(eakv):
    """A turn that is aborted after begin (the engine will not compute its KV): the units it
    admitted leave the host index, the blocks it was to fill leave the GPU index, what was
    resident before stays, and the slots and blocks are handed out again."""
    b = 4
    ctx = cp_ctx(eakv, b, 32, 32)
    first = np.arange(1, 5, dtype=np.uint64)
    ctx.eakv_turn_begin(0, 4 * b, first, 0, 0)
    ctx.eakv_turn_end()
    longer = np.arange(1, 11, dtype=np.uint64)                # the same 4 blocks + 6 new ones + a tail
    v = ctx.eakv_turn_begin(0, 10 * b + 2, longer, 0, 1)
    assert v["hit"].tolist() == [1] * 4 + [0] * 6 and v["admit"].tolist() == [0] * 4 + [1] * 6
    assert v["needs_fill"].tolist() == [0] * 4 + [1] * 6 and v["tail_block"] >= 0
    with pytest.raises(eakv.EakvError):
        ctx.eakv_turn_begin(0, 4 * b, first, 1, 1)            # one turn at a time
    ctx.eakv_turn_abort()
    assert ctx.eakv_match(longer)[:2] == (4, 4)               # only what existed before is listed
    assert ctx.eakv_get_stats()["resident"] == 4
    with pytest.raises(eakv.EakvError):
        ctx.eakv_turn_abort()                                 # nothing open any more
    # the withdrawn slots, blocks and the tail block are free again: the same turn repeats exactly
    v2 = ctx.eakv_turn_begin(0, 10 * b + 2, longer, 0, 2)
    assert v2["slot"].tolist() == v["slot"].tolist()
    assert sorted(v2["gpu_block"].tolist() + [v2["tail_block"]]) == sorted(v["gpu_block"].tolist() + [v["tail_block"]])
    ctx.eakv_turn_end()
    assert ctx.eakv_match(longer)[:2] == (10, 10)
    ctx.close()


def test_requests_overlap_and_an_unstored_release_takes_its_turn_back(eakv):
    """eakv_request_*: two requests open at once share a prefix block; a request released before
    its store is taken back like an aborted turn; refused ids and orders."""
    b = 4
    ctx = cp_ctx(eakv, b, 16, 32)
    sys_key = 900
    a = np.asarray([sys_key, 1, 2, 3], dtype=np.uint64)
    c = np.asarray([sys_key, 11, 12], dtype=np.uint64)
    va = ctx.eakv_request_begin(1, 0, 4 * b + 1, a, 0, 0)
    vc = ctx.eakv_request_begin(2, 0, 3 * b, c, 1, 1)
    assert va["gpu_block"][0] == vc["gpu_block"][0]                    # the shared first block
    assert vc["gpu_resident"].tolist() == [1, 0, 0] and vc["hit"].tolist() == [1, 0, 0]
    assert va["tail_block"] >= 0 and vc["tail_block"] == -1
    for bad in (lambda: ctx.eakv_request_begin(1, 0, 4, a[:1], 0, 2),  # id in use
                lambda: ctx.eakv_turn_begin(0, 4, a[:1], 0, 2),        # single turn while requests are open
                lambda: ctx.eakv_request_store(3), lambda: ctx.eakv_request_release(3)):
        with pytest.raises(eakv.EakvError) as ei:
            bad()
        assert ei.value.code == eakv.E_INVAL
    # a third request that does not fit beside the two is refused and changes nothing
    before = ctx.eakv_get_stats()
    big = np.arange(100, 112, dtype=np.uint64)
    assert ctx.eakv_request_begin(3, 0, 12 * b, big, 2, 3) is None
    assert ctx.eakv_get_stats() == before and ctx.eakv_match(big)[:2] == (0, 0)
    ctx.eakv_request_store(1)
    with pytest.raises(eakv.EakvError):
        ctx.eakv_request_store(1)                                      # once per begin
    ctx.eakv_request_release(1)                                        # finished: everything stays listed
    assert ctx.eakv_match(a)[:2] == (4, 4)
    # request 2 is released without a store: its two new units and blocks are taken back, the shared
    # block (stored by request 1) stays
    ctx.eakv_request_release(2)
    assert ctx.eakv_match(c)[:2] == (1, 1)
    assert ctx.eakv_get_stats()["resident"] == 4
    # now the big request fits
    assert ctx.eakv_request_begin(3, 0, 12 * b, big, 2, 4) is not None
    ctx.eakv_request_store(3)
    ctx.eakv_request_release(3)
    assert ctx.eakv_match(big)[:2] == (12, 12)
    ctx.close()


def test_units_admitted_by_an_open_request_are_not_restorable_until_it_stored(eakv):
    """Request 1 admits the units of a prompt; before it has stored them request 2 arrives with the
    same prompt (another GPU tier state is simulated by a tiny GPU tier that request 1 does not
    share: different keys cannot be used, so request 2 simply repeats the prompt).  Its lookup
    must not count the unwritten slots as host coverage, and must not store them a second time."""
    b = 4
    ctx = cp_ctx(eakv, b, 32, 32)
    keys = np.arange(1, 7, dtype=np.uint64)
    v1 = ctx.eakv_request_begin(1, 0, 6 * b, keys, 0, 0)
    assert v1["admit"].tolist() == [1] * 6 and v1["host_prefix_blocks"] == 0
    v2 = ctx.eakv_request_begin(2, 0, 6 * b, keys, 1, 1)
    assert v2["hit"].tolist() == [1] * 6 and v2["admit"].tolist() == [0] * 6      # listed: no second store
    assert v2["host_prefix_blocks"] == 0                                           # but nothing to restore yet
    assert v2["gpu_prefix_blocks"] == 6 and v2["restore_hi"] == v2["restore_lo"]   # (the GPU blocks are shared)
    ctx.eakv_request_store(1)
    ctx.eakv_request_store(2)
    v3 = ctx.eakv_request_begin(3, 0, 6 * b, keys, 2, 2)
    assert v3["host_prefix_blocks"] == 6                                           # stored: restorable now
    for rid in (1, 2, 3):
        ctx.eakv_request_release(rid)
    # a request released before its store leaves nothing pending behind
    other = np.arange(50, 53, dtype=np.uint64)
    ctx.eakv_request_begin(4, 0, 3 * b, other, 0, 3)
    ctx.eakv_request_release(4)
    v5 = ctx.eakv_request_begin(5, 0, 3 * b, other, 0, 4)
    assert v5["admit"].tolist() == [1, 1, 1]
    ctx.eakv_request_store(5)
    ctx.eakv_request_release(5)
    assert ctx.eakv_match(other)[:2] == (3, 3)
    ctx.close()


@pytest.mark.parametrize("R,seed", [(1, 5), (1, 6), (2, 7), (4, 8)])
def test_deferred_stores_interleaved_with_other_lookups_equal_the_oracle(eakv, R, seed):
    """eakv_request_begin ... (other requests' lookups) ... eakv_request_store: every view equals
    the oracle's deferred-store record, and the tier's final recency order and slots are equal.
    (The bytes of the same interleavings are checked on the GPU.)"""
    from deferred_util import drive, operations
    shape = SHAPES["tiny"]
    b = shape.block_size
    kh = 160 // R
    oracle = TraceOracle(shape, 160, kh, chunk_blocks=R)
    ctx = cp_ctx(eakv, b, 160, kh, chunk_blocks=R)
    seen = dict(begins=0, refused=0)

    def on_begin(rid, agent, tokens, now):
        w = oracle.begin(rid, tokens, agent, now, defer_store=True)
        v = ctx.eakv_request_begin(rid, 0, len(tokens), keys_of(tokens, b), agent, now)
        assert (v is None) == (w is None)
        if v is None:
            seen["refused"] += 1
            return False
        seen["begins"] += 1
        compare_view(v, w, R)
        return True

    def on_store(rid):
        oracle.store(rid)
        ctx.eakv_request_store(rid)

    def on_finish(rid):
        oracle.finish(rid)
        ctx.eakv_request_release(rid)

    drive(operations(seed, 500, b, 60 * b, max_open=4), on_begin, on_store, on_finish)
    keys, slots = ctx.eakv_tier_export()
    assert list(zip(keys.tolist(), slots.tolist())) == list(oracle.host.order.items())
    assert seen["begins"] > 100
    ctx.close()


def test_a_release_before_the_store_takes_back_only_units_the_request_still_owns(eakv):
    """Request 1 admits six units; request 2's lookup evicts four of them unwritten and reuses
    their slots; request 3 admits two of the evicted keys again.  Request 1, released without a
    store, may take back only the two units it still owns: not request 3's, although they carry
    keys request 1 once admitted, and not the slots request 2 now owns."""
    b = 4
    ctx = cp_ctx(eakv, b, 64, 8)
    k1 = np.arange(1, 7, dtype=np.uint64)
    k2 = np.arange(11, 17, dtype=np.uint64)
    v1 = ctx.eakv_request_begin(1, 0, 6 * b, k1, 0, 0)
    assert v1["slot"].tolist() == [0, 1, 2, 3, 4, 5]
    v2 = ctx.eakv_request_begin(2, 0, 6 * b, k2, 1, 1)
    assert v2["slot"].tolist() == [6, 7, 0, 1, 2, 3] and v2["evicted_keys"].tolist() == [1, 2, 3, 4]
    ctx.eakv_request_store(2)
    # keys 1, 2 come back through request 3 (evicting request 1's last two units, 5 and 6)
    k3 = np.asarray([1, 2], dtype=np.uint64)
    v3 = ctx.eakv_request_begin(3, 0, 2 * b, k3, 2, 2)
    assert v3["admit"].tolist() == [1, 1] and v3["evicted_keys"].tolist() == [5, 6]
    # request 1 owns nothing any more: its release changes no listing
    before = ctx.eakv_tier_export()
    ctx.eakv_request_release(1)
    after = ctx.eakv_tier_export()
    assert before[0].tolist() == after[0].tolist() and before[1].tolist() == after[1].tolist()
    ctx.eakv_request_store(3)
    assert ctx.eakv_match(k3)[1] == 2 and ctx.eakv_match(k2)[1] == 6
    for rid in (2, 3):
        ctx.eakv_request_release(rid)
    # and a request that still owns some of its units takes back exactly those
    k4 = np.arange(21, 25, dtype=np.uint64)
    k5 = np.arange(31, 37, dtype=np.uint64)
    ctx.eakv_request_begin(4, 0, 4 * b, k4, 0, 3)          # evicts 11..14
    v5 = ctx.eakv_request_begin(5, 0, 6 * b, k5, 1, 4)     # evicts 15, 16, 1, 2, then 21, 22 of request 4
    assert v5["evicted_keys"].tolist() == [15, 16, 1, 2, 21, 22]
    ctx.eakv_request_release(4)                            # owns 23, 24 only
    keys = ctx.eakv_tier_export()[0].tolist()
    assert keys == [31, 32, 33, 34, 35, 36]
    ctx.eakv_request_store(5)
    ctx.eakv_request_release(5)
    assert ctx.eakv_match(k5)[1] == 6
    ctx.close()


def test_injected_transfer_failures_withdraw_what_the_turn_registered(eakv):
    """The paths that only a CUDA error reaches otherwise, with a failure made on the host
    (eakv_selfcheck_fail_next_transfer): a restore that fails in begin and a store that fails in
    end / request_store leave no key listed whose bytes were never written, close the turn, and
    leave the context usable."""
    b = 4
    E = eakv
    p = np.arange(1, 7, dtype=np.uint64)                    # 6 blocks, stored by the first turn
    q = np.arange(101, 111, dtype=np.uint64)                # pushes them out of the 10-block GPU tier
    grown = np.concatenate([p, np.arange(7, 10, dtype=np.uint64)])

    def fresh():
        ctx = cp_ctx(eakv, b, 10, 64)
        for keys, agent in ((p, 0), (q, 1)):
            ctx.eakv_turn_begin(0, len(keys) * b, keys, agent, 0)
            ctx.eakv_turn_end()
        assert ctx.eakv_match(grown)[:2] == (0, 6)
        return ctx

    # restore fails in eakv_turn_begin
    ctx = fresh()
    listed = ctx.eakv_tier_export()[0].tolist()
    ctx.eakv_selfcheck_fail_next_transfer(E.E_CUDA)
    with pytest.raises(E.EakvError) as ei:
        ctx.eakv_turn_begin(0, len(grown) * b, grown, 0, 1)
    assert ei.value.code == E.E_CUDA
    with pytest.raises(E.EakvError):
        ctx.eakv_turn_end()                                   # no turn is open
    assert sorted(ctx.eakv_tier_export()[0].tolist()) == sorted(listed)      # the three new units are gone
    assert ctx.eakv_match(grown)[:2] == (0, 6)               # and no block of it is keyed on the GPU
    v = ctx.eakv_turn_begin(0, len(grown) * b, grown, 0, 2)  # the same turn again goes through
    assert (v["host_prefix_blocks"], v["admit"].tolist()) == (6, [0] * 6 + [1] * 3)
    ctx.eakv_turn_end()
    assert ctx.eakv_match(grown)[1] == 9
    ctx.close()

    # store fails in eakv_turn_end
    ctx = fresh()
    ctx.eakv_turn_begin(0, len(grown) * b, grown, 0, 1)
    ctx.eakv_selfcheck_fail_next_transfer(E.E_CUDA)
    with pytest.raises(E.EakvError) as ei:
        ctx.eakv_turn_end()
    assert ei.value.code == E.E_CUDA
    assert ctx.eakv_match(grown)[1] == 6                     # restored prefix stays, unwritten units do not
    with pytest.raises(E.EakvError):
        ctx.eakv_turn_abort()
    ctx.close()

    # the same for overlapping requests, with another request open meanwhile
    ctx = cp_ctx(eakv, b, 64, 64)
    other = np.arange(201, 205, dtype=np.uint64)
    ctx.eakv_request_begin(9, 0, 4 * b, other, 3, 0)
    ctx.eakv_request_begin(1, 0, 6 * b, p, 0, 0)
    ctx.eakv_selfcheck_fail_next_transfer(E.E_CUDA)
    with pytest.raises(E.EakvError):
        ctx.eakv_request_store(1)
    assert ctx.eakv_match(p)[1] == 0                          # nothing of request 1 is listed
    with pytest.raises(E.EakvError):
        ctx.eakv_request_release(1)                           # the failure closed it
    ctx.eakv_request_store(9)
    ctx.eakv_request_release(9)
    assert ctx.eakv_match(other)[1] == 4
    # restore fails in eakv_request_begin: the units it admitted (registered as its own) go too
    ctx2 = cp_ctx(eakv, b, 10, 64)
    for keys, agent in ((p, 0), (q, 1)):
        ctx2.eakv_turn_begin(0, len(keys) * b, keys, agent, 0)
        ctx2.eakv_turn_end()
    ctx2.eakv_selfcheck_fail_next_transfer(E.E_NOMEM)
    with pytest.raises(E.EakvError) as ei:
        ctx2.eakv_request_begin(5, 0, len(grown) * b, grown, 0, 1)
    assert ei.value.code == E.E_NOMEM
    assert ctx2.eakv_match(grown)[:2] == (0, 6)
    v = ctx2.eakv_request_begin(6, 0, len(grown) * b, grown, 0, 2)
    assert v["admit"].tolist() == [0] * 6 + [1] * 3
    ctx2.eakv_request_store(6)
    ctx2.eakv_request_release(6)
    assert ctx2.eakv_match(grown)[1] == 9
    ctx2.close()
    ctx.close()


def test_layered_end_refuses_a_wrong_event_count_and_keeps_the_turn_open(eakv):
    """eakv_turn_end_layers / eakv_request_store_layers: one event per layer group; a wrong count
    is refused before anything happens, and the turn can still be ended."""
    b = 4
    ctx = eakv.Context(num_layers=5, kv_heads=1, head_dim=8, block_size=b, gpu_blocks=32, host_blocks=32,
                       kv_base=None, control_plane_only=True)
    keys = np.arange(1, 5, dtype=np.uint64)
    ctx.eakv_turn_begin(0, 4 * b, keys, 0, 0)
    for bad in ([None], [None] * 4):                      # 5 layers in groups of 2 -> 3 events
        with pytest.raises(eakv.EakvError) as ei:
            ctx.eakv_turn_end_layers(2, bad)
        assert ei.value.code == eakv.E_INVAL
    ctx.eakv_turn_end_layers(2, [None] * 3)
    assert ctx.eakv_match(keys)[1] == 4
    more = np.arange(1, 7, dtype=np.uint64)
    ctx.eakv_request_begin(7, 0, 6 * b, more, 0, 1)
    with pytest.raises(eakv.EakvError) as ei:
        ctx.eakv_request_store_layers(7, 5, [None] * 2)   # one group of 5 layers -> 1 event
    assert ei.value.code == eakv.E_INVAL
    ctx.eakv_request_store_layers(7, 5, [None])
    ctx.eakv_request_release(7)
    assert ctx.eakv_match(more)[1] == 6
    ctx.close()


def test_layered_begin_refuses_bad_events_before_anything_changes(eakv):
    b = 4
    ctx = eakv.Context(num_layers=5, kv_heads=1, head_dim=8, block_size=b, gpu_blocks=32, host_blocks=32,
                       kv_base=None, control_plane_only=True)
    keys = np.arange(1, 5, dtype=np.uint64)
    before = ctx.eakv_get_stats()
    for bad in ((2, [1, 2]), (2, [1, None, 3]), (5, [])):          # 3 events needed; a NULL one; 1 needed
        with pytest.raises(eakv.EakvError) as ei:
            ctx.eakv_turn_begin(0, 4 * b, keys, 0, 0, layers=bad)
        assert ei.value.code == eakv.E_INVAL
        with pytest.raises(eakv.EakvError) as ei:
            ctx.eakv_request_begin(3, 0, 4 * b, keys, 0, 0, layers=bad)
        assert ei.value.code == eakv.E_INVAL
    assert ctx.eakv_get_stats() == before and ctx.eakv_match(keys)[:2] == (0, 0)
    v = ctx.eakv_turn_begin(0, 4 * b, keys, 0, 0, layers=(2, [1, 2, 3]))     # (bookkeeping only: never touched)
    assert v["admit"].tolist() == [1] * 4
    ctx.eakv_turn_end()
    ctx.close()


@pytest.mark.parametrize("seed", range(12))
def test_every_listed_unit_is_written_or_pending_under_random_begin_store_release(eakv, seed):
    """Requests begin, store and are released in random order, some of them released before their
    store.  A model of which slot holds whose bytes follows the views: a slot is written by the
    store of the request that owns it, an eviction forgets it, a release before the store takes
    the owner's pending units back.  After every call the tier lists exactly the written and the
    pending units at those slots, and a restore only ever reads a written slot of the right key."""
    import random
    from deferred_util import Prompts
    rng = random.Random(1000 + seed)
    b = 4
    R = rng.choice([1, 1, 2, 4])
    kh = 60 // R + 1 + rng.choice([0, 10, 40]) // R
    nb = rng.choice([130, 160, 220])
    ctx = cp_ctx(eakv, b, nb, kh, chunk_blocks=R, policy=rng.choice([0, 2]), kappa_blocks=max(1, 8 // R),
                 window_ms=20_000, len_window=8)
    prompts = Prompts(rng, b, agents=6)
    written, pending, begun, stored, busy = {}, {}, {}, set(), set()
    rid = now = restored = withdrawn = 0
    for step in range(400):
        now += rng.randrange(0, 3000)
        choices = []
        if len(begun) < 5 and len(busy) < 6:
            choices += ["begin"] * 3
        if any(r not in stored for r in begun):
            choices += ["store"] * 2
        if begun:
            choices += ["release"] * 2
        op = rng.choice(choices)
        if op == "begin":
            agent = rng.choice([a for a in range(6) if a not in busy])
            rid += 1
            toks = prompts.next_prompt(agent, 60 * b)
            keys = keys_of(toks, b)
            v = ctx.eakv_request_begin(rid, 0, len(toks), keys, agent, now)
            if v is None:
                continue
            ukeys = [int(k) for k in keys[R - 1::R]]
            for k in v["evicted_keys"].tolist():
                written.pop(k, None)
                pending.pop(k, None)
            if v["restore_hi"] > v["restore_lo"]:
                for c in range(v["restore_lo"] // R, -(-v["restore_hi"] // R)):
                    assert written.get(ukeys[c]) == int(v["slot"][c]), "restore of a slot that was never written"
                    restored += 1
            for c, a in enumerate(v["admit"].tolist()):
                if a:
                    pending[ukeys[c]] = (rid, int(v["slot"][c]))
            begun[rid] = agent
            busy.add(agent)
        elif op == "store":
            r = rng.choice([r for r in begun if r not in stored])
            ctx.eakv_request_store(r)
            stored.add(r)
            for k, (owner, s) in list(pending.items()):
                if owner == r:
                    written[k] = s
                    del pending[k]
        else:
            r = rng.choice(list(begun))
            ctx.eakv_request_release(r)
            if r not in stored:
                for k, (owner, s) in list(pending.items()):
                    if owner == r:
                        del pending[k]
                        withdrawn += 1
            stored.discard(r)
            busy.discard(begun.pop(r))
        ek, es = ctx.eakv_tier_export()
        assert dict(zip(ek.tolist(), es.tolist())) == {**written, **{k: s for k, (_, s) in pending.items()}}, step
    assert withdrawn > 0
    ctx.close()
