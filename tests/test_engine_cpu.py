"""The engine model (running-request cap, pinned GPU blocks, preemption with recomputation) on
the CPU: the library's bookkeeping (eakv_gpu_tier_acquire / eakv_gpu_tier_release_request,
eakv_tier_step_again) and the package's scheduler against oracle.engine, event for event."""
import random
from dataclasses import replace

import numpy as np
import pytest

from eakv_workloads import CONFIGS, SHAPES, make_trace
from oracle import closedloop as ocl
from oracle import engine as oen
from oracle import hash as ohash
from oracle.trace import GpuTier, TraceOracle


@pytest.fixture(scope="module")
def mods():
    from paper_2609_33762_b200 import build, closedloop, eakv
    build.build()
    return eakv, closedloop


def cp_ctx(eakv, b, gpu_blocks, host_blocks, **kw):
    return eakv.Context(num_layers=1, kv_heads=1, head_dim=8, block_size=b, gpu_blocks=gpu_blocks,
                        host_blocks=host_blocks, kv_base=None, control_plane_only=True, **kw)


def as_keys(keys):
    return np.asarray(keys, dtype=np.uint64)


@pytest.mark.parametrize("free_order", [0, 1])
def test_pinned_gpu_tier_random_requests(mods, free_order):
    """Random overlapping requests, some sharing a prefix: every acquire (fitting or refused) and
    every release leaves the library's GPU tier where the oracle's is."""
    eakv, _ = mods
    rng = random.Random(21 + free_order)
    for case in range(25):
        nb = rng.randrange(6, 30)
        g = GpuTier(nb, free_order)
        ctx = cp_ctx(eakv, 4, nb, 4, gpu_free_order=free_order)
        holders = []
        for rid in range(120):
            if holders and rng.random() < 0.45:
                victim = holders.pop(rng.randrange(len(holders)))
                g.release_request(victim)
                ctx.eakv_gpu_tier_release_request(victim)
            n = rng.randrange(0, nb)
            shared = rng.randrange(0, 3)
            keys = [1000 + j for j in range(shared)] + [rng.randrange(12) * 100 + j + 1 for j in range(n - shared)]
            keys = list(dict.fromkeys(keys))
            tail = rng.random() < 0.5
            want = g.acquire(rid, keys, tail)
            got = ctx.eakv_gpu_tier_acquire(rid, as_keys(keys), tail)
            if want is None:
                assert got is None
            else:
                assert got is not None
                assert (got[0].tolist(), got[1].tolist(), got[2]) == (want[0], want[1], want[2])
                holders.append(rid)
            # both tiers list the same keys in the same blocks
            probe = as_keys(sorted(set(list(g.order) + list(g.pinned))))
            for k in probe:
                G, _, ids, _ = ctx.eakv_match(as_keys([k]))
                assert G == 1 and ids[0] == (g.order.get(int(k)) if int(k) in g.order else g.pinned[int(k)][0])
        for rid in holders:
            g.release_request(rid)
            ctx.eakv_gpu_tier_release_request(rid)
        # everything released: a plain single-request step now behaves as in the oracle, which
        # shows that the recency order (not only the contents) was the same all along
        keys = [5000 + j for j in range(nb - 1)]
        want = g.step(keys, False)
        got = ctx.eakv_gpu_tier_step(as_keys(keys), False)
        assert (got[0].tolist(), got[1].tolist()) == (want[0], want[1])
        with pytest.raises(eakv.EakvError):
            ctx.eakv_gpu_tier_release_request(12345)           # holds nothing
        ctx.close()


def test_single_request_calls_are_refused_while_requests_hold_blocks(mods):
    eakv, _ = mods
    ctx = cp_ctx(eakv, 4, 16, 16)
    assert ctx.eakv_gpu_tier_acquire(7, as_keys([1, 2, 3]), True) is not None
    with pytest.raises(eakv.EakvError) as ei:
        ctx.eakv_gpu_tier_step(as_keys([9]), False)
    assert ei.value.code == eakv.E_INVAL
    with pytest.raises(eakv.EakvError) as ei:
        ctx.eakv_turn_begin(0, 4, as_keys([9]), 0, 0)
    assert ei.value.code == eakv.E_INVAL
    with pytest.raises(eakv.EakvError) as ei:
        ctx.eakv_gpu_tier_acquire(7, as_keys([4]), False)     # the id is in use
    assert ei.value.code == eakv.E_INVAL
    # too large for the tier even alone: an error, not "try again later"
    with pytest.raises(eakv.EakvError) as ei:
        ctx.eakv_gpu_tier_acquire(8, as_keys(range(100, 117)), False)
    assert ei.value.code == eakv.E_CAPACITY
    assert ctx.eakv_gpu_tier_acquire(8, as_keys(range(100, 114)), False) is None      # 14 > 16 - 4 held: busy
    ctx.eakv_gpu_tier_release_request(7)
    assert ctx.eakv_gpu_tier_acquire(8, as_keys(range(100, 114)), False) is not None
    ctx.eakv_gpu_tier_release_request(8)
    ctx.eakv_gpu_tier_step(as_keys([9]), False)
    ctx.close()


def test_later_lookup_keeps_the_decision_and_stays_out_of_the_windows(mods):
    """eakv_tier_step_again against the oracle's resumed lookup: same walk with the kept choice,
    and the admission windows afterwards decide as if the later lookup had not happened."""
    eakv, _ = mods
    from oracle.tier import HostTier
    rng = random.Random(5)
    for policy in (0, 1, 2):
        kw = dict(policy=policy, kappa_blocks=3, theta_percent=60, window_ms=40, len_window=6)
        o = HostTier(24, 4, **kw)
        ctx = cp_ctx(eakv, 4, 8, 24, **kw)
        now = 0
        for i in range(300):
            now += rng.randrange(0, 12)
            n = rng.randrange(0, 20)
            start = rng.randrange(0, 8) * 50
            keys = [start + j + 1 for j in range(n)]
            n_tok = 4 * n + rng.randrange(0, 4)
            agent = rng.randrange(5)
            decided = None if rng.random() < 0.7 else (rng.random() < 0.5)
            w = o.step(keys, n_tok, agent, now, decided=decided)
            g = ctx.eakv_tier_step(as_keys(keys), agent, n_tok, now, decided=decided)
            assert (g["hit"].tolist(), g["admit"].tolist(), g["slot"].tolist()) == (w.hit, w.admit, w.slot)
            assert list(zip(g["evicted_keys"].tolist(), g["evicted_slots"].tolist())) == w.evicted
            assert (g["save"], g["pressure"], g["new_chunks"], g["host_prefix_blocks"]) == \
                   (w.save, w.pressure, w.new_chunks, w.host_prefix_blocks)
        st = ctx.eakv_get_stats()
        for f in ("requests", "references", "hits", "admitted", "declined", "evicted", "declined_requests",
                  "pressure_requests"):
            assert st[f] == o.stats[f], f
        ctx.close()


def engine_begin(ctx, b, keys_of):
    """Test-only driver of one running request through the C-ABI bookkeeping."""
    def begin(request_id, tokens, agent, now_ms, decided):
        n = len(tokens)
        keys = keys_of(tokens)
        G, H, _, _ = ctx.eakv_match(keys)
        got = ctx.eakv_gpu_tier_acquire(request_id, keys, n % b != 0)
        if got is None:
            return None
        step = ctx.eakv_tier_step(keys, agent, n, now_ms, decided=decided)
        return dict(fresh_tokens=n - max(G, H) * b, loaded=max(H - G, 0), stored=int(step["admit"].sum()),
                    save=step["save"], G=G, H=H, gpu_block=got[1].tolist(), gpu_resident=got[0].tolist(),
                    hit=step["hit"].tolist(), admit=step["admit"].tolist(), slot=step["slot"].tolist(),
                    evicted=list(zip(step["evicted_keys"].tolist(), step["evicted_slots"].tolist())))
    return begin


def request_begin(ctx, b, keys_of):
    """The same through the library's request calls (bookkeeping only: every key is supplied)."""
    def begin(request_id, tokens, agent, now_ms, decided):
        v = ctx.eakv_request_begin(request_id, 0, len(tokens), keys_of(tokens), agent, now_ms, decided=decided)
        if v is None:
            return None
        ctx.eakv_request_store(request_id)
        return dict(fresh_tokens=v["fresh_tokens"], loaded=v["restore_hi"] - v["restore_lo"],
                    stored=v["n_stored_blocks"], save=bool(v["save"]), G=v["gpu_prefix_blocks"],
                    H=v["host_prefix_blocks"], gpu_block=v["gpu_block"].tolist(),
                    gpu_resident=v["gpu_resident"].tolist(), hit=v["hit"].tolist(), admit=v["admit"].tolist(),
                    slot=v["slot"].tolist(),
                    evicted=list(zip(v["evicted_keys"].tolist(), v["evicted_slots"].tolist())))
    return begin


@pytest.mark.parametrize("api", ["single-calls", "request-calls"])
@pytest.mark.parametrize("policy,kh,gpu_blocks,A,S,decode_us", [
    (0, 1024, 130, 8, 4, 20_000), (0, 160, 140, 8, 3, 60_000), (2, 200, 200, 6, 6, 40_000),
    (1, 300, 300, 8, 2, 10_000), (2, 160, 135, 8, 8, 100_000), (0, 1024, 130, 5, 1, 700)])
def test_engine_replay_matches_oracle(mods, policy, kh, gpu_blocks, A, S, decode_us, api):
    eakv, closedloop = mods
    cfg = CONFIGS["c0_big_tier"]
    shape = SHAPES[cfg.shape]
    b = shape.block_size
    trace = make_trace(cfg, agents=8, turns=8)
    kw = dict(policy=policy, kappa_blocks=10, window_ms=50, len_window=16)
    om = ocl.ServiceModel(t_pf_ns=40_000, h2d_bytes_per_us=9_000, d2h_bytes_per_us=7_000, tau_load_us=120)
    orc = TraceOracle(shape, gpu_blocks, kh, **kw)
    want = oen.replay(trace, orc, om, A, S, decode_us, shape.bytes_per_token)
    pm = closedloop.ServiceModel(t_pf_ns=40_000, h2d_bytes_per_us=9_000, d2h_bytes_per_us=7_000, tau_load_us=120)
    ctx = cp_ctx(eakv, b, gpu_blocks, kh, **kw)
    recs = []
    keys_of = lambda t: as_keys(ohash.hash_blocks(t.tolist(), b))
    begin = engine_begin(ctx, b, keys_of) if api == "single-calls" else request_begin(ctx, b, keys_of)
    release = ctx.eakv_gpu_tier_release_request if api == "single-calls" else ctx.eakv_request_release

    def logged_begin(*a):
        r = begin(*a)
        if r is not None:
            recs.append(r)
        return r

    got = closedloop.replay_engine(trace, logged_begin, release, pm, A, S, decode_us, shape.bytes_per_token, b)
    st = ctx.eakv_get_stats()
    ctx.close()
    assert got["events"] == want["events"]
    assert got["order"] == want["order"] and got["makespan_us"] == want["makespan_us"]
    assert got["preemptions"] == want["preemptions"]
    assert got["recomputed_after_preemption"] == want["totals"]["preempt_recomputed_tokens"]
    assert got["resumed_lookups"] == want["preemptions"]
    assert len(recs) == len(orc.records)
    for g, w in zip(recs, orc.records):
        for f in ("G", "H", "hit", "admit", "slot", "evicted", "gpu_resident", "gpu_block", "loaded", "stored",
                  "fresh_tokens", "save"):
            assert g[f] == w[f], f
    for f in ("requests", "references", "hits", "admitted", "declined", "evicted"):
        assert st[f] == orc.host.stats[f], f
    if S > 1 and gpu_blocks <= 200:
        assert got["preemptions"] > 0


def test_config3_full_trace_engine_parity(mods):
    """All 1,280 calls of config 3 (conditioned admission, 32 GiB host tier) on the engine model
    with the paper's cap of 16 running requests and a GPU tier of 96 GiB, against the oracle."""
    eakv, closedloop = mods
    from full_trace_util import trace_and_keys
    cfg, shape, trace, agent_keys = trace_and_keys("c3")
    b = shape.block_size
    gpu_blocks = (96 << 30) // shape.block_bytes
    kh = cfg.host_blocks
    kw = dict(policy=2, kappa_blocks=cfg.kappa_blocks)
    om = ocl.ServiceModel()
    want = oen.replay(trace, TraceOracle(shape, gpu_blocks, kh, **kw), om, 16, 16, 2_000_000,
                      shape.bytes_per_token, agent_keys=agent_keys)
    ctx = cp_ctx(eakv, b, gpu_blocks, kh, **kw)
    np_keys = {a: as_keys(k) for a, k in agent_keys.items()}
    tasks = sorted(trace.agent_tokens)
    by_len = {}

    def keys_of(tokens):            # the caller passes a prefix of some agent's stream: find whose
        return by_len[id(tokens.base if tokens.base is not None else tokens)][: len(tokens) // b]

    for a in tasks:
        by_len[id(trace.agent_tokens[a])] = np_keys[a]
    got = closedloop.replay_engine(trace, request_begin(ctx, b, keys_of), ctx.eakv_request_release,
                                   closedloop.ServiceModel(), 16, 16, 2_000_000, shape.bytes_per_token, b)
    ctx.close()
    assert got["events"] == want["events"] and got["makespan_us"] == want["makespan_us"]
    assert got["preemptions"] == want["preemptions"]
    assert got["recomputed_after_preemption"] == want["totals"]["preempt_recomputed_tokens"]
    assert len(got["order"]) == 1280
