"""The C++ control plane (eakv_match, eakv_tier_step, eakv_gpu_tier_step) against the oracle,
on the CPU: a control-plane-only context makes no CUDA call, so this runs without a GPU.
Keys come from the oracle's hash here; the GPU tests check the hash kernel itself."""
import random
from dataclasses import replace

import numpy as np
import pytest

from eakv_workloads import CONFIGS, SHAPES, make_trace
from oracle import hash as ohash
from oracle.tier import CapacityError, HostTier
from oracle.trace import GpuTier, TraceOracle


@pytest.fixture(scope="module")
def eakv():
    from paper_2609_33762_b200 import build, eakv as m
    build.build()
    return m


def drive_chunked(ctx, trace, b, R):
    """Two granularities: block keys for the GPU tier, one key per full chunk for the host."""
    recs = []
    for req in trace.requests:
        toks = trace.prompt(req)
        keys = as_keys(ohash.hash_blocks(toks.tolist(), b))
        G = ctx.eakv_match(keys)[0]
        chunk_keys = np.ascontiguousarray(keys[R - 1::R])
        _, Hc, _, _ = ctx.eakv_match(chunk_keys)
        step = ctx.eakv_tier_step(chunk_keys, req.agent, len(toks), req.time_ms)
        res, blk, tail = ctx.eakv_gpu_tier_step(keys, len(toks) % b != 0)
        if tail >= 0:
            ctx.eakv_gpu_tier_release(tail)
        recs.append((keys, G, Hc * R, step, res, blk))
    return recs


def cp_ctx(eakv, block_size, gpu_blocks, host_blocks, **kw):
    return eakv.Context(num_layers=1, kv_heads=1, head_dim=8, block_size=block_size,
                        gpu_blocks=gpu_blocks, host_blocks=host_blocks, kv_base=None,
                        control_plane_only=True, **kw)


def as_keys(keys):
    return np.asarray(keys, dtype=np.uint64)


@pytest.mark.parametrize("policy", [0, 1, 2])
@pytest.mark.parametrize("telemetry", [1, 0])
def test_tier_step_random_requests(eakv, policy, telemetry):
    rng = random.Random(100 + 10 * policy + telemetry)
    for case in range(40):
        K = rng.randrange(3, 40)
        b = rng.choice([1, 4, 16])
        kappa = rng.choice([0, 1, 2, 5, 100])
        theta = rng.choice([50, 95, 100])
        window = rng.choice([5, 50, 10_000])
        lw = rng.choice([1, 3, 256])
        ctx = cp_ctx(eakv, b, 8, K, policy=policy, kappa_blocks=kappa, theta_percent=theta,
                     window_ms=window, len_window=lw, telemetry=telemetry)
        tier = HostTier(K, b, policy, kappa, theta, window, lw, bool(telemetry))
        now = 0
        for _ in range(rng.randrange(5, 60)):
            agent = rng.randrange(5)
            n = rng.randrange(0, K + 1)
            start = rng.randrange(0, 4)
            keys = [1000 * agent + start + j for j in range(n)]
            if n > 2 and rng.random() < 0.3:            # a foreign key in the middle: isolated hits after it
                keys[rng.randrange(1, n)] = 999_000 + rng.randrange(50)
            n_tokens = n * b + rng.randrange(0, b)
            now += rng.choice([0, 1, 7, 100])
            G, H, _, slots = ctx.eakv_match(as_keys(keys))
            assert H == tier.leading_run(keys)
            assert slots.tolist() == [tier.slot_of(k) for k in keys[:H]]
            want = tier.step(keys, n_tokens, agent, now)
            got = ctx.eakv_tier_step(as_keys(keys), agent, n_tokens, now)
            assert got["hit"].tolist() == want.hit and got["admit"].tolist() == want.admit
            assert got["slot"].tolist() == want.slot
            assert list(zip(got["evicted_keys"].tolist(), got["evicted_slots"].tolist())) == want.evicted
            assert (got["host_prefix_blocks"], got["new_chunks"], got["pressure"], got["save"]) == \
                   (want.host_prefix_blocks, want.new_chunks, want.pressure, want.save)
        st = ctx.eakv_get_stats()
        for f in ("requests", "references", "hits", "admitted", "declined", "evicted",
                  "declined_requests", "pressure_requests"):
            assert st[f] == tier.stats[f], f
        assert st["resident"] == len(tier.order)
        ctx.close()


@pytest.mark.parametrize("free_order", [0, 1])
def test_gpu_tier_random_requests(eakv, free_order):
    rng = random.Random(7 + free_order)
    for case in range(60):
        NB = rng.randrange(2, 30)
        ctx = cp_ctx(eakv, 4, NB, 4, gpu_free_order=free_order)
        g = GpuTier(NB, free_order)
        for _ in range(rng.randrange(3, 40)):
            agent = rng.randrange(4)
            tail = rng.random() < 0.5
            n = rng.randrange(0, NB - int(tail) + 1)
            keys = [100 * agent + j for j in range(n)]
            G, _, gids, _ = ctx.eakv_match(as_keys(keys))
            lead = 0
            for k in keys:
                if k not in g:
                    break
                lead += 1
            assert G == lead and gids.tolist() == [g.order[k] for k in keys[:G]]
            want = g.step(keys, tail)
            res, blk, t = ctx.eakv_gpu_tier_step(as_keys(keys), tail)
            assert (res.tolist(), blk.tolist(), t) == want
            if tail:
                g.release(t)
                ctx.eakv_gpu_tier_release(t)
        ctx.close()


def drive(ctx, trace, b, limit=None):
    """The harness's control sequence with oracle keys instead of the hash kernel."""
    recs = []
    for i, req in enumerate(trace.requests):
        if limit is not None and i >= limit:
            break
        toks = trace.prompt(req)
        keys = as_keys(ohash.hash_blocks(toks.tolist(), b))
        G, H, _, slots = ctx.eakv_match(keys)
        step = ctx.eakv_tier_step(keys, req.agent, len(toks), req.time_ms)
        res, blk, tail = ctx.eakv_gpu_tier_step(keys, len(toks) % b != 0)
        if tail >= 0:
            ctx.eakv_gpu_tier_release(tail)
        recs.append((keys, G, H, step, res, blk))
    return recs


def compare(recs, oracle_records):
    assert len(recs) == len(oracle_records)
    for (keys, G, H, step, res, blk), w in zip(recs, oracle_records):
        assert [int(k) for k in keys] == w["keys"]
        assert (G, H, step["new_chunks"], step["pressure"], step["save"]) == \
               (w["G"], w["H"], w["new_chunks"], w["pressure"], w["save"])
        assert step["hit"].tolist() == w["hit"] and step["admit"].tolist() == w["admit"]
        assert step["slot"].tolist() == w["slot"]
        assert list(zip(step["evicted_keys"].tolist(), step["evicted_slots"].tolist())) == w["evicted"]
        assert res.tolist() == w["gpu_resident"] and blk.tolist() == w["gpu_block"]


@pytest.mark.parametrize("cfg_name", ["c0", "c0_big_tier"])
def test_config0_control_plane_on_cpu(eakv, cfg_name):
    cfg = CONFIGS[cfg_name]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg)
    oracle = TraceOracle(shape, cfg.gpu_blocks, cfg.host_blocks)
    oracle.run(trace)
    ctx = cp_ctx(eakv, shape.block_size, cfg.gpu_blocks, cfg.host_blocks)
    compare(drive(ctx, trace, shape.block_size), oracle.records)
    ctx.close()


@pytest.mark.parametrize("policy", [1, 2])
def test_policies_on_a_scaled_down_config2_trace(eakv, policy):
    cfg = replace(CONFIGS["c2"], shape="tiny", agents=8, turns=16, first_prompt=400,
                  append_median=150.0, context_cap=3000, tool_gap_mean_ms=15_000.0)
    shape = SHAPES["tiny"]
    trace = make_trace(cfg, seed=31)
    kw = dict(policy=policy, kappa_blocks=6, window_ms=60_000, len_window=32)
    oracle = TraceOracle(shape, 256, 300, **kw)
    oracle.run(trace)
    ctx = cp_ctx(eakv, shape.block_size, 256, 300, **kw)
    compare(drive(ctx, trace, shape.block_size), oracle.records)
    assert oracle.host.stats["declined_requests"] > 0
    ctx.close()


@pytest.mark.parametrize("policy,R", [(0, 4), (2, 4), (2, 8), (1, 2)])
def test_two_granularities(eakv, policy, R):
    """Host chunks of R blocks over single GPU blocks: u and kappa count chunks, the tier holds
    chunks, coverage is chunk-aligned."""
    cfg = replace(CONFIGS["c2"], shape="tiny", agents=6, turns=14, first_prompt=500,
                  append_median=200.0, context_cap=3500, tool_gap_mean_ms=15_000.0)
    shape = SHAPES["tiny"]
    trace = make_trace(cfg, seed=41)
    kw = dict(policy=policy, kappa_blocks=2, window_ms=60_000, len_window=32)
    kh = 700 // R                                            # about 700 blocks of host tier
    oracle = TraceOracle(shape, 256, kh, chunk_blocks=R, **kw)
    oracle.run(trace)
    ctx = cp_ctx(eakv, shape.block_size, 256, kh, chunk_blocks=R, **kw)
    compare(drive_chunked(ctx, trace, shape.block_size, R), oracle.records)
    assert all(r["H"] % R == 0 for r in oracle.records)
    if policy != 1:                                             # the fixed filter declines it all
        assert any(r["H"] > r["G"] for r in oracle.records)      # restores do happen
    ctx.close()


def test_capacity_and_argument_errors(eakv):
    ctx = cp_ctx(eakv, 4, 6, 3)
    keys = as_keys([1, 2, 3, 4])
    ctx.eakv_tier_step(keys[:2], 0, 8, 0)
    before = ctx.eakv_get_stats()
    with pytest.raises(eakv.EakvError) as ei:
        ctx.eakv_tier_step(keys, 0, 16, 1)                 # 4 blocks > K_H = 3
    assert ei.value.code == eakv.E_CAPACITY and ctx.eakv_get_stats() == before
    with pytest.raises(eakv.EakvError) as ei:
        ctx.eakv_gpu_tier_step(as_keys(range(1, 7)), True)  # 6 blocks + tail > 6
    assert ei.value.code == eakv.E_CAPACITY
    res, blk, tail = ctx.eakv_gpu_tier_step(as_keys([1, 2]), True)
    assert tail == 2
    with pytest.raises(eakv.EakvError) as ei:
        ctx.eakv_gpu_tier_step(as_keys([1, 2, 3, 4, 5]), True)   # the outstanding tail counts
    assert ei.value.code == eakv.E_CAPACITY
    for bad, code in ((0, eakv.E_INVAL), (7, eakv.E_RANGE), (-1, eakv.E_RANGE)):
        with pytest.raises(eakv.EakvError) as ei:
            ctx.eakv_gpu_tier_release(bad)                 # 0 is a keyed block, 7/-1 out of range
        assert ei.value.code == code
    ctx.eakv_gpu_tier_release(tail)
    # data-plane calls are refused on a control-plane-only context; sync and stats still work
    for call in (lambda: ctx.eakv_store([0], None, [0]), lambda: ctx.eakv_load([0], [0]),
                 lambda: ctx.eakv_hash_blocks(16, 64, 1, 16)):
        with pytest.raises(eakv.EakvError) as ei:
            call()
        assert ei.value.code == eakv.E_INVAL
    ctx.eakv_sync()
    ctx.close()


def test_oracle_capacity_error_matches(eakv):
    t = HostTier(2, 4)
    with pytest.raises(CapacityError):
        t.step([1, 2, 3], 12, 0, 0)


def test_shared_system_prompt_is_deduplicated_across_agents(eakv):
    """A prefix common to all agents (a weakly shared pool): its chunks are stored once and hit
    by every other agent; product and oracle agree request by request."""
    cfg = replace(CONFIGS["c0_big_tier"], shared_prefix_tokens=256)
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg)
    oracle = TraceOracle(shape, cfg.gpu_blocks, cfg.host_blocks)
    oracle.run(trace)
    ctx = cp_ctx(eakv, shape.block_size, cfg.gpu_blocks, cfg.host_blocks)
    compare(drive(ctx, trace, shape.block_size), oracle.records)
    ctx.close()
    first_turns = [r for r in oracle.records[:8]]
    assert first_turns[0]["H"] == 0 and all(r["H"] == 16 for r in first_turns[1:])   # 256 tokens = 16 blocks
    plain = TraceOracle(shape, cfg.gpu_blocks, cfg.host_blocks)
    plain.run(make_trace(CONFIGS["c0_big_tier"]))
    assert oracle.totals["stored_blocks"] < plain.totals["stored_blocks"]


def test_config3_full_trace_control_plane_on_cpu(eakv):
    """All 1,280 requests (3.88 M references) of the config 2/3 trace at the 32 GiB tier under
    capacity-conditioned admission, through the C++ control plane and the oracle."""
    cfg = CONFIGS["c3"]
    shape = SHAPES[cfg.shape]
    b = shape.block_size
    trace = make_trace(cfg)
    agent_keys = {a: ohash.hash_blocks(t.tolist(), b) for a, t in trace.agent_tokens.items()}
    kw = dict(policy=2, kappa_blocks=cfg.kappa_blocks)
    oracle = TraceOracle(shape, cfg.gpu_blocks, cfg.host_blocks, **kw)
    ctx = cp_ctx(eakv, b, cfg.gpu_blocks, cfg.host_blocks, **kw)
    for r in trace.requests:
        keys = agent_keys[r.agent][: r.n_tokens // b]
        w = oracle.turn(range(r.n_tokens), r.agent, r.time_ms, keys=keys)
        k = as_keys(keys)
        G, H, _, _ = ctx.eakv_match(k)
        st = ctx.eakv_tier_step(k, r.agent, r.n_tokens, r.time_ms)
        res, blk, tail = ctx.eakv_gpu_tier_step(k, r.n_tokens % b != 0)
        if tail >= 0:
            ctx.eakv_gpu_tier_release(tail)
        assert (G, H, st["pressure"], st["save"]) == (w["G"], w["H"], w["pressure"], w["save"])
        assert np.array_equal(st["admit"], np.asarray(w["admit"], dtype=np.uint8))
        assert np.array_equal(st["slot"], np.asarray(w["slot"], dtype=np.int32))
        assert np.array_equal(blk, np.asarray(w["gpu_block"], dtype=np.int32))
        oracle.records.clear()
    st = ctx.eakv_get_stats()
    for f in ("requests", "references", "hits", "admitted", "declined", "evicted", "declined_requests",
              "pressure_requests"):
        assert st[f] == oracle.host.stats[f], f
    assert 0 < st["declined_requests"] < st["requests"]
    ctx.close()


def test_reverse_free_order_whole_trace(eakv):
    """C0 with the tail-first GPU recency order: every record equals the oracle's, and the GPU
    tier keeps more prefix blocks than with the ascending order."""
    cfg = CONFIGS["c0_big_tier"]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg, agents=3)      # three agents: the pool holds a part of each prompt
    totals = {}
    for order in (0, 1):
        orc = TraceOracle(shape, cfg.gpu_blocks, cfg.host_blocks, gpu_free_order=order)
        orc.run(trace)
        ctx = cp_ctx(eakv, shape.block_size, cfg.gpu_blocks, cfg.host_blocks, gpu_free_order=order)
        compare(drive(ctx, trace, shape.block_size), orc.records)
        ctx.close()
        totals[order] = orc.totals["gpu_hit_blocks"]
    assert totals[1] > totals[0]


def test_free_order_argument_is_checked(eakv):
    with pytest.raises(eakv.EakvError):
        cp_ctx(eakv, 4, 8, 8, gpu_free_order=2)


@pytest.mark.parametrize("policy", [0, 1, 2])
def test_tier_export_import_restart(eakv, policy):
    """Stop after half of the trace, export the host tier's index and the admission windows, import
    them into a fresh context and go on: every later decision equals the uninterrupted oracle run
    whose GPU tier was emptied at the same point."""
    cfg = CONFIGS["c0_big_tier"]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg, agents=5)
    # first prompts (32 blocks) pass the filter; short windows so that the pressure signal moves
    kw = dict(policy=policy, kappa_blocks=40, window_ms=30, len_window=8)
    half = len(trace.requests) // 2
    orc = TraceOracle(shape, cfg.gpu_blocks, 300, **kw)
    for i, req in enumerate(trace.requests):
        if i == half:
            orc.gpu = GpuTier(cfg.gpu_blocks)                # the engine's blocks do not survive
        orc.turn(trace.prompt(req), req.agent, req.time_ms)
    first, second = replace_requests(trace, 0, half), replace_requests(trace, half, None)
    ctx = cp_ctx(eakv, shape.block_size, cfg.gpu_blocks, 300, **kw)
    recs = drive(ctx, first, shape.block_size)
    keys, slots = ctx.eakv_tier_export()
    windows = ctx.eakv_admission_export()
    assert list(zip(keys.tolist(), slots.tolist())) == list(orc_order_at(trace, shape, cfg, half, kw))
    ctx.close()
    ctx = cp_ctx(eakv, shape.block_size, cfg.gpu_blocks, 300, **kw)
    ctx.eakv_tier_import(keys, slots)
    ctx.eakv_admission_import(windows)
    assert ctx.eakv_admission_export().tolist() == windows.tolist()
    for bad in ([], [5], [1, 3], [0, 2, 7], [0, 0, 3, 1], [0, 9, 1, 2, 3, 4, 5, 6, 7, 8, 9, 0]):
        with pytest.raises(eakv.EakvError):
            ctx.eakv_admission_import(np.array(bad, dtype=np.int64))
    assert ctx.eakv_admission_export().tolist() == windows.tolist()
    assert ctx.eakv_get_stats()["resident"] == len(keys)
    recs += drive(ctx, second, shape.block_size)
    compare(recs, orc.records)
    if policy == 2:
        # the windows matter: with the index alone the restarted context decides differently
        assert sum(int(r["pressure"]) for r in orc.records[half:]) > 0
        cold = cp_ctx(eakv, shape.block_size, cfg.gpu_blocks, 300, **kw)
        cold.eakv_tier_import(keys, slots)
        cold_recs = drive(cold, second, shape.block_size)
        cold.close()
        assert [int(r[3]["save"]) for r in cold_recs] != [int(w["save"]) for w in orc.records[half:]]
    # import is refused into a tier that is not empty, and for repeated slots or keys
    with pytest.raises(eakv.EakvError):
        ctx.eakv_tier_import(keys[:1], slots[:1])
    ctx.close()
    ctx = cp_ctx(eakv, shape.block_size, cfg.gpu_blocks, 300, **kw)
    for bad_k, bad_s in (([1, 2], [0, 0]), ([1, 1], [0, 1]), ([1], [300]), ([1], [-1])):
        with pytest.raises(eakv.EakvError):
            ctx.eakv_tier_import(np.array(bad_k, np.uint64), np.array(bad_s, np.int32))
        assert ctx.eakv_get_stats()["resident"] == 0 and len(ctx.eakv_tier_export()[0]) == 0
    ctx.eakv_tier_import(np.array([7, 9], np.uint64), np.array([5, 0], np.int32))
    st = ctx.eakv_tier_step(as_keys([11, 12, 13]), 0, 12, 0)          # unused slots, ascending
    assert st["slot"].tolist() == [1, 2, 3]
    ctx.close()


def replace_requests(trace, lo, hi):
    from copy import copy
    t = copy(trace)
    t.requests = trace.requests[lo:hi]
    return t


def orc_order_at(trace, shape, cfg, n, kw):
    """Host tier order (key, slot), least recent first, after the first n requests."""
    o = TraceOracle(shape, cfg.gpu_blocks, 300, **kw)
    for req in trace.requests[:n]:
        o.turn(trace.prompt(req), req.agent, req.time_ms)
    return o.host.order.items()


def test_random_traces_across_every_option(eakv):
    """Small random traces through every combination of policy, chunking, telemetry and GPU free
    order: the C++ control plane and the oracle must agree on every record."""
    rng = random.Random(2024)
    cfg0 = CONFIGS["c0_big_tier"]
    shape = SHAPES[cfg0.shape]
    for case in range(24):
        policy = case % 3
        R = (1, 2, 4)[(case // 3) % 3]
        telemetry = (case // 9) % 2
        order = rng.randrange(2)
        agents = rng.randrange(2, 7)
        cfg = replace(cfg0, seed=100 + case, append_median=float(rng.choice([60, 200, 500])),
                      first_prompt=rng.choice([96, 256, 512]))
        trace = make_trace(cfg, agents=agents, turns=rng.randrange(3, 8))
        kh = max(trace.config.context_cap // (shape.block_size * R) + 1, rng.randrange(40, 400) // R)
        kw = dict(policy=policy, kappa_blocks=rng.choice([0, 2, 8, 30]), theta_percent=rng.choice([50, 95, 100]),
                  window_ms=rng.choice([5, 40, 60000]), len_window=rng.choice([4, 256]), telemetry=telemetry)
        orc = TraceOracle(shape, cfg.gpu_blocks, kh, chunk_blocks=R, gpu_free_order=order, **kw)
        orc.run(trace)
        ctx = cp_ctx(eakv, shape.block_size, cfg.gpu_blocks, kh, chunk_blocks=R, gpu_free_order=order, **kw)
        recs = drive_chunked(ctx, trace, shape.block_size, R) if R > 1 else drive(ctx, trace, shape.block_size)
        compare(recs, orc.records)
        ctx.close()


@pytest.mark.parametrize("period,max_age", [(1, 5), (10, 0), (10, 25), (100, 50), (1000, 5000)])
def test_published_reports_random_requests(eakv, period, max_age):
    """Tier reports published at intervals (Appendix D): capacity-conditioned admission that reads
    the latest report, fresh or stale, against the oracle on random request streams."""
    rng = random.Random(300 + period + max_age)
    engaged = stale = 0
    for case in range(40):
        K = rng.randrange(3, 40)
        b = rng.choice([1, 4, 16])
        kw = dict(policy=2, kappa_blocks=rng.choice([0, 1, 2, 5]), theta_percent=rng.choice([50, 95, 100]),
                  window_ms=rng.choice([50, 400, 10_000]), len_window=rng.choice([1, 3, 256]),
                  telemetry_period_ms=period, telemetry_max_age_ms=max_age)
        ctx = cp_ctx(eakv, b, 8, K, **kw)
        tier = HostTier(K, b, **kw)
        now = 0
        for _ in range(rng.randrange(5, 80)):
            agent = rng.randrange(5)
            n = rng.randrange(0, K + 1)
            keys = [1000 * agent + rng.randrange(0, 4) + j for j in range(n)]
            n_tokens = n * b + rng.randrange(0, b)
            now += rng.choice([0, 1, 7, 100, 3 * period])
            decided = None if rng.random() < 0.85 else (rng.random() < 0.5)
            want = tier.step(keys, n_tokens, agent, now, decided=decided)
            got = ctx.eakv_tier_step(as_keys(keys), agent, n_tokens, now, decided=decided)
            assert got["hit"].tolist() == want.hit and got["admit"].tolist() == want.admit
            assert got["slot"].tolist() == want.slot
            assert (got["pressure"], got["save"]) == (want.pressure, want.save)
            engaged += want.pressure
            stale += tier.report is not None and max_age > 0 and now - tier.report[0] > max_age
        ctx.close()
    assert engaged > 0
    if 0 < max_age < period:
        assert stale > 0


def test_scaled_config2_trace_with_the_papers_report_interval(eakv):
    """Config 2's generator scaled down, capacity-conditioned admission reading reports published
    every second that stay fresh for five (the paper's parameter table), whole trace against the
    oracle; and the decisions differ from the synchronous reading somewhere, so the reports matter."""
    cfg = replace(CONFIGS["c2"], shape="tiny", agents=8, turns=16, first_prompt=400,
                  append_median=150.0, context_cap=3000, tool_gap_mean_ms=5_000.0)
    shape = SHAPES["tiny"]
    trace = make_trace(cfg, seed=31)
    base = dict(policy=2, kappa_blocks=6, window_ms=60_000, len_window=32)
    kw = dict(base, telemetry_period_ms=1000, telemetry_max_age_ms=5000)
    oracle = TraceOracle(shape, 256, 300, **kw)
    oracle.run(trace)
    ctx = cp_ctx(eakv, shape.block_size, 256, 300, **kw)
    compare(drive(ctx, trace, shape.block_size), oracle.records)
    ctx.close()
    sync = TraceOracle(shape, 256, 300, **base)
    sync.run(trace)
    assert [r["pressure"] for r in sync.records] != [r["pressure"] for r in oracle.records]
    assert oracle.host.stats["declined_requests"] > 0


def test_admission_export_carries_the_latest_report(eakv):
    kw = dict(policy=2, kappa_blocks=0, theta_percent=50, window_ms=60_000, telemetry_period_ms=1000,
              telemetry_max_age_ms=5000)
    ctx = cp_ctx(eakv, 4, 8, 4, **kw)
    tier = HostTier(4, 4, **kw)
    steps = [([1, 2, 3, 4], 40, 0, 100), ([5, 6], 40, 1, 1500), ([1, 2], 40, 0, 1900), ([7], 40, 1, 2100)]
    for keys, n, agent, now in steps:
        tier.step(keys, n, agent, now)
        ctx.eakv_tier_step(as_keys(keys), agent, n, now)
    assert tier.report == (2000, 4, 4)
    state = ctx.eakv_admission_export()
    assert state[-3:].tolist() == [2000, 4, 4]
    k, s = ctx.eakv_tier_export()
    ctx.close()
    ctx = cp_ctx(eakv, 4, 8, 4, **kw)
    ctx.eakv_tier_import(k, s)
    ctx.eakv_admission_import(state)
    # 2,900 ms: still the report of 2,000 ms, which the restarted context can only know from the import
    want = tier.step([8], 40, 0, 2900)
    got = ctx.eakv_tier_step(as_keys([8]), 0, 40, 2900)
    assert want.pressure and got["pressure"] and not got["save"]
    ctx.close()
