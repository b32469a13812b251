"""GPU parity on whole agent traces: every per-request output (keys, G, H, hit/admit/slot
sequences, evictions, GPU block assignment) and every byte of KV in both tiers must equal
the oracle's, for config 0, its large-tier sibling, and both admission policies."""
import numpy as np
import pytest

from eakv_workloads import CONFIGS, SHAPES, key_words_numpy, key_words_torch, make_trace, normal_bf16_words
from oracle.trace import TraceOracle

from gpu_util import require_gpu, torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def normal_payload(keys, q, n_words):
    """Config 0's payload: bf16(N(0,1)) drawn per (block key, piece)."""
    return np.stack([normal_bf16_words((0, int(k), q), n_words) for k in keys])


def compare_records(got, want):
    assert len(got) == len(want)
    for g, w in zip(got, want):
        assert [int(x) for x in g["keys"]] == w["keys"]
        for f in ("n_tokens", "G", "H", "new_chunks", "pressure", "save", "loaded", "stored",
                  "fresh_tokens", "filled"):
            assert g[f] == w[f], f
        for f in ("hit", "admit", "slot", "gpu_resident", "gpu_block"):
            assert [int(x) for x in g[f]] == [int(x) for x in w[f]], f
        assert [(int(k), int(s)) for k, s in g["evicted"]] == w["evicted"]


def compare_bytes(server, oracle):
    server.ctx.eakv_sync()
    for q, t in enumerate(server.pool.pieces):
        got = t.cpu().numpy().view(np.uint8)
        # only key-indexed GPU blocks have defined content
        for key, blk in oracle.gpu.order.items():
            assert np.array_equal(got[blk], oracle.pool[q][blk]), (q, blk)
    tier = server.ctx.tier_host_view()
    for key, slot in oracle.host.order.items():
        assert np.array_equal(tier[slot], oracle.tier[slot]), slot


@pytest.mark.parametrize("cfg_name", ["c0", "c0_big_tier"])
@pytest.mark.parametrize("link", [0, 1])
def test_config0_bit_exact(cfg_name, link):
    from paper_2609_33762_b200.harness import AgentServer
    cfg = CONFIGS[cfg_name]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg)
    payload = normal_payload if cfg_name == "c0" and link == 0 else key_words_numpy
    oracle = TraceOracle(shape, cfg.gpu_blocks, cfg.host_blocks, payload=payload)
    oracle.run(trace)
    server = AgentServer(shape, cfg.gpu_blocks, cfg.host_blocks, payload, native_turn=False, link_strategy=link,
                         staging_bytes=7 * shape.block_bytes, incremental_hash=(link == 1),
                         min_staged_run_bytes=-1 if link == 1 else 0)
    server.run(trace)
    compare_records(server.records, oracle.records)
    assert server.totals == oracle.totals
    compare_bytes(server, oracle)
    st = server.ctx.eakv_get_stats()
    for f in ("requests", "references", "hits", "admitted", "declined", "evicted",
              "declined_requests", "pressure_requests"):
        assert st[f] == oracle.host.stats[f], f
    assert st["blocks_stored"] == oracle.totals["stored_blocks"]
    assert st["blocks_loaded"] == oracle.totals["loaded_blocks"]
    server.close()


@pytest.mark.parametrize("policy,kappa", [(1, 8), (2, 8), (2, 2), (1, 40)])
def test_admission_policies_bit_exact(policy, kappa):
    """Tool-gap interleave (config 2's recipe) on the tiny KV shape with a tier far below
    the working set, so the pressure signal engages; device payload generator."""
    from dataclasses import replace
    from paper_2609_33762_b200.harness import AgentServer
    cfg = replace(CONFIGS["c2"], shape="tiny", agents=6, turns=14, first_prompt=300,
                  append_median=120.0, context_cap=1800, tool_gap_mean_ms=20_000.0)
    shape = SHAPES["tiny"]
    trace = make_trace(cfg, seed=21)
    kw = dict(policy=policy, kappa_blocks=kappa, window_ms=60_000, len_window=16)
    oracle = TraceOracle(shape, 128, 160, payload=key_words_numpy, **kw)
    oracle.run(trace)
    dev_payload = lambda keys, q, n: key_words_torch(keys.astype(np.int64), q, n, "cuda")
    server = AgentServer(shape, 128, 160, dev_payload, native_turn=False, **kw)
    server.run(trace)
    compare_records(server.records, oracle.records)
    compare_bytes(server, oracle)
    assert oracle.host.stats["declined_requests"] > 0          # the filter did engage
    if policy == 2:
        assert 0 < oracle.host.stats["pressure_requests"] < len(trace.requests)
    server.close()


def test_telemetry_off_uses_estimate_alone():
    from dataclasses import replace
    from paper_2609_33762_b200.harness import AgentServer
    cfg = replace(CONFIGS["c2"], shape="tiny", agents=5, turns=8, first_prompt=300,
                  append_median=100.0, context_cap=1500)
    shape = SHAPES["tiny"]
    trace = make_trace(cfg, seed=22)
    kw = dict(policy=2, kappa_blocks=4, telemetry=0)
    oracle = TraceOracle(shape, 128, 100, **{**kw, "telemetry": False})
    oracle.run(trace)
    server = AgentServer(shape, 128, 100, None, data_plane=False, **kw)
    server.run(trace)
    compare_records(server.records, oracle.records)
    server.close()


def test_tier_step_capacity_error_changes_nothing():
    from paper_2609_33762_b200 import eakv
    from paper_2609_33762_b200.harness import AgentServer
    shape = SHAPES["tiny"]
    server = AgentServer(shape, 16, 4, None, data_plane=False)
    keys = np.arange(1, 6, dtype=np.uint64)
    server.ctx.eakv_tier_step(keys[:2], 0, 32, 0)
    before = server.ctx.eakv_get_stats()
    with pytest.raises(eakv.EakvError) as ei:
        server.ctx.eakv_tier_step(keys, 0, 80, 1)
    assert ei.value.code == eakv.E_CAPACITY
    assert server.ctx.eakv_get_stats() == before
    with pytest.raises(eakv.EakvError) as ei:
        server.ctx.eakv_gpu_tier_step(np.arange(1, 18, dtype=np.uint64), False)
    assert ei.value.code == eakv.E_CAPACITY
    G, H, gids, slots = server.ctx.eakv_match(keys)
    assert (G, H) == (0, 2) and slots.tolist() == [0, 1]
    server.close()


@pytest.mark.parametrize("R,policy,link", [(4, 0, 1), (4, 2, 0), (8, 0, 1)])
def test_two_granularities_bit_exact(R, policy, link):
    """Host chunks of R GPU blocks (the paper's 1,024-token chunks over 16-token blocks, scaled
    down): records and every resident byte against the oracle."""
    from dataclasses import replace
    from paper_2609_33762_b200.harness import AgentServer
    cfg = replace(CONFIGS["c2"], shape="tiny", agents=6, turns=12, first_prompt=500,
                  append_median=200.0, context_cap=3500, tool_gap_mean_ms=15_000.0)
    shape = SHAPES["tiny"]
    trace = make_trace(cfg, seed=42)
    kw = dict(policy=policy, kappa_blocks=2, window_ms=60_000, len_window=32)
    kh = 700 // R
    oracle = TraceOracle(shape, 256, kh, payload=key_words_numpy, chunk_blocks=R, **kw)
    oracle.run(trace)
    server = AgentServer(shape, 256, kh, key_words_numpy, chunk_blocks=R, native_turn=False, link_strategy=link,
                         staging_bytes=6 * shape.block_bytes, **kw)
    server.run(trace)
    compare_records(server.records, oracle.records)
    assert server.totals == oracle.totals and oracle.totals["loaded_blocks"] > 0
    server.ctx.eakv_sync()
    tier = server.ctx.tier_host_view()
    for key, slot in oracle.host.order.items():
        for i in range(R):
            assert np.array_equal(tier[slot * R + i], oracle.tier[slot * R + i]), (slot, i)
    for q, t in enumerate(server.pool.pieces):
        got = t.cpu().numpy().view(np.uint8)
        for key, blk in oracle.gpu.order.items():
            assert np.array_equal(got[blk], oracle.pool[q][blk])
    server.close()


@pytest.mark.parametrize("cfg_name,R,policy,incremental", [
    ("c0", 1, 0, False), ("c0_big_tier", 1, 0, True), ("c0_big_tier", 4, 0, True),
    ("c0", 1, 2, True), ("c0", 2, 1, False)])
def test_native_turn_engine_bit_exact(cfg_name, R, policy, incremental):
    """eakv_turn_begin / eakv_turn_end (lookup, bookkeeping, restore and store inside the
    library) against the oracle: every record and every resident byte."""
    from paper_2609_33762_b200 import eakv
    from paper_2609_33762_b200.harness import AgentServer
    cfg = CONFIGS[cfg_name]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg)
    kh = cfg.host_blocks // R
    kw = dict(policy=policy, kappa_blocks=20, window_ms=40, len_window=16)
    oracle = TraceOracle(shape, cfg.gpu_blocks, kh, payload=key_words_numpy, chunk_blocks=R, **kw)
    oracle.run(trace)
    server = AgentServer(shape, cfg.gpu_blocks, kh, key_words_numpy, chunk_blocks=R, native_turn=True,
                         incremental_hash=incremental, **kw)
    server.run(trace)
    compare_records(server.records, oracle.records)
    assert server.totals == oracle.totals
    server.ctx.eakv_sync()
    tier = server.ctx.tier_host_view()
    for key, slot in oracle.host.order.items():
        for i in range(R):
            assert np.array_equal(tier[slot * R + i], oracle.tier[slot * R + i])
    for q, t in enumerate(server.pool.pieces):
        got = t.cpu().numpy().view(np.uint8)
        for key, blk in oracle.gpu.order.items():
            assert np.array_equal(got[blk], oracle.pool[q][blk])
    # protocol errors: end without begin, begin twice
    with pytest.raises(eakv.EakvError) as ei:
        server.ctx.eakv_turn_end()
    assert ei.value.code == eakv.E_INVAL
    toks = torch.zeros(64, dtype=torch.int32).pin_memory()
    server.ctx.eakv_turn_begin(toks.data_ptr(), 40, None, 99, 10**6)
    with pytest.raises(eakv.EakvError) as ei:
        server.ctx.eakv_turn_begin(toks.data_ptr(), 40, None, 99, 10**6)
    assert ei.value.code == eakv.E_INVAL
    server.ctx.eakv_turn_end()
    server.close()


@pytest.mark.parametrize("native", [False, True])
def test_reverse_free_order_bit_exact(native):
    """Tail-first GPU recency order (a request's last block is its least recent): records and
    resident bytes equal the oracle's, with the step-by-step harness and the turn engine."""
    from paper_2609_33762_b200 import eakv
    from paper_2609_33762_b200.harness import AgentServer
    cfg = CONFIGS["c0_big_tier"]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg, agents=3)
    oracle = TraceOracle(shape, cfg.gpu_blocks, cfg.host_blocks, payload=key_words_numpy, gpu_free_order=1)
    oracle.run(trace)
    assert oracle.totals["gpu_hit_blocks"] > 0 and oracle.totals["loaded_blocks"] > 0
    server = AgentServer(shape, cfg.gpu_blocks, cfg.host_blocks, key_words_numpy, native_turn=native,
                         incremental_hash=True, gpu_free_order=eakv.FREE_REVERSE)
    server.run(trace)
    compare_records(server.records, oracle.records)
    assert server.totals == oracle.totals
    compare_bytes(server, oracle)
    server.close()


@pytest.mark.parametrize("policy,kh,pool,native", [(0, 1024, 3, False), (2, 200, 4, True), (0, 160, 8, False)])
def test_closed_loop_replay_bit_exact(policy, kh, pool, native):
    """Closed-loop replay on the GPU path: the call order that the service times produce, the
    makespan, every record and every resident byte equal the oracle's closed-loop replay."""
    from oracle import closedloop as ocl
    from paper_2609_33762_b200 import closedloop
    from paper_2609_33762_b200.harness import AgentServer
    cfg = CONFIGS["c0_big_tier"]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg, agents=8, turns=8)
    kw = dict(policy=policy, kappa_blocks=10, window_ms=50, len_window=16)
    rates = dict(t_pf_ns=40_000, h2d_bytes_per_us=9_000, d2h_bytes_per_us=7_000, tau_load_us=120,
                 call_overhead_us=33)
    oracle = TraceOracle(shape, cfg.gpu_blocks, kh, payload=key_words_numpy, **kw)
    want = ocl.replay(trace, oracle, ocl.ServiceModel(**rates), pool, shape.bytes_per_token)
    server = AgentServer(shape, cfg.gpu_blocks, kh, key_words_numpy, incremental_hash=True,
                         native_turn=native, **kw)
    order, makespan, _ = closedloop.replay_trace(trace, server.turn, closedloop.ServiceModel(**rates), pool,
                                                 shape.bytes_per_token, shape.block_size)
    assert order == want["order"] and makespan == want["makespan_us"]
    compare_records(server.records, oracle.records)
    assert server.totals == oracle.totals
    compare_bytes(server, oracle)
    server.close()


@pytest.mark.parametrize("native", [True, False], ids=["request-calls", "single-calls"])
@pytest.mark.parametrize("policy,kh,gpu_blocks,S,decode_us,R,link", [
    (0, 1024, 130, 4, 20_000, 1, 1), (0, 160, 140, 3, 60_000, 1, 0), (2, 200, 200, 6, 40_000, 1, 1),
    (0, 64, 136, 4, 50_000, 4, 1)])
def test_engine_replay_with_preemption_bit_exact(policy, kh, gpu_blocks, S, decode_us, R, link, native):
    """The engine model (several running requests with pinned GPU blocks, suspension when GPU KV
    memory is short, resumption by restoring and recomputing) on the GPU path with bytes: every
    scheduler event, every record of every first and resumed lookup, J, and every resident byte of
    both tiers equal the oracle's."""
    from oracle import closedloop as ocl
    from oracle import engine as oen
    from paper_2609_33762_b200 import closedloop
    from paper_2609_33762_b200.harness import AgentServer
    cfg = CONFIGS["c0_big_tier"]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg, agents=8, turns=8)
    kw = dict(policy=policy, kappa_blocks=10 if R == 1 else 2, window_ms=50, len_window=16)
    rates = dict(t_pf_ns=40_000, h2d_bytes_per_us=9_000, d2h_bytes_per_us=7_000, tau_load_us=120)
    oracle = TraceOracle(shape, gpu_blocks, kh, payload=key_words_numpy, chunk_blocks=R, **kw)
    want = oen.replay(trace, oracle, ocl.ServiceModel(**rates), 8, S, decode_us, shape.bytes_per_token)
    server = AgentServer(shape, gpu_blocks, kh, key_words_numpy, incremental_hash=True, chunk_blocks=R,
                         link_strategy=link, native_turn=native, **kw)
    got = closedloop.replay_engine(trace, server.begin, server.finish, closedloop.ServiceModel(**rates), 8, S,
                                   decode_us, shape.bytes_per_token, shape.block_size)
    assert got["events"] == want["events"] and got["order"] == want["order"]
    assert got["makespan_us"] == want["makespan_us"] and got["preemptions"] == want["preemptions"] > 0
    assert got["recomputed_after_preemption"] == want["totals"]["preempt_recomputed_tokens"]
    compare_records(server.records, oracle.records)
    assert [r["resumed"] for r in server.records] == [r["resumed"] for r in oracle.records]
    want_totals = dict(oracle.totals)
    want_totals.setdefault("preempt_recomputed_tokens", 0)
    got_totals = dict(server.totals)
    got_totals.setdefault("preempt_recomputed_tokens", 0)
    assert got_totals == want_totals
    assert any(r["resumed"] and r["loaded"] > 0 for r in oracle.records) or policy == 2 or kh <= 160
    compare_bytes(server, oracle)
    server.close()


@pytest.mark.parametrize("R,link,seed,write_behind,layers", [(1, 1, 5, False, 0), (1, 0, 6, False, 0), (2, 1, 11, False, 0),
                                                              (1, 1, 8, True, 0), (1, 1, 6, False, 2)])
def test_deferred_stores_interleaved_with_other_lookups_with_bytes(R, link, seed, write_behind, layers):
    """Requests whose host write comes only after other requests have been looked up
    (eakv_request_begin ... eakv_request_store): a unit that a later lookup evicted before its
    bytes arrived must not be written, or the slot's new owner would read a stranger's KV.  Every
    record equals the oracle's, and after every store each listed unit whose write is not pending
    holds the oracle's bytes (which tests/test_oracle_deferred_store.py pins to the payload)."""
    from deferred_util import drive, operations
    from paper_2609_33762_b200.harness import AgentServer
    shape = SHAPES["tiny"]
    b = shape.block_size
    gpu_blocks, kh = 200, 64 // R               # a tier a few running requests overrun
    oracle = TraceOracle(shape, gpu_blocks, kh, payload=key_words_numpy, chunk_blocks=R)
    server = AgentServer(shape, gpu_blocks, kh, key_words_numpy, incremental_hash=False, chunk_blocks=R,
                         link_strategy=link, native_turn=True, write_behind=write_behind, store_layers=layers,
                         load_layers=layers)
    seen = dict(begins=0, skipped=0)

    def check_listed_bytes():
        server.ctx.eakv_sync()
        tier = server.ctx.tier_host_view()
        for ukey, slot in oracle.host.order.items():
            if ukey not in oracle.pending:
                for i in range(R):
                    assert np.array_equal(tier[slot * R + i], oracle.tier[slot * R + i]), (ukey, slot, i)

    def on_begin(rid, agent, tokens, now):
        w = oracle.begin(rid, tokens, agent, now, defer_store=True)
        g = server.begin(rid, tokens, agent, now, defer_store=True)
        assert (g is None) == (w is None)
        if g is None:
            return False
        seen["begins"] += 1
        compare_records([g], [w])
        return True

    def on_store(rid):
        admitted = sum(oracle.open[rid]["admit_b"])
        seen["skipped"] += admitted - oracle.store(rid)
        server.store(rid)
        check_listed_bytes()

    def on_finish(rid):
        oracle.finish(rid)
        server.finish(rid)

    drive(operations(seed, 260, b, 60 * b, max_open=4), on_begin, on_store, on_finish)
    assert seen["begins"] > 60 and seen["skipped"] > 0          # evicted-before-written did occur
    compare_bytes(server, oracle)
    server.close()


@pytest.mark.parametrize("cfg_name,R,policy,link,group,write_behind", [
    ("c0", 1, 0, 1, 1, False), ("c0", 1, 2, 0, 3, False), ("c0_big_tier", 4, 0, 1, 2, False), ("c0", 1, 0, 1, 4, True)])
def test_turn_engine_with_layered_host_writes_bit_exact(cfg_name, R, policy, link, group, write_behind):
    """The turn engine with the prefill on a stream of its own, a layer group at a time, the host
    write following it group by group (eakv_turn_end_layers), and the restore in layer groups with
    one event each (eakv_turn_begin_layers): records and every resident byte equal the oracle's."""
    from paper_2609_33762_b200.harness import AgentServer
    cfg = CONFIGS[cfg_name]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg)
    kh = cfg.host_blocks // R
    kw = dict(policy=policy, kappa_blocks=20, window_ms=40, len_window=16)
    oracle = TraceOracle(shape, cfg.gpu_blocks, kh, payload=key_words_numpy, chunk_blocks=R, **kw)
    oracle.run(trace)
    server = AgentServer(shape, cfg.gpu_blocks, kh, key_words_numpy, native_turn=True, incremental_hash=True,
                         chunk_blocks=R, link_strategy=link, store_layers=group, load_layers=group,
                         write_behind=write_behind, **kw)
    server.run(trace)
    assert len(server.last_restore_events) == -(-shape.num_layers // group)
    for ev in server.last_restore_events:
        ev.synchronize()
    compare_records(server.records, oracle.records)
    assert server.totals == oracle.totals and oracle.totals["stored_blocks"] > 0
    compare_bytes(server, oracle)
    server.close()


def test_warm_restart_with_adopted_tier_memory():
    """Half of the trace, then the process 'restarts': the host tier's index is exported, the
    context destroyed, a new one adopts the same pinned tier memory and imports the index.  The
    rest of the trace restores the old bytes: records and resident bytes equal the oracle run
    whose GPU tier was emptied at the same point."""
    from oracle.trace import GpuTier
    from paper_2609_33762_b200.harness import AgentServer
    cfg = CONFIGS["c0_big_tier"]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg, agents=5)
    kh = cfg.host_blocks                                  # large enough that prefixes survive
    half = len(trace.requests) // 2
    oracle = TraceOracle(shape, cfg.gpu_blocks, kh, payload=key_words_numpy)
    for i, req in enumerate(trace.requests):
        if i == half:
            oracle.gpu = GpuTier(cfg.gpu_blocks)
        oracle.turn(trace.prompt(req), req.agent, req.time_ms)
    tier_mem = torch.zeros(kh * shape.block_bytes, dtype=torch.uint8).pin_memory()
    server = AgentServer(shape, cfg.gpu_blocks, kh, key_words_numpy, tier_memory=tier_mem.data_ptr())
    for req in trace.requests[:half]:
        server.turn(trace.prompt(req), req.agent, req.time_ms)
    server.ctx.eakv_sync()
    recs = list(server.records)
    keys, slots = server.ctx.eakv_tier_export()
    assert len(keys) > 0
    server.close()
    del server
    server = AgentServer(shape, cfg.gpu_blocks, kh, key_words_numpy, tier_memory=tier_mem.data_ptr())
    server.ctx.eakv_tier_import(keys, slots)
    for req in trace.requests[half:]:
        server.turn(trace.prompt(req), req.agent, req.time_ms)
    recs += server.records
    compare_records(recs, oracle.records)
    assert sum(r["loaded"] for r in server.records) > 0          # restores came from the old bytes
    compare_bytes(server, oracle)
    server.close()


@pytest.mark.parametrize("cfg_name,R,policy", [("c0", 1, 0), ("c0_big_tier", 1, 0), ("c0_big_tier", 4, 2)])
def test_write_behind_turn_engine_bit_exact(cfg_name, R, policy):
    """Deferred host writes (eakv_turn_end returns with the caller's stream free): records and every
    resident byte still equal the oracle's.  Config 0's GPU tier turns over completely every turn, so
    blocks are handed to new keys while their write is still pending and the library has to make the
    caller's stream wait; the large-tier sibling also restores from slots written by deferred stores."""
    from paper_2609_33762_b200.harness import AgentServer
    cfg = CONFIGS[cfg_name]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg)
    kh = cfg.host_blocks // R
    kw = dict(policy=policy, kappa_blocks=20, window_ms=40, len_window=16)
    oracle = TraceOracle(shape, cfg.gpu_blocks, kh, payload=key_words_numpy, chunk_blocks=R, **kw)
    oracle.run(trace)
    server = AgentServer(shape, cfg.gpu_blocks, kh, key_words_numpy, chunk_blocks=R, native_turn=True,
                         incremental_hash=True, write_behind=True, **kw)
    server.run(trace)
    compare_records(server.records, oracle.records)
    assert server.totals == oracle.totals
    server.ctx.eakv_sync()
    tier = server.ctx.tier_host_view()
    for key, slot in oracle.host.order.items():
        for i in range(R):
            assert np.array_equal(tier[slot * R + i], oracle.tier[slot * R + i])
    for q, t in enumerate(server.pool.pieces):
        got = t.cpu().numpy().view(np.uint8)
        for key, blk in oracle.gpu.order.items():
            assert np.array_equal(got[blk], oracle.pool[q][blk])
    server.close()


def test_write_behind_orders_block_reuse_and_slot_reads():
    """A deferred write of ~0.9 GiB is still on the link when the next turn is handed the same GPU
    blocks and fills them at once, and when a third turn restores from the slots being written:
    the tier must receive the first turn's bytes and the restore must return them."""
    from paper_2609_33762_b200 import eakv
    from paper_2609_33762_b200.harness import PagedPool
    shape = SHAPES["qwen3_30b_a3b"]
    nb, kh, m = 700, 1400, 640                       # the second prompt has to take 580 of the first's blocks
    pool = PagedPool(shape, nb, "cuda:0")
    ctx = eakv.Context(num_layers=shape.num_layers, kv_heads=shape.kv_heads, head_dim=shape.head_dim,
                       block_size=shape.block_size, gpu_blocks=nb, host_blocks=kh, kv_base=pool.kv_base,
                       write_behind=True)
    stream = torch.cuda.current_stream()
    rng = np.random.default_rng(77)
    n = m * shape.block_size
    prompts = [torch.from_numpy(rng.integers(0, 151936, size=n, dtype=np.int32)).pin_memory() for _ in range(2)]

    def turn(p, value, fill=True):
        v = ctx.eakv_turn_begin(prompts[p].data_ptr(), n, None, p, 0, stream)
        ids = torch.as_tensor(v["gpu_block"][v["needs_fill"] != 0].astype(np.int64), device="cuda")
        if fill and len(ids):
            for piece in pool.pieces:
                piece[ids] = value                   # the engine's prefill, on the same stream, at once
        ctx.eakv_turn_end(stream)
        return v

    a = turn(0, 0x1111)
    assert a["n_stored_blocks"] == m and a["n_fill"] == m
    b = turn(1, 0x2222)                              # reuses most of a's GPU blocks while a's write is pending
    assert len(set(a["gpu_block"].tolist()) & set(b["gpu_block"][b["needs_fill"] != 0].tolist())) >= 500
    c = turn(0, 0x3333, fill=False)                  # a's prompt again: restored from the slots just written
    assert c["restore_hi"] - c["restore_lo"] == m and c["n_fill"] == 0
    ctx.eakv_sync()
    tier = ctx.tier_host_view().view(np.uint16)
    for slot in a["slot"].tolist():
        assert (tier[slot] == 0x1111).all(), slot
    for slot in b["slot"].tolist():
        assert (tier[slot] == 0x2222).all(), slot
    ids = torch.as_tensor(c["gpu_block"].astype(np.int64), device="cuda")
    for piece in pool.pieces[::17]:
        assert bool((piece[ids].view(torch.int16) == 0x1111).all())
    ctx.close()


@pytest.mark.parametrize("R,link,seed", [(1, 1, 21), (2, 0, 22), (1, 1, 23)])
def test_written_units_hold_their_payload_under_random_begin_store_release(R, link, seed):
    """Requests begin, store and are released in random order on the GPU path with bytes, some of
    them released before their store (their pending units are taken back).  A model follows the
    views (a slot is written by the store of the request that owns it; an eviction forgets it);
    after every store each written unit's slot must hold the payload of its blocks' keys, and
    every restored GPU block the payload of the key it was restored for."""
    import random
    from deferred_util import Prompts
    from paper_2609_33762_b200.harness import AgentServer
    shape = SHAPES["tiny"]
    b = shape.block_size
    W = shape.piece_bytes // 2
    rng = random.Random(seed)
    kh, nb, max_blocks = 120 // R, 60, 30       # the host tier outlives the GPU tier (restores) and still evicts
    server = AgentServer(shape, nb, kh, key_words_numpy, incremental_hash=False, chunk_blocks=R,
                         link_strategy=link, native_turn=True)
    prompts = Prompts(rng, b, agents=6)
    written, pending, begun, stored, busy, unit_blocks = {}, {}, {}, set(), set(), {}
    rid = now = withdrawn = restored = 0

    def payload_of(keys):
        return [key_words_numpy(np.asarray(keys, dtype=np.uint64), q, W) for q in range(shape.pieces_per_block)]

    def check_written():
        server.ctx.eakv_sync()
        tier = server.ctx.tier_host_view().view(np.uint16)
        for ukey, slot in written.items():
            want = payload_of(unit_blocks[ukey])
            for i in range(R):
                for q in range(shape.pieces_per_block):
                    assert np.array_equal(tier[slot * R + i, q], want[q][i]), (ukey, slot, i, q)

    for step in range(300):
        now += rng.randrange(0, 3000)
        choices = []
        if len(begun) < 4 and len(busy) < 6:
            choices += ["begin"] * 3
        if any(r not in stored for r in begun):
            choices += ["store"] * 2
        if begun:
            choices += ["release"] * 2
        op = rng.choice(choices)
        if op == "begin":
            agent = rng.choice([a for a in range(6) if a not in busy])
            rid += 1
            toks = prompts.next_prompt(agent, max_blocks * b)
            rec = server.begin(rid, toks, agent, now, defer_store=True)
            if rec is None:
                continue
            keys = [int(k) for k in rec["keys"]]
            ukeys = keys[R - 1::R]
            for c, uk in enumerate(ukeys):
                unit_blocks[uk] = keys[c * R:(c + 1) * R]
            for k, _ in rec["evicted"]:
                written.pop(int(k), None)
                pending.pop(int(k), None)
            if rec["loaded"]:
                lo = rec["G"]
                ids = torch.as_tensor(np.asarray(rec["gpu_block"][lo:lo + rec["loaded"]], dtype=np.int64), device="cuda")
                want = payload_of(keys[lo:lo + rec["loaded"]])
                torch.cuda.synchronize()
                for q in (0, shape.pieces_per_block - 1):
                    got = server.pool.pieces[q][ids].cpu().numpy().view(np.uint16)
                    assert np.array_equal(got, want[q])
                restored += rec["loaded"]
            for c, a in enumerate(rec["admit"]):
                if a:
                    pending[ukeys[c]] = (rid, int(rec["slot"][c]))
            begun[rid] = agent
            busy.add(agent)
        elif op == "store":
            r = rng.choice([r for r in begun if r not in stored])
            server.store(r)
            stored.add(r)
            for k, (owner, sl) in list(pending.items()):
                if owner == r:
                    written[k] = sl
                    del pending[k]
            check_written()
        else:
            r = rng.choice(list(begun))
            server.finish(r)
            if r not in stored:
                for k, (owner, sl) in list(pending.items()):
                    if owner == r:
                        del pending[k]
                        withdrawn += 1
            stored.discard(r)
            busy.discard(begun.pop(r))
    check_written()
    ek, es = server.ctx.eakv_tier_export()
    assert dict(zip(ek.tolist(), es.tolist())) == {**written, **{k: sl for k, (_, sl) in pending.items()}}
    assert withdrawn > 0 and restored > 0
    server.close()


def test_a_failed_store_or_restore_leaves_no_stale_slot_readable():
    """With bytes: a store that fails in eakv_turn_end (made to fail on the host) withdraws the
    turn's units, so that the same prompt afterwards is computed and stored again rather than
    restored from slots that were never written; a restore that fails in eakv_turn_begin
    withdraws that turn, and the retry restores the right bytes."""
    from paper_2609_33762_b200 import eakv
    from paper_2609_33762_b200.harness import PagedPool
    shape = SHAPES["tiny"]
    nb, kh, m = 24, 64, 12
    pool = PagedPool(shape, nb, "cuda:0")
    ctx = eakv.Context(num_layers=shape.num_layers, kv_heads=shape.kv_heads, head_dim=shape.head_dim,
                       block_size=shape.block_size, gpu_blocks=nb, host_blocks=kh, kv_base=pool.kv_base)
    stream = torch.cuda.current_stream()
    rng = np.random.default_rng(78)
    n = m * shape.block_size
    prompts = [torch.from_numpy(rng.integers(0, 50000, size=n, dtype=np.int32)).pin_memory() for _ in range(3)]

    def begin(p, value):
        v = ctx.eakv_turn_begin(prompts[p].data_ptr(), n, None, p, 0, stream)
        ids = torch.as_tensor(v["gpu_block"][v["needs_fill"] != 0].astype(np.int64), device="cuda")
        for piece in pool.pieces:
            piece[ids] = value
        return v

    tier = ctx.tier_host_view().view(np.uint16)
    tier[:] = 0x7777                                    # what a never-written slot would return
    a = begin(0, 0x1111)
    ctx.eakv_selfcheck_fail_next_transfer(eakv.E_CUDA)
    with pytest.raises(eakv.EakvError):
        ctx.eakv_turn_end(stream)
    ctx.eakv_sync()
    assert (tier[a["slot"]] == 0x7777).all()            # nothing was written ...
    assert ctx.eakv_match(a["keys"])[1] == 0            # ... and nothing is listed
    for p, value in ((1, 0x2222), (2, 0x3333)):         # two other prompts take prompt 0 off the GPU
        begin(p, value)
        ctx.eakv_turn_end(stream)
    a2 = begin(0, 0x4444)                               # computed again (not restored), stored now
    assert a2["restore_hi"] == a2["restore_lo"] and a2["n_fill"] == m and a2["n_stored_blocks"] == m
    ctx.eakv_turn_end(stream)
    begin(1, 0x5555)                                    # (prompt 1 is restored: nothing to fill)
    ctx.eakv_turn_end(stream)
    begin(2, 0x6666)
    ctx.eakv_turn_end(stream)
    # prompt 0 is off the GPU again: its restore is made to fail once, then retried
    ctx.eakv_selfcheck_fail_next_transfer(eakv.E_CUDA)
    with pytest.raises(eakv.EakvError):
        ctx.eakv_turn_begin(prompts[0].data_ptr(), n, None, 0, 0, stream)
    assert ctx.eakv_match(a["keys"])[:2] == (0, m)      # still only on the host
    a3 = begin(0, 0x0BAD)
    assert a3["restore_hi"] - a3["restore_lo"] == m and a3["n_fill"] == 0
    ctx.eakv_turn_end(stream)
    ctx.eakv_sync()
    ids = torch.as_tensor(a3["gpu_block"].astype(np.int64), device="cuda")
    for piece in pool.pieces:
        assert bool((piece[ids].view(torch.int16) == 0x4444).all())
    ctx.close()


def test_write_behind_orders_a_direct_load_of_pending_slots():
    """eakv_load of slots that a deferred write is still filling, into GPU blocks the write does
    not touch: only the slot marks can make it wait, and it must return the written bytes."""
    from paper_2609_33762_b200 import eakv
    from paper_2609_33762_b200.harness import PagedPool
    shape = SHAPES["qwen3_30b_a3b"]
    nb, kh, m = 1400, 700, 640
    pool = PagedPool(shape, nb, "cuda:0")
    ctx = eakv.Context(num_layers=shape.num_layers, kv_heads=shape.kv_heads, head_dim=shape.head_dim,
                       block_size=shape.block_size, gpu_blocks=nb, host_blocks=kh, kv_base=pool.kv_base,
                       write_behind=True)
    stream = torch.cuda.current_stream()
    n = m * shape.block_size
    toks = torch.from_numpy(np.random.default_rng(78).integers(0, 151936, size=n, dtype=np.int32)).pin_memory()
    v = ctx.eakv_turn_begin(toks.data_ptr(), n, None, 0, 0, stream)
    ids = torch.as_tensor(v["gpu_block"].astype(np.int64), device="cuda")
    for piece in pool.pieces:
        piece[ids] = 0x4444
    ctx.eakv_turn_end(stream)                        # ~0.9 GiB now on its way to the tier
    used = set(v["gpu_block"].tolist())
    spare = np.array([b for b in range(nb) if b not in used][:m], dtype=np.int32)
    # at once, into blocks the write never touches, last-written slots first
    ctx.eakv_load(np.ascontiguousarray(v["slot"][::-1]), spare, stream)
    ctx.eakv_sync()
    dst = torch.as_tensor(spare.astype(np.int64), device="cuda")
    for piece in pool.pieces[::13]:
        assert bool((piece[dst].view(torch.int16) == 0x4444).all())
    ctx.close()


@pytest.mark.parametrize("link", [1, 0], ids=["staged", "zero-copy"])
def test_a_store_waits_for_a_restore_on_another_stream_that_reads_its_slots(link):
    """The bookkeeping may hand a slot on while a restore enqueued on another stream still reads it
    (several lookups can pass while 0.9 GiB cross the link).  The library orders the write behind
    that read: the restore must deliver the old bytes, the tier must end up with the new ones.
    Likewise a restore enqueued on another stream while a store still fills its slots waits for it."""
    from paper_2609_33762_b200 import eakv
    from paper_2609_33762_b200.harness import PagedPool
    shape = SHAPES["qwen3_30b_a3b"]
    nb, kh, m = 2000, 1300, 640
    pool = PagedPool(shape, nb, "cuda:0")
    ctx = eakv.Context(num_layers=shape.num_layers, kv_heads=shape.kv_heads, head_dim=shape.head_dim,
                       block_size=shape.block_size, gpu_blocks=nb, host_blocks=kh, kv_base=pool.kv_base,
                       link_strategy=link)
    a, b_, c = (np.arange(m, dtype=np.int32) + k * m for k in range(3))       # three disjoint block sets
    slots = np.arange(m, dtype=np.int32)
    for blocks, value in ((a, 0x1111), (b_, 0x2222), (c, 0x3333)):
        ids = torch.as_tensor(blocks.astype(np.int64), device="cuda")
        for piece in pool.pieces:
            piece[ids] = value
    torch.cuda.synchronize()
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    ctx.eakv_store(a, None, slots, sa)                   # the slots hold 0x1111
    ctx.eakv_sync()
    ctx.eakv_load(slots, c, sa)                          # restore them into set c on one stream ...
    ctx.eakv_store(b_, None, slots[::-1].copy(), sb)     # ... and at once overwrite them from another
    ctx.eakv_sync()
    torch.cuda.synchronize()
    ids = torch.as_tensor(c.astype(np.int64), device="cuda")
    for piece in pool.pieces[::7]:
        assert bool((piece[ids].view(torch.int16) == 0x1111).all())
    tier = ctx.tier_host_view().view(np.uint16)
    assert (tier[slots] == 0x2222).all()
    # the same stream needs no wait and a later restore sees the new bytes
    ctx.eakv_load(slots, a, sb)
    ctx.eakv_sync()
    ids = torch.as_tensor(a.astype(np.int64), device="cuda")
    for piece in pool.pieces[::7]:
        assert bool((piece[ids].view(torch.int16) == 0x2222).all())
    # and the other way round: a restore, on another stream, of slots that a store is still filling
    ctx.eakv_store(c, None, slots, sa)                   # (set c holds 0x1111 since the first restore)
    ctx.eakv_load(slots[::-1].copy(), b_, sb)
    ctx.eakv_sync()
    torch.cuda.synchronize()
    ids = torch.as_tensor(b_.astype(np.int64), device="cuda")
    for piece in pool.pieces[::7]:
        assert bool((piece[ids].view(torch.int16) == 0x1111).all())
    # pool blocks: a restore into blocks that a store on another stream still reads waits for it
    slots2 = slots + m
    ids_c = torch.as_tensor(c.astype(np.int64), device="cuda")
    for piece in pool.pieces:
        piece[ids_c] = 0x5555
    torch.cuda.synchronize()
    ctx.eakv_store(c, None, slots2, sa)                  # a second set of slots holds 0x5555
    ctx.eakv_sync()
    ctx.eakv_store(a, None, slots, sa)                   # set a (0x2222) on its way to the first slots ...
    ctx.eakv_load(slots2, a[::-1].copy(), sb)            # ... while another stream restores into set a
    ctx.eakv_sync()
    torch.cuda.synchronize()
    tier = ctx.tier_host_view().view(np.uint16)
    assert (tier[slots] == 0x2222).all()                 # the store read set a before it changed
    ids = torch.as_tensor(a.astype(np.int64), device="cuda")
    for piece in pool.pieces[::7]:
        assert bool((piece[ids].view(torch.int16) == 0x5555).all())
    ctx.close()


def test_random_traces_with_bytes_across_options():
    """Small random traces with KV bytes through combinations of policy, chunking, link strategy,
    copy path, GPU free order, the turn engine and deferred writes: records and resident bytes
    equal the oracle's in every case."""
    import random
    from dataclasses import replace
    from paper_2609_33762_b200.harness import AgentServer
    rng = random.Random(77)
    cfg0 = CONFIGS["c0_big_tier"]
    shape = SHAPES[cfg0.shape]
    for case in range(12):
        policy = case % 3
        R = (1, 2, 4)[(case // 3) % 3]
        native = case % 2 == 1
        wb = native and case % 4 == 3
        link = rng.randrange(2)
        order = rng.randrange(2)
        cfg = replace(cfg0, seed=300 + case, append_median=float(rng.choice([60, 200, 500])),
                      first_prompt=rng.choice([96, 256, 512]))
        trace = make_trace(cfg, agents=rng.randrange(2, 6), turns=rng.randrange(3, 7))
        kh = max(cfg.context_cap // (shape.block_size * R) + 1, rng.randrange(60, 500) // R)
        kw = dict(policy=policy, kappa_blocks=rng.choice([0, 2, 8, 30]), window_ms=rng.choice([5, 40, 60000]),
                  len_window=rng.choice([4, 256]))
        oracle = TraceOracle(shape, cfg.gpu_blocks, kh, payload=key_words_numpy, chunk_blocks=R,
                             gpu_free_order=order, **kw)
        oracle.run(trace)
        server = AgentServer(shape, cfg.gpu_blocks, kh, key_words_numpy, chunk_blocks=R, native_turn=native,
                             incremental_hash=bool(case & 1), link_strategy=link, copy_path=rng.randrange(2),
                             gpu_free_order=order, write_behind=wb,
                             staging_bytes=rng.choice([3, 9]) * shape.block_bytes, **kw)
        server.run(trace)
        compare_records(server.records, oracle.records)
        assert server.totals == oracle.totals, case
        server.ctx.eakv_sync()
        tier = server.ctx.tier_host_view()
        for key, slot in oracle.host.order.items():
            for i in range(R):
                assert np.array_equal(tier[slot * R + i], oracle.tier[slot * R + i]), (case, slot)
        for q, t in enumerate(server.pool.pieces):
            got = t.cpu().numpy().view(np.uint8)
            for key, blk in oracle.gpu.order.items():
                assert np.array_equal(got[blk], oracle.pool[q][blk]), (case, q, blk)
        server.close()
