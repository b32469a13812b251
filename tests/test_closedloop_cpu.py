"""Closed-loop replay: the library's scheduler and control plane against the oracle's, on the
CPU (a control-plane-only context makes no CUDA call; keys come from the oracle's hash).
Every call's (task, turn, eligible, start, finish), the makespan and the counters must agree."""
import random

import numpy as np
import pytest

from eakv_workloads import CONFIGS, SHAPES, make_trace
from oracle import closedloop as ocl
from oracle import hash as ohash
from oracle.trace import TraceOracle


@pytest.fixture(scope="module")
def mods():
    from paper_2609_33762_b200 import build, closedloop, eakv
    build.build()
    return eakv, closedloop


def control_plane_turn(eakv, ctx, b):
    """One turn through the C++ bookkeeping; returns what the service-time model needs."""
    def turn(tokens, agent, now_ms):
        n = len(tokens)
        keys = np.asarray(ohash.hash_blocks(tokens.tolist(), b), dtype=np.uint64)
        G, H, _, _ = ctx.eakv_match(keys)
        step = ctx.eakv_tier_step(keys, agent, n, now_ms)
        _, _, tail = ctx.eakv_gpu_tier_step(keys, n % b != 0)
        if tail >= 0:
            ctx.eakv_gpu_tier_release(tail)
        return dict(fresh_tokens=n - max(G, H) * b, loaded=max(H - G, 0), stored=int(step["admit"].sum()))
    return turn


@pytest.mark.parametrize("policy,kh,pool", [(0, 1024, 3), (0, 160, 5), (2, 200, 4), (1, 300, 2), (2, 160, 8)])
def test_closed_loop_matches_oracle(mods, policy, kh, pool):
    eakv, closedloop = mods
    cfg = CONFIGS["c0_big_tier"]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg, agents=8, turns=8)
    kw = dict(policy=policy, kappa_blocks=10, window_ms=50, len_window=16)
    om = ocl.ServiceModel(t_pf_ns=40_000, h2d_bytes_per_us=9_000, d2h_bytes_per_us=7_000,
                          tau_load_us=120, call_overhead_us=33)
    want = ocl.replay(trace, TraceOracle(shape, cfg.gpu_blocks, kh, **kw), om, pool, shape.bytes_per_token)
    pm = closedloop.ServiceModel(t_pf_ns=40_000, h2d_bytes_per_us=9_000, d2h_bytes_per_us=7_000,
                                 tau_load_us=120, call_overhead_us=33)
    ctx = eakv.Context(num_layers=1, kv_heads=1, head_dim=8, block_size=shape.block_size,
                       gpu_blocks=cfg.gpu_blocks, host_blocks=kh, kv_base=None, control_plane_only=True, **kw)
    order, makespan, busy = closedloop.replay_trace(
        trace, control_plane_turn(eakv, ctx, shape.block_size), pm, pool, shape.bytes_per_token,
        shape.block_size)
    st = ctx.eakv_get_stats()
    ctx.close()
    assert order == want["order"]
    assert makespan == want["makespan_us"]
    # the engine is busy exactly for the sum of the three service terms plus the fixed overheads
    assert sum(busy.values()) + pm.call_overhead_us * len(order) == sum(o[4] - o[3] for o in order)
    assert st["requests"] == len(order) == 64


def test_service_model_equals_oracle_on_random_arguments(mods):
    _, closedloop = mods
    rng = random.Random(1)
    for _ in range(500):
        kw = dict(t_pf_ns=rng.randrange(0, 50_000), h2d_bytes_per_us=rng.randrange(1, 10**5),
                  d2h_bytes_per_us=rng.randrange(1, 10**5), tau_load_us=rng.randrange(0, 1000),
                  call_overhead_us=rng.randrange(0, 100), store_blocking=rng.random() < 0.5)
        args = (rng.randrange(0, 10**6), rng.choice([0, rng.randrange(1, 10**11)]),
                rng.choice([0, rng.randrange(1, 10**11)]))
        assert closedloop.ServiceModel(**kw).service_us(*args) == ocl.service_us(ocl.ServiceModel(**kw), *args)


def test_smaller_pool_shrinks_the_working_set(mods):
    """Section 5.3: halving the active pool lowers computed prefill at a fixed tier (fewer
    histories compete), here with recomputation only (a one-chunk host tier cannot help)."""
    eakv, closedloop = mods
    cfg = CONFIGS["c0_big_tier"]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg, agents=8, turns=8)
    fresh = {}
    for pool in (8, 2):
        ctx = eakv.Context(num_layers=1, kv_heads=1, head_dim=8, block_size=shape.block_size,
                           gpu_blocks=2 * cfg.gpu_blocks, host_blocks=128, kv_base=None,
                           control_plane_only=True, policy=1, kappa_blocks=0)
        tot = {"fresh": 0}

        def turn(tokens, agent, now_ms, _t=control_plane_turn(eakv, ctx, shape.block_size)):
            r = _t(tokens, agent, now_ms)
            tot["fresh"] += r["fresh_tokens"]
            return r
        closedloop.replay_trace(trace, turn, closedloop.ServiceModel(), pool, shape.bytes_per_token,
                                shape.block_size)
        ctx.close()
        fresh[pool] = tot["fresh"]
    assert fresh[2] < fresh[8]


def test_config3_full_closed_loop_parity():
    """All 1,280 calls of config 3 under conditioned admission, active pool 16, 32 GiB tier: the
    library's scheduler and control plane give the oracle's call order and makespan (a few seconds;
    keys come from the oracle's hash, once per agent)."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, os.path.join(root, "tests", "check_full_traces.py"), "--config", "c3",
                          "--policy", "2", "--host-gib", "32", "--closed-loop", "16"],
                         capture_output=True, text=True, timeout=600, cwd=root)
    assert out.returncode == 0, out.stderr[-2000:]
    assert "1280 calls in identical order" in out.stdout
    assert "makespan 595.6 s" in out.stdout and "computed prefill 44250953" in out.stdout
