"""Pins for the closed-loop replay oracle: closed forms (single task, work conservation,
no queueing, sequential pool), a tick-by-tick brute force of the scheduler, and the service
time of Eq. 2 on hand values."""
import random

from eakv_workloads import CONFIGS, SHAPES, make_trace
from oracle import closedloop as cl
from oracle.trace import TraceOracle


def test_service_time_hand_values():
    m = cl.ServiceModel(t_pf_ns=10_000, h2d_bytes_per_us=50_000, d2h_bytes_per_us=25_000,
                        tau_load_us=300, call_overhead_us=7, store_blocking=True)
    # 100 tokens recomputed at 10 us each = 1000 us
    assert cl.service_us(m, 100, 0, 0) == 7 + 1000
    # restoring 1,000,001 bytes at 50,000 B/us = 20.00002 us -> 21, plus tau_load
    assert cl.service_us(m, 0, 1_000_001, 0) == 7 + 300 + 21
    # nothing restored: no fixed restoration overhead either
    assert cl.service_us(m, 0, 0, 50_000) == 7 + 2
    off = cl.ServiceModel(store_blocking=False, call_overhead_us=0)
    assert cl.service_us(off, 0, 0, 10**9) == 0
    # Eq. 2 at the paper's H20 figures: 0.86 us per restored token against 5.6 us per recomputed
    # token gives OBR = 1 - 0.86 / 5.6 for long prefixes
    m2 = cl.ServiceModel(t_pf_ns=5600, h2d_bytes_per_us=1000, tau_load_us=0)
    n, beta = 10**6, 860
    t_load = cl.service_us(m2, 0, n * beta, 0)
    t_rec = cl.service_us(m2, n, 0, 0)
    assert abs((1 - t_load / t_rec) - (1 - 0.86 / 5.6)) < 1e-9


def run(n_tasks, turns, gaps, A, svc):
    return cl.simulate(n_tasks, lambda i: turns[i], lambda i, t: gaps[i][t], A,
                       lambda i, t, s: svc[i][t])


def test_single_task_is_the_sum_of_services_and_gaps():
    svc = [[5, 7, 11, 2]]
    gaps = [[0, 100, 3, 40]]
    order, mk = run(1, [4], gaps, 1, svc)
    assert mk == sum(svc[0]) + sum(gaps[0])
    assert [o[:2] for o in order] == [(0, t) for t in range(4)]


def test_zero_gaps_keep_the_engine_busy():
    rng = random.Random(0)
    turns = [rng.randrange(1, 6) for _ in range(7)]
    svc = [[rng.randrange(1, 50) for _ in range(t)] for t in turns]
    gaps = [[0] * t for t in turns]
    for A in (1, 3, 7):
        order, mk = run(7, turns, gaps, A, svc)
        assert mk == sum(map(sum, svc))
        assert len(order) == sum(turns)
        # never two calls at once, never idle
        for x, y in zip(order, order[1:]):
            assert y[3] == x[4]


def test_long_gaps_mean_no_queueing():
    # services of 1 us, gaps of distinct large sizes: every call starts when it is eligible
    turns = [3, 3, 3]
    svc = [[1] * 3 for _ in range(3)]
    gaps = [[0, 1000 + 10 * i, 5000 + 7 * i] for i in range(3)]
    order, mk = run(3, turns, gaps, 3, svc)
    per_task = [sum(svc[i]) + sum(gaps[i]) + (i if False else 0) for i in range(3)]
    # the three first calls queue behind each other at time 0 (task i waits i us)
    assert mk == max(per_task[i] + i for i in range(3))
    for task, turn, when, start, finish in order:
        if turn > 0:
            assert start == when


def test_pool_of_one_runs_tasks_back_to_back():
    turns = [2, 3, 1]
    svc = [[4, 5], [1, 1, 1], [9]]
    gaps = [[0, 10], [0, 20, 30], [0]]
    order, mk = run(3, turns, gaps, 1, svc)
    assert mk == sum(map(sum, svc)) + sum(map(sum, gaps))
    assert [o[0] for o in order] == [0, 0, 1, 1, 1, 2]


def brute_force(n_tasks, turns, gaps, A, svc):
    """One microsecond per tick: an idle engine takes the eligible call that has waited longest."""
    waiting = list(range(n_tasks))
    nxt = {}
    while waiting and len(nxt) < A:
        nxt[waiting.pop(0)] = (0, 0)
    busy_until, running = 0, None
    order, t = [], 0
    while nxt or running:
        if running and t == busy_until:
            task, turn = running
            running = None
            if turn + 1 < turns[task]:
                nxt[task] = (turn + 1, t + gaps[task][turn + 1])
            elif waiting:
                nxt[waiting.pop(0)] = (0, t)
        if running is None:
            ready = [(w, k) for k, (_, w) in nxt.items() if w <= t]
            if ready:
                w, task = min(ready)
                turn, _ = nxt.pop(task)
                running = (task, turn)
                busy_until = t + svc[task][turn]
                order.append((task, turn, w, t, busy_until))
                continue          # a zero-length call may finish in this same tick
        t += 1
    return order, max(o[4] for o in order)


def test_scheduler_against_tick_brute_force():
    rng = random.Random(5)
    for case in range(60):
        n = rng.randrange(1, 6)
        A = rng.randrange(1, n + 1)
        turns = [rng.randrange(1, 5) for _ in range(n)]
        svc = [[rng.randrange(1, 9) for _ in range(t)] for t in turns]
        gaps = [[0] + [rng.randrange(0, 12) for _ in range(t - 1)] for t in turns]
        assert run(n, turns, gaps, A, svc) == brute_force(n, turns, gaps, A, svc)


def test_replay_counts_every_call_once_and_order_depends_on_the_tier():
    cfg = CONFIGS["c0_big_tier"]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg, agents=5, turns=6)
    model = cl.ServiceModel(t_pf_ns=50_000, tau_load_us=50)
    out = {}
    for kh in (1024, 160):
        orc = TraceOracle(shape, cfg.gpu_blocks, kh)
        out[kh] = cl.replay(trace, orc, model, active_pool=3, bytes_per_token=shape.bytes_per_token)
        seen = sorted((o[0], o[1]) for o in out[kh]["order"])
        assert seen == [(a, t) for a in range(5) for t in range(6)]
        assert out[kh]["totals"]["prompt_tokens"] == int(sum(trace.agent_lengths[a].sum() for a in range(5)))
    # a tier that loses prefixes recomputes more and takes longer
    assert out[160]["totals"]["fresh_tokens"] > out[1024]["totals"]["fresh_tokens"]
    assert out[160]["makespan_us"] > out[1024]["makespan_us"]
