"""Pins for the engine model of the closed-loop replay oracle (several running requests, pinned
GPU blocks, preemption with recomputation: Section 2, Appendix A, Appendix C of the paper).

  * the pinned GPU tier: acquire + release is the single-request step; pinned blocks are never
    taken; the fit test is exact (brute force over the block sets);
  * a running cap of one reproduces the one-call-at-a-time closed loop exactly;
  * a GPU tier that holds every running context never preempts, J = 0;
  * a hand-computed case of two requests that cannot co-reside: one preemption, J = the
    victim's uncovered tokens (0 when the host tier covers them);
  * a tick-by-tick brute force of the scheduler on small random cases;
  * conservation: every call finishes once, every suspension is resumed, J is the sum over the
    resumed lookups.
"""
import random

import numpy as np
import pytest

from eakv_workloads import CONFIGS, SHAPES, make_trace
from oracle import closedloop as cl
from oracle import engine as en
from oracle.tier import FILTER_FIXED
from oracle.trace import GpuTier, TraceOracle


# ---------------------------------------------------------------------------------------------
# pinned GPU tier
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("free_order", [0, 1])
def test_acquire_then_release_is_the_single_request_step(free_order):
    rng = random.Random(7 + free_order)
    for case in range(40):
        nb = rng.randrange(4, 20)
        a, c = GpuTier(nb, free_order), GpuTier(nb, free_order)
        for rid in range(60):
            start = rng.randrange(0, 30)
            n = rng.randrange(0, nb)
            keys = [f"k{start}-{j}" if rng.random() < 0.2 else f"s{j}" for j in range(n)]
            keys = list(dict.fromkeys(keys))
            tail = rng.random() < 0.5 and len(keys) + 1 <= nb
            want = a.step(keys, tail)
            a.release(want[2])
            got = c.acquire(rid, keys, tail)
            assert got == want
            c.release_request(rid)
            assert list(a.order.items()) == list(c.order.items()) and a.free == c.free
            assert not c.pinned and not c.held


def check_tier_invariants(g, holders):
    blocks = list(g.free) + list(g.order.values()) + [v[0] for v in g.pinned.values()] + \
             [t for _, t in g.held.values() if t >= 0]
    assert sorted(blocks) == list(range(g.NB))                 # every block in exactly one place
    for rid, (keys, ids) in holders.items():
        for k, blk in zip(keys, ids):
            assert g.pinned[k][0] == blk                       # a held block stays where it is
    for k, (blk, cnt) in g.pinned.items():
        assert cnt == sum(1 for keys, _ in holders.values() if k in keys) and cnt > 0


def test_pinned_blocks_are_never_taken_and_the_fit_test_is_exact():
    rng = random.Random(11)
    for case in range(60):
        nb = rng.randrange(6, 24)
        g = GpuTier(nb, rng.randrange(2))
        holders = {}
        for rid in range(80):
            if holders and rng.random() < 0.4:
                victim = rng.choice(list(holders))
                g.release_request(victim)
                del holders[victim]
            n = rng.randrange(1, nb)
            shared = rng.randrange(0, 3)                        # prompts may share a prefix
            keys = [f"sys{j}" for j in range(shared)] + [f"r{rng.randrange(12)}-{j}" for j in range(n - shared)]
            keys = list(dict.fromkeys(keys))
            tail = rng.random() < 0.5
            # brute force: blocks held by others are untouchable; everything else is available
            held_blocks = {v[0] for v in g.pinned.values()} | {t for _, t in g.held.values() if t >= 0}
            own_free_of_charge = sum(1 for k in keys if k in g.pinned)
            fits = (len(keys) - own_free_of_charge + int(tail)) <= nb - len(held_blocks)
            assert g.fits(keys, tail) == fits
            before = (list(g.order.items()), list(g.free), {k: list(v) for k, v in g.pinned.items()})
            got = g.acquire(rid, keys, tail)
            if not fits:
                assert got is None
                assert before == (list(g.order.items()), list(g.free), {k: list(v) for k, v in g.pinned.items()})
            else:
                res, ids, t = got
                assert len(set(ids)) == len(ids) and not (set(ids) & (held_blocks - {g.pinned[k][0] for k in keys}))
                holders[rid] = (keys, ids)
            check_tier_invariants(g, holders)


# ---------------------------------------------------------------------------------------------
# scheduler
# ---------------------------------------------------------------------------------------------
class BlockCountBackend:
    """Abstract GPU: request (task, turn) needs w blocks of K; it fits iff the running ones leave
    room.  Prefill takes svc us the first time and re_svc us after a suspension."""

    def __init__(self, K, need, svc, re_svc):
        self.K, self.need, self.svc, self.re_svc = K, need, svc, re_svc
        self.held = {}
        self.log = []

    def try_start(self, task, turn, now, resumed):
        w = self.need[task][turn]
        if sum(self.held.values()) + w > self.K:
            return None
        self.held[(task, turn)] = w
        self.log.append((now, task, turn, resumed))
        return self.re_svc[task][turn] if resumed else self.svc[task][turn]

    def release(self, task, turn):
        del self.held[(task, turn)]


def run_engine(n, turns, gaps, A, S, decode, backend):
    return en.simulate(n, lambda i: turns[i], lambda i, t: gaps[i][t], A, S, decode,
                       backend.try_start, backend.release)


def test_running_cap_of_one_is_the_one_call_at_a_time_closed_loop():
    rng = random.Random(3)
    for case in range(80):
        n = rng.randrange(1, 6)
        A = rng.randrange(1, n + 1)
        turns = [rng.randrange(1, 5) for _ in range(n)]
        svc = [[rng.randrange(0, 9) for _ in range(t)] for t in turns]
        gaps = [[0] + [rng.randrange(0, 12) for _ in range(t - 1)] for t in turns]
        decode = rng.randrange(0, 6)
        want = cl.simulate(n, lambda i: turns[i], lambda i, t: gaps[i][t], A,
                           lambda i, t, s: svc[i][t] + decode)
        be = BlockCountBackend(1, [[1] * t for t in turns], svc, svc)
        got = run_engine(n, turns, gaps, A, 1, decode, be)
        assert got["order"] == sorted(want[0], key=lambda o: (o[3], o[0])) and got["makespan_us"] == want[1]
        assert got["preemptions"] == 0


def tick_brute_force(n, turns, gaps, A, S, decode, K, need, svc, re_svc):
    """The same rules, one microsecond per tick, no event queue: at every tick first end what
    ends, then start what may start."""
    not_entered = list(range(n))
    fresh = {}
    while not_entered and len(fresh) < A:
        fresh[not_entered.pop(0)] = (0, 0)
    running = {}          # (task, turn) -> dict(seq, phase, until, rem, first, eligible)
    suspended = []
    order, preemptions, seq, t = [], 0, 0, 0
    held = lambda: sum(need[k[0]][k[1]] for k in running)
    while fresh or running or suspended:
        progressed = True
        while progressed:
            progressed = False
            for k, r in sorted(running.items(), key=lambda kv: kv[1]["seq"]):
                if r["phase"] == "prefill" and r["until"] <= t:
                    r["phase"], r["until"] = "decode", t + r["rem"]
                    progressed = True
            for k, r in sorted(running.items(), key=lambda kv: (kv[1]["until"], kv[1]["seq"])):
                if r["phase"] == "decode" and r["until"] <= t:
                    del running[k]
                    order.append((k[0], k[1], r["eligible"], r["first"], t))
                    if k[1] + 1 < turns[k[0]]:
                        fresh[k[0]] = (k[1] + 1, t + gaps[k[0]][k[1] + 1])
                    elif not_entered:
                        fresh[not_entered.pop(0)] = (0, t)
                    progressed = True
            while not any(r["phase"] == "prefill" for r in running.values()) and len(running) < S:
                if suspended:
                    k, r = suspended[0]
                    if held() + need[k[0]][k[1]] > K:
                        break
                    suspended.pop(0)
                    r.update(seq=seq, phase="prefill", until=t + re_svc[k[0]][k[1]])
                else:
                    ready = [(w, task) for task, (_, w) in fresh.items() if w <= t]
                    if not ready:
                        break
                    w, task = min(ready)
                    turn, _ = fresh.pop(task)
                    k = (task, turn)
                    while held() + need[task][turn] > K:
                        vk = max(running, key=lambda q: running[q]["seq"])
                        v = running.pop(vk)
                        v["rem"] = v["until"] - t
                        suspended.insert(0, (vk, v))
                        preemptions += 1
                    r = dict(seq=seq, phase="prefill", until=t + svc[task][turn], rem=decode, first=t, eligible=w)
                seq += 1
                running[k] = r
                progressed = True
        t += 1
    order.sort(key=lambda o: (o[3], o[0]))
    return order, max(o[4] for o in order), preemptions


def test_scheduler_against_tick_brute_force():
    rng = random.Random(9)
    seen_preemption = 0
    for case in range(150):
        n = rng.randrange(1, 6)
        A = rng.randrange(1, n + 1)
        S = rng.randrange(1, 4)
        turns = [rng.randrange(1, 4) for _ in range(n)]
        svc = [[rng.randrange(0, 7) for _ in range(t)] for t in turns]
        re_svc = [[rng.randrange(0, 7) for _ in range(t)] for t in turns]
        need = [[rng.randrange(1, 6) for _ in range(t)] for t in turns]
        gaps = [[0] + [rng.randrange(0, 10) for _ in range(t - 1)] for t in turns]
        decode = rng.randrange(0, 12)
        K = rng.randrange(5, 12)
        got = run_engine(n, turns, gaps, A, S, decode, BlockCountBackend(K, need, svc, re_svc))
        want = tick_brute_force(n, turns, gaps, A, S, decode, K, need, svc, re_svc)
        assert (got["order"], got["makespan_us"], got["preemptions"]) == want, case
        seen_preemption += got["preemptions"] > 0
        # conservation
        assert sorted(o[:2] for o in got["order"]) == [(i, t) for i in range(n) for t in range(turns[i])]
        kinds = [e[0] for e in got["events"]]
        assert kinds.count("suspend") == kinds.count("resume") == got["preemptions"]
        assert kinds.count("start") == kinds.count("finish") == sum(turns)
    assert seen_preemption > 10


def test_room_for_every_running_request_means_no_preemption():
    rng = random.Random(4)
    for case in range(30):
        n, S = 5, 3
        turns = [3] * n
        svc = [[rng.randrange(1, 7) for _ in range(3)] for _ in range(n)]
        need = [[rng.randrange(1, 5) for _ in range(3)] for _ in range(n)]
        gaps = [[0, 2, 3] for _ in range(n)]
        be = BlockCountBackend(S * 4, need, svc, svc)
        got = run_engine(n, turns, gaps, n, S, 20, be)
        assert got["preemptions"] == 0
        # and the cap is what limits concurrency: three requests do run at once
        level, peak = 0, 0
        for e in sorted(got["events"], key=lambda e: (e[1], e[0] != "finish")):
            level += {"start": 1, "finish": -1}[e[0]]
            peak = max(peak, level)
        assert peak == S


# ---------------------------------------------------------------------------------------------
# replay against the trace oracle
# ---------------------------------------------------------------------------------------------
class TwoTaskTrace:
    """Two tasks with one call of 24 tokens each (six 4-token blocks), different tokens."""

    def __init__(self):
        rng = np.random.default_rng(1)
        self.agent_tokens = {a: rng.integers(0, 1000, size=24, dtype=np.int32) for a in (0, 1)}
        self.agent_lengths = {a: np.array([24]) for a in (0, 1)}
        self.agent_gaps_ms = {a: np.array([0]) for a in (0, 1)}


def tiny_shape():
    from eakv_workloads import KVShape
    return KVShape(1, 1, 8, 4)


def test_hand_case_two_requests_that_cannot_co_reside():
    """K_G = 10 blocks, two requests of 6 blocks, 1 us per computed token, decode 100 us, cap 2.
    t = 0: request 0 starts, prefill 24 us, decodes until 124.  t = 24: request 1 does not fit
    (4 free blocks) and suspends request 0 with 100 us of decoding left; it takes the 4 free blocks
    and the 2 least recent of request 0's; prefill until 48, decode until 148.  Request 0 cannot
    resume at 48 (needs 6, only its own 4 surviving blocks are not pinned).  t = 148: request 1
    finishes, request 0 resumes."""
    model = cl.ServiceModel(t_pf_ns=1000, h2d_bytes_per_us=4, d2h_bytes_per_us=4, tau_load_us=0,
                            store_blocking=False)
    trace = TwoTaskTrace()
    # (a) nothing reaches the host tier (fixed admission, kappa 0): the victim recomputes all 24
    # tokens: J = 24, finish = 148 + 24 + 100
    o = TraceOracle(tiny_shape(), 10, 64, policy=FILTER_FIXED, kappa_blocks=0)
    out = en.replay(trace, o, model, active_pool=2, running_cap=2, decode_us=100, bytes_per_token=1)
    assert out["order"] == [(0, 0, 0, 0, 272), (1, 0, 0, 24, 148)]
    assert out["preemptions"] == 1 and out["makespan_us"] == 272
    assert out["events"] == [("start", 0, 0, 0), ("suspend", 24, 0, 0), ("start", 24, 1, 0),
                             ("finish", 148, 1, 0), ("resume", 148, 0, 0), ("finish", 272, 0, 0)]
    assert out["totals"]["preempt_recomputed_tokens"] == 24 and out["totals"]["fresh_tokens"] == 48
    assert out["totals"]["prompt_tokens"] == 48 and out["totals"]["loaded_blocks"] == 0
    resumed = [r for r in o.records if r["resumed"]]
    assert len(resumed) == 1 and resumed[0]["G"] == 0 and resumed[0]["save"] is False
    assert o.host.stats["requests"] == 2                       # the resumed lookup is not a new request
    # (b) write-all: the host tier holds the victim's 6 blocks, so the resume restores them
    # (24 bytes at 4 bytes per us = 6 us) and recomputes nothing: J = 0, finish = 148 + 6 + 100
    o = TraceOracle(tiny_shape(), 10, 64)
    out = en.replay(trace, o, model, active_pool=2, running_cap=2, decode_us=100, bytes_per_token=1)
    assert out["order"] == [(0, 0, 0, 0, 254), (1, 0, 0, 24, 148)]
    assert out["totals"]["preempt_recomputed_tokens"] == 0 and out["totals"]["loaded_blocks"] == 6
    assert out["totals"]["stored_blocks"] == 12                # nothing is stored twice (deduplication)
    # (c) a cap of one never preempts: the requests run back to back
    o = TraceOracle(tiny_shape(), 10, 64)
    out = en.replay(trace, o, model, active_pool=2, running_cap=1, decode_us=100, bytes_per_token=1)
    assert out["order"] == [(0, 0, 0, 0, 124), (1, 0, 0, 124, 248)] and out["preemptions"] == 0
    # (d) room for both: they overlap, no preemption
    o = TraceOracle(tiny_shape(), 12, 64)
    out = en.replay(trace, o, model, active_pool=2, running_cap=2, decode_us=100, bytes_per_token=1)
    assert out["order"] == [(0, 0, 0, 0, 124), (1, 0, 0, 24, 148)] and out["preemptions"] == 0


@pytest.mark.parametrize("policy,kh", [(0, 1024), (0, 160), (2, 160)])
def test_replay_with_a_cap_of_one_equals_the_closed_loop_replay(policy, kh):
    cfg = CONFIGS["c0_big_tier"]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg, agents=5, turns=6)
    model = cl.ServiceModel(t_pf_ns=50_000, tau_load_us=50, call_overhead_us=700)
    kw = dict(policy=policy, kappa_blocks=4, window_ms=10, len_window=8)
    a = TraceOracle(shape, cfg.gpu_blocks, kh, **kw)
    want = cl.replay(trace, a, model, active_pool=3, bytes_per_token=shape.bytes_per_token)
    c = TraceOracle(shape, cfg.gpu_blocks, kh, **kw)
    got = en.replay(trace, c, model, active_pool=3, running_cap=1, decode_us=700,
                    bytes_per_token=shape.bytes_per_token)
    assert got["order"] == want["order"] and got["makespan_us"] == want["makespan_us"]
    assert got["preemptions"] == 0 and got["totals"]["preempt_recomputed_tokens"] == 0
    for k, v in want["totals"].items():
        assert got["totals"][k] == v, k
    for ra, rc in zip(a.records, c.records):
        for f in ("keys", "G", "H", "hit", "admit", "slot", "evicted", "gpu_resident", "gpu_block",
                  "loaded", "stored", "fresh_tokens", "filled", "save", "pressure", "new_chunks"):
            assert ra[f] == rc[f], f
    assert a.host.stats == c.host.stats


def test_replay_under_gpu_pressure_preempts_and_accounts_for_it():
    cfg = CONFIGS["c0_big_tier"]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg, agents=6, turns=6)
    model = cl.ServiceModel(t_pf_ns=2_000, tau_load_us=20)
    results = {}
    for gpu_blocks in (10_000, 160):
        o = TraceOracle(shape, gpu_blocks, 4096)
        out = en.replay(trace, o, model, active_pool=6, running_cap=4, decode_us=30_000,
                        bytes_per_token=shape.bytes_per_token)
        results[gpu_blocks] = out
        assert sorted(x[:2] for x in out["order"]) == [(a, t) for a in range(6) for t in range(6)]
        resumed = [r for r in o.records if r["resumed"]]
        assert len(resumed) == out["preemptions"]
        assert out["totals"]["preempt_recomputed_tokens"] == sum(r["fresh_tokens"] for r in resumed)
        assert out["totals"]["prompt_tokens"] == int(sum(trace.agent_lengths[a].sum() for a in range(6)))
        assert not o.gpu.pinned and not o.gpu.held                 # everything was let go
    assert results[10_000]["preemptions"] == 0
    assert results[160]["preemptions"] > 0
    assert results[160]["makespan_us"] > results[10_000]["makespan_us"]
