"""Closed-loop replay: the order of the calls follows from how long each one takes.

Section 2 ("A closed-loop workload"), Section 5.1 and Appendix B of the paper: A tasks are
active at a time, admitted in list order; a task may issue its next call only after the previous
response is complete and the recorded gap has gone by; a finished task frees its place for the
next one in the list; the makespan is when the last response of all completes.  The engine is one call at a time, first come first served by eligibility (lower
task id first among equals).  A call's response time follows Eq. 2 in integer microseconds:

    overhead + ceil(computed_tokens * t_pf) + [restored > 0] (tau_load + ceil(restored_bytes / B_H2D))
             + [blocking write] ceil(stored_bytes / B_D2H)

so a cache policy changes the interleaving, which changes what the tiers see next.

    python -m paper_2609_33762_b200.closedloop --config c3 --active-pool 16 --host-gib 32
    python -m paper_2609_33762_b200.closedloop --config c3 --active-pool 8,16 --policy conditioned
    python -m paper_2609_33762_b200.closedloop --config c3 --theta 50,80,95,100 --policy conditioned

    python -m paper_2609_33762_b200.closedloop --config c3 --active-pool 16 --running-cap 16 --gpu-gib 96

With ``--running-cap`` the engine runs that many requests at once (class EngineLoop below): a running
request's GPU blocks are pinned, and a request that finds no room suspends a running one, which later
resumes by restoring and recomputing its KV; the output then carries the preemption count and the
recomputed tokens.

With ``--measured-transfers`` the restore and write terms are the device times of the real
``eakv_load`` / ``eakv_store`` calls on this GPU instead of bytes / bandwidth (the prefill
term stays modelled: there is no model to run).
"""
from __future__ import annotations

import argparse
import heapq
import json
import time
from dataclasses import dataclass

import numpy as np

from . import eakv

GIB = 1 << 30


@dataclass(frozen=True)
class ServiceModel:
    """Rates of Eq. 2.  Defaults: one B200 serving the Qwen3-30B-A3B shape (3.3 B activated
    parameters, 6.6 GFLOP per token, 40 % of the measured dense bf16 rate: about 10 us per
    computed token) over the measured pinned host link (about 55 GB/s each way)."""
    t_pf_ns: int = 10_000
    h2d_bytes_per_us: int = 55_000
    d2h_bytes_per_us: int = 55_000
    tau_load_us: int = 200
    call_overhead_us: int = 0
    store_blocking: bool = True

    def service_us(self, computed_tokens: int, restored_bytes: int, stored_bytes: int) -> int:
        t = self.call_overhead_us + -(-computed_tokens * self.t_pf_ns // 1000)
        if restored_bytes > 0:
            t += self.tau_load_us + -(-restored_bytes // self.h2d_bytes_per_us)
        if self.store_blocking and stored_bytes > 0:
            t += -(-stored_bytes // self.d2h_bytes_per_us)
        return int(t)


class ClosedLoop:
    """Event-queue scheduler.  ``serve(task, turn, start_us) -> service time in us`` performs the
    call; tasks are 0 .. n_tasks-1 in pool-entry order."""

    def __init__(self, turns, gaps_us, active_pool):
        self.turns = [int(t) for t in turns]
        self.gaps_us = gaps_us
        self.active_pool = int(active_pool)
        if self.active_pool < 1:
            raise ValueError("the active pool holds at least one task")

    def run(self, serve):
        n_tasks = len(self.turns)
        heap = []                                  # (eligible time, task, turn)
        next_task = 0
        while next_task < n_tasks and next_task < self.active_pool:
            heapq.heappush(heap, (0, next_task, 0))
            next_task += 1
        free_at = 0
        order = []
        while heap:
            when, task, turn = heapq.heappop(heap)
            start = when if when > free_at else free_at
            finish = start + int(serve(task, turn, start))
            free_at = finish
            order.append((task, turn, when, start, finish))
            if turn + 1 < self.turns[task]:
                heapq.heappush(heap, (finish + int(self.gaps_us[task][turn + 1]), task, turn + 1))
            elif next_task < n_tasks:
                heapq.heappush(heap, (finish, next_task, 0))
                next_task += 1
        return order, (max(o[4] for o in order) if order else 0)


class EngineLoop:
    """Closed loop against an engine that runs up to ``running_cap`` requests at once (Section 2 and
    Appendix A of the paper: the engine's own cap on running requests, 16 there, beside the active
    pool) and suspends a running request if the GPU cannot hold every running request's KV, to resume
    it later by recomputing its KV (Section 2; the recomputed tokens are the J terms of Appendix C).

    The engine model: a response is a prefill phase, served one request at a time, followed by
    ``decode_us`` of decoding during which the request stays running (its GPU blocks stay pinned)
    but no longer holds up the next prefill.  A request starts when the prefill engine and a
    running place are free and ``try_start`` finds room for its blocks.  Suspended requests go
    first, the most recently suspended at the front, then waiting requests by eligibility (lower
    task id among equals).  A new request that finds no room suspends the most recently started
    running request until it fits; a suspended request never suspends another one, it waits (and
    everything behind it waits) until its blocks fit.

    ``try_start(task, turn, now_us, resumed) -> prefill microseconds or None`` (None: no room, nothing
    changed); ``release(task, turn)`` lets a finished or suspended request's blocks go."""

    def __init__(self, turns, gaps_us, active_pool, running_cap, decode_us):
        self.turns = [int(t) for t in turns]
        self.gaps_us = gaps_us
        self.active_pool, self.running_cap, self.decode_us = int(active_pool), int(running_cap), int(decode_us)
        if self.active_pool < 1 or self.running_cap < 1:
            raise ValueError("the active pool and the running cap hold at least one request")

    def run(self, try_start, release):
        n_tasks = len(self.turns)
        waiting = []                               # heap of (eligible, task, turn)
        next_task = 0
        while next_task < n_tasks and next_task < self.active_pool:
            heapq.heappush(waiting, (0, next_task, 0))
            next_task += 1
        suspended = []                             # stack: last suspended on top
        running = {}                               # (task, turn) -> [start seq, decode end or None while prefilling]
        info = {}                                  # (task, turn) -> [eligible, first start, decode time left]
        in_prefill, prefill_end = None, 0
        now = seq = preemptions = 0
        order, events = [], []
        while waiting or suspended or running:
            if in_prefill is not None and prefill_end <= now:
                running[in_prefill][1] = now + info[in_prefill][2]
                in_prefill = None
            done = sorted((st[1], st[0], k) for k, st in running.items() if k != in_prefill and st[1] <= now)
            for _, _, k in done:
                del running[k]
                release(*k)
                events.append(("finish", now, k[0], k[1]))
                order.append((k[0], k[1], info[k][0], info[k][1], now))
                if k[1] + 1 < self.turns[k[0]]:
                    heapq.heappush(waiting, (now + int(self.gaps_us[k[0]][k[1] + 1]), k[0], k[1] + 1))
                elif next_task < n_tasks:
                    heapq.heappush(waiting, (now, next_task, 0))
                    next_task += 1
            zero_length = False
            while in_prefill is None and len(running) < self.running_cap and not zero_length:
                if suspended:
                    k = suspended[-1]
                    t = try_start(k[0], k[1], now, True)
                    if t is None:
                        break
                    suspended.pop()
                    events.append(("resume", now, k[0], k[1]))
                else:
                    if not waiting or waiting[0][0] > now:
                        break
                    eligible, task, turn = waiting[0]
                    k = (task, turn)
                    t = try_start(task, turn, now, False)
                    while t is None:
                        if not running:
                            raise RuntimeError("a request does not fit the GPU tier on its own")
                        victim = max(running, key=lambda q: running[q][0])
                        info[victim][2] = running[victim][1] - now
                        del running[victim]
                        release(*victim)
                        suspended.append(victim)
                        preemptions += 1
                        events.append(("suspend", now, victim[0], victim[1]))
                        t = try_start(task, turn, now, False)
                    heapq.heappop(waiting)
                    info[k] = [eligible, now, self.decode_us]
                    events.append(("start", now, task, turn))
                running[k] = [seq, None]
                seq += 1
                in_prefill, prefill_end = k, now + int(t)
                if t == 0:
                    running[k][1] = now + info[k][2]
                    in_prefill = None
                    zero_length = info[k][2] == 0
            if any(k != in_prefill and st[1] <= now for k, st in running.items()):
                continue
            times = [st[1] for k, st in running.items() if k != in_prefill]
            if in_prefill is not None:
                times.append(prefill_end)
            elif len(running) < self.running_cap and not suspended and waiting:
                times.append(waiting[0][0])
            if not times:
                if waiting or suspended:
                    raise RuntimeError("the engine cannot make progress")
                break
            now = min(times)
        order.sort(key=lambda o: (o[3], o[0]))
        return dict(order=order, makespan_us=max((o[4] for o in order), default=0), preemptions=preemptions,
                    events=events)


def replay_engine(trace, begin_fn, finish_fn, model: ServiceModel, active_pool, running_cap, decode_us,
                  bytes_per_token, block_size):
    """Closed-loop replay of ``trace`` on the engine model above.  ``begin_fn(request_id, tokens, agent,
    now_ms, decided) -> record or None`` (None: the request's GPU blocks do not fit; ``decided`` is None
    for a first lookup, else the store/skip choice of the request's first lookup);
    ``finish_fn(request_id)``.  Returns EngineLoop.run's dict plus ``recomputed_after_preemption``
    (J of Appendix C), ``busy`` (engine microseconds by kind) and ``resumed_lookups``."""
    tasks = sorted(trace.agent_tokens)
    block_bytes = block_size * bytes_per_token
    decided = {}
    acc = {"J": 0, "resumed": 0, "compute_us": 0, "restore_us": 0, "write_us": 0}

    def rid(i, turn):
        return i * 1_000_000 + turn

    def try_start(i, turn, now_us, resumed):
        a = tasks[i]
        n = int(trace.agent_lengths[a][turn])
        rec = begin_fn(rid(i, turn), trace.agent_tokens[a][:n], a, now_us // 1000,
                       decided[(i, turn)] if resumed else None)
        if rec is None:
            return None
        if resumed:
            acc["J"] += rec["fresh_tokens"]
            acc["resumed"] += 1
        else:
            decided[(i, turn)] = bool(rec["save"])
        c = -(-rec["fresh_tokens"] * model.t_pf_ns // 1000)
        r = model.tau_load_us + -(-rec["loaded"] * block_bytes // model.h2d_bytes_per_us) if rec["loaded"] > 0 else 0
        w = -(-rec["stored"] * block_bytes // model.d2h_bytes_per_us) if (model.store_blocking and rec["stored"] > 0) else 0
        acc["compute_us"] += c
        acc["restore_us"] += r
        acc["write_us"] += w
        return c + r + w

    loop = EngineLoop([len(trace.agent_lengths[a]) for a in tasks],
                      [trace.agent_gaps_ms[a].astype(np.int64) * 1000 for a in tasks],
                      active_pool, running_cap, decode_us)
    out = loop.run(try_start, lambda i, turn: finish_fn(rid(i, turn)))
    out["recomputed_after_preemption"] = acc["J"]
    out["resumed_lookups"] = acc["resumed"]
    out["busy"] = {k: acc[k] for k in ("compute_us", "restore_us", "write_us")}
    return out


def replay_trace(trace, turn_fn, model: ServiceModel, active_pool, bytes_per_token, block_size,
                 measured=None):
    """Closed-loop replay of ``trace``.  ``turn_fn(tokens, agent, now_ms) -> record`` with
    ``fresh_tokens``, ``loaded`` and ``stored`` (blocks).  ``measured()``, if given, returns the
    device microseconds the call's transfers took and replaces the bandwidth terms."""
    tasks = sorted(trace.agent_tokens)
    block_bytes = block_size * bytes_per_token
    busy = {"compute_us": 0, "restore_us": 0, "write_us": 0}

    def serve(i, turn, start_us):
        a = tasks[i]
        n = int(trace.agent_lengths[a][turn])
        rec = turn_fn(trace.agent_tokens[a][:n], a, start_us // 1000)
        if measured is None:
            t = model.service_us(rec["fresh_tokens"], rec["loaded"] * block_bytes, rec["stored"] * block_bytes)
            busy["compute_us"] += model.service_us(rec["fresh_tokens"], 0, 0) - model.call_overhead_us
            busy["restore_us"] += model.service_us(0, rec["loaded"] * block_bytes, 0) - model.call_overhead_us
            busy["write_us"] += model.service_us(0, 0, rec["stored"] * block_bytes) - model.call_overhead_us
            return t
        load_us, store_us = measured()
        compute = model.service_us(rec["fresh_tokens"], 0, 0)
        busy["compute_us"] += compute - model.call_overhead_us
        busy["restore_us"] += load_us
        busy["write_us"] += store_us if model.store_blocking else 0
        return compute + load_us + (store_us if model.store_blocking else 0)

    loop = ClosedLoop([len(trace.agent_lengths[a]) for a in tasks],
                      [trace.agent_gaps_ms[a].astype(np.int64) * 1000 for a in tasks], active_pool)
    order, makespan = loop.run(serve)
    return order, makespan, busy


def run(config, *, policy="write_all", host_gib=None, active_pool=None, model=ServiceModel(),
        data_plane=False, device="cuda:0", chunk_blocks=1, kappa=None, theta=95, agents=None,
        turns=None, measured_transfers=False, gpu_free_order=eakv.FREE_ASCENDING,
        running_cap=None, decode_us=0, gpu_gib=None):
    import torch
    from eakv_workloads import CONFIGS, SHAPES, key_words_torch, make_trace
    from .harness import AgentServer
    from .replay import POLICIES, plan

    cfg = CONFIGS[config]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg, agents=agents, turns=turns)
    A = active_pool or len(trace.agent_tokens)
    kh, why = plan(cfg, trace, shape, host_gib, data_plane)
    kh = max(1, kh // chunk_blocks)
    if measured_transfers and not data_plane:
        raise ValueError("measured transfers need the data plane")
    if running_cap and measured_transfers:
        raise ValueError("the engine model takes its transfer times from the service model")
    gpu_blocks = cfg.gpu_blocks if gpu_gib is None else int(gpu_gib * GIB) // shape.block_bytes
    payload = (lambda keys, q, n: key_words_torch(keys.astype(np.int64), q, n, device)) if data_plane else None
    server = AgentServer(shape, gpu_blocks, kh, payload, device=device, data_plane=data_plane,
                         incremental_hash=True, policy=POLICIES[policy],
                         kappa_blocks=max(1, cfg.kappa_blocks // chunk_blocks) if kappa is None else kappa,
                         theta_percent=theta, chunk_blocks=chunk_blocks, gpu_free_order=gpu_free_order)
    seen = {"load": 0, "store": 0}

    def measured():
        torch.cuda.synchronize()
        out = []
        for kind in ("load", "store"):
            items = server._timed[kind][seen[kind]:]
            seen[kind] = len(server._timed[kind])
            out.append(int(round(sum(e0.elapsed_time(e1) for _, e0, e1 in items) * 1000)))
        return out

    t0 = time.perf_counter()
    engine = None
    if running_cap:
        engine = replay_engine(trace, server.begin, server.finish, model, A, running_cap, decode_us,
                               shape.bytes_per_token, shape.block_size)
        order, makespan, busy = engine["order"], engine["makespan_us"], engine["busy"]
    else:
        order, makespan, busy = replay_trace(trace, server.turn, model, A, shape.bytes_per_token,
                                             shape.block_size, measured if measured_transfers else None)
    server.ctx.eakv_sync()
    wall = time.perf_counter() - t0
    st = server.ctx.eakv_get_stats()
    tot = server.totals
    queue_us = sum(o[3] - o[2] for o in order)
    benefit = eakv.eakv_offload_benefit(prefix_tokens=max(1, trace.total_prompt_tokens // max(1, len(trace.requests))),
                                        beta_rank_bytes=shape.bytes_per_token, t_prefill_ps=model.t_pf_ns * 1000,
                                        h2d_bytes_per_s=model.h2d_bytes_per_us * 1_000_000,
                                        tau_load_ps=model.tau_load_us * 1_000_000)
    out = {
        "config": config, "policy": policy, "active_pool": A, "tasks": len(trace.agent_tokens),
        "requests": len(order), "host_gib": kh * chunk_blocks * shape.block_bytes / GIB,
        "host_sizing": why, "chunk_blocks": chunk_blocks, "theta_percent": theta,
        "data_plane": data_plane, "measured_transfers": measured_transfers,
        "service_model": model.__dict__,
        # Eq. 2: the long-prefix limit of OBR and the prefix length from which a restore pays (eakv_offload_benefit)
        "offload_benefit": {k: benefit[k] for k in ("obr_long_prefix", "break_even_tokens")},
        "makespan_s": makespan / 1e6, "mean_queue_delay_ms": queue_us / max(1, len(order)) / 1e3,
        "engine_busy_s": {k[:-3]: v / 1e6 for k, v in busy.items()},
        "prompt_tokens": tot["prompt_tokens"], "computed_prefill_tokens": tot["fresh_tokens"],
        "restored_tokens": tot["loaded_blocks"] * shape.block_size,
        "stored_tokens": tot["stored_blocks"] * shape.block_size,
        "gpu_hit_tokens": tot["gpu_hit_blocks"] * shape.block_size,
        "tier": {k: st[k] for k in ("hits", "admitted", "declined", "evicted", "declined_requests",
                                    "pressure_requests", "resident")},
        "wall_s": wall,
    }
    if engine is not None:
        # Appendix C: total computed prefill = first-pass prefill + the tokens recomputed after preemptions
        out["engine"] = {"running_cap": running_cap, "decode_us": decode_us,
                         "gpu_gib": gpu_blocks * shape.block_bytes / GIB,
                         "preemptions": engine["preemptions"],
                         "recomputed_after_preemption_tokens": engine["recomputed_after_preemption"],
                         "computed_prefill_incl_preemption_tokens":
                             tot["fresh_tokens"] + engine["recomputed_after_preemption"]}
    server.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="c3", choices=["c0", "c0_big_tier", "c2", "c3", "c4"])
    ap.add_argument("--policy", default="write_all", choices=["write_all", "fixed", "conditioned"])
    ap.add_argument("--host-gib", type=float, default=None)
    ap.add_argument("--active-pool", default=None, help="comma-separated pool sizes (default: every task)")
    ap.add_argument("--theta", default="95", help="comma-separated occupancy thresholds in percent")
    ap.add_argument("--kappa", type=int, default=None)
    ap.add_argument("--chunk-blocks", type=int, default=1)
    ap.add_argument("--t-pf-ns", type=int, default=ServiceModel.t_pf_ns)
    ap.add_argument("--h2d-gbps", type=float, default=55.0)
    ap.add_argument("--d2h-gbps", type=float, default=55.0)
    ap.add_argument("--tau-load-us", type=int, default=ServiceModel.tau_load_us)
    ap.add_argument("--call-overhead-us", type=int, default=0)
    ap.add_argument("--async-writes", action="store_true", help="responses do not wait for host writes")
    ap.add_argument("--data-plane", action="store_true", help="move the KV bytes as well")
    ap.add_argument("--measured-transfers", action="store_true")
    ap.add_argument("--reverse-free", action="store_true")
    ap.add_argument("--agents", type=int, default=None)
    ap.add_argument("--turns", type=int, default=None)
    ap.add_argument("--running-cap", type=int, default=None,
                    help="engine model: this many requests run at once, GPU blocks pinned while they run, "
                         "preemption if the GPU pool cannot hold all running requests (default: one call at a time)")
    ap.add_argument("--decode-ms", type=float, default=2000.0, help="engine model: decoding time per call")
    ap.add_argument("--gpu-gib", type=float, default=None, help="GPU KV tier size (default: the configuration's)")
    args = ap.parse_args()
    model = ServiceModel(t_pf_ns=args.t_pf_ns, h2d_bytes_per_us=int(args.h2d_gbps * 1000),
                         d2h_bytes_per_us=int(args.d2h_gbps * 1000), tau_load_us=args.tau_load_us,
                         call_overhead_us=args.call_overhead_us, store_blocking=not args.async_writes)
    pools = [int(x) for x in args.active_pool.split(",")] if args.active_pool else [None]
    for A in pools:
        for theta in [int(x) for x in args.theta.split(",")]:
            print(json.dumps(run(args.config, policy=args.policy, host_gib=args.host_gib, active_pool=A,
                                 model=model, data_plane=args.data_plane or args.measured_transfers,
                                 chunk_blocks=args.chunk_blocks, kappa=args.kappa, theta=theta,
                                 agents=args.agents, turns=args.turns,
                                 measured_transfers=args.measured_transfers,
                                 gpu_free_order=eakv.FREE_REVERSE if args.reverse_free else eakv.FREE_ASCENDING,
                                 running_cap=args.running_cap, decode_us=int(args.decode_ms * 1000),
                                 gpu_gib=args.gpu_gib)))


if __name__ == "__main__":
    main()
