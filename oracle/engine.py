"""Closed-loop replay against an engine that runs several requests at once and preempts
(test infrastructure, CPU only).

What the paper fixes (Section 2, "A closed-loop workload"; Appendix A; Appendix C): tasks in an
active pool of size A issue their next call after the previous response and the recorded
interval; the engine has a limit of its own on concurrently running requests (16 in the
paper's setup); if the GPU cannot hold the KV of all of them it suspends one, which later resumes by
recomputing its KV, and the tokens recomputed that way (J) add to computed prefill.  The store
or skip choice of a request's first lookup is kept for its later lookups, including those after
a preemption (Appendix D).

What it leaves to the engine, and this build's reading of it:
  * A response has two phases.  Prefill (Eq. 2: computed tokens * t_pf, restore, blocking host
    write) runs on the engine one request at a time; decoding then takes a fixed ``decode_us``
    during which the request stays running -- its GPU blocks stay pinned -- without holding up
    the prefill of the next request.  At most ``running_cap`` requests are running.
  * A request starts when the prefill engine is free, a running place is free and its GPU
    blocks can be had.  Waiting requests are taken first come first served by eligibility
    (lower task id first among equals); suspended requests come before all of them, the most
    recently suspended first.
  * A new request whose blocks do not fit beside the running ones suspends the most recently
    started running request (again and again until it fits): the victim's blocks become
    evictable, in the same recency position as if it had finished, and the victim keeps what is
    left of its decoding time.  A suspended request never suspends another: it resumes when its
    blocks fit, and until then nothing behind it starts.  (Without that rule two requests that
    cannot co-reside would suspend each other for ever.)
  * A resumed request looks its prompt up again (GPU tier, host tier with the kept store/skip
    choice), restores what the host covers, recomputes the rest -- those tokens are J -- stores
    what the choice admits and the tier does not hold, then decodes for its remaining time.
All times are integer microseconds.
"""
from dataclasses import replace

from .closedloop import service_us


class EngineError(Exception):
    pass


class _Req:
    __slots__ = ("task", "turn", "eligible", "first_start", "seq", "rem_decode", "end", "resumes")

    def __init__(self, task, turn, eligible):
        self.task, self.turn, self.eligible = task, turn, eligible
        self.first_start = None
        self.seq = -1
        self.rem_decode = None
        self.end = None
        self.resumes = 0


def simulate(n_tasks, turns_of, gap_us_of, active_pool, running_cap, decode_us, try_start, release):
    """Run the closed loop.

    try_start(task, turn, now_us, resumed) -> prefill time in us, or None (nothing changed) when
    the request's GPU blocks do not fit; release(task, turn) lets a finished or suspended
    request's blocks go.  Returns dict(order, makespan_us, preemptions, events): order holds
    (task, turn, eligible_us, first_start_us, finish_us) by first start; events holds
    ("start" | "resume" | "suspend" | "finish", time_us, task, turn) as they happen."""
    if running_cap < 1 or active_pool < 1:
        raise ValueError("the active pool and the running cap hold at least one request")
    not_entered = list(range(n_tasks))
    fresh = []                                  # eligible or future first starts: _Req
    while not_entered and len(fresh) < active_pool:
        fresh.append(_Req(not_entered.pop(0), 0, 0))
    suspended = []                              # most recently suspended first
    running = []                                # in start order
    prefill = None                              # the request in its prefill phase
    prefill_end = 0
    now = 0
    seq = 0
    order, events = [], []
    preemptions = 0
    makespan = 0

    def retire(r):
        nonlocal makespan
        running.remove(r)
        release(r.task, r.turn)
        events.append(("finish", now, r.task, r.turn))
        order.append((r.task, r.turn, r.eligible, r.first_start, now))
        makespan = max(makespan, now)
        if r.turn + 1 < turns_of(r.task):
            fresh.append(_Req(r.task, r.turn + 1, now + gap_us_of(r.task, r.turn + 1)))
        elif not_entered:
            fresh.append(_Req(not_entered.pop(0), 0, now))

    while fresh or suspended or running:
        # 1. the prefill that ends now hands over to decoding; decodes that end now retire
        if prefill is not None and prefill_end <= now:
            prefill.end = now + prefill.rem_decode
            prefill = None
        for r in sorted([r for r in running if r is not prefill and r.end <= now], key=lambda r: (r.end, r.seq)):
            retire(r)
        # 2. start what can start
        while prefill is None and len(running) < running_cap:
            if suspended:
                cand, resumed = suspended[0], True
            else:
                ready = [r for r in fresh if r.eligible <= now]
                if not ready:
                    break
                cand, resumed = min(ready, key=lambda r: (r.eligible, r.task)), False
            t = try_start(cand.task, cand.turn, now, resumed)
            if t is None and resumed:
                break                            # waits for room; nothing behind it starts
            while t is None:
                victims = [r for r in running if r is not prefill]
                if not victims:
                    raise EngineError("a request does not fit the GPU tier on its own")
                v = max(victims, key=lambda r: r.seq)
                v.rem_decode = v.end - now
                running.remove(v)
                release(v.task, v.turn)
                suspended.insert(0, v)
                preemptions += 1
                events.append(("suspend", now, v.task, v.turn))
                t = try_start(cand.task, cand.turn, now, False)
            if resumed:
                suspended.pop(0)
                cand.resumes += 1
            else:
                fresh.remove(cand)
                cand.first_start = now
                cand.rem_decode = decode_us
            cand.seq = seq
            seq += 1
            running.append(cand)
            events.append(("resume" if resumed else "start", now, cand.task, cand.turn))
            prefill, prefill_end = cand, now + t
            if t == 0:                           # nothing to prefill: straight to decoding
                prefill.end = now + prefill.rem_decode
                prefill = None
                if cand.end <= now:
                    break                        # and nothing to decode: it retires before anything else starts
        if any(r is not prefill and r.end <= now for r in running):
            continue                             # a zero-length phase ended in this same instant
        # 3. advance to the next instant at which something can happen
        nxt = []
        if prefill is not None:
            nxt.append(prefill_end)
        nxt += [r.end for r in running if r is not prefill]
        if prefill is None and len(running) < running_cap and not suspended:
            nxt += [r.eligible for r in fresh if r.eligible > now]
        if not nxt:
            if fresh or suspended:
                raise EngineError("nothing can make progress")
            break
        now = min(nxt)
    order.sort(key=lambda o: (o[3], o[0]))
    return dict(order=order, makespan_us=makespan, preemptions=preemptions, events=events)


def replay(trace, oracle, model, active_pool, running_cap, decode_us, bytes_per_token, agent_keys=None):
    """Closed-loop replay of ``trace`` against a TraceOracle through ``begin`` / ``finish``.
    ``model``'s call_overhead_us is not used: decoding is ``decode_us``.  Returns simulate()'s
    dict plus the oracle's totals (``preempt_recomputed_tokens`` is J of Appendix C)."""
    tasks = sorted(trace.agent_tokens)
    b = oracle.b
    prefill_model = replace(model, call_overhead_us=0)
    decided = {}

    def rid(i, turn):
        return i * 1_000_000 + turn

    def try_start(i, turn, now_us, resumed):
        a = tasks[i]
        n = int(trace.agent_lengths[a][turn])
        keys = None if agent_keys is None else agent_keys[a][: n // b]
        rec = oracle.begin(rid(i, turn), trace.agent_tokens[a][:n], a, now_us // 1000, keys=keys,
                           decided=decided[(i, turn)] if resumed else None)
        if rec is None:
            return None
        if not resumed:
            decided[(i, turn)] = rec["save"]
        return service_us(prefill_model, rec["fresh_tokens"], rec["loaded"] * b * bytes_per_token,
                          rec["stored"] * b * bytes_per_token)

    out = simulate(len(tasks), lambda i: len(trace.agent_lengths[tasks[i]]),
                   lambda i, t: int(trace.agent_gaps_ms[tasks[i]][t]) * 1000,
                   active_pool, running_cap, decode_us, try_start,
                   lambda i, turn: oracle.finish(rid(i, turn)))
    out["totals"] = dict(oracle.totals)
    out["totals"].setdefault("preempt_recomputed_tokens", 0)
    return out
