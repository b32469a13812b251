"""Closed-loop replay with a service-time model (test infrastructure, CPU only).

Section 2 ("A closed-loop workload"), Section 5.1 and Appendix B ("Workload construction",
"Timing boundary"): A tasks are active at a time, admitted in list order; a task may issue call
k+1 only after call k's response is complete and the recorded gap between the two has gone by;
a task that has finished all of its calls frees its place for the next one in the list; the
makespan is when the last response of all completes, gaps included.  Serving decisions therefore change the order in which the tiers see
the calls.

The engine here is this build's reading (the paper runs a real engine): one call at a time,
taken in order of eligibility (ties: lower task id).  Its response time follows Eq. 2:
recomputing n tokens costs n * t_pf, restoring n tokens costs n * beta / B_H2D + tau_load;
a blocking host write costs bytes / B_D2H; every call pays a fixed overhead that stands for
decoding.  All times are integer microseconds, every division rounds up.
"""
from dataclasses import dataclass


@dataclass(frozen=True)
class ServiceModel:
    t_pf_ns: int = 10_000            # prefill time per computed token, nanoseconds
    h2d_bytes_per_us: int = 55_000   # effective host-to-GPU bandwidth (55,000 B/us = 55 GB/s)
    d2h_bytes_per_us: int = 55_000   # GPU-to-host bandwidth for writes
    tau_load_us: int = 200           # fixed restoration overhead, paid when anything is restored
    call_overhead_us: int = 0        # fixed part of a response (decoding, frontend)
    store_blocking: bool = True      # the response waits for its host write


def ceil_div(a, b):
    return -(-a // b)


def service_us(model, computed_tokens, restored_bytes, stored_bytes):
    t = model.call_overhead_us + ceil_div(computed_tokens * model.t_pf_ns, 1000)
    if restored_bytes > 0:
        t += model.tau_load_us + ceil_div(restored_bytes, model.h2d_bytes_per_us)
    if model.store_blocking and stored_bytes > 0:
        t += ceil_div(stored_bytes, model.d2h_bytes_per_us)
    return t


def simulate(n_tasks, turns_of, gap_us_of, active_pool, serve):
    """Run the closed loop.

    turns_of(task) -> number of calls; gap_us_of(task, turn) -> interval before that call
    (turn >= 1); serve(task, turn, start_us) -> service time in microseconds (it performs the
    call against the tiers).  Returns (order, makespan_us) with order = list of
    (task, turn, eligible_us, start_us, finish_us)."""
    waiting = list(range(n_tasks))            # tasks not yet in the pool, in order
    eligible = {}                             # task -> (turn, eligible time) of its next call
    while waiting and len(eligible) < active_pool:
        eligible[waiting.pop(0)] = (0, 0)
    server_free = 0
    order = []
    makespan = 0
    while eligible:
        # first come, first served by eligibility; lower task id breaks ties
        task = min(eligible, key=lambda k: (eligible[k][1], k))
        turn, when = eligible.pop(task)
        start = max(when, server_free)
        finish = start + serve(task, turn, start)
        server_free = finish
        order.append((task, turn, when, start, finish))
        makespan = max(makespan, finish)
        if turn + 1 < turns_of(task):
            eligible[task] = (turn + 1, finish + gap_us_of(task, turn + 1))
        elif waiting:
            eligible[waiting.pop(0)] = (0, finish)
    return order, makespan


def replay(trace, oracle, model, active_pool, bytes_per_token, agent_keys=None):
    """Closed-loop replay of ``trace`` against a TraceOracle.  Returns dict(order, makespan_us,
    totals) where totals are the oracle's token/block counters.  ``agent_keys`` (agent -> block
    keys of its final prompt) spares re-hashing: prompts only grow by appends, so a call's keys are
    a prefix of that list."""
    tasks = sorted(trace.agent_tokens)
    b = oracle.b

    def serve(i, turn, start_us):
        a = tasks[i]
        n = int(trace.agent_lengths[a][turn])
        keys = None if agent_keys is None else agent_keys[a][: n // b]
        rec = oracle.turn(trace.agent_tokens[a][:n], a, start_us // 1000, keys=keys)
        return service_us(model, rec["fresh_tokens"], rec["loaded"] * b * bytes_per_token,
                          rec["stored"] * b * bytes_per_token)

    order, makespan = simulate(len(tasks), lambda i: len(trace.agent_lengths[tasks[i]]),
                               lambda i, t: int(trace.agent_gaps_ms[tasks[i]][t]) * 1000,
                               active_pool, serve)
    return dict(order=order, makespan_us=makespan, totals=dict(oracle.totals))
