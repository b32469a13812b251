"""Whole-trace control-plane parity on the CPU from the command line, for tier sizes and policies
beyond the ones tests/test_full_traces_cpu.py runs.

    python tests/check_full_traces.py --config c4 --host-gib 64,512
    python tests/check_full_traces.py --config c3 --policy 2
    python tests/check_full_traces.py --config c3 --policy 2 --host-gib 32 --closed-loop 16

Runs every request of a configuration's trace through the library's control plane
(control-plane-only context: no GPU needed) and through the oracle, and compares every output
of every request.  Block keys come from the oracle's hash, computed once per agent: prompts only
grow by appends, so a request's keys are a prefix of its agent's final key list.
"""
import argparse
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

from eakv_workloads import CONFIGS, SHAPES, make_trace  # noqa: E402
from oracle import hash as ohash  # noqa: E402
from oracle.trace import TraceOracle  # noqa: E402
from paper_2609_33762_b200 import build, eakv  # noqa: E402


def closed_loop(args, cfg, shape, trace, agent_keys, kh, kw, gib):
    """The library's scheduler and control plane against the oracle's closed-loop replay."""
    from oracle import closedloop as ocl
    from paper_2609_33762_b200 import closedloop
    b = shape.block_size
    t0 = time.time()
    want = ocl.replay(trace, TraceOracle(shape, cfg.gpu_blocks, kh, **kw), ocl.ServiceModel(), args.closed_loop,
                      shape.bytes_per_token, agent_keys=agent_keys)
    ctx = eakv.Context(num_layers=1, kv_heads=1, head_dim=8, block_size=b, gpu_blocks=cfg.gpu_blocks,
                       host_blocks=kh, kv_base=None, control_plane_only=True, **kw)
    np_keys = {a: np.asarray(k, dtype=np.uint64) for a, k in agent_keys.items()}

    def turn(tokens, agent, now_ms):
        n = len(tokens)
        k = np_keys[agent][: n // b]
        G, H, _, _ = ctx.eakv_match(k)
        st = ctx.eakv_tier_step(k, agent, n, now_ms)
        _, _, tail = ctx.eakv_gpu_tier_step(k, n % b != 0)
        if tail >= 0:
            ctx.eakv_gpu_tier_release(tail)
        return dict(fresh_tokens=n - max(G, H) * b, loaded=max(H - G, 0), stored=int(st["admit"].sum()))

    order, makespan, _ = closedloop.replay_trace(trace, turn, closedloop.ServiceModel(), args.closed_loop,
                                                 shape.bytes_per_token, b)
    stats = ctx.eakv_get_stats()
    ctx.close()
    assert order == want["order"], "call order differs"
    assert makespan == want["makespan_us"]
    print(f"{args.config} policy {args.policy} tier {gib} GiB closed loop A={args.closed_loop}: {len(order)} calls "
          f"in identical order, makespan {makespan / 1e6:.1f} s, computed prefill {want['totals']['fresh_tokens']}, "
          f"hits {stats['hits']} ({time.time() - t0:.0f} s)", flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="c4")
    ap.add_argument("--host-gib", default="64")
    ap.add_argument("--policy", type=int, default=0)
    ap.add_argument("--limit", type=int, default=None)
    ap.add_argument("--turn-engine", action="store_true", help="drive eakv_turn_begin / eakv_turn_end")
    ap.add_argument("--closed-loop", type=int, default=0, metavar="A",
                    help="closed-loop replay with an active pool of A tasks: call order, makespan and totals")
    args = ap.parse_args()
    build.build()
    from full_trace_util import compare_full_trace, trace_and_keys
    cfg, shape, trace, agent_keys = trace_and_keys(args.config)
    for gib in [float(x) for x in args.host_gib.split(",")]:
        kh = int(gib * (1 << 30) // shape.block_bytes)
        if args.closed_loop:
            kw = dict(policy=args.policy, kappa_blocks=cfg.kappa_blocks)
            closed_loop(args, cfg, shape, trace, agent_keys, kh, kw, gib)
            continue
        out = compare_full_trace(eakv, args.config, gib, policy=args.policy, limit=args.limit,
                                 turn_engine=args.turn_engine)
        print(f"{args.config} policy {args.policy} tier {gib} GiB ({kh} blocks): {out['requests']} requests, "
              f"{out['references']} references identical; computed prefill {out['computed_prefill']}, "
              f"restored blocks {out['restored_blocks']}, stored blocks {out['stored_blocks']} "
              f"({out['seconds']:.0f} s)", flush=True)


if __name__ == "__main__":
    main()
