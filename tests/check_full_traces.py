"""Whole-trace control-plane parity on the CPU (not collected by pytest: it takes minutes).

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
    ap.add_argument("--closed-loop", type=int, default=0, metavar="A",
                    help="closed-loop replay with an active pool of A tasks: call order, makespan and totals")
    args = ap.parse_args()
    build.build()
    cfg = CONFIGS[args.config]
    shape = SHAPES[cfg.shape]
    b = shape.block_size
    trace = make_trace(cfg)
    t0 = time.time()
    agent_keys = {a: ohash.hash_blocks(toks.tolist(), b) for a, toks in trace.agent_tokens.items()}
    print(f"keys of {len(agent_keys)} agents in {time.time() - t0:.1f} s", flush=True)
    for gib in [float(x) for x in args.host_gib.split(",")]:
        kh = int(gib * (1 << 30) // shape.block_bytes)
        kw = dict(policy=args.policy, kappa_blocks=cfg.kappa_blocks)
        if args.closed_loop:
            closed_loop(args, cfg, shape, trace, agent_keys, kh, kw, gib)
            continue
        oracle = TraceOracle(shape, cfg.gpu_blocks, kh, **kw)
        ctx = eakv.Context(num_layers=1, kv_heads=1, head_dim=8, block_size=b, gpu_blocks=cfg.gpu_blocks,
                           host_blocks=kh, kv_base=None, control_plane_only=True, **kw)
        t0 = time.time()
        refs = 0
        for i, r in enumerate(trace.requests):
            if args.limit and i >= args.limit:
                break
            keys = agent_keys[r.agent][: r.n_tokens // b]
            w = oracle.turn(range(r.n_tokens), r.agent, r.time_ms, keys=keys)
            k = np.asarray(keys, dtype=np.uint64)
            G, H, _, _ = ctx.eakv_match(k)
            st = ctx.eakv_tier_step(k, r.agent, r.n_tokens, r.time_ms)
            res, blk, tail = ctx.eakv_gpu_tier_step(k, r.n_tokens % b != 0)
            if tail >= 0:
                ctx.eakv_gpu_tier_release(tail)
            assert (G, H, st["new_chunks"], st["pressure"], st["save"]) == \
                   (w["G"], w["H"], w["new_chunks"], w["pressure"], w["save"]), i
            assert np.array_equal(st["hit"], np.asarray(w["hit"], dtype=np.uint8)), i
            assert np.array_equal(st["admit"], np.asarray(w["admit"], dtype=np.uint8)), i
            assert np.array_equal(st["slot"], np.asarray(w["slot"], dtype=np.int32)), i
            assert list(zip(st["evicted_keys"].tolist(), st["evicted_slots"].tolist())) == w["evicted"], i
            assert np.array_equal(res, np.asarray(w["gpu_resident"], dtype=np.uint8)), i
            assert np.array_equal(blk, np.asarray(w["gpu_block"], dtype=np.int32)), i
            oracle.records.clear()
            refs += len(keys)
        stats = ctx.eakv_get_stats()
        for f in ("requests", "references", "hits", "admitted", "declined", "evicted"):
            assert stats[f] == oracle.host.stats[f], f
        ctx.close()
        print(f"{args.config} policy {args.policy} tier {gib} GiB ({kh} blocks): {i + 1} requests, "
              f"{refs} references identical; computed prefill {oracle.totals['fresh_tokens']}, "
              f"restored blocks {oracle.totals['loaded_blocks']}, stored blocks "
              f"{oracle.totals['stored_blocks']} ({time.time() - t0:.0f} s)", flush=True)


if __name__ == "__main__":
    main()
