"""Replay a synthetic agent trace through the eakv path and report what the paper reports
for its replays: computed (fresh) prefill tokens, host writes and restores, hit tokens —
plus the achieved store/load rates.

    python -m paper_2609_33762_b200.replay --config c2              # tier sized by Eq. 5
    python -m paper_2609_33762_b200.replay --config c3 --policy conditioned
    python -m paper_2609_33762_b200.replay --config c4 --host-gib 64 --limit 2000

Sizing follows the paper's rule: working-set scale (A - 1) * N_mean * beta (Eq. 5) for
configurations whose tier capacity is defined as that working-set size, capped by the pinned memory
the box can spare.  With --no-data-plane only keys, matching and both tiers' bookkeeping run.
"""
from __future__ import annotations

import argparse
import json
import time

import numpy as np

from . import eakv

POLICIES = {"write_all": eakv.POLICY_WRITE_ALL, "fixed": eakv.POLICY_FILTER_FIXED,
            "conditioned": eakv.POLICY_FILTER_CONDITIONED}
GIB = 1 << 30


def working_set_blocks(trace, shape):
    """Eq. 5 in blocks: (A - 1) * mean prompt length * beta / block bytes (eakv_working_set)."""
    return eakv.eakv_working_set(num_layers=shape.num_layers, kv_heads=shape.kv_heads, head_dim=shape.head_dim,
                                 elem_bytes=shape.elem_bytes, block_size=shape.block_size,
                                 active_pool=len(trace.agent_tokens),
                                 total_prompt_tokens=trace.total_prompt_tokens,
                                 n_requests=len(trace.requests))["working_set_blocks"]


def mem_available_bytes():
    try:
        for line in open("/proc/meminfo"):
            if line.startswith("MemAvailable:"):
                return int(line.split()[1]) * 1024
    except OSError:
        pass
    return 0


def plan(cfg, trace, shape, host_gib=None, data_plane=True, ram_fraction=0.6):
    """Tier capacity in blocks for a configuration and the reason for it."""
    if host_gib is not None:
        kh, why = int(host_gib * GIB // shape.block_bytes), f"{host_gib} GiB requested"
    elif cfg.host_blocks:
        kh, why = cfg.host_blocks, "fixed by the configuration"
    else:
        kh, why = working_set_blocks(trace, shape), "working-set scale (A-1)*N_mean*beta"
    if data_plane:
        cap = int(mem_available_bytes() * ram_fraction // shape.block_bytes)
        if cap and kh > cap:
            kh, why = cap, why + f", capped at {ram_fraction:.0%} of available host memory"
    return kh, why


def run(config, *, policy="write_all", host_gib=None, limit=None, data_plane=True,
        incremental_hash=True, device="cuda:0", link_strategy=eakv.LINK_STAGED, agents=None,
        turns=None, server_hook=None, chunk_blocks=1, kappa=None, native_turn=True,
        gpu_free_order=eakv.FREE_ASCENDING, write_behind=False):
    import torch
    from eakv_workloads import CONFIGS, SHAPES, key_words_torch, make_trace
    from .harness import AgentServer

    cfg = CONFIGS[config]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg, agents=agents, turns=turns)
    kh, why = plan(cfg, trace, shape, host_gib, data_plane)
    kh = max(1, kh // chunk_blocks)                  # the tier counts chunks of chunk_blocks blocks
    payload = (lambda keys, q, n: key_words_torch(keys.astype(np.int64), q, n, device)) if data_plane else None
    t0 = time.perf_counter()
    server = AgentServer(shape, cfg.gpu_blocks, kh, payload, device=device, data_plane=data_plane,
                         incremental_hash=incremental_hash, policy=POLICIES[policy],
                         kappa_blocks=max(1, cfg.kappa_blocks // chunk_blocks) if kappa is None else kappa,
                         link_strategy=link_strategy, chunk_blocks=chunk_blocks,
                         native_turn=native_turn, gpu_free_order=gpu_free_order,
                         write_behind=write_behind)
    t_setup = time.perf_counter() - t0
    t0 = time.perf_counter()
    server.run(trace, limit=limit)
    torch.cuda.synchronize()
    wall = time.perf_counter() - t0
    rates = server.transfer_rates() if data_plane else None
    if server_hook is not None:
        server_hook(server, trace)
    st = server.ctx.eakv_get_stats()
    if server.hash_ctx is not server.ctx:            # bookkeeping-only run: the hashing context counts the hashing
        hs = server.hash_ctx.eakv_get_stats()
        st["tokens_hashed"], st["kernel_launches"] = hs["tokens_hashed"], hs["kernel_launches"]
    tot = server.totals
    n_req = len(server.records)
    out = {
        "config": config, "policy": policy, "requests": n_req, "kv_shape": cfg.shape,
        "gpu_blocks": cfg.gpu_blocks, "host_chunks": kh, "chunk_blocks": chunk_blocks,
        "gpu_free_order": "reverse" if gpu_free_order == eakv.FREE_REVERSE else "ascending",
        "write_behind": bool(write_behind),
        "host_gib": kh * chunk_blocks * shape.block_bytes / GIB,
        "host_sizing": why, "data_plane": data_plane, "native_turn": bool(native_turn),
        "working_set_blocks_eq5": working_set_blocks(trace, shape),
        "prompt_tokens": tot["prompt_tokens"], "computed_prefill_tokens": tot["fresh_tokens"],
        "gpu_hit_tokens": tot["gpu_hit_blocks"] * shape.block_size,
        "host_hit_tokens": tot["host_hit_blocks"] * shape.block_size,
        "restored_tokens": tot["loaded_blocks"] * shape.block_size,
        "stored_tokens": tot["stored_blocks"] * shape.block_size,
        "restored_gib": tot["loaded_blocks"] * shape.block_bytes / GIB,
        "stored_gib": tot["stored_blocks"] * shape.block_bytes / GIB,
        "declined_requests": st["declined_requests"], "pressure_requests": st["pressure_requests"],
        "declined_blocks": st["declined"], "evicted_blocks": st["evicted"],
        "tokens_hashed": st["tokens_hashed"], "kernel_launches": st["kernel_launches"],
        "wall_s": wall, "setup_s": t_setup, "transfer_rates": rates,
        "moved_gb_per_s_wall": (tot["loaded_blocks"] + tot["stored_blocks"]) * shape.block_bytes / wall / 1e9
        if data_plane else None,
    }
    server.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="c2", choices=["c0", "c0_big_tier", "c2", "c3", "c4"])
    ap.add_argument("--policy", default="write_all", choices=sorted(POLICIES))
    ap.add_argument("--host-gib", type=float, default=None)
    ap.add_argument("--limit", type=int, default=None, help="replay only the first N requests")
    ap.add_argument("--no-data-plane", dest="data_plane", action="store_false")
    ap.add_argument("--zero-copy", action="store_true", help="zero-copy host link instead of staged")
    ap.add_argument("--chunk-blocks", type=int, default=1,
                    help="host-tier chunk in GPU blocks (64 = the paper's 1,024-token chunks at block 16)")
    ap.add_argument("--kappa", type=int, default=None, help="write threshold in tier units")
    ap.add_argument("--single-calls", dest="native_turn", action="store_false",
                    help="drive the single calls one by one instead of eakv_turn_begin / eakv_turn_end")
    ap.add_argument("--write-behind", action="store_true",
                    help="host writes are deferred to a stream of the context (turn engine only)")
    ap.add_argument("--reverse-free", action="store_true",
                    help="GPU tier keeps a request's blocks tail-first in its recency order")
    args = ap.parse_args()
    out = run(args.config, policy=args.policy, host_gib=args.host_gib, limit=args.limit,
              data_plane=args.data_plane, chunk_blocks=args.chunk_blocks, kappa=args.kappa,
              native_turn=args.native_turn, write_behind=args.write_behind,
              gpu_free_order=eakv.FREE_REVERSE if args.reverse_free else eakv.FREE_ASCENDING,
              link_strategy=eakv.LINK_ZERO_COPY if args.zero_copy else eakv.LINK_STAGED)
    print(json.dumps(out))


if __name__ == "__main__":
    main()
