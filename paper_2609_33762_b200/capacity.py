"""Capacity model of a trace on the GPU (the paper's stack-distance model, Section 3.2 and
Appendix C): predicted computed prefill and restored volume for a sweep of host-tier sizes,
and the working-set sizes that go with them.

    python -m paper_2609_33762_b200.capacity --config c2 --host-gib 8,16,32,64,128,256

The reference stream (each request touches all full blocks of its prompt, in request
order) is built from one batched hash launch: prompts only grow by appends, so a request's
keys are a prefix of its agent's final key list.
"""
from __future__ import annotations

import argparse
import json
import time

import numpy as np

from . import eakv

GIB = 1 << 30


def reference_stream(trace, shape, device="cuda:0"):
    """(stream keys on the device as int64 tensor, request offsets, request tokens, host keys)."""
    import torch
    b = shape.block_size
    agents = sorted(trace.agent_tokens)
    lens = [len(trace.agent_tokens[a]) for a in agents]
    # pad every agent's tokens to a multiple of 4 so each prompt starts 16-byte aligned
    starts, cur = [], 0
    for n in lens:
        starts.append(cur)
        cur += (n + 3) // 4 * 4
    flat = np.zeros(cur, dtype=np.int32)
    for a, s0, n in zip(agents, starts, lens):
        flat[s0:s0 + n] = trace.agent_tokens[a]
    # one launch per agent (each agent's final prompt once)
    tok_dev = torch.from_numpy(flat).to(device)
    ctx = eakv.Context(num_layers=1, kv_heads=1, head_dim=8, block_size=b, gpu_blocks=1, host_blocks=1,
                       kv_base=[tok_dev.data_ptr(), tok_dev.data_ptr()], tier_location=eakv.TIER_DEVICE,
                       tier_memory=tok_dev.data_ptr(), hash_scratch_blocks=max(1, cur // b + len(agents)))
    agent_keys = {}
    seed = ctx.eakv_hash_seed()
    for a, s0, n in zip(agents, starts, lens):
        nblk = n // b
        out = torch.empty(max(nblk, 1), dtype=torch.int64, device=device)
        ctx.eakv_hash_blocks(tok_dev.data_ptr() + 4 * s0, n, seed, out.data_ptr())
        agent_keys[a] = out[:nblk]
    torch.cuda.synchronize()
    ctx.close()
    pieces, offsets, tokens = [], [0], []
    for r in trace.requests:
        nblk = r.n_tokens // b
        pieces.append(agent_keys[r.agent][:nblk])
        offsets.append(offsets[-1] + nblk)
        tokens.append(r.n_tokens)
    stream = torch.cat(pieces) if pieces else torch.empty(0, dtype=torch.int64, device=device)
    return stream, np.asarray(offsets, dtype=np.int64), np.asarray(tokens, dtype=np.int64)


def gpu_prefixes(trace, shape, gpu_blocks, stream_host, offsets, gpu_free_order=eakv.FREE_ASCENDING):
    """G_j of every request from the library's GPU-tier bookkeeping (control plane only)."""
    b = shape.block_size
    ctx = eakv.Context(num_layers=1, kv_heads=1, head_dim=8, block_size=b, gpu_blocks=gpu_blocks,
                       host_blocks=1, kv_base=None, control_plane_only=True, gpu_free_order=gpu_free_order)
    G = np.zeros(len(trace.requests), dtype=np.int64)
    for j, r in enumerate(trace.requests):
        keys = stream_host[offsets[j]:offsets[j + 1]]
        G[j] = ctx.eakv_match(keys)[0]
        _, _, tail = ctx.eakv_gpu_tier_step(keys, r.n_tokens % b != 0)
        if tail >= 0:
            ctx.eakv_gpu_tier_release(tail)
    ctx.close()
    return G


def working_set_within(dist_ptr, n_refs, offsets, tokens, G, block_size, ws_full=None, percent=1):
    """Smallest tier (in blocks) whose predicted computed prefill is within ``percent`` % of the
    unbounded tier's (eakv_working_set_sizes: the search runs in the library)."""
    return eakv.eakv_working_set_sizes(dist_ptr, n_refs, offsets, tokens, G, block_size, percent)[1]


def model(config, host_gib, device="cuda:0", limit=None, agents=None, shared_prefix=0,
          gpu_free_order=eakv.FREE_ASCENDING):
    import torch
    from dataclasses import replace
    from eakv_workloads import CONFIGS, SHAPES, make_trace
    cfg = CONFIGS[config]
    if shared_prefix:
        cfg = replace(cfg, shared_prefix_tokens=shared_prefix)
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg, agents=agents)
    if limit:
        trace.requests = trace.requests[:limit]
    t0 = time.perf_counter()
    stream, offsets, tokens = reference_stream(trace, shape, device)
    t_stream = time.perf_counter() - t0
    n_refs = int(offsets[-1])
    dist = torch.empty(max(n_refs, 1), dtype=torch.int64, device=device)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    eakv.eakv_reuse_distances(stream.data_ptr(), n_refs, dist.data_ptr())
    t_dist = time.perf_counter() - t0
    stream_host = stream.cpu().numpy().view(np.uint64)
    G = gpu_prefixes(trace, shape, cfg.gpu_blocks, stream_host, offsets, gpu_free_order)
    caps = [max(1, int(g * GIB // shape.block_bytes)) for g in host_gib] + [1 << 40]
    t0 = time.perf_counter()
    out = eakv.eakv_capacity_curve(dist.data_ptr(), n_refs, offsets, tokens, G, shape.block_size, caps)
    t_curve = time.perf_counter() - t0
    ws_full, ws_99 = eakv.eakv_working_set_sizes(dist.data_ptr(), n_refs, offsets, tokens, G, shape.block_size, 1)
    # Eq. 5 and the pressure ratios of Section 3.2, integer arithmetic in the library
    sizing = eakv.eakv_working_set(num_layers=shape.num_layers, kv_heads=shape.kv_heads, head_dim=shape.head_dim,
                                   elem_bytes=shape.elem_bytes, block_size=shape.block_size,
                                   active_pool=len(trace.agent_tokens),
                                   total_prompt_tokens=trace.total_prompt_tokens, n_requests=len(trace.requests),
                                   gpu_blocks=cfg.gpu_blocks, host_blocks=0)
    ws_eq5 = sizing["working_set_blocks"]
    inf_computed = int(out["computed_tokens"][-1])
    rows = []
    for c, g in enumerate(host_gib):
        rows.append({"host_gib": g, "blocks": caps[c], "hits": int(out["hits"][c]),
                     # gamma_H = C_reuse / C_H (Section 3.2), with C_reuse the Eq. 5 scale
                     "gamma_h": eakv.eakv_working_set(
                         num_layers=shape.num_layers, kv_heads=shape.kv_heads, head_dim=shape.head_dim,
                         elem_bytes=shape.elem_bytes, block_size=shape.block_size,
                         active_pool=len(trace.agent_tokens), total_prompt_tokens=trace.total_prompt_tokens,
                         n_requests=len(trace.requests), host_blocks=caps[c])["gamma_h"],
                     "restored_tokens": int(out["restored_blocks"][c]) * shape.block_size,
                     "computed_prefill_tokens": int(out["computed_tokens"][c])})
    return {"config": config, "agents": len(trace.agent_tokens), "shared_prefix_tokens": shared_prefix,
            "gpu_free_order": "reverse" if gpu_free_order == eakv.FREE_REVERSE else "ascending",
            "gpu_hit_tokens": int(G.sum()) * shape.block_size,
            "requests": len(trace.requests), "references": n_refs,
            "prompt_tokens": int(tokens.sum()), "rows": rows,
            "computed_prefill_tokens_infinite_tier": inf_computed,
            # gamma_G = A * N_bar / K_G (Section 3.2), K_G in tokens
            "gamma_g": sizing["gamma_g"],
            "working_set_blocks": {"eq5": ws_eq5, "full": ws_full, "within_1_percent": ws_99},
            "working_set_gib": {"eq5": ws_eq5 * shape.block_bytes / GIB, "full": ws_full * shape.block_bytes / GIB,
                                "within_1_percent": ws_99 * shape.block_bytes / GIB},
            "seconds": {"stream": t_stream, "distances": t_dist, "curve": t_curve},
            "distance_refs_per_s": n_refs / t_dist if t_dist > 0 else None}


def audit(config, policy, host_gib, kappa=None, chunk_blocks=1, device="cuda:0", limit=None):
    """Declined-chunk audit (Appendix D): run the tier bookkeeping under an admission policy,
    then ask of every declined chunk whether its next reference lies beyond the tier's reach
    (reuse distance D >= K_H from the GPU model) or never comes."""
    import torch
    from eakv_workloads import CONFIGS, SHAPES, make_trace
    from .replay import POLICIES
    cfg = CONFIGS[config]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg)
    if limit:
        trace.requests = trace.requests[:limit]
    R = max(1, chunk_blocks)
    b = shape.block_size
    stream, offsets, tokens = reference_stream(trace, shape, device)
    keys_host = stream.cpu().numpy().view(np.uint64)
    # the tier's own reference stream: one key per full chunk
    chunk_keys, chunk_off = [], [0]
    for j in range(len(trace.requests)):
        k = keys_host[offsets[j]:offsets[j + 1]][R - 1::R]
        chunk_keys.append(k)
        chunk_off.append(chunk_off[-1] + len(k))
    cstream = np.concatenate(chunk_keys) if chunk_keys else np.zeros(0, np.uint64)
    kh = max(1, int(host_gib * GIB // (R * shape.block_bytes)))
    kap = max(1, cfg.kappa_blocks // R) if kappa is None else kappa     # the config's threshold, in tier units
    ctx = eakv.Context(num_layers=1, kv_heads=1, head_dim=8, block_size=b, gpu_blocks=1, host_blocks=kh,
                       kv_base=None, control_plane_only=True, policy=POLICIES[policy],
                       kappa_blocks=kap, chunk_blocks=R)
    declined = np.zeros(len(cstream), dtype=bool)
    for j, r in enumerate(trace.requests):
        st = ctx.eakv_tier_step(chunk_keys[j], r.agent, r.n_tokens, r.time_ms)
        declined[chunk_off[j]:chunk_off[j + 1]] = (st["hit"] == 0) & (st["admit"] == 0)
    stats = ctx.eakv_get_stats()
    ctx.close()
    n = len(cstream)
    cdev = torch.from_numpy(cstream.view(np.int64)).to(device)
    ddev = torch.from_numpy(declined.astype(np.uint8)).to(device)
    next_dist = torch.empty(max(n, 1), dtype=torch.int64, device=device)
    # the audit itself (reuse distances, next references, the condition of Proposition 1) runs in the library
    n_declined, meets, never = eakv.eakv_declined_audit(cdev.data_ptr(), ddev.data_ptr(), n, kh,
                                                        next_dist.data_ptr())
    nd = next_dist[:n]
    d_next = nd[nd >= 0].cpu().numpy()             # declined chunks that are referenced again: their D
    idx = range(n_declined)
    return {"config": config, "policy": policy, "host_gib": host_gib, "tier_units": kh, "chunk_blocks": R,
            "kappa": kap, "declined_chunks": int(len(idx)), "meet_condition": meets,
            "share_meeting_condition": meets / len(idx) if len(idx) else None,
            "never_referenced_again": never,
            "median_distance_over_capacity": float(np.median(d_next / kh)) if len(d_next) else None,
            "declined_requests": stats["declined_requests"], "pressure_requests": stats["pressure_requests"],
            "admitted_chunks": stats["admitted"]}


def kappa_sweep(config, host_gib, kappas, chunk_blocks=1, limit=None, device="cuda:0"):
    """Threshold sensitivity (Appendix D): under fixed admission, the requests each kappa filters
    and the share of new-chunk writes it declines, relative to a write-all run."""
    from eakv_workloads import CONFIGS, SHAPES, make_trace
    cfg = CONFIGS[config]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg)
    if limit:
        trace.requests = trace.requests[:limit]
    R = max(1, chunk_blocks)
    stream, offsets, _ = reference_stream(trace, shape, device)
    keys_host = stream.cpu().numpy().view(np.uint64)
    chunk_keys = [np.ascontiguousarray(keys_host[offsets[j]:offsets[j + 1]][R - 1::R])
                  for j in range(len(trace.requests))]
    kh = max(1, int(host_gib * GIB // (R * shape.block_bytes)))
    rows = []
    for kappa in kappas:
        ctx = eakv.Context(num_layers=1, kv_heads=1, head_dim=8, block_size=shape.block_size, gpu_blocks=1,
                           host_blocks=kh, kv_base=None, control_plane_only=True,
                           policy=eakv.POLICY_FILTER_FIXED, kappa_blocks=kappa, chunk_blocks=R)
        for j, r in enumerate(trace.requests):
            ctx.eakv_tier_step(chunk_keys[j], r.agent, r.n_tokens, r.time_ms)
        st = ctx.eakv_get_stats()
        ctx.close()
        new_chunks = st["admitted"] + st["declined"]
        rows.append({"kappa": kappa, "filtered_requests": st["declined_requests"],
                     "declined_chunks": st["declined"], "admitted_chunks": st["admitted"],
                     "share_of_new_chunk_writes_declined": st["declined"] / new_chunks if new_chunks else None,
                     "hits": st["hits"]})
    return {"config": config, "host_gib": host_gib, "tier_units": kh, "chunk_blocks": R, "rows": rows}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="c2", choices=["c0", "c0_big_tier", "c2", "c3", "c4"])
    ap.add_argument("--host-gib", default="8,16,32,64,128,256")
    ap.add_argument("--limit", type=int, default=None)
    ap.add_argument("--audit", default=None, choices=["fixed", "conditioned"],
                    help="declined-chunk audit under this policy instead of the capacity sweep")
    ap.add_argument("--chunk-blocks", type=int, default=1)
    ap.add_argument("--kappa", type=int, default=None)
    ap.add_argument("--kappa-sweep", default=None, help="comma-separated thresholds, fixed admission")
    ap.add_argument("--agents", type=int, default=None, help="active pool size (default: the config's)")
    ap.add_argument("--shared-prefix", type=int, default=0, help="system-prompt tokens shared by all agents")
    ap.add_argument("--reverse-free", action="store_true",
                    help="GPU tier keeps a request's blocks tail-first in its recency order")
    args = ap.parse_args()
    gib = [float(x) for x in args.host_gib.split(",")]
    if args.kappa_sweep:
        for g in gib:
            print(json.dumps(kappa_sweep(args.config, g, [int(k) for k in args.kappa_sweep.split(",")],
                                         chunk_blocks=args.chunk_blocks, limit=args.limit)))
        return
    if args.audit:
        for g in gib:
            print(json.dumps(audit(args.config, args.audit, g, kappa=args.kappa,
                                   chunk_blocks=args.chunk_blocks, limit=args.limit)))
        return
    out = model(args.config, gib, limit=args.limit, agents=args.agents, shared_prefix=args.shared_prefix,
                gpu_free_order=eakv.FREE_REVERSE if args.reverse_free else eakv.FREE_ASCENDING)
    print(json.dumps(out))


if __name__ == "__main__":
    main()
