"""Whole-trace control-plane parity on the CPU: every request of a configuration's trace through
the library's bookkeeping (a control-plane-only context: no GPU needed) and through the oracle,
every output of every request compared.  Block keys come from the oracle's hash, computed once
per agent: prompts only grow by appends, so a request's keys are a prefix of its agent's final
key list.  Used by tests/test_full_traces_cpu.py and by the command line in check_full_traces.py."""
import time

import numpy as np

from eakv_workloads import CONFIGS, SHAPES, make_trace
from oracle import hash as ohash
from oracle.trace import TraceOracle

_cache = {}


def trace_and_keys(config):
    """(cfg, shape, trace, agent -> oracle keys of its final prompt), cached per configuration."""
    if config not in _cache:
        cfg = CONFIGS[config]
        shape = SHAPES[cfg.shape]
        trace = make_trace(cfg)
        keys = {a: ohash.hash_blocks(toks.tolist(), shape.block_size) for a, toks in trace.agent_tokens.items()}
        _cache[config] = (cfg, shape, trace, keys)
    return _cache[config]


def compare_full_trace(eakv, config, host_gib, policy=0, limit=None, turn_engine=False, stride=1, **ctx_kw):
    """Returns a summary dict; raises AssertionError at the first request whose outputs differ.
    ``turn_engine``: drive the library through eakv_turn_begin / eakv_turn_end instead of the
    single calls.  ``stride`` > 1 compares the arrays of every stride-th request only (both sides
    still process every request; the scalars are compared for all)."""
    cfg, shape, trace, agent_keys = trace_and_keys(config)
    b = shape.block_size
    kh = int(host_gib * (1 << 30) // shape.block_bytes)
    kw = dict(policy=policy, kappa_blocks=cfg.kappa_blocks)
    kw.update(ctx_kw)
    oracle = TraceOracle(shape, cfg.gpu_blocks, kh, **kw)
    ctx = eakv.Context(num_layers=1, kv_heads=1, head_dim=8, block_size=b, gpu_blocks=cfg.gpu_blocks,
                       host_blocks=kh, kv_base=None, control_plane_only=True, **kw)
    t0 = time.time()
    refs = n = 0
    for i, r in enumerate(trace.requests):
        if limit and i >= limit:
            break
        keys = agent_keys[r.agent][: r.n_tokens // b]
        w = oracle.turn(range(r.n_tokens), r.agent, r.time_ms, keys=keys)
        k = np.asarray(keys, dtype=np.uint64)
        if turn_engine:
            v = ctx.eakv_turn_begin(0, r.n_tokens, k, r.agent, r.time_ms)
            ctx.eakv_turn_end()
            G, H = v["gpu_prefix_blocks"], v["host_prefix_blocks"]
            st = dict(v, pressure=bool(v["pressure"]), save=bool(v["save"]))
            res, blk = v["gpu_resident"], v["gpu_block"]
            assert (v["fresh_tokens"], v["restore_hi"] - v["restore_lo"], v["n_stored_blocks"], v["n_fill"]) == \
                   (w["fresh_tokens"], w["loaded"], w["stored"], w["filled"]), i
        else:
            G, H, _, _ = ctx.eakv_match(k)
            st = ctx.eakv_tier_step(k, r.agent, r.n_tokens, r.time_ms)
            res, blk, tail = ctx.eakv_gpu_tier_step(k, r.n_tokens % b != 0)
            if tail >= 0:
                ctx.eakv_gpu_tier_release(tail)
        assert (G, H, st["new_chunks"], st["pressure"], st["save"]) == \
               (w["G"], w["H"], w["new_chunks"], w["pressure"], w["save"]), i
        if i % stride == 0:
            assert np.array_equal(st["hit"], np.asarray(w["hit"], dtype=np.uint8)), i
            assert np.array_equal(st["admit"], np.asarray(w["admit"], dtype=np.uint8)), i
            assert np.array_equal(st["slot"], np.asarray(w["slot"], dtype=np.int32)), i
            assert list(zip(st["evicted_keys"].tolist(), st["evicted_slots"].tolist())) == w["evicted"], i
            assert np.array_equal(res, np.asarray(w["gpu_resident"], dtype=np.uint8)), i
            assert np.array_equal(blk, np.asarray(w["gpu_block"], dtype=np.int32)), i
        oracle.records.clear()
        refs += len(keys)
        n += 1
    stats = ctx.eakv_get_stats()
    for f in ("requests", "references", "hits", "admitted", "declined", "evicted"):
        assert stats[f] == oracle.host.stats[f], f
    ctx.close()
    return dict(config=config, policy=policy, host_gib=host_gib, host_blocks=kh, requests=n, references=refs,
                computed_prefill=oracle.totals["fresh_tokens"], restored_blocks=oracle.totals["loaded_blocks"],
                stored_blocks=oracle.totals["stored_blocks"], seconds=time.time() - t0)
