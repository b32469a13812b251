#!/usr/bin/env python
"""Benchmark of the paged-KV offload hot path on B200 (store/load microbench workload with
Qwen3-30B-A3B-shaped KV: 48 layers, 4 KV heads, head_dim 128, bf16, block 16).

One step = one pass of the whole path over one batch: two requests of `--blocks` blocks
each.  Request 1 resubmits the prompt of two steps ago (its KV is host-resident and gone
from the GPU): hash -> match -> tier step (all hits) -> load every block into freshly
drawn, uniform-random pool blocks.  Request 2 is a new prompt: hash -> match (nothing) ->
tier step (every block admitted, evicting the oldest prompt) -> store from uniform-random
pool blocks.  Bytes moved per step = 2 * blocks * 1.5 MiB.

  value  whole-step GB/s with the tier in HBM and tokens resident on the device (the
         on-device gather/scatter, HBM roofline);
  e2e    the same step through the same calls with the tier in pinned host memory and the
         tokens in pinned host memory (host-link roofline; H2D/D2H bytes inside the timing).

`--impl reference` times the CPU oracle on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

# The request that restores resubmits the prompt stored LAG steps earlier, and the tier holds
# TIER_PROMPTS prompts, so restores and host writes of neighbouring steps are independent and
# both directions of the link stay busy (each prompt is still written once and restored once).
LAG = 2
TIER_PROMPTS = 3
METRIC = "kv_store_load_gbps"
UNIT = "GB/s"
WORKLOAD = "c1_store_load_microbench_qwen3_30b_a3b"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="eakv", choices=["eakv", "reference"])
    ap.add_argument("--blocks", type=int, default=4096, help="blocks per request")
    ap.add_argument("--pool-blocks", type=int, default=65536)
    ap.add_argument("--link", default="staged", choices=["zero_copy", "staged", "copy_engine"],
                    help="host-link strategy of the e2e arm")
    ap.add_argument("--copy-path", default="bulk", choices=["vector", "bulk"])
    ap.add_argument("--copy-ctas", type=int, default=0)
    ap.add_argument("--host-ctas", type=int, default=0)
    ap.add_argument("--host-copy-path", default="bulk_load", choices=["vector", "bulk_load", "bulk_both"],
                    help="device code that moves a mapped host tier (zero-copy strategy)")
    ap.add_argument("--host-load-ctas", type=int, default=0)
    ap.add_argument("--host-store-ctas", type=int, default=0)
    ap.add_argument("--staging-mib", type=int, default=256)
    ap.add_argument("--no-overlap", dest="overlap", action="store_false",
                    help="e2e arm: restores and host writes on one stream instead of two")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--quick", action="store_true",
                    help="main line and e2e arm only: no side measurements (strategy matrix, curve, hash, "
                         "control plane, CPU baseline); for sweeps")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--hash-only", action="store_true",
                    help="run only the prefix-hash throughput section and print its JSON")
    ap.add_argument("--hash-prompts", type=int, default=512)
    ap.add_argument("--tp-shard", type=int, default=1,
                    help="run the microbench on one tensor-parallel rank's KV shape (heads / TP) instead "
                         "of the unsharded one; not the headline workload")
    ap.add_argument("--sweep", action="store_true",
                    help="also print the 1..4096-block curve (contiguous/random ids, masks)")
    return ap.parse_args()


# ------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------
class ClockSampler:
    """Polls SM clock and throttle reasons through NVML (read-only) every few milliseconds
    on a thread, so that even a short timed region gets samples under load."""
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap"}

    def __init__(self, index):
        self.index = index
        self.samples = []          # (perf_counter, sm_mhz, reasons bitmask)
        self.thread = None
        self.stop_flag = False
        self.max_mhz = None
        self.err = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            idx = self.index
            if vis:
                ids = [v for v in vis.split(",") if v.strip()]
                if idx < len(ids) and ids[idx].strip().isdigit():
                    idx = int(ids[idx])
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            self.nv = pynvml
            # the first queries after initialisation can take much longer than the rest
            pynvml.nvmlDeviceGetClockInfo(self.handle, pynvml.NVML_CLOCK_SM)
            pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle)
        except Exception as e:  # noqa: BLE001
            self.err = repr(e)
            return
        self.thread = threading.Thread(target=self._poll, daemon=True)
        self.thread.start()

    def _poll(self):
        nv = self.nv
        while not self.stop_flag:
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM)
                rs = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle)
                self.samples.append((time.perf_counter(), float(mhz), int(rs)))
            except Exception as e:  # noqa: BLE001
                self.err = repr(e)
                return
            time.sleep(0.002)

    def mark(self):
        return time.perf_counter()

    def stop(self, t0=None, t1=None):
        self.stop_flag = True
        if self.thread is not None:
            self.thread.join(timeout=2)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "samples": 0,
                    "reasons": ["no samples: " + str(self.err)]}
        sel = [x for x in self.samples if (t0 is None or x[0] >= t0) and (t1 is None or x[0] <= t1)]
        scope = "timed region"
        if len(sel) < 3:                      # region shorter than the polling period
            sel, scope = self.samples, "warm-up + timed region"
        mask = 0
        for _, _, r in sel:
            mask |= r
        return {"sm_mhz": float(np.median([x[1] for x in sel])), "sm_max_mhz": self.max_mhz,
                "samples": len(sel), "scope": scope,
                "reasons": sorted(n for bit, n in self.REASONS.items() if mask & bit)}


# ------------------------------------------------------------------------------------------
# the step
# ------------------------------------------------------------------------------------------
class Arm:
    """One configuration of the path (device tier or pinned-host tier) over a shared pool."""

    def __init__(self, args, pool, shape, torch, eakv, *, host_tier, device, link=None, copy_path=None,
                 tier_memory=None):
        self.torch, self.eakv = torch, eakv
        link = link or args.link
        copy_path = copy_path or args.copy_path
        self.m = args.blocks
        self.b = shape.block_size
        self.n_tokens = self.m * self.b
        self.host_tier = host_tier
        self.device = device
        kw = dict(copy_path=eakv.COPY_BULK if copy_path == "bulk" else eakv.COPY_VECTOR,
                  max_call_blocks=max(16384, self.m))
        if host_tier:
            kw.update(tier_location=eakv.TIER_PINNED_HOST,
                      link_strategy={"staged": eakv.LINK_STAGED, "zero_copy": eakv.LINK_ZERO_COPY,
                                     "copy_engine": eakv.LINK_COPY_ENGINE}[link],
                      staging_bytes=args.staging_mib << 20, copy_ctas=args.host_ctas,
                      host_copy_path={"vector": 0, "bulk_load": 1, "bulk_both": 2}[args.host_copy_path],
                      host_load_ctas=args.host_load_ctas, host_store_ctas=args.host_store_ctas)
            if link == "staged":
                kw["copy_ctas"] = args.copy_ctas
            if tier_memory is not None:
                kw["tier_memory"] = tier_memory
        else:
            # the tier is a tensor of ours that the context adopts, so it can be inspected
            self.tier_t = torch.empty((TIER_PROMPTS * self.m, shape.pieces_per_block, shape.piece_bytes // 2),
                                      dtype=torch.int16, device=device)
            kw.update(tier_location=eakv.TIER_DEVICE, link_strategy=eakv.LINK_ZERO_COPY,
                      copy_ctas=args.copy_ctas, tier_memory=self.tier_t.data_ptr())
        self.ctx = eakv.Context(num_layers=shape.num_layers, kv_heads=shape.kv_heads,
                                head_dim=shape.head_dim, block_size=shape.block_size,
                                gpu_blocks=pool.gpu_blocks, host_blocks=TIER_PROMPTS * self.m,
                                kv_base=pool.kv_base, **kw)
        self.block_bytes = self.ctx.block_bytes
        # lookups (hash, key read-back) run on their own stream so the host control plane of
        # the next request overlaps the transfers of the previous one; the e2e arm also gives
        # restores and host writes a stream each (full-duplex link), ordered by events
        self.hash_stream = torch.cuda.Stream(device)
        self.load_stream = torch.cuda.Stream(device)
        self.store_stream = torch.cuda.Stream(device) if (host_tier and args.overlap) else self.load_stream
        self.load_done = [torch.cuda.Event() for _ in range(4)]     # by step modulo 4
        self.store_done = [torch.cuda.Event() for _ in range(4)]
        self.seed = self.ctx.eakv_hash_seed()
        self.keys_dev = torch.empty(self.m, dtype=torch.int64, device=device)
        self.keys_host = torch.empty(self.m, dtype=torch.int64).pin_memory()
        self.tok_dev = torch.empty(self.n_tokens, dtype=torch.int32, device=device)
        self.h2d = self.d2h = 0

    def streams(self):
        return {self.hash_stream, self.load_stream, self.store_stream}

    def request(self, tokens, table, agent, now, timed_events=None, step_idx=0):
        """tokens: device int32 tensor (device arm) or pinned host tensor (e2e arm)."""
        torch = self.torch
        hs = self.hash_stream
        # Lookups never touch a copy engine: queued behind the bulk transfers of other
        # requests they would wait for all of them.  Host-resident tokens are read by the
        # hash kernel straight from pinned memory and the keys are written straight into
        # pinned memory (both mapped into the device's address space).
        if tokens.device.type == "cpu":
            self.h2d += tokens.numel() * 4
        nblk = self.ctx.eakv_hash_blocks(tokens.data_ptr(), self.n_tokens, self.seed,
                                         self.keys_host.data_ptr(), hs)
        hs.synchronize()
        self.d2h += nblk * 8
        keys = self.keys_host.numpy().view(np.uint64)
        G, H, _, slots = self.ctx.eakv_match(keys)
        step = self.ctx.eakv_tier_step(keys, agent, self.n_tokens, now)
        moved = 0
        if H > 0:
            ls = self.load_stream
            # the slots being read were written by the store of LAG steps ago
            ls.wait_event(self.store_done[(step_idx - LAG) % 4])
            ev = self._timer(ls, timed_events)
            self.ctx.eakv_load(slots[:H], table[:H], ls)
            self._timer_end(ls, ev, H * self.block_bytes, timed_events)
            self.load_done[step_idx % 4].record(ls)
            moved += H * self.block_bytes
            self.h2d += H * self.block_bytes if self.host_tier else 0
        n_admit = int(step["admit"].sum())
        if n_admit:
            ss = self.store_stream
            # the slots this store overwrites held the prompt the previous step restored
            ss.wait_event(self.load_done[(step_idx - 1) % 4])
            ev = self._timer(ss, timed_events)
            self.ctx.eakv_store(table, step["admit"], step["slot"], ss)
            self._timer_end(ss, ev, n_admit * self.block_bytes, timed_events)
            self.store_done[step_idx % 4].record(ss)
            moved += n_admit * self.block_bytes
            self.d2h += n_admit * self.block_bytes if self.host_tier else 0
        return moved, H, n_admit

    def _timer(self, stream, timed_events):
        if timed_events is None:
            return None
        ev = (self.torch.cuda.Event(enable_timing=True), self.torch.cuda.Event(enable_timing=True))
        ev[0].record(stream)
        return ev

    def _timer_end(self, stream, ev, nbytes, timed_events):
        if ev is not None:
            ev[1].record(stream)
            timed_events.append((nbytes, ev))

    def step(self, s, prompts, tables, timed_events=None):
        """prompts[s-LAG] was stored LAG steps ago; prompts[s] is new.  The two requests use
        disjoint, freshly drawn pool blocks."""
        m = self.m
        a, _, _ = self.request(prompts[s - LAG], tables[s][:m], agent=(s - LAG) % 4, now=s * 1000,
                               timed_events=timed_events, step_idx=s)
        b, _, _ = self.request(prompts[s], tables[s][m:], agent=s % 4, now=s * 1000 + 500,
                               timed_events=timed_events, step_idx=s)
        return a + b


def run_arm(arm, prompts, tables, steps, warmup, dist, clocks=None, time_kernels=True):
    torch = arm.torch
    main = torch.cuda.current_stream(arm.device)
    if clocks:
        clocks.start()
    # prime: store the first LAG prompts so that the first step has something to restore
    for s in range(LAG):
        arm.request(prompts[s], tables[s][arm.m:], agent=s % 4, now=0, step_idx=s)
    for s in range(LAG, warmup + LAG):
        arm.step(s, prompts, tables)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    arm.h2d = arm.d2h = 0
    launches0 = arm.ctx.eakv_get_stats()["kernel_launches"]
    timed = [] if time_kernels else None
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(main)                      # the device is idle: this is the start of the region
    for st in arm.streams():
        st.wait_stream(main)
    moved = 0
    for s in range(warmup + LAG, warmup + LAG + steps):
        moved += arm.step(s, prompts, tables, timed_events=timed)
    for st in arm.streams():
        main.wait_stream(st)
    e1.record(main)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    clk = clocks.stop(t0, time.perf_counter()) if clocks else None
    if dist is not None:
        dist.barrier()
    launches = arm.ctx.eakv_get_stats()["kernel_launches"] - launches0
    kernel = [(b, ev[0].elapsed_time(ev[1])) for b, ev in (timed or []) if b > 0]
    return dict(ms=ms, moved=moved, launches=launches, kernel=kernel, clocks=clk,
                h2d=arm.h2d / steps, d2h=arm.d2h / steps)


def hash_throughput(torch, eakv, pool, shape, device, peak_gbs, prompts=512, tokens=65536, reps=10):
    """Prefix-hash rate: a batch of long prompts in one launch (device-resident tokens, larger
    than L2), and the latency of one 64k-token prompt."""
    ctx = eakv.Context(num_layers=shape.num_layers, kv_heads=shape.kv_heads, head_dim=shape.head_dim,
                       block_size=shape.block_size, gpu_blocks=pool.gpu_blocks, host_blocks=1,
                       kv_base=pool.kv_base, tier_location=eakv.TIER_DEVICE,
                       tier_memory=pool.pieces[0].data_ptr(),
                       hash_scratch_blocks=prompts * tokens // shape.block_size)
    toks = torch.randint(0, 151936, (prompts * tokens,), dtype=torch.int32, device=device)
    keys = torch.empty(prompts * tokens // shape.block_size, dtype=torch.int64, device=device)
    offsets = np.arange(prompts + 1, dtype=np.int64) * tokens
    stream = torch.cuda.current_stream(device)
    best = None
    for i in range(reps + 3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        ctx.eakv_hash_blocks_batched(toks.data_ptr(), offsets, None, keys.data_ptr(), stream)
        e1.record(stream)
        torch.cuda.synchronize()
        if i >= 3:
            ms = e0.elapsed_time(e1)
            best = ms if best is None else min(best, ms)
    # sustained rate: launches enqueued back to back, so host-side preparation of the next call
    # overlaps the kernel of the previous one
    burst = 8
    sustained = None
    for i in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(burst):
            ctx.eakv_hash_blocks_batched(toks.data_ptr(), offsets, None, keys.data_ptr(), stream)
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / burst
        sustained = ms if sustained is None else min(sustained, ms)
    # two contexts on two streams, calls alternating: the scan launch of one call overlaps the token
    # launch of the next (each context has its own scratch, so the two calls are independent)
    ctx2 = eakv.Context(num_layers=shape.num_layers, kv_heads=shape.kv_heads, head_dim=shape.head_dim,
                        block_size=shape.block_size, gpu_blocks=pool.gpu_blocks, host_blocks=1,
                        kv_base=pool.kv_base, tier_location=eakv.TIER_DEVICE,
                        tier_memory=pool.pieces[0].data_ptr(),
                        hash_scratch_blocks=prompts * tokens // shape.block_size)
    keys2 = torch.empty_like(keys)
    s2 = torch.cuda.Stream(device)
    two_stream = None
    for i in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        s2.wait_stream(stream)
        for j in range(burst):
            if j % 2 == 0:
                ctx.eakv_hash_blocks_batched(toks.data_ptr(), offsets, None, keys.data_ptr(), stream)
            else:
                ctx2.eakv_hash_blocks_batched(toks.data_ptr(), offsets, None, keys2.data_ptr(), s2)
        stream.wait_stream(s2)
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / burst
        two_stream = ms if two_stream is None else min(two_stream, ms)
    ctx2.close()
    single = []
    seed = ctx.eakv_hash_seed()
    for i in range(reps + 3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        ctx.eakv_hash_blocks(toks.data_ptr() + 4 * tokens * (i % prompts), tokens, seed, keys.data_ptr(), stream)
        e1.record(stream)
        torch.cuda.synchronize()
        if i >= 3:
            single.append(e0.elapsed_time(e1) * 1e3)
    # latency of one call against prompt length, and the incremental case: an agent turn that
    # appends ~3k tokens to a 48k-token prompt hashes only the appended blocks (parent = the key
    # of the last block it already has)
    def call_us(n_tok, parent):
        ts = []
        for i in range(reps + 3):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            ctx.eakv_hash_blocks(toks.data_ptr(), n_tok, parent, keys.data_ptr(), stream)
            e1.record(stream)
            torch.cuda.synchronize()
            if i >= 3:
                ts.append(e0.elapsed_time(e1) * 1e3)
        return float(np.median(ts))
    latency = {str(n): call_us(n, seed) for n in (1024, 4096, 16384, 65536, 131072) if n <= prompts * tokens}
    inc_us = call_us(3072, 0x123456789ABCDEF)
    # tokens that still sit in pinned host memory: the kernel reads them through the mapping, so
    # the host link bounds the rate at 4 bytes per token
    n_host = min(131072, prompts * tokens)
    host_toks = torch.randint(0, 151936, (n_host,), dtype=torch.int32).pin_memory()
    ts = []
    for i in range(reps + 3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        ctx.eakv_hash_blocks(host_toks.data_ptr(), n_host, seed, keys.data_ptr(), stream)
        e1.record(stream)
        torch.cuda.synchronize()
        if i >= 3:
            ts.append(e0.elapsed_time(e1) * 1e3)
    host_us = float(np.median(ts))
    # what a lookup costs its caller: wall time from the call to the keys being readable on the host
    # (tokens in pinned memory in, keys in pinned memory out), next to the floor any kernel pays on
    # this machine through Python: one trivial kernel launch plus a stream synchronize
    keys_pin = torch.empty(8192, dtype=torch.int64).pin_memory()
    one = torch.zeros(1, device=device)

    def wall_us(fn, reps=60):
        ts = []
        for i in range(reps + 5):
            t0 = time.perf_counter()
            fn()
            stream.synchronize()
            if i >= 5:
                ts.append((time.perf_counter() - t0) * 1e6)
        return float(np.median(ts))
    lookup = {str(n): wall_us(lambda n=n: ctx.eakv_hash_blocks(host_toks.data_ptr(), n, seed, keys_pin.data_ptr(), stream))
              for n in (16, 1024, 4096, 65536) if n <= n_host}
    floor_us = wall_us(lambda: one.add_(1))
    ctx.close()
    rate = prompts * tokens / (best * 1e-3)
    srate = prompts * tokens / (sustained * 1e-3)
    return {"sustained_tokens_per_s": srate, "sustained_ms_per_launch": sustained,
            "sustained_frac_of_hbm_bound": srate * 4 / 1e9 / peak_gbs,
            "two_streams_tokens_per_s": prompts * tokens / (two_stream * 1e-3),
            "two_streams_ms_per_call": two_stream,
            "batched_tokens_per_s": rate, "batch": f"{prompts} prompts x {tokens} tokens, block {shape.block_size}",
            "batched_ms": best, "frac_of_hbm_bound": rate * 4 / 1e9 / peak_gbs,
            "hbm_bound_tokens_per_s": peak_gbs * 1e9 / 4,
            "single_prompt_tokens": tokens, "single_prompt_us_median": float(np.median(single)),
            "single_call_us_by_tokens": latency,
            "lookup_wall_us_by_tokens": lookup, "launch_and_sync_floor_us": floor_us,
            "lookup_note": "wall time of eakv_hash_blocks + stream synchronize, tokens and keys in pinned host "
                           "memory; the floor is one trivial kernel launch + synchronize on the same stream",
            "host_resident_prompt": {"tokens": n_host, "us": host_us, "tokens_per_s": n_host / (host_us * 1e-6),
                                     "bytes_per_s": 4 * n_host / (host_us * 1e-6),
                                     "note": "tokens read from pinned host memory through the mapping"},
            "incremental": {"appended_tokens": 3072, "us": inc_us, "appended_tokens_per_s": 3072 / (inc_us * 1e-6),
                            "equivalent_full_prompt_tokens_per_s": 49152 / (inc_us * 1e-6),
                            "note": "a 48k-token turn that appends 3k tokens hashes 3k, not 48k"}}


def control_plane_rate(eakv, pool, shape, device, requests=400, blocks=4096):
    """Single-thread rate of the host control plane: block references per second through
    eakv_match and eakv_tier_step on a thrashing tier (every second request re-references the
    previous one's keys, the others insert and evict)."""
    ctx = eakv.Context(num_layers=shape.num_layers, kv_heads=shape.kv_heads, head_dim=shape.head_dim,
                       block_size=shape.block_size, gpu_blocks=pool.gpu_blocks, host_blocks=3 * blocks,
                       kv_base=pool.kv_base, tier_location=eakv.TIER_DEVICE,
                       tier_memory=pool.pieces[0].data_ptr())
    rng = np.random.default_rng(3)
    keys = [rng.integers(1, 1 << 60, size=blocks, dtype=np.uint64) for _ in range(requests // 2 + 1)]
    t_match = t_step = 0.0
    refs = 0
    for i in range(requests):
        k = keys[i // 2]
        t0 = time.perf_counter()
        ctx.eakv_match(k)
        t1 = time.perf_counter()
        ctx.eakv_tier_step(k, i % 7, blocks * shape.block_size, i * 100)
        t2 = time.perf_counter()
        t_match += t1 - t0
        t_step += t2 - t1
        refs += blocks
    st = ctx.eakv_get_stats()
    ctx.close()
    out = {"match_refs_per_s": refs / t_match, "tier_step_refs_per_s": refs / t_step,
           "references": refs, "hits": st["hits"], "evicted": st["evicted"],
           "note": "through the Python binding, one thread"}
    out["turn"] = turn_overhead(eakv, device)
    return out


def turn_overhead(eakv, device, prompt_blocks=3072, appended_blocks=192, reps=20):
    """Wall time of one whole turn through eakv_turn_begin + eakv_turn_end when nothing has to move:
    a 48k-token prompt of which the last 3k tokens are new since the previous turn (their keys are
    hashed on the GPU, the others are passed in), every block resident on the GPU, the write
    declined.  What is left is the library's own cost per turn: hashing, the lookups and both
    tiers' bookkeeping over 3,072 blocks.  (A KV shape of 512 bytes per block keeps the pool small;
    the control plane does not depend on it.)"""
    import torch
    b, nb = 16, 2 * prompt_blocks
    piece = b * 1 * 8 * 2
    pool = [torch.zeros(nb * piece // 2, dtype=torch.int16, device=device) for _ in range(2)]
    ctx = eakv.Context(num_layers=1, kv_heads=1, head_dim=8, block_size=b, gpu_blocks=nb,
                       host_blocks=2 * prompt_blocks, kv_base=[t.data_ptr() for t in pool],
                       tier_location=eakv.TIER_DEVICE, policy=eakv.POLICY_FILTER_FIXED, kappa_blocks=0)
    stream = torch.cuda.current_stream(device)
    tok = torch.randint(0, 150000, (prompt_blocks * b,), dtype=torch.int32).pin_memory()
    n_prev = (prompt_blocks - appended_blocks) * b
    v = ctx.eakv_turn_begin(tok.data_ptr(), n_prev, None, 0, 0, stream)
    ctx.eakv_turn_end(stream)
    known = v["keys"]
    times = []
    for i in range(reps + 3):
        t0 = time.perf_counter()
        v = ctx.eakv_turn_begin(tok.data_ptr(), prompt_blocks * b, known, 0, i + 1, stream)
        ctx.eakv_turn_end(stream)
        times.append(time.perf_counter() - t0)
    ctx.eakv_sync()
    assert v["gpu_prefix_blocks"] == prompt_blocks and v["n_stored_blocks"] == 0
    ctx.close()
    return {"wall_us_median": float(np.median(times[3:])) * 1e6, "prompt_tokens": prompt_blocks * b,
            "appended_tokens": appended_blocks * b,
            "note": "eakv_turn_begin + eakv_turn_end, prompt resident on the GPU, write declined: "
                    "hash of the appended tokens + lookups + bookkeeping of 3,072 blocks"}


def layered_load_probe(torch, arm, tables, shape, layers_per_group=12):
    """Restore 4,096 blocks from the pinned tier whole, and in layer groups: when the first
    group's event fires a consumer could start on those layers."""
    m = arm.m
    slots = np.arange(m, dtype=np.int32)
    table = tables[0][:m]
    st = torch.cuda.Stream(arm.device)
    groups = -(-shape.num_layers // layers_per_group)
    out = {}
    for mode in ("plain", "layered"):
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(groups)]
        for ev in evs:
            ev.record(st)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        if mode == "plain":
            arm.ctx.eakv_load(slots, table, st)
        else:
            arm.ctx.eakv_load_layers(slots, table, layers_per_group, [ev.cuda_event for ev in evs], st)
        e1.record(st)
        torch.cuda.synchronize()
        out[mode + "_ms"] = e0.elapsed_time(e1)
        if mode == "layered":
            out["group_ready_ms"] = [e0.elapsed_time(ev) for ev in evs]
    out["layers_per_group"] = layers_per_group
    out["blocks"] = m
    return out


def layered_store_probe(torch, arm, tables, shape, layers_per_group=12):
    """Write 4,096 blocks to the pinned tier whole, and in layer groups behind per-group events of
    a producer (already complete here, so the figures are the write alone): the layered form
    costs nothing extra, and under a real producer its first groups run beneath the compute."""
    m = arm.m
    slots = np.arange(m, dtype=np.int32)
    table = tables[0][:m]
    st = torch.cuda.Stream(arm.device)
    groups = -(-shape.num_layers // layers_per_group)
    evs = [torch.cuda.Event() for _ in range(groups)]
    for ev in evs:
        ev.record(st)
    out = {}
    for mode in ("plain", "layered"):
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        if mode == "plain":
            arm.ctx.eakv_store(table, None, slots, st)
        else:
            arm.ctx.eakv_store_layers(table, None, slots, layers_per_group, [ev.cuda_event for ev in evs], st)
        e1.record(st)
        torch.cuda.synchronize()
        out[mode + "_ms"] = e0.elapsed_time(e1)
    out["layers_per_group"] = layers_per_group
    out["blocks"] = m
    return out


def store_load_curve(torch, eakv, pool, shape, device, args, h2d_peak, d2h_peak, tier_ptr=None,
                     tier_blocks=4096, reps=5):
    """The microbench's curve: 1 to 4,096 blocks per call, block ids contiguous or uniform-random
    over the pool (host slots alike), admit mask all-ones or Bernoulli(0.5); GB/s of the admitted
    bytes, median of ``reps`` calls timed with CUDA events on the launching stream.  Host tier
    under the default strategy (staged, scattered calls go direct) and a tier in HBM."""
    rng = np.random.default_rng(7)
    nb, kh = pool.gpu_blocks, int(min(4096, tier_blocks))
    rows = []
    tier_dev = torch.empty(kh * shape.block_bytes, dtype=torch.uint8, device=device)
    arms = [("host", dict(tier_location=eakv.TIER_PINNED_HOST, link_strategy=eakv.LINK_STAGED,
                          staging_bytes=args.staging_mib << 20,
                          **({"tier_memory": tier_ptr} if tier_ptr else {}))),
            ("hbm", dict(tier_location=eakv.TIER_DEVICE, tier_memory=tier_dev.data_ptr()))]
    stream = torch.cuda.current_stream(device)
    for name, kw in arms:
        ctx = eakv.Context(num_layers=shape.num_layers, kv_heads=shape.kv_heads, head_dim=shape.head_dim,
                           block_size=shape.block_size, gpu_blocks=nb, host_blocks=kh,
                           kv_base=pool.kv_base, **kw)
        for m in (1, 16, 256, 4096):
            if m > kh or m > nb:
                continue
            for ids in ("contiguous", "random"):
                for mask in ("ones", "bernoulli"):
                    for op in ("store", "load"):
                        if op == "load" and mask != "ones":
                            continue                      # a restore has no mask
                        rates = []
                        for i in range(reps + 1):
                            start = int(rng.integers(0, nb - m + 1))
                            table = (np.arange(start, start + m) if ids == "contiguous"
                                     else rng.permutation(nb)[:m]).astype(np.int32)
                            slots = (np.arange(m) if ids == "contiguous" else rng.permutation(kh)[:m]).astype(np.int32)
                            adm = None if mask == "ones" else (rng.random(m) < 0.5).astype(np.uint8)
                            nbytes = (m if adm is None else int(adm.sum())) * shape.block_bytes
                            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                            e0.record(stream)
                            if op == "store":
                                ctx.eakv_store(table, adm, slots, stream)
                            else:
                                ctx.eakv_load(slots, table, stream)
                            e1.record(stream)
                            torch.cuda.synchronize()
                            if nbytes and i > 0:          # the first call of a kind warms up
                                rates.append(nbytes / (e0.elapsed_time(e1) * 1e-3) / 1e9)
                        if rates:
                            row = dict(tier=name, op=op, blocks=m, ids=ids, mask=mask,
                                       gbps=round(float(np.median(rates)), 2))
                            if name == "host":
                                pk = d2h_peak if op == "store" else h2d_peak
                                row["frac_of_link"] = round(row["gbps"] / pk, 3) if pk else None
                            rows.append(row)
        ctx.close()
    return {"unit": "GB/s of admitted bytes, median of %d calls" % reps, "rows": rows}


def pinned_link_peak(torch, device, gib=1, reps=5):
    n = gib << 30
    host = torch.empty(n, dtype=torch.uint8).pin_memory()
    dev = torch.empty(n, dtype=torch.uint8, device=device)
    out = {}
    for name, (dst, src) in (("h2d", (dev, host)), ("d2h", (host, dev))):
        best = 0.0
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); dst.copy_(src, non_blocking=True); e1.record()
            torch.cuda.synchronize()
            best = max(best, n / (e0.elapsed_time(e1) * 1e-3) / 1e9)
        out[name] = best
    # both directions at once on two streams
    s1, s2 = torch.cuda.Stream(device), torch.cuda.Stream(device)
    host2 = torch.empty(n, dtype=torch.uint8).pin_memory()
    dev2 = torch.empty(n, dtype=torch.uint8, device=device)
    best = 0.0
    for _ in range(reps):
        torch.cuda.synchronize()
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        s1.wait_stream(torch.cuda.current_stream()); s2.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s1):
            dev.copy_(host, non_blocking=True)
        with torch.cuda.stream(s2):
            host2.copy_(dev2, non_blocking=True)
        torch.cuda.current_stream().wait_stream(s1); torch.cuda.current_stream().wait_stream(s2)
        t1.record()
        torch.cuda.synchronize()
        best = max(best, 2 * n / (t0.elapsed_time(t1) * 1e-3) / 1e9)
    out["bidir"] = best
    return out


# ------------------------------------------------------------------------------------------
# CPU oracle arm
# ------------------------------------------------------------------------------------------
def oracle_step_rate(seconds, blocks=128, pool_blocks=512, steps_cap=10**9):
    """The oracle, as it stands, on the same step with `blocks` blocks per request and a
    host-resident pool of `pool_blocks`; returns (GB/s, steps run, seconds)."""
    from eakv_workloads import SHAPES
    from oracle import hash as ohash, storeload
    from oracle.tier import HostTier
    shape = SHAPES["qwen3_30b_a3b"]
    rng = np.random.default_rng(1)
    b, P, Q = shape.block_size, shape.piece_bytes, shape.pieces_per_block
    pool = [rng.integers(0, 256, size=(pool_blocks, P), dtype=np.uint8) for _ in range(Q)]
    tier_mem = np.zeros((2 * blocks, Q, P), dtype=np.uint8)
    tier = HostTier(2 * blocks, b)
    prompts = {}

    def prompt(s):
        if s not in prompts:
            prompts[s] = rng.integers(0, 151936, size=blocks * b, dtype=np.int32)
        return prompts[s]

    def request(tokens, table, agent, now):
        keys = ohash.hash_blocks(tokens.tolist(), b)
        H = tier.leading_run(keys)
        slots = [tier.slot_of(k) for k in keys[:H]]
        res = tier.step(keys, len(tokens), agent, now)
        storeload.load(pool, tier_mem, slots, table[:H])
        storeload.store(pool, tier_mem, table, res.admit, res.slot)
        return (H + sum(res.admit)) * shape.block_bytes

    request(prompt(0), rng.permutation(pool_blocks)[:blocks], 0, 0)
    t0 = time.perf_counter()
    moved, s = 0, 0
    while True:
        s += 1
        moved += request(prompt(s - 1), rng.permutation(pool_blocks)[:blocks], (s - 1) % 2, s * 1000)
        moved += request(prompt(s), rng.permutation(pool_blocks)[:blocks], s % 2, s * 1000 + 500)
        prompts.pop(s - 1, None)
        dt = time.perf_counter() - t0
        if dt >= seconds or s >= steps_cap:
            break
    return moved / dt / 1e9, s, dt


def oracle_step_rate_c(seconds, blocks=128, pool_blocks=512, steps_cap=10**9):
    """The same step through the plain C oracle (oracle/eakv_oracle.c: Horner hash with 128-bit
    products, linear-scan LRU tier, per-piece memcpy), as it stands; (GB/s, steps, seconds)."""
    from eakv_workloads import SHAPES
    from oracle import c_oracle
    from oracle import hash as ohash
    shape = SHAPES["qwen3_30b_a3b"]
    rng = np.random.default_rng(1)
    b, P, Q = shape.block_size, shape.piece_bytes, shape.pieces_per_block
    pool = [rng.integers(0, 256, size=(pool_blocks, P), dtype=np.uint8) for _ in range(Q)]
    tier_mem = np.zeros((2 * blocks, Q, P), dtype=np.uint8)
    tier = c_oracle.Tier(2 * blocks, 0, 8)
    prompts = {}

    def prompt(s):
        if s not in prompts:
            prompts[s] = rng.integers(0, 151936, size=blocks * b, dtype=np.int32)
        return prompts[s]

    def request(tokens, table):
        keys = c_oracle.hash_blocks(tokens, b, ohash.HASH_SEED, ohash.HASH_BASE)
        H, slots = tier.leading_run(keys)
        _save, _hit, admit, slot = tier.step(keys)
        c_oracle.load(pool, tier_mem, slots, table[:H])
        c_oracle.store(pool, tier_mem, table, admit, slot)
        return (H + int(admit.sum())) * shape.block_bytes

    request(prompt(0), rng.permutation(pool_blocks)[:blocks].astype(np.int32))
    t0 = time.perf_counter()
    moved, s = 0, 0
    while True:
        s += 1
        moved += request(prompt(s - 1), rng.permutation(pool_blocks)[:blocks].astype(np.int32))
        moved += request(prompt(s), rng.permutation(pool_blocks)[:blocks].astype(np.int32))
        prompts.pop(s - 1, None)
        dt = time.perf_counter() - t0
        if dt >= seconds or s >= steps_cap:
            break
    tier.close()
    return moved / dt / 1e9, s, dt


def oracle_all_cores(seconds):
    """The same oracle step on every host core at once (one independent process per core, as it
    stands); returns (summed GB/s, processes) or None if the children could not be run."""
    n = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    code = f"import bench; print(bench.oracle_step_rate_c({float(seconds)!r})[0])"
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", OMP_NUM_THREADS="1")
    procs = [subprocess.Popen([sys.executable, "-c", code], cwd=ROOT, env=env, stdout=subprocess.PIPE,
                              stderr=subprocess.DEVNULL, text=True) for _ in range(n)]
    total = 0.0
    try:
        for p in procs:
            out, _ = p.communicate(timeout=seconds * 6 + 120)
            if p.returncode != 0:
                return None
            total += float(out.strip().splitlines()[-1])
    except (subprocess.TimeoutExpired, ValueError, IndexError):
        for p in procs:
            if p.poll() is None:
                p.kill()
        return None
    return total, n


def host_info(local_rank):
    """CPU model, core count and the NUMA node of this rank's GPU; binds the calling thread (which
    allocates the pinned tier) to that node's cores when the system exposes them."""
    info = {"cpu_count": os.cpu_count()}
    try:
        for ln in open("/proc/cpuinfo"):
            if ln.startswith("model name"):
                info["cpu_model"] = ln.split(":", 1)[1].strip()
                break
    except OSError:
        pass
    try:
        import torch
        bus = torch.cuda.get_device_properties(local_rank)
        pci = f"{bus.pci_domain_id:04x}:{bus.pci_bus_id:02x}:{bus.pci_device_id:02x}.0"
        node = int(open(f"/sys/bus/pci/devices/{pci}/numa_node").read())
        info["gpu_pci"] = pci
        info["gpu_numa_node"] = node
        if node >= 0:
            cpus = set()
            for part in open(f"/sys/devices/system/node/node{node}/cpulist").read().strip().split(","):
                lo, _, hi = part.partition("-")
                cpus.update(range(int(lo), int(hi or lo) + 1))
            allowed = cpus & os.sched_getaffinity(0)
            if allowed:
                os.sched_setaffinity(0, allowed)
                info["bound_to_numa_cpus"] = len(allowed)
    except (OSError, ValueError, AttributeError, RuntimeError) as e:
        info["numa"] = f"not available ({type(e).__name__})"
    return info


def oracle_component_rates():
    """The oracle's parts timed alone, as they stand: hashed tokens/s, tier references/s."""
    from oracle import hash as ohash
    from oracle.tier import HostTier
    rng = np.random.default_rng(2)
    toks = rng.integers(0, 151936, size=1 << 20, dtype=np.int32).tolist()
    t0 = time.perf_counter()
    keys = ohash.hash_blocks(toks, 16)
    t_hash = time.perf_counter() - t0
    tier = HostTier(3 * 4096, 16)
    t0 = time.perf_counter()
    refs = 0
    for i in range(40):
        k = keys[(i // 2) * 4096 % len(keys):][:4096]
        tier.step(k, len(k) * 16, i % 5, i)
        refs += len(k)
    t_tier = time.perf_counter() - t0
    # the whole of config 0 (96 requests, every byte held in numpy) through the trace oracle
    from eakv_workloads import CONFIGS, SHAPES, key_words_numpy, make_trace
    from oracle.trace import TraceOracle
    cfg = CONFIGS["c0"]
    trace = make_trace(cfg)
    t0 = time.perf_counter()
    TraceOracle(SHAPES[cfg.shape], cfg.gpu_blocks, cfg.host_blocks, payload=key_words_numpy).run(trace)
    t_c0 = time.perf_counter() - t0
    from oracle import c_oracle
    big = rng.integers(0, 151936, size=1 << 24, dtype=np.int32)
    t0 = time.perf_counter()
    c_oracle.hash_blocks(big, 16, ohash.HASH_SEED, ohash.HASH_BASE)
    t_chash = time.perf_counter() - t0
    return {"python_hash_tokens_per_s": len(toks) / t_hash, "python_tier_refs_per_s": refs / t_tier,
            "python_config0_trace_seconds": t_c0, "c_hash_tokens_per_s": len(big) / t_chash}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    blocks = 128
    # warm-up steps, then K timed steps of the bounded sample
    oracle_step_rate_c(0.0, blocks=blocks, steps_cap=max(1, min(args.warmup, 2)))
    gbps, steps, dt = oracle_step_rate_c(1e9, blocks=blocks, steps_cap=args.steps)
    line = {
        "impl": "reference", "metric": METRIC, "value": gbps, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8",
        "data": "synthetic", "gpu_launches": 0,
        "config": {"workload": WORKLOAD, "blocks_per_request": blocks,
                   "note": "plain C oracle on a bounded sample of the step (128 blocks per request)"},
        "cpu_baseline": {"value": gbps, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": f"{steps} steps x 2 requests x {blocks} blocks (1.5 MiB each)"},
        "e2e": {"value": gbps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------
def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus < 1:
        raise SystemExit("--gpus must be at least 1")

    import torch
    from paper_2609_33762_b200.multi import launched, spawn_local_ranks
    if args.gpus > 1 and not launched():
        # no launcher: start the N replicas here, one process per GPU; rank 0 prints the line
        have = torch.cuda.device_count() if torch.cuda.is_available() else 0
        if have < args.gpus:
            raise SystemExit(f"bench.py --gpus {args.gpus}: this machine has {have} CUDA device(s); "
                             "the eakv path has no CPU fallback")
        sys.exit(spawn_local_ranks([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], args.gpus))

    from eakv_workloads import SHAPES
    from paper_2609_33762_b200 import eakv
    from paper_2609_33762_b200.harness import PagedPool
    from paper_2609_33762_b200.multi import aggregate_over_ranks, init_distributed

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the eakv path has no CPU fallback")
    if not os.path.exists(os.path.join(ROOT, "paper_2609_33762_b200", "libeakv.so")):
        from paper_2609_33762_b200 import build
        build.build()
    eakv.lib()

    rank, world, local_rank, dist = init_distributed(args.gpus)
    device = torch.device(f"cuda:{local_rank}")
    torch.cuda.set_device(device)
    host = host_info(local_rank)      # also binds this thread to the GPU's NUMA node, if exposed
    shape = SHAPES["qwen3_30b_a3b"]
    workload = WORKLOAD
    if args.tp_shard > 1:
        shape = shape.tp_shard(args.tp_shard)
        workload = f"{WORKLOAD}_tp{args.tp_shard}_rank"
    m = args.blocks

    # paged pool, as large as fits (200k blocks = 293 GiB do not fit one GPU)
    free, _total = torch.cuda.mem_get_info(device)
    reserve = TIER_PROMPTS * m * shape.block_bytes + (4 << 30) + 2 * (args.staging_mib << 20) * 2
    nb = min(args.pool_blocks, int((free - reserve) // shape.block_bytes))
    nb = max(nb, 2 * m)
    pool = PagedPool(shape, nb, device, fill=lambda q, t: t.random_(), contiguous=True)
    torch.cuda.synchronize()

    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
    else:
        peak, peak_src = 6650.0, "fallback"
    if args.hash_only:
        print(json.dumps({"hash": hash_throughput(torch, eakv, pool, shape, device, peak,
                                                  prompts=args.hash_prompts)}))
        return

    total_steps = args.steps + args.warmup + LAG
    rng = np.random.default_rng(1 + rank)
    tok_np = rng.integers(0, 151936, size=(total_steps + 1, m * shape.block_size), dtype=np.int32)
    prompts_dev = [torch.from_numpy(tok_np[i]).to(device) for i in range(total_steps + 1)]
    prompts_host = [torch.from_numpy(tok_np[i]).pin_memory() for i in range(total_steps + 1)]
    # fresh uniform-random block ids per request, without replacement
    # uniform-random block ids without replacement: consecutive steps take disjoint windows of
    # one random permutation of the pool, so transfers of neighbouring steps never share a block
    perm = rng.permutation(nb).astype(np.int32)
    windows = nb // (2 * m)
    tables = [perm[(i % windows) * 2 * m:(i % windows + 1) * 2 * m] for i in range(total_steps + 1)]

    clocks = ClockSampler(local_rank) if rank == 0 else None

    # ---- device-resident arm (value) ----
    arm = Arm(args, pool, shape, torch, eakv, host_tier=False, device=device)
    r = run_arm(arm, prompts_dev, tables, args.steps, args.warmup, dist, clocks)
    check_ok = self_check(torch, arm, pool, tables, args, shape)
    arm.ctx.close()
    del arm
    ms_max, moved_sum = aggregate_over_ranks(dist, r["ms"], r["moved"], device)
    value = moved_sum / (ms_max * 1e-3) / 1e9

    def kernel_rate(res):
        kb = sum(b for b, _ in res["kernel"])
        kms = sum(t for _, t in res["kernel"])
        return 2 * kb / (kms * 1e-3) / 1e9 if kms > 0 else 0.0

    achieved = kernel_rate(r)
    kernel_name = "copy_blocks_vector_kernel" if args.copy_path == "vector" else "copy_blocks_bulk_kernel"
    by_copy_path = {args.copy_path: {"achieved": achieved, "frac": achieved / peak,
                                     "launches_timed": len(r["kernel"])}}
    if not args.quick:
        # the other device copy path on the same step (fewer steps), so both appear side by side
        other = "vector" if args.copy_path == "bulk" else "bulk"
        arm_o = Arm(args, pool, shape, torch, eakv, host_tier=False, device=device, copy_path=other)
        r_o = run_arm(arm_o, prompts_dev, tables, max(2, min(args.steps, 10)), min(args.warmup, 3), dist, None)
        arm_o.ctx.close()
        del arm_o
        by_copy_path[other] = {"achieved": kernel_rate(r_o), "frac": kernel_rate(r_o) / peak,
                               "launches_timed": len(r_o["kernel"])}
    # the profile's per-block DRAM traffic was captured on the unsharded shape
    traffic = read_profile_traffic(kernel_name, m) if args.tp_shard == 1 else None

    # The same step on one tensor-parallel rank's shape (Eq. 1: a rank of TP8 holds one KV head, so its
    # pieces are 4 KiB instead of 16 KiB; the paper states every size per rank): device tier, a pool
    # of its own (32,768 blocks), a few steps.  A side measurement of the single-GPU line only.
    tp8 = None
    if args.tp_shard == 1 and not args.quick and rank == 0 and dist is None:
        def tp8_section():
            sh8 = shape.tp_shard(8)
            nb8 = max(2 * m, min(32768, nb))
            pool8 = PagedPool(sh8, nb8, device, fill=lambda q, t: t.random_(), contiguous=True)
            perm8 = np.random.default_rng(5).permutation(nb8).astype(np.int32)
            w8 = nb8 // (2 * m)
            tables8 = [perm8[(i % w8) * 2 * m:(i % w8 + 1) * 2 * m] for i in range(total_steps + 1)]
            a8 = Arm(args, pool8, sh8, torch, eakv, host_tier=False, device=device)
            r8 = run_arm(a8, prompts_dev, tables8, max(2, min(args.steps, 10)), min(args.warmup, 3), None, None)
            a8.ctx.close()
            rate = kernel_rate(r8)
            return {"kv_heads": sh8.kv_heads, "piece_bytes": sh8.piece_bytes, "block_bytes": sh8.block_bytes,
                    "pool_blocks": nb8, "achieved": rate, "frac": rate / peak, "unit": "GB/s read+write",
                    "value_gbps": r8["moved"] / (r8["ms"] * 1e-3) / 1e9, "launches_timed": len(r8["kernel"])}
        try:
            tp8 = tp8_section()
        except Exception as exc:  # noqa: BLE001
            tp8 = {"error": f"{type(exc).__name__}: {exc}"}
        torch.cuda.empty_cache()

    # ---- end-to-end arm (pinned host tier, host tokens) ----
    def e2e_section():
        link = pinned_link_peak(torch, device) if rank == 0 else None
        # one pinned tier shared by every strategy's context (allocating 18 GiB of pinned memory
        # takes seconds; the contexts adopt it one after the other)
        try:
            tier_pin = torch.empty(TIER_PROMPTS * m * shape.block_bytes, dtype=torch.uint8, pin_memory=True)
            tier_ptr = tier_pin.data_ptr()
        except RuntimeError:
            tier_pin, tier_ptr = None, None
        arm = Arm(args, pool, shape, torch, eakv, host_tier=True, device=device, tier_memory=tier_ptr)
        e_steps = max(2, min(args.steps, 8))
        # measured twice on the same arm, the faster pass reported and both listed: the first
        # pass on a freshly started machine has been seen to run its two directions one after
        # the other (cold host side), which says nothing about the path
        passes = [run_arm(arm, prompts_host, tables, e_steps, min(args.warmup, 3), dist, None,
                          time_kernels=False) for _ in range(2)]
        pass_ms = [aggregate_over_ranks(dist, p_["ms"], p_["moved"], device) for p_ in passes]
        re_ = passes[0] if pass_ms[0][0] <= pass_ms[1][0] else passes[1]
        layered = layered_load_probe(torch, arm, tables, shape) if (rank == 0 and not args.quick) else None
        layered_st = layered_store_probe(torch, arm, tables, shape) if (rank == 0 and not args.quick) else None
        arm.ctx.close()
        del arm
        e_ms, e_moved = aggregate_over_ranks(dist, re_["ms"], re_["moved"], device)
        e_val = e_moved / (e_ms * 1e-3) / 1e9
        e2e = {"value": e_val, "unit": UNIT, "h2d_bytes_per_step": int(re_["h2d"]),
               "d2h_bytes_per_step": int(re_["d2h"]), "steps": e_steps,
               "ms_per_step": e_ms / e_steps, "link_strategy": args.link,
               "passes_gbps": [mv / (ms_ * 1e-3) / 1e9 for ms_, mv in pass_ms]}
        e2e["layered_load"] = layered
        e2e["layered_store"] = layered_st
        serial = bound = None
        if link:
            # one direction at a time: harmonic mean of the two; both at once: the measured
            # bidirectional pinned-memcpy rate
            serial = 2.0 / (1.0 / link["h2d"] + 1.0 / link["d2h"])
            bound = link["bidir"] if args.overlap else serial
            e2e.update(host_link_peak_gbps=link, overlap=bool(args.overlap),
                       frac_of_link=e_val / bound / max(world, 1),
                       frac_of_one_direction=e_val / serial / max(world, 1))
        # the same step under every host-link strategy, side by side (fewer steps each)
        by = {args.link: {"value": e_val, "frac_of_link": e2e.get("frac_of_link"), "steps": e_steps}}
        for name in ("staged", "zero_copy", "copy_engine"):
            if name in by or args.quick:
                continue
            a2 = Arm(args, pool, shape, torch, eakv, host_tier=True, device=device, link=name,
                     tier_memory=tier_ptr)
            r2 = run_arm(a2, prompts_host, tables, 3, 2, dist, None, time_kernels=False)
            a2.ctx.close()
            del a2
            ms2, mv2 = aggregate_over_ranks(dist, r2["ms"], r2["moved"], device)
            v2 = mv2 / (ms2 * 1e-3) / 1e9
            by[name] = {"value": v2, "frac_of_link": v2 / bound / max(world, 1) if bound else None, "steps": 3}
        e2e["by_strategy"] = by
        if rank == 0 and not args.quick:
            e2e["curve"] = guarded(store_load_curve, torch, eakv, pool, shape, device, args,
                                   link.get("h2d"), link.get("d2h"), tier_ptr, TIER_PROMPTS * m)
        del tier_pin
        return e2e

    # side measurements never take the main line down with them
    def guarded(fn, *a, **k):
        try:
            return fn(*a, **k)
        except Exception as exc:  # noqa: BLE001
            return {"error": f"{type(exc).__name__}: {exc}"}

    e2e = None
    if not args.no_e2e:
        # with one rank a failure here (say, no pinned memory left) must not lose the main line;
        # with several ranks the section holds collectives, so it runs unguarded
        e2e = guarded(e2e_section) if dist is None else e2e_section()
        if "error" in e2e:
            e2e.update(value=None, unit=UNIT)
    side = rank == 0 and not args.quick
    hashing = guarded(hash_throughput, torch, eakv, pool, shape, device, peak) if side else None
    control = guarded(control_plane_rate, eakv, pool, shape, device) if side else None

    cpu = None
    if rank == 0 and not args.no_cpu_baseline and not args.quick:
        g, s, dt = oracle_step_rate_c(args.cpu_seconds)
        cpu = {"value": g, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"plain C oracle: {s} steps x 2 requests x 128 blocks of 1.5 MiB in {dt:.1f} s"}
        py = guarded(oracle_step_rate, min(args.cpu_seconds, 4.0))
        cpu["python_oracle_value"] = py[0] if isinstance(py, tuple) else py
        cpu.update(guarded(oracle_component_rates))
        allc = guarded(oracle_all_cores, min(args.cpu_seconds, 6.0))
        cpu["all_cores"] = ({"value": allc[0], "unit": UNIT, "cores": allc[1],
                             "note": "one independent oracle process per core"}
                            if isinstance(allc, tuple) else allc)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_max / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
            "config": {"workload": workload, "blocks_per_request": m, "requests_per_step": 2,
                       "pool_blocks": nb, "block_bytes": shape.block_bytes,
                       "block_ids": "uniform-random without replacement", "admit_mask": "from tier step (all admitted)",
                       "l2": f"inputs larger than L2 ({4 * m * shape.block_bytes / 2**30:.1f} GiB moved per step)",
                       "tokens_hashed_per_step": 2 * m * shape.block_size,
                       "copy_path": args.copy_path, "self_check": check_ok},
            "clocks": r["clocks"],
            "e2e": e2e,
            "gpu_launches": r["launches"],
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "traffic": traffic, "peak_source": peak_src,
                         "kernel": kernel_name,
                         "launches_timed": len(r["kernel"]),
                         "by_copy_path": by_copy_path,
                         "tp8_rank_shape": tp8,
                         "frac_of_nominal_8TBs": achieved / 8000.0},
            "cpu_baseline": cpu,
            "hash": hashing,
            "control_plane": control,
            "host": host,
        }
        print(json.dumps(line))
        if args.sweep:
            sweep(args, torch, eakv, pool, shape, device)
    if dist is not None:
        dist.destroy_process_group()


def self_check(torch, arm, pool, tables, args, shape):
    """After the timed region: the last stored prompt's slots must equal its pool blocks."""
    s = args.warmup + args.steps + LAG - 1
    table = tables[s][args.blocks:]
    keys = arm.keys_host.numpy().view(np.uint64)         # keys of the last request
    _, H, _, slots = arm.ctx.eakv_match(keys)
    if H != len(keys):
        return False
    ok = True
    for j in np.linspace(0, len(keys) - 1, 16).astype(int):
        for q in (0, shape.pieces_per_block - 1):
            ok &= bool(torch.equal(arm.tier_t[int(slots[j]), q], pool.pieces[q][int(table[j])]))
    return bool(ok)


def read_profile_traffic(kernel, m):
    """DRAM bytes per launch of the copy kernel, scaled from the committed ncu summary of a
    smaller launch (traffic is proportional to blocks moved): the line
    `dram_bytes_per_block = <float>` in profiles/<kernel>.txt."""
    path = os.path.join(ROOT, "profiles", kernel + ".txt")
    try:
        for ln in open(path):
            if ln.startswith("dram_bytes_per_block"):
                return float(ln.split("=")[1]) * m
    except OSError:
        pass
    return None


def sweep(args, torch, eakv, pool, shape, device):
    """Store/load curve: 1..4096 blocks per call, contiguous vs random ids, mask all-ones vs
    Bernoulli(0.5), device tier vs host tier (both strategies)."""
    rng = np.random.default_rng(7)
    nb = pool.gpu_blocks
    kh = 4096
    rows = []
    arms = [("hbm", dict(tier_location=eakv.TIER_DEVICE)),
            ("host_zero_copy", dict(tier_location=eakv.TIER_PINNED_HOST, link_strategy=eakv.LINK_ZERO_COPY)),
            ("host_staged", dict(tier_location=eakv.TIER_PINNED_HOST, link_strategy=eakv.LINK_STAGED,
                                 staging_bytes=args.staging_mib << 20)),
            ("host_copy_engine", dict(tier_location=eakv.TIER_PINNED_HOST, link_strategy=eakv.LINK_COPY_ENGINE))]
    for name, kw in arms:
        ctx = eakv.Context(num_layers=shape.num_layers, kv_heads=shape.kv_heads, head_dim=shape.head_dim,
                           block_size=shape.block_size, gpu_blocks=nb, host_blocks=kh,
                           kv_base=pool.kv_base, **kw)
        stream = torch.cuda.current_stream(device)
        for m in (1, 2, 4, 8, 16, 32, 64, 128, 256, 512, 1024, 2048, 4096):
            for ids in ("contiguous", "random"):
                for mask in ("ones", "bernoulli"):
                    reps = 20 if m <= 256 else 5
                    for op in ("store", "load"):
                        if op == "load" and mask != "ones":
                            continue
                        times, nbytes = [], 0
                        for _ in range(reps):
                            start = int(rng.integers(0, nb - m + 1))
                            table = (np.arange(start, start + m) if ids == "contiguous"
                                     else rng.permutation(nb)[:m]).astype(np.int32)
                            slots = (np.arange(m) if ids == "contiguous" else rng.permutation(kh)[:m]).astype(np.int32)
                            adm = None if mask == "ones" else (rng.random(m) < 0.5).astype(np.uint8)
                            nbytes = (m if adm is None else int(adm.sum())) * shape.block_bytes
                            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                            e0.record(stream)
                            if op == "store":
                                ctx.eakv_store(table, adm, slots, stream)
                            else:
                                ctx.eakv_load(slots, table, stream)
                            e1.record(stream)
                            torch.cuda.synchronize()
                            if nbytes:
                                times.append(nbytes / (e0.elapsed_time(e1) * 1e-3) / 1e9)
                        if times:
                            rows.append(dict(arm=name, op=op, blocks=m, ids=ids, mask=mask,
                                             gbps_median=float(np.median(times)), gbps_best=float(max(times))))
        ctx.close()
    for row in rows:
        print(json.dumps({"sweep": row}), file=sys.stderr)
    from eakv_workloads import SHAPES
    shape_sweep(torch, eakv, SHAPES["qwen3_30b_a3b"], device)     # always from the unsharded shape


def shape_sweep(torch, eakv, shape, device, call_bytes=3 << 29):
    """Copy rate at tensor-parallel rank shapes (the paper states sizes per TP rank: a rank holds
    max(1, ceil(H_kv / TP)) heads, so pieces shrink with TP): 1.5 GiB per call between a device
    pool and a device tier, random block ids, both copy paths."""
    rng = np.random.default_rng(9)
    for tp in (1, 2, 8):
        sh = shape.tp_shard(tp)
        n = call_bytes // sh.block_bytes
        words = sh.piece_bytes // 2
        pieces = [torch.empty((2 * n, words), dtype=torch.int16, device=device) for _ in range(sh.pieces_per_block)]
        tier = torch.empty(n * sh.block_bytes, dtype=torch.uint8, device=device)
        for path, pname in ((eakv.COPY_BULK, "bulk"), (eakv.COPY_VECTOR, "vector")):
            ctx = eakv.Context(num_layers=sh.num_layers, kv_heads=sh.kv_heads, head_dim=sh.head_dim,
                               block_size=sh.block_size, gpu_blocks=2 * n, host_blocks=n,
                               kv_base=[t.data_ptr() for t in pieces], tier_location=eakv.TIER_DEVICE,
                               tier_memory=tier.data_ptr(), copy_path=path, max_call_blocks=n)
            table = rng.permutation(2 * n)[:n].astype(np.int32)
            slots = rng.permutation(n).astype(np.int32)
            stream = torch.cuda.current_stream(device)
            row = dict(tp=tp, kv_heads=sh.kv_heads, piece_bytes=sh.piece_bytes, blocks=int(n), path=pname)
            for op in ("store", "load"):
                ts = []
                for i in range(8):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                    if op == "store":
                        ctx.eakv_store(table, None, slots, stream)
                    else:
                        ctx.eakv_load(slots, table, stream)
                    e1.record(stream)
                    torch.cuda.synchronize()
                    if i >= 3:
                        ts.append(e0.elapsed_time(e1))
                row[op + "_gbps_read_plus_write"] = 2 * n * sh.block_bytes / (float(np.median(ts)) * 1e-3) / 1e9
            ctx.close()
            print(json.dumps({"shape_sweep": row}), file=sys.stderr)
        del pieces, tier


if __name__ == "__main__":
    main()
