"""Agent-turn driver over the eakv C-ABI.  PyTorch supplies device memory and streams
only; every step of the path (block keys, prefix match, tier bookkeeping, restore, store)
runs inside libeakv.  The "prefill" of a real serving engine is replaced by writing each
fresh block's synthetic payload into the paged pool.

One turn (the order follows the paper: lookup at scheduling time, restore before compute,
store after): hash -> match -> GPU tier step -> host tier step -> load blocks [G, H) ->
fill fresh blocks -> store admitted blocks.

By default the server drives the library's turn engine (eakv_turn_begin / eakv_turn_end, and
eakv_request_begin / _store / _release for requests that overlap): the whole turn, including
what to restore, what the engine must compute and what to store, is decided inside the
library.  ``native_turn=False`` drives the single calls (eakv_hash_blocks, eakv_match,
eakv_tier_step, eakv_gpu_tier_step, eakv_load, eakv_store) one by one instead; that path exists
to test those calls and to run bookkeeping-only replays, and is the only place where this module
combines their results itself.
"""
from __future__ import annotations

import numpy as np
import torch

from . import eakv


class PagedPool:
    """2L paged arrays [gpu_blocks, piece_bytes] as int16 tensors on one CUDA device.  With
    ``contiguous`` they are the slices of one [2L, gpu_blocks, piece] allocation, i.e. they sit
    at one constant pitch (what the copy-engine-only link strategy needs)."""

    def __init__(self, shape, gpu_blocks, device="cuda:0", fill=None, contiguous=False):
        self.shape = shape
        self.gpu_blocks = int(gpu_blocks)
        self.device = torch.device(device)
        W = shape.piece_bytes // 2
        self.words = W
        alloc = torch.zeros if fill is None else torch.empty
        if contiguous:
            self.whole = alloc((shape.pieces_per_block, self.gpu_blocks, W), dtype=torch.int16, device=self.device)
            self.pieces = [self.whole[q] for q in range(shape.pieces_per_block)]
        else:
            self.pieces = [alloc((self.gpu_blocks, W), dtype=torch.int16, device=self.device)
                           for _ in range(shape.pieces_per_block)]
        if fill is not None:
            for q, t in enumerate(self.pieces):
                fill(q, t)

    @property
    def kv_base(self):
        return [t.data_ptr() for t in self.pieces]


class AgentServer:
    def __init__(self, shape, gpu_blocks, host_blocks, payload, *, device="cuda:0",
                 gpu_index_blocks=0, incremental_hash=False, data_plane=True, chunk_blocks=1,
                 native_turn=None, store_layers=0, load_layers=0, **ctx_kwargs):
        """``payload(keys, q, n_words)`` returns the int16/uint16 words of piece q for the
        blocks with these keys, as a numpy array or a tensor on ``device``.  With
        ``chunk_blocks`` = R > 1 the host tier works in chunks of R blocks (``host_blocks``
        then counts chunks): one key per full chunk goes to the tier step, and chunk slot s
        maps to block slots s*R .. s*R+R-1 for store and load.  ``store_layers`` = g > 0 (turn
        engine, data plane): the "prefill" runs on a stream of its own, g layers at a time with an
        event after each group, and the host write follows it group by group
        (eakv_turn_end_layers / eakv_request_store_layers).  ``load_layers`` = g > 0: the restore
        runs in groups of g layers with one event per group (eakv_turn_begin_layers /
        eakv_request_begin_layers); ``last_restore_events`` holds the latest turn's events."""
        self.shape = shape
        self.store_layers = int(store_layers)
        self.load_layers = int(load_layers)
        self.last_restore_events = []
        self._fill_stream = None
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        # data_plane=False runs keys, matching and both tiers' bookkeeping only: no KV bytes move.
        # The bookkeeping then lives in a control-plane-only context (no tier memory, no staging),
        # which runs the library's turn engine from keys alone; a second, minimal context on the
        # device does nothing but hash.
        self.data_plane = data_plane
        self.pool = PagedPool(shape, gpu_blocks if data_plane else 1, device)
        common = dict(num_layers=shape.num_layers, kv_heads=shape.kv_heads, head_dim=shape.head_dim,
                      block_size=shape.block_size, elem_bytes=shape.elem_bytes)
        if data_plane:
            self.ctx = eakv.Context(gpu_blocks=gpu_blocks, host_blocks=host_blocks,
                                    gpu_index_blocks=gpu_index_blocks, kv_base=self.pool.kv_base,
                                    chunk_blocks=chunk_blocks, **common, **ctx_kwargs)
            self.hash_ctx = self.ctx
        else:
            self._no_tier = torch.zeros(16, dtype=torch.uint8, device=self.device)
            hash_kw = {k: ctx_kwargs[k] for k in ("hash_base", "hash_seed", "hash_scratch_blocks") if k in ctx_kwargs}
            self.hash_ctx = eakv.Context(gpu_blocks=1, host_blocks=1, kv_base=self.pool.kv_base,
                                         tier_memory=self._no_tier.data_ptr(), tier_location=eakv.TIER_DEVICE,
                                         **common, **hash_kw)
            book_kw = {k: v for k, v in ctx_kwargs.items()
                       if k not in ("tier_memory", "tier_location", "link_strategy", "copy_path", "copy_ctas",
                                    "staging_bytes", "hash_scratch_blocks", "write_behind")}
            self.ctx = eakv.Context(gpu_blocks=gpu_blocks, host_blocks=host_blocks,
                                    gpu_index_blocks=gpu_index_blocks, kv_base=None, control_plane_only=True,
                                    chunk_blocks=chunk_blocks, **common, **book_kw)
        self.payload = payload
        self.incremental = incremental_hash
        self.stream = torch.cuda.current_stream(self.device)
        self._ready = {}
        self.b = shape.block_size
        self.R = max(1, int(chunk_blocks))
        if native_turn is None:
            native_turn = True
        self.native_turn = native_turn     # drive turns through the library's turn engine
        self.seed = self.hash_ctx.eakv_hash_seed()
        self._agent_keys = {}          # agent -> np.uint64 keys of its previous prompt
        self._timed = {"load": [], "store": []}     # (bytes, start event, end event)
        self.records = []
        self.totals = dict(prompt_tokens=0, fresh_tokens=0, loaded_blocks=0, stored_blocks=0,
                           gpu_hit_blocks=0, host_hit_blocks=0)

    def close(self):
        self.ctx.close()
        if self.hash_ctx is not self.ctx:
            self.hash_ctx.close()

    def _time(self, kind, nbytes):
        """Context manager bracketing one store/load call with CUDA events on its stream."""
        server = self

        class _T:
            def __enter__(self_t):
                self_t.e0 = torch.cuda.Event(enable_timing=True)
                self_t.e1 = torch.cuda.Event(enable_timing=True)
                self_t.e0.record(server.stream)

            def __exit__(self_t, *exc):
                self_t.e1.record(server.stream)
                server._timed[kind].append((nbytes, self_t.e0, self_t.e1))
        return _T()

    def _timed_since(self, e0, kind, nbytes):
        """Close a timing bracket opened with event ``e0`` on the server's stream (turn engine: the
        restore is enqueued inside eakv_turn_begin, the store inside eakv_turn_end)."""
        if nbytes > 0:
            e1 = torch.cuda.Event(enable_timing=True)
            e1.record(self.stream)
            self._timed[kind].append((nbytes, e0, e1))

    def transfer_rates(self):
        """GB/s of the store and load calls so far (device time between the events that
        bracket each call); call after a synchronize."""
        out = {}
        for kind, items in self._timed.items():
            nbytes = sum(b for b, _, _ in items)
            ms = sum(e0.elapsed_time(e1) for _, e0, e1 in items)
            out[kind] = {"calls": len(items), "gib": nbytes / (1 << 30),
                         "gb_per_s": nbytes / (ms * 1e-3) / 1e9 if ms > 0 else None}
        return out

    def _ensure_pinned(self, n_tokens):
        if getattr(self, "_tok_pin", None) is None or self._tok_pin.numel() < n_tokens:
            cap = 1 << max(12, int(n_tokens - 1).bit_length())
            self._tok_pin = torch.empty(cap, dtype=torch.int32).pin_memory()
            self._keys_pin = torch.empty(cap // self.b + 1, dtype=torch.int64).pin_memory()

    # -- block keys -------------------------------------------------------------------------
    def block_keys(self, tokens: np.ndarray, agent) -> np.ndarray:
        n = len(tokens)
        nblk = n // self.b
        prev = self._agent_keys.get(agent) if self.incremental else None
        start = 0 if prev is None else min(len(prev), nblk)
        out = np.empty(nblk, dtype=np.uint64)
        if start:
            out[:start] = prev[:start]
        if nblk > start:
            # tokens are handed over in pinned host memory and keys come back into pinned host
            # memory: the hash kernel reads and writes both directly (they are mapped into
            # the device's address space), so a lookup never queues behind bulk KV copies
            seg_len = (nblk - start) * self.b
            self._ensure_pinned(seg_len)
            self._tok_pin.numpy()[:seg_len] = tokens[start * self.b: nblk * self.b]
            parent = int(out[start - 1]) if start else self.seed
            got = self.hash_ctx.eakv_hash_blocks(self._tok_pin.data_ptr(), seg_len, parent,
                                                 self._keys_pin.data_ptr(), self.stream)
            assert got == nblk - start
            self.stream.synchronize()
            out[start:] = self._keys_pin.numpy()[:got].view(np.uint64)
        if self.incremental:
            self._agent_keys[agent] = out
        return out

    # -- one request ------------------------------------------------------------------------
    def _turn_native(self, tokens, agent, now_ms):
        """The same turn through the library's two-call engine: lookup, bookkeeping and the
        restore happen inside eakv_turn_begin, the store inside eakv_turn_end."""
        n = len(tokens)
        if self.data_plane:
            self._ensure_pinned(max(n, 1))
            self._tok_pin.numpy()[:n] = tokens
            known = self._agent_keys.get(agent) if self.incremental else None
            e0 = torch.cuda.Event(enable_timing=True)
            e0.record(self.stream)
            v = self.ctx.eakv_turn_begin(self._tok_pin.data_ptr(), n, known, agent, now_ms, self.stream,
                                         layers=self._restore_layers())
            self._timed_since(e0, "load", (v["restore_hi"] - v["restore_lo"]) * self.ctx.block_bytes)
        else:       # bookkeeping only: the hashing context supplies every key
            v = self.ctx.eakv_turn_begin(0, n, self.block_keys(tokens, agent), agent, now_ms)
        keys, blocks = v["keys"], v["gpu_block"]
        if self.incremental and self.data_plane:
            self._agent_keys[agent] = keys
        ready = self._fill(keys, blocks, np.nonzero(v["needs_fill"])[0])
        if self.data_plane:
            e0 = torch.cuda.Event(enable_timing=True)
            e0.record(self.stream)
        if ready is None:
            self.ctx.eakv_turn_end(self.stream)
        else:
            self.ctx.eakv_turn_end_layers(self.store_layers, [ev.cuda_event for ev in ready], self.stream)
            self.stream.wait_stream(self._fill_stream)
        if self.data_plane:
            self._timed_since(e0, "store", v["n_stored_blocks"] * self.ctx.block_bytes)
        rec = self._record_from_view(v, agent, now_ms, n)
        G, H = rec["G"], rec["H"]
        return rec, G, H

    def begin(self, request_id, tokens, agent, now_ms, decided=None, defer_store=False):
        """A turn of a request that stays running: the same steps as ``turn`` up to and including
        the store, with the request's GPU blocks pinned under ``request_id`` until ``finish``
        (eakv_gpu_tier_acquire).  Returns None, with nothing changed, when the blocks do not fit
        beside the running requests.  ``decided``: None for the request's first lookup, else the
        store/skip choice made then (a resumed request: eakv_tier_step_again).  ``defer_store``
        (turn engine only): the host write waits for ``store(request_id)``, as in an engine that
        looks other requests up while this one computes."""
        tokens = np.asarray(tokens, dtype=np.int32)
        n = len(tokens)
        if self.native_turn:
            return self._begin_native(request_id, tokens, agent, now_ms, decided, defer_store)
        if defer_store:
            raise ValueError("defer_store needs the turn engine (native_turn)")
        keys = self.block_keys(tokens, agent)
        nblk = len(keys)
        R = self.R
        # lookups first (they change nothing), then the GPU side: if the blocks cannot be had,
        # neither tier may change
        if R == 1:
            G, H, _, host_slots = self.ctx.eakv_match(keys)
            unit_keys = keys
        else:
            G = self.ctx.eakv_match(keys)[0]
            unit_keys = np.ascontiguousarray(keys[R - 1::R])
            _, Hc, _, chunk_slots = self.ctx.eakv_match(unit_keys)
            H = Hc * R
            host_slots = (chunk_slots.astype(np.int64)[:, None] * R + np.arange(R)).reshape(-1).astype(np.int32)
        got = self.ctx.eakv_gpu_tier_acquire(request_id, keys, n % self.b != 0)
        if got is None:
            return None
        resident, blocks, tail = got
        step = self.ctx.eakv_tier_step(unit_keys, agent, n, now_ms, decided=decided)
        if R == 1:
            admit_b, slot_b = step["admit"], step["slot"]
        else:
            admit_b = np.zeros(nblk, dtype=np.uint8)
            slot_b = np.full(nblk, -1, dtype=np.int32)
            nc = len(unit_keys)
            admit_b[:nc * R] = np.repeat(step["admit"], R)
            base = np.repeat(step["slot"].astype(np.int64), R) * R + np.tile(np.arange(R), nc)
            slot_b[:nc * R] = np.where(np.repeat(step["slot"], R) >= 0, base, -1).astype(np.int32)
        cover = max(G, H)
        lo, hi = (G, H) if H > G else (G, G)
        if hi > lo and self.data_plane:
            with self._time("load", (hi - lo) * self.ctx.block_bytes):
                self.ctx.eakv_load(host_slots[lo:hi], blocks[lo:hi], self.stream)
        fill = [j for j in range(cover, nblk) if not resident[j]]
        if fill and self.data_plane:
            ids = torch.as_tensor(blocks[fill].astype(np.int64), device=self.device)
            fkeys = keys[fill]
            for q, piece in enumerate(self.pool.pieces):
                w = self.payload(fkeys, q, self.pool.words)
                if isinstance(w, np.ndarray):
                    w = torch.from_numpy(w.view(np.int16)).to(self.device)
                piece[ids] = w.view(torch.int16)
        if self.data_plane and admit_b.any():
            with self._time("store", int(admit_b.sum()) * self.ctx.block_bytes):
                self.ctx.eakv_store(blocks, admit_b, slot_b, self.stream)
        rec = dict(agent=agent, now_ms=now_ms, n_tokens=n, keys=keys, G=G, H=H,
                   new_chunks=step["new_chunks"], pressure=step["pressure"], save=step["save"],
                   hit=step["hit"], admit=step["admit"], slot=step["slot"],
                   evicted=list(zip(step["evicted_keys"].tolist(), step["evicted_slots"].tolist())),
                   gpu_resident=resident, gpu_block=blocks, loaded=hi - lo,
                   stored=int(admit_b.sum()), fresh_tokens=n - cover * self.b,
                   filled=len(fill), request_id=request_id, resumed=decided is not None, tail_block=tail)
        t = self.totals
        if decided is None:
            t["prompt_tokens"] += n
            t["fresh_tokens"] += rec["fresh_tokens"]
            t["gpu_hit_blocks"] += G
            t["host_hit_blocks"] += H
        else:
            t["preempt_recomputed_tokens"] = t.get("preempt_recomputed_tokens", 0) + rec["fresh_tokens"]
        t["loaded_blocks"] += rec["loaded"]
        t["stored_blocks"] += rec["stored"]
        self.records.append(rec)
        return rec

    def _restore_layers(self):
        """(layers per group, event handles) for a layered restore, or None."""
        if self.load_layers <= 0:
            return None
        groups = -(-self.shape.num_layers // self.load_layers)
        self.last_restore_events = [torch.cuda.Event() for _ in range(groups)]
        for ev in self.last_restore_events:
            ev.record(self.stream)                       # materialises the handle
        return self.load_layers, [ev.cuda_event for ev in self.last_restore_events]

    def store(self, request_id):
        """The deferred host write of ``begin(..., defer_store=True)`` (eakv_request_store)."""
        self._request_store(request_id, self._ready.pop(request_id, None))

    def _request_store(self, request_id, ready):
        if ready is None:
            self.ctx.eakv_request_store(request_id, self.stream if self.data_plane else None)
        else:
            self.ctx.eakv_request_store_layers(request_id, self.store_layers, [ev.cuda_event for ev in ready],
                                               self.stream)
            self.stream.wait_stream(self._fill_stream)

    def _begin_native(self, request_id, tokens, agent, now_ms, decided, defer_store=False):
        """The same through eakv_request_begin / eakv_request_store."""
        n = len(tokens)
        if self.data_plane:
            self._ensure_pinned(max(n, 1))
            self._tok_pin.numpy()[:n] = tokens
            known = self._agent_keys.get(agent) if self.incremental else None
            v = self.ctx.eakv_request_begin(request_id, self._tok_pin.data_ptr(), n, known, agent, now_ms,
                                            decided=decided, stream=self.stream, layers=self._restore_layers())
        else:
            v = self.ctx.eakv_request_begin(request_id, 0, n, self.block_keys(tokens, agent), agent, now_ms,
                                            decided=decided)
        if v is None:
            return None
        keys, blocks = v["keys"], v["gpu_block"]
        if self.incremental and self.data_plane:
            prev = self._agent_keys.get(agent)
            if prev is None or len(keys) >= len(prev):
                self._agent_keys[agent] = keys
        ready = self._fill(keys, blocks, np.nonzero(v["needs_fill"])[0])
        if defer_store:
            self._ready[request_id] = ready
        else:
            self._request_store(request_id, ready)
        rec = self._record_from_view(v, agent, now_ms, n)
        rec.update(request_id=request_id, resumed=decided is not None)
        t = self.totals
        if decided is None:
            t["prompt_tokens"] += n
            t["fresh_tokens"] += rec["fresh_tokens"]
            t["gpu_hit_blocks"] += rec["G"]
            t["host_hit_blocks"] += rec["H"]
        else:
            t["preempt_recomputed_tokens"] = t.get("preempt_recomputed_tokens", 0) + rec["fresh_tokens"]
        t["loaded_blocks"] += rec["loaded"]
        t["stored_blocks"] += rec["stored"]
        self.records.append(rec)
        return rec

    def _fill(self, keys, blocks, fill):
        """The engine's part: produce the KV of the blocks the library flagged (synthetic payload).
        With ``store_layers`` the layers are produced on a stream of their own, a group at a time,
        and the per-group events are returned for the layered host write."""
        layered = self.store_layers > 0 and self.data_plane and self.native_turn
        if not layered:
            if len(fill) and self.data_plane:
                ids = torch.as_tensor(blocks[fill].astype(np.int64), device=self.device)
                for q, piece in enumerate(self.pool.pieces):
                    w = self.payload(keys[fill], q, self.pool.words)
                    if isinstance(w, np.ndarray):
                        w = torch.from_numpy(w.view(np.int16)).to(self.device)
                    piece[ids] = w.view(torch.int16)
            return None
        if self._fill_stream is None:
            self._fill_stream = torch.cuda.Stream(self.device)
        g = self.store_layers
        groups = -(-self.shape.num_layers // g)
        events = [torch.cuda.Event() for _ in range(groups)]    # (the caller keeps them until the store is enqueued)
        ids = torch.as_tensor(blocks[fill].astype(np.int64), device=self.device) if len(fill) else None
        self._fill_stream.wait_stream(self.stream)      # the blocks may still be read by earlier work
        with torch.cuda.stream(self._fill_stream):
            for grp in range(groups):
                for q in range(2 * grp * g, min(2 * (grp + 1) * g, len(self.pool.pieces))):
                    if ids is not None:
                        w = self.payload(keys[fill], q, self.pool.words)
                        if isinstance(w, np.ndarray):
                            w = torch.from_numpy(w.view(np.int16)).to(self.device)
                        self.pool.pieces[q][ids] = w.view(torch.int16)
                events[grp].record(self._fill_stream)
        return events

    @staticmethod
    def _record_from_view(v, agent, now_ms, n):
        return dict(agent=agent, now_ms=now_ms, n_tokens=n, keys=v["keys"], G=v["gpu_prefix_blocks"],
                    H=v["host_prefix_blocks"], new_chunks=v["new_chunks"], pressure=bool(v["pressure"]),
                    save=bool(v["save"]), hit=v["hit"], admit=v["admit"], slot=v["slot"],
                    evicted=list(zip(v["evicted_keys"].tolist(), v["evicted_slots"].tolist())),
                    gpu_resident=v["gpu_resident"], gpu_block=v["gpu_block"],
                    loaded=v["restore_hi"] - v["restore_lo"], stored=v["n_stored_blocks"],
                    fresh_tokens=v["fresh_tokens"], filled=int(v["n_fill"]), tail_block=v["tail_block"])

    def finish(self, request_id):
        """The request finished, or the engine suspended it: its GPU blocks become evictable."""
        self._ready.pop(request_id, None)
        if self.native_turn:
            self.ctx.eakv_request_release(request_id)
        else:
            self.ctx.eakv_gpu_tier_release_request(request_id)

    def turn(self, tokens, agent, now_ms):
        tokens = np.asarray(tokens, dtype=np.int32)
        if self.native_turn:
            rec, G, H = self._turn_native(tokens, agent, now_ms)
            return self._account(rec, G, H)
        n = len(tokens)
        keys = self.block_keys(tokens, agent)
        nblk = len(keys)
        R = self.R
        if R == 1:
            G, H, _gids, host_slots = self.ctx.eakv_match(keys)
            step = self.ctx.eakv_tier_step(keys, agent, n, now_ms)
            admit_b, slot_b = step["admit"], step["slot"]
        else:
            # block keys locate the GPU prefix, chunk keys (the key at each full chunk's last
            # block) the host prefix; chunk decisions are then spread over their blocks
            G = self.ctx.eakv_match(keys)[0]
            chunk_keys = np.ascontiguousarray(keys[R - 1::R])
            _, Hc, _, chunk_slots = self.ctx.eakv_match(chunk_keys)
            H = Hc * R
            host_slots = (chunk_slots.astype(np.int64)[:, None] * R + np.arange(R)).reshape(-1).astype(np.int32)
            step = self.ctx.eakv_tier_step(chunk_keys, agent, n, now_ms)
            admit_b = np.zeros(nblk, dtype=np.uint8)
            slot_b = np.full(nblk, -1, dtype=np.int32)
            nc = len(chunk_keys)
            admit_b[:nc * R] = np.repeat(step["admit"], R)
            base = np.repeat(step["slot"].astype(np.int64), R) * R + np.tile(np.arange(R), nc)
            slot_b[:nc * R] = np.where(np.repeat(step["slot"], R) >= 0, base, -1).astype(np.int32)
        resident, blocks, tail = self.ctx.eakv_gpu_tier_step(keys, n % self.b != 0)
        cover = max(G, H)
        lo, hi = (G, H) if H > G else (G, G)
        if hi > lo and self.data_plane:
            with self._time("load", (hi - lo) * self.ctx.block_bytes):
                self.ctx.eakv_load(host_slots[lo:hi], blocks[lo:hi], self.stream)
        fill = [j for j in range(cover, nblk) if not resident[j]]
        if fill and self.data_plane:
            ids = torch.as_tensor(blocks[fill].astype(np.int64), device=self.device)
            fkeys = keys[fill]
            for q, piece in enumerate(self.pool.pieces):
                w = self.payload(fkeys, q, self.pool.words)
                if isinstance(w, np.ndarray):
                    w = torch.from_numpy(w.view(np.int16)).to(self.device)
                piece[ids] = w.view(torch.int16)
        if self.data_plane and admit_b.any():
            with self._time("store", int(admit_b.sum()) * self.ctx.block_bytes):
                self.ctx.eakv_store(blocks, admit_b, slot_b, self.stream)
        if tail >= 0:
            self.ctx.eakv_gpu_tier_release(tail)
        rec = dict(agent=agent, now_ms=now_ms, n_tokens=n, keys=keys, G=G, H=H,
                   new_chunks=step["new_chunks"], pressure=step["pressure"], save=step["save"],
                   hit=step["hit"], admit=step["admit"], slot=step["slot"],
                   evicted=list(zip(step["evicted_keys"].tolist(), step["evicted_slots"].tolist())),
                   gpu_resident=resident, gpu_block=blocks, loaded=hi - lo,
                   stored=int(admit_b.sum()), fresh_tokens=n - cover * self.b,
                   filled=len(fill))
        return self._account(rec, G, H)

    def _account(self, rec, G, H):
        t = self.totals
        t["prompt_tokens"] += rec["n_tokens"]
        t["fresh_tokens"] += rec["fresh_tokens"]
        t["loaded_blocks"] += rec["loaded"]
        t["stored_blocks"] += rec["stored"]
        t["gpu_hit_blocks"] += G
        t["host_hit_blocks"] += H
        self.records.append(rec)
        return rec

    def run(self, trace, limit=None):
        for i, req in enumerate(trace.requests):
            if limit is not None and i >= limit:
                break
            self.turn(trace.prompt(req), req.agent, req.time_ms)
        self.ctx.eakv_sync()
        return self.records
