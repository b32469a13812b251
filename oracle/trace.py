"""Whole-trace driver: what one agent turn does to the two tiers and to the KV bytes.

Per request (Section 4 and Appendix D for the order: lookup first, restore before
compute, store after): hash the prompt's full blocks; G / H = leading runs resident in
the GPU index / host tier; run the host-tier step (promotions, admission, insertions);
reference the same keys in the GPU tier (harness-owned LRU of K_G blocks, ascending
order, fresh blocks from a free stack, a partial tail takes a temporary block);
load the host-covered blocks [G, H) into their GPU blocks; "prefill" = fill every block
at or beyond max(G, H) that was not already GPU-resident with its payload; store the
admitted blocks to their host slots.

The GPU tier is never specified by the paper (it belongs to the serving engine); the
model above is this build's reading.  KV payloads are a function of (block key, piece).

Two granularities (Section 5.1 and Appendix A: 1,024-token host chunks over the engine's
16-token blocks; Appendix C: restoration is counted "after chunk and block alignment"):
with ``chunk_blocks`` = R > 1 the host tier's unit is a chunk of R consecutive blocks, keyed
by the prefix hash at the chunk's last token.  Only full chunks are looked up and stored;
host coverage is H_chunks * R blocks; the restore run is blocks [G, H_chunks * R); chunk
slot s occupies block slots s*R .. s*R + R - 1 of the tier.
"""
from collections import OrderedDict

import numpy as np

from . import hash as ohash
from . import storeload
from .tier import HostTier


class GpuTier:
    """LRU of keyed GPU blocks with a free stack that first yields 0, 1, 2, ...

    ``free_order``: how a finished request leaves its blocks in the recency order.  0: as
    referenced (the prompt's first block is the least recent of the request).  1: reversed,
    the way a paged engine returns a sequence's blocks tail first, so that the tail is
    evicted before the head and what survives of a sequence is still a prefix."""

    def __init__(self, num_blocks, free_order=0):
        self.NB = int(num_blocks)
        self.free_order = int(free_order)
        self.order = OrderedDict()                 # key -> block id, least recent first (evictable)
        self.free = list(range(self.NB - 1, -1, -1))
        self.pinned = {}                           # key -> [block id, holders]: out of the recency order
        self.held = {}                             # request id -> (keys in prompt order, tail block)

    def __contains__(self, key):
        return key in self.order or key in self.pinned

    def _alloc(self):
        if not self.free:
            _, vb = self.order.popitem(last=False)
            self.free.append(vb)
        return self.free.pop()

    def step(self, keys, need_tail):
        """Reference ``keys`` in order.  Returns (was_resident[], block_id[], tail_block)."""
        if len(keys) + int(need_tail) > self.NB:
            raise ValueError("request does not fit the GPU cache")
        resident, ids = [], []
        for k in keys:
            if k in self.order:
                self.order.move_to_end(k)
                resident.append(1)
                ids.append(self.order[k])
            else:
                blk = self._alloc()
                self.order[k] = blk
                resident.append(0)
                ids.append(blk)
        tail = self._alloc() if need_tail else -1
        if self.free_order == 1:
            for k in reversed(keys):
                self.order.move_to_end(k)
        return resident, ids, tail

    def release(self, block_id):
        if block_id >= 0:
            self.free.append(block_id)

    # ---- several requests at once: a running request's blocks cannot be evicted -------------
    # (Section 2: the engine runs several requests at once and suspends one if their KV no
    # longer fits on the GPU.)  A pinned block is out of the recency order; when its last holder lets go it
    # re-enters at the most-recent end.  acquire() followed at once by release_request() leaves
    # the tier exactly as step() does.
    def fits(self, keys, need_tail):
        """Can ``keys`` (+ a tail block) be acquired without touching a pinned block?  Every key
        whose block nobody holds yet takes one block out of the free and the evictable ones."""
        pinned = self.pinned
        cost = int(need_tail) + sum(1 for k in dict.fromkeys(keys) if k not in pinned)
        return cost <= len(self.free) + len(self.order)

    def acquire(self, request_id, keys, need_tail):
        """Reference ``keys`` in order and pin their blocks for ``request_id``.  Returns
        (was_resident[], block_id[], tail_block) or None, with nothing changed, if they do not fit."""
        pinned = self.pinned
        if request_id in self.held:
            raise ValueError("request already holds blocks")
        if not self.fits(keys, need_tail):
            return None
        resident, ids = [], []
        for k in keys:
            if k in pinned:                       # held by a running request (maybe this one)
                pinned[k][1] += 1
                resident.append(1)
                ids.append(pinned[k][0])
            elif k in self.order:
                blk = self.order.pop(k)
                pinned[k] = [blk, 1]
                resident.append(1)
                ids.append(blk)
            else:
                blk = self._alloc()
                pinned[k] = [blk, 1]
                resident.append(0)
                ids.append(blk)
        tail = self._alloc() if need_tail else -1
        self.held[request_id] = (list(keys), tail)
        return resident, ids, tail

    def release_request(self, request_id):
        """The request finished or was suspended: its blocks become evictable again, entering
        the recency order in prompt order (or tail first, see ``free_order``)."""
        keys, tail = self.held.pop(request_id)
        for k in (reversed(keys) if self.free_order == 1 else keys):
            ent = self.pinned[k]
            ent[1] -= 1
            if ent[1] == 0:
                del self.pinned[k]
                self.order[k] = ent[0]
        self.release(tail)


class TraceOracle:
    def __init__(self, shape, gpu_blocks, host_blocks, policy=0, kappa_blocks=8,
                 theta_percent=95, window_ms=60_000, len_window=256, telemetry=True,
                 payload=None, hash_base=ohash.HASH_BASE, hash_seed=ohash.HASH_SEED,
                 chunk_blocks=1, gpu_free_order=0, telemetry_period_ms=0, telemetry_max_age_ms=0):
        """``payload(keys, q, n_words) -> uint16[len(keys), n_words]`` enables full-bytes
        mode (pool and tier held in numpy); None runs metadata only."""
        self.shape = shape
        self.b = shape.block_size
        self.R = int(chunk_blocks)
        self.gpu = GpuTier(gpu_blocks, gpu_free_order)
        self.host = HostTier(host_blocks, self.b * self.R, policy, kappa_blocks, theta_percent,
                             window_ms, len_window, telemetry, telemetry_period_ms, telemetry_max_age_ms)
        self.payload = payload
        self.hash_base, self.hash_seed = hash_base, hash_seed
        self.pool = self.tier = None
        if payload is not None:
            P = shape.piece_bytes
            self.pool = [np.zeros((gpu_blocks, P), dtype=np.uint8)
                         for _ in range(shape.pieces_per_block)]
            self.tier = np.zeros((host_blocks * self.R, shape.pieces_per_block, P), dtype=np.uint8)
        self.records = []
        self.pending = {}        # unit key -> the open request that admitted it and has not written it yet
        self.open = {}           # request id -> what its deferred store still needs
        self.totals = dict(prompt_tokens=0, fresh_tokens=0, loaded_blocks=0, stored_blocks=0,
                           gpu_hit_blocks=0, host_hit_blocks=0)

    def turn(self, tokens, agent, now_ms, keys=None):
        """``keys``: the prompt's block keys if the caller already has them (prompts that only
        grow by appends share their prefix keys with the previous turn); else they are hashed."""
        n = len(tokens)
        if keys is None:
            keys = ohash.hash_blocks(tokens, self.b, self.hash_seed, self.hash_base)
        G = 0
        for k in keys:
            if k not in self.gpu:
                break
            G += 1
        R = self.R
        chunk_keys = keys[R - 1::R]                      # key at each full chunk's last block
        Hc = self.host.leading_run(chunk_keys)
        H = Hc * R
        # block slots of the host-covered prefix, chunk by chunk
        host_slots = [self.host.slot_of(k) * R + i for k in chunk_keys[:Hc] for i in range(R)]
        res = self.host.step(chunk_keys, n, agent, now_ms)
        resident, gpu_ids, tail = self.gpu.step(keys, n % self.b != 0)
        cover = max(G, H)
        lo, hi = (G, H) if H > G else (G, G)
        fill = [j for j in range(cover, len(keys)) if not resident[j]]
        # per-block view of the chunk decisions (blocks past the last full chunk: no host part)
        admit_b = [0] * len(keys)
        slot_b = [-1] * len(keys)
        for c, (a, s) in enumerate(zip(res.admit, res.slot)):
            for i in range(R):
                admit_b[c * R + i] = a
                slot_b[c * R + i] = s * R + i if s >= 0 else -1
        if self.payload is not None:
            storeload.load(self.pool, self.tier, host_slots[lo:hi], gpu_ids[lo:hi])
            if fill:
                W = self.shape.piece_bytes // 2
                for q in range(self.shape.pieces_per_block):
                    words = self.payload([keys[j] for j in fill], q, W)
                    for r, j in enumerate(fill):
                        self.pool[q][gpu_ids[j], :] = words[r].view(np.uint8)
            storeload.store(self.pool, self.tier, gpu_ids, admit_b, slot_b)
        self.gpu.release(tail)
        rec = dict(agent=agent, now_ms=now_ms, n_tokens=n, keys=keys, G=G, H=H,
                   new_chunks=res.new_chunks, pressure=res.pressure, save=res.save,
                   hit=res.hit, admit=res.admit, slot=res.slot, evicted=res.evicted,
                   gpu_resident=resident, gpu_block=gpu_ids, loaded=hi - lo,
                   stored=sum(admit_b), fresh_tokens=n - cover * self.b, filled=len(fill))
        t = self.totals
        t["prompt_tokens"] += n
        t["fresh_tokens"] += rec["fresh_tokens"]
        t["loaded_blocks"] += rec["loaded"]
        t["stored_blocks"] += rec["stored"]
        t["gpu_hit_blocks"] += G
        t["host_hit_blocks"] += H
        self.records.append(rec)
        return rec

    # ---- requests that overlap: begin pins the GPU blocks, finish lets them go ---------------
    def begin(self, request_id, tokens, agent, now_ms, keys=None, decided=None, defer_store=False):
        """The same turn as ``turn`` up to and including the store, with the request's GPU blocks
        pinned until ``finish``.  Returns None, with nothing changed, if the GPU tier cannot hold
        the request beside the running ones.  ``decided``: the save decision of the request's
        first lookup when this is a later one (a resumed request), else None.

        ``defer_store``: the host write happens later, at ``store(request_id)`` (an engine writes a
        request's KV once it has computed it, and other requests may be looked up in between).
        The bookkeeping is that of the reference model all the same, every write registered at its
        lookup; what changes is physical: a unit whose bytes are not there yet cannot be restored,
        so another request's host prefix ends before the first such unit, and a unit that a later
        lookup evicts before its bytes arrive is never written (its slot has a new owner)."""
        n = len(tokens)
        if keys is None:
            keys = ohash.hash_blocks(tokens, self.b, self.hash_seed, self.hash_base)
        need_tail = n % self.b != 0
        if not self.gpu.fits(keys, need_tail):
            return None
        G = 0
        for k in keys:
            if k not in self.gpu:
                break
            G += 1
        R = self.R
        chunk_keys = keys[R - 1::R]
        Hc = self.host.leading_run(chunk_keys)
        for c in range(Hc):
            if chunk_keys[c] in self.pending:          # listed, but its bytes have not been written yet
                Hc = c
                break
        H = Hc * R
        host_slots = [self.host.slot_of(k) * R + i for k in chunk_keys[:Hc] for i in range(R)]
        res = self.host.step(chunk_keys, n, agent, now_ms, decided=decided)
        for k, _ in res.evicted:
            self.pending.pop(k, None)                  # a pending write lost its slot
        resident, gpu_ids, tail = self.gpu.acquire(request_id, keys, need_tail)
        cover = max(G, H)
        lo, hi = (G, H) if H > G else (G, G)
        fill = [j for j in range(cover, len(keys)) if not resident[j]]
        admit_b = [0] * len(keys)
        slot_b = [-1] * len(keys)
        for c, (a, s) in enumerate(zip(res.admit, res.slot)):
            for i in range(R):
                admit_b[c * R + i] = a
                slot_b[c * R + i] = s * R + i if s >= 0 else -1
        if self.payload is not None:
            storeload.load(self.pool, self.tier, host_slots[lo:hi], gpu_ids[lo:hi])
            if fill:
                W = self.shape.piece_bytes // 2
                for q in range(self.shape.pieces_per_block):
                    words = self.payload([keys[j] for j in fill], q, W)
                    for r, j in enumerate(fill):
                        self.pool[q][gpu_ids[j], :] = words[r].view(np.uint8)
            if not defer_store:
                storeload.store(self.pool, self.tier, gpu_ids, admit_b, slot_b)
        if defer_store:
            for c, a in enumerate(res.admit):
                if a:
                    self.pending[chunk_keys[c]] = request_id
            self.open[request_id] = dict(chunk_keys=chunk_keys, admit=list(res.admit), gpu_ids=gpu_ids,
                                         admit_b=admit_b, slot_b=slot_b)
        rec = dict(agent=agent, now_ms=now_ms, n_tokens=n, keys=keys, G=G, H=H,
                   new_chunks=res.new_chunks, pressure=res.pressure, save=res.save,
                   hit=res.hit, admit=res.admit, slot=res.slot, evicted=res.evicted,
                   gpu_resident=resident, gpu_block=gpu_ids, loaded=hi - lo,
                   stored=sum(admit_b), fresh_tokens=n - cover * self.b, filled=len(fill),
                   request_id=request_id, resumed=decided is not None, tail_block=tail)
        t = self.totals
        if decided is None:
            t["prompt_tokens"] += n
            t["fresh_tokens"] += rec["fresh_tokens"]
            t["gpu_hit_blocks"] += G
            t["host_hit_blocks"] += H
        else:       # Appendix C: tokens recomputed after a preemption add to computed prefill (J)
            t["preempt_recomputed_tokens"] = t.get("preempt_recomputed_tokens", 0) + rec["fresh_tokens"]
        t["loaded_blocks"] += rec["loaded"]
        t["stored_blocks"] += rec["stored"]
        self.records.append(rec)
        return rec

    def store(self, request_id):
        """The deferred host write of ``begin(..., defer_store=True)``: the admitted units that are
        still this request's (no later lookup evicted them) are written; returns how many blocks."""
        o = self.open.pop(request_id)
        R = self.R
        admit_b = list(o["admit_b"])
        for c, a in enumerate(o["admit"]):
            if not a:
                continue
            if self.pending.get(o["chunk_keys"][c]) == request_id:
                del self.pending[o["chunk_keys"][c]]
            else:
                for i in range(R):
                    admit_b[c * R + i] = 0
        if self.payload is not None:
            storeload.store(self.pool, self.tier, o["gpu_ids"], admit_b, o["slot_b"])
        return sum(admit_b)

    def finish(self, request_id):
        """The request finished, or the engine suspended it: its blocks become evictable."""
        assert request_id not in self.open, "store first"
        self.gpu.release_request(request_id)

    def run(self, trace, limit=None):
        for i, req in enumerate(trace.requests):
            if limit is not None and i >= limit:
                break
            self.turn(trace.prompt(req), req.agent, req.time_ms)
        return self.records
