"""ctypes binding of libeakv.so: same names as the C entry points, argument marshalling
only.  Device buffers are passed as integer addresses (``tensor.data_ptr()``), host arrays
as numpy arrays; a negative status raises ``EakvError``.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

OK, E_INVAL, E_RANGE, E_CAPACITY, E_NOMEM, E_CUDA, E_TIMEOUT, E_BUSY = 0, -1, -2, -3, -4, -5, -6, -7
POLICY_WRITE_ALL, POLICY_FILTER_FIXED, POLICY_FILTER_CONDITIONED = 0, 1, 2
LINK_ZERO_COPY, LINK_STAGED, LINK_COPY_ENGINE = 0, 1, 2
TIER_PINNED_HOST, TIER_DEVICE = 0, 1
FREE_ASCENDING, FREE_REVERSE = 0, 1
COPY_VECTOR, COPY_BULK = 0, 1
HOST_COPY_VECTOR, HOST_COPY_BULK_LOAD, HOST_COPY_BULK_BOTH = 0, 1, 2

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libeakv.so")
_lib = None


class EakvError(RuntimeError):
    def __init__(self, code, where, detail=""):
        self.code = code
        msg = f"{where}: {lib().eakv_strerror(code).decode()} ({code})"
        if detail:
            msg += f": {detail}"
        super().__init__(msg)


class Config(C.Structure):
    _fields_ = [
        ("num_layers", C.c_int32), ("kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("block_size", C.c_int32), ("elem_bytes", C.c_int32),
        ("gpu_blocks", C.c_int64), ("host_blocks", C.c_int64), ("gpu_index_blocks", C.c_int64),
        ("kv_base", C.POINTER(C.c_void_p)),
        ("hash_base", C.c_uint64), ("hash_seed", C.c_uint64),
        ("policy", C.c_int32), ("kappa_blocks", C.c_int32), ("theta_percent", C.c_int32),
        ("len_window", C.c_int32), ("window_ms", C.c_int64), ("telemetry", C.c_int32),
        ("link_strategy", C.c_int32), ("tier_location", C.c_int32), ("copy_path", C.c_int32),
        ("copy_ctas", C.c_int32),
        ("staging_bytes", C.c_int64), ("max_call_blocks", C.c_int64),
        ("hash_scratch_blocks", C.c_int64), ("min_staged_run_bytes", C.c_int64),
        ("control_plane_only", C.c_int32), ("chunk_blocks", C.c_int32),
        ("tier_memory", C.c_void_p),
        ("gpu_free_order", C.c_int32), ("write_behind", C.c_int32),
        ("telemetry_period_ms", C.c_int64), ("telemetry_max_age_ms", C.c_int64),
        ("host_copy_path", C.c_int32), ("host_load_ctas", C.c_int32), ("host_store_ctas", C.c_int32),
        ("reserved0", C.c_int32),
    ]


class Stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in (
        "requests", "references", "hits", "admitted", "declined", "evicted",
        "declined_requests", "pressure_requests", "resident",
        "tokens_hashed", "blocks_stored", "blocks_loaded", "bytes_stored", "bytes_loaded",
        "kernel_launches", "memcpy_calls")]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class StepInfo(C.Structure):
    _fields_ = [("host_prefix_blocks", C.c_int64), ("new_chunks", C.c_int64),
                ("pressure", C.c_int32), ("save", C.c_int32)]


class OffloadIn(C.Structure):
    _fields_ = [("prefix_tokens", C.c_int64), ("beta_rank_bytes", C.c_int64), ("t_prefill_ps", C.c_int64),
                ("h2d_bytes_per_s", C.c_int64), ("tau_load_ps", C.c_int64)]


class OffloadOut(C.Structure):
    _fields_ = [("t_load_ps", C.c_int64), ("t_rec_ps", C.c_int64), ("break_even_tokens", C.c_int64),
                ("obr", C.c_double), ("obr_long_prefix", C.c_double), ("restore_is_faster", C.c_int32),
                ("reserved", C.c_int32)]


class WorkingSetIn(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("num_layers", "kv_heads", "head_dim", "elem_bytes", "tensor_parallel",
                                         "block_size")] + \
               [(n, C.c_int64) for n in ("active_pool", "total_prompt_tokens", "n_requests", "gpu_blocks",
                                         "host_blocks")]


class WorkingSetOut(C.Structure):
    _fields_ = [("beta_rank_bytes", C.c_int64), ("working_set_bytes", C.c_int64),
                ("working_set_blocks", C.c_int64), ("gamma_g", C.c_double), ("gamma_h", C.c_double),
                ("pool_exceeds_gpu", C.c_int32), ("working_set_exceeds_host", C.c_int32)]


class TurnView(C.Structure):
    _fields_ = [(n, C.c_int64) for n in (
        "n_blocks", "n_units", "gpu_prefix_blocks", "host_prefix_blocks", "restore_lo", "restore_hi",
        "fresh_tokens", "new_chunks", "n_fill", "n_stored_blocks", "n_evicted")] + [
        ("pressure", C.c_int32), ("save", C.c_int32), ("tail_block", C.c_int32), ("reserved", C.c_int32),
        ("keys", C.c_void_p), ("gpu_block", C.c_void_p), ("gpu_resident", C.c_void_p),
        ("needs_fill", C.c_void_p), ("hit", C.c_void_p), ("admit", C.c_void_p), ("slot", C.c_void_p),
        ("evicted_keys", C.c_void_p), ("evicted_slots", C.c_void_p)]


def _view_array(ptr, n, dtype):
    """Copy n items of a context-owned host array (valid until the next turn) into numpy."""
    if n <= 0 or not ptr:
        return np.zeros(0, dtype=dtype)
    nbytes = n * np.dtype(dtype).itemsize
    buf = (C.c_uint8 * nbytes).from_address(ptr)
    return np.frombuffer(buf, dtype=dtype).copy()


EXPORTS = [
    "eakv_config_init", "eakv_create", "eakv_destroy", "eakv_hash_blocks",
    "eakv_hash_blocks_batched", "eakv_match", "eakv_tier_step", "eakv_gpu_tier_step",
    "eakv_gpu_tier_release", "eakv_store", "eakv_load", "eakv_sync", "eakv_get_stats",
    "eakv_tier_ptr", "eakv_hash_seed", "eakv_hash_base", "eakv_strerror", "eakv_last_cuda_error",
    "eakv_hash_blocks_static", "eakv_hash_blocks_static_status", "eakv_load_layers", "eakv_reuse_distances", "eakv_capacity_curve",
    "eakv_turn_begin", "eakv_turn_end", "eakv_turn_abort", "eakv_tier_export", "eakv_tier_import",
    "eakv_admission_export", "eakv_admission_import",
    "eakv_selfcheck_limits", "eakv_selfcheck_wait_probe",
    "eakv_gpu_tier_acquire", "eakv_gpu_tier_release_request", "eakv_tier_step_again",
    "eakv_declined_audit", "eakv_working_set",
    "eakv_request_begin", "eakv_request_store", "eakv_request_release", "eakv_working_set_sizes", "eakv_selfcheck_fail_next_transfer", "eakv_store_layers", "eakv_turn_end_layers", "eakv_request_store_layers",
    "eakv_turn_begin_layers", "eakv_request_begin_layers", "eakv_offload_benefit",
]
STATIC_MAX_BLOCKS = 65536


def lib():
    """Load libeakv.so (once).  Raises if it has not been built: there is no fallback."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2609_33762_b200.build` "
            "(the eakv path has no CPU or PyTorch fallback)")
    L = C.CDLL(_LIB_PATH)
    vp, i32, i64, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64
    L.eakv_config_init.argtypes = [C.POINTER(Config)]
    L.eakv_create.argtypes = [C.POINTER(Config), C.POINTER(vp)]
    L.eakv_destroy.argtypes = [vp]
    L.eakv_hash_blocks.argtypes = [vp, vp, i64, u64, vp, C.POINTER(i64), vp]
    L.eakv_hash_blocks_static.argtypes = [vp, i64, i32, u64, u64, vp, C.POINTER(i64), vp]
    L.eakv_hash_blocks_static_status.argtypes = [vp]
    L.eakv_hash_blocks_batched.argtypes = [vp, vp, vp, i64, vp, vp, vp, vp]
    L.eakv_match.argtypes = [vp, vp, i64, C.POINTER(i64), C.POINTER(i64), vp, vp]
    L.eakv_tier_step.argtypes = [vp, vp, i64, i64, i64, i64, vp, vp, vp, vp, vp,
                                 C.POINTER(i64), C.POINTER(StepInfo)]
    L.eakv_gpu_tier_step.argtypes = [vp, vp, i64, i32, vp, vp, C.POINTER(i32)]
    L.eakv_gpu_tier_release.argtypes = [vp, i32]
    L.eakv_gpu_tier_acquire.argtypes = [vp, i64, vp, i64, i32, vp, vp, C.POINTER(i32)]
    L.eakv_gpu_tier_release_request.argtypes = [vp, i64]
    L.eakv_tier_step_again.argtypes = [vp, vp, i64, i64, i64, i32, vp, vp, vp, vp, vp,
                                       C.POINTER(i64), C.POINTER(StepInfo)]
    L.eakv_store.argtypes = [vp, vp, vp, vp, i64, vp]
    L.eakv_load.argtypes = [vp, vp, vp, i64, vp]
    L.eakv_load_layers.argtypes = [vp, vp, vp, i64, i32, vp, i32, vp]
    L.eakv_reuse_distances.argtypes = [vp, i64, vp, vp]
    L.eakv_capacity_curve.argtypes = [vp, i64, vp, vp, vp, i64, i32, vp, i32, vp, vp, vp, vp, vp]
    L.eakv_declined_audit.argtypes = [vp, vp, i64, i64, C.POINTER(i64), C.POINTER(i64), C.POINTER(i64), vp, vp]
    L.eakv_selfcheck_fail_next_transfer.argtypes = [vp, i32]
    L.eakv_store_layers.argtypes = [vp, vp, vp, vp, i64, i32, vp, i32, vp]
    L.eakv_turn_end_layers.argtypes = [vp, i32, vp, i32, vp]
    L.eakv_turn_begin_layers.argtypes = [vp, vp, i64, vp, i64, i64, i64, i32, vp, i32, vp, vp]
    L.eakv_request_begin_layers.argtypes = [vp, i64, vp, i64, vp, i64, i64, i64, i32, i32, vp, i32, vp, vp]
    L.eakv_request_store_layers.argtypes = [vp, i64, i32, vp, i32, vp]
    L.eakv_offload_benefit.argtypes = [C.POINTER(OffloadIn), C.POINTER(OffloadOut)]
    L.eakv_working_set_sizes.argtypes = [vp, i64, vp, vp, vp, i64, i32, i32, C.POINTER(i64), C.POINTER(i64), vp]
    L.eakv_working_set.argtypes = [C.POINTER(WorkingSetIn), C.POINTER(WorkingSetOut)]
    L.eakv_turn_begin.argtypes = [vp, vp, i64, vp, i64, i64, i64, vp, C.POINTER(TurnView)]
    L.eakv_turn_end.argtypes = [vp, vp]
    L.eakv_turn_abort.argtypes = [vp]
    L.eakv_request_begin.argtypes = [vp, i64, vp, i64, vp, i64, i64, i64, i32, vp, C.POINTER(TurnView)]
    L.eakv_request_store.argtypes = [vp, i64, vp]
    L.eakv_request_release.argtypes = [vp, i64]
    L.eakv_tier_export.argtypes = [vp, vp, vp, i64, C.POINTER(i64)]
    L.eakv_tier_import.argtypes = [vp, vp, vp, i64]
    L.eakv_admission_export.argtypes = [vp, vp, i64, C.POINTER(i64)]
    L.eakv_admission_import.argtypes = [vp, vp, i64]
    L.eakv_sync.argtypes = [vp]
    L.eakv_selfcheck_limits.argtypes = [vp, i64, i64, i64]
    L.eakv_selfcheck_wait_probe.argtypes = [vp, vp]
    L.eakv_get_stats.argtypes = [vp, C.POINTER(Stats)]
    L.eakv_tier_ptr.argtypes = [vp]
    L.eakv_tier_ptr.restype = vp
    L.eakv_hash_seed.argtypes = [vp]
    L.eakv_hash_seed.restype = u64
    L.eakv_hash_base.argtypes = [vp]
    L.eakv_hash_base.restype = u64
    L.eakv_strerror.argtypes = [C.c_int]
    L.eakv_strerror.restype = C.c_char_p
    L.eakv_last_cuda_error.argtypes = [vp]
    L.eakv_last_cuda_error.restype = C.c_char_p
    _lib = L
    return L


def _np(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a, a.ctypes.data


def _stream(s):
    if s is None:
        return None
    return C.c_void_p(int(getattr(s, "cuda_stream", s)))


def eakv_hash_blocks_static(tokens_dev, n_tokens, block_size, hash_base, parent_hash,
                            hashes_dev, stream=None):
    """Context-free, allocation-free block keys (scratch lives inside the library; at most
    STATIC_MAX_BLOCKS keys per call; calls on one device must not overlap on the GPU)."""
    n = C.c_int64(0)
    rc = lib().eakv_hash_blocks_static(C.c_void_p(int(tokens_dev)), int(n_tokens), int(block_size),
                                       C.c_uint64(int(hash_base)), C.c_uint64(int(parent_hash)),
                                       C.c_void_p(int(hashes_dev)), C.byref(n), _stream(stream))
    if rc != OK:
        raise EakvError(rc, "eakv_hash_blocks_static")
    return n.value


def eakv_hash_blocks_static_status(stream=None):
    """Raise EakvError(E_RANGE) if a self-check of the allocation-free hash tripped since the
    last query (the word is cleared by the query); waits for ``stream``."""
    rc = lib().eakv_hash_blocks_static_status(_stream(stream))
    if rc != OK:
        raise EakvError(rc, "eakv_hash_blocks_static_status")


def eakv_reuse_distances(keys_dev, n_refs, dist_dev, stream=None):
    """Reuse distances of the uint64 keys at device address ``keys_dev`` into int64 ``dist_dev``
    (-1 = first reference)."""
    rc = lib().eakv_reuse_distances(C.c_void_p(int(keys_dev)), int(n_refs), C.c_void_p(int(dist_dev)),
                                    _stream(stream))
    if rc != OK:
        raise EakvError(rc, "eakv_reuse_distances")


def eakv_declined_audit(keys_dev, declined_dev, n_refs, capacity, next_dist_dev=0, stream=None):
    """(declined, meets, never) of the declined references at device address ``declined_dev`` (uint8)."""
    d, m, nv = C.c_int64(0), C.c_int64(0), C.c_int64(0)
    rc = lib().eakv_declined_audit(C.c_void_p(int(keys_dev)), C.c_void_p(int(declined_dev)), int(n_refs),
                                   int(capacity), C.byref(d), C.byref(m), C.byref(nv),
                                   C.c_void_p(int(next_dist_dev)) if next_dist_dev else None, _stream(stream))
    if rc != OK:
        raise EakvError(rc, "eakv_declined_audit")
    return d.value, m.value, nv.value


def eakv_offload_benefit(*, prefix_tokens, beta_rank_bytes, t_prefill_ps, h2d_bytes_per_s, tau_load_ps=0):
    """Eq. 2: restore time, recompute time (picoseconds), OBR(n), its long-prefix limit and the
    break-even prefix length."""
    i = OffloadIn(int(prefix_tokens), int(beta_rank_bytes), int(t_prefill_ps), int(h2d_bytes_per_s), int(tau_load_ps))
    o = OffloadOut()
    rc = lib().eakv_offload_benefit(C.byref(i), C.byref(o))
    if rc != OK:
        raise EakvError(rc, "eakv_offload_benefit")
    return {f: getattr(o, f) for f, _ in OffloadOut._fields_ if f != "reserved"}


def eakv_working_set_sizes(dist_dev, n_refs, req_offsets, req_tokens, req_gpu_prefix, block_size, percent=1,
                           stream=None):
    """(full, within): smallest tier that hits every re-reference, and smallest tier whose predicted
    computed prefill is within ``percent`` % of the unbounded tier's."""
    off, offp = _np(req_offsets, np.int64)
    tok, tokp = _np(req_tokens, np.int64)
    gpu, gpup = _np(req_gpu_prefix, np.int64)
    full, within = C.c_int64(0), C.c_int64(0)
    rc = lib().eakv_working_set_sizes(C.c_void_p(int(dist_dev)), int(n_refs), offp, tokp, gpup, len(off) - 1,
                                      int(block_size), int(percent), C.byref(full), C.byref(within),
                                      _stream(stream))
    if rc != OK:
        raise EakvError(rc, "eakv_working_set_sizes")
    return full.value, within.value


def eakv_working_set(*, num_layers, kv_heads, head_dim, block_size, active_pool, total_prompt_tokens,
                     n_requests, gpu_blocks=0, host_blocks=0, elem_bytes=2, tensor_parallel=1):
    """Eq. 1, Eq. 5 and the pressure ratios of Section 3.2 as a dict (integer arithmetic in the library)."""
    i = WorkingSetIn(num_layers, kv_heads, head_dim, elem_bytes, tensor_parallel, block_size, active_pool,
                     total_prompt_tokens, n_requests, gpu_blocks, host_blocks)
    o = WorkingSetOut()
    rc = lib().eakv_working_set(C.byref(i), C.byref(o))
    if rc != OK:
        raise EakvError(rc, "eakv_working_set")
    return {n: getattr(o, n) for n, _ in WorkingSetOut._fields_}


def eakv_capacity_curve(dist_dev, n_refs, req_offsets, req_tokens, req_gpu_prefix, block_size,
                        capacities, want_cover=False, stream=None):
    """Hits, restored blocks and computed tokens per capacity (and H_j per request if asked)."""
    off, offp = _np(req_offsets, np.int64)
    tok, tokp = _np(req_tokens, np.int64)
    gpu, gpup = _np(req_gpu_prefix, np.int64)
    caps, capsp = _np(capacities, np.int64)
    J, Cn = len(off) - 1, len(caps)
    hits = np.zeros(Cn, dtype=np.int64)
    restored = np.zeros(Cn, dtype=np.int64)
    computed = np.zeros(Cn, dtype=np.int64)
    cover = np.zeros((Cn, J), dtype=np.int64) if want_cover else None
    vp = lambda a: a.ctypes.data
    rc = lib().eakv_capacity_curve(C.c_void_p(int(dist_dev)), int(n_refs), offp, tokp, gpup, J,
                                   int(block_size), capsp, Cn, vp(hits), vp(restored), vp(computed),
                                   vp(cover) if want_cover else None, _stream(stream))
    if rc != OK:
        raise EakvError(rc, "eakv_capacity_curve")
    return dict(hits=hits, restored_blocks=restored, computed_tokens=computed, cover=cover)


class Context:
    """Owns one eakv_ctx.  Method names mirror the C entry points."""

    def __init__(self, *, num_layers, kv_heads, head_dim, block_size, gpu_blocks, host_blocks,
                 kv_base, elem_bytes=2, gpu_index_blocks=0, hash_base=0, hash_seed=0,
                 policy=POLICY_WRITE_ALL, kappa_blocks=8, theta_percent=95, len_window=256,
                 window_ms=60_000, telemetry=1, link_strategy=LINK_STAGED,
                 tier_location=TIER_PINNED_HOST, copy_path=COPY_BULK, copy_ctas=0,
                 staging_bytes=0, max_call_blocks=0, hash_scratch_blocks=0, min_staged_run_bytes=0,
                 tier_memory=0, control_plane_only=False, chunk_blocks=1,
                 gpu_free_order=FREE_ASCENDING, write_behind=False, telemetry_period_ms=0,
                 telemetry_max_age_ms=0, host_copy_path=HOST_COPY_BULK_LOAD, host_load_ctas=0, host_store_ctas=0):
        L = lib()
        cfg = Config()
        L.eakv_config_init(C.byref(cfg))
        kv_base = list(kv_base) if kv_base is not None else []
        if not control_plane_only and len(kv_base) != 2 * num_layers:
            raise ValueError("kv_base must hold 2 * num_layers device pointers")
        ptrs = (C.c_void_p * max(len(kv_base), 1))(*[int(p) for p in kv_base])
        cfg.num_layers, cfg.kv_heads, cfg.head_dim = num_layers, kv_heads, head_dim
        cfg.block_size, cfg.elem_bytes = block_size, elem_bytes
        cfg.gpu_blocks, cfg.host_blocks, cfg.gpu_index_blocks = gpu_blocks, host_blocks, gpu_index_blocks
        cfg.kv_base = C.cast(ptrs, C.POINTER(C.c_void_p)) if kv_base else None
        cfg.control_plane_only = int(bool(control_plane_only))
        cfg.chunk_blocks = int(chunk_blocks)
        cfg.gpu_free_order = int(gpu_free_order)
        cfg.write_behind = int(bool(write_behind))
        cfg.telemetry_period_ms, cfg.telemetry_max_age_ms = int(telemetry_period_ms), int(telemetry_max_age_ms)
        cfg.host_copy_path = int(host_copy_path)
        cfg.host_load_ctas, cfg.host_store_ctas = int(host_load_ctas), int(host_store_ctas)
        cfg.hash_base, cfg.hash_seed = hash_base, hash_seed
        cfg.policy, cfg.kappa_blocks, cfg.theta_percent = policy, kappa_blocks, theta_percent
        cfg.len_window, cfg.window_ms, cfg.telemetry = len_window, window_ms, telemetry
        cfg.link_strategy, cfg.tier_location = link_strategy, tier_location
        cfg.copy_path, cfg.copy_ctas = copy_path, copy_ctas
        cfg.staging_bytes, cfg.max_call_blocks = staging_bytes, max_call_blocks
        cfg.hash_scratch_blocks = hash_scratch_blocks
        cfg.min_staged_run_bytes = min_staged_run_bytes
        cfg.tier_memory = int(tier_memory) if tier_memory else None
        self._h = C.c_void_p()
        rc = L.eakv_create(C.byref(cfg), C.byref(self._h))
        if rc != OK:
            self._h = None
            raise EakvError(rc, "eakv_create")
        self.block_size = block_size
        self.host_blocks = host_blocks
        self.chunk_blocks = max(1, int(chunk_blocks))
        self.tier_slots = host_blocks * self.chunk_blocks
        self.piece_bytes = block_size * kv_heads * head_dim * elem_bytes
        self.block_bytes = 2 * num_layers * self.piece_bytes
        self.tier_location = tier_location

    # -- lifetime ---------------------------------------------------------------------------
    def eakv_destroy(self):
        if self._h:
            lib().eakv_destroy(self._h)
            self._h = None

    close = eakv_destroy

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.eakv_destroy()

    def __del__(self):
        try:
            self.eakv_destroy()
        except Exception:
            pass

    def _check(self, rc, where):
        if rc != OK:
            detail = lib().eakv_last_cuda_error(self._h).decode() if rc == E_CUDA else ""
            raise EakvError(rc, where, detail)

    # -- hashing ----------------------------------------------------------------------------
    def eakv_hash_blocks(self, tokens_dev, n_tokens, parent_hash, hashes_dev, stream=None):
        n = C.c_int64(0)
        rc = lib().eakv_hash_blocks(self._h, C.c_void_p(int(tokens_dev)), int(n_tokens),
                                    C.c_uint64(int(parent_hash)), C.c_void_p(int(hashes_dev)),
                                    C.byref(n), _stream(stream))
        self._check(rc, "eakv_hash_blocks")
        return n.value

    def eakv_hash_blocks_batched(self, tokens_dev, offsets, parents, hashes_dev, stream=None):
        off, off_p = _np(offsets, np.int64)
        n_prompts = len(off) - 1
        par_p = None
        if parents is not None:
            par, par_p = _np(parents, np.uint64)
        out = np.zeros(n_prompts + 1, dtype=np.int64)
        rc = lib().eakv_hash_blocks_batched(self._h, C.c_void_p(int(tokens_dev)), off_p, n_prompts,
                                            par_p, C.c_void_p(int(hashes_dev)),
                                            out.ctypes.data, _stream(stream))
        self._check(rc, "eakv_hash_blocks_batched")
        return out

    # -- control plane ----------------------------------------------------------------------
    def eakv_match(self, hashes):
        h, hp = _np(hashes, np.uint64)
        n = len(h)
        G, H = C.c_int64(0), C.c_int64(0)
        gids = np.full(n, -1, dtype=np.int32)
        slots = np.full(n, -1, dtype=np.int32)
        rc = lib().eakv_match(self._h, hp, n, C.byref(G), C.byref(H),
                              gids.ctypes.data, slots.ctypes.data)
        self._check(rc, "eakv_match")
        return G.value, H.value, gids[:G.value], slots[:H.value]

    def eakv_tier_export(self):
        """(keys, slots) of the host tier's residents, least recent first."""
        n = C.c_int64(0)
        self._check(lib().eakv_tier_export(self._h, None, None, 0, C.byref(n)), "eakv_tier_export")
        keys = np.zeros(n.value, dtype=np.uint64)
        slots = np.zeros(n.value, dtype=np.int32)
        rc = lib().eakv_tier_export(self._h, keys.ctypes.data, slots.ctypes.data,
                                    n.value, C.byref(n))
        self._check(rc, "eakv_tier_export")
        return keys, slots

    def eakv_tier_import(self, keys, slots):
        k, kp = _np(keys, np.uint64)
        s_, sp = _np(slots, np.int32)
        if len(k) != len(s_):
            raise ValueError("keys and slots differ in length")
        self._check(lib().eakv_tier_import(self._h, kp, sp, len(k)), "eakv_tier_import")

    def eakv_admission_export(self):
        """The admission windows as an opaque int64 array (see eakv_admission_import)."""
        n = C.c_int64(0)
        self._check(lib().eakv_admission_export(self._h, None, 0, C.byref(n)), "eakv_admission_export")
        vals = np.zeros(n.value, dtype=np.int64)
        self._check(lib().eakv_admission_export(self._h, vals.ctypes.data, n.value, C.byref(n)),
                    "eakv_admission_export")
        return vals

    def eakv_admission_import(self, values):
        v, vp_ = _np(values, np.int64)
        self._check(lib().eakv_admission_import(self._h, vp_, len(v)), "eakv_admission_import")

    def eakv_tier_step(self, hashes, agent_id, n_tokens, now_ms, decided=None):
        """``decided``: None for a request's first lookup; True / False = the store / skip choice
        of that first lookup when this is a later one (eakv_tier_step_again)."""
        h, hp = _np(hashes, np.uint64)
        n = len(h)
        hit = np.zeros(n, dtype=np.uint8)
        admit = np.zeros(n, dtype=np.uint8)
        slot = np.zeros(n, dtype=np.int32)
        ek = np.zeros(n, dtype=np.uint64)
        es = np.zeros(n, dtype=np.int32)
        nev = C.c_int64(n)
        info = StepInfo()
        vp = lambda a: a.ctypes.data
        if decided is None:
            rc = lib().eakv_tier_step(self._h, hp, n, int(agent_id), int(n_tokens), int(now_ms),
                                      vp(hit), vp(admit), vp(slot), vp(ek), vp(es), C.byref(nev),
                                      C.byref(info))
        else:
            rc = lib().eakv_tier_step_again(self._h, hp, n, int(n_tokens), int(now_ms), int(bool(decided)),
                                            vp(hit), vp(admit), vp(slot), vp(ek), vp(es), C.byref(nev),
                                            C.byref(info))
        self._check(rc, "eakv_tier_step")
        k = nev.value
        return dict(hit=hit, admit=admit, slot=slot, evicted_keys=ek[:k], evicted_slots=es[:k],
                    host_prefix_blocks=info.host_prefix_blocks, new_chunks=info.new_chunks,
                    pressure=bool(info.pressure), save=bool(info.save))

    def eakv_gpu_tier_step(self, hashes, need_tail):
        h, hp = _np(hashes, np.uint64)
        n = len(h)
        res = np.zeros(n, dtype=np.uint8)
        blk = np.zeros(n, dtype=np.int32)
        tail = C.c_int32(-1)
        rc = lib().eakv_gpu_tier_step(self._h, hp, n, int(bool(need_tail)),
                                      res.ctypes.data,
                                      blk.ctypes.data, C.byref(tail))
        self._check(rc, "eakv_gpu_tier_step")
        return res, blk, tail.value

    def eakv_gpu_tier_acquire(self, request_id, hashes, need_tail):
        """(resident, blocks, tail) with the blocks pinned under ``request_id``, or None when they
        do not fit beside the running requests (nothing changed)."""
        h, hp = _np(hashes, np.uint64)
        n = len(h)
        res = np.zeros(n, dtype=np.uint8)
        blk = np.zeros(n, dtype=np.int32)
        tail = C.c_int32(-1)
        rc = lib().eakv_gpu_tier_acquire(self._h, int(request_id), hp, n, int(bool(need_tail)),
                                         res.ctypes.data, blk.ctypes.data,
                                         C.byref(tail))
        if rc == E_BUSY:
            return None
        self._check(rc, "eakv_gpu_tier_acquire")
        return res, blk, tail.value

    def eakv_gpu_tier_release_request(self, request_id):
        self._check(lib().eakv_gpu_tier_release_request(self._h, int(request_id)),
                    "eakv_gpu_tier_release_request")

    def eakv_gpu_tier_release(self, block_id):
        self._check(lib().eakv_gpu_tier_release(self._h, int(block_id)), "eakv_gpu_tier_release")

    # -- data plane -------------------------------------------------------------------------
    def eakv_store(self, block_table, admit_mask, host_slots, stream=None):
        bt, btp = _np(block_table, np.int32)
        hs, hsp = _np(host_slots, np.int32)
        amp = None
        if admit_mask is not None:
            am, amp = _np(admit_mask, np.uint8)
        rc = lib().eakv_store(self._h, btp, amp, hsp, len(bt), _stream(stream))
        self._check(rc, "eakv_store")

    def eakv_load(self, host_slots, block_table, stream=None):
        bt, btp = _np(block_table, np.int32)
        hs, hsp = _np(host_slots, np.int32)
        rc = lib().eakv_load(self._h, hsp, btp, len(bt), _stream(stream))
        self._check(rc, "eakv_load")

    def eakv_load_layers(self, host_slots, block_table, layers_per_group, events, stream=None):
        """``events``: sequence of cudaEvent_t handles as integers (torch.cuda.Event.cuda_event)."""
        bt, btp = _np(block_table, np.int32)
        hs, hsp = _np(host_slots, np.int32)
        ev = (C.c_void_p * max(len(events), 1))(*[int(e) for e in events])
        rc = lib().eakv_load_layers(self._h, hsp, btp, len(bt), int(layers_per_group),
                                    C.cast(ev, C.c_void_p), len(events), _stream(stream))
        self._check(rc, "eakv_load_layers")

    def eakv_store_layers(self, block_table, admit_mask, host_slots, layers_per_group, ready_events, stream=None):
        """``ready_events``: per layer group a cudaEvent_t handle as integer (already recorded by the
        producer) or None for no wait."""
        bt, btp = _np(block_table, np.int32)
        hs, hsp = _np(host_slots, np.int32)
        amp = None
        if admit_mask is not None:
            am, amp = _np(admit_mask, np.uint8)
        ev = (C.c_void_p * max(len(ready_events), 1))(*[None if e is None else int(e) for e in ready_events])
        rc = lib().eakv_store_layers(self._h, btp, amp, hsp, len(bt), int(layers_per_group),
                                     C.cast(ev, C.c_void_p), len(ready_events), _stream(stream))
        self._check(rc, "eakv_store_layers")

    def eakv_turn_begin(self, tokens_ptr, n_tokens, known_keys, agent_id, now_ms, stream=None, layers=None):
        """First half of a turn; returns a dict of the view's scalars and (copied) arrays.
        ``layers`` = (layers_per_group, events): the restore runs in layer groups and records one
        event per group (eakv_turn_begin_layers)."""
        kp, nk = None, 0
        if known_keys is not None and len(known_keys):
            kk, kp = _np(known_keys, np.uint64)
            nk = len(kk)
        v = TurnView()
        if layers is None:
            rc = lib().eakv_turn_begin(self._h, C.c_void_p(int(tokens_ptr)), int(n_tokens), kp, nk,
                                       int(agent_id), int(now_ms), _stream(stream), C.byref(v))
        else:
            ev = self._event_array(layers[1])
            rc = lib().eakv_turn_begin_layers(self._h, C.c_void_p(int(tokens_ptr)), int(n_tokens), kp, nk,
                                              int(agent_id), int(now_ms), int(layers[0]), C.cast(ev, C.c_void_p),
                                              len(layers[1]), _stream(stream), C.byref(v))
        self._check(rc, "eakv_turn_begin")
        return self._view_dict(v)

    def eakv_request_begin(self, request_id, tokens_ptr, n_tokens, known_keys, agent_id, now_ms,
                           decided=None, stream=None, layers=None):
        """First half of a running request's turn (its GPU blocks stay pinned until
        eakv_request_release); None when the blocks do not fit beside the running requests.
        ``decided``: None for the first lookup, else the store/skip choice made then."""
        kp, nk = None, 0
        if known_keys is not None and len(known_keys):
            kk, kp = _np(known_keys, np.uint64)
            nk = len(kk)
        v = TurnView()
        d = -1 if decided is None else int(bool(decided))
        if layers is None:
            rc = lib().eakv_request_begin(self._h, int(request_id), C.c_void_p(int(tokens_ptr)), int(n_tokens), kp, nk,
                                          int(agent_id), int(now_ms), d, _stream(stream), C.byref(v))
        else:
            ev = self._event_array(layers[1])
            rc = lib().eakv_request_begin_layers(self._h, int(request_id), C.c_void_p(int(tokens_ptr)), int(n_tokens),
                                                 kp, nk, int(agent_id), int(now_ms), d, int(layers[0]),
                                                 C.cast(ev, C.c_void_p), len(layers[1]), _stream(stream), C.byref(v))
        if rc == E_BUSY:
            return None
        self._check(rc, "eakv_request_begin")
        return self._view_dict(v)

    def eakv_selfcheck_fail_next_transfer(self, code):
        self._check(lib().eakv_selfcheck_fail_next_transfer(self._h, int(code)), "eakv_selfcheck_fail_next_transfer")

    def eakv_request_store(self, request_id, stream=None):
        self._check(lib().eakv_request_store(self._h, int(request_id), _stream(stream)), "eakv_request_store")

    @staticmethod
    def _event_array(ready_events):
        return (C.c_void_p * max(len(ready_events), 1))(*[None if e is None else int(e) for e in ready_events])

    def eakv_request_store_layers(self, request_id, layers_per_group, ready_events, stream=None):
        ev = self._event_array(ready_events)
        rc = lib().eakv_request_store_layers(self._h, int(request_id), int(layers_per_group), C.cast(ev, C.c_void_p),
                                             len(ready_events), _stream(stream))
        self._check(rc, "eakv_request_store_layers")

    def eakv_turn_end_layers(self, layers_per_group, ready_events, stream=None):
        ev = self._event_array(ready_events)
        rc = lib().eakv_turn_end_layers(self._h, int(layers_per_group), C.cast(ev, C.c_void_p),
                                        len(ready_events), _stream(stream))
        self._check(rc, "eakv_turn_end_layers")

    def eakv_request_release(self, request_id):
        self._check(lib().eakv_request_release(self._h, int(request_id)), "eakv_request_release")

    @staticmethod
    def _view_dict(v):
        nb, nu, ne = v.n_blocks, v.n_units, v.n_evicted
        out = {n: getattr(v, n) for n, _ in TurnView._fields_[:15] if n != "reserved"}
        out.update(keys=_view_array(v.keys, nb, np.uint64), gpu_block=_view_array(v.gpu_block, nb, np.int32),
                   gpu_resident=_view_array(v.gpu_resident, nb, np.uint8),
                   needs_fill=_view_array(v.needs_fill, nb, np.uint8),
                   hit=_view_array(v.hit, nu, np.uint8), admit=_view_array(v.admit, nu, np.uint8),
                   slot=_view_array(v.slot, nu, np.int32),
                   evicted_keys=_view_array(v.evicted_keys, ne, np.uint64),
                   evicted_slots=_view_array(v.evicted_slots, ne, np.int32))
        return out

    def eakv_turn_end(self, stream=None):
        self._check(lib().eakv_turn_end(self._h, _stream(stream)), "eakv_turn_end")

    def eakv_turn_abort(self):
        self._check(lib().eakv_turn_abort(self._h), "eakv_turn_abort")

    def eakv_sync(self):
        self._check(lib().eakv_sync(self._h), "eakv_sync")

    def eakv_selfcheck_limits(self, gpu_blocks=0, tier_slots=0, hash_blocks=0):
        self._check(lib().eakv_selfcheck_limits(self._h, int(gpu_blocks), int(tier_slots), int(hash_blocks)),
                    "eakv_selfcheck_limits")

    def eakv_selfcheck_wait_probe(self, stream=None):
        self._check(lib().eakv_selfcheck_wait_probe(self._h, _stream(stream)), "eakv_selfcheck_wait_probe")

    # -- introspection ----------------------------------------------------------------------
    def eakv_get_stats(self):
        s = Stats()
        self._check(lib().eakv_get_stats(self._h, C.byref(s)), "eakv_get_stats")
        return s.as_dict()

    def eakv_tier_ptr(self):
        return lib().eakv_tier_ptr(self._h)

    def eakv_hash_seed(self):
        return lib().eakv_hash_seed(self._h)

    def eakv_hash_base(self):
        return lib().eakv_hash_base(self._h)

    def tier_host_view(self):
        """numpy uint8 view [block slots, 2L, piece_bytes] of a pinned-host tier."""
        if self.tier_location != TIER_PINNED_HOST:
            raise ValueError("tier is not in host memory")
        n = self.tier_slots * self.block_bytes
        buf = (C.c_uint8 * n).from_address(self.eakv_tier_ptr())
        return np.frombuffer(buf, dtype=np.uint8).reshape(
            self.tier_slots, self.block_bytes // self.piece_bytes, self.piece_bytes)
