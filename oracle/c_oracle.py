"""ctypes access to the plain C oracle (oracle/eakv_oracle.c) -- TEST INFRASTRUCTURE ONLY.

Compiled on demand with gcc into oracle/libeakv_oracle.so.  Used by the tests (which check it
against the Python oracle, so that it inherits that oracle's pins) and by the benchmark's
CPU-baseline legs, never by the product."""
import ctypes as C
import os
import subprocess

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "eakv_oracle.c")
LIB = os.path.join(HERE, "libeakv_oracle.so")
_lib = None


def build(force=False):
    if force or not os.path.exists(LIB) or os.path.getmtime(LIB) < os.path.getmtime(SRC):
        subprocess.run(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-o", LIB, SRC], check=True)
    return LIB


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        vp, i32, i64, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64
        L.oracle_hash_blocks.argtypes = [vp, i64, i32, u64, u64, vp]
        L.oracle_hash_blocks.restype = i64
        L.oracle_store.argtypes = [vp, vp, i32, i64, vp, vp, vp, i64]
        L.oracle_load.argtypes = [vp, vp, i32, i64, vp, vp, i64]
        L.oracle_tier_new.argtypes = [i64, i32, i32]
        L.oracle_tier_new.restype = vp
        L.oracle_tier_free.argtypes = [vp]
        L.oracle_tier_leading_run.argtypes = [vp, vp, i64, vp]
        L.oracle_tier_leading_run.restype = i64
        L.oracle_tier_step.argtypes = [vp, vp, i64, vp, vp, vp]
        L.oracle_tier_step.restype = i32
        _lib = L
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def hash_blocks(tokens, block_size, parent, base):
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    out = np.zeros(len(tokens) // block_size + 1, dtype=np.uint64)
    n = lib().oracle_hash_blocks(_p(tokens), len(tokens), block_size, parent, base, _p(out))
    return out[:n]


def _pool_ptrs(pool):
    return (C.c_void_p * len(pool))(*[a.ctypes.data for a in pool])


def store(pool, tier, block_table, admit, slots):
    """pool: list of 2L uint8 arrays [blocks, piece_bytes]; tier: uint8 [slots, 2L, piece_bytes]."""
    bt = np.ascontiguousarray(block_table, dtype=np.int32)
    sl = np.ascontiguousarray(slots, dtype=np.int32)
    ad = None if admit is None else np.ascontiguousarray(admit, dtype=np.uint8)
    lib().oracle_store(_pool_ptrs(pool), _p(tier), len(pool), pool[0].shape[1], _p(bt),
                       None if ad is None else _p(ad), _p(sl), len(bt))


def load(pool, tier, slots, block_table):
    bt = np.ascontiguousarray(block_table, dtype=np.int32)
    sl = np.ascontiguousarray(slots, dtype=np.int32)
    lib().oracle_load(_pool_ptrs(pool), _p(tier), len(pool), pool[0].shape[1], _p(sl), _p(bt), len(bt))


class Tier:
    """LRU reference model under write-all (policy 0) or fixed admission (policy 1)."""

    def __init__(self, capacity, policy=0, kappa=8):
        self._t = lib().oracle_tier_new(capacity, policy, kappa)

    def close(self):
        if self._t:
            lib().oracle_tier_free(self._t)
            self._t = None

    def leading_run(self, keys):
        k = np.ascontiguousarray(keys, dtype=np.uint64)
        slots = np.full(len(k), -1, dtype=np.int32)
        h = lib().oracle_tier_leading_run(self._t, _p(k), len(k), _p(slots))
        return h, slots[:h]

    def step(self, keys):
        k = np.ascontiguousarray(keys, dtype=np.uint64)
        hit = np.zeros(len(k), dtype=np.uint8)
        admit = np.zeros(len(k), dtype=np.uint8)
        slot = np.zeros(len(k), dtype=np.int32)
        save = lib().oracle_tier_step(self._t, _p(k), len(k), _p(hit), _p(admit), _p(slot))
        if save < 0:
            raise ValueError("request references more keys than the tier holds")
        return bool(save), hit, admit, slot
