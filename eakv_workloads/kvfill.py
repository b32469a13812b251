"""KV payload bits.  The path under test never interprets them; these generators only
make the bytes reproducible so that either side can regenerate any block on demand.

Two families:
  * ``normal_bf16_words``: N(0,1) fp32 rounded to bf16 (round-to-nearest-even), used by
    the tiny configuration;
  * counter words: a pure integer function of (salt, element index), finite bf16 bit
    patterns, available for numpy (CPU side) and torch (device side) with identical
    results, used where a second full copy of the pool would not fit anywhere.
"""
from __future__ import annotations

import numpy as np

_M1 = 0x9E3779B97F4A7C15
_M2 = 0xD6E8FEB86659FD93
_MASK64 = (1 << 64) - 1


def normal_bf16_words(seed_tuple, n_words: int) -> np.ndarray:
    """uint16 bit patterns of bf16(N(0,1)), seeded by an integer tuple."""
    rng = np.random.default_rng(list(seed_tuple))
    x = rng.standard_normal(n_words, dtype=np.float32)
    bits = x.view(np.uint32).astype(np.uint64)
    rounded = (bits + 0x7FFF + ((bits >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def _signed(v: int) -> int:
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def counter_words_numpy(salt: int, start: int, n_words: int) -> np.ndarray:
    """uint16 words w[i] = f(salt, start + i); finite bf16 patterns (|x| < 2)."""
    idx = np.arange(start, start + n_words, dtype=np.uint64)
    with np.errstate(over="ignore"):
        v = (idx * np.uint64(_M1) + np.uint64(salt & _MASK64)) * np.uint64(_M2)
    return ((v >> np.uint64(29)) & np.uint64(0xBFFF)).astype(np.uint16)


def counter_words_torch(salt: int, start: int, n_words: int, device):
    """Same words as ``counter_words_numpy`` as an int16 torch tensor on ``device``."""
    import torch
    idx = torch.arange(start, start + n_words, dtype=torch.int64, device=device)
    v = (idx * _signed(_M1) + _signed(salt)) * _signed(_M2)
    return ((v >> 29) & 0xBFFF).to(torch.int16)


def counter_words_at_torch(salt: int, idx):
    """``counter_words_torch`` evaluated at arbitrary int64 element indices ``idx``."""
    import torch
    v = (idx.to(torch.int64) * _signed(_M1) + _signed(salt)) * _signed(_M2)
    return ((v >> 29) & 0xBFFF).to(torch.int16)


_PATTERNS = {}


def _key_scalar_numpy(keys) -> np.ndarray:
    """2 x 16 payload bits per key (finite bf16 patterns: exponent's top bit clear)."""
    keys = np.asarray(keys, dtype=np.uint64)
    with np.errstate(over="ignore"):
        v = keys * np.uint64(_M2)
    lo = ((v >> np.uint64(37)) & np.uint64(0xBFFF)).astype(np.uint16)
    hi = ((v >> np.uint64(13)) & np.uint64(0xBFFF)).astype(np.uint16)
    return np.stack([lo, hi], axis=-1)            # [n, 2]: even and odd words get different bits


def key_words_numpy(keys, q: int, n_words: int) -> np.ndarray:
    """[len(keys), n_words] uint16: payload of piece ``q`` of the blocks with these keys: a
    fixed per-piece pattern XOR 16 bits derived from the key (cheap enough that generating the
    "prefill" of a replay does not dominate it)."""
    pat = _PATTERNS.get(("np", q, n_words))
    if pat is None:
        pat = _PATTERNS[("np", q, n_words)] = counter_words_numpy(q + 1, 0, n_words)
    kv = _key_scalar_numpy(keys)                               # [n, 2]
    return (pat.reshape(1, -1, 2) ^ kv.reshape(-1, 1, 2)).reshape(len(kv), n_words)


def key_words_torch(keys, q: int, n_words: int, device):
    """Same as ``key_words_numpy`` as an int16 tensor on ``device``.  ``keys`` is an int64
    tensor (or sequence) holding the 61-bit keys."""
    import torch
    dev = torch.device(device)
    pat = _PATTERNS.get((str(dev), q, n_words))
    if pat is None:
        pat = _PATTERNS[(str(dev), q, n_words)] = counter_words_torch(q + 1, 0, n_words, dev)
    keys = torch.as_tensor(keys, dtype=torch.int64, device=dev).reshape(-1, 1)
    v = keys * _signed(_M2)
    kv = torch.cat([((v >> 37) & 0xBFFF), ((v >> 13) & 0xBFFF)], dim=1).to(torch.int16)   # [n, 2]
    return (pat.reshape(1, -1, 2) ^ kv.reshape(-1, 1, 2)).reshape(kv.shape[0], n_words)
