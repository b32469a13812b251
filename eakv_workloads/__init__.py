"""Seeded synthetic inputs for the paged-KV offload path.

This package only *generates inputs*: KV shapes, agent traces (who asks what, when),
token ids and KV payload bits.  It contains none of the method's arithmetic (no
hashing, matching, tier bookkeeping or copying) so that the CPU oracle and the CUDA
path can both consume it without sharing any of the code under test.
"""
from .shapes import KVShape, SHAPES, CONFIGS, TraceConfig  # noqa: F401
from .traces import Trace, Request, make_trace  # noqa: F401
from .kvfill import (  # noqa: F401
    normal_bf16_words, counter_words_numpy, counter_words_torch, counter_words_at_torch,
    key_words_numpy, key_words_torch,
)
