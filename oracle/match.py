"""Longest cached prefix (Section 2 "Exact-prefix reuse"; Appendix C "Prefix coverage
from a reference stream", and the restore equation R_j = max{0, H_j - G_j} there).

A lookup walks the block keys from the start and stops at the first absent one: a resident
block behind a gap does not count, since only an unbroken prefix can be restored.
"""


def leading_run(keys, index):
    """Number of leading keys present in ``index`` (any container with ``in``)."""
    n = 0
    for k in keys:
        if k not in index:
            break
        n += 1
    return n


def match(keys, gpu_index, host_index):
    """Return (G, H): leading blocks resident on the GPU and in the host tier."""
    return leading_run(keys, gpu_index), leading_run(keys, host_index)


def restore_run(G, H):
    """Blocks [lo, hi) that a restore brings from the host: those the host covers beyond
    the GPU-resident prefix; empty when H <= G."""
    return (G, H) if H > G else (G, G)


def fresh_tokens(n_tokens, block_size, G, H):
    """Prompt tokens no tier covers (computed prefill): n - max(G, H) * b."""
    return n_tokens - max(G, H) * block_size


def fresh_prefill(submitted_tokens, cache_stable_tokens):
    """Appendix F: with resident history, fresh prefill = submitted - cache-stable."""
    return submitted_tokens - cache_stable_tokens
