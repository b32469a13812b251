"""Prefix-dependent block keys (Section 3.2: each full chunk's key depends on its
entire prefix; Section 4: only *full* chunks count).

The paper's stack hashes with a cryptographic hash on the CPU; this build fixes a
polynomial hash modulo the Mersenne prime p = 2^61 - 1 instead:

    h_{-1} = parent,   h_i = (h_{i-1} * B + (token_i + 1)) mod p,

kept canonical in [0, p).  Block j's key is h after its last token; a partial tail
block has no key.  Hashing may resume at a block boundary by passing the previous
block's key as ``parent``.
"""
P61 = (1 << 61) - 1
HASH_BASE = 6364136223846793005 % P61   # 1752450205419405103
HASH_SEED = 0x9E3779B97F4A7C15 % P61    # 2177342782468422681


def hash_blocks(tokens, block_size, parent=HASH_SEED, base=HASH_BASE):
    """Keys of the full blocks of ``tokens`` (any int sequence), as Python ints."""
    h = int(parent) % P61
    keys = []
    filled = 0
    for t in tokens:
        h = (h * base + (int(t) + 1)) % P61
        filled += 1
        if filled == block_size:
            keys.append(h)
            filled = 0
    return keys


def hash_prefix(tokens, parent=HASH_SEED, base=HASH_BASE):
    """Running hash after all of ``tokens`` (no block structure)."""
    h = int(parent) % P61
    for t in tokens:
        h = (h * base + (int(t) + 1)) % P61
    return h
