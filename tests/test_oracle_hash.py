"""Pins for oracle.hash: the closed-form polynomial, special cases and invariants."""
import random

from oracle import hash as oh

P = (1 << 61) - 1


def closed_form(tokens, parent, base):
    n = len(tokens)
    s = parent * pow(base, n, P)
    for i, t in enumerate(tokens):
        s += (t + 1) * pow(base, n - 1 - i, P)
    return s % P


def test_constants_and_vectors(golden):
    g = golden("hash_vectors.txt")
    assert oh.P61 == int(g["p"]) == 2**61 - 1
    assert oh.HASH_BASE == int(g["base"])
    assert oh.HASH_SEED == int(g["seed"])
    assert oh.hash_prefix([]) == int(g["hash_empty"])
    assert oh.hash_prefix([0]) == int(g["hash_0"])
    assert oh.hash_prefix([0, 1, 2, 3]) == int(g["hash_0_1_2_3"])
    # the vectors themselves follow from the closed form
    assert closed_form([0], oh.HASH_SEED, oh.HASH_BASE) == int(g["hash_0"])
    assert closed_form([0, 1, 2, 3], oh.HASH_SEED, oh.HASH_BASE) == int(g["hash_0_1_2_3"])


def test_matches_closed_form_random():
    rng = random.Random(1)
    for _ in range(50):
        n = rng.randrange(0, 200)
        toks = [rng.randrange(0, 2**31 - 1) for _ in range(n)]
        parent = rng.randrange(0, P)
        base = rng.randrange(2, P)
        assert oh.hash_prefix(toks, parent, base) == closed_form(toks, parent, base)


def test_constant_sequence_geometric_sum():
    # all tokens equal: S*B^n + x*(B^n - 1)/(B - 1)
    B, S = oh.HASH_BASE, oh.HASH_SEED
    inv = pow(B - 1, P - 2, P)
    for x_tok, n in [(0, 1), (7, 16), (151935, 333), (2**31 - 2, 64)]:
        x = x_tok + 1
        expect = (S * pow(B, n, P) + x * (pow(B, n, P) - 1) * inv) % P
        assert oh.hash_prefix([x_tok] * n) == expect


def test_block_keys_are_prefix_hashes_and_tail_has_no_key():
    rng = random.Random(2)
    toks = [rng.randrange(0, 151936) for _ in range(16 * 5 + 9)]
    keys = oh.hash_blocks(toks, 16)
    assert len(keys) == 5
    for j, k in enumerate(keys):
        assert k == closed_form(toks[: 16 * (j + 1)], oh.HASH_SEED, oh.HASH_BASE)
    assert oh.hash_blocks(toks[:15], 16) == []
    assert oh.hash_blocks([], 16) == []


def test_resume_from_parent_equals_one_shot():
    rng = random.Random(3)
    toks = [rng.randrange(0, 151936) for _ in range(32 * 9 + 5)]
    full = oh.hash_blocks(toks, 32)
    for j in range(1, 9):
        resumed = oh.hash_blocks(toks[32 * j:], 32, parent=full[j - 1])
        assert resumed == full[j:]


def test_keys_depend_on_entire_prefix():
    a = list(range(64))
    b = list(a)
    b[0] += 1           # edit the very first token
    ka, kb = oh.hash_blocks(a, 16), oh.hash_blocks(b, 16)
    assert all(x != y for x, y in zip(ka, kb))   # every later key changes
    c = list(a)
    c[40] += 1          # edit inside block 2
    kc = oh.hash_blocks(c, 16)
    assert kc[:2] == ka[:2] and kc[2] != ka[2] and kc[3] != ka[3]


def test_canonical_zero_representative():
    # choose parent so that parent*B + x == 0 (mod p): result must be 0, never p
    B = oh.HASH_BASE
    for tok in [0, 5, 151935]:
        parent = (-(tok + 1) * pow(B, P - 2, P)) % P
        assert oh.hash_prefix([tok], parent) == 0
    # and the largest representative p-1 is reachable and stays p-1
    parent = ((P - 1 - 1) * pow(B, P - 2, P)) % P
    assert oh.hash_prefix([0], parent) == P - 1


def test_leading_zero_tokens_do_not_collide():
    # x = token + 1 is never zero, so [0]*k for different k give different hashes
    seen = {oh.hash_prefix([0] * k) for k in range(64)}
    assert len(seen) == 64
