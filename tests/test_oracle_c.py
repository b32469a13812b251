"""The plain C oracle against the Python oracle (which carries the pins): hash keys, store/load
bytes and the LRU tier under write-all and fixed admission must agree exactly."""
import random

import numpy as np
import pytest

from oracle import c_oracle, hash as ohash, storeload
from oracle.tier import FILTER_FIXED, WRITE_ALL, HostTier


def test_hash_agrees_with_python_oracle_and_printed_vectors():
    rng = np.random.default_rng(0)
    assert c_oracle.hash_blocks([0, 1, 2, 3], 4, ohash.HASH_SEED, ohash.HASH_BASE).tolist() == [1550033248144644936]
    assert c_oracle.hash_blocks([0], 1, ohash.HASH_SEED, ohash.HASH_BASE).tolist() == [978183904022676520]
    for b in (1, 3, 16, 32):
        for n in (0, 1, b - 1, b, 5 * b + 2, 1000):
            toks = rng.integers(0, 151936, size=max(n, 0), dtype=np.int32)
            for parent in (ohash.HASH_SEED, 0, ohash.P61 - 1, int(rng.integers(0, ohash.P61))):
                got = c_oracle.hash_blocks(toks, b, parent, ohash.HASH_BASE).tolist()
                assert got == ohash.hash_blocks(toks.tolist(), b, parent)


def test_store_load_agree_with_python_oracle():
    rng = np.random.default_rng(1)
    Q, P, nb, kh = 6, 96, 20, 12
    pool_a = [rng.integers(0, 256, size=(nb, P), dtype=np.uint8) for _ in range(Q)]
    pool_b = [a.copy() for a in pool_a]
    tier_a = rng.integers(0, 256, size=(kh, Q, P), dtype=np.uint8)
    tier_b = tier_a.copy()
    table = rng.permutation(nb)[:kh].astype(np.int32)
    slots = rng.permutation(kh).astype(np.int32)
    admit = (rng.random(kh) < 0.6).astype(np.uint8)
    c_oracle.store(pool_a, tier_a, table, admit, slots)
    storeload.store(pool_b, tier_b, table, admit, slots)
    assert np.array_equal(tier_a, tier_b)
    dst = rng.permutation(nb)[:5].astype(np.int32)
    src = rng.permutation(kh)[:5].astype(np.int32)
    c_oracle.load(pool_a, tier_a, src, dst)
    storeload.load(pool_b, tier_b, src, dst)
    for a, b in zip(pool_a, pool_b):
        assert np.array_equal(a, b)


@pytest.mark.parametrize("policy", [WRITE_ALL, FILTER_FIXED])
def test_tier_agrees_with_python_oracle(policy):
    rng = random.Random(5 + policy)
    for case in range(40):
        K = rng.randrange(2, 24)
        kappa = rng.randrange(0, 8)
        py = HostTier(K, 4, policy, kappa)
        ct = c_oracle.Tier(K, policy, kappa)
        for step in range(rng.randrange(3, 30)):
            agent = rng.randrange(4)
            n = rng.randrange(0, K + 1)
            keys = [1000 * agent + j for j in range(n)]
            assert ct.leading_run(keys)[0] == py.leading_run(keys)
            want = py.step(keys, 4 * n, agent, step)
            save, hit, admit, slot = ct.step(keys)
            assert (save, hit.tolist(), admit.tolist(), slot.tolist()) == \
                   (bool(want.save), want.hit, want.admit, want.slot)
        with pytest.raises(ValueError):
            ct.step(list(range(K + 1)))
        ct.close()
