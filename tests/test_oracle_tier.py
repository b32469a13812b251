"""Pins for oracle.tier and oracle.stackdist: Mattson inclusion (Eq. 4), Lemma 1,
Proposition 1 and the write rule (Eq. 6 / Eq. 10), against brute force on tiny traces.
The brute-force LRU below is written differently on purpose (timestamps + linear scan).
"""
import math
import random

import pytest

from oracle import stackdist as sd
from oracle import tier as ot


def brute_lru(stream, K, declined=frozenset()):
    """LRU by last-use timestamps; returns (hits, promoted_flags)."""
    last_use = {}            # resident key -> timestamp of last promotion
    hits, promoted = [], []
    for i, k in enumerate(stream):
        if k in last_use:
            hits.append(True); promoted.append(True)
            last_use[k] = i
            continue
        hits.append(False)
        if i in declined:
            promoted.append(False)
            continue
        if len(last_use) >= K:
            victim = min(last_use, key=lambda x: last_use[x])
            del last_use[victim]
        last_use[k] = i
        promoted.append(True)
    return hits, promoted


def rand_stream(rng, T, U):
    return [rng.randrange(U) for _ in range(T)]


def test_reuse_distance_hand_case():
    #          a  b  c  a  b  b  d  c  a
    stream = [1, 2, 3, 1, 2, 2, 4, 3, 1]
    expect = [math.inf, math.inf, math.inf, 2, 2, 0, math.inf, 3, 3]
    assert sd.reuse_distances_definition(stream) == expect
    assert sd.reuse_distances(stream) == expect


def test_fast_distances_equal_definition():
    rng = random.Random(5)
    for _ in range(100):
        s = rand_stream(rng, rng.randrange(0, 80), rng.randrange(1, 15))
        assert sd.reuse_distances(s) == sd.reuse_distances_definition(s)


def test_mattson_inclusion_and_monotone_hits():
    rng = random.Random(6)
    for _ in range(150):
        s = rand_stream(rng, rng.randrange(1, 120), rng.randrange(1, 20))
        D = sd.reuse_distances(s)
        prev = None
        for K in range(1, 22):
            model = ot.simulate_stream(s, K)
            brute, _ = brute_lru(s, K)
            assert model == brute
            assert model == sd.predicted_hits(D, K)            # hit  <=>  D < K
            if prev is not None:                                 # inclusion: hits grow with K
                assert all((not p) or m for p, m in zip(prev, model))
            prev = model
        # a tier that holds everything hits every re-reference
        assert ot.simulate_stream(s, 10**9) == [d != math.inf for d in D]
        assert sd.working_set_full(D) == (max([d for d in D if d != math.inf], default=-1) + 1)


def test_lemma1_resident_iff_promotions_below_capacity():
    rng = random.Random(7)
    for _ in range(300):
        s = rand_stream(rng, rng.randrange(2, 60), rng.randrange(2, 10))
        K = rng.randrange(1, 8)
        declined = {i for i in range(len(s)) if rng.random() < 0.3}
        hits, promoted = brute_lru(s, K, declined)
        assert hits == ot.simulate_stream(s, K, declined)
        for t, y in enumerate(s):
            prev = [i for i in range(t) if s[i] == y]
            if not prev:
                continue
            sref = prev[-1]
            if not promoted[sref]:
                continue
            P = len({s[i] for i in range(sref + 1, t) if promoted[i] and s[i] != y})
            assert hits[t] == (P < K)


def test_proposition1_declinable_writes_lose_no_hit():
    rng = random.Random(8)
    for _ in range(300):
        s = rand_stream(rng, rng.randrange(2, 70), rng.randrange(2, 12))
        K = rng.randrange(1, 8)
        D = sd.reuse_distances(s)
        # next-reference distance of every reference (inf if never referenced again)
        nxt = [math.inf] * len(s)
        last = {}
        for i, k in enumerate(s):
            if k in last:
                nxt[last[k]] = D[i]
            last[k] = i
        full = ot.simulate_stream(s, K)
        eligible = [i for i in range(len(s)) if nxt[i] >= K]
        declined = {i for i in eligible if rng.random() < 0.6}
        restricted = ot.simulate_stream(s, K, declined)
        assert all((not f) or r for f, r in zip(full, restricted))
        assert sum(restricted) >= sum(full)


def test_proposition1_coverage_never_shrinks():
    rng = random.Random(9)
    for _ in range(100):
        # requests = prefixes of a few "agents", so coverage (leading run) is meaningful
        reqs = []
        for _ in range(rng.randrange(2, 10)):
            a = rng.randrange(3)
            n = rng.randrange(1, 8)
            reqs.append([(a, j) for j in range(n)])
        s = [k for r in reqs for k in r]
        K = rng.randrange(1, 10)
        D = sd.reuse_distances(s)
        nxt = [math.inf] * len(s)
        last = {}
        for i, k in enumerate(s):
            if k in last:
                nxt[last[k]] = D[i]
            last[k] = i
        declined = {i for i in range(len(s)) if nxt[i] >= K and rng.random() < 0.5}
        full = ot.simulate_stream(s, K)
        rest = ot.simulate_stream(s, K, declined)
        pos = 0
        for r in reqs:
            cf = sd.request_coverage(full[pos:pos + len(r)])
            cr = sd.request_coverage(rest[pos:pos + len(r)])
            assert cr >= cf
            pos += len(r)


def run_requests(tier, reqs, b=4):
    out = []
    for i, (agent, keys) in enumerate(reqs):
        out.append(tier.step(keys, len(keys) * b + 1, agent, i * 1000))
    return out


def test_host_tier_equals_stream_model_under_write_all():
    rng = random.Random(10)
    for _ in range(100):
        reqs = [(rng.randrange(4), [(a, j) for j in range(rng.randrange(0, 7))])
                for a in [rng.randrange(4) for _ in range(rng.randrange(1, 12))]]
        K = rng.randrange(7, 15)
        t = ot.HostTier(K, 4)
        res = run_requests(t, reqs)
        s = [k for _, keys in reqs for k in keys]
        flat = [h for r in res for h in r.hit]
        assert [bool(h) for h in flat] == ot.simulate_stream(s, K)
        # admit = miss (write-all), dedup = resident chunks are never copied
        assert all(a == 1 - h for r in res for a, h in zip(r.admit, r.hit))
        # slots of resident keys are unique and in range
        slots = list(t.order.values())
        assert len(set(slots)) == len(slots) and all(0 <= x < K for x in slots)
        assert len(slots) + len(t.free) == K


def test_slot_assignment_free_stack():
    t = ot.HostTier(3, 4)
    r = t.step(["a", "b", "c"], 13, 0, 0)
    assert r.slot == [0, 1, 2] and r.evicted == []
    r = t.step(["d"], 5, 1, 1)                 # evicts "a" (least recent), reuses slot 0
    assert r.evicted == [("a", 0)] and r.slot == [0] and r.admit == [1]
    r = t.step(["b", "e"], 9, 0, 2)            # b hits (slot 1); e evicts c (slot 2)
    assert r.hit == [1, 0] and r.slot == [1, 2] and r.evicted == [("c", 2)]
    assert r.host_prefix_blocks == 1 and r.new_chunks == 1


def test_isolated_resident_chunk_hits_but_does_not_extend_coverage():
    t = ot.HostTier(8, 4)
    t.step(["a", "b", "c"], 12, 0, 0)
    r = t.step(["a", "x", "c"], 12, 0, 1)
    assert r.host_prefix_blocks == 1
    assert r.hit == [1, 0, 1] and r.admit == [0, 1, 0]
    assert r.new_chunks == 2


def test_capacity_error_changes_nothing():
    t = ot.HostTier(2, 4)
    t.step(["a"], 4, 0, 0)
    before = (list(t.order.items()), list(t.free), dict(t.stats))
    with pytest.raises(ot.CapacityError):
        t.step(["p", "q", "r"], 12, 0, 1)
    assert before == (list(t.order.items()), list(t.free), dict(t.stats))


def test_write_rule_endpoints_and_threshold():
    keys = lambda a, n: [(a, j) for j in range(n)]
    # u = floor(n/b) - floor(h/b): 10 blocks, host holds first 4 -> u = 6
    for kappa, expect_save in [(5, False), (6, True), (7, True)]:
        t = ot.HostTier(64, 4, policy=ot.FILTER_FIXED, kappa_blocks=kappa)
        t.step(keys(0, 4), 16, 0, 0)           # u = 4 <= kappa: saved
        assert all(k in t for k in keys(0, 4))
        r = t.step(keys(0, 10), 43, 0, 1)
        assert r.new_chunks == 6 and r.pressure and r.save == expect_save
        assert r.hit[:4] == [1] * 4
        assert r.admit[4:] == [int(expect_save)] * 6
        if not expect_save:
            assert r.slot[4:] == [-1] * 6 and r.evicted == []
    # fixed admission: a long first prompt is declined, and stays declined as u only grows
    t = ot.HostTier(64, 4, policy=ot.FILTER_FIXED, kappa_blocks=8)
    for turn, n in enumerate([9, 10, 12]):
        r = t.step(keys(1, n), n * 4, 1, turn)
        assert not r.save and sum(r.admit) == 0
    assert len(t.order) == 0
    # kappa = infinity reproduces write-all; p == 0 reproduces write-all
    rng = random.Random(11)
    reqs = [(a, keys(a, rng.randrange(1, 9))) for a in [rng.randrange(3) for _ in range(30)]]
    base = run_requests(ot.HostTier(10, 4), reqs)
    for pol, kap in [(ot.FILTER_FIXED, 10**9), (ot.FILTER_CONDITIONED, 10**9), (ot.WRITE_ALL, 0)]:
        other = run_requests(ot.HostTier(10, 4, policy=pol, kappa_blocks=kap), reqs)
        assert [(r.hit, r.admit, r.slot, r.evicted) for r in base] == \
               [(r.hit, r.admit, r.slot, r.evicted) for r in other]


def test_conditioned_pressure_needs_estimate_and_full_evicting_tier():
    b = 4
    keys = lambda a, lo, hi: [(a, j) for j in range(lo, hi)]
    # K = 8 blocks = 32 tokens of capacity.  Two agents with 5-block prompts: estimate
    # (A-1)*mean = 1*20 tokens <= 32 -> never pressure, even once the tier evicts.
    t = ot.HostTier(8, b, policy=ot.FILTER_CONDITIONED, kappa_blocks=2)
    for i in range(6):
        r = t.step(keys(i % 2, 0, 5) if i < 2 else keys(i, 0, 5), 20, i % 2, i)
        assert not r.pressure and r.save
    assert t.stats["evicted"] > 0
    # Three agents with 5-block prompts: estimate 2*20 = 40 > 32.  Pressure engages only
    # after the tier is >= 95 % full AND has evicted inside the window.
    t = ot.HostTier(8, b, policy=ot.FILTER_CONDITIONED, kappa_blocks=2)
    r0 = t.step(keys(0, 0, 5), 20, 0, 0)       # A=1: estimate 0
    r1 = t.step(keys(1, 0, 5), 20, 1, 1)       # A=2: 20 <= 32; evicts 2 while inserting
    r2 = t.step(keys(2, 0, 5), 20, 2, 2)       # A=3: 40 > 32, tier full (8/8), e_t = 2 > 0
    assert (r0.pressure, r1.pressure, r2.pressure) == (False, False, True)
    assert r1.evicted and len(r1.evicted) == 2
    assert not r2.save and sum(r2.admit) == 0 and r2.new_chunks == 5
    # a small extension of a resident prefix is still saved under pressure
    r3 = t.step(keys(1, 0, 6), 24, 1, 3)
    assert r3.pressure and r3.host_prefix_blocks == 5 and r3.new_chunks == 1 and r3.save
    assert r3.admit == [0, 0, 0, 0, 0, 1]
    # evictions older than the window no longer count: pressure subsides
    r4 = t.step(keys(2, 0, 5), 20, 2, 3 + 60_000)
    assert not r4.pressure and r4.save
    # agents outside the window drop out of A_t (only agent 2 is recent now)
    assert sum(1 for v in t.agent_last.values() if v > 3 + 60_000 - t.window_ms) == 1


def test_conditioned_without_telemetry_uses_estimate_alone():
    b = 4
    keys = lambda a: [(a, j) for j in range(5)]
    t = ot.HostTier(8, b, policy=ot.FILTER_CONDITIONED, kappa_blocks=2, telemetry=False)
    flags = [t.step(keys(a), 20, a, a).pressure for a in range(3)]
    assert flags == [False, False, True]      # third request: 2*20 > 32 although nothing evicted
    assert len(t.order) == 8 or len(t.order) == 10 - 2


def test_length_window_keeps_last_256():
    t = ot.HostTier(4, 4, policy=ot.FILTER_CONDITIONED, len_window=3)
    for i, n in enumerate([100, 200, 300, 400]):
        t.step([], n, 0, i)
    assert list(t.lengths) == [200, 300, 400]


def test_declined_audit_hand_case_and_kappa_sensitivity():
    from oracle import audit
    # positions 1 (key 2) and 2 (key 3) declined, K = 2: key 2 returns after {3, 1} (D = 2 >= K),
    # key 3 never returns: both meet Proposition 1's condition
    a = audit.declined_audit([1, 2, 3, 1, 2, 4, 1], [1, 2], 2)
    assert (a["declined"], a["meets"], a["never_again"], a["ratios"]) == (2, 2, 1, [1.0])
    # with K = 3 the returning chunk is within reach: declining it costs a hit
    a = audit.declined_audit([1, 2, 3, 1, 2, 4, 1], [1, 2], 3)
    assert (a["meets"], a["never_again"]) == (1, 1)
    # brute force on random streams: the condition is "next D >= K or no next reference"
    rng = random.Random(12)
    for _ in range(50):
        s = rand_stream(rng, rng.randrange(2, 50), rng.randrange(2, 9))
        K = rng.randrange(1, 6)
        dec = sorted(rng.sample(range(len(s)), rng.randrange(0, len(s))))
        a = audit.declined_audit(s, dec, K)
        want = 0
        for i in dec:
            later = [j for j in range(i + 1, len(s)) if s[j] == s[i]]
            if not later or len(set(s[i + 1:later[0]]) - {s[i]}) >= K:
                want += 1
        assert a["meets"] == want
    # kappa sensitivity: filtered requests shrink as kappa grows; kappa = infinity filters none
    reqs = [([(a_, j) for j in range(n)], n * 4, a_, t) for t, (a_, n) in
            enumerate([(0, 3), (1, 9), (0, 5), (2, 20), (1, 12), (0, 30), (2, 21)])]
    out = audit.kappa_sensitivity(reqs, 40, 4, [0, 2, 8, 10**9])
    filt = [out[k]["filtered_requests"] for k in (0, 2, 8, 10**9)]
    assert filt == sorted(filt, reverse=True) and filt[-1] == 0 and filt[0] > 0
    assert out[10**9]["declined_chunks"] == 0
    assert audit.median([3, 1, 2]) == 2 and audit.median([4, 1, 2, 3]) == 2.5


def test_gpu_tier_free_order_closed_cases():
    """Pool of 10 blocks, request A = 6 blocks, then request B = 5 blocks: one block of A has to
    go.  Ascending order loses A's first block (nothing of A is a resident prefix any more);
    tail-first order loses A's last block (five of six stay a prefix)."""
    from oracle.trace import GpuTier
    A = [("a", j) for j in range(6)]
    B = [("b", j) for j in range(5)]
    lead = lambda g, ks: next((i for i, k in enumerate(ks) if k not in g), len(ks))
    for order, want in ((0, 0), (1, 5)):
        g = GpuTier(10, order)
        g.step(A, False)
        g.step(B, False)
        assert lead(g, A) == want and lead(g, B) == 5
        assert len(g.order) == 10


def test_gpu_tier_free_order_against_timestamp_brute_force():
    """Brute force with explicit time stamps: a request's block j gets stamp (t, j) in ascending
    order and (t, -j) in tail-first order; the victim is always the smallest stamp."""
    import random
    from oracle.trace import GpuTier
    rng = random.Random(3)
    for order in (0, 1):
        for case in range(40):
            NB = rng.randrange(3, 16)
            g = GpuTier(NB, order)
            stamp = {}
            for t in range(30):
                agent = rng.randrange(3)
                n = rng.randrange(1, NB + 1)
                keys = [(agent, j) for j in range(n)]
                # brute force: residents after the request = its keys plus the newest others
                for j, k in enumerate(keys):
                    stamp[k] = (t, -j if order else j)
                while len(stamp) > NB:
                    del stamp[min(stamp, key=stamp.get)]
                g.step(keys, False)
                assert set(g.order) == set(stamp)
                assert list(g.order) == sorted(stamp, key=stamp.get)


def test_working_set_within_hand_case():
    """Two requests of 4 keys each, alternating: between two references of a key lie the other 7
    keys, so every reuse distance is 7; a tier of 8 recovers everything and smaller tiers nothing:
    both the full working set and the 1 % size are 8; with a GPU prefix covering all of it, nothing
    is left to recover and the size is 0."""
    from oracle import stackdist as sd
    a, b = [1, 2, 3, 4], [5, 6, 7, 8]
    reqs = [a, b, a, b]
    toks = [16, 16, 16, 16]
    assert sd.working_set_full(sd.reuse_distances([k for r in reqs for k in r])) == 8
    assert sd.working_set_within(reqs, toks, [0, 0, 0, 0], 4, percent=1) == 8
    assert sd.working_set_within(reqs, toks, [4, 4, 4, 4], 4, percent=1) == 0
    # half of the benefit is not within 1 % but is within 100 %
    assert sd.working_set_within(reqs, toks, [0, 0, 0, 0], 4, percent=10**6) == 0


# ---- tier reports published at intervals (Appendix D: 1 s report interval, 5 s maximum age) --------
def test_published_reports_hand_case():
    """K_H = 4 chunks of 4 tokens, theta 50 %, kappa 0, reports every 1,000 ms, fresh for 5,000 ms.
    Two agents with 40-token prompts make the estimate (A-1) * sum(len) > K_H * b * count true
    from the second request on."""
    from oracle.tier import FILTER_CONDITIONED, HostTier
    kw = dict(policy=FILTER_CONDITIONED, kappa_blocks=0, theta_percent=50, window_ms=60_000)
    t = HostTier(4, 4, telemetry_period_ms=1000, telemetry_max_age_ms=5000, **kw)
    sync = HostTier(4, 4, **kw)
    # 100 ms: first request; one agent, estimate false -> saved, the tier is full afterwards
    for x in (t, sync):
        r = x.step([1, 2, 3, 4], 40, agent=0, now_ms=100)
        assert r.save and not r.pressure
    # 200 ms: no report has been published yet (the first one comes at 1,000 ms): p_t is
    # the working-set test by itself, and it says pressure.  Read synchronously, the tier is full but has not
    # evicted anything, so there is no pressure.
    r = t.step([5, 6], 40, agent=1, now_ms=200)
    assert r.pressure and not r.save and r.admit == [0, 0] and t.report is None
    assert not sync.step([5, 6], 40, agent=1, now_ms=200).pressure          # (it stores 5, 6, evicting 1, 2)
    # 1,500 ms: the report of 1,000 ms says 4 registered chunks, no evictions -> no pressure
    r = t.step([5, 6], 40, agent=1, now_ms=1500)
    assert t.report == (1000, 4, 0) and not r.pressure and r.save
    assert r.evicted == [(1, 0), (2, 1)]                                     # evictions at 1,500 ms
    # 1,900 ms: 0.4 s after those evictions the latest report is still the one of 1,000 ms
    r = t.step([1, 2], 40, agent=0, now_ms=1900)
    assert t.report == (1000, 4, 0) and not r.pressure and r.save and len(r.evicted) == 2
    # 2,100 ms: the report of 2,000 ms counts the four evictions -> full and evicting -> pressure
    r = t.step([7], 40, agent=1, now_ms=2100)
    assert t.report == (2000, 4, 4) and r.pressure and not r.save
    # a request exactly at a publication time reads that report, which does not yet see what the
    # request itself (or another request of the same millisecond) does
    r = t.step([8], 4, agent=1, now_ms=3000)
    assert t.report == (3000, 4, 4)
    # the eviction window of a report is (t - 60 s, t): the report of 61,000 ms still counts the
    # evictions of 1,500 and 1,900 ms, the report of 62,000 ms none of them
    t.step([1], 4, agent=0, now_ms=61_400)
    assert t.report == (61_000, 4, 4)
    t.step([1], 4, agent=0, now_ms=62_000)
    assert t.report == (62_000, 4, 0)


def test_stale_report_falls_back_to_the_estimate():
    """Reports every 10 s, fresh for 5 s; K_H * b = 16 tokens.  The report of 10,000 ms says
    "3 of 4 chunks, no evictions", i.e. no pressure whatever the estimate says."""
    from oracle.tier import FILTER_CONDITIONED, HostTier
    kw = dict(policy=FILTER_CONDITIONED, kappa_blocks=0, theta_percent=50, window_ms=600_000)
    t = HostTier(4, 4, telemetry_period_ms=10_000, telemetry_max_age_ms=5_000, **kw)
    assert t.step([1, 2, 3], 12, agent=0, now_ms=100).save              # one agent: estimate false
    # 12,000 ms: the report is 2 s old, fresh.  Estimate (2-1) * (12+100) = 112 > 16 * 2 is true,
    # the tier is full (75 % >= 50 %) but the report shows no eviction: no pressure, saved
    r = t.step([4], 100, agent=1, now_ms=12_000)
    assert t.report == (10_000, 3, 0) and not r.pressure and r.save
    # 16,500 ms: the same report is 6.5 s old and no newer one exists (the next comes at 20,000 ms):
    # not fresh, so p_t is the working-set test only: (2-1) * 212 > 16 * 3 -> pressure, declined
    r = t.step([5], 100, agent=0, now_ms=16_500)
    assert t.report == (10_000, 3, 0) and r.pressure and not r.save and r.new_chunks == 25
    # with no age limit the old report is still used: no pressure
    t3 = HostTier(4, 4, telemetry_period_ms=10_000, telemetry_max_age_ms=0, **kw)
    t3.step([1, 2, 3], 12, agent=0, now_ms=100)
    t3.step([4], 100, agent=1, now_ms=12_000)
    assert not t3.step([5], 100, agent=0, now_ms=16_500).pressure
    # a stale report and an estimate that says no: no pressure (window of one prompt length)
    t2 = HostTier(4, 4, telemetry_period_ms=10_000, telemetry_max_age_ms=5_000, len_window=1, **kw)
    t2.step([1, 2, 3], 12, agent=0, now_ms=100)
    assert not t2.step([4], 100, agent=1, now_ms=12_000).pressure       # fresh report without evictions
    assert not t2.step([5], 4, agent=0, now_ms=16_500).pressure         # stale; (2-1) * 4 <= 16
    assert t2.step([6], 100, agent=0, now_ms=16_600).pressure           # stale; (2-1) * 100 > 16
    # at 20,000 ms the next report appears and is read again
    t2.step([7], 100, agent=1, now_ms=20_000)
    assert t2.report[0] == 20_000


def test_reports_every_millisecond_equal_the_synchronous_reading():
    """With a report every millisecond and requests at distinct times the latest report is the tier
    as the request finds it, so the decisions must be those of the synchronous reading (which has
    its own hand-computed pins above)."""
    import random as _random
    from oracle.tier import FILTER_CONDITIONED, HostTier
    rng = _random.Random(17)
    for case in range(20):
        kw = dict(policy=FILTER_CONDITIONED, kappa_blocks=rng.randrange(0, 4), theta_percent=rng.choice([50, 95]),
                  window_ms=rng.choice([30, 200]), len_window=rng.choice([4, 64]))
        a = HostTier(12, 4, **kw)
        c = HostTier(12, 4, telemetry_period_ms=1, telemetry_max_age_ms=5, **kw)
        now = 0
        engaged = 0
        for i in range(300):
            now += rng.randrange(1, 9)
            start = rng.randrange(6) * 20
            keys = [start + j for j in range(rng.randrange(0, 10))]
            n_tok = 4 * len(keys) + rng.randrange(4)
            agent = rng.randrange(4)
            ra, rc = a.step(keys, n_tok, agent, now), c.step(keys, n_tok, agent, now)
            assert (ra.pressure, ra.save, ra.hit, ra.admit, ra.slot, ra.evicted) == \
                   (rc.pressure, rc.save, rc.hit, rc.admit, rc.slot, rc.evicted)
            engaged += ra.pressure
        assert engaged > 0
