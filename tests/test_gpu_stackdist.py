"""GPU parity of the stack-distance capacity model (eakv_reuse_distances, eakv_capacity_curve)
against oracle.stackdist: reuse distances, Mattson hits, prefix coverage, restored blocks and
computed prefill per capacity, all integers and bit-exact."""
import math

import numpy as np
import pytest

from eakv_workloads import CONFIGS, SHAPES, make_trace
from oracle import stackdist as sd
from oracle.trace import TraceOracle

from gpu_util import require_gpu, torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def gpu_distances(stream_keys):
    from paper_2609_33762_b200 import eakv
    keys = np.asarray(stream_keys, dtype=np.uint64)
    dev = torch.from_numpy(keys.view(np.int64)).cuda()
    out = torch.full((max(len(keys), 1) + 1,), -7, dtype=torch.int64, device="cuda")
    eakv.eakv_reuse_distances(dev.data_ptr(), len(keys), out.data_ptr())
    res = out.cpu().numpy()
    assert res[len(keys)] == -7
    return res[:len(keys)], out


def as_oracle(dist):
    return [math.inf if d < 0 else int(d) for d in dist]


def test_hand_case_and_tiny_streams():
    got, _ = gpu_distances([1, 2, 3, 1, 2, 2, 4, 3, 1])
    assert as_oracle(got) == [math.inf, math.inf, math.inf, 2, 2, 0, math.inf, 3, 3]
    for s in ([], [5], [5, 5], [5, 6, 5], [7] * 10, list(range(10)), [1, 2] * 8):
        got, _ = gpu_distances(s)
        assert as_oracle(got) == sd.reuse_distances_definition(s)


@pytest.mark.parametrize("T,U", [(1000, 7), (1023, 50), (1024, 300), (1025, 1000), (5000, 40),
                                 (40000, 3000), (70000, 70000), (65536, 2)])
def test_random_streams(T, U):
    rng = np.random.default_rng(T + U)
    universe = rng.integers(0, 1 << 61, size=U, dtype=np.uint64)      # full-width keys
    idx = rng.integers(0, U, size=T)
    if T > 2000:                                   # make it bursty: long runs and far re-references
        idx = np.sort(idx.reshape(-1, 8), axis=1).reshape(-1)[:T]
    stream = universe[idx]
    got, _ = gpu_distances(stream)
    assert as_oracle(got) == sd.reuse_distances(stream.tolist())


def test_capacity_curve_on_config0():
    from paper_2609_33762_b200 import eakv
    cfg = CONFIGS["c0_big_tier"]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg)
    oracle = TraceOracle(shape, cfg.gpu_blocks, cfg.host_blocks)
    recs = oracle.run(trace)
    req_keys = [r["keys"] for r in recs]
    n_tok = [r["n_tokens"] for r in recs]
    G = [r["G"] for r in recs]
    stream = [k for ks in req_keys for k in ks]
    offsets = np.concatenate([[0], np.cumsum([len(k) for k in req_keys])])
    dist, dist_dev = gpu_distances(stream)
    assert as_oracle(dist) == sd.reuse_distances(stream)
    caps = [1, 16, 100, 256, 1024, 5000, 10**9]
    out = eakv.eakv_capacity_curve(dist_dev.data_ptr(), len(stream), offsets, n_tok, G,
                                   shape.block_size, caps, want_cover=True)
    for c, K in enumerate(caps):
        want = sd.predict_trace(req_keys, n_tok, G, K, shape.block_size)
        assert out["hits"][c] == sum(want["hit_flags"])
        assert out["cover"][c].tolist() == want["host_cover"]
        assert out["restored_blocks"][c] == want["restored_blocks"]
        assert out["computed_tokens"][c] == want["computed_tokens"]
    # the model at the configured capacity equals what the simulated tier did (Mattson)
    c = caps.index(1024)
    assert out["cover"][c].tolist() == [r["H"] for r in recs]
    assert out["restored_blocks"][c] == oracle.totals["loaded_blocks"]
    assert out["computed_tokens"][c] == oracle.totals["fresh_tokens"]
    assert np.all(np.diff(out["hits"]) >= 0)             # hits are monotone in capacity
    # smallest tier within 1 % (and 10 %) of the unbounded tier's computed prefill: GPU narrowing
    # against the oracle's plain scan over every capacity
    ws_full = sd.working_set_full(sd.reuse_distances(stream))
    for pct in (0, 1, 10):
        full, within = eakv.eakv_working_set_sizes(dist_dev.data_ptr(), len(stream), offsets, n_tok, G,
                                                   shape.block_size, pct)
        assert full == ws_full
        assert within == sd.working_set_within(req_keys, n_tok, G, shape.block_size, percent=pct)


def test_config3_prefix_distances_and_product_tier_agree():
    """627k references of the config 2/3 trace: distances against the oracle, and the hit
    count at the 32 GiB capacity against the library's own tier bookkeeping (write-all)."""
    from paper_2609_33762_b200 import eakv
    cfg = CONFIGS["c3"]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg)
    oracle = TraceOracle(shape, cfg.gpu_blocks, cfg.host_blocks)
    recs = oracle.run(trace, limit=400)
    stream = [k for r in recs for k in r["keys"]]
    dist, dist_dev = gpu_distances(stream)
    assert as_oracle(dist) == sd.reuse_distances(stream)
    offsets = np.concatenate([[0], np.cumsum([len(r["keys"]) for r in recs])])
    out = eakv.eakv_capacity_curve(dist_dev.data_ptr(), len(stream), offsets,
                                   [r["n_tokens"] for r in recs], [r["G"] for r in recs],
                                   shape.block_size, [cfg.host_blocks, 10**9], want_cover=True)
    assert out["hits"][0] == oracle.host.stats["hits"]
    assert out["cover"][0].tolist() == [r["H"] for r in recs]
    assert out["computed_tokens"][0] == oracle.totals["fresh_tokens"]
    ctx = eakv.Context(num_layers=1, kv_heads=1, head_dim=8, block_size=shape.block_size,
                       gpu_blocks=8, host_blocks=cfg.host_blocks, kv_base=None, control_plane_only=True)
    for r in recs:
        ctx.eakv_tier_step(np.asarray(r["keys"], dtype=np.uint64), r["agent"], r["n_tokens"], r["now_ms"])
    assert ctx.eakv_get_stats()["hits"] == out["hits"][0]
    ctx.close()


def test_argument_errors():
    from paper_2609_33762_b200 import eakv
    d = torch.zeros(4, dtype=torch.int64, device="cuda")
    with pytest.raises(eakv.EakvError):
        eakv.eakv_reuse_distances(0, 4, d.data_ptr())
    with pytest.raises(eakv.EakvError):                      # offsets do not end at n_refs
        eakv.eakv_capacity_curve(d.data_ptr(), 4, [0, 3], [48], [0], 16, [4])
    with pytest.raises(eakv.EakvError):                      # too many capacities
        eakv.eakv_capacity_curve(d.data_ptr(), 4, [0, 4], [64], [0], 16, list(range(1, 70)))


@pytest.mark.parametrize("T,U,K", [(1, 1, 1), (50, 5, 3), (3000, 200, 64), (40_000, 3000, 500), (20_000, 50, 10)])
def test_declined_audit_entry_point_on_random_streams(T, U, K):
    """eakv_declined_audit against the oracle's definition-level audit: random reference streams,
    random sets of declined positions; the three counts and, per declined position, the reuse
    distance of the chunk's next reference."""
    from oracle import audit as oaudit
    from paper_2609_33762_b200 import eakv
    rng = np.random.default_rng(T + U)
    stream = rng.integers(1, U + 1, size=T, dtype=np.int64)
    mask = (rng.random(T) < 0.3).astype(np.uint8)
    declined = np.nonzero(mask)[0].tolist()
    want = oaudit.declined_audit(stream.tolist(), declined, K)
    kd = torch.from_numpy(stream).cuda()
    md = torch.from_numpy(mask).cuda()
    nd = torch.full((T + 1,), 7, dtype=torch.int64, device="cuda")
    got = eakv.eakv_declined_audit(kd.data_ptr(), md.data_ptr(), T, K, nd.data_ptr())
    assert got == (want["declined"], want["meets"], want["never_again"])
    nd = nd.cpu().numpy()
    assert nd[T] == 7                                                  # nothing written past the end
    assert ((nd[:T] == -2) == (mask == 0)).all()
    assert int((nd[:T] == -1).sum()) == want["never_again"]
    again = nd[:T][nd[:T] >= 0]
    assert sorted((again / K).tolist()) == sorted(want["ratios"])
    # without the per-reference output, and an empty stream
    assert eakv.eakv_declined_audit(kd.data_ptr(), md.data_ptr(), T, K) == got
    assert eakv.eakv_declined_audit(0, 0, 0, K) == (0, 0, 0)


def test_declined_chunk_audit_matches_oracle():
    """The audit of declined writes (next reuse distance >= K_H or never again) on a scaled
    config-2 trace under both filters, against the oracle's definition-level audit."""
    from dataclasses import replace
    import eakv_workloads
    from oracle import audit as oaudit
    from oracle import hash as ohash
    from oracle.tier import HostTier
    from paper_2609_33762_b200 import capacity
    small = replace(CONFIGS["c2"], shape="tiny", agents=6, turns=12, first_prompt=400,
                    append_median=150.0, context_cap=3000, tool_gap_mean_ms=15_000.0, kappa_blocks=4)
    eakv_workloads.CONFIGS["_audit"] = small
    try:
        shape = SHAPES["tiny"]
        trace = make_trace(small)
        kh = 300
        gib = kh * shape.block_bytes / (1 << 30)
        for policy, pol_id in (("fixed", 1), ("conditioned", 2)):
            got = capacity.audit("_audit", policy, gib)
            tier = HostTier(kh, shape.block_size, pol_id, small.kappa_blocks)
            stream, declined = [], []
            for r in trace.requests:
                keys = ohash.hash_blocks(trace.prompt(r).tolist(), shape.block_size)
                res = tier.step(keys, r.n_tokens, r.agent, r.time_ms)
                for k, h, a in zip(keys, res.hit, res.admit):
                    if not h and not a:
                        declined.append(len(stream))
                    stream.append(k)
            want = oaudit.declined_audit(stream, declined, kh)
            assert got["tier_units"] == kh
            assert got["declined_chunks"] == want["declined"] > 0
            assert got["meet_condition"] == want["meets"]
            assert got["never_referenced_again"] == want["never_again"]
            assert got["declined_requests"] == tier.stats["declined_requests"]
    finally:
        del eakv_workloads.CONFIGS["_audit"]
