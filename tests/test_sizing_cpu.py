"""Host logic of the replay and capacity drivers that needs no GPU: tier sizing by the
working-set scale (Eq. 5) agrees with the oracle's arithmetic, and the plan honours the
configuration, explicit requests and the host-memory cap."""
import pytest

from eakv_workloads import CONFIGS, SHAPES, make_trace
from oracle import sizing
from paper_2609_33762_b200 import replay


def test_working_set_blocks_matches_oracle_arithmetic():
    for name in ("c0", "c2", "c4"):
        cfg = CONFIGS[name]
        shape = SHAPES[cfg.shape]
        trace = make_trace(cfg)
        beta = sizing.beta_rank(shape.num_layers, shape.head_dim, shape.elem_bytes, shape.kv_heads)
        assert beta == shape.bytes_per_token
        n_mean = trace.total_prompt_tokens / len(trace.requests)
        ws = sizing.working_set_bytes(cfg.agents, n_mean, beta)
        assert replay.working_set_blocks(trace, shape) == int(ws // shape.block_bytes)


def test_plan_sources(monkeypatch):
    cfg2, cfg3 = CONFIGS["c2"], CONFIGS["c3"]
    shape = SHAPES[cfg2.shape]
    trace = make_trace(cfg2, agents=4, turns=3)
    monkeypatch.setattr(replay, "mem_available_bytes", lambda: 0)          # no cap known
    kh, why = replay.plan(cfg3, trace, shape)
    assert kh == cfg3.host_blocks == (32 << 30) // shape.block_bytes and "configuration" in why
    kh, why = replay.plan(cfg2, trace, shape)
    assert kh == replay.working_set_blocks(trace, shape) and "working-set" in why
    kh, why = replay.plan(cfg2, trace, shape, host_gib=3)
    assert kh == (3 << 30) // shape.block_bytes and "requested" in why
    # a data-plane run is capped by what the host can pin; a bookkeeping run is not
    monkeypatch.setattr(replay, "mem_available_bytes", lambda: 10 << 30)
    kh, why = replay.plan(cfg3, trace, shape)
    assert kh == int((10 << 30) * 0.6 // shape.block_bytes) and "capped" in why
    kh, _ = replay.plan(cfg3, trace, shape, data_plane=False)
    assert kh == cfg3.host_blocks


def test_eakv_working_set_against_oracle_sizing_and_the_papers_printed_values():
    """eakv_working_set (Eq. 1, Eq. 5, gamma_G, gamma_H in integers) against oracle.sizing evaluated
    in exact fractions, and on the paper's own H20 numbers (Section 3.2, Appendix C)."""
    import random
    from fractions import Fraction
    from paper_2609_33762_b200 import eakv
    # the paper: 4,427 requests with 147,124,984 prompt tokens, A = 16, Qwen3 at TP8 (24 KiB per
    # token per rank), GPU KV capacity 343,408 tokens, host tier 5 GiB in 1,024-token chunks (213)
    out = eakv.eakv_working_set(num_layers=48, kv_heads=4, head_dim=128, tensor_parallel=8, block_size=1024,
                                active_pool=16, total_prompt_tokens=147_124_984, n_requests=4427,
                                gpu_blocks=335, host_blocks=213)
    assert out["beta_rank_bytes"] == 24 * 1024
    assert abs(out["working_set_bytes"] / 2**30 - 11.4) < 0.05                 # "11.4 GiB per rank"
    assert abs(out["gamma_h"] - 2.3) < 0.05 and out["working_set_exceeds_host"] == 1
    assert abs(out["gamma_g"] - 16 * 33_234 / (335 * 1024)) < 0.01 and out["pool_exceeds_gpu"] == 1
    a8 = eakv.eakv_working_set(num_layers=48, kv_heads=4, head_dim=128, tensor_parallel=8, block_size=1024,
                               active_pool=8, total_prompt_tokens=147_124_984, n_requests=4427, host_blocks=853)
    assert abs(a8["working_set_bytes"] / 2**30 - 5.3) < 0.05                   # "5.3 GiB" at A = 8
    assert a8["working_set_exceeds_host"] == 0                                 # a 20 GiB tier holds it
    rng = random.Random(8)
    for _ in range(300):
        L, H, d, s = rng.randrange(1, 80), rng.randrange(1, 33), rng.choice([64, 128]), rng.choice([1, 2, 4])
        tp, b = rng.choice([1, 2, 4, 8, 16]), rng.choice([1, 16, 32, 1024])
        A, n = rng.randrange(1, 300), rng.randrange(1, 10**5)
        total = rng.randrange(0, 10**12)
        kg, kh = rng.randrange(0, 10**6), rng.randrange(0, 10**6)
        got = eakv.eakv_working_set(num_layers=L, kv_heads=H, head_dim=d, elem_bytes=s, tensor_parallel=tp,
                                    block_size=b, active_pool=A, total_prompt_tokens=total, n_requests=n,
                                    gpu_blocks=kg, host_blocks=kh)
        beta = sizing.beta_rank(L, d, s, H, tp)
        n_bar = Fraction(total, n)
        ws = sizing.working_set_bytes(A, n_bar, beta)
        assert got["beta_rank_bytes"] == beta
        assert got["working_set_bytes"] == ws.numerator // ws.denominator
        assert got["working_set_blocks"] == sizing.tier_chunks(ws, b, beta).__floor__()
        if kg:
            g = sizing.gamma_g(A, n_bar, kg * b)
            assert abs(got["gamma_g"] - float(g)) <= 1e-12 * max(1.0, float(g)) and got["pool_exceeds_gpu"] == (g > 1)
        if kh:
            h = sizing.gamma_h(ws, kh * b * beta)
            assert abs(got["gamma_h"] - float(h)) <= 1e-12 * max(1.0, float(h))
            assert got["working_set_exceeds_host"] == (h > 1)
    import pytest
    with pytest.raises(eakv.EakvError):
        eakv.eakv_working_set(num_layers=0, kv_heads=1, head_dim=8, block_size=16, active_pool=2,
                              total_prompt_tokens=10, n_requests=1)


def test_eakv_offload_benefit_against_the_oracle_and_the_papers_ratio():
    """Eq. 2 in the library (integers, picoseconds) against oracle.sizing.obr / load_time, on the
    paper's own deployment (24 KiB per token and rank, 26.6 GiB/s: 0.86 us of restore per token
    against 5.6 us of prefill, OBR > 0.84) and on random inputs; the break-even length is the first
    n at which the restore is not slower."""
    import math
    import random
    from oracle import sizing as sz
    from paper_2609_33762_b200 import build, eakv
    build.build()
    GIB = 1 << 30
    beta = sz.beta_rank(48, 128, 2, 4, 8)
    bw = int(26.6 * GIB)
    t_pf_ps = round(6.6e9 / (8 * 148e12) * 1e12)
    o = eakv.eakv_offload_benefit(prefix_tokens=10**9, beta_rank_bytes=beta, t_prefill_ps=t_pf_ps, h2d_bytes_per_s=bw)
    assert round(o["t_load_ps"] / 10**9 / 1e6, 2) == 0.86 and round(t_pf_ps / 1e6, 1) == 5.6
    assert o["obr"] > 0.84 and math.isclose(o["obr"], 1 - 0.86 / 5.6, abs_tol=0.01)
    assert math.isclose(o["obr_long_prefix"], o["obr"], abs_tol=1e-9) and o["break_even_tokens"] == 0
    rng = random.Random(4)
    for _ in range(200):
        n = rng.randrange(1, 200_000)
        b_ = rng.randrange(1 << 10, 1 << 19)
        t = rng.randrange(100_000, 20_000_000)
        w = rng.randrange(1 << 30, 1 << 37)
        tau = rng.randrange(0, 400_000_000)
        o = eakv.eakv_offload_benefit(prefix_tokens=n, beta_rank_bytes=b_, t_prefill_ps=t, h2d_bytes_per_s=w, tau_load_ps=tau)
        want = sz.obr(n, t * 1e-12, b_, w, tau_load=tau * 1e-12)
        assert math.isclose(o["obr"], want, rel_tol=1e-9, abs_tol=1e-9)
        assert math.isclose(o["t_load_ps"], sz.load_time(n, b_, w, tau * 1e-12) * 1e12, rel_tol=1e-9, abs_tol=1.0)
        assert o["restore_is_faster"] == (o["t_load_ps"] < o["t_rec_ps"]) or abs(o["t_load_ps"] - o["t_rec_ps"]) <= 1
        ne = o["break_even_tokens"]
        gain = t * w - b_ * 10**12                     # per token, times B_H2D
        if gain <= 0:
            assert ne == -1
        else:
            assert ne * gain >= tau * w and (ne == 0 or (ne - 1) * gain < tau * w)
    with pytest.raises(eakv.EakvError):
        eakv.eakv_offload_benefit(prefix_tokens=0, beta_rank_bytes=1, t_prefill_ps=1, h2d_bytes_per_s=1)
