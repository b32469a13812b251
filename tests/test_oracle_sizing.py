"""Pins for oracle.sizing and oracle.match against values the paper prints."""
import math

from oracle import match as om
from oracle import sizing as sz

GIB = 1 << 30
KIB = 1 << 10


def test_footprints_table(golden):
    g = golden("paper_constants.txt")
    assert sz.beta_rank(48, 128, 2, 4, 1) == int(g["qwen3_bytes_per_token_unsharded"])
    assert sz.beta_rank(64, 128, 2, 8, 1) == int(g["qwen25_bytes_per_token_unsharded"])
    for tp in (1, 2, 4, 8):
        assert sz.beta_rank(48, 128, 2, 4, tp) == int(g[f"qwen3_kib_rank_tp{tp}"]) * KIB
        assert sz.beta_rank(64, 128, 2, 8, tp) == int(g[f"qwen25_kib_rank_tp{tp}"]) * KIB
    assert 8 * sz.beta_rank(48, 128, 2, 4, 8) == int(g["qwen3_aggregate_kib_tp8"]) * KIB


def test_working_set_scale_and_pressure(golden):
    g = golden("paper_constants.txt")
    beta = sz.beta_rank(48, 128, 2, 4, 8)
    nbar = int(g["mean_prompt_tokens"])
    ws16 = sz.working_set_bytes(16, nbar, beta)
    ws8 = sz.working_set_bytes(8, nbar, beta)
    assert round(ws16 / GIB, 1) == float(g["ws_gib_a16"])
    assert round(ws8 / GIB, 1) == float(g["ws_gib_a8"])
    assert round(sz.working_set_bytes(64, 64 * 1024, beta) / GIB, 1) == float(g["ws_gib_64x64k"])
    assert round(sz.working_set_bytes(128, 128 * 1024, beta) / GIB) == float(g["ws_gib_128x128k"])
    assert round(sz.gamma_g(16, nbar, int(g["gpu_kv_tokens_h20"])), 2) == float(g["gamma_g_a16"])
    assert round(sz.gamma_h(ws16, 5 * GIB), 1) == float(g["gamma_h_5gib"])
    assert round(sz.gamma_h(ws16, 10 * GIB), 1) == float(g["gamma_h_10gib"])
    assert round(sz.gamma_h(ws16, 20 * GIB), 2) == float(g["gamma_h_20gib"])


def test_tier_chunks(golden):
    g = golden("paper_constants.txt")
    beta = sz.beta_rank(48, 128, 2, 4, 8)
    assert 1024 * beta == 24 << 20
    assert sz.tier_chunks(5 * GIB, 1024, beta) == int(g["kh_5gib"])
    assert sz.tier_chunks(10 * GIB, 1024, beta) == int(g["kh_10gib"])
    assert sz.tier_chunks(40 * GIB, 1024, beta) == int(g["kh_40gib"])


def test_obr_bound(golden):
    g = golden("paper_constants.txt")
    beta = sz.beta_rank(48, 128, 2, 4, 8)
    bw = float(g["restore_gib_per_s"]) * GIB
    us = sz.load_time(1, beta, bw) * 1e6
    assert round(us, 2) == float(g["restore_us_per_token"])
    t_pf = 6.6e9 / (8 * 148e12)          # 6.6 GFLOP/token over eight 148-TFLOPS GPUs
    assert round(t_pf * 1e6, 1) == float(g["prefill_us_per_token_bound"])
    big = sz.obr(10**9, t_pf, beta, bw)
    assert big > float(g["obr_lower_bound"])
    assert math.isclose(big, 1 - 0.86 / 5.6, abs_tol=0.01)
    # a fixed overhead lowers OBR for short prefixes and is amortised for long ones
    assert sz.obr(16, t_pf, beta, bw, tau_load=1e-4) < sz.obr(10**6, t_pf, beta, bw, tau_load=1e-4) < big


def test_fold_example(golden):
    g = golden("paper_constants.txt")
    assert om.fresh_prefill(int(g["fold_submitted_a"]), int(g["fold_stable_a"])) == int(g["fold_fresh_a"])
    assert om.fresh_prefill(int(g["fold_submitted_b"]), int(g["fold_stable_b"])) == int(g["fold_fresh_b"])
    # the same numbers through the block-level coverage with b = 1000 "omitting rounding"
    assert om.fresh_tokens(51000, 1000, G=50, H=0) == 1000
    assert om.fresh_tokens(20000, 1000, G=0, H=2) == 18000


def test_match_stops_at_first_absent_block():
    keys = [10, 11, 12, 13, 14]
    assert om.match(keys, {10, 11}, {10, 11, 12, 14}) == (2, 3)      # isolated 14 ignored
    assert om.match(keys, set(), set()) == (0, 0)
    assert om.match(keys, set(keys), {10}) == (5, 1)
    assert om.restore_run(2, 3) == (2, 3)
    assert om.restore_run(5, 1) == (5, 5)
    assert om.fresh_tokens(5 * 16 + 3, 16, 2, 3) == 5 * 16 + 3 - 48


def test_match_brute_force():
    import random
    rng = random.Random(0)
    for _ in range(200):
        n = rng.randrange(0, 12)
        keys = rng.sample(range(100), n)
        gpu = {k for k in keys if rng.random() < 0.7}
        host = {k for k in keys if rng.random() < 0.7}
        G = next((i for i, k in enumerate(keys) if k not in gpu), n)
        H = next((i for i, k in enumerate(keys) if k not in host), n)
        assert om.match(keys, gpu, host) == (G, H)
