"""Host logic of the replay and capacity drivers that needs no GPU: tier sizing by the
working-set scale (Eq. 5) agrees with the oracle's arithmetic, and the plan honours the
configuration, explicit requests and the host-memory cap."""
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
