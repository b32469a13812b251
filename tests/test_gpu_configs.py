"""GPU parity on the larger configurations (2, 3 and 4): every per-request output of the
control plane against the oracle on the configuration's own trace and KV shape, and the KV
bytes of sampled resident blocks on a data-plane prefix of each trace."""
import gc

import numpy as np
import pytest

from eakv_workloads import CONFIGS, SHAPES, key_words_numpy, key_words_torch, make_trace
from oracle import sizing
from oracle.trace import TraceOracle

from gpu_util import require_gpu, torch

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _gpu_and_clean():
    require_gpu()
    gc.collect()
    torch.cuda.empty_cache()
    yield
    gc.collect()
    torch.cuda.empty_cache()


def compare_records_fast(got, want):
    assert len(got) == len(want)
    for i, (g, w) in enumerate(zip(got, want)):
        assert np.array_equal(np.asarray(g["keys"], dtype=np.uint64), np.asarray(w["keys"], dtype=np.uint64)), i
        for f in ("n_tokens", "G", "H", "new_chunks", "pressure", "save", "loaded", "stored",
                  "fresh_tokens", "filled"):
            assert g[f] == w[f], (i, f)
        for f in ("hit", "admit", "slot", "gpu_resident", "gpu_block"):
            assert np.array_equal(np.asarray(g[f], dtype=np.int64), np.asarray(w[f], dtype=np.int64)), (i, f)
        assert [(int(k), int(s)) for k, s in g["evicted"]] == w["evicted"], i


def eq5_blocks(trace, shape):
    beta = sizing.beta_rank(shape.num_layers, shape.head_dim, shape.elem_bytes, shape.kv_heads)
    n_mean = trace.total_prompt_tokens / len(trace.requests)
    ws = sizing.working_set_bytes(len(trace.agent_tokens), n_mean, beta)
    return int(ws // (shape.block_size * beta))


def run_both(cfg_name, *, policy, host_blocks, limit=None, data_plane=False, link=1, chunk_blocks=1, native=False):
    from paper_2609_33762_b200.harness import AgentServer
    cfg = CONFIGS[cfg_name]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg)
    kw = dict(policy=policy, kappa_blocks=cfg.kappa_blocks)
    if chunk_blocks > 1:
        kw["chunk_blocks"] = chunk_blocks
    oracle = TraceOracle(shape, cfg.gpu_blocks, host_blocks, **kw)
    oracle.run(trace, limit=limit)
    payload = (lambda keys, q, n: key_words_torch(keys.astype(np.int64), q, n, "cuda")) if data_plane else None
    server = AgentServer(shape, cfg.gpu_blocks, host_blocks, payload, data_plane=data_plane, native_turn=native,
                         incremental_hash=True, link_strategy=link, **kw)
    server.run(trace, limit=limit)
    compare_records_fast(server.records, oracle.records)
    assert server.totals == oracle.totals
    return server, oracle, shape, trace


def check_sampled_bytes(server, oracle, shape, n=48):
    """Resident blocks named by the oracle's indices must hold their key's payload."""
    server.ctx.eakv_sync()
    W = shape.piece_bytes // 2
    rng = np.random.default_rng(5)
    gpu = list(oracle.gpu.order.items())
    host = list(oracle.host.order.items())
    for items, kind in ((gpu, "gpu"), (host, "host")):
        if not items:
            continue
        pick = [items[i] for i in rng.choice(len(items), size=min(n, len(items)), replace=False)]
        keys = np.array([k for k, _ in pick], dtype=np.uint64)
        where = np.array([s for _, s in pick], dtype=np.int64)
        for q in (0, shape.pieces_per_block // 2, shape.pieces_per_block - 1):
            want = key_words_numpy(keys, q, W)
            if kind == "gpu":
                got = server.pool.pieces[q][torch.as_tensor(where, device="cuda")].cpu().numpy().view(np.uint16)
            else:
                got = server.ctx.tier_host_view()[where, q].view(np.uint16)
            assert np.array_equal(got, want), (kind, q)


def test_config2_full_trace_control_plane():
    """Write-all, tier capacity = the Eq. 5 working-set size, all 1,280 requests."""
    from paper_2609_33762_b200 import replay
    cfg = CONFIGS["c2"]
    shape = SHAPES[cfg.shape]
    trace = make_trace(cfg)
    kh = eq5_blocks(trace, shape)
    assert replay.working_set_blocks(trace, shape) == kh       # the product sizes the tier alike
    server, oracle, *_ = run_both("c2", policy=0, host_blocks=kh)
    assert oracle.host.stats["evicted"] == 0 or kh < oracle.host.stats["admitted"]
    server.close()


@pytest.mark.parametrize("policy,limit", [(2, None), (0, 500), (1, 200)])
def test_config3_policies_control_plane(policy, limit):
    """Fixed 32 GiB tier: conditioned admission on the full trace; write-all and the fixed
    filter (which declines every request of this trace) on a prefix."""
    cfg = CONFIGS["c3"]
    # the conditioned run goes through the library's turn engine (bookkeeping-only context fed with the
    # GPU's keys), the other two through the single calls
    server, oracle, *_ = run_both("c3", policy=policy, host_blocks=cfg.host_blocks, limit=limit, native=policy == 2)
    st = oracle.host.stats
    if policy == 2:
        assert 0 < st["declined_requests"] < st["requests"] and st["pressure_requests"] > 0
    if policy == 1:
        assert st["admitted"] == 0 and st["declined_requests"] == st["requests"]
    server.close()


@pytest.mark.parametrize("host_gib,limit", [(64, 1000), (512, 700)])
def test_config4_prefix_control_plane(host_gib, limit):
    """128 agents, Llama-3-8B shape, block 32, the two ends of the 64-512 GiB tier sweep
    (bookkeeping only, so no pinned memory of that size is needed): a prefix of the trace."""
    shape = SHAPES["llama3_8b"]
    kh = (host_gib << 30) // shape.block_bytes
    server, oracle, *_ = run_both("c4", policy=0, host_blocks=kh, limit=limit)
    server.close()


def test_config3_data_plane_prefix():
    """First 120 requests of the config 2/3 trace with KV bytes moving through the staged
    host link; sampled resident blocks on both tiers hold exactly their payload."""
    cfg = CONFIGS["c3"]
    kh = 8192                                             # 12 GiB of pinned tier
    server, oracle, shape, _ = run_both("c3", policy=2, host_blocks=kh, limit=120, data_plane=True)
    assert oracle.totals["loaded_blocks"] > 0 and oracle.totals["stored_blocks"] > 0
    check_sampled_bytes(server, oracle, shape)
    server.close()


def test_config4_data_plane_prefix():
    """First 60 requests of config 4 (4 MiB blocks, 64-KiB pieces) through the zero-copy link."""
    kh = 4096                                             # 16 GiB of pinned tier
    server, oracle, shape, _ = run_both("c4", policy=0, host_blocks=kh, limit=60, data_plane=True, link=0)
    assert oracle.totals["stored_blocks"] > 0
    check_sampled_bytes(server, oracle, shape)
    server.close()


def test_config3_paper_granularity_control_plane():
    """The paper's own granularities on config 3's trace: 1,024-token host chunks (64 blocks of
    16 tokens), a 32 GiB tier = 341 chunks of 96 MiB, kappa = 8 chunks, conditioned admission."""
    from dataclasses import replace
    cfg = CONFIGS["c3"]
    shape = SHAPES[cfg.shape]
    R = 64
    kh = (32 << 30) // (R * shape.block_bytes)
    assert kh == 341
    import eakv_workloads
    old = eakv_workloads.CONFIGS["c3"]
    try:
        CONFIGS["c3"] = replace(old, kappa_blocks=8)
        server, oracle, *_ = run_both("c3", policy=2, host_blocks=kh, limit=600, chunk_blocks=R)
    finally:
        CONFIGS["c3"] = old
    assert oracle.host.stats["declined_requests"] > 0
    assert all(r["H"] % R == 0 for r in oracle.records)
    server.close()
