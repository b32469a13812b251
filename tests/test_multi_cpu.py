"""World-size-2 gloo test of the multi-GPU plumbing (no GPU needed): max-over-ranks timing,
summed work and the agent sharding that replicas use."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    from paper_2609_33762_b200.multi import aggregate_over_ranks, init_distributed, shard_agents
    rank, world, local_rank, dist = init_distributed(2, backend="gloo")
    dist.barrier()
    ms, units = aggregate_over_ranks(dist, 10.0 + 5 * rank, 100.0 * (rank + 1))
    dist.barrier()
    print(json.dumps(dict(rank=rank, world=world, ms=ms, units=units, agents=shard_agents(5, rank, world))))
    dist.destroy_process_group()
""") % ROOT


def test_two_rank_aggregation(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    import json
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err
        outs.append(json.loads(out.strip().splitlines()[-1]))
    outs.sort(key=lambda d: d["rank"])
    for d in outs:
        assert d["world"] == 2 and d["ms"] == 15.0 and d["units"] == 300.0
    assert outs[0]["agents"] == [0, 2, 4] and outs[1]["agents"] == [1, 3]


def test_single_process_is_identity():
    from paper_2609_33762_b200.multi import aggregate_over_ranks, init_distributed
    env = {k: os.environ.pop(k, None) for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    try:
        assert init_distributed(1)[:2] == (0, 1)
        assert aggregate_over_ranks(None, 3.5, 7) == (3.5, 7.0)
    finally:
        for k, v in env.items():
            if v is not None:
                os.environ[k] = v


TP_WORKER = textwrap.dedent("""
    import json, os, sys
    import numpy as np
    sys.path.insert(0, %r)
    from eakv_workloads import CONFIGS, SHAPES, make_trace
    from oracle import hash as ohash
    from paper_2609_33762_b200 import eakv
    from paper_2609_33762_b200.multi import decisions_digest, init_distributed, tp_rank_plan
    rank, world, local_rank, dist = init_distributed(2, backend="gloo")
    cfg = CONFIGS["c0"]
    full = SHAPES[cfg.shape]
    shard, kh = tp_rank_plan(full, world, 4 << 20)          # 4 MiB of host memory per rank
    trace = make_trace(cfg)
    ctx = eakv.Context(num_layers=shard.num_layers, kv_heads=shard.kv_heads, head_dim=shard.head_dim,
                       block_size=shard.block_size, gpu_blocks=cfg.gpu_blocks, host_blocks=kh,
                       kv_base=None, control_plane_only=True, policy=eakv.POLICY_FILTER_CONDITIONED)
    recs, stored_bytes = [], 0
    for req in trace.requests:
        toks = trace.prompt(req)
        keys = np.asarray(ohash.hash_blocks(toks.tolist(), shard.block_size), dtype=np.uint64)
        st = ctx.eakv_tier_step(keys, req.agent, len(toks), req.time_ms)
        recs.append(dict(hit=st["hit"], admit=st["admit"], slot=st["slot"],
                         evicted=list(zip(st["evicted_keys"].tolist(), st["evicted_slots"].tolist()))))
        stored_bytes += int(st["admit"].sum()) * ctx.block_bytes
    ctx.close()
    mine = dict(rank=rank, digest=decisions_digest(recs), kh=kh, stored_bytes=stored_bytes,
                heads=shard.kv_heads, block_bytes=shard.block_bytes)
    gathered = [None] * world
    dist.all_gather_object(gathered, mine)
    dist.barrier()
    if rank == 0:
        print(json.dumps(gathered))
    dist.destroy_process_group()
""") % ROOT


def test_tensor_parallel_ranks_take_the_same_decisions(tmp_path):
    """Two TP ranks, each with its head shard and its own tier of the same byte budget: identical
    K_H and decisions, half the bytes per block of the unsharded shape (Eq. 1)."""
    import json
    from eakv_workloads import CONFIGS, SHAPES
    from oracle import sizing
    script = tmp_path / "tp_worker.py"
    script.write_text(TP_WORKER)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=180) for p in procs]
    for p, (out, err) in zip(procs, outs):
        assert p.returncode == 0, err
    got = json.loads(outs[0][0].strip().splitlines()[-1])
    full = SHAPES[CONFIGS["c0"].shape]
    beta = sizing.beta_rank(full.num_layers, full.head_dim, full.elem_bytes, full.kv_heads, tp=2)
    assert got[0]["digest"] == got[1]["digest"]
    assert got[0]["stored_bytes"] == got[1]["stored_bytes"] > 0
    for g in got:
        assert g["heads"] == 1 and g["block_bytes"] == full.block_size * beta == full.block_bytes // 2
        assert g["kh"] == sizing.tier_chunks(4 << 20, full.block_size, beta)


SPAWNED = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    from paper_2609_33762_b200.multi import aggregate_over_ranks, init_distributed, launched
    assert launched()
    rank, world, local_rank, dist = init_distributed(int(sys.argv[1]), backend="gloo")
    dist.barrier()
    ms, units = aggregate_over_ranks(dist, 1.0 + rank, 10.0)
    dist.barrier()
    if rank == 0:
        print(json.dumps(dict(world=world, ms=ms, units=units, local_rank=local_rank)))
    else:
        print("a line from another rank that must not reach the caller's stdout")
    dist.destroy_process_group()
    sys.exit(int(sys.argv[2]) if rank == 1 else 0)
""") % ROOT

SPAWNER = textwrap.dedent("""
    import sys
    sys.path.insert(0, %r)
    from paper_2609_33762_b200.multi import spawn_local_ranks
    sys.exit(spawn_local_ranks([sys.executable, sys.argv[1], sys.argv[2], sys.argv[3]], int(sys.argv[2])))
""") % ROOT


def test_spawned_local_ranks_rendezvous_and_only_rank0_prints(tmp_path):
    """The path `bench.py --gpus N` takes without a launcher, with a stub in place of the arm: N
    local ranks meet over gloo, rank 0's line is the only output, the worst exit code comes back."""
    import json
    worker, spawner = tmp_path / "spawned.py", tmp_path / "spawner.py"
    worker.write_text(SPAWNED)
    spawner.write_text(SPAWNER)
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, str(spawner), str(worker), "3", "0"], env=env, capture_output=True,
                         text=True, timeout=180)
    assert out.returncode == 0, out.stderr
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    assert json.loads(lines[0]) == dict(world=3, ms=3.0, units=30.0, local_rank=0)
    # a failing rank makes the whole command fail
    out = subprocess.run([sys.executable, str(spawner), str(worker), "2", "7"], env=env, capture_output=True,
                         text=True, timeout=180)
    assert out.returncode == 7


def test_world_size_mismatch_is_an_error():
    from paper_2609_33762_b200.multi import init_distributed
    import pytest
    saved = {k: os.environ.get(k) for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    try:
        os.environ.update(WORLD_SIZE="1", RANK="0", LOCAL_RANK="0")
        with pytest.raises(RuntimeError, match="WORLD_SIZE=1"):
            init_distributed(8)                      # asked for 8, launched as 1: used to run one replica silently
        for k in saved:
            os.environ.pop(k, None)
        with pytest.raises(RuntimeError, match="WORLD_SIZE=1"):
            init_distributed(2)                      # no launcher at all
    finally:
        for k, v in saved.items():
            if v is None:
                os.environ.pop(k, None)
            else:
                os.environ[k] = v


def test_bench_gpus_2_without_devices_fails_loudly():
    """On a machine without CUDA devices `bench.py --gpus 2` must not print a one-replica line."""
    import torch
    if torch.cuda.is_available() and torch.cuda.device_count() >= 2:
        import pytest
        pytest.skip("this machine has the devices")
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1"],
                         env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode != 0
    assert "CUDA device" in out.stderr and not out.stdout.strip()
