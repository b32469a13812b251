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
