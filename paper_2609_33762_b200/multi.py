"""Multi-GPU plumbing.  The path shards by rank with no exchange step (in the paper every
tensor-parallel rank holds its own head shard of each token's KV and its own host tier),
so N GPUs run N independent replicas: a barrier brackets the timed region, the time is the
maximum over ranks and the work is the sum.  No data-path collective exists."""
from __future__ import annotations

import os


def init_distributed(expected_world: int, backend: str | None = None):
    """Join the process group the launcher set up (torchrun, or spawn_local_ranks below); returns
    (rank, world, local_rank, dist|None).  The launcher's WORLD_SIZE must be the number of
    replicas the caller asked for: a mismatch raises instead of silently running another count."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if expected_world and expected_world != world:
        raise RuntimeError(f"{expected_world} replicas were asked for but the launcher set WORLD_SIZE={world}")
    if world <= 1:
        return 0, 1, local_rank, None
    import torch
    import torch.distributed as dist
    if backend is None:
        backend = "nccl" if torch.cuda.is_available() else "gloo"
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    if backend == "nccl":
        torch.cuda.set_device(local_rank)
    dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world, local_rank, dist


def launched() -> bool:
    """Did a launcher (torchrun or spawn_local_ranks) start this process as one rank of several?"""
    return "WORLD_SIZE" in os.environ and "RANK" in os.environ


def spawn_local_ranks(argv, n_ranks: int, timeout_s: float | None = None) -> int:
    """Run ``argv`` (a command line) as ``n_ranks`` local processes, one replica each, with the
    rendezvous variables a launcher would set (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_ADDR =
    127.0.0.1, a free MASTER_PORT).  Rank 0 inherits this process's stdout, so its single result
    line is this command's; the other ranks' stdout is dropped, every rank's stderr passes through.
    Returns the largest exit code (a rank that had to be killed counts as 1).  No data-path
    collective is involved anywhere: the replicas only meet at barriers and at the final max/sum."""
    import socket
    import subprocess
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(n_ranks):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(n_ranks),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen(list(argv), env=env, stdout=None if rank == 0 else subprocess.DEVNULL))
    worst = 0
    try:
        for p in procs:
            rc = p.wait(timeout=timeout_s)
            worst = max(worst, rc if rc >= 0 else 1)
    except subprocess.TimeoutExpired:
        worst = 1
    finally:
        for p in procs:                 # exactly the processes started here, by handle
            if p.poll() is None:
                p.kill()
                p.wait()
                worst = max(worst, 1)
    return worst


def aggregate_over_ranks(dist, elapsed_ms: float, units: float, device=None):
    """(max over ranks of elapsed_ms, sum over ranks of units)."""
    if dist is None:
        return float(elapsed_ms), float(units)
    import torch
    dev = device if (device is not None and dist.get_backend() == "nccl") else "cpu"
    t = torch.tensor([float(elapsed_ms)], dtype=torch.float64, device=dev)
    u = torch.tensor([float(units)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def shard_agents(n_agents: int, rank: int, world: int):
    """Agents served by this rank when a trace is split across replicas (round-robin)."""
    return [a for a in range(n_agents) if a % world == rank]


def tp_rank_plan(shape, tp: int, host_bytes_per_rank: int):
    """Tensor-parallel serving (Eq. 1 and Section 2 of the paper: every rank holds its head shard
    of each token's KV and its own host tier, so sizes are stated per rank).  Returns the rank's
    KV shape and K_H = floor(C_H / (b * beta_rank)).  Every rank sees the same keys and the same
    K_H, hence takes the same decisions; only the bytes per block differ from the unsharded
    shape.  No exchange step exists between the ranks' tiers."""
    shard = shape.tp_shard(tp)
    return shard, int(host_bytes_per_rank) // shard.block_bytes


def decisions_digest(records) -> str:
    """Order-sensitive digest of the per-request decisions (hit / admit / slot / evictions), to
    compare ranks without shipping the records."""
    import hashlib
    h = hashlib.sha256()
    for r in records:
        for f in ("hit", "admit", "slot"):
            h.update(bytes(memoryview(r[f]).cast("B")))
        for k, s in r["evicted"]:
            h.update(int(k).to_bytes(8, "little") + int(s).to_bytes(4, "little", signed=True))
    return h.hexdigest()
