"""Multi-GPU plumbing.  The path shards by rank with no exchange step (in the paper every
tensor-parallel rank holds its own head shard of each token's KV and its own host tier),
so N GPUs run N independent replicas: a barrier brackets the timed region, the time is the
maximum over ranks and the work is the sum.  No data-path collective exists."""
from __future__ import annotations

import os


def init_distributed(expected_world: int, backend: str | None = None):
    """Join the process group torchrun set up; returns (rank, world, local_rank, dist|None)."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
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
    if expected_world and expected_world != world:
        raise RuntimeError(f"--gpus {expected_world} but WORLD_SIZE={world}")
    return rank, world, local_rank, dist


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
