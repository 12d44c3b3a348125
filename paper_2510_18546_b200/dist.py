"""Multi-GPU plumbing.  The path shards by episode with no exchange step (independent episodes,
independent kv heads), so ranks run replicas / disjoint episode shards and the only collective is
the max-over-ranks of the measured time.  One process per GPU; torch.distributed does the plumbing."""
from __future__ import annotations

from typing import List, Sequence

import torch

_world = 1


def init_process_group(world: int, rank: int, backend: str = "nccl") -> None:
    """Joins the job's process group (env:// rendezvous) when there is more than one rank."""
    global _world
    _world = world
    if world > 1:
        import torch.distributed as dist
        if not dist.is_initialized():
            dist.init_process_group(backend=backend, world_size=world, rank=rank)


def barrier() -> None:
    if _world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(x: float) -> float:
    """The slowest rank's time: multi-GPU numbers are reported as the max over ranks."""
    if _world == 1:
        return float(x)
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(x)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def shard_episodes(n_q: Sequence[int], world: int) -> List[List[int]]:
    """Splits a batch of independent episodes over ranks, longest first onto the least loaded rank
    (work grows with the number of query tokens).  Returns, per rank, the episode indices in order."""
    order = sorted(range(len(n_q)), key=lambda b: (-int(n_q[b]), b))
    load = [0] * world
    out: List[List[int]] = [[] for _ in range(world)]
    for b in order:
        r = min(range(world), key=lambda i: (load[i], i))
        out[r].append(b)
        load[r] += int(n_q[b])
    return [sorted(x) for x in out]
