"""Host-side helpers for running the compression step on several GPUs.

The path shards over independent (batch, KV head) units and has no exchange step, so N
GPUs run N replicas, each on its own sequences; the only collectives are the ones a
benchmark needs to agree on a time: a barrier and a max over ranks.  Works with the
`nccl` backend on GPUs and with `gloo` on CPU (used by the tests).
"""
from __future__ import annotations

import os

import torch


def env_rank_world():
    """(rank, world_size, local_rank) from the torchrun environment (defaults 0, 1, 0)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str | None = None):
    """Join the process group when WORLD_SIZE > 1; returns (rank, world, local_rank)."""
    rank, world, local = env_rank_world()
    if world > 1:
        import torch.distributed as dist

        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if not dist.is_initialized():
            dist.init_process_group(backend or ("nccl" if torch.cuda.is_available() else "gloo"))
    return rank, world, local


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist

        dist.barrier()


def max_over_ranks(x: float, world: int, device: str = "cpu") -> float:
    """The slowest rank's value: the time a multi-GPU step really took."""
    if world == 1:
        return float(x)
    import torch.distributed as dist

    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def layer_seed_offset(rank: int) -> int:
    """Every rank draws its own sequences (weak scaling): layer ids are shifted per rank."""
    return 1000 * rank


def aggregate_throughput(units_per_rank: float, world: int, max_ms: float) -> float:
    """Whole-job units per second: all ranks' units over the slowest rank's time."""
    return units_per_rank * world / (max_ms * 1e-3)


def finish(world: int):
    if world > 1:
        import torch.distributed as dist

        if dist.is_initialized():
            dist.destroy_process_group()
