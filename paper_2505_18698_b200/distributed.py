"""Multi-GPU plumbing: one process per GPU, (batch, head) units partitioned across ranks.

Every equation of the method is per head, so ranks never exchange data on the hot path; the only
collectives are the barrier around the timed region and the max-over-ranks of the step time.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist

from .workloads import shard_units


def env_world():
    """(rank, local_rank, world_size) from the launcher's environment (1 process if absent)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str):
    """Joins the process group the launcher described (MASTER_ADDR/PORT, RANK, WORLD_SIZE)."""
    rank, local, world = env_world()
    if world > 1 and not dist.is_initialized():
        dist.init_process_group(backend, rank=rank, world_size=world)
    return rank, local, world


def my_units(total_units: int):
    """Half-open range of (batch*heads) units this rank owns."""
    rank, _, world = env_world()
    return shard_units(total_units, world, rank)


def barrier():
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def gather_units(local: torch.Tensor, total_units: int) -> torch.Tensor:
    """All ranks' unit-major results concatenated in unit order (for tests and small outputs)."""
    if not dist.is_initialized():
        return local
    world = dist.get_world_size()
    sizes = [shard_units(total_units, world, r) for r in range(world)]
    biggest = max(hi - lo for lo, hi in sizes)
    pad = torch.zeros((biggest,) + tuple(local.shape[1:]), dtype=local.dtype, device=local.device)
    pad[: local.shape[0]] = local
    out = [torch.empty_like(pad) for _ in range(world)]
    dist.all_gather(out, pad)
    return torch.cat([out[r][: hi - lo] for r, (lo, hi) in enumerate(sizes)], dim=0)
