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


def monarch_attn_fwd_sharded(Q, K, V, b, T, gather=True, fwd=None):
    """MonarchAttention forward of a whole [batch, heads, N, d] problem split over the ranks of the
    default process group: the (batch, head) units are independent (every equation of the method
    is per head), so rank r runs its contiguous slice of units through the library on its own GPU
    and no collective touches the data path; only the optional gather of the results does.

    Q, K, V: the full tensors, present on every rank (host tensors, or on this rank's GPU).
    fwd: the per-shard call, `fwd(Qs, Ks, Vs, b, T) -> Ys` on tensors [1, units, N, d]; the default
         moves the slice to the current CUDA device if needed and calls `binding.monarch_attn_fwd`
         (tests on CPU pass a stand-in here: the partition and the gather are what they exercise).
    gather=True: returns the full [batch, heads, N, d] result on every rank (all_gather over the
         group; on the device the shard results live on).  gather=False: returns
         (Y_shard [units, N, d], (lo, hi)) and communicates nothing.
    Without an initialised process group it is the single-GPU call."""
    batch, heads, N, d = (int(x) for x in Q.shape)
    total = batch * heads
    lo, hi = my_units(total) if dist.is_initialized() else (0, total)
    if fwd is None:
        from . import binding

        def fwd(Qs, Ks, Vs, b_, T_):
            dev = torch.device("cuda", torch.cuda.current_device())
            Qs, Ks, Vs = (x if x.is_cuda else x.to(dev, non_blocking=True) for x in (Qs, Ks, Vs))
            return binding.monarch_attn_fwd(Qs.contiguous(), Ks.contiguous(), Vs.contiguous(), b_, T_)

    def shard(x):
        return x.reshape(total, N, d)[lo:hi].unsqueeze(0)

    if hi > lo:
        Ys = fwd(shard(Q), shard(K), shard(V), b, T).reshape(hi - lo, N, d)
    else:                                   # more ranks than units: this rank has nothing to do
        Ys = Q.new_zeros((0, N, d))
    if not gather:
        return Ys, (lo, hi)
    return gather_units(Ys, total).reshape(batch, heads, N, d)
