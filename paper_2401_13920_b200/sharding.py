"""Host-side helpers for running the router on several GPUs (one process per GPU).

The capacity of the LocMoE router is counted per (source device, expert) pair,
so the gate, route and dispatch of a logical source device depend on that
device's tokens only.  A batch can therefore be split by source device across
ranks with no exchange before the All-to-All: every rank routes the tokens of
its own logical devices and the count matrices of the ranks add up to those of
the whole batch.  These helpers do the integer bookkeeping; they contain no
router arithmetic and run on any torch.distributed backend.
"""
from __future__ import annotations

import numpy as np
import torch
import torch.distributed as dist


def devices_of_rank(D: int, world: int, rank: int) -> range:
    """Contiguous block of logical source devices owned by a rank (D divisible by world)."""
    if D % world != 0:
        raise ValueError("logical devices (%d) must divide evenly over %d ranks" % (D, world))
    per = D // world
    return range(rank * per, (rank + 1) * per)


def shard_by_source(src: np.ndarray, D: int, world: int, rank: int) -> np.ndarray:
    """Indices (ascending, i.e. in token order) of the tokens whose source device belongs to this rank."""
    devs = devices_of_rank(D, world, rank)
    return np.nonzero((src >= devs.start) & (src < devs.stop))[0]


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time: what a multi-GPU throughput has to be computed from."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(arr: np.ndarray, device="cpu") -> np.ndarray:
    """Element-wise sum of an integer array over the ranks (count matrices of disjoint source devices add up)."""
    if not (dist.is_available() and dist.is_initialized()):
        return arr.copy()
    t = torch.as_tensor(arr.astype(np.int64), device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return t.cpu().numpy()


def aggregate_throughput(units_per_rank: int, steps: int, elapsed_ms_local: float, world: int, device="cpu") -> float:
    """Whole-job units per second: all ranks' units over the slowest rank's time."""
    ms = max_over_ranks(elapsed_ms_local, device)
    return world * units_per_rank * steps / (ms * 1e-3)


def global_capacity_inputs(delta_e_local: torch.Tensor, T_local: int, group=None):
    """What every rank needs to evaluate the capacity rule of the WHOLE batch from its own share.

    delta_e_local: float32[E], the per-expert minimum cosines of this rank's tokens as written by the capacity
    call (1.0 for an expert without tokens).  Returns (delta, T_global): the batch-wide minimum over experts and
    ranks, clamped to [0, 1] exactly as the single-GPU call clamps it (the library's ``locmoe_batch_delta`` does
    that; this function only all-reduces), and the total token count.  Pass them to the capacity rule as
    ``delta_override`` and ``T_global``; every rank then derives the same capacities.
    """
    from . import binding
    d = delta_e_local.detach().to(torch.float32).clone()
    n = torch.tensor([int(T_local)], dtype=torch.int64, device=d.device)
    if dist.is_available() and dist.is_initialized():
        dist.all_reduce(d, op=dist.ReduceOp.MIN, group=group)
        dist.all_reduce(n, op=dist.ReduceOp.SUM, group=group)
    return binding.batch_delta(d), int(n.item())
