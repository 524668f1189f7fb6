"""Batch sharding across GPUs: one process per GPU, no data-path collective.

Sequences of a verification step are independent (Algorithm 1 runs per prompt),
so a batch is split by sequence: rank r of N owns a contiguous slice, every rank
holds its own copy of the vocabulary map and of the n-gram cache, and the step's
three kernels run unchanged on the slice. The only exchanges are for the
scheduler / the benchmark: an all-gather of the per-sequence results and a
max / sum reduction of timings and counts. They use torch.distributed (NCCL on
GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from dataclasses import replace
from typing import Tuple

import torch
import torch.distributed as dist


def split_batch(B: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous slice [lo, hi) of a batch of B sequences owned by `rank`;
    sizes differ by at most one, earlier ranks take the larger slices."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(B, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def weak_shard(w, rank: int, world: int):
    """Weak scaling: every rank runs a full-size batch of its own sequences
    (its own generator stream), so total work grows with the world size."""
    if world == 1:
        return w
    return replace(w, name=f"{w.name}.r{rank}", gen_seed=w.gen_seed + 0x1000 * (rank + 1))


def reduce_timing(ms_local: float, units_local: int, device) -> Tuple[float, int]:
    """(max over ranks of the elapsed time, sum over ranks of the processed units)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms_local), int(units_local)
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), int(u.item())


def gather_step_results(n_accepted: torch.Tensor, out_token: torch.Tensor, B: int):
    """All ranks receive the whole batch's (n_accepted, out_token), in sequence
    order, from slices made by split_batch. Slices may differ in length by one:
    they are padded to the longest for the collective."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return n_accepted.clone(), out_token.clone()
    world, rank = dist.get_world_size(), dist.get_rank()
    longest = (B + world - 1) // world
    lo, hi = split_batch(B, rank, world)
    if n_accepted.shape[0] != hi - lo or out_token.shape[0] != hi - lo:
        raise ValueError("slice length does not match split_batch")
    pack = torch.zeros(2, longest, dtype=torch.int32, device=n_accepted.device)
    pack[0, :hi - lo] = n_accepted
    pack[1, :hi - lo] = out_token
    parts = [torch.empty_like(pack) for _ in range(world)]
    dist.all_gather(parts, pack)
    n_all = torch.empty(B, dtype=torch.int32, device=pack.device)
    t_all = torch.empty(B, dtype=torch.int32, device=pack.device)
    for r in range(world):
        a, b = split_batch(B, r, world)
        n_all[a:b] = parts[r][0, :b - a]
        t_all[a:b] = parts[r][1, :b - a]
    return n_all, t_all
