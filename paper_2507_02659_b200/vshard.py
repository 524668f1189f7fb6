"""Vocabulary sharding across GPUs: the target's output layer split by columns.

With the target model under tensor parallelism every GPU holds, for every row,
only the logits of its own range of target ids. Steps 2 and 3 then run as four
kernels-only calls with three small exchanges between them (all of them
torch.distributed collectives: NCCL on GPUs, gloo in the CPU tests):

    od_verify_shard_stats  -> all-gather of 16 bytes per row
    od_verify_shard_finish -> od_sample_shard_mass -> all-gather of 16 bytes per sequence
    od_sample_shard_pick   -> all-gather of 12 bytes per sequence, reduced by `combine_picks`

Step 1 (od_map_proposals) is replicated: every rank translates the same
proposals, so all ranks take identical decisions from identical bits.
`emulate_step` runs all shards of a step one after the other on ONE GPU through
the same calls (no collective); the tests and the benchmark use it where only
one GPU is at hand.
"""
from __future__ import annotations

from typing import List, Tuple

import torch
import torch.distributed as dist

from . import binding as od

TILE = 256      # shards are whole 256-id tiles (the sampler's tile)


def split_vocab(v_p: int, rank: int, world: int) -> Tuple[int, int]:
    """Target ids [lo, hi) owned by `rank`: contiguous, in rank order, whole tiles
    (the last shard ends at v_p); tile counts differ by at most one, earlier ranks
    take the larger shards. Needs at least one tile per rank."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    tiles = (v_p + TILE - 1) // TILE
    if world > tiles:
        raise ValueError("more shards than 256-id tiles")
    base, extra = divmod(tiles, world)
    t_lo = rank * base + min(rank, extra)
    t_hi = t_lo + base + (1 if rank < extra else 0)
    return t_lo * TILE, min(v_p, t_hi * TILE)


def gather_shards(x: torch.Tensor) -> torch.Tensor:
    """[world, *x.shape]: every rank's `x`, in rank order, on every rank."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return x.unsqueeze(0).contiguous()
    world = dist.get_world_size()
    out = torch.empty((world,) + tuple(x.shape), dtype=x.dtype, device=x.device)
    dist.all_gather(list(out.unbind(0)), x.contiguous())
    return out


def combine_picks(tokens: torch.Tensor, masses: torch.Tensor, flags: torch.Tensor):
    """The step's (out_token, resid_mass, sample_flags) from the per-shard outputs
    stacked along dim 0: only the owning shard wrote a token (the others -1, 0, 0),
    so the result is the maximum of tokens and masses and the OR of the flags."""
    f = flags[0].clone()
    for k in range(1, flags.shape[0]):
        f |= flags[k]
    return tokens.max(dim=0).values, masses.max(dim=0).values, f


def step(ctx: od.Context, shard_lo: int, shard_logits: torch.Tensor, mp: od.MapOut, q_rows, draft_ids,
         temperature, seed, step_index: int):
    """Steps 2 and 3 on this rank's shard (`shard_logits` = columns [shard_lo,
    shard_lo + shard_len) of the step's rows); every rank returns the same
    (VerifyOut, SampleOut)."""
    rank = dist.get_rank() if dist.is_available() and dist.is_initialized() else 0
    stats_all = gather_shards(od.od_verify_shard_stats(ctx, shard_lo, shard_logits, mp, temperature))
    vo = od.od_verify_shard_finish(ctx, stats_all, mp, temperature, seed, step_index)
    mass_all = gather_shards(od.od_sample_shard_mass(ctx, shard_lo, shard_logits, vo, q_rows, draft_ids,
                                                     mp, temperature))
    so = od.od_sample_shard_pick(ctx, rank, shard_lo, mass_all, shard_logits, vo, q_rows, draft_ids, mp,
                                 temperature, seed, step_index)
    pack = torch.stack([so.out_token, so.resid_mass.view(torch.int32), so.flags])      # 12 bytes / sequence
    allp = gather_shards(pack)
    tok, mass, fl = combine_picks(allp[:, 0], allp[:, 1].view(torch.float32), allp[:, 2])
    return vo, od.SampleOut(tok, mass, fl)


def emulate_step(ctx: od.Context, logits: torch.Tensor, n_shards: int, mp: od.MapOut, q_rows, draft_ids,
                 temperature, seed, step_index: int, copy_shards: bool = False):
    """All `n_shards` shards of one step on one GPU, through the calls `step` makes
    and in its order. Shards are column slices of the full rows (views with the
    full row stride), or separate dense buffers with `copy_shards`."""
    v_p = logits.shape[2]
    bounds = [split_vocab(v_p, r, n_shards) for r in range(n_shards)]
    parts: List[torch.Tensor] = []
    per16 = 16 // logits.element_size()
    for lo, hi in bounds:
        v = logits[:, :, lo:hi]
        if copy_shards:
            # a buffer of its own whose rows start on 16-byte boundaries (the last shard's length is arbitrary)
            width = (hi - lo + per16 - 1) // per16 * per16
            buf = torch.zeros(v.shape[0], v.shape[1], width, dtype=v.dtype, device=v.device)
            buf[:, :, :hi - lo] = v
            v = buf[:, :, :hi - lo]
        parts.append(v)
    stats_all = torch.stack([od.od_verify_shard_stats(ctx, lo, p, mp, temperature)
                             for (lo, _), p in zip(bounds, parts)])
    vo = od.od_verify_shard_finish(ctx, stats_all, mp, temperature, seed, step_index)
    mass_all = torch.stack([od.od_sample_shard_mass(ctx, lo, p, vo, q_rows, draft_ids, mp, temperature)
                            for (lo, _), p in zip(bounds, parts)])
    picks = [od.od_sample_shard_pick(ctx, r, lo, mass_all, p, vo, q_rows, draft_ids, mp, temperature,
                                     seed, step_index)
             for r, ((lo, _), p) in enumerate(zip(bounds, parts))]
    tok, mass, fl = combine_picks(torch.stack([s.out_token for s in picks]),
                                  torch.stack([s.resid_mass for s in picks]),
                                  torch.stack([s.flags for s in picks]))
    return vo, od.SampleOut(tok, mass, fl), picks
