"""Lane sharding over ranks (App. A: codes are handed out once, every rank then decodes on its
own, and nothing is exchanged until the sequences are collected at the end).

Host logic only: which lanes a rank owns, and the single collection of the results through
`torch.distributed` (NCCL for device tensors, gloo for host tensors).  No kernel here."""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist


def shard_range(n: int, rank: int, world: int) -> Tuple[int, int]:
    """[lo, hi) of the n units (lanes, or start tokens with their whole code groups) that `rank`
    owns: contiguous, in rank order, sizes differing by at most one."""
    if world < 1 or not 0 <= rank < world or n < 0:
        raise ValueError("need 0 <= rank < world and n >= 0")
    base, extra = divmod(n, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def step_lattice_args(N: int, rank: int, world: int) -> dict:
    """Arguments of this rank's as_step_lattice call when the N lanes of one lattice are sharded:
    lanes j0 .. j0+lanes-1 of the same lattice (same N, same shift u on every rank)."""
    lo, hi = shard_range(N, rank, world)
    return {"N": N, "j0": lo, "lanes": hi - lo}


def decode_args(S: int, N: int, rank: int, world: int) -> dict:
    """Arguments of this rank's as_decode_bigram call when a job of S start tokens x N codes is
    sharded by start token (a start token keeps its whole lattice, so the code set of every group
    is untouched): start tokens s_lo .. s_hi-1, i.e. lanes s_lo*N .. s_hi*N-1 of the whole job."""
    lo, hi = shard_range(S, rank, world)
    return {"s_lo": lo, "s_hi": hi, "S": hi - lo, "N": N, "lane_lo": lo * N, "lane_hi": hi * N}


def gather_sequences(seq: torch.Tensor, length: torch.Tensor, n_total: int, group=None, unit: int = 1):
    """All ranks' decoded sequences in lane order: (seq[n_total, T], length[n_total]) on every rank.
    `seq`/`length` are this rank's shard: the job's n_total lanes are cut in units of `unit` lanes
    (1 = by lane; N = by start token, each with its whole lattice of N codes) and rank r owns the
    units shard_range(n_total // unit, r, world).  One all-gather of equal-sized (padded) blocks:
    the only exchange of a sharded decode."""
    if unit < 1 or n_total % unit:
        raise ValueError("n_total must be a multiple of unit")
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    if world == 1:
        return seq, length
    rank = dist.get_rank(group)

    def lanes_of(r):
        a, b = shard_range(n_total // unit, r, world)
        return a * unit, b * unit
    lo, hi = lanes_of(rank)
    if seq.shape[0] != hi - lo or length.shape[0] != hi - lo:
        raise ValueError("shard has %d lanes, rank %d of %d owns %d" % (seq.shape[0], rank, world, hi - lo))
    T = seq.shape[1]
    rows = -(-(n_total // unit) // world) * unit      # largest shard
    block = torch.full((rows, T + 1), -1, dtype=torch.int32, device=seq.device)
    block[: hi - lo, :T] = seq
    block[: hi - lo, T] = length
    out = [torch.empty_like(block) for _ in range(world)]
    dist.all_gather(out, block, group=group)
    parts = []
    for r in range(world):
        a, b = lanes_of(r)
        parts.append(out[r][: b - a])
    full = torch.cat(parts, dim=0)
    return full[:, :T].contiguous(), full[:, T].contiguous()
