"""Replicate chains across GPUs: one process per GPU, no collective on the per-step path.

The chains of a BMGD job are independent (each has its own theta and its own partitions; they only share the
buffer), so a job with Rc chains splits into contiguous shares of chains, one share per rank.  Rank r creates its
handle with `first_chain` = the id of its first chain, so chain c of the whole job draws the same partitions on
whichever rank it lands: N GPUs with Rc/N chains each give, bit for bit, what one GPU with Rc chains gives.  The one
collective is an all-gather of theta at the end (NCCL when the tensors are on GPUs, gloo for host tensors).

The paper's own multi-GPU use (Section 2.1: several GPUs work on one mini-batch; Section 4.3: 5 GPUs x 150 rows) puts
one all-reduce of p values on every step's critical path; that is not what this module does.
"""
from __future__ import annotations

from typing import List, Tuple

import torch


def chain_share(Rc: int, world: int, rank: int) -> Tuple[int, int]:
    """(first, count): the contiguous run of chain ids that rank `rank` of `world` works on.

    Shares differ by at most one chain; the first Rc % world ranks hold the longer ones; a rank may get none."""
    if Rc < 0 or world < 1 or not (0 <= rank < world):
        raise ValueError("chain_share: need Rc >= 0 and 0 <= rank < world")
    q, r = divmod(Rc, world)
    first = rank * q + min(rank, r)
    return first, q + (1 if rank < r else 0)


def gather_theta(local: torch.Tensor, Rc: int, group=None) -> torch.Tensor:
    """All-gather the ranks' theta shares [count_r, ...] into the job's theta [Rc, ...], in chain order, on every rank.

    `local` holds this rank's chains in the order of chain_share; ranks with a shorter share are padded for the
    collective and the padding is dropped again."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    first, count = chain_share(Rc, world, rank)
    if local.shape[0] != count:
        raise ValueError(f"rank {rank} holds {local.shape[0]} chains, its share is {count}")
    longest = -(-Rc // world)
    tail = tuple(local.shape[1:])
    padded = torch.zeros((longest,) + tail, dtype=local.dtype, device=local.device)
    padded[:count] = local
    parts: List[torch.Tensor] = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(parts, padded, group=group)
    out = torch.empty((Rc,) + tail, dtype=local.dtype, device=local.device)
    for r, part in enumerate(parts):
        f, c = chain_share(Rc, world, r)
        out[f:f + c] = part[:c]
    return out
