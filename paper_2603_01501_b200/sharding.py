"""Data-parallel form of the GAC step (App. A.1, "Efficient computation under
data parallelism"): every rank holds a shard of the flattened gradient and of
the stored direction, reduces its shard locally, ONE all-reduce sums three
numbers, and every rank then takes the same decision and updates its shard.

Only host logic lives here: how a flat vector made of many tensors is cut into
per-rank shards, and the order of the calls around the collective.  The
arithmetic is in the CUDA library.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist

Piece = Tuple[int, int, int]          # (tensor index, first element, one past the last element)


def flat_shard_plan(numels: Sequence[int], world: int, align: int = 8) -> List[List[Piece]]:
    """Cuts the concatenation of tensors with the given element counts into
    `world` contiguous shards of (almost) equal length, as FSDP / ZeRO flat
    sharding does.  Shard boundaries are multiples of `align` elements of the
    flat vector, so an aligned tensor stays vector-aligned on both sides of a
    cut whenever its own offset is.  Every element belongs to exactly one shard;
    trailing ranks may get an empty shard when there are few elements."""
    if world < 1:
        raise ValueError("world must be >= 1")
    total = sum(numels)
    per = -(-total // world)
    per = -(-per // align) * align
    plan: List[List[Piece]] = [[] for _ in range(world)]
    offset = 0
    for i, n in enumerate(numels):
        lo = 0
        while lo < n:
            r = min((offset + lo) // per, world - 1)
            room = (r + 1) * per - (offset + lo) if r < world - 1 else n - lo
            hi = min(n, lo + room)
            plan[r].append((i, lo, hi))
            lo = hi
        offset += n
    return plan


def shard_views(tensors: Sequence[torch.Tensor], pieces: Sequence[Piece]) -> List[torch.Tensor]:
    """Views of the shard's pieces (no copy): what this rank passes to gac_init."""
    return [tensors[i].view(-1)[lo:hi] for i, lo, hi in pieces]


def sharded_step(gb, ctx, step: int, sums: torch.Tensor, group=None, staleness: int = 0,
                 fetch: bool = False, coef_override=None, mark=None, peer_exchange: bool = False):
    """One GAC step on this rank's shard: local sums -> all-reduce of three
    doubles -> decision -> in-place update.  `gb` is the binding module, `sums`
    a float64 CUDA tensor of 3 elements reused across steps.  All calls are
    enqueued on the current stream; the collective is the process group's
    (NCCL on GPUs) -- or, with `peer_exchange` on a context prepared by
    `attach_peer_exchange`, the library's own: the reduction kernel stores the
    three sums into every rank's slot array and a small kernel adds them in
    rank order.  `mark`, if given, is called once the decision has been
    enqueued and before the update is (a caller that times the two passes
    records an event there).  Returns the decision record when `fetch`."""
    if peer_exchange:
        gb.gac_stats_exchange(ctx, step, staleness=staleness)
        res = gb.gac_decide_exchange(ctx, fetch=fetch)
    else:
        gb.gac_stats_partial(ctx, step, sums, staleness=staleness)
        if dist.is_available() and dist.is_initialized():
            dist.all_reduce(sums, op=dist.ReduceOp.SUM, group=group)
        res = gb.gac_decide(ctx, sums, fetch=fetch)
    if mark is not None:
        mark()
    gb.gac_project(ctx, coef_override=coef_override)
    return res


def attach_peer_exchange(gb, ctx, group=None, timeout_ms: int = 0):
    """Prepares a context for `sharded_step(..., peer_exchange=True)`: allocates this rank's slot
    array in symmetric memory, lets every rank map every other rank's array (a collective over
    `group`; PyTorch's symmetric memory does the mapping), zero-fills it and hands the addresses
    to the library.  Returns the symmetric-memory tensor, which the caller must keep alive as long
    as the context is used.  Raises if symmetric memory cannot be set up; NCCL's all-reduce (the
    default path of `sharded_step`) needs none of this."""
    import torch.distributed._symmetric_memory as symm
    if not (dist.is_available() and dist.is_initialized()):
        raise RuntimeError("attach_peer_exchange needs an initialised process group")
    pg = group if group is not None else dist.group.WORLD
    world, rank = dist.get_world_size(pg), dist.get_rank(pg)
    buf = symm.empty(gb.gac_exchange_bytes(world), dtype=torch.uint8, device=torch.device("cuda", torch.cuda.current_device()))
    handle = symm.rendezvous(buf, pg)
    buf.zero_()
    torch.cuda.synchronize()
    dist.barrier(group=pg)                 # nobody posts before every array reads zero
    slots = [int(p) for p in handle.buffer_ptrs]
    if len(slots) != world or slots[rank] != buf.data_ptr():
        raise RuntimeError("symmetric memory returned an unexpected set of buffer addresses")
    gb.gac_exchange_attach(ctx, rank, world, slots, timeout_ms)
    ctx._keep_symm = (buf, handle)
    return buf
