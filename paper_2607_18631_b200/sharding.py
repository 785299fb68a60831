"""One plan space split over several GPUs (one process per GPU, torch.distributed).

Candidates are independent, so a rank scores a contiguous slice of the index range with `pf_score` and only
the k-entry top-k lists travel: one all-gather of k * 12 bytes per rank, then a fold with `pf_topk_merge` on
every rank.  Dense per-candidate outputs stay sharded.  No kernel of this library waits on another rank.

The list exchange and the fold are host logic and are written so that they can be exercised without a GPU:
`merge` defaults to the CUDA merge of the library, and a test may pass its own.
"""
from __future__ import annotations

from typing import Callable, Optional, Tuple


def shard_range(n: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous, near-equal slices: (first, count) of `rank`; the first n % world ranks get one extra."""
    if world < 1 or not (0 <= rank < world):
        raise ValueError("bad rank / world")
    base, extra = divmod(n, world)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)


def _cuda_merge(k, a, b):
    from .binding import pf_topk_merge
    return pf_topk_merge(k, a[0], a[1], a[2], b[0], b[1], b[2])


def gather_and_merge(idx, score, count, k: int, group=None, merge: Optional[Callable] = None):
    """All-gather the ranks' top-k lists (idx int64[k], score float32[k], count int32[1], on the device the
    process group communicates from) and fold them into the global top-k on every rank.
    Returns (idx, score, count) tensors."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    merge = merge or _cuda_merge
    idx_all = [torch.empty_like(idx) for _ in range(world)]
    sc_all = [torch.empty_like(score) for _ in range(world)]
    cnt_all = [torch.empty_like(count) for _ in range(world)]
    dist.all_gather(idx_all, idx, group=group)
    dist.all_gather(sc_all, score, group=group)
    dist.all_gather(cnt_all, count, group=group)
    acc = (idx_all[0], sc_all[0], cnt_all[0])
    for r in range(1, world):
        acc = merge(k, acc, (idx_all[r], sc_all[r], cnt_all[r]))
    return acc


def sharded_score_topk(plan, k: int, group=None, dense: bool = False):
    """Score this rank's slice of `plan` (a binding.Plan) and return (local outputs dict, global top-k)."""
    import torch.distributed as dist
    rank, world = dist.get_rank(group), dist.get_world_size(group)
    first, count = shard_range(plan.size, rank, world)
    out = plan.score(first=first, count=count, k=k, dense=dense)
    top = gather_and_merge(out["topk_idx"], out["topk_score"], out["topk_count"], k, group=group)
    return out, top
