"""One plan space split over several GPUs (one process per GPU, torch.distributed).

Candidates are independent, so a rank scores a contiguous slice of the index range and only small things travel:
  - the k-entry top-k lists (one all-gather of k * 12 bytes per rank, folded with `pf_topk_merge` on every rank);
  - for the survivor selection, two 65,536-bin histograms of score bits (all-reduced between the selection's
    passes, so that the cut to the s_max best is exact across ranks) and one count per rank (how many candidates
    at the threshold each rank holds: ties are taken in ascending index order, i.e. rank by rank);
  - the simulator tier's top-k lists (each rank simulates its own survivors).
Dense per-candidate outputs and survivor lists stay sharded.  No kernel of this library waits on another rank, and
none reads a peer's memory: the collectives are torch.distributed's.

The exchange and the folds are host logic and are written so that they can be exercised without a GPU: the
per-rank work goes through an `ops` object (`CudaOps`: the library's calls) and the collectives through a `comm`
object (`DistComm`: a process group); a test may pass its own.
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


class DistComm:
    """The collectives `sharded_search` needs, on a torch.distributed process group."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self._dist, self.group = dist, group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)

    def all_reduce_sum(self, t):
        self._dist.all_reduce(t, op=self._dist.ReduceOp.SUM, group=self.group)
        return t

    def all_gather(self, t):
        import torch
        out = [torch.empty_like(t) for _ in range(self.world)]
        self._dist.all_gather(out, t, group=self.group)
        return out


class CudaOps:
    """A rank's share of the work through the library (binding.Plan on this rank's GPU)."""

    def __init__(self, plan):
        self.plan = plan
        self.size = plan.size

    def score(self, first, count, k):
        return self.plan.score(first=first, count=count, k=k)

    def hist(self, out, first, cut):
        return self.plan.select_hist(out["reason"], out["tput"], first=first, cut=cut)

    def cut(self, hist_sum, level, s_max, cut):
        from .binding import pf_select_cut
        return pf_select_cut(hist_sum, level, s_max, cut)

    def cut_info(self, cut):
        from .binding import cut_to_numpy
        c = cut_to_numpy(cut)
        return int(c["thr_bits"]) & 0xFFFF, bool(c["take_all"])

    def write(self, out, first, cut, eq_before, cap):
        return self.plan.select_write(out["reason"], out["tput"], cut, eq_before, cap, first=first)

    def simulate(self, surv, n, jitter_seed, k_sim):
        r = self.plan.simulate(surv, surv.numel(), jitter_seed, k=k_sim, d_n=n, dense=False)
        return r["topk_idx"], r["topk_score"], r["topk_count"]

    def merge(self, k, a, b):
        from .binding import pf_topk_merge
        return pf_topk_merge(k, a[0], a[1], a[2], b[0], b[1], b[2])


def _fold(comm, merge, lists, k):
    """All-gather every rank's (idx, score, count) list and fold them into the global top-k on every rank."""
    import torch
    idx, score, count = (t.contiguous() for t in lists)
    if comm.world == 1:
        return idx, score, count
    # one collective instead of three: the list travels as one byte string (idx | score | count)
    nb_i, nb_s = idx.numel() * idx.element_size(), score.numel() * score.element_size()
    packed = torch.cat([idx.view(torch.uint8), score.view(torch.uint8), count.view(torch.uint8)])
    parts = comm.all_gather(packed)

    def unpack(buf):
        return (buf[:nb_i].view(idx.dtype), buf[nb_i:nb_i + nb_s].view(score.dtype), buf[nb_i + nb_s:].view(count.dtype))
    acc = unpack(parts[0])
    for r in range(1, comm.world):
        acc = merge(k, acc, unpack(parts[r]))
    return acc


def gather_and_merge(idx, score, count, k: int, group=None, merge: Optional[Callable] = None):
    """All-gather the ranks' top-k lists (idx int64[k], score float32[k], count int32[1], on the device the
    process group communicates from) and fold them into the global top-k on every rank.
    Returns (idx, score, count) tensors."""
    if merge is None:
        from .binding import pf_topk_merge
        merge = lambda kk, a, b: pf_topk_merge(kk, a[0], a[1], a[2], b[0], b[1], b[2])  # noqa: E731
    return _fold(DistComm(group), merge, (idx, score, count), k)


def sharded_score_topk(plan, k: int, group=None, dense: bool = False):
    """Score this rank's slice of `plan` (a binding.Plan) and return (local outputs dict, global top-k)."""
    comm = DistComm(group)
    first, count = shard_range(plan.size, comm.rank, comm.world)
    out = plan.score(first=first, count=count, k=k, dense=dense)
    top = gather_and_merge(out["topk_idx"], out["topk_score"], out["topk_count"], k, group=group)
    return out, top


def sharded_search(ops, k: int, s_max: int, k_sim: int, jitter_seed: int, comm=None, group=None) -> dict:
    """The whole search on one space split over the ranks of `comm` (default: DistComm(group)).

    Every rank scores its slice, the analytic top-k lists are folded, the s_max best feasible plans of the WHOLE
    space are selected (exactly: histograms all-reduced between the passes, ties at the cut taken rank by rank),
    each rank simulates the survivors of its own slice and the re-ranked lists are folded.  Returns, on every rank:
      local      this rank's dense outputs (dict with reason / tput / mem of its slice) and `first`, `count`
      topk       (idx, score, count): the global analytic top-k
      surv       (idx, count): this rank's survivors, ascending; the ranks' lists in rank order are the global list
      n_survivors_total
      sim_topk   (idx, score, count): the global simulator-refined top-k_sim
    """
    import torch
    comm = comm or DistComm(group)
    first, count = shard_range(ops.size, comm.rank, comm.world)
    out = ops.score(first, count, k)
    topk = _fold(comm, ops.merge, (out["topk_idx"], out["topk_score"], out["topk_count"]), k)
    # the cut to the s_max best of the whole space: two histogram levels, summed over the ranks
    h_hi = comm.all_reduce_sum(ops.hist(out, first, None).to(torch.int64))
    cut = ops.cut(h_hi, 0, s_max, None)
    h_lo_local = ops.hist(out, first, cut)
    h_lo = comm.all_reduce_sum(h_lo_local.to(torch.int64))
    cut = ops.cut(h_lo, 1, 0, cut)
    thr_lo, take_all = ops.cut_info(cut)
    # candidates exactly at the threshold are taken in ascending index order: this rank's come after those of
    # the lower ranks
    eq_local = h_lo_local[thr_lo:thr_lo + 1].to(torch.int64) if not take_all else torch.zeros_like(h_lo[:1])
    eq_all = comm.all_gather(eq_local.contiguous())
    eq_before = int(sum(int(t.item()) for t in eq_all[:comm.rank]))
    surv, n = ops.write(out, first, cut, eq_before, max(min(count, s_max), 1))
    n_all = comm.all_gather(n)
    sim = ops.simulate(surv, n, jitter_seed, k_sim)
    sim_topk = _fold(comm, ops.merge, sim, k_sim)
    local = dict(out)
    local.update(first=first, count=count)
    return dict(local=local, topk=topk, surv=(surv, n), n_survivors_total=int(sum(int(t.item()) for t in n_all)),
                sim_topk=sim_topk)
