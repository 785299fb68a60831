"""Helpers for the split-space tests: ranks played by threads of one process, and the oracle standing in for a
rank's share of the work."""
from __future__ import annotations

import threading

import numpy as np


class ThreadComm:
    """The collectives of sharded_search among threads of one process (one thread per rank)."""

    def __init__(self, shared: dict, rank: int):
        self.shared, self.rank, self.world = shared, rank, shared["world"]

    @staticmethod
    def make_shared(world: int) -> dict:
        return dict(world=world, barrier=threading.Barrier(world, timeout=120), slots=[None] * world)

    def _exchange(self, t):
        self.shared["slots"][self.rank] = t
        self.shared["barrier"].wait()
        vals = list(self.shared["slots"])
        self.shared["barrier"].wait()
        return vals

    def all_reduce_sum(self, t):
        vals = self._exchange(t.clone())
        total = vals[0].clone()
        for v in vals[1:]:
            total += v
        t.copy_(total)
        return t

    def all_gather(self, t):
        return [v.clone() for v in self._exchange(t.clone())]


def run_ranks(world: int, fn):
    """Run fn(rank, comm) on `world` threads; returns the list of results, re-raising the first failure."""
    shared = ThreadComm.make_shared(world)
    results, errors = [None] * world, [None] * world

    def body(r):
        try:
            results[r] = fn(r, ThreadComm(shared, r))
        except BaseException as e:  # noqa: BLE001
            errors[r] = e
            shared["barrier"].abort()

    threads = [threading.Thread(target=body, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    for e in errors:
        if e is not None and not isinstance(e, threading.BrokenBarrierError):
            raise e
    for e in errors:
        if e is not None:
            raise e
    return results


class OracleOps:
    """A rank's share of the work done by the CPU oracle (numpy / torch CPU tensors): lets the host logic of
    sharded_search run without a GPU."""

    def __init__(self, orc, threads: int = 2):
        self.orc, self.size, self.threads = orc, orc.size, threads

    def score(self, first, count, k):
        import torch
        reason, tput, mem, _ = self.orc.score_range(first, count, threads=self.threads)
        idx, sc = self.orc.topk(reason, tput, first, k)
        ti = torch.full((k,), -1, dtype=torch.int64)
        ts = torch.zeros(k, dtype=torch.float32)
        ti[:len(idx)] = torch.from_numpy(idx.astype(np.int64))
        ts[:len(idx)] = torch.from_numpy(sc.astype(np.float32))
        return dict(reason=reason, tput=tput.astype(np.float32), mem=mem, topk_idx=ti, topk_score=ts,
                    topk_count=torch.tensor([len(idx)], dtype=torch.int32))

    def _eligible_bits(self, out):
        feas = (out["reason"] & 0x7F) == 0
        return out["tput"].view(np.uint32)[feas], np.flatnonzero(feas)

    def hist(self, out, first, cut):
        import torch
        bits, _ = self._eligible_bits(out)
        if cut is None:
            h = np.bincount(bits >> 16, minlength=65536)
        elif cut["take_all"]:
            h = np.zeros(65536, dtype=np.int64)
        else:
            h = np.bincount(bits[(bits >> 16) == cut["bin_hi"]] & 0xFFFF, minlength=65536)
        return torch.from_numpy(h.astype(np.int32))

    def cut(self, hist_sum, level, s_max, cut):
        h = hist_sum.numpy()
        from_top = np.cumsum(h[::-1])                      # from_top[i]: count in the i + 1 highest bins
        if level == 0:
            total = int(h.sum())
            cut = dict(total=total, target=s_max, take_all=total <= s_max, bin_hi=0, above_hi=0, thr_bits=0,
                       n_gt=total, need_eq=0)
            if cut["take_all"]:
                return cut
            i = int(np.searchsorted(from_top, s_max))       # first position where the running count reaches s_max
            cut["bin_hi"], cut["above_hi"] = 65535 - i, int(from_top[i] - h[65535 - i])
            return cut
        if cut["take_all"]:
            return cut
        want = cut["target"] - cut["above_hi"]
        i = int(np.searchsorted(from_top, want))
        lo = 65535 - i
        cut["thr_bits"] = (cut["bin_hi"] << 16) | lo
        cut["n_gt"] = cut["above_hi"] + int(from_top[i] - h[lo])
        cut["need_eq"] = cut["target"] - cut["n_gt"]
        return cut

    def cut_info(self, cut):
        return cut["thr_bits"] & 0xFFFF, bool(cut["take_all"])

    def write(self, out, first, cut, eq_before, cap):
        import torch
        bits, pos = self._eligible_bits(out)
        if cut["take_all"]:
            keep = pos
        else:
            eq = pos[bits == cut["thr_bits"]]
            need = max(cut["need_eq"] - eq_before, 0)
            keep = np.sort(np.concatenate([pos[bits > cut["thr_bits"]], eq[:need]]))
        surv = torch.zeros(max(cap, 1), dtype=torch.int64)
        surv[:len(keep)] = torch.from_numpy((keep + first).astype(np.int64))
        return surv, torch.tensor([len(keep)], dtype=torch.int64)

    def simulate(self, surv, n, jitter_seed, k_sim):
        import torch
        from oracle import Oracle
        idx = surv[:int(n.item())].numpy().astype(np.uint64)
        ts, _, _ = self.orc.simulate_list(idx, jitter_seed, threads=self.threads)
        ti, tsc = Oracle.topk_list(idx, ts, k_sim)
        oi = torch.full((k_sim,), -1, dtype=torch.int64)
        os_ = torch.zeros(k_sim, dtype=torch.float32)
        oi[:len(ti)] = torch.from_numpy(ti.astype(np.int64))
        os_[:len(ti)] = torch.from_numpy(tsc.astype(np.float32))
        return oi, os_, torch.tensor([len(ti)], dtype=torch.int32)

    def merge(self, k, a, b):
        import torch
        na, nb = int(a[2].item()), int(b[2].item())
        idx = np.concatenate([a[0][:na].numpy(), b[0][:nb].numpy()]).astype(np.int64)
        sc = np.concatenate([a[1][:na].numpy(), b[1][:nb].numpy()]).astype(np.float64)
        order = np.lexsort((idx, -sc))[:k]
        oi = torch.full((k,), -1, dtype=torch.int64)
        os_ = torch.zeros(k, dtype=torch.float32)
        oi[:len(order)] = torch.from_numpy(idx[order])
        os_[:len(order)] = torch.from_numpy(sc[order].astype(np.float32))
        return oi, os_, torch.tensor([len(order)], dtype=torch.int32)
