"""Helpers for the GPU parity tests: run the CUDA path through the binding and bring results to numpy."""
from __future__ import annotations

import numpy as np

from helpers import TPUT_RTOL, check_topk


def gpu_score(plan, first=0, count=None, k=0, dense=True):
    import torch
    out = plan.score(first=first, count=count, k=k, dense=dense)
    torch.cuda.synchronize()
    res = {}
    if dense:
        res["reason"] = out["reason"].cpu().numpy()
        res["tput"] = out["tput"].cpu().numpy()
        res["mem"] = out["mem"].cpu().numpy()
    if k > 0:
        n = int(out["topk_count"].item())
        idx = out["topk_idx"].cpu().numpy().view(np.uint64)
        sc = out["topk_score"].cpu().numpy()
        assert np.all(idx[n:] == np.uint64(0xFFFFFFFFFFFFFFFF)) and np.all(sc[n:] == 0)
        res["topk_idx"], res["topk_score"] = idx[:n], sc[:n]
    return res


def compare_dense(res, reason, tput, mem):
    """Parity bar: reason codes and int64 byte counts bit-exact; throughput within 1e-4 relative
    (fp32 device arithmetic against the fp64 oracle); exact zeros where infeasible."""
    np.testing.assert_array_equal(res["reason"], reason)
    feas = (reason & 0x7F) == 0
    np.testing.assert_array_equal(res["mem"], mem)
    assert np.all(res["tput"][~feas] == 0.0)
    np.testing.assert_allclose(res["tput"][feas], tput[feas], rtol=TPUT_RTOL, atol=0)


def compare_topk(res, oracle_obj, reason, tput, first, k):
    idx, sc = oracle_obj.topk(reason, tput, first, k)
    check_topk(res["topk_idx"], res["topk_score"], idx, sc)
    # every returned plan passes the predicate
    rel = (res["topk_idx"] - np.uint64(first)).astype(np.int64)
    assert np.all((reason[rel] & 0x7F) == 0)
