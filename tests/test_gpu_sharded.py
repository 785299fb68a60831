"""One space split over several ranks, on one GPU: four ranks are played by four threads of this process, each with
its own plan handle, going through the library's real entry points (pf_score on a slice, pf_select_hist /
pf_select_cut / pf_select_write, pf_simulate, pf_topk_merge) and through sharded_search's host logic, with the
collectives done among the threads.  No kernel waits on another rank, so the ranks' launches may interleave in any
order.  The result must equal the unsplit pf_search on the same space, and the oracle."""
from __future__ import annotations

import numpy as np
import pytest

from oracle import Oracle
from workloads import make_config

from helpers import TPUT_RTOL, check_topk, variant
from sharded_common import run_ranks

pytestmark = pytest.mark.gpu


def _split(cfg, world, k, s_max, k_sim):
    import torch
    from paper_2607_18631_b200 import Plan
    from paper_2607_18631_b200.sharding import CudaOps, sharded_search

    def rank_fn(rank, comm):
        plan = Plan(cfg)
        r = sharded_search(CudaOps(plan), k, s_max, k_sim, 4, comm=comm)
        torch.cuda.synchronize()
        n = int(r["surv"][1].item())
        res = dict(first=r["local"]["first"], count=r["local"]["count"],
                   reason=r["local"]["reason"].cpu().numpy(), tput=r["local"]["tput"].cpu().numpy(),
                   mem=r["local"]["mem"].cpu().numpy(), surv=r["surv"][0][:n].cpu().numpy().view(np.uint64),
                   total=r["n_survivors_total"], topk=[t.cpu().numpy() for t in r["topk"]],
                   sim_topk=[t.cpu().numpy() for t in r["sim_topk"]])
        plan.close()
        return res
    return run_ranks(world, rank_fn)


def _check_against_unsplit(cfg, world, k, s_max, k_sim, with_oracle=True):
    import torch
    from paper_2607_18631_b200 import Plan
    parts = _split(cfg, world, k, s_max, k_sim)
    plan = Plan(cfg)
    b = plan.search(k, s_max, k_sim, 4)
    torch.cuda.synchronize()
    # dense outputs: the slices, concatenated, are the unsplit arrays
    for key in ("reason", "tput", "mem"):
        np.testing.assert_array_equal(np.concatenate([p[key] for p in parts]), b[key].cpu().numpy())
    n = int(b["surv_count"].item())
    surv = np.concatenate([p["surv"] for p in parts])
    np.testing.assert_array_equal(surv, b["surv_idx"][:n].cpu().numpy().view(np.uint64))
    kc, ks = int(b["topk_count"].item()), int(b["sim_topk_count"].item())
    for p in parts:
        assert p["total"] == n
        assert int(p["topk"][2][0]) == kc and int(p["sim_topk"][2][0]) == ks
        np.testing.assert_array_equal(p["topk"][0][:kc], b["topk_idx"][:kc].cpu().numpy())
        np.testing.assert_array_equal(p["topk"][1][:kc], b["topk_score"][:kc].cpu().numpy())
        np.testing.assert_array_equal(p["sim_topk"][0][:ks], b["sim_topk_idx"][:ks].cpu().numpy())
        np.testing.assert_array_equal(p["sim_topk"][1][:ks], b["sim_topk_score"][:ks].cpu().numpy())
    plan.close()
    if with_oracle:
        orc = Oracle(cfg)
        reason, tput, mem, _ = orc.score_range(threads=16)
        np.testing.assert_array_equal(np.concatenate([p["reason"] for p in parts]), reason)
        np.testing.assert_array_equal(np.concatenate([p["mem"] for p in parts]), mem)
        got_t = np.concatenate([p["tput"] for p in parts])
        feas = (reason & 0x7F) == 0
        np.testing.assert_allclose(got_t[feas], tput[feas], rtol=TPUT_RTOL, atol=0)
        want = orc.select_survivors(reason, got_t.astype(np.float64), 0, s_max)
        np.testing.assert_array_equal(surv, want)
        ref, _, _ = orc.simulate_list(surv, 4, threads=16)
        ref_idx, ref_sc = Oracle.topk_list(surv, ref, k_sim)
        p0 = parts[0]
        check_topk(p0["sim_topk"][0][:ks].view(np.uint64), p0["sim_topk"][1][:ks], ref_idx, ref_sc)
        idx, sc = orc.topk(reason, tput, 0, k)
        check_topk(p0["topk"][0][:kc].view(np.uint64), p0["topk"][1][:kc], idx, sc)
    return n


@pytest.mark.parametrize("world,s_max", [(4, 10 ** 6), (4, 700), (3, 1), (2, 3000)])
def test_split_search_equals_the_unsplit_search_mid(world, s_max):
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15), rules=dict(enforce_realizability=0))
    n = _check_against_unsplit(cfg, world, 128, s_max, 100)
    assert n == min(s_max, n) and n > 0


def test_split_search_with_the_cut_inside_a_run_of_equal_scores():
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15))
    for kv in (1, 2, 3):
        cfg["kern"][kv] = dict(cfg["kern"][0])
    for s_max in (7, 501, 2001, 4001):          # 2,144 plans are feasible: the last cut keeps them all
        assert _check_against_unsplit(cfg, 4, 128, s_max, 64) == min(s_max, 2144)


def test_split_search_large_space():
    assert _check_against_unsplit(make_config("large"), 4, 1024, 10 ** 6, 100, with_oracle=False) == 12_905
    cfg = variant("large_unconstrained", cluster=dict(budget_bytes=10 ** 15))
    assert _check_against_unsplit(cfg, 4, 1024, 300_000, 100, with_oracle=False) == 300_000
