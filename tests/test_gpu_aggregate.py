"""GPU parity of the per-plan serving aggregate (one score per plan over the request-length mix)."""
from __future__ import annotations

import numpy as np
import pytest

from oracle import Oracle
from workloads import make_config

from helpers import TPUT_RTOL, check_topk, variant

pytestmark = pytest.mark.gpu


def _run(cfg, k):
    import torch
    from paper_2607_18631_b200 import Plan
    plan, orc = Plan(cfg), Oracle(cfg)
    out = plan.score(k=0)
    agg = plan.aggregate_serving(out["reason"], out["tput"], k=k)
    torch.cuda.synchronize()
    # the aggregate is a function of the per-candidate scores: give the oracle the device's own fp32 scores, so
    # that the comparison isolates the reduction
    reason = out["reason"].cpu().numpy()
    tput = out["tput"].cpu().numpy().astype(np.float64)
    pr, pt = orc.aggregate_serving(reason, tput)
    assert plan.serve_plan_count() == len(pr)
    np.testing.assert_array_equal(agg["plan_reason"].cpu().numpy(), pr)
    got = agg["plan_tput"].cpu().numpy()
    feas = (pr & 0x7F) == 0
    assert np.all(got[~feas] == 0)
    np.testing.assert_allclose(got[feas], pt[feas], rtol=TPUT_RTOL, atol=0)
    n = int(agg["topk_count"].item())
    order = np.flatnonzero(feas)
    order = order[np.lexsort((order, -pt[order]))][:k]
    check_topk(agg["topk_idx"].cpu().numpy().view(np.uint64)[:n], agg["topk_score"].cpu().numpy()[:n],
               order.astype(np.uint64), pt[order])
    # and end to end against the fp64 oracle's own scores
    r64, t64, _, _ = orc.score_range(threads=8)
    pr64, pt64 = orc.aggregate_serving(r64, t64)
    np.testing.assert_array_equal(pr, pr64)
    np.testing.assert_allclose(got[feas], pt64[feas], rtol=TPUT_RTOL, atol=0)
    plan.close()
    return pr, pt


def test_serving_aggregate_matches_oracle():
    pr, pt = _run(make_config("serve"), 128)
    assert ((pr & 0x7F) == 0).sum() > 100 and ((pr & 0x7F) == 11).sum() > 100


def test_serving_aggregate_small_mix_and_k_edges():
    cfg = variant("serve", cluster=dict(budget_bytes=10 ** 15))
    for kn in cfg["kern"]:
        kn["avail_mask"] = 255
    cfg["axes"][6] = ("scen", [5, 9, 5])          # a repeated scenario, three digits
    _run(cfg, 1024)
    cfg["axes"][6] = ("scen", [17])
    _run(cfg, 1)


def test_aggregate_rejects_training_plans():
    import torch
    from paper_2607_18631_b200 import Plan, PlanfrontError
    plan = Plan(make_config("tiny"))
    out = plan.score(k=0)
    assert plan.serve_plan_count() == 0
    with pytest.raises(PlanfrontError):
        plan.aggregate_serving(out["reason"], out["tput"], k=4,
                               workspace=torch.empty(4096, dtype=torch.uint8, device="cuda"))
    plan.close()
