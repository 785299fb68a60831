"""GPU parity of the calibration-domain overlay and of pf_report (the extrapolation report of a plan list)."""
from __future__ import annotations

import numpy as np
import pytest

from oracle import Oracle
from workloads import make_config

from gpu_common import compare_dense, compare_topk, gpu_score
from helpers import variant

pytestmark = pytest.mark.gpu


def _plan(cfg):
    from paper_2607_18631_b200 import Plan
    return Plan(cfg)


def _variants():
    roomy = variant("mid", cluster=dict(budget_bytes=10 ** 15))
    for k in roomy["kern"]:
        k["avail_mask"] = 255
    roomy["kern"][3]["dtype"] = 1
    out = {"default": roomy}
    for name, dom in (("none", dict(attached=0)), ("gpu7", dict(gpu_id=7)), ("bf16", dict(dtype_mask=1)),
                      ("narrow", dict(m_lo=96, m_hi=1536))):
        c = variant("mid", cluster=dict(budget_bytes=10 ** 15))
        for k in c["kern"]:
            k["avail_mask"] = 255
        c["kern"][3]["dtype"] = 1
        c["domain"].update(dom)
        out[name] = c
    return out


@pytest.mark.parametrize("name", ["default", "none", "gpu7", "bf16", "narrow"])
def test_domain_flags_match_the_oracle(name):
    cfg = _variants()[name]
    plan, orc = _plan(cfg), Oracle(cfg)
    reason, tput, mem, _ = orc.score_range(threads=8)
    res = gpu_score(plan, k=128)
    compare_dense(res, reason, tput, mem)
    compare_topk(res, orc, reason, tput, 0, 128)
    flagged = int((reason & 0x80 != 0).sum())
    feas = int(((reason & 0x7F) == 0).sum())
    assert {"none": flagged == 0, "gpu7": flagged == feas}.get(name, 0 < flagged < feas)
    plan.close()


def test_report_of_a_topk_list_and_of_arbitrary_plans():
    import torch
    cfg = _variants()["narrow"]
    plan, orc = _plan(cfg), Oracle(cfg)
    out = plan.score(k=128)
    rep = plan.report(out["topk_idx"], 128, d_n=out["topk_count"])
    torch.cuda.synchronize()
    n = int(out["topk_count"].item())
    rec = plan.report_to_numpy(rep, n)
    idx = out["topk_idx"].cpu().numpy().view(np.uint64)[:n]
    for i, r in zip(idx, rec):
        d = orc.eval(int(i))
        assert (r["reason"], r["why"], r["m_e"], r["bucket"]) == (d["reason"], d["why"], d["m_e"], d["bucket"])
    assert np.any(rec["why"] != 0) and np.all((rec["reason"] & 0x7F) == 0)
    # every kind of plan: rejected early (no m_e), rejected late, feasible; an unused slot and an index past the end
    pick = np.concatenate([np.arange(0, plan.size, 997, dtype=np.uint64),
                           np.array([0xFFFFFFFFFFFFFFFF, plan.size], dtype=np.uint64)])
    t = torch.from_numpy(pick.view(np.int64).copy()).cuda()
    rec = plan.report_to_numpy(plan.report(t), len(pick))
    torch.cuda.synchronize()
    for i, r in zip(pick[:-2], rec[:-2]):
        d = orc.eval(int(i))
        assert r["reason"] == d["reason"] and r["why"] == d["why"], (i, r, d["reason"], d["why"])
        if (d["reason"] & 0x7F) == 0 or (d["reason"] & 0x7F) >= 8:
            assert r["m_e"] == d["m_e"] and r["bucket"] == d["bucket"]
        else:
            assert r["m_e"] == 0
    assert rec[-1]["reason"] == 0xFF and rec[-2]["reason"] == 0xFF
    plan.close()


def test_report_on_the_serving_space():
    import torch
    cfg = make_config("serve")
    plan, orc = _plan(cfg), Oracle(cfg)
    pick = np.arange(0, plan.size, 4099, dtype=np.uint64)
    t = torch.from_numpy(pick.view(np.int64).copy()).cuda()
    rec = plan.report_to_numpy(plan.report(t), len(pick))
    torch.cuda.synchronize()
    seen = set()
    for i, r in zip(pick, rec):
        d = orc.eval(int(i))
        assert r["reason"] == d["reason"] and r["why"] == d["why"]
        if (d["reason"] & 0x7F) in (0, 8, 11):
            assert r["m_e"] == d["m_e"] and r["bucket"] == d["bucket"]
        seen.add(int(d["reason"]))
    assert 0 in seen or 0x80 in seen
    plan.close()
