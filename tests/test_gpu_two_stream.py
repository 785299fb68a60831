"""GPU parity of the simulator tier's two-stream layer timeline (comm chunking + SM budget per schedule)."""
from __future__ import annotations

import numpy as np
import pytest

from oracle import Oracle

from helpers import TPUT_RTOL, check_topk, variant

pytestmark = pytest.mark.gpu


def _plan(cfg):
    from paper_2607_18631_b200 import Plan
    return Plan(cfg)


def _cfg(n_chunks, sm_frac, **model):
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15), rules=dict(enforce_realizability=0))
    cfg["model"].update(model)
    for s in cfg["sched"]:
        if s["overlap"]:
            s["n_chunks"] = n_chunks
            s["sm_frac"] = float(np.float32(sm_frac))
    return cfg


@pytest.mark.parametrize("n_chunks,sm_frac,model", [(1, 0.0, {}), (4, 0.15, {}), (16, 0.3, {}), (3, 0.1, dict(L_dense=2, F_dense=8192))])
def test_simulator_parity_with_the_two_stream_timeline(n_chunks, sm_frac, model):
    import torch
    cfg = _cfg(n_chunks, sm_frac, **model)
    plan, orc = _plan(cfg), Oracle(cfg)
    out = plan.score(k=0)
    sel = plan.select_survivors(out["reason"], out["tput"], 10 ** 6)
    torch.cuda.synchronize()
    ns = int(sel["surv_count"].item())
    idx = sel["surv_idx"][:ns].cpu().numpy().view(np.uint64)
    assert ns > 3000
    sim = plan.simulate(sel["surv_idx"], ns, 4, k=100)
    torch.cuda.synchronize()
    ref, ref_st, _ = orc.simulate_list(idx, 4, threads=16)
    np.testing.assert_array_equal(sim["sim_status"][:ns].cpu().numpy(), ref_st)
    got = sim["tput_sim"][:ns].cpu().numpy()
    np.testing.assert_allclose(got, ref, rtol=TPUT_RTOL, atol=0)
    # the timeline really is in use: overlapped plans differ from the alpha-table simulation
    base = _cfg(0, 0.0, **model)
    ref0, _, _ = Oracle(base).simulate_list(idx, 4, threads=16)
    assert np.any(np.abs(ref / ref0 - 1) > 1e-3)
    c = int(sim["topk_count"].item())
    ref_idx, ref_sc = Oracle.topk_list(idx[ref > 0], ref[ref > 0], 100)
    check_topk(sim["topk_idx"].cpu().numpy().view(np.uint64)[:c], sim["topk_score"].cpu().numpy()[:c], ref_idx, ref_sc)
    plan.close()


def test_scoring_ignores_the_chunking_and_bad_values_are_rejected():
    import torch
    from paper_2607_18631_b200 import PlanfrontError
    a, b = _plan(_cfg(0, 0.0)), _plan(_cfg(8, 0.2))
    ra, rb = a.score(k=0), b.score(k=0)
    torch.cuda.synchronize()
    for key in ("reason", "tput", "mem"):
        assert torch.equal(ra[key], rb[key])
    a.close()
    b.close()
    for n_chunks, sm in ((17, 0.0), (-1, 0.0), (2, 0.95), (2, -0.1)):
        with pytest.raises(PlanfrontError):
            _plan(_cfg(n_chunks, sm))
