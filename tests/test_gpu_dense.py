"""GPU parity of the leading-dense-layer model (L_dense, F_dense) and the separate query head width (hd_q)."""
from __future__ import annotations

import numpy as np
import pytest

from oracle import Oracle
from workloads import make_config

from gpu_common import compare_dense, compare_topk, gpu_score
from helpers import TPUT_RTOL, check_topk, variant

pytestmark = pytest.mark.gpu


def _plan(cfg):
    from paper_2607_18631_b200 import Plan
    return Plan(cfg)


def _cases():
    out = {}
    c = variant("mid", cluster=dict(budget_bytes=10 ** 15))
    c["model"].update(L_dense=3, F_dense=11008, hd_q=192)
    out["mid_roomy"] = c
    c = make_config("mid")
    c["model"].update(L_dense=1, F_dense=16384)
    out["mid_gated"] = c
    c = variant("mid", cluster=dict(budget_bytes=60_000_000_000), rules=dict(enforce_realizability=0))
    c["model"].update(L_dense=5, F_dense=2048)              # dense layers cheaper than MoE ones
    out["mid_unconstrained_cheap_dense"] = c
    c = variant("mid", cluster=dict(budget_bytes=10 ** 15), rules=dict(enforce_realizability=0))
    c["model"].update(L_dense=2, F_dense=65536)             # dense layers dearer: the first rank is the slow one
    out["mid_dear_dense"] = c
    c = make_config("tiny")
    c["model"].update(L_dense=3, F_dense=4096)
    out["tiny"] = c
    return out


@pytest.mark.parametrize("name", list(_cases()))
def test_scoring_parity_with_leading_dense_layers(name):
    cfg = _cases()[name]
    plan, orc = _plan(cfg), Oracle(cfg)
    reason, tput, mem, _ = orc.score_range(threads=8)
    res = gpu_score(plan, k=cfg["k"])
    compare_dense(res, reason, tput, mem)
    compare_topk(res, orc, reason, tput, 0, cfg["k"])
    assert ((reason & 0x7F) == 0).sum() > 10
    plan.close()


@pytest.mark.parametrize("name", ["mid_unconstrained_cheap_dense", "mid_dear_dense"])
def test_simulator_parity_with_leading_dense_layers(name):
    import torch
    cfg = _cases()[name]
    plan, orc = _plan(cfg), Oracle(cfg)
    out = plan.score(k=0)
    sel = plan.select_survivors(out["reason"], out["tput"], 10 ** 6)
    torch.cuda.synchronize()
    ns = int(sel["surv_count"].item())
    idx = sel["surv_idx"][:ns].cpu().numpy().view(np.uint64)
    assert ns > 500
    sim = plan.simulate(sel["surv_idx"], ns, 4, k=100)
    torch.cuda.synchronize()
    ref, ref_st, _ = orc.simulate_list(idx, 4, threads=16)
    np.testing.assert_array_equal(sim["sim_status"][:ns].cpu().numpy(), ref_st)
    np.testing.assert_allclose(sim["tput_sim"][:ns].cpu().numpy(), ref, rtol=TPUT_RTOL, atol=0)
    kinds = {orc.eval(int(i))["kind"] for i in idx[::53]}
    assert kinds == {0, 1, 2}
    c = int(sim["topk_count"].item())
    ref_idx, ref_sc = Oracle.topk_list(idx[ref > 0], ref[ref > 0], 100)
    check_topk(sim["topk_idx"].cpu().numpy().view(np.uint64)[:c], sim["topk_score"].cpu().numpy()[:c], ref_idx, ref_sc)
    plan.close()


def test_reference_like_model_memory_on_the_device():
    """The reconstructed 27-layer reference model: the device reproduces the oracle's bytes, i.e. the paper's
    optimizer sizes, bit for bit."""
    from test_oracle_dense_pins import reference_like
    cfg = reference_like()
    plan, orc = _plan(cfg), Oracle(cfg)
    reason, tput, mem, _ = orc.score_range()
    res = gpu_score(plan, k=0)
    compare_dense(res, reason, tput, mem)
    plan.close()


def test_invalid_dense_layer_inputs():
    from paper_2607_18631_b200 import PlanfrontError
    cfg = make_config("tiny")
    cfg["model"].update(L_dense=8, F_dense=1024)      # every layer dense: not a MoE model
    with pytest.raises(PlanfrontError):
        _plan(cfg)
    cfg = make_config("tiny")
    cfg["model"].update(L_dense=1, F_dense=0)
    with pytest.raises(PlanfrontError):
        _plan(cfg)


@pytest.mark.parametrize("l_dense,f_dense,hd_q", [(1, 12288, 0), (3, 18432, 192), (47, 1024, 0)])
def test_serving_space_with_leading_dense_layers(l_dense, f_dense, hd_q):
    """The serving space with the first layers dense (and a separate query width): every candidate and the per-plan
    aggregate against the oracle."""
    import torch
    cfg = make_config("serve")
    cfg["model"].update(L_dense=l_dense, F_dense=f_dense, hd_q=hd_q)
    plan, orc = _plan(cfg), Oracle(cfg)
    res = gpu_score(plan, k=128)
    reason, tput, mem, _ = orc.score_range(threads=16)
    compare_dense(res, reason, tput, mem)
    compare_topk(res, orc, reason, tput, 0, 128)
    assert ((reason & 0x7F) == 0).sum() > 10_000
    base = Oracle(make_config("serve")).score_range(threads=16)
    assert not np.array_equal(base[2], mem)                  # the dense layers do change the byte counts
    plan.close()
