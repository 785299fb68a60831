"""GPU parity of the memory-sharding axis {zero1, zero1_offload, fsdp}: scoring, top-k, survivor selection and
the simulator on spaces that carry the axis as their most significant digit."""
from __future__ import annotations

import copy

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


def with_shard(cfg, values=(0, 1, 2)):
    cfg = copy.deepcopy(cfg)
    cfg["axes"] = list(cfg["axes"]) + [("shard", list(values))]
    return cfg


@pytest.mark.parametrize("base", ["tiny", "mid", "mid_roomy", "mid_unconstrained"])
def test_sharded_spaces_full_parity(base):
    if base == "mid_roomy":
        cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15))
    elif base == "mid_unconstrained":
        cfg = variant("mid", cluster=dict(budget_bytes=40_000_000_000), rules=dict(enforce_realizability=0))
    else:
        cfg = make_config(base)
    cfg = with_shard(cfg, (2, 0, 1) if base == "tiny" else (0, 1, 2))
    plan, orc = _plan(cfg), Oracle(cfg)
    assert plan.size == orc.size == 3 * Oracle(make_config("tiny" if base == "tiny" else "mid")).size
    reason, tput, mem, _ = orc.score_range(threads=8)
    k = cfg["k"]
    res = gpu_score(plan, k=k)
    compare_dense(res, reason, tput, mem)
    compare_topk(res, orc, reason, tput, 0, k)
    if base != "tiny":
        n = plan.size // 3
        feas = (reason & 0x7F) == 0
        # the three regimes admit different sets (offload frees the optimizer state, fsdp trades it for a buffer)
        counts = [int(feas[s * n:(s + 1) * n].sum()) for s in range(3)]
        assert counts[1] >= counts[0] and len(set(counts)) > 1 or base == "mid_roomy"
    t = plan.decode(plan.size - 1)
    assert t["shard"] == cfg["axes"][10][1][-1]
    plan.close()


def test_space_without_the_axis_equals_the_zero1_block():
    import torch
    base = variant("mid", cluster=dict(budget_bytes=10 ** 15))
    p10, p11 = _plan(base), _plan(with_shard(base))
    a = p10.score(k=0)
    b = p11.score(k=0)
    torch.cuda.synchronize()
    n = p10.size
    for key in ("reason", "tput", "mem"):
        assert torch.equal(a[key], b[key][:n])
    assert p10.decode(5)["shard"] == 0
    p10.close()
    p11.close()


def test_select_and_simulate_on_a_sharded_space():
    """Survivors of all three regimes go through the simulator; its step time carries the regime's optimizer
    and data-parallel terms and the contention penalty."""
    import torch
    cfg = with_shard(variant("mid", cluster=dict(budget_bytes=10 ** 15), rules=dict(enforce_realizability=0)))
    plan, orc = _plan(cfg), Oracle(cfg)
    out = plan.score(k=0)
    sel = plan.select_survivors(out["reason"], out["tput"], 10 ** 6)
    torch.cuda.synchronize()
    ns = int(sel["surv_count"].item())
    got = sel["surv_idx"][:ns].cpu().numpy().view(np.uint64)
    reason = out["reason"].cpu().numpy()
    want = orc.select_survivors(reason, out["tput"].cpu().numpy().astype(np.float64), 0, 10 ** 6)
    np.testing.assert_array_equal(got, want)
    n = plan.size // 3
    assert all(((got >= s * n) & (got < (s + 1) * n)).sum() > 1000 for s in range(3))
    sim = plan.simulate(sel["surv_idx"], ns, 4, k=100)
    torch.cuda.synchronize()
    tput_sim = sim["tput_sim"][:ns].cpu().numpy()
    status = sim["sim_status"][:ns].cpu().numpy()
    ref, ref_st, _ = orc.simulate_list(got, 4, threads=16)
    np.testing.assert_array_equal(status, ref_st)
    np.testing.assert_allclose(tput_sim, ref, rtol=TPUT_RTOL, atol=0)
    c = int(sim["topk_count"].item())
    ref_idx, ref_sc = Oracle.topk_list(got[ref > 0], ref[ref > 0], 100)
    check_topk(sim["topk_idx"].cpu().numpy().view(np.uint64)[:c], sim["topk_score"].cpu().numpy()[:c], ref_idx, ref_sc)
    plan.close()


def test_bad_sharding_inputs_are_rejected():
    from paper_2607_18631_b200 import PlanfrontError
    cfg = with_shard(make_config("tiny"), (0, 3))
    with pytest.raises(PlanfrontError):
        _plan(cfg)
    cfg = with_shard(make_config("tiny"))
    cfg["cluster"]["bw_host"] = 0.0
    with pytest.raises(PlanfrontError):
        _plan(cfg)


def test_large_space_with_the_sharding_axis_slices():
    """The large training space tripled by the sharding axis (539,725,824 candidates) in one call; the oracle
    checks a 20 M-candidate slice inside each regime's block, element by element, and the top-1024 of one."""
    import torch
    cfg = with_shard(make_config("large"))
    plan, orc = _plan(cfg), Oracle(cfg)
    n = plan.size // 3
    assert plan.size == 539_725_824
    out = plan.score(k=1024)
    torch.cuda.synchronize()
    for s in range(3):
        first, count = s * n + 70_000_000, 20_000_000
        reason, tput, mem, _ = orc.score_range(first, count, threads=64)
        res = dict(reason=out["reason"][first:first + count].cpu().numpy(),
                   tput=out["tput"][first:first + count].cpu().numpy(),
                   mem=out["mem"][first:first + count].cpu().numpy())
        compare_dense(res, reason, tput, mem)
    del out
    first, count = n + 60_000_000, 50_000_000
    reason, tput, mem, _ = orc.score_range(first, count, threads=64)
    res = gpu_score(plan, first=first, count=count, k=1024)
    compare_dense(res, reason, tput, mem)
    compare_topk(res, orc, reason, tput, first, 1024)
    plan.close()
