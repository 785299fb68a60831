"""GPU parity of survivor selection, the pipeline simulator and the host-buffer search call."""
from __future__ import annotations

import numpy as np
import pytest

from oracle import Oracle
from workloads import make_config

from gpu_common import gpu_score
from helpers import TPUT_RTOL, axis_index, check_topk, variant

pytestmark = pytest.mark.gpu


def _plan(cfg):
    from paper_2607_18631_b200 import Plan
    return Plan(cfg)


def _select(plan, reason_t, tput_t, s_max, first=0):
    import torch
    out = plan.select_survivors(reason_t, tput_t, s_max, first=first)
    torch.cuda.synchronize()
    n = int(out["surv_count"].item())
    return out["surv_idx"][:n].cpu().numpy().view(np.uint64), out


def _simulate(plan, idx_np, seed, k):
    import torch
    t = torch.from_numpy(idx_np.view(np.int64).copy()).cuda()
    out = plan.simulate(t, len(idx_np), seed, k=k)
    torch.cuda.synchronize()
    n = int(out["topk_count"].item()) if k else 0
    return (out["tput_sim"][:len(idx_np)].cpu().numpy(), out["sim_status"][:len(idx_np)].cpu().numpy(),
            out["topk_idx"].cpu().numpy().view(np.uint64)[:n] if k else None,
            out["topk_score"].cpu().numpy()[:n] if k else None)


@pytest.mark.parametrize("s_max", [1, 50, 3000, 10 ** 6])
def test_select_survivors_matches_oracle(s_max):
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15), rules=dict(enforce_realizability=0))
    plan, orc = _plan(cfg), Oracle(cfg)
    out = plan.score(k=0)
    got, _ = _select(plan, out["reason"], out["tput"], s_max)
    # selection runs on the device's own fp32 scores: give the oracle the same numbers to rank
    reason = out["reason"].cpu().numpy()
    tput = out["tput"].cpu().numpy().astype(np.float64)
    want = orc.select_survivors(reason, tput, 0, s_max)
    np.testing.assert_array_equal(got, want)
    plan.close()


def _check_selection_against_oracle_scores(got, orc, o_reason, o_tput, first, s_max):
    """The device's survivor list against the oracle's own selection on the oracle's own fp64 scores: same length,
    ascending, and the two sets may differ only in members whose oracle score lies within the throughput tolerance
    of the S-th best score (near-ties at the cut, which fp32 and fp64 may order differently)."""
    want = orc.select_survivors(o_reason, o_tput, first, s_max)
    assert len(got) == len(want)
    assert np.all(np.diff(got.astype(np.int64)) > 0)
    only_gpu = np.setdiff1d(got, want).astype(np.int64) - first
    only_ref = np.setdiff1d(want, got).astype(np.int64) - first
    if len(only_gpu) or len(only_ref):
        cut = o_tput[want.astype(np.int64) - first].min()        # the S-th best oracle score
        assert np.all(np.abs(o_tput[only_gpu] - cut) <= TPUT_RTOL * cut)
        assert np.all(np.abs(o_tput[only_ref] - cut) <= TPUT_RTOL * cut)
    assert np.all((o_reason[got.astype(np.int64) - first] & 0x7F) == 0)
    return len(only_gpu)


@pytest.mark.parametrize("s_max", [1, 50, 3000, 10 ** 6])
def test_select_survivors_against_the_oracles_own_scores(s_max):
    """End to end: device scores (fp32) -> device selection, against oracle scores (fp64) -> oracle selection."""
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15), rules=dict(enforce_realizability=0))
    plan, orc = _plan(cfg), Oracle(cfg)
    out = plan.score(k=0)
    got, _ = _select(plan, out["reason"], out["tput"], s_max)
    o_reason, o_tput, _, _ = orc.score_range(threads=8)
    _check_selection_against_oracle_scores(got, orc, o_reason, o_tput, 0, s_max)
    plan.close()


def test_select_with_many_equal_scores_and_subrange():
    """Serving-like ties do not exist in training spaces, so force them: two kernel variants with identical
    tables make every score appear twice; the cut must fall on the smaller indices."""
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15))
    for kv in (1, 2, 3):
        cfg["kern"][kv] = dict(cfg["kern"][0])
    plan, orc = _plan(cfg), Oracle(cfg)
    first, count = 1000, 100_003
    out = plan.score(first=first, count=count, k=0)
    reason = out["reason"].cpu().numpy()
    tput = out["tput"].cpu().numpy().astype(np.float64)
    for s_max in (7, 500, 501, 4000):
        got, _ = _select(plan, out["reason"], out["tput"], s_max, first=first)
        want = orc.select_survivors(reason, tput, first, s_max)
        np.testing.assert_array_equal(got, want)
    plan.close()


def test_select_excludes_plans_outside_the_simulator_domain():
    cfg = variant("large_unconstrained", cluster=dict(budget_bytes=10 ** 15))
    cfg["model"]["L"] = 128
    cfg["axes"][4] = ("v", [1, 2, 9])
    cfg["axes"][5] = ("ep", [8, 64])
    cfg["axes"][6] = ("pp", [1, 4, 32, 64])
    cfg["axes"][7] = ("tp", [1, 2])
    cfg["axes"][8] = ("dp", [8, 16, 64])
    plan, orc = _plan(cfg), Oracle(cfg)
    out = plan.score(k=0)
    reason = out["reason"].cpu().numpy()
    tput = out["tput"].cpu().numpy().astype(np.float64)
    got, _ = _select(plan, out["reason"], out["tput"], 10 ** 6)
    want = orc.select_survivors(reason, tput, 0, 10 ** 6)
    np.testing.assert_array_equal(got, want)
    feas = int(((reason & 0x7F) == 0).sum())
    assert 0 < len(got) < feas          # some feasible plans have pp = 64 or 9 virtual stages
    plan.close()


def _sim_parity(cfg, idx, seed=4, k=100):
    plan, orc = _plan(cfg), Oracle(cfg)
    tput_sim, status, tk_idx, tk_sc = _simulate(plan, idx, seed, k)
    want, want_st, _ = orc.simulate_list(idx, seed, threads=16)
    np.testing.assert_array_equal(status, want_st)
    np.testing.assert_allclose(tput_sim, want, rtol=TPUT_RTOL, atol=0)
    ok = want > 0
    ref_idx, ref_sc = Oracle.topk_list(idx[ok], want[ok], k)
    check_topk(tk_idx, tk_sc, ref_idx, ref_sc)
    plan.close()
    return tput_sim, status


def test_simulate_every_schedule_class_small():
    """All feasible candidates of a space with 1F1B, interleaved and DualPipe-style plans, pp up to 8."""
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15), rules=dict(enforce_realizability=0))
    orc = Oracle(cfg)
    reason, _, _, _ = orc.score_range(threads=8)
    idx = np.flatnonzero((reason & 0x7F) == 0).astype(np.uint64)
    assert len(idx) > 3000
    kinds = {orc.eval(int(i))["kind"] for i in idx[::97]}
    assert kinds == {0, 1, 2}
    _, status = _sim_parity(cfg, idx)
    assert np.all(status == 0)


def test_simulate_deep_pipelines_and_long_windows():
    """pp up to 32, up to 8 virtual stages, m beyond the 64-microbatch window, uneven layer splits."""
    cfg = variant("large_unconstrained", cluster=dict(budget_bytes=10 ** 15))
    for kn in cfg["kern"]:
        kn["avail_mask"] = 255
    orc = Oracle(cfg)
    picks = []
    for sched, v in ((0, 1), (1, 1), (2, 2), (2, 3), (2, 7), (3, 1)):
        for pp in (1, 2, 4, 8, 16, 32):
            for mb, dp in ((1, 8), (15, 64), (16, 32), (5, 1024 // max(pp, 1) // 2)):
                for rec in (0, 1, 2):
                    i = axis_index(cfg, kv=1, rec=rec, sched=sched, mb=mb, v=v, ep=8, pp=pp, tp=2, dp=dp)
                    if orc.eval(i)["reason"] & 0x7F == 0:
                        picks.append(i)
    idx = np.unique(np.array(picks, dtype=np.uint64))
    assert len(idx) > 100
    ds = [orc.eval(int(i)) for i in idx]
    assert {d["kind"] for d in ds} == {0, 1, 2}
    assert max(d["pp"] for d in ds) == 32 and max(d["Q"] for d in ds) > 32
    assert any(d["m"] > 64 for d in ds) and any(d["m"] < 64 for d in ds)
    _, status = _sim_parity(cfg, idx, k=64)
    assert np.all(status == 0)


def test_simulate_every_interleaved_shape_of_the_large_space():
    """Interleaved schedules keep their timelines on a ring of 2 pp microbatch slots per stage where that is smaller;
    a ring that were too short for some shape would leave its readers waiting (status STALL).  Every interleaved
    shape the large space offers -- pp 1..32, 1..8 virtual stages, every microbatch size, short and long windows --
    must finish and agree with the oracle.  (The list is repeated so that the call is large enough for the rings to
    be used: small calls keep full timelines, which are faster per simulated op.)"""
    cfg = variant("large_unconstrained", cluster=dict(budget_bytes=10 ** 15))
    for kn in cfg["kern"]:
        kn["avail_mask"] = 255
    orc = Oracle(cfg)
    axes = dict(cfg["axes"])
    picks = []
    for v in axes["v"]:
        for pp in (1, 2, 4, 8, 16, 32):
            for mb in axes["mb"]:
                for dp in (8, 32, 256):
                    i = axis_index(cfg, kv=1, rec=0, sched=2, mb=mb, v=v, ep=8, pp=pp, tp=2, dp=dp)
                    if orc.eval(i)["reason"] & 0x7F == 0:
                        picks.append(i)
    idx = np.unique(np.array(picks, dtype=np.uint64))
    ds = [orc.eval(int(i)) for i in idx]
    assert len(idx) > 300 and {d["kind"] for d in ds} == {1}
    assert {d["v_eff"] for d in ds} == set(range(2, 9)) and {d["pp"] for d in ds} == {2, 4, 8, 16}
    assert any(d["m"] >= 64 and d["pp"] * 2 < 64 for d in ds)          # rings that wrap
    assert any(d["m"] <= 2 * d["pp"] for d in ds)                      # and windows too short to need one
    _, status = _sim_parity(cfg, idx, k=64)                            # a small call: full timelines
    assert np.all(status == 0)
    big = np.tile(idx, 80)                                             # 40,320 entries: ring timelines
    plan = _plan(cfg)
    tput_big, status_big, _, _ = _simulate(plan, big, 4, 16)
    plan.close()
    want, want_st, _ = orc.simulate_list(idx, 4, threads=16)
    assert np.all(status_big == 0)
    np.testing.assert_allclose(tput_big, np.tile(want, 80), rtol=TPUT_RTOL, atol=0)


def test_simulate_infeasible_and_out_of_domain_entries():
    cfg = variant("large_unconstrained", cluster=dict(budget_bytes=10 ** 15))
    cfg["model"]["L"] = 128
    for kn in cfg["kern"]:
        kn["avail_mask"] = 255
    orc = Oracle(cfg)
    a = axis_index(cfg, sched=0, pp=64, tp=1, dp=16, ep=16, mb=1, v=1)     # feasible, 64 ranks: unsupported
    b = axis_index(cfg, sched=0, pp=3, tp=1, dp=16, ep=16, mb=1, v=1) if 3 in dict(cfg["axes"])["pp"] else 1
    c = axis_index(cfg, sched=0, pp=4, tp=1, dp=16, ep=16, mb=1, v=1)
    idx = np.array(sorted({a, b, c, 0}), dtype=np.uint64)
    plan = _plan(cfg)
    tput_sim, status, _, _ = _simulate(plan, idx, 4, 0)
    want, want_st, _ = orc.simulate_list(idx, 4)
    np.testing.assert_array_equal(status, want_st)
    np.testing.assert_allclose(tput_sim, want, rtol=TPUT_RTOL, atol=0)
    assert set(status.tolist()) == {0, 1}
    plan.close()


def test_jitter_seed_changes_scores_deterministically():
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15))
    orc = Oracle(cfg)
    reason, _, _, _ = orc.score_range(threads=8)
    idx = np.flatnonzero((reason & 0x7F) == 0).astype(np.uint64)[:500]
    plan = _plan(cfg)
    a, _, _, _ = _simulate(plan, idx, 4, 0)
    b, _, _, _ = _simulate(plan, idx, 4, 0)
    c, _, _, _ = _simulate(plan, idx, 5, 0)
    np.testing.assert_array_equal(a, b)
    assert np.mean(a != c) > 0.9
    plan.close()


def test_large_space_simulator_tier_end_to_end():
    """score -> select -> simulate -> re-rank on the 1.8e8 space, device side, against the oracle run on the
    same survivor list."""
    import torch
    for name in ("large", "large_unconstrained"):
        cfg = make_config(name)
        plan, orc = _plan(cfg), Oracle(cfg)
        out = plan.score(k=1024)
        got, sel = _select(plan, out["reason"], out["tput"], 10 ** 6)
        reason = out["reason"].cpu().numpy()
        tput = out["tput"].cpu().numpy().astype(np.float64)
        want = orc.select_survivors(reason, tput, 0, 10 ** 6)
        np.testing.assert_array_equal(got, want)
        sim = plan.simulate(sel["surv_idx"], 10 ** 6, 4, k=100, d_n=sel["surv_count"])
        torch.cuda.synchronize()
        n = len(got)
        ts = sim["tput_sim"][:n].cpu().numpy()
        st = sim["sim_status"][:n].cpu().numpy()
        ref, ref_st, _ = orc.simulate_list(got, 4, threads=64)
        np.testing.assert_array_equal(st, ref_st)
        np.testing.assert_allclose(ts, ref, rtol=TPUT_RTOL, atol=0)
        k = int(sim["topk_count"].item())
        ref_idx, ref_sc = Oracle.topk_list(got, ref, 100)
        check_topk(sim["topk_idx"].cpu().numpy().view(np.uint64)[:k], sim["topk_score"].cpu().numpy()[:k],
                   ref_idx, ref_sc)
        plan.close()
        del out, sel, sim
        torch.cuda.empty_cache()


def test_search_host_returns_the_same_results():
    import torch
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15), rules=dict(enforce_realizability=0))
    plan, orc = _plan(cfg), Oracle(cfg)
    N = plan.size
    ws = torch.empty(plan.search_workspace(128, 2000, 100), dtype=torch.uint8, device="cuda")
    h_reason = np.empty(N, dtype=np.uint8)
    h_tput = np.empty(N, dtype=np.float32)
    h_mem = np.empty(N, dtype=np.int64)
    r = plan.search_host(128, 2000, 100, 4, ws, h_reason=h_reason, h_tput=h_tput, h_mem=h_mem)
    reason, tput, mem, _ = orc.score_range(threads=8)
    np.testing.assert_array_equal(h_reason, reason)
    np.testing.assert_array_equal(h_mem, mem)
    feas = (reason & 0x7F) == 0
    np.testing.assert_allclose(h_tput[feas], tput[feas], rtol=TPUT_RTOL)
    idx, sc = orc.topk(reason, tput, 0, 128)
    check_topk(r["topk_idx"], r["topk_score"], idx, sc)
    surv = orc.select_survivors(h_reason, h_tput.astype(np.float64), 0, 2000)
    assert r["n_survivors"] == len(surv) == 2000
    ref, _, _ = orc.simulate_list(surv, 4, threads=8)
    ref_idx, ref_sc = Oracle.topk_list(surv, ref, 100)
    check_topk(r["sim_topk_idx"], r["sim_topk_score"], ref_idx, ref_sc)
    # dense outputs are optional
    r2 = plan.search_host(128, 2000, 100, 4, ws)
    np.testing.assert_array_equal(r2["topk_idx"], r["topk_idx"])
    np.testing.assert_array_equal(r2["sim_topk_idx"], r["sim_topk_idx"])
    plan.close()


def test_one_million_survivors_against_the_oracle():
    """The simulator tier at its nominal size: with the memory gate lifted the unconstrained large space has
    more than a million feasible plans, so select returns exactly 1e6 survivors.  The list is checked against the
    oracle's selection on the oracle's own scores (near-ties at the cut allowed), every one of the million
    simulations against the oracle's, and the re-ranked top-100 against the oracle's ranking of its own results."""
    import torch
    cfg = variant("large_unconstrained", cluster=dict(budget_bytes=10 ** 15))
    plan, orc = _plan(cfg), Oracle(cfg)
    out = plan.score(k=0)
    sel = plan.select_survivors(out["reason"], out["tput"], 10 ** 6)
    sim = plan.simulate(sel["surv_idx"], 10 ** 6, 4, k=100, d_n=sel["surv_count"])
    torch.cuda.synchronize()
    S = int(sel["surv_count"].item())
    assert S == 10 ** 6
    surv = sel["surv_idx"][:S].cpu().numpy().view(np.uint64)
    o_reason, o_tput, _, _ = orc.score_range(threads=64, want_mem=False)
    np.testing.assert_array_equal(out["reason"].cpu().numpy(), o_reason)
    _check_selection_against_oracle_scores(surv, orc, o_reason, o_tput, 0, 10 ** 6)
    del o_reason, o_tput
    ref, ref_st, _ = orc.simulate_list(surv, 4, threads=64)
    np.testing.assert_array_equal(sim["sim_status"][:S].cpu().numpy(), ref_st)
    np.testing.assert_allclose(sim["tput_sim"][:S].cpu().numpy(), ref, rtol=TPUT_RTOL, atol=0)
    k = int(sim["topk_count"].item())
    assert k == 100
    ref_idx, ref_sc = Oracle.topk_list(surv, ref, 100)
    check_topk(sim["topk_idx"].cpu().numpy().view(np.uint64)[:k], sim["topk_score"].cpu().numpy()[:k], ref_idx,
               ref_sc)
    plan.close()


def test_both_simulator_instances_give_the_same_bits_at_the_threshold():
    """A call of 32,767 survivors runs the small-call kernel (full timelines, eight-lane groups, plain indices), one
    of 32,768 the large-call kernel (ring timelines, four-lane groups, permuted indices).  The arithmetic per
    candidate is the same sequence of fp32 operations either way, so the survivors the two calls share must get the
    same bits; and a list with room for more than it holds must be served by the instance its actual length asks
    for."""
    import torch
    from paper_2607_18631_b200 import Plan
    plan = Plan(make_config("large_unconstrained"))
    b = plan.search(1024, 10 ** 6, 100, 4)
    torch.cuda.synchronize()
    ns = int(b["surv_count"].item())
    surv = b["surv_idx"][:ns].clone()
    T = 32768
    assert ns > T
    small = plan.simulate(surv[:T - 1].contiguous(), T - 1, 4)
    large = plan.simulate(surv[:T].contiguous(), T, 4)
    d_n = torch.tensor([T - 1], dtype=torch.int64, device="cuda")
    roomy = plan.simulate(surv.contiguous(), ns, 4, d_n=d_n)
    torch.cuda.synchronize()
    s_small, s_large = small["tput_sim"].cpu().numpy(), large["tput_sim"][:T - 1].cpu().numpy()
    assert (s_small > 0).all()
    np.testing.assert_array_equal(s_small, s_large)
    np.testing.assert_array_equal(small["sim_status"].cpu().numpy(), large["sim_status"][:T - 1].cpu().numpy())
    np.testing.assert_array_equal(s_small, roomy["tput_sim"][:T - 1].cpu().numpy())
    plan.close()
