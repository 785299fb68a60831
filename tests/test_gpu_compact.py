"""The compact view of dense scoring outputs (pf_compact, pf_search_host_compact) against the oracle: the reason
histogram is the bincount of the oracle's reason codes, the mask its feasibility bits, the records its feasible set
in ascending index order with its scores and byte counts."""
from __future__ import annotations

import numpy as np
import pytest

from oracle import Oracle
from workloads import make_config

from helpers import TPUT_RTOL, check_topk, variant

pytestmark = pytest.mark.gpu


def _plan(cfg):
    from paper_2607_18631_b200 import Plan
    return Plan(cfg)


def _check_view(hist, mask, recs, n_feasible, o_reason, o_tput, o_mem, first):
    count = len(o_reason)
    np.testing.assert_array_equal(hist[:12].astype(np.int64), np.bincount(o_reason & 0x7F, minlength=12)[:12])
    assert np.all(hist[12:] == 0)
    feas = (o_reason & 0x7F) == 0
    assert n_feasible == int(feas.sum())
    if mask is not None:
        bits = np.unpackbits(np.asarray(mask, dtype=np.uint8), bitorder="little")[:count].astype(bool)
        np.testing.assert_array_equal(bits, feas)
        assert not np.unpackbits(np.asarray(mask, dtype=np.uint8), bitorder="little")[count:].any()
    if recs is not None:
        want = np.flatnonzero(feas)[:len(recs)]
        np.testing.assert_array_equal(recs["idx"].astype(np.int64), want + first)
        np.testing.assert_array_equal(recs["mem"], o_mem[want])
        np.testing.assert_array_equal(recs["reason"], o_reason[want])
        np.testing.assert_allclose(recs["tput"], o_tput[want], rtol=TPUT_RTOL, atol=0)


@pytest.mark.parametrize("name,first,count", [("tiny", 0, None), ("mid", 0, None), ("mid", 1003, 70_001),
                                              ("serve", 16, 500_000)])
def test_compact_view_matches_the_oracle(name, first, count):
    import torch
    cfg = variant(name, cluster=dict(budget_bytes=10 ** 15)) if name == "mid" else make_config(name)
    plan, orc = _plan(cfg), Oracle(cfg)
    count = plan.size - first if count is None else count
    out = plan.score(first=first, count=count, k=0)
    o_reason, o_tput, o_mem, _ = orc.score_range(first, count, threads=8)
    n_feas = int(((o_reason & 0x7F) == 0).sum())
    for cap in (n_feas + 5, max(n_feas // 3, 1), 0):
        c = plan.compact(out["reason"], out["tput"], out["mem"], cap, first=first)
        torch.cuda.synchronize()
        n = int(c["n_feasible"].item())
        recs = plan.records_to_numpy(c["records"], min(n, cap)) if cap else None
        _check_view(c["hist"].cpu().numpy().astype(np.uint64), c["mask"].cpu().numpy(), recs, n, o_reason, o_tput,
                    o_mem, first)
    # without the mask and without the memory array
    c = plan.compact(out["reason"], out["tput"], None, n_feas, first=first, want_mask=False)
    torch.cuda.synchronize()
    recs = plan.records_to_numpy(c["records"], n_feas)
    assert np.all(recs["mem"] == 0)
    plan.close()


def test_search_host_compact_on_the_large_space():
    """The whole search through host buffers with the compact view: the 1.8e8-candidate space comes back as a
    histogram, 22.5 MB of feasibility bits and 12,905 records instead of 2.3 GB of dense arrays."""
    import torch
    cfg = make_config("large")
    plan, orc = _plan(cfg), Oracle(cfg)
    N = plan.size
    cap = 100_000
    ws = torch.empty(plan.search_compact_workspace(1024, 10 ** 6, 100, cap), dtype=torch.uint8, device="cuda")
    h_mask = np.empty((N + 7) // 8, dtype=np.uint8)
    r = plan.search_host_compact(1024, 10 ** 6, 100, 4, ws, cap, h_mask=h_mask)
    o_reason, o_tput, o_mem, _ = orc.score_range(threads=64)
    assert r["n_records"] == r["n_feasible"] == 12_905
    _check_view(r["hist"], r["mask"], r["records"][:r["n_records"]], r["n_feasible"], o_reason, o_tput, o_mem, 0)
    idx, sc = orc.topk(o_reason, o_tput, 0, 1024)
    check_topk(r["topk_idx"], r["topk_score"], idx, sc)
    surv = orc.select_survivors(o_reason, o_tput, 0, 10 ** 6)
    assert r["n_survivors"] == len(surv)
    ref, _, _ = orc.simulate_list(surv, 4, threads=64)
    ref_idx, ref_sc = Oracle.topk_list(surv, ref, 100)
    check_topk(r["sim_topk_idx"], r["sim_topk_score"], ref_idx, ref_sc)
    # the view is taken while the constant blocks of the dense arrays are still being streamed out: whatever the
    # workspace held before (all zero bytes read as "feasible everywhere") must not show in it
    for poison in (0, 0x85):
        ws.fill_(poison)
        h_mask2 = np.full((N + 7) // 8, 0xFF, dtype=np.uint8)
        rp = plan.search_host_compact(1024, 10 ** 6, 100, 4, ws, cap, h_mask=h_mask2)
        np.testing.assert_array_equal(rp["hist"], r["hist"])
        np.testing.assert_array_equal(h_mask2, h_mask)
        assert rp["n_records"] == r["n_records"]
        np.testing.assert_array_equal(rp["records"][:rp["n_records"]], r["records"][:r["n_records"]])
        np.testing.assert_array_equal(rp["sim_topk_idx"], r["sim_topk_idx"])
    # pinned host buffers take the bits and the records beside the search (pageable ones, above, at its end)
    from paper_2607_18631_b200 import binding
    p_mask = torch.full(((N + 7) // 8,), 0xFF, dtype=torch.uint8).pin_memory()
    p_recs = torch.zeros(cap * binding.RECORD_DTYPE.itemsize, dtype=torch.uint8).pin_memory()
    ws.fill_(0x85)
    rq = plan.search_host_compact(1024, 10 ** 6, 100, 4, ws, cap, h_mask=p_mask, h_records=p_recs)
    np.testing.assert_array_equal(rq["hist"], r["hist"])
    np.testing.assert_array_equal(p_mask.numpy(), h_mask)
    assert rq["n_records"] == r["n_records"] and rq["n_survivors"] == r["n_survivors"]
    q_recs = p_recs.numpy().view(binding.RECORD_DTYPE)[:rq["n_records"]]
    np.testing.assert_array_equal(q_recs, r["records"][:r["n_records"]])
    np.testing.assert_array_equal(rq["topk_idx"], r["topk_idx"])
    np.testing.assert_array_equal(rq["sim_topk_idx"], r["sim_topk_idx"])
    np.testing.assert_array_equal(rq["sim_topk_score"], r["sim_topk_score"])
    # the device writes into the pinned mask itself: nothing outside it may change, and a mask that starts at an odd
    # address (the device writes whole words) must come out the same
    nb = (N + 7) // 8
    for lead in (64, 61):
        guard = torch.full((lead + nb + 64,), 0xA5, dtype=torch.uint8).pin_memory()
        ws.fill_(0)
        rg = plan.search_host_compact(1024, 10 ** 6, 100, 4, ws, cap, h_mask=guard[lead:lead + nb], h_records=p_recs)
        g = guard.numpy()
        np.testing.assert_array_equal(g[lead:lead + nb], h_mask)
        assert (g[:lead] == 0xA5).all() and (g[lead + nb:] == 0xA5).all()
        np.testing.assert_array_equal(rg["hist"], r["hist"])
    # records and mask are optional, and a short record buffer is filled from the front
    r2 = plan.search_host_compact(1024, 10 ** 6, 100, 4, ws, 1000)
    assert r2["n_feasible"] == 12_905 and r2["n_records"] == 1000
    np.testing.assert_array_equal(r2["records"][:1000]["idx"], r["records"][:1000]["idx"])
    np.testing.assert_array_equal(r2["hist"], r["hist"])
    r3 = plan.search_host_compact(1024, 10 ** 6, 100, 4, ws, 0)
    assert r3["n_feasible"] == 12_905 and r3["records"] is None
    plan.close()


@pytest.mark.parametrize("name,k,s_max,k_sim", [("mid", 64, 1000, 10), ("tiny", 16, 100, 5), ("serve", 64, 0, 0)])
def test_search_host_compact_small_spaces_pinned_and_pageable(name, k, s_max, k_sim):
    """The host call's two ways of filling the mask (device writes into a pinned buffer over a copy of zeros; one copy
    into a pageable one) on spaces whose last chunk is partial, with the mask at an even and at an odd address, on a
    training space with and a serving space without the simulator tier."""
    import torch
    cfg = make_config(name)
    plan, orc = _plan(cfg), Oracle(cfg)
    N = plan.size
    reason, _, _, _ = orc.score_range(threads=8)
    feas = (reason & 0x7F) == 0
    n_feas = int(feas.sum())
    cap = n_feas + 10
    ks = max(k_sim, 1) if s_max else 0
    ws = torch.empty(plan.search_compact_workspace(k, s_max, ks, cap), dtype=torch.uint8, device="cuda")
    nb = (N + 7) // 8
    for pinned in (False, True):
        for lead in (0, 3):
            buf = torch.full((lead + nb + 8,), 0xA5, dtype=torch.uint8)
            if pinned:
                buf = buf.pin_memory()
            ws.fill_(0x85)
            r = plan.search_host_compact(k, s_max, ks, 4, ws, cap, h_mask=buf[lead:lead + nb])
            g = buf.numpy()
            bits = np.unpackbits(g[lead:lead + nb], bitorder="little")[:N].astype(bool)
            np.testing.assert_array_equal(bits, feas)
            assert (g[:lead] == 0xA5).all() and (g[lead + nb:] == 0xA5).all()
            assert r["n_feasible"] == n_feas and r["n_records"] == n_feas
            np.testing.assert_array_equal(r["records"][:n_feas]["idx"], np.nonzero(feas)[0].astype(np.uint64))
    plan.close()
