"""The one-call search on device buffers (pf_search): same results as pf_score -> pf_select_survivors -> pf_simulate
called one after the other, on spaces where the selection keeps everything and where it has to cut."""
from __future__ import annotations

import numpy as np
import pytest

from workloads import make_config

from helpers import variant

pytestmark = pytest.mark.gpu


def _plan(cfg):
    from paper_2607_18631_b200 import Plan
    return Plan(cfg)


def _separate(plan, k, s_max, k_sim, seed):
    import torch
    out = plan.score(k=k)
    sel = plan.select_survivors(out["reason"], out["tput"], s_max)
    sim = plan.simulate(sel["surv_idx"], s_max, seed, k=k_sim, d_n=sel["surv_count"], dense=False)
    torch.cuda.synchronize()
    return out, sel, sim


def _same(plan, k, s_max, k_sim, seed=4):
    import torch
    out, sel, sim = _separate(plan, k, s_max, k_sim, seed)
    b = plan.search(k, s_max, k_sim, seed)
    torch.cuda.synchronize()
    for key in ("reason", "tput", "mem", "topk_idx", "topk_score", "topk_count"):
        assert torch.equal(out[key], b[key]), key
    n = int(sel["surv_count"].item())
    assert int(b["surv_count"].item()) == n
    assert torch.equal(sel["surv_idx"][:n], b["surv_idx"][:n])
    assert torch.equal(sim["topk_count"], b["sim_topk_count"])
    c = int(sim["topk_count"].item())
    assert torch.equal(sim["topk_idx"][:c], b["sim_topk_idx"][:c])
    assert torch.equal(sim["topk_score"][:c], b["sim_topk_score"][:c])
    # a second call on the same buffers gives the same again (the scratch is re-initialised by the call)
    b2 = plan.search(k, s_max, k_sim, seed, bufs=b)
    torch.cuda.synchronize()
    assert int(b2["surv_count"].item()) == n and torch.equal(sel["surv_idx"][:n], b2["surv_idx"][:n])
    return n


@pytest.mark.parametrize("s_max", [10 ** 6, 700, 1])
def test_search_equals_the_three_calls_mid(s_max):
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15), rules=dict(enforce_realizability=0))
    plan = _plan(cfg)
    n = _same(plan, 128, s_max, 100)
    assert n == min(s_max, n) and n > 0
    plan.close()


def test_search_equals_the_three_calls_large_and_out_of_domain_plans():
    plan = _plan(make_config("large"))
    assert _same(plan, 1024, 10 ** 6, 100) == 12_905
    plan.close()
    # feasible plans outside the simulator's domain must not reach the digest
    cfg = variant("large_unconstrained", cluster=dict(budget_bytes=10 ** 15))
    cfg["model"]["L"] = 128
    cfg["axes"][4] = ("v", [1, 2, 9])
    cfg["axes"][5] = ("ep", [8, 64])
    cfg["axes"][6] = ("pp", [1, 4, 32, 64])
    cfg["axes"][7] = ("tp", [1, 2])
    cfg["axes"][8] = ("dp", [8, 16, 64])
    plan = _plan(cfg)
    _same(plan, 256, 5000, 64)
    _same(plan, 256, 10 ** 6, 64)
    plan.close()


def test_search_on_a_serving_space_scores_only():
    import torch
    plan = _plan(make_config("serve"))
    out = plan.score(k=128)
    b = plan.search(128, 1000, 10, 4)
    torch.cuda.synchronize()
    for key in ("reason", "tput", "mem", "topk_idx", "topk_score", "topk_count"):
        assert torch.equal(out[key], b[key]), key
    plan.close()


def test_search_replays_from_a_cuda_graph():
    """The whole search enqueues on one stream without synchronizing or allocating, so it can be captured once and
    replayed; each replay re-initialises its scratch and gives the same results."""
    import torch
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15), rules=dict(enforce_realizability=0))
    plan = _plan(cfg)
    b = plan.search(128, 2000, 100, 4)                 # allocates the buffers, builds the plan's order table
    torch.cuda.synchronize()
    want = {k: v.clone() for k, v in b.items() if k != "workspace"}
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        plan.search(128, 2000, 100, 4, bufs=b)
    for _ in range(3):
        for k in ("reason", "surv_idx", "sim_topk_score"):
            b[k].zero_()
        graph.replay()
        torch.cuda.synchronize()
        n = int(b["surv_count"].item())
        assert n == int(want["surv_count"].item()) == 2000
        for k in ("reason", "tput", "mem", "topk_idx", "topk_score", "sim_topk_idx", "sim_topk_score"):
            assert torch.equal(b[k], want[k]), k
        assert torch.equal(b["surv_idx"][:n], want["surv_idx"][:n])
    plan.close()


def test_search_ignores_what_the_output_buffers_held_before():
    """Inside one search the constant blocks of the dense outputs are streamed out while the selection already
    reads the evaluated ones.  Whatever the buffers held before the call -- here: every reason byte 0 ("feasible")
    and huge scores -- must not leak into the survivor list, and the dense outputs are complete when the call's
    stream work is done."""
    import torch
    import oracle
    plan = _plan(make_config("large"))
    orc = oracle.Oracle(make_config("large"))
    b = plan.search(1024, 10 ** 6, 100, 4)
    torch.cuda.synchronize()
    want = {k: v.clone() for k, v in b.items() if k != "workspace"}
    for s_max in (10 ** 6, 3000):
        b["reason"].zero_()
        b["tput"].fill_(3.0e38)
        b["mem"].fill_(-1)
        b["surv_idx"].fill_(-1)
        b = plan.search(1024, s_max, 100, 4, bufs=b)
        torch.cuda.synchronize()
        for key in ("reason", "tput", "mem", "topk_idx", "topk_score", "topk_count"):
            assert torch.equal(b[key], want[key]), key
        n = int(b["surv_count"].item())
        assert n == min(s_max, 12_905)
        if s_max >= 12_905:
            assert torch.equal(b["surv_idx"][:n], want["surv_idx"][:n])
        else:
            feas = torch.nonzero((want["reason"] & 0x7F) == 0).flatten()
            ref = orc.select_survivors(want["reason"].cpu().numpy(), want["tput"].cpu().numpy().astype(np.float64),
                                       0, s_max)
            assert np.array_equal(b["surv_idx"][:n].cpu().numpy().view(np.uint64), ref)
            assert n < feas.numel()
    plan.close()


def test_search_streams_constant_blocks_of_odd_size_exactly():
    """Blocks of 6,615 candidates: the constant blocks' reason / tput / mem spans start at every 16-byte phase, so the
    streaming kernel's bulk copies are preceded and followed by ragged ends.  The one-call search must give, byte
    for byte, what pf_score gives (which writes every block with plain stores), whatever the buffers held before;
    three ranges are also compared with the oracle."""
    import torch
    import oracle
    from helpers import TPUT_RTOL
    cfg = make_config("large")
    cut = {"kv": 7, "sched": 3, "mb": 15, "v": 7}
    cfg["axes"] = [(n, (list(v)[:cut[n]] if n in cut else v)) for n, v in cfg["axes"]]
    plan = _plan(cfg)
    assert plan.size == 6615 * 11 ** 4
    out = plan.score(k=256)
    b = plan.search(256, 10 ** 6, 50, 4)
    for fill in (0xFF, 0x00):
        b["reason"].fill_(fill)
        b["tput"].fill_(1.5e30)
        b["mem"].fill_(-7)
        b = plan.search(256, 10 ** 6, 50, 4, bufs=b)
        torch.cuda.synchronize()
        for key in ("reason", "tput", "mem", "topk_idx", "topk_score", "topk_count"):
            assert torch.equal(out[key], b[key]), key
    span = plan.fill_span()
    assert span["block_candidates"] == 6615 and span["n_blocks"] == 11 ** 4
    assert 0 < span["scored_blocks"] < span["n_blocks"]          # the streaming kernel had work to do
    orc = oracle.Oracle(cfg)
    for first in (0, 6615 * 5000 + 17, plan.size - 300_001):
        r, t, m, _ = orc.score_range(first, 300_001, threads=4)
        sl = slice(first, first + 300_001)
        assert np.array_equal(b["reason"][sl].cpu().numpy(), r)
        assert np.array_equal(b["mem"][sl].cpu().numpy(), m)
        assert np.allclose(b["tput"][sl].cpu().numpy(), t, rtol=TPUT_RTOL, atol=0)
    plan.close()


@pytest.mark.parametrize("name", ["large"])
def test_search_gives_the_same_bits_call_after_call(name):
    """Back-to-back calls overlap one call's last kernels with the next call's first ones on four streams (the
    caller's, two of the plan's, the chained launches in between); every output must come out bit for bit the
    same, whatever the buffers held."""
    import torch
    from paper_2607_18631_b200 import Plan
    plan = Plan(make_config(name))
    b = plan.search(1024, 10 ** 6, 100, 4)
    torch.cuda.synchronize()
    keys = ("reason", "tput", "mem", "topk_idx", "topk_score", "topk_count", "surv_count", "sim_topk_idx",
            "sim_topk_score", "sim_topk_count")
    ref = {k: b[k].clone() for k in keys}
    ns = int(ref["surv_count"].item())
    ref_surv = b["surv_idx"][:ns].clone()
    for it in range(120):
        if it % 3 == 0:
            b["reason"].fill_(0)
            b["tput"].fill_(7.0)
            b["mem"].fill_(-1)
        plan.search(1024, 10 ** 6, 100, 4, bufs=b)
        if it % 3 == 0 or it % 10 == 9:
            torch.cuda.synchronize()
            for k in keys:
                assert torch.equal(b[k], ref[k]), (it, k)
            assert torch.equal(b["surv_idx"][:ns], ref_surv), it
    plan.close()
