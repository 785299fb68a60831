"""GPU parity of pf_score against the CPU oracle, element by element, through the C ABI."""
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


def _full_parity(cfg, threads=8):
    plan, orc = _plan(cfg), Oracle(cfg)
    assert plan.size == orc.size
    reason, tput, mem, _ = orc.score_range(threads=threads)
    res = gpu_score(plan, k=cfg["k"])
    compare_dense(res, reason, tput, mem)
    compare_topk(res, orc, reason, tput, 0, cfg["k"])
    plan.close()
    return reason


@pytest.mark.parametrize("name", ["tiny", "mid", "serve"])
def test_small_spaces_full_parity(name):
    reason = _full_parity(make_config(name))
    assert ((reason & 0x7F) == 0).sum() > 0


def test_mid_variants_dense_in_feasible_candidates():
    """The stock mid space admits only 80 plans; lift the budget (and the dry-run rules) so that thousands
    of candidates reach the cost model and the block top-k has to prune."""
    big = 10 ** 15
    r = _full_parity(variant("mid", cluster=dict(budget_bytes=big)))
    assert ((r & 0x7F) == 0).sum() > 1500
    r = _full_parity(variant("mid", cluster=dict(budget_bytes=big), rules=dict(enforce_realizability=0)))
    assert ((r & 0x7F) == 0).sum() > 3000
    cfg = variant("mid", cluster=dict(budget_bytes=big), rules=dict(ep_scope=0))
    cfg["k"] = 1024
    _full_parity(cfg)


def test_serve_variant_all_kernels_available():
    cfg = variant("serve", cluster=dict(budget_bytes=10 ** 15))
    for k in cfg["kern"]:
        k["avail_mask"] = 255
    cfg["k"] = 1024
    _full_parity(cfg)


def test_dense_space_with_exact_ties_prunes_the_block_buffers():
    """Nearly every candidate feasible and every score repeated 64 times (the kernel-variant axis lists each
    variant 64 times): each block sees thousands of admissible keys, so its shared-memory buffer is pruned
    repeatedly, and the cut at k falls inside a run of exact ties that only the index order resolves."""
    cfg = variant("large", cluster=dict(budget_bytes=10 ** 15), rules=dict(world_min=1, enforce_realizability=0))
    for kn in cfg["kern"]:
        kn["avail_mask"] = 255
    cfg["axes"] = [("kv", [i % 8 for i in range(512)]), ("rec", [0, 1, 2]), ("sched", [0, 1]),
                   ("mb", [1, 2, 4, 8, 16]), ("v", [1]), ("ep", [1, 2, 4, 8]), ("pp", [1]), ("tp", [1, 2, 4, 8]),
                   ("dp", [8, 16, 32, 64, 128, 256, 512, 1024]), ("world", [0])]
    for k in (1024, 100):
        cfg["k"] = k
        r = _full_parity(cfg)
    assert ((r & 0x7F) == 0).mean() > 0.5 and len(r) == 1_966_080


def test_derived_axes_and_wide_integers():
    """dp derived from the world size; and a space whose products need the 64-bit rule path."""
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15))
    cfg["axes"][8] = ("dp", [0])
    _full_parity(cfg)
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15, G=8), rules=dict(world_min=1, world_max=1 << 20))
    cfg["workload"]["gbs"] = 3 * (1 << 31)
    cfg["axes"][8] = ("dp", [1, 2, 4, 1 << 19, 1 << 20])
    cfg["axes"][9] = ("world", [0])
    _full_parity(cfg)


def test_ranges_chunks_and_alignment():
    """pf_score on sub-ranges with ragged, unaligned starts; chunk top-k lists merged with pf_topk_merge
    equal the top-k of the whole space."""
    import torch
    from paper_2607_18631_b200 import pf_topk_merge
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15))
    plan, orc = _plan(cfg), Oracle(cfg)
    reason, tput, mem, _ = orc.score_range(threads=8)
    k = 128
    for first, count in ((0, 1), (1, 7), (13, 4099), (431, 433), (110_000, 592), (5, 110_587)):
        res = gpu_score(plan, first=first, count=count, k=k)
        compare_dense(res, reason[first:first + count], tput[first:first + count], mem[first:first + count])
        compare_topk(res, orc, reason[first:first + count], tput[first:first + count], first, k)
    # three ragged chunks -> merge
    cuts = [0, 33_333, 77_001, plan.size]
    acc = None
    for a, b in zip(cuts[:-1], cuts[1:]):
        out = plan.score(first=a, count=b - a, k=k, dense=False)
        cur = (out["topk_idx"], out["topk_score"], out["topk_count"])
        acc = cur if acc is None else pf_topk_merge(k, *acc, *cur)
    torch.cuda.synchronize()
    n = int(acc[2].item())
    idx, sc = orc.topk(reason, tput, 0, k)
    assert n == len(idx)
    from helpers import check_topk
    check_topk(acc[0].cpu().numpy().view(np.uint64)[:n], acc[1].cpu().numpy()[:n], idx, sc)
    plan.close()


def test_optional_outputs_and_errors():
    import torch
    from paper_2607_18631_b200 import PlanfrontError
    cfg = make_config("tiny")
    plan, orc = _plan(cfg), Oracle(cfg)
    reason, tput, mem, _ = orc.score_range()
    # top-k only (no dense outputs)
    res = gpu_score(plan, k=16, dense=False)
    compare_topk(res, orc, reason, tput, 0, 16)
    # dense only
    res = gpu_score(plan, k=0)
    compare_dense(res, reason, tput, mem)
    # single outputs
    r = torch.full((plan.size,), 77, dtype=torch.uint8, device="cuda")
    plan.score(k=0, reason=r, dense=False)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(r.cpu().numpy(), reason)
    with pytest.raises(PlanfrontError):
        plan.score(first=plan.size, count=1)
    with pytest.raises(PlanfrontError):
        plan.score(first=0, count=plan.size + 1)
    with pytest.raises(PlanfrontError):
        plan.score(k=2048)
    with pytest.raises(PlanfrontError):
        plan.score(k=4, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    # decode helper agrees with the axis lists
    t = plan.decode(150)
    d = orc.eval(150)
    assert (t["kv"], t["rec"], t["sched"], t["mb"], t["ep"], t["pp"], t["tp"]) == \
           (d["kv"], d["rec"], d["sched"], d["mb"], d["ep"], d["pp"], d["tp"])
    plan.close()


def test_invalid_specs_are_rejected():
    from paper_2607_18631_b200 import PlanfrontError
    for mutate in (lambda c: c["axes"].__setitem__(3, ("mb", [])),
                   lambda c: c["axes"].__setitem__(0, ("kv", [0, 5])),
                   lambda c: c["axes"].__setitem__(9, ("world", [0])),       # dp and world both derived
                   lambda c: c["model"].__setitem__("H", 0),
                   lambda c: c["axes"].pop()):
        cfg = make_config("tiny")
        mutate(cfg)
        with pytest.raises(PlanfrontError):
            _plan(cfg)


def test_large_space_full_size():
    """The 1.8e8-candidate space in the launch configuration the benchmark times: reason codes and bytes
    bit-exact over the WHOLE space, throughput on every feasible candidate, top-1024."""
    cfg = make_config("large")
    plan, orc = _plan(cfg), Oracle(cfg)
    assert plan.size == 179_908_608
    reason, tput, mem, _ = orc.score_range(threads=64)
    res = gpu_score(plan, k=1024)
    assert np.array_equal(res["reason"], reason)
    assert np.array_equal(res["mem"], mem)
    feas = (reason & 0x7F) == 0
    assert np.all(res["tput"][~feas] == 0.0)
    np.testing.assert_allclose(res["tput"][feas], tput[feas], rtol=1e-4, atol=0)
    compare_topk(res, orc, reason, tput, 0, 1024)
    plan.close()


def test_slab_order_table_follows_the_range_and_is_ignored_when_stale():
    """The plan keeps the slab visiting order of its latest pf_score range.  Alternating ranges rebuild it; a
    table that does not hold the call's range (here: its rebuild was only captured into a CUDA graph, not run)
    is ignored on the device and the call still gives the oracle's results."""
    import torch
    cfg = make_config("large")
    plan, orc = _plan(cfg), Oracle(cfg)
    ranges = ((50_000_000, 30_000_000), (12_345, 40_000_000), (50_000_000, 30_000_000))
    expect = {}
    for first, count in ranges:
        if (first, count) not in expect:
            expect[(first, count)] = orc.score_range(first, count, threads=64)
        reason, tput, mem, _ = expect[(first, count)]
        res = gpu_score(plan, first=first, count=count, k=256)
        compare_dense(res, reason, tput, mem)
        compare_topk(res, orc, reason, tput, first, 256)
    # capture a call on a new range: the table rebuild is recorded, not executed
    first, count = 100_000_000, 20_000_000
    reason, tput, mem, _ = orc.score_range(first, count, threads=64)
    out = plan.score(first=ranges[0][0], count=count, k=256)          # allocates the buffers, old range
    torch.cuda.synchronize()
    kw = dict(first=first, count=count, k=256, reason=out["reason"], tput=out["tput"], mem=out["mem"],
              topk_idx=out["topk_idx"], topk_score=out["topk_score"], topk_count=out["topk_count"],
              workspace=out["workspace"])
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        plan.score(**kw)

    def check():
        torch.cuda.synchronize()
        res = dict(reason=out["reason"].cpu().numpy(), tput=out["tput"].cpu().numpy(), mem=out["mem"].cpu().numpy())
        n = int(out["topk_count"].item())
        res["topk_idx"] = out["topk_idx"].cpu().numpy().view(np.uint64)[:n]
        res["topk_score"] = out["topk_score"].cpu().numpy()[:n]
        compare_dense(res, reason, tput, mem)
        compare_topk(res, orc, reason, tput, first, 256)

    out["reason"].fill_(99)
    plan.score(**kw)                # eager: the host believes the table is current, the device sees it is not
    check()
    out["reason"].fill_(99)
    graph.replay()                  # now the rebuild runs, followed by the scoring kernel
    check()
    out["reason"].fill_(99)
    plan.score(**kw)                # and the eager call uses the rebuilt table
    check()
    plan.close()


def test_large_unconstrained_topk():
    cfg = make_config("large_unconstrained")
    plan, orc = _plan(cfg), Oracle(cfg)
    first, count = 60_000_000, 40_000_000     # a slice keeps the oracle side short
    reason, tput, mem, _ = orc.score_range(first, count, threads=64)
    res = gpu_score(plan, first=first, count=count, k=1024)
    compare_dense(res, reason, tput, mem)
    compare_topk(res, orc, reason, tput, first, 1024)
    plan.close()


def test_degenerate_spaces():
    """Edge shapes: a 4096-entry axis, single-entry axes everywhere else, a space with no feasible plan at all
    (empty top-k, empty survivor list, empty simulation), k = 1."""
    import torch
    # (a) one long axis (the kernel-variant list repeated up to the axis limit), everything else fixed
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15))
    cfg["axes"] = [("kv", [i % 4 for i in range(4096)]), ("rec", [1]), ("sched", [0]), ("mb", [2]), ("v", [1]),
                   ("ep", [2]), ("pp", [2]), ("tp", [2]), ("dp", [2]), ("world", [8])]
    cfg["k"] = 1
    r = _full_parity(cfg)
    assert len(r) == 4096 and ((r & 0x7F) == 0).sum() > 3000
    # (b) a first axis longer than a slab may be: slabs degenerate to single candidates of the second axis
    cfg = variant("tiny")
    cfg["axes"][0] = ("kv", [i % 2 for i in range(3000)])
    cfg["k"] = 7
    _full_parity(cfg)
    # (c) nothing feasible: budget of one byte
    cfg = variant("mid", cluster=dict(budget_bytes=1))
    plan, orc = _plan(cfg), Oracle(cfg)
    reason, tput, mem, _ = orc.score_range(threads=8)
    assert ((reason & 0x7F) == 0).sum() == 0
    res = gpu_score(plan, k=128)
    compare_dense(res, reason, tput, mem)
    assert len(res["topk_idx"]) == 0
    out = plan.score(k=0)
    sel = plan.select_survivors(out["reason"], out["tput"], 1000)
    sim = plan.simulate(sel["surv_idx"], 1000, 4, k=10, d_n=sel["surv_count"])
    torch.cuda.synchronize()
    assert int(sel["surv_count"].item()) == 0 and int(sim["topk_count"].item()) == 0
    assert torch.all(sim["topk_idx"] == -1)
    plan.close()
