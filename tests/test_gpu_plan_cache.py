"""Plans take their device block, streams and events from per-device caches and hand them back when destroyed.
What one plan left in a block must not show in the next plan's results, and plans alive at the same time must not
share anything."""
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


def _parity(plan, cfg, ref):
    reason, tput, mem, orc = ref
    res = gpu_score(plan, k=cfg["k"])
    compare_dense(res, reason, tput, mem)
    compare_topk(res, orc, reason, tput, 0, cfg["k"])


def _ref(cfg):
    orc = Oracle(cfg)
    reason, tput, mem, _ = orc.score_range(threads=8)
    return reason, tput, mem, orc


def test_recycled_blocks_and_streams_give_the_same_results():
    cfgs = [make_config("mid"), make_config("tiny"), make_config("serve"),
            variant("mid", cluster=dict(budget_bytes=10 ** 15))]
    refs = [_ref(c) for c in cfgs]
    # one after the other: each plan gets the block the one before it released (training and serving plans, spaces of
    # different sizes: the block holds the former plan's tables wherever the new image does not reach)
    for rnd in range(3):
        for cfg, ref in zip(cfgs, refs):
            plan = _plan(cfg)
            _parity(plan, cfg, ref)
            plan.close()
    # several alive at once (more than the cache keeps), destroyed in another order than created, then again
    for rnd in range(2):
        plans = [_plan(c) for c in cfgs + cfgs]
        for plan, cfg, ref in zip(plans, cfgs + cfgs, refs + refs):
            _parity(plan, cfg, ref)
        for i in (3, 0, 6, 1, 7, 2, 5, 4):
            plans[i].close()


def test_search_after_recycling_matches_a_fresh_process_result():
    """The one-call search uses every cached resource (both streams, all events, the order table in the block)."""
    import torch
    cfg = make_config("mid")
    cfg_big = variant("mid", cluster=dict(budget_bytes=10 ** 15))
    first = None
    for rnd in range(4):
        # a plan of another space in between, so that the block and the order table it holds are really reused
        other = _plan(cfg_big if rnd % 2 else make_config("tiny"))
        other.search(64, 1000, 10, 3)
        torch.cuda.synchronize()
        other.close()
        plan = _plan(cfg)
        out = plan.search(64, 1000, 10, 3)
        torch.cuda.synchronize()
        nk, ns = int(out["topk_count"].item()), int(out["sim_topk_count"].item())
        got = {k: out[k].cpu().numpy().copy() for k in ("reason", "tput", "mem")}
        got["topk_idx"] = out["topk_idx"][:nk].cpu().numpy().copy()
        got["sim_topk_idx"] = out["sim_topk_idx"][:ns].cpu().numpy().copy()
        got["sim_topk_score"] = out["sim_topk_score"][:ns].cpu().numpy().copy()
        assert nk > 0 and ns > 0
        plan.close()
        if first is None:
            first = got
            orc = Oracle(cfg)
            reason, tput, mem, _ = orc.score_range(threads=8)
            np.testing.assert_array_equal(got["reason"], reason)
        else:
            for k in first:
                np.testing.assert_array_equal(got[k], first[k])


def test_plans_created_and_destroyed_from_several_threads():
    """The caches, and the kernels' shared-memory limits, are shared by every thread of the process (ctypes calls run
    without the interpreter lock): plans of different spaces scored and searched from four threads at once."""
    import threading
    import torch
    cfgs = [make_config("mid"), make_config("tiny"), variant("mid", cluster=dict(budget_bytes=10 ** 15))]
    refs = [_ref(c) for c in cfgs]

    def search_result(cfg):
        plan = _plan(cfg)
        out = plan.search(64, 1000, 10, 3)
        torch.cuda.current_stream().synchronize()
        ns = int(out["sim_topk_count"].item())
        res = (out["reason"].cpu().numpy().copy(), out["sim_topk_idx"][:ns].cpu().numpy().copy(),
               out["sim_topk_score"][:ns].cpu().numpy().copy(), int(out["surv_count"].item()))
        plan.close()
        return res
    searched = [search_result(c) for c in cfgs]
    errors = []

    def work(seed):
        try:
            torch.cuda.set_device(0)
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                for i in range(12):
                    j = (seed + i) % len(cfgs)
                    plan = _plan(cfgs[j])
                    _parity(plan, cfgs[j], refs[j])
                    plan.close()
                    got = search_result(cfgs[j])
                    for x, y in zip(got, searched[j]):
                        assert np.array_equal(x, y)
        except Exception as ex:   # noqa: BLE001 -- reported by the main thread
            errors.append(repr(ex))

    threads = [threading.Thread(target=work, args=(s,)) for s in range(4)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
