"""pf_score_static: the no-allocation variant of pf_score, through the C ABI.

Some users of the library cannot allocate device memory at the point where they score plans: their GPU memory
was handed to a pool at start-up, or they run in a loop that must not hit the device-wide synchronization an
allocation implies, or they are a plugin that only ever receives buffers.  For them the workspace of pf_score
is replaced by an array built into the library.  This test makes the variant's call the first scoring call on a fresh plan (its
set-up -- the look-up of the array's device address -- runs before anything else has touched the library's
kernels), calls it twice in a row on the same buffers' worth of work (the array keeps the first call's contents,
so the second call checks that everything that must start from zero is cleared), compares both calls with the
ordinary entry point and with the CPU oracle, and checks that a call leaves the device's free memory and the
process's allocator counters where they were.

Collected last on purpose: a run that stops at the first failure has then already run every other test.
"""
from __future__ import annotations

import numpy as np
import pytest

from gpu_common import compare_dense, compare_topk
from helpers import TPUT_RTOL, check_topk, variant

pytestmark = pytest.mark.gpu


def test_static_scratch_variant_matches_pf_score_twice_in_a_row():
    import torch
    from paper_2607_18631_b200 import Plan, PlanfrontError
    from paper_2607_18631_b200.binding import PF_EWORKSPACE, STATIC_SCRATCH_BYTES

    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15), rules=dict(enforce_realizability=0))
    plan = Plan(cfg)
    N, k = plan.size, 128
    assert plan.score_workspace(N, k) <= STATIC_SCRATCH_BYTES

    # every buffer the static variant needs is allocated here, before the calls
    reason = torch.empty(N, dtype=torch.uint8, device="cuda")
    tput = torch.empty(N, dtype=torch.float32, device="cuda")
    mem = torch.empty(N, dtype=torch.int64, device="cuda")
    tk_idx = torch.empty(k, dtype=torch.int64, device="cuda")
    tk_sc = torch.empty(k, dtype=torch.float32, device="cuda")
    tk_cnt = torch.empty(1, dtype=torch.int32, device="cuda")
    got = []
    unchanged = []
    for call in range(3):
        reason.fill_(0xEE)
        tput.fill_(-1.0)
        mem.fill_(-1)
        tk_cnt.fill_(-1)
        torch.cuda.synchronize()
        before = (torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_reserved())
        plan.score_static(reason, tput, mem, k, tk_idx, tk_sc, tk_cnt)   # call 0: the plan's first scoring call
        torch.cuda.synchronize()
        after = (torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_reserved())
        # the process's allocator never moves; the device's free memory may move on the first call only (the
        # runtime may load the library's device image then)
        assert after[1:] == before[1:], f"call {call}"
        unchanged.append(after[0] == before[0])
        got.append(dict(reason=reason.cpu().numpy(), tput=tput.cpu().numpy(), mem=mem.cpu().numpy(),
                        n=int(tk_cnt.item()), idx=tk_idx.cpu().numpy().view(np.uint64).copy(),
                        sc=tk_sc.cpu().numpy().copy()))
    assert any(unchanged[1:]), "free device memory changed across every repeated call"

    ref = plan.score(k=k)                      # ordinary entry point, caller-provided workspace
    torch.cuda.synchronize()
    n_ref = int(ref["topk_count"].item())
    ref_idx = ref["topk_idx"].cpu().numpy().view(np.uint64)[:n_ref]
    ref_sc = ref["topk_score"].cpu().numpy()[:n_ref]
    assert n_ref == k
    import oracle
    orc = oracle.Oracle(cfg)
    o_reason, o_tput, o_mem, _ = orc.score_range(threads=8)
    for call, g in enumerate(got):
        np.testing.assert_array_equal(g["reason"], ref["reason"].cpu().numpy(), err_msg=f"call {call}")
        np.testing.assert_array_equal(g["mem"], ref["mem"].cpu().numpy(), err_msg=f"call {call}")
        np.testing.assert_allclose(g["tput"], ref["tput"].cpu().numpy(), rtol=TPUT_RTOL, atol=0)
        assert g["n"] == n_ref
        check_topk(g["idx"][:g["n"]], g["sc"][:g["n"]], ref_idx, ref_sc)
        # and against the oracle, like every other scoring call
        res = dict(reason=g["reason"], tput=g["tput"], mem=g["mem"], topk_idx=g["idx"][:g["n"]],
                   topk_score=g["sc"][:g["n"]])
        compare_dense(res, o_reason, o_tput, o_mem)
        compare_topk(res, orc, o_reason, o_tput, 0, k)

    # a sub-range and a top-k-only call share the same array without trouble
    tk_cnt.fill_(-1)
    plan.score_static(None, None, None, 16, tk_idx, tk_sc, tk_cnt, first=1000, count=50_000)
    sub = plan.score(first=1000, count=50_000, k=16, dense=False)
    torch.cuda.synchronize()
    assert int(tk_cnt.item()) == int(sub["topk_count"].item())
    np.testing.assert_array_equal(tk_idx[:16].cpu().numpy(), sub["topk_idx"].cpu().numpy())
    plan.close()

    # a request that does not fit the built-in array is refused, not truncated
    # (the 1.8e8-candidate space with k = 1024 wants several hundred blocks' key lists, more than the array)
    big = Plan(variant("large"))
    assert big.score_workspace(big.size, 1024) > STATIC_SCRATCH_BYTES
    big_idx = torch.empty(1024, dtype=torch.int64, device="cuda")
    big_sc = torch.empty(1024, dtype=torch.float32, device="cuda")
    with pytest.raises(PlanfrontError) as e:
        big.score_static(None, None, None, 1024, big_idx, big_sc, tk_cnt)
    assert e.value.status == PF_EWORKSPACE
    big.close()
