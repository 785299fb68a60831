"""Pins of the calibration-domain overlay (principle P4; Appendix "Testbeds and calibration domains"): every
calibrated constant carries the GPU, the dtypes and the tokens-per-expert range it was fit over; a query outside
is flagged extrapolated, never rejected or re-scored; with no domain attached nothing is flagged."""
from __future__ import annotations

import numpy as np

from oracle import Oracle
from workloads import make_config

from helpers import axis_index, variant

WHY_GPU, WHY_DTYPE, WHY_LOW, WHY_HIGH = 1, 2, 4, 8


def _roomy():
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15))
    for k in cfg["kern"]:
        k["avail_mask"] = 255
    return cfg


def test_paper_domain_is_the_default_and_its_range_is_inclusive():
    """The printed domain: m_range [64, 8192].  m_e = 64 and 8192 are inside, 48 and 24576 outside, on the
    low and on the high side."""
    cfg = _roomy()
    assert cfg["domain"] == dict(attached=1, gpu_id=-1, dtype_mask=0xFFFF, m_lo=64, m_hi=8192)
    cfg["domain"]["m_lo"], cfg["domain"]["m_hi"] = 96, 1536
    o = Oracle(cfg)
    # m_e = mb*4096*6*ep / (64*tp)
    for mb, ep, tp, me, why in ((1, 1, 8, 48, WHY_LOW), (1, 1, 4, 96, 0), (4, 1, 1, 1536, 0), (8, 1, 1, 3072, WHY_HIGH),
                                (8, 8, 1, 24576, WHY_HIGH)):
        d = o.eval(axis_index(cfg, kv=0, mb=mb, ep=ep, tp=tp, pp=1, dp=8 // tp, sched=0, v=1))
        assert d["m_e"] == me and d["why"] == why and bool(d["reason"] & 0x80) == (why != 0), d


def test_no_domain_attached_flags_nothing_and_scores_are_bit_identical():
    """An uncalibrated model is the factory model to the bit: the flag is the only thing a domain changes."""
    a, b = _roomy(), _roomy()
    b["domain"]["attached"] = 0
    ra, ta, ma, _ = Oracle(a).score_range()
    rb, tb, mb_, _ = Oracle(b).score_range()
    assert np.any(ra & 0x80) and not np.any(rb & 0x80)
    assert np.array_equal(ra & 0x7F, rb) and np.array_equal(ta, tb) and np.array_equal(ma, mb_)


def test_flag_marks_only_feasible_plans_and_never_changes_feasibility():
    cfg = make_config("mid")
    r, t, _, _ = Oracle(cfg).score_range()
    flagged = (r & 0x80) != 0
    assert np.all((r[flagged] & 0x7F) == 0) and np.all(t[flagged] > 0)


def test_another_gpu_or_an_uncovered_dtype_is_outside_the_domain():
    """A domain fit on GPU 7 says nothing about GPU 0: every feasible plan is extrapolated.  A domain covering
    bf16 only flags exactly the fp8 variants (and whatever the range flags)."""
    base = _roomy()
    base["kern"][3]["dtype"] = 1
    r0, _, _, _ = Oracle(base).score_range()
    feas = (r0 & 0x7F) == 0
    other = _roomy()
    other["kern"][3]["dtype"] = 1
    other["domain"]["gpu_id"] = 7
    r1, _, _, _ = Oracle(other).score_range()
    assert np.array_equal(r1 & 0x7F, r0 & 0x7F) and np.all((r1[feas] & 0x80) != 0)
    same = _roomy()
    same["kern"][3]["dtype"] = 1
    same["domain"]["gpu_id"] = 0
    assert np.array_equal(Oracle(same).score_range()[0], r0)
    bf16 = _roomy()
    bf16["kern"][3]["dtype"] = 1
    bf16["domain"]["dtype_mask"] = 1
    o2 = Oracle(bf16)
    r2, _, _, _ = o2.score_range()
    kv = np.arange(o2.size) % 4
    assert np.all((r2[feas & (kv == 3)] & 0x80) != 0)
    assert np.array_equal(r2[kv != 3], r0[kv != 3])
    d = o2.eval(int(np.flatnonzero(feas & (kv == 3) & ((r0 & 0x80) == 0))[0]))
    assert d["why"] == WHY_DTYPE


def test_serving_plans_carry_the_flag_too():
    cfg = make_config("serve")
    o = Oracle(cfg)
    r, _, _, _ = o.score_range(0, 200_000)
    feas = np.flatnonzero((r & 0x7F) == 0)
    assert len(feas) > 100
    for i in feas[:: max(1, len(feas) // 50)]:
        d = o.eval(int(i))
        assert bool(d["reason"] & 0x80) == (d["m_e"] < 64 or d["m_e"] > 8192)
        assert d["why"] == (WHY_LOW if d["m_e"] < 64 else WHY_HIGH if d["m_e"] > 8192 else 0)
