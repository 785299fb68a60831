"""Pins for the CPU oracle: every check here compares the oracle with something OTHER than itself --
numbers the paper prints, closed forms, brute-force counting on the tiny space, stated rule outcomes,
and invariants.  No GPU."""
from __future__ import annotations

import itertools

import numpy as np
import pytest

import oracle
from oracle import Oracle
from workloads import make_config
from workloads.configs import space_size

from helpers import axis_index, load_kv, load_rows, v2lite_like, variant

GB = 1e9


# ----------------------------------------------------------------------------- memory gate (paper numbers)

def test_budget_is_point_nine_of_capacity():
    """Sec. 2.1: 72 GB budget = 80 GB HBM at a 0.9 usable fraction (decimal GB)."""
    g = load_kv("paper_memory_gate.txt")
    assert oracle.budget_bytes(int(g["hbm_gb"] * GB)) == int(g["budget_gb"] * GB)
    assert oracle.budget_bytes(24_000_000_000) == 21_600_000_000


def test_expert_optimizer_state_is_ep_invariant_and_matches_paper():
    """Sec. 5 RQ1: the expert optimizer state is ep-invariant at 21.59 GB on dp = 8."""
    g = load_kv("paper_memory_gate.txt")
    o = Oracle(v2lite_like())
    vals = []
    for i in range(o.size):
        d = o.eval(i)
        assert d["reason"] & 0x7F == 0
        vals.append(d["bytes_o_expert"])
    assert len(set(vals)) == 1
    # 12 B per parameter (fp32 master + two Adam moments) over the expert-DP group times ep ranks = dp
    n_exp_total = int(g["moe_layers"] * g["experts"] * 3 * g["hidden"] * g["expert_ffn"])
    assert vals[0] == 12 * n_exp_total // int(g["dp"]) == 21_592_276_992
    assert round(vals[0] / GB, 2) == g["expert_optimizer_gb"]


def test_admitted_memory_increments_match_paper():
    """Sec. 5 RQ1: ep8 47.0 GB, ep4 57.8 GB, ep2 79.39 GB.  The differences are weight + gradient bytes of
    the experts a rank gains: 6 B/param x expert params x (1/ep' - 1/ep)."""
    g = load_kv("paper_memory_gate.txt")
    cfg = v2lite_like()
    o = Oracle(cfg)
    mem = {}
    for i in range(o.size):
        d = o.eval(i)
        mem[d["ep"]] = d["mem"]
    d48 = (mem[4] - mem[8]) / GB
    d24 = (mem[2] - mem[4]) / GB
    assert round(d48, 1) == round(g["mem_ep4_gb"] - g["mem_ep8_gb"], 1) == 10.8
    assert round(d24, 2) == round(g["mem_ep2_gb"] - g["mem_ep4_gb"], 2) == 21.59
    # and the ep2 - ep4 increment equals the (ep-invariant) expert optimizer state, as in the paper
    assert mem[2] - mem[4] == o.eval(0)["bytes_o_expert"]


def test_gate_direction_and_strictness():
    """Sec. 5 RQ1: 79.39 > 72 is rejected, 57.8 and 47.0 are admitted: reject iff peak > budget."""
    base = Oracle(v2lite_like())
    mem = {base.eval(i)["ep"]: base.eval(i)["mem"] for i in range(base.size)}
    # budget exactly at the ep4 peak: ep4 (== budget) and ep8 pass, ep2 fails with MEMORY
    o = Oracle(v2lite_like(budget=mem[4]))
    got = {o.eval(i)["ep"]: o.eval(i)["reason"] & 0x7F for i in range(o.size)}
    assert got == {2: 11, 4: 0, 8: 0}
    o = Oracle(v2lite_like(budget=mem[4] - 1))
    got = {o.eval(i)["ep"]: o.eval(i)["reason"] & 0x7F for i in range(o.size)}
    assert got == {2: 11, 4: 11, 8: 0}


def test_dense_optimizer_shards_over_dp():
    """Sec. 5 RQ1: total optimizer 22.93 GB = expert 21.59 GB + a dense part sharded over dp.
    Structure check: dense optimizer bytes = 12 * ceil(N_dense / dp)."""
    o = Oracle(v2lite_like())
    d = o.eval(0)
    assert d["bytes_o_dense"] == 12 * -(-d["N_dense"] // d["dp"])
    assert d["bytes_o"] == d["bytes_o_dense"] + d["bytes_o_expert"]
    # weights bf16 (2 B) and gradients fp32 (4 B): the 6 B/param the paper's increments imply
    assert d["bytes_w"] == 2 * (d["N_dense"] + d["N_exp"])
    assert d["bytes_g"] == 4 * (d["N_dense"] + d["N_exp"])


def test_memory_formula_hand_computed():
    """Tiny space, candidate 0 (tp = pp = ep = 1, dp = 2, mb = 1, 1F1B, no recompute), worked by hand:
      attention params 4*1024*1024 = 4,194,304; router 1024*8 = 8,192; expert 3*1024*2816 = 8,650,752
      embeddings 32000*1024 = 32,768,000, held twice (embedding + head) when pp = 1
      N_dense = 8*(4,194,304 + 8,192) + 65,536,000 = 99,155,968;  N_exp = 8*8*8,650,752 = 553,648,128
      weights + grads = 6 * 652,804,096 = 3,916,824,576;  optimizer = 12 * 652,804,096 / 2 = 3,916,824,576
      activation bytes/token/layer = 12,288 + 10,272 + 33,792 = 56,352;  t = 2048;  per layer 115,408,896
      in flight: min(pp, m) * 8 layers = 8 -> 923,271,168;  fp32 logits 4*2048*32000 = 262,144,000
      total 9,019,064,320 B."""
    o = Oracle(make_config("tiny"))
    d = o.eval(0)
    assert (d["tp"], d["pp"], d["ep"], d["dp"], d["mb"], d["kind"], d["rec"]) == (1, 1, 1, 2, 1, 0, 0)
    assert d["N_dense"] == 99_155_968 and d["N_exp"] == 553_648_128
    assert d["bytes_w"] + d["bytes_g"] == 3_916_824_576
    assert d["bytes_o"] == 3_916_824_576
    assert d["bytes_a"] == 923_271_168 + 262_144_000
    assert d["mem"] == 9_019_064_320
    dv = o.derived()
    assert (dv["a_attn"], dv["a_fix"], dv["a_ffn"]) == (12_288, 10_272, 33_792)


def test_memory_non_increasing_in_dp():
    """More data parallelism only shards optimizer state further (nothing else grows) when the
    microbatch count stays at or above the pipeline depth."""
    c = variant("mid", cluster=dict(budget_bytes=10 ** 15, G=64), rules=dict(world_max=64, world_min=1))
    c["axes"][-1] = ("world", [0])
    o = Oracle(c)
    for tp, pp in ((1, 1), (2, 1), (1, 2)):
        prev = None
        for dp in (1, 2, 4, 8):
            d = o.eval(axis_index(c, tp=tp, pp=pp, dp=dp, ep=1, mb=1, sched=0, v=1))
            assert d["reason"] & 0x7F == 0, d
            if prev is not None:
                assert d["mem"] < prev
            prev = d["mem"]


# ----------------------------------------------------------------------------- realization tax

def test_tax_rule_divides_by_one_plus_frac():
    """Sec. 3.2 / Table 'tax': throughput / (1 + frac); a negative frac raises the score; unset (0)
    leaves it bit-identical."""
    g = load_kv("paper_ratios.txt")
    for frac in (g["tax_serve_h800"], g["tax_serve_4090"], g["tax_train_4090"], g["tax_train_h800"], 0.0):
        cfg = make_config("tiny")
        cfg["kern"][1]["patch_ovh"] = float(np.float32(frac))
        o = Oracle(cfg)
        i = axis_index(cfg, kv=1)
        d = o.eval(i)
        assert d["reason"] == 0
        f32frac = float(np.float32(frac))
        assert d["tput"] == d["tput_unpriced"] / (1.0 + f32frac)
        if frac < 0:
            assert d["tput"] > d["tput_unpriced"]
        if frac == 0.0:
            assert d["tput"] == d["tput_unpriced"]
        # the native variant (kv = 0) never pays the patch overhead
        d0 = o.eval(axis_index(cfg, kv=0))
        assert d0["tput"] == d0["tput_unpriced"]


def test_schedule_overhead_applies_only_with_overlap():
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15))
    o = Oracle(cfg)
    i0 = axis_index(cfg, sched=0, tp=1, pp=2, dp=4, ep=4, v=1)   # 1F1B, no overlap
    i1 = axis_index(cfg, sched=1, tp=1, pp=2, dp=4, ep=4, v=2)   # interleaved + overlap
    d0, d1 = o.eval(i0), o.eval(i1)
    assert d0["reason"] & 0x7F == 0 and d1["reason"] & 0x7F == 0
    assert d0["tput"] == d0["tput_unpriced"]
    assert d1["tput"] == d1["tput_unpriced"] / (1.0 + cfg["sched"][1]["sched_ovh"])


def test_paper_ratio_arithmetic():
    """Sec. 5 RQ1 prints +10.84% = 26174.91 / 23614.55 - 1; RQ2 prints the overlap penalty as the mean
    of 0.0294 and 0.0248 (0.0271 at the printed precision).  These fix how scores are compared (a plain
    ratio of tokens/s/GPU)."""
    g = load_kv("paper_ratios.txt")
    assert round((g["constrained_top1"] / g["fallback_top1"] - 1) * 100, 2) == g["gain_percent"]
    assert round((g["overlap_pair_a"] + g["overlap_pair_b"]) / 2, 4) == round(g["overlap_penalty"], 4)


# ----------------------------------------------------------------------------- rules

def test_tiny_space_brute_force_histogram():
    """Nested loops over the tiny space, most-significant axis outermost, with the rule outcomes counted
    from the rule statements directly (not through the oracle's decode):
      world = 2: tp*pp must divide 2 -> (tp, pp) = (2, 2) fails WORLD: 1/4 of 432 = 108
      EP inside DP: ep = 2 needs dp = 2, i.e. only (tp, pp) = (1, 1): 2 of the 6 remaining
        (layout, ep) pairs fail -> 108
      interleaved (auto v = 2) needs pp >= 2: 3 of 4 feasible layouts x 18 = 54 fail VSTAGE
      DualPipe is unmapped: 4 layouts x 18 = 72 fail UNMAPPED_SCHEDULE;  the rest (90) pass."""
    cfg = make_config("tiny")
    o = Oracle(cfg)
    assert o.size == space_size(cfg) == 432
    reason, tput, mem, _ = o.score_range()
    names = [n for n, _ in cfg["axes"]]
    lists = [v for _, v in cfg["axes"]]
    expect = np.zeros(432, dtype=np.uint8)
    feasible_layouts = set()
    # itertools.product varies the LAST factor fastest, so feed the axes most-significant first
    for lin, combo in enumerate(itertools.product(*reversed(lists))):
        c = dict(zip(reversed(names), combo))
        tp, pp, ep, s = c["tp"], c["pp"], c["ep"], c["sched"]
        if 2 % (tp * pp) != 0:
            r = 1
        else:
            dp = 2 // (tp * pp)
            if dp % ep != 0:
                r = 3
            elif s == 1 and pp < 2:
                r = 5
            elif s == 2:
                r = 9
            else:
                r = 0
            if r in (0, 5, 9):
                feasible_layouts.add((tp, pp, ep))
        expect[lin] = r
    assert feasible_layouts == {(1, 1, 1), (1, 1, 2), (2, 1, 1), (1, 2, 1)}
    np.testing.assert_array_equal(reason & 0x7F, expect)
    assert np.bincount(expect, minlength=12).tolist() == [90, 108, 0, 108, 0, 54, 0, 0, 0, 72, 0, 0]
    # infeasible candidates carry no score
    assert np.all(tput[(reason & 0x7F) != 0] == 0.0)
    assert np.all(tput[(reason & 0x7F) == 0] > 0.0)


def test_decode_is_least_significant_axis_first():
    cfg = make_config("mid")
    o = Oracle(cfg)
    rng = np.random.default_rng(1)
    for idx in rng.integers(0, o.size, size=200).tolist():
        d = o.eval(idx)
        rem = idx
        for name, vals in cfg["axes"]:
            digit = rem % len(vals)
            rem //= len(vals)
            if name in ("kv", "rec", "sched", "mb", "v", "ep", "pp", "tp"):
                assert d[name] == vals[digit], (name, idx)


def test_twenty_seven_layers_vs_pipeline_depth():
    """Fig. 2 / Sec. 5 RQ1: an interleaved schedule needs pp*v | 27; 3, 9, 27 pass, even products fail."""
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15, G=32), rules=dict(world_max=4096, world_min=1))
    cfg["model"]["L"] = 27
    cfg["workload"]["gbs"] = 27 * 64
    cfg["axes"] = [("kv", [0]), ("rec", [0]), ("sched", [1]), ("mb", [1]), ("v", [1, 2, 3, 4, 9]), ("ep", [1]),
                   ("pp", [1, 2, 3, 4, 9, 27]), ("tp", [1]), ("dp", [1]), ("world", [0])]
    o = Oracle(cfg)
    for i in range(o.size):
        d = o.eval(i)
        r = d["reason"] & 0x7F
        q = d["pp"] * d["v"]
        if d["v"] < 2 or d["pp"] < 2:
            assert r == 5
        elif 27 % q != 0:
            assert r == 6, d
        else:
            assert r != 6 and q in (9, 27)


def test_serving_dp_attention_needs_dp_equal_ep():
    """Sec. 2.1: on 8 GPUs tp1/ep4 with dp-attention is unrealizable (dp = 8 != ep); tp1/ep8 and a
    plain tp8 are fine."""
    cfg = variant("serve", cluster=dict(budget_bytes=10 ** 15))
    for k in cfg["kern"]:
        k["avail_mask"] = 255
    o = Oracle(cfg)
    r = lambda **kw: o.eval(axis_index(cfg, **kw))["reason"] & 0x7F
    assert r(tp=1, ep=4, dpa=1, batch=512) == 1
    assert r(tp=1, ep=8, dpa=1, batch=512) == 0
    assert r(tp=8, ep=1, dpa=0, batch=512) == 0
    assert r(tp=2, ep=4, dpa=1, batch=512) == 0      # dp = 8/2 = 4 == ep
    assert r(tp=2, ep=4, dpa=0, batch=512) == 1      # EP inside TP needs ep | tp
    assert r(tp=4, ep=2, dpa=0, batch=512) == 0


def test_unmapped_schedule_and_unconstrained_mode():
    """Sec. 2.1 / 3.3: DualPipe has no realization -> rejected by the dry run; the unconstrained mode
    keeps it; switching the constraint on never admits anything new."""
    cfg_on = variant("mid", cluster=dict(budget_bytes=10 ** 15))
    cfg_off = variant("mid", cluster=dict(budget_bytes=10 ** 15), rules=dict(enforce_realizability=0))
    r_on, t_on, _, _ = Oracle(cfg_on).score_range()
    r_off, t_off, _, _ = Oracle(cfg_off).score_range()
    f_on, f_off = (r_on & 0x7F) == 0, (r_off & 0x7F) == 0
    assert np.all(f_off[f_on])                       # constrained-feasible => unconstrained-feasible
    assert np.all(t_on[f_on] == t_off[f_on])         # and scored identically ("bit-for-bit")
    assert set(np.unique(r_on & 0x7F)) >= {9, 10}
    assert not ({9, 10} & set(np.unique(r_off & 0x7F)))
    # every candidate rejected by 9 uses the DualPipe class (schedule 2); rule 10 hits overlap schedules
    sched = (np.arange(len(r_on)) // (4 * 3)) % 3
    assert np.all(sched[(r_on & 0x7F) == 9] == 2)
    assert np.all(sched[(r_on & 0x7F) == 10] == 1)


def test_overlap_preconditions():
    """Sec. 4 'Emitters': full recompute + EP overlap raises; pp > 1 under 1f1b with overlap raises."""
    cfg = variant("large", cluster=dict(budget_bytes=10 ** 15))
    for k in cfg["kern"]:
        k["avail_mask"] = 255
    o = Oracle(cfg)
    base = dict(tp=1, ep=8, dp=16, mb=1, v=1, kv=0)
    r = lambda **kw: o.eval(axis_index(cfg, **{**base, **kw}))["reason"] & 0x7F
    assert r(sched=1, pp=1, rec=0) == 0        # 1f1b + overlap at pp = 1
    assert r(sched=1, pp=1, rec=2) == 10       # full recompute + overlap
    assert r(sched=1, pp=2, dp=8, rec=0) == 10  # pp > 1 under 1f1b + overlap
    assert r(sched=0, pp=2, dp=8, rec=2) == 0  # no overlap: no precondition
    assert r(sched=2, pp=2, dp=8, v=2, rec=0) == 0   # interleaved + overlap is allowed at pp > 1
    assert r(sched=3, pp=2, dp=8, rec=0) == 9  # dualpipe: unmapped comes first


def test_large_space_rule_counts_match_independent_probe():
    """Rules 1-7 on the large space against counts made by a separate brute-force probe."""
    g = load_kv("large_space_rule_counts.txt")
    cfg = variant("large", cluster=dict(budget_bytes=10 ** 15))
    for k in cfg["kern"]:
        k["avail_mask"] = 255
    # one recompute mode and one kernel variant: the structural rules do not look at them
    cfg["axes"][0] = ("kv", [0])
    cfg["axes"][1] = ("rec", [0])
    cfg["rules"]["enforce_realizability"] = 0
    o = Oracle(cfg)
    assert o.size == 7_496_192
    reason, _, _, _ = o.score_range(threads=8, want_mem=False, want_tput=False)
    h = np.bincount(reason & 0x7F, minlength=12)
    assert h[1] == g["WORLD"] and h[2] == g["TP"] and h[3] == g["EP"] and h[4] == g["BATCH"]
    assert h[5] == g["VSTAGE"] and h[6] == g["LAYERS"] and h[7] == g["MICROBATCH"]
    assert h[0] + h[8] + h[11] == g["PASS"]


def test_kernel_missing_and_extrapolated_flag():
    """Sec. 3.3 kernel tier + calibration domain [64, 8192] tokens per expert."""
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15))
    for k in cfg["kern"]:
        k["avail_mask"] = 255
    cfg["kern"][2]["avail_mask"] = 255 & ~(1 << 3)          # no entry for 512 <= m_e < 1024
    cfg["kern"][3]["needs_caps"] = 1                        # needs fp8, cluster has none
    o = Oracle(cfg)
    # m_e = t*K*ep/(E*tp) with t = mb*4096, K = 6, E = 64
    i = axis_index(cfg, kv=2, mb=2, ep=1, tp=1, pp=1, dp=8, sched=0, v=1)   # m_e = 768 -> bucket 3
    d = o.eval(i)
    assert d["m_e"] == 768 and d["bucket"] == 3 and d["reason"] == 8
    i = axis_index(cfg, kv=2, mb=4, ep=1, tp=1, pp=1, dp=8, sched=0, v=1)   # m_e = 1536 -> bucket 4
    assert o.eval(i)["reason"] & 0x7F == 0
    i = axis_index(cfg, kv=3, mb=4, ep=1, tp=1, pp=1, dp=8, sched=0, v=1)
    assert o.eval(i)["reason"] == 8
    # bucket edges
    for mb, ep, tp, me, b in ((1, 1, 8, 48, 0), (1, 1, 4, 96, 0), (1, 1, 2, 192, 1), (8, 8, 1, 24576, 7)):
        d = o.eval(axis_index(cfg, kv=0, mb=mb, ep=ep, tp=tp, pp=1, dp=8 // tp, sched=0, v=1))
        assert d["m_e"] == me and d["bucket"] == b, d
        flagged = bool(d["reason"] & 0x80)
        assert flagged == (me < 64 or me > 8192)


# ----------------------------------------------------------------------------- analytic time

def test_single_gpu_reduces_to_flops_over_peak():
    """tp = pp = ep = dp = 1 with uniform efficiency: no communication, no bubble, so the step is
    3 x forward FLOPs / (peak x efficiency) plus the optimizer sweep -- the textbook 6ND/peak rule."""
    cfg = variant("tiny", cluster=dict(budget_bytes=10 ** 15, G=1), rules=dict(world_min=1, world_max=1))
    cfg["axes"] = [("kv", [0]), ("rec", [0]), ("sched", [0]), ("mb", [1, 4]), ("v", [0]), ("ep", [1]),
                   ("pp", [1]), ("tp", [1]), ("dp", [0]), ("world", [1])]
    for b in range(8):
        cfg["kern"][0]["eff"][b] = cfg["consts"]["eff_dense"]
    o = Oracle(cfg)
    M, C = cfg["model"], cfg["cluster"]
    dv = o.derived()
    for i in range(o.size):
        d = o.eval(i)
        fwd_per_token = M["L"] * (dv["f_dense"] + dv["f_exp"]) + dv["f_head"]
        tokens = cfg["workload"]["gbs"] * M["seq"]
        t_compute = 3 * fwd_per_token * tokens / (C["peak_flops"] * cfg["consts"]["eff_dense"])
        t_opt = 2 * d["bytes_o"] / C["hbm_bw"]
        assert d["tput"] == pytest.approx(tokens / (t_compute + t_opt), rel=1e-12)
        assert d["tpc"] == 0 and d["a2a"] == 0 and d["p"] == 0 and d["T_dp"] == 0


def test_forward_flops_hand_computed():
    """Tiny model: attention 2*4,194,304 + 2*2048*16*64 = 12,582,912; router 2*1024*8 = 16,384;
    experts 2*2*8,650,752 = 34,603,008; head 2*32000*1024 = 65,536,000."""
    dv = Oracle(make_config("tiny")).derived()
    assert dv["f_attn"] == 12_582_912 and dv["f_rt"] == 16_384 and dv["f_exp"] == 34_603_008
    assert dv["f_head"] == 65_536_000 and dv["f_dense"] == 12_582_912 + 16_384


def test_1f1b_analytic_bubble_closed_form():
    """spec: 1F1B bubble fraction (pp - 1)/(m + pp - 1) when stage-to-stage latency is zero."""
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15, alpha_intra=0.0, alpha_inter=0.0,
                                      bw_intra=float(np.float32(1e30)), bw_inter=float(np.float32(1e30))))
    o = Oracle(cfg)
    for pp, dp in ((2, 4), (4, 2), (8, 1)):
        d = o.eval(axis_index(cfg, sched=0, tp=1, pp=pp, dp=dp, ep=1, mb=2, v=1))
        assert d["reason"] & 0x7F == 0
        m = d["m"]
        ideal = m * (d["F"] + d["B"])
        bubble = (d["T_pipe"] - ideal) / d["T_pipe"]
        assert bubble == pytest.approx((pp - 1) / (m + pp - 1), rel=1e-9)


def _sweep(cfg_a, cfg_b):
    ra, ta, _, _ = Oracle(cfg_a).score_range(threads=4)
    rb, tb, _, _ = Oracle(cfg_b).score_range(threads=4)
    np.testing.assert_array_equal(ra, rb)
    f = (ra & 0x7F) == 0
    assert f.sum() > 50
    return ta[f], tb[f]


@pytest.mark.parametrize("field,factor", [("bw_intra", 2.0), ("bw_inter", 2.0), ("alpha_intra", 0.5),
                                           ("alpha_inter", 0.5)])
def test_throughput_monotone_in_links(field, factor):
    """spec invariant: throughput never falls when a link gets faster (or its latency shorter)."""
    big = 10 ** 15
    a = variant("mid", cluster=dict(budget_bytes=big, G=4))
    b = variant("mid", cluster=dict(budget_bytes=big, G=4))
    b["cluster"][field] = float(np.float32(a["cluster"][field] * factor))
    ta, tb = _sweep(a, b)
    assert np.all(tb >= ta)
    assert np.any(tb > ta)


def test_hiding_reduces_exposed_all_to_all_but_never_below_zero():
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15))
    o = Oracle(cfg)
    n = 0
    for i in range(0, o.size, 7):
        d = o.eval(i)
        if d["reason"] & 0x7F:
            continue
        n += 1
        assert 0.0 <= d["xF"] <= d["a2a"] and 0.0 <= d["xB"] <= d["a2a"]
        if not d["ov"]:
            assert d["xF"] == d["a2a"]
    assert n > 100


# ----------------------------------------------------------------------------- top-k

def test_topk_invariants():
    """Sec. 3.3: every returned plan passes the predicate; ranking by score, ties by index."""
    for name in ("tiny", "mid", "serve"):
        cfg = make_config(name)
        o = Oracle(cfg)
        reason, tput, _, _ = o.score_range(threads=4)
        idx, sc = o.topk(reason, tput, 0, cfg["k"])
        nfeas = int(((reason & 0x7F) == 0).sum())
        assert len(idx) == min(cfg["k"], nfeas)
        assert np.all((reason[idx.astype(np.int64)] & 0x7F) == 0)
        assert np.all(np.diff(sc) <= 0)
        ties = np.diff(sc) == 0
        assert np.all(np.diff(idx.astype(np.int64))[ties] > 0)
        # against numpy's own ordering
        feas = np.flatnonzero((reason & 0x7F) == 0)
        order = feas[np.lexsort((feas, -tput[feas]))][:cfg["k"]]
        np.testing.assert_array_equal(idx.astype(np.int64), order)


def test_survivors_are_best_feasible_sorted_by_index():
    cfg = make_config("mid")
    o = Oracle(cfg)
    reason, tput, _, _ = o.score_range(threads=4)
    s = o.select_survivors(reason, tput, 0, 50)
    assert len(s) == 50 and np.all(np.diff(s.astype(np.int64)) > 0)
    top, _ = o.topk(reason, tput, 0, 50)
    assert set(s.tolist()) == set(top.tolist())
    allf = o.select_survivors(reason, tput, 0, 10 ** 6)
    assert len(allf) == int(((reason & 0x7F) == 0).sum())


# ----------------------------------------------------------------------------- serving: one score per plan

def test_serving_plan_aggregate_is_tokens_over_time():
    """Sec. 5 RQ3 ranks serving plans, not (plan, request-shape) pairs.  The aggregate must equal total output
    tokens over total time, rebuilt here from the per-scenario prefill / decode times, and must reduce to the
    per-scenario score when the mix has one scenario or all scenarios score alike."""
    cfg = variant("serve", cluster=dict(budget_bytes=10 ** 15))
    for k in cfg["kern"]:
        k["avail_mask"] = 255
    # a small length mix keeps the per-candidate loop short
    cfg["workload"]["scen_P"] = cfg["workload"]["scen_P"][:5]
    cfg["workload"]["scen_O"] = cfg["workload"]["scen_O"][:5]
    cfg["axes"][6] = ("scen", [0, 1, 2, 3, 4])
    o = Oracle(cfg)
    reason, tput, _, _ = o.score_range(threads=4)
    pr, pt = o.aggregate_serving(reason, tput)
    n_plans = o.size // 5
    assert len(pr) == n_plans
    checked = 0
    for p in range(0, n_plans, 37):
        ds = [o.eval(p + n_plans * i) for i in range(5)]
        if any(d["reason"] & 0x7F for d in ds):
            first = next(d["reason"] & 0x7F for d in ds if d["reason"] & 0x7F)
            assert pr[p] == first and pt[p] == 0.0
            continue
        checked += 1
        d0 = ds[0]
        n_eng = d0["tp"] * d0["ep"] if d0["dpa"] else d0["tp"]
        b_loc = d0["batch"] // d0["ep"] if d0["dpa"] else d0["batch"]
        O = cfg["workload"]["scen_O"]
        tokens = sum(d0["batch"] * O[i] for i in range(5))
        time = sum(b_loc * ds[i]["T_pre"] + O[i] * ds[i]["T_dec"] for i in range(5))
        want = tokens / time / n_eng
        if not cfg["kern"][d0["kv"]]["is_native"]:
            want /= 1 + cfg["kern"][d0["kv"]]["patch_ovh"]
        assert pt[p] == pytest.approx(want, rel=1e-12)
        per = [d["tput"] for d in ds]
        assert min(per) * (1 - 1e-12) <= pt[p] <= max(per) * (1 + 1e-12)
        assert pr[p] == (0x80 if any(d["reason"] & 0x80 for d in ds) else 0)
    assert checked > 20
    # one scenario: the aggregate is the scenario's own score
    one = variant("serve", cluster=dict(budget_bytes=10 ** 15))
    one["axes"][6] = ("scen", [3])
    oo = Oracle(one)
    r1, t1, _, _ = oo.score_range(threads=4)
    pr1, pt1 = oo.aggregate_serving(r1, t1)
    f = (r1 & 0x7F) == 0
    np.testing.assert_allclose(pt1[f], t1[f], rtol=1e-15)
    np.testing.assert_array_equal(pr1, r1)
    # the same scenario listed three times: still the scenario's own score
    rep = variant("serve", cluster=dict(budget_bytes=10 ** 15))
    rep["axes"][6] = ("scen", [3, 3, 3])
    orp = Oracle(rep)
    r3, t3, _, _ = orp.score_range(threads=4)
    pr3, pt3 = orp.aggregate_serving(r3, t3)
    np.testing.assert_allclose(pt3[f], t1[f], rtol=1e-14)


def test_serving_plan_is_infeasible_if_any_scenario_is():
    """The KV cache grows with prompt + output length, so the memory gate can reject a plan for the long requests
    only; such a plan cannot serve the mix."""
    cfg = make_config("serve")
    o = Oracle(cfg)
    reason, tput, _, _ = o.score_range(threads=8)
    pr, pt = o.aggregate_serving(reason, tput)
    n_plans = o.size // 128
    per = (reason.reshape(128, n_plans) & 0x7F)
    any_bad = (per != 0).any(axis=0)
    all_bad = (per != 0).all(axis=0)
    assert (any_bad & ~all_bad).sum() > 0                      # mixed plans exist in this space
    np.testing.assert_array_equal((pr & 0x7F) != 0, any_bad)
    assert np.all(pt[any_bad] == 0) and np.all(pt[~any_bad] > 0)


# --------------------------------------------------------------------------- operation tally (counting build)

def test_operation_tally_charges_by_how_far_a_candidate_gets():
    """Hand counts: a candidate rejected by the first rule pays the decode (one mod and one div per axis) and
    that rule's ten integer operators (fifteen when dp is derived from the world size), nothing else; a feasible candidate pays for every block, floating part
    included; the tally build computes the same reasons as the plain build."""
    cfg = make_config("tiny")
    orc = Oracle(cfg)
    reason, _, _, _ = orc.score_range(0, orc.size)
    n_axes = len(cfg["axes"])
    rule1 = 15 if list(dict(cfg["axes"])["dp"]) == [0] else 10
    first_rule = [i for i in range(orc.size) if reason[i] == 1]
    feasible = [i for i in range(orc.size) if (reason[i] & 0x7F) == 0]
    assert first_rule and feasible
    c = oracle.count_ops(orc, first_rule[0], 1)
    assert c == {"int_ops": 2 * n_axes + rule1, "fp_ops": 0, "candidates": 1}
    c = oracle.count_ops(orc, feasible[0], 1)
    assert c["fp_ops"] == 110 and c["int_ops"] > 150 and c["candidates"] == 1
    # totals add up candidate by candidate and do not depend on the thread count
    whole = oracle.count_ops(orc, 0, orc.size, threads=1)
    assert whole == oracle.count_ops(orc, 0, orc.size, threads=4)
    assert whole["candidates"] == orc.size
    assert whole["fp_ops"] == 110 * len(feasible)
    parts = [oracle.count_ops(orc, i, 1)["int_ops"] for i in range(0, orc.size, 7)]
    assert min(parts) >= 2 * n_axes + rule1
