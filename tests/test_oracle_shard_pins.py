"""Pins of the oracle's sharding dimension {zero1, zero1_offload, fsdp} (Sec. 3.1, memory plan; Sec. 3.2,
contention penalty; Sec. 5 RQ2, hiding conditioned out in the offload domain).

None of these retype the oracle's formulas: they use what the paper fixes (zero1 = prior behaviour to the bit,
the printed optimizer-state sizes, the 0.0271 penalty and the divide-by-(1+frac) rule), special cases with an
obvious value (a one-rank group shards nothing), and invariants."""
from __future__ import annotations

import copy

import numpy as np
import pytest

from oracle import Oracle
from workloads import make_config

from helpers import axis_index, v2lite_like, variant

ZERO1, OFFLOAD, FSDP = 0, 1, 2


def with_shard(cfg, values=(ZERO1, OFFLOAD, FSDP)):
    cfg = copy.deepcopy(cfg)
    cfg["axes"] = list(cfg["axes"]) + [("shard", list(values))]
    return cfg


@pytest.mark.parametrize("name", ["tiny", "mid"])
def test_zero1_reproduces_the_space_without_the_axis_bit_for_bit(name):
    """Sharding defaults to zero1, which reproduces prior behaviour bit for bit; the axis is the most
    significant digit, so block s of the widened space is the old space under sharding s."""
    base = make_config(name)
    ob = Oracle(base)
    r0, t0, m0, _ = ob.score_range()
    o3 = Oracle(with_shard(base))
    assert o3.size == 3 * ob.size
    r, t, m, _ = o3.score_range()
    n = ob.size
    assert np.array_equal(r[:n], r0) and np.array_equal(m[:n], m0) and np.array_equal(t[:n], t0)
    # structural rules do not look at the sharding
    for s in (1, 2):
        same = (r0 != 0) & (r0 != 11) & (r0 != 0x80)
        assert np.array_equal(r[s * n:(s + 1) * n][same], r0[same])


def test_offload_frees_exactly_the_optimizer_state_the_paper_prints():
    """Reference-like model at dp = 8: the expert optimizer state is 21.59 GB whatever ep is (Sec. 5 RQ1);
    keeping the optimizer state in host memory lowers the peak by exactly the state's size and by nothing else."""
    cfg = with_shard(v2lite_like())
    orc = Oracle(cfg)
    for ep in (2, 4, 8):
        z = orc.eval(axis_index(cfg, ep=ep, shard=ZERO1))
        o = orc.eval(axis_index(cfg, ep=ep, shard=OFFLOAD))
        assert z["bytes_o_expert"] == 21_592_276_992
        assert o["bytes_o"] == 0 and o["bytes_buf"] == 0
        assert z["mem"] - o["mem"] == z["bytes_o"]
        assert z["bytes_o"] == z["bytes_o_expert"] + z["bytes_o_dense"] > 21_592_276_992
        assert o["bytes_w"] == z["bytes_w"] and o["bytes_g"] == z["bytes_g"] and o["bytes_a"] == z["bytes_a"]


def test_fsdp_on_one_rank_shards_nothing_and_adds_only_the_gather_buffer():
    """dp = 1 and expert-DP = 1: sharding over one rank leaves parameters and gradients whole, so the only
    difference to zero1 is the working buffer -- two layers of bf16 parameters: per layer
    4*H*H (attention, nh*hd = H) + H*E (router) + E * 3*H*F (all experts local at ep = 1)."""
    cfg = with_shard(v2lite_like(ep_values=(1,)))
    cfg["cluster"]["G"] = 1
    cfg["workload"].update(gbs=8, world=1)
    cfg["rules"].update(world_min=1, world_max=1)
    cfg["axes"][9] = ("world", [1])
    orc = Oracle(cfg)
    z = orc.eval(axis_index(cfg, ep=1, shard=ZERO1))
    f = orc.eval(axis_index(cfg, ep=1, shard=FSDP))
    assert z["dp"] == 1 and z["edp"] == 1 and (z["reason"] & 0x7F) == 0
    assert f["bytes_w"] == z["bytes_w"] and f["bytes_g"] == z["bytes_g"] and f["bytes_o"] == z["bytes_o"]
    H, E, F = 2048, 64, 1408
    per_layer = 4 * H * H + H * E + E * 3 * H * F
    assert f["bytes_buf"] == 2 * 2 * per_layer
    assert f["mem"] - z["mem"] == f["bytes_buf"]


def test_fsdp_divides_parameters_and_gradients_by_the_group_sizes():
    """dp = 8, ep = 8 (expert-DP = 1): dense parameters and gradients drop to an eighth (they divide evenly
    here), expert ones stay whole; weights keep the 2 : 4 byte ratio to gradients."""
    cfg = with_shard(v2lite_like())
    orc = Oracle(cfg)
    z = orc.eval(axis_index(cfg, ep=8, shard=ZERO1))
    f = orc.eval(axis_index(cfg, ep=8, shard=FSDP))
    assert z["N_dense"] % 8 == 0 and z["edp"] == 1
    assert f["bytes_w"] == 2 * (z["N_dense"] // 8 + z["N_exp"])
    assert f["bytes_g"] == 2 * f["bytes_w"]
    assert f["bytes_o"] == z["bytes_o"]
    # ep = 2: expert-DP = 4, experts shard four ways as well
    z2 = orc.eval(axis_index(cfg, ep=2, shard=ZERO1))
    f2 = orc.eval(axis_index(cfg, ep=2, shard=FSDP))
    assert z2["edp"] == 4 and z2["N_exp"] % 4 == 0
    assert f2["bytes_w"] == 2 * (z2["N_dense"] // 8 + z2["N_exp"] // 4)


def _overlap_cfg(penalty, hide=None):
    """mid space with an admitting budget; schedule 1 (interleaved) has overlap on."""
    cfg = with_shard(variant("mid", cluster=dict(budget_bytes=10 ** 15)))
    cfg["consts"]["offload_overlap_penalty"] = float(np.float32(penalty))
    if hide is not None:
        for s in cfg["sched"]:
            if s["overlap"]:
                s["hide_frac"] = float(np.float32(hide))
    return cfg


def test_contention_penalty_prices_exactly_the_offloaded_and_overlapped_plans():
    """throughput / (1 + frac) with the paper's measured 0.0271, on offload-and-overlap plans only; an unset
    (zero) penalty leaves every score identical to the bit."""
    assert abs(make_config("mid")["consts"]["offload_overlap_penalty"] - 0.0271) < 1e-7
    c0, c1 = _overlap_cfg(0.0), _overlap_cfg(0.0271)
    o0, o1 = Oracle(c0), Oracle(c1)
    r0, t0, _, _ = o0.score_range()
    r1, t1, _, _ = o1.score_range()
    assert np.array_equal(r0, r1)
    n = o0.size // 3
    sched_digit = (np.arange(o0.size) // (4 * 3)) % 3
    ov = np.array([c0["sched"][s]["overlap"] for s in range(3)])[sched_digit] == 1
    shard = np.arange(o0.size) // n
    feas = (r0 & 0x7F) == 0
    taxed = feas & ov & (shard == OFFLOAD)
    assert taxed.sum() > 50 and (feas & ~taxed).sum() > 50
    assert np.array_equal(t0[~taxed], t1[~taxed])
    frac = float(np.float32(0.0271))
    np.testing.assert_allclose(t1[taxed], t0[taxed] / (1.0 + frac), rtol=1e-14)


def test_hiding_is_conditioned_out_in_the_offload_domain():
    """With the optimizer offloaded the hidden fraction of the all-to-all does not enter the score; under
    zero1 and fsdp it does."""
    ca, cb = _overlap_cfg(0.0271, hide=0.2), _overlap_cfg(0.0271, hide=0.8)
    oa, ob = Oracle(ca), Oracle(cb)
    ra, ta, _, _ = oa.score_range()
    rb, tb, _, _ = ob.score_range()
    assert np.array_equal(ra, rb)
    n = oa.size // 3
    feas = (ra & 0x7F) == 0
    off = slice(n, 2 * n)
    assert np.array_equal(ta[off], tb[off])
    for blk in (slice(0, n), slice(2 * n, 3 * n)):
        f = feas[blk]
        assert np.all(tb[blk][f] >= ta[blk][f]) and np.any(tb[blk][f] > ta[blk][f])


def test_offloaded_step_speeds_up_with_the_host_link_and_zero1_ignores_it():
    slow = with_shard(variant("mid", cluster=dict(budget_bytes=10 ** 15, bw_host=float(np.float32(10e9)))))
    fast = with_shard(variant("mid", cluster=dict(budget_bytes=10 ** 15, bw_host=float(np.float32(100e9)))))
    os_, of = Oracle(slow), Oracle(fast)
    rs, ts, _, _ = os_.score_range()
    rf, tf, _, _ = of.score_range()
    n = os_.size // 3
    feas = (rs & 0x7F) == 0
    assert np.array_equal(ts[:n], tf[:n]) and np.array_equal(ts[2 * n:], tf[2 * n:])
    f = feas[n:2 * n]
    assert f.sum() > 50 and np.all(tf[n:2 * n][f] > ts[n:2 * n][f])
    # the offloaded optimizer step: (gradient + weight bytes of the rank's shard) / link rate, so the step
    # time difference between the two links is that many bytes times (1/10e9 - 1/100e9)
    i = int(np.flatnonzero(f)[0]) + n
    a, b = os_.eval(i), of.eval(i)
    shard_params = (a["N_dense"] + a["dp"] - 1) // a["dp"] + (a["N_exp"] + a["edp"] - 1) // a["edp"]
    want = 6 * shard_params * (1 / float(np.float32(10e9)) - 1 / float(np.float32(100e9)))
    assert abs((a["T_step"] - b["T_step"]) - want) <= 1e-9 * want


def test_fsdp_replaces_the_gradient_all_reduce_by_per_microbatch_gathers():
    """On one rank there is nothing to gather: fsdp and zero1 then take the same time; with dp > 1 the
    per-microbatch traffic grows with the number of microbatches, so halving the microbatch size (twice the
    microbatches) doubles the fsdp data-parallel term."""
    cfg = with_shard(variant("mid", cluster=dict(budget_bytes=10 ** 15)))
    orc = Oracle(cfg)
    z = orc.eval(axis_index(cfg, tp=8, pp=1, dp=1, ep=8, mb=2, v=1, sched=0, shard=ZERO1))
    f = orc.eval(axis_index(cfg, tp=8, pp=1, dp=1, ep=8, mb=2, v=1, sched=0, shard=FSDP))
    assert (z["reason"] & 0x7F) == 0 and (f["reason"] & 0x7F) == 0 and z["edp"] == 1
    assert f["T_dp"] == 0.0 and z["T_dp"] == 0.0 and f["T_step"] == z["T_step"]
    a = orc.eval(axis_index(cfg, tp=1, pp=1, dp=8, ep=1, mb=2, v=1, sched=0, shard=FSDP))
    b = orc.eval(axis_index(cfg, tp=1, pp=1, dp=8, ep=1, mb=1, v=1, sched=0, shard=FSDP))
    assert (a["reason"] & 0x7F) == 0 and b["m"] == 2 * a["m"]
    assert abs(b["T_dp"] / a["T_dp"] - 2.0) < 1e-12
    zz = orc.eval(axis_index(cfg, tp=1, pp=1, dp=8, ep=1, mb=2, v=1, sched=0, shard=ZERO1))
    assert a["T_dp"] > zz["T_dp"] > 0.0
