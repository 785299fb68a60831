"""Pins for the oracle's pipeline-schedule simulator: closed forms, a hand-worked timeline, golden
makespans from an independent implementation, order validity and jitter properties.  No GPU."""
from __future__ import annotations

import numpy as np
import pytest

import oracle
from oracle import Oracle
from workloads import make_config

from helpers import axis_index, load_rows, variant

K1F1B, KINT, KDUAL = 0, 1, 2


def test_1f1b_closed_form_every_shape():
    """Uniform stages, zero latency: makespan (m + pp - 1)(F + B), i.e. bubble (pp-1)/(m+pp-1)."""
    for pp in range(1, 33):
        for m in range(1, 70):
            for F, B in ((1.0, 2.0), (1.0, 1.0), (2.0, 3.0)):
                got = oracle.makespan(K1F1B, pp, 1, m, [F] * pp, [B] * pp, 0.0)
                assert got == (m + pp - 1) * (F + B), (pp, m, F, B)


def test_interleaved_closed_form():
    """Uniform chunk times f, b, zero latency, m a multiple of pp: (m*v + pp - 1)(f + b)."""
    for pp in range(1, 17):
        for v in (1, 2, 3, 4, 8):
            for m in range(pp, 65, pp):
                got = oracle.makespan(KINT, pp, v, m, [1.0] * (pp * v), [2.0] * (pp * v), 0.0)
                assert got == (m * v + pp - 1) * 3.0, (pp, v, m)


def test_interleaved_needs_m_multiple_of_pp():
    with pytest.raises(ValueError):
        oracle.schedule_order(KINT, 4, 2, 6)


def test_dualpipe_style_golden_makespans():
    for F, B, pp, m, want in load_rows("dualpipe_style_makespans.txt"):
        got = oracle.makespan(KDUAL, pp, 1, m, [float(F)] * pp, [float(B)] * pp, 0.0)
        assert got == float(want), (F, B, pp, m)


def test_dualpipe_style_trivial_depths():
    """pp = 1 and pp = 2: each rank is busy the whole time, makespan = m (F + B)."""
    for m in (2, 4, 10, 64):
        assert oracle.makespan(KDUAL, 1, 1, m, [1.0], [2.0], 0.0) == 3.0 * m
        assert oracle.makespan(KDUAL, 2, 1, m, [1.0] * 2, [2.0] * 2, 0.0) == 3.0 * m


def test_hand_worked_timeline_with_latency():
    """1F1B, pp = 2, m = 2, F = [1, 2], B = [3, 4], latency 0.5.
    rank 0 runs F(0,0) F(0,1) B(0,0) B(0,1); rank 1 runs F(1,0) B(1,0) F(1,1) B(1,1).
    F(0,0) 0-1, F(0,1) 1-2, F(1,0) 1.5-3.5, B(1,0) 3.5-7.5, F(1,1) 7.5-9.5, B(1,1) 9.5-13.5,
    B(0,0) starts at 7.5 + 0.5 = 8 -> 11, B(0,1) starts at 13.5 + 0.5 = 14 -> 17."""
    order = oracle.schedule_order(K1F1B, 2, 1, 2)
    assert order[0] == [(0, 0, 0, 0), (0, 1, 0, 0), (0, 0, 0, 1), (0, 1, 0, 1)]
    assert order[1] == [(1, 0, 0, 0), (1, 0, 0, 1), (1, 1, 0, 0), (1, 1, 0, 1)]
    assert oracle.makespan(K1F1B, 2, 1, 2, [1.0, 2.0], [3.0, 4.0], 0.5) == 17.0


def _check_order_complete(order, Q, nj, ndir):
    seen = set()
    for ops in order:
        for op in ops:
            assert op not in seen
            seen.add(op)
    want = {(q, j, d, b) for q in range(Q) for j in range(nj) for d in range(ndir) for b in (0, 1)}
    assert seen == want


def test_orders_run_every_op_exactly_once_and_inflight_bounds():
    for pp in (1, 2, 3, 4, 8):
        for m in (1, 2, 5, 8, 16):
            order = oracle.schedule_order(K1F1B, pp, 1, m)
            _check_order_complete(order, pp, m, 1)
            for s, ops in enumerate(order):
                # ops of rank s belong to stage s; peak forwards-minus-backwards in flight = min(pp - s, m)
                assert all(q == s for q, _, _, _ in ops)
                live = peak = 0
                for _, _, _, b in ops:
                    live += -1 if b else 1
                    peak = max(peak, live)
                assert peak == min(pp - s, m)
    for pp, v, m in ((2, 2, 4), (4, 2, 8), (4, 3, 4), (8, 2, 16)):
        order = oracle.schedule_order(KINT, pp, v, m)
        _check_order_complete(order, pp * v, m, 1)
        for s, ops in enumerate(order):
            assert all(q % pp == s for q, _, _, _ in ops)
    for pp, m in ((1, 4), (2, 8), (4, 8), (8, 16), (16, 8)):
        order = oracle.schedule_order(KDUAL, pp, 1, m)
        _check_order_complete(order, pp, m // 2, 2)
        for r, ops in enumerate(order):
            assert all((q if d == 0 else pp - 1 - q) == r for q, _, d, _ in ops)
            live = peak = 0
            for _, _, _, b in ops:
                live += -1 if b else 1
                peak = max(peak, live)
            assert peak <= pp + 1


def test_interleaved_inflight_matches_memory_model():
    """The interleaved order's peak number of forward chunks in flight on rank 0, pp*v + pp - 1 (capped by
    m*v), is the unit count the memory model charges for that schedule class: the two statements were
    written separately and must agree.  Rank s warms up with 2(pp-s-1) + (v-1)pp forward chunks."""
    for pp, v, m in ((2, 2, 2), (2, 2, 8), (4, 2, 8), (4, 3, 16), (8, 4, 8), (8, 2, 64)):
        order = oracle.schedule_order(KINT, pp, v, m)
        for s, ops in enumerate(order):
            live = peak = 0
            for _, _, _, b in ops:
                live += -1 if b else 1
                peak = max(peak, live)
            assert peak == min(2 * (pp - s - 1) + (v - 1) * pp + 1, m * v), (pp, v, m, s)
        cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15, G=64), rules=dict(world_max=64, world_min=1, enforce_realizability=0))
        cfg["model"]["L"] = 96
        cfg["workload"]["gbs"] = m
        cfg["axes"] = [("kv", [0]), ("rec", [0, 2]), ("sched", [1]), ("mb", [1]), ("v", [v]), ("ep", [1]),
                       ("pp", [pp]), ("tp", [1]), ("dp", [1]), ("world", [0])]
        o = Oracle(cfg)
        d0, d2 = o.eval(0), o.eval(1)
        assert d0["reason"] & 0x7F == 0 and d0["m"] == m
        dv = o.derived()
        t = cfg["model"]["seq"]
        units = min(pp * v + pp - 1, m * v) * d0["Lc"]
        # pp >= 2 and not DualPipe: rank 0 holds no logits, so the activation term is units x layer bytes
        assert d0["bytes_a"] == units * t * dv["a_full"]
        assert d2["bytes_a"] == units * t * dv["a_ckpt"] + t * dv["a_full"]


def test_latency_only_delays():
    rng = np.random.default_rng(3)
    for kind, pp, v, m in ((K1F1B, 4, 1, 8), (KINT, 4, 2, 8), (KDUAL, 4, 1, 8), (K1F1B, 1, 1, 5), (KINT, 1, 3, 4),
                           (KDUAL, 1, 1, 6)):
        Q = pp * v
        F = rng.uniform(0.5, 1.5, Q)
        B = rng.uniform(1.0, 3.0, Q)
        prev = oracle.makespan(kind, pp, v, m, F, B, 0.0)
        # lower bounds: the busiest rank's total work, and one microbatch's full traversal
        ranks = [[q for q in range(Q) if (q % pp == r if kind != KDUAL else q in (r, pp - 1 - r))] for r in range(pp)]
        per_rank = max(sum(F[q] + B[q] for q in qs) * (m if kind != KDUAL else m / 2) for qs in ranks)
        assert prev >= per_rank - 1e-12
        assert prev >= F.sum() + B.sum() - 1e-12
        for p in (0.1, 0.5, 2.0):
            cur = oracle.makespan(kind, pp, v, m, F, B, p)
            assert cur >= prev
            if pp == 1:
                assert cur == prev
            prev = cur


def test_mix32_and_jitter():
    # the avalanche hash in wrapping 32-bit arithmetic, restated in Python integers
    def mix(x):
        x &= 0xFFFFFFFF
        x ^= x >> 16
        x = (x * 0x7FEB352D) & 0xFFFFFFFF
        x ^= x >> 15
        x = (x * 0x846CA68B) & 0xFFFFFFFF
        x ^= x >> 16
        return x
    for x in (0, 1, 2, 0x9E3779B9, 0xFFFFFFFF, 123456789):
        assert oracle.mix32(x) == mix(x)
    assert oracle.mix32(0) == 0
    seen = {oracle.mix32(i) for i in range(4096)}
    assert len(seen) == 4096
    js = np.array([oracle.jitter(4, idx, q, b) for idx in (0, 7, 2 ** 33 + 5) for q in range(40) for b in (0, 1)])
    assert js.min() >= 0.9 and js.max() < 1.1
    assert abs(js.mean() - 1.0) < 0.02
    assert len(np.unique(js)) > 200
    # the uniform draw has 24 bits, so it is exact in fp32
    u = (js - 0.9) / 0.2
    assert np.allclose(u * 2 ** 24, np.round(u * 2 ** 24), atol=1e-6)
    h = mix(mix(mix(mix(4 + 0x9E3779B9) ^ 5) ^ 2) ^ (2 * 3 + 1))
    assert oracle.jitter(4, 2 ** 33 + 5, 3, 1) == 0.9 + 0.2 * ((h >> 8) / 2 ** 24)


def _stage_times(o: Oracle, cfg, idx, seed):
    d = o.eval(idx)
    L = cfg["model"]["L"]
    kind, pp, v = d["kind"], d["pp"], d["v_eff"]
    Q = pp if kind == KDUAL else pp * v
    F, B = [], []
    for q in range(Q):
        nq = L // Q + (1 if q < L % Q else 0)
        f = nq * d["F_l"] + (d["headF"] if q == Q - 1 else 0.0)
        b = nq * d["B_l"] + (cfg["consts"]["bwd_factor"] * d["headF"] if q == Q - 1 else 0.0)
        F.append(f * oracle.jitter(seed, idx, q, 0))
        B.append(b * oracle.jitter(seed, idx, q, 1))
    return d, np.array(F), np.array(B)


def test_simulate_wiring_window_and_pricing():
    """orc_simulate = stage durations (balanced layer split, head on the last stage, jitter) -> fixed
    order -> makespan over min(m, 64) microbatches + steady-state extension -> same step terms and
    pricing as the analytic scorer."""
    cfg = variant("large_unconstrained", cluster=dict(budget_bytes=10 ** 15))
    for k in cfg["kern"]:
        k["avail_mask"] = 255
    o = Oracle(cfg)
    cases = [dict(sched=0, pp=4, tp=2, dp=8, ep=8, mb=1, v=1),     # 1F1B, m = 1920 > 64
             dict(sched=0, pp=16, tp=1, dp=64, ep=64, mb=15, v=1),  # m = 16
             dict(sched=2, pp=4, tp=2, dp=8, ep=8, mb=4, v=3),     # interleaved, Q = 12
             dict(sched=2, pp=8, tp=1, dp=16, ep=16, mb=15, v=2),  # m = 64
             dict(sched=3, pp=8, tp=1, dp=16, ep=16, mb=15, v=1),  # DualPipe-style
             dict(sched=3, pp=2, tp=4, dp=8, ep=32, mb=1, v=1),
             dict(sched=1, pp=1, tp=8, dp=8, ep=8, mb=2, v=1)]
    for c in cases:
        idx = axis_index(cfg, kv=1, rec=1, **c)
        d, F, B = _stage_times(o, cfg, idx, 4)
        assert d["reason"] & 0x7F == 0, (c, d["reason"])
        st, tput_sim, T_sim = o.simulate(idx, 4)
        assert st == 0
        kind, pp, v, m = d["kind"], d["pp"], d["v_eff"], d["m"]
        m_sim = min(m, 64)
        if kind == KINT:
            m_sim = (m_sim // pp) * pp
        T = oracle.makespan(kind, pp, v, m_sim, F, B, d["p"])
        if kind == KDUAL:
            W = max(0.5 * (F[r] + B[r] + F[pp - 1 - r] + B[pp - 1 - r]) for r in range(pp))
        else:
            W = max(sum(F[c2 * pp + r] + B[c2 * pp + r] for c2 in range(v)) for r in range(pp))
        T += (m - m_sim) * W
        assert T_sim == pytest.approx(T, rel=1e-13)
        T_step = T + (1 - cfg["consts"]["dp_overlap_frac"]) * d["T_dp"] + d["T_opt"] + cfg["consts"]["step_overhead"]
        tput = cfg["workload"]["gbs"] * cfg["model"]["seq"] / (T_step * d["world"])
        if not cfg["kern"][d["kv"]]["is_native"]:
            tput /= 1 + cfg["kern"][d["kv"]]["patch_ovh"]
        if d["ov"]:
            tput /= 1 + cfg["sched"][d["sched"]]["sched_ovh"]
        assert tput_sim == pytest.approx(tput, rel=1e-13)
        # jitter is +-10%, so the simulated score stays near the analytic one
        assert 0.6 * d["tput"] < tput_sim < 1.4 * d["tput"]


def test_window_extension_is_exact_for_uniform_1f1b():
    """With uniform stages the 1F1B makespan is linear in m with slope F + B, so simulating 64
    microbatches and extending with the bottleneck rank's work reproduces the closed form for any m."""
    for pp in (1, 2, 8):
        F, B = [1.5] * pp, [2.5] * pp
        for m in (65, 100, 1000):
            T = oracle.makespan(K1F1B, pp, 1, 64, F, B, 0.0) + (m - 64) * 4.0
            assert T == (m + pp - 1) * 4.0


def test_simulate_outside_domain_keeps_analytic_score():
    cfg = variant("large_unconstrained", cluster=dict(budget_bytes=10 ** 15))
    for k in cfg["kern"]:
        k["avail_mask"] = 255
    o = Oracle(cfg)
    idx = axis_index(cfg, sched=0, pp=64, tp=1, dp=16, ep=16, mb=1, v=1)
    d = o.eval(idx)
    # L = 61 < 64 stages: rejected by LAYERS, so widen the model for this check
    assert d["reason"] & 0x7F == 6
    cfg["model"]["L"] = 128
    o = Oracle(cfg)
    d = o.eval(idx)
    assert d["reason"] & 0x7F == 0
    st, tput_sim, _ = o.simulate(idx, 4)
    assert st == 1 and tput_sim == d["tput"]
    # and such candidates are never selected as survivors
    reason = np.zeros(1, dtype=np.uint8)
    assert len(o.select_survivors(reason, np.array([d["tput"]]), idx, 10)) == 0


def test_simulate_infeasible_candidate_scores_zero():
    cfg = make_config("tiny")
    o = Oracle(cfg)
    idx = axis_index(cfg, sched=2)  # DualPipe: unmapped
    st, t, _ = o.simulate(idx, 4)
    assert st == 1 and t == 0.0
