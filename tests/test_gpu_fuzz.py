"""Seeded random plan spaces: odd axis lengths and values, both EP scopes, both layer modes, derived and listed dp /
world, with and without the sharding axis, leading dense layers, calibration domains and two-stream schedules.
Every space is compared with the oracle element by element (scores, top-k, survivors, simulator)."""
from __future__ import annotations

import copy

import numpy as np
import pytest

from oracle import Oracle
from workloads import make_config

from gpu_common import compare_dense, compare_topk, gpu_score
from helpers import TPUT_RTOL

pytestmark = pytest.mark.gpu


def random_space(seed: int, big: bool = False) -> dict:
    rng = np.random.default_rng(seed)
    cfg = copy.deepcopy(make_config("mid"))
    pick = lambda pool, lo, hi: sorted(rng.choice(pool, size=int(rng.integers(lo, hi + 1)), replace=False).tolist())
    m = cfg["model"]
    m["L"] = int(rng.choice([12, 24, 27, 30, 32, 61]))
    m["nh"] = int(rng.choice([16, 24, 32, 48]))
    m["nkv"] = m["nh"]
    m["E"] = int(rng.choice([16, 48, 64, 96]))
    m["K"] = int(rng.choice([2, 4, 6]))
    m["S"] = int(rng.choice([0, 1, 2]))
    m["Fs"] = m["F"] if m["S"] else 0
    m["attn_kind"] = int(rng.integers(0, 2))
    if m["attn_kind"]:
        m["kv_latent"], m["rope_dim"] = 512, 64
    m["count_embeddings"] = int(rng.integers(0, 2))
    if rng.random() < 0.5:
        m["L_dense"], m["F_dense"] = int(rng.integers(1, 4)), int(rng.choice([2048, 11008, 40960]))
    if rng.random() < 0.3:
        m["hd_q"] = 192
    cfg["cluster"]["G"] = 8
    cfg["cluster"]["budget_bytes"] = int(rng.choice([30e9, 72e9, 1e15]))
    cfg["cluster"]["gpu_id"] = int(rng.integers(0, 2))
    cfg["workload"]["gbs"] = int(rng.choice([768, 1536, 3840, 7680]))
    cfg["workload"]["world"] = 0
    cfg["rules"].update(ep_scope=int(rng.integers(0, 2)), layer_mode=int(rng.choice([0, 2])), tp_max=8, world_min=1,
                        world_max=512, enforce_realizability=int(rng.integers(0, 2)))
    # either dp is derived from a few world sizes, or the world from listed dp values: most layouts then hold
    lo = 2 if big else 0   # big spaces: longer axes, hundreds of slabs (the slab-order and table paths)
    if rng.random() < 0.5:
        dp_axis, world_axis = [0], pick([8, 16, 24, 32, 48, 64, 96, 128], 2 + lo, 4 + lo)
    else:
        dp_axis, world_axis = pick([1, 2, 3, 4, 6, 8, 12, 16], 2 + lo, 5 + lo), [0]
    axes = [("kv", pick([0, 1, 2, 3], 1 + lo, 4)), ("rec", pick([0, 1, 2], 1 + lo, 3)), ("sched", pick([0, 1, 2], 2, 3)),
            ("mb", pick([1, 2, 3, 4, 6, 8], 2 + lo, 4 + lo)),
            ("v", [0] if rng.random() < 0.3 else pick([1, 2, 3, 4], 1 + lo, 3 + lo // 2)),
            ("ep", pick([1, 2, 3, 4, 6, 8, 12, 16], 2 + lo, 4 + lo)), ("pp", pick([1, 2, 3, 4, 6, 8], 2 + lo, 4 + lo)),
            ("tp", pick([1, 2, 4, 8], 1 + lo, 3 + lo // 2)), ("dp", dp_axis), ("world", world_axis)]
    if rng.random() < 0.5:
        axes.append(("shard", pick([0, 1, 2], 1, 3)))
    cfg["axes"] = axes
    for k in cfg["kern"]:
        k["avail_mask"] = int(rng.integers(1, 256))
        k["dtype"] = int(rng.integers(0, 2))
    for s in cfg["sched"]:
        s["mapped"] = int(rng.random() < 0.8)
        if s["overlap"] and rng.random() < 0.5:
            s["n_chunks"], s["sm_frac"] = int(rng.integers(1, 9)), float(np.float32(rng.uniform(0.0, 0.3)))
    cfg["domain"].update(attached=int(rng.random() < 0.8), gpu_id=int(rng.choice([-1, 0, 1])),
                         dtype_mask=int(rng.choice([1, 2, 3])), m_lo=int(rng.choice([16, 64, 256])),
                         m_hi=int(rng.choice([2048, 8192])))
    return cfg


@pytest.mark.parametrize("seed", list(range(24)) + [100 + i for i in range(8)])
def test_random_space_full_pipeline(seed):
    import torch
    from paper_2607_18631_b200 import Plan
    cfg = random_space(1000 + seed, big=seed >= 100)
    plan, orc = Plan(cfg), Oracle(cfg)
    assert plan.size == orc.size
    reason, tput, mem, _ = orc.score_range(threads=8)
    k = 64
    res = gpu_score(plan, k=k)
    compare_dense(res, reason, tput, mem)
    compare_topk(res, orc, reason, tput, 0, k)
    # an unaligned sub-range
    a, b = plan.size // 7 + 3, plan.size - plan.size // 5
    sub = gpu_score(plan, first=a, count=b - a, k=16)
    compare_dense(sub, reason[a:b], tput[a:b], mem[a:b])
    # the one-call search against the oracle's selection (on the device's own scores) and simulation
    s_max = int(np.random.default_rng(seed).choice([5, 200, 10 ** 6]))
    bufs = plan.search(k, s_max, 32, 4)
    torch.cuda.synchronize()
    n = int(bufs["surv_count"].item())
    got = bufs["surv_idx"][:n].cpu().numpy().view(np.uint64)
    want = orc.select_survivors(bufs["reason"].cpu().numpy(), bufs["tput"].cpu().numpy().astype(np.float64), 0, s_max)
    np.testing.assert_array_equal(got, want)
    if n:
        sim = plan.simulate(bufs["surv_idx"], n, 4, k=0)
        torch.cuda.synchronize()
        ref, ref_st, _ = orc.simulate_list(got, 4, threads=8)
        np.testing.assert_array_equal(sim["sim_status"][:n].cpu().numpy(), ref_st)
        np.testing.assert_allclose(sim["tput_sim"][:n].cpu().numpy(), ref, rtol=TPUT_RTOL, atol=0)
    plan.close()


def random_serving_space(seed: int) -> dict:
    rng = np.random.default_rng(seed)
    cfg = copy.deepcopy(make_config("serve"))
    pick = lambda pool, lo, hi: sorted(rng.choice(pool, size=int(rng.integers(lo, hi + 1)), replace=False).tolist())
    m = cfg["model"]
    m["L"] = int(rng.choice([24, 48, 61]))
    m["nh"] = int(rng.choice([24, 40, 64]))
    m["nkv"] = m["nh"]
    m["E"] = int(rng.choice([48, 128, 160]))
    m["K"] = int(rng.choice([4, 6, 8]))
    m["attn_kind"] = int(rng.integers(0, 2))
    world = int(rng.choice([4, 8, 16]))
    cfg["workload"]["world"] = world
    cfg["cluster"]["budget_bytes"] = int(rng.choice([40e9, 72e9, 1e15]))
    n_scen = int(rng.choice([1, 7, 32]))
    cfg["workload"]["scen_P"] = [int(x) for x in rng.integers(16, 20000, size=n_scen)]
    cfg["workload"]["scen_O"] = [int(x) for x in rng.integers(1, 4000, size=n_scen)]
    cfg["axes"] = [("kv", pick(list(range(6)), 1, 6)), ("chunk", pick([512, 1000, 2048, 4096, 8192], 1, 4)),
                   ("batch", pick([1, 2, 3, 8, 16, 48, 128, 512], 2, 6)), ("dpa", pick([0, 1], 1, 2)),
                   ("ep", pick([1, 2, 4, 8, 16], 1, 4)), ("tp", pick([1, 2, 4, 8], 1, 4)), ("scen", list(range(n_scen)))]
    for k in cfg["kern"]:
        k["avail_mask"] = int(rng.integers(1, 256))
    cfg["domain"].update(m_lo=int(rng.choice([1, 64])), m_hi=int(rng.choice([16, 8192])))
    # drawn last, so that the spaces above keep their earlier draws: leading dense layers and a query head width
    if rng.random() < 0.5:
        m["L_dense"] = int(rng.choice([1, 3]))
        m["F_dense"] = int(rng.choice([4096, 12288]))
        m["hd_q"] = int(rng.choice([0, 192]))
    return cfg


@pytest.mark.parametrize("seed", range(10))
def test_random_serving_space(seed):
    import torch
    from paper_2607_18631_b200 import Plan
    cfg = random_serving_space(2000 + seed)
    plan, orc = Plan(cfg), Oracle(cfg)
    reason, tput, mem, _ = orc.score_range(threads=8)
    res = gpu_score(plan, k=32)
    compare_dense(res, reason, tput, mem)
    compare_topk(res, orc, reason, tput, 0, 32)
    out = plan.score(k=0)
    agg = plan.aggregate_serving(out["reason"], out["tput"], k=8)
    torch.cuda.synchronize()
    pr, pt = orc.aggregate_serving(out["reason"].cpu().numpy(), out["tput"].cpu().numpy().astype(np.float64))
    np.testing.assert_array_equal(agg["plan_reason"].cpu().numpy(), pr)
    np.testing.assert_allclose(agg["plan_tput"].cpu().numpy(), pt, rtol=TPUT_RTOL, atol=0)
    plan.close()
