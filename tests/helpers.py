"""Shared test helpers: golden-file loading, config variants, comparison rules."""
from __future__ import annotations

import copy
import os

import numpy as np

from workloads import make_config

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")

TPUT_RTOL = 1e-4  # fp32 GPU vs fp64 oracle, relative


def load_kv(name: str) -> dict:
    """'key value' lines, '#' comments."""
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split()
            out[k] = float(v)
    return out


def load_rows(name: str):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            rows.append([int(x) for x in line.split()])
    return rows


def axis_index(cfg: dict, **values) -> int:
    """Linear index of the candidate whose axis VALUES are given (least-significant axis first)."""
    idx, stride = 0, 1
    for name, vals in cfg["axes"]:
        v = values.get(name, vals[0])
        idx += vals.index(v) * stride
        stride *= len(vals)
    return idx


def v2lite_like(ep_values=(2, 4, 8), budget=10 ** 15) -> dict:
    """An 8-GPU training space shaped like the paper's reference model as far as it is printed:
    64 experts of 2048 x 1408 (three matrices each), 26 MoE layers, dp = 8 at tp = pp = 1,
    embeddings not counted.  Everything else is a free choice that the pinned quantities do not
    depend on."""
    cfg = make_config("tiny")
    cfg["name"] = "v2lite_like"
    cfg["model"].update(L=26, H=2048, nh=16, nkv=16, hd=128, E=64, K=6, F=1408, S=0, Fs=0, seq=4096,
                        vocab=102400, count_embeddings=0)
    cfg["cluster"].update(G=8, budget_bytes=budget)
    cfg["workload"].update(gbs=64, world=8)
    cfg["rules"].update(world_min=1, world_max=8, ep_scope=0)
    cfg["axes"] = [("kv", [0]), ("rec", [0]), ("sched", [0]), ("mb", [1]), ("v", [0]), ("ep", list(ep_values)),
                   ("pp", [1]), ("tp", [1]), ("dp", [0]), ("world", [8])]
    return cfg


def variant(name: str, **sections) -> dict:
    """make_config(name) with per-section overrides, e.g. variant('mid', cluster=dict(budget_bytes=...))."""
    cfg = copy.deepcopy(make_config(name))
    for sec, upd in sections.items():
        if isinstance(cfg[sec], dict):
            cfg[sec].update(upd)
        else:
            cfg[sec] = upd
    return cfg


def check_topk(idx_gpu, score_gpu, idx_ref, score_ref, rtol=TPUT_RTOL):
    """Top-k parity: same length; scores agree position by position; index sets identical except for
    members whose reference score is within rtol of the k-th reference score (near-ties at the cut)
    -- and positions may swap only between entries whose scores are within rtol of each other."""
    idx_gpu = np.asarray(idx_gpu, dtype=np.uint64)
    idx_ref = np.asarray(idx_ref, dtype=np.uint64)
    assert len(idx_gpu) == len(idx_ref), (len(idx_gpu), len(idx_ref))
    if len(idx_ref) == 0:
        return
    score_gpu = np.asarray(score_gpu, dtype=np.float64)
    score_ref = np.asarray(score_ref, dtype=np.float64)
    np.testing.assert_allclose(score_gpu, score_ref, rtol=rtol)
    assert np.all(np.diff(score_gpu) <= 0), "top-k not sorted by score"
    kth = score_ref[-1]
    only_gpu = np.setdiff1d(idx_gpu, idx_ref)
    only_ref = np.setdiff1d(idx_ref, idx_gpu)
    ref_map = dict(zip(idx_ref.tolist(), score_ref.tolist()))
    gpu_map = dict(zip(idx_gpu.tolist(), score_gpu.tolist()))
    for i in only_ref.tolist():
        assert abs(ref_map[i] - kth) <= rtol * abs(kth), f"reference member {i} missing and not a near-tie"
    for i in only_gpu.tolist():
        assert abs(gpu_map[i] - kth) <= 2 * rtol * abs(kth), f"extra member {i} is not a near-tie"
    # order: wherever the two lists disagree at a position, the two scores there must be near-ties
    for a, b, sa, sb in zip(idx_gpu.tolist(), idx_ref.tolist(), score_gpu.tolist(), score_ref.tolist()):
        if a != b:
            assert abs(sa - sb) <= rtol * abs(sb)
