"""The five synthetic plan spaces.

Each config is a plain dict:
  name, phase (0 train / 1 serve), k (top-k size),
  model{...ints}, cluster{ints + fp32 floats}, workload{gbs | world, scen_P, scen_O},
  consts{fp32}, sched[list of dict], kern[list of dict], rules{ints},
  axes: list of (axis name, [int values]) least-significant axis first.

Every float is rounded to fp32 once here, so the fp32 GPU path and the fp64 oracle read the same
numbers.  Tables are drawn from numpy's default_rng(seed) in a fixed order (see table_draws).
The spaces stand in for the paper's workloads (a v2-lite-class model on 8 GPUs, a DeepSeek-V3-class
model on up to 1024 GPUs, a large-EP serving deployment), whose constant sets are not published:
they keep the structure -- divisor-structured parallel axes, three schedule classes, a kernel-variant
axis, multiplicative overhead tables -- with seeded random tables.
"""
from __future__ import annotations

import numpy as np

CONFIG_NAMES = ("tiny", "mid", "serve", "large", "large_unconstrained")

KIND_1F1B, KIND_INTERLEAVED, KIND_DUALPIPE = 0, 1, 2
CAP_FP8, CAP_DEVICE_COMM = 1, 2

TRAIN_AXES = ("kv", "rec", "sched", "mb", "v", "ep", "pp", "tp", "dp", "world")
SERVE_AXES = ("kv", "chunk", "batch", "dpa", "ep", "tp", "scen")


def f32(x) -> float:
    """Round to fp32 and return as a Python float (exactly representable in both widths)."""
    return float(np.float32(x))


def table_draws(seed: int, n_kern: int, n_sched: int, p_avail: float):
    """Seeded tables, drawn in this order: eff[kv][0..7] ~ U[0.3, 0.8] (kv-major), patch_ovh[kv] ~
    U[0, 0.15], sched_ovh[s] ~ U[0, 0.15], availability draws a[kv][0..7] ~ U[0, 1) (bucket available
    iff a < p_avail).  Returns (rng, eff, patch_ovh, sched_ovh, avail_mask) with fp32-rounded floats."""
    rng = np.random.default_rng(seed)
    eff = rng.uniform(0.3, 0.8, size=(n_kern, 8)).astype(np.float32)
    patch = rng.uniform(0.0, 0.15, size=n_kern).astype(np.float32)
    sovh = rng.uniform(0.0, 0.15, size=n_sched).astype(np.float32)
    a = rng.random(size=(n_kern, 8))
    masks = [int(sum(1 << b for b in range(8) if a[kv, b] < p_avail)) for kv in range(n_kern)]
    return rng, eff, patch, sovh, masks


def _consts():
    # offload_overlap_penalty: the measured contention penalty the paper reports (0.0271)
    return dict(eff_dense=f32(0.5), bwd_factor=f32(2.0), dp_overlap_frac=f32(0.5),
                dualpipe_startup_div=f32(8.0), step_overhead=f32(0.0), offload_overlap_penalty=f32(0.0271))


# hidden fraction of the expert all-to-all per schedule class when overlap is on
HIDE = {KIND_1F1B: 0.3147, KIND_INTERLEAVED: 0.5073, KIND_DUALPIPE: 0.9}


def _sched(kind, overlap, mapped, sched_ovh):
    return dict(kind=kind, overlap=overlap, mapped=mapped,
                hide_frac=f32(HIDE[kind] if overlap else 0.0), sched_ovh=f32(sched_ovh))


def _kern(eff_row, patch, mask, is_native, fp8=False):
    return dict(needs_caps=CAP_FP8 if fp8 else 0, avail_mask=mask, is_native=is_native,
                wbytes=1 if fp8 else 2, dtype_mult=f32(2.0 if fp8 else 1.0),
                eff=[f32(e) for e in eff_row], patch_ovh=f32(patch), dtype=1 if fp8 else 0)


def _model(**kw):
    m = dict(L=0, H=0, nh=0, nkv=0, hd=0, attn_kind=0, kv_latent=0, rope_dim=0, E=0, K=0, F=0, S=0, Fs=0,
             seq=0, vocab=0, wb=2, gb=4, ob=12, ab=2, n_mats=3, count_embeddings=1)
    m.update(kw)
    return m


def _cluster(G, budget_bytes, peak, hbm_bw, bw_intra, bw_inter, a_intra, a_inter, caps=0, bw_host=55e9):
    # budget_bytes: usable HBM per modeled GPU (0.9 of a 24 GB / 80 GB part), given as integer bytes
    return dict(G=G, budget_bytes=budget_bytes, reserved_bytes=0, caps=caps,
                peak_flops=f32(peak), hbm_bw=f32(hbm_bw), bw_intra=f32(bw_intra), bw_inter=f32(bw_inter),
                alpha_intra=f32(a_intra), alpha_inter=f32(a_inter), bw_host=f32(bw_host), gpu_id=0)


def _tiny():
    _, eff, patch, sovh, masks = table_draws(0, 2, 3, 1.0)
    return dict(
        name="tiny", phase=0, k=16,
        model=_model(L=8, H=1024, nh=16, nkv=16, hd=64, E=8, K=2, F=2816, S=0, Fs=0, seq=2048, vocab=32000),
        cluster=_cluster(2, 21_600_000_000, 165e12, 1008e9, 32e9, 32e9, 10e-6, 10e-6),
        workload=dict(gbs=64, world=2, scen_P=[], scen_O=[]),
        consts=_consts(),
        sched=[_sched(KIND_1F1B, 0, 1, sovh[0]), _sched(KIND_INTERLEAVED, 0, 1, sovh[1]),
               _sched(KIND_DUALPIPE, 1, 0, sovh[2])],
        kern=[_kern(eff[0], patch[0], masks[0], 1), _kern(eff[1], patch[1], masks[1], 0)],
        rules=dict(ep_scope=0, layer_mode=0, tp_max=8, world_min=1, world_max=2, enforce_realizability=1),
        axes=[("kv", [0, 1]), ("rec", [0, 1, 2]), ("sched", [0, 1, 2]), ("mb", [1, 2, 4]), ("v", [0]),
              ("ep", [1, 2]), ("pp", [1, 2]), ("tp", [1, 2]), ("dp", [0]), ("world", [2])],
    )


def _mid():
    _, eff, patch, sovh, masks = table_draws(0, 4, 3, 0.9)
    p2 = [1, 2, 4, 8]
    return dict(
        name="mid", phase=0, k=128,
        model=_model(L=24, H=4096, nh=32, nkv=32, hd=128, E=64, K=6, F=1408, S=2, Fs=1408, seq=4096,
                     vocab=102400),
        cluster=_cluster(8, 72_000_000_000, 990e12, 3350e9, 200e9, 200e9, 5e-6, 5e-6),
        workload=dict(gbs=512, world=8, scen_P=[], scen_O=[]),
        consts=_consts(),
        sched=[_sched(KIND_1F1B, 0, 1, sovh[0]), _sched(KIND_INTERLEAVED, 1, 1, sovh[1]),
               _sched(KIND_DUALPIPE, 1, 0, sovh[2])],
        kern=[_kern(eff[i], patch[i], masks[i], 1 if i == 0 else 0) for i in range(4)],
        rules=dict(ep_scope=1, layer_mode=0, tp_max=8, world_min=1, world_max=8, enforce_realizability=1),
        axes=[("kv", [0, 1, 2, 3]), ("rec", [0, 1, 2]), ("sched", [0, 1, 2]), ("mb", [1, 2, 4, 8]),
              ("v", [1, 2, 4]), ("ep", p2), ("pp", p2), ("tp", p2), ("dp", p2), ("world", [8])],
    )


def _serve():
    rng, eff, patch, sovh, masks = table_draws(2, 6, 1, 0.9)
    # prompt / output lengths: lognormal with means 2048 / 512 (sigma 1), drawn after the tables
    z = rng.standard_normal(size=(128, 2))
    P = np.clip(np.rint(np.exp(np.log(2048.0) - 0.5 + z[:, 0])), 16, 32768).astype(np.int64)
    O = np.clip(np.rint(np.exp(np.log(512.0) - 0.5 + z[:, 1])), 1, 8192).astype(np.int64)
    return dict(
        name="serve", phase=1, k=128,
        model=_model(L=48, H=5120, nh=40, nkv=40, hd=128, attn_kind=1, kv_latent=512, rope_dim=64, E=128, K=8,
                     F=1536, S=1, Fs=1536, seq=4096, vocab=128000),
        cluster=_cluster(8, 72_000_000_000, 990e12, 3350e9, 200e9, 200e9, 5e-6, 5e-6, caps=CAP_FP8),
        workload=dict(gbs=0, world=8, scen_P=[int(x) for x in P], scen_O=[int(x) for x in O]),
        consts=_consts(),
        sched=[_sched(KIND_1F1B, 0, 1, sovh[0])],
        kern=[_kern(eff[i], patch[i], masks[i], 1 if i in (0, 3) else 0, fp8=(i >= 3)) for i in range(6)],
        rules=dict(ep_scope=0, layer_mode=0, tp_max=8, world_min=1, world_max=8, enforce_realizability=1),
        axes=[("kv", list(range(6))), ("chunk", [1024, 2048, 4096, 8192]),
              ("batch", [1 << i for i in range(10)]), ("dpa", [0, 1]), ("ep", [1, 2, 4, 8]),
              ("tp", [1, 2, 4, 8]), ("scen", list(range(128)))],
    )


def _large(enforce: int, seed: int = 0):
    _, eff, patch, sovh, masks = table_draws(seed, 8, 4, 0.9)
    p2 = [1 << i for i in range(11)]
    return dict(
        name="large" if enforce else "large_unconstrained", phase=0, k=1024,
        model=_model(L=61, H=7168, nh=128, nkv=128, hd=128, attn_kind=1, kv_latent=512, rope_dim=64, E=256,
                     K=8, F=2048, S=1, Fs=2048, seq=4096, vocab=129280),
        cluster=_cluster(8, 72_000_000_000, 990e12, 3350e9, 450e9, 400e9, 5e-6, 10e-6, caps=CAP_FP8),
        workload=dict(gbs=15360, world=0, scen_P=[], scen_O=[]),
        consts=_consts(),
        sched=[_sched(KIND_1F1B, 0, 1, sovh[0]), _sched(KIND_1F1B, 1, 1, sovh[1]),
               _sched(KIND_INTERLEAVED, 1, 1, sovh[2]), _sched(KIND_DUALPIPE, 1, 0, sovh[3])],
        kern=[_kern(eff[i], patch[i], masks[i], 1 if i in (0, 4) else 0, fp8=(i >= 4)) for i in range(8)],
        rules=dict(ep_scope=1, layer_mode=2, tp_max=8, world_min=16, world_max=1024,
                   enforce_realizability=enforce),
        axes=[("kv", list(range(8))), ("rec", [0, 1, 2]), ("sched", [0, 1, 2, 3]),
              ("mb", list(range(1, 17))), ("v", list(range(1, 9))), ("ep", p2), ("pp", p2), ("tp", p2),
              ("dp", p2), ("world", [0])],
    )


# The calibration domain the constants carry (paper, Appendix: tokens per expert in [64, 8192]); any GPU and any
# dtype by default, so that attaching it flags exactly the plans outside the fitted tokens-per-expert range.
def default_domain() -> dict:
    return dict(attached=1, gpu_id=-1, dtype_mask=0xFFFF, m_lo=64, m_hi=8192)


def make_config(name: str, seed: int = 0) -> dict:
    """Return a fresh config dict.  'large_unconstrained' is 'large' with the dry-run rules off
    (the paper's unconstrained search mode), used by the simulator tier.  `seed` re-draws the tables of
    the large spaces (independent problems of the same shape, one per GPU in a multi-GPU benchmark);
    the other spaces keep their fixed seeds."""
    if name == "tiny":
        cfg = _tiny()
    elif name == "mid":
        cfg = _mid()
    elif name == "serve":
        cfg = _serve()
    elif name == "large":
        cfg = _large(1, seed)
    elif name == "large_unconstrained":
        cfg = _large(0, seed)
    else:
        raise KeyError(name)
    cfg["domain"] = default_domain()
    return cfg


def space_size(cfg: dict) -> int:
    n = 1
    for _, vals in cfg["axes"]:
        n *= len(vals)
    return n
