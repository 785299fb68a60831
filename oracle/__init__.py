"""CPU oracle for plan scoring (fp64 / int64, plain C).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package.  It shares
no code with the CUDA library and the CUDA library never falls back to it.

`build()` compiles planfront_oracle.c with gcc into liborc.so next to the source; `Oracle(cfg)` wraps a
problem description (a dict from `workloads.make_config`) and exposes the C entry points.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "planfront_oracle.c")
_HDR = os.path.join(_HERE, "planfront_oracle.h")
_LIB = os.path.join(_HERE, "liborc.so")
_LIB_COUNT = os.path.join(_HERE, "liborc_count.so")

MAX_SCHED, MAX_KERN, NBUCKET, MAX_AXES = 8, 16, 8, 11

REASON_NAMES = {0: "FEASIBLE", 1: "WORLD", 2: "TP", 3: "EP", 4: "BATCH", 5: "VSTAGE", 6: "LAYERS",
                7: "MICROBATCH", 8: "KERNEL_MISSING", 9: "UNMAPPED_SCHEDULE", 10: "OVERLAP_PRECOND",
                11: "MEMORY"}

i64, f64 = C.c_int64, C.c_double


def build(force: bool = False, count_ops: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP for the range/list helpers).  Returns the .so path.

    `count_ops=True` makes the operation-tallying build (-DORACLE_COUNT_OPS, liborc_count.so): same results,
    plus per-candidate integer/floating operation counts for an ALU roofline."""
    out = _LIB_COUNT if count_ops else _LIB
    if not force and os.path.exists(out):
        newest = max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))
        if os.path.getmtime(out) >= newest:
            return out
    cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off", "-Wall", "-Wextra"]
    if count_ops:
        cmd.append("-DORACLE_COUNT_OPS")
    cmd += ["-o", out, _SRC, "-lm"]
    subprocess.run(cmd, check=True, cwd=_HERE)
    return out


class Model(C.Structure):
    _fields_ = [(n, i64) for n in ("L", "H", "nh", "nkv", "hd", "attn_kind", "kv_latent", "rope_dim", "E", "K",
                                   "F", "S", "Fs", "seq", "vocab", "wb", "gb", "ob", "ab", "n_mats",
                                   "count_embeddings", "L_dense", "F_dense", "hd_q")]


class Cluster(C.Structure):
    _fields_ = [(n, i64) for n in ("G", "budget_bytes", "reserved_bytes", "caps")] + \
               [(n, f64) for n in ("peak_flops", "hbm_bw", "bw_intra", "bw_inter", "alpha_intra", "alpha_inter",
                                   "bw_host")] + [("gpu_id", i64)]


class Workload(C.Structure):
    _fields_ = [("phase", i64), ("gbs", i64), ("world", i64), ("n_scen", i64),
                ("scen_P", C.POINTER(i64)), ("scen_O", C.POINTER(i64))]


class Consts(C.Structure):
    _fields_ = [(n, f64) for n in ("eff_dense", "bwd_factor", "dp_overlap_frac", "dualpipe_startup_div",
                                   "step_overhead", "offload_overlap_penalty")]


class Sched(C.Structure):
    _fields_ = [("kind", i64), ("overlap", i64), ("mapped", i64), ("hide_frac", f64), ("sched_ovh", f64),
                ("n_chunks", i64), ("sm_frac", f64)]


class Kern(C.Structure):
    _fields_ = [("needs_caps", i64), ("avail_mask", i64), ("is_native", i64), ("wbytes", i64),
                ("dtype_mult", f64), ("eff", f64 * NBUCKET), ("patch_ovh", f64), ("dtype", i64)]


class Rules(C.Structure):
    _fields_ = [(n, i64) for n in ("ep_scope", "layer_mode", "tp_max", "world_min", "world_max",
                                   "enforce_realizability")]


class Domain(C.Structure):
    _fields_ = [(n, i64) for n in ("attached", "gpu_id", "dtype_mask", "m_lo", "m_hi")]


class Axes(C.Structure):
    _fields_ = [("n_axes", i64), ("len", i64 * MAX_AXES), ("val", C.POINTER(i64) * MAX_AXES)]


class Problem(C.Structure):
    _fields_ = [("model", Model), ("cluster", Cluster), ("workload", Workload), ("consts", Consts),
                ("n_sched", i64), ("sched", Sched * MAX_SCHED), ("n_kern", i64), ("kern", Kern * MAX_KERN),
                ("rules", Rules), ("axes", Axes), ("domain", Domain)]


class Derived(C.Structure):
    _fields_ = [(n, i64) for n in ("dk", "P_attn", "P_rt", "P_e", "P_sh", "P_dl", "P_emb", "a_attn", "a_fix",
                                   "a_ffn", "a_full", "a_sel", "a_ckpt", "f_attn", "f_rt", "f_sh", "f_dense",
                                   "f_exp", "f_head", "P_dld", "a_full_d", "a_sel_d", "f_mlp_d", "f_dense_d")]


class Detail(C.Structure):
    _fields_ = [(n, i64) for n in ("kv", "rec", "sched", "mb", "v", "ep", "pp", "tp", "dp", "world", "shard", "chunk",
                                   "batch", "dpa", "scen", "kind", "ov", "v_eff", "m", "t", "Q", "Lc", "Ls",
                                   "edp", "m_e", "bucket", "bucket_pre", "nd0", "nd_last", "N_dense", "N_exp", "bytes_w",
                                   "bytes_g", "bytes_o_dense", "bytes_o_expert", "bytes_o", "bytes_a", "bytes_buf",
                                   "mem")] + \
               [(n, f64) for n in ("cF", "cB", "rc", "tpc", "a2a", "xF", "xB", "F_l", "B_l", "headF", "F", "B",
                                   "p", "T_pipe", "T_dp", "T_opt", "T_step", "T_dec", "T_pre", "F_ld", "B_ld", "cD", "cE",
                                   "tput_unpriced",
                                   "tput")] + [("reason", i64), ("why", i64)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        L = _lib
        u64, u32, u8p = C.c_uint64, C.c_uint32, C.POINTER(C.c_uint8)
        PP = C.POINTER(Problem)
        L.orc_budget_bytes.restype = i64
        L.orc_budget_bytes.argtypes = [i64]
        L.orc_derive.restype = None
        L.orc_derive.argtypes = [C.POINTER(Model), C.POINTER(Derived)]
        L.orc_space_size.restype = u64
        L.orc_space_size.argtypes = [PP]
        L.orc_eval.restype = C.c_int
        L.orc_eval.argtypes = [PP, u64, C.POINTER(Detail)]
        L.orc_score_range.restype = C.c_int
        L.orc_score_range.argtypes = [PP, u64, u64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int]
        L.orc_topk.restype = u64
        L.orc_topk.argtypes = [C.c_void_p, C.c_void_p, u64, u64, u64, C.c_void_p, C.c_void_p]
        L.orc_topk_list.restype = u64
        L.orc_topk_list.argtypes = [C.c_void_p, C.c_void_p, u64, u64, C.c_void_p, C.c_void_p]
        L.orc_select_survivors.restype = u64
        L.orc_select_survivors.argtypes = [PP, C.c_void_p, C.c_void_p, u64, u64, u64, C.c_void_p]
        L.orc_serve_plan_count.restype = u64
        L.orc_serve_plan_count.argtypes = [PP]
        L.orc_aggregate_serving.restype = None
        L.orc_aggregate_serving.argtypes = [PP, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_schedule_order.restype = C.c_int
        L.orc_schedule_order.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_int]
        L.orc_makespan.restype = f64
        L.orc_makespan.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, f64]
        L.orc_two_stream_layer.restype = f64
        L.orc_two_stream_layer.argtypes = [f64, f64, f64, f64, C.c_int]
        L.orc_mix32.restype = u32
        L.orc_mix32.argtypes = [u32]
        L.orc_jitter.restype = f64
        L.orc_jitter.argtypes = [u32, u64, C.c_int, C.c_int]
        L.orc_simulate.restype = C.c_int
        L.orc_simulate.argtypes = [PP, u64, u32, C.POINTER(f64), C.POINTER(f64)]
        L.orc_simulate_list.restype = C.c_int
        L.orc_simulate_list.argtypes = [PP, C.c_void_p, u64, u32, C.c_void_p, C.c_void_p, C.c_int]
        del u8p
    return _lib


_lib_count = None


def count_ops(oracle: "Oracle", first: int = 0, count: int | None = None, threads: int = 1) -> dict:
    """Run the operation-tallying build over [first, first+count) of `oracle`'s space.

    Returns {"int_ops", "fp_ops", "candidates"} (totals); the reasons it computes are checked against nothing
    here -- the tally build differs from the plain one only by its counters."""
    global _lib_count
    if _lib_count is None:
        _lib_count = C.CDLL(build(count_ops=True))
        _lib_count.orc_score_range.restype = C.c_int
        _lib_count.orc_score_range.argtypes = [C.POINTER(Problem), C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p,
                                               C.c_void_p, C.c_int]
        _lib_count.orc_ops_enabled.restype = C.c_int
        _lib_count.orc_ops_reset.restype = None
        _lib_count.orc_ops_read.restype = None
        _lib_count.orc_ops_read.argtypes = [C.POINTER(i64 * 3)]
    L = _lib_count
    if not L.orc_ops_enabled():
        raise RuntimeError("liborc_count.so was not built with -DORACLE_COUNT_OPS")
    if count is None:
        count = oracle.size - first
    L.orc_ops_reset()
    L.orc_score_range(C.byref(oracle.pb), first, count, None, None, None, threads)
    out = (i64 * 3)()
    L.orc_ops_read(C.byref(out))
    return {"int_ops": int(out[0]), "fp_ops": int(out[1]), "candidates": int(out[2])}


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def budget_bytes(hbm_bytes: int) -> int:
    return int(lib().orc_budget_bytes(hbm_bytes))


def schedule_order(kind: int, pp: int, v: int, m: int):
    """Per-rank op order as a list (one per rank) of (q, j, direction, is_backward) tuples."""
    stride = 2 * m * max(v, 1)
    out = np.zeros(pp * stride, dtype=np.int32)
    n = lib().orc_schedule_order(kind, pp, v, m, _ptr(out), stride)
    if n < 0:
        raise ValueError(f"no order for kind={kind} pp={pp} v={v} m={m} (code {n})")
    res = []
    for r in range(pp):
        ops = out[r * stride:r * stride + n]
        res.append([((int(o) >> 2) & 255, int(o) >> 10, (int(o) >> 1) & 1, int(o) & 1) for o in ops])
    return res


def makespan(kind: int, pp: int, v: int, m: int, Fq, Bq, p: float) -> float:
    Fq = np.ascontiguousarray(Fq, dtype=np.float64)
    Bq = np.ascontiguousarray(Bq, dtype=np.float64)
    return float(lib().orc_makespan(kind, pp, v, m, _ptr(Fq), _ptr(Bq), float(p)))


def two_stream_layer(A: float, e_tot: float, d_tot: float, c_tot: float, n: int) -> float:
    return float(lib().orc_two_stream_layer(A, e_tot, d_tot, c_tot, n))


def mix32(x: int) -> int:
    return int(lib().orc_mix32(x & 0xFFFFFFFF))


def jitter(seed: int, idx: int, q: int, is_backward: int) -> float:
    return float(lib().orc_jitter(seed, idx, q, is_backward))


class Oracle:
    """A problem instance bound to the C oracle.  `cfg` is a dict from workloads.make_config()."""

    def __init__(self, cfg: dict):
        self.cfg = cfg
        self._keep = []
        pb = Problem()
        for n, _ in Model._fields_:
            setattr(pb.model, n, int(cfg["model"].get(n, 0)))
        for n, _ in Cluster._fields_:
            setattr(pb.cluster, n, cfg["cluster"][n])
        w = cfg["workload"]
        pb.workload.phase = int(cfg["phase"])
        pb.workload.gbs = int(w.get("gbs", 0))
        pb.workload.world = int(w.get("world", 0))
        sp = np.asarray(w.get("scen_P", []), dtype=np.int64)
        so = np.asarray(w.get("scen_O", []), dtype=np.int64)
        self._keep += [sp, so]
        pb.workload.n_scen = len(sp)
        pb.workload.scen_P = sp.ctypes.data_as(C.POINTER(i64))
        pb.workload.scen_O = so.ctypes.data_as(C.POINTER(i64))
        for n, _ in Consts._fields_:
            setattr(pb.consts, n, float(cfg["consts"][n]))
        pb.n_sched = len(cfg["sched"])
        for i, s in enumerate(cfg["sched"]):
            for n, _ in Sched._fields_:
                setattr(pb.sched[i], n, s.get(n, 0))
        pb.n_kern = len(cfg["kern"])
        for i, k in enumerate(cfg["kern"]):
            for n in ("needs_caps", "avail_mask", "is_native", "wbytes"):
                setattr(pb.kern[i], n, int(k[n]))
            pb.kern[i].dtype_mult = float(k["dtype_mult"])
            pb.kern[i].patch_ovh = float(k["patch_ovh"])
            pb.kern[i].dtype = int(k.get("dtype", 0))
            for b in range(NBUCKET):
                pb.kern[i].eff[b] = float(k["eff"][b])
        for n, _ in Rules._fields_:
            setattr(pb.rules, n, int(cfg["rules"][n]))
        for n, _ in Domain._fields_:
            setattr(pb.domain, n, int(cfg["domain"][n]))
        pb.axes.n_axes = len(cfg["axes"])
        for a, (_, vals) in enumerate(cfg["axes"]):
            arr = np.asarray(vals, dtype=np.int64)
            self._keep.append(arr)
            pb.axes.len[a] = len(arr)
            pb.axes.val[a] = arr.ctypes.data_as(C.POINTER(i64))
        self.pb = pb
        self.size = int(lib().orc_space_size(C.byref(pb)))

    def derived(self) -> dict:
        d = Derived()
        lib().orc_derive(C.byref(self.pb.model), C.byref(d))
        return {n: getattr(d, n) for n, _ in Derived._fields_}

    def eval(self, idx: int) -> dict:
        d = Detail()
        lib().orc_eval(C.byref(self.pb), idx, C.byref(d))
        return d.as_dict()

    def score_range(self, first: int = 0, count: int | None = None, threads: int = 1,
                    want_mem: bool = True, want_tput: bool = True):
        """Returns (reason uint8[count], tput float64[count], mem int64[count], threads_used)."""
        if count is None:
            count = self.size - first
        reason = np.zeros(count, dtype=np.uint8)
        tput = np.zeros(count, dtype=np.float64) if want_tput else None
        mem = np.zeros(count, dtype=np.int64) if want_mem else None
        used = lib().orc_score_range(C.byref(self.pb), first, count, _ptr(reason),
                                     _ptr(tput) if want_tput else None, _ptr(mem) if want_mem else None,
                                     threads)
        return reason, tput, mem, int(used)

    def topk(self, reason, tput, first: int, k: int):
        oi = np.zeros(k, dtype=np.uint64)
        os_ = np.zeros(k, dtype=np.float64)
        n = lib().orc_topk(_ptr(reason), _ptr(tput), first, len(reason), k, _ptr(oi), _ptr(os_))
        return oi[:n], os_[:n]

    @staticmethod
    def topk_list(idx, score, k: int):
        idx = np.ascontiguousarray(idx, dtype=np.uint64)
        score = np.ascontiguousarray(score, dtype=np.float64)
        oi = np.zeros(k, dtype=np.uint64)
        os_ = np.zeros(k, dtype=np.float64)
        n = lib().orc_topk_list(_ptr(idx), _ptr(score), len(idx), k, _ptr(oi), _ptr(os_))
        return oi[:n], os_[:n]

    def aggregate_serving(self, reason, tput):
        """Per-plan (reason uint8[n_plans], tput float64[n_plans]) over all length scenarios."""
        n = int(lib().orc_serve_plan_count(C.byref(self.pb)))
        reason = np.ascontiguousarray(reason, dtype=np.uint8)
        tput = np.ascontiguousarray(tput, dtype=np.float64)
        pr = np.zeros(n, dtype=np.uint8)
        pt = np.zeros(n, dtype=np.float64)
        lib().orc_aggregate_serving(C.byref(self.pb), _ptr(reason), _ptr(tput), _ptr(pr), _ptr(pt))
        return pr, pt

    def select_survivors(self, reason, tput, first: int, s_max: int):
        out = np.zeros(max(min(s_max, len(reason)), 1), dtype=np.uint64)
        n = lib().orc_select_survivors(C.byref(self.pb), _ptr(reason), _ptr(tput), first, len(reason), s_max,
                                       _ptr(out))
        return out[:n]

    def simulate(self, idx: int, seed: int):
        t, tp = f64(0.0), f64(0.0)
        st = lib().orc_simulate(C.byref(self.pb), idx, seed, C.byref(t), C.byref(tp))
        return int(st), t.value, tp.value

    def simulate_list(self, idx, seed: int, threads: int = 1):
        idx = np.ascontiguousarray(idx, dtype=np.uint64)
        t = np.zeros(len(idx), dtype=np.float64)
        st = np.zeros(len(idx), dtype=np.uint8)
        used = lib().orc_simulate_list(C.byref(self.pb), _ptr(idx), len(idx), seed, _ptr(t), _ptr(st), threads)
        return t, st, int(used)
