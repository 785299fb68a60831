"""Thin ctypes binding over libplanfront.so: argument marshalling only.

Every step of the path (decode, rules, memory, cost, pricing, top-k, survivor selection, simulation) runs in
the library's CUDA kernels.  PyTorch provides device memory and the current stream, nothing else.  There is
no CPU fallback: if the library is missing or no CUDA device is present, the calls raise.

Function names mirror the C ABI declared in include/planfront.h.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
# PLANFRONT_LIB: another build of the same library (the checked build, build.build(bounds_check=True))
LIB_PATH = os.environ.get("PLANFRONT_LIB") or os.path.join(HERE, "libplanfront.so")

MAX_AXES, MAX_SCHED, MAX_KERN, NBUCKET, K_MAX = 11, 8, 16, 8, 1024
PF_OK, PF_EINVAL, PF_ERANGE, PF_EWORKSPACE, PF_ECUDA, PF_EUNSUPPORTED = 0, -1, -2, -3, -4, -5
UINT64_MAX = 0xFFFFFFFFFFFFFFFF

EXPORTS = ("pf_version", "pf_strerror", "pf_reason_str", "pf_last_cuda_error", "pf_plan_create", "pf_plan_destroy",
           "pf_plan_size", "pf_decode", "pf_score_workspace", "pf_score", "pf_topk_merge", "pf_select_workspace",
           "pf_select_survivors", "pf_simulate_workspace", "pf_simulate", "pf_search_workspace", "pf_search_host",
           "pf_dualpipe_order", "pf_score_static", "pf_serve_plan_count", "pf_aggregate_workspace", "pf_aggregate_serving",
           "pf_report", "pf_search", "pf_search_device_workspace", "pf_compact_workspace", "pf_compact",
           "pf_search_compact_workspace", "pf_search_host_compact", "pf_select_hist", "pf_select_cut",
           "pf_select_write")
# measurement hooks of include/planfront_bench.h that this library exports (the probes live in probes.py)
BENCH_EXPORTS = ("pf_launch_count", "pf_timing_enable", "pf_timing_classes", "pf_timing_read", "pf_bench_fill_span", "pf_check_read", "pf_check_selftest")
STATIC_SCRATCH_BYTES = 4 << 20
T_CLASSES = ("score", "topk", "select", "simulate", "aggregate", "fill", "simprep", "compact")
REASON_BINS = 16
RECORD_DTYPE = np.dtype([("idx", "<u8"), ("mem", "<i8"), ("tput", "<f4"), ("reason", "u1"), ("pad", "u1", (3,))])

i32, u32, i64, u64, f32 = C.c_int32, C.c_uint32, C.c_int64, C.c_uint64, C.c_float


class PfModel(C.Structure):
    _fields_ = [(n, i32) for n in ("L", "H", "nh", "nkv", "hd", "attn_kind", "kv_latent", "rope_dim", "E", "K", "F",
                                   "S", "Fs", "seq", "vocab", "wb", "gb", "ob", "ab", "n_mats", "count_embeddings",
                                   "L_dense", "F_dense", "hd_q")]


class PfCluster(C.Structure):
    _fields_ = [("G", i32), ("caps", u32), ("budget_bytes", i64), ("reserved_bytes", i64)] + \
               [(n, f32) for n in ("peak_flops", "hbm_bw", "bw_intra", "bw_inter", "alpha_intra", "alpha_inter",
                                   "bw_host")] + [("gpu_id", i32)]


class PfWorkload(C.Structure):
    _fields_ = [("phase", i32), ("n_scen", i32), ("gbs", i64), ("world", i64),
                ("scen_P", C.POINTER(i32)), ("scen_O", C.POINTER(i32))]


class PfAxes(C.Structure):
    _fields_ = [("n_axes", i32), ("len", i32 * MAX_AXES), ("val", C.POINTER(i32) * MAX_AXES)]


class PfSched(C.Structure):
    _fields_ = [("kind", i32), ("overlap", i32), ("mapped", i32), ("hide_frac", f32), ("sched_ovh", f32),
                ("n_chunks", i32), ("sm_frac", f32)]


class PfKern(C.Structure):
    _fields_ = [("needs_caps", u32), ("avail_mask", u32), ("is_native", i32), ("wbytes", i32),
                ("dtype_mult", f32), ("eff", f32 * NBUCKET), ("patch_ovh", f32), ("dtype", i32)]


class PfDomain(C.Structure):
    _fields_ = [("attached", i32), ("gpu_id", i32), ("dtype_mask", u32), ("m_lo", i32), ("m_hi", i32)]


class PfReport(C.Structure):
    _fields_ = [("reason", C.c_uint8), ("why", C.c_uint8), ("bucket", C.c_uint16), ("reserved", u32), ("m_e", i64)]


REPORT_DTYPE = np.dtype([("reason", np.uint8), ("why", np.uint8), ("bucket", np.uint16), ("reserved", np.uint32),
                         ("m_e", np.int64)])


class PfTables(C.Structure):
    _fields_ = [(n, f32) for n in ("eff_dense", "bwd_factor", "dp_overlap_frac", "dualpipe_startup_div",
                                   "step_overhead", "offload_overlap_penalty")] + \
               [("n_sched", i32), ("sched", PfSched * MAX_SCHED), ("n_kern", i32), ("kern", PfKern * MAX_KERN),
                ("domain", PfDomain)]


class PfRules(C.Structure):
    _fields_ = [(n, i32) for n in ("ep_scope", "layer_mode", "tp_max", "world_min", "world_max",
                                   "enforce_realizability")]


class PfTuple(C.Structure):
    _fields_ = [(n, i32) for n in ("kv", "rec", "sched", "mb", "v", "ep", "pp", "tp", "dp", "world", "chunk",
                                   "batch", "dpa", "scen", "shard")]


class PlanfrontError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(what)


_lib = None


def load_library(path: str | None = None):
    """dlopen libplanfront.so and declare the signatures.  Raises if the library has not been built."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or LIB_PATH
    if not os.path.exists(path):
        raise PlanfrontError(PF_EINVAL, f"{path} not found: build it with `python -m paper_2607_18631_b200.build`")
    L = C.CDLL(path)
    vp, sz = C.c_void_p, C.c_size_t
    L.pf_version.restype = C.c_int
    L.pf_strerror.restype = C.c_char_p
    L.pf_strerror.argtypes = [C.c_int]
    L.pf_reason_str.restype = C.c_char_p
    L.pf_reason_str.argtypes = [C.c_uint8]
    L.pf_last_cuda_error.restype = C.c_char_p
    L.pf_plan_create.restype = C.c_int
    L.pf_plan_create.argtypes = [C.POINTER(PfModel), C.POINTER(PfCluster), C.POINTER(PfWorkload), C.POINTER(PfAxes),
                                 C.POINTER(PfTables), C.POINTER(PfRules), C.POINTER(vp)]
    L.pf_plan_destroy.restype = None
    L.pf_plan_destroy.argtypes = [vp]
    L.pf_plan_size.restype = u64
    L.pf_plan_size.argtypes = [vp]
    L.pf_decode.restype = C.c_int
    L.pf_decode.argtypes = [vp, u64, C.POINTER(PfTuple)]
    L.pf_score_workspace.restype = sz
    L.pf_score_workspace.argtypes = [vp, u64, u32]
    L.pf_score.restype = C.c_int
    L.pf_score.argtypes = [vp, u64, u64, vp, vp, vp, u32, vp, vp, vp, vp, sz, vp]
    L.pf_score_static.restype = C.c_int
    L.pf_score_static.argtypes = [vp, u64, u64, vp, vp, vp, u32, vp, vp, vp, vp]
    L.pf_serve_plan_count.restype = u64
    L.pf_serve_plan_count.argtypes = [vp]
    L.pf_aggregate_workspace.restype = sz
    L.pf_aggregate_workspace.argtypes = [vp, u32]
    L.pf_aggregate_serving.restype = C.c_int
    L.pf_aggregate_serving.argtypes = [vp, vp, vp, vp, vp, u32, vp, vp, vp, vp, sz, vp]
    L.pf_topk_merge.restype = C.c_int
    L.pf_topk_merge.argtypes = [u32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    L.pf_select_workspace.restype = sz
    L.pf_select_workspace.argtypes = [vp, u64, u64]
    L.pf_select_survivors.restype = C.c_int
    L.pf_select_survivors.argtypes = [vp, u64, u64, vp, vp, u64, vp, vp, vp, sz, vp]
    L.pf_simulate_workspace.restype = sz
    L.pf_simulate_workspace.argtypes = [vp, u64, u32]
    L.pf_simulate.restype = C.c_int
    L.pf_simulate.argtypes = [vp, vp, u64, vp, u32, vp, vp, u32, vp, vp, vp, vp, sz, vp]
    L.pf_search_workspace.restype = sz
    L.pf_search_workspace.argtypes = [vp, u32, u64, u32]
    L.pf_search_host.restype = C.c_int
    L.pf_search_host.argtypes = [vp, u32, u64, u32, u32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    L.pf_launch_count.restype = u64
    L.pf_timing_enable.restype = C.c_int
    L.pf_timing_enable.argtypes = [vp, C.c_int]
    L.pf_timing_classes.restype = C.c_int
    L.pf_timing_classes.argtypes = [vp, C.c_uint32, C.c_uint32]
    L.pf_timing_read.restype = C.c_int
    L.pf_timing_read.argtypes = [vp, vp, vp]
    L.pf_check_selftest.restype = C.c_int
    L.pf_check_selftest.argtypes = [vp]
    L.pf_check_read.restype = C.c_int
    L.pf_check_read.argtypes = [vp, vp]
    L.pf_bench_fill_span.restype = C.c_int
    L.pf_bench_fill_span.argtypes = [vp, C.POINTER(u64), C.POINTER(u64), C.POINTER(u64), C.POINTER(u64)]
    L.pf_dualpipe_order.restype = C.c_int
    L.pf_dualpipe_order.argtypes = [C.c_int, C.c_int, vp]
    L.pf_select_hist.restype = C.c_int
    L.pf_select_hist.argtypes = [vp, u64, u64, vp, vp, vp, vp, vp, sz, vp]
    L.pf_select_cut.restype = C.c_int
    L.pf_select_cut.argtypes = [vp, C.c_int, u64, vp, vp]
    L.pf_select_write.restype = C.c_int
    L.pf_select_write.argtypes = [vp, u64, u64, vp, vp, vp, u64, vp, u64, vp, vp, sz, vp]
    L.pf_compact_workspace.restype = sz
    L.pf_compact_workspace.argtypes = [u64]
    L.pf_compact.restype = C.c_int
    L.pf_compact.argtypes = [vp, u64, u64, vp, vp, vp, vp, vp, vp, u64, vp, vp, sz, vp]
    L.pf_search_compact_workspace.restype = sz
    L.pf_search_compact_workspace.argtypes = [vp, u32, u64, u32, u64]
    L.pf_search_host_compact.restype = C.c_int
    L.pf_search_host_compact.argtypes = [vp, u32, u64, u32, u32, vp, vp, vp, u64] + [vp] * 8 + [vp, sz, vp]
    L.pf_search_device_workspace.restype = sz
    L.pf_search_device_workspace.argtypes = [vp, u32, u64, u32]
    L.pf_search.restype = C.c_int
    L.pf_search.argtypes = [vp, u32, u64, u32, u32] + [vp] * 12 + [sz, vp]
    L.pf_report.restype = C.c_int
    L.pf_report.argtypes = [vp, vp, u32, vp, vp, vp]
    if path == LIB_PATH:
        _lib = L
    return L


def _check(status: int, what: str):
    if status != PF_OK:
        L = load_library()
        msg = L.pf_strerror(status).decode()
        if status == PF_ECUDA:
            msg += " (" + L.pf_last_cuda_error().decode() + ")"
        raise PlanfrontError(status, f"{what}: {msg}")


def pf_version() -> int:
    return int(load_library().pf_version())


def pf_strerror(status: int) -> str:
    return load_library().pf_strerror(status).decode()


def pf_reason_str(reason: int) -> str:
    return load_library().pf_reason_str(reason).decode()


def pf_launch_count() -> int:
    return int(load_library().pf_launch_count())


def pf_dualpipe_order(pp: int, m: int):
    """Host helper, needs no GPU: per-rank op order as lists of (position, microbatch, direction, is_backward)."""
    out = np.zeros(pp * 2 * m, dtype=np.uint8)
    _check(load_library().pf_dualpipe_order(pp, m, out.ctypes.data_as(C.c_void_p)), "pf_dualpipe_order")
    res = []
    for r in range(pp):
        ops = out[r * 2 * m:(r + 1) * 2 * m]
        res.append([((pp - 1 - r) if (int(o) >> 1) & 1 else r, int(o) >> 2, (int(o) >> 1) & 1, int(o) & 1)
                    for o in ops])
    return res


def _torch():
    import torch
    if not torch.cuda.is_available():
        raise PlanfrontError(PF_ECUDA, "no CUDA device: the plan-scoring path has no CPU fallback")
    return torch


def _dptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else None


def _stream_ptr(torch, stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


class Plan:
    """A plan space on the current CUDA device (pf_plan_create / pf_plan_destroy)."""

    def __init__(self, cfg: dict):
        torch = _torch()
        self._L = load_library()
        self.cfg = cfg
        self._keep = []
        m = PfModel(**{n: int(cfg["model"].get(n, 0)) for n, _ in PfModel._fields_})
        c = cfg["cluster"]
        cl = PfCluster(G=int(c["G"]), caps=int(c["caps"]), budget_bytes=int(c["budget_bytes"]),
                       reserved_bytes=int(c["reserved_bytes"]),
                       **{n: float(c[n]) for n in ("peak_flops", "hbm_bw", "bw_intra", "bw_inter", "alpha_intra",
                                                   "alpha_inter")}, bw_host=float(c.get("bw_host", 0.0)), gpu_id=int(c.get("gpu_id", 0)))
        w = cfg["workload"]
        sp = np.asarray(w.get("scen_P", []), dtype=np.int32)
        so = np.asarray(w.get("scen_O", []), dtype=np.int32)
        self._keep += [sp, so]
        wl = PfWorkload(phase=int(cfg["phase"]), n_scen=len(sp), gbs=int(w.get("gbs", 0)), world=int(w.get("world", 0)),
                        scen_P=sp.ctypes.data_as(C.POINTER(i32)), scen_O=so.ctypes.data_as(C.POINTER(i32)))
        ax = PfAxes()
        ax.n_axes = len(cfg["axes"])
        for a, (_, vals) in enumerate(cfg["axes"]):
            arr = np.asarray(vals, dtype=np.int32)
            self._keep.append(arr)
            ax.len[a] = len(arr)
            ax.val[a] = arr.ctypes.data_as(C.POINTER(i32))
        tb = PfTables(**{n: float(cfg["consts"][n]) for n in ("eff_dense", "bwd_factor", "dp_overlap_frac",
                                                               "dualpipe_startup_div", "step_overhead")},
                      offload_overlap_penalty=float(cfg["consts"].get("offload_overlap_penalty", 0.0)))
        tb.n_sched = len(cfg["sched"])
        for i, s in enumerate(cfg["sched"]):
            tb.sched[i] = PfSched(kind=int(s["kind"]), overlap=int(s["overlap"]), mapped=int(s["mapped"]),
                                  hide_frac=float(s["hide_frac"]), sched_ovh=float(s["sched_ovh"]),
                                  n_chunks=int(s.get("n_chunks", 0)), sm_frac=float(s.get("sm_frac", 0.0)))
        tb.n_kern = len(cfg["kern"])
        for i, k in enumerate(cfg["kern"]):
            kk = PfKern(needs_caps=int(k["needs_caps"]), avail_mask=int(k["avail_mask"]), is_native=int(k["is_native"]),
                        wbytes=int(k["wbytes"]), dtype_mult=float(k["dtype_mult"]), patch_ovh=float(k["patch_ovh"]),
                        dtype=int(k.get("dtype", 0)))
            for b in range(NBUCKET):
                kk.eff[b] = float(k["eff"][b])
            tb.kern[i] = kk
        dm = cfg.get("domain", dict(attached=0, gpu_id=-1, dtype_mask=0, m_lo=0, m_hi=0))
        tb.domain = PfDomain(attached=int(dm["attached"]), gpu_id=int(dm["gpu_id"]), dtype_mask=int(dm["dtype_mask"]),
                             m_lo=int(dm["m_lo"]), m_hi=int(dm["m_hi"]))
        ru = PfRules(**{n: int(cfg["rules"][n]) for n, _ in PfRules._fields_})
        h = C.c_void_p()
        _check(self._L.pf_plan_create(C.byref(m), C.byref(cl), C.byref(wl), C.byref(ax), C.byref(tb), C.byref(ru),
                                      C.byref(h)), "pf_plan_create")
        self._h = h
        self.size = int(self._L.pf_plan_size(h))
        self.device = torch.device("cuda", torch.cuda.current_device())

    def close(self):
        if getattr(self, "_h", None):
            self._L.pf_plan_destroy(self._h)
            self._h = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    # ---- pf_timing_enable / pf_timing_read
    def timing_enable(self, on: bool = True):
        _check(self._L.pf_timing_enable(self._h, 1 if on else 0), "pf_timing_enable")

    def timing_classes(self, names=None, every: int = 1):
        """pf_timing_classes: time only the named classes (names of T_CLASSES; None: all), every `every`-th time."""
        mask = 0xFFFFFFFF if names is None else sum(1 << T_CLASSES.index(n) for n in names)
        _check(self._L.pf_timing_classes(self._h, mask, every), "pf_timing_classes")

    def check_selftest(self) -> int:
        return int(self._L.pf_check_selftest(self._h))

    def check_read(self):
        """pf_check_read: (status, record of six words) of the checked build; status PF_EUNSUPPORTED otherwise."""
        out = np.zeros(6, dtype=np.uint32)
        st = self._L.pf_check_read(self._h, out.ctypes.data_as(C.c_void_p))
        return int(st), out

    def fill_span(self) -> dict:
        """pf_bench_fill_span: how the latest pf_search split the space between the scoring and the fill kernel."""
        a, b, c, d = u64(0), u64(0), u64(0), u64(0)
        _check(self._L.pf_bench_fill_span(self._h, C.byref(a), C.byref(b), C.byref(c), C.byref(d)),
               "pf_bench_fill_span")
        return dict(n_blocks=int(a.value), block_candidates=int(b.value), scored_blocks=int(c.value),
                    filled_blocks=int(d.value))

    def timing_read(self) -> dict:
        """{class: (milliseconds, kernels)} accumulated since the last read; waits for the recorded events."""
        ms = np.zeros(len(T_CLASSES), dtype=np.float32)
        nk = np.zeros(len(T_CLASSES), dtype=np.uint32)
        _check(self._L.pf_timing_read(self._h, ms.ctypes.data_as(C.c_void_p), nk.ctypes.data_as(C.c_void_p)),
               "pf_timing_read")
        return {n: (float(ms[i]), int(nk[i])) for i, n in enumerate(T_CLASSES)}

    # ---- pf_decode
    def decode(self, idx: int) -> dict:
        t = PfTuple()
        _check(self._L.pf_decode(self._h, idx, C.byref(t)), "pf_decode")
        return {n: getattr(t, n) for n, _ in PfTuple._fields_}

    # ---- pf_score
    def score_workspace(self, count: int, k: int) -> int:
        return int(self._L.pf_score_workspace(self._h, count, k))

    def score(self, first: int = 0, count: int | None = None, k: int = 0, reason=None, tput=None, mem=None,
              topk_idx=None, topk_score=None, topk_count=None, workspace=None, stream=None, dense: bool = True):
        """Enqueue pf_score.  Missing output tensors are allocated here (dense ones only if dense=True);
        returns a dict of the tensors used.  Does not synchronize."""
        torch = _torch()
        if count is None:
            count = self.size - first
        dev = self.device
        if dense:
            reason = torch.empty(count, dtype=torch.uint8, device=dev) if reason is None else reason
            tput = torch.empty(count, dtype=torch.float32, device=dev) if tput is None else tput
            mem = torch.empty(count, dtype=torch.int64, device=dev) if mem is None else mem
        if k > 0:
            topk_idx = torch.empty(k, dtype=torch.int64, device=dev) if topk_idx is None else topk_idx
            topk_score = torch.empty(k, dtype=torch.float32, device=dev) if topk_score is None else topk_score
            topk_count = torch.empty(1, dtype=torch.int32, device=dev) if topk_count is None else topk_count
        if workspace is None:
            workspace = torch.empty(self.score_workspace(count, k), dtype=torch.uint8, device=dev)
        _check(self._L.pf_score(self._h, first, count, _dptr(reason), _dptr(tput), _dptr(mem), k, _dptr(topk_idx),
                                _dptr(topk_score), _dptr(topk_count), _dptr(workspace), workspace.numel(),
                                _stream_ptr(torch, stream)), "pf_score")
        return dict(reason=reason, tput=tput, mem=mem, topk_idx=topk_idx, topk_score=topk_score,
                    topk_count=topk_count, workspace=workspace)

    # ---- pf_score_static
    def score_static(self, reason, tput, mem, k: int, topk_idx, topk_score, topk_count, first: int = 0,
                     count: int | None = None, stream=None):
        """Enqueue pf_score_static: the caller passes every buffer, nothing is allocated here or in the library
        (the scratch is the library's built-in array).  Does not synchronize."""
        torch = _torch()
        if count is None:
            count = self.size - first
        _check(self._L.pf_score_static(self._h, first, count, _dptr(reason), _dptr(tput), _dptr(mem), k,
                                       _dptr(topk_idx), _dptr(topk_score), _dptr(topk_count),
                                       _stream_ptr(torch, stream)), "pf_score_static")

    # ---- pf_select_survivors
    def select_workspace(self, count: int, s_max: int) -> int:
        return int(self._L.pf_select_workspace(self._h, count, s_max))

    def select_survivors(self, reason, tput, s_max: int, first: int = 0, surv_idx=None, surv_count=None,
                         workspace=None, stream=None):
        torch = _torch()
        count = reason.numel()
        dev = self.device
        surv_idx = torch.empty(max(s_max, 1), dtype=torch.int64, device=dev) if surv_idx is None else surv_idx
        surv_count = torch.empty(1, dtype=torch.int64, device=dev) if surv_count is None else surv_count
        if workspace is None:
            workspace = torch.empty(self.select_workspace(count, s_max), dtype=torch.uint8, device=dev)
        _check(self._L.pf_select_survivors(self._h, first, count, _dptr(reason), _dptr(tput), s_max, _dptr(surv_idx),
                                           _dptr(surv_count), _dptr(workspace), workspace.numel(),
                                           _stream_ptr(torch, stream)), "pf_select_survivors")
        return dict(surv_idx=surv_idx, surv_count=surv_count, workspace=workspace)

    # ---- the selection in steps (one space split over several GPUs)
    def select_hist(self, reason, tput, first: int = 0, cut=None, workspace=None, stream=None):
        """pf_select_hist: int32[65536] histogram of the high (cut None) or low (inside the cut's bin) 16 score bits
        of this slice's eligible candidates.  Does not synchronize."""
        torch = _torch()
        count = reason.numel()
        hist = torch.empty(65536, dtype=torch.int32, device=self.device)
        if workspace is None:
            workspace = torch.empty(self.select_workspace(count, 1), dtype=torch.uint8, device=self.device)
        _check(self._L.pf_select_hist(self._h, first, count, _dptr(reason), _dptr(tput), _dptr(cut), _dptr(hist),
                                      _dptr(workspace), workspace.numel(), _stream_ptr(torch, stream)),
               "pf_select_hist")
        return hist

    def select_write(self, reason, tput, cut, eq_before: int, cap: int, first: int = 0, workspace=None, stream=None):
        """pf_select_write: this slice's survivors under a cut.  Returns (surv_idx int64[cap], surv_count int64[1])."""
        torch = _torch()
        count = reason.numel()
        surv = torch.empty(max(cap, 1), dtype=torch.int64, device=self.device)
        n = torch.empty(1, dtype=torch.int64, device=self.device)
        if workspace is None:
            workspace = torch.empty(self.select_workspace(count, 1), dtype=torch.uint8, device=self.device)
        _check(self._L.pf_select_write(self._h, first, count, _dptr(reason), _dptr(tput), _dptr(cut), int(eq_before),
                                       _dptr(surv), max(cap, 1), _dptr(n), _dptr(workspace), workspace.numel(),
                                       _stream_ptr(torch, stream)), "pf_select_write")
        return surv, n

    # ---- pf_simulate
    def simulate_workspace(self, n: int, k: int) -> int:
        return int(self._L.pf_simulate_workspace(self._h, n, k))

    def simulate(self, surv_idx, n: int, jitter_seed: int, k: int = 0, d_n=None, tput_sim=None, sim_status=None,
                 topk_idx=None, topk_score=None, topk_count=None, workspace=None, stream=None, dense: bool = True):
        torch = _torch()
        dev = self.device
        if dense:
            tput_sim = torch.empty(max(n, 1), dtype=torch.float32, device=dev) if tput_sim is None else tput_sim
            sim_status = torch.empty(max(n, 1), dtype=torch.uint8, device=dev) if sim_status is None else sim_status
        if k > 0:
            topk_idx = torch.empty(k, dtype=torch.int64, device=dev) if topk_idx is None else topk_idx
            topk_score = torch.empty(k, dtype=torch.float32, device=dev) if topk_score is None else topk_score
            topk_count = torch.empty(1, dtype=torch.int32, device=dev) if topk_count is None else topk_count
        if workspace is None:
            workspace = torch.empty(self.simulate_workspace(n, k), dtype=torch.uint8, device=dev)
        _check(self._L.pf_simulate(self._h, _dptr(surv_idx), n, _dptr(d_n), jitter_seed, _dptr(tput_sim),
                                   _dptr(sim_status), k, _dptr(topk_idx), _dptr(topk_score), _dptr(topk_count),
                                   _dptr(workspace), workspace.numel(), _stream_ptr(torch, stream)), "pf_simulate")
        return dict(tput_sim=tput_sim, sim_status=sim_status, topk_idx=topk_idx, topk_score=topk_score,
                    topk_count=topk_count, workspace=workspace)

    # ---- pf_aggregate_serving
    # ---- pf_search (device buffers)
    def search_device_workspace(self, k: int, s_max: int, k_sim: int) -> int:
        return int(self._L.pf_search_device_workspace(self._h, k, s_max, k_sim))

    def search(self, k: int, s_max: int, k_sim: int, jitter_seed: int, bufs: dict | None = None, stream=None,
               want_mem: bool = True):
        """Enqueue pf_search: score + select + simulate in one call, everything on the device.  `bufs` (as returned
        by an earlier call) is reused; missing buffers are allocated here.  Does not synchronize."""
        torch = _torch()
        dev, N = self.device, self.size
        b = dict(bufs) if bufs else {}

        def get(name, n, dtype):
            if name not in b:
                b[name] = torch.empty(max(n, 1), dtype=dtype, device=dev)
            return b[name]
        reason, tput = get("reason", N, torch.uint8), get("tput", N, torch.float32)
        mem = get("mem", N, torch.int64) if want_mem else None
        tk_i, tk_s, tk_c = get("topk_idx", k, torch.int64), get("topk_score", k, torch.float32), get("topk_count", 1, torch.int32)
        sv, sv_c = get("surv_idx", s_max, torch.int64), get("surv_count", 1, torch.int64)
        si_i, si_s, si_c = (get("sim_topk_idx", k_sim, torch.int64), get("sim_topk_score", k_sim, torch.float32),
                            get("sim_topk_count", 1, torch.int32))
        ws = get("workspace", self.search_device_workspace(k, s_max, k_sim), torch.uint8)
        _check(self._L.pf_search(self._h, k, s_max, k_sim, jitter_seed, _dptr(reason), _dptr(tput), _dptr(mem),
                                 _dptr(tk_i), _dptr(tk_s), _dptr(tk_c), _dptr(sv), _dptr(sv_c), _dptr(si_i),
                                 _dptr(si_s), _dptr(si_c), _dptr(ws), ws.numel(), _stream_ptr(torch, stream)),
               "pf_search")
        return b

    # ---- pf_report
    def report(self, idx, n: int | None = None, d_n=None, out=None, stream=None):
        """Enqueue pf_report for the plan indices in `idx` (int64/uint64 device tensor).  Returns a uint8 device
        tensor of n x 16 bytes; `report_to_numpy` views it as records (reason, why, bucket, m_e)."""
        torch = _torch()
        n = idx.numel() if n is None else n
        out = torch.empty(max(n, 1) * C.sizeof(PfReport), dtype=torch.uint8, device=self.device) if out is None else out
        _check(self._L.pf_report(self._h, _dptr(idx), n, _dptr(d_n), _dptr(out), _stream_ptr(torch, stream)),
               "pf_report")
        return out

    @staticmethod
    def report_to_numpy(out, n: int):
        return out.cpu().numpy()[:n * REPORT_DTYPE.itemsize].view(REPORT_DTYPE)

    def serve_plan_count(self) -> int:
        return int(self._L.pf_serve_plan_count(self._h))

    def aggregate_serving(self, reason, tput, k: int = 0, plan_reason=None, plan_tput=None, topk_idx=None,
                          topk_score=None, topk_count=None, workspace=None, stream=None):
        """Enqueue pf_aggregate_serving on the dense outputs of a whole-space pf_score.  Does not synchronize."""
        torch = _torch()
        dev = self.device
        n = self.serve_plan_count()
        plan_reason = torch.empty(n, dtype=torch.uint8, device=dev) if plan_reason is None else plan_reason
        plan_tput = torch.empty(n, dtype=torch.float32, device=dev) if plan_tput is None else plan_tput
        if k > 0:
            topk_idx = torch.empty(k, dtype=torch.int64, device=dev) if topk_idx is None else topk_idx
            topk_score = torch.empty(k, dtype=torch.float32, device=dev) if topk_score is None else topk_score
            topk_count = torch.empty(1, dtype=torch.int32, device=dev) if topk_count is None else topk_count
        if workspace is None:
            workspace = torch.empty(int(self._L.pf_aggregate_workspace(self._h, k)), dtype=torch.uint8, device=dev)
        _check(self._L.pf_aggregate_serving(self._h, _dptr(reason), _dptr(tput), _dptr(plan_reason), _dptr(plan_tput),
                                            k, _dptr(topk_idx), _dptr(topk_score), _dptr(topk_count),
                                            _dptr(workspace), workspace.numel(), _stream_ptr(torch, stream)),
               "pf_aggregate_serving")
        return dict(plan_reason=plan_reason, plan_tput=plan_tput, topk_idx=topk_idx, topk_score=topk_score,
                    topk_count=topk_count, workspace=workspace)

    # ---- pf_compact
    def compact(self, reason, tput, mem, record_cap: int, first: int = 0, want_mask: bool = True, stream=None):
        """Enqueue pf_compact on dense outputs of candidates [first, first + len(reason)).  Returns device tensors:
        hist (int64[16]), mask (uint8[ceil(count / 8)] or None), records (uint8 view of record_cap records),
        n_feasible (int64[1]).  Does not synchronize."""
        torch = _torch()
        dev, count = self.device, reason.numel()
        hist = torch.empty(REASON_BINS, dtype=torch.int64, device=dev)
        mask = torch.empty((count + 7) // 8, dtype=torch.uint8, device=dev) if want_mask else None
        records = torch.empty(max(record_cap, 1) * RECORD_DTYPE.itemsize, dtype=torch.uint8, device=dev)
        n_feas = torch.empty(1, dtype=torch.int64, device=dev)
        ws = torch.empty(int(self._L.pf_compact_workspace(count)), dtype=torch.uint8, device=dev)
        _check(self._L.pf_compact(self._h, first, count, _dptr(reason), _dptr(tput), _dptr(mem), _dptr(hist),
                                  _dptr(mask), _dptr(records), record_cap, _dptr(n_feas), _dptr(ws), ws.numel(),
                                  _stream_ptr(torch, stream)), "pf_compact")
        return dict(hist=hist, mask=mask, records=records, n_feasible=n_feas, workspace=ws)

    @staticmethod
    def records_to_numpy(records, n: int):
        return records.cpu().numpy()[:n * RECORD_DTYPE.itemsize].view(RECORD_DTYPE)

    # ---- pf_search_host_compact
    def search_compact_workspace(self, k: int, s_max: int, k_sim: int, record_cap: int) -> int:
        return int(self._L.pf_search_compact_workspace(self._h, k, s_max, k_sim, record_cap))

    def search_host_compact(self, k: int, s_max: int, k_sim: int, jitter_seed: int, workspace, record_cap: int,
                            h_mask=None, h_records=None, stream=None):
        """pf_search_host_compact: the whole search with the compact view as the per-candidate result.  h_mask
        (uint8[N / 8]) and h_records (RECORD_DTYPE[record_cap]) may be numpy arrays or pinned torch tensors (bytes);
        both optional.  Returns a dict of numpy results; synchronous."""
        torch = _torch()

        def hptr(x):
            if x is None:
                return None
            return C.c_void_p(x.data_ptr()) if hasattr(x, "data_ptr") else x.ctypes.data_as(C.c_void_p)
        if record_cap > 0 and h_records is None:
            h_records = np.empty(record_cap, dtype=RECORD_DTYPE)
        hist = np.zeros(REASON_BINS, dtype=np.uint64)
        nfeas = np.zeros(1, dtype=np.uint64)
        ti = np.empty(max(k, 1), dtype=np.uint64)
        ts = np.empty(max(k, 1), dtype=np.float32)
        tc = np.zeros(1, dtype=np.uint32)
        si = np.empty(max(k_sim, 1), dtype=np.uint64)
        ss = np.empty(max(k_sim, 1), dtype=np.float32)
        sc = np.zeros(1, dtype=np.uint32)
        nsurv = np.zeros(1, dtype=np.uint64)
        _check(self._L.pf_search_host_compact(self._h, k, s_max, k_sim, jitter_seed, hptr(hist), hptr(h_mask),
                                              hptr(h_records), record_cap, hptr(nfeas), hptr(ti), hptr(ts), hptr(tc),
                                              hptr(si), hptr(ss), hptr(sc), hptr(nsurv), _dptr(workspace),
                                              workspace.numel(), _stream_ptr(torch, stream)),
               "pf_search_host_compact")
        n_rec = int(min(int(nfeas[0]), record_cap))
        return dict(hist=hist, n_feasible=int(nfeas[0]), n_records=n_rec, mask=h_mask, records=h_records,
                    topk_idx=ti[:tc[0]], topk_score=ts[:tc[0]], sim_topk_idx=si[:sc[0]], sim_topk_score=ss[:sc[0]],
                    n_survivors=int(nsurv[0]))

    # ---- pf_search_host
    def search_workspace(self, k: int, s_max: int, k_sim: int) -> int:
        return int(self._L.pf_search_workspace(self._h, k, s_max, k_sim))

    def search_host(self, k: int, s_max: int, k_sim: int, jitter_seed: int, workspace, h_reason=None, h_tput=None,
                    h_mem=None, stream=None):
        """pf_search_host with numpy / pinned-torch HOST buffers for the dense outputs (each may be None).
        Returns a dict of numpy results; synchronous."""
        torch = _torch()

        def hptr(x):
            if x is None:
                return None
            return C.c_void_p(x.data_ptr()) if hasattr(x, "data_ptr") else x.ctypes.data_as(C.c_void_p)
        ti = np.empty(max(k, 1), dtype=np.uint64)
        ts = np.empty(max(k, 1), dtype=np.float32)
        tc = np.zeros(1, dtype=np.uint32)
        si = np.empty(max(k_sim, 1), dtype=np.uint64)
        ss = np.empty(max(k_sim, 1), dtype=np.float32)
        sc = np.zeros(1, dtype=np.uint32)
        nsurv = np.zeros(1, dtype=np.uint64)
        _check(self._L.pf_search_host(self._h, k, s_max, k_sim, jitter_seed, hptr(h_reason), hptr(h_tput), hptr(h_mem),
                                      hptr(ti), hptr(ts), hptr(tc), hptr(si), hptr(ss), hptr(sc), hptr(nsurv),
                                      _dptr(workspace), workspace.numel(), _stream_ptr(torch, stream)),
               "pf_search_host")
        return dict(topk_idx=ti[:tc[0]], topk_score=ts[:tc[0]], sim_topk_idx=si[:sc[0]], sim_topk_score=ss[:sc[0]],
                    n_survivors=int(nsurv[0]))


CUT_DTYPE = np.dtype([("total", "<u8"), ("above_hi", "<u8"), ("n_gt", "<u8"), ("need_eq", "<u8"), ("target", "<u8"),
                      ("bin_hi", "<u4"), ("thr_bits", "<u4"), ("take_all", "<i4"), ("reserved", "<u4")])


def pf_select_cut(hist_sum, level: int, s_max: int, cut=None, stream=None):
    """pf_select_cut on a summed histogram (int64[65536] device tensor).  `cut`: the uint8[48] device tensor of the
    level-0 call when level is 1.  Returns the cut tensor.  Does not synchronize."""
    torch = _torch()
    if cut is None:
        cut = torch.zeros(CUT_DTYPE.itemsize, dtype=torch.uint8, device=hist_sum.device)
    _check(load_library().pf_select_cut(_dptr(hist_sum), level, s_max, _dptr(cut), _stream_ptr(torch, stream)),
           "pf_select_cut")
    return cut


def cut_to_numpy(cut):
    return cut.cpu().numpy().view(CUT_DTYPE)[0]


def pf_topk_merge(k: int, idx_a, score_a, count_a, idx_b, score_b, count_b, stream=None):
    """Merge two device top-k lists; returns (idx, score, count) device tensors."""
    torch = _torch()
    dev = idx_a.device
    oi = torch.empty(k, dtype=torch.int64, device=dev)
    os_ = torch.empty(k, dtype=torch.float32, device=dev)
    oc = torch.empty(1, dtype=torch.int32, device=dev)
    _check(load_library().pf_topk_merge(k, _dptr(idx_a), _dptr(score_a), _dptr(count_a), _dptr(idx_b), _dptr(score_b),
                                        _dptr(count_b), _dptr(oi), _dptr(os_), _dptr(oc), _stream_ptr(torch, stream)),
           "pf_topk_merge")
    return oi, os_, oc
