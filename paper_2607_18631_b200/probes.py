"""ctypes binding of libplanfront_probe.so: the roofline probes a benchmark times (include/planfront_bench.h).

Measurement utilities only; the scoring path does not use them."""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libplanfront_probe.so")
EXPORTS = ("pf_probe_alu", "pf_probe_write")
PROBE_KINDS = {"ffma": 0, "imad": 1, "logic": 2}

_lib = None


def load_library():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run paper_2607_18631_b200.build.build()")
        L = C.CDLL(LIB_PATH)
        L.pf_probe_alu.restype = C.c_int
        L.pf_probe_alu.argtypes = [C.c_int, C.c_uint32, C.c_void_p, C.POINTER(C.c_uint64), C.c_void_p]
        L.pf_probe_write.restype = C.c_int
        L.pf_probe_write.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p]
        _lib = L
    return _lib


class ProbeError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: status {status}")
        self.status = status


def pf_probe_alu(kind: str, iters: int, sink) -> int:
    """Launch one issue-rate probe on the current stream; returns the thread-level instructions it executes."""
    import torch
    n = C.c_uint64(0)
    st = load_library().pf_probe_alu(PROBE_KINDS[kind], iters, sink.data_ptr(), C.byref(n),
                                     torch.cuda.current_stream().cuda_stream)
    if st != 0:
        raise ProbeError(st, "pf_probe_alu")
    return int(n.value)


def pf_probe_write(buf) -> int:
    """Fill `buf` (a device tensor, 16-byte aligned, size a multiple of 16 bytes) with streaming stores."""
    import torch
    nbytes = buf.numel() * buf.element_size()
    st = load_library().pf_probe_write(buf.data_ptr(), nbytes, torch.cuda.current_stream().cuda_stream)
    if st != 0:
        raise ProbeError(st, "pf_probe_write")
    return nbytes
