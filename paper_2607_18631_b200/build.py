"""In-tree build of libplanfront.so with nvcc for sm_100a (no JIT cache: the .so sits next to this file)."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(HERE, "libplanfront.so")
SOURCES = ["pf_api.cu", "pf_score.cu", "pf_select.cu", "pf_simulate.cu", "pf_search.cu", "pf_aggregate.cu", "pf_report.cu", "pf_compact.cu"]
# the roofline probes of the benchmark: a library of their own, not part of the scoring ABI
PROBE_LIB = os.path.join(HERE, "libplanfront_probe.so")
# the same library with every device-side index range-checked (-DPF_BOUNDS_CHECK): for the checked test run
CHECK_LIB = os.path.join(HERE, "libplanfront_check.so")
PROBE_SOURCES = ["pf_probe.cu"]


def _newest_source() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, f) for f in os.listdir(INCLUDE)]
    return max(os.path.getmtime(p) for p in paths)


def _compile(lib: str, sources, verbose: bool, defines=()) -> None:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-I" + INCLUDE, "-Xcompiler", "-fPIC", "-shared", "-o", lib]
    cmd += ["-D" + d for d in defines]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in sources]
    subprocess.run(cmd, check=True)


def build(force: bool = False, verbose: bool = False, bounds_check: bool = False) -> str:
    """Compile the scoring library (every scoring .cu into libplanfront.so) and the benchmark's probe library.
    Returns the scoring library's path.  bounds_check=True builds (only) the checked variant,
    libplanfront_check.so, and returns its path; PLANFRONT_LIB=<that path> makes the binding load it."""
    newest = _newest_source()
    if bounds_check:
        if force or not os.path.exists(CHECK_LIB) or os.path.getmtime(CHECK_LIB) < newest:
            _compile(CHECK_LIB, SOURCES, verbose, defines=("PF_BOUNDS_CHECK",))
        return CHECK_LIB
    if force or not os.path.exists(LIB) or os.path.getmtime(LIB) < newest:
        _compile(LIB, SOURCES, verbose)
    if force or not os.path.exists(PROBE_LIB) or os.path.getmtime(PROBE_LIB) < newest:
        _compile(PROBE_LIB, PROBE_SOURCES, verbose)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
