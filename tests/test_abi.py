"""CPU checks of the C-ABI library: it loads, exports what the header declares, and its host-only helpers
agree with the oracle.  No compute calls (no GPU here)."""
from __future__ import annotations

import os
import re

import pytest

import oracle
from paper_2607_18631_b200 import binding as B
from paper_2607_18631_b200 import build as pf_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    pf_build.build()
    return B.load_library()


def _declared_functions(header="planfront.h"):
    text = open(os.path.join(ROOT, "include", header)).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pf_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = _declared_functions()
    assert len(names) >= 18
    for n in names:
        assert hasattr(lib, n), f"{n} declared in planfront.h but not exported"
    assert set(names) == set(B.EXPORTS)


def test_measurement_hooks_are_declared_apart_and_exported_by_their_libraries(lib):
    """The scoring header declares no measurement utility; the benchmark header's hooks are exported by the scoring
    library (timing, launch count) and by the probe library (the roofline probes)."""
    from paper_2607_18631_b200 import probes
    product = set(_declared_functions())
    assert not {n for n in product if "probe" in n or "timing" in n or "launch_count" in n}
    bench = set(_declared_functions("planfront_bench.h"))
    assert bench == set(B.BENCH_EXPORTS) | set(probes.EXPORTS)
    for n in B.BENCH_EXPORTS:
        assert hasattr(lib, n)
    plib = probes.load_library()
    for n in probes.EXPORTS:
        assert hasattr(plib, n)
        assert not hasattr(lib, n), f"{n} must not be part of the scoring library"


def test_version_and_strings(lib):
    assert B.pf_version() == 100
    assert B.pf_strerror(0) == "ok"
    for st in (-1, -2, -3, -4, -5):
        assert B.pf_strerror(st) not in ("ok", "unknown status")
    assert B.pf_reason_str(11) == "memory_infeasible"      # the paper's own name for the memory-gate verdict
    assert "extrapolated" in B.pf_reason_str(0x80)
    assert all(B.pf_reason_str(r) != "unknown reason" for r in range(12))
    assert B.pf_launch_count() == 0


def test_create_rejects_bad_arguments_before_touching_the_device(lib):
    import ctypes as C
    h = C.c_void_p()
    assert lib.pf_plan_create(None, None, None, None, None, None, C.byref(h)) == B.PF_EINVAL
    assert lib.pf_plan_size(None) == 0
    assert lib.pf_score_workspace(None, 10, 1) == 256
    assert lib.pf_decode(None, 0, None) == B.PF_EINVAL
    assert lib.pf_topk_merge(0, None, None, None, None, None, None, None, None, None, None) == B.PF_EINVAL


def test_product_path_fails_loudly_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    from workloads import make_config
    with pytest.raises(B.PlanfrontError):
        B.Plan(make_config("tiny"))


def test_dualpipe_order_tables_match_the_oracle_definition(lib):
    """The library builds its DualPipe-style order tables on the host with its own list scheduler; the
    oracle has another.  Same definition, separately written: the orders must be identical."""
    for pp in (1, 2, 4, 6, 8, 10, 16, 32):
        for m in (2, 4, 6, 8, 16, 30, 32, 64):
            assert B.pf_dualpipe_order(pp, m) == oracle.schedule_order(2, pp, 1, m), (pp, m)
    with pytest.raises(B.PlanfrontError):
        B.pf_dualpipe_order(3, 8)
    with pytest.raises(B.PlanfrontError):
        B.pf_dualpipe_order(4, 7)


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2607_18631_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower() or f == "binding.py" and "oracle" not in text, (dirpath, f)
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c", ".h")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2607_18631_b200" not in text and "planfront.h" not in text
