"""The roofline probes run, report their instruction counts and reject bad arguments."""
from __future__ import annotations

import pytest

pytestmark = pytest.mark.gpu


def test_probes_report_counts_and_plausible_rates():
    import torch
    from paper_2607_18631_b200 import build as pf_build, probes as binding
    pf_build.build()

    dev = torch.device("cuda", 0)
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    sink = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    for kind in ("ffma", "imad", "logic"):
        binding.pf_probe_alu(kind, 64, sink)                     # warm-up
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        n = binding.pf_probe_alu(kind, 2048, sink)
        b.record(stream)
        torch.cuda.synchronize()
        assert n == sms * 8 * 256 * 2048 * 8 * 4
        rate = n / (a.elapsed_time(b) * 1e-3)
        # between a tenth of and slightly above SMs x 4 schedulers x 32 lanes x 2.1 GHz
        assert 0.1 * sms * 128 * 2.1e9 < rate < 1.05 * sms * 128 * 2.1e9, (kind, rate)
    assert int(sink.item()) == 0

    buf = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    binding.pf_probe_write(buf)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    nbytes = binding.pf_probe_write(buf)
    b.record(stream)
    torch.cuda.synchronize()
    assert nbytes == 512 << 20
    assert bool((buf == 0x5A).all())
    gbs = nbytes / (a.elapsed_time(b) * 1e-3) / 1e9
    assert 1000.0 < gbs < 12000.0, gbs


def test_probes_reject_bad_arguments():
    import torch
    from paper_2607_18631_b200 import build as pf_build, probes as binding
    pf_build.build()

    dev = torch.device("cuda", 0)
    sink = torch.zeros(1, dtype=torch.int32, device=dev)
    with pytest.raises(binding.ProbeError):
        binding.pf_probe_alu("ffma", 0, sink)
    with pytest.raises(binding.ProbeError):
        binding.pf_probe_alu("ffma", (1 << 24) + 1, sink)
    buf = torch.empty(64, dtype=torch.uint8, device=dev)
    with pytest.raises(binding.ProbeError):
        binding.pf_probe_write(buf[:24])                         # not a multiple of 16 bytes
    with pytest.raises(binding.ProbeError):
        binding.pf_probe_write(buf[8:40])                        # not 16-byte aligned


def test_timing_hooks_count_kernels_by_class_mask_and_stride():
    """pf_timing_enable / pf_timing_classes / pf_timing_read: every class of a search is reported with its kernel count;
    a class mask leaves the others at zero; a stride times every n-th launch group of a class; the results of the
    search do not depend on any of it."""
    import torch
    from paper_2607_18631_b200 import Plan
    from workloads import make_config
    plan = Plan(make_config("mid"))
    b = plan.search(64, 1000, 10, 3)
    torch.cuda.synchronize()
    ref = {k: b[k].clone() for k in ("reason", "tput", "sim_topk_idx", "sim_topk_score", "surv_count")}

    def run(n):
        for _ in range(n):
            plan.search(64, 1000, 10, 3, bufs=b)
        torch.cuda.synchronize()
        for k in ref:
            assert torch.equal(b[k], ref[k]), k
        return plan.timing_read()

    assert all(v == (0.0, 0) for v in run(2).values())          # off by default
    plan.timing_enable(True)
    pc = run(4)
    assert pc["score"][1] == 4 and pc["fill"][1] == 4            # one scoring kernel and one fill kernel per call
    assert pc["select"][1] == 4 * 6 and pc["simprep"][1] == 4 * 3
    assert pc["simulate"][1] == 4 and pc["topk"][1] >= 8          # (a list that holds < 32,768 survivors: one instance)
    assert all(pc[c][0] > 0.0 for c in ("score", "fill", "select", "simprep", "simulate", "topk"))
    assert pc["aggregate"] == (0.0, 0) and pc["compact"] == (0.0, 0)
    plan.timing_classes(["fill"])
    pc = run(4)
    assert pc["fill"][1] == 4 and pc["fill"][0] > 0.0
    assert all(pc[c] == (0.0, 0) for c in pc if c != "fill")
    plan.timing_classes(["fill", "simulate"], every=3)
    pc = run(7)                                                   # launches 0, 3 and 6 of each class are timed
    assert pc["fill"][1] == 3 and pc["simulate"][1] == 3
    assert all(pc[c] == (0.0, 0) for c in pc if c not in ("fill", "simulate"))
    plan.timing_classes(None)
    plan.timing_enable(False)
    assert all(v == (0.0, 0) for v in run(2).values())
    plan.close()
