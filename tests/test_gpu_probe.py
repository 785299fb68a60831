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
