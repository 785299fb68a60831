#!/usr/bin/env python
"""Benchmark of the plan-scoring hot path on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one pass of the whole path over the large training space (179,908,608 candidates): score every
candidate (reason byte, tokens/s/GPU, peak bytes, top-1024), select the best feasible survivors (up to 1e6),
simulate each survivor's pipeline schedule and re-rank the top-100 -- one pf_search call.  Rank 0 prints ONE JSON
line.

N > 1 (launched under torch.distributed.run): every rank scores an independent space of the same shape
(tables re-drawn from seed = rank); no data-path collective; value = all ranks' candidates / max time.
With --split the ranks share ONE space instead (contiguous index slices, strong scaling): the selection's
histograms are all-reduced and the top-k lists all-gathered over NCCL (paper_2607_18631_b200/sharding.py).

--impl reference times the CPU oracle (fp64, OpenMP over the host cores) on the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from workloads import make_config  # noqa: E402

METRIC = "candidate plans scored/sec on 1 B200 (feasibility+cost+top-k)"
UNIT = "candidates/s"
K_TOP, S_MAX, K_SIM, JITTER_SEED = 1024, 1_000_000, 100, 4
FILL_TIMING_EVERY = 8   # inside the timed region the fill kernel is bracketed by events on every eighth launch
BYTES_PER_CANDIDATE = 13          # dense outputs: reason u8 + tput f32 + mem i64
FALLBACK_HBM_GBS = 6650.0         # used only when MEASURED_PEAKS.json is absent
NOMINAL_HBM_GBS = 7700.0          # HGX B200 data-sheet figure, for context
# DRAM traffic of the fill kernel (the dominant kernel of a step), from one ncu capture on the profiling slice
# (profile_case.py: a 49 M-candidate cut of the same space; summary under profiles/): dram__bytes_read.sum +
# dram__bytes_write.sum of one fill_tail_kernel launch there, and the candidates that launch covers.  The kernel
# writes every byte once and reads nothing (0.1 MB read): the capture shows 542.4 MB of DRAM traffic for 602.1 MB
# of dense outputs -- the difference, 59.7 MB, is what still sat dirty in the 126 MB L2 when the kernel ended, a
# constant of the cache, not of the workload.  A full-space launch is therefore reported as its algorithmic bytes
# minus that residue.
FILL_KERNEL_SLICE_DRAM_BYTES = 542_420_224
FILL_KERNEL_SLICE_CANDIDATES = 46_313_472
# thread-level instructions the scoring kernel issues per plan that goes through the memory model, the step-time
# model and the price: smsp__thread_inst_executed.sum with the memory gate lifted minus with the gate on, over the
# plans the gate had rejected (ncu, profile_case.py --config large_unconstrained --topk-only; summary under profiles/)
COSTED_PLAN_THREAD_INSTRUCTIONS = 2780
# thread-level instructions one simulated op needs at least: load the dependency's end, add the hand-over latency,
# max with the rank's clock, add the duration, store the result, advance the cursor
SIM_INSTR_PER_OP = 6


def workload_config(world: int, n: int) -> dict:
    """The `config` object both arms print (identical for the same N)."""
    return {"workload": "large training space (config 4: 179,908,608 candidates, top-1024) + simulator tier on its "
                        "survivors (config 5: the s_max best feasible plans, top-100)",
            "candidates_per_gpu": n, "k": K_TOP, "s_max": S_MAX, "k_sim": K_SIM, "parallelism": f"dp{world}"}


def _measured_hbm():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML every 10 ms while running."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        names = {"hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
                 "hw_power_brake_slowdown": 0x80, "sw_power_cap": 0x4}
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                for n, bit in names.items():
                    if r & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            time.sleep(0.01)

    def start(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def _dist_setup(n_gpus: int):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return world, rank, local


# --------------------------------------------------------------------------------------------- oracle side

def oracle_step(orc, threads: int, sample_stride: int = 1):
    """The oracle's pass over the workload, as it stands: score (all host cores), full-sort top-k, survivor
    selection, simulation of the survivors, re-rank.  sample_stride > 1 scores every stride-th block of
    1,228,800 candidates (a bounded sample of the same space).  Returns candidates scored."""
    from oracle import Oracle
    N = orc.size
    block = 1_228_800
    scored = 0
    if sample_stride == 1:
        reason, tput, _mem, _ = orc.score_range(0, N, threads=threads)
        scored = N
        orc.topk(reason, tput, 0, K_TOP)
        surv = orc.select_survivors(reason, tput, 0, S_MAX)
        ts, _, _ = orc.simulate_list(surv, JITTER_SEED, threads=threads)
        Oracle.topk_list(surv, ts, K_SIM)
    else:
        for b0 in range(0, N, block * sample_stride):
            cnt = min(block, N - b0)
            reason, tput, _mem, _ = orc.score_range(b0, cnt, threads=threads)
            scored += cnt
            orc.topk(reason, tput, b0, K_TOP)
            surv = orc.select_survivors(reason, tput, b0, S_MAX)
            ts, _, _ = orc.simulate_list(surv, JITTER_SEED, threads=threads)
            Oracle.topk_list(surv, ts, K_SIM)
    return scored


def run_reference(args):
    world, rank, _ = _dist_setup(args.gpus)
    if rank != 0:
        return
    import oracle
    oracle.build()
    cfg = make_config("large")
    orc = oracle.Oracle(cfg)
    threads = os.cpu_count() or 1
    # bound the run: one probe block decides the sampling stride so that (steps + warmup) passes end in minutes
    t0 = time.perf_counter()
    orc.score_range(60_000_000, 1_228_800, threads=threads)
    probe = time.perf_counter() - t0
    est_full = probe * orc.size / 1_228_800
    budget = 150.0 / max(args.steps + args.warmup, 1)
    stride = max(1, int(np.ceil(est_full / budget)))
    used = orc.score_range(0, 1024, threads=threads)[3]
    for _ in range(args.warmup):
        oracle_step(orc, threads, stride)
    t0 = time.perf_counter()
    scored = 0
    for _ in range(args.steps):
        scored += oracle_step(orc, threads, stride)
    dt = time.perf_counter() - t0
    value = scored / dt
    sample = "whole space per step" if stride == 1 else f"every {stride}-th block of 1,228,800 candidates per step"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(world, orc.size),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": used, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------- CUDA side

def _time_launches(torch, stream, fn, reps=5, warm=2):
    """Average device time (ms) of fn() over `reps` launches on `stream`, after `warm` untimed ones."""
    for _ in range(warm):
        fn()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record(stream)
    for _ in range(reps):
        fn()
    b.record(stream)
    torch.cuda.synchronize()
    return a.elapsed_time(b) / reps


def _probe_peaks(torch, probes, stream, big):
    """Issue-rate peaks (thread-instructions/s) per instruction kind and the pure streaming-write rate (GB/s),
    measured with the probe library's kernels; `big` is a device buffer far larger than L2."""
    sink = torch.zeros(1, dtype=torch.int32, device=big.device)
    out = {}
    for kind in ("ffma", "imad", "logic"):
        n = [0]

        def go():
            n[0] = probes.pf_probe_alu(kind, 8192, sink)
        ms = _time_launches(torch, stream, go)
        out[kind] = n[0] / (ms * 1e-3)
    nbytes = big.numel() * big.element_size()
    ms = _time_launches(torch, stream, lambda: probes.pf_probe_write(big))
    return out, nbytes / (ms * 1e-3) / 1e9


def _survivor_shapes(plan, cfg, surv_host):
    """(simulated ops, longest per-rank op chain) of these survivors: 2 * (simulated microbatches) * (virtual
    stages) ops each, with the 64-microbatch window (for an interleaved schedule, a multiple of pp); a rank's chain
    is its 2 * m_sim * v ops plus the pipeline's fill."""
    gbs = int(cfg["workload"]["gbs"])
    total, longest = 0, 0
    for idx in surv_host:
        t = plan.decode(int(idx))
        kind = int(cfg["sched"][t["sched"]]["kind"])
        dp = t["dp"] if t["dp"] else t["world"] // (t["tp"] * t["pp"])
        m = gbs // (dp * t["mb"])
        v_eff = t["v"] if t["v"] else (2 if kind == 1 else 1)
        m_sim = min(m, 64)
        if kind == 1:
            m_sim = m if m <= 64 else (64 // t["pp"]) * t["pp"]
        v_sim = v_eff if kind == 1 else 1
        total += 2 * m_sim * t["pp"] * v_sim
        longest = max(longest, 2 * (m_sim * v_sim + t["pp"]))
    return total, longest


class SearchRig:
    """A plan with every buffer one pf_search call needs, allocated once."""

    def __init__(self, torch, cfg, k, s_max, k_sim):
        from paper_2607_18631_b200 import Plan
        self.torch, self.cfg, self.k, self.s_max, self.k_sim = torch, cfg, k, s_max, k_sim
        self.plan = Plan(cfg)
        N, dev = self.plan.size, self.plan.device
        self.N = N
        e = lambda n, dt: torch.empty(max(n, 1), dtype=dt, device=dev)
        self.bufs = dict(reason=e(N, torch.uint8), tput=e(N, torch.float32), mem=e(N, torch.int64),
                         topk_idx=e(k, torch.int64), topk_score=e(k, torch.float32), topk_count=e(1, torch.int32),
                         surv_idx=e(s_max, torch.int64), surv_count=e(1, torch.int64),
                         sim_topk_idx=e(k_sim, torch.int64), sim_topk_score=e(k_sim, torch.float32),
                         sim_topk_count=e(1, torch.int32),
                         workspace=e(self.plan.search_device_workspace(k, s_max, k_sim), torch.uint8))

    def step(self, stream):
        self.plan.search(self.k, self.s_max, self.k_sim, JITTER_SEED, bufs=self.bufs, stream=stream)

    def timed(self, stream, reps, warm=3):
        """(ms per call, per-class ms per call) over `reps` calls."""
        for _ in range(warm):
            self.step(stream)
        self.torch.cuda.synchronize()
        self.plan.timing_enable(True)
        self.plan.timing_read()
        a, b = self.torch.cuda.Event(enable_timing=True), self.torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(reps):
            self.step(stream)
        b.record(stream)
        self.torch.cuda.synchronize()
        pc = self.plan.timing_read()
        self.plan.timing_enable(False)
        return a.elapsed_time(b) / reps, {c: pc[c][0] / reps for c in pc if pc[c][1]}

    def close(self):
        self.plan.close()
        self.bufs = None


def _config_lines(torch, stream, hbm, peaks):
    """Device time per call on every benchmark space besides the headline one: configs 1-3, the large space scored
    alone, the unconstrained large space through the whole search (config 5b: 45,116 survivors), the same with the
    memory gate lifted (the cost-heavy scoring case: 1.17 M plans through the cost model; the simulator tier at its
    nominal 1e6 survivors).  Each line names what bounds it."""
    import oracle
    from paper_2607_18631_b200 import Plan
    out = {}
    for name, k in (("tiny", 16), ("mid", 128), ("serve", 128)):
        cfg = make_config(name)
        plan = Plan(cfg)
        o = plan.score(k=k)
        ms = _time_launches(torch, stream, lambda: plan.score(k=k, reason=o["reason"], tput=o["tput"], mem=o["mem"],
                                                              topk_idx=o["topk_idx"], topk_score=o["topk_score"],
                                                              topk_count=o["topk_count"], workspace=o["workspace"],
                                                              stream=stream), reps=20, warm=3)
        line = {"candidates": plan.size, "call": "pf_score", "ms_per_call": ms, "candidates_per_s": plan.size / (ms * 1e-3),
                "bound": "launch latency (the space is smaller than one wave of the GPU)" if plan.size < 5e5
                else "latency / issue (0.98 M candidates, every one evaluated)"}
        if name == "serve":
            ag = plan.aggregate_serving(o["reason"], o["tput"], k=k)
            ms_a = _time_launches(torch, stream, lambda: plan.aggregate_serving(
                o["reason"], o["tput"], k=k, plan_reason=ag["plan_reason"], plan_tput=ag["plan_tput"],
                topk_idx=ag["topk_idx"], topk_score=ag["topk_score"], topk_count=ag["topk_count"],
                workspace=ag["workspace"], stream=stream), reps=20, warm=3)
            line["aggregate_ms_per_call"] = ms_a
            line["plans"] = plan.serve_plan_count()
        out[name] = line
        plan.close()
        del o
    # the large space scored alone (one kernel writes everything): HBM-write bound
    cfg = make_config("large")
    plan = Plan(cfg)
    o = plan.score(k=K_TOP)
    ms = _time_launches(torch, stream, lambda: plan.score(k=K_TOP, reason=o["reason"], tput=o["tput"], mem=o["mem"],
                                                          topk_idx=o["topk_idx"], topk_score=o["topk_score"],
                                                          topk_count=o["topk_count"], workspace=o["workspace"],
                                                          stream=stream), reps=10, warm=3)
    out["large_pf_score"] = {"candidates": plan.size, "call": "pf_score", "ms_per_call": ms,
                             "candidates_per_s": plan.size / (ms * 1e-3), "bound": "hbm",
                             "achieved_gbs": BYTES_PER_CANDIDATE * plan.size / (ms * 1e-3) / 1e9,
                             "frac_of_measured_hbm": BYTES_PER_CANDIDATE * plan.size / (ms * 1e-3) / 1e9 / hbm}
    plan.close()
    del o
    torch.cuda.empty_cache()
    # config 5b and the nominal-size simulator tier
    for label, lift in (("large_unconstrained", False), ("large_unconstrained_gate_lifted", True)):
        cfg = make_config("large_unconstrained")
        if lift:
            cfg["cluster"]["budget_bytes"] = 10 ** 15
        rig = SearchRig(torch, cfg, K_TOP, S_MAX, K_SIM)
        ms, cls = rig.timed(stream, reps=10 if lift else 20)
        n_surv = int(rig.bufs["surv_count"].item())
        n_feas = int(((rig.bufs["reason"] & 0x7F) == 0).sum().item())
        ops, chain = _survivor_shapes(rig.plan, cfg, rig.bufs["surv_idx"][:n_surv].cpu().numpy()[::max(1, n_surv // 20000)])
        ops *= max(1, n_surv // 20000) if n_surv > 20000 else 1
        line = {"candidates": rig.N, "call": "pf_search", "ms_per_call": ms, "candidates_per_s": rig.N / (ms * 1e-3),
                "feasible": n_feas, "survivors": n_surv, "class_ms": cls,
                "simulator": {"ms": cls.get("simulate", 0.0), "survivors_per_s": n_surv / (cls["simulate"] * 1e-3),
                              "simulated_ops": ops, "longest_chain_steps": chain,
                              "alu_frac": SIM_INSTR_PER_OP * ops / peaks["logic"] / (cls["simulate"] * 1e-3)},
                "bound": "hbm (the fill kernel) beside the latency-bound simulator" if not lift
                else "alu / latency: the simulator's 1e6 survivors dominate the call"}
        if lift:
            # cost-heavy scoring: every feasible plan goes through the memory and step-time model.  ALU bound from
            # the oracle's operation tally over a sample of the FEASIBLE candidates only (the work the kernel cannot
            # skip), against the measured issue rates; HBM bound from the dense outputs.
            oracle.build()
            orc = oracle.Oracle(cfg)
            feas = torch.nonzero((rig.bufs["reason"] & 0x7F) == 0).flatten().cpu().numpy()
            pick = feas[:: max(1, len(feas) // 1500)]
            io = fo = 0
            for i in pick:
                c = oracle.count_ops(orc, int(i), 1)
                io += c["int_ops"]
                fo += c["fp_ops"]
            i_per, f_per = io / len(pick), fo / len(pick)
            t_alu = n_feas * (i_per / min(peaks["imad"], peaks["logic"]) + f_per / peaks["ffma"])
            t_hbm = rig.N * BYTES_PER_CANDIDATE / (hbm * 1e9)
            head_ms = cls.get("score", 0.0)
            line["cost_heavy_scoring"] = {
                "feasible_through_cost_model": n_feas, "int_ops_per_feasible": i_per, "fp_ops_per_feasible": f_per,
                "ops_source": f"oracle operation tally over {len(pick)} sampled feasible candidates",
                "t_alu_ms": t_alu * 1e3, "t_hbm_ms": t_hbm * 1e3, "score_kernel_ms": head_ms,
                "note": "the scoring kernel of this call writes the evaluated blocks only; its ALU work is the feasible "
                        "candidates' cost model plus the rule tables",
                "alu_frac_of_score_kernel": t_alu * 1e3 / head_ms if head_ms else None,
                # from the ncu capture summarised under profiles/ (score kernel, cost-heavy slice): what the
                # compiled kernel issues per plan it takes through the cost model, and the issue-rate bound on that
                "issued_thread_instructions_per_costed_plan": COSTED_PLAN_THREAD_INSTRUCTIONS,
                "t_issue_ms": n_feas * COSTED_PLAN_THREAD_INSTRUCTIONS / peaks["logic"] * 1e3,
                "issue_frac_of_score_kernel": (n_feas * COSTED_PLAN_THREAD_INSTRUCTIONS / peaks["logic"] * 1e3 / head_ms
                                               if head_ms else None)}
        out[label] = line
        rig.close()
        del rig
        torch.cuda.empty_cache()
    return out


def run_split(args, torch, dist, world, rank, local):
    """--split: ONE space cut into contiguous slices over the ranks (strong scaling).  A step is sharded_search:
    every rank scores and selects inside its slice, the selection's histograms are all-reduced so that the cut to the
    s_max best is exact across ranks, each rank simulates its own survivors, the top-k lists are all-gathered and
    folded.  The collectives are NCCL's through torch.distributed; one small device-to-host read per step (the cut)
    sits inside the timed region."""
    from paper_2607_18631_b200 import Plan, binding
    from paper_2607_18631_b200.sharding import CudaOps, sharded_search, shard_range
    cfg = make_config("large")
    plan = Plan(cfg)
    ops = CudaOps(plan)
    N = plan.size
    stream = torch.cuda.current_stream()

    def step():
        return sharded_search(ops, K_TOP, S_MAX, K_SIM, JITTER_SEED)

    for _ in range(max(args.warmup, 3)):
        r = step()
    dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    launches0 = binding.pf_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.start()
    dist.barrier()
    torch.cuda.synchronize()
    ev0.record(stream)
    for _ in range(args.steps):
        r = step()
    ev1.record(stream)
    torch.cuda.synchronize()
    dist.barrier()
    clocks = sampler.stop()
    t = torch.tensor([ev0.elapsed_time(ev1)], dtype=torch.float64, device=plan.device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_step = float(t.item()) / args.steps
    launches = binding.pf_launch_count() - launches0
    if rank == 0:
        first, count = shard_range(N, 0, world)
        cfgd = workload_config(world, count)
        cfgd["parallelism"] = f"one space split over {world} rank(s): contiguous index slices"
        line = {"metric": METRIC, "value": N / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
                "scaling": "strong", "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": cfgd,
                "survivors": r["n_survivors_total"], "clocks": clocks, "gpu_launches": int(launches),
                "collectives_per_step": {"all_reduce": 2, "all_reduce_bytes": 2 * 65536 * 8, "all_gather": 4,
                                         "all_gather_bytes_per_rank": (K_TOP + K_SIM) * 12 + 8 + 16},
                "note": "host-driven: per step one device-to-host read of the cut (48 bytes) sits between the "
                        "selection's passes; dense outputs and survivor lists stay on their ranks"}
        print(json.dumps(line))
    dist.destroy_process_group()


def run_ours(args):
    import torch
    from paper_2607_18631_b200 import Plan, binding

    world, rank, local = _dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (the scoring path has no CPU fallback)")
    torch.cuda.set_device(local)
    dist = None
    if world > 1 or args.split:
        import torch.distributed as dist
        if "MASTER_ADDR" not in os.environ:          # a single process asked for the split path
            os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT="29531", RANK="0", WORLD_SIZE="1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if args.split:
        return run_split(args, torch, dist, world, rank, local)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    cfg = make_config("large", seed=rank)
    rig = SearchRig(torch, cfg, K_TOP, S_MAX, K_SIM)
    plan, bufs, N, dev = rig.plan, rig.bufs, rig.N, rig.plan.device
    stream = torch.cuda.current_stream()

    def step():
        # one call: score (dense outputs + top-1024) -> select survivors -> simulate + top-100, all on the device
        rig.step(stream)

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()

    # ---- timed region: exactly K steps, device time on the launching stream
    # Inside the timed region only the dominant kernel (the fill kernel, on its own stream) is bracketed by the
    # library's event pairs, and only every eighth of its launches: an event between two kernels of the caller's
    # stream costs that chain its overlapped launches, and a timed event in front of the kernel the step waits for
    # last costs the step itself (0.411 ms per step untimed, 0.415 with every fill launch timed, 0.418 with every
    # class timed).  The other classes are timed in a pass of the same length right after the timed region.
    sampler = ClockSampler(local)
    plan.timing_classes(["fill"], every=FILL_TIMING_EVERY)
    plan.timing_enable(True)
    launches0 = binding.pf_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.start()
    barrier()
    ev0.record(stream)
    for _ in range(args.steps):
        step()
    ev1.record(stream)
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop()
    ms_total = ev0.elapsed_time(ev1)
    launches = binding.pf_launch_count() - launches0
    per_class = plan.timing_read()
    plan.timing_classes(None)
    for _ in range(args.steps):
        step()
    torch.cuda.synchronize()
    per_class_all = plan.timing_read()
    plan.timing_enable(False)
    fill_timed = per_class.get("fill", (0.0, 0))   # (ms, launches) of the launches timed inside the timed region
    per_class = dict(per_class_all)
    n_surv = int(bufs["surv_count"].item())

    t = torch.tensor([ms_total], dtype=torch.float64, device=dev)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_step = float(t.item()) / args.steps
    value = world * N / (ms_step * 1e-3)

    # ---- sustained region: the same step back to back for at least two seconds, clocks sampled throughout
    sustained = None
    if not args.no_sustained:
        n_sus = max(int(2.2e3 / ms_step), args.steps)
        sampler2 = ClockSampler(local)
        plan.timing_classes(["fill"], every=FILL_TIMING_EVERY)   # as in the timed region
        plan.timing_enable(True)
        plan.timing_read()
        sa, sb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        sampler2.start()
        sa.record(stream)
        for i in range(n_sus):
            step()
            if (i & 255) == 255:
                plan.timing_read()       # keeps the event pool bounded; the last block's figures are reported
        sb.record(stream)
        torch.cuda.synchronize()
        clocks2 = sampler2.stop()
        pc2 = plan.timing_read()
        plan.timing_enable(False)
        plan.timing_classes(None)
        n_last = (n_sus & 255) or 256
        if "fill" in pc2 and pc2["fill"][1]:
            pc2 = {"fill": (pc2["fill"][0] * n_last / pc2["fill"][1], pc2["fill"][1])}   # sampled: per timed launch
        ms_sus = sa.elapsed_time(sb) / n_sus
        sustained = {"steps": n_sus, "seconds": sa.elapsed_time(sb) * 1e-3, "ms_per_step": ms_sus,
                     "value": world * N / (ms_sus * 1e-3), "clocks": clocks2,
                     "ms_x_median_sm_mhz": ms_sus * clocks2["sm_mhz"] if clocks2["sm_mhz"] else None,
                     "class_ms_per_step": {c: pc2[c][0] / n_last for c in pc2 if pc2[c][1]}}
    barrier()

    # ---- end to end through the host-buffer calls: plan creation (uploads the inputs), the whole search, and the
    # results into pinned host memory, per step.  Compact: reason histogram + feasibility bits + records of the
    # feasible plans + the two top-k lists.  Dense: all thirteen bytes per candidate.
    h2d = sum(4 * len(v) for _, v in cfg["axes"])
    REC_CAP = 1 << 20
    ws_c = torch.empty(plan.search_compact_workspace(K_TOP, S_MAX, K_SIM, REC_CAP), dtype=torch.uint8, device=dev)
    h_mask = torch.empty((N + 7) // 8, dtype=torch.uint8, pin_memory=True)
    h_recs = torch.empty(REC_CAP * binding.RECORD_DTYPE.itemsize, dtype=torch.uint8, pin_memory=True)
    n_rec = [0]

    def e2e_compact():
        p2 = Plan(cfg)
        r = p2.search_host_compact(K_TOP, S_MAX, K_SIM, JITTER_SEED, ws_c, REC_CAP, h_mask=h_mask, h_records=h_recs,
                                   stream=stream)
        n_rec[0] = r["n_records"]
        p2.close()

    def _wall(fn, reps):
        fn()
        barrier()
        t0 = time.perf_counter()
        for _ in range(reps):
            fn()
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        te = torch.tensor([dt], dtype=torch.float64, device=dev)
        if dist is not None:
            dist.all_reduce(te, op=dist.ReduceOp.MAX)
        return float(te.item()) / reps

    e2e_steps = max(5, min(args.steps, 50))
    s_compact = _wall(e2e_compact, e2e_steps)
    d2h_compact = 16 * 8 + 8 + (N + 7) // 8 + n_rec[0] * binding.RECORD_DTYPE.itemsize + K_TOP * 12 + 4 + K_SIM * 12 + 4 + 8
    del ws_c
    e2e = {"value": world * N / s_compact, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h_compact,
           "steps": e2e_steps, "ms_per_step": s_compact * 1e3,
           "mode": "pf_plan_create + pf_search_host_compact + pf_plan_destroy per step: reason histogram, feasibility "
                   "bits (a copy of zeros to the whole pinned mask beside the search + device writes of the 2 KB "
                   "stretches that hold feasible plans), records of every feasible plan, both top-k lists"}
    if not args.no_dense_e2e:
        h_reason = torch.empty(N, dtype=torch.uint8, pin_memory=True)
        h_tput = torch.empty(N, dtype=torch.float32, pin_memory=True)
        h_mem = torch.empty(N, dtype=torch.int64, pin_memory=True)
        ws_search = torch.empty(plan.search_workspace(K_TOP, S_MAX, K_SIM), dtype=torch.uint8, device=dev)

        def e2e_dense():
            p2 = Plan(cfg)
            p2.search_host(K_TOP, S_MAX, K_SIM, JITTER_SEED, ws_search, h_reason=h_reason, h_tput=h_tput, h_mem=h_mem,
                           stream=stream)
            p2.close()
        s_dense = _wall(e2e_dense, 3)
        e2e["dense"] = {"value": world * N / s_dense, "unit": UNIT, "ms_per_step": s_dense * 1e3, "steps": 3,
                        "d2h_bytes_per_step": N * BYTES_PER_CANDIDATE + K_TOP * 12 + 4 + K_SIM * 12 + 4 + 8,
                        "mode": "pf_search_host with every dense array copied back (PCIe-bound)"}
        del ws_search, h_reason, h_tput, h_mem

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel: the kernel that streams the constant blocks of the dense outputs
    hbm, how = _measured_hbm()
    cls_ms = {c: per_class[c][0] / args.steps for c in per_class if per_class[c][1]}
    dom = max(cls_ms, key=lambda c: cls_ms[c])
    span = plan.fill_span()
    fill_cands = (span["n_blocks"] - span["scored_blocks"]) * span["block_candidates"]
    # the fill kernel runs once per step, from right behind the scoring kernel to the end of the call
    fill_ms = cls_ms.get("fill", 0.0)
    if fill_timed[1]:                        # the live figure: the launches timed inside the timed region
        fill_ms = fill_timed[0] / fill_timed[1]
        cls_ms["fill"] = fill_ms
    if fill_ms > 0:
        kernel, k_ms, k_bytes = "fill_tail_kernel", fill_ms, BYTES_PER_CANDIDATE * fill_cands
    else:                                    # no separate fill kernel ran: the scoring kernel wrote everything
        kernel, k_ms, k_bytes = "score_kernel", cls_ms["score"], BYTES_PER_CANDIDATE * N
    achieved = k_bytes / (k_ms * 1e-3) / 1e9
    traffic = None
    if FILL_KERNEL_SLICE_DRAM_BYTES and kernel == "fill_tail_kernel":
        residue = BYTES_PER_CANDIDATE * FILL_KERNEL_SLICE_CANDIDATES - FILL_KERNEL_SLICE_DRAM_BYTES
        traffic = int(k_bytes - residue)
    roofline = {"kernel": kernel, "bound": "hbm", "achieved": achieved, "peak": hbm, "unit": "GB/s",
                "frac": achieved / hbm, "traffic": traffic, "peak_source": how,
                "algorithmic_bytes_per_launch": k_bytes, "ms_per_launch": k_ms,
                "frac_of_nominal_hbm": achieved / NOMINAL_HBM_GBS,
                "dominant_class": dom, "class_ms_per_step": cls_ms,
                "class_ms_source": "fill: the library's event pair around every eighth launch inside the timed region; the other classes: a pass of "
                                   "the same number of steps right after it with every class timed (events between the "
                                   "kernels of the caller's stream cost that chain its overlapped launches, so the "
                                   "timed region has none)",
                "launch_split": {"blocks": span["n_blocks"], "candidates_per_block": span["block_candidates"],
                                 "scoring_kernel_blocks": span["scored_blocks"], "fill_kernel_candidates": fill_cands,
                                 "fill_kernel_blocks": span["filled_blocks"]},
                "whole_step": {"bytes": BYTES_PER_CANDIDATE * N, "ms": ms_step,
                               "achieved": BYTES_PER_CANDIDATE * N / (ms_step * 1e-3) / 1e9,
                               "frac": BYTES_PER_CANDIDATE * N / (ms_step * 1e-3) / 1e9 / hbm},
                "note": "the fill kernel (bulk copies from shared memory, one 128-thread block per SM) runs on a stream "
                        "of its own beside everything else in the call, from right behind the scoring kernel to the "
                        "end: it shares the memory system with the kernels it runs beside and is what the step waits "
                        "for last; classes on different streams overlap, so class times add up to more than the step"}

    # ---- side measurements (single-GPU runs): probes, top-k-only mode, simulator figures, the other configs
    extra = {}
    if world == 1 and not args.no_report:
        from paper_2607_18631_b200 import probes
        ws_score = torch.empty(plan.score_workspace(N, K_TOP), dtype=torch.uint8, device=dev)
        ms_topk_only = _time_launches(
            torch, stream, lambda: plan.score(0, N, K_TOP, topk_idx=bufs["topk_idx"], topk_score=bufs["topk_score"],
                                              topk_count=bufs["topk_count"], workspace=ws_score, stream=stream,
                                              dense=False), reps=10, warm=3)
        extra["topk_only"] = {"ms_per_launch": ms_topk_only, "value": N / (ms_topk_only * 1e-3), "unit": UNIT,
                              "note": "dense outputs not written (NULL): rules + cost + top-1024 only"}
        peaks, write_gbs = _probe_peaks(torch, probes, stream, bufs["mem"])
        step()                                   # the write probe overwrote `mem`: restore the step's outputs
        torch.cuda.synchronize()
        roofline["write_ceiling_gbs"] = write_gbs
        roofline["frac_of_write_ceiling"] = achieved / write_gbs
        n_feas = int(((bufs["reason"] & 0x7F) == 0).sum().item())
        sim_ms = cls_ms["simulate"]
        sim_ops, chain = _survivor_shapes(plan, cfg, bufs["surv_idx"][:n_surv].cpu().numpy())
        extra["simulator"] = {
            "kernel": "simulate_kernel", "bound": "alu", "survivors": n_surv, "ms_per_launch": sim_ms,
            "prepass_ms": cls_ms.get("simprep", 0.0), "survivors_per_s": n_surv / (sim_ms * 1e-3),
            "simulated_ops": sim_ops, "simulated_ops_per_s": sim_ops / (sim_ms * 1e-3),
            "thread_instructions_per_op": SIM_INSTR_PER_OP,
            "achieved": SIM_INSTR_PER_OP * sim_ops / (sim_ms * 1e-3), "peak": peaks["logic"],
            "unit": "thread-instructions/s", "frac": SIM_INSTR_PER_OP * sim_ops / (sim_ms * 1e-3) / peaks["logic"],
            "longest_chain_steps": chain, "ns_per_chain_step": sim_ms * 1e6 / chain,
            "note": "a dependency-bound event simulation: the kernel cannot end before the longest per-rank op chain "
                    "has been walked (one shared-memory round trip per step), which is what ns_per_chain_step measures; "
                    "the ALU fraction is the algorithmic instructions against the measured issue rate"}
        extra["probes"] = {"thread_inst_per_s": peaks, "stream_write_gbs": write_gbs, "feasible": n_feas,
                           "feasible_fraction": n_feas / N}
        del ws_score
        if not args.no_configs:
            rig.close()
            torch.cuda.empty_cache()
            extra["configs"] = _config_lines(torch, stream, hbm, peaks)

    # ---- the oracle on the host cores (rank 0, single-GPU runs only)
    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        import oracle
        oracle.build()
        orc = oracle.Oracle(make_config("large"))
        threads = os.cpu_count() or 1
        used = orc.score_range(0, 1024, threads=threads)[3]
        t0 = time.perf_counter()
        scored = oracle_step(orc, threads, 1)
        dt = time.perf_counter() - t0
        t1 = time.perf_counter()
        orc.score_range(60_000_000, 2_457_600, threads=1)
        single = 2_457_600 / (time.perf_counter() - t1)
        cpu_baseline = {"value": scored / dt, "unit": UNIT, "cores": used, "kind": "oracle",
                        "sample": f"one whole step (all {scored:,} candidates + {n_surv:,} simulated survivors), "
                                  f"{dt:.1f} s",
                        "single_thread_value": single,
                        "single_thread_sample": "scoring only, candidates [60,000,000, 62,457,600)"}
        if "probes" in extra:
            # what evaluating every candidate on its own would cost in ALU time (the oracle's tally over the whole
            # space): the bound a kernel WITHOUT per-block hoisting of the rules would face, next to the HBM bound
            ops = oracle.count_ops(orc, 0, N, threads=threads)
            pk = extra["probes"]["thread_inst_per_s"]
            i_per, f_per = ops["int_ops"] / ops["candidates"], ops["fp_ops"] / ops["candidates"]
            t_alu = N * (i_per / min(pk["imad"], pk["logic"]) + f_per / pk["ffma"])
            t_hbm = N * BYTES_PER_CANDIDATE / (hbm * 1e9)
            extra["per_candidate_bounds"] = {
                "int_ops_per_candidate": i_per, "fp_ops_per_candidate": f_per,
                "ops_source": "oracle operation tally, every candidate of the space",
                "t_alu_ms": t_alu * 1e3, "t_hbm_ms": t_hbm * 1e3, "bound": "hbm" if t_hbm >= t_alu else "alu",
                "note": "t_alu is what one-thread-per-candidate evaluation would need; the kernels decide whole "
                        "blocks of candidates from their outer axes and never do most of that work"}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": workload_config(world, N),
            "survivors": n_surv,
            "l2": "no flush: each step rewrites 2.34 GB of dense outputs, far beyond the 126 MB L2",
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
            "cpu_baseline": cpu_baseline}
    if sustained is not None:
        line["sustained"] = sustained
    line.update(extra)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=("ours", "reference"), default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing leg")
    ap.add_argument("--no-report", action="store_true", help="skip the side measurements (probes, top-k-only)")
    ap.add_argument("--no-configs", action="store_true", help="skip the per-config lines")
    ap.add_argument("--no-sustained", action="store_true", help="skip the two-second sustained region")
    ap.add_argument("--no-dense-e2e", action="store_true", help="skip the dense-output end-to-end leg")
    ap.add_argument("--split", action="store_true",
                    help="one space split over the ranks (strong scaling) instead of one space per rank")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
