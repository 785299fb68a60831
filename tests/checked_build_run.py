"""Runs the scoring path in the CHECKED build of the library (every device-side index range-checked, violations
recorded instead of trapping) over the small spaces, a set of randomized spaces and the deep-pipeline simulator
cases, and prints one line per case: `<case> status=<pf_check_read status> record=<six words>`.  Started by
tests/test_gpu_bounds_check.py in a process of its own with PLANFRONT_LIB pointing at libplanfront_check.so."""
from __future__ import annotations

import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))


def main():
    import torch
    from paper_2607_18631_b200 import Plan
    from workloads import make_config
    from helpers import axis_index, variant
    from test_gpu_fuzz import random_space

    def report(name, plan):
        torch.cuda.synchronize()
        st, rec = plan.check_read()
        print(f"{name} status={st} record={' '.join(str(int(x)) for x in rec)}", flush=True)

    # the checks' own check first: a deliberately bad index must show up in the record (and be redirected)
    plan = Plan(make_config("tiny"))
    assert plan.check_selftest() == 0
    report("selftest", plan)
    report("selftest_cleared", plan)
    plan.close()

    cases = [("tiny", make_config("tiny"), 16), ("mid", make_config("mid"), 128),
             ("mid_open", variant("mid", cluster=dict(budget_bytes=10 ** 15), rules=dict(enforce_realizability=0)), 128),
             ("serve", make_config("serve"), 128)]
    for seed in range(8):
        cases.append((f"fuzz{seed}", random_space(seed), 64))
    for name, cfg, k in cases:
        plan = Plan(cfg)
        out = plan.score(k=k)
        n = plan.size
        if n > 3000:                                   # a ragged, unaligned sub-range as well
            plan.score(first=1001, count=min(n - 1001, 70_003), k=k)
        if cfg["phase"] == 0:
            b = plan.search(k, 5000, 50, 4)
            sel = plan.select_survivors(out["reason"], out["tput"], 300)
            plan.simulate(sel["surv_idx"], 300, 4, k=20, d_n=sel["surv_count"])
            del b, sel
        else:
            plan.aggregate_serving(out["reason"], out["tput"], k=k)
        c = plan.compact(out["reason"], out["tput"], out["mem"], 1000)
        del c, out
        report(name, plan)
        plan.close()
    # deep pipelines, long windows, every schedule class
    cfg = variant("large_unconstrained", cluster=dict(budget_bytes=10 ** 15))
    for kn in cfg["kern"]:
        kn["avail_mask"] = 255
    picks = []
    for sched, v in ((0, 1), (1, 1), (2, 2), (2, 3), (2, 7), (2, 8), (3, 1)):
        for pp in (1, 2, 4, 8, 16, 32):
            for mb, dp in ((1, 8), (15, 64), (16, 32)):
                picks.append(axis_index(cfg, kv=1, rec=0, sched=sched, mb=mb, v=v, ep=8, pp=pp, tp=2, dp=dp))
    plan = Plan(cfg)
    idx = torch.from_numpy(np.unique(np.array(picks, dtype=np.int64))).cuda()
    plan.simulate(idx, idx.numel(), 4, k=64)
    report("deep_pipelines", plan)
    plan.close()
    # many blocks of odd size: the one-call search with the streaming kernel at work on the fill stream
    cfg = make_config("large")
    cut = {"kv": 7, "sched": 3, "mb": 15, "v": 7}
    cfg["axes"] = [(n, (list(v)[:cut[n]] if n in cut else v)) for n, v in cfg["axes"]]
    plan = Plan(cfg)
    b = plan.search(256, 10 ** 6, 50, 4)
    b = plan.search(256, 3000, 50, 4, bufs=b)
    report("odd_blocks_search", plan)
    plan.close()


if __name__ == "__main__":
    main()
