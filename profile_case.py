"""A small, fixed workload for profiler captures (ncu): a cut of the large training space.

  python profile_case.py [--launches 3] [--stage search|score|select|simulate] [--config large] [--lift-gate]
                         [--topk-only]

The cut keeps every axis of the benchmark's large space but three of its eleven expert-parallel degrees
(49,065,984 candidates): 638 MB of dense outputs per call, larger than the 126 MB L2 but well under a few GB on the
device, so that a multi-pass capture of one launch ends by itself quickly.  `search` runs the one-call search (the
benchmark's step: scoring kernel, selection, simulator kernel and re-rank beside the fill kernel); the other stages run
the separate entry points.
"""
from __future__ import annotations

import argparse
import os
import sys

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def slice_config(name: str = "large") -> dict:
    from workloads import make_config
    cfg = make_config(name)
    axes = dict(cfg["axes"])
    cfg["axes"] = [(n, ([8, 64, 256] if n == "ep" else v)) for n, v in cfg["axes"]]
    assert len(axes["ep"]) == 11
    return cfg


def main():
    import torch

    from paper_2607_18631_b200 import Plan

    ap = argparse.ArgumentParser()
    ap.add_argument("--launches", type=int, default=3)
    ap.add_argument("--stage", default="search", choices=("search", "score", "select", "simulate"))
    ap.add_argument("--config", default="large")
    ap.add_argument("--lift-gate", action="store_true",
                    help="raise the memory budget so that no plan is rejected by the gate (with --config "
                         "large_unconstrained: every plan that passes the integer rules goes through the cost model)")
    ap.add_argument("--topk-only", action="store_true", help="stage score: no dense outputs, top-k only")
    args = ap.parse_args()

    cfg = slice_config(args.config)
    if args.lift_gate:
        cfg["cluster"]["budget_bytes"] = 10 ** 15
    plan = Plan(cfg)
    bufs = out = sel = None
    for _ in range(args.launches):
        if args.stage == "search":
            bufs = plan.search(1024, 1_000_000, 100, 4, bufs=bufs)
            continue
        out = plan.score(k=1024, dense=not args.topk_only)
        if args.stage in ("select", "simulate"):
            sel = plan.select_survivors(out["reason"], out["tput"], 1_000_000)
        if args.stage == "simulate":
            plan.simulate(sel["surv_idx"], 1_000_000, 4, k=100, d_n=sel["surv_count"], dense=False)
    torch.cuda.synchronize()
    if args.stage == "search":
        span = plan.fill_span()
        fill = (span["n_blocks"] - span["scored_blocks"]) * span["block_candidates"]
        print(f"searched {plan.size} candidates; {int(bufs['surv_count'].item())} survivors; the fill kernel covers "
              f"{fill} candidates ({span['filled_blocks']} of {span['n_blocks']} blocks)")
    else:
        print(f"scored {plan.size} candidates; top-k holds {int(out['topk_count'].item())}"
              + (f"; {int(sel['surv_count'].item())} survivors" if sel is not None else ""))
    plan.close()


if __name__ == "__main__":
    main()
