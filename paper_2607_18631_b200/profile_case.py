"""A small, fixed workload for profiler captures (ncu): a slice of the large training space.

  python -m paper_2607_18631_b200.profile_case [--count 50000000] [--launches 3] [--stage score|select|simulate|all]

The slice is larger than the 126 MB L2 (50M candidates write 650 MB of dense outputs) but holds well under a
few GB on the device, so a multi-pass capture of one launch ends by itself quickly.
"""
from __future__ import annotations

import argparse
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def main():
    import torch

    from paper_2607_18631_b200 import Plan
    from workloads import make_config

    ap = argparse.ArgumentParser()
    ap.add_argument("--count", type=int, default=50_000_000)
    ap.add_argument("--first", type=int, default=60_000_000)
    ap.add_argument("--launches", type=int, default=3)
    ap.add_argument("--stage", default="all", choices=("score", "select", "simulate", "all"))
    ap.add_argument("--config", default="large")
    args = ap.parse_args()

    plan = Plan(make_config(args.config))
    count = min(args.count, plan.size - args.first)
    out = sel = None
    for _ in range(args.launches):
        out = plan.score(first=args.first, count=count, k=1024)
        if args.stage in ("select", "simulate", "all"):
            sel = plan.select_survivors(out["reason"], out["tput"], 1_000_000, first=args.first)
        if args.stage in ("simulate", "all"):
            plan.simulate(sel["surv_idx"], 1_000_000, 4, k=100, d_n=sel["surv_count"], dense=False)
    torch.cuda.synchronize()
    n = int(out["topk_count"].item())
    print(f"scored {count} candidates from {args.first}; top-k holds {n}"
          + (f"; {int(sel['surv_count'].item())} survivors" if sel is not None else ""))
    plan.close()


if __name__ == "__main__":
    main()
