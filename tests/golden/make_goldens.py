"""Regenerates the two golden files that no printed number backs:

  large_space_rule_counts.txt     first-failing-rule histogram (rules 1-7) of the large training space
  dualpipe_style_makespans.txt    makespans of the DualPipe-style order for uniform stage durations

from implementations written for this purpose only: vectorised numpy predicates for the rules, and a pure-Python
event simulation for the schedule.  Nothing here imports `oracle/` or the CUDA package, so the files cross-check two
separate readings of the same definitions.  The comment header of each file is kept; only the value lines are made.

    python tests/golden/make_goldens.py            # rewrite both files
    python tests/golden/make_goldens.py --check    # compare with the stored files, exit 1 on a difference
"""
from __future__ import annotations

import argparse
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))

# --------------------------------------------------------------------------- rules 1-7 on the large space

# The large space as the benchmark defines it: 61 layers, 128 heads, 256 experts, shared and expert FFN width 2048,
# 8 GPUs per node, plans of 16..1024 GPUs, 15,360 sequences per step, experts may span dp x tp, uneven layer split.
LARGE = dict(L=61, nh=128, E=256, Fs=2048, G=8, world_min=16, world_max=1024, gbs=15360, tp_max=8)
# schedule classes of the four schedule entries: 1F1B, 1F1B + overlap, interleaved + overlap, DualPipe-style
KINDS = np.array([0, 0, 1, 2])


def large_space_rule_counts() -> dict:
    """One pass over (dp, tp, pp, ep, v, mb, schedule) with boolean masks; a candidate is charged to the first rule it
    breaks, in the predicate's order."""
    p2 = 2 ** np.arange(11)
    dp, tp, pp, ep, v, mb, s = np.meshgrid(p2, p2, p2, p2, np.arange(1, 9), np.arange(1, 17), np.arange(4),
                                           indexing="ij", sparse=True)
    c = LARGE
    shape = np.broadcast_shapes(dp.shape, tp.shape, pp.shape, ep.shape, v.shape, mb.shape, s.shape)
    kind = KINDS[s]
    world = tp * pp * dp
    fails = []
    fails.append((world < c["world_min"]) | (world > c["world_max"]) | ((world > c["G"]) & (world % c["G"] != 0)))
    fails.append((tp > c["tp_max"]) | (tp > c["G"]) | (c["nh"] % tp != 0) | (c["Fs"] % tp != 0))
    fails.append((c["E"] % ep != 0) | ((dp * tp) % ep != 0))
    fails.append(c["gbs"] % (dp * mb) != 0)
    fails.append(np.where(kind == 1, (v < 2) | (pp < 2), v != 1))
    fails.append(pp * v > c["L"])
    m = c["gbs"] // np.maximum(dp * mb, 1)
    fails.append(np.where(kind == 1, m % pp != 0, np.where(kind == 2, (m % 2 != 0) | ((pp > 1) & (pp % 2 != 0)), False)))
    alive = np.ones(shape, dtype=bool)
    names = ["WORLD", "TP", "EP", "BATCH", "VSTAGE", "LAYERS", "MICROBATCH"]
    out = {}
    for name, f in zip(names, fails):
        hit = alive & np.broadcast_to(f, shape)
        out[name] = int(hit.sum())
        alive &= ~hit
    out["PASS"] = int(alive.sum())
    return out


# --------------------------------------------------------------------------- DualPipe-style order and its makespan

def dualpipe_style_order(pp: int, m: int):
    """Per-rank op sequences from the nominal schedule: forward 1 tick, backward 2 ticks, free hand-overs; two
    directions with m/2 microbatches each; direction 0 puts position q on rank q, direction 1 on rank pp-1-q.  An idle
    rank starts the ready op with the smallest (ready time, backward first, microbatch, direction); a forward at
    position q waits while pp - q microbatches of its direction are in flight on the rank.  Ops are tuples
    (is_backward, direction, position, microbatch)."""
    n = m // 2
    done_at = {}                                   # op -> nominal completion tick
    seq = [[] for _ in range(pp)]
    idle_from = [0] * pp
    flying = [[0, 0] for _ in range(pp)]
    todo = {r: [(b, d, (r if d == 0 else pp - 1 - r), j) for d in (0, 1) for b in (0, 1) for j in range(n)]
            for r in range(pp)}
    clock, left = 0, 4 * n * pp
    while left:
        for r in range(pp):
            if idle_from[r] > clock:
                continue
            best = None
            for op in todo[r]:
                b, d, q, j = op
                needs = []
                if b == 0:
                    if q > 0:
                        needs.append((0, d, q - 1, j))
                    if flying[r][d] >= pp - q:
                        continue
                else:
                    needs.append((0, d, q, j))
                    if q < pp - 1:
                        needs.append((1, d, q + 1, j))
                if any(done_at.get(x, 1 << 30) > clock for x in needs):
                    continue
                ready = max([done_at[x] for x in needs], default=0)
                key = (ready, 1 - b, j, d)
                if best is None or key < best[0]:
                    best = (key, op)
            if best is None:
                continue
            op = best[1]
            b, d, q, j = op
            todo[r].remove(op)
            done_at[op] = idle_from[r] = clock + (2 if b else 1)
            flying[r][d] += -1 if b else 1
            seq[r].append(op)
            left -= 1
        later = [t for t in idle_from if t > clock]
        if not later:
            raise RuntimeError("the nominal schedule stalled")
        clock = min(later)
    return seq


def makespan(seq, pp: int, F: int, B: int) -> int:
    """Run the fixed per-rank sequences with durations F / B and free hand-overs; an op starts when its rank is free
    and its predecessors are done."""
    end, at, free = {}, [0] * pp, [0] * pp
    total = sum(len(s) for s in seq)
    while total:
        moved = False
        for r in range(pp):
            while at[r] < len(seq[r]):
                b, d, q, j = seq[r][at[r]]
                needs = [(0, d, q - 1, j)] if (b == 0 and q > 0) else []
                if b == 1:
                    needs = [(0, d, q, j)] + ([(1, d, q + 1, j)] if q < pp - 1 else [])
                if any(x not in end for x in needs):
                    break
                start = max([free[r]] + [end[x] for x in needs])
                end[(b, d, q, j)] = free[r] = start + (B if b else F)
                at[r] += 1
                total -= 1
                moved = True
        if not moved:
            raise RuntimeError("the order deadlocked")
    return max(end.values())


DUALPIPE_CASES = [(1, 2, pp, m) for pp in (4, 8, 16) for m in (8, 16, 32, 64)] + \
                 [(1, 1, 4, 16), (1, 1, 8, 16), (1, 1, 16, 16), (1, 1, 16, 64),
                  (1, 3, 4, 16), (1, 3, 8, 64), (1, 3, 16, 64)]


def dualpipe_rows():
    orders = {}
    rows = []
    for F, B, pp, m in DUALPIPE_CASES:
        if (pp, m) not in orders:
            orders[(pp, m)] = dualpipe_style_order(pp, m)
        rows.append((F, B, pp, m, makespan(orders[(pp, m)], pp, F, B)))
    return rows


# --------------------------------------------------------------------------- files

def _header(path):
    with open(path) as f:
        return [ln for ln in f if ln.startswith("#")]


def _values(path):
    with open(path) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--check", action="store_true")
    args = ap.parse_args()
    counts = large_space_rule_counts()
    files = {
        "large_space_rule_counts.txt": [[k, str(v)] for k, v in counts.items()],
        "dualpipe_style_makespans.txt": [[str(x) for x in row] for row in dualpipe_rows()],
    }
    bad = 0
    for name, rows in files.items():
        path = os.path.join(HERE, name)
        if args.check:
            same = sorted(_values(path)) == sorted(rows)
            print(f"{name}: {'same' if same else 'DIFFERENT'}")
            bad += not same
        else:
            head = _header(path)
            with open(path, "w") as f:
                f.writelines(head)
                f.writelines(" ".join(r) + "\n" for r in rows)
            print(f"wrote {path}")
    return 1 if bad else 0


if __name__ == "__main__":
    sys.exit(main())
