"""Pins of the two-stream layer timeline of the simulator tier (Sec. 3.2: a list-scheduling timeline that models
the overlap of compute and communication explicitly and derives the hidden fraction of communication).

The oracle runs a generic list scheduler over the layer's op DAG.  Here it is held to an independent event-driven
simulation written differently (discrete event queue), to closed forms of the regimes where one stream dominates,
and to the no-overlap sum."""
from __future__ import annotations

import heapq
import itertools

import numpy as np
import pytest

import oracle
from oracle import Oracle

from helpers import axis_index, variant


def event_sim(A, e_tot, d_tot, c_tot, n):
    """Independent restatement: two servers, FIFO by ready time (ties by op number), driven by an event heap."""
    e, d, c = e_tot / n, d_tot / n, c_tot / n
    dur = [A] + [d] * n + [e] * n + [c] * n
    stream = [0] + [1] * n + [0] * n + [1] * n
    deps = [[]] + [[0]] * n + [[1 + i] + ([n + i] if i else []) for i in range(n)] + [[n + 1 + i] for i in range(n)]
    n_ops = len(dur)
    end = [None] * n_ops
    ready_q = {0: [], 1: []}            # per stream: heap of (ready time, op)
    waiting = set(range(n_ops))
    busy_until = {0: 0.0, 1: 0.0}
    running = {}
    events = []                         # (time, op) completions
    now = 0.0

    def release():
        for i in sorted(waiting):
            if all(end[j] is not None for j in deps[i]):
                heapq.heappush(ready_q[stream[i]], (max([end[j] for j in deps[i]], default=0.0), i))
                waiting.discard(i)

    def start():
        for s in (0, 1):
            if s not in running and ready_q[s]:
                rt, i = heapq.heappop(ready_q[s])
                t0 = max(now, rt, busy_until[s])
                running[s] = i
                heapq.heappush(events, (t0 + dur[i], i))

    release()
    start()
    while events:
        now, i = heapq.heappop(events)
        end[i] = now
        busy_until[stream[i]] = now
        del running[stream[i]]
        release()
        start()
    return max(end)


@pytest.mark.parametrize("n", [1, 2, 3, 4, 8, 16])
def test_list_scheduler_matches_an_independent_event_simulation(n):
    rng = np.random.default_rng(100 + n)
    for _ in range(200):
        A, e, d, c = (float(x) for x in rng.uniform(0.01, 3.0, size=4) * rng.choice([0.1, 1.0, 10.0], size=4))
        got = oracle.two_stream_layer(A, e, d, c, n)
        want = event_sim(A, e, d, c, n)
        assert abs(got - want) <= 1e-12 * want, (A, e, d, c, n, got, want)


def test_one_chunk_is_the_plain_sum_and_closed_forms_of_the_dominated_regimes():
    # no chunking: dispatch, experts, combine strictly one after the other
    assert oracle.two_stream_layer(0.7, 1.1, 0.4, 0.3, 1) == pytest.approx(0.7 + 0.4 + 1.1 + 0.3, rel=1e-15)
    for n in (2, 4, 8):
        # compute-bound: every chunk of experts takes longer than a chunk of either transfer, so only the first
        # dispatch chunk and the last combine chunk are exposed: hidden fraction (n-1)/n
        A, e, d, c = 0.5, 8.0, 2.0, 1.0
        assert oracle.two_stream_layer(A, e, d, c, n) == pytest.approx(A + d / n + e + c / n, rel=1e-14)
        # transfer-bound (a dispatch chunk outlasts an expert chunk): the communication stream runs all dispatches,
        # then all combines without a gap -- unless the last combine chunk has to wait for the last expert chunk
        A, e, d, c = 0.5, 0.8, 8.0, 4.0
        want = max(A + d + c, A + d + e / n + c / n)
        assert oracle.two_stream_layer(A, e, d, c, n) == pytest.approx(want, rel=1e-14)
    # more chunks never hurt, and the layer is never faster than either stream's own work
    for A, e, d, c in itertools.product((0.2, 1.0), (0.5, 4.0), (0.3, 2.0), (0.3, 2.0)):
        spans = [oracle.two_stream_layer(A, e, d, c, n) for n in (1, 2, 4, 8, 16)]
        assert all(b <= a * (1 + 1e-12) for a, b in zip(spans, spans[1:]))
        assert spans[-1] >= max(A + e, A + d + c) * (1 - 1e-12)


def _two_stream_cfg(n_chunks, sm_frac, hide=None):
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15), rules=dict(enforce_realizability=0))
    for s in cfg["sched"]:
        if s["overlap"]:
            s["n_chunks"] = n_chunks
            s["sm_frac"] = float(np.float32(sm_frac))
            if hide is not None:
                s["hide_frac"] = float(np.float32(hide))
    return cfg


def test_simulator_uses_the_timeline_only_where_the_schedule_asks_for_it():
    """n_chunks = 0 keeps the alpha-table in the simulator (scores identical to a table without the new
    fields); schedules without overlap are never touched; the analytic tier ignores the chunking."""
    base = variant("mid", cluster=dict(budget_bytes=10 ** 15), rules=dict(enforce_realizability=0))
    zero, four = _two_stream_cfg(0, 0.0), _two_stream_cfg(4, 0.1)
    ob, oz, o4 = Oracle(base), Oracle(zero), Oracle(four)
    r, t, _, _ = ob.score_range()
    idx = np.flatnonzero((r & 0x7F) == 0).astype(np.uint64)[::7]
    sb, _, _ = ob.simulate_list(idx, 4, threads=8)
    sz, _, _ = oz.simulate_list(idx, 4, threads=8)
    assert np.array_equal(sb, sz)
    r4, t4, _, _ = o4.score_range()
    assert np.array_equal(r, r4) and np.array_equal(t, t4)          # the analytic scorer does not look at it
    s4, _, _ = o4.simulate_list(idx, 4, threads=8)
    ov = np.array([base["sched"][ob.eval(int(i))["sched"]]["overlap"] for i in idx]) == 1
    assert np.array_equal(s4[~ov], sb[~ov]) and np.any(s4[ov] != sb[ov])


def test_timeline_reduces_to_known_cases_inside_the_simulator():
    """pp = 1, one stage: the step is m (F + B) with F, B the stage times; with one chunk and no SM budget the
    timeline exposes the whole all-to-all, i.e. the simulator equals itself with hiding switched off; chunking
    then only helps."""
    idx_of = lambda cfg: axis_index(cfg, sched=1, pp=2, v=2, tp=1, dp=4, ep=4, mb=2, kv=0, rec=0)
    c1, c8 = _two_stream_cfg(1, 0.0), _two_stream_cfg(8, 0.0)
    nohide = _two_stream_cfg(0, 0.0, hide=0.0)
    i = idx_of(c1)
    assert (Oracle(c1).eval(i)["reason"] & 0x7F) == 0 and Oracle(c1).eval(i)["ov"] == 1
    st1, t1, _ = Oracle(c1).simulate(i, 4)
    st0, t0, _ = Oracle(nohide).simulate(i, 4)
    st8, t8, _ = Oracle(c8).simulate(i, 4)
    assert st1 == st0 == st8 == 0
    assert t1 == pytest.approx(t0, rel=1e-12)
    assert t8 > t1
    # an SM budget slows compute: with one chunk there is nothing to gain from it
    st, ts, _ = Oracle(_two_stream_cfg(1, 0.25)).simulate(i, 4)
    assert ts < t1
