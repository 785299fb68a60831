"""Host logic of the multi-GPU path with two gloo ranks on CPU: slice arithmetic, list exchange, fold.
The per-slice scoring and the merge step are stood in for by the oracle (no GPU here); on a GPU the same
functions run with pf_score and pf_topk_merge."""
from __future__ import annotations

import os
import socket

import numpy as np
import pytest

from paper_2607_18631_b200.sharding import shard_range


def test_shard_range_covers_the_space_exactly():
    for n in (0, 1, 7, 432, 110_592, 179_908_608):
        for world in (1, 2, 3, 8):
            spans = [shard_range(n, r, world) for r in range(world)]
            assert spans[0][0] == 0
            for (f0, c0), (f1, _) in zip(spans[:-1], spans[1:]):
                assert f0 + c0 == f1
            assert spans[-1][0] + spans[-1][1] == n
            counts = [c for _, c in spans]
            assert max(counts) - min(counts) <= 1
    with pytest.raises(ValueError):
        shard_range(10, 2, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, k, ret):
    import torch
    import torch.distributed as dist
    from oracle import Oracle
    from paper_2607_18631_b200.sharding import gather_and_merge, shard_range
    from helpers import variant
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15))
        orc = Oracle(cfg)
        first, count = shard_range(orc.size, rank, world)
        reason, tput, _, _ = orc.score_range(first, count)
        li, ls = orc.topk(reason, tput, first, k)
        idx = torch.full((k,), -1, dtype=torch.int64)
        sc = torch.zeros(k, dtype=torch.float32)
        idx[:len(li)] = torch.from_numpy(li.astype(np.int64))
        sc[:len(ls)] = torch.from_numpy(ls.astype(np.float32))
        cnt = torch.tensor([len(li)], dtype=torch.int32)

        def merge(k_, a, b):   # stand-in for pf_topk_merge with the same contract
            na, nb = int(a[2]), int(b[2])
            ii = np.concatenate([a[0][:na].numpy(), b[0][:nb].numpy()]).astype(np.uint64)
            ss = np.concatenate([a[1][:na].numpy(), b[1][:nb].numpy()]).astype(np.float64)
            oi, os_ = Oracle.topk_list(ii, ss, k_)
            ri = torch.full((k_,), -1, dtype=torch.int64)
            rs = torch.zeros(k_, dtype=torch.float32)
            ri[:len(oi)] = torch.from_numpy(oi.astype(np.int64))
            rs[:len(os_)] = torch.from_numpy(os_.astype(np.float32))
            return ri, rs, torch.tensor([len(oi)], dtype=torch.int32)

        gi, gs, gc = gather_and_merge(idx, sc, cnt, k, merge=merge)
        ret[rank] = (gi.numpy().copy(), gs.numpy().copy(), int(gc))
    finally:
        dist.destroy_process_group()


def test_two_rank_gather_and_merge_equals_global_topk():
    import torch.multiprocessing as mp
    from oracle import Oracle
    from helpers import variant
    world, k = 2, 64
    port = _free_port()
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(world, port, k, ret), nprocs=world, join=True)
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15))
    orc = Oracle(cfg)
    reason, tput, _, _ = orc.score_range()
    want_idx, want_sc = orc.topk(reason, tput, 0, k)
    assert len(ret) == world
    for r in range(world):
        gi, gs, gc = ret[r]
        assert gc == len(want_idx)
        np.testing.assert_array_equal(gi[:gc].astype(np.uint64), want_idx)
        np.testing.assert_allclose(gs[:gc], want_sc, rtol=1e-6)


# ----------------------------------------------------------------------------- the whole search, split

def _search_cfg(ties: bool):
    from helpers import variant
    cfg = variant("mid", cluster=dict(budget_bytes=10 ** 15), rules=dict(enforce_realizability=0))
    if ties:
        for kv in (1, 2, 3):          # four identical kernel variants: every score appears four times
            cfg["kern"][kv] = dict(cfg["kern"][0])
    return cfg


def _search_worker(rank, world, port, k, s_max, k_sim, ties, ret):
    import torch.distributed as dist
    from oracle import Oracle
    from paper_2607_18631_b200.sharding import sharded_search
    from sharded_common import OracleOps
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        r = sharded_search(OracleOps(Oracle(_search_cfg(ties))), k, s_max, k_sim, 4)
        n = int(r["surv"][1].item())
        ret[rank] = dict(first=r["local"]["first"], count=r["local"]["count"],
                         topk=tuple(t.numpy().copy() for t in r["topk"]),
                         surv=r["surv"][0][:n].numpy().copy(), total=r["n_survivors_total"],
                         sim_topk=tuple(t.numpy().copy() for t in r["sim_topk"]))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("s_max,ties", [(10 ** 6, False), (700, False), (501, True), (1, True)])
def test_two_rank_sharded_search_equals_the_unsplit_search(s_max, ties):
    """sharded_search itself on two gloo ranks (the oracle doing each rank's share of the work): the folded top-k,
    the concatenated survivor lists and the folded simulator top-k are those of the unsplit space -- with a cut that
    falls inside a run of equal scores spread over both ranks."""
    import torch.multiprocessing as mp
    from oracle import Oracle
    world, k, k_sim = 2, 64, 50
    port = _free_port()
    ret = mp.Manager().dict()
    mp.spawn(_search_worker, args=(world, port, k, s_max, k_sim, ties, ret), nprocs=world, join=True)
    orc = Oracle(_search_cfg(ties))
    reason, tput, _, _ = orc.score_range(threads=4)
    tput32 = tput.astype(np.float32).astype(np.float64)       # the ranks rank fp32 scores, like the device
    want_idx, want_sc = orc.topk(reason, tput32, 0, k)
    want_surv = orc.select_survivors(reason, tput32, 0, s_max)
    sim, _, _ = orc.simulate_list(want_surv, 4, threads=4)
    want_sim_idx, want_sim_sc = Oracle.topk_list(want_surv, sim, k_sim)
    got_surv = np.concatenate([ret[r]["surv"] for r in range(world)]).astype(np.uint64)
    np.testing.assert_array_equal(got_surv, want_surv)
    for r in range(world):
        assert ret[r]["total"] == len(want_surv)
        gi, gs, gc = ret[r]["topk"]
        np.testing.assert_array_equal(gi[:int(gc[0])].astype(np.uint64), want_idx)
        si, ss, sc = ret[r]["sim_topk"]
        n = int(sc[0])
        assert n == len(want_sim_idx)
        np.testing.assert_array_equal(si[:n].astype(np.uint64), want_sim_idx)
        np.testing.assert_allclose(ss[:n], want_sim_sc, rtol=1e-6)
    if ties and s_max > 1:
        # the cut did fall inside a run of equal scores
        cut_score = tput32[want_surv.astype(np.int64)].min()
        assert (tput32[(reason & 0x7F) == 0] == cut_score).sum() > (tput32[want_surv.astype(np.int64)] == cut_score).sum()
