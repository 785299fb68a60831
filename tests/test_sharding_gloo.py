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
