"""The N > 1 host logic on CPU: two gloo ranks split a candidate range, evaluate their slices
(with the CPU oracle standing in for the device) and merge their winners."""
import os
import socket

import numpy as np
import pytest

from paper_2306_08423_b200 import sharding
from paper_2306_08423_b200 import workloads as W


def test_shard_ranges_cover_exactly_once():
    for n in (0, 1, 7, 88, 1000, 38_838_764):
        for world in (1, 2, 3, 8):
            seen = 0
            sizes = []
            for r in range(world):
                first, count = sharding.shard_range(n, r, world)
                assert first == seen
                seen += count
                sizes.append(count)
            assert seen == n and max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.shard_range(10, 2, 2)
    assert sharding.rank_seed(1, 3) == 4


def _worker(rank, world, port, out):
    import torch.distributed as dist
    import oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = W.config0()
        n = oracle.count(w.table, w.space)
        first, count = sharding.shard_range(n, rank, world)
        batch, _ = oracle.eval_indices(w.table, w.space, np.arange(first, first + count))
        local_order = np.lexsort((np.arange(count), batch))
        k = int(local_order[0])
        best = sharding.merge_argmin(first + k, int(batch[k]))
        # the ranks' lists of their 10 fastest, gathered; their 10 smallest are the global 10 fastest
        import torch
        kk = 10
        lt = torch.from_numpy(batch[local_order[:kk]].copy())
        li = torch.from_numpy((first + local_order[:kk]).astype(np.int64))
        gt, gi = sharding.gather_topk_lists(lt, li)
        sel = np.lexsort((gi.numpy(), gt.numpy()))[:kk]
        merged = (gi.numpy()[sel].tolist(), gt.numpy()[sel].tolist())
        slowest = sharding.max_over_ranks(float(rank + 1))
        empty = sharding.merge_argmin(-1 if rank else 5, 0 if rank else 42)   # one rank has nothing
        out.put((rank, best, slowest, empty, merged))
    finally:
        dist.destroy_process_group()


def test_two_ranks_merge_their_winners():
    import torch.multiprocessing as mp
    import oracle
    oracle.build()
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    results = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    w = W.config0()
    batch, _ = oracle.eval_indices(w.table, w.space, np.arange(88))
    want = int(np.lexsort((np.arange(88), batch))[0])
    order = np.lexsort((np.arange(88), batch))[:10]
    for rank, best, slowest, empty, merged in results:
        assert merged == (order.tolist(), batch[order].tolist())
        assert best == (want, int(batch[want]))
        assert slowest == 2.0
        assert empty == (5, 42)
