"""Parity of the CUDA engine against the CPU oracle, through the C ABI.

Integer outputs (batch time, activity time, argmin, top-k, every emitted record and
offset) must be bit-exact; utilisation is fp64 within 1e-12 relative.
"""
import copy
import os

import numpy as np
import pytest

import oracle
from paper_2306_08423_b200 import workloads as W

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
THREADS = max(1, min(32, (os.cpu_count() or 2)))


@pytest.fixture(scope="module")
def E():
    from paper_2306_08423_b200 import engine
    return engine


@pytest.fixture()
def ctx(E):
    c = E.Context(0)
    yield c
    c.close()


def dev(n, dtype=torch.int64):
    return torch.empty(n, dtype=dtype, device="cuda")


def load(E, ctx, w):
    E.distsim_load_event_table(ctx, w.table)
    n = E.distsim_set_space(ctx, w.space)
    assert n == oracle.count(w.table, w.space)
    return n


def eval_all(E, ctx, n, busy=True):
    batch = dev(n)
    sb = dev(n * ctx.pp_max) if busy else None
    E.distsim_eval_strategies(ctx, 0, n, batch, sb)
    torch.cuda.synchronize()
    return batch, (sb.view(n, ctx.pp_max) if busy else None)


def stream_checksum(rec):
    """The order-sensitive checksum distsim_checksum_timelines defines, of one record list
    (int64 [r, 5]), restated with numpy."""
    with np.errstate(over="ignore"):
        wds = rec.reshape(-1).astype(np.uint64)
        z = wds + np.arange(1, wds.size + 1, dtype=np.uint64) * np.uint64(0x9E3779B97F4A7C15)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        z = z ^ (z >> np.uint64(31))
        return int(z.sum(dtype=np.uint64))


def device_checksums(E, ctx, records, offsets, n_lists):
    out = dev(max(1, n_lists))
    E.distsim_checksum_timelines(ctx, records, offsets, n_lists, out)
    torch.cuda.synchronize()
    return out.cpu().numpy()[:n_lists].view(np.uint64)


def check_emission(E, ctx, w, indices):
    """Emits the given candidates and compares every record with the oracle."""
    N = w.table.n_devices
    idx = torch.tensor(list(indices), dtype=torch.int64, device="cuda")
    n = len(indices)
    offsets, busy, util = dev(n * N + 1), dev(n * N), dev(n * N, torch.float64)
    total = E.distsim_emit_timelines(ctx, idx, n, None, 0, offsets, busy, util)
    records = dev(max(1, total) * 5)
    records.fill_(-7)
    total2 = E.distsim_emit_timelines(ctx, idx, n, records, total, offsets, busy, util)
    assert total2 == total
    torch.cuda.synchronize()
    rec = records.cpu().numpy()[: total * 5].reshape(total, 5)
    off = offsets.cpu().numpy(); bz = busy.cpu().numpy(); ut = util.cpu().numpy()
    assert off[0] == 0 and off[-1] == total
    # the call that never waits on the host, provisioned by the shape of the pass above: the same output
    shape = E.distsim_emit_shape_of_last_plan(ctx)
    assert shape.records == total
    records2, offsets2, busy2, util2 = dev(max(1, total) * 5), dev(n * N + 1), dev(n * N), dev(n * N, torch.float64)
    records2.fill_(-7)
    E.distsim_emit_timelines_async(ctx, idx, n, records2, total, shape, offsets2, busy2, util2)
    torch.cuda.synchronize()
    assert torch.equal(records2, records) and torch.equal(offsets2, offsets) and torch.equal(busy2, busy) and torch.equal(util2, util)
    sums = device_checksums(E, ctx, records, offsets, n * N)
    order = np.argsort(np.asarray(indices), kind="stable")
    cands = oracle.enumerate_at(w.table, w.space, np.asarray(indices)[order])
    for pos, c in zip(order, cands):
        r = oracle.simulate(w.table, c, replicate=True)
        base = off[pos * N]
        assert (off[pos * N: pos * N + N + 1] - base == r.offsets).all(), c
        got = rec[base: base + r.offsets[-1]]
        if not (got == r.records).all():
            bad = np.argwhere((got != r.records).any(axis=1))[0, 0]
            raise AssertionError(f"{c}: record {bad}: got {got[bad]}, want {r.records[bad]}")
        assert (bz[pos * N: pos * N + N] == r.busy_ns).all(), c
        np.testing.assert_allclose(ut[pos * N: pos * N + N], r.util, rtol=1e-12, atol=0)
        for k in (0, N // 2, N - 1):              # the stream checksum of some of its devices
            assert int(sums[pos * N + k]) == stream_checksum(r.records[r.offsets[k]:r.offsets[k + 1]]), (c, k)
    return total


def test_config0_everything(E, ctx):
    w = W.config0()
    n = load(E, ctx, w)
    assert n == 88
    batch, sb = eval_all(E, ctx, n)
    ob, obusy = oracle.eval_indices(w.table, w.space, np.arange(n), replicate=True, pp_stride=w.space.pp_max)
    assert (batch.cpu().numpy() == ob).all()
    assert (sb.cpu().numpy() == obusy).all()
    # host decode == oracle's loop enumeration
    for i, c in enumerate(oracle.enumerate_at(w.table, w.space, np.arange(n))):
        d = E.distsim_decode(ctx, i)
        assert (d["mp"], d["pp"], d["dp"], d["m"], d["sched"], d["bounds"]) == (c.mp, c.pp, c.dp, c.m, c.sched, c.bounds)
    bi, bt = E.distsim_argmin(ctx, batch, 0, n)
    order = np.lexsort((np.arange(n), ob))
    assert (bi, bt) == (order[0], ob[order[0]])
    ki, kt = dev(10), dev(10)
    E.distsim_topk(ctx, batch, 0, n, 10, ki, kt)
    assert (ki.cpu().numpy() == order[:10]).all() and (kt.cpu().numpy() == ob[order[:10]]).all()
    check_emission(E, ctx, w, list(range(n)))


@pytest.mark.parametrize("seed", range(8))
def test_random_small_full_parity(E, ctx, seed):
    kw = dict(dp_overlap=seed % 2, dp_bucket_bytes=0 if seed % 4 == 3 else 3000)
    if seed >= 4:
        kw.update(n_devices=16, gpus_per_node=2, n_layers=9, global_batch=24, mp_max=4, pp_max=8,
                  m_list=(1, 2, 3, 5, 6, 12), partition_mode=W.PARTITION_ALL)
    w = W.random_small(100 + seed, **kw)
    n = load(E, ctx, w)
    batch, sb = eval_all(E, ctx, n)
    ob, obusy = oracle.eval_indices_parallel(w.table, w.space, np.arange(n), THREADS, replicate=False,
                                             pp_stride=w.space.pp_max)
    gb = batch.cpu().numpy()
    assert (gb == ob).all(), np.argwhere(gb != ob)[:5]
    assert (sb.cpu().numpy() == obusy).all()
    bi, bt = E.distsim_argmin(ctx, batch, 0, n)
    order = np.lexsort((np.arange(n), ob))
    assert (bi, bt) == (order[0], ob[order[0]])
    k = min(n, 37)
    ki = dev(k)
    E.distsim_topk(ctx, batch, 0, n, k, ki)
    assert (ki.cpu().numpy() == order[:k]).all()
    rng = np.random.default_rng(seed)
    pick = rng.choice(n, size=min(n, 24), replace=False).tolist()
    check_emission(E, ctx, w, pick)


@pytest.mark.parametrize("sched_mask", [7, 4, 5, 6])
def test_asynchronous_1f1b_schedule(E, ctx, sched_mask):
    """Spaces with the asynchronous schedule (bit 2) alone and beside the others: every candidate
    of a small space (lock-step kernel), sampled candidates of a space with enough partitions for
    the one-partition-per-thread kernel, emitted timelines without gradient buckets."""
    w = W.random_small(300 + sched_mask, dp_overlap=sched_mask % 2, sched_mask=sched_mask)
    n = load(E, ctx, w)
    batch, sb = eval_all(E, ctx, n)
    ob, obusy = oracle.eval_indices_parallel(w.table, w.space, np.arange(n), THREADS, replicate=False,
                                             pp_stride=w.space.pp_max)
    assert (batch.cpu().numpy() == ob).all() and (sb.cpu().numpy() == obusy).all()
    cands = oracle.enumerate_at(w.table, w.space, np.arange(n))
    for i in range(0, n, max(1, n // 50)):
        assert E.distsim_decode(ctx, i)["sched"] == cands[i].sched
    pick = [i for i, c in enumerate(cands) if c.sched == 2 and c.dp > 1][:: max(1, n // 60)][:16]
    assert pick
    check_emission(E, ctx, w, pick + [0, n - 1])
    # 50 388 partitions at pp = 8: the thread kernel, 32-bit and relative-frame paths included
    w = W.random_small(310 + sched_mask, n_devices=16, gpus_per_node=4, n_layers=20, global_batch=64,
                       mp_max=2, pp_max=8, m_list=(1, 3, 8, 16, 32), sched_mask=sched_mask,
                       partition_mode=W.PARTITION_ALL)
    n = load(E, ctx, w)
    batch, sb = eval_all(E, ctx, n)
    rng = np.random.default_rng(sched_mask)
    idx = np.unique(np.concatenate([rng.integers(0, n, 3000), [0, n - 1]]))
    ob, obusy = oracle.eval_indices_parallel(w.table, w.space, idx, THREADS, replicate=False,
                                             pp_stride=w.space.pp_max)
    sel = torch.from_numpy(idx).cuda()
    assert (batch[sel].cpu().numpy() == ob).all()
    assert (sb[sel].cpu().numpy() == obusy).all()
    bi, bt = E.distsim_argmin(ctx, batch, 0, n)
    assert oracle.eval_indices(w.table, w.space, np.array([bi]))[0][0] == bt == int(batch.min().item())


@pytest.mark.parametrize("case", range(6))
def test_interleaved_1f1b_every_candidate(E, ctx, case):
    """Spaces with interleaved 1F1B candidates (sched_mask bit 3: v = 2, 4 chunks per device)
    beside the other schedules and alone, every composition into pp * v virtual stages or the
    balanced one, both gradient-overlap modes, one bucket or many: every candidate's batch time
    and per-device activity time, the decoded candidates, the best one and the k fastest."""
    mask = (15, 8, 11, 15, 9, 8)[case]
    kw = dict(n_devices=8, gpus_per_node=(4, 2, 4, 8, 4, 2)[case], n_layers=(9, 8, 10, 9, 12, 16)[case],
              global_batch=16, mp_max=2, pp_max=(4, 4, 4, 8, 4, 8)[case], m_list=(1, 2, 4, 6, 8, 16),
              partition_mode=(W.PARTITION_ALL, W.PARTITION_ALL, W.PARTITION_BALANCED, W.PARTITION_ALL,
                              W.PARTITION_ALL, W.PARTITION_BALANCED)[case],
              dp_overlap=case % 2, dp_bucket_bytes=0 if case == 2 else 3000, sched_mask=mask, v_max=(4, 2, 4, 2, 2, 4)[case])
    w = W.random_small(700 + case, **kw)
    n = load(E, ctx, w)
    cands = oracle.enumerate_at(w.table, w.space, np.arange(n))
    assert any(c.sched == 3 and c.v == kw["v_max"] for c in cands) and (mask == 8 or any(c.sched != 3 for c in cands))
    batch, sb = eval_all(E, ctx, n)
    ob, obusy = oracle.eval_indices_parallel(w.table, w.space, np.arange(n), THREADS, replicate=False,
                                             pp_stride=w.space.pp_max)
    gb = batch.cpu().numpy()
    assert (gb == ob).all(), [(i, cands[i]) for i in np.argwhere(gb != ob)[:3, 0]]
    assert (sb.cpu().numpy() == obusy).all()
    for i in range(0, n, max(1, n // 97)):
        d = E.distsim_decode(ctx, i)
        c = cands[i]
        assert (d["mp"], d["pp"], d["dp"], d["m"], d["sched"], d["bounds"], d["v"]) == (c.mp, c.pp, c.dp, c.m, c.sched, c.bounds, c.v)
    order = np.lexsort((np.arange(n), ob))
    k = min(n, 64)
    ki, kt, got = dev(k), dev(k), dev(n)
    assert E.distsim_eval_select(ctx, 0, n, got, k, ki, kt) == (order[0], ob[order[0]])
    assert (ki.cpu().numpy() == order[:k]).all() and (kt.cpu().numpy() == ob[order[:k]]).all()
    # odd sub-ranges across the rows
    rng = np.random.default_rng(case)
    for _ in range(6):
        first = int(rng.integers(0, n)); count = int(rng.integers(1, n - first + 1))
        out = dev(count)
        E.distsim_eval_strategies(ctx, first, count, out)
        assert (out.cpu().numpy() == ob[first:first + count]).all()
    cells, _ = E.distsim_testing_space_cells(ctx)
    assert cells == W.count_candidates_and_cells(w.table, w.space)[1]
    # every record of the timelines of interleaved candidates (and some of the others beside them)
    ilv = [i for i, c in enumerate(cands) if c.sched == 3]
    pick = ilv[:: max(1, len(ilv) // 14)][:14] + [ilv[-1], 0, n - 1]
    check_emission(E, ctx, w, pick)


def test_interleaved_1f1b_on_the_64_device_shape(E, ctx):
    """The 64-device workload with two chunks per device added to its schedules: sampled
    candidates of every row against the oracle, the best candidate over the whole space."""
    w = W.config1()
    w.space.sched_mask, w.space.v_max = 11, 2
    n = load(E, ctx, w)
    assert n > 38_838_764
    idx, total = stratified_indices(w.table, w.space, 60, 5)
    assert total == n
    cands = oracle.enumerate_at(w.table, w.space, idx)
    assert sum(c.sched == 3 for c in cands) > 500
    batch, _ = eval_all(E, ctx, n, busy=False)
    ob, _ = oracle.eval_indices_parallel(w.table, w.space, idx, THREADS, replicate=False)
    gb = batch[torch.from_numpy(idx).cuda()].cpu().numpy()
    assert (gb == ob).all(), idx[np.argwhere(gb != ob)[:5, 0]]
    bi, bt = E.distsim_argmin(ctx, batch, 0, n)
    assert oracle.eval_indices(w.table, w.space, np.array([bi]))[0][0] == bt == int(batch.min().item())
    # timelines: interleaved candidates with few and many micro-batches, one of the others beside them
    ilv = [int(i) for i, c in zip(idx, cands) if c.sched == 3]
    check_emission(E, ctx, w, [ilv[0], ilv[len(ilv) // 2], ilv[-1], 0])


@pytest.mark.parametrize("case", range(6))
def test_bidirectional_pipelines_every_candidate(E, ctx, case):
    """Spaces with bidirectional-pipeline candidates (sched_mask bit 4) beside the other schedules
    and alone: every candidate's batch time and per-device activity time, the decoded candidates,
    the best one and the k fastest, sub-ranges; emission of such a candidate is refused."""
    mask = (31, 16, 19, 23, 17, 24)[case]
    kw = dict(n_devices=(8, 8, 8, 16, 4, 8)[case], gpus_per_node=(4, 2, 4, 8, 4, 2)[case],
              n_layers=(9, 8, 10, 9, 12, 16)[case], global_batch=16, mp_max=2, pp_max=(4, 4, 4, 8, 4, 8)[case],
              m_list=(1, 2, 4, 6, 8, 16), partition_mode=(W.PARTITION_ALL, W.PARTITION_ALL, W.PARTITION_BALANCED,
                                                          W.PARTITION_ALL, W.PARTITION_ALL, W.PARTITION_BALANCED)[case],
              dp_overlap=case % 2, dp_bucket_bytes=0 if case == 2 else 3000, sched_mask=mask, v_max=2)
    w = W.random_small(720 + case, **kw)
    n = load(E, ctx, w)
    cands = oracle.enumerate_at(w.table, w.space, np.arange(n))
    assert any(c.sched == 4 and c.pp == kw["pp_max"] for c in cands) and (mask == 16 or any(c.sched != 4 for c in cands))
    batch, sb = eval_all(E, ctx, n)
    ob, obusy = oracle.eval_indices_parallel(w.table, w.space, np.arange(n), THREADS, replicate=False,
                                             pp_stride=w.space.pp_max)
    gb = batch.cpu().numpy()
    assert (gb == ob).all(), [(i, cands[i]) for i in np.argwhere(gb != ob)[:3, 0]]
    assert (sb.cpu().numpy() == obusy).all()
    for i in range(0, n, max(1, n // 97)):
        d = E.distsim_decode(ctx, i)
        c = cands[i]
        assert (d["mp"], d["pp"], d["dp"], d["m"], d["sched"], d["bounds"], d["v"]) == (c.mp, c.pp, c.dp, c.m, c.sched, c.bounds, c.v)
    order = np.lexsort((np.arange(n), ob))
    k = min(n, 64)
    ki, kt, got = dev(k), dev(k), dev(n)
    assert E.distsim_eval_select(ctx, 0, n, got, k, ki, kt) == (order[0], ob[order[0]])
    assert (ki.cpu().numpy() == order[:k]).all() and (kt.cpu().numpy() == ob[order[:k]]).all()
    rng = np.random.default_rng(case)
    for _ in range(6):
        first = int(rng.integers(0, n)); count = int(rng.integers(1, n - first + 1))
        out = dev(count)
        E.distsim_eval_strategies(ctx, first, count, out)
        assert (out.cpu().numpy() == ob[first:first + count]).all()
    cells, _ = E.distsim_testing_space_cells(ctx)
    assert cells == W.count_candidates_and_cells(w.table, w.space)[1]
    # every record of the timelines of bidirectional candidates (and some of the others beside them)
    two_way = [i for i, c in enumerate(cands) if c.sched == 4]
    pick = two_way[:: max(1, len(two_way) // 14)][:14] + [two_way[-1], 0, n - 1]
    check_emission(E, ctx, w, pick)


def test_bidirectional_pipelines_on_the_64_device_shape(E, ctx):
    """The 64-device workload with bidirectional pipelines added to its schedules: sampled
    candidates of every row against the oracle, the best candidate over the whole space."""
    w = W.config1()
    w.space.sched_mask = 19
    n = load(E, ctx, w)
    assert n > 38_838_764
    idx, total = stratified_indices(w.table, w.space, 60, 5)
    assert total == n
    cands = oracle.enumerate_at(w.table, w.space, idx)
    assert sum(c.sched == 4 for c in cands) > 500 and any(c.sched == 4 and c.pp == 16 and c.m == 128 for c in cands)
    batch, _ = eval_all(E, ctx, n, busy=False)
    ob, _ = oracle.eval_indices_parallel(w.table, w.space, idx, THREADS, replicate=False)
    gb = batch[torch.from_numpy(idx).cuda()].cpu().numpy()
    assert (gb == ob).all(), idx[np.argwhere(gb != ob)[:5, 0]]
    bi, bt = E.distsim_argmin(ctx, batch, 0, n)
    assert oracle.eval_indices(w.table, w.space, np.array([bi]))[0][0] == bt == int(batch.min().item())
    # timelines: bidirectional candidates with few and many micro-batches, one of the others beside them
    two_way = [int(i) for i, c in zip(idx, cands) if c.sched == 4]
    deep = [int(i) for i, c in zip(idx, cands) if c.sched == 4 and c.pp == 16 and c.m == 128]
    check_emission(E, ctx, w, [two_way[0], two_way[len(two_way) // 2], deep[0], deep[-1], 0])


@pytest.mark.parametrize("case", range(12))
def test_randomised_spaces_sampled_parity(E, ctx, case):
    """Randomly drawn clusters, layer counts, micro-batch lists (around m = pp, where the
    recurrence changes form), duration scales (time bounds far below, around and above 2^32, so
    rows mix 32-bit and 64-bit entries), bucket sizes, overlap modes, schedule masks and jitter:
    sampled candidates and their per-stage activity times against the oracle."""
    rng = np.random.default_rng(4000 + case)
    hi = int(rng.choice([5000, 400_000, 30_000_000, 400_000_000]))
    ms = sorted(set(int(x) for x in rng.choice([1, 2, 3, 4, 7, 8, 9, 15, 16, 17, 24, 31, 32, 33, 48, 64], size=6)))
    w = W.random_small(2000 + case, n_devices=int(rng.choice([16, 32, 64])), gpus_per_node=int(rng.choice([2, 4, 8])),
                       n_layers=int(rng.choice([17, 20, 24])), global_batch=int(rng.choice([64, 96, 128])),
                       mp_max=int(rng.choice([1, 2, 4])), pp_max=int(rng.choice([4, 8, 16, 16])), m_list=tuple(ms),
                       partition_mode=W.PARTITION_ALL, dp_overlap=int(rng.integers(0, 2)),
                       dp_bucket_bytes=int(rng.choice([0, 3000, 100_000])), lo=50, hi=hi,
                       moe=bool(rng.integers(0, 2)), sched_mask=int(rng.choice([3, 3, 7, 2, 5])))
    if case % 4 == 3:
        w = W.add_jitter(w, 4, hi // 7 + 1, case)
    if W.count_candidates_and_cells(w.table, w.space)[0] < 10:
        pytest.skip("the draw gave an empty space")
    n = load(E, ctx, w)
    batch, sb = eval_all(E, ctx, n, busy=n * ctx.pp_max < 2e8)
    idx = np.unique(np.concatenate([rng.integers(0, n, 1500), [0, n - 1]]))
    ob, obusy = oracle.eval_indices_parallel(w.table, w.space, idx, THREADS, replicate=False,
                                             pp_stride=w.space.pp_max)
    sel = torch.from_numpy(idx).cuda()
    gb = batch[sel].cpu().numpy()
    assert (gb == ob).all(), idx[np.argwhere(gb != ob)[:5, 0]]
    if sb is not None:
        assert (sb[sel].cpu().numpy() == obusy).all()


def test_many_layers(E, ctx):
    """200 layers: tables too large to stage in shared memory (bucket-lane tables and binomials
    are read from global memory), long item templates and one-item runs in emission."""
    w = W.random_small(77, n_devices=8, gpus_per_node=4, n_layers=200, global_batch=32, mp_max=2, pp_max=4,
                       m_list=(1, 3, 4, 8), partition_mode=W.PARTITION_ALL, dp_bucket_bytes=30_000, hi=3000)
    n = load(E, ctx, w)
    assert n > 10**6
    batch, sb = eval_all(E, ctx, n)
    rng = np.random.default_rng(77)
    idx = np.unique(np.concatenate([rng.integers(0, n, 400), [0, n - 1]]))
    ob, obusy = oracle.eval_indices_parallel(w.table, w.space, idx, THREADS, replicate=False,
                                             pp_stride=w.space.pp_max)
    sel = torch.from_numpy(idx).cuda()
    assert (batch[sel].cpu().numpy() == ob).all()
    assert (sb[sel].cpu().numpy() == obusy).all()
    check_emission(E, ctx, w, [int(idx[0]), int(idx[len(idx) // 2]), int(idx[-1])])


def test_many_microbatches(E, ctx):
    """m = 1000 and 4096 (the largest the interface takes): thousands of lock-step slots, item
    runs spanning many blocks in emission."""
    w = W.random_small(78, n_devices=8, gpus_per_node=4, n_layers=9, global_batch=8192, mp_max=2, pp_max=8,
                       m_list=(1000, 4096), m_rule=W.M_RULE_CEIL, partition_mode=W.PARTITION_BALANCED,
                       dp_bucket_bytes=3000, hi=900)
    n = load(E, ctx, w)
    batch, sb = eval_all(E, ctx, n)
    ob, obusy = oracle.eval_indices_parallel(w.table, w.space, np.arange(n), THREADS, replicate=False,
                                             pp_stride=w.space.pp_max)
    assert (batch.cpu().numpy() == ob).all() and (sb.cpu().numpy() == obusy).all()
    cands = oracle.enumerate_at(w.table, w.space, np.arange(n))
    pick = [i for i, c in enumerate(cands) if c.pp == 8][:2] + [i for i, c in enumerate(cands) if c.m == 4096 and c.pp == 2][:1]
    check_emission(E, ctx, w, pick)


@pytest.mark.parametrize("n_devices,n_layers,batch", [(1, 1, 1), (1, 3, 4), (2, 1, 2), (2, 2, 6), (4, 3, 4)])
def test_degenerate_shapes(E, ctx, n_devices, n_layers, batch):
    """One device, one layer, one sample: spaces of a handful of candidates, every candidate
    evaluated, selected (k = whole range) and emitted."""
    w = W.random_small(90 + n_devices + n_layers, n_devices=n_devices, gpus_per_node=min(2, n_devices),
                       n_layers=n_layers, global_batch=batch, mp_max=4, pp_max=4, m_list=(1, 2, 3, 4),
                       partition_mode=W.PARTITION_ALL, dp_bucket_bytes=0, hi=300)
    n = load(E, ctx, w)
    assert 1 <= n < 200
    batch_t, sb = eval_all(E, ctx, n)
    ob, obusy = oracle.eval_indices(w.table, w.space, np.arange(n), replicate=True, pp_stride=w.space.pp_max)
    assert (batch_t.cpu().numpy() == ob).all() and (sb.cpu().numpy() == obusy).all()
    order = np.lexsort((np.arange(n), ob))
    assert E.distsim_argmin(ctx, batch_t, 0, n) == (order[0], ob[order[0]])
    ki, kt = dev(n), dev(n)
    E.distsim_topk(ctx, batch_t, 0, n, n, ki, kt)
    assert (ki.cpu().numpy() == order).all() and (kt.cpu().numpy() == ob[order]).all()
    check_emission(E, ctx, w, list(range(n)))


def test_ranges_straddle_rows_and_empty(E, ctx):
    w = W.random_small(7, partition_mode=W.PARTITION_ALL)
    n = load(E, ctx, w)
    full, _ = eval_all(E, ctx, n, busy=False)
    full = full.cpu().numpy()
    rng = np.random.default_rng(0)
    for _ in range(12):
        first = int(rng.integers(0, n))
        count = int(rng.integers(0, n - first + 1))
        out = dev(max(1, count)); out.fill_(-1)
        E.distsim_eval_strategies(ctx, first, count, out)
        torch.cuda.synchronize()
        assert (out.cpu().numpy()[:count] == full[first:first + count]).all()
        if count:
            bi, bt = E.distsim_argmin(ctx, out, first, count)
            seg = full[first:first + count]
            assert bt == seg.min() and bi == first + int(np.argmin(seg))
    with pytest.raises(E.DistsimError) as ei:
        E.distsim_eval_strategies(ctx, n - 1, 2, dev(2))
    assert ei.value.code == E.E_RANGE


def test_config2_long_pipelines(E, ctx):
    w = W.config2()
    n = load(E, ctx, w)
    assert n == 4176
    batch, sb = eval_all(E, ctx, n)
    ob, obusy = oracle.eval_indices_parallel(w.table, w.space, np.arange(n), THREADS, replicate=False,
                                             pp_stride=w.space.pp_max)
    gb = batch.cpu().numpy()
    assert (gb == ob).all(), np.argwhere(gb != ob)[:5]
    assert (sb.cpu().numpy() == obusy).all()
    order = np.lexsort((np.arange(n), ob))
    bi, bt = E.distsim_argmin(ctx, batch, 0, n)
    assert (bi, bt) == (order[0], ob[order[0]])
    ki, kt = dev(1024), dev(1024)
    E.distsim_topk(ctx, batch, 0, n, 1024, ki, kt)
    assert (ki.cpu().numpy() == order[:1024]).all() and (kt.cpu().numpy() == ob[order[:1024]]).all()
    # full timelines of three of the fastest (1024 devices each) and two pp = 64 candidates
    cands = oracle.enumerate_at(w.table, w.space, np.arange(n))
    pp64 = [i for i, c in enumerate(cands) if c.pp == 64 and c.m == 7]
    check_emission(E, ctx, w, [int(order[0]), int(order[517]), int(order[1023]), pp64[0], pp64[1]])


def _sampled_parity(E, ctx, w, n_sample, seed):
    n = load(E, ctx, w)
    batch, _ = eval_all(E, ctx, n, busy=False)
    rng = np.random.default_rng(seed)
    idx = np.unique(np.concatenate([np.linspace(0, n - 1, n_sample // 2).astype(np.int64),
                                    rng.integers(0, n, n_sample // 2), [0, n - 1]]))
    ob, obusy = oracle.eval_indices_parallel(w.table, w.space, idx, THREADS, replicate=False,
                                             pp_stride=w.space.pp_max)
    gb = batch[torch.from_numpy(idx).cuda()].cpu().numpy()
    assert (gb == ob).all(), idx[np.argwhere(gb != ob)[:5, 0]]
    # per-stage activity time on sampled candidates (evaluated one by one)
    for i in idx[:: max(1, len(idx) // 64)]:
        b1, s1 = dev(1), dev(ctx.pp_max)
        E.distsim_eval_strategies(ctx, int(i), 1, b1, s1)
        k = int(np.searchsorted(idx, i))
        assert b1.item() == ob[k] and (s1.cpu().numpy() == obusy[k]).all()
    # argmin over the whole space: agrees with a reduction of the device array, and the
    # winner's time agrees with the oracle
    bi, bt = E.distsim_argmin(ctx, batch, 0, n)
    tmin = int(batch.min().item())
    assert bt == tmin and bi == int((batch == tmin).nonzero()[0].item())
    assert oracle.eval_indices(w.table, w.space, np.array([bi]))[0][0] == bt
    # top-k: sorted by (time, index), equal to a stable sort of the device array
    k = 1024
    ki, kt = dev(k), dev(k)
    E.distsim_topk(ctx, batch, 0, n, k, ki, kt)
    st, si = torch.sort(batch, stable=True)
    assert (kt == st[:k]).all() and (ki == si[:k]).all()
    return n, batch, ki


def test_config3_moe_sampled(E, ctx):
    w = W.config3()
    n, batch, ki = _sampled_parity(E, ctx, w, 3000, 3)
    assert n == 650_420
    pick = ki.cpu().numpy()[[0, 1, 500]].tolist() + [12345, n - 1]
    check_emission(E, ctx, w, pick)


def test_config1_full_size_sampled(E, ctx):
    w = W.config1()
    n, batch, ki = _sampled_parity(E, ctx, w, 6000, 1)
    assert n == 38_838_764
    pick = ki.cpu().numpy()[[0, 7, 1023]].tolist() + [0, 20_000_001, n - 1]
    check_emission(E, ctx, w, pick)


def test_config3_every_candidate(E, ctx):
    """All 650 420 candidates of the 256-device MoE workload against the oracle."""
    w = W.config3()
    n = load(E, ctx, w)
    batch, _ = eval_all(E, ctx, n, busy=False)
    ob, _ = oracle.eval_indices_parallel(w.table, w.space, np.arange(n), THREADS, replicate=False)
    gb = batch.cpu().numpy()
    assert (gb == ob).all(), np.argwhere(gb != ob)[:5]
    order = np.lexsort((np.arange(n), ob))
    assert E.distsim_argmin(ctx, batch, 0, n) == (order[0], ob[order[0]])
    ki, kt = dev(1024), dev(1024)
    E.distsim_topk(ctx, batch, 0, n, 1024, ki, kt)
    assert (ki.cpu().numpy() == order[:1024]).all() and (kt.cpu().numpy() == ob[order[:1024]]).all()


def stratified_indices(table, space, per_cell, seed):
    """Indices that hit every (row, micro-batch count, schedule) cell of a space with up to
    `per_cell` partitions each - the first and the last partition among them, hence both ends of
    every row."""
    rng = np.random.default_rng(seed)
    out, off = [], 0
    for mp, pp, dp, ms, parts, n_sched, _v in W.space_shape(table, space):
        for e in range(len(ms)):
            if parts <= per_cell:
                p = np.arange(parts, dtype=np.int64)
            else:
                p = np.unique(np.concatenate([[0, parts - 1], rng.integers(0, parts, per_cell - 2)])).astype(np.int64)
            for sc in range(n_sched):
                out.append(off + (e * parts + p) * n_sched + sc)
        off += len(ms) * parts * n_sched
    return np.unique(np.concatenate(out)), off


def test_config1_stratified_million(E, ctx):
    """More than a million candidates of the 64-device workload, drawn so that every (row,
    micro-batch count, schedule) cell and both ends of every row are compared with the oracle."""
    w = W.config1()
    n = load(E, ctx, w)
    idx, total = stratified_indices(w.table, w.space, 10000, 11)
    assert total == n == 38_838_764 and len(idx) >= 1_000_000 and idx[0] == 0 and idx[-1] == n - 1
    batch, _ = eval_all(E, ctx, n, busy=False)
    ob, _ = oracle.eval_indices_parallel(w.table, w.space, idx, THREADS, replicate=False)
    gb = batch[torch.from_numpy(idx).cuda()].cpu().numpy()
    assert (gb == ob).all(), idx[np.argwhere(gb != ob)[:5, 0]]


def test_stalled_table_copies_fall_back_exactly(E, ctx):
    """The kernels' first wait for their staged tables is made to give up at once (a host-set poll
    limit of 0; the second wait keeps its limit, so every copy has landed before its block goes
    on and nothing hangs): every block then reads its tables from global memory.  Results must be
    bit-exact, and the next synchronising call must still deliver its outputs while returning
    DISTSIM_E_TIMEOUT."""
    for cfg, k in ((1, 64), (3, 64), (2, 16)):      # thread kernel in 32- and 64-bit arithmetic, lock-step kernel
        w = W.CONFIGS[cfg]()
        n = load(E, ctx, w)
        want, wb = eval_all(E, ctx, n)
        best = E.distsim_argmin(ctx, want, 0, n)
        E.distsim_testing_set_stage_wait_polls(ctx, 0)
        try:
            got, gbz = eval_all(E, ctx, n)
            assert torch.equal(got, want) and torch.equal(gbz, wb)
            with pytest.raises(E.DistsimError) as ei:
                E.distsim_argmin(ctx, got, 0, n)
            assert ei.value.code == E.E_TIMEOUT and ei.value.result == best
            assert E.distsim_argmin(ctx, got, 0, n) == best          # the status word was cleared
            # emission after a stalled evaluation: outputs complete, code reported once
            got2, _ = eval_all(E, ctx, n, busy=False)
            top = dev(k)
            E.distsim_topk(ctx, got2, 0, n, k, top)
            N = w.table.n_devices
            off = dev(k * N + 1)
            with pytest.raises(E.DistsimError) as ei:
                E.distsim_emit_timelines(ctx, top, k, None, 0, off)
            assert ei.value.code == E.E_TIMEOUT and ei.value.total_records == int(off[-1]) > 0
        finally:
            E.distsim_testing_set_stage_wait_polls(ctx, 1 << 16)
        again, _ = eval_all(E, ctx, n, busy=False)
        assert torch.equal(again, want)
        assert E.distsim_argmin(ctx, again, 0, n) == best


def _flat_table(n_layers, n_devices, gpus_per_node, global_batch, space, per_layer_ns, seed):
    """Table whose layer times do not depend on the micro-batch size, so that an entry's time
    bound grows with m: small m fits 32 bits, large m does not."""
    rng = np.random.default_rng(seed)
    classes = W.event_classes(n_devices, global_batch, n_layers, space)
    f = rng.integers(per_layer_ns // 2, per_layer_ns, n_layers)
    g = 2 * f + rng.integers(0, 1000, n_layers)
    return W.EventTable(
        n_layers=n_layers, n_devices=n_devices, gpus_per_node=gpus_per_node, global_batch=global_batch,
        seq=128, hidden=64, class_mp=[c[0] for c in classes], class_b=[c[1] for c in classes],
        fwd_ns=np.tile(f, (len(classes), 1)), bwd_ns=np.tile(g, (len(classes), 1)),
        layer_is_expert=(np.arange(n_layers) % 3 == 0).astype(np.uint8),
        grad_bytes=rng.integers(1, 5 * 10**6, n_layers), dp_bucket_bytes=2 * 10**6)


def test_rows_mixing_32_and_64_bit_entries(E, ctx):
    # per micro-batch ~ 16 layers x 3 x 2^24 ns: the bound crosses 2^32 between m = 4 and m = 8,
    # so one row is evaluated partly in uint32 and partly in int64 arithmetic
    space = W.SearchSpace(mp_max=2, pp_max=8, m_list=[1, 2, 4, 8, 16], m_rule=W.M_RULE_CEIL,
                          partition_mode=W.PARTITION_ALL)
    table = _flat_table(16, 16, 4, 64, space, 1 << 24, 5)
    w = W.Workload("mixed_width", table, space, 5)
    n = load(E, ctx, w)
    cells, cells32 = E.distsim_testing_space_cells(ctx)
    assert cells == W.count_candidates_and_cells(table, space)[1] and 0 < cells32 < cells
    batch, sb = eval_all(E, ctx, n)
    rng = np.random.default_rng(0)
    idx = np.unique(np.concatenate([rng.integers(0, n, 4000), np.arange(0, n, max(1, n // 500)), [n - 1]]))
    ob, obusy = oracle.eval_indices_parallel(table, space, idx, THREADS, pp_stride=space.pp_max)
    sel = torch.from_numpy(idx).cuda()
    assert (batch[sel].cpu().numpy() == ob).all()
    assert (sb[sel].cpu().numpy() == obusy).all()
    # an odd-aligned sub-range exercises the unpaired store path
    first, count = 12345, 40001
    out = dev(count + 1)[1:]
    E.distsim_eval_strategies(ctx, first, count, out)
    assert torch.equal(out, batch[first:first + count])
    check_emission(E, ctx, w, [0, 7, int(idx[len(idx) // 2]), n - 1])


@pytest.mark.parametrize("pp,n_layers", [(32, 34), (64, 66)])
def test_long_pipelines_every_composition(E, ctx, pp, n_layers):
    # lock-step kernel with all compositions: one and two stages per lane
    space = W.SearchSpace(mp_max=1, pp_max=pp, m_list=[1, 3, 40, 70], m_rule=W.M_RULE_CEIL,
                          partition_mode=W.PARTITION_ALL)
    # an odd global batch admits dp = 1 only, so the space holds the pp = n_devices row alone
    table = _flat_table(n_layers, pp, 8, 141, space, 50_000, pp)
    w = W.Workload(f"long_{pp}", table, space, pp)
    n = load(E, ctx, w)
    batch, sb = eval_all(E, ctx, n)
    cands = oracle.enumerate_at(table, space, np.arange(n))
    assert all(c.pp == pp for c in cands)
    idx = np.unique(np.concatenate([np.arange(0, n, 37), [n - 1]]))
    ob, obusy = oracle.eval_indices_parallel(table, space, idx, THREADS, pp_stride=space.pp_max)
    sel = torch.from_numpy(idx).cuda()
    assert (batch[sel].cpu().numpy() == ob).all()
    assert (sb[sel].cpu().numpy() == obusy).all()
    check_emission(E, ctx, w, [int(idx[1]), int(idx[-2])])


def test_long_pipelines_with_chunks_and_two_ways(E, ctx):
    # the longest pipelines the warp-per-candidate kernel takes: up to 32 devices running
    # interleaved 1F1B with two chunks each (64 virtual stages) and bidirectional pipelines (one
    # candidate per warp, the largest shared-memory arrays), few and many micro-batches, balanced
    # partitions of an odd number of layers: every candidate
    space = W.SearchSpace(mp_max=1, pp_max=32, m_list=[2, 32, 64, 70, 96], m_rule=W.M_RULE_CEIL,
                          partition_mode=W.PARTITION_BALANCED, sched_mask=24, v_max=2)
    table = _flat_table(67, 32, 8, 141, space, 50_000, 32)        # odd global batch: dp = 1 only
    w = W.Workload("long_32_chunks_two_ways", table, space, 32)
    n = load(E, ctx, w)
    cands = oracle.enumerate_at(table, space, np.arange(n))
    kinds = {(c.pp, c.sched, c.m) for c in cands}
    assert (32, 3, 96) in kinds and (32, 4, 70) in kinds and (32, 4, 2) in kinds, kinds
    batch, sb = eval_all(E, ctx, n)
    ob, obusy = oracle.eval_indices_parallel(table, space, np.arange(n), THREADS, pp_stride=space.pp_max)
    assert (batch.cpu().numpy() == ob).all()
    assert (sb.cpu().numpy() == obusy).all()
    pick = [i for i, c in enumerate(cands) if (c.pp, c.sched, c.m) in ((32, 3, 96), (32, 4, 70), (32, 4, 2))]
    check_emission(E, ctx, w, pick)


@pytest.mark.parametrize("cfg,stride", [(1, 39_119), (2, 1), (3, 653)])
def test_index_decoding_matches_loop_enumeration(E, ctx, cfg, stride):
    # the library's index -> candidate mapping against the oracle's nested loops
    w = W.CONFIGS[cfg]()
    n = load(E, ctx, w)
    idx = np.unique(np.concatenate([np.arange(0, n, stride), [n - 1]]))
    for i, c in zip(idx.tolist(), oracle.enumerate_at(w.table, w.space, idx)):
        d = E.distsim_decode(ctx, i)
        assert (d["mp"], d["pp"], d["dp"], d["m"], d["sched"], d["bounds"]) == (c.mp, c.pp, c.dp, c.m, c.sched, c.bounds), i
        assert d["micro_batch_size"] == -(-(w.table.global_batch // c.dp) // c.m)


def test_paper_grid_with_extrapolated_allreduce(E, ctx):
    # the paper's own search shape (16 GPUs, 48 layers, 15 valid (mp, pp) settings), with
    # all-reduces above 8 devices extrapolated from the 8-device time
    w = W.paper_grid()
    n = load(E, ctx, w)
    batch, sb = eval_all(E, ctx, n)
    ob, obusy = oracle.eval_indices_parallel(w.table, w.space, np.arange(n), THREADS, replicate=False,
                                             pp_stride=w.space.pp_max)
    assert (batch.cpu().numpy() == ob).all() and (sb.cpu().numpy() == obusy).all()
    cands = oracle.enumerate_at(w.table, w.space, np.arange(n))
    dp16 = [i for i, c in enumerate(cands) if c.dp == 16]
    mp16 = [i for i, c in enumerate(cands) if c.mp == 16]
    check_emission(E, ctx, w, dp16[:2] + mp16[:2] + [n // 2, n - 1])
    # and a small irregular space where even 4- and 8-way all-reduces are extrapolated
    w2 = W.random_small(41)
    w2.table.allreduce_profile_max = 2
    n2 = load(E, ctx, w2)
    b2, s2 = eval_all(E, ctx, n2)
    o2, ob2 = oracle.eval_indices_parallel(w2.table, w2.space, np.arange(n2), THREADS, pp_stride=w2.space.pp_max)
    assert (b2.cpu().numpy() == o2).all() and (s2.cpu().numpy() == ob2).all()
    check_emission(E, ctx, w2, list(range(0, n2, max(1, n2 // 12))))


@pytest.mark.parametrize("seed", range(4))
def test_per_microbatch_jitter_full_parity(E, ctx, seed):
    kw = dict(dp_overlap=seed % 2, dp_bucket_bytes=3000)
    if seed >= 2:
        kw.update(n_devices=16, gpus_per_node=2, n_layers=9, global_batch=24, mp_max=4, pp_max=8,
                  m_list=(1, 2, 3, 5, 6, 12), partition_mode=W.PARTITION_ALL)
    w = W.add_jitter(W.random_small(200 + seed, **kw), 4 if seed % 2 else 1, 2500, seed)
    n = load(E, ctx, w)
    batch, sb = eval_all(E, ctx, n)
    ob, obusy = oracle.eval_indices_parallel(w.table, w.space, np.arange(n), THREADS, replicate=False,
                                             pp_stride=w.space.pp_max)
    gb = batch.cpu().numpy()
    assert (gb == ob).all(), np.argwhere(gb != ob)[:5]
    assert (sb.cpu().numpy() == obusy).all()
    rng = np.random.default_rng(seed)
    check_emission(E, ctx, w, rng.choice(n, size=min(n, 20), replace=False).tolist())


def test_jitter_on_benchmark_shapes(E, ctx):
    # 256-device MoE workload (int64 times, every composition) and the long pipelines of the
    # 1024-device workload, each with an 8-slot jitter table
    # and the 64-device workload (uint32 arithmetic in the one-partition-per-thread kernel)
    for cfg, amp, n_sample in ((3, 200_000, 1500), (2, 5_000_000, 4176), (1, 50_000, 3000)):
        w = W.add_jitter(W.CONFIGS[cfg](), 8, amp)
        n = load(E, ctx, w)
        batch, sb = eval_all(E, ctx, n)
        idx = np.unique(np.linspace(0, n - 1, n_sample).astype(np.int64))
        ob, obusy = oracle.eval_indices_parallel(w.table, w.space, idx, THREADS, pp_stride=w.space.pp_max)
        sel = torch.from_numpy(idx).cuda()
        assert (batch[sel].cpu().numpy() == ob).all()
        assert (sb[sel].cpu().numpy() == obusy).all()
        ki = dev(4)
        E.distsim_topk(ctx, batch, 0, n, 4, ki)
        check_emission(E, ctx, w, ki.cpu().numpy().tolist()[:2] + [int(idx[len(idx) // 3])])
    # tables the engine refuses
    import copy
    t = copy.deepcopy(W.config0().table)
    t.jitter_fwd_ns = np.zeros((3, 4), np.int64); t.jitter_bwd_ns = np.zeros((3, 4), np.int64)
    with pytest.raises(E.DistsimError) as ei:
        E.distsim_load_event_table(ctx, t)
    assert ei.value.code == E.E_UNSUPPORTED                   # slots must be a power of two
    t.jitter_fwd_ns = np.zeros((2, 2), np.int64); t.jitter_bwd_ns = np.zeros((2, 2), np.int64)
    E.distsim_load_event_table(ctx, t)
    with pytest.raises(E.DistsimError) as ei:
        E.distsim_set_space(ctx, W.config0().space)           # pp = 4 needs 4 columns
    assert ei.value.code == E.E_ARG


def test_integer_probes_run():
    from paper_2306_08423_b200 import probes
    sink = dev(1)
    for mode in range(5):
        assert probes.distsim_bench_int_issue_probe(148, 64, mode, sink) > 0
    torch.cuda.synchronize()
    with pytest.raises(RuntimeError):
        probes.distsim_bench_int_issue_probe(148, 64, 9, sink)


def _emit_chunk_and_check(E, ctx, w, top, sample_positions):
    """Emits the selections `top` (device tensor) in one call, checks structure on the device
    and the sampled selections record by record against the oracle."""
    N = w.table.n_devices
    n = top.numel()
    offsets, busy, util = dev(n * N + 1), dev(n * N), dev(n * N, torch.float64)
    total = E.distsim_emit_timelines(ctx, top, n, None, 0)
    records = dev(total * 5)
    records.fill_(-7)                                  # no field of any record is ever -7
    assert E.distsim_emit_timelines(ctx, top, n, records, total, offsets, busy, util) == total
    assert int((records == -7).sum()) == 0             # every word was written
    rec = records.view(total, 5)
    # properties that hold at any size
    assert int(offsets[0]) == 0 and int(offsets[-1]) == total
    assert bool((offsets[1:] >= offsets[:-1]).all())
    assert bool(((rec[:, 0] >= 0) & (rec[:, 0] <= 10)).all())
    assert bool((rec[:, 4] >= rec[:, 3]).all()) and bool((rec[:, 3] >= 0).all())
    assert bool((util > 0).all()) and bool((util <= 1.0).all())
    idx = top.cpu().numpy()
    sums = device_checksums(E, ctx, records, offsets, n * N)
    for pos in sample_positions:
        c = oracle.enumerate_at(w.table, w.space, np.array([idx[pos]]))[0]
        r = oracle.simulate(w.table, c, replicate=True)
        want = [stream_checksum(r.records[r.offsets[k]:r.offsets[k + 1]]) for k in range(N)]
        assert sums[pos * N: (pos + 1) * N].tolist() == want, (pos, c)
        lo, hi = int(offsets[pos * N]), int(offsets[(pos + 1) * N])
        assert hi - lo == r.offsets[-1]
        assert (offsets[pos * N: (pos + 1) * N + 1].cpu().numpy() - lo == r.offsets).all()
        assert (rec[lo:hi].cpu().numpy() == r.records).all(), (pos, c)
        assert (busy[pos * N: (pos + 1) * N].cpu().numpy() == r.busy_ns).all()
        np.testing.assert_allclose(util[pos * N: (pos + 1) * N].cpu().numpy(), r.util, rtol=1e-12, atol=0)
    return total


def test_emission_in_the_benchmark_launch_configurations(E, ctx):
    # (a) the search step of the benchmark: the 1024 fastest of the 64-device workload, one call
    w = W.config1()
    n = load(E, ctx, w)
    batch, _ = eval_all(E, ctx, n, busy=False)
    top = dev(1024)
    E.distsim_topk(ctx, batch, 0, n, 1024, top)
    _emit_chunk_and_check(E, ctx, w, top, [0, 333, 1023])
    del batch
    # (b) the emission workload: the 1024 fastest of the 1024-device workload, 128 per call
    w = W.config4()
    n = load(E, ctx, w)
    batch, _ = eval_all(E, ctx, n, busy=False)
    top = dev(w.top_k)
    E.distsim_topk(ctx, batch, 0, n, w.top_k, top)
    grand = 0
    for k, i in enumerate(range(0, w.top_k, 128)):
        grand += _emit_chunk_and_check(E, ctx, w, top[i:i + 128], [(17 * k) % 128])
        torch.cuda.empty_cache()
    assert grand > 10**9                              # about 2e9 records, 8e10 bytes in all


@pytest.mark.parametrize("cfg", [1, 3])
def test_small_windows_agree_with_the_full_evaluation(E, ctx, cfg):
    # a window of under 2048 partitions is evaluated by the lock-step kernel, the whole space by
    # the one-partition-per-thread kernel: two implementations, one answer
    w = W.CONFIGS[cfg]()
    n = load(E, ctx, w)
    full, fb = eval_all(E, ctx, n)
    rng = np.random.default_rng(cfg)
    out, ob = dev(3001), dev(3001 * ctx.pp_max)
    for _ in range(48):
        count = int(rng.integers(1, 3001))
        first = int(rng.integers(0, n - count))
        E.distsim_eval_strategies(ctx, first, count, out, ob)
        assert torch.equal(out[:count], full[first:first + count])
        assert torch.equal(ob[:count * ctx.pp_max].view(count, -1), fb[first:first + count])


def _check_eval_select(E, ctx, first, count, k):
    want = dev(count)
    E.distsim_eval_strategies(ctx, first, count, want)
    wi, wt = dev(max(1, k)), dev(max(1, k))
    if k:
        E.distsim_topk(ctx, want, first, count, k, wi, wt)
    best = E.distsim_argmin(ctx, want, first, count)
    got = dev(count); got.fill_(-1)
    gi, gt = dev(max(1, k)), dev(max(1, k))
    assert E.distsim_eval_select(ctx, first, count, got, k, gi if k else None, gt if k else None) == best
    torch.cuda.synchronize()
    assert torch.equal(got, want)
    if k:
        assert torch.equal(gi, wi) and torch.equal(gt, wt)
    # without host outputs: asynchronous, the best candidate goes to device memory
    got.fill_(-1); gi.fill_(-1); gt.fill_(-1)
    d_best = dev(2)
    assert E.distsim_eval_select(ctx, first, count, got, k, gi if k else None, gt if k else None, d_best,
                                 to_host=False) is None
    torch.cuda.synchronize()
    assert torch.equal(got, want) and tuple(d_best.tolist()) == (best[1], best[0])
    if k:
        assert torch.equal(gi, wi) and torch.equal(gt, wt)
    return want


def test_eval_select_matches_separate_calls(E, ctx):
    """Evaluation with the best candidate and the k fastest folded into its kernels against the
    separate calls, which the other tests compare with the oracle: thread kernel in 32- and 64-bit
    arithmetic, lock-step kernel, sub-ranges, short arrays, ties, times too wide to pack."""
    for cfg, k in ((1, 1024), (3, 1024), (2, 1024), (0, 10)):
        w = W.CONFIGS[cfg]()
        n = load(E, ctx, w)
        _check_eval_select(E, ctx, 0, n, k)
        _check_eval_select(E, ctx, 0, n, 0)
        if n > 10_000:
            rng = np.random.default_rng(cfg)
            for _ in range(3):
                first = int(rng.integers(0, n - 9000))
                count = int(rng.integers(4097, min(n - first, 3_000_000)))
                _check_eval_select(E, ctx, first, count, int(rng.integers(1, 4097)))
            _check_eval_select(E, ctx, 12345, 4000, 77)                # short: sorted directly
    # coarse times: many ties at the threshold, resolved by index
    space = W.SearchSpace(mp_max=2, pp_max=8, m_list=[1, 2, 4, 8, 16], m_rule=W.M_RULE_CEIL,
                          partition_mode=W.PARTITION_ALL)
    table = _flat_table(16, 16, 4, 64, space, 3, 5)                    # layer times of 1 or 2 ns
    table.grad_bytes[:] = 0
    w = W.Workload("ties", table, space, 5)
    n = load(E, ctx, w)
    full = _check_eval_select(E, ctx, 0, n, 4096)
    assert int((full == full.min()).sum()) > 1
    ob, _ = oracle.eval_indices_parallel(table, space, np.arange(0, n, 97), THREADS)
    assert (full[::97].cpu().numpy() == ob).all()
    # times near 2^45: time and position do not fit one key, the calls fall back to separate passes
    w = W.random_small(3, lo=2**44, hi=2**45, partition_mode=W.PARTITION_ALL, n_layers=16, pp_max=4,
                       m_list=(1, 2, 4, 8))
    n = load(E, ctx, w)
    assert n > 4096
    _check_eval_select(E, ctx, 0, n, 500)


def test_asynchronous_emission_provisioning(E, ctx):
    """distsim_emit_timelines_async with shapes larger than needed (same records), with a shape or a
    capacity that is too small (nothing written, DISTSIM_E_CAPACITY from the next synchronising call,
    the count of records needed in the last offset), and the context usable afterwards."""
    w = W.config3()
    n = load(E, ctx, w)
    N = w.table.n_devices
    batch, _ = eval_all(E, ctx, n, busy=False)
    k = 48
    top = dev(k)
    E.distsim_topk(ctx, batch, 0, n, k, top)
    offsets, busy, util = dev(k * N + 1), dev(k * N), dev(k * N, torch.float64)
    total = E.distsim_emit_timelines(ctx, top, k, None, 0, offsets, busy, util)
    want = dev(total * 5)
    E.distsim_emit_timelines(ctx, top, k, want, total, offsets, busy, util)
    shape = E.distsim_emit_shape_of_last_plan(ctx)
    # a selection of another kind through a shape sized on this one, with headroom
    roomy = E.EmitShape(2 * shape.records, 2 * shape.item_tiles + 3, 2 * shape.bucket_tiles + 1, shape.tmpl_words + 40,
                        shape.bucket_recs + 7, shape.run_words)
    got, off2 = dev(total * 5 + 50), dev(k * N + 1)
    got.fill_(-7)
    E.distsim_emit_timelines_async(ctx, top, k, got, total + 10, roomy, off2, None, None)
    torch.cuda.synchronize()
    assert torch.equal(got[: total * 5], want) and bool((got[total * 5:] == -7).all()) and torch.equal(off2, offsets)
    other = torch.arange(0, n, n // 8, dtype=torch.int64, device="cuda")[:8].contiguous()
    t8 = E.distsim_emit_timelines(ctx, other, 8, None, 0)
    want8 = dev(t8 * 5)
    E.distsim_emit_timelines(ctx, other, 8, want8, t8)
    s8 = E.distsim_emit_shape_of_last_plan(ctx)
    big = E.EmitShape(*[max(getattr(roomy, f), getattr(s8, f)) for f, _ in E.EmitShape._fields_])
    got8 = dev(t8 * 5)
    E.distsim_emit_timelines_async(ctx, other, 8, got8, t8, big)
    torch.cuda.synchronize()
    assert torch.equal(got8, want8)
    # too little: each in turn
    for what in ("capacity", "item_tiles", "run_words", "tmpl_words", "bucket_recs", "bucket_tiles"):
        small = E.EmitShape(*[getattr(shape, f) for f, _ in E.EmitShape._fields_])
        cap = total
        if what == "capacity":
            cap = total - 1
        elif getattr(shape, what) == 0:
            continue
        else:
            setattr(small, what, getattr(shape, what) - 1)
        got.fill_(-7); off2.fill_(-1)
        E.distsim_emit_timelines_async(ctx, top, k, got, cap, small, off2, None, None)
        torch.cuda.synchronize()
        assert bool((got == -7).all()), what
        assert int(off2[-1]) == total and torch.equal(off2, offsets), what
        with pytest.raises(E.DistsimError) as err:
            E.distsim_argmin(ctx, batch, 0, n)
        assert err.value.code == E.E_CAPACITY, what
        assert E.distsim_argmin(ctx, batch, 0, n)[1] == int(batch.min().item())       # the status is cleared
    with pytest.raises(E.DistsimError):
        E.distsim_emit_timelines_async(ctx, top, k, got, total, E.EmitShape(total, 1 << 40, 1, 1, 1, 1))


def test_merged_rank_lists_equal_the_global_topk(E, ctx):
    """One search split over 1, 2, 3 and 8 slices (as sharding.shard_range gives them to ranks):
    every slice evaluated and selected on its own, the slices' lists merged by distsim_merge_topk,
    against the selection over the whole range."""
    from paper_2306_08423_b200 import sharding
    for cfg, k in ((3, 1024), (0, 7), (2, 300)):
        w = W.CONFIGS[cfg]()
        n = load(E, ctx, w)
        full, wi, wt = dev(n), dev(k), dev(k)
        best = E.distsim_eval_select(ctx, 0, n, full, k, wi, wt)
        for world in (1, 2, 3, 8):
            lists_t, lists_i, bests = [], [], []
            for rank in range(world):
                first, count = sharding.shard_range(n, rank, world)
                kk = min(k, count)
                part, li, lt = dev(count), dev(k), dev(k)
                li.fill_(torch.iinfo(torch.int64).max); lt.fill_(torch.iinfo(torch.int64).max)     # padding of short slices
                bests.append(E.distsim_eval_select(ctx, first, count, part, kk, li[:kk], lt[:kk]))
                lists_t.append(lt); lists_i.append(li)
            gt, gi = torch.cat(lists_t), torch.cat(lists_i)
            mi, mt = dev(k), dev(k)
            E.distsim_merge_topk(ctx, gt, gi, gt.numel(), k, mi, mt)
            torch.cuda.synchronize()
            assert torch.equal(mi, wi) and torch.equal(mt, wt), (cfg, world)
            assert min((t, i) for i, t in bests) == (best[1], best[0])


def test_two_pass_argmin_for_wide_times(E, ctx):
    # times near 2^55 with a large count cannot be packed with the index into 64 bits
    w = W.random_small(3, lo=2**44, hi=2**45, partition_mode=W.PARTITION_ALL, n_layers=12, pp_max=4,
                       m_list=(1, 2, 4, 8))
    n = load(E, ctx, w)
    batch, _ = eval_all(E, ctx, n, busy=False)
    ob, _ = oracle.eval_indices_parallel(w.table, w.space, np.arange(n), THREADS)
    assert (batch.cpu().numpy() == ob).all()
    reps = (1 << 21) // n + 1
    big = batch.repeat(reps)                       # duplicates: ties must go to the first copy
    bi, bt = E.distsim_argmin(ctx, big, 5, big.numel())
    assert bt == ob.min() and bi == 5 + int(np.argmin(ob))
    # top-k with massive ties: the k smallest indices among equal times
    k = 300
    ki, kt = dev(k), dev(k)
    E.distsim_topk(ctx, big, 0, big.numel(), k, ki, kt)
    st, si = torch.sort(big, stable=True)
    assert (kt == st[:k]).all() and (ki == si[:k]).all()
    # the one pass over a long array reads 16-byte pairs: arrays that start off a 16-byte
    # boundary, of odd and even length, with distinct times so that the refined path is taken
    gen = torch.Generator(device="cuda").manual_seed(7)
    distinct = torch.randperm((1 << 21) + 3, generator=gen, device="cuda").to(torch.int64) * 1000 + 17
    for off, length in ((1, (1 << 21) + 1), (1, 1 << 21), (0, (1 << 21) + 1), (2, 1 << 21)):
        view = distinct[off:off + length]
        st, si = torch.sort(view, stable=True)
        for k in (1, 1024, 4096):
            ki, kt = dev(k), dev(k)
            E.distsim_topk(ctx, view, 0, length, k, ki, kt)
            assert (kt == st[:k]).all() and (ki == si[:k]).all(), (off, length, k)
        bi, bt = E.distsim_argmin(ctx, view, 0, length)
        assert (bt, bi) == (int(st[0]), int(si[0]))


def test_api_errors(E, ctx):
    w = W.config0()
    with pytest.raises(E.DistsimError) as ei:
        E.distsim_set_space(ctx, w.space)
    assert ei.value.code == E.E_STATE
    with pytest.raises(E.DistsimError) as ei:
        E.distsim_eval_strategies(ctx, 0, 1, dev(1))
    assert ei.value.code == E.E_STATE
    t = copy.deepcopy(w.table); t.n_devices = 12
    with pytest.raises(E.DistsimError) as ei:
        E.distsim_load_event_table(ctx, t)
    assert ei.value.code == E.E_UNSUPPORTED
    t = copy.deepcopy(w.table); t.fwd_ns[0, 0] = -1
    with pytest.raises(E.DistsimError) as ei:
        E.distsim_load_event_table(ctx, t)
    assert ei.value.code == E.E_ARG
    t = copy.deepcopy(w.table); t.fwd_ns[:] = 2**60
    E.distsim_load_event_table(ctx, t)
    with pytest.raises(E.DistsimError) as ei:
        E.distsim_set_space(ctx, w.space)
    assert ei.value.code == E.E_OVERFLOW
    # a class the space needs is missing from the table
    t = copy.deepcopy(w.table)
    t.class_mp, t.class_b, t.fwd_ns, t.bwd_ns = t.class_mp[1:], t.class_b[1:], t.fwd_ns[1:], t.bwd_ns[1:]
    E.distsim_load_event_table(ctx, t)
    with pytest.raises(E.DistsimError) as ei:
        E.distsim_set_space(ctx, w.space)
    assert ei.value.code == E.E_ARG and "not in the table" in str(ei.value)
    # capacity and range errors of emission
    n = load(E, ctx, w)
    idx = torch.tensor([0, 5], dtype=torch.int64, device="cuda")
    total = E.distsim_emit_timelines(ctx, idx, 2, None, 0)
    small = dev(5 * (total - 1)); small.fill_(-1)
    with pytest.raises(E.DistsimError) as ei:
        E.distsim_emit_timelines(ctx, idx, 2, small, total - 1)
    assert ei.value.code == E.E_CAPACITY and ei.value.total_records == total
    assert (small == -1).all()                     # nothing was written
    bad = torch.tensor([0, n], dtype=torch.int64, device="cuda")
    with pytest.raises(E.DistsimError) as ei:
        E.distsim_emit_timelines(ctx, bad, 2, None, 0)
    assert ei.value.code == E.E_RANGE
    with pytest.raises(E.DistsimError) as ei:
        E.distsim_topk(ctx, dev(n), 0, n, n + 1, dev(n + 1))
    assert ei.value.code == E.E_ARG
    with pytest.raises(E.DistsimError):
        E.distsim_decode(ctx, n)
    # the context is still usable afterwards
    batch, _ = eval_all(E, ctx, n, busy=False)
    assert (batch.cpu().numpy() == oracle.eval_indices(w.table, w.space, np.arange(n))[0]).all()


def test_search_host_matches_device_path(E, ctx):
    w = W.config0()
    n, bi, bt, ki, kt = E.distsim_search_host(ctx, w.table, w.space, 16)
    ob, _ = oracle.eval_indices(w.table, w.space, np.arange(n))
    order = np.lexsort((np.arange(n), ob))
    assert (bi, bt) == (order[0], ob[order[0]])
    assert (ki == order[:16]).all() and (kt == ob[order[:16]]).all()
