"""Pins of the CPU oracle against what the paper and the mathematics fix.

Nothing here touches the CUDA engine.  Each test names the fact it pins; together
they are chosen so that a dropped term, a wrong sign or index, or a transposed
operand in the oracle fails at least one.
"""
import itertools
import math
import os

import numpy as np
import pytest

import oracle
from oracle import Candidate, KINDS
from paper_2306_08423_b200 import workloads as W
from tests.dag_bruteforce import bidirectional_order, longest_path_bidirectional, longest_path_timeline

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def make_table(f, g, *, n_devices, gpus_per_node, global_batch, classes, seq=0, hidden=1,
               expert=None, grad=None, scale_by_b=False, **kw):
    """Table whose every class has the same per-layer times f, g (or b*f, b*g)."""
    L = len(f)
    fwd = np.array([[(b if scale_by_b else 1) * v for v in f] for (_, b) in classes], np.int64)
    bwd = np.array([[(b if scale_by_b else 1) * v for v in g] for (_, b) in classes], np.int64)
    return W.EventTable(
        n_layers=L, n_devices=n_devices, gpus_per_node=gpus_per_node, global_batch=global_batch,
        seq=seq, hidden=hidden, class_mp=[c[0] for c in classes], class_b=[c[1] for c in classes],
        fwd_ns=fwd, bwd_ns=bwd,
        layer_is_expert=np.zeros(L, np.uint8) if expert is None else expert,
        grad_bytes=np.zeros(L, np.int64) if grad is None else grad, **kw)


def balanced(L, pp):
    return tuple(j * L // pp for j in range(pp + 1))


# --------------------------------------------------------------------------- #
# communication cost formulas

def test_ring_allreduce_volume_matches_paper_formula():
    # Sec. 4.2: per-device volume of an N-device ring all-reduce of P bytes is 2(N-1)P/N.
    for n in (2, 3, 8, 64, 1024):
        for p in (1, 7, 1000, 26214400):
            assert oracle.ring_allreduce_ns(n, p, 0, 1) == math.ceil(2 * (n - 1) * p / n) == -(-2 * (n - 1) * p // n)
    # ... which tends to 2P for large N
    assert oracle.ring_allreduce_ns(10**6, 10**6, 0, 1) == 2 * 10**6 - 2
    # latency term: 2(N-1) steps; bandwidth divides
    assert oracle.ring_allreduce_ns(8, 0, 5, 3) == 70
    assert oracle.ring_allreduce_ns(2, 300, 0, 300) == 1
    assert oracle.ring_allreduce_ns(2, 301, 0, 300) == 2  # rounds up


def test_allreduce_extrapolation_above_profiled_size():
    # Sec. 4.2: up to k devices the all-reduce is taken as profiled; above, the k-device time is
    # scaled by the per-device volume 2(N-1)P/N of the actual device count
    k, a, be = 8, 10_000, 25
    for p in (1, 4096, 26214400):
        t8 = oracle.ring_allreduce_ns(8, p, a, be)
        for n in (2, 4, 8):
            assert oracle.allreduce_ns(k, n, p, a, be) == oracle.ring_allreduce_ns(n, p, a, be)
        for n in (16, 64, 1024):
            got = oracle.allreduce_ns(k, n, p, a, be)
            want = t8 * (2 * (n - 1) / n) / (2 * 7 / 8)
            assert got == -(-t8 * 8 * (n - 1) // (7 * n)) and abs(got - want) <= 1
            assert got < 8 * t8 / 7 + 1                       # bounded: tends to T(8) * 8/7
        assert oracle.allreduce_ns(0, 64, p, a, be) == oracle.ring_allreduce_ns(64, p, a, be)
    # end to end: pure DP on 16 devices with one bucket
    f, g = [5, 11, 3], [9, 20, 8]
    grad = np.array([1000, 555, 77], np.int64)
    T = make_table(f, g, n_devices=16, gpus_per_node=4, global_batch=16, classes=[(1, 1)], grad=grad,
                   dp_bucket_bytes=0, dp_overlap=0, alpha_intra_ns=3, beta_intra=16, alpha_inter_ns=40,
                   beta_inter=2, allreduce_profile_max=8)
    r = oracle.simulate(T, Candidate(1, 1, 16, 1, 0, (0, 3)))
    t8 = 2 * 7 * 40 + -(-2 * 7 * 1632 // (8 * 2))
    assert r.batch_ns == sum(f) + sum(g) + -(-t8 * 8 * 15 // (7 * 16))


def test_paper_grid_workload_shape():
    w = W.paper_grid()
    assert oracle.count(w.table, w.space) == 2 * sum(
        len([m for m in (1, 2, 4, 8, 16) if (16 // dp) % m == 0])
        for mp in (1, 2, 4, 8, 16) for pp in (1, 2, 4, 8, 16) if mp * pp <= 16 for dp in [16 // (mp * pp)])
    cands = oracle.enumerate_at(w.table, w.space, np.arange(oracle.count(w.table, w.space)))
    assert len({(c.mp, c.pp) for c in cands}) == 15           # Sec. 6: 15 valid settings of 25


def test_p2p_and_all_to_all_formulas():
    assert oracle.p2p_ns(1000, 7, 10) == 107
    assert oracle.p2p_ns(1001, 7, 10) == 108
    assert oracle.all_to_all_ns(4, 1000, 3, 5) == 3 * 3 + 150
    assert oracle.all_to_all_ns(1, 1000, 3, 5) == 0


# --------------------------------------------------------------------------- #
# P-1: uniform stages, zero comm, dp = 1: batch = (m + pp - 1)(t_f + t_b)

@pytest.mark.parametrize("sched", [0, 1])
@pytest.mark.parametrize("pp,m", [(1, 1), (2, 2), (4, 8), (8, 3), (4, 1), (16, 5), (2, 9)])
def test_uniform_pipeline_closed_form(pp, m, sched):
    tf, tb, per_stage = 7, 13, 3
    L = pp * per_stage
    T = make_table([tf] * L, [tb] * L, n_devices=pp, gpus_per_node=1, global_batch=m,
                   classes=[(1, 1)], alpha_intra_ns=0, alpha_inter_ns=0)
    r = oracle.simulate(T, Candidate(1, pp, 1, m, sched, balanced(L, pp)))
    assert r.batch_ns == (m + pp - 1) * per_stage * (tf + tb)
    assert (r.busy_ns == m * per_stage * (tf + tb)).all()


# P-2: pure data parallelism, one all-reduce after the last event
@pytest.mark.parametrize("n", [2, 4, 16])
def test_pure_data_parallel_closed_form(n):
    f, g = [5, 11, 3], [9, 20, 8]
    grad = np.array([1000, 555, 77], np.int64)
    T = make_table(f, g, n_devices=n, gpus_per_node=4, global_batch=n, classes=[(1, 1)],
                   grad=grad, dp_bucket_bytes=0, dp_overlap=0,
                   alpha_intra_ns=3, beta_intra=16, alpha_inter_ns=40, beta_inter=2)
    r = oracle.simulate(T, Candidate(1, 1, n, 1, 0, (0, 3)))
    a, be = (3, 16) if n <= 4 else (40, 2)
    S = int(grad.sum())
    expect = sum(f) + sum(g) + 2 * (n - 1) * a + -(-2 * (n - 1) * S // (n * be))
    assert r.batch_ns == expect
    assert (r.busy_ns == expect).all() and np.allclose(r.util, 1.0, rtol=0, atol=0)


# P-3: GPipe with per-stage-constant item times: identical-job flow-shop identity
@pytest.mark.parametrize("seed", range(6))
def test_gpipe_flow_shop_identity(seed):
    rng = np.random.default_rng(seed)
    pp, m, L = int(rng.integers(2, 6)), int(rng.integers(1, 7)), 11
    cuts = sorted(rng.choice(np.arange(1, L), pp - 1, replace=False).tolist())
    bounds = (0, *cuts, L)
    f = rng.integers(1, 50, L).tolist()
    g = rng.integers(1, 90, L).tolist()
    T = make_table(f, g, n_devices=pp, gpus_per_node=2, global_batch=m, classes=[(1, 1)],
                   seq=10, hidden=10, alpha_intra_ns=4, beta_intra=7, alpha_inter_ns=30, beta_inter=3)
    r = oracle.simulate(T, Candidate(1, pp, 1, m, 0, bounds))
    act = 1 * 10 * 10 * 2
    p2p = [(4 + -(-act // 7)) if (d // 2 == (d + 1) // 2) else (30 + -(-act // 3)) for d in range(pp - 1)]
    a = [sum(f[bounds[d]:bounds[d + 1]]) + (p2p[d] if d < pp - 1 else 0) for d in range(pp)]
    gg = [sum(g[bounds[d]:bounds[d + 1]]) + (p2p[d - 1] if d > 0 else 0) for d in range(pp)]
    for d in range(pp):
        rec = r.records[r.offsets[d]:r.offsets[d + 1]]
        for j in range(m):
            endF = rec[(rec[:, 2] == j) & np.isin(rec[:, 0], [0, 2, 4, 6])][:, 4].max()
            endB = rec[(rec[:, 2] == j) & np.isin(rec[:, 0], [1, 3, 5, 7])][:, 4].max()
            assert endF == sum(a[:d + 1]) + j * max(a[:d + 1])
            last_f = sum(a) + (m - 1) * max(a)
            assert endB == last_f + sum(gg[d:]) + j * max(gg[d:])


# P-4: no pipeline: m sequential forward+backward passes with their all-reduces
def test_single_stage_sum():
    f, g = [3, 4, 5], [6, 8, 10]
    T = make_table(f, g, n_devices=4, gpus_per_node=4, global_batch=8, classes=[(4, 2)], seq=3,
                   hidden=5, alpha_intra_ns=2, beta_intra=4)
    r = oracle.simulate(T, Candidate(4, 1, 1, 4, 1, (0, 3)))
    act = 2 * 3 * 5 * 2
    ar = 2 * 3 * 2 + -(-2 * 3 * 2 * act // (4 * 4))
    assert r.batch_ns == 4 * (sum(f) + sum(g) + 6 * ar)
    assert r.offsets[-1] == 4 * (4 * 2 * 3 * 2)    # 4 devices x 4 mb x (F,B) x 3 layers x (compute, AR)


# P-10: hand-worked examples (tests/golden/worked_pipeline_examples.txt)
def test_hand_worked_examples():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "worked_pipeline_examples.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 6
    for name, p2p, sched, batch, busy0, busy1 in rows:
        jit = {}
        if name == "W3":
            jit = dict(jitter_fwd_ns=np.array([[0, 0], [3, 0]]), jitter_bwd_ns=np.zeros((2, 2), np.int64))
        T = make_table([1, 1], [2, 2], n_devices=2, gpus_per_node=1, global_batch=2, classes=[(1, 1)],
                       alpha_intra_ns=int(p2p), alpha_inter_ns=int(p2p), **jit)
        r = oracle.simulate(T, Candidate(1, 2, 1, 2, int(sched), (0, 1, 2)))
        assert r.batch_ns == int(batch), name
        assert r.busy_ns.tolist() == [int(busy0), int(busy1)]
        assert r.util.tolist() == [int(busy0) / int(batch), int(busy1) / int(batch)]


# --------------------------------------------------------------------------- #
# P-6: brute-force longest path over the explicit event DAG, every record

def _tiny_cases():
    for seed in range(10):
        w = W.random_small(seed, n_devices=8, gpus_per_node=4, n_layers=4, global_batch=8,
                           mp_max=2, pp_max=4, m_list=(1, 2, 3), dp_overlap=seed % 2,
                           dp_bucket_bytes=0 if seed % 5 == 4 else 700)
        yield w


@pytest.mark.parametrize("w", list(_tiny_cases()), ids=lambda w: w.name)
def test_brute_force_longest_path(w):
    n = oracle.count(w.table, w.space)
    cands = oracle.enumerate_at(w.table, w.space, np.arange(n))
    assert any(c.pp == 4 and c.sched == 1 for c in cands)
    for c in cands:
        r = oracle.simulate(w.table, c, replicate=False)
        batch, lanes = longest_path_timeline(w.table, c)
        assert r.batch_ns == batch
        for d in range(c.pp):
            got = [tuple(x) for x in r.records[r.offsets[d]:r.offsets[d + 1]].tolist()]
            assert got == lanes[d], (c, d)


# asynchronous 1F1B: the 1F1B order without the gradient all-reduce events
@pytest.mark.parametrize("seed", range(20, 26))
def test_async_1f1b_is_1f1b_without_gradient_allreduce(seed):
    w = W.random_small(seed, n_devices=8, gpus_per_node=4, n_layers=4, global_batch=8, mp_max=2,
                       pp_max=4, m_list=(1, 2, 3, 5), dp_overlap=seed % 2,
                       dp_bucket_bytes=0 if seed % 3 == 2 else 700, sched_mask=7)
    n = oracle.count(w.table, w.space)
    cands = oracle.enumerate_at(w.table, w.space, np.arange(n))
    assert [c.sched for c in cands[:6]] == [0, 1, 2, 0, 1, 2]          # the schedule varies fastest
    seen_dp = False
    for i in range(0, n, 3):
        sync, asyn = cands[i + 1], cands[i + 2]
        assert (sync.sched, asyn.sched) == (1, 2) and sync.bounds == asyn.bounds and sync.m == asyn.m
        r1 = oracle.simulate(w.table, sync, replicate=True)
        r2 = oracle.simulate(w.table, asyn, replicate=True)
        ends = []
        for dev in range(w.table.n_devices):
            a = r1.records[r1.offsets[dev]:r1.offsets[dev + 1]]
            b = r2.records[r2.offsets[dev]:r2.offsets[dev + 1]]
            main = a[a[:, 0] != 8]
            assert (b == main).all()                                   # identical main lanes, no buckets
            assert r2.busy_ns[dev] == int((main[:, 4] - main[:, 3]).sum())
            ends.append(int(main[:, 4].max()))
        assert r2.batch_ns == max(ends) <= r1.batch_ns
        if sync.dp == 1:
            assert r2.batch_ns == r1.batch_ns
        else:
            seen_dp = True
        batch, lanes = longest_path_timeline(w.table, asyn)            # independent DAG without all-reduce nodes
        assert batch == r2.batch_ns
    assert seen_dp


# interleaved 1F1B (v model chunks per device): simulated for candidates given explicitly
@pytest.mark.parametrize("pp,v,groups", [(2, 2, 1), (2, 2, 3), (2, 4, 2), (4, 2, 1), (4, 3, 2), (8, 2, 3), (8, 4, 1), (16, 2, 2)])
def test_interleaved_uniform_closed_form(pp, v, groups):
    # Uniform virtual stages, no communication cost: the schedule's bubble is (pp - 1) items of
    # one chunk, 1 / v of the plain pipeline's: batch = (m v + pp - 1)(t_f + t_b) with per-chunk
    # item times.  Any slip in the item order shows up as a longer batch or a deadlock.
    tf, tb, per, m = 7, 13, 2, pp * groups
    L = pp * v * per
    T = make_table([tf] * L, [tb] * L, n_devices=pp, gpus_per_node=1, global_batch=m,
                   classes=[(1, 1)], alpha_intra_ns=0, alpha_inter_ns=0)
    r = oracle.simulate(T, Candidate(1, pp, 1, m, 3, tuple(j * per for j in range(pp * v + 1)), v))
    assert r.batch_ns == (m * v + pp - 1) * per * (tf + tb)
    assert (r.busy_ns == m * v * per * (tf + tb)).all()
    # the same model on the plain pipeline (v times longer stages) has the v times larger bubble
    plain = oracle.simulate(T, Candidate(1, pp, 1, m, 1, balanced(L, pp)))
    assert plain.batch_ns == (m + pp - 1) * v * per * (tf + tb) > r.batch_ns


def _interleaved_cases():
    for seed in range(12):
        rng = np.random.default_rng(700 + seed)
        pp, v = [(2, 2), (2, 3), (4, 2)][seed % 3]
        mp = 1 + seed % 2
        dp = [1, 2][(seed // 2) % 2]
        m = pp * int(rng.integers(1, 3))
        P = pp * v
        L = P + int(rng.integers(0, 4))
        cuts = sorted(rng.choice(np.arange(1, L), size=P - 1, replace=False).tolist())
        w = W.random_small(800 + seed, n_devices=pp * mp * dp, gpus_per_node=2, n_layers=L,
                           global_batch=dp * m * int(rng.integers(1, 3)), mp_max=2, pp_max=4, m_list=(m,),
                           dp_overlap=seed % 2, dp_bucket_bytes=0 if seed % 5 == 4 else 700)
        yield w, Candidate(mp, pp, dp, m, 3, (0, *cuts, L), v)


@pytest.mark.parametrize("w,cand", list(_interleaved_cases()), ids=lambda x: getattr(x, "name", None))
def test_interleaved_brute_force_and_invariants(w, cand):
    T = w.table
    r = oracle.simulate(T, cand, replicate=False)
    batch, lanes = longest_path_timeline(T, cand)          # independent DAG over virtual stages
    assert r.batch_ns == batch
    for d in range(cand.pp):
        got = [tuple(x) for x in r.records[r.offsets[d]:r.offsets[d + 1]].tolist()]
        assert got == lanes[d], (cand, d)
    # the scan order of the pick step (Algorithm 1) does not matter; replicas are identical
    assert oracle.simulate(T, cand, replicate=False, reverse_scan=True).batch_ns == r.batch_ns
    full = oracle.simulate(T, cand, replicate=True)
    assert full.batch_ns == r.batch_ns
    for rr in range(cand.dp):
        for d in range(cand.pp):
            for q in range(cand.mp):
                dev = (rr * cand.pp + d) * cand.mp + q
                a = full.records[full.offsets[dev]:full.offsets[dev + 1]]
                assert (a == r.records[r.offsets[d]:r.offsets[d + 1]]).all()
    # every device's main lane is serial and holds each (chunk, micro-batch) item once
    for d in range(cand.pp):
        a = r.records[r.offsets[d]:r.offsets[d + 1]]
        main = a[a[:, 0] != 8]
        assert (main[1:, 3] >= main[:-1, 4]).all()
        comp_f = main[main[:, 0] == 0]
        layers_d = [l for c in range(cand.v) for l in range(cand.bounds[c * cand.pp + d], cand.bounds[c * cand.pp + d + 1])]
        assert sorted(set(comp_f[:, 1].tolist())) == sorted(layers_d)
        assert len(comp_f) == cand.m * len(layers_d)
        if not T.dp_overlap or cand.dp == 1:
            assert r.busy_ns[d] == int((a[:, 4] - a[:, 3]).sum())
    assert r.batch_ns >= int(r.busy_ns.max())


def test_interleaved_rejects_what_the_schedule_does_not_define():
    T = make_table([5] * 8, [9] * 8, n_devices=2, gpus_per_node=2, global_batch=6, classes=[(1, 1), (1, 2), (1, 3)],
                   alpha_intra_ns=1, alpha_inter_ns=1, beta_intra=1, beta_inter=1)
    ok = Candidate(1, 2, 1, 6, 3, (0, 2, 4, 6, 8), 2)
    assert oracle.simulate(T, ok).batch_ns > 0
    with pytest.raises(Exception):
        oracle.simulate(T, Candidate(1, 2, 1, 3, 3, (0, 2, 4, 6, 8), 2))      # m is not a multiple of pp
    with pytest.raises(Exception):
        oracle.simulate(T, Candidate(1, 2, 1, 6, 3, (0, 4, 8), 2))            # bounds for pp stages, not pp * v


# --------------------------------------------------------------------------- #
# bidirectional pipelines (schedule 4)

@pytest.mark.parametrize("pp,groups", [(2, 1), (2, 3), (4, 1), (4, 2), (6, 1), (8, 1), (8, 3), (16, 1)])
def test_bidirectional_uniform_closed_form(pp, groups):
    # Equal forward and backward item times on uniform stages, no communication: the timeline is
    # the schedule's grid of unit slots, 2 m + pp - 2 of them - for m = pp the published property
    # of the schedule (pp - 2 idle slots per device, against 2 (pp - 1) of the plain pipeline) -
    # and every device is busy in 2 m of them.
    t, per, m = 11, 3, pp * groups
    L = pp * per
    T = make_table([t] * L, [t] * L, n_devices=pp, gpus_per_node=1, global_batch=m, classes=[(1, 1)],
                   alpha_intra_ns=0, alpha_inter_ns=0)
    r = oracle.simulate(T, Candidate(1, pp, 1, m, 4, balanced(L, pp)))
    assert r.batch_ns == (2 * m + pp - 2) * per * t
    assert (r.busy_ns == 2 * m * per * t).all()
    if groups == 1:
        assert r.batch_ns == (3 * pp - 2) * per * t
    plain = oracle.simulate(T, Candidate(1, pp, 1, m, 1, balanced(L, pp)))
    assert plain.batch_ns == 2 * (m + pp - 1) * per * t >= r.batch_ns
    # the device order used is the unit-slot order, restated independently as a token game
    order, slots = bidirectional_order(pp, m)
    assert slots == 2 * m + pp - 2
    for d in range(pp):
        a = r.records[r.offsets[d]:r.offsets[d + 1]]
        firsts = a[(a[:, 0] <= 1) & (a[:, 1] == np.where(a[:, 0] == 0, d * per, (d + 1) * per - 1))]
        # (the first layer event of each item of the device's stage in pipeline "down" ...)
        down = [(k, j) for (k, j, u) in order[d] if u == 0]
        assert [("F" if k == 0 else "B", j) for k, _, j in firsts[:, :3].tolist()] == down


def test_hand_worked_bidirectional_example():
    # tests/golden/worked_bidirectional_example.txt: four devices, four micro-batches, every item
    # one time unit, worked by hand on squared paper; rows "device slot kind micro-batch pipeline"
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "worked_bidirectional_example.txt"))
            if ln.strip() and not ln.startswith("#")]
    T = make_table([1] * 4, [1] * 4, n_devices=4, gpus_per_node=1, global_batch=4, classes=[(1, 1)],
                   alpha_intra_ns=0, alpha_inter_ns=0)
    r = oracle.simulate(T, Candidate(1, 4, 1, 4, 4, (0, 1, 2, 3, 4)))
    assert r.batch_ns == 10
    want = {d: [] for d in range(4)}
    for dev, slot, kind, mb, pipe in rows:
        d, u = int(dev), int(pipe)
        layer = d if u == 0 else 3 - d
        want[d].append((0 if kind == "F" else 1, layer, int(mb), int(slot), int(slot) + 1))
    for d in range(4):
        got = [tuple(x) for x in r.records[r.offsets[d]:r.offsets[d + 1]].tolist()]
        assert all(e[3] == e[4] for e in got if e[0] in (6, 7))              # transfers cost nothing here
        assert [e for e in got if e[0] <= 1] == sorted(want[d], key=lambda e: e[3]), d


def _bidirectional_cases():
    for seed in range(12):
        rng = np.random.default_rng(900 + seed)
        pp = [2, 4, 4, 6][seed % 4] if seed % 4 != 3 else 2
        mp = 1 + seed % 2
        dp = [1, 2][(seed // 2) % 2]
        m = 2 * int(rng.integers(1, 4))
        L = pp + int(rng.integers(0, 4))
        cuts = sorted(rng.choice(np.arange(1, L), size=pp - 1, replace=False).tolist())
        w = W.random_small(950 + seed, n_devices=pp * mp * dp, gpus_per_node=2, n_layers=L,
                           global_batch=dp * m * int(rng.integers(1, 3)), mp_max=2, pp_max=4, m_list=(m,),
                           dp_overlap=seed % 2, dp_bucket_bytes=0 if seed % 5 == 4 else 700)
        yield w, Candidate(mp, pp, dp, m, 4, (0, *cuts, L))


@pytest.mark.parametrize("w,cand", list(_bidirectional_cases()), ids=lambda x: getattr(x, "name", None))
def test_bidirectional_brute_force_and_invariants(w, cand):
    T = w.table
    r = oracle.simulate(T, cand, replicate=False)
    batch, lanes = longest_path_bidirectional(T, cand)     # independent DAG, order from the token game
    assert r.batch_ns == batch
    for d in range(cand.pp):
        got = [tuple(x) for x in r.records[r.offsets[d]:r.offsets[d + 1]].tolist()]
        assert got == lanes[d], (cand, d)
    assert oracle.simulate(T, cand, replicate=False, reverse_scan=True).batch_ns == r.batch_ns
    full = oracle.simulate(T, cand, replicate=True)
    assert full.batch_ns == r.batch_ns
    for rr in range(cand.dp):
        for d in range(cand.pp):
            for q in range(cand.mp):
                dev = (rr * cand.pp + d) * cand.mp + q
                a = full.records[full.offsets[dev]:full.offsets[dev + 1]]
                assert (a == r.records[r.offsets[d]:r.offsets[d + 1]]).all()
    for d in range(cand.pp):
        a = r.records[r.offsets[d]:r.offsets[d + 1]]
        main, buckets = a[a[:, 0] != 8], a[a[:, 0] == 8]
        assert (main[1:, 3] >= main[:-1, 4]).all() and (buckets[1:, 3] >= buckets[:-1, 4]).all()
        # the device runs every micro-batch of pipeline "down" through stage d and every one of
        # pipeline "up" through stage pp - 1 - d, forward and backward
        comp_f = main[main[:, 0] == 0]
        for u, s in ((0, d), (1, cand.pp - 1 - d)):
            mine = comp_f[comp_f[:, 1] == cand.bounds[s]]
            assert sorted(mine[:, 2].tolist()) == list(range(u * cand.m // 2, (u + 1) * cand.m // 2))
        # the weights of a stage are on two devices even without data parallelism: gradient
        # events whenever the stage has gradient bytes
        has_grad = any(T.grad_bytes[l] > 0 for s in (d, cand.pp - 1 - d) for l in range(cand.bounds[s], cand.bounds[s + 1]))
        assert (len(buckets) > 0) == has_grad
    assert r.batch_ns >= int(r.busy_ns.max())


def test_bidirectional_on_unequal_links():
    # six devices on nodes of four: the link between devices 3 and 4 is the slow one, so the two
    # pipelines cross it at different stages (pipeline "down" after its stage 3, pipeline "up"
    # after its stage 1), and the gradient groups {0, 5}, {1, 4} span nodes while {2, 3} does not
    T = make_table([5, 7, 4, 6, 8, 9, 3], [9, 11, 8, 7, 13, 12, 6], n_devices=6, gpus_per_node=4, global_batch=4,
                   classes=[(1, 1), (1, 2)], seq=16, hidden=8, alpha_intra_ns=3, alpha_inter_ns=50, beta_intra=64,
                   beta_inter=4, grad=np.array([100, 0, 300, 50, 0, 700, 20]), dp_bucket_bytes=256, dp_overlap=1)
    for m in (2, 4):
        c = Candidate(1, 6, 1, m, 4, (0, 1, 2, 3, 4, 5, 7))
        r = oracle.simulate(T, c, replicate=False)
        batch, lanes = longest_path_bidirectional(T, c)
        assert r.batch_ns == batch
        for d in range(6):
            assert [tuple(x) for x in r.records[r.offsets[d]:r.offsets[d + 1]].tolist()] == lanes[d], d
        sends = {d: sorted({(int(e[0]), int(e[4] - e[3])) for e in r.records[r.offsets[d]:r.offsets[d + 1]] if e[0] in (6, 7)})
                 for d in range(6)}
        slow, fast = 50 + -(-(4 // m) * 16 * 8 * 2 // 4), 3 + -(-(4 // m) * 16 * 8 * 2 // 64)
        assert sends[3] == [(6, fast), (6, slow), (7, fast), (7, slow)]      # forward down and backward up cross 3|4
        assert sends[0] == [(6, fast), (7, fast)] and sends[5] == [(6, fast), (7, fast)]


def test_bidirectional_rejects_what_the_schedule_does_not_define():
    T = make_table([5] * 8, [9] * 8, n_devices=4, gpus_per_node=2, global_batch=6, classes=[(1, 1), (1, 2), (1, 3), (1, 6)],
                   alpha_intra_ns=1, alpha_inter_ns=1, beta_intra=1, beta_inter=1)
    assert oracle.simulate(T, Candidate(1, 4, 1, 6, 4, (0, 2, 4, 6, 8))).batch_ns > 0
    with pytest.raises(Exception):
        oracle.simulate(T, Candidate(1, 4, 1, 3, 4, (0, 2, 4, 6, 8)))         # an odd number of micro-batches
    T1 = make_table([5] * 8, [9] * 8, n_devices=1, gpus_per_node=1, global_batch=6, classes=[(1, 1)],
                    alpha_intra_ns=1, alpha_inter_ns=1, beta_intra=1, beta_inter=1)
    with pytest.raises(Exception):
        oracle.simulate(T1, Candidate(1, 1, 1, 6, 4, (0, 8)))                  # one device: nothing to run against


# per-micro-batch jitter
def _jittered(seed, **kw):
    w = W.random_small(seed, n_devices=8, gpus_per_node=4, n_layers=4, global_batch=8, mp_max=2,
                       pp_max=4, m_list=(1, 2, 3, 5), dp_bucket_bytes=700, **kw)
    return W.add_jitter(w, 4, 900, seed)


@pytest.mark.parametrize("seed", range(60, 66))
def test_jitter_brute_force_longest_path(seed):
    w = _jittered(seed, dp_overlap=seed % 2)
    n = oracle.count(w.table, w.space)
    for c in oracle.enumerate_at(w.table, w.space, np.arange(n)):
        r = oracle.simulate(w.table, c, replicate=False)
        batch, lanes = longest_path_timeline(w.table, c)
        assert r.batch_ns == batch
        for d in range(c.pp):
            got = [tuple(x) for x in r.records[r.offsets[d]:r.offsets[d + 1]].tolist()]
            assert got == lanes[d], (c, d)


def test_jitter_special_cases():
    import copy
    w = _jittered(70)
    n = oracle.count(w.table, w.space)
    cands = oracle.enumerate_at(w.table, w.space, np.arange(0, n, 7))
    plain = copy.deepcopy(w.table); plain.jitter_fwd_ns = None; plain.jitter_bwd_ns = None
    zero = copy.deepcopy(w.table); zero.jitter_fwd_ns[:] = 0; zero.jitter_bwd_ns[:] = 0
    more = copy.deepcopy(w.table); more.jitter_fwd_ns[2, 1] += 55
    for c in cands:
        r0 = oracle.simulate(plain, c, replicate=False)
        rz = oracle.simulate(zero, c, replicate=False)
        rj = oracle.simulate(w.table, c, replicate=False)
        # an all-zero table changes no time; it only adds one zero-length event per item
        assert rz.batch_ns == r0.batch_ns and (rz.busy_ns == r0.busy_ns).all()
        keep = ~np.isin(rz.records[:, 0], [9, 10])
        assert (rz.records[keep] == r0.records).all()
        assert (~keep).sum() == 2 * c.m * c.pp and (rz.records[~keep, 4] == rz.records[~keep, 3]).all()
        # jitter only delays, and more jitter delays more
        assert rj.batch_ns >= r0.batch_ns
        assert oracle.simulate(more, c, replicate=False).batch_ns >= rj.batch_ns
        # busy time = sum of durations on the main lane (+ bucket excess): check the main lane
        for d in range(c.pp):
            rec = rj.records[rj.offsets[d]:rj.offsets[d + 1]]
            main = rec[rec[:, 0] != 8]
            jit = main[np.isin(main[:, 0], [9, 10])]
            want = sum(int(w.table.jitter_fwd_ns[j % 4, d]) + int(w.table.jitter_bwd_ns[j % 4, d]) for j in range(c.m))
            assert int((jit[:, 4] - jit[:, 3]).sum()) == want
    # constant jitter on uniform stages: the closed form with longer items
    pp, m, tf, tb, cj = 4, 6, 7, 13, 5
    T = make_table([tf] * pp, [tb] * pp, n_devices=pp, gpus_per_node=1, global_batch=m, classes=[(1, 1)],
                   alpha_intra_ns=0, alpha_inter_ns=0, jitter_fwd_ns=np.full((2, pp), cj),
                   jitter_bwd_ns=np.full((2, pp), cj))
    for sched in (0, 1):
        r = oracle.simulate(T, Candidate(1, pp, 1, m, sched, balanced(pp, pp)))
        assert r.batch_ns == (m + pp - 1) * (tf + tb + 2 * cj)


# --------------------------------------------------------------------------- #
# P-5: invariants

def _cases(seeds, **kw):
    for seed in seeds:
        w = W.random_small(seed, **kw)
        n = oracle.count(w.table, w.space)
        idx = np.unique(np.linspace(0, n - 1, 12).astype(np.int64))
        for c in oracle.enumerate_at(w.table, w.space, idx):
            yield w, c


def test_replicas_identical_busy_is_sum_and_batch_dominates():
    for w, c in _cases(range(20, 26)):
        r = oracle.simulate(w.table, c, replicate=True)
        red = oracle.simulate(w.table, c, replicate=False)
        rev = oracle.simulate(w.table, c, replicate=True, reverse_scan=True)
        assert r.batch_ns == red.batch_ns == rev.batch_ns
        assert (r.records == rev.records).all() and (r.offsets == rev.offsets).all()
        assert len(r.offsets) == w.table.n_devices + 1          # MP x PP x DP event lists (Sec. 4.3)
        for rr in range(c.dp):
            for d in range(c.pp):
                for q in range(c.mp):
                    k = (rr * c.pp + d) * c.mp + q                # Algorithm 1: F[d*MP + m_p]
                    a = r.records[r.offsets[k]:r.offsets[k + 1]]
                    bq = red.records[red.offsets[d]:red.offsets[d + 1]]
                    assert (a == bq).all()
                    assert r.busy_ns[k] == red.busy_ns[d]
        assert r.batch_ns >= r.busy_ns.max()
        assert (r.records[:, 4] >= r.records[:, 3]).all() and (r.records[:, 3] >= 0).all()
        assert r.records[:, 3].min() == 0                         # time origin: first item starts at 0


def test_busy_equals_sum_of_durations_without_overlap():
    for w, c in _cases(range(30, 34), dp_overlap=0):
        r = oracle.simulate(w.table, c, replicate=False)
        for d in range(c.pp):
            rec = r.records[r.offsets[d]:r.offsets[d + 1]]
            assert r.busy_ns[d] == int((rec[:, 4] - rec[:, 3]).sum())


def _coverage_measure(rec):
    """Measure of the union of the records' [start, end) intervals by a coverage count over the
    distinct end points (no sorting of intervals, no merging)."""
    pts = np.unique(np.concatenate([rec[:, 3], rec[:, 4]]))
    diff = np.zeros(len(pts) + 1, np.int64)
    np.add.at(diff, np.searchsorted(pts, rec[:, 3]), 1)
    np.add.at(diff, np.searchsorted(pts, rec[:, 4]), -1)
    covered = np.cumsum(diff)[:-1] > 0                      # segment [pts[i], pts[i+1])
    return int((np.diff(pts) * covered[:-1]).sum())


def _merge_that_forgets_the_running_end(rec):
    """The plausible mistake in an interval merge: the running end is overwritten by the next
    interval's end instead of the later of the two."""
    iv = sorted((int(s), int(e)) for s, e in rec[:, 3:5])
    total, lo, hi = 0, iv[0][0], iv[0][1]
    for s, e in iv[1:]:
        if s > hi:
            total += hi - lo; lo, hi = s, e
        else:
            hi = e
    return total + hi - lo


def test_busy_is_the_union_of_intervals_when_buckets_overlap_the_main_lane():
    # Sec. 3.2 activity time under DP modeling with overlapped buckets (dp > 1): buckets start
    # inside main-lane events, so the union is smaller than the sum of the durations.
    n_nested = n_strict = 0
    for w, c in _cases(range(70, 82), dp_overlap=1, dp_bucket_bytes=900, n_layers=6):
        if c.dp == 1 or c.sched == 2:
            continue
        r = oracle.simulate(w.table, c, replicate=False)
        for d in range(c.pp):
            rec = r.records[r.offsets[d]:r.offsets[d + 1]]
            main, bk = rec[rec[:, 0] != 8], rec[rec[:, 0] == 8]
            want = _coverage_measure(rec)
            assert r.busy_ns[d] == want, (c, d)
            # the same on a boolean time grid when it is small enough
            if rec[:, 4].max() < 4_000_000:
                grid = np.zeros(int(rec[:, 4].max()), bool)
                for s, e in rec[:, 3:5]:
                    grid[s:e] = True
                assert int(grid.sum()) == want
            # main lane without gaps after its first event, bucket lane busy after the main lane
            # ends: activity = sum of the main-lane durations + what the buckets add past its end
            main_sum = int((main[:, 4] - main[:, 3]).sum())
            dp_end = int(bk[:, 4].max()) if len(bk) else 0
            assert r.busy_ns[d] == main_sum + max(0, dp_end - int(main[:, 4].max())), (c, d)
            n_strict += r.busy_ns[d] < int((rec[:, 4] - rec[:, 3]).sum())
            n_nested += _merge_that_forgets_the_running_end(rec) != want
    assert n_strict >= 10 and n_nested >= 5      # the cases do exercise overlap and nesting


def test_hand_worked_bucket_overlap_examples():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "worked_bucket_overlap_examples.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 4
    for name, sched, overlap, batch, *busy in rows:
        if name == "W4":
            T = make_table([1, 1], [10, 10], n_devices=2, gpus_per_node=1, global_batch=2, classes=[(1, 1)],
                           grad=np.array([100, 200], np.int64), dp_bucket_bytes=100, dp_overlap=int(overlap),
                           alpha_intra_ns=50, beta_intra=1, alpha_inter_ns=1, beta_inter=100)
            c = Candidate(1, 1, 2, 1, int(sched), (0, 2))
        else:
            T = make_table([1, 1], [2, 2], n_devices=4, gpus_per_node=2, global_batch=4, classes=[(1, 1)],
                           grad=np.array([100, 200], np.int64), dp_bucket_bytes=100, dp_overlap=int(overlap),
                           alpha_intra_ns=7, beta_intra=1, alpha_inter_ns=1, beta_inter=100)
            c = Candidate(1, 2, 2, 2, int(sched), (0, 1, 2))
        r = oracle.simulate(T, c, replicate=False)
        assert r.batch_ns == int(batch), (name, sched)
        assert r.busy_ns.tolist() == [int(x) for x in busy], (name, sched)
        assert r.util.tolist() == [int(x) / int(batch) for x in busy]
        full = oracle.simulate(T, c, replicate=True)
        assert full.busy_ns.tolist() == [int(busy[(k // c.mp) % c.pp]) for k in range(T.n_devices)]


def test_main_lane_is_serial_and_bucket_lane_is_serial():
    for w, c in _cases(range(40, 44)):
        r = oracle.simulate(w.table, c, replicate=False)
        for d in range(c.pp):
            rec = r.records[r.offsets[d]:r.offsets[d + 1]]
            main, bk = rec[rec[:, 0] != 8], rec[rec[:, 0] == 8]
            assert (main[1:, 3] >= main[:-1, 4]).all()
            assert (bk[1:, 3] >= bk[:-1, 4]).all()
            assert (bk[:, 1] == np.arange(len(bk))).all() and (bk[:, 2] == -1).all()
            if c.dp == 1:
                assert len(bk) == 0


def _batch(table, c):
    return oracle.simulate(table, c, replicate=False, want_records=False).batch_ns


def test_monotone_in_durations_and_link_constants():
    import copy
    for w, c in _cases(range(50, 54)):
        base = _batch(w.table, c)
        rng = np.random.default_rng(w.seed)
        for _ in range(4):
            t = copy.deepcopy(w.table)
            k, l = int(rng.integers(t.n_classes)), int(rng.integers(t.n_layers))
            (t.fwd_ns if rng.integers(2) else t.bwd_ns)[:, l] += int(rng.integers(1, 5000))
            assert _batch(t, c) >= base
        for name, sign in (("alpha_intra_ns", 1), ("alpha_inter_ns", 1), ("beta_intra", -1), ("beta_inter", -1)):
            t = copy.deepcopy(w.table)
            setattr(t, name, getattr(t, name) + 3)
            assert sign * (_batch(t, c) - base) >= 0
        t = copy.deepcopy(w.table); t.dp_overlap = 0
        appended = _batch(t, c)
        assert appended >= base                                    # overlapping never hurts
        # gradient volume: monotone when every bucket waits for the end of the lane (with
        # overlap, more bytes can move a fixed-size bucket's last byte into an earlier layer)
        t.grad_bytes = t.grad_bytes + 999
        assert _batch(t, c) >= appended


# P-11: bucket properties
def test_bucket_chain_properties():
    f, g = [10, 10, 10, 10], [20, 20, 20, 20]
    grad = np.array([400, 400, 400, 400], np.int64)
    kw = dict(n_devices=4, gpus_per_node=4, global_batch=4, classes=[(1, 1), (1, 2)], grad=grad,
              alpha_intra_ns=1, beta_intra=1)
    # one layer per stage and bucket >= W_d: overlapped equals appended only for the first
    # stage (no trailing transfer there); with a transfer, overlap starts the bucket earlier.
    for bucket in (0, 400, 1000):
        Ta = make_table(f, g, dp_bucket_bytes=bucket, dp_overlap=1, **kw)
        Tb = make_table(f, g, dp_bucket_bytes=bucket, dp_overlap=0, **kw)
        c = Candidate(1, 2, 2, 1, 0, (0, 2, 4))
        ra, rb = oracle.simulate(Ta, c, replicate=False), oracle.simulate(Tb, c, replicate=False)
        a0 = ra.records[ra.offsets[0]:ra.offsets[1]]; b0 = rb.records[rb.offsets[0]:rb.offsets[1]]
        if bucket in (0, 1000):
            assert (a0 == b0).all()                                # stage 0: last layer ends the lane
    # identical ready times: K full buckets back to back = K * T_full
    T0 = make_table(f, g, dp_bucket_bytes=100, dp_overlap=0, **kw)
    r = oracle.simulate(T0, Candidate(1, 1, 4, 1, 0, (0, 4)), replicate=False)
    bk = r.records[r.records[:, 0] == 8]
    t_full = oracle.ring_allreduce_ns(4, 100, 1, 1)
    assert len(bk) == 16 and (bk[:, 4] - bk[:, 3] == t_full).all()
    assert bk[-1, 4] - bk[0, 3] == 16 * t_full
    # partial last bucket carries the remainder
    T1 = make_table(f, g, dp_bucket_bytes=300, dp_overlap=1, **kw)
    r = oracle.simulate(T1, Candidate(1, 1, 4, 1, 0, (0, 4)), replicate=False)
    bk = r.records[r.records[:, 0] == 8]
    assert len(bk) == 6 and bk[-1, 4] - bk[-1, 3] == oracle.ring_allreduce_ns(4, 100, 1, 1)
    # bucket k (bytes [300k, 300k+300)) ends inside layer 3 - (300k+299)//400; ready when that
    # layer's backward of the last microbatch ends; layers run 3,2,1,0 taking 20 ns each after
    # the forward pass (40 ns)
    fwd_end = 40
    prev = 0
    for k in range(6):
        last = min(300 * k + 299, 1599)
        ready = fwd_end + 20 * (last // 400 + 1)
        start = max(ready, prev)
        assert bk[k, 3] == start
        prev = bk[k, 4]


# --------------------------------------------------------------------------- #
# enumeration pins

def test_paper_grid_has_15_valid_settings():
    # Sec. 6: degrees {1,2,4,8,16} on 16 GPUs -> 15 valid (mp, pp) settings, dp = GPUs/mp/pp
    sp = W.SearchSpace(mp_max=16, pp_max=16, m_list=[1], sched_mask=1)
    T = make_table([1] * 48, [1] * 48, n_devices=16, gpus_per_node=4, global_batch=16, classes=[(1, 1)])
    n = oracle.count(T, sp)
    assert n == 15
    cands = oracle.enumerate_at(T, sp, np.arange(n))
    assert len({(c.mp, c.pp) for c in cands}) == 15
    assert all(c.mp * c.pp * c.dp == 16 for c in cands)


def test_paper_per_stage_example_item_counts():
    # Sec. 5.4: "2m4p1d", 4 micro-batches -> 32 forward and backward items, 4 (each) per GPU
    T = make_table([5] * 8, [9] * 8, n_devices=8, gpus_per_node=4, global_batch=4, classes=[(2, 1)],
                   seq=4, hidden=4)
    for sched in (0, 1):
        r = oracle.simulate(T, Candidate(2, 4, 1, 4, sched, (0, 2, 4, 6, 8)))
        assert len(r.offsets) == 9
        tot_f = tot_b = 0
        for k in range(8):
            rec = r.records[r.offsets[k]:r.offsets[k + 1]]
            first_layer = (k // 2) * 2
            nf = int(((rec[:, 0] == 0) & (rec[:, 1] == first_layer)).sum())
            nb = int(((rec[:, 0] == 1) & (rec[:, 1] == first_layer)).sum())
            assert nf == 4 and nb == 4
            tot_f += nf; tot_b += nb
        assert tot_f == 32 and tot_b == 32
        # the two GPUs of an MP group behave identically (Sec. 5.4)
        for k in range(0, 8, 2):
            assert (r.records[r.offsets[k]:r.offsets[k + 1]] == r.records[r.offsets[k + 1]:r.offsets[k + 2]]).all()


def test_composition_count_and_lexicographic_order():
    L = 9
    T = make_table([1] * L, [1] * L, n_devices=4, gpus_per_node=4, global_batch=4, classes=[(1, 1), (1, 2), (1, 4)])
    sp = W.SearchSpace(mp_max=1, pp_max=4, m_list=[1], partition_mode=W.PARTITION_ALL, sched_mask=2)
    n = oracle.count(T, sp)
    assert n == sum(math.comb(L - 1, pp - 1) for pp in (1, 2, 4))
    cands = oracle.enumerate_at(T, sp, np.arange(n))
    expect = []
    for pp in (1, 2, 4):
        for cut in itertools.combinations(range(1, L), pp - 1):     # lexicographic
            expect.append((pp, (0, *cut, L)))
    assert [(c.pp, c.bounds) for c in cands] == expect


def test_canonical_order_against_python_loops():
    for cfg in (0, 2):
        w = W.CONFIGS[cfg]()
        T, sp = w.table, w.space
        expect = []
        mp = 1
        while mp <= sp.mp_max:
            pp = 1
            while pp <= min(sp.pp_max, T.n_layers):
                if T.n_devices % (mp * pp) == 0 and T.global_batch % (T.n_devices // (mp * pp)) == 0:
                    dp = T.n_devices // (mp * pp)
                    bp = T.global_batch // dp
                    for m in sp.m_list.tolist():
                        ok = m <= bp and (bp % m == 0 if sp.m_rule == 0 else True)
                        if ok:
                            for sc in (0, 1):
                                expect.append((mp, pp, dp, m, sc, balanced(T.n_layers, pp)))
                pp *= 2
            mp *= 2
        n = oracle.count(T, sp)
        assert n == len(expect) == {0: 88, 2: 4176}[cfg]
        got = oracle.enumerate_at(T, sp, np.arange(n))
        assert [(c.mp, c.pp, c.dp, c.m, c.sched, c.bounds) for c in got] == expect


def test_canonical_order_with_interleaved_rows():
    # every (mp, pp) is followed by its interleaved candidates: v ascending over powers of two, m
    # among the multiples of pp, partitions of the layers into pp * v virtual stages in
    # lexicographic order
    for mask, mode in ((15, W.PARTITION_ALL), (8, W.PARTITION_ALL), (11, W.PARTITION_BALANCED),
                       (31, W.PARTITION_ALL), (16, W.PARTITION_ALL), (19, W.PARTITION_BALANCED)):
        w = W.random_small(5, n_devices=8, gpus_per_node=4, n_layers=9, global_batch=16, mp_max=2, pp_max=4,
                           m_list=(1, 2, 4, 6, 8), partition_mode=mode, sched_mask=mask, v_max=4)
        T, sp = w.table, w.space
        L = T.n_layers
        expect = []
        for mp in (1, 2):
            for pp in (1, 2, 4):
                dp = T.n_devices // (mp * pp)
                if T.global_batch % dp:
                    continue
                bp = T.global_batch // dp
                ms = [m for m in sp.m_list.tolist() if m <= bp]
                parts = (lambda P: [balanced(L, P)] if mode == W.PARTITION_BALANCED else
                         [(0, *c, L) for c in itertools.combinations(range(1, L), P - 1)])
                for m in ms:
                    for b in parts(pp):
                        for sc in (0, 1, 2):
                            if mask & (1 << sc):
                                expect.append((mp, pp, dp, m, sc, b, 1))
                if pp >= 2 and mask & 8:
                    for v in (2, 4):
                        if pp * v > L:
                            continue
                        for m in ms:
                            if m % pp == 0:
                                expect += [(mp, pp, dp, m, 3, b, v) for b in parts(pp * v)]
                # ... and then by its bidirectional candidates: even m, partitions into pp stages
                if pp >= 2 and mask & 16:
                    for m in ms:
                        if m % 2 == 0:
                            expect += [(mp, pp, dp, m, 4, b, 1) for b in parts(pp)]
        n = oracle.count(T, sp)
        assert n == len(expect) == W.count_candidates_and_cells(T, sp)[0] and any(e[4] >= 3 for e in expect)
        got = oracle.enumerate_at(T, sp, np.arange(n))
        assert [(c.mp, c.pp, c.dp, c.m, c.sched, c.bounds, c.v) for c in got] == expect
        # and the enumerated interleaved candidates simulate like the same candidates given explicitly
        for c in [c for c in got if c.sched >= 3][::7]:
            b, _ = oracle.eval_indices(T, sp, np.array([got.index(c)]))
            assert b[0] == oracle.simulate(T, c, replicate=False, want_records=False).batch_ns


def test_candidate_counts_of_the_benchmark_spaces():
    assert oracle.count(W.config1().table, W.config1().space) == 38_838_764
    assert oracle.count(W.config3().table, W.config3().space) == 650_420


def test_locality_of_collectives():
    w = W.config0()
    cands = oracle.enumerate_at(w.table, w.space, np.arange(88))
    T = w.table
    for c in cands:
        if c.m != 1 or c.sched != 0:
            continue
        r = oracle.simulate(T, c, replicate=False)
        rec = r.records
        b = T.global_batch // c.dp
        act = b * T.seq * T.hidden * 2
        ar = rec[rec[:, 0] == KINDS["MP_AR_F"]]
        if c.mp > 1:
            inter = c.mp > T.gpus_per_node                  # 8-way MP spans both 4-GPU nodes
            a, be = (T.alpha_inter_ns, T.beta_inter) if inter else (T.alpha_intra_ns, T.beta_intra)
            assert (ar[:, 4] - ar[:, 3] == oracle.ring_allreduce_ns(c.mp, 2 * act, a, be)).all()
        else:
            assert len(ar) == 0
        snd = rec[rec[:, 0] == KINDS["SEND_F"]]
        for row in snd:
            d = list(c.bounds).index(row[1] + 1) - 1
            inter = (d * c.mp) // 4 != ((d + 1) * c.mp) // 4
            a, be = (T.alpha_inter_ns, T.beta_inter) if inter else (T.alpha_intra_ns, T.beta_intra)
            assert row[4] - row[3] == oracle.p2p_ns(act, a, be)


def test_errors():
    T = make_table([1, 1], [1, 1], n_devices=2, gpus_per_node=1, global_batch=2, classes=[(1, 1)])
    with pytest.raises(oracle.OracleError):
        oracle.simulate(T, Candidate(1, 2, 1, 1, 0, (0, 1, 2)))      # class (1, 2) missing
    with pytest.raises(oracle.OracleError):
        oracle.simulate(T, Candidate(1, 2, 1, 2, 0, (0, 2, 2)))      # empty stage
    with pytest.raises(oracle.OracleError):
        oracle.simulate(T, Candidate(1, 1, 1, 2, 0, (0, 2)))         # degrees do not multiply to N
