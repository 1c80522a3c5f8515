"""Independent brute-force pin for the oracle (tiny cases only).

Builds the explicit event DAG of one candidate - every computation, all-reduce,
all-to-all, transfer and gradient-bucket event is a node; edges are device order
and data dependencies - and finds every event's start as the longest path into
it by exhaustive memoised depth-first search.  It does not share a line with the
oracle: the 1F1B order is restated as "greedy under an activation cap" (a stage
runs a forward whenever fewer than min(pp - d, m) micro-batches are in flight,
else a backward), costs are written directly from the alpha-beta formulas, and
locality is worked out per pair of ranks.
"""
import sys
from functools import lru_cache


def ceil_div(a, b):
    return -(-a // b)


def stage_order(sched, pp, d, m):
    """List of ('F'|'B', j) in the order stage d executes them."""
    if sched == 0:
        return [("F", j) for j in range(m)] + [("B", j) for j in range(m)]
    cap = min(pp - d, m)
    order, nf, nb = [], 0, 0
    while nb < m:
        if nf < m and nf - nb < cap:
            order.append(("F", nf)); nf += 1
        else:
            order.append(("B", nb)); nb += 1
    return order


def longest_path_timeline(table, cand):
    """Returns (batch_ns, {stage d: [(kind, layer, mb, start, end), ...] main lane then buckets})."""
    T = table
    pp, mp, dp, m = cand.pp, cand.mp, cand.dp, cand.m
    c = cand.bounds
    G = T.gpus_per_node
    Bp = T.global_batch // dp
    b = ceil_div(Bp, m)
    kappa = [k for k in range(len(T.class_mp)) if T.class_mp[k] == mp and T.class_b[k] == b][0]
    f = [int(v) for v in T.fwd_ns[kappa]]
    g = [int(v) for v in T.bwd_ns[kappa]]
    act = b * T.seq * T.hidden * T.act_bytes_per_elem

    def rank(r, d, q):
        return (r * pp + d) * mp + q

    def ab(inter):
        return (T.alpha_inter_ns, T.beta_inter) if inter else (T.alpha_intra_ns, T.beta_intra)

    # locality for replica r = 0, q = 0 (tiny power-of-two cases: all replicas agree)
    mp_inter = len({rank(0, 0, q) // G for q in range(mp)}) > 1
    dp_inter = len({rank(r, 0, 0) // G for r in range(dp)}) > 1
    AR = 0
    if mp > 1:
        a, be = ab(mp_inter)
        AR = 2 * (mp - 1) * a + ceil_div(2 * (mp - 1) * 2 * act, mp * be)
    A2A = 0
    if dp > 1:
        a, be = ab(dp_inter)
        A2A = (dp - 1) * a + ceil_div((dp - 1) * act, dp * be)
    P2P = []
    for d in range(pp - 1):
        a, be = ab(rank(0, d, 0) // G != rank(0, d + 1, 0) // G)
        P2P.append(a + ceil_div(act, be))

    # nodes: id -> (duration, [predecessor ids]); names are tuples
    dur, preds, label = {}, {}, {}
    first_of_op, last_of_op = {}, {}
    layer_done = {}                      # (d, layer) -> node id finishing that layer in B(d, m-1)
    lane = {d: [] for d in range(pp)}
    for d in range(pp):
        prev = None
        for (typ, j) in stage_order(cand.sched, pp, d, m):
            evs = []
            layers = range(c[d], c[d + 1]) if typ == "F" else range(c[d + 1] - 1, c[d] - 1, -1)
            jt = getattr(T, "jitter_fwd_ns" if typ == "F" else "jitter_bwd_ns", None)
            if jt is not None:
                evs.append((9 if typ == "F" else 10, layers[0], int(jt[j % len(jt)][d])))
            for l in layers:
                evs.append((0 if typ == "F" else 1, l, f[l] if typ == "F" else g[l]))
                if mp > 1:
                    evs.append((2 if typ == "F" else 3, l, AR))
                if T.layer_is_expert[l] and dp > 1:
                    evs.append((4 if typ == "F" else 5, l, A2A))
            if typ == "F" and d < pp - 1:
                evs.append((6, c[d + 1] - 1, P2P[d]))
            if typ == "B" and d > 0:
                evs.append((7, c[d], P2P[d - 1]))
            for i, (kind, l, du) in enumerate(evs):
                nid = (d, typ, j, i)
                dur[nid] = du
                preds[nid] = [prev] if prev is not None else []
                label[nid] = (kind, l, j)
                lane[d].append(nid)
                if i == 0:
                    first_of_op[(d, typ, j)] = nid
                if typ == "B" and j == m - 1 and kind in (1, 3, 5):
                    layer_done[(d, l)] = nid
                prev = nid
            last_of_op[(d, typ, j)] = prev
    # data edges
    for d in range(pp):
        for j in range(m):
            if d > 0:
                preds[first_of_op[(d, "F", j)]].append(last_of_op[(d - 1, "F", j)])
            if d < pp - 1:
                preds[first_of_op[(d, "B", j)]].append(last_of_op[(d + 1, "B", j)])
            else:
                preds[first_of_op[(d, "B", j)]].append(last_of_op[(d, "F", j)])
    # gradient buckets on a separate lane
    buckets = {d: [] for d in range(pp)}
    if dp > 1 and cand.sched != 2:       # the asynchronous schedule has no gradient all-reduce
        a, be = ab(dp_inter)
        for d in range(pp):
            stream = [(l, ceil_div(int(T.grad_bytes[l]), mp)) for l in range(c[d + 1] - 1, c[d] - 1, -1)]
            W = sum(x[1] for x in stream)
            if W == 0:
                continue
            size = T.dp_bucket_bytes if T.dp_bucket_bytes > 0 else W
            k, lo, prevb = 0, 0, None
            while lo < W:
                hi = min(W, lo + size)
                pos, owner = 0, None
                for (l, gl) in stream:
                    if pos <= hi - 1 < pos + gl:
                        owner = l
                    pos += gl
                nid = (d, "G", k, 0)
                dur[nid] = 2 * (dp - 1) * a + ceil_div(2 * (dp - 1) * (hi - lo), dp * be)
                ready = layer_done[(d, owner)] if T.dp_overlap else lane[d][-1]
                preds[nid] = [ready] + ([prevb] if prevb is not None else [])
                label[nid] = (8, k, -1)
                buckets[d].append(nid)
                prevb = nid
                k += 1
                lo = hi

    sys.setrecursionlimit(max(10000, 4 * len(dur) + 1000))

    @lru_cache(maxsize=None)
    def end(nid):
        return start(nid) + dur[nid]

    @lru_cache(maxsize=None)
    def start(nid):
        return max([end(p) for p in preds[nid]], default=0)

    out = {}
    batch = 0
    for d in range(pp):
        recs = []
        for nid in lane[d] + buckets[d]:
            k, l, j = label[nid]
            recs.append((k, l, j, start(nid), end(nid)))
            batch = max(batch, end(nid))
        out[d] = recs
    return batch, out
