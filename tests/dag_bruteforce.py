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


def interleaved_order(pp, v, d, m):
    """('F'|'B', j, chunk) in the order device d runs them under interleaved 1F1B: micro-batches
    go in groups of pp; a group passes chunk 0, 1, .. forward and v-1, v-2, .. backward.  The
    device launches forwards until the first micro-batch can have come back to it through all
    later devices and chunks (all of them when there is a single group), then alternates."""
    fseq = [(c, g * pp + i) for g in range(m // pp) for c in range(v) for i in range(pp)]
    bseq = [(c, g * pp + i) for g in range(m // pp) for c in reversed(range(v)) for i in range(pp)]
    warm = len(fseq) if m == pp else min(len(fseq), 2 * (pp - d - 1) + (v - 1) * pp)
    order = [("F", j, c) for (c, j) in fseq[:warm]]
    rest_f, b = fseq[warm:], list(bseq)
    while rest_f:
        c, j = rest_f.pop(0); order.append(("F", j, c))
        c, j = b.pop(0); order.append(("B", j, c))
    order += [("B", j, c) for (c, j) in b]
    return order


def longest_path_timeline(table, cand):
    """Returns (batch_ns, {stage d: [(kind, layer, mb, start, end), ...] main lane then buckets})."""
    T = table
    pp, mp, dp, m = cand.pp, cand.mp, cand.dp, cand.m
    v = cand.v if cand.sched == 3 else 1       # model chunks per device
    P = pp * v                                  # virtual stages; stage vs = chunk * pp + device
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
    for vs in range(P - 1):
        a, be = ab(rank(0, vs % pp, 0) // G != rank(0, (vs + 1) % pp, 0) // G)
        P2P.append(a + ceil_div(act, be))

    # nodes: id -> (duration, [predecessor ids]); names are tuples
    dur, preds, label = {}, {}, {}
    first_of_op, last_of_op = {}, {}
    layer_done = {}                      # (d, layer) -> node id finishing that layer in B(d, m-1)
    lane = {d: [] for d in range(pp)}
    for d in range(pp):
        prev = None
        items = (interleaved_order(pp, v, d, m) if cand.sched == 3
                 else [(typ, j, 0) for (typ, j) in stage_order(cand.sched, pp, d, m)])
        for (typ, j, ch) in items:
            evs = []
            vs = ch * pp + d
            layers = range(c[vs], c[vs + 1]) if typ == "F" else range(c[vs + 1] - 1, c[vs] - 1, -1)
            jt = getattr(T, "jitter_fwd_ns" if typ == "F" else "jitter_bwd_ns", None)
            if jt is not None:
                evs.append((9 if typ == "F" else 10, layers[0], int(jt[j % len(jt)][d])))
            for l in layers:
                evs.append((0 if typ == "F" else 1, l, f[l] if typ == "F" else g[l]))
                if mp > 1:
                    evs.append((2 if typ == "F" else 3, l, AR))
                if T.layer_is_expert[l] and dp > 1:
                    evs.append((4 if typ == "F" else 5, l, A2A))
            if typ == "F" and vs < P - 1:
                evs.append((6, c[vs + 1] - 1, P2P[vs]))
            if typ == "B" and vs > 0:
                evs.append((7, c[vs], P2P[vs - 1]))
            for i, (kind, l, du) in enumerate(evs):
                nid = (vs, typ, j, i)
                dur[nid] = du
                preds[nid] = [prev] if prev is not None else []
                label[nid] = (kind, l, j)
                lane[d].append(nid)
                if i == 0:
                    first_of_op[(vs, typ, j)] = nid
                if typ == "B" and j == m - 1 and kind in (1, 3, 5):
                    layer_done[(d, l)] = nid
                prev = nid
            last_of_op[(vs, typ, j)] = prev
    # data edges between neighbouring (virtual) stages
    for vs in range(P):
        for j in range(m):
            if vs > 0:
                preds[first_of_op[(vs, "F", j)]].append(last_of_op[(vs - 1, "F", j)])
            if vs < P - 1:
                preds[first_of_op[(vs, "B", j)]].append(last_of_op[(vs + 1, "B", j)])
            else:
                preds[first_of_op[(vs, "B", j)]].append(last_of_op[(vs, "F", j)])
    # gradient buckets on a separate lane
    buckets = {d: [] for d in range(pp)}
    if dp > 1 and cand.sched != 2:       # the asynchronous schedule has no gradient all-reduce
        a, be = ab(dp_inter)
        for d in range(pp):
            k, prevb = 0, None                  # one lane per device; bucket numbers run on over the chunks
            for ch in reversed(range(v)):       # a stream per chunk, the chunk whose last backward runs first first
                vs = ch * pp + d
                stream = [(l, ceil_div(int(T.grad_bytes[l]), mp)) for l in range(c[vs + 1] - 1, c[vs] - 1, -1)]
                W = sum(x[1] for x in stream)
                if W == 0:
                    continue
                size = T.dp_bucket_bytes if T.dp_bucket_bytes > 0 else W
                lo = 0
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


# ---- bidirectional pipelines (schedule 4) ----------------------------------------------------------

def bidirectional_order(pp, m):
    """[device] -> [('F'|'B', micro-batch, pipeline)] in the order the device runs them.

    Restated as a token game on a grid of unit time slots: pipeline 0 runs down the devices with
    micro-batches 0 .. m/2-1, pipeline 1 runs up with m/2 .. m-1, each keeps its own 1F1B order
    ("forward while fewer than min(pp - stage, m/2) of its micro-batches are in flight, else
    backward"), and in every slot a device runs, of its two pipelines' next items, one whose input
    existed before the slot began - the earlier micro-batch of its pipeline first (a tie, which
    does not occur, would go to a backward item, then to pipeline 0)."""
    half = m // 2
    stage = lambda d, u: d if u == 0 else pp - 1 - d
    queue = {}
    for d in range(pp):
        for u in (0, 1):
            cap, first = min(pp - stage(d, u), half), u * half
            q, nf, nb = [], 0, 0
            while nb < half:
                if nf < half and nf - nb < cap:
                    q.append(("F", first + nf)); nf += 1
                else:
                    q.append(("B", first + nb)); nb += 1
            queue[(d, u)] = q
    done = {}                                  # (pipeline, stage, kind, micro-batch) -> slot after it ran
    order = {d: [] for d in range(pp)}
    slot = 0
    while any(queue.values()):
        chosen = []
        for d in range(pp):
            options = []
            for u in (0, 1):
                if not queue[(d, u)]:
                    continue
                kind, j = queue[(d, u)][0]
                s = stage(d, u)
                if kind == "F":
                    need = None if s == 0 else (u, s - 1, "F", j)
                else:
                    need = (u, s, "F", j) if s == pp - 1 else (u, s + 1, "B", j)
                if need is None or done.get(need, slot + 1) <= slot:
                    options.append((j - u * half, kind != "B", u, kind, j))
            if options:
                chosen.append((d,) + min(options)[2:])
        assert chosen, "the token game is stuck"
        for d, u, kind, j in chosen:
            queue[(d, u)].pop(0)
            done[(u, stage(d, u), kind, j)] = slot + 1
            order[d].append((kind, j, u))
        slot += 1
    return order, slot


def longest_path_bidirectional(table, cand):
    """As longest_path_timeline, for the bidirectional schedule: (batch_ns, {device: records})."""
    T = table
    pp, mp, dp, m = cand.pp, cand.mp, cand.dp, cand.m
    c, G = cand.bounds, T.gpus_per_node
    b = ceil_div(T.global_batch // dp, m)
    kappa = [k for k in range(len(T.class_mp)) if T.class_mp[k] == mp and T.class_b[k] == b][0]
    f = [int(x) for x in T.fwd_ns[kappa]]
    g = [int(x) for x in T.bwd_ns[kappa]]
    act = b * T.seq * T.hidden * T.act_bytes_per_elem
    rank = lambda r, d, q: (r * pp + d) * mp + q
    ab = lambda inter: (T.alpha_inter_ns, T.beta_inter) if inter else (T.alpha_intra_ns, T.beta_intra)
    AR = A2A = 0
    if mp > 1:
        a, be = ab(len({rank(0, 0, q) // G for q in range(mp)}) > 1)
        AR = 2 * (mp - 1) * a + ceil_div(2 * (mp - 1) * 2 * act, mp * be)
    if dp > 1:
        a, be = ab(len({rank(r, 0, 0) // G for r in range(dp)}) > 1)
        A2A = (dp - 1) * a + ceil_div((dp - 1) * act, dp * be)
    link = []                                   # transfer across the boundary between devices a and a + 1
    for a_dev in range(pp - 1):
        a, be = ab(rank(0, a_dev, 0) // G != rank(0, a_dev + 1, 0) // G)
        link.append(a + ceil_div(act, be))
    stage = lambda d, u: d if u == 0 else pp - 1 - d
    device = stage                              # the map is its own inverse
    order, _ = bidirectional_order(pp, m)

    dur, preds, label = {}, {}, {}
    first_of, last_of, layer_done = {}, {}, {}
    lane = {d: [] for d in range(pp)}
    last_mb = {0: m // 2 - 1, 1: m - 1}
    for d in range(pp):
        prev = None
        for (typ, j, u) in order[d]:
            s = stage(d, u)
            layers = range(c[s], c[s + 1]) if typ == "F" else range(c[s + 1] - 1, c[s] - 1, -1)
            evs = []
            for l in layers:
                evs.append((0 if typ == "F" else 1, l, f[l] if typ == "F" else g[l]))
                if mp > 1:
                    evs.append((2 if typ == "F" else 3, l, AR))
                if T.layer_is_expert[l] and dp > 1:
                    evs.append((4 if typ == "F" else 5, l, A2A))
            if typ == "F" and s < pp - 1:       # to the device of the pipeline's next stage
                evs.append((6, c[s + 1] - 1, link[min(d, device(s + 1, u))]))
            if typ == "B" and s > 0:
                evs.append((7, c[s], link[min(d, device(s - 1, u))]))
            for i, (kind, l, du) in enumerate(evs):
                nid = (u, s, typ, j, i)
                dur[nid], preds[nid], label[nid] = du, ([prev] if prev is not None else []), (kind, l, j)
                lane[d].append(nid)
                if i == 0:
                    first_of[(u, s, typ, j)] = nid
                if typ == "B" and j == last_mb[u] and kind in (1, 3, 5):
                    layer_done[(d, l)] = nid
                prev = nid
            last_of[(u, s, typ, j)] = prev
    for u in (0, 1):
        for s in range(pp):
            for j in range(u * (m // 2), (u + 1) * (m // 2)):
                if s > 0:
                    preds[first_of[(u, s, "F", j)]].append(last_of[(u, s - 1, "F", j)])
                if s < pp - 1:
                    preds[first_of[(u, s, "B", j)]].append(last_of[(u, s + 1, "B", j)])
                else:
                    preds[first_of[(u, s, "B", j)]].append(last_of[(u, s, "F", j)])
    # gradients of a stage are reduced over the 2 dp devices holding it (both pipelines, every
    # replica); a device's two streams share its one lane, the later stage's stream first
    buckets = {d: [] for d in range(pp)}
    n = 2 * dp
    for d in range(pp):
        members = [rank(r, dd, 0) for r in range(dp) for dd in (d, pp - 1 - d)]
        a, be = ab(len({x // G for x in members}) > 1)
        k, prevb = 0, None
        for s in sorted((d, pp - 1 - d), reverse=True):
            stream = [(l, ceil_div(int(T.grad_bytes[l]), mp)) for l in range(c[s + 1] - 1, c[s] - 1, -1)]
            Wt = sum(x[1] for x in stream)
            if Wt == 0:
                continue
            size = T.dp_bucket_bytes if T.dp_bucket_bytes > 0 else Wt
            lo = 0
            while lo < Wt:
                hi = min(Wt, lo + size)
                pos, owner = 0, None
                for (l, gl) in stream:
                    if pos <= hi - 1 < pos + gl:
                        owner = l
                    pos += gl
                nid = (d, "G", k, 0)
                dur[nid] = 2 * (n - 1) * a + ceil_div(2 * (n - 1) * (hi - lo), n * be)
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

    out, batch = {}, 0
    for d in range(pp):
        recs = []
        for nid in lane[d] + buckets[d]:
            kk, l, j = label[nid]
            recs.append((kk, l, j, start(nid), end(nid)))
            batch = max(batch, end(nid))
        out[d] = recs
    return batch, out
