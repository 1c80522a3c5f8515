/*
 * distsim_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-threaded CPU restatement of DistSim's hierarchical
 * modeling (paper Sec. 4.3): MP modeling, PP modeling (Algorithm 1, run as a
 * literal worklist over explicit event objects), DP modeling, and the timeline
 * analyses (batch time, per-device busy time, utilisation; paper Sec. 3.2).
 * It exists so that the CUDA engine can be compared against something that can
 * be checked against the paper by eye.  It shares no code, header, table or
 * helper with the CUDA path and must never be called from the product path:
 * only the test-suite, the smoke check and the benchmark's CPU-baseline leg
 * may build, load or run it.
 *
 * Nothing here is blocked, fused, vectorised or reordered.  All times are
 * int64 nanoseconds; the only arithmetic is +, max and round-up division in
 * the communication cost formulas; utilisation is one fp64 division.
 *
 * Notation (paper Sec. 4.3 / Algorithm 1 plus the alpha-beta cost model):
 *   N devices, G per node, L layers, B global batch, s sequence, h hidden,
 *   e bytes per activation element.  A candidate strategy is
 *   x = (mp, pp, dp = N/(mp*pp), stage bounds 0=c_0<..<c_pp=L, m, sched);
 *   Bp = B/dp, b = ceil(Bp/m); the event class is (mp, b).
 *   Device index: rank(r,d,q) = (r*pp + d)*mp + q  (Algorithm 1 indexes the
 *   pipeline lists as d*MP + m_p; DP modeling duplicates them DP times, so the
 *   replica index r is outermost).  node(rank) = rank / G.
 *
 * Schedules: GPipe, 1F1B (Dapple), asynchronous 1F1B (no gradient all-reduce) and, for
 * candidates given explicitly, interleaved 1F1B over v model chunks per device (see the
 * comment above orc_simulate).
 *
 * Pins for every function here live in tests/test_oracle_pins.py (closed
 * forms, invariants, brute-force longest path, hand-worked examples, printed
 * counts from the paper).  The paper's measured accuracy against real clusters
 * cannot be reproduced here: parity with measured reality is unpinned.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_MAX_PP 64

enum {
    ORC_OK = 0,
    ORC_E_ARG = -1,       /* malformed argument                                 */
    ORC_E_CLASS = -2,     /* event class (mp, b) missing from the table         */
    ORC_E_LOCALITY = -3,  /* replicas of one stage would see different links    */
    ORC_E_DEADLOCK = -4,  /* the worklist found no available schedule item      */
    ORC_E_NOMEM = -5
};

/* Event kinds written to the `kind` field of a record. */
enum {
    ORC_COMPUTE_F = 0, ORC_COMPUTE_B = 1,
    ORC_MP_AR_F = 2,   ORC_MP_AR_B = 3,
    ORC_A2A_F = 4,     ORC_A2A_B = 5,
    ORC_SEND_F = 6,    ORC_SEND_B = 7,
    ORC_DP_AR = 8,
    ORC_JITTER_F = 9,  ORC_JITTER_B = 10   /* per-micro-batch fluctuation at the start of an item */
};

/* The event table: profiled (here: synthetic) event times per class, plus the
 * cluster constants of the alpha-beta communication model. */
typedef struct {
    int32_t n_layers, n_classes, n_devices, gpus_per_node;
    int64_t global_batch, seq, hidden;
    int64_t alpha_intra_ns, beta_intra;   /* beta in bytes per ns */
    int64_t alpha_inter_ns, beta_inter;
    int64_t dp_bucket_bytes;              /* 0: one all-reduce per stage          */
    int32_t dp_overlap;                   /* 0: after the last event; 1: overlap  */
    int32_t act_bytes_per_elem;
    const int32_t *class_mp, *class_b;    /* [n_classes]                          */
    const int64_t *fwd_ns, *bwd_ns;       /* [n_classes][n_layers]                */
    const uint8_t *layer_is_expert;       /* [n_layers]                           */
    const int64_t *grad_bytes;            /* [n_layers], at mp = 1                */
    int32_t allreduce_profile_max;        /* 0: every all-reduce size is modelled directly;
                                             k > 0: all-reduces over more than k devices are
                                             the k-device time scaled by the volume formula */
    int32_t n_jitter;                     /* P: number of micro-batch slots of the jitter table
                                             (0: all micro-batches of a stage cost the same)  */
    int32_t jitter_stages;                /* columns of the jitter tables (>= pp of any strategy) */
    int32_t pad;
    const int64_t *jitter_fwd_ns;         /* [P][jitter_stages]: extra time of the forward item of
                                             micro-batch j on stage d is [j mod P][d]          */
    const int64_t *jitter_bwd_ns;         /* same for backward items                           */
} orc_table;

/* The search space (paper Sec. 6: grid search over parallel degrees). */
typedef struct {
    int32_t mp_max, pp_max, n_m;
    const int32_t *m_list;                /* ascending                            */
    int32_t m_rule;                       /* 0: m divides Bp; 1: any m <= Bp      */
    int32_t partition_mode;               /* 0: balanced; 1: all compositions     */
    int32_t sched_mask;                   /* bit 0: GPipe, bit 1: 1F1B (Dapple),
                                             bit 2: 1F1B without gradient synchronisation,
                                             bit 3: interleaved 1F1B with v = 2, 4, .. v_max chunks,
                                             bit 4: bidirectional pipelines */
    int32_t v_max;                        /* largest number of model chunks per device (bit 3)    */
} orc_space;

typedef struct {
    int32_t mp, pp, dp, m, sched;         /* sched 0: GPipe, 1: 1F1B, 2: asynchronous 1F1B,
                                             3: interleaved 1F1B, 4: bidirectional pipelines */
    int32_t bounds[ORC_MAX_PP + 1];       /* c_0 .. c_P, P = pp (P = pp * v for sched 3)  */
    int32_t v;                            /* sched 3: model chunks per device (0 or 1 otherwise) */
} orc_candidate;

typedef struct { int64_t kind, layer, mb, start, end; } orc_event;
typedef struct { orc_event *ev; int64_t n, cap; } orc_list;

typedef struct {
    int32_t n_lists;          /* N (replicate) or pp (one device per stage)       */
    int64_t batch_ns;
    orc_list *lists;          /* final per-device event lists                     */
    int64_t *busy_ns;         /* [n_lists] union measure of the event intervals   */
    double *util;             /* [n_lists] busy / batch                           */
} orc_result;

/* ------------------------------------------------------------------------- */
/* small helpers                                                              */

static int64_t cdiv(int64_t a, int64_t b) { return (a + b - 1) / b; }
static int64_t max64(int64_t a, int64_t b) { return a > b ? a : b; }

static int list_push(orc_list *l, orc_event e)
{
    if (l->n == l->cap) {
        int64_t nc = l->cap ? 2 * l->cap : 64;
        orc_event *p = (orc_event *)realloc(l->ev, (size_t)nc * sizeof(orc_event));
        if (!p) return ORC_E_NOMEM;
        l->ev = p; l->cap = nc;
    }
    l->ev[l->n++] = e;
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Communication events: alpha-beta costs.                                    */
/* The per-device volume of a ring all-reduce over n devices of a P-byte      */
/* tensor is 2(n-1)P/n (paper Sec. 4.2, all-reduce profiling); each of its    */
/* 2(n-1) steps also pays the link latency alpha.                             */

int64_t orc_ring_allreduce_ns(int64_t n, int64_t bytes, int64_t alpha, int64_t beta)
{
    return 2 * (n - 1) * alpha + cdiv(2 * (n - 1) * bytes, n * beta);
}
/* All-reduce event time.  The paper (Sec. 4.2) profiles all-reduces of up to 8 devices directly
 * and, above that, takes the 8-device time and scales it by the per-device volume
 * 2(N-1)P/N of the actual device count: T(n) = T(k) * [2(n-1)/n] / [2(k-1)/k], rounded up.
 * Here the "profiled" times come from the ring alpha-beta form; k = 0 switches the
 * extrapolation off (every size modelled directly). */
int64_t orc_allreduce_ns(int64_t k, int64_t n, int64_t bytes, int64_t alpha, int64_t beta)
{
    if (k <= 1 || n <= k) return orc_ring_allreduce_ns(n, bytes, alpha, beta);
    return cdiv(orc_ring_allreduce_ns(k, bytes, alpha, beta) * k * (n - 1), (k - 1) * n);
}
/* Pairwise-exchange all-to-all: n-1 steps, each moving 1/n of the buffer. */
int64_t orc_all_to_all_ns(int64_t n, int64_t bytes, int64_t alpha, int64_t beta)
{
    return (n - 1) * alpha + cdiv((n - 1) * bytes, n * beta);
}
/* Point-to-point activation transfer between adjacent stages. */
int64_t orc_p2p_ns(int64_t bytes, int64_t alpha, int64_t beta)
{
    return alpha + cdiv(bytes, beta);
}

/* Intra/inter-node attribute of communication events (paper Sec. 4.1): a
 * transfer is intra-node iff source and destination rank share a node; a
 * collective is intra-node iff all its members do.  Found by brute force over
 * every group the strategy creates; all replicas must agree, because the
 * method models them with one event.  Returns 0 intra, 1 inter, -1 mixed. */
static int64_t rank_of(const orc_candidate *x, int64_t r, int64_t d, int64_t q)
{
    return (r * x->pp + d) * x->mp + q;
}
static int merge_loc(int cur, int v) { return cur == -2 ? v : (cur == v ? cur : -1); }

static int loc_mp_groups(const orc_table *T, const orc_candidate *x)
{
    int cur = -2;
    for (int64_t r = 0; r < x->dp; ++r)
        for (int64_t d = 0; d < x->pp; ++d) {
            int inter = 0;
            int64_t n0 = rank_of(x, r, d, 0) / T->gpus_per_node;
            for (int64_t q = 1; q < x->mp; ++q)
                if (rank_of(x, r, d, q) / T->gpus_per_node != n0) inter = 1;
            cur = merge_loc(cur, inter);
        }
    return cur;
}
static int loc_dp_groups(const orc_table *T, const orc_candidate *x)
{
    int cur = -2;
    for (int64_t d = 0; d < x->pp; ++d)
        for (int64_t q = 0; q < x->mp; ++q) {
            int inter = 0;
            int64_t n0 = rank_of(x, 0, d, q) / T->gpus_per_node;
            for (int64_t r = 1; r < x->dp; ++r)
                if (rank_of(x, r, d, q) / T->gpus_per_node != n0) inter = 1;
            cur = merge_loc(cur, inter);
        }
    return cur;
}
/* Bidirectional pipelines: the weights of stage s live on device s (pipeline "down") and on
 * device pp - 1 - s (pipeline "up") of every replica; their gradients are reduced over those
 * 2 dp devices. */
static int loc_mirror_group(const orc_table *T, const orc_candidate *x, int64_t d)
{
    int cur = -2;
    for (int64_t q = 0; q < x->mp; ++q) {
        int inter = 0;
        int64_t n0 = rank_of(x, 0, d, q) / T->gpus_per_node;
        for (int64_t r = 0; r < x->dp; ++r)
            if (rank_of(x, r, d, q) / T->gpus_per_node != n0 ||
                rank_of(x, r, x->pp - 1 - d, q) / T->gpus_per_node != n0) inter = 1;
        cur = merge_loc(cur, inter);
    }
    return cur;
}
/* Transfer from pipeline device da to pipeline device db (db = da + 1 between neighbouring
 * stages; the interleaved schedule also sends from the last device back to the first). */
static int loc_transfer(const orc_table *T, const orc_candidate *x, int64_t da, int64_t db)
{
    int cur = -2;
    for (int64_t r = 0; r < x->dp; ++r)
        for (int64_t q = 0; q < x->mp; ++q) {
            int inter = rank_of(x, r, da, q) / T->gpus_per_node !=
                        rank_of(x, r, db, q) / T->gpus_per_node;
            cur = merge_loc(cur, inter);
        }
    return cur;
}
static int64_t alpha_of(const orc_table *T, int loc) { return loc ? T->alpha_inter_ns : T->alpha_intra_ns; }
static int64_t beta_of(const orc_table *T, int loc) { return loc ? T->beta_inter : T->beta_intra; }

/* ------------------------------------------------------------------------- */
/* Search-space enumeration by nested loops, outermost first:                  */
/*   mp ascending over powers of two <= mp_max;                                */
/*   pp ascending over powers of two <= min(pp_max, L) with mp*pp | N, dp | B; */
/*   m ascending over the valid entries of m_list;                             */
/*   stage partition in lexicographic order of (c_1..c_{pp-1});                */
/*   schedule: GPipe, then 1F1B, then asynchronous 1F1B.                       */
/* With bit 3 of sched_mask every (mp, pp) with pp >= 2 is followed, for       */
/* v = 2, 4, .. <= v_max with pp*v <= min(64, L), by the interleaved 1F1B       */
/* candidates of v chunks per device: m ascending over the valid entries that  */
/* are multiples of pp, then the partition of the L layers into pp*v virtual    */
/* stages (balanced, or every composition in lexicographic order).             */
/* With bit 4 every (mp, pp) with pp >= 2 is then followed by the candidates of */
/* the bidirectional schedule: m ascending over the valid even entries, the    */
/* partition into pp stages as for the plain schedules.                        */
/* The paper's own grid (Sec. 6) walks mp and pp over powers of two and takes  */
/* dp = GPUs/mp/pp, dropping the invalid combinations.                         */

static int valid_m(const orc_space *S, int64_t Bp, int64_t m)
{
    if (m < 1 || m > Bp) return 0;
    return S->m_rule == 0 ? (Bp % m == 0) : 1;
}

/* Advances bounds c_1..c_{pp-1} to the next (pp-1)-subset of {1..L-1} in
 * lexicographic order; returns 0 when the last one has been passed. */
static int next_partition(int32_t *c, int pp, int L)
{
    int i = pp - 1;
    while (i >= 1 && c[i] == L - (pp - i)) --i;
    if (i < 1) return 0;
    ++c[i];
    for (int j = i + 1; j <= pp - 1; ++j) c[j] = c[j - 1] + 1;
    return 1;
}

typedef int (*orc_visit_fn)(void *ctx, int64_t index, const orc_candidate *x);

/* Walks the whole space in canonical order; stops early when visit returns
 * non-zero.  Returns the number of candidates visited (or the full count). */
static int64_t walk_space(const orc_table *T, const orc_space *S, orc_visit_fn visit, void *ctx)
{
    int64_t index = 0;
    const int L = T->n_layers;
    for (int64_t mp = 1; mp <= S->mp_max; mp *= 2)
        for (int64_t pp = 1; pp <= S->pp_max && pp <= L; pp *= 2) {
            if (T->n_devices % (mp * pp) != 0) continue;
            int64_t dp = T->n_devices / (mp * pp);
            if (T->global_batch % dp != 0) continue;
            int64_t Bp = T->global_batch / dp;
            for (int mi = 0; mi < S->n_m; ++mi) {
                int64_t m = S->m_list[mi];
                if (!valid_m(S, Bp, m)) continue;
                orc_candidate x;
                memset(&x, 0, sizeof x);
                x.mp = (int32_t)mp; x.pp = (int32_t)pp; x.dp = (int32_t)dp; x.m = (int32_t)m;
                x.bounds[0] = 0; x.bounds[pp] = L;
                if (S->partition_mode == 0)
                    for (int j = 1; j < pp; ++j) x.bounds[j] = (int32_t)((int64_t)j * L / pp);
                else
                    for (int j = 1; j < pp; ++j) x.bounds[j] = j;
                do {
                    for (int sc = 0; sc < 3; ++sc) {
                        if (!(S->sched_mask & (1 << sc))) continue;
                        x.sched = sc;
                        if (visit && visit(ctx, index, &x)) return index + 1;
                        ++index;
                    }
                } while (S->partition_mode == 1 && next_partition(x.bounds, (int)pp, L));
            }
            /* interleaved 1F1B: candidates with v chunks per device, P = pp * v virtual stages */
            if (pp < 2) continue;
            for (int64_t v = 2; (S->sched_mask & 8) && v <= S->v_max && pp * v <= ORC_MAX_PP && pp * v <= L; v *= 2) {
                const int P = (int)(pp * v);
                for (int mi = 0; mi < S->n_m; ++mi) {
                    int64_t m = S->m_list[mi];
                    if (!valid_m(S, Bp, m) || m % pp != 0) continue;
                    orc_candidate x;
                    memset(&x, 0, sizeof x);
                    x.mp = (int32_t)mp; x.pp = (int32_t)pp; x.dp = (int32_t)dp; x.m = (int32_t)m;
                    x.sched = 3; x.v = (int32_t)v;
                    x.bounds[0] = 0; x.bounds[P] = L;
                    if (S->partition_mode == 0)
                        for (int j = 1; j < P; ++j) x.bounds[j] = (int32_t)((int64_t)j * L / P);
                    else
                        for (int j = 1; j < P; ++j) x.bounds[j] = j;
                    do {
                        if (visit && visit(ctx, index, &x)) return index + 1;
                        ++index;
                    } while (S->partition_mode == 1 && next_partition(x.bounds, P, L));
                }
            }
            /* bidirectional pipelines: half of the (even number of) micro-batches each way */
            if (!(S->sched_mask & 16)) continue;
            for (int mi = 0; mi < S->n_m; ++mi) {
                int64_t m = S->m_list[mi];
                if (!valid_m(S, Bp, m) || m % 2 != 0) continue;
                orc_candidate x;
                memset(&x, 0, sizeof x);
                x.mp = (int32_t)mp; x.pp = (int32_t)pp; x.dp = (int32_t)dp; x.m = (int32_t)m;
                x.sched = 4;
                x.bounds[0] = 0; x.bounds[pp] = L;
                if (S->partition_mode == 0)
                    for (int j = 1; j < pp; ++j) x.bounds[j] = (int32_t)((int64_t)j * L / pp);
                else
                    for (int j = 1; j < pp; ++j) x.bounds[j] = j;
                do {
                    if (visit && visit(ctx, index, &x)) return index + 1;
                    ++index;
                } while (S->partition_mode == 1 && next_partition(x.bounds, (int)pp, L));
            }
        }
    return index;
}

int64_t orc_count(const orc_table *T, const orc_space *S)
{
    return walk_space(T, S, NULL, NULL);
}

typedef struct { const int64_t *idx; int64_t n, next; orc_candidate *out; } pick_ctx;
static int pick_visit(void *vc, int64_t index, const orc_candidate *x)
{
    pick_ctx *c = (pick_ctx *)vc;
    while (c->next < c->n && c->idx[c->next] == index) c->out[c->next++] = *x;
    return c->next >= c->n;
}
/* Decodes the candidates at the given ascending indices by walking the loops. */
int orc_enumerate_at(const orc_table *T, const orc_space *S, const int64_t *sorted_idx,
                     int64_t n, orc_candidate *out)
{
    for (int64_t i = 1; i < n; ++i) if (sorted_idx[i] < sorted_idx[i - 1]) return ORC_E_ARG;
    if (n > 0 && sorted_idx[0] < 0) return ORC_E_ARG;
    pick_ctx c = { sorted_idx, n, 0, out };
    walk_space(T, S, pick_visit, &c);
    return c.next == n ? ORC_OK : ORC_E_ARG;
}

/* ------------------------------------------------------------------------- */
/* The simulation of one candidate.                                           */

typedef struct { int32_t is_bwd, mb, chunk; } orc_op;

static int find_class(const orc_table *T, int64_t mp, int64_t b)
{
    for (int k = 0; k < T->n_classes; ++k)
        if (T->class_mp[k] == mp && T->class_b[k] == b) return k;
    return -1;
}

void orc_result_free(orc_result *R)
{
    if (!R) return;
    if (R->lists) { for (int i = 0; i < R->n_lists; ++i) free(R->lists[i].ev); free(R->lists); }
    free(R->busy_ns); free(R->util); free(R);
}

static int cmp_event_start(const void *a, const void *b)
{
    const orc_event *x = (const orc_event *)a, *y = (const orc_event *)b;
    if (x->start != y->start) return x->start < y->start ? -1 : 1;
    if (x->end != y->end) return x->end < y->end ? -1 : 1;
    return 0;
}
/* Measure of the union of a device's event intervals (its activity time). */
static int64_t union_measure(const orc_list *l)
{
    if (l->n == 0) return 0;
    orc_event *tmp = (orc_event *)malloc((size_t)l->n * sizeof(orc_event));
    memcpy(tmp, l->ev, (size_t)l->n * sizeof(orc_event));
    qsort(tmp, (size_t)l->n, sizeof(orc_event), cmp_event_start);
    int64_t total = 0, lo = tmp[0].start, hi = tmp[0].end;
    for (int64_t i = 1; i < l->n; ++i) {
        if (tmp[i].start > hi) { total += hi - lo; lo = tmp[i].start; hi = tmp[i].end; }
        else hi = max64(hi, tmp[i].end);
    }
    total += hi - lo;
    free(tmp);
    return total;
}

/*
 * Bidirectional pipelines (sched 4; Chimera, which the paper names among the pipeline scheduling
 * algorithms in Sec. 2; the schedule is, as for the others, the input of the pipeline modeling
 * of Sec. 4.3).  Two pipelines run over the same pp devices (pp even) in opposite directions:
 * pipeline "down" has stage s on device s and takes micro-batches 0 .. m/2 - 1, pipeline "up" has
 * stage s on device pp - 1 - s and takes micro-batches m/2 .. m - 1 (m even).  Each pipeline, on
 * its own, runs the 1F1B order.  A device holds one stage of each and merges the two orders; the
 * merged order is the one in which the items run when every item takes one time slot and every
 * device, slot by slot, runs the first of its two pipelines' next items whose input was produced
 * in an earlier slot - preferring the item whose micro-batch comes earlier within its pipeline
 * (the two never hold the same position when both could run - checked for pp <= 32, m <= 64 -
 * a backward item, then pipeline "down", would go first).  With m = pp that takes 3 pp - 2 slots (pp - 2 idle
 * slots per device, the published property of the schedule), with any even m, 2 m + pp - 2.
 * ops[d * 2m + k]: the k-th item of device d (chunk = pipeline).  Returns 0, or -1 (no memory).
 */
static int bidirectional_order(int pp, int m, orc_op *ops)
{
    const int half = m / 2, n_ops = 2 * m;
    /* the two 1F1B orders of every device, and when each item finished (slot number; -1: not yet) */
    orc_op *q = (orc_op *)malloc((size_t)2 * pp * m * sizeof(orc_op));     /* [device][pipeline][m] */
    int *endF = (int *)malloc((size_t)2 * pp * m * sizeof(int));           /* [pipeline][stage][micro-batch] */
    int *endB = (int *)malloc((size_t)2 * pp * m * sizeof(int));
    if (!q || !endF || !endB) { free(q); free(endF); free(endB); return -1; }
    for (int i = 0; i < 2 * pp * m; ++i) endF[i] = endB[i] = -1;
    for (int d = 0; d < pp; ++d)
        for (int u = 0; u < 2; ++u) {
            const int s = u ? pp - 1 - d : d, first = u ? half : 0;
            orc_op *o = q + ((int64_t)d * 2 + u) * m;
            const int w = pp - s < half ? pp - s : half;
            int k = 0, nf = 0, nb = 0;
            for (; nf < w; ++nf) { o[k].is_bwd = 0; o[k].chunk = u; o[k++].mb = first + nf; }
            while (nb < half) {
                o[k].is_bwd = 1; o[k].chunk = u; o[k++].mb = first + nb++;
                if (nf < half) { o[k].is_bwd = 0; o[k].chunk = u; o[k++].mb = first + nf++; }
            }
        }
    int head[ORC_MAX_PP][2], n_done[ORC_MAX_PP], pick[ORC_MAX_PP];
    for (int d = 0; d < pp; ++d) { head[d][0] = head[d][1] = 0; n_done[d] = 0; }
    int left = pp * n_ops;
    for (int t = 0; left > 0; ++t) {
        if (t > 4 * (m + pp)) { free(q); free(endF); free(endB); return -1; }
        /* every device chooses on what earlier slots produced ... */
        for (int d = 0; d < pp; ++d) {
            pick[d] = -1;
            int best_mb = 0, best_bwd = 0;
            for (int u = 0; u < 2; ++u) {
                if (head[d][u] == m) continue;
                const orc_op o = q[((int64_t)d * 2 + u) * m + head[d][u]];
                const int s = u ? pp - 1 - d : d;
                const int64_t at = ((int64_t)u * pp + s) * m + o.mb;
                int dep;
                if (!o.is_bwd) dep = s == 0 ? 0 : endF[at - m];
                else dep = s == pp - 1 ? endF[at] : endB[at + m];
                if (dep < 0 || dep > t) continue;
                const int local = o.mb - (u ? half : 0);
                if (pick[d] < 0 || local < best_mb || (local == best_mb && o.is_bwd > best_bwd)) {
                    pick[d] = u; best_mb = local; best_bwd = o.is_bwd;
                }
            }
        }
        /* ... then the chosen items run, one slot each */
        for (int d = 0; d < pp; ++d) {
            const int u = pick[d];
            if (u < 0) continue;
            const orc_op o = q[((int64_t)d * 2 + u) * m + head[d][u]];
            const int s = u ? pp - 1 - d : d;
            (o.is_bwd ? endB : endF)[((int64_t)u * pp + s) * m + o.mb] = t + 1;
            ops[(int64_t)d * n_ops + n_done[d]++] = o;
            ++head[d][u]; --left;
        }
    }
    free(q); free(endF); free(endB);
    return 0;
}

/*
 * Interleaved 1F1B (sched 3; the paper names further scheduling algorithms as input to the same
 * pipeline modeling, Sec. 4.3 "the pipeline schedule generated from the pipeline algorithm",
 * and cites Megatron-LM, whose interleaved schedule this is).  Every device holds v model
 * chunks: the model is cut into P = pp * v virtual stages, virtual stage s = c * pp + d being
 * chunk c of device d, so consecutive virtual stages sit on consecutive devices and the last
 * device sends to the first between chunks.  A device runs its m * v forward and m * v backward
 * items in this order (m must be a multiple of pp): the k-th forward item is chunk
 * (k / pp) mod v of micro-batch (k / (pp v)) pp + k mod pp, the k-th backward item the same
 * with chunk v - 1 - (k / pp) mod v; device d first runs min(m v, 2 (pp - d - 1) + (v - 1) pp)
 * forward items (all of them when m = pp), then alternates one forward, one backward, and
 * finishes with the remaining backward items.  Dependencies, events, transfers and the
 * device-is-busy rule are those of Algorithm 1, with virtual stages in the place of stages.
 * Gradient buckets are cut per chunk (each chunk's gradients in backward order), chunks in the
 * order their last micro-batch's backward runs (v - 1 first), on the device's one lane.
 *
 * orc_simulate
 *   replicate    1: keep a list for every one of the N devices;
 *                0: keep only the device (r=0, q=0) of every stage (pp lists).
 *   reverse_scan 0: the pick step scans stages 0..pp-1; 1: pp-1..0.  The
 *                result must not depend on it (each item's start depends only
 *                on its two predecessors).
 */
orc_result *orc_simulate(const orc_table *T, const orc_candidate *x, int replicate,
                         int reverse_scan, int *err)
{
    int e = ORC_OK;
    orc_result *R = NULL;
    orc_list *F = NULL;          /* Algorithm 1's event lists, pipeline only      */
    orc_op *ops = NULL;          /* schedule S: per stage, 2m items in order      */
    int64_t *endF = NULL, *endB = NULL;
    orc_event *tmp = NULL;
    const int pp = x->pp, mp = x->mp, dp = x->dp, m = x->m, L = T->n_layers;
    const int v = x->sched == 3 ? x->v : 1;      /* model chunks per device               */
    const int P = pp * v;                        /* virtual stages                         */

    if (pp < 1 || pp > ORC_MAX_PP || mp < 1 || dp < 1 || m < 1 || v < 1 || P > ORC_MAX_PP ||
        (int64_t)mp * pp * dp != T->n_devices || T->global_batch % dp != 0 ||
        x->bounds[0] != 0 || x->bounds[P] != L || x->sched < 0 || x->sched > 4 ||
        (x->sched == 3 && (m % pp != 0 || T->n_jitter > 0)) ||
        (x->sched == 4 && (pp % 2 != 0 || m % 2 != 0 || T->n_jitter > 0)) ||
        (T->n_jitter > 0 && (T->jitter_stages < pp || !T->jitter_fwd_ns || !T->jitter_bwd_ns))) {
        e = ORC_E_ARG; goto fail;
    }
    for (int s = 0; s < P; ++s) if (x->bounds[s + 1] <= x->bounds[s]) { e = ORC_E_ARG; goto fail; }

    /* ---- Step 1: events and their elapsed times (MP modeling) ------------- */
    const int64_t Bp = T->global_batch / dp;
    const int64_t b = cdiv(Bp, m);
    const int kappa = find_class(T, mp, b);
    if (kappa < 0) { e = ORC_E_CLASS; goto fail; }
    const int64_t *f = T->fwd_ns + (int64_t)kappa * L;
    const int64_t *g = T->bwd_ns + (int64_t)kappa * L;
    const int64_t act = b * T->seq * T->hidden * T->act_bytes_per_elem;

    int64_t AR = 0, A2A = 0, P2P[ORC_MAX_PP];
    int loc_dp = 0;
    const int two_way = x->sched == 4;           /* bidirectional pipelines                */
    const int64_t n_sync = two_way ? 2 * (int64_t)dp : dp;      /* devices that hold a stage's weights */
    int loc_sync[ORC_MAX_PP];                    /* per device: locality of its gradient groups */
    if (mp > 1) {
        int loc = loc_mp_groups(T, x);
        if (loc < 0) { e = ORC_E_LOCALITY; goto fail; }
        AR = orc_allreduce_ns(T->allreduce_profile_max, mp, 2 * act, alpha_of(T, loc), beta_of(T, loc));
    }
    if (dp > 1) {
        loc_dp = loc_dp_groups(T, x);
        if (loc_dp < 0) { e = ORC_E_LOCALITY; goto fail; }
        A2A = orc_all_to_all_ns(dp, act, alpha_of(T, loc_dp), beta_of(T, loc_dp));
    }
    for (int d = 0; d < pp; ++d) {
        loc_sync[d] = two_way ? loc_mirror_group(T, x, d) : loc_dp;
        if (loc_sync[d] < 0) { e = ORC_E_LOCALITY; goto fail; }
    }
    /* P2P[s]: transfer between virtual stages s and s + 1, i.e. between devices s mod pp and
     * (s + 1) mod pp */
    for (int s = 0; s + 1 < P; ++s) {
        int loc = loc_transfer(T, x, s % pp, (s + 1) % pp);
        if (loc < 0) { e = ORC_E_LOCALITY; goto fail; }
        P2P[s] = orc_p2p_ns(act, alpha_of(T, loc), beta_of(T, loc));
    }

    /* ---- Step 2: the pipeline schedule S(D, L, M) -------------------------- */
    const int n_ops = 2 * m * v;                 /* items of one device                    */
    ops = (orc_op *)malloc((size_t)pp * n_ops * sizeof(orc_op));
    const int n_vs = two_way ? 2 * pp : P;       /* rows of endF / endB: virtual stages, or
                                                    [pipeline][stage] of the bidirectional schedule */
    endF = (int64_t *)malloc((size_t)n_vs * m * sizeof(int64_t));   /* [virtual stage][micro-batch] */
    endB = (int64_t *)malloc((size_t)n_vs * m * sizeof(int64_t));
    tmp = (orc_event *)malloc((size_t)(3 * L + 2) * sizeof(orc_event));
    const int mp_lists = replicate ? mp : 1;
    F = (orc_list *)calloc((size_t)pp * mp_lists, sizeof(orc_list));
    if (!ops || !endF || !endB || !tmp || !F) { e = ORC_E_NOMEM; goto fail; }
    for (int64_t i = 0; i < (int64_t)n_vs * m; ++i) endF[i] = endB[i] = -1;
    if (two_way && bidirectional_order(pp, m, ops) != 0) { e = ORC_E_NOMEM; goto fail; }
    for (int d = 0; d < pp && !two_way; ++d) {
        orc_op *o = ops + (int64_t)d * n_ops;
        int k = 0;
        for (int i = 0; i < n_ops; ++i) o[i].chunk = 0;
        if (x->sched == 3) {                      /* interleaved 1F1B over v chunks        */
            const int total = m * v;
            int warm = (pp - d - 1) * 2 + (v - 1) * pp;
            if (m == pp || warm > total) warm = total;
            int nf = 0, nb = 0;
            for (int step = 0; step < 2 * total; ++step) {
                /* warm-up forwards; then forward, backward alternately; then the backwards left */
                int is_b;
                if (nf < warm) is_b = 0;
                else if (nf < total) is_b = ((step - warm) & 1);
                else is_b = 1;
                const int idx = is_b ? nb++ : nf++;
                const int c = (idx / pp) % v;
                o[k].is_bwd = is_b;
                o[k].chunk = is_b ? v - 1 - c : c;
                o[k].mb = (idx / (pp * v)) * pp + idx % pp;
                ++k;
            }
        } else if (x->sched == 0) {               /* GPipe: all forwards, then all backwards */
            for (int j = 0; j < m; ++j) { o[k].is_bwd = 0; o[k++].mb = j; }
            for (int j = 0; j < m; ++j) { o[k].is_bwd = 1; o[k++].mb = j; }
        } else {                                  /* 1F1B (Dapple): warm-up, then one-B-one-F;
                                                     the asynchronous variant keeps this order */
            int w = pp - d < m ? pp - d : m;
            int nf = 0, nb = 0;
            for (; nf < w; ++nf) { o[k].is_bwd = 0; o[k++].mb = nf; }
            while (nb < m) {
                o[k].is_bwd = 1; o[k++].mb = nb++;
                if (nf < m) { o[k].is_bwd = 0; o[k++].mb = nf++; }
            }
        }
    }

    /* ---- Step 3: Algorithm 1 as a worklist ---------------------------------- */
    {
        int32_t head[ORC_MAX_PP];
        int64_t device_free[ORC_MAX_PP];
        int64_t remaining = (int64_t)pp * n_ops;
        for (int d = 0; d < pp; ++d) { head[d] = 0; device_free[d] = 0; }
        while (remaining > 0) {
            /* Pick step of Algorithm 1 (Sec. 4.3): the first device whose next schedule item
             * has its input data ready and its micro-batch matched; the item belongs to virtual
             * stage vs = chunk * pp + d (vs = d without chunks) */
            int pick = -1; int64_t t = 0;
            for (int s = 0; s < pp && pick < 0; ++s) {
                int d = reverse_scan ? pp - 1 - s : s;
                if (head[d] == n_ops) continue;
                orc_op o = ops[(int64_t)d * n_ops + head[d]];
                /* the item's stage in its chain of stages, and its row in endF / endB */
                const int st = two_way ? (o.chunk ? pp - 1 - d : d) : o.chunk * pp + d;
                const int vs = two_way ? o.chunk * pp + st : st;
                const int n_st = two_way ? pp : P;
                int64_t dep;
                if (!o.is_bwd) dep = st == 0 ? 0 : endF[(int64_t)(vs - 1) * m + o.mb];
                else dep = st == n_st - 1 ? endF[(int64_t)vs * m + o.mb] : endB[(int64_t)(vs + 1) * m + o.mb];
                if (dep < 0) continue;
                pick = d; t = max64(device_free[d], dep);
            }
            if (pick < 0) { e = ORC_E_DEADLOCK; goto fail; }
            const int d = pick;
            const orc_op o = ops[(int64_t)d * n_ops + head[d]];
            const int st = two_way ? (o.chunk ? pp - 1 - d : d) : o.chunk * pp + d;
            const int vs = two_way ? o.chunk * pp + st : st;
            const int n_st = two_way ? pp : P;
            const int la = x->bounds[st], le = x->bounds[st + 1];   /* the item's layers [la, le) */
            /* transfers to the next / previous stage of the item's pipeline: pipeline "up" of the
             * bidirectional schedule crosses the device boundaries the other way round */
            const int64_t send_f = st < n_st - 1 ? (two_way && o.chunk ? P2P[pp - 2 - st] : P2P[st]) : 0;
            const int64_t send_b = st > 0 ? (two_way && o.chunk ? P2P[pp - 1 - st] : P2P[st - 1]) : 0;
            /* Look-up step of Algorithm 1: the events MP modeling mapped the item's layers to -
             * per layer a computation event, then its all-reduce event (mp > 1) and its
             * all-to-all event (expert layer, dp > 1) - followed by the communication event of
             * the item, the transfer to the neighbouring stage. */
            int n = 0;
            /* Fluctuation between micro-batches (the paper's error analysis, Sec. 5.3, blames
             * profiling fluctuation that accumulates along the stages): when a jitter table is
             * given, the item of micro-batch j on stage d begins with a jitter event of
             * [j mod P][d] ns, before its first computation event. */
            if (T->n_jitter > 0) {
                const int64_t *jt = o.is_bwd ? T->jitter_bwd_ns : T->jitter_fwd_ns;
                const int64_t jit = jt[(int64_t)(o.mb % T->n_jitter) * T->jitter_stages + d];
                const int first_layer = o.is_bwd ? le - 1 : la;
                tmp[n++] = (orc_event){ o.is_bwd ? ORC_JITTER_B : ORC_JITTER_F, first_layer, o.mb, t, t + jit };
                t += jit;
            }
            if (!o.is_bwd) {
                for (int l = la; l < le; ++l) {
                    tmp[n++] = (orc_event){ ORC_COMPUTE_F, l, o.mb, t, t + f[l] }; t += f[l];
                    if (mp > 1) { tmp[n++] = (orc_event){ ORC_MP_AR_F, l, o.mb, t, t + AR }; t += AR; }
                    if (T->layer_is_expert[l] && dp > 1) { tmp[n++] = (orc_event){ ORC_A2A_F, l, o.mb, t, t + A2A }; t += A2A; }
                }
                if (st < n_st - 1) { tmp[n++] = (orc_event){ ORC_SEND_F, le - 1, o.mb, t, t + send_f }; t += send_f; }
                endF[(int64_t)vs * m + o.mb] = t;
            } else {
                for (int l = le - 1; l >= la; --l) {
                    tmp[n++] = (orc_event){ ORC_COMPUTE_B, l, o.mb, t, t + g[l] }; t += g[l];
                    if (mp > 1) { tmp[n++] = (orc_event){ ORC_MP_AR_B, l, o.mb, t, t + AR }; t += AR; }
                    if (T->layer_is_expert[l] && dp > 1) { tmp[n++] = (orc_event){ ORC_A2A_B, l, o.mb, t, t + A2A }; t += A2A; }
                }
                if (st > 0) { tmp[n++] = (orc_event){ ORC_SEND_B, la, o.mb, t, t + send_b }; t += send_b; }
                endB[(int64_t)vs * m + o.mb] = t;
            }
            device_free[d] = t;
            for (int q = 0; q < mp_lists; ++q)          /* every device of the MP group */
                for (int i = 0; i < n; ++i)
                    if ((e = list_push(&F[d * mp_lists + q], tmp[i])) != ORC_OK) goto fail;
            ++head[d]; --remaining;                      /* the item leaves the schedule */
        }
    }

    /* ---- Step 4: DP modeling -------------------------------------------------- */
    R = (orc_result *)calloc(1, sizeof(orc_result));
    if (!R) { e = ORC_E_NOMEM; goto fail; }
    R->n_lists = replicate ? T->n_devices : pp;
    R->lists = (orc_list *)calloc((size_t)R->n_lists, sizeof(orc_list));
    R->busy_ns = (int64_t *)calloc((size_t)R->n_lists, sizeof(int64_t));
    R->util = (double *)calloc((size_t)R->n_lists, sizeof(double));
    if (!R->lists || !R->busy_ns || !R->util) { e = ORC_E_NOMEM; goto fail; }
    {
        const int dp_lists = replicate ? dp : 1;
        for (int r = 0; r < dp_lists; ++r)
            for (int d = 0; d < pp; ++d)
                for (int q = 0; q < mp_lists; ++q) {
                    /* duplicate the pipeline list of (d, q) for replica r */
                    orc_list *src = &F[d * mp_lists + q];
                    orc_list *dst = &R->lists[(r * pp + d) * mp_lists + q];
                    for (int64_t i = 0; i < src->n; ++i)
                        if ((e = list_push(dst, src->ev[i])) != ORC_OK) goto fail;
                    if (n_sync == 1) continue;
                    /* Asynchronous pipeline parallelism (the paper's discussion of new
                     * algorithms in "Related Work And Discussion": the pipeline schedule
                     * is built in the same way, only without the global synchronisation
                     * event, usually an all-reduce): every replica updates its own
                     * weights, so no gradient all-reduce event is appended. */
                    if (x->sched == 2) continue;
                    /* gradient all-reduce events: the stage's gradients, in the
                     * order the backward pass produces them (last layer first),
                     * cut into buckets; each bucket is a ring all-reduce over
                     * the dp replicas on a separate communication lane. */
                    const int64_t main_end = src->n ? src->ev[src->n - 1].end : 0;
                    int64_t prev_end = 0, kb = 0;      /* the device's one lane; bucket numbers run on */
                    /* one gradient stream per model chunk (one stream without chunks), the
                     * chunks in the order their last backward runs: chunk v - 1 first.
                     * Bidirectional pipelines: one stream per pipeline - the device's stage in
                     * it, reduced over the 2 dp devices that hold that stage - and the stream of
                     * the later stage first (its backward items end first). */
                    const int n_streams = two_way ? 2 : v;
                    for (int c = n_streams - 1; c >= 0; --c) {
                        int vs = c * pp + d, last_mb = m - 1;
                        if (two_way) {
                            const int up_first = pp - 1 - d > d;            /* the stage held in pipeline "up" is the later one */
                            const int u = (c == 1) == up_first;             /* c = 1 comes first */
                            vs = u ? pp - 1 - d : d;
                            last_mb = u ? m - 1 : m / 2 - 1;
                        }
                        const int la = x->bounds[vs], le = x->bounds[vs + 1];
                        int64_t W = 0;
                        for (int l = la; l < le; ++l) W += cdiv(T->grad_bytes[l], mp);
                        if (W == 0) continue;
                        const int64_t bucket = T->dp_bucket_bytes > 0 ? T->dp_bucket_bytes : W;
                        const int64_t nb = cdiv(W, bucket);
                        for (int64_t k = 0; k < nb; ++k) {
                            const int64_t lo = k * bucket;
                            const int64_t hi = lo + bucket < W ? lo + bucket : W;
                            int64_t ready = main_end;
                            if (T->dp_overlap) {
                                /* the layer holding the bucket's last byte (position hi-1) */
                                int64_t pos = 0; int last = -1;
                                for (int l = le - 1; l >= la; --l) {
                                    int64_t gl = cdiv(T->grad_bytes[l], mp);
                                    if (hi - 1 >= pos && hi - 1 < pos + gl) { last = l; break; }
                                    pos += gl;
                                }
                                /* ready when that layer's backward events of the LAST
                                 * microbatch's backward pass have all finished */
                                ready = -1;
                                for (int64_t i = 0; i < src->n; ++i) {
                                    const orc_event *ev = &src->ev[i];
                                    if (ev->layer == last && ev->mb == last_mb &&
                                        (ev->kind == ORC_COMPUTE_B || ev->kind == ORC_MP_AR_B || ev->kind == ORC_A2A_B))
                                        ready = max64(ready, ev->end);
                                }
                                if (ready < 0) { e = ORC_E_ARG; goto fail; }
                            }
                            const int64_t start = max64(ready, prev_end);
                            const int64_t end = start + orc_allreduce_ns(T->allreduce_profile_max, n_sync, hi - lo, alpha_of(T, loc_sync[d]), beta_of(T, loc_sync[d]));
                            if ((e = list_push(dst, (orc_event){ ORC_DP_AR, kb++, -1, start, end })) != ORC_OK) goto fail;
                            prev_end = end;
                        }
                    }
                }
    }

    /* ---- Step 5: timeline analyses --------------------------------------------- */
    R->batch_ns = 0;
    for (int i = 0; i < R->n_lists; ++i)
        for (int64_t k = 0; k < R->lists[i].n; ++k)
            R->batch_ns = max64(R->batch_ns, R->lists[i].ev[k].end);
    for (int i = 0; i < R->n_lists; ++i) {
        R->busy_ns[i] = union_measure(&R->lists[i]);
        R->util[i] = R->batch_ns > 0 ? (double)R->busy_ns[i] / (double)R->batch_ns : 0.0;
    }

    for (int i = 0; i < pp * mp_lists; ++i) free(F[i].ev);
    free(F); free(ops); free(endF); free(endB); free(tmp);
    if (err) *err = ORC_OK;
    return R;

fail:
    if (F) { for (int i = 0; i < pp * (replicate ? mp : 1); ++i) free(F[i].ev); free(F); }
    free(ops); free(endF); free(endB); free(tmp);
    orc_result_free(R);
    if (err) *err = e;
    return NULL;
}

/* ------------------------------------------------------------------------- */
/* Accessors for callers that cannot see the struct layout.                    */

int64_t orc_result_batch(const orc_result *R) { return R->batch_ns; }
int32_t orc_result_n_lists(const orc_result *R) { return R->n_lists; }
int64_t orc_result_total_records(const orc_result *R)
{
    int64_t t = 0;
    for (int i = 0; i < R->n_lists; ++i) t += R->lists[i].n;
    return t;
}
/* offsets[n_lists+1] (in records), records[total][5], busy[n_lists], util[n_lists] */
void orc_result_copy(const orc_result *R, int64_t *offsets, int64_t *records, int64_t *busy, double *util)
{
    int64_t t = 0;
    for (int i = 0; i < R->n_lists; ++i) {
        if (offsets) offsets[i] = t;
        if (records) memcpy(records + 5 * t, R->lists[i].ev, (size_t)R->lists[i].n * sizeof(orc_event));
        if (busy) busy[i] = R->busy_ns[i];
        if (util) util[i] = R->util[i];
        t += R->lists[i].n;
    }
    if (offsets) offsets[R->n_lists] = t;
}

/* Batch time and per-stage busy time (device r=0, q=0 of each stage) of the
 * candidates at the given ascending indices.  stage_busy is [n][pp_stride],
 * unused entries set to 0; nullable.  Single-threaded. */
int orc_eval_indices(const orc_table *T, const orc_space *S, const int64_t *sorted_idx, int64_t n,
                     int replicate, int64_t *batch_ns, int64_t *stage_busy, int32_t pp_stride)
{
    orc_candidate *c = (orc_candidate *)malloc((size_t)(n > 0 ? n : 1) * sizeof(orc_candidate));
    if (!c) return ORC_E_NOMEM;
    int e = orc_enumerate_at(T, S, sorted_idx, n, c);
    for (int64_t i = 0; i < n && e == ORC_OK; ++i) {
        orc_result *R = orc_simulate(T, &c[i], replicate, 0, &e);
        if (!R) break;
        batch_ns[i] = R->batch_ns;
        if (stage_busy) {
            for (int d = 0; d < pp_stride; ++d) stage_busy[i * pp_stride + d] = 0;
            for (int d = 0; d < c[i].pp && d < pp_stride; ++d) {
                /* with replicate, stage d's first device is rank (0*pp + d)*mp + 0 */
                int li = replicate ? d * c[i].mp : d;
                stage_busy[i * pp_stride + d] = R->busy_ns[li];
            }
        }
        orc_result_free(R);
    }
    free(c);
    return e;
}

int orc_sizeof_candidate(void) { return (int)sizeof(orc_candidate); }
