// Bidirectional pipelines (schedule 4): evaluation of candidates whose devices run two pipelines
// in opposite directions.
//
// Pipeline 0 ("down") has stage s on device s and takes micro-batches 0 .. m/2 - 1, pipeline 1
// ("up") has stage s on device pp - 1 - s and takes m/2 .. m - 1 (pp and m even); both cut the
// model at the same pp - 1 bounds.  A device holds one stage of each and runs their items in the
// merged order the host worked out for (pp, m) (DeviceView::order, 2 m + 1 slots per device): each pipeline keeps its 1F1B
// order, the merge is the one of unit time slots.  Algorithm 1 of the paper runs unchanged over
// the 2 pp (pipeline, stage) pairs with one free time per device.  The weights of a stage are on
// two devices of every replica, so its gradients are reduced over 2 dp devices - also when
// dp = 1 - and a device sends two streams of buckets down its one lane, the later stage's first.
//
// One warp evaluates a candidate, a lane per device, in rounds, exactly as for interleaved 1F1B
// (interleaved.cuh): the item ends travel through rings of pp ends per (pipeline, stage) and
// direction, indexed by the micro-batch's number within its pipeline; a pipeline on its own never
// has more than pp - s micro-batches in flight at stage s, so pp ends per ring are enough.
#pragma once

#include "costs.cuh"
#include "interleaved.cuh"

namespace distsim {

constexpr int kOrderUp = 1 << 15, kOrderBackward = 1 << 14, kOrderMicroBatch = (1 << 14) - 1;

// Shared memory of one candidate, in int64 words: the arrays of interleaved.cuh for 2 pp
// (pipeline, stage) pairs and `kt` kept items per device, with pp + 1 bounds.
__host__ __device__ inline int bidirectional_words(int pp, int kt)
{
    const int P = 2 * pp;
    return 2 * P * pp + 2 * P + P + 2 * pp * kt + (2 * P + pp + 1 + 1) / 2;
}

__device__ __forceinline__ IlvArrays bidirectional_arrays(int64_t *base, int pp, int kt)
{
    const int P = 2 * pp;
    IlvArrays A;
    A.ring_f = base;
    A.ring_b = A.ring_f + P * pp;
    A.cost = A.ring_b + P * pp;                    // [2 x]: forward item of pair x = pipeline * pp + stage, [2 x + 1]: backward
    A.last_b = A.cost + 2 * P;                     // start of the pair's last backward item
    A.kt = kt;
    A.tail = A.last_b + P;                         // [device][item mod kt][start, end]
    A.cnt_f = reinterpret_cast<int *>(A.tail + 2 * pp * kt);
    A.cnt_b = A.cnt_f + P;
    A.bounds = A.cnt_b + P;
    return A;
}

// How many items of each kind precede position `pos` (0 .. 2 m) of device d's order.
struct ItemsBefore { int f0, b0, f1, b1; };
__device__ __forceinline__ ItemsBefore items_before(const DeviceView &v, int64_t entry_off, int m, int d, int pos)
{
    const uint32_t w = __ldg(&v.order_before[entry_off + (int64_t)d * (2 * m + 1) + pos]);
    ItemsBefore n;
    n.f0 = (int)(w & 511u); n.b0 = (int)((w >> 9) & 511u); n.f1 = (int)((w >> 18) & 511u);
    n.b1 = pos - n.f0 - n.b0 - n.f1;
    return n;
}

// No (pp, m) keeps more items than this per device (the host checks it when it builds the orders):
// the shared memory of a candidate is sized with it.
__host__ __device__ inline int bidirectional_kept_cap(int pp) { return pp / 2 + 2; }

// Where an entry's orders start in DeviceView::order, and its kept items per device.
__device__ __forceinline__ int64_t order_offset(const DeviceView &v, int entry) { return __ldg(&v.order_off[entry]) & (((int64_t)1 << 48) - 1); }
__device__ __forceinline__ int order_kept(const DeviceView &v, int entry) { return (int)(__ldg(&v.order_off[entry]) >> 48); }

// True if the 2 dp devices that hold the stages of device d and of device pp - 1 - d share a node.
__device__ __forceinline__ bool mirror_group_near(const DeviceView &v, const Row &row, int d)
{
    if (v.tc.n_devices <= v.tc.gpus_per_node) return true;
    if (row.dp > 1 || row.mp >= v.tc.gpus_per_node) return false;
    const int per_node = v.tc.gpus_per_node / row.mp;          // pipeline devices of one replica per node
    return d / per_node == (row.pp - 1 - d) / per_node;
}

// The gradient buckets of stage [a, e) appended to a device's lane (see bucket_lane_chain), for a
// row whose partial-bucket table holds bytes: a full bucket costs t_full, the partial one is
// priced here, as an all-reduce over n devices.
template <class Visit>
__device__ __forceinline__ int64_t mirror_bucket_chain(const DeviceView &v, const int64_t *pb, const int64_t *nbt,
                                                       const int64_t *tpt, int a, int e, int64_t tb, int64_t main_end,
                                                       int64_t end, bool &any, int64_t t_full, int64_t n,
                                                       int64_t alpha, int64_t beta, Visit visit)
{
    const int L1 = v.tc.n_layers + 1;
    const int64_t *nbe = nbt + (int64_t)e * L1;
    const int64_t part_bytes = __ldg(&tpt[(int64_t)e * L1 + a]);
    const int64_t part = part_bytes > 0 ? allreduce_cost(v.tc, n, part_bytes, alpha, beta) : 0;
    if (!v.tc.overlap) {
        const int64_t full = __ldg(&nbe[a]);
        if (full == 0 && part_bytes == 0) return end;
        any = true;
        const int64_t start = max64(end, main_end);
        visit(start, start + full * t_full + part);
        return start + full * t_full + part;
    }
    const int64_t pbe = pb[e];
    if (v.tc.bucket > 0) {
        int64_t nb_prev = 0;
        for (int l = e - 1; l >= a; --l) {
            const int64_t nb_l = __ldg(&nbe[l]);
            const int64_t n_l = nb_l - nb_prev;     // full buckets whose last byte lies in layer l
            if (n_l > 0) {
                const int64_t start = max64(end, tb + (pbe - pb[l]));
                end = start + n_l * t_full;
                visit(start, end);
                any = true;
            }
            nb_prev = nb_l;
        }
    }
    if (part_bytes > 0) {
        const int lstar = __ldg(&v.next_grad[a]);
        const int64_t start = max64(end, tb + (pbe - pb[lstar]));
        end = start + part;
        visit(start, end);
        any = true;
    }
    return end;
}

// Evaluates one candidate of a two_way row by `seg` consecutive lanes of the calling warp (seg a
// power of two >= pp, pp <= 32; lane d < pp of the segment owns device d), every lane of the warp
// calling this together.  A: the candidate's arrays; afterwards A.bounds, A.cost and A.last_b
// describe the candidate.  rec (nullable): item start times go to rec[d * 2 m + position in the
// device's order].
__device__ __forceinline__ IlvResult bidirectional_candidate(const DeviceView &v, const Row &row, const Entry &en,
                                                             const CandidateCoords &cc, const int64_t *binom,
                                                             const IlvArrays &A, int64_t *rec, int seg)
{
    const int lane = (threadIdx.x & 31) & (seg - 1);         // lane within the candidate's segment
    const int pp = row.pp, P = 2 * pp, m = en.m, half = m >> 1, L = v.tc.n_layers;
    int64_t *ring_f = A.ring_f, *ring_b = A.ring_b, *cost = A.cost, *last_b = A.last_b, *tail = A.tail;
    int *cnt_f = A.cnt_f, *cnt_b = A.cnt_b, *bounds = A.bounds;
    const int kt = A.kt;

    // ---- the partition into pp stages -------------------------------------------------------
    if (v.sc.partition_mode == 0) {
        for (int s = lane; s <= pp; s += seg) bounds[s] = (int)((int64_t)s * L / pp);
    } else if (lane == 0) {
        // the (pp-1)-subsets of {1..L-1} in lexicographic order (combinatorial number system)
        int64_t r = cc.part_rank;
        int c = 0;
        bounds[0] = 0; bounds[pp] = L;
        for (int i = 1; i < pp; ++i) {
            ++c;
            while (true) {
                const int64_t n = binom[(int64_t)(L - 1 - c) * v.sc.binom_k + (pp - 1 - i)];
                if (r < n) break;
                r -= n;
                ++c;
            }
            bounds[i] = c;
        }
    }
    __syncwarp();
    const int64_t *pf = v.etf + (int64_t)cc.entry * v.tc.lp;
    const int64_t *pb = v.etb + (int64_t)cc.entry * v.tc.lp;
    for (int x = lane; x < P; x += seg) {
        const int u = x >= pp, s = x - u * pp;
        const int a = bounds[s], e = bounds[s + 1];
        // pipeline "down" sends across the boundary s | s + 1 (forward) and s - 1 | s (backward);
        // pipeline "up" runs on device pp - 1 - s and crosses the boundaries the other way round
        const int64_t send_f = s < pp - 1 ? p2p_cost(row, en, u ? pp - 2 - s : s) : 0;
        const int64_t send_b = s > 0 ? p2p_cost(row, en, u ? pp - 1 - s : s - 1) : 0;
        cost[2 * x] = __ldg(&pf[e]) - __ldg(&pf[a]) + send_f;
        cost[2 * x + 1] = __ldg(&pb[e]) - __ldg(&pb[a]) + send_b;
        cnt_f[x] = 0; cnt_b[x] = 0; last_b[x] = 0;
    }
    __syncwarp();

    // ---- the rounds: every device whose next item has its input runs it ---------------------
    const int d = lane;
    const uint16_t *mine = v.order + order_offset(v, cc.entry) + (int64_t)d * (2 * m + 1);
    int n_done = 0;
    int kept_at = 0;                                // n_done mod kt: where the next kept interval goes
    int64_t free_at = 0;
    // the merged order takes 2 m + pp - 2 rounds when m >= pp, never more than 2 (m + pp); the
    // segments of a warp may differ in m: all of them make the rounds of the longest
    const int limit = __reduce_max_sync(0xffffffffu, 2 * (m + pp) + 8);
    for (int round = 0; round < limit; ++round) {
        const bool pending = d < pp && n_done < 2 * m;
        if (!__any_sync(0xffffffffu, pending)) break;
        bool run = false, is_b = false;
        int x = 0, j = 0;
        int64_t dep = 0;
        if (pending) {
            const int item = mine[n_done];
            const int u = (item & kOrderUp) ? 1 : 0;
            is_b = (item & kOrderBackward) != 0;
            j = item & kOrderMicroBatch;
            const int s = u ? pp - 1 - d : d;
            x = u * pp + s;
            if (!is_b) {
                run = s == 0 || cnt_f[x - 1] > j;
                if (run && s > 0) dep = ring_f[(x - 1) * pp + (j & (pp - 1))];
            } else if (s == pp - 1) {
                run = true;                          // its own forward item came earlier in the device's order
                dep = ring_f[x * pp + (j & (pp - 1))];
            } else {
                run = cnt_b[x + 1] > j;
                if (run) dep = ring_b[(x + 1) * pp + (j & (pp - 1))];
            }
        }
        __syncwarp();                                // every device has read before any writes
        if (run) {
            const int64_t start = max64(dep, free_at);
            free_at = start + cost[2 * x + (is_b ? 1 : 0)];
            int64_t *slot = tail + 2 * (d * kt + kept_at);
            slot[0] = start; slot[1] = free_at;
            kept_at = kept_at + 1 == kt ? 0 : kept_at + 1;
            if (rec) rec[(int64_t)d * 2 * m + n_done] = start;
            if (is_b) {
                ring_b[x * pp + (j & (pp - 1))] = free_at;
                cnt_b[x] = j + 1;
                if (j == half - 1) last_b[x] = start;
            } else {
                ring_f[x * pp + (j & (pp - 1))] = free_at;
                cnt_f[x] = j + 1;
            }
            ++n_done;
        }
        __syncwarp();
    }
    if (d < pp && n_done < 2 * m) atomicCAS(v.status, 0, kStatusScheduleStuck);

    // ---- gradient buckets: the stream of the later stage first, both on the device's one lane --
    IlvResult R{0, 0, 0, 0};
    if (d < pp) {
        const int64_t main_end = free_at;
        int64_t dp_end = main_end, extra = 0;       // extra: time the buckets run while the main lane is idle
        {
            const int64_t *nbt = v.nb + row.row_tab_off, *tpt = v.tp + row.row_tab_off;
            const int64_t *kept = tail + 2 * d * kt;
            const int n_kept = min(kt, 2 * m);
            const bool near = mirror_group_near(v, row, d);
            const int64_t alpha = near ? v.tc.alpha_intra : v.tc.alpha_inter, beta = near ? v.tc.beta_intra : v.tc.beta_inter;
            const int64_t t_full = near ? row.t_full_near : row.t_full;
            int64_t end = 0;
            bool any = false;
            // activity is the union of all event intervals: a run of buckets adds its length less
            // what the kept items cover of it (no bucket starts before the first kept item does)
            auto visit = [&](int64_t bs, int64_t be) {
                int64_t covered = 0;
                for (int k = 0; k < n_kept; ++k) {
                    const int64_t lo = max64(bs, kept[2 * k]), hi = min(be, kept[2 * k + 1]);
                    covered += hi > lo ? hi - lo : 0;
                }
                extra += (be - bs) - covered;
            };
            const int s_hi = max(d, pp - 1 - d), s_lo = min(d, pp - 1 - d);
            for (int k = 0; k < 2; ++k) {
                const int s = k == 0 ? s_hi : s_lo;
                const int x = (s == d ? 0 : pp) + s;
                end = mirror_bucket_chain(v, pb, nbt, tpt, bounds[s], bounds[s + 1], last_b[x], main_end, end, any, t_full,
                                          2 * (int64_t)row.dp, alpha, beta, visit);
            }
            if (any) dp_end = end;
        }
        const int x_down = d, x_up = pp + (pp - 1 - d);
        R.busy = (int64_t)half * (cost[2 * x_down] + cost[2 * x_down + 1] + cost[2 * x_up] + cost[2 * x_up + 1]) + extra;
        R.main_end = main_end; R.dp_end = dp_end;
    }
    int64_t mx = max64(R.main_end, R.dp_end);
    for (int o = seg >> 1; o > 0; o >>= 1) mx = max64(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    R.batch = mx;
    return R;
}

}  // namespace distsim
