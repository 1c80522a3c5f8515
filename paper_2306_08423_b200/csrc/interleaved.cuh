// Interleaved 1F1B: evaluation of candidates whose devices hold v model chunks each.
//
// The model is cut into P = pp * v virtual stages; virtual stage s = c * pp + d is chunk c of
// device d, so consecutive virtual stages sit on consecutive devices and the last device sends
// to the first between chunks.  Algorithm 1 of the paper runs unchanged over virtual stages with
// one free time per device; what the schedule fixes is the order of a device's 2 m v items
// (m a multiple of pp): the k-th forward item is chunk (k / pp) mod v of micro-batch
// (k / (pp v)) pp + k mod pp, the k-th backward item the same with chunk v - 1 - (k / pp) mod v;
// device d first runs min(m v, 2 (pp - d - 1) + (v - 1) pp) forward items (all of them when
// m = pp), then one forward and one backward item in turn, then the backward items left.
//
// One warp evaluates a candidate, a lane per device, in rounds: in a round every device whose
// next item has its input (produced in an earlier round) runs it.  That is list scheduling with
// unit item times, which takes 2 (m v + pp - 1) rounds; the simulated times ride along:
//   end = max(arrival of the input, device free) + cost of the item.
// An item's end is handed to the item that consumes it through a ring per virtual stage and
// direction in shared memory, indexed by micro-batch mod pp: in round order no more than pp
// ends of one ring are ever waiting (the forward items of a group of pp micro-batches on the
// last virtual stage, when m = pp), and a counter per ring says how many have been produced.
#pragma once

#include "recurrence.cuh"

namespace distsim {

constexpr int kIlvThreads = 64;                 // two warps of 32 / pp candidates each
constexpr int32_t kStatusScheduleStuck = -71;   // device status: the rounds ran out (never seen)

// The last items of a device that are kept with their start and end: from the last backward item
// of the chunk that finishes first (chunk v - 1) on, (v - 1) pp + 2 items at most.  Gradient
// buckets can run while the device idles between them, which counts as activity.
__host__ __device__ inline int interleaved_tail_items(int pp, int v) { return (v - 1) * pp + 2; }

// Shared memory of one candidate, in int64 words: two rings of pp ends per virtual stage, the
// forward and backward item cost of every virtual stage, the start of its last backward item,
// the (start, end) of every device's last items, then (as 32-bit values) the two production
// counters per virtual stage and the P + 1 bounds.
__host__ __device__ inline int interleaved_words(int pp, int v)
{
    const int P = pp * v;
    return 2 * P * pp + 2 * P + P + 2 * pp * interleaved_tail_items(pp, v) + (2 * P + P + 1 + 1) / 2;
}

// Cost of the transfer from virtual stage s to s + 1 (devices s mod pp and (s + 1) mod pp): the
// usual neighbour transfer, or from the last device back to the first, which stays inside a node
// only if a whole pipeline replica does.
__device__ __forceinline__ int64_t virtual_p2p_cost(const DeviceView &v, const Row &row, const Entry &en, int s)
{
    const int d = s & (row.pp - 1);
    if (d < row.pp - 1) return p2p_cost(row, en, d);
    return row.mp * row.pp <= v.tc.gpus_per_node ? en.p2p_intra : en.p2p_inter;
}

// A candidate's arrays in the shared memory of its warp (see interleaved_words).
struct IlvArrays {
    int64_t *ring_f, *ring_b, *cost, *last_b, *tail;
    int *cnt_f, *cnt_b, *bounds;
    int kt;
};
__device__ __forceinline__ IlvArrays interleaved_arrays(int64_t *base, int pp, int vch)
{
    const int P = pp * vch;
    IlvArrays A;
    A.ring_f = base;
    A.ring_b = A.ring_f + P * pp;
    A.cost = A.ring_b + P * pp;                    // [2 s]: forward item of virtual stage s, [2 s + 1]: backward
    A.last_b = A.cost + 2 * P;                     // start of the last backward item (micro-batch m - 1)
    A.kt = interleaved_tail_items(pp, vch);
    A.tail = A.last_b + P;                         // [device][item mod kt][start, end]
    A.cnt_f = reinterpret_cast<int *>(A.tail + 2 * pp * A.kt);
    A.cnt_b = A.cnt_f + P;
    A.bounds = A.cnt_b + P;
    return A;
}

// What a lane knows of its device after the evaluation.
struct IlvResult { int64_t main_end, dp_end, busy, batch; };

// Evaluates one interleaved candidate by `seg` consecutive lanes of the calling warp (seg a power
// of two >= pp; lane d < pp of the segment owns device d), every lane of the warp calling this
// together: the other segments work on candidates of their own.  A: the candidate's arrays;
// afterwards A.bounds, A.cost and A.last_b describe the candidate.
// rec (nullable): item start times go to rec[d * 2 m v + position in the device's order].
__device__ __forceinline__ IlvResult interleaved_candidate(const DeviceView &v, const Row &row, const Entry &en,
                                                           const CandidateCoords &cc, const int64_t *binom,
                                                           const IlvArrays &A, int64_t *rec, int seg)
{
    const int lane = (threadIdx.x & 31) & (seg - 1);         // lane within the candidate's segment
    const int pp = row.pp, vch = row.v, P = pp * vch, m = en.m, L = v.tc.n_layers;
    const int log_pp = 31 - __clz(pp), log_v = 31 - __clz(vch);
    int64_t *ring_f = A.ring_f, *ring_b = A.ring_b, *cost = A.cost, *last_b = A.last_b, *tail = A.tail;
    int *cnt_f = A.cnt_f, *cnt_b = A.cnt_b, *bounds = A.bounds;
    const int kt = A.kt;

    // ---- the partition into P virtual stages --------------------------------------------------
    if (v.sc.partition_mode == 0) {
        for (int s = lane; s <= P; s += seg) bounds[s] = (int)((int64_t)s * L / P);
    } else if (lane == 0) {
        // the (P-1)-subsets of {1..L-1} in lexicographic order (combinatorial number system)
        int64_t r = cc.part_rank;
        int c = 0;
        bounds[0] = 0; bounds[P] = L;
        for (int i = 1; i < P; ++i) {
            ++c;
            while (true) {
                const int64_t n = binom[(int64_t)(L - 1 - c) * v.sc.binom_k + (P - 1 - i)];
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
    for (int s = lane; s < P; s += seg) {
        const int a = bounds[s], e = bounds[s + 1];
        cost[2 * s] = __ldg(&pf[e]) - __ldg(&pf[a]) + (s < P - 1 ? virtual_p2p_cost(v, row, en, s) : 0);
        cost[2 * s + 1] = __ldg(&pb[e]) - __ldg(&pb[a]) + (s > 0 ? virtual_p2p_cost(v, row, en, s - 1) : 0);
        cnt_f[s] = 0; cnt_b[s] = 0; last_b[s] = 0;
    }
    __syncwarp();

    // ---- the rounds ---------------------------------------------------------------------------
    const int d = lane;
    const int total = m * vch;                      // forward (and backward) items of a device
    int warm = (pp - d - 1) * 2 + (vch - 1) * pp;
    if (m == pp || warm > total) warm = total;
    int n_f = 0, n_b = 0;
    int kept_at = 0;                                // (items run) mod kt: where the next kept interval goes
    int64_t free_at = 0;
    // (the segments of a warp may differ in m: all of them make the rounds of the longest)
    const int limit = __reduce_max_sync(0xffffffffu, 2 * (total + pp) + 8);
    for (int round = 0; round < limit; ++round) {
        const bool pending = d < pp && n_f + n_b < 2 * total;
        if (!__any_sync(0xffffffffu, pending)) break;
        // the device's next item and, if it is there, its input
        bool run = false, is_b = false;
        int s = 0, j = 0;
        int64_t dep = 0;
        if (pending) {
            const int step = n_f + n_b;
            is_b = n_f < warm ? false : (n_f < total ? ((step - warm) & 1) : true);
            const int idx = is_b ? n_b : n_f;
            const int c0 = (idx >> log_pp) & (vch - 1);
            const int c = is_b ? vch - 1 - c0 : c0;
            j = ((idx >> (log_pp + log_v)) << log_pp) + (idx & (pp - 1));
            s = c * pp + d;
            if (!is_b) {
                run = s == 0 || cnt_f[s - 1] > j;
                if (run && s > 0) dep = ring_f[(s - 1) * pp + (j & (pp - 1))];
            } else if (s == P - 1) {
                run = true;                          // its own forward item came earlier in the device's order
                dep = ring_f[s * pp + (j & (pp - 1))];
            } else {
                run = cnt_b[s + 1] > j;
                if (run) dep = ring_b[(s + 1) * pp + (j & (pp - 1))];
            }
        }
        __syncwarp();                                // every device has read before any writes
        if (run) {
            const int64_t start = max64(dep, free_at);
            free_at = start + cost[2 * s + (is_b ? 1 : 0)];
            int64_t *slot = tail + 2 * (d * kt + kept_at);
            slot[0] = start; slot[1] = free_at;
            kept_at = kept_at + 1 == kt ? 0 : kept_at + 1;
            if (rec) rec[(int64_t)d * 2 * total + n_f + n_b] = start;
            if (is_b) {
                ring_b[s * pp + (j & (pp - 1))] = free_at;
                cnt_b[s] = j + 1;
                if (j == m - 1) last_b[s] = start;
                ++n_b;
            } else {
                ring_f[s * pp + (j & (pp - 1))] = free_at;
                cnt_f[s] = j + 1;
                ++n_f;
            }
        }
        __syncwarp();
    }
    if (d < pp && n_f + n_b < 2 * total) atomicCAS(v.status, 0, kStatusScheduleStuck);

    // ---- gradient buckets: one stream per chunk, the chunk whose backward finishes first (the
    //      last one) first, chained on the device's one lane; then the reduction --------------
    IlvResult R{0, 0, 0, 0};
    if (d < pp) {
        const int64_t main_end = free_at;
        int64_t dp_end = main_end, extra = 0;       // extra: time the buckets run while the main lane is idle
        if (row.dp > 1) {
            const int64_t *nbt = v.nb + row.row_tab_off, *tpt = v.tp + row.row_tab_off;
            const int64_t *mine = tail + 2 * d * kt;
            const int n_kept = min(kt, 2 * total);
            int64_t end = 0;
            bool any = false;
            // activity is the union of all event intervals: a run of buckets adds its length less
            // what the kept items cover of it (no bucket starts before the first kept item does)
            auto visit = [&](int64_t bs, int64_t be) {
                int64_t covered = 0;
                for (int k = 0; k < n_kept; ++k) {
                    const int64_t lo = max64(bs, mine[2 * k]), hi = min(be, mine[2 * k + 1]);
                    covered += hi > lo ? hi - lo : 0;
                }
                extra += (be - bs) - covered;
            };
            for (int c = vch - 1; c >= 0; --c) {
                const int s = c * pp + d;
                end = bucket_lane_chain(v, row, pb, nbt, tpt, bounds[s], bounds[s + 1], last_b[s], main_end, end, any, visit);
            }
            if (any) dp_end = end;
        }
        for (int c = 0; c < vch; ++c) R.busy += (int64_t)m * (cost[2 * (c * pp + d)] + cost[2 * (c * pp + d) + 1]);
        R.busy += extra;
        R.main_end = main_end; R.dp_end = dp_end;
    }
    int64_t mx = max64(R.main_end, R.dp_end);
    for (int o = seg >> 1; o > 0; o >>= 1) mx = max64(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    R.batch = mx;
    return R;
}

}  // namespace distsim
