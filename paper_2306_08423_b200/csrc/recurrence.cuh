// Device code shared by the evaluation and the emission-planning kernels: candidate decoding
// and the lock-step form of the pipeline recurrence.
//
// Pipeline recurrence (Algorithm 1 of the paper): a schedule item (forward or backward pass of
// one micro-batch on one stage) starts at the later of (a) the end of the item it takes its
// input from on the neighbouring stage, including that item's trailing transfer event, and
// (b) the end of the previous item on its own device.  Because every micro-batch of a stage
// costs the same, an item is described by its stage's forward cost `fop` or backward cost `bop`.
//
// Lock-step form.  Give every item a unit-time "slot" s; then in both schedules
//   GPipe : F(d,j) runs in slot d + j,              B(d,j) in slot (m + 2pp - 2 - d) + j
//   1F1B  : F(d,j) runs in slot d + j  (j <  w_d),  B(d,j) in slot (2pp - 1 - d) + 2j
//           F(d,j) runs in slot d + 2j (j >= w_d),  with w_d = min(pp - d, m)
// all items finish within 2(m + pp - 1) slots, a stage runs at most one item per slot in its
// schedule's order, and when an item runs, the *most recent* forward (backward) item finished
// by the previous (next) stage before this slot is exactly the one it depends on.  So a lane
// that owns a stage keeps only the end of its latest item and fetches the neighbour's with a
// shuffle per slot (see lockstep_candidate).
#pragma once

#include "engine.h"

namespace distsim {

__device__ __forceinline__ int64_t max64(int64_t a, int64_t b) { return a > b ? a : b; }

// Bounds c_{d0} .. c_{d0+S} of partition number `part_rank` of the row's partitions.
// Balanced mode: c_j = floor(j L / pp).  All-compositions mode: the (pp-1)-subsets of
// {1..L-1} in lexicographic order, decoded with the combinatorial number system: position i
// takes the smallest value c whose block of C(L-1-c, pp-1-i) completions contains the rank.
// `binom`: the binomial table, in global memory (v.binom) or a block's copy of it in shared memory.
template <int S>
__device__ __forceinline__ void partition_bounds(const DeviceView &v, const int64_t *binom, int pp, int64_t part_rank,
                                                 int d0, int (&out)[S + 1])
{
    const int L = v.tc.n_layers;
    if (v.sc.partition_mode == 0) {
#pragma unroll
        for (int k = 0; k <= S; ++k) out[k] = (int)((int64_t)(d0 + k) * L / pp);
        return;
    }
#pragma unroll
    for (int k = 0; k <= S; ++k) out[k] = (d0 + k == 0) ? 0 : L;
    int64_t r = part_rank;
    int c = 0;
    const int last = min(pp - 1, d0 + S);
    for (int i = 1; i <= last; ++i) {
        ++c;
        const int kk = pp - 1 - i;
        while (true) {
            const int64_t cnt = binom[(int64_t)(L - 1 - c) * v.sc.binom_k + kk];
            if (r < cnt) break;
            r -= cnt;
            ++c;
        }
#pragma unroll
        for (int k = 0; k <= S; ++k) if (i == d0 + k) out[k] = c;
    }
}

// Copies the binomial table into shared memory when it fits `cap_words` (decoding a partition
// walks it with dependent loads); returns the table to use.  Every thread of the block calls it;
// contains a block-wide barrier.
__device__ __forceinline__ const int64_t *stage_binom(const DeviceView &v, int64_t *smem, int cap_words)
{
    const int words = v.sc.partition_mode ? v.tc.n_layers * v.sc.binom_k : 0;
    const bool fits = words > 0 && words <= cap_words;
    if (fits)
        for (int i = threadIdx.x; i < words; i += blockDim.x) smem[i] = __ldg(&v.binom[i]);
    __syncthreads();
    return fits ? smem : v.binom;
}

struct CandidateCoords {
    int entry;           // global entry index
    int sched;           // 0 GPipe, 1 1F1B, 2 asynchronous 1F1B (1F1B order, no gradient all-reduce)
    int64_t part_rank;
};

// Row-local index -> (entry, partition, schedule); the schedule varies fastest.
__device__ __forceinline__ CandidateCoords split_local(const Row &row, int64_t local)
{
    CandidateCoords cc;
    if (row.size < ((int64_t)1 << 32)) {
        const uint32_t l32 = (uint32_t)local;
        const uint32_t per_entry = (uint32_t)(row.n_part * row.n_sched);
        const uint32_t e = l32 / per_entry;
        const uint32_t rem = l32 - e * per_entry;
        cc.entry = row.entry0 + (int)e;
        cc.part_rank = rem / (uint32_t)row.n_sched;
        cc.sched = row_sched(row, (int)(rem - (uint32_t)cc.part_rank * (uint32_t)row.n_sched));
    } else {
        const int64_t per_entry = row.n_part * row.n_sched;
        const int64_t e = local / per_entry;
        const int64_t rem = local - e * per_entry;
        cc.entry = row.entry0 + (int)e;
        cc.part_rank = rem / row.n_sched;
        cc.sched = row_sched(row, (int)(rem - cc.part_rank * row.n_sched));
    }
    return cc;
}

// A stage's place in the lock-step slots, in a form both schedules share: the forward items
// j < w run in slot d + j and the others in slot d + 2j; the backward item j runs in slot
// b0 + (j << sh).  GPipe: w = m, b0 = m + 2pp - 2 - d, sh = 0; 1F1B: w = min(pp - d, m),
// b0 = 2pp - 1 - d, sh = 1.  A stage never has a forward and a backward item in one slot.
struct SlotPlan { int w, b0, sh; };
__device__ __forceinline__ SlotPlan slot_plan(int sched, int pp, int m, int d)
{
    SlotPlan sp;
    if (sched == 0) { sp.w = m; sp.b0 = m + 2 * pp - 2 - d; sp.sh = 0; }
    else { sp.w = min(pp - d, m); sp.b0 = 2 * pp - 1 - d; sp.sh = 1; }
    return sp;
}
// Activity of a stage over the kChunk slots s0 .. s0 + kChunk - 1 as bit masks (bit i: slot
// s0 + i): `fwd` the slots with a forward item, `bwd` those with a backward item.  Computed once
// per chunk, so that the slots themselves only test a bit.
constexpr int kChunk = 16;
__device__ __forceinline__ uint32_t slot_range_mask(int lo_slot, int hi_slot, int s0)
{
    const int lo = min(max(lo_slot - s0, 0), kChunk), hi = min(max(hi_slot - s0, 0), kChunk);
    return hi > lo ? (1u << hi) - (1u << lo) : 0u;
}
__device__ __forceinline__ void chunk_activity(const SlotPlan &sp, int m, int d, int s0, uint32_t &fwd, uint32_t &bwd)
{
    // bits of the slots whose distance from slot `from` is even
    auto alternate = [&](int from) { return ((from - s0) & 1) ? 0xAAAAAAAAu : 0x55555555u; };
    fwd = slot_range_mask(d, d + sp.w, s0) |                                          // d + j, j < w
          (slot_range_mask(d + 2 * sp.w, d + 2 * m - 1, s0) & alternate(d));          // d + 2j, w <= j < m
    bwd = slot_range_mask(sp.b0, sp.b0 + ((m - 1) << sp.sh) + 1, s0) & (sp.sh ? alternate(sp.b0) : 0xFFFFFFFFu);
}

// Extra time of the item of micro-batch j on stage d (0 without a jitter table).
__device__ __forceinline__ int64_t jitter_of(const DeviceView &v, const int64_t *table, int j, int d)
{
    return v.tc.n_jitter ? __ldg(&table[(j & (v.tc.n_jitter - 1)) * v.tc.jitter_stages + d]) : 0;
}

// Gradient all-reduce buckets of one stage [a, e) appended to a communication lane (DP modeling).
// `tb` is the start of the stage's last backward item, `main_end` the end of the device's main
// lane, `end` the end of the lane's buckets so far (0: none yet).  pb: the entry's backward prefix
// row; nbt/tpt: the row's bucket tables.  Returns the lane's new end and sets `any` if the stage
// has a bucket; visit(start, end) is called for every run of buckets that follow each other
// without a gap.
template <class Visit>
__device__ __forceinline__ int64_t bucket_lane_chain(const DeviceView &v, const Row &row,
                                                     const int64_t *pb, const int64_t *nbt,
                                                     const int64_t *tpt, int a, int e, int64_t tb,
                                                     int64_t main_end, int64_t end, bool &any, Visit visit)
{
    const int L1 = v.tc.n_layers + 1;
    const int64_t *nbe = nbt + (int64_t)e * L1;
    const int64_t part = __ldg(&tpt[(int64_t)e * L1 + a]);
    if (!v.tc.overlap) {
        const int64_t full = __ldg(&nbe[a]);
        if (full == 0 && part == 0) return end;
        any = true;
        const int64_t start = max64(end, main_end);
        visit(start, start + full * row.t_full + part);
        return start + full * row.t_full + part;
    }
    // a bucket is ready when the layer holding its last byte has finished its backward
    // composite in the last backward item; buckets then run back to back
    const int64_t pbe = pb[e];
    if (v.tc.bucket > 0) {
        int64_t nb_prev = 0;                   // nb[e][l+1]
        for (int l = e - 1; l >= a; --l) {
            const int64_t nb_l = __ldg(&nbe[l]);
            const int64_t n_l = nb_l - nb_prev; // full buckets whose last byte lies in layer l
            if (n_l > 0) {
                const int64_t start = max64(end, tb + (pbe - pb[l]));
                end = start + n_l * row.t_full;
                visit(start, end);
                any = true;
            }
            nb_prev = nb_l;
        }
    }
    if (part > 0) {
        // the trailing bucket ends in the stage's first layer that has any gradient bytes
        const int lstar = __ldg(&v.next_grad[a]);
        const int64_t start = max64(end, tb + (pbe - pb[lstar]));
        end = start + part;
        visit(start, end);
        any = true;
    }
    return end;
}

// The same for a device with one stage: the end of its bucket lane (main_end when the stage
// sends no gradients).
__device__ __forceinline__ int64_t bucket_lane_end(const DeviceView &v, const Row &row,
                                                   const int64_t *pb, const int64_t *nbt,
                                                   const int64_t *tpt, int a, int e, int64_t tb,
                                                   int64_t main_end)
{
    if (row.dp == 1) return main_end;
    bool any = false;
    const int64_t end = bucket_lane_chain(v, row, pb, nbt, tpt, a, e, tb, main_end, 0, any, [](int64_t, int64_t) {});
    return any ? end : main_end;
}

// Result of one candidate on the lanes that own its stages (S stages per lane).
template <int S>
struct StageResult {
    int a[S], e[S];              // layer range [a, e) of each owned stage
    int64_t fop[S], bop[S];      // cost of a forward / backward item incl. trailing transfer
    int64_t main_end[S];         // end of the stage's last item
    int64_t last_b_start[S];     // start of the first layer event of the stage's last backward item
    int64_t dp_end[S];           // end of the gradient-bucket lane
    int64_t busy[S];             // activity time of a device of the stage
    int64_t batch;               // max over all stages (same on every lane of the segment)
};

// Cost of the transfer across boundary d | d+1 for this entry.
__device__ __forceinline__ int64_t p2p_cost(const Row &row, const Entry &en, int d)
{
    return (((d + 1) & (row.p2p_period - 1)) == 0) ? en.p2p_inter : en.p2p_intra;
}

__device__ __forceinline__ int64_t shfl_idx64(int64_t x, int src_lane)
{
    const uint32_t lo = __shfl_sync(0xffffffffu, (uint32_t)x, src_lane);
    const uint32_t hi = __shfl_sync(0xffffffffu, (uint32_t)((uint64_t)x >> 32), src_lane);
    return (int64_t)(((uint64_t)hi << 32) | lo);
}
// Stores `value` at `where` on the lanes where `on` holds: a predicated store, so that the slots
// of the lock-step form stay free of branches.
__device__ __forceinline__ void store_if(bool on, int64_t *where, int64_t value)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.s32 p, %0, 0;\n\t@p st.global.b64 [%1], %2;\n\t}"
                 :: "r"((int)on), "l"(where), "l"(value) : "memory");
}
// The state word of the lock-step form in either width (uint32_t: entries whose time bound is
// below 2^32, one shuffle and single-word compares per slot).
__device__ __forceinline__ int64_t shfl_idx(int64_t x, int src_lane) { return shfl_idx64(x, src_lane); }
__device__ __forceinline__ uint32_t shfl_idx(uint32_t x, int src_lane) { return __shfl_sync(0xffffffffu, x, src_lane); }

// Lock-step evaluation of one candidate by `wl` consecutive lanes (wl * S == pp), every lane of
// the warp calling this together (lanes of other segments work on their own candidates).
//   entry_index  global index of `en`;  seg_lane: lane index inside the segment;
//   n_slots_warp loop bound, uniform over the warp
//   pf, pb     the entry's forward / backward prefix rows (shared or global memory)
//   rec        if kRecord and non-null: item start times go to rec[d * 2m + position in stage order]
//   binom      the binomial table of the partition decoding (global, or the block's shared copy)
//   kJit       the table has per-micro-batch jitter (otherwise none of its code is generated)
// Per stage the only state is t, the end of the stage's latest item (= when its device is free).
// When an item runs, the item it takes its input from ran on the neighbouring stage in the slot
// before, or (the first forward item after a 1F1B warm-up) is still that stage's latest item; so
// the input's arrival is the neighbour's t as of the previous slot, and a slot is
//   t = max(neighbour's t, t) + cost
// with the neighbour chosen by the kind of item (previous stage for a forward item, next stage
// for a backward one, the stage itself - a no-op - when it idles or has no such neighbour: the
// first stage's forward items and the last stage's backward items wait for their own device only).
// One stage per lane fetches exactly that value with one indexed shuffle per slot.
//   T          type of the times inside the slots: int64_t, or uint32_t when the entry's time
//              bound is below 2^32 (exact: no time of the candidate can reach the bound)
template <int S, bool kRecord, bool kJit, class T = int64_t>
__device__ __forceinline__ StageResult<S> lockstep_candidate(
    const DeviceView &v, const Row &row, const Entry &en, int entry_index, const int64_t *pf,
    const int64_t *pb, int sched, int64_t part_rank, int seg_lane, int wl, int n_slots_warp, int64_t *rec,
    const int64_t *binom)
{
    StageResult<S> R;
    const int pp = row.pp, m = en.m;
    const int d0 = seg_lane * S;
    int bounds[S + 1];
    partition_bounds<S>(v, binom, pp, part_rank, d0, bounds);
    SlotPlan sp[S];
#pragma unroll
    for (int k = 0; k < S; ++k) {
        const int d = d0 + k;
        R.a[k] = bounds[k]; R.e[k] = bounds[k + 1];
        R.fop[k] = pf[R.e[k]] - pf[R.a[k]] + (d < pp - 1 ? p2p_cost(row, en, d) : 0);
        R.bop[k] = pb[R.e[k]] - pb[R.a[k]] + (d > 0 ? p2p_cost(row, en, d - 1) : 0);
        sp[k] = slot_plan(sched, pp, m, d);
    }
    T t[S], fop[S], bop[S];
    int n_f[S], n_b[S];                  // forward / backward items done: the next item's micro-batch
    int64_t *rp[S];                      // where the next item's start goes (a stage's items are consecutive)
    const bool recording = kRecord && rec != nullptr;
#pragma unroll
    for (int k = 0; k < S; ++k) {
        t[k] = 0; n_f[k] = 0; n_b[k] = 0;
        fop[k] = (T)R.fop[k]; bop[k] = (T)R.bop[k];
        rp[k] = (kRecord && rec) ? rec + (int64_t)(d0 + k) * 2 * m : nullptr;
    }
    const int lane = threadIdx.x & 31;
    // where a forward (backward) item's input comes from: the previous (next) lane, or the lane
    // itself when there is no such stage (one stage per lane)
    const int src_f = d0 > 0 ? lane - 1 : lane, src_b = d0 < pp - 1 ? lane + 1 : lane;

    for (int s0 = 0; s0 < n_slots_warp; s0 += kChunk) {
        uint32_t fm[S], bm[S];
#pragma unroll
        for (int k = 0; k < S; ++k) chunk_activity(sp[k], m, d0 + k, s0, fm[k], bm[k]);
#pragma unroll
        for (int i = 0; i < kChunk; ++i) {
            if (S == 1) {
                const bool do_f = (fm[0] >> i) & 1u, do_b = (bm[0] >> i) & 1u;
                T cost = do_f ? fop[0] : (do_b ? bop[0] : (T)0);
                if (kJit) {
                    if (do_f) cost += (T)jitter_of(v, v.raw.jit_f, n_f[0], d0);
                    if (do_b) cost += (T)jitter_of(v, v.raw.jit_b, n_b[0], d0);
                }
                const T dep = shfl_idx(t[0], do_f ? src_f : (do_b ? src_b : lane));
                const T own = t[0] + cost, via = dep + cost;             // both ready before the compare ends
                const bool late = dep > t[0];
                if (kRecord) {
                    const bool item = recording && (do_f || do_b);
                    store_if(item, rp[0], (int64_t)(late ? dep : t[0]));
                    rp[0] += item ? 1 : 0;
                }
                t[0] = late ? via : own;
                if (kJit) { n_f[0] += do_f ? 1 : 0; n_b[0] += do_b ? 1 : 0; }
            } else {
                // several stages per lane: the lane's first (last) stage takes the previous (next)
                // lane's last (first) stage, the others their neighbour inside the lane
                const T up_f = __shfl_up_sync(0xffffffffu, t[S - 1], 1, wl);
                const T dn_b = __shfl_down_sync(0xffffffffu, t[0], 1, wl);
                T old[S];
#pragma unroll
                for (int k = 0; k < S; ++k) old[k] = t[k];
#pragma unroll
                for (int k = 0; k < S; ++k) {
                    const int d = d0 + k;
                    const bool do_f = (fm[k] >> i) & 1u, do_b = (bm[k] >> i) & 1u;
                    T cost = do_f ? fop[k] : (do_b ? bop[k] : (T)0);
                    if (kJit) {
                        if (do_f) cost += (T)jitter_of(v, v.raw.jit_f, n_f[k], d);
                        if (do_b) cost += (T)jitter_of(v, v.raw.jit_b, n_b[k], d);
                    }
                    const T dep_f = (k == 0) ? (d == 0 ? (T)0 : up_f) : old[k > 0 ? k - 1 : 0];
                    const T dep_b = (k == S - 1) ? (d == pp - 1 ? (T)0 : dn_b) : old[k < S - 1 ? k + 1 : 0];
                    const T dep = do_f ? dep_f : (do_b ? dep_b : (T)0);
                    const T own = old[k] + cost, via = dep + cost;
                    const bool late = dep > old[k];
                    if (kRecord) {
                        const bool item = recording && (do_f || do_b);
                        store_if(item, rp[k], (int64_t)(late ? dep : old[k]));
                        rp[k] += item ? 1 : 0;
                    }
                    t[k] = late ? via : own;
                    if (kJit) { n_f[k] += do_f ? 1 : 0; n_b[k] += do_b ? 1 : 0; }
                }
            }
        }
    }

    const int64_t *nbt = v.nb + row.row_tab_off;
    const int64_t *tpt = v.tp + row.row_tab_off;
    int64_t mx = 0;
#pragma unroll
    for (int k = 0; k < S; ++k) {
        R.main_end[k] = (int64_t)t[k];
        // every stage's last item is the backward item of the last micro-batch; its first layer
        // event starts one backward item cost before its end
        R.last_b_start[k] = (int64_t)t[k] - R.bop[k];
        // the asynchronous schedule has no gradient all-reduce events
        if (sched == 2 || row.dp == 1) {
            R.dp_end[k] = R.main_end[k];
        } else if (v.dt) {
            // per-entry bucket-lane table: the lane's end relative to the start of the last
            // backward item (overlap; negative: no buckets) or the buckets' total cost
            const int64_t val = __ldg(&v.dt[(int64_t)entry_index * v.tab_words + R.e[k] * (v.tc.n_layers + 1) + R.a[k]]);
            R.dp_end[k] = v.tc.overlap ? (val < 0 ? R.main_end[k] : R.last_b_start[k] + val) : R.main_end[k] + val;
        } else {
            R.dp_end[k] = bucket_lane_end(v, row, pb, nbt, tpt, R.a[k], R.e[k], R.last_b_start[k], R.main_end[k]);
        }
        const int64_t extra = R.dp_end[k] - R.main_end[k];
        R.busy[k] = (int64_t)m * (R.fop[k] + R.bop[k]) + (extra > 0 ? extra : 0) +
                    (kJit ? __ldg(&v.jsum[(int64_t)entry_index * DISTSIM_MAX_PP + d0 + k]) : 0);
        mx = max64(mx, max64(R.main_end[k], R.dp_end[k]));
    }
    for (int off = 1; off < wl; off <<= 1) mx = max64(mx, __shfl_xor_sync(0xffffffffu, mx, off, wl));
    R.batch = mx;
    return R;
}

}  // namespace distsim
