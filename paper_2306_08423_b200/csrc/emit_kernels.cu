// Timeline emission: per-device event records (kind, layer, microbatch, start_ns, end_ns) of
// selected candidates, plus per-device activity time and utilisation.
//
//   emit_plan_kernel     one warp per selected candidate: decode it, run the lock-step recurrence
//                        while recording every item's start time into scratch, count records; the
//                        last block to finish scans the per-candidate record totals.
//   emit_devices_kernel  per (candidate, device): record offset, activity time, utilisation.
//   emit_items_kernel    the bandwidth-bound part.  A block owns (candidate, stage, run of
//                        consecutive items, chunk of replicas).  It builds the stage's forward
//                        and backward item templates (records relative to the item's start) in
//                        shared memory once, then an image of the whole run: a warp per item, a
//                        word is template word + {0, 0, microbatch, start, start}.  The stage's
//                        mp*dp replicas hold identical lists, so the image is computed once and
//                        written to each replica of the chunk by one bulk asynchronous copy
//                        (cp.async.bulk shared -> global) issued by one lane per replica.
//   emit_buckets_kernel  gradient-bucket records of every stage.
#include "recurrence.cuh"
#include "smem_stage.cuh"
#include "bidirectional.cuh"

namespace distsim {

namespace {

constexpr int kItemThreads = 256;
constexpr int kMaxTileItems = 256;  // most schedule items per block (a plan picks its own count)
constexpr int kTileWords = 3872;    // largest capacity of a block's image of its run, in int64 words
constexpr int kRunWords = 3872;     // run length the plans aim at (three blocks per SM; shorter runs
                                    // measured slower: the per-block set-up weighs more)
constexpr int kTileReplicas = 16;   // replicas per block
constexpr int kBucketRun = 768;     // gradient buckets per shared-memory image (5 words each)
constexpr int kBucketReplicas = 32; // replicas per block of the bucket kernel: one lane of the first warp each
// the longest item: every layer with computation, all-reduce and all-to-all, a jitter event, a transfer
static_assert((3 * DISTSIM_MAX_LAYERS + 2) * 5 <= kTileWords && kTileWords % 2 == 0, "an item must fit the image");

// The row that holds candidate `index`.  Every lane of the warp calls this with the same index;
// the lanes look at 32 rows at a time (the rows' offsets ascend from 0).
__device__ __forceinline__ int find_row(const DeviceView &v, int64_t index)
{
    const int lane = threadIdx.x & 31;
    int found = 0;
    for (int base = 0; base < v.sc.n_rows; base += 32) {
        const int r = base + lane;
        const bool at_or_before = r < v.sc.n_rows && __ldg(&v.rows[r].offset) <= index;
        const unsigned int mask = __ballot_sync(0xffffffffu, at_or_before);
        if (!mask) break;
        found = base + 31 - __clz(mask);
    }
    return found;
}

// Words of a selection's summary: what the scan over all selections needs of its plan.
enum { kSumRecords = 0, kSumItemTiles, kSumBucketTiles, kSumTmplWords, kSumBucketRecs, kSumRunWords, kSumWords = 8 };
static_assert(kSumWords == kEmitSumWords, "the context sizes the summaries");

template <int S>
__device__ __forceinline__ void plan_candidate(const DeviceView &v, const Row &row, int row_index,
                                               int64_t index, EmitPlan *plan, int64_t *rec, const int64_t *binom,
                                               int64_t *sum /* the selection's words of the summary the scan reads */)
{
    const int lane = threadIdx.x & 31;
    const int wl = row.pp / S;
    const int seg_lane = lane % wl;
    const bool owner = lane < wl;          // the other segments of the warp shadow the same candidate
    const CandidateCoords cc = split_local(row, index - row.offset);
    const Entry en = v.entries[cc.entry];
    const int64_t *pf = v.etf + (int64_t)cc.entry * v.tc.lp;
    const int64_t *pb = v.etb + (int64_t)cc.entry * v.tc.lp;
    const int n_slots = 2 * (en.m + row.pp - 1);
    // times of an entry whose bound is below 2^32 fit 32 bits: half the instructions per slot
    const bool narrow = S == 1 && v.tc.n_jitter == 0 && en.bound < ((int64_t)1 << 32);
    const StageResult<S> R = v.tc.n_jitter > 0
        ? lockstep_candidate<S, true, true>(v, row, en, cc.entry, pf, pb, cc.sched, cc.part_rank, seg_lane, wl,
                                            n_slots, owner ? rec : nullptr, binom)
        : narrow
        ? lockstep_candidate<S, true, false, uint32_t>(v, row, en, cc.entry, pf, pb, cc.sched, cc.part_rank, seg_lane,
                                                       wl, n_slots, owner ? rec : nullptr, binom)
        : lockstep_candidate<S, true, false>(v, row, en, cc.entry, pf, pb, cc.sched, cc.part_rank, seg_lane, wl,
                                             n_slots, owner ? rec : nullptr, binom);
    // per stage: records of a forward / backward item, gradient buckets, records of one device;
    // their prefix over the stages and the widest item by shuffles over the lanes that own stages
    int64_t recs[S], kbs[S];
    int widest = 1, both = 2;
    int64_t lane_recs = 0;
    if (owner) {
        const int L1 = v.tc.n_layers + 1;
#pragma unroll
        for (int k = 0; k < S; ++k) {
            const int d = seg_lane * S + k;
            const int a = R.a[k], e = R.e[k];
            const int n_layers = e - a;
            const int n_exp = v.pe[e] - v.pe[a];
            const int64_t per_dir = (int64_t)n_layers * (row.mp > 1 ? 2 : 1) + (row.dp > 1 ? n_exp : 0) +
                                    (v.tc.n_jitter > 0 ? 1 : 0);      // an item starts with its jitter event
            const int64_t rf = per_dir + (d < row.pp - 1 ? 1 : 0);
            const int64_t rb = per_dir + (d > 0 ? 1 : 0);
            int64_t kb = 0;
            if (row.dp > 1 && cc.sched != 2) {              // no buckets in the asynchronous schedule
                const int64_t *nbt = v.nb + row.row_tab_off, *tpt = v.tp + row.row_tab_off;
                kb = nbt[(int64_t)e * L1 + a] + (tpt[(int64_t)e * L1 + a] > 0 ? 1 : 0);
            }
            recs[k] = (int64_t)en.m * (rf + rb) + kb;
            kbs[k] = kb;
            lane_recs += recs[k];
            widest = max(widest, (int)max(rf, rb));
            both = max(both, (int)(rf + rb));
            plan->bounds[d] = a;
            if (d == row.pp - 1) plan->bounds[row.pp] = e;
            plan->rf[d] = (int32_t)rf; plan->rb[d] = (int32_t)rb;
            plan->n_buckets[d] = kb;
            plan->stage_recs[d] = recs[k];
            plan->busy[d] = R.busy[k];
            plan->main_end[d] = R.main_end[k];
            plan->last_b_start[d] = R.last_b_start[k];
        }
    }
    int64_t incl = lane_recs;                      // lanes that own no stage contribute nothing
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int64_t up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    const int64_t total = __shfl_sync(0xffffffffu, incl, 31);
    int64_t most_buckets = 0;
    if (owner) {
#pragma unroll
        for (int k = 0; k < S; ++k) most_buckets = max64(most_buckets, kbs[k]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        widest = max(widest, __shfl_xor_sync(0xffffffffu, widest, o));
        both = max(both, __shfl_xor_sync(0xffffffffu, both, o));
        most_buckets = max64(most_buckets, __shfl_xor_sync(0xffffffffu, most_buckets, o));
    }
    if (owner) {
        int64_t acc = incl - lane_recs;
#pragma unroll
        for (int k = 0; k < S; ++k) { plan->stage_rec_prefix[seg_lane * S + k] = acc; acc += recs[k]; }
    }
    if (lane == 0) {
        plan->index = index; plan->batch_ns = R.batch;
        plan->row = row_index; plan->entry = cc.entry; plan->m = en.m; plan->sched = cc.sched;
        plan->pp = row.pp; plan->mp = row.mp; plan->dp = row.dp; plan->ok = 1; plan->v = 1; plan->two_way = 0;
        plan->stage_rec_prefix[row.pp] = total;
        plan->rec_total = total * row.mp * row.dp;
        // a run of tile_items items of any mix must fit the image of kTileWords words
        // a run aims at kRunWords words (small images: more blocks per SM), holds at least one item
        const int cap = max(1, min(kMaxTileItems, kRunWords / (widest * 5)));
        const int n_chunks = (2 * en.m + cap - 1) / cap;          // equal runs rather than full ones and a rest
        plan->tile_items = (2 * en.m + n_chunks - 1) / n_chunks;
        plan->run_words = plan->tile_items * widest * 5;          // no run of this selection is longer
        plan->tmpl_words = both * 5;
        const int64_t reps = (int64_t)row.mp * row.dp;
        sum[kSumRecords] = plan->rec_total;
        sum[kSumItemTiles] = (int64_t)row.pp * ((2 * en.m + plan->tile_items - 1) / plan->tile_items) *
                             ((reps + kTileReplicas - 1) / kTileReplicas);
        sum[kSumBucketTiles] = (int64_t)row.pp * ((reps + kBucketReplicas - 1) / kBucketReplicas);
        sum[kSumTmplWords] = plan->tmpl_words;
        sum[kSumBucketRecs] = most_buckets;
        sum[kSumRunWords] = plan->run_words;
    }
}

// The same for a candidate of the interleaved schedule (a lane per device, v chunks each): A is
// the warp's shared memory for the evaluation.  Record counts, bounds and last backward starts
// are kept per virtual stage c * pp + d, the rest per device.
__device__ __forceinline__ void plan_interleaved(const DeviceView &v, const Row &row, int row_index, int64_t index,
                                                 EmitPlan *plan, int64_t *rec, const int64_t *binom, int64_t *sum,
                                                 const IlvArrays &A)
{
    const int lane = threadIdx.x & 31;
    const int pp = row.pp, vch = row.v, P = pp * vch;
    const CandidateCoords cc = split_local(row, index - row.offset);
    const Entry en = v.entries[cc.entry];
    const IlvResult R = interleaved_candidate(v, row, en, cc, binom, A, rec, 32);
    const int L1 = v.tc.n_layers + 1;
    int widest = 1, both = 0;
    int64_t dev_recs = 0, dev_buckets = 0;
    if (lane < pp) {
        const int d = lane;
        for (int c = 0; c < vch; ++c) {
            const int s = c * pp + d;
            const int a = A.bounds[s], e = A.bounds[s + 1];
            const int64_t per_dir = (int64_t)(e - a) * (row.mp > 1 ? 2 : 1) + (row.dp > 1 ? v.pe[e] - v.pe[a] : 0);
            const int64_t rf = per_dir + (s < P - 1 ? 1 : 0);
            const int64_t rb = per_dir + (s > 0 ? 1 : 0);
            int64_t kb = 0;
            if (row.dp > 1) {
                const int64_t *nbt = v.nb + row.row_tab_off, *tpt = v.tp + row.row_tab_off;
                kb = nbt[(int64_t)e * L1 + a] + (tpt[(int64_t)e * L1 + a] > 0 ? 1 : 0);
            }
            plan->bounds[s] = a;
            if (s == P - 1) plan->bounds[P] = e;
            plan->rf[s] = (int32_t)rf; plan->rb[s] = (int32_t)rb;
            plan->last_b_start[s] = A.last_b[s];
            dev_recs += (int64_t)en.m * (rf + rb) + kb;
            dev_buckets += kb;
            widest = max(widest, (int)max(rf, rb));
            both += (int)(rf + rb);
        }
        plan->n_buckets[d] = dev_buckets;
        plan->stage_recs[d] = dev_recs;
        plan->busy[d] = R.busy;
        plan->main_end[d] = R.main_end;
    }
    int64_t incl = dev_recs, most_buckets = dev_buckets;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int64_t up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    const int64_t total = __shfl_sync(0xffffffffu, incl, 31);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        widest = max(widest, __shfl_xor_sync(0xffffffffu, widest, o));
        both = max(both, __shfl_xor_sync(0xffffffffu, both, o));
        most_buckets = max64(most_buckets, __shfl_xor_sync(0xffffffffu, most_buckets, o));
    }
    if (lane < pp) plan->stage_rec_prefix[lane] = incl - dev_recs;
    if (lane == 0) {
        plan->index = index; plan->batch_ns = R.batch;
        plan->row = row_index; plan->entry = cc.entry; plan->m = en.m; plan->sched = 3;
        plan->pp = pp; plan->mp = row.mp; plan->dp = row.dp; plan->ok = 1; plan->v = vch; plan->two_way = 0;
        plan->stage_rec_prefix[pp] = total;
        plan->rec_total = total * row.mp * row.dp;
        const int n_items = 2 * en.m * vch;                       // items of a device
        const int cap = max(1, min(kMaxTileItems, kRunWords / (widest * 5)));
        const int n_chunks = (n_items + cap - 1) / cap;
        plan->tile_items = (n_items + n_chunks - 1) / n_chunks;
        plan->run_words = plan->tile_items * widest * 5;
        plan->tmpl_words = both * 5;                              // the templates of all chunks of the widest device
        const int64_t reps = (int64_t)row.mp * row.dp;
        sum[kSumRecords] = plan->rec_total;
        sum[kSumItemTiles] = (int64_t)pp * ((n_items + plan->tile_items - 1) / plan->tile_items) *
                             ((reps + kTileReplicas - 1) / kTileReplicas);
        sum[kSumBucketTiles] = (int64_t)pp * ((reps + kBucketReplicas - 1) / kBucketReplicas);
        sum[kSumTmplWords] = plan->tmpl_words;
        sum[kSumBucketRecs] = most_buckets;
        sum[kSumRunWords] = plan->run_words;
    }
}

// The same for a bidirectional-pipeline candidate: the plan's "chunks" are its two pipelines, the
// per-stage arrays are indexed pipeline * pp + device, bounds holds the pp + 1 shared bounds.
__device__ __forceinline__ void plan_bidirectional(const DeviceView &v, const Row &row, int row_index, int64_t index,
                                                   EmitPlan *plan, int64_t *rec, const int64_t *binom, int64_t *sum,
                                                   const IlvArrays &A)
{
    const int lane = threadIdx.x & 31;
    const int pp = row.pp;
    const CandidateCoords cc = split_local(row, index - row.offset);
    const Entry en = v.entries[cc.entry];
    const IlvResult R = bidirectional_candidate(v, row, en, cc, binom, A, rec, 32);
    const int L1 = v.tc.n_layers + 1, half = en.m / 2;
    int widest = 1, both = 0;
    int64_t dev_recs = 0, dev_buckets = 0;
    if (lane < pp) {
        const int d = lane;
        for (int c = 0; c < 2; ++c) {
            const int st = c ? pp - 1 - d : d;                     // the device's stage in pipeline c
            const int a = A.bounds[st], e = A.bounds[st + 1];
            const int64_t per_dir = (int64_t)(e - a) * (row.mp > 1 ? 2 : 1) + (row.dp > 1 ? v.pe[e] - v.pe[a] : 0);
            const int64_t rf = per_dir + (st < pp - 1 ? 1 : 0);
            const int64_t rb = per_dir + (st > 0 ? 1 : 0);
            // the stage's gradients go to its other holder at least: buckets whenever it has gradient bytes
            const int64_t *nbt = v.nb + row.row_tab_off, *tpt = v.tp + row.row_tab_off;
            const int64_t kb = nbt[(int64_t)e * L1 + a] + (tpt[(int64_t)e * L1 + a] > 0 ? 1 : 0);
            const int x = c * pp + d;
            plan->rf[x] = (int32_t)rf; plan->rb[x] = (int32_t)rb;
            plan->last_b_start[x] = A.last_b[c * pp + st];
            dev_recs += (int64_t)half * (rf + rb) + kb;
            dev_buckets += kb;
            widest = max(widest, (int)max(rf, rb));
            both += (int)(rf + rb);
        }
        plan->bounds[d] = A.bounds[d];
        if (d == pp - 1) plan->bounds[pp] = A.bounds[pp];
        plan->n_buckets[d] = dev_buckets;
        plan->stage_recs[d] = dev_recs;
        plan->busy[d] = R.busy;
        plan->main_end[d] = R.main_end;
    }
    int64_t incl = dev_recs, most_buckets = dev_buckets;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int64_t up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    const int64_t total = __shfl_sync(0xffffffffu, incl, 31);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        widest = max(widest, __shfl_xor_sync(0xffffffffu, widest, o));
        both = max(both, __shfl_xor_sync(0xffffffffu, both, o));
        most_buckets = max64(most_buckets, __shfl_xor_sync(0xffffffffu, most_buckets, o));
    }
    if (lane < pp) plan->stage_rec_prefix[lane] = incl - dev_recs;
    if (lane == 0) {
        plan->index = index; plan->batch_ns = R.batch;
        plan->row = row_index; plan->entry = cc.entry; plan->m = en.m; plan->sched = 4;
        plan->pp = pp; plan->mp = row.mp; plan->dp = row.dp; plan->ok = 1; plan->v = 2; plan->two_way = 1;
        plan->stage_rec_prefix[pp] = total;
        plan->rec_total = total * row.mp * row.dp;
        const int n_items = 2 * en.m;                             // items of a device
        const int cap = max(1, min(kMaxTileItems, kRunWords / (widest * 5)));
        const int n_chunks = (n_items + cap - 1) / cap;
        plan->tile_items = (n_items + n_chunks - 1) / n_chunks;
        plan->run_words = plan->tile_items * widest * 5;
        plan->tmpl_words = both * 5;                              // the templates of both pipelines of the widest device
        const int64_t reps = (int64_t)row.mp * row.dp;
        sum[kSumRecords] = plan->rec_total;
        sum[kSumItemTiles] = (int64_t)pp * ((n_items + plan->tile_items - 1) / plan->tile_items) *
                             ((reps + kTileReplicas - 1) / kTileReplicas);
        sum[kSumBucketTiles] = (int64_t)pp * ((reps + kBucketReplicas - 1) / kBucketReplicas);
        sum[kSumTmplWords] = plan->tmpl_words;
        sum[kSumBucketRecs] = most_buckets;
        sum[kSumRunWords] = plan->run_words;
    }
}

// Totals over all selections and the exclusive scan of their record counts, by one block, from
// the selections' summaries.
__device__ __forceinline__ void scan_plans(EmitPlan *plans, const int64_t *sums, int n, int64_t *totals /* the words of EmitTotals */)
{
    __shared__ int64_t warp_sum[32];
    const int t = threadIdx.x, nt = blockDim.x, lane = t & 31, warp = t >> 5;
    const int per = (n + nt - 1) / nt;
    const int b = min(n, t * per), e = min(n, b + per);
    int64_t s = 0, mx[kSumWords] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll 4
    for (int i = b; i < e; ++i) {
        s += __ldcg(&sums[(int64_t)i * kSumWords + kSumRecords]);
#pragma unroll
        for (int w = kSumItemTiles; w <= kSumRunWords; ++w) mx[w] = max64(mx[w], __ldcg(&sums[(int64_t)i * kSumWords + w]));
    }
    // exclusive scan of the per-thread sums over the block: inside warps, then over the warp totals
    int64_t incl = s;
    for (int off = 1; off < 32; off <<= 1) {
        const int64_t up = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += up;
    }
    if (lane == 31) warp_sum[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const int64_t w = lane < (nt >> 5) ? warp_sum[lane] : 0;
        int64_t wi = w;
        for (int off = 1; off < 32; off <<= 1) {
            const int64_t up = __shfl_up_sync(0xffffffffu, wi, off);
            if (lane >= off) wi += up;
        }
        warp_sum[lane] = wi - w;                       // exclusive
        if (lane == 31) totals[0] = wi;
        if (lane >= kSumItemTiles && lane <= kSumRunWords) totals[lane] = 0;      // maxima: from zero
    }
    __syncthreads();
    int64_t acc = warp_sum[warp] + incl - s;
#pragma unroll 4
    for (int i = b; i < e; ++i) { plans[i].rec_base = acc; acc += __ldcg(&sums[(int64_t)i * kSumWords + kSumRecords]); }
    // totals[1..5]: item tiles, bucket tiles, template words, bucket records, run words (the order of the summary)
#pragma unroll
    for (int w = kSumItemTiles; w <= kSumRunWords; ++w)
        if (mx[w] > 0) atomicMax((unsigned long long *)&totals[w], (unsigned long long)mx[w]);
}

// One warp per selection plans it; the last block to finish then scans the plans (totals[6]
// counts the finished blocks: zero before the first launch, and the last block leaves it zero).
constexpr int kPlanBinomWords = 512;
__global__ void __launch_bounds__(128)
emit_plan_kernel(DeviceView v, const int64_t *__restrict__ indices, int n, EmitPlan *plans,
                 int64_t *op_start, int64_t op_words_per_cand, int64_t *sums, int64_t *totals,
                 int ilv_words /* shared-memory words per warp for interleaved candidates */,
                 int64_t *h_totals /* nullable; host memory the device can write: the totals' words, then
                                      (word 7) the device status word as this kernel leaves it */,
                 EmitTotals limits /* limits.pad[0] != 0: what the caller has provisioned; word 7 of the
                                      totals then says whether the plans stay within it */)
{
    extern __shared__ __align__(16) int64_t plan_dyn[];
    __shared__ int64_t binom_s[kPlanBinomWords];
    __shared__ bool last;
    const int64_t *binom = stage_binom(v, binom_s, kPlanBinomWords);
    const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (i < n) {
        EmitPlan *plan = plans + i;
        const int64_t index = indices[i];
        if (index < 0 || index >= v.sc.n_candidates) {
            if ((threadIdx.x & 31) == 0) {
                plan->ok = 0; plan->rec_total = 0; plan->index = index; plan->pp = 0; plan->m = 0; plan->v = 1; plan->two_way = 0;
                plan->mp = 1; plan->dp = 1; plan->tile_items = 8; plan->tmpl_words = 0; plan->run_words = 0;
                for (int w = 0; w < kSumWords; ++w) sums[(int64_t)i * kSumWords + w] = 0;
                atomicCAS(v.status, 0, DISTSIM_E_RANGE);
            }
        } else {
            const int r = find_row(v, index);
            const Row row = v.rows[r];
            if (row.two_way) {
                int64_t *rec_i = op_start + (int64_t)i * op_words_per_cand;
                const CandidateCoords cc = split_local(row, index - row.offset);
                plan_bidirectional(v, row, r, index, plan, rec_i, binom, sums + (int64_t)i * kSumWords,
                                   bidirectional_arrays(plan_dyn + (int64_t)(threadIdx.x >> 5) * ilv_words, row.pp,
                                                        order_kept(v, cc.entry)));
            } else {
            int64_t *rec_i = op_start + (int64_t)i * op_words_per_cand;
            if (row.v > 1) {
                plan_interleaved(v, row, r, index, plan, rec_i, binom, sums + (int64_t)i * kSumWords,
                                 interleaved_arrays(plan_dyn + (int64_t)(threadIdx.x >> 5) * ilv_words, row.pp, row.v));
            } else {
            int64_t *rec = op_start + (int64_t)i * op_words_per_cand;
            if (row.pp > 32) plan_candidate<2>(v, row, r, index, plan, rec, binom, sums + (int64_t)i * kSumWords);
            else plan_candidate<1>(v, row, r, index, plan, rec, binom, sums + (int64_t)i * kSumWords);
            }
            }
        }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last = atomicAdd((unsigned long long *)&totals[6], 1ull) == (unsigned long long)gridDim.x - 1;
    __syncthreads();
    if (!last) return;
    __threadfence();
    if (threadIdx.x == 0) totals[6] = 0;               // the next launch counts its blocks from zero
    scan_plans(plans, sums, n, totals);
    if (limits.pad[0]) {
        __syncthreads();
        if (threadIdx.x == 0) {
            const int64_t *lim = reinterpret_cast<const int64_t *>(&limits);
            bool fits = true;
            for (int w = 0; w <= kSumRunWords; ++w) fits = fits && __ldcg(&totals[w]) <= lim[w];
            totals[7] = fits ? 1 : 0;
            if (!fits) atomicCAS(v.status, 0, DISTSIM_E_CAPACITY);
        }
    }
    if (!h_totals) return;
    __syncthreads();
    if (threadIdx.x == 0) {
        // the host reads these once an event recorded behind this kernel has completed
        for (int w = 0; w <= kSumRunWords; ++w) h_totals[w] = __ldcg(&totals[w]);
        h_totals[7] = (int64_t)*((volatile int32_t *)v.status);
        __threadfence_system();
    }
}

__global__ void __launch_bounds__(256)
emit_devices_kernel(DeviceView v, const EmitPlan *__restrict__ plans, int n, int64_t *offsets,
                    int64_t *busy, double *util, const int64_t *totals)
{
    const int64_t N = v.tc.n_devices;
    const int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g == 0 && offsets) offsets[(int64_t)n * N] = totals[0];
    if (g >= (int64_t)n * N) return;
    const int i = (int)(g / N);
    const int k = (int)(g - (int64_t)i * N);
    const EmitPlan &p = plans[i];
    if (!p.ok) {
        if (offsets) offsets[g] = p.rec_base;
        if (busy) busy[g] = 0;
        if (util) util[g] = 0.0;
        return;
    }
    const int q = k % p.mp, d = (k / p.mp) % p.pp, r = k / (p.mp * p.pp);
    if (offsets)
        offsets[g] = p.rec_base + (int64_t)r * p.mp * p.stage_rec_prefix[p.pp] +
                     (int64_t)p.mp * p.stage_rec_prefix[d] + (int64_t)q * p.stage_recs[d];
    if (busy) busy[g] = p.busy[d];
    if (util) util[g] = p.batch_ns > 0 ? (double)p.busy[d] / (double)p.batch_ns : 0.0;
}

// Position `s` in stage d's schedule order -> (is backward, micro-batch, items of each kind before it).
__device__ __forceinline__ void item_at(int sched, int pp, int m, int d, int s, bool &bwd, int &j, int &nf, int &nb)
{
    if (sched == 0) {
        if (s < m) { bwd = false; j = s; nf = s; nb = 0; }
        else { bwd = true; j = s - m; nf = m; nb = s - m; }
        return;
    }
    const int w = min(pp - d, m);
    if (s < w) { bwd = false; j = s; nf = s; nb = 0; }
    else if (s < 2 * m - w) {
        const int t = s - w;
        if (!(t & 1)) { bwd = true; j = t >> 1; nf = w + (t >> 1); nb = t >> 1; }
        else { bwd = false; j = w + (t >> 1); nf = w + (t >> 1); nb = (t >> 1) + 1; }
    } else { bwd = true; j = s - m; nf = m; nb = s - m; }
}

// Gradient-bucket records.  A block owns (selection, stage, chunk of replicas).  Buckets whose last byte lies in the same layer share a ready time, so once the
// first of them has started the rest follow back to back: per layer one serial step (lane 0),
// inside a layer a closed form (a thread per bucket).  The records of up to `run` buckets
// are assembled in shared memory once and sent to every replica by a bulk copy, as in
// emit_items_kernel.
// The work of one block (tile: its number inside the selection).
__device__ __forceinline__ void emit_buckets_block(const DeviceView &v, const EmitPlan &p, int tile,
                                                   int64_t *__restrict__ out, int run /* buckets per image */,
                                                   int64_t *dyn_s)
{
    int64_t *img_a = dyn_s;                             // word x of the run at img_a[x]
    int64_t *img_b = dyn_s + run * 5 + 1;               // the same word at img_b[x + 1] (run * 5 + 1 is even)
    int64_t *g_start = img_b + run * 5 + 1;             // [L + 1] start of the first bucket ending in layer a+i
    int64_t *g_first = g_start + DISTSIM_MAX_LAYERS + 1;  // [L + 1] number of that bucket
    __shared__ int64_t part_start_s, lane_end_s;
    const bool two_way = p.two_way != 0;                // two streams (pipelines), each reduced over 2 dp devices
    if (!p.ok || (p.dp == 1 && !two_way)) return;
    const int mp = p.mp, reps = mp * p.dp;
    const int rep_chunks = (reps + kBucketReplicas - 1) / kBucketReplicas;
    const int d = tile / rep_chunks, rc = tile - d * rep_chunks;
    if (d >= p.pp) return;
    if (p.n_buckets[d] == 0) return;
    const Row &row = v.rows[p.row];
    const int L1 = v.tc.n_layers + 1;
    const int64_t *pb = v.etb + (int64_t)p.entry * v.tc.lp;
    const bool near = two_way && mirror_group_near(v, row, d);
    const int64_t t_full = near ? row.t_full_near : row.t_full, main_end = p.main_end[d];
    const int64_t stage_words = p.stage_recs[d] * 5;
    const int64_t replica_words = (int64_t)mp * p.stage_rec_prefix[p.pp] * 5;
    // the device's bucket records follow its main-lane records
    int64_t *base = out + (p.rec_base + (int64_t)mp * p.stage_rec_prefix[d]) * 5 + (p.stage_recs[d] - p.n_buckets[d]) * 5;
    if (threadIdx.x == 0) lane_end_s = 0;
    int64_t kb0 = 0;                                    // buckets of the chunks already written
    // one gradient stream per model chunk the device holds (one without chunks), the last chunk
    // first, all on the device's one lane
    for (int k = p.v - 1; k >= 0; --k) {
        // bidirectional candidates: the stream of the device's later stage first
        const int c = two_way ? ((k == 1) == (p.pp - 1 - d > d) ? 1 : 0) : k;
        const int s = c * p.pp + d;                     // (virtual) stage; index of the per-stage arrays
        const int st = two_way ? (c ? p.pp - 1 - d : d) : s;
        const int a = p.bounds[st], e = p.bounds[st + 1];
        const int64_t *nbe = v.nb + row.row_tab_off + (int64_t)e * L1;
        int64_t part = v.tp[row.row_tab_off + (int64_t)e * L1 + a];
        // (the table of a two_way row holds the trailing bucket's bytes: its cost depends on the device)
        if (two_way && part > 0)
            part = allreduce_cost(v.tc, 2 * (int64_t)p.dp, part, near ? v.tc.alpha_intra : v.tc.alpha_inter,
                                  near ? v.tc.beta_intra : v.tc.beta_inter);
        const int64_t n_full = nbe[a];
        const int64_t kb = n_full + (part > 0 ? 1 : 0);
        if (kb == 0) continue;
        const int64_t tbs = p.last_b_start[s];
        __syncthreads();                                // the previous chunk's reads of g_start / g_first are done
        // all threads fetch the per-layer inputs (independent loads), then thread 0 runs the short chain
        for (int l = a + threadIdx.x; l < e; l += blockDim.x) {
            g_first[l - a] = l + 1 < e ? nbe[l + 1] : 0;                       // buckets before layer l's group
            g_start[l - a] = v.tc.overlap ? tbs + (pb[e] - pb[l]) : main_end;    // ready time of the group
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int64_t end = lane_end_s, part_start = 0;
            for (int l = e - 1; l >= a; --l) {
                const int64_t nb_prev = g_first[l - a];
                const int64_t nb_l = l > a ? g_first[l - 1 - a] : n_full;       // nb[e][l]
                const int64_t start = max64(end, g_start[l - a]);
                g_start[l - a] = start;
                if (nb_l > nb_prev) end = start + (nb_l - nb_prev) * t_full;
            }
            if (part > 0) {
                const int ls = v.next_grad[a];
                const int64_t ready = v.tc.overlap ? tbs + (pb[e] - pb[ls]) : main_end;
                part_start = max64(end, ready);
                end = part_start + part;
            }
            part_start_s = part_start;
            lane_end_s = end;
        }
        __syncthreads();
        const int64_t part_start = part_start_s;
        for (int64_t k0 = 0; k0 < kb; k0 += run) {
            const int nk = (int)min((int64_t)run, kb - k0);
            for (int kk = threadIdx.x; kk < nk; kk += blockDim.x) {
                const int64_t k = k0 + kk;
                int64_t start, dur;
                if (k >= n_full) { start = part_start; dur = part; }
                else {
                    // the layer whose group holds bucket k: the largest l with nb[e][l] > k
                    // (nb[e][l] = g_first[l-1-a] for l > a grows as l decreases, and nb[e][a] = n_full > k)
                    int lo = a, hi = e - 1;
                    while (lo < hi) {
                        const int mid = (lo + hi + 1) >> 1;
                        if (g_first[mid - 1 - a] > k) lo = mid; else hi = mid - 1;
                    }
                    start = g_start[lo - a] + (k - g_first[lo - a]) * t_full;
                    dur = t_full;
                }
                const int64_t rec[5] = {DISTSIM_DP_AR, kb0 + k, -1, start, start + dur};
#pragma unroll
                for (int f = 0; f < 5; ++f) { img_a[kk * 5 + f] = rec[f]; img_b[kk * 5 + f + 1] = rec[f]; }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncthreads();
            const int total = nk * 5;
            const int rep = rc * kBucketReplicas + threadIdx.x;
            if (threadIdx.x < kBucketReplicas && rep < reps) {
                const int r = rep / mp, q = rep - r * mp;
                int64_t *dst = base + (int64_t)r * replica_words + (int64_t)q * stage_words + (kb0 + k0) * 5;
                // 16-byte aligned copies take img_a from word 0, the others img_b from word 1
                const bool odd = ((reinterpret_cast<uintptr_t>(dst) >> 3) & 1) != 0;
                const int head = odd ? 1 : 0;
                const int bulk_words = (total - head) & ~1;
                if (odd) __stcs(dst, img_a[0]);
                if (head + bulk_words < total) __stcs(dst + total - 1, img_a[total - 1]);
                // the image is rewritten by the next run, and the block's shared memory must outlive
                // the copy engine's reads of it
                if (bulk_words > 0) {
                    const int64_t *src = odd ? img_b + 2 : img_a;
                    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                                 :: "l"(dst + head), "r"(smem_addr(src)), "r"(bulk_words * 8) : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                }
            }
            __syncthreads();
        }
        kb0 += kb;
    }
}

// Gradient-bucket records: a launch of its own with small blocks (measured: as extra blocks of
// the item launch they take the places of item blocks and cost more than they save).
constexpr int kBucketThreads = 128;
__global__ void __launch_bounds__(kBucketThreads)
emit_buckets_kernel(DeviceView v, const EmitPlan *__restrict__ plans, int64_t *__restrict__ out, int run /* buckets per image */,
                    const int64_t *__restrict__ gate /* nullable: totals whose word 7 says whether to write at all */)
{
    if (gate && __ldcg(&gate[7]) == 0) return;
    extern __shared__ __align__(16) int64_t dyn_b[];
    emit_buckets_block(v, plans[blockIdx.y], (int)blockIdx.x, out, run, dyn_b);
}

// Interleaved 1F1B: position `pos` in device d's order -> (is backward, chunk, micro-batch, forward
// and backward items before it); see interleaved.cuh for the order.
__device__ __forceinline__ void interleaved_item_at(int pp, int vch, int m, int d, int pos, bool &bwd, int &c, int &j,
                                                    int &nf, int &nb)
{
    const int total = m * vch;
    int warm = (pp - d - 1) * 2 + (vch - 1) * pp;
    if (m == pp || warm > total) warm = total;
    if (pos < warm) { bwd = false; nf = pos; nb = 0; }
    else if (pos - warm < 2 * (total - warm)) { const int t = pos - warm; bwd = t & 1; nf = warm + (t + 1) / 2; nb = t / 2; }
    else { bwd = true; nf = total; nb = pos - total; }
    const int idx = bwd ? nb : nf;
    const int c0 = (idx / pp) % vch;
    c = bwd ? vch - 1 - c0 : c0;
    j = (idx / (pp * vch)) * pp + idx % pp;
}
// ... and the words of the records of the device's first nf forward and nb backward items: of the
// first n forward items, chunk c has (n / (pp v)) pp + clamp(n mod (pp v) - c pp, 0, pp); the
// backward items take the chunks in reverse.
__device__ __forceinline__ int64_t interleaved_words_before(const EmitPlan &p, int d, int nf, int nb)
{
    const int pp = p.pp, vch = p.v, cyc = pp * vch;
    const int qf = nf / cyc, rf_ = nf - qf * cyc, qb = nb / cyc, rb_ = nb - qb * cyc;
    int64_t recs = 0;
    for (int c = 0; c < vch; ++c) {
        const int s = c * pp + d;
        const int cf = qf * pp + min(max(rf_ - c * pp, 0), pp);
        const int cb = qb * pp + min(max(rb_ - (vch - 1 - c) * pp, 0), pp);
        recs += (int64_t)cf * p.rf[s] + (int64_t)cb * p.rb[s];
    }
    return recs * 5;
}

__global__ void __launch_bounds__(kItemThreads)
emit_items_kernel(DeviceView v, const EmitPlan *__restrict__ plans, const int64_t *__restrict__ op_start,
                  int64_t op_words_per_cand, int64_t *__restrict__ out /* records as flat words */,
                  int cap /* words of one image: even, at least the longest run of any selection */,
                  const int64_t *__restrict__ gate /* nullable: totals whose word 7 says whether to write at all */)
{
    if (gate && __ldcg(&gate[7]) == 0) return;
    extern __shared__ __align__(16) int64_t dyn_s[];
    int64_t *img_a = dyn_s;                             // word x of the run at img_a[x]
    int64_t *img_b = dyn_s + cap;                       // the same word at img_b[x + 1]
    int64_t *tmpl = dyn_s + 2 * cap + 2;                // per chunk: [rf*5] forward, then [rb*5] backward
    __shared__ int64_t rep_off_s[kTileReplicas];
    __shared__ int64_t start_s[kMaxTileItems];          // start time of each item of the run
    __shared__ int64_t jit_s[kMaxTileItems];            // jitter at the start of each item
    __shared__ int32_t ioff[kMaxTileItems + 1];         // word offset of each item inside the run
    __shared__ int32_t meta_s[kMaxTileItems];           // micro-batch << 6 | chunk << 1 | is-backward
    __shared__ int32_t toff_s[DISTSIM_MAX_PP / 2][2];   // word offset of each chunk's forward / backward template
    __shared__ int64_t run_base_s;                      // words of the device's records before the run
    const int i = blockIdx.y;
    const EmitPlan &p = plans[i];
    if (!p.ok) return;
    const int m = p.m, pp = p.pp, sched = p.sched, mp = p.mp, vch = p.v, P = pp * vch;
    const bool two_way = p.two_way != 0;                // vch = 2 stands for the two pipelines
    const int reps = mp * p.dp;
    const int tile_items = p.tile_items;
    const int dev_items = two_way ? 2 * m : 2 * m * vch;   // items of a device
    const int item_chunks = (dev_items + tile_items - 1) / tile_items;
    const int rep_chunks = (reps + kTileReplicas - 1) / kTileReplicas;
    int tile = blockIdx.x;
    if (tile >= pp * item_chunks * rep_chunks) return;
    const int rc = tile % rep_chunks; tile /= rep_chunks;
    const int ic = tile % item_chunks;
    const int d = tile / item_chunks;

    const Row &row = v.rows[p.row];
    const Entry &en = v.entries[p.entry];
    const int64_t *pf = v.etf + (int64_t)p.entry * v.tc.lp;
    const int64_t *pb = v.etb + (int64_t)p.entry * v.tc.lp;
    const int64_t *f = v.raw.fwd + (int64_t)en.cls * v.tc.n_layers;
    const int64_t *g = v.raw.bwd + (int64_t)en.cls * v.tc.n_layers;
    const int row_mp = row.mp, row_dp = row.dp;
    const int per_layer = row_mp > 1 ? 2 : 1;
    const int64_t ar = en.ar, a2a = en.a2a;
    const int jr = v.tc.n_jitter > 0 ? 1 : 0;           // record 0 of an item is its jitter event

    // ---- item templates: records relative to the end of the item's jitter event; one pair of
    //      templates per model chunk of the device (one without chunks) ----------------------
    int tmpl_acc = 0;
    for (int c = 0; c < vch; ++c) {
        const int s = c * pp + d;                       // (virtual) stage; index of the per-stage arrays
        // the stage's place in its chain of stages: a bidirectional candidate has two chains of pp
        const int st = two_way ? (c ? pp - 1 - d : d) : s, n_st = two_way ? pp : P;
        const int a = p.bounds[st], e = p.bounds[st + 1];
        const int rf = p.rf[s], rb = p.rb[s];
        int64_t *tf = tmpl + tmpl_acc, *tb = tf + (int64_t)rf * 5;
        if (threadIdx.x == 0) { toff_s[c][0] = tmpl_acc; toff_s[c][1] = tmpl_acc + rf * 5; }
        tmpl_acc += (rf + rb) * 5;
        if (jr && threadIdx.x == 32) {
            tf[0] = DISTSIM_JITTER_F; tf[1] = a; tf[2] = 0; tf[3] = 0; tf[4] = 0;
            tb[0] = DISTSIM_JITTER_B; tb[1] = e - 1; tb[2] = 0; tb[3] = 0; tb[4] = 0;
        }
        for (int l = a + threadIdx.x; l < e; l += blockDim.x) {
            const bool ex = row_dp > 1 && v.raw.expert[l];
            {   // forward: layers ascending
                const int r = jr + (l - a) * per_layer + (row_dp > 1 ? v.pe[l] - v.pe[a] : 0);
                int64_t t = pf[l] - pf[a];
                int64_t *w = tf + (int64_t)r * 5;
                w[0] = DISTSIM_COMPUTE_F; w[1] = l; w[2] = 0; w[3] = t; t += f[l]; w[4] = t; w += 5;
                if (row_mp > 1) { w[0] = DISTSIM_MP_AR_F; w[1] = l; w[2] = 0; w[3] = t; t += ar; w[4] = t; w += 5; }
                if (ex) { w[0] = DISTSIM_A2A_F; w[1] = l; w[2] = 0; w[3] = t; t += a2a; w[4] = t; }
            }
            {   // backward: layers descending
                const int r = jr + (e - 1 - l) * per_layer + (row_dp > 1 ? v.pe[e] - v.pe[l + 1] : 0);
                int64_t t = pb[e] - pb[l + 1];
                int64_t *w = tb + (int64_t)r * 5;
                w[0] = DISTSIM_COMPUTE_B; w[1] = l; w[2] = 0; w[3] = t; t += g[l]; w[4] = t; w += 5;
                if (row_mp > 1) { w[0] = DISTSIM_MP_AR_B; w[1] = l; w[2] = 0; w[3] = t; t += ar; w[4] = t; w += 5; }
                if (ex) { w[0] = DISTSIM_A2A_B; w[1] = l; w[2] = 0; w[3] = t; t += a2a; w[4] = t; }
            }
        }
        if (threadIdx.x == 0) {
            if (st < n_st - 1) {
                int64_t *w = tf + (int64_t)(rf - 1) * 5;
                const int64_t t = pf[e] - pf[a];
                w[0] = DISTSIM_SEND_F; w[1] = e - 1; w[2] = 0; w[3] = t;
                w[4] = t + (two_way ? p2p_cost(row, en, c ? pp - 2 - st : st)
                                    : vch > 1 ? virtual_p2p_cost(v, row, en, s) : p2p_cost(row, en, d));
            }
            if (st > 0) {
                int64_t *w = tb + (int64_t)(rb - 1) * 5;
                const int64_t t = pb[e] - pb[a];
                w[0] = DISTSIM_SEND_B; w[1] = a; w[2] = 0; w[3] = t;
                w[4] = t + (two_way ? p2p_cost(row, en, c ? pp - 1 - st : st - 1)
                                    : vch > 1 ? virtual_p2p_cost(v, row, en, s - 1) : p2p_cost(row, en, d - 1));
            }
        }
    }
    // ---- the run: its items' start times, kinds, micro-batches and word offsets ------------
    // an item's offset follows from how many forward / backward items (of each chunk) precede it
    const int s0 = ic * tile_items;
    const int n_items = min(dev_items, s0 + tile_items) - s0;
    int64_t base0;                                       // words of the device's records before the run
    const int64_t order_at = two_way ? order_offset(v, p.entry) : 0;
    // words of the device's records before position `pos` of its order (bidirectional candidates)
    auto two_way_words_before = [&](int pos) {
        const ItemsBefore n = items_before(v, order_at, m, d, pos);
        return ((int64_t)n.f0 * p.rf[d] + (int64_t)n.b0 * p.rb[d] + (int64_t)n.f1 * p.rf[pp + d] + (int64_t)n.b1 * p.rb[pp + d]) * 5;
    };
    if (two_way) base0 = two_way_words_before(s0);
    else {
        bool bwd0; int c0, j0, nf0, nb0;
        if (vch > 1) {
            interleaved_item_at(pp, vch, m, d, s0, bwd0, c0, j0, nf0, nb0);
            base0 = interleaved_words_before(p, d, nf0, nb0);
        } else {
            item_at(sched, pp, m, d, s0, bwd0, j0, nf0, nb0);
            base0 = ((int64_t)nf0 * p.rf[d] + (int64_t)nb0 * p.rb[d]) * 5;
        }
    }
    for (int k = threadIdx.x; k <= n_items; k += blockDim.x) {
        bool bwd; int c = 0, j, nf, nb;
        int64_t before;
        if (two_way) {
            before = two_way_words_before(s0 + k);                             // k == n_items: one past the run
            const int item = k < n_items ? v.order[order_at + (int64_t)d * (2 * m + 1) + s0 + k] : 0;
            c = (item & kOrderUp) ? 1 : 0;
            bwd = (item & kOrderBackward) != 0;
            j = (item & kOrderMicroBatch) + c * (m / 2);
        } else if (vch > 1) {
            interleaved_item_at(pp, vch, m, d, s0 + k, bwd, c, j, nf, nb);     // k == n_items: one past the run
            before = interleaved_words_before(p, d, nf, nb);
        } else {
            item_at(sched, pp, m, d, s0 + k, bwd, j, nf, nb);
            before = ((int64_t)nf * p.rf[d] + (int64_t)nb * p.rb[d]) * 5;
        }
        ioff[k] = (int)(before - base0);
        if (k < n_items) {
            start_s[k] = op_start[(int64_t)i * op_words_per_cand + (int64_t)d * dev_items + s0 + k];
            meta_s[k] = (j << 6) | (c << 1) | (bwd ? 1 : 0);
            jit_s[k] = jitter_of(v, bwd ? v.raw.jit_b : v.raw.jit_f, j, d);
        }
    }
    // word offset of every replica (r, q) of this tile relative to replica 0 of the stage
    const int rep0 = rc * kTileReplicas;
    const int n_rep = min(reps, rep0 + kTileReplicas) - rep0;
    if (threadIdx.x >= 64 && threadIdx.x < 64 + kTileReplicas) {
        const int k = threadIdx.x - 64;
        int64_t off = 0;
        if (k < n_rep) {
            const int rep = rep0 + k;
            const int r = rep / mp, q = rep - r * mp;
            off = (int64_t)r * mp * p.stage_rec_prefix[pp] * 5 + (int64_t)q * p.stage_recs[d] * 5;
        }
        rep_off_s[k] = off;
    }
    if (threadIdx.x == 0) run_base_s = base0;
    __syncthreads();

    // ---- the run's image: one warp per item, a word is template word + {0, 0, j, start, start} ----
    const int total = ioff[n_items];                 // <= cap by the plans' choice of tile_items
    {
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        const int lane_field = lane - (lane / 5) * 5;
        for (int it = warp; it < n_items; it += kItemThreads / 32) {
            const int off = ioff[it], len = ioff[it + 1] - off;
            const int meta = meta_s[it];
            const int64_t *tp = tmpl + toff_s[(meta >> 1) & 31][meta & 1];
            const int64_t j = meta >> 6;
            // the jitter event runs [start, start + jitter); every later event is relative to its end
            const int64_t t0 = start_s[it], t1 = t0 + (jr ? jit_s[it] : 0);
            int field = lane_field;                  // w mod 5, kept without dividing
            for (int w = lane; w < len; w += 32) {
                int64_t val = tp[w];
                if (field == 2) val += j;
                else if (field >= 3) val += (w == 3 ? t0 : t1);
                img_a[off + w] = val;
                img_b[off + w + 1] = val;
                field += 2;                          // 32 mod 5
                if (field >= 5) field -= 5;
            }
        }
    }
    // make the image visible to the bulk-copy engine, then hand it one copy per replica
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    if (threadIdx.x >= n_rep || total == 0) return;
    // Records are 40 bytes, so a replica's copy of the run starts on a 16-byte boundary or 8 bytes
    // past one.  Bulk copies need both ends 16-byte aligned: aligned replicas take img_a from word 0,
    // the others take img_b (the run shifted by one word) from word 1; single words at the ends are
    // stored directly.
    int64_t *dst = out + (p.rec_base + (int64_t)mp * p.stage_rec_prefix[d]) * 5 + run_base_s + rep_off_s[threadIdx.x];
    const bool odd = ((reinterpret_cast<uintptr_t>(dst) >> 3) & 1) != 0;
    const int head = odd ? 1 : 0;                    // words stored directly before the bulk copy
    const int bulk_words = (total - head) & ~1;
    if (odd) __stcs(dst, img_a[0]);
    if (bulk_words > 0) {
        const int64_t *src = odd ? img_b + 2 : img_a;
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                     :: "l"(dst + head), "r"(smem_addr(src)), "r"(bulk_words * 8) : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    }
    if (head + bulk_words < total) __stcs(dst + total - 1, img_a[total - 1]);
    // the block's shared memory must outlive the copy engine's reads of it
    if (bulk_words > 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

// Order-sensitive 64-bit checksum of every device's record stream: the sum over the stream's
// words w_i (five per record, i counted from the start of the device's list) of
// mix(w_i + (i + 1) * 0x9E3779B97F4A7C15) modulo 2^64, mix being the SplitMix64 finaliser.  Moving,
// dropping or altering a word changes the sum.  One block per list.
__device__ __forceinline__ uint64_t mix64(uint64_t z)
{
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
__global__ void __launch_bounds__(256)
checksum_lists_kernel(const int64_t *__restrict__ words, const int64_t *__restrict__ offsets, int64_t n_lists,
                      unsigned long long *__restrict__ out)
{
    __shared__ unsigned long long part[8];
    for (int64_t list = blockIdx.x; list < n_lists; list += gridDim.x) {
        const int64_t w0 = offsets[list] * 5, n = (offsets[list + 1] - offsets[list]) * 5;
        unsigned long long acc = 0;
        for (int64_t i = threadIdx.x; i < n; i += blockDim.x)
            acc += mix64((uint64_t)__ldcs(words + w0 + i) + (uint64_t)(i + 1) * 0x9E3779B97F4A7C15ull);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
        __syncthreads();
        if (threadIdx.x == 0) {
            unsigned long long sum = 0;
            for (int k = 0; k < 8; ++k) sum += part[k];
            out[list] = sum;
        }
        __syncthreads();
    }
}

}  // namespace

void launch_checksum_lists(cudaStream_t s, const distsim_record *records, const int64_t *offsets, int64_t n_lists,
                           uint64_t *out, int64_t *launches)
{
    if (n_lists <= 0) return;
    const unsigned grid = (unsigned)(n_lists < (1 << 20) ? n_lists : (1 << 20));
    checksum_lists_kernel<<<grid, 256, 0, s>>>(reinterpret_cast<const int64_t *>(records), offsets, n_lists,
                                               reinterpret_cast<unsigned long long *>(out));
    ++*launches;
}

int interleaved_words_of(int pp, int v) { return interleaved_words(pp, v); }
int bidirectional_words_of(int pp, int kept) { return bidirectional_words(pp, kept); }
int bidirectional_kept_cap_of(int pp) { return bidirectional_kept_cap(pp); }

void launch_emit_plan(cudaStream_t s, const DeviceView &v, const int64_t *d_indices, int n,
                      EmitPlan *plans, int64_t *op_start, int64_t op_words_per_cand, int64_t *sums,
                      int64_t *offsets, int64_t *busy, double *util, int64_t *d_totals, int ilv_words,
                      int64_t *h_totals, cudaEvent_t planned, int64_t *launches, const EmitTotals *limits)
{
    EmitTotals lim{};
    if (limits) { lim = *limits; lim.pad[0] = 1; }
    const size_t plan_smem = (size_t)4 * ilv_words * sizeof(int64_t);
    ensure_dynamic_smem(reinterpret_cast<const void *>(&emit_plan_kernel), plan_smem);
    emit_plan_kernel<<<(n + 3) / 4, 128, plan_smem, s>>>(v, d_indices, n, plans, op_start, op_words_per_cand, sums, d_totals,
                                                     ilv_words, h_totals, lim);
    ++*launches;
    if (planned) cudaEventRecord(planned, s);       // the host can go on while the per-device words are written
    launch_emit_devices(s, v, plans, n, offsets, busy, util, d_totals, launches);
}

void launch_emit_devices(cudaStream_t s, const DeviceView &v, const EmitPlan *plans, int n, int64_t *offsets,
                         int64_t *busy, double *util, const int64_t *d_totals, int64_t *launches)
{
    if (!offsets && !busy && !util) return;
    const int64_t total = (int64_t)n * v.tc.n_devices + 1;
    emit_devices_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(v, plans, n, offsets, busy, util, d_totals);
    ++*launches;
}

void launch_emit_records(cudaStream_t s, const SideStream &ss, const DeviceView &v, int n, const EmitPlan *plans,
                         const int64_t *op_start, int64_t op_words_per_cand, const EmitTotals &t,
                         distsim_record *records, int64_t *launches, const int64_t *gate, const EmitDeviceWords *words)
{
    if (n == 0 || t.item_tiles == 0) {
        if (words) launch_emit_devices(s, v, plans, n, words->offsets, words->busy, words->util, words->d_totals, launches);
        return;
    }
    // two images of the run, then the forward and backward item templates of the widest stage
    const int cap = (int)((t.run_words + 1) & ~(int64_t)1);
    const size_t smem = (size_t)(2 * cap + 2 + t.tmpl_words) * sizeof(int64_t);
    ensure_dynamic_smem(reinterpret_cast<const void *>(&emit_items_kernel), smem);
    int64_t *out = reinterpret_cast<int64_t *>(records);
    const bool buckets = t.bucket_tiles > 0 && t.bucket_recs > 0;
    // The bucket records are few and their blocks wait more than they write: on the side stream
    // they run beside the item kernel (both only read the plans and write disjoint records).  The
    // fork event is recorded before the item kernel is enqueued, the item kernel goes first.
    const bool beside = (buckets || words) && ss.side[0];
    if (beside) cudaEventRecord(ss.fork, s);
    emit_items_kernel<<<dim3((unsigned)t.item_tiles, (unsigned)n), kItemThreads, smem, s>>>(
        v, plans, op_start, op_words_per_cand, out, cap, gate);
    ++*launches;
    if (beside) cudaStreamWaitEvent(ss.side[0], ss.fork, 0);
    if (words) launch_emit_devices(beside ? ss.side[0] : s, v, plans, n, words->offsets, words->busy, words->util, words->d_totals, launches);
    if (buckets) {
        // an odd number of buckets per image keeps both images 16-byte aligned
        const int run = (int)(t.bucket_recs < kBucketRun ? t.bucket_recs : kBucketRun) | 1;
        const size_t bsmem = (size_t)(2 * (run * 5 + 1) + 2 * (DISTSIM_MAX_LAYERS + 1)) * sizeof(int64_t);
        ensure_dynamic_smem(reinterpret_cast<const void *>(&emit_buckets_kernel), bsmem);
        const cudaStream_t bs = beside ? ss.side[0] : s;
        emit_buckets_kernel<<<dim3((unsigned)t.bucket_tiles, (unsigned)n), kBucketThreads, bsmem, bs>>>(v, plans, out, run, gate);
        ++*launches;
    }
    if (beside) {
        cudaEventRecord(ss.join[0], ss.side[0]);
        cudaStreamWaitEvent(s, ss.join[0], 0);
    }
}

}  // namespace distsim
