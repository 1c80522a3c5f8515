// Evaluation kernels: batch time (and optionally per-stage activity time) of a range of
// candidates of one row.
//
// eval_lockstep_kernel: a segment of pp/S consecutive lanes evaluates one candidate, lane =
// stage (S = 2 stages per lane when pp = 64), 32/(pp/S) candidates per warp, all segments of a
// warp advancing through the slots of the lock-step recurrence together.  The prefix rows of
// the entries a block touches are staged into shared memory with one bulk copy per table
// (cp.async.bulk, completion on the block's own mbarrier, no multicast).
#include "recurrence.cuh"
#include "smem_stage.cuh"
#include "eval_thread.cuh"

namespace distsim {

namespace {

constexpr int kEvalThreads = 256;

template <int S>
__global__ void __launch_bounds__(kEvalThreads)
eval_lockstep_kernel(DeviceView v, int row_index, int64_t lo, int64_t hi, int64_t first,
                     int64_t *__restrict__ batch_out, int64_t *__restrict__ busy_out,
                     int max_stage_entries)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t bar;
    const Row row = v.rows[row_index];
    const int pp = row.pp;
    const int wl = pp / S;                         // lanes per candidate
    const int cpw = 32 / wl;                       // candidates per warp
    const int warps = blockDim.x >> 5;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t cta_first = lo + (int64_t)blockIdx.x * warps * cpw;
    if (cta_first >= hi) return;
    const int64_t cta_last = min(hi, cta_first + (int64_t)warps * cpw) - 1;

    // ---- stage the prefix rows of the entries this block touches -----------------------
    const int e_lo = split_local(row, cta_first).entry;
    const int e_hi = split_local(row, cta_last).entry;
    const int n_stage = e_hi - e_lo + 1;
    const int lp = v.tc.lp;
    int64_t *sm_f = reinterpret_cast<int64_t *>(smem_raw);
    int64_t *sm_b = sm_f + (int64_t)max_stage_entries * lp;
    bool staged = false;
    if (max_stage_entries > 0 && n_stage <= max_stage_entries) {
        const uint32_t bytes = (uint32_t)(n_stage * lp * sizeof(int64_t));
        staged = stage_two_tables(&bar, sm_f, v.etf + (int64_t)e_lo * lp, sm_b,
                                  v.etb + (int64_t)e_lo * lp, bytes, v.status);
    }

    const int seg = lane / wl, seg_lane = lane - seg * wl;
    int64_t local = cta_first + (int64_t)warp * cpw + seg;
    const bool valid = local < hi;
    if (!valid) local = hi - 1;                    // idle segments shadow a real candidate
    const CandidateCoords cc = split_local(row, local);
    const Entry en = v.entries[cc.entry];
    const int64_t *pf = staged ? sm_f + (int64_t)(cc.entry - e_lo) * lp : v.etf + (int64_t)cc.entry * lp;
    const int64_t *pb = staged ? sm_b + (int64_t)(cc.entry - e_lo) * lp : v.etb + (int64_t)cc.entry * lp;

    int n_slots = 2 * (en.m + pp - 1);
    n_slots = __reduce_max_sync(0xffffffffu, n_slots);

    const StageResult<S> R = lockstep_candidate<S, false>(v, row, en, pf, pb, cc.sched, cc.part_rank,
                                                          seg_lane, wl, n_slots, nullptr);
    if (!valid) return;
    const int64_t out = row.offset + local - first;
    if (seg_lane == 0) batch_out[out] = R.batch;
    if (busy_out) {
        int64_t *bo = busy_out + out * v.sc.pp_max;
#pragma unroll
        for (int k = 0; k < S; ++k) bo[seg_lane * S + k] = R.busy[k];
        for (int d = pp + seg_lane; d < v.sc.pp_max; d += wl) bo[d] = 0;
    }
}

template <int PP, typename T>
void launch_thread_kernel(cudaStream_t s, const DeviceView &v, int row_index, const Row &row, int64_t lo,
                          int64_t hi, int64_t first, int e_begin, int e_end, int ept, int64_t p_lo,
                          int64_t p_hi, int64_t *batch_out, int64_t *busy_out)
{
    const int lp = v.tc.lp;
    ThreadKernelSmem plan{};
    size_t words = 0;
    // prefix rows of every entry of the row; the row's two bucket tables only when there is no
    // per-entry bucket-lane table to look the result up in
    if ((size_t)row.n_entries * lp * 2 <= 8192) {
        plan.n_entries_staged = row.n_entries;
        plan.off_etb = row.n_entries * lp;
        words = (size_t)row.n_entries * lp * 2;
    }
    if (!v.dt && words + 2 * (size_t)v.tab_words <= 12288) {
        plan.tables_staged = 1;
        plan.off_nb = (int32_t)words;
        plan.off_tp = (int32_t)words + v.tab_words;
        words += 2 * (size_t)v.tab_words;
    }
    const size_t smem = words * sizeof(int64_t);
    const int64_t n_threads = p_hi - p_lo;
    dim3 grid((unsigned)((n_threads + kThreadBlock - 1) / kThreadBlock), (unsigned)((e_end - e_begin + ept - 1) / ept));
    if (busy_out) {
        if (smem > 24 * 1024)
            cudaFuncSetAttribute(eval_thread_kernel<PP, T, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        eval_thread_kernel<PP, T, true><<<grid, kThreadBlock, smem, s>>>(v, row_index, lo, hi, first, e_begin, e_end, ept,
                                                                         p_lo, p_hi, batch_out, busy_out, plan);
    } else {
        if (smem > 24 * 1024)
            cudaFuncSetAttribute(eval_thread_kernel<PP, T, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        eval_thread_kernel<PP, T, false><<<grid, kThreadBlock, smem, s>>>(v, row_index, lo, hi, first, e_begin, e_end, ept,
                                                                          p_lo, p_hi, batch_out, busy_out, plan);
    }
}

template <typename T>
void launch_thread_kernel_pp(cudaStream_t s, const DeviceView &v, int row_index, const Row &row, int64_t lo,
                             int64_t hi, int64_t first, int e_begin, int e_end, int ept, int64_t p_lo,
                             int64_t p_hi, int64_t *batch_out, int64_t *busy_out)
{
    switch (row.pp) {
    case 1: launch_thread_kernel<1, T>(s, v, row_index, row, lo, hi, first, e_begin, e_end, ept, p_lo, p_hi, batch_out, busy_out); break;
    case 2: launch_thread_kernel<2, T>(s, v, row_index, row, lo, hi, first, e_begin, e_end, ept, p_lo, p_hi, batch_out, busy_out); break;
    case 4: launch_thread_kernel<4, T>(s, v, row_index, row, lo, hi, first, e_begin, e_end, ept, p_lo, p_hi, batch_out, busy_out); break;
    case 8: launch_thread_kernel<8, T>(s, v, row_index, row, lo, hi, first, e_begin, e_end, ept, p_lo, p_hi, batch_out, busy_out); break;
    default: launch_thread_kernel<16, T>(s, v, row_index, row, lo, hi, first, e_begin, e_end, ept, p_lo, p_hi, batch_out, busy_out); break;
    }
}

void launch_lockstep(cudaStream_t s, const DeviceView &v, int row_index, const Row &row, int64_t lo, int64_t hi,
                     int64_t first, int64_t *batch_out, int64_t *busy_out);

}  // namespace

void launch_eval_row(cudaStream_t s, const DeviceView &v, int row_index, const Row &row, const Entry *row_entries,
                     int64_t lo, int64_t hi, int64_t first, int64_t *batch_out, int64_t *busy_out,
                     int64_t *launches)
{
    if (hi <= lo) return;
    if (row.pp > 16) {
        launch_lockstep(s, v, row_index, row, lo, hi, first, batch_out, busy_out);
        ++*launches;
        return;
    }
    // Short pipelines: cut the range into runs of entries with the same arithmetic width; a run
    // with enough partitions goes to the one-partition-per-thread kernel, the rest to lock-step.
    const int64_t per_entry = row.n_part * row.n_sched;
    const int e_begin = (int)(lo / per_entry), e_end = (int)((hi - 1) / per_entry) + 1;
    int r0 = e_begin;
    while (r0 < e_end) {
        const bool narrow = row_entries[r0].bound < ((int64_t)1 << 32);
        int r1 = r0 + 1;
        while (r1 < e_end && (row_entries[r1].bound < ((int64_t)1 << 32)) == narrow) ++r1;
        const int64_t lo_r = lo > (int64_t)r0 * per_entry ? lo : (int64_t)r0 * per_entry;
        const int64_t hi_r = hi < (int64_t)r1 * per_entry ? hi : (int64_t)r1 * per_entry;
        int64_t p_lo = 0, p_hi = row.n_part;
        if (r1 - r0 == 1) {
            p_lo = (lo_r - (int64_t)r0 * per_entry) / row.n_sched;
            p_hi = (hi_r - 1 - (int64_t)r0 * per_entry) / row.n_sched + 1;
        }
        const int64_t n_parts = p_hi - p_lo;
        const int n_e = r1 - r0;
        const int ept = n_parts >= 148 * 4 * kThreadBlock ? n_e : 1;       // entries per thread
        if (n_parts * ((n_e + ept - 1) / ept) >= 2048) {
            if (narrow) launch_thread_kernel_pp<uint32_t>(s, v, row_index, row, lo_r, hi_r, first, r0, r1, ept, p_lo, p_hi, batch_out, busy_out);
            else launch_thread_kernel_pp<int64_t>(s, v, row_index, row, lo_r, hi_r, first, r0, r1, ept, p_lo, p_hi, batch_out, busy_out);
        } else {
            launch_lockstep(s, v, row_index, row, lo_r, hi_r, first, batch_out, busy_out);
        }
        ++*launches;
        r0 = r1;
    }
}

namespace {

void launch_lockstep(cudaStream_t s, const DeviceView &v, int row_index, const Row &row, int64_t lo, int64_t hi,
                     int64_t first, int64_t *batch_out, int64_t *busy_out)
{
    const int S = row.pp > 32 ? 2 : 1;
    const int wl = row.pp / S;
    const int cpb = (kEvalThreads / 32) * (32 / wl);      // candidates per block
    const int64_t blocks = (hi - lo + cpb - 1) / cpb;
    // entries a block can touch: its candidates span at most this many entries
    const int64_t per_entry = row.n_part * row.n_sched;
    int64_t span = (cpb + per_entry - 1) / per_entry + 1;
    if (span > row.n_entries) span = row.n_entries;
    int max_stage = (int)span;
    size_t smem = (size_t)max_stage * v.tc.lp * sizeof(int64_t) * 2;
    if (smem > 96 * 1024) { max_stage = 0; smem = 0; }   // too wide: read the rows from global
    if (S == 1) {
        if (smem > 48 * 1024)
            cudaFuncSetAttribute(eval_lockstep_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        eval_lockstep_kernel<1><<<(unsigned)blocks, kEvalThreads, smem, s>>>(v, row_index, lo, hi, first,
                                                                           batch_out, busy_out, max_stage);
    } else {
        if (smem > 48 * 1024)
            cudaFuncSetAttribute(eval_lockstep_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        eval_lockstep_kernel<2><<<(unsigned)blocks, kEvalThreads, smem, s>>>(v, row_index, lo, hi, first,
                                                                           batch_out, busy_out, max_stage);
    }
}

}  // namespace

}  // namespace distsim
