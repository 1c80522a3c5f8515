// Evaluation kernels: batch time (and optionally per-stage activity time) of a range of
// candidates.
//
// eval_thread_kernel (eval_thread.cuh): one stage partition per thread, for rows with many
// partitions and pp <= 16.
// eval_lockstep_kernel: a segment of pp consecutive lanes evaluates one candidate, lane = stage,
// 32/pp candidates per warp, all segments of a warp advancing through the slots of the
// lock-step recurrence together; for pp = 64 a lane owns two neighbouring stages and a warp one
// candidate.  The prefix rows of the entries a block touches are staged into shared memory with
// one bulk copy per table (cp.async.bulk, completion on the block's own mbarrier, no multicast).
//
// A search space has a few dozen rows, many of them tiny; launching them one by one would leave
// the device idle between kernels, so one launch carries a list of (row, range) work items and
// every block looks up the item it belongs to.
#include <vector>

#include "recurrence.cuh"
#include "smem_stage.cuh"
#include "eval_thread.cuh"
#include "bidirectional.cuh"

namespace distsim {

namespace {

// Threads per block of the lock-step kernel.  Blocks are small so that the long candidates of
// a row (many micro-batches: hundreds of slots) spread over all SMs instead of sharing a few.
constexpr int kEvalThreads = 64;
constexpr int kLockstepBinomWords = 512;          // binomial tables up to this size are copied to shared memory

// The part of a block's work that depends on the number of stages a lane owns.
template <int S, bool kJit>
__device__ __forceinline__ void lockstep_block(const DeviceView &v, const EvalWork &wk, const Row &row, int local_block,
                                               int64_t first, int64_t *__restrict__ batch_out,
                                               int64_t *__restrict__ busy_out, int smem_words,
                                               unsigned char *smem_raw, uint64_t *bar, const int64_t *binom)
{
    const int64_t lo = wk.lo, hi = wk.hi;
    const int pp = row.pp;
    const int wl = pp / S;                         // lanes of a warp per candidate
    const int warps = blockDim.x >> 5;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int cpb = warps * (32 / wl);             // candidates per block
    const int64_t cta_first = lo + (int64_t)local_block * cpb;
    if (cta_first >= hi) return;                   // the whole block leaves: no barrier is left waiting
    const int64_t cta_last = min(hi, cta_first + (int64_t)cpb) - 1;

    // ---- stage the prefix rows of the entries this block touches -----------------------
    const int e_lo = split_local(row, cta_first).entry;
    const int e_hi = split_local(row, cta_last).entry;
    const int n_stage = e_hi - e_lo + 1;
    const int lp = v.tc.lp;
    const int max_stage_entries = smem_words / (2 * lp);
    int64_t *sm_f = reinterpret_cast<int64_t *>(smem_raw);
    int64_t *sm_b = sm_f + (int64_t)max_stage_entries * lp;
    bool staged = false;
    if (max_stage_entries > 0 && n_stage <= max_stage_entries) {
        const uint32_t bytes = (uint32_t)(n_stage * lp * sizeof(int64_t));
        staged = stage_two_tables(bar, sm_f, v.etf + (int64_t)e_lo * lp, sm_b,
                                  v.etb + (int64_t)e_lo * lp, bytes, v.status, v.stage_polls);
    }

    const int seg = lane / wl, seg_lane = lane - seg * wl;
    int64_t local = cta_first + warp * (32 / wl) + seg;
    const bool valid = local < hi;
    if (!valid) local = hi - 1;                    // idle segments shadow a real candidate
    const CandidateCoords cc = split_local(row, local);
    const Entry en = v.entries[cc.entry];
    const int64_t *pf = staged ? sm_f + (int64_t)(cc.entry - e_lo) * lp : v.etf + (int64_t)cc.entry * lp;
    const int64_t *pb = staged ? sm_b + (int64_t)(cc.entry - e_lo) * lp : v.etb + (int64_t)cc.entry * lp;

    int n_slots = 2 * (en.m + pp - 1);
    n_slots = __reduce_max_sync(0xffffffffu, n_slots);

    const StageResult<S> R = lockstep_candidate<S, false, kJit>(v, row, en, cc.entry, pf, pb, cc.sched, cc.part_rank,
                                                                seg_lane, wl, n_slots, nullptr, binom);
    if (!valid) return;
    const int64_t out = row.offset + local - first;
    if (seg_lane == 0) batch_out[out] = R.batch;
    if (busy_out) {
        int64_t *bo = busy_out + out * v.sc.pp_max;
#pragma unroll
        for (int k = 0; k < S; ++k) bo[seg_lane * S + k] = R.busy[k];
        for (int z = pp + seg_lane; z < v.sc.pp_max; z += wl) bo[z] = 0;
    }
}

template <bool kJit>
__global__ void __launch_bounds__(kEvalThreads)
eval_lockstep_kernel(DeviceView v, EvalBatch batch, int64_t first, int64_t *__restrict__ batch_out,
                     int64_t *__restrict__ busy_out, int smem_words)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t bar;
    __shared__ int64_t binom_s[kLockstepBinomWords];
    const int64_t *binom = stage_binom(v, binom_s, kLockstepBinomWords);
    int wi = 0;
    while (wi + 1 < batch.n && (int)blockIdx.x >= batch.w[wi + 1].block_begin) ++wi;
    const EvalWork &wk = batch.w[wi];
    const Row row = v.rows[wk.row];
    // A row's candidates grow in micro-batch count, hence in slots, with their index: its last
    // blocks are the long ones and take the first block numbers, so that they start first.
    const int local_block = wk.nx - 1 - ((int)blockIdx.x - wk.block_begin);
    if (row.pp > 32) lockstep_block<2, kJit>(v, wk, row, local_block, first, batch_out, busy_out, smem_words, smem_raw, &bar, binom);
    else lockstep_block<1, kJit>(v, wk, row, local_block, first, batch_out, busy_out, smem_words, smem_raw, &bar, binom);
}

// Interleaved 1F1B and bidirectional-pipeline candidates (interleaved.cuh, bidirectional.cuh):
// pp lanes per candidate, 32 / pp candidates per warp, each with arrays of its own in shared memory.
__host__ __device__ inline int warp_candidate_words(const Row &row)
{
    return row.two_way ? bidirectional_words(row.pp, bidirectional_kept_cap(row.pp)) : interleaved_words(row.pp, row.v);
}
__host__ __device__ inline int warp_candidate_lanes(const Row &row) { return row.pp < 32 ? row.pp : 32; }

__global__ void __launch_bounds__(kIlvThreads)
eval_interleaved_kernel(DeviceView v, EvalBatch batch, int64_t first, int64_t *__restrict__ batch_out,
                        int64_t *__restrict__ busy_out)
{
    extern __shared__ __align__(16) int64_t ilv_s[];
    __shared__ int64_t binom_s[512];
    const int64_t *binom = stage_binom(v, binom_s, 512);
    int wi = 0;
    while (wi + 1 < batch.n && (int)blockIdx.x >= batch.w[wi + 1].block_begin) ++wi;
    const EvalWork &wk = batch.w[wi];
    const Row row = v.rows[wk.row];
    const int seg = warp_candidate_lanes(row), per_warp = 32 / seg;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int slot = warp * per_warp + lane / seg;          // the candidate's number inside the block
    int64_t local = wk.lo + (int64_t)((int)blockIdx.x - wk.block_begin) * (kIlvThreads / 32) * per_warp + slot;
    const bool valid = local < wk.hi;
    if (!valid) local = wk.hi - 1;                 // an idle segment shadows a real candidate
    const CandidateCoords cc = split_local(row, local);
    const Entry en = v.entries[cc.entry];
    int64_t *mine = ilv_s + (int64_t)slot * warp_candidate_words(row);
    const IlvResult R = row.two_way
        ? bidirectional_candidate(v, row, en, cc, binom, bidirectional_arrays(mine, row.pp, order_kept(v, cc.entry)), nullptr, seg)
        : interleaved_candidate(v, row, en, cc, binom, interleaved_arrays(mine, row.pp, row.v), nullptr, seg);
    if (!valid) return;
    const int d = lane & (seg - 1);
    const int64_t out = row.offset + local - first;
    if (d == 0) batch_out[out] = R.batch;
    if (busy_out) {
        int64_t *bo = busy_out + out * v.sc.pp_max;
        if (d < row.pp) bo[d] = R.busy;
        for (int z = row.pp + d; z < v.sc.pp_max; z += seg) bo[z] = 0;
    }
}

// Work items collected for one kernel instance, launched when full or at the end.
struct Pending {
    EvalBatch batch{};
    int blocks = 0;
    int smem_words = 0;
};

constexpr int kMaxBlocks = 1 << 30;                // blocks of one launch

// Candidates per block of the lock-step kernel: 32 / pp per warp, one per warp (two stages per lane) at pp = 64.
int lockstep_cpb(const Row &row)
{
    return row.pp > 32 ? kEvalThreads / 32 : (kEvalThreads / 32) * (32 / row.pp);
}

int lockstep_smem_words(const DeviceView &v, const Row &row)
{
    const int cpb = lockstep_cpb(row);
    const int64_t per_entry = row.n_part * row.n_sched;
    int64_t span = (cpb + per_entry - 1) / per_entry + 1;
    if (span > row.n_entries) span = row.n_entries;
    const int64_t words = span * v.tc.lp * 2;
    return words * (int64_t)sizeof(int64_t) > 96 * 1024 ? 0 : (int)words;     // too wide: global reads
}

void flush_lockstep(cudaStream_t s, const DeviceView &v, Pending &p, int64_t first, int64_t *batch_out,
                    int64_t *busy_out, int64_t *launches)
{
    if (p.batch.n == 0) return;
    const size_t smem = (size_t)p.smem_words * sizeof(int64_t);
    if (v.tc.n_jitter > 0) {
        ensure_dynamic_smem(reinterpret_cast<const void *>(&eval_lockstep_kernel<true>), smem);
        eval_lockstep_kernel<true><<<p.blocks, kEvalThreads, smem, s>>>(v, p.batch, first, batch_out, busy_out, p.smem_words);
    } else {
        ensure_dynamic_smem(reinterpret_cast<const void *>(&eval_lockstep_kernel<false>), smem);
        eval_lockstep_kernel<false><<<p.blocks, kEvalThreads, smem, s>>>(v, p.batch, first, batch_out, busy_out, p.smem_words);
    }
    ++*launches;
    p = Pending{};
}

template <int PP, typename T, bool kBusy>
void flush_thread(cudaStream_t s, const DeviceView &v, Pending &p, int64_t first, int64_t *batch_out,
                  int64_t *busy_out, int64_t *launches)
{
    if (p.batch.n == 0) return;
    const size_t smem = (size_t)p.smem_words * sizeof(int64_t);
    if (v.tc.n_jitter > 0) {
        ensure_dynamic_smem(reinterpret_cast<const void *>(&eval_thread_kernel<PP, T, kBusy, true>), smem);
        eval_thread_kernel<PP, T, kBusy, true><<<p.blocks, kThreadBlock, smem, s>>>(v, p.batch, first, batch_out, busy_out);
    } else {
        ensure_dynamic_smem(reinterpret_cast<const void *>(&eval_thread_kernel<PP, T, kBusy, false>), smem);
        eval_thread_kernel<PP, T, kBusy, false><<<p.blocks, kThreadBlock, smem, s>>>(v, p.batch, first, batch_out, busy_out);
    }
    ++*launches;
    p = Pending{};
}

// Thread-kernel instances are indexed by (log2 pp, narrow).
template <typename T, bool kBusy>
void flush_thread_pp(int log2pp, cudaStream_t s, const DeviceView &v, Pending &p, int64_t first,
                     int64_t *batch_out, int64_t *busy_out, int64_t *launches)
{
    switch (log2pp) {
    case 0: flush_thread<1, T, kBusy>(s, v, p, first, batch_out, busy_out, launches); break;
    case 1: flush_thread<2, T, kBusy>(s, v, p, first, batch_out, busy_out, launches); break;
    case 2: flush_thread<4, T, kBusy>(s, v, p, first, batch_out, busy_out, launches); break;
    case 3: flush_thread<8, T, kBusy>(s, v, p, first, batch_out, busy_out, launches); break;
    default: flush_thread<16, T, kBusy>(s, v, p, first, batch_out, busy_out, launches); break;
    }
}

void flush_thread_any(int log2pp, bool narrow, cudaStream_t s, const DeviceView &v, Pending &p, int64_t first,
                      int64_t *batch_out, int64_t *busy_out, int64_t *launches)
{
    if (narrow) {
        if (busy_out) flush_thread_pp<uint32_t, true>(log2pp, s, v, p, first, batch_out, busy_out, launches);
        else flush_thread_pp<uint32_t, false>(log2pp, s, v, p, first, batch_out, busy_out, launches);
    } else {
        if (busy_out) flush_thread_pp<int64_t, true>(log2pp, s, v, p, first, batch_out, busy_out, launches);
        else flush_thread_pp<int64_t, false>(log2pp, s, v, p, first, batch_out, busy_out, launches);
    }
}

int ilog2(int v) { int b = 0; while ((1 << (b + 1)) <= v) ++b; return b; }

// The shared-memory budget of the kernel instance that evaluates rows of this pp and arithmetic width.
int thread_budget_words(int pp, bool narrow, bool jitter)
{
    switch (ilog2(pp)) {
    case 0: return narrow ? thread_kernel_budget_words<1, uint32_t>(jitter) : thread_kernel_budget_words<1, int64_t>(jitter);
    case 1: return narrow ? thread_kernel_budget_words<2, uint32_t>(jitter) : thread_kernel_budget_words<2, int64_t>(jitter);
    case 2: return narrow ? thread_kernel_budget_words<4, uint32_t>(jitter) : thread_kernel_budget_words<4, int64_t>(jitter);
    case 3: return narrow ? thread_kernel_budget_words<8, uint32_t>(jitter) : thread_kernel_budget_words<8, int64_t>(jitter);
    default: return narrow ? thread_kernel_budget_words<16, uint32_t>(jitter) : thread_kernel_budget_words<16, int64_t>(jitter);
    }
}

}  // namespace

// Cuts candidates [lo, hi) of a row of `pp` stages into pieces of at most max_blocks blocks of the
// lock-step kernel each (block counts are computed in 64 bits: a range of billions of candidates
// must not overflow a launch's grid).  Returns the number of pieces; the first max_pieces are
// written.
int64_t lockstep_pieces(int pp, int64_t lo, int64_t hi, int64_t max_blocks, int64_t max_pieces,
                        int64_t *piece_lo, int64_t *piece_hi, int32_t *piece_blocks)
{
    Row row{};
    row.pp = pp;
    const int64_t cpb = lockstep_cpb(row);
    const int64_t per_piece = max_blocks * cpb;            // candidates
    int64_t n = 0;
    for (int64_t a = lo; a < hi; a += per_piece, ++n) {
        const int64_t b = hi - a < per_piece ? hi : a + per_piece;
        if (n < max_pieces) {
            piece_lo[n] = a; piece_hi[n] = b;
            piece_blocks[n] = (int32_t)((b - a + cpb - 1) / cpb);
        }
    }
    return n;
}

void launch_eval(cudaStream_t s, const SideStream &ss, const DeviceView &v, const Row *rows, int n_rows,
                 const Entry *entries, int64_t first, int64_t count, int64_t *batch_out, int64_t *busy_out,
                 int64_t *launches)
{
    const int64_t last = first + count;
    struct ThreadItem { EvalWork w; int lg; bool narrow; int blocks, words; };
    std::vector<EvalWork> lock_items;              // lock-step kernel
    std::vector<int> lock_words;
    std::vector<ThreadItem> thread_items;          // one-partition-per-thread kernel
    std::vector<EvalWork> ilv_items;               // interleaved 1F1B kernel (a candidate per warp)
    int ilv_words = 0;
    constexpr int64_t kPieceBlocks = 1 << 24;

    auto add_lockstep = [&](int r, int64_t lo, int64_t hi) {
        for (int64_t a = lo; a < hi;) {
            int64_t pl, ph; int32_t blocks;
            lockstep_pieces(rows[r].pp, a, hi, kPieceBlocks, 1, &pl, &ph, &blocks);
            EvalWork w{};
            w.row = r; w.lo = pl; w.hi = ph; w.nx = blocks;
            lock_items.push_back(w);
            lock_words.push_back(lockstep_smem_words(v, rows[r]));
            a = ph;
        }
    };

    for (int r = 0; r < n_rows; ++r) {
        const Row &row = rows[r];
        const int64_t lo = first > row.offset ? first - row.offset : 0;
        const int64_t hi = last < row.offset + row.size ? last - row.offset : row.size;
        if (hi <= lo) continue;
        if (row.v > 1 || row.two_way) {
            const int64_t cpb = (kIlvThreads / 32) * (32 / warp_candidate_lanes(row));      // candidates per block
            for (int64_t a = lo; a < hi; a += kPieceBlocks * cpb) {
                EvalWork w{};
                w.row = r; w.lo = a; w.hi = hi - a < kPieceBlocks * cpb ? hi : a + kPieceBlocks * cpb;
                w.nx = (int)((w.hi - w.lo + cpb - 1) / cpb);
                ilv_items.push_back(w);
            }
            const int words = (int)cpb * warp_candidate_words(row);                        // of a block
            if (words > ilv_words) ilv_words = words;
            continue;
        }
        if (row.pp > 16) { add_lockstep(r, lo, hi); continue; }
        // Short pipelines: cut the range into runs of entries with the same arithmetic width; a
        // run with enough partitions goes to the one-partition-per-thread kernel, the rest to
        // the lock-step kernel.
        const Entry *row_entries = entries + row.entry0;
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
            const int64_t nx = (n_parts + kThreadBlock - 1) / kThreadBlock;
            const int64_t ny = (n_e + ept - 1) / ept;
            if (n_parts * ny >= 2048 && nx * ny < kMaxBlocks) {
                ThreadItem it{};
                it.lg = ilog2(row.pp); it.narrow = narrow; it.blocks = (int)(nx * ny);
                EvalWork &w = it.w;
                w.row = r; w.e_begin = r0; w.e_end = r1; w.ept = ept; w.p_lo = p_lo; w.p_hi = p_hi;
                w.lo = lo_r; w.hi = hi_r; w.nx = (int)nx;
                const int binom_words = v.sc.partition_mode ? v.tc.n_layers * v.sc.binom_k : 0;
                const int budget = thread_budget_words(row.pp, narrow, v.tc.n_jitter > 0);
                const bool use32 = narrow && v.pfb32 != nullptr && (row.dp == 1 || v.dt32 != nullptr);   // as in the kernel
                it.words =
                    use32 ? thread_kernel_smem32(row.n_entries, v.tc.lp, v.tab_words32, v.dt32 != nullptr, binom_words, budget).words
                          : thread_kernel_smem(row.n_entries, v.tc.lp, v.tab_words, v.dt != nullptr, binom_words, budget).words;
                thread_items.push_back(it);
            } else {
                add_lockstep(r, lo_r, hi_r);
            }
            r0 = r1;
        }
    }

    // The lock-step launches (few warps that run for long) go first, on a high-priority side
    // stream forked from `s` and joined to it at the end, so that they run beside the
    // thread-kernel launches (largest first) that fill the rest of the device.  Without
    // thread-kernel work there is nothing to run beside: everything goes to `s` directly.
    const bool use_side = ss.side[0] != nullptr && !thread_items.empty() && !lock_items.empty();
    cudaStream_t ls = s;
    if (use_side) {
        cudaEventRecord(ss.fork, s);
        cudaStreamWaitEvent(ss.side[0], ss.fork, 0);
        ls = ss.side[0];
    }
    Pending p;
    for (size_t i = 0; i < lock_items.size(); ++i) {
        if (p.batch.n == kMaxEvalWork || p.blocks > kMaxBlocks - lock_items[i].nx)
            flush_lockstep(ls, v, p, first, batch_out, busy_out, launches);
        EvalWork &w = p.batch.w[p.batch.n++];
        w = lock_items[i];
        w.block_begin = p.blocks;
        p.blocks += w.nx;
        // one dynamic size per launch: the largest any item wants (items that want none still work)
        if (lock_words[i] > p.smem_words) p.smem_words = lock_words[i];
    }
    flush_lockstep(ls, v, p, first, batch_out, busy_out, launches);
    // interleaved candidates: a kernel of their own, on the caller's stream
    auto flush_interleaved = [&]() {
        if (p.batch.n == 0) return;
        const size_t smem = (size_t)ilv_words * sizeof(int64_t);
        ensure_dynamic_smem(reinterpret_cast<const void *>(&eval_interleaved_kernel), smem);
        eval_interleaved_kernel<<<p.blocks, kIlvThreads, smem, s>>>(v, p.batch, first, batch_out, busy_out);
        ++*launches;
        p = Pending{};
    };
    for (const EvalWork &item : ilv_items) {
        if (p.batch.n == kMaxEvalWork || p.blocks > kMaxBlocks - item.nx) flush_interleaved();
        EvalWork &w = p.batch.w[p.batch.n++];
        w = item;
        w.block_begin = p.blocks;
        p.blocks += w.nx;
    }
    flush_interleaved();
    for (int lg = 4; lg >= 0; --lg)
        for (int nw = 1; nw >= 0; --nw) {
            for (const ThreadItem &it : thread_items) {
                if (it.lg != lg || it.narrow != (nw == 1)) continue;
                if (p.batch.n == kMaxEvalWork || p.blocks > kMaxBlocks - it.blocks)
                    flush_thread_any(lg, nw == 1, s, v, p, first, batch_out, busy_out, launches);
                EvalWork &w = p.batch.w[p.batch.n++];
                w = it.w;
                w.block_begin = p.blocks;
                p.blocks += it.blocks;
                if (it.words > p.smem_words) p.smem_words = it.words;
            }
            flush_thread_any(lg, nw == 1, s, v, p, first, batch_out, busy_out, launches);
        }
    if (use_side) {
        cudaEventRecord(ss.join[0], ss.side[0]);
        cudaStreamWaitEvent(s, ss.join[0], 0);
    }
}

}  // namespace distsim
