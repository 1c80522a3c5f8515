// One stage partition per thread: the evaluation kernel for rows with many partitions and
// pp <= 16.
//
// A thread owns one stage partition of the row and walks the row's entries (micro-batch
// counts) and schedules with it, so the partition is decoded once and the stage costs once
// per entry.  All per-stage state of the pipeline recurrence - forward/backward item cost,
// device-free time, latest forward end - lives in registers (the stage loops are fully
// unrolled, pp is a template parameter), so a recurrence cell is exactly one max and one add
// with no memory traffic and no shuffles, and every lane does useful work in every
// instruction.  Item order per schedule (any order consistent with every device's own order and
// with the data dependencies gives the same times):
//   GPipe  forward waves j = 0..m-1 over stages 0..pp-1, then backward waves over pp-1..0.
//   1F1B   warm-up: forward wave j covers stages 0..pp-1-j (j < min(pp, m));
//          then backward wave i over stages pp-1..0, each stage following its backward item
//          with forward item w_d + i while that exists (w_d = min(pp-d, m)); the forward item
//          takes its input from the previous wave's forward end of stage d-1.
// Gradient buckets: the end of a stage's bucket lane is start-of-last-backward + DT where
//   DT = max over bucket groups of (ready offset of the group + cost of all buckets from it on),
// which does not depend on the schedule; with X = max(0, DT - backward item cost) the stage's
// contribution to the batch time is main_end + X and its activity time m(fop+bop) + X.
//
// Relative time frames (tables without jitter).  Along a wave the cell t_d = max(t_{d-1}, free_d)
// + c_d chains a max and an add per stage.  Measuring stage d's times from the cost prefix
// C_d = c_0 + .. + c_d (w_d = t_d - C_d) turns the wave into
//   w_d = max(r_d + c_d, w_{d-1}),   r_d = w_d of the previous wave,
// a single fused add-max per cell (__viaddmax_u32 on 32-bit times).  Backward waves use the
// suffix sums of the backward costs, shifted by their total so that every value stays
// non-negative (entries whose time bound plus that shift does not fit 32 bits keep the plain
// form in 32-bit arithmetic).  In a steady 1F1B wave - a
// backward and a forward item per stage - the same change of variables, with
// h_d = latest forward end of stage d - fop_d + bop_0 + .. + bop_{d-1} and fb_d = fop_d + bop_d:
//   w_d = max(h_d + fb_d, w_{d+1}),   h_d <- max(h_{d-1} + fb_{d-1}, w_d),
// again one fused add-max per cell.  All of it is exact integer arithmetic.
//
// Arithmetic width.  On this GPU a 64-bit max + add costs six integer instructions, a 32-bit
// one two (one when fused).  Every entry carries an upper bound on every time any of its
// candidates can produce; the entries whose bound is below 2^32 are evaluated with T = uint32_t
// (exactly: nothing can overflow), the others with T = int64_t.
//
// Tables.  Before the recurrence of an entry a thread works out its pp stage costs and
// bucket-lane excesses; for entries with few micro-batches that part outweighs the cells.  The
// block therefore stages what it reads in shared memory with bulk copies: the prefix rows of
// the row's entries, the binomial table of the unranking and the bucket-lane tables of as many
// of the row's last entries as fit the budget that keeps the kernel's resident blocks per SM.
// The 32-bit instance reads 32-bit copies of the tables (forward and backward prefix packed
// into one 8-byte word), which halves the shared memory and the arithmetic of that part.
#pragma once

#include "recurrence.cuh"
#include "smem_stage.cuh"

namespace distsim {

constexpr int kThreadBlock = 128;
constexpr int kMaxRowEntries = 16;      // entries whose scalars are kept in shared memory

// Resident blocks per SM asked of the compiler (caps the registers per thread).
template <int PP, typename T>
__host__ __device__ constexpr int thread_kernel_min_blocks()
{
    return sizeof(T) == 8 ? (PP >= 16 ? 3 : 4) : (PP >= 16 ? 5 : 8);
}

template <typename T> __device__ __forceinline__ T vmax(T a, T b) { return a > b ? a : b; }

// One recurrence cell: end = max(input arrival, device free) + cost.
template <typename T> __device__ __forceinline__ T cell(T arrival, T free_at, T cost)
{
    return (T)(vmax(arrival, free_at) + cost);
}

template <int PP, typename T>
struct ThreadState {
    T fop[PP], bop[PP];
};

// Per-micro-batch jitter: extra time of the item of micro-batch j on stage d, from tables in
// shared memory ([slot][stage], the slot count a power of two).  Every thread of a block asks
// for the same (j, d), so the reads are broadcasts.  Without a jitter table (kJit false) the
// accessors fold to zero at compile time.
template <int PP, typename T, bool kJit>
struct JitterTab {
    const T *f, *b;
    int mask;
    __device__ __forceinline__ T fwd(int j, int d) const { return kJit ? f[(j & mask) * PP + d] : (T)0; }
    __device__ __forceinline__ T bwd(int j, int d) const { return kJit ? b[(j & mask) * PP + d] : (T)0; }
};

// GPipe: returns main-lane end of every stage in free_at.
template <int PP, typename T, bool kJit>
__device__ __forceinline__ void run_gpipe(const ThreadState<PP, T> &c, int m, T (&free_at)[PP],
                                          const JitterTab<PP, T, kJit> &jt)
{
#pragma unroll
    for (int d = 0; d < PP; ++d) free_at[d] = 0;
#pragma unroll 2
    for (int j = 0; j < m; ++j) {
        T t = free_at[0] + c.fop[0] + jt.fwd(j, 0);
        free_at[0] = t;
#pragma unroll
        for (int d = 1; d < PP; ++d) { t = cell(t, free_at[d], (T)(c.fop[d] + jt.fwd(j, d))); free_at[d] = t; }
    }
#pragma unroll 2
    for (int j = 0; j < m; ++j) {
        T t = free_at[PP - 1] + c.bop[PP - 1] + jt.bwd(j, PP - 1);
        free_at[PP - 1] = t;
#pragma unroll
        for (int d = PP - 2; d >= 0; --d) { t = cell(t, free_at[d], (T)(c.bop[d] + jt.bwd(j, d))); free_at[d] = t; }
    }
}

// 1F1B backward wave i in which the stages d >= D0 also run a forward item (D0 may be PP): the
// backward item is B(d, i), the forward item F(d, PP - d + i).
template <int PP, int D0, typename T, bool kJit>
__device__ __forceinline__ void wave_1f1b(const ThreadState<PP, T> &c, T (&free_at)[PP], T (&last_f)[PP],
                                          const JitterTab<PP, T, kJit> &jt, int i)
{
    T t = 0;
#pragma unroll
    for (int d = PP - 1; d >= 0; --d) {
        const T cb = c.bop[d] + jt.bwd(i, d);
        t = d == PP - 1 ? (T)(free_at[d] + cb) : cell(t, free_at[d], cb);
        free_at[d] = t;
        if (d >= D0) {
            const T cf = c.fop[d] + jt.fwd(PP - d + i, d);
            const T f = d == 0 ? (T)(free_at[0] + cf) : cell(last_f[d > 0 ? d - 1 : 0], free_at[d], cf);
            free_at[d] = f;
            last_f[d] = f;
        }
    }
}

// A steady-state 1F1B wave: every stage runs its backward item and then a forward item.  After
// a forward item the device's free time IS that item's end, so inside the steady state the
// free times are not kept separately: last_f doubles as the free time.
template <int PP, typename T, bool kJit>
__device__ __forceinline__ void wave_1f1b_steady(const ThreadState<PP, T> &c, T (&last_f)[PP],
                                                 const JitterTab<PP, T, kJit> &jt, int i)
{
    T t = 0;
#pragma unroll
    for (int d = PP - 1; d >= 0; --d) {
        const T cb = c.bop[d] + jt.bwd(i, d);
        const T cf = c.fop[d] + jt.fwd(PP - d + i, d);
        t = d == PP - 1 ? (T)(last_f[d] + cb) : cell(t, last_f[d], cb);
        last_f[d] = d == 0 ? (T)(t + cf) : cell(last_f[d > 0 ? d - 1 : 0], t, cf);
    }
}

// Runs the last waves, in which fewer and fewer stages still have a forward item: with K waves
// to go (wave i = m - K), the stages with pp - d < K do (statically unrolled over K = PP .. 1).
template <int PP, int K, typename T, bool kJit>
struct TailWaves {
    static __device__ __forceinline__ void run(const ThreadState<PP, T> &c, int m, T (&free_at)[PP], T (&last_f)[PP],
                                               const JitterTab<PP, T, kJit> &jt)
    {
        if (K <= m) wave_1f1b<PP, PP - K + 1, T, kJit>(c, free_at, last_f, jt, m - K);
        TailWaves<PP, K - 1, T, kJit>::run(c, m, free_at, last_f, jt);
    }
};
template <int PP, typename T, bool kJit>
struct TailWaves<PP, 0, T, kJit> {
    static __device__ __forceinline__ void run(const ThreadState<PP, T> &, int, T (&)[PP], T (&)[PP],
                                               const JitterTab<PP, T, kJit> &) {}
};

// Warm-up forward wave J over stages 0 .. PP-1-J.
template <int PP, int J, typename T, bool kJit>
struct WarmWaves {
    static __device__ __forceinline__ void run(const ThreadState<PP, T> &c, int m, T (&free_at)[PP], T (&last_f)[PP],
                                               const JitterTab<PP, T, kJit> &jt)
    {
        if (J < m) {
            T t = free_at[0] + c.fop[0] + jt.fwd(J, 0);
            free_at[0] = t; last_f[0] = t;
#pragma unroll
            for (int d = 1; d < PP - J; ++d) {
                t = cell(t, free_at[d], (T)(c.fop[d] + jt.fwd(J, d)));
                free_at[d] = t; last_f[d] = t;
            }
        }
        WarmWaves<PP, J + 1, T, kJit>::run(c, m, free_at, last_f, jt);
    }
};
template <int PP, typename T, bool kJit>
struct WarmWaves<PP, PP, T, kJit> {
    static __device__ __forceinline__ void run(const ThreadState<PP, T> &, int, T (&)[PP], T (&)[PP],
                                               const JitterTab<PP, T, kJit> &) {}
};

// max(a + b, c): one instruction on 32-bit operands (the GPU's fused add-max).
template <typename T> __device__ __forceinline__ T addmax(T a, T b, T c) { return vmax((T)(a + b), c); }
template <> __device__ __forceinline__ uint32_t addmax<uint32_t>(uint32_t a, uint32_t b, uint32_t c)
{
    return __viaddmax_u32(a, b, c);
}

// GPipe without jitter, in relative frames (see the header): returns main-lane ends in free_at.
template <int PP, typename T>
__device__ __forceinline__ void run_gpipe_rel(const ThreadState<PP, T> &c, int m, T (&free_at)[PP])
{
    // forward, frame w_d = t_d - (fop[0] + .. + fop[d]): r[d] holds w_d of the previous wave;
    // wave 0 has w = 0 on every stage
    T r[PP];
#pragma unroll
    for (int d = 0; d < PP; ++d) r[d] = 0;
#pragma unroll 2
    for (int j = 1; j < m; ++j) {
        T w = r[0] + c.fop[0];
        r[0] = w;
#pragma unroll
        for (int d = 1; d < PP; ++d) { w = addmax(r[d], c.fop[d], w); r[d] = w; }
    }
    // backward, frame w_d = t_d + (bop[0] + .. + bop[d-1]): r[d] = (device-free time of stage d)
    // + that prefix; the stage is free at r[d] + fop[0] + .. + fop[d] after its last forward item
    T cf = 0, pb = 0;
#pragma unroll
    for (int d = 0; d < PP; ++d) { cf += c.fop[d]; r[d] = (T)(r[d] + cf + pb); pb += c.bop[d]; }
#pragma unroll 2
    for (int j = 0; j < m; ++j) {
        T w = r[PP - 1] + c.bop[PP - 1];
        r[PP - 1] = w;
#pragma unroll
        for (int d = PP - 2; d >= 0; --d) { w = addmax(r[d], c.bop[d], w); r[d] = w; }
    }
    pb = 0;
#pragma unroll
    for (int d = 0; d < PP; ++d) { free_at[d] = (T)(r[d] - pb); pb += c.bop[d]; }
}

// A steady-state 1F1B wave without jitter.  fb[d] = fop[d] + bop[d];
// h[d] = latest forward end of stage d - fop[d] + (bop[0] + .. + bop[d-1]).
template <int PP, typename T>
__device__ __forceinline__ void wave_1f1b_steady_rel(const T (&fb)[PP], T (&h)[PP])
{
    T w = 0;
#pragma unroll
    for (int d = PP - 1; d >= 0; --d) {
        w = d == PP - 1 ? (T)(h[d] + fb[d]) : addmax(h[d], fb[d], w);                  // backward item
        h[d] = d == 0 ? w : addmax(h[d > 0 ? d - 1 : 0], fb[d > 0 ? d - 1 : 0], w);   // forward item
    }
}

// 1F1B without jitter and with m >= PP, entirely in relative frames.
//   warm-up   forward frame as in run_gpipe_rel: r[d] = w_d of stage d's latest forward item.
//   then      h[d] = (end of stage d's latest forward item) - fop[d] + bop[0] + .. + bop[d-1]
//             while the stage's latest item is a forward one ("after F"), and
//             h[d] = (end of its latest backward item) + bop[0] + .. + bop[d-1] once it is a
//             backward one ("after B", in the last waves); the backward item of the next wave is
//             w_d = max(h[d] + y_d, w_{d+1}) with y_d = fop[d] + bop[d] after F and bop[d] after B.
// Wave K of the tail (K waves to go, i = m - K): stages d >= PP-K+1 still run a forward item; a
// stage is "after F" iff it ran one in the wave before (d >= PP-K; in the first wave, K = PP,
// that is every stage).  Requires m >= PP: all PP warm-up waves and all PP tail waves exist.
template <int PP, int K, typename T>
struct TailWavesRel {
    static __device__ __forceinline__ void run(const ThreadState<PP, T> &c, const T (&fb)[PP], int m, T (&h)[PP])
    {
        {
            T w = 0;
#pragma unroll
            for (int d = PP - 1; d >= 0; --d) {
                const T y = d >= PP - K ? fb[d] : c.bop[d];
                w = d == PP - 1 ? (T)(h[d] + y) : addmax(h[d], y, w);
                if (d >= PP - K + 1) h[d] = d == 0 ? w : addmax(h[d > 0 ? d - 1 : 0], fb[d > 0 ? d - 1 : 0], w);
                else h[d] = w;
            }
        }
        TailWavesRel<PP, K - 1, T>::run(c, fb, m, h);
    }
};
template <int PP, typename T>
struct TailWavesRel<PP, 0, T> {
    static __device__ __forceinline__ void run(const ThreadState<PP, T> &, const T (&)[PP], int, T (&)[PP]) {}
};

// Warm-up forward wave J >= 1 over stages 0 .. PP-1-J (wave 0 leaves w = 0 everywhere).
template <int PP, int J, typename T>
struct WarmWavesRel {
    static __device__ __forceinline__ void run(const ThreadState<PP, T> &c, int m, T (&r)[PP])
    {
        {
            T w = r[0] + c.fop[0];
            r[0] = w;
#pragma unroll
            for (int d = 1; d < PP - J; ++d) { w = addmax(r[d], c.fop[d], w); r[d] = w; }
        }
        WarmWavesRel<PP, J + 1, T>::run(c, m, r);
    }
};
template <int PP, typename T>
struct WarmWavesRel<PP, PP, T> {
    static __device__ __forceinline__ void run(const ThreadState<PP, T> &, int, T (&)[PP]) {}
};

template <int PP, typename T>
__device__ __forceinline__ void run_1f1b_rel(const ThreadState<PP, T> &c, int m, T (&free_at)[PP])
{
    T h[PP], fb[PP];
#pragma unroll
    for (int d = 0; d < PP; ++d) { h[d] = 0; fb[d] = c.fop[d] + c.bop[d]; }
    WarmWavesRel<PP, (PP > 1 ? 1 : PP), T>::run(c, m, h);
    // forward frame -> the frame of h: add fop[0] + .. + fop[d-1] and bop[0] + .. + bop[d-1]
    T off = 0;
#pragma unroll
    for (int d = 0; d < PP; ++d) { h[d] += off; off += fb[d]; }
    if (m > PP) {
#pragma unroll 2
        for (int i = 0; i < m - PP; ++i) wave_1f1b_steady_rel<PP, T>(fb, h);
    }
    TailWavesRel<PP, PP, T>::run(c, fb, m, h);
    // every stage's latest item is now its last backward item
    T pb = 0;
#pragma unroll
    for (int d = 0; d < PP; ++d) { free_at[d] = (T)(h[d] - pb); pb += c.bop[d]; }
}

template <int PP, typename T, bool kJit>
__device__ __forceinline__ void run_1f1b(const ThreadState<PP, T> &c, int m, T (&free_at)[PP],
                                         const JitterTab<PP, T, kJit> &jt)
{
    T last_f[PP];
#pragma unroll
    for (int d = 0; d < PP; ++d) { free_at[d] = 0; last_f[d] = 0; }
    WarmWaves<PP, 0, T, kJit>::run(c, m, free_at, last_f, jt);
    // waves i = 0 .. m-PP-1: every stage still has a forward item to pair with its backward;
    // entering them every stage's latest item is a forward one (free_at == last_f)
    if (m > PP) {
#pragma unroll 2
        for (int i = 0; i < m - PP; ++i) wave_1f1b_steady<PP, T, kJit>(c, last_f, jt, i);
#pragma unroll
        for (int d = 0; d < PP; ++d) free_at[d] = last_f[d];
    }
    // the last min(PP, m) waves
    TailWaves<PP, PP, T, kJit>::run(c, m, free_at, last_f, jt);
}

// The same schedule with the warm-up and last waves as loops over the wave number (the set of
// stages that run a forward item is tested per stage at run time) instead of one unrolled copy
// per wave: an eighth of the code.  Used for the few entries of a table without jitter that
// cannot take the relative form (m < pp, or a time bound too close to 2^32), where a smaller
// kernel is worth more than their speed.
template <int PP, typename T>
__device__ __forceinline__ void run_1f1b_compact(const ThreadState<PP, T> &c, int m, T (&free_at)[PP])
{
    T last_f[PP];
#pragma unroll
    for (int d = 0; d < PP; ++d) { free_at[d] = 0; last_f[d] = 0; }
    const int n_edge = min(PP, m);
#pragma unroll 1
    for (int J = 0; J < n_edge; ++J) {           // warm-up wave J: forward items on stages 0 .. PP-1-J
        T t = 0;
#pragma unroll
        for (int d = 0; d < PP; ++d)
            if (d < PP - J) {
                t = d == 0 ? (T)(free_at[0] + c.fop[0]) : cell(t, free_at[d], c.fop[d]);
                free_at[d] = t; last_f[d] = t;
            }
    }
    const JitterTab<PP, T, false> none{nullptr, nullptr, 0};
    if (m > PP) {
#pragma unroll 1
        for (int i = 0; i < m - PP; ++i) wave_1f1b_steady<PP, T, false>(c, last_f, none, i);
#pragma unroll
        for (int d = 0; d < PP; ++d) free_at[d] = last_f[d];
    }
#pragma unroll 1
    for (int K = n_edge; K >= 1; --K) {          // K waves to go: stages d >= PP-K+1 still run a forward item
        T t = 0;
#pragma unroll
        for (int d = PP - 1; d >= 0; --d) {
            t = d == PP - 1 ? (T)(free_at[d] + c.bop[d]) : cell(t, free_at[d], c.bop[d]);
            free_at[d] = t;
            if (d >= PP - K + 1) {
                const T f = d == 0 ? (T)(t + c.fop[0]) : cell(last_f[d > 0 ? d - 1 : 0], t, c.fop[d]);
                free_at[d] = f; last_f[d] = f;
            }
        }
    }
}

// Shared-memory plan of a block (offsets in int64 words from the dynamic shared base): the
// prefix rows of every entry of the row; then, when per-entry bucket-lane tables exist, the
// binomial table of the unranking and the bucket-lane tables of the row's last entries (as many
// as the budget allows: the entries with the most micro-batches come last); otherwise the row's
// two bucket tables - each as far as it fits.
struct ThreadKernelSmem {
    int32_t n_entries_staged;   // 0: read prefix rows from global
    int32_t tables_staged;      // 1: NB / TP tables of the row are in shared memory
    int32_t n_dt_staged;        // bucket-lane tables of the row's last n_dt_staged entries are in shared memory
    int32_t binom_staged;       // 1: the binomial table is in shared memory
    int32_t off_etb, off_nb, off_tp, off_dt, off_binom;
    int32_t words;              // dynamic shared memory needed, in int64 words
};
// Dynamic shared memory (int64 words) a block may use without lowering the number of resident
// blocks the kernel is compiled for: an SM's 228 KB, less 1 KB per block, less the kernel's
// static arrays.
template <int PP, typename T>
__host__ __device__ constexpr int thread_kernel_budget_words(bool jitter)
{
    const int per_block = 233472 / thread_kernel_min_blocks<PP, T>() - 1024;
    const int fixed = PP * kThreadBlock * (int)sizeof(T) + (PP + 1) * kThreadBlock * 2 + 16 * 24 + 256 +
                      (jitter ? 2 * 64 * PP * (int)sizeof(T) : 0);
    return (per_block - fixed) / 8 > 0 ? (per_block - fixed) / 8 : 0;
}
__host__ __device__ inline ThreadKernelSmem thread_kernel_smem(int n_entries, int lp, int tab_words, bool have_dt,
                                                               int binom_words, int budget_words)
{
    ThreadKernelSmem plan{};
    int words = 0;
    if (n_entries * lp * 2 <= 8192 && n_entries * lp * 2 <= budget_words) {
        plan.n_entries_staged = n_entries;
        plan.off_etb = n_entries * lp;
        words = n_entries * lp * 2;
    }
    if (!have_dt) {
        if (words + 2 * tab_words <= 12288 && words + 2 * tab_words <= budget_words) {
            plan.tables_staged = 1;
            plan.off_nb = words;
            plan.off_tp = words + tab_words;
            words += 2 * tab_words;
        }
    } else {
        // bulk copies move multiples of 16 bytes: an odd-sized binomial table stays in global memory
        if (binom_words > 0 && !(binom_words & 1) && words + binom_words <= budget_words) {
            plan.binom_staged = 1;
            plan.off_binom = words;
            words += binom_words;
        }
        int k = tab_words > 0 ? (budget_words - words) / tab_words : 0;
        if (k > n_entries) k = n_entries;
        if (k > 0 && (int64_t)k * tab_words * 8 < (1 << 20)) {       // one bulk copy, one barrier transaction count
            plan.n_dt_staged = k;
            plan.off_dt = words;
            words += k * tab_words;
        }
    }
    plan.words = words;
    return plan;
}

// The same plan for a launch in 32-bit arithmetic, which reads the 32-bit copies of the tables:
// one (forward, backward) prefix row per entry (lp words), the binomial table, and the 32-bit
// bucket-lane tables (tab_words32 / 2 words each) of the row's last entries.
__host__ __device__ inline ThreadKernelSmem thread_kernel_smem32(int n_entries, int lp, int tab_words32, bool have_dt,
                                                                 int binom_words, int budget_words)
{
    ThreadKernelSmem plan{};
    int words = 0;
    if (n_entries * lp <= 8192 && n_entries * lp <= budget_words) {
        plan.n_entries_staged = n_entries;
        words = n_entries * lp;                      // lp is even: the next table stays 16-byte aligned
    }
    if (binom_words > 0 && !(binom_words & 1) && words + binom_words <= budget_words) {
        plan.binom_staged = 1;
        plan.off_binom = words;
        words += binom_words;
    }
    if (have_dt) {
        const int tw = tab_words32 / 2;
        int k = (budget_words - words) / tw;
        if (k > n_entries) k = n_entries;
        if (k > 0 && (int64_t)k * tw * 8 < (1 << 20)) {
            plan.n_dt_staged = k;
            plan.off_dt = words;
            words += k * tw;
        }
    }
    plan.words = words;
    return plan;
}

// Entry scalars the hot path needs, kept in shared memory for the whole row.
struct EntryLite { int64_t p2p_intra, p2p_inter; int32_t m, rel_fits32; };

constexpr int kMaxJitterSlots = 64;

template <int PP, typename T, bool kBusy, bool kJit>
__global__ void __launch_bounds__(kThreadBlock, thread_kernel_min_blocks<PP, T>())
eval_thread_kernel(DeviceView v, EvalBatch batch, int64_t first,
                   int64_t *__restrict__ batch_out, int64_t *__restrict__ busy_out)
{
    // which work item (row and range) this block belongs to
    int wi = 0;
    while (wi + 1 < batch.n && (int)blockIdx.x >= batch.w[wi + 1].block_begin) ++wi;
    const EvalWork &wk = batch.w[wi];
    const int row_index = wk.row, e_begin = wk.e_begin, e_end = wk.e_end, entries_per_thread = wk.ept;
    const int64_t lo = wk.lo, hi = wk.hi, p_lo = wk.p_lo, p_hi = wk.p_hi;
    const int local_block = (int)blockIdx.x - wk.block_begin;
    const int block_x = local_block % wk.nx, block_y = local_block / wk.nx;
    extern __shared__ __align__(16) int64_t dsm[];
    __shared__ __align__(8) uint64_t bar;
    __shared__ T xs[PP][kThreadBlock];                // per thread, per stage: bucket-lane excess X
    __shared__ uint16_t cs[PP + 1][kThreadBlock];     // per thread: stage bounds c_0 .. c_PP
    __shared__ EntryLite ents[kMaxRowEntries];
    __shared__ T jit_f_s[kJit ? kMaxJitterSlots * PP : 1], jit_b_s[kJit ? kMaxJitterSlots * PP : 1];
    const Row &row = v.rows[row_index];
    const int lp = v.tc.lp;
    const int L1 = v.tc.n_layers + 1;
    const int binom_words = v.sc.partition_mode ? v.tc.n_layers * v.sc.binom_k : 0;
    // 32-bit arithmetic reads 32-bit copies of the prefix rows and bucket-lane tables
    const bool use32 = sizeof(T) == 4 && v.pfb32 != nullptr && (row.dp == 1 || v.dt32 != nullptr);
    const ThreadKernelSmem plan =
        use32 ? thread_kernel_smem32(row.n_entries, lp, v.tab_words32, v.dt32 != nullptr, binom_words,
                                     thread_kernel_budget_words<PP, T>(kJit))
              : thread_kernel_smem(row.n_entries, lp, v.tab_words, v.dt != nullptr, binom_words,
                                   thread_kernel_budget_words<PP, T>(kJit));
    const int dp = row.dp, n_sched = row.n_sched, sched_list = row.sched_list, period = row.p2p_period;
    const int64_t t_full = row.t_full;

    // ---- stage the row's prefix rows (and bucket tables when no per-entry table exists) ----
    const int64_t *etf_g = v.etf + (int64_t)row.entry0 * lp;
    const int64_t *etb_g = v.etb + (int64_t)row.entry0 * lp;
    const int64_t *nb_g = v.nb + row.row_tab_off;
    const int64_t *tp_g = v.tp + row.row_tab_off;
    if (threadIdx.x < kMaxRowEntries && threadIdx.x < row.n_entries) {
        const Entry &en = v.entries[row.entry0 + threadIdx.x];
        ents[threadIdx.x].p2p_intra = en.p2p_intra;
        ents[threadIdx.x].p2p_inter = en.p2p_inter;
        ents[threadIdx.x].m = en.m;
        ents[threadIdx.x].rel_fits32 = en.rel_bound < ((int64_t)1 << 32) ? 1 : 0;
    }
    if (kJit)
        for (int k = threadIdx.x; k < v.tc.n_jitter * PP; k += blockDim.x) {
            const int p = k / PP, d = k - p * PP;
            jit_f_s[k] = (T)v.raw.jit_f[p * v.tc.jitter_stages + d];
            jit_b_s[k] = (T)v.raw.jit_b[p * v.tc.jitter_stages + d];
        }
    const JitterTab<PP, T, kJit> jt{jit_f_s, jit_b_s, v.tc.n_jitter - 1};
    bool staged = false;
    const int dt_first = row.n_entries - plan.n_dt_staged;      // first entry whose bucket-lane table is staged
    if (use32) {
        const uint32_t pbytes = (uint32_t)(plan.n_entries_staged * lp * sizeof(uint2));
        const uint32_t bbytes = plan.binom_staged ? (uint32_t)(binom_words * sizeof(int64_t)) : 0u;
        const uint32_t dbytes = (uint32_t)(plan.n_dt_staged * v.tab_words32 * sizeof(uint32_t));
        const uint32_t *dt_g = v.dt32 ? v.dt32 + (int64_t)(row.entry0 + dt_first) * v.tab_words32 : nullptr;
        const StageCopy cp[kMaxCopies] = {{dsm, v.pfb32 + (int64_t)row.entry0 * lp, pbytes},
                                          {dsm + plan.off_binom, v.binom, bbytes},
                                          {dsm + plan.off_dt, dt_g, dbytes}, {nullptr, nullptr, 0u}};
        if (pbytes + bbytes + dbytes > 0) staged = stage_tables(&bar, cp, v.status, v.stage_polls);
        else __syncthreads();
    } else if (plan.n_entries_staged > 0 || plan.tables_staged || plan.n_dt_staged > 0 || plan.binom_staged) {
        const uint32_t pbytes = (uint32_t)(plan.n_entries_staged * lp * sizeof(int64_t));
        const uint32_t tbytes = plan.tables_staged ? (uint32_t)(v.tab_words * sizeof(int64_t)) : 0u;
        const uint32_t dbytes = (uint32_t)(plan.n_dt_staged * v.tab_words * sizeof(int64_t));
        const uint32_t bbytes = plan.binom_staged ? (uint32_t)(binom_words * sizeof(int64_t)) : 0u;
        const int64_t *dt_g = v.dt ? v.dt + (int64_t)(row.entry0 + dt_first) * v.tab_words : nullptr;
        // with per-entry bucket-lane tables the row's NB / TP tables are not needed here
        const StageCopy cp[kMaxCopies] = {{dsm, etf_g, pbytes}, {dsm + plan.off_etb, etb_g, pbytes},
                                          v.dt ? StageCopy{dsm + plan.off_dt, dt_g, dbytes}
                                               : StageCopy{dsm + plan.off_nb, nb_g, tbytes},
                                          v.dt ? StageCopy{dsm + plan.off_binom, v.binom, bbytes}
                                               : StageCopy{dsm + plan.off_tp, tp_g, tbytes}};
        staged = stage_tables(&bar, cp, v.status, v.stage_polls);      // contains the block-wide barriers
    } else {
        __syncthreads();
    }
    const int64_t *binom_p = (staged && plan.binom_staged) ? dsm + plan.off_binom : v.binom;
    const int64_t *etf = (staged && plan.n_entries_staged) ? dsm : etf_g;
    const int64_t *etb = (staged && plan.n_entries_staged) ? dsm + plan.off_etb : etb_g;
    const int64_t *nbt = (staged && plan.tables_staged) ? dsm + plan.off_nb : nb_g;
    const int64_t *tpt = (staged && plan.tables_staged) ? dsm + plan.off_tp : tp_g;

    const int64_t part = p_lo + (int64_t)block_x * kThreadBlock + threadIdx.x;
    if (part >= p_hi) return;
    const int e0 = e_begin + block_y * entries_per_thread;
    const int e1 = min(e_end, e0 + entries_per_thread);

    // ---- decode the partition once (bounds are parked in shared memory) ----------------------
    cs[0][threadIdx.x] = 0; cs[PP][threadIdx.x] = (uint16_t)v.tc.n_layers;
    if (v.sc.partition_mode == 0) {
#pragma unroll
        for (int j = 1; j < PP; ++j) cs[j][threadIdx.x] = (uint16_t)((int64_t)j * v.tc.n_layers / PP);
    } else {
        int64_t r = part;
        int cur = 0;
#pragma unroll
        for (int i = 1; i < PP; ++i) {
            ++cur;
            while (true) {
                const int64_t cnt = binom_p[(v.tc.n_layers - 1 - cur) * v.sc.binom_k + (PP - 1 - i)];
                if (r < cnt) break;
                r -= cnt;
                ++cur;
            }
            cs[i][threadIdx.x] = (uint16_t)cur;
        }
    }

    const int64_t per_entry = row.n_part * n_sched;
    for (int e = e0; e < e1; ++e) {                     // e: entry index inside the row
        int m;
        int64_t p2p_intra, p2p_inter;
        bool rel = sizeof(T) == 8;      // the relative frames' shift must fit the arithmetic width as well
        if (e < kMaxRowEntries) { m = ents[e].m; p2p_intra = ents[e].p2p_intra; p2p_inter = ents[e].p2p_inter; rel = rel || ents[e].rel_fits32; }
        else {
            const Entry &en = v.entries[row.entry0 + e];
            m = en.m; p2p_intra = en.p2p_intra; p2p_inter = en.p2p_inter;
            rel = rel || en.rel_bound < ((int64_t)1 << 32);
        }

        // ---- stage costs and bucket-lane excess (schedule independent) -------------------
        ThreadState<PP, T> st;
        if (use32) {
            // everything of this entry fits 32 bits: packed prefix rows, 32-bit table values
            const uint2 *pr = (staged && plan.n_entries_staged) ? reinterpret_cast<const uint2 *>(dsm) + e * lp
                                                                : v.pfb32 + (int64_t)(row.entry0 + e) * lp;
            const uint32_t *d32 = nullptr;
            if (v.dt32)
                d32 = (staged && e >= dt_first)
                          ? reinterpret_cast<const uint32_t *>(dsm + plan.off_dt) + (e - dt_first) * v.tab_words32
                          : v.dt32 + (int64_t)(row.entry0 + e) * v.tab_words32;
            const uint32_t p_in = (uint32_t)p2p_intra, p_out = (uint32_t)p2p_inter;
            uint2 prev = pr[0];
            int a = 0;
#pragma unroll
            for (int d = 0; d < PP; ++d) {
                const int ee = cs[d + 1][threadIdx.x];
                const uint2 cur = pr[ee];
                const uint32_t send_f = d < PP - 1 ? ((((d + 1) & (period - 1)) == 0) ? p_out : p_in) : 0u;
                const uint32_t send_b = d > 0 ? (((d & (period - 1)) == 0) ? p_out : p_in) : 0u;
                const uint32_t fop = cur.x - prev.x + send_f;
                const uint32_t bop = cur.y - prev.y + send_b;
                uint32_t x = 0;
                if (dp > 1) {
                    const uint32_t val = d32[ee * L1 + a];
                    x = v.tc.overlap ? max(val, bop) - bop : val;
                }
                st.fop[d] = (T)fop; st.bop[d] = (T)bop;
                xs[d][threadIdx.x] = (T)x;
                a = ee; prev = cur;
            }
        } else {
            const int64_t *pf = etf + (int64_t)e * lp;
            const int64_t *pb = etb + (int64_t)e * lp;
            const int64_t *dte = nullptr;
            if (v.dt)
                dte = (staged && e >= dt_first) ? dsm + plan.off_dt + (e - dt_first) * v.tab_words
                                                : v.dt + (int64_t)(row.entry0 + e) * v.tab_words;
            int a = 0;
            int64_t pfa = pf[0], pba = pb[0];
#pragma unroll
            for (int d = 0; d < PP; ++d) {
                const int ee = cs[d + 1][threadIdx.x];
                const int64_t pfe = pf[ee], pbe = pb[ee];
                const int64_t send_f = d < PP - 1 ? ((((d + 1) & (period - 1)) == 0) ? p2p_inter : p2p_intra) : 0;
                const int64_t send_b = d > 0 ? (((d & (period - 1)) == 0) ? p2p_inter : p2p_intra) : 0;
                const int64_t fop = pfe - pfa + send_f;
                const int64_t bop = pbe - pba + send_b;
                int64_t x = 0;
                if (dp > 1) {
                    if (dte) {
                        const int64_t val = dte[ee * L1 + a];
                        x = v.tc.overlap ? val - bop : val;
                    } else {
                        const int64_t *nbe = nbt + (int64_t)ee * L1;
                        const int64_t partial = tpt[(int64_t)ee * L1 + a];
                        const int64_t n_full = nbe[a];
                        if (!v.tc.overlap) {
                            x = n_full * t_full + partial;
                        } else {
                            int64_t dt = -1;
                            if (n_full > 0) {
                                int64_t nb_prev = 0;
                                for (int l = ee - 1; l >= a; --l) {
                                    const int64_t nb_l = nbe[l];
                                    if (nb_l != nb_prev)
                                        dt = max64(dt, (pbe - pb[l]) + (n_full - nb_prev) * t_full + partial);
                                    nb_prev = nb_l;
                                }
                            }
                            if (partial > 0) dt = max64(dt, (pbe - pb[__ldg(&v.next_grad[a])]) + partial);
                            x = dt - bop;
                        }
                    }
                    if (x < 0) x = 0;
                }
                st.fop[d] = (T)fop; st.bop[d] = (T)bop;
                xs[d][threadIdx.x] = (T)x;
                a = ee; pfa = pfe; pba = pbe;
            }
        }

        // ---- the row's schedules -------------------------------------------------------------
        const int64_t local0 = (int64_t)e * per_entry + part * n_sched;
        int64_t res0 = 0, res1 = 0, res2 = 0;      // result per schedule position (scalars: no indexed local array)
        int64_t main_only = -1;            // batch time of the 1F1B main lanes alone, once known
#pragma unroll 1
        for (int sc = 0; sc < n_sched; ++sc) {
            const int64_t local = local0 + sc;
            if (local < lo || local >= hi) continue;
            const int id = (sched_list >> (2 * sc)) & 3;
            // the asynchronous schedule is the 1F1B main lane without the gradient buckets
            const bool with_buckets = id != 2;
            int64_t res_sc;
            if (id == 2 && main_only >= 0) {
                res_sc = main_only;
            } else {
                T free_at[PP];
                // (with one micro-batch every stage runs its forward, then its backward item: the GPipe order)
                if (id == 0 || (m == 1 && !kJit)) {
                    if (kJit || !rel) run_gpipe<PP, T, kJit>(st, m, free_at, jt);
                    else run_gpipe_rel<PP, T>(st, m, free_at);
                } else {
                    if (kJit) run_1f1b<PP, T, kJit>(st, m, free_at, jt);
                    else if (!rel || m < PP) run_1f1b_compact<PP, T>(st, m, free_at);
                    else run_1f1b_rel<PP, T>(st, m, free_at);
                }
                T batch = 0;
                if (with_buckets) {
#pragma unroll
                    for (int d = 0; d < PP; ++d) batch = vmax(batch, (T)(free_at[d] + xs[d][threadIdx.x]));
                }
                if (id == 2 || (id == 1 && sc + 1 < n_sched)) {      // an asynchronous twin follows (or this is it)
                    T plain = 0;
#pragma unroll
                    for (int d = 0; d < PP; ++d) plain = vmax(plain, free_at[d]);
                    main_only = (int64_t)plain;
                    if (id == 2) batch = plain;
                }
                res_sc = (int64_t)batch;
            }
            if (sc == 0) res0 = res_sc; else if (sc == 1) res1 = res_sc; else res2 = res_sc;
            if (kBusy) {
                int64_t *bo = busy_out + (row.offset + local - first) * v.sc.pp_max;
#pragma unroll
                for (int d = 0; d < PP; ++d)
                    bo[d] = (int64_t)m * ((int64_t)st.fop[d] + (int64_t)st.bop[d]) +
                            (with_buckets ? (int64_t)xs[d][threadIdx.x] : 0) +
                            (kJit ? __ldg(&v.jsum[(int64_t)(row.entry0 + e) * DISTSIM_MAX_PP + d]) : 0);
                for (int d = PP; d < v.sc.pp_max; ++d) bo[d] = 0;
            }
        }
        // results of the two schedules are neighbours in the output: one 16-byte store if aligned
        const int64_t out0 = row.offset + local0 - first;
        if (n_sched == 2 && local0 >= lo && local0 + 1 < hi && !(reinterpret_cast<uintptr_t>(batch_out + out0) & 15)) {
            *reinterpret_cast<longlong2 *>(batch_out + out0) = make_longlong2(res0, res1);
        } else {
            if (local0 >= lo && local0 < hi) batch_out[out0] = res0;
            if (n_sched > 1 && local0 + 1 >= lo && local0 + 1 < hi) batch_out[out0 + 1] = res1;
            if (n_sched > 2 && local0 + 2 >= lo && local0 + 2 < hi) batch_out[out0 + 2] = res2;
        }
    }
}

}  // namespace distsim
