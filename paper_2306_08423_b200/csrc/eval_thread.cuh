// One stage partition per thread: the evaluation kernel for rows with many partitions and
// pp <= 16.
//
// A thread owns one stage partition of the row and walks the row's entries (micro-batch
// counts) and both schedules with it, so the partition is decoded once and the stage costs once
// per entry.  All per-stage state of the pipeline recurrence - forward/backward item cost,
// device-free time, latest forward end - lives in registers (the stage loops are fully
// unrolled, pp is a template parameter), so a recurrence cell is exactly one 64-bit max and one
// 64-bit add with no memory traffic and no shuffles, and every lane does useful work in every
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
#pragma once

#include "recurrence.cuh"
#include "smem_stage.cuh"

namespace distsim {

constexpr int kThreadBlock = 128;

// Tunables (overridable at compile time for experiments).
#ifndef DS_MINBLOCKS_WIDE
#define DS_MINBLOCKS_WIDE 3       // resident blocks per SM asked for when pp == 16
#endif
#ifndef DS_MINBLOCKS_NARROW
#define DS_MINBLOCKS_NARROW 4     // ... when pp <= 8
#endif
#ifndef DS_UNROLL_MAIN
#define DS_UNROLL_MAIN 1          // unroll factor of the steady-state wave loops
#endif
#ifndef DS_ROLLED_TRIANGLES
#define DS_ROLLED_TRIANGLES 0     // 1: warm-up / drain waves as predicated rolled loops
#endif
#define DS_PRAGMA(x) _Pragma(#x)
#define DS_UNROLL(n) DS_PRAGMA(unroll n)

template <int PP>
struct ThreadState {
    int64_t fop[PP], bop[PP];
};

// GPipe: returns main-lane end of every stage in free_at.
template <int PP>
__device__ __forceinline__ void run_gpipe(const ThreadState<PP> &c, int m, int64_t (&free_at)[PP])
{
#pragma unroll
    for (int d = 0; d < PP; ++d) free_at[d] = 0;
DS_UNROLL(DS_UNROLL_MAIN)
    for (int j = 0; j < m; ++j) {
        int64_t t = free_at[0] + c.fop[0];
        free_at[0] = t;
#pragma unroll
        for (int d = 1; d < PP; ++d) { t = max64(t, free_at[d]) + c.fop[d]; free_at[d] = t; }
    }
DS_UNROLL(DS_UNROLL_MAIN)
    for (int j = 0; j < m; ++j) {
        int64_t t = free_at[PP - 1] + c.bop[PP - 1];
        free_at[PP - 1] = t;
#pragma unroll
        for (int d = PP - 2; d >= 0; --d) { t = max64(t, free_at[d]) + c.bop[d]; free_at[d] = t; }
    }
}

// One 1F1B backward wave in which the stages d >= D0 also run a forward item (D0 may be PP).
template <int PP, int D0>
__device__ __forceinline__ void wave_1f1b(const ThreadState<PP> &c, int64_t (&free_at)[PP], int64_t (&last_f)[PP])
{
    int64_t t = 0;
#pragma unroll
    for (int d = PP - 1; d >= 0; --d) {
        t = (d == PP - 1 ? free_at[d] : max64(t, free_at[d])) + c.bop[d];
        free_at[d] = t;
        if (d >= D0) {
            const int64_t f = (d == 0 ? free_at[0] : max64(last_f[d > 0 ? d - 1 : 0], free_at[d])) + c.fop[d];
            free_at[d] = f;
            last_f[d] = f;
        }
    }
}

// Runs the last waves, in which fewer and fewer stages still have a forward item: with K waves
// to go, the stages with pp - d < K do (statically unrolled over K = KMAX .. 1).
template <int PP, int K>
struct TailWaves {
    static __device__ __forceinline__ void run(const ThreadState<PP> &c, int m, int64_t (&free_at)[PP], int64_t (&last_f)[PP])
    {
        // stage d runs a forward item in this wave iff pp - d < K, i.e. d >= PP - K + 1
        if (K <= m) wave_1f1b<PP, PP - K + 1>(c, free_at, last_f);
        TailWaves<PP, K - 1>::run(c, m, free_at, last_f);
    }
};
template <int PP>
struct TailWaves<PP, 0> {
    static __device__ __forceinline__ void run(const ThreadState<PP> &, int, int64_t (&)[PP], int64_t (&)[PP]) {}
};

// Warm-up forward wave J over stages 0 .. PP-1-J.
template <int PP, int J>
struct WarmWaves {
    static __device__ __forceinline__ void run(const ThreadState<PP> &c, int m, int64_t (&free_at)[PP], int64_t (&last_f)[PP])
    {
        if (J < m) {
            int64_t t = free_at[0] + c.fop[0];
            free_at[0] = t; last_f[0] = t;
#pragma unroll
            for (int d = 1; d < PP - J; ++d) { t = max64(t, free_at[d]) + c.fop[d]; free_at[d] = t; last_f[d] = t; }
        }
        WarmWaves<PP, J + 1>::run(c, m, free_at, last_f);
    }
};
template <int PP>
struct WarmWaves<PP, PP> {
    static __device__ __forceinline__ void run(const ThreadState<PP> &, int, int64_t (&)[PP], int64_t (&)[PP]) {}
};

template <int PP>
__device__ __forceinline__ void run_1f1b(const ThreadState<PP> &c, int m, int64_t (&free_at)[PP])
{
    int64_t last_f[PP];
#pragma unroll
    for (int d = 0; d < PP; ++d) { free_at[d] = 0; last_f[d] = 0; }
#if DS_ROLLED_TRIANGLES
    // warm-up wave j covers the stages d < PP - j
    for (int j = 0; j < min(PP, m); ++j) {
        int64_t t = 0;
#pragma unroll
        for (int d = 0; d < PP; ++d)
            if (d < PP - j) { t = (d == 0 ? free_at[0] : max64(t, free_at[d])) + c.fop[d]; free_at[d] = t; last_f[d] = t; }
    }
DS_UNROLL(DS_UNROLL_MAIN)
    for (int i = 0; i < m - PP; ++i) wave_1f1b<PP, 0>(c, free_at, last_f);
    // with k waves to go, stage d still runs a forward item iff PP - d < k
    for (int k = min(PP, m); k >= 1; --k) {
        int64_t t = 0;
#pragma unroll
        for (int d = PP - 1; d >= 0; --d) {
            t = (d == PP - 1 ? free_at[d] : max64(t, free_at[d])) + c.bop[d];
            free_at[d] = t;
            if (PP - d < k) {
                const int64_t f = (d == 0 ? free_at[0] : max64(last_f[d > 0 ? d - 1 : 0], free_at[d])) + c.fop[d];
                free_at[d] = f; last_f[d] = f;
            }
        }
    }
#else
    WarmWaves<PP, 0>::run(c, m, free_at, last_f);
    // waves i = 0 .. m-PP-1: every stage still has a forward item to pair with its backward
DS_UNROLL(DS_UNROLL_MAIN)
    for (int i = 0; i < m - PP; ++i) wave_1f1b<PP, 0>(c, free_at, last_f);
    // the last min(PP, m) waves
    TailWaves<PP, PP>::run(c, m, free_at, last_f);
#endif
}

// Shared-memory plan of a block (offsets in int64 words from the dynamic shared base).
struct ThreadKernelSmem {
    int32_t n_entries_staged;   // 0: read prefix rows from global
    int32_t tables_staged;      // 1: NB / TP tables of the row are in shared memory
    int32_t off_etb, off_nb, off_tp;
};

template <int PP, bool kBusy>
__global__ void __launch_bounds__(kThreadBlock, (PP >= 16 ? DS_MINBLOCKS_WIDE : DS_MINBLOCKS_NARROW))
eval_thread_kernel(DeviceView v, int row_index, int64_t lo, int64_t hi, int64_t first,
                   int e_begin, int e_end, int entries_per_thread, int64_t p_lo, int64_t p_hi,
                   int64_t *__restrict__ batch_out, int64_t *__restrict__ busy_out,
                   ThreadKernelSmem plan, int tab_words)
{
    extern __shared__ __align__(16) int64_t dsm[];
    __shared__ __align__(8) uint64_t bar;
    __shared__ int64_t xs[PP][kThreadBlock];          // per thread, per stage: bucket-lane excess X
    __shared__ uint16_t cs[PP + 1][kThreadBlock];      // per thread: stage bounds c_0 .. c_PP
    const Row &row = v.rows[row_index];
    const int lp = v.tc.lp;
    const int L1 = v.tc.n_layers + 1;

    // ---- stage the row's prefix rows and bucket tables ---------------------------------
    const int64_t *etf_g = v.etf + (int64_t)row.entry0 * lp;
    const int64_t *etb_g = v.etb + (int64_t)row.entry0 * lp;
    const int64_t *nb_g = v.nb + row.row_tab_off;
    const int64_t *tp_g = v.tp + row.row_tab_off;
    bool staged = false;
    if (plan.n_entries_staged > 0 || plan.tables_staged) {
        const uint32_t pbytes = (uint32_t)(plan.n_entries_staged * lp * sizeof(int64_t));
        const uint32_t tbytes = plan.tables_staged ? (uint32_t)(tab_words * sizeof(int64_t)) : 0u;
        const StageCopy cp[kMaxCopies] = {{dsm, etf_g, pbytes}, {dsm + plan.off_etb, etb_g, pbytes},
                                          {dsm + plan.off_nb, nb_g, tbytes}, {dsm + plan.off_tp, tp_g, tbytes}};
        staged = stage_tables(&bar, cp, v.status);
    }
    const int64_t *etf = (staged && plan.n_entries_staged) ? dsm : etf_g;
    const int64_t *etb = (staged && plan.n_entries_staged) ? dsm + plan.off_etb : etb_g;
    const int64_t *nbt = (staged && plan.tables_staged) ? dsm + plan.off_nb : nb_g;
    const int64_t *tpt = (staged && plan.tables_staged) ? dsm + plan.off_tp : tp_g;

    const int64_t part = p_lo + (int64_t)blockIdx.x * kThreadBlock + threadIdx.x;
    if (part >= p_hi) return;
    const int e0 = e_begin + (int)blockIdx.y * entries_per_thread;
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
                const int64_t cnt = __ldg(&v.binom[(int64_t)(v.tc.n_layers - 1 - cur) * v.sc.binom_k + (PP - 1 - i)]);
                if (r < cnt) break;
                r -= cnt;
                ++cur;
            }
            cs[i][threadIdx.x] = (uint16_t)cur;
        }
    }

    const int64_t per_entry = row.n_part * row.n_sched;
    for (int e = e0; e < e1; ++e) {                     // e: entry index inside the row
        const Entry &en = v.entries[row.entry0 + e];
        const int64_t *pf = etf + (int64_t)e * lp;
        const int64_t *pb = etb + (int64_t)e * lp;
        const int m = en.m;
        ThreadState<PP> st;
#pragma unroll
        for (int d = 0; d < PP; ++d) {
            const int a = cs[d][threadIdx.x], ee = cs[d + 1][threadIdx.x];
            st.fop[d] = pf[ee] - pf[a] + (d < PP - 1 ? p2p_cost(row, en, d) : 0);
            st.bop[d] = pb[ee] - pb[a] + (d > 0 ? p2p_cost(row, en, d - 1) : 0);
        }
        // ---- bucket-lane excess per stage (schedule independent) ------------------------
#pragma unroll
        for (int d = 0; d < PP; ++d) {
            int64_t x = 0;
            if (row.dp > 1) {
                const int a = cs[d][threadIdx.x], ee = cs[d + 1][threadIdx.x];
                const int64_t *nbe = nbt + (int64_t)ee * L1;
                const int64_t partial = tpt[(int64_t)ee * L1 + a];
                const int64_t n_full = nbe[a];
                if (!v.tc.overlap) {
                    x = n_full * row.t_full + partial;
                } else {
                    int64_t dt = -1;                     // latest bucket-lane end relative to the last backward start
                    const int64_t pbe = pb[ee];
                    if (n_full > 0) {
                        int64_t nb_prev = 0;
                        for (int l = ee - 1; l >= a; --l) {
                            const int64_t nb_l = nbe[l];
                            if (nb_l != nb_prev)
                                dt = max64(dt, (pbe - pb[l]) + (n_full - nb_prev) * row.t_full + partial);
                            nb_prev = nb_l;
                        }
                    }
                    if (partial > 0) dt = max64(dt, (pbe - pb[__ldg(&v.next_grad[a])]) + partial);
                    x = dt - st.bop[d];
                    if (x < 0) x = 0;
                }
            }
            xs[d][threadIdx.x] = x;
        }

        for (int sc = 0; sc < row.n_sched; ++sc) {
            const int64_t local = (int64_t)e * per_entry + part * row.n_sched + sc;
            if (local < lo || local >= hi) continue;
            int64_t free_at[PP];
            if (row.sched0 + sc == 0) run_gpipe<PP>(st, m, free_at);
            else run_1f1b<PP>(st, m, free_at);
            int64_t batch = 0;
#pragma unroll
            for (int d = 0; d < PP; ++d) batch = max64(batch, free_at[d] + xs[d][threadIdx.x]);
            const int64_t out = row.offset + local - first;
            batch_out[out] = batch;
            if (kBusy) {
                int64_t *bo = busy_out + out * v.sc.pp_max;
#pragma unroll
                for (int d = 0; d < PP; ++d) bo[d] = (int64_t)m * (st.fop[d] + st.bop[d]) + xs[d][threadIdx.x];
                for (int d = PP; d < v.sc.pp_max; ++d) bo[d] = 0;
            }
        }
    }
}

}  // namespace distsim
