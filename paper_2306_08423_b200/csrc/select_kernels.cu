// Selection kernels: best candidate (argmin) and the k fastest candidates (top-k) of an array
// of batch times.  Ordering is always by (batch time, index): ties go to the smaller index.
#include "engine.h"

namespace distsim {

namespace {

using u64 = unsigned long long;
constexpr int kSelThreads = 256;

__device__ __forceinline__ u64 warp_min_u64(u64 x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const u64 y = __shfl_xor_sync(0xffffffffu, x, o);
        x = y < x ? y : x;
    }
    return x;
}

__device__ __forceinline__ u64 block_min_u64(u64 x)
{
    __shared__ u64 part[kSelThreads / 32];
    x = warp_min_u64(x);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = x;
    __syncthreads();
    if (threadIdx.x < 32) {
        x = threadIdx.x < kSelThreads / 32 ? part[threadIdx.x] : ~0ull;
        x = warp_min_u64(x);
    }
    __syncthreads();
    return x;   // valid on thread 0
}

// Packed argmin: key = (time << idx_bits) | index fits 64 bits, one atomicMin per block.
__global__ void __launch_bounds__(kSelThreads)
argmin_packed_kernel(const int64_t *__restrict__ t, int64_t n, int idx_bits, u64 *key)
{
    u64 best = ~0ull;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const u64 k = ((u64)t[i] << idx_bits) | (u64)i;
        best = k < best ? k : best;
    }
    best = block_min_u64(best);
    if (threadIdx.x == 0 && best != ~0ull) atomicMin(key, best);
}

// Two-pass argmin for times too wide to pack: first the smallest time, then the smallest index
// among the elements that have it.
__global__ void __launch_bounds__(kSelThreads)
argmin_time_kernel(const int64_t *__restrict__ t, int64_t n, u64 *key)
{
    u64 best = ~0ull;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const u64 k = (u64)t[i];
        best = k < best ? k : best;
    }
    best = block_min_u64(best);
    if (threadIdx.x == 0 && best != ~0ull) atomicMin(key, best);
}
__global__ void __launch_bounds__(kSelThreads)
argmin_index_kernel(const int64_t *__restrict__ t, int64_t n, u64 *key)
{
    const u64 tmin = key[0];
    u64 best = ~0ull;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        if ((u64)t[i] == tmin) { best = (u64)i < best ? (u64)i : best; }
    best = block_min_u64(best);
    if (threadIdx.x == 0 && best != ~0ull) atomicMin(key + 1, best);
}
__global__ void argmin_unpack_kernel(const u64 *key, int idx_bits, int packed, int64_t *result)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    if (packed) {
        result[0] = (int64_t)(key[0] >> idx_bits);
        result[1] = (int64_t)(key[0] & ((1ull << idx_bits) - 1ull));
    } else {
        result[0] = (int64_t)key[0];
        result[1] = (int64_t)key[1];
    }
}

// ---- top-k ---------------------------------------------------------------------------------
// Radix select with 11-bit digits, most significant first: first on the time, then (only if the
// threshold time is shared by more elements than are still wanted) on the index among the
// elements that have it.  `rank` is the rank still to resolve inside the current group.
// After the first pass only the elements whose top digit does not exceed the chosen bin can
// still matter; they are copied to a compact (time, index) buffer and the remaining passes read
// that buffer instead of the whole array (if they fit; otherwise everything stays on the array).
constexpr int kRadixBits = 11;
constexpr int kBins = 1 << kRadixBits;
struct SelState {
    u64 tprefix, tmask, rank, iprefix, imask, blocks_done, cursor, skip_index;
    u64 use_compact, cn;         // remaining passes read the compact buffer of cn pairs
    u64 stride;                  // > 1: the passes read every stride-th element of the array (sampling phase);
                                 // with kSampleGathered set, the first pass has copied those elements to the
                                 // head of the compact buffer and the later passes read them there
    u64 k;                       // elements wanted
    u64 threshold;               // sampled selection: a time that at least k elements do not exceed
    u64 tmin;                    // sampled selection: smallest time of the array
    u64 small;                   // sampled selection: the candidates fit one sort (n_cand of them)
    u64 n_cand;
};

// The source a pass reads: the array itself (index = position) or the compact buffer.
constexpr u64 kSampleGathered = 1ull << 63;
struct SelSource { const int64_t *t; const int64_t *idx; int64_t n; int64_t stride; };
__device__ __forceinline__ SelSource sel_source(const SelState *st, const int64_t *batch, int64_t count,
                                                const SelectScratch &sc)
{
    if (st->use_compact) return SelSource{sc.comp_time, sc.comp_idx, (int64_t)st->cn, 1};
    if (st->stride > 1) {
        const int64_t stride = (int64_t)(st->stride & ~kSampleGathered), n = (count + stride - 1) / stride;
        if (st->stride & kSampleGathered) return SelSource{sc.comp_time, nullptr, n, 1};
        return SelSource{batch, nullptr, n, stride};
    }
    return SelSource{batch, nullptr, count, 1};
}

// Run by one whole block once a histogram is complete: finds the bin that holds rank `rank`.
// On thread 0 (only) the results are valid after the call: the bin, the number of elements in
// the bins before it and in it.  Ends with a block-wide barrier.
struct PickedBin { int bin; u64 before, in_bin; };
__device__ __forceinline__ PickedBin find_bin(u64 rank, const u64 *hist, u64 *partial /* shared, [kSelThreads] */)
{
    __threadfence();
    constexpr int kPer = kBins / kSelThreads;
    u64 mine = 0;
    for (int k = 0; k < kPer; ++k) mine += *((volatile const u64 *)&hist[threadIdx.x * kPer + k]);
    partial[threadIdx.x] = mine;
    __syncthreads();
    // chunk (a thread's kPer bins) that holds the wanted rank: exclusive scan of the chunk sums by
    // the first warp, each lane taking kSelThreads / 32 consecutive chunks
    __shared__ int chunk_s;
    __shared__ u64 cum_s;
    if (threadIdx.x < 32) {
        constexpr int kEach = kSelThreads / 32;
        u64 sum = 0;
        for (int c = 0; c < kEach; ++c) sum += partial[threadIdx.x * kEach + c];
        u64 incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const u64 up = __shfl_up_sync(0xffffffffu, incl, o);
            if ((int)threadIdx.x >= o) incl += up;
        }
        const u64 total = __shfl_sync(0xffffffffu, incl, 31);
        const bool mine_has = rank >= incl - sum && rank < incl;
        const unsigned who = __ballot_sync(0xffffffffu, mine_has);
        if (who == 0 && threadIdx.x == 0) { chunk_s = kSelThreads - 1; cum_s = total - partial[kSelThreads - 1]; }   // rank beyond the data
        if (mine_has) {
            u64 cum = incl - sum;
            int chunk = threadIdx.x * kEach + kEach - 1;
            for (int c = 0; c < kEach; ++c) {
                const u64 pc = partial[threadIdx.x * kEach + c];
                if (rank < cum + pc) { chunk = threadIdx.x * kEach + c; break; }
                cum += pc;
            }
            chunk_s = chunk; cum_s = cum;
        }
    }
    __syncthreads();
    PickedBin p{0, 0, 0};
    if (threadIdx.x == 0) {
        u64 cum = cum_s;
        const int chunk = chunk_s;
        p.bin = chunk * kPer + kPer - 1;
        for (int k = 0; k < kPer; ++k) {
            const u64 h = *((volatile const u64 *)&hist[chunk * kPer + k]);
            if (rank < cum + h) { p.bin = chunk * kPer + k; p.in_bin = h; break; }
            cum += h;
        }
        p.before = cum;
    }
    return p;
}

// The pick step of a radix pass: narrows the prefix / mask to the bin that holds the wanted
// rank and clears the histogram for the next digit.
template <bool kIndexPhase>
__device__ __forceinline__ void pick_bin(SelState *st, u64 *hist, u64 *partial /* shared, [kSelThreads] */, int shift,
                                         unsigned dmask, bool last_time_pass)
{
    const u64 tprefix = st->tprefix, tmask = st->tmask, iprefix = st->iprefix, imask = st->imask;
    const u64 rank = st->rank;
    const PickedBin p = find_bin(rank, hist, partial);
    if (threadIdx.x == 0) {
        const u64 cum = p.before, in_bin = p.in_bin;
        const int bin = p.bin;
        st->rank = rank - cum;
        if (!kIndexPhase && last_time_pass && in_bin == rank - cum + 1) {
            // the elements equal to the threshold time are exactly the ones still needed
            st->skip_index = 1; st->iprefix = ~0ull;
        }
        if (kIndexPhase) { st->iprefix = iprefix | ((u64)bin << shift); st->imask = imask | ((u64)dmask << shift); }
        else { st->tprefix = tprefix | ((u64)bin << shift); st->tmask = tmask | ((u64)dmask << shift); }
        st->blocks_done = 0;
        // everything at or below the chosen bin may still matter: this many pairs to compact
        // (once the compact buffer is in use, cn is its size and must stay)
        if (!st->use_compact) st->cn = cum + in_bin;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kBins; i += blockDim.x) hist[i] = 0;
}

template <bool kIndexPhase>
__global__ void __launch_bounds__(kSelThreads)
radix_pass_kernel(const int64_t *__restrict__ batch, int64_t count, SelectScratch sc, int shift, int width,
                  bool last_time_pass)
{
    __shared__ unsigned int sh[kBins];
    __shared__ u64 partial[kSelThreads];
    __shared__ bool last;
    SelState *st = reinterpret_cast<SelState *>(sc.sel_state);
    u64 *hist = sc.hist;
    // no ties at the threshold time: every element equal to it is wanted, no index pass needed
    if (kIndexPhase && st->skip_index) return;
    for (int i = threadIdx.x; i < kBins; i += blockDim.x) sh[i] = 0;
    __syncthreads();
    const SelSource src = sel_source(st, batch, count, sc);
    const u64 tprefix = st->tprefix, tmask = st->tmask, iprefix = st->iprefix, imask = st->imask;
    const unsigned dmask = (1u << width) - 1u;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < src.n; i += (int64_t)gridDim.x * blockDim.x) {
        const u64 x = (u64)src.t[i * src.stride];
        // the first pass over a strided sample leaves a dense copy for the passes that follow
        if (!kIndexPhase && src.stride > 1 && src.n <= sc.comp_cap) sc.comp_time[i] = (int64_t)x;
        if ((x & tmask) != tprefix) continue;
        if (kIndexPhase) {
            const u64 id = src.idx ? (u64)src.idx[i] : (u64)i;
            if ((id & imask) != iprefix) continue;
            atomicAdd(&sh[(unsigned)(id >> shift) & dmask], 1u);
        } else {
            atomicAdd(&sh[(unsigned)(x >> shift) & dmask], 1u);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kBins; i += blockDim.x) if (sh[i]) atomicAdd(&hist[i], (u64)sh[i]);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last = atomicAdd(&st->blocks_done, 1ull) == (u64)gridDim.x - 1;
    __syncthreads();
    if (!last) return;
    pick_bin<kIndexPhase>(st, hist, partial, shift, dmask, last_time_pass);
    if (!kIndexPhase && threadIdx.x == 0 && src.stride > 1 && src.n <= sc.comp_cap) st->stride |= kSampleGathered;
}

__global__ void sel_init_kernel(SelState *st, u64 *hist, int k, int64_t stride, u64 *key /* nullable: [2], set to all ones */)
{
    for (int i = threadIdx.x; i < kBins; i += blockDim.x) hist[i] = 0;
    if (key && threadIdx.x < 2) key[threadIdx.x] = ~0ull;
    if (threadIdx.x == 0) {
        SelState z{};
        z.rank = (u64)(k - 1); z.k = (u64)k; z.stride = (u64)stride; z.tmin = ~0ull;
        *st = z;
    }
}

// The one pass over a long array (after the sampling phase has left, in tprefix, a time that at
// least k elements do not exceed): the minimum of the packed (time, position) key, and every
// element up to the threshold copied to the compact buffer.  The last block to finish resets the
// selection state for the selection proper, which then reads the compact buffer - or, should
// the elements not fit it (masses of ties), the array itself.
__global__ void __launch_bounds__(kSelThreads)
scan_select_kernel(const int64_t *__restrict__ batch, int64_t count, SelectScratch sc, int idx_bits, int want_min,
                   int want_compact, int low_bits /* time bits the sampling passes left open */)
{
    __shared__ bool last;
    // Elements up to the threshold are few (about k times the sampling stride out of the whole
    // array, a few hundred per block), but one counter in global memory cannot take an atomic
    // for each: a block collects its own in shared memory and takes one range of the compact
    // buffer at its end; what does not fit the block's buffer goes there directly.
    constexpr int kHeld = 512;
    __shared__ int64_t held_t[kHeld], held_i[kHeld];
    __shared__ unsigned int n_held;
    __shared__ u64 held_base;
    if (threadIdx.x == 0) n_held = 0;
    __syncthreads();
    SelState *st = reinterpret_cast<SelState *>(sc.sel_state);
    const u64 threshold = want_compact ? (st->tprefix | ((1ull << low_bits) - 1ull)) : 0;
    // A thread meets its elements in ascending position, so "strictly smaller" keeps the first
    // of equal times: (xmin, imin) is the thread's smallest (time, position) pair.
    u64 xmin = ~0ull;
    int64_t imin = 0;
    auto consider = [&](u64 x, int64_t i) {
        if (x < xmin) { xmin = x; imin = i; }
        if (want_compact && x <= threshold) {
            const unsigned int h = atomicAdd(&n_held, 1u);
            if (h < (unsigned)kHeld) { held_t[h] = (int64_t)x; held_i[h] = i; }
            else {
                const u64 pos = atomicAdd(&st->cursor, 1ull);
                if (pos < (u64)sc.comp_cap) { sc.comp_time[pos] = (int64_t)x; sc.comp_idx[pos] = i; }
            }
        }
    };
    // 16-byte loads of pairs (the array from its first 16-byte boundary on), four of them in
    // flight per thread; the element before that boundary and an odd last one go to one thread
    const int64_t head = (count > 0 && (reinterpret_cast<uintptr_t>(batch) & 15)) ? 1 : 0;
    const int64_t n_pairs = (count - head) >> 1;
    const bool edges = blockIdx.x == 0 && threadIdx.x == 0;
    if (edges && head) consider((u64)batch[0], 0);
    const longlong2 *pairs = reinterpret_cast<const longlong2 *>(batch + head);
    constexpr int kUnroll = 4;
    const int64_t step = (int64_t)gridDim.x * blockDim.x;
    for (int64_t p0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p0 < n_pairs; p0 += step * kUnroll) {
        longlong2 x[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int64_t p = p0 + u * step;
            if (p < n_pairs) x[u] = __ldcs(pairs + p);
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int64_t p = p0 + u * step;
            if (p >= n_pairs) break;
            consider((u64)x[u].x, head + 2 * p);
            consider((u64)x[u].y, head + 2 * p + 1);
        }
    }
    if (edges && head + 2 * n_pairs < count) consider((u64)batch[count - 1], count - 1);
    if (want_min) {
        u64 best = xmin != ~0ull ? (xmin << idx_bits) | (u64)imin : ~0ull;
        best = block_min_u64(best);
        if (threadIdx.x == 0 && best != ~0ull) atomicMin(sc.key, best);
    }
    if (!want_compact) return;
    __syncthreads();
    const unsigned int n_mine = n_held < (unsigned)kHeld ? n_held : (unsigned)kHeld;
    if (threadIdx.x == 0 && n_mine) held_base = atomicAdd(&st->cursor, (u64)n_mine);
    __syncthreads();
    for (unsigned int h = threadIdx.x; h < n_mine; h += blockDim.x)
        if (held_base + h < (u64)sc.comp_cap) { sc.comp_time[held_base + h] = held_t[h]; sc.comp_idx[held_base + h] = held_i[h]; }
    xmin = block_min_u64(xmin);
    if (threadIdx.x == 0 && xmin != ~0ull) atomicMin(&st->tmin, xmin);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last = atomicAdd(&st->blocks_done, 1ull) == (u64)gridDim.x - 1;
    __syncthreads();
    if (last && threadIdx.x == 0) {
        const u64 n = *((volatile u64 *)&st->cursor);
        st->use_compact = n <= (u64)sc.comp_cap ? 1 : 0;
        st->cn = n;
        st->threshold = threshold;
        st->tprefix = 0; st->tmask = 0; st->iprefix = 0; st->imask = 0; st->skip_index = 0;
        st->rank = st->k - 1; st->stride = 0; st->cursor = 0; st->blocks_done = 0;
    }
}

// After the first time pass: copies the elements whose time does not exceed the chosen top
// digit into the compact buffer, if they fit; the last block then switches the source over.
__global__ void __launch_bounds__(kSelThreads)
compact_kernel(const int64_t *__restrict__ batch, int64_t count, SelectScratch sc, int shift)
{
    __shared__ bool last;
    SelState *st = reinterpret_cast<SelState *>(sc.sel_state);
    const u64 cn = st->cn;
    if (cn > (u64)sc.comp_cap) return;              // does not fit: later passes keep reading the array
    const u64 limit = st->tprefix >> shift;         // the chosen top digit
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x) {
        const u64 x = (u64)batch[i];
        if ((x >> shift) <= limit) {
            const u64 pos = atomicAdd(&st->cursor, 1ull);
            if (pos < (u64)sc.comp_cap) { sc.comp_time[pos] = (int64_t)x; sc.comp_idx[pos] = i; }
        }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last = atomicAdd(&st->blocks_done, 1ull) == (u64)gridDim.x - 1;
    __syncthreads();
    if (last && threadIdx.x == 0) { st->use_compact = 1; st->cursor = 0; st->blocks_done = 0; }
}

// Collects the elements that are not above the threshold pair (time, index), at most k of them,
// in any order.  only_small: the refined path of the sampled selection - nothing to do unless its
// candidates fit one sort.
__global__ void __launch_bounds__(kSelThreads)
collect_kernel(const int64_t *__restrict__ batch, int64_t count, SelectScratch sc, int k, int only_small)
{
    SelState *st = reinterpret_cast<SelState *>(sc.sel_state);
    if (only_small && !st->small) return;
    const SelSource src = sel_source(st, batch, count, sc);
    const u64 T = st->tprefix, I = st->iprefix;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < src.n; i += (int64_t)gridDim.x * blockDim.x) {
        const u64 x = (u64)src.t[i];
        const u64 id = src.idx ? (u64)src.idx[i] : (u64)i;
        if (x < T || (x == T && id <= I)) {
            const u64 pos = atomicAdd(&st->cursor, 1ull);
            if (pos < (u64)k) { sc.cand_time[pos] = (int64_t)x; sc.cand_idx[pos] = (int64_t)id; }
        }
    }
}

// Bitonic sort of np2 (a power of two) (time, index) pairs in shared memory, ascending, by the
// whole block.
__device__ __forceinline__ void bitonic_sort_pairs(int64_t *st, int64_t *si, int np2)
{
    for (int size = 2; size <= np2; size <<= 1)
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            for (int i = threadIdx.x; i < np2 / 2; i += blockDim.x) {
                const int a = 2 * i - (i & (stride - 1));
                const int b = a + stride;
                const bool up = (a & size) == 0;
                const bool gt = st[a] > st[b] || (st[a] == st[b] && si[a] > si[b]);
                if (gt == up) {
                    const int64_t x = st[a]; st[a] = st[b]; st[b] = x;
                    const int64_t y = si[a]; si[a] = si[b]; si[b] = y;
                }
            }
            // a step of stride <= 32 exchanges inside aligned groups of 64 elements, each the work
            // of one warp (comparator i belongs to thread i mod 1024, group to warp i / 32 mod 32)
            const int next = stride > 1 ? stride >> 1 : size;
            if (stride >= 64 || next >= 64) __syncthreads(); else __syncwarp();
        }
}

// The same on packed keys (time << idx_bits | index): half the shared-memory traffic.
__device__ __forceinline__ void bitonic_sort_keys(u64 *key, int np2)
{
    for (int size = 2; size <= np2; size <<= 1)
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            for (int i = threadIdx.x; i < np2 / 2; i += blockDim.x) {
                const int a = 2 * i - (i & (stride - 1));
                const int b = a + stride;
                const bool up = (a & size) == 0;
                const u64 x = key[a], y = key[b];
                if ((x > y) == up) { key[a] = y; key[b] = x; }
            }
            const int next = stride > 1 ? stride >> 1 : size;
            if (stride >= 64 || next >= 64) __syncthreads(); else __syncwarp();
        }
}

// One block sorts up to 4096 (time, index) pairs ascending (bitonic network in shared memory)
// and writes the first k.  Also the whole top-k for arrays of at most 4096 elements.
// state != nullptr: the refined path of the sampled selection - the number of pairs is the
// state's n_cand, and there is nothing to do unless the candidates fit (state->small).
constexpr int kSortMax = 4096;
__global__ void __launch_bounds__(1024)
sort_pairs_kernel(const int64_t *__restrict__ ct, const int64_t *__restrict__ ci, int n_in, int k,
                  int64_t first, int64_t *out_idx, int64_t *out_time, const SelState *state,
                  int idx_bits /* > 0: time and index fit one 64-bit key with this many index bits */)
{
    extern __shared__ __align__(16) unsigned char sm[];
    int64_t *st = reinterpret_cast<int64_t *>(sm);
    int64_t *si = st + kSortMax;
    if (state) {
        if (!state->small) return;
        n_in = (int)state->n_cand;
    }
    int np2 = 64;                        // whole groups of 64 (see the sort's barriers)
    while (np2 < n_in) np2 <<= 1;
    if (idx_bits > 0) {
        u64 *key = reinterpret_cast<u64 *>(sm);
        for (int i = threadIdx.x; i < np2; i += blockDim.x)
            key[i] = i < n_in ? ((u64)ct[i] << idx_bits) | (u64)(ci ? ci[i] : (int64_t)i) : ~0ull;
        __syncthreads();
        bitonic_sort_keys(key, np2);
        for (int i = threadIdx.x; i < k; i += blockDim.x) {
            out_idx[i] = first + (int64_t)(key[i] & ((1ull << idx_bits) - 1ull));
            if (out_time) out_time[i] = (int64_t)(key[i] >> idx_bits);
        }
        return;
    }
    for (int i = threadIdx.x; i < np2; i += blockDim.x) {
        st[i] = i < n_in ? ct[i] : INT64_MAX;
        si[i] = i < n_in ? (ci ? ci[i] : (int64_t)i) : INT64_MAX;
    }
    __syncthreads();
    bitonic_sort_pairs(st, si, np2);
    for (int i = threadIdx.x; i < k; i += blockDim.x) {
        out_idx[i] = first + si[i];
        if (out_time) out_time[i] = st[i];
    }
}

// Sampled selection, after the one pass over the array: the compact buffer holds the cn elements
// between the array's smallest time and the sample's threshold.  One histogram over that range
// (2048 bins of equal width, a power of two) finds a cut that at least k of them do not exceed;
// if those candidates fit one sort (the usual case: about k plus one bin's worth), `small` is
// set and collect + sort finish the selection; otherwise the general kernel below does.
__global__ void __launch_bounds__(kSelThreads)
refine_kernel(SelectScratch sc)
{
    __shared__ unsigned int sh[kBins];
    __shared__ u64 partial[kSelThreads];
    __shared__ bool last;
    SelState *st = reinterpret_cast<SelState *>(sc.sel_state);
    if (!st->use_compact) return;                      // the elements did not fit: `small` stays 0
    const u64 tmin = st->tmin, range = st->threshold - tmin;
    const int shift = range >> kRadixBits ? 64 - __clzll((long long)range) - kRadixBits : 0;     // (range >> shift) < 2048
    for (int i = threadIdx.x; i < kBins; i += blockDim.x) sh[i] = 0;
    __syncthreads();
    const int64_t n = (int64_t)st->cn;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        atomicAdd(&sh[(unsigned)(((u64)sc.comp_time[i] - tmin) >> shift)], 1u);
    __syncthreads();
    for (int i = threadIdx.x; i < kBins; i += blockDim.x) if (sh[i]) atomicAdd(&sc.hist[i], (u64)sh[i]);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last = atomicAdd(&st->blocks_done, 1ull) == (u64)gridDim.x - 1;
    __syncthreads();
    if (!last) return;
    const PickedBin p = find_bin(st->k - 1, sc.hist, partial);
    if (threadIdx.x == 0) {
        // candidates: everything up to the upper edge of the chosen bin, any index
        st->tprefix = tmin + (((u64)p.bin + 1) << shift) - 1;
        st->iprefix = ~0ull;
        st->n_cand = p.before + p.in_bin;
        st->small = p.before + p.in_bin <= (u64)kSortMax ? 1 : 0;
        st->blocks_done = 0; st->cursor = 0;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kBins; i += blockDim.x) sc.hist[i] = 0;
}

// The general selection by one block, for the rare inputs the refined path cannot finish
// (masses of equal times): a radix select over all time digits, then over the index digits among
// the elements with the threshold time, on the compact buffer or, if that overflowed, the array
// itself; then the k winners are sorted.  Slow on long inputs, exact on all.
__global__ void __launch_bounds__(kSelThreads)
general_select_kernel(const int64_t *__restrict__ batch, int64_t count, SelectScratch sc, int k, int tb, int ib,
                      int64_t first, int64_t *out_idx, int64_t *out_time)
{
    extern __shared__ __align__(16) unsigned char sm[];
    int64_t *pt = reinterpret_cast<int64_t *>(sm);          // [kSortMax] winners' times
    int64_t *pi = pt + kSortMax;                            // [kSortMax] winners' indices
    u64 *h = reinterpret_cast<u64 *>(pi + kSortMax);        // [kBins]
    __shared__ u64 partial[kSelThreads];
    __shared__ PickedBin picked;
    __shared__ unsigned int n_won;
    SelState *st = reinterpret_cast<SelState *>(sc.sel_state);
    if (st->small) return;
    const SelSource src = sel_source(st, batch, count, sc);
    u64 tprefix = 0, tmask = 0, iprefix = 0, imask = 0, rank = (u64)(k - 1);
    bool skip_index = false;
    for (int phase = 0; phase < 2; ++phase) {              // 0: time digits, 1: index digits
        const int bits = phase == 0 ? tb : ib;
        if (phase == 1 && skip_index) break;
        for (int shift = ((bits + kRadixBits - 1) / kRadixBits - 1) * kRadixBits; shift >= 0; shift -= kRadixBits) {
            const int width = bits - shift < kRadixBits ? bits - shift : kRadixBits;
            const unsigned dmask = (1u << width) - 1u;
            for (int i = threadIdx.x; i < kBins; i += blockDim.x) h[i] = 0;
            __syncthreads();
            for (int64_t i = threadIdx.x; i < src.n; i += blockDim.x) {
                const u64 x = (u64)src.t[i];
                if ((x & tmask) != tprefix) continue;
                if (phase == 0) { atomicAdd(&h[(unsigned)(x >> shift) & dmask], 1ull); continue; }
                const u64 id = src.idx ? (u64)src.idx[i] : (u64)i;
                if ((id & imask) == iprefix) atomicAdd(&h[(unsigned)(id >> shift) & dmask], 1ull);
            }
            __syncthreads();
            const PickedBin p = find_bin(rank, h, partial);
            if (threadIdx.x == 0) picked = p;
            __syncthreads();
            rank -= picked.before;
            if (phase == 0) {
                tprefix |= (u64)picked.bin << shift; tmask |= (u64)dmask << shift;
                // the elements equal to the threshold time are exactly the ones still needed
                if (shift == 0 && picked.in_bin == rank + 1) skip_index = true;
            } else {
                iprefix |= (u64)picked.bin << shift; imask |= (u64)dmask << shift;
            }
            __syncthreads();
        }
    }
    if (skip_index) iprefix = ~0ull;
    if (threadIdx.x == 0) n_won = 0;
    __syncthreads();
    for (int64_t i = threadIdx.x; i < src.n; i += blockDim.x) {
        const u64 x = (u64)src.t[i];
        const u64 id = src.idx ? (u64)src.idx[i] : (u64)i;
        if (x < tprefix || (x == tprefix && id <= iprefix)) {
            const unsigned pos = atomicAdd(&n_won, 1u);
            if (pos < (unsigned)k) { pt[pos] = (int64_t)x; pi[pos] = (int64_t)id; }
        }
    }
    __syncthreads();
    int np2 = 1;
    while (np2 < k) np2 <<= 1;
    for (int i = k + threadIdx.x; i < np2; i += blockDim.x) { pt[i] = INT64_MAX; pi[i] = INT64_MAX; }
    __syncthreads();
    bitonic_sort_pairs(pt, pi, np2);
    for (int i = threadIdx.x; i < k; i += blockDim.x) {
        out_idx[i] = first + pi[i];
        if (out_time) out_time[i] = pt[i];
    }
}

int bits_for(int64_t v)       // number of bits needed to represent v >= 0
{
    int b = 0;
    while (v > 0) { ++b; v >>= 1; }
    return b;
}

// Blocks for a pass over n elements: two elements per thread while that fits eight blocks per SM
// (short passes are bound by the latency of a thread's loads, not by their number), the
// blocks striding over the rest.
int grid_for(int64_t n)
{
    int64_t g = (n + kSelThreads * 2 - 1) / (kSelThreads * 2);
    if (g < 1) g = 1;
    if (g > 148 * 8) g = 148 * 8;
    return (int)g;
}

}  // namespace

void launch_argmin(cudaStream_t s, const int64_t *batch, int64_t count, int64_t time_bound,
                   const SelectScratch &sc, int64_t *d_result, int64_t *launches)
{
    const int idx_bits = bits_for(count - 1) > 0 ? bits_for(count - 1) : 1;
    const bool packed = bits_for(time_bound) + idx_bits <= 63;
    cudaMemsetAsync(sc.key, 0xFF, 2 * sizeof(u64), s);
    const int g = grid_for(count);
    if (packed) {
        argmin_packed_kernel<<<g, kSelThreads, 0, s>>>(batch, count, idx_bits, sc.key);
        ++*launches;
    } else {
        argmin_time_kernel<<<g, kSelThreads, 0, s>>>(batch, count, sc.key);
        argmin_index_kernel<<<g, kSelThreads, 0, s>>>(batch, count, sc.key);
        *launches += 2;
    }
    argmin_unpack_kernel<<<1, 32, 0, s>>>(sc.key, idx_bits, packed ? 1 : 0, d_result);
    ++*launches;
}

namespace {

// Bits of the times that the radix select looks at.
int time_bits(int64_t time_bound)
{
    // bits above the bound on any time are zero everywhere: start below them
    return bits_for(time_bound) > 0 ? bits_for(time_bound) : 1;
}

// Radix passes over all time digits (most significant first) of the current source.
// min_shift > 0 leaves the digits below that bit open: the prefix found is then the top of a
// range of times, not one time.
void time_passes(cudaStream_t s, const int64_t *batch, int64_t count, int64_t n_source, int64_t time_bound,
                 const SelectScratch &sc, bool compact_after_first, int64_t *launches, int min_shift = 0)
{
    const int g = grid_for(n_source);
    const int tb = time_bits(time_bound);
    bool first_pass = true;
    for (int shift = ((tb + kRadixBits - 1) / kRadixBits - 1) * kRadixBits; shift >= min_shift; shift -= kRadixBits) {
        const int width = tb - shift < kRadixBits ? tb - shift : kRadixBits;
        radix_pass_kernel<false><<<g, kSelThreads, 0, s>>>(batch, count, sc, shift, width, shift == 0);
        ++*launches;
        if (compact_after_first && first_pass && shift > 0 && sc.comp_cap > 0) {
            compact_kernel<<<grid_for(count), kSelThreads, 0, s>>>(batch, count, sc, shift);
            ++*launches;
        }
        first_pass = false;
    }
}

// Index passes, collection and the final sort of the k winners.
void finish_passes(cudaStream_t s, const int64_t *batch, int64_t first, int64_t count, int64_t n_source, int k,
                   const SelectScratch &sc, int64_t *d_indices, int64_t *d_times, int64_t *launches)
{
    const size_t sort_smem = (size_t)kSortMax * 2 * sizeof(int64_t);
    const int g = grid_for(n_source);
    const int ib = bits_for(count - 1) > 0 ? bits_for(count - 1) : 1;
    for (int shift = ((ib + kRadixBits - 1) / kRadixBits - 1) * kRadixBits; shift >= 0; shift -= kRadixBits) {
        const int width = ib - shift < kRadixBits ? ib - shift : kRadixBits;
        radix_pass_kernel<true><<<g, kSelThreads, 0, s>>>(batch, count, sc, shift, width, false);
        ++*launches;
    }
    collect_kernel<<<g, kSelThreads, 0, s>>>(batch, count, sc, k, 0);
    sort_pairs_kernel<<<1, 1024, sort_smem, s>>>(sc.cand_time, sc.cand_idx, k, k, first, d_indices, d_times, nullptr, 0);
    *launches += 2;
}

constexpr int64_t kSampledMin = (int64_t)1 << 20;     // arrays at least this long are sampled first

}  // namespace

namespace {
__global__ void add_scalar_kernel(int64_t *word, int64_t value) { if (threadIdx.x == 0 && blockIdx.x == 0) *word += value; }
}  // namespace
void launch_add_scalar(cudaStream_t s, int64_t *d_word, int64_t value, int64_t *launches)
{
    add_scalar_kernel<<<1, 32, 0, s>>>(d_word, value);
    ++*launches;
}

namespace {
__global__ void merge_init_kernel(SelState *st, int64_t n)
{
    if (threadIdx.x == 0 && blockIdx.x == 0) { SelState z{}; z.use_compact = 1; z.cn = (u64)n; *st = z; }
}
}  // namespace

void launch_merge_pairs(cudaStream_t s, const int64_t *times, const int64_t *indices, int64_t n, int k,
                        const SelectScratch &sc, int64_t *d_indices, int64_t *d_times, int64_t *launches)
{
    // the general selection kernel, reading the given pairs in the place of the compact buffer
    SelectScratch src = sc;
    src.comp_time = const_cast<int64_t *>(times);
    src.comp_idx = const_cast<int64_t *>(indices);
    src.comp_cap = n;
    merge_init_kernel<<<1, 32, 0, s>>>(reinterpret_cast<SelState *>(sc.sel_state), n);
    const size_t gen_smem = (size_t)kSortMax * 2 * sizeof(int64_t) + (size_t)kBins * sizeof(u64);
    ensure_dynamic_smem(reinterpret_cast<const void *>(&general_select_kernel), gen_smem);
    general_select_kernel<<<1, kSelThreads, gen_smem, s>>>(nullptr, n, src, k, 63, 63, 0, d_indices, d_times);
    *launches += 2;
}

void launch_topk(cudaStream_t s, const int64_t *batch, int64_t first, int64_t count, int k,
                 int64_t time_bound, const SelectScratch &sc, int64_t *d_indices, int64_t *d_times,
                 int64_t *launches)
{
    launch_select(s, batch, first, count, k, time_bound, sc, nullptr, d_indices, d_times, launches);
}

void launch_select(cudaStream_t s, const int64_t *batch, int64_t first, int64_t count, int k, int64_t time_bound,
                   const SelectScratch &sc, int64_t *d_result, int64_t *d_indices, int64_t *d_times,
                   int64_t *launches)
{
    const size_t sort_smem = (size_t)kSortMax * 2 * sizeof(int64_t);
    ensure_dynamic_smem(reinterpret_cast<const void *>(&sort_pairs_kernel), sort_smem);     // per device
    const int idx_bits = bits_for(count - 1) > 0 ? bits_for(count - 1) : 1;
    const bool packed = bits_for(time_bound) + idx_bits <= 63;
    const bool sampled = k > 0 && count >= kSampledMin && sc.comp_cap > 0;
    if (!sampled) {
        // short arrays (or no compact buffer): the best element and the selection as separate passes
        if (d_result) launch_argmin(s, batch, count, time_bound, sc, d_result, launches);
        if (k == 0) return;
        if (count <= kSortMax) {
            sort_pairs_kernel<<<1, 1024, sort_smem, s>>>(batch, nullptr, (int)count, k, first, d_indices, d_times, nullptr, 0);
            ++*launches;
            return;
        }
        sel_init_kernel<<<1, 256, 0, s>>>(reinterpret_cast<SelState *>(sc.sel_state), sc.hist, k, 0, nullptr);
        ++*launches;
        time_passes(s, batch, count, count, time_bound, sc, true, launches);
        finish_passes(s, batch, first, count, count, k, sc, d_indices, d_times, launches);
        return;
    }
    // 1. the k-th smallest time of a strided sample: about 2^16 elements, but a stride small enough
    //    for the expected k * stride elements up to that time to fit the compact buffer four times
    int64_t stride = count >> 16;
    if (stride > sc.comp_cap / (4 * (int64_t)k)) stride = sc.comp_cap / (4 * (int64_t)k);
    if (stride < 64) stride = 64;
    const int64_t n_sample = (count + stride - 1) / stride;
    const bool min_here = d_result != nullptr && packed;
    sel_init_kernel<<<1, 256, 0, s>>>(reinterpret_cast<SelState *>(sc.sel_state), sc.hist, k, stride,
                                      min_here ? sc.key : nullptr);
    ++*launches;
    //    The last digit of the times is left open when there are two digits above it: the threshold
    //    is then the top of the 2048-wide range of times that holds the sample's k-th smallest -
    //    still a time that k elements do not exceed, for one pass over the sample less.
    const int low_bits = time_bits(time_bound) > 2 * kRadixBits ? kRadixBits : 0;
    time_passes(s, batch, count, n_sample, time_bound, sc, false, launches, low_bits);
    // 2. one pass: minimum of the packed key, elements up to that time into the compact buffer
    scan_select_kernel<<<grid_for(count), kSelThreads, 0, s>>>(batch, count, sc, idx_bits, min_here ? 1 : 0, 1, low_bits);
    ++*launches;
    if (min_here) {
        argmin_unpack_kernel<<<1, 32, 0, s>>>(sc.key, idx_bits, 1, d_result);
        ++*launches;
    } else if (d_result) {
        launch_argmin(s, batch, count, time_bound, sc, d_result, launches);     // times too wide to pack
    }
    // 3. the selection proper on the compact buffer (about k * stride pairs when the sample is
    //    representative; the grid is sized for that, the kernels stride over whatever there is):
    //    one histogram over its range of times cuts it down to what one sort takes
    const int64_t n_expect = (int64_t)k * stride * 4 < count ? (int64_t)k * stride * 4 : count;
    SelState *st = reinterpret_cast<SelState *>(sc.sel_state);
    const int g_small = grid_for(n_expect) < 148 ? grid_for(n_expect) : 148;     // a block's histogram costs more than its elements
    refine_kernel<<<g_small, kSelThreads, 0, s>>>(sc);
    collect_kernel<<<g_small, kSelThreads, 0, s>>>(batch, count, sc, kSortMax, 1);
    sort_pairs_kernel<<<1, 1024, sort_smem, s>>>(sc.cand_time, sc.cand_idx, 0, k, first, d_indices, d_times, st,
                                         packed ? idx_bits : 0);
    // ... and the general kernel for what that path cannot finish (it returns at once otherwise)
    const size_t gen_smem = sort_smem + (size_t)kBins * sizeof(u64);
    ensure_dynamic_smem(reinterpret_cast<const void *>(&general_select_kernel), gen_smem);
    general_select_kernel<<<1, kSelThreads, gen_smem, s>>>(batch, count, sc, k, time_bits(time_bound), idx_bits, first,
                                                          d_indices, d_times);
    *launches += 4;
}

}  // namespace distsim

// ---- top-k without any allocation --------------------------------------------------------------
// Same kernels as launch_topk, but the radix-select scratch (histogram, selection state and the
// k collected pairs) lives in a fixed device array that is part of the loaded library, so the
// call neither needs a context nor touches the CUDA allocator.
namespace {

constexpr int kStaticWords = 8 + distsim::kBins + 16 + 2 * DISTSIM_TOPK_STATIC_MAX_K;   // 64-bit words
static __device__ __align__(256) unsigned long long g_topk_static_scratch[kStaticWords];

constexpr int kMaxDevices = 64;
unsigned long long *g_static_scratch_addr[kMaxDevices];    // device address of the array, per device

}  // namespace

extern "C" int distsim_topk_static(void *stream, const int64_t *d_batch_ns, int64_t first,
                                   int64_t count, int32_t k, int64_t *d_indices, int64_t *d_times)
{
    if (!d_batch_ns || !d_indices || first < 0 || count < 1 || k < 1 || k > count) return DISTSIM_E_ARG;
    if (k > DISTSIM_TOPK_STATIC_MAX_K) return DISTSIM_E_CAPACITY;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return DISTSIM_E_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return DISTSIM_E_UNSUPPORTED;
    if (!g_static_scratch_addr[dev]) {
        // In host code the array's name is only a handle for the runtime, not a pointer a kernel
        // could use: ask the runtime for the address the array has on the current device.
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_topk_static_scratch) != cudaSuccess || !p) return DISTSIM_E_CUDA;
        g_static_scratch_addr[dev] = static_cast<unsigned long long *>(p);
    }
    unsigned long long *base = g_static_scratch_addr[dev];
    distsim::SelectScratch sc{};
    sc.key = base; sc.hist = base + 8; sc.sel_state = base + 8 + distsim::kBins;
    sc.cand_time = reinterpret_cast<int64_t *>(base + 8 + distsim::kBins + 16);
    sc.cand_idx = sc.cand_time + DISTSIM_TOPK_STATIC_MAX_K;
    int64_t launches = 0;
    // launch_topk begins by clearing the histogram, the selection state and the output cursor,
    // so whatever the previous call left in the array is never read
    distsim::launch_topk(static_cast<cudaStream_t>(stream), d_batch_ns, first, count, k, INT64_MAX, sc,
                         d_indices, d_times, &launches);
    return cudaGetLastError() == cudaSuccess ? DISTSIM_OK : DISTSIM_E_CUDA;
}
