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
    u64 pad[6];
};

// The source a pass reads: the array itself (index = position) or the compact buffer.
struct SelSource { const int64_t *t; const int64_t *idx; int64_t n; };
__device__ __forceinline__ SelSource sel_source(const SelState *st, const int64_t *batch, int64_t count,
                                                const SelectScratch &sc)
{
    if (st->use_compact) return SelSource{sc.comp_time, sc.comp_idx, (int64_t)st->cn};
    return SelSource{batch, nullptr, count};
}

// Run by one whole block once a digit's histogram is complete: picks the bin that holds the
// wanted rank, narrows the prefix / mask to it and clears the histogram for the next digit.
template <bool kIndexPhase>
__device__ __forceinline__ void pick_bin(SelState *st, u64 *hist, u64 *partial /* shared, [kSelThreads] */, int shift,
                                         unsigned dmask, bool last_time_pass)
{
    const u64 tprefix = st->tprefix, tmask = st->tmask, iprefix = st->iprefix, imask = st->imask;
    __threadfence();
    constexpr int kPer = kBins / kSelThreads;
    u64 mine = 0;
    for (int k = 0; k < kPer; ++k) mine += *((volatile u64 *)&hist[threadIdx.x * kPer + k]);
    partial[threadIdx.x] = mine;
    __syncthreads();
    if (threadIdx.x == 0) {
        u64 rank = st->rank, cum = 0, in_bin = 0;
        int chunk = kSelThreads - 1;
        for (int c = 0; c < kSelThreads; ++c) {
            if (rank < cum + partial[c]) { chunk = c; break; }
            cum += partial[c];
        }
        int bin = chunk * kPer + kPer - 1;
        for (int k = 0; k < kPer; ++k) {
            const u64 h = *((volatile u64 *)&hist[chunk * kPer + k]);
            if (rank < cum + h) { bin = chunk * kPer + k; in_bin = h; break; }
            cum += h;
        }
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
        const u64 x = (u64)src.t[i];
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
}

__global__ void sel_init_kernel(SelState *st, u64 *hist, int k)
{
    for (int i = threadIdx.x; i < kBins; i += blockDim.x) hist[i] = 0;
    if (threadIdx.x == 0) { SelState z{}; z.rank = (u64)(k - 1); *st = z; }
}

// The pick step alone, for a first digit whose histogram an evaluation has filled.
__global__ void __launch_bounds__(kSelThreads)
radix_pick_kernel(SelectScratch sc, int shift, int width, bool last_time_pass)
{
    __shared__ u64 partial[kSelThreads];
    pick_bin<false>(reinterpret_cast<SelState *>(sc.sel_state), sc.hist, partial, shift, (1u << width) - 1u, last_time_pass);
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

// Collects the k elements that are not above the threshold pair (time, index), in any order.
__global__ void __launch_bounds__(kSelThreads)
collect_kernel(const int64_t *__restrict__ batch, int64_t count, SelectScratch sc, int k)
{
    SelState *st = reinterpret_cast<SelState *>(sc.sel_state);
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

// One block sorts up to 4096 (time, index) pairs ascending (bitonic network in shared memory)
// and writes the first k.  Also the whole top-k for arrays of at most 4096 elements.
constexpr int kSortMax = 4096;
__global__ void __launch_bounds__(1024)
sort_pairs_kernel(const int64_t *__restrict__ ct, const int64_t *__restrict__ ci, int n_in, int k,
                  int64_t first, int64_t *out_idx, int64_t *out_time)
{
    extern __shared__ __align__(16) unsigned char sm[];
    int64_t *st = reinterpret_cast<int64_t *>(sm);
    int64_t *si = st + kSortMax;
    int np2 = 1;
    while (np2 < n_in) np2 <<= 1;
    for (int i = threadIdx.x; i < np2; i += blockDim.x) {
        st[i] = i < n_in ? ct[i] : INT64_MAX;
        si[i] = i < n_in ? (ci ? ci[i] : (int64_t)i) : INT64_MAX;
    }
    __syncthreads();
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
            __syncthreads();
        }
    for (int i = threadIdx.x; i < k; i += blockDim.x) {
        out_idx[i] = first + si[i];
        if (out_time) out_time[i] = st[i];
    }
}

int bits_for(int64_t v)       // number of bits needed to represent v >= 0
{
    int b = 0;
    while (v > 0) { ++b; v >>= 1; }
    return b;
}

int grid_for(int64_t n)
{
    int64_t g = (n + kSelThreads * 8 - 1) / (kSelThreads * 8);
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

// Bits of the times that the radix select looks at, and its first digit.
struct TimeDigits { int tb, shift0, width0; };
TimeDigits time_digits(int64_t time_bound)
{
    TimeDigits d;
    // bits above the bound on any time are zero everywhere: start below them
    d.tb = bits_for(time_bound) > 0 ? bits_for(time_bound) : 1;
    d.shift0 = ((d.tb + kRadixBits - 1) / kRadixBits - 1) * kRadixBits;
    d.width0 = d.tb - d.shift0 < kRadixBits ? d.tb - d.shift0 : kRadixBits;
    return d;
}

// The radix select for more than kSortMax elements.  first_digit_done: the histogram of the first
// digit has been filled already (by an evaluation), only its bin is still to be picked.
void select_passes(cudaStream_t s, const int64_t *batch, int64_t first, int64_t count, int k, int64_t time_bound,
                   const SelectScratch &sc, bool first_digit_done, int64_t *d_indices, int64_t *d_times,
                   int64_t *launches)
{
    const size_t sort_smem = (size_t)kSortMax * 2 * sizeof(int64_t);
    const int g = grid_for(count);
    const TimeDigits td = time_digits(time_bound);
    bool first_pass = true;
    for (int shift = td.shift0; shift >= 0; shift -= kRadixBits) {
        const int width = td.tb - shift < kRadixBits ? td.tb - shift : kRadixBits;
        if (first_pass && first_digit_done) radix_pick_kernel<<<1, kSelThreads, 0, s>>>(sc, shift, width, shift == 0);
        else radix_pass_kernel<false><<<g, kSelThreads, 0, s>>>(batch, count, sc, shift, width, shift == 0);
        ++*launches;
        if (first_pass && shift > 0 && sc.comp_cap > 0) {
            compact_kernel<<<g, kSelThreads, 0, s>>>(batch, count, sc, shift);
            ++*launches;
        }
        first_pass = false;
    }
    const int ib = bits_for(count - 1) > 0 ? bits_for(count - 1) : 1;
    for (int shift = ((ib + kRadixBits - 1) / kRadixBits - 1) * kRadixBits; shift >= 0; shift -= kRadixBits) {
        const int width = ib - shift < kRadixBits ? ib - shift : kRadixBits;
        radix_pass_kernel<true><<<g, kSelThreads, 0, s>>>(batch, count, sc, shift, width, false);
        ++*launches;
    }
    collect_kernel<<<g, kSelThreads, 0, s>>>(batch, count, sc, k);
    sort_pairs_kernel<<<1, 1024, sort_smem, s>>>(sc.cand_time, sc.cand_idx, k, k, first, d_indices, d_times);
    *launches += 2;
}

}  // namespace

void launch_topk(cudaStream_t s, const int64_t *batch, int64_t first, int64_t count, int k,
                 int64_t time_bound, const SelectScratch &sc, int64_t *d_indices, int64_t *d_times,
                 int64_t *launches)
{
    const size_t sort_smem = (size_t)kSortMax * 2 * sizeof(int64_t);
    ensure_dynamic_smem(reinterpret_cast<const void *>(&sort_pairs_kernel), sort_smem);     // per device
    if (count <= kSortMax) {
        sort_pairs_kernel<<<1, 1024, sort_smem, s>>>(batch, nullptr, (int)count, k, first, d_indices, d_times);
        ++*launches;
        return;
    }
    sel_init_kernel<<<1, 256, 0, s>>>(reinterpret_cast<SelState *>(sc.sel_state), sc.hist, k);
    ++*launches;
    select_passes(s, batch, first, count, k, time_bound, sc, false, d_indices, d_times, launches);
}

FusedSelect begin_fused_select(cudaStream_t s, int64_t count, int k, int64_t time_bound, const SelectScratch &sc,
                               int64_t *launches)
{
    static_assert(kBins == kSelectBins, "the evaluation kernels fill the radix select's histogram");
    FusedSelect fs{};
    fs.key = sc.key; fs.hist = sc.hist;
    fs.idx_bits = bits_for(count - 1) > 0 ? bits_for(count - 1) : 1;
    const TimeDigits td = time_digits(time_bound);
    fs.shift = td.shift0; fs.width = td.width0;
    // folded in when time and position fit one key and the array is too long to be sorted directly
    fs.enabled = (bits_for(time_bound) + fs.idx_bits <= 63 && count > kSortMax) ? 1 : 0;
    if (fs.enabled) {
        cudaMemsetAsync(sc.key, 0xFF, 2 * sizeof(u64), s);
        sel_init_kernel<<<1, 256, 0, s>>>(reinterpret_cast<SelState *>(sc.sel_state), sc.hist, k > 0 ? k : 1);
        ++*launches;
    }
    return fs;
}

void finish_fused_argmin(cudaStream_t s, const FusedSelect &fs, const SelectScratch &sc, int64_t *d_result,
                         int64_t *launches)
{
    argmin_unpack_kernel<<<1, 32, 0, s>>>(sc.key, fs.idx_bits, 1, d_result);
    ++*launches;
}

void finish_fused_topk(cudaStream_t s, const FusedSelect &fs, const int64_t *batch, int64_t first, int64_t count, int k,
                       int64_t time_bound, const SelectScratch &sc, int64_t *d_indices, int64_t *d_times,
                       int64_t *launches)
{
    (void)fs;
    const size_t sort_smem = (size_t)kSortMax * 2 * sizeof(int64_t);
    ensure_dynamic_smem(reinterpret_cast<const void *>(&sort_pairs_kernel), sort_smem);     // per device
    select_passes(s, batch, first, count, k, time_bound, sc, true, d_indices, d_times, launches);
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
