// Integer-issue probes: dependency-free streams of integer ALU work, used by the benchmark to
// measure the device's plain-integer peaks under the clocks of the moment (the denominators of
// the evaluation kernel's roofline).
//   mode 0  32-bit add / xor pairs                      (16 instructions per round and thread)
//   mode 1  recurrence cells x = max(x, y) + c on int64 (8 cells per round and thread, counted
//           as 6 instructions each: compare pair, two selects, add, add-with-carry)
//   mode 2  32-bit compare + select pairs               (16 instructions per round and thread)
//   mode 3  recurrence cells x = max(x, y) + c on uint32 (8 cells per round and thread, counted
//           as 2 instructions each)
//   mode 4  recurrence cells x = max(x + c, y) on uint32 with the fused add-max instruction
//           (8 cells per round and thread, counted as 2 instructions each, as in mode 3)
//
// This file is a library of its own (libdistsim_bench.so, declared in include/distsim_bench.h):
// measurement code stays out of the engine's library.
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/distsim_bench.h"

namespace {

constexpr int kChains = 8;

template <int kMode>
__global__ void __launch_bounds__(256) int_issue_probe_kernel(int iters, int64_t *sink)
{
    uint32_t x[kChains], y[kChains];
    int64_t a[kChains], b[kChains], c[kChains];
#pragma unroll
    for (int k = 0; k < kChains; ++k) {
        x[k] = threadIdx.x + k; y[k] = blockIdx.x * 7u + k;
        a[k] = threadIdx.x * 3 + k; b[k] = (int64_t)blockIdx.x * 1000003 + k; c[k] = k + 1 + (sink == nullptr);
    }
    // 8 rounds per loop trip, so that loop overhead is about 1 %
    for (int it = 0; it < iters; it += 8) {
#pragma unroll
        for (int rep = 0; rep < 8; ++rep) {
#pragma unroll
            for (int k = 0; k < kChains; ++k) {
                if (kMode == 0) {
                    asm volatile("add.u32 %0, %0, %1;" : "+r"(x[k]) : "r"(y[k]));
                    asm volatile("xor.b32 %0, %0, %1;" : "+r"(y[k]) : "r"(x[k]));
                } else if (kMode == 1) {
                    // chain k: a = max(a, b) + c; b alternates with a through the other chain
                    const int64_t mx = a[k] > b[k] ? a[k] : b[k];
                    a[k] = mx + c[k];
                } else if (kMode == 3) {
                    const uint32_t mx = x[k] > y[k] ? x[k] : y[k];
                    x[k] = mx + (uint32_t)c[k];
                } else if (kMode == 4) {
                    x[k] = __viaddmax_u32(x[k], (uint32_t)c[k], y[k]);
                } else {
                    asm volatile("{ .reg .pred p; setp.gt.u32 p, %0, %1; selp.u32 %0, %0, %1, p; }" : "+r"(x[k]) : "r"(y[k]));
                    asm volatile("{ .reg .pred p; setp.lt.u32 p, %0, %1; selp.u32 %0, %1, %0, p; }" : "+r"(y[k]) : "r"(x[k]));
                }
            }
        }
    }
    uint32_t acc = 0;
#pragma unroll
    for (int k = 0; k < kChains; ++k) acc += x[k] ^ y[k] ^ (uint32_t)a[k] ^ (uint32_t)(a[k] >> 32);
    if (acc == 0x12345678u && sink) sink[0] = acc;       // keeps the work alive; practically never taken
}

}  // namespace

extern "C" int distsim_bench_int_issue_probe(void *stream, int32_t mode, int32_t blocks, int32_t iters,
                                             int64_t *d_sink, int64_t *h_ops)
{
    if (!h_ops || !d_sink || blocks < 1 || iters < 1 || mode < 0 || mode > 4) return -1;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    iters = (iters + 7) & ~7;                    // the kernel runs whole groups of 8 rounds
    if (mode == 1) int_issue_probe_kernel<1><<<blocks, 256, 0, s>>>(iters, d_sink);
    else if (mode == 2) int_issue_probe_kernel<2><<<blocks, 256, 0, s>>>(iters, d_sink);
    else if (mode == 3) int_issue_probe_kernel<3><<<blocks, 256, 0, s>>>(iters, d_sink);
    else if (mode == 4) int_issue_probe_kernel<4><<<blocks, 256, 0, s>>>(iters, d_sink);
    else int_issue_probe_kernel<0><<<blocks, 256, 0, s>>>(iters, d_sink);
    const int64_t per_round = mode == 1 ? kChains * 6 : kChains * 2;   // modes 0, 2: 16 = 8 x 2; modes 3, 4: 8 x 2
    *h_ops = (int64_t)blocks * 256 * iters * per_round;
    return cudaGetLastError() == cudaSuccess ? 0 : -6;
}
