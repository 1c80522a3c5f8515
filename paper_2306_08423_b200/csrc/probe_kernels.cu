// Integer-issue probe: a dependency-free stream of 32-bit integer ALU instructions, used by the
// benchmark to measure the device's plain-integer issue peak under the clocks of the moment
// (the denominator of the evaluation kernel's roofline).
#include "engine.h"

namespace distsim {

namespace {

constexpr int kChains = 8;

// Each thread advances 8 independent (x, y) pairs: x += y (integer add) and y ^= x (logic op),
// i.e. 16 integer instructions per iteration that cannot be fused with one another.
__global__ void __launch_bounds__(256) int_issue_probe_kernel(int iters, int64_t *sink)
{
    uint32_t x[kChains], y[kChains];
#pragma unroll
    for (int k = 0; k < kChains; ++k) { x[k] = threadIdx.x + k; y[k] = blockIdx.x * 7u + k; }
    // 8 rounds per loop trip: 128 counted instructions against 2 of loop overhead
    for (int it = 0; it < iters; it += 8) {
#pragma unroll
        for (int rep = 0; rep < 8; ++rep) {
#pragma unroll
            for (int k = 0; k < kChains; ++k) {
                asm volatile("add.u32 %0, %0, %1;" : "+r"(x[k]) : "r"(y[k]));
                asm volatile("xor.b32 %0, %0, %1;" : "+r"(y[k]) : "r"(x[k]));
            }
        }
    }
    uint32_t acc = 0;
#pragma unroll
    for (int k = 0; k < kChains; ++k) acc += x[k] ^ y[k];
    if (acc == 0x12345678u) sink[0] = acc;       // keeps the work alive; practically never taken
}

}  // namespace

int64_t launch_int_issue_probe(cudaStream_t s, int blocks, int iters, int64_t *sink, int64_t *launches)
{
    iters = (iters + 7) & ~7;                    // the kernel runs whole groups of 8 rounds
    int_issue_probe_kernel<<<blocks, 256, 0, s>>>(iters, sink);
    ++*launches;
    return (int64_t)blocks * 256 * iters * kChains * 2;
}

}  // namespace distsim
