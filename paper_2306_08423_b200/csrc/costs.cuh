// Communication cost model (alpha-beta), shared by the set-up kernels and the kernels that
// price a collective themselves.
#pragma once

#include "engine.h"

namespace distsim {

__device__ __forceinline__ int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// Ring all-reduce over n devices of `bytes`: 2(n-1) steps, each paying the latency and moving
// 1/n of the tensor, i.e. a per-device volume of 2(n-1)*bytes/n (paper Sec. 4.2).
__device__ __forceinline__ int64_t ring_cost(int64_t n, int64_t bytes, int64_t alpha, int64_t beta)
{
    return 2 * (n - 1) * alpha + ceil_div(2 * (n - 1) * bytes, n * beta);
}

// All-reduce event time: directly modelled up to k = ar_profile_max devices; above, the k-device
// time scaled by the per-device volume 2(n-1)S/n of the actual device count (paper Sec. 4.2).
__device__ __forceinline__ int64_t allreduce_cost(const TableConst &tc, int64_t n, int64_t bytes, int64_t alpha, int64_t beta)
{
    const int64_t k = tc.ar_profile_max;
    if (k <= 1 || n <= k) return ring_cost(n, bytes, alpha, beta);
    return ceil_div(ring_cost(k, bytes, alpha, beta) * k * (n - 1), (k - 1) * n);
}

}  // namespace distsim
