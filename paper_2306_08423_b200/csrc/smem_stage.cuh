// Staging of read-only tables into shared memory with bulk asynchronous copies.
//
// One thread arms the block's mbarrier with the expected byte count and issues the copies
// (cp.async.bulk global -> shared of the issuing block, no multicast); every thread then waits
// on the barrier's phase with a bounded number of polls.  If the wait gives up, the block records
// DISTSIM_E_TIMEOUT in the status word and reads the tables from global memory instead; it
// polls once more (again bounded) before leaving so that no copy is still in flight when the
// block's shared memory is released.
// Requirements: source and destination 16-byte aligned, size a multiple of 16 bytes.
#pragma once

#include "engine.h"

namespace distsim {

__device__ __forceinline__ uint32_t smem_addr(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ bool mbar_poll(uint32_t bar, uint32_t phase, int max_polls)
{
    for (int i = 0; i < max_polls; ++i) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done) : "r"(bar), "r"(phase) : "memory");
        if (done) return true;
    }
    return false;
}

// Copies `bytes` from src_a to dst_a and from src_b to dst_b (both shared destinations).
// Must be called by every thread of the block.  Returns true when the shared copies are usable.
__device__ __forceinline__ bool stage_two_tables(uint64_t *bar_ptr, void *dst_a, const void *src_a,
                                                 void *dst_b, const void *src_b, uint32_t bytes,
                                                 int32_t *status)
{
    const uint32_t bar = smem_addr(bar_ptr);
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(bar) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                     :: "r"(bar), "r"(2 * bytes) : "memory");
        asm volatile(
            "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
            :: "r"(smem_addr(dst_a)), "l"(src_a), "r"(bytes), "r"(bar) : "memory");
        asm volatile(
            "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
            :: "r"(smem_addr(dst_b)), "l"(src_b), "r"(bytes), "r"(bar) : "memory");
    }
    // each try_wait already blocks for a bounded, implementation-defined time
    bool ok = mbar_poll(bar, 0, 1 << 16);
    if (!ok) {
        atomicCAS(status, 0, DISTSIM_E_TIMEOUT);
        mbar_poll(bar, 0, 1 << 16);          // drain before the block can exit
    }
    // the block must agree: a table that one thread could not see is read from global by all
    ok = __syncthreads_and(ok);
    return ok;
}

}  // namespace distsim
