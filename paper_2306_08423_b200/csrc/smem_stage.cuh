// Staging of read-only tables into shared memory with bulk asynchronous copies.
//
// One thread arms the block's mbarrier with the expected byte count and issues the copies
// (cp.async.bulk global -> shared of the issuing block, no multicast); every thread then waits
// on the barrier's phase with a bounded number of polls.  If the wait gives up, the block records
// DISTSIM_E_TIMEOUT in the status word and reads the tables from global memory instead (the same
// values, so results stay exact); it polls once more (again bounded) before going on so that no
// copy is still in flight when the block's shared memory is released.  Should that second wait
// give up as well, the status word takes kStatusCopyPending: the block may leave with a copy in
// flight and nothing computed on the device afterwards can be trusted.
// Requirements: sources and destinations 16-byte aligned, sizes multiples of 16 bytes.
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

struct StageCopy { void *dst; const void *src; uint32_t bytes; };

// Issues up to kMaxCopies bulk copies (entries with bytes == 0 are skipped) and waits for all of
// them.  Must be called once per block, by every thread.  Returns true when the shared copies
// are usable by the whole block.
constexpr int kMaxCopies = 4;
constexpr int kDrainPolls = 1 << 16;
__device__ __forceinline__ bool stage_tables(uint64_t *bar_ptr, const StageCopy (&c)[kMaxCopies], int32_t *status,
                                             int first_polls)
{
    const uint32_t bar = smem_addr(bar_ptr);
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(bar) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t total = 0;
#pragma unroll
        for (int i = 0; i < kMaxCopies; ++i) total += c[i].bytes;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                     :: "r"(bar), "r"(total) : "memory");
#pragma unroll
        for (int i = 0; i < kMaxCopies; ++i)
            if (c[i].bytes)
                asm volatile(
                    "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                    :: "r"(smem_addr(c[i].dst)), "l"(c[i].src), "r"(c[i].bytes), "r"(bar) : "memory");
    }
    // each try_wait already blocks for a bounded, implementation-defined time
    bool ok = mbar_poll(bar, 0, first_polls);
    if (!ok) {
        atomicCAS(status, 0, DISTSIM_E_TIMEOUT);
        if (!mbar_poll(bar, 0, kDrainPolls))                  // drain before the block can exit
            atomicMin(status, kStatusCopyPending);
    }
    // the block must agree: a table that one thread could not see is read from global by all
    ok = __syncthreads_and(ok);
    return ok;
}

__device__ __forceinline__ bool stage_two_tables(uint64_t *bar_ptr, void *dst_a, const void *src_a,
                                                 void *dst_b, const void *src_b, uint32_t bytes,
                                                 int32_t *status, int first_polls)
{
    const StageCopy c[kMaxCopies] = {{dst_a, src_a, bytes}, {dst_b, src_b, bytes}, {nullptr, nullptr, 0}, {nullptr, nullptr, 0}};
    return stage_tables(bar_ptr, c, status, first_polls);
}

}  // namespace distsim
