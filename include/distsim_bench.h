/*
 * distsim_bench.h -- measurement helpers of the benchmark (libdistsim_bench.so).  Not part of
 * the engine's ABI and not linked into the engine's library; the paper has no counterpart.
 */
#ifndef DISTSIM_BENCH_H
#define DISTSIM_BENCH_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Enqueues, on the current device, a kernel of `blocks` x 256 threads that issues a
 * dependency-free stream of integer work, `iters` rounds per thread, and stores the total
 * instruction count (threads x instructions) in *h_ops (host).  mode 0: 16 32-bit add / xor
 * instructions per round; mode 1: 8 recurrence cells x = max(x, y) + c on int64 per round,
 * counted as 6 instructions each; mode 2: 16 32-bit compare / select instructions per round;
 * mode 3: 8 recurrence cells on uint32 per round, counted as 2 instructions each; mode 4: the
 * same cells in the form x = max(x + c, y), issued as one fused add-max instruction each (still
 * counted as 2).  Timed by the caller with events on `stream` (a cudaStream_t as void*), it
 * gives the device's plain-integer issue rate under the clocks of the moment.
 *   d_sink  device memory, at least 8 bytes, caller-owned (keeps the work alive; practically
 *           never written).
 * Returns 0, -1 on a bad argument, -6 when the launch failed.  Asynchronous; allocates nothing.
 */
int distsim_bench_int_issue_probe(void *stream, int32_t mode, int32_t blocks, int32_t iters,
                                  int64_t *d_sink, int64_t *h_ops);

#ifdef __cplusplus
}
#endif
#endif /* DISTSIM_BENCH_H */
