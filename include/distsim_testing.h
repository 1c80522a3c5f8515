/*
 * distsim_testing.h -- hooks into a context for the test-suite and the benchmark's accounting.
 * They are exported by the engine's library because they need the context, but they are not
 * part of its stable ABI; the paper has no counterpart for any of them.
 */
#ifndef DISTSIM_TESTING_H
#define DISTSIM_TESTING_H

#include <stdint.h>

#include "distsim.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Sets how often the evaluation kernels poll, in their FIRST wait, for the bulk copies that
 * stage tables into shared memory (default 65 536).  With 0 that wait gives up at once: every
 * block takes the path a stalled copy engine would force - it records the stall, waits for the
 * copy once more with the full limit (so nothing is in flight when the block goes on) and reads
 * its tables from global memory.  Results stay exact; the next synchronising call returns
 * DISTSIM_E_TIMEOUT after writing its outputs.  Nothing hangs, traps or faults in either setting.
 */
int distsim_testing_set_stage_wait_polls(distsim_ctx *ctx, int32_t polls);

/*
 * Host arithmetic of the evaluation launches (no device involved): cuts the candidates [lo, hi)
 * of a row with pp stages into pieces of at most max_blocks blocks of the long-pipeline kernel,
 * as the library does before it launches (so that no range, however large, overflows a grid).
 * Returns the number of pieces (or DISTSIM_E_ARG) and writes the first max_pieces of them:
 * h_lo[i], h_hi[i] the piece's candidates, h_blocks[i] its blocks.
 */
int64_t distsim_testing_lockstep_pieces(int32_t pp, int64_t lo, int64_t hi, int64_t max_blocks, int64_t max_pieces,
                                        int64_t *h_lo, int64_t *h_hi, int32_t *h_blocks);

/*
 * Host logic of the bidirectional schedule (no device involved): the merged item order the library
 * builds for pp devices and m micro-batches (both even, 2 <= pp <= 32, 2 <= m <= DISTSIM_MAX_M).
 * h_order[d * 2 m + k] = pipeline << 15 | is-backward << 14 | micro-batch within its pipeline for
 * the k-th item of device d; *h_kept = the items a device may run from the last backward item of
 * its later stage on.  Returns DISTSIM_OK or DISTSIM_E_ARG.
 */
int distsim_testing_bidirectional_order(int32_t pp, int32_t m, uint16_t *h_order, int32_t *h_kept);

/*
 * Phase timing of distsim_eval_select for the benchmark: with enable != 0 the call records CUDA
 * events on its stream before the evaluation launches, after them and after the selection
 * launches; distsim_testing_last_phase_ms returns the two durations of the most recent such
 * call (it must have completed: distsim_eval_select synchronises before it returns).
 */
int distsim_testing_time_phases(distsim_ctx *ctx, int32_t enable);
int distsim_testing_last_phase_ms(distsim_ctx *ctx, float *h_eval_ms, float *h_select_ms);

/* Number of kernels this context has launched so far (launch accounting of the benchmark). */
int64_t distsim_testing_launch_count(const distsim_ctx *ctx);

/*
 * Recurrence cells of the current space (a candidate has 2 m pp cells, one per schedule item),
 * and how many of them belong to entries that the engine evaluates in 32-bit arithmetic
 * (exactly: their time bound is below 2^32).  Host outputs.
 */
int distsim_testing_space_cells(distsim_ctx *ctx, int64_t *h_cells, int64_t *h_cells_32bit);

#ifdef __cplusplus
}
#endif
#endif /* DISTSIM_TESTING_H */
