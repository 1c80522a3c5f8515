/*
 * distsim.h -- C ABI of the batched strategy-timeline engine (CUDA, sm_100a).
 *
 * The engine evaluates DistSim's event-based activity timeline (paper Sec. 3.2
 * and 4.3) for very many candidate hybrid-parallel training strategies at once.
 * A candidate is x = (mp, pp, dp = N/(mp*pp), stage bounds 0=c_0<..<c_pp=L,
 * micro-batch count m, pipeline schedule); the model enters as an event table:
 * per event class (mp, micro-batch size b) the elapsed time of every layer's
 * forward and backward computation event, and alpha-beta constants for the
 * communication events.
 *
 * Conventions
 *   - Every function returns DISTSIM_OK (0) or a negative DISTSIM_E_* code; it
 *     never throws, aborts or prints.  distsim_last_error() gives the text of
 *     the most recent failure on that context.
 *   - "h_" pointers are HOST memory, "d_" pointers are DEVICE memory on the
 *     context's device.  Host inputs are copied before the call returns.
 *     Device buffers are allocated and owned by the caller; the library owns
 *     only its copies of the tables and its scratch.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Calls enqueue work on it and return without synchronising,
 *     except where a result is returned to host memory (stated per function).
 *   - All times are int64 nanoseconds.  A context is not thread-safe: use one
 *     per host thread.
 *   - There is no CPU fallback: without a CUDA device distsim_create fails.
 *   - DISTSIM_E_TIMEOUT.  Kernels stage their tables into shared memory with bulk copies and
 *     wait for them a bounded number of times.  A block whose wait gives up reads the same
 *     tables from global memory instead, so its results are exact.  The stall is reported by
 *     the next synchronising call (distsim_argmin, distsim_emit_timelines), which still writes
 *     all its outputs and then returns DISTSIM_E_TIMEOUT: the code tells the caller that the
 *     device's copy engine stalled, not that the outputs are wrong.  Only if a block's second,
 *     equally bounded wait gives up too (a copy may then still be in flight) does that call
 *     write nothing; distsim_last_error says which of the two happened.
 */
#ifndef DISTSIM_H
#define DISTSIM_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DISTSIM_MAX_PP      64     /* pipeline stages                              */
#define DISTSIM_MAX_LAYERS  256
#define DISTSIM_MAX_M       4096   /* micro-batches per candidate                  */

enum {
    DISTSIM_OK = 0,
    DISTSIM_E_ARG = -1,        /* null pointer, malformed table or space            */
    DISTSIM_E_STATE = -2,      /* table or space not loaded yet                     */
    DISTSIM_E_RANGE = -3,      /* candidate index outside [0, n_candidates)         */
    DISTSIM_E_CAPACITY = -4,   /* caller's output buffer too small                  */
    DISTSIM_E_OVERFLOW = -5,   /* a time or count bound does not fit 62 bits        */
    DISTSIM_E_CUDA = -6,       /* a CUDA runtime call failed                        */
    DISTSIM_E_TIMEOUT = -7,    /* a bounded device-side wait gave up (see below)    */
    DISTSIM_E_UNSUPPORTED = -8 /* e.g. degrees that are not powers of two           */
};

/* Event kinds in distsim_record.kind. */
enum {
    DISTSIM_COMPUTE_F = 0, DISTSIM_COMPUTE_B = 1,   /* layer computation event       */
    DISTSIM_MP_AR_F = 2,   DISTSIM_MP_AR_B = 3,     /* model-parallel all-reduce     */
    DISTSIM_A2A_F = 4,     DISTSIM_A2A_B = 5,       /* expert-layer all-to-all       */
    DISTSIM_SEND_F = 6,    DISTSIM_SEND_B = 7,      /* transfer to the neighbour     */
    DISTSIM_DP_AR = 8,                              /* gradient all-reduce bucket    */
    DISTSIM_JITTER_F = 9,  DISTSIM_JITTER_B = 10    /* fluctuation at an item's start */
};

typedef struct distsim_ctx distsim_ctx;

/* Creates a context on the given CUDA device.  Fails with DISTSIM_E_CUDA when
 * there is no such device or it is not compute capability 10.x. */
int distsim_create(distsim_ctx **out, int cuda_device);
void distsim_destroy(distsim_ctx *ctx);
/* Text of the last error on this context ("" if none); valid until the next call. */
const char *distsim_last_error(const distsim_ctx *ctx);

/*
 * The event table (paper Sec. 3.2 "event", Sec. 4.1-4.2; the layer-to-events
 * mapping MAP(L->E) that Algorithm 1 takes as input).  All pointers are host
 * memory, read during the call only.
 *   fwd_ns/bwd_ns [n_classes][n_layers]  elapsed time of the layer's computation
 *                                        event for class k = (class_mp[k], class_b[k])
 *   layer_is_expert [n_layers]           1: the layer also has an all-to-all event
 *   grad_bytes [n_layers]                gradient bytes of the layer at mp = 1
 *   alpha_*_ns, beta_* (bytes per ns)    link latency / bandwidth inside a node
 *                                        and between nodes (the intra/inter-node
 *                                        attribute of communication events, Sec. 4.1)
 *   dp_bucket_bytes                      gradient all-reduce bucket size; 0 = one
 *                                        all-reduce event per stage (paper Sec. 4.3,
 *                                        DP modeling)
 *   dp_overlap                           0: buckets start after the device's last
 *                                        event; 1: a bucket starts once the layer
 *                                        holding its last byte has finished the
 *                                        last micro-batch's backward
 *   allreduce_profile_max                0: every all-reduce size is modelled directly;
 *                                        k > 1: an all-reduce over n > k devices takes the
 *                                        k-device time scaled by the per-device volume,
 *                                        ceil(T(k) * k (n-1) / ((k-1) n))  (the paper profiles
 *                                        up to 8 devices and extrapolates, Sec. 4.2)
 *   n_jitter, jitter_*                   fluctuation between micro-batches (the paper's error
 *                                        analysis, Sec. 5.3, blames profiling fluctuation that
 *                                        accumulates along the stages): with P = n_jitter > 0 the
 *                                        forward (backward) item of micro-batch j on stage d
 *                                        begins with a jitter event of jitter_fwd_ns
 *                                        (jitter_bwd_ns) [j mod P][d] ns.  Every strategy of the
 *                                        space must have pp <= jitter_stages.
 * Communication costs: ring all-reduce over n devices of S bytes
 * 2(n-1)alpha + ceil(2(n-1)S / (n beta)) (per-device volume 2(n-1)S/n, Sec. 4.2);
 * transfer alpha + ceil(S/beta); all-to-all (n-1)alpha + ceil((n-1)S/(n beta)).
 * Requirements: n_devices, gpus_per_node powers of two; 1 <= n_layers <=
 * DISTSIM_MAX_LAYERS; all times, bytes and constants >= 0, betas >= 1.
 * Returns DISTSIM_E_OVERFLOW if an upper bound on any batch time reaches 2^62.
 * Loading a table invalidates the current search space.
 */
typedef struct {
    int32_t n_layers, n_classes, n_devices, gpus_per_node;
    int64_t global_batch, seq, hidden;
    int64_t alpha_intra_ns, beta_intra, alpha_inter_ns, beta_inter;
    int64_t dp_bucket_bytes;
    int32_t dp_overlap;
    int32_t act_bytes_per_elem;
    const int32_t *class_mp, *class_b;
    const int64_t *fwd_ns, *bwd_ns;
    const uint8_t *layer_is_expert;
    const int64_t *grad_bytes;
    int32_t allreduce_profile_max;
    int32_t n_jitter;               /* P: 0, or a power of two <= 64                */
    int32_t jitter_stages;          /* columns of the jitter tables, <= 64         */
    int32_t reserved;               /* must be 0                                   */
    const int64_t *jitter_fwd_ns, *jitter_bwd_ns;   /* [P][jitter_stages], NULL if P == 0 */
} distsim_event_table;

int distsim_load_event_table(distsim_ctx *ctx, const distsim_event_table *h_table);

/*
 * The search space (paper Sec. 6: grid over parallel degrees with dp =
 * GPUs/mp/pp, invalid combinations dropped).  Candidates are numbered in this
 * canonical order, outermost first: mp ascending over powers of two <= mp_max;
 * pp ascending over powers of two <= min(pp_max, n_layers) with mp*pp | N and
 * dp | global_batch; m ascending over the valid entries of m_list (m_rule 0: m
 * divides Bp = global_batch/dp; 1: any m <= Bp, micro-batch size ceil(Bp/m));
 * stage partition (partition_mode 0: the balanced one, c_j = floor(j L / pp);
 * 1: every composition, lexicographic in (c_1..c_{pp-1})); schedule GPipe, 1F1B,
 * asynchronous 1F1B as enabled in sched_mask (bit 0 GPipe, bit 1 1F1B/Dapple, bit 2
 * asynchronous 1F1B: the 1F1B item order without gradient all-reduce events - the paper's
 * discussion of new algorithms reads an asynchronous pipeline as the same schedule minus the
 * global synchronisation event).
 * Bit 3 of sched_mask adds the interleaved 1F1B schedule (Sec. 4.3 takes the pipeline algorithm's
 * schedule as Algorithm 1's input; the paper builds on Megatron-LM, whose interleaved schedule
 * this is): every (mp, pp) with pp >= 2 is followed, for v = 2, 4, .. <= v_max with
 * pp*v <= min(DISTSIM_MAX_PP, L), by the candidates whose devices hold v model chunks each -
 * m ascending over the valid entries that are multiples of pp, then the partition of the layers
 * into pp*v virtual stages (virtual stage c*pp + d is chunk c of device d).  Such candidates have
 * schedule id 3; tables with per-micro-batch jitter do not combine with them
 * (DISTSIM_E_UNSUPPORTED).
 * Bit 4 adds bidirectional pipelines (Chimera, which Sec. 2 names among the pipeline scheduling
 * algorithms; schedule id 4): every (mp, pp) with pp >= 2 is then followed by the candidates
 * that run two pipelines in opposite directions over the same devices - pipeline "down" with
 * stage s on device s and the first m/2 micro-batches, pipeline "up" with stage s on device
 * pp-1-s and the others, each in 1F1B order, merged on a device in the order they would
 * interleave with unit item times - m ascending over the valid even entries, then the partition
 * into pp stages.  A stage's gradients are reduced over the 2 dp devices that hold it (also when
 * dp = 1).  Needs pp_max <= 32 and a table without jitter (DISTSIM_E_UNSUPPORTED otherwise).
 * Candidates are never materialised: the device decodes them from the index.
 * Fails with DISTSIM_E_ARG if a needed class (mp, b) is not in the table, with
 * DISTSIM_E_OVERFLOW if the count does not fit 62 bits.  *n_candidates receives
 * the size of the space.
 */
typedef struct {
    int32_t mp_max, pp_max, n_m;
    const int32_t *m_list;          /* host, ascending, 1 <= m <= DISTSIM_MAX_M */
    int32_t m_rule;
    int32_t partition_mode;
    int32_t sched_mask;
    int32_t v_max;                  /* interleaved 1F1B (sched_mask bit 3): chunks per device up to v_max */
} distsim_space;

int distsim_set_space(distsim_ctx *ctx, const distsim_space *h_space, int64_t *n_candidates);

typedef struct {
    int32_t mp, pp, dp, m, sched;   /* sched 0: GPipe, 1: 1F1B, 2: asynchronous 1F1B, 3: interleaved 1F1B,
                                       4: bidirectional pipelines */
    int32_t micro_batch_size;       /* b = ceil(Bp / m)                            */
    int32_t class_index;            /* row of the event table                      */
    int32_t bounds[DISTSIM_MAX_PP + 1];   /* c_0 .. c_pp (c_0 .. c_{pp*v} for sched 3) */
    int32_t v;                      /* model chunks per device (1 unless sched 3)  */
} distsim_candidate;

/* Host-side decode of one index, for reporting (the device decodes on its own). */
int distsim_decode(distsim_ctx *ctx, int64_t index, distsim_candidate *h_out);

/*
 * Batch time of candidates [first, first + count): for each, MP modeling, the
 * pipeline recurrence of Algorithm 1 (an item starts at the later of its input's
 * arrival and its device becoming free), DP modeling, and the critical path.
 *   d_batch_ns      [count]            out
 *   d_stage_busy_ns [count][pp_max]    out, nullable: activity time of one device
 *                                      of each stage (all replicas are identical);
 *                                      entries d >= pp are 0
 * Asynchronous on `stream`.
 */
int distsim_eval_strategies(distsim_ctx *ctx, void *stream, int64_t first, int64_t count,
                            int64_t *d_batch_ns, int64_t *d_stage_busy_ns);

/*
 * Evaluation and selection in one call (paper Sec. 6: the grid search keeps the fastest):
 * evaluates candidates [first, first + count) like distsim_eval_strategies and returns the best
 * candidate and the k fastest like distsim_argmin and distsim_topk.  For a long range the
 * selection reads the batch times little more than once: a strided sample of them gives a time
 * that at least k candidates do not exceed, one pass then finds the best candidate and gathers
 * the candidates up to that time, and the k fastest are selected among those few.
 *   d_batch_ns [count] out;  k in [0, min(count, 4096)], 0: no top-k;
 *   d_indices [k] out, d_times [k] out (nullable): ascending by (batch time, index);
 *   d_best [2] out, nullable (device): batch time and index of the best candidate;
 *   h_best_index, h_best_batch_ns: host out, both or neither.  With host outputs the call
 *   synchronises `stream`; without them it is asynchronous, and a stalled table copy
 *   (DISTSIM_E_TIMEOUT, see above) is reported by the next synchronising call instead.
 */
int distsim_eval_select(distsim_ctx *ctx, void *stream, int64_t first, int64_t count, int64_t *d_batch_ns,
                        int32_t k, int64_t *d_indices, int64_t *d_times, int64_t *d_best, int64_t *h_best_index,
                        int64_t *h_best_batch_ns);

/*
 * Best strategy of a range (paper Sec. 6: the grid search keeps the fastest):
 * smallest d_batch_ns[i], ties to the smallest index.  d_batch_ns[i] belongs to
 * candidate first + i.  Results go to host memory; the call synchronises `stream`.
 */
int distsim_argmin(distsim_ctx *ctx, void *stream, const int64_t *d_batch_ns, int64_t first,
                   int64_t count, int64_t *h_best_index, int64_t *h_best_batch_ns);

/*
 * The k fastest candidates of a range, ascending by (batch time, index).
 *   d_indices [k] out (candidate indices, first + i);  d_times [k] out, nullable.
 * Requires 1 <= k <= min(count, 4096).  Asynchronous on `stream`.
 * distsim_argmin and distsim_topk assume that d_batch_ns holds batch times produced by
 * distsim_eval_strategies for the current table and space (they use the load-time upper bound
 * on any batch time to skip empty high-order bits).
 */
int distsim_topk(distsim_ctx *ctx, void *stream, const int64_t *d_batch_ns, int64_t first,
                 int64_t count, int32_t k, int64_t *d_indices, int64_t *d_times);

/*
 * The k smallest of n given (batch time, candidate index) pairs, ascending by (time, index):
 * the merge step of a search whose candidate range was split over several GPUs (Sec. 6: the
 * candidates are independent, so every GPU selects among its own and only these short lists
 * are exchanged).  d_times_in, d_indices_in [n]: the gathered lists, times and indices >= 0;
 * d_indices [k] out, d_times [k] out (nullable).  Requires 1 <= k <= min(n, 4096).
 * Asynchronous on `stream`.
 */
int distsim_merge_topk(distsim_ctx *ctx, void *stream, const int64_t *d_times_in, const int64_t *d_indices_in,
                       int64_t n, int32_t k, int64_t *d_indices, int64_t *d_times);

/* One timeline record: event `kind` of `layer` for micro-batch `microbatch`
 * occupying [start_ns, end_ns) on its device.  For transfers, `layer` is the
 * stage's boundary layer; for gradient buckets it is the bucket number and
 * microbatch is -1. */
typedef struct { int64_t kind, layer, microbatch, start_ns, end_ns; } distsim_record;

/*
 * Full per-device timelines of n selected candidates (the simulator's output,
 * paper Sec. 3.2; the per-device event lists F of Algorithm 1 after DP
 * modeling).  Device rank (r*pp + d)*mp + q holds stage d of replica r.
 * A device's records are its main lane in time order, then its gradient buckets.
 *   d_indices  [n]                 candidate indices (device memory)
 *   d_records  [capacity_records]  out, nullable: NULL = sizing pass only
 *   d_offsets  [n*N + 1]           out: record offset of device k of selection i at
 *                                  [i*N + k]; last entry = total
 *   d_busy_ns  [n*N], d_util [n*N] out: activity time (union of the device's event
 *                                  intervals) and busy / batch time
 *   h_total_records                out (host): records needed
 * If capacity_records is too small nothing is written to d_records and the call
 * returns DISTSIM_E_CAPACITY with *h_total_records set.  The indices are read from device
 * memory so that the output of distsim_topk feeds this call without a trip through the host.
 * The call synchronises `stream` once,
 * after planning, to size the output (that is when *h_total_records, d_offsets, d_busy_ns and
 * d_util are final); the record kernels are then enqueued and the call returns without waiting
 * for them: d_records is complete when the work enqueued on `stream` so far has finished.  The
 * context's planning scratch is reused by the next call, so issue a context's calls on one
 * stream or order them yourself.
 */
int distsim_emit_timelines(distsim_ctx *ctx, void *stream, const int64_t *d_indices, int32_t n,
                           distsim_record *d_records, int64_t capacity_records,
                           int64_t *d_offsets, int64_t *d_busy_ns, double *d_util,
                           int64_t *h_total_records);

/*
 * The same without any wait on the host, for a loop that emits timelines step after step (the
 * paper's search loop, Sec. 6, keeps the host out of the way of the device).  What the
 * synchronising call learns from its planning pass - how much output and how much of the
 * kernels' resources the selection needs - the caller passes in instead:
 * distsim_emit_shape_of_last_plan() returns those figures for the context's most recent
 * synchronising planning pass (a sizing call, say, on a selection of the kind the loop will see),
 * and the caller may enlarge any of them for headroom.
 *   h_shape    host: upper bounds this call provisions for (the fields of distsim_emit_shape)
 * The call plans the n selections, then writes their records, all in stream order.  If the
 * selection needs more than `shape` or capacity_records allow, no record is written, the device
 * status becomes DISTSIM_E_CAPACITY and the next synchronising call on the context returns it;
 * d_offsets, d_busy_ns and d_util are written either way, and d_offsets[n*N] is the number of
 * records needed.  Errors found on the host (arguments, state) are returned at once.
 */
typedef struct {
    int64_t records;        /* records of all selections                                    */
    int64_t item_tiles;     /* most blocks of the item kernel any selection needs            */
    int64_t bucket_tiles;   /* most blocks of the gradient-bucket kernel any selection needs */
    int64_t tmpl_words;     /* most 64-bit words of a device's item templates                */
    int64_t bucket_recs;    /* most gradient-bucket records of a device                      */
    int64_t run_words;      /* most 64-bit words of one block's run of items                 */
} distsim_emit_shape;
int distsim_emit_shape_of_last_plan(distsim_ctx *ctx, distsim_emit_shape *h_shape);
int distsim_emit_timelines_async(distsim_ctx *ctx, void *stream, const int64_t *d_indices, int32_t n,
                                 distsim_record *d_records, int64_t capacity_records,
                                 const distsim_emit_shape *h_shape,
                                 int64_t *d_offsets, int64_t *d_busy_ns, double *d_util);

/*
 * Order-sensitive 64-bit checksum of every device's record stream (the paper has no counterpart:
 * a way to check emitted timelines, e.g. after they have been moved, without comparing gigabytes).
 * List k holds the records [d_offsets[k], d_offsets[k+1]) of d_records, as written by
 * distsim_emit_timelines (n_lists = n * N).  With w_0 .. w_{5r-1} the int64 words of its r
 * records in order, d_checksums[k] = sum over i of mix(w_i + (i + 1) * 0x9E3779B97F4A7C15) modulo
 * 2^64, where mix(z) is the SplitMix64 finaliser: z ^= z >> 30; z *= 0xBF58476D1CE4E5B9;
 * z ^= z >> 27; z *= 0x94D049BB133111EB; z ^= z >> 31.
 *   d_records, d_offsets [n_lists + 1] in; d_checksums [n_lists] out.  Asynchronous on `stream`.
 */
int distsim_checksum_timelines(distsim_ctx *ctx, void *stream, const distsim_record *d_records,
                               const int64_t *d_offsets, int64_t n_lists, uint64_t *d_checksums);

/*
 * Whole search from host memory: loads the table and space, evaluates every
 * candidate, and returns the best one and the k fastest to host buffers.
 *   h_topk_indices/h_topk_times [k]  out, nullable when k == 0
 * Synchronises.  Uses internal device scratch for the batch times.
 */
int distsim_search_host(distsim_ctx *ctx, const distsim_event_table *h_table,
                        const distsim_space *h_space, int32_t k, int64_t *h_n_candidates,
                        int64_t *h_best_index, int64_t *h_best_batch_ns,
                        int64_t *h_topk_indices, int64_t *h_topk_times);

/*
 * Top-k for callers that must not allocate device memory (the paper has no counterpart; this
 * is a deployment convenience).  Every other entry point works on a distsim_ctx, and creating
 * one calls cudaMalloc.  Some hosts cannot afford that: a latency-critical loop that may not
 * block on the allocator's device-wide synchronisation, a process whose whole GPU memory has
 * already been handed to a pool, or a plug-in inside a host application that forbids it.
 * This variant needs no context and calls no allocator (neither CUDA's nor any library's):
 * its radix-select scratch is a fixed array of about 33 KB that is part of the library image,
 * present on every GPU that has loaded the library until the process exits.
 *   d_batch_ns [count] in; d_indices [k] out (first + position), d_times [k] out, nullable;
 *   result ascending by (batch time, index), identical to distsim_topk's.
 *   Requires 1 <= k <= min(count, DISTSIM_TOPK_STATIC_MAX_K); a larger k is refused with
 *   DISTSIM_E_CAPACITY and nothing is launched.  Other errors: DISTSIM_E_ARG (null pointer, bad
 *   range), DISTSIM_E_CUDA, DISTSIM_E_UNSUPPORTED (device ordinal above 63).
 * It runs on the current device.  The first call on each device looks up the array's device
 * address (cudaGetSymbolAddress); make that first call before any stream capture begins and
 * not concurrently from several host threads.  Asynchronous on `stream`.
 * All calls on a device share the one array, and it keeps the previous call's contents; each
 * call clears the parts it reads before using them.  Two calls whose kernels can overlap on the
 * GPU (different streams or host threads of one process on the same device) race on it: issue
 * them on one stream or order them yourself.
 */
#define DISTSIM_TOPK_STATIC_MAX_K 1024
int distsim_topk_static(void *stream, const int64_t *d_batch_ns, int64_t first, int64_t count,
                        int32_t k, int64_t *d_indices, int64_t *d_times);

#ifdef __cplusplus
}
#endif
#endif /* DISTSIM_H */
