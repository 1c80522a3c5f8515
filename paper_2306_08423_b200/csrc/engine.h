// Internal declarations shared by the engine's translation units (not part of the C ABI).
//
// Device-resident data (all built by kernels in setup_kernels.cu from the raw event table):
//
//   Row      one per valid (mp, pp) pair, in canonical order.  A row owns a contiguous block of
//            candidate indices: (entry, partition, schedule) with the schedule fastest.
//   Entry    one per valid micro-batch count m of a row: m, micro-batch size b, event class and
//            the communication-event costs that depend on (dp, b).
//   ETF/ETB  per entry, exclusive prefix sums over layers of the layer composites
//              phi(l)   = fwd(l) + AR + [expert l] * A2A      (MP modeling, paper Sec. 4.3)
//              gamma(l) = bwd(l) + AR + [expert l] * A2A
//            so that any contiguous stage's item cost is one subtraction.  Row stride `lp` is
//            n_layers + 1 rounded up to an even count, which keeps every row 16-byte aligned for
//            bulk copies into shared memory.
//   NB/TP    per row, [e][l] tables for the gradient buckets of a stage that ends at layer e:
//            NB = number of full buckets completed once layers e-1..l have produced their
//            gradients; TP = cost of the trailing partial bucket of the stage [l, e).
//   DT       per entry, [e][l]: for the stage [l, e), with gradient overlap the end of its bucket
//            lane relative to the start of its last backward item (-1 if it has no buckets);
//            without overlap the total cost of its buckets.  Optional (memory budget).
//   binom    C(n, k), saturated at 2^62, for unranking stage partitions.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>
#include <vector>

#include "../../include/distsim.h"

namespace distsim {

constexpr int64_t kSat = (int64_t)1 << 62;
// Device status word beyond the DISTSIM_E_* codes: a block gave up waiting for a bulk copy twice
// and may have left with the copy still in flight.
constexpr int32_t kStatusCopyPending = -70;

struct TableConst {
    int32_t n_layers, n_classes, n_devices, gpus_per_node;
    int64_t global_batch, seq, hidden;
    int64_t alpha_intra, beta_intra, alpha_inter, beta_inter;
    int64_t bucket;       // dp_bucket_bytes
    int32_t overlap;
    int32_t elem_bytes;
    int32_t lp;           // padded prefix-row length (int64 words)
    int32_t ar_profile_max;   // all-reduces over more devices are extrapolated (0: never)
    int32_t n_jitter;         // P: micro-batch slots of the jitter tables (0 or a power of two)
    int32_t jitter_stages;    // columns of the jitter tables
};

struct Row {
    int64_t offset;       // first candidate index of the row
    int64_t n_part;       // stage partitions per entry
    int64_t size;         // n_entries * n_part * n_sched
    int64_t t_full;       // cost of one full gradient bucket (0 if dp == 1)   [device-filled]
    int64_t row_tab_off;  // offset (words) of this row's NB / TP tables
    int32_t mp, pp, dp, log2_mp;
    int32_t n_entries, entry0;
    int32_t n_sched, sched_list;   // enabled schedules in canonical order, two bits each (see row_sched)
    int32_t p2p_period;   // boundary d|d+1 is inter-node iff ((d+1) & (p2p_period-1)) == 0
    int32_t v;            // model chunks per device: 1, or > 1 for a row of interleaved 1F1B candidates
                          // (one schedule, id 3; partitions into pp * v virtual stages)
    int32_t two_way;      // 1 for a row of bidirectional-pipeline candidates (one schedule, id 4; v = 1;
                          // even micro-batch counts), else 0
    int64_t t_full_near;  // two_way rows: t_full is the cost of a full gradient bucket over the 2 dp holders
                          // of a stage when they span nodes, this one when a node holds them all   [device-filled]
};

// Schedule id (0 GPipe, 1 1F1B, 2 asynchronous 1F1B, 3 interleaved 1F1B, 4 bidirectional pipelines)
// of position sc among a row's schedules.
__host__ __device__ inline int row_sched(const Row &row, int sc) { return row.two_way ? 4 : (row.sched_list >> (2 * sc)) & 3; }

struct Entry {
    int32_t m, b, cls, row;
    int64_t p2p_intra, p2p_inter, a2a, ar;   // [device-filled]
    int64_t bound;        // [device-filled] upper bound on every time of every candidate of the entry
    int64_t rel_bound;    // [device-filled] bound + the largest shift of a relative time frame
};

struct SpaceConst {
    int32_t n_rows, n_entries, pp_max, partition_mode;   // partition_mode 0 balanced, 1 all
    int32_t binom_k;      // second dimension of binom
    int32_t pad;
    int64_t n_candidates;
};

// Raw table on the device (inputs of the set-up kernels; the emission kernels read the
// per-class layer times from it as well).
struct RawTable {
    const int32_t *class_mp, *class_b;
    const int64_t *fwd, *bwd;        // [n_classes][n_layers]
    const uint8_t *expert;           // [n_layers]
    const int64_t *grad;             // [n_layers]
    const int64_t *jit_f, *jit_b;    // [n_jitter][jitter_stages] extra item time (nullptr if none)
};

// Everything a kernel needs, passed by value.
struct DeviceView {
    TableConst tc;
    SpaceConst sc;
    RawTable raw;
    const Row *rows;
    const Entry *entries;
    const int64_t *etf, *etb;        // [n_entries][lp]
    const int64_t *nb, *tp;          // per row [L+1][L+1]
    const int64_t *dt;               // per entry [L+1][L+1] bucket-lane table (nullptr: not built)
    int32_t tab_words;               // words of one [L+1][L+1] table, rounded up to even
    int32_t tab_words32;             // 32-bit words of one dt32 table, rounded up to a multiple of 4
    const uint2 *pfb32;              // [n_entries][lp] (forward, backward) prefix sums of the entries whose
                                     // time bound is below 2^32 (zeros for the others); nullptr: not built
    const uint32_t *dt32;            // [n_entries][tab_words32] bucket-lane tables of those entries, negative
                                     // values stored as 0 (nullptr: not built)
    const int64_t *binom;            // [n_layers][binom_k]
    const int32_t *next_grad;        // [L+1] smallest l' >= l with grad_bytes[l'] > 0 (L if none)
    const int32_t *pe;               // [L+1] number of expert layers before layer l
    const int64_t *jsum;             // [n_entries][DISTSIM_MAX_PP] total jitter of the m forward and
                                     // m backward items of a stage (nullptr without jitter)
    const uint16_t *order;           // bidirectional schedule: every device's items in its order,
                                     // [entry's offset + device * (2 m + 1) + position]: pipeline << 15 |
                                     // is-backward << 14 | micro-batch within its pipeline
    const uint32_t *order_before;    // same index, position 0 .. 2 m: how many forward items of pipeline 0,
                                     // backward items of pipeline 0 and forward items of pipeline 1 come before
                                     // that position in the device's order, 9 bits each
    const int64_t *order_off;        // [n_entries] offset of the entry's orders in `order` (low 48 bits) and,
                                     // above them, the items a device may run from the last backward item
                                     // of its earlier-finishing pipeline on (nullptr: no such rows)
    int32_t *status;                 // device status word: 0 ok, else first error code
    int32_t stage_polls;             // polls of the first wait for staged tables (the drain wait keeps its own limit)
};

// A kernel's limit on dynamic shared memory is an attribute of (kernel, device): raise it when a
// launch needs more than this process has asked for so far on the current device, not on every
// launch.  `kernel` is the address of the __global__ function.
inline cudaError_t ensure_dynamic_smem(const void *kernel, size_t bytes)
{
    struct Granted { const void *kernel; int device; size_t bytes; };
    static std::mutex mu;
    static std::vector<Granted> granted;
    if (bytes == 0) return cudaSuccess;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    for (Granted &g : granted)
        if (g.kernel == kernel && g.device == dev) {
            if (bytes <= g.bytes) return cudaSuccess;
            e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
            if (e == cudaSuccess) g.bytes = bytes;
            return e;
        }
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess) granted.push_back(Granted{kernel, dev, bytes});
    return e;
}

// ---- set-up kernels (setup_kernels.cu) -------------------------------------------------
void launch_fill_entries(cudaStream_t s, const TableConst &tc, Row *rows, int n_rows,
                         Entry *entries, int n_entries, int64_t *launches);
void launch_build_prefix(cudaStream_t s, const TableConst &tc, const RawTable &raw,
                         const Entry *entries, int n_entries, int64_t *etf, int64_t *etb,
                         int64_t *launches);
void launch_build_bucket_tables(cudaStream_t s, const TableConst &tc, const RawTable &raw,
                                const Row *rows, int n_rows, int64_t *nb, int64_t *tp,
                                int64_t *launches);
// 32-bit copies of the prefix rows and bucket-lane tables for the entries whose time bound is
// below 2^32 (after launch_build_entry_tables: reads the entries' bounds).  dt32 may be null.
void launch_build_narrow_tables(cudaStream_t s, const DeviceView &v, uint2 *pfb32, uint32_t *dt32,
                                int64_t *launches);
// Per entry: the bucket-lane table (if dt != nullptr) and the time bound of the entry.
void launch_build_entry_tables(cudaStream_t s, const DeviceView &v, Entry *entries, int64_t *dt,
                               int64_t *jsum, int64_t *launches);
void launch_build_layer_tables(cudaStream_t s, const TableConst &tc, const RawTable &raw,
                               int32_t *next_grad, int32_t *pe, int64_t *launches);

// ---- evaluation (eval_kernels.cu) ------------------------------------------------------
// One launch covers several (row, range) work items; a block finds its item from block_begin.
struct EvalWork {
    int32_t row;                 // row index
    int32_t e_begin, e_end, ept; // thread kernel: entries [e_begin, e_end) of the row, per thread
    int64_t p_lo, p_hi;          // thread kernel: partitions [p_lo, p_hi)
    int64_t lo, hi;              // candidates [lo, hi), local to the row
    int32_t block_begin;         // first block of the item inside the launch
    int32_t nx;                  // thread kernel: blocks along the partition axis
};
constexpr int kMaxEvalWork = 24;
struct EvalBatch {
    int32_t n, pad;
    EvalWork w[kMaxEvalWork];
};
// One more stream for the latency-bound lock-step launch of an evaluation, so that it runs
// beside the throughput-bound launches instead of before them (side[0] == nullptr: everything
// on the caller's stream).
struct SideStream {
    cudaStream_t side[1] = {nullptr};
    cudaEvent_t fork = nullptr, join[1] = {nullptr};
};
// Evaluates candidates [first, first + count); rows / entries: host copies.  Results go to
// batch_out[index - first] and, if non-null, busy_out[(index - first) * pp_max + d].  All work
// is ordered after what `s` held before the call and before what is enqueued on `s` after it.
void launch_eval(cudaStream_t s, const SideStream &ss, const DeviceView &v, const Row *rows, int n_rows,
                 const Entry *entries, int64_t first, int64_t count, int64_t *batch_out, int64_t *busy_out,
                 int64_t *launches);
// Cuts candidates [lo, hi) of a row of pp stages into pieces of at most max_blocks lock-step
// blocks each; returns the number of pieces and writes the first max_pieces of them.
int64_t lockstep_pieces(int pp, int64_t lo, int64_t hi, int64_t max_blocks, int64_t max_pieces,
                        int64_t *piece_lo, int64_t *piece_hi, int32_t *piece_blocks);

// ---- selection (select_kernels.cu) -----------------------------------------------------
struct SelectScratch {
    unsigned long long *key;        // [2] packed / two-pass argmin keys
    unsigned long long *hist;       // [2048] radix histogram
    unsigned long long *sel_state;  // [16] radix-select state
    int64_t *cand_time, *cand_idx;  // [4096] selected pairs before sorting
    int64_t *comp_time, *comp_idx;  // [comp_cap] compact buffer of the surviving pairs (optional)
    int64_t comp_cap;               // 0: no compact buffer
};
// d_result[0] = smallest time, d_result[1] = its smallest position in `batch`.
void launch_argmin(cudaStream_t s, const int64_t *batch, int64_t count, int64_t time_bound,
                   const SelectScratch &sc, int64_t *d_result, int64_t *launches);
// The best element and the k fastest of a long array in little more than one pass over it: a
// strided sample gives a threshold that at least k elements do not exceed (the k-th smallest of
// a subset is never below the k-th smallest of the whole); one pass then takes the minimum of
// the packed (time, position) key and copies the elements up to the threshold to the compact
// buffer, and the selection proper runs on that buffer.  d_result (nullable): [0] smallest
// time, [1] its smallest position.  k == 0: the best element only.
void launch_select(cudaStream_t s, const int64_t *batch, int64_t first, int64_t count, int k, int64_t time_bound,
                   const SelectScratch &sc, int64_t *d_result, int64_t *d_indices, int64_t *d_times,
                   int64_t *launches);
// The k smallest of n given (time, index) pairs, ascending (merging the lists of several ranks).
void launch_merge_pairs(cudaStream_t s, const int64_t *times, const int64_t *indices, int64_t n, int k,
                        const SelectScratch &sc, int64_t *d_indices, int64_t *d_times, int64_t *launches);
void launch_add_scalar(cudaStream_t s, int64_t *d_word, int64_t value, int64_t *launches);    // *d_word += value
// time_bound: an upper bound on every element of `batch` (INT64_MAX if unknown).
void launch_topk(cudaStream_t s, const int64_t *batch, int64_t first, int64_t count, int k,
                 int64_t time_bound, const SelectScratch &sc, int64_t *d_indices, int64_t *d_times,
                 int64_t *launches);

// ---- emission (emit_kernels.cu) --------------------------------------------------------
struct EmitPlan {                    // per selected candidate, written by the planning kernel
    int64_t index;
    int64_t batch_ns;
    int64_t rec_base;                // first record of the selection (after the scan)
    int64_t rec_total;               // records of all its devices
    int32_t row, entry, m, sched, pp, mp, dp, ok;
    int32_t v, two_way;              // model chunks per device (1 unless interleaved 1F1B); then the arrays
                                     // indexed "per stage" below are per virtual stage c * pp + d where noted.
                                     // two_way: a bidirectional-pipeline candidate - v = 2 stands for its two
                                     // pipelines, rf / rb / last_b_start are indexed pipeline * pp + device, and
                                     // bounds holds the pp + 1 bounds both pipelines share
    int32_t bounds[DISTSIM_MAX_PP + 1];              // per (virtual) stage
    int32_t tile_items;              // schedule items per block of the record kernel
    int32_t tmpl_words;              // words of the widest stage's forward + backward item templates
    int32_t run_words;               // upper bound on the words of any run of items of this selection
    int32_t rf[DISTSIM_MAX_PP], rb[DISTSIM_MAX_PP];   // records of one forward / backward item, per (virtual) stage
    int64_t n_buckets[DISTSIM_MAX_PP];                // per device
    int64_t stage_recs[DISTSIM_MAX_PP];               // records of one device of stage d
    int64_t stage_rec_prefix[DISTSIM_MAX_PP + 1];
    int64_t busy[DISTSIM_MAX_PP];
    int64_t main_end[DISTSIM_MAX_PP];
    int64_t last_b_start[DISTSIM_MAX_PP];             // per (virtual) stage
};
// Totals over the planned selections (device words written by the scan kernel, read by the host).
struct EmitTotals {
    int64_t records;        // records of all selections
    int64_t item_tiles;     // most item tiles of any selection
    int64_t bucket_tiles;   // most (stage, replica chunk) tiles of any selection's bucket lanes
    int64_t tmpl_words;     // most words of any stage's forward + backward item templates
    int64_t bucket_recs;    // most gradient-bucket records of any stage
    int64_t run_words;      // most words of any run of items (capacity of the record kernel's images)
    int64_t pad[2];
};
// Plans the n selections: item start times into op_start (op_words_per_cand words each), record
// counts, offsets / busy / util (each nullable); sums: scratch of kEmitSumWords words per
// selection; d_totals: the words of an EmitTotals.
constexpr int kEmitSumWords = 8;
void launch_emit_plan(cudaStream_t s, const DeviceView &v, const int64_t *d_indices, int n,
                      EmitPlan *plans, int64_t *op_start, int64_t op_words_per_cand, int64_t *sums,
                      int64_t *offsets, int64_t *busy, double *util, int64_t *d_totals,
                      int ilv_words /* shared-memory words a warp needs for the space's interleaved rows (0: none) */,
                      int64_t *h_totals /* nullable: host memory the device can write; receives the totals' words
                                           and, in word 7, the device status word after planning */,
                      cudaEvent_t planned /* nullable: recorded behind the planning kernel */,
                      int64_t *launches,
                      const EmitTotals *limits = nullptr /* nullable: what the caller has provisioned (records:
                                           its capacity); the last block sets word 7 of d_totals to 1 if the
                                           plans stay within it, else to 0 and the status to DISTSIM_E_CAPACITY */);
// Offsets, activity times and utilisations of every device of the planned selections (each nullable).
void launch_emit_devices(cudaStream_t s, const DeviceView &v, const EmitPlan *plans, int n, int64_t *offsets,
                         int64_t *busy, double *util, const int64_t *d_totals, int64_t *launches);
int interleaved_words_of(int pp, int v);           // those words for one row
int bidirectional_words_of(int pp, int kept);      // shared-memory words a bidirectional candidate needs
int bidirectional_kept_cap_of(int pp);             // most items the kernels keep per device of such a candidate
// out[k] = order-sensitive checksum of the records [offsets[k], offsets[k + 1]).
void launch_checksum_lists(cudaStream_t s, const distsim_record *records, const int64_t *offsets, int64_t n_lists,
                           uint64_t *out, int64_t *launches);
// gate (nullable): device words of an EmitTotals; the kernels write nothing unless word 7 is non-zero.
// words (nullable): the per-device outputs, written beside the item kernel (on the side stream) rather
// than by launch_emit_plan before it.
struct EmitDeviceWords { int64_t *offsets, *busy; double *util; const int64_t *d_totals; };
void launch_emit_records(cudaStream_t s, const SideStream &ss, const DeviceView &v, int n, const EmitPlan *plans,
                         const int64_t *op_start, int64_t op_words_per_cand, const EmitTotals &totals,
                         distsim_record *records, int64_t *launches, const int64_t *gate = nullptr,
                         const EmitDeviceWords *words = nullptr);

}  // namespace distsim
