// Host side of the C ABI: context, validation, search-space bookkeeping, kernel launches.
// No timeline arithmetic happens here; the host only counts the space, looks up event classes
// and decides launch shapes.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <map>
#include <new>
#include <string>
#include <utility>
#include <vector>

#include "engine.h"
#include "../../include/distsim_testing.h"

using namespace distsim;

namespace {

struct DevBuf {
    void *p = nullptr;
    size_t cap = 0;
    ~DevBuf() { if (p) cudaFree(p); }
    cudaError_t reserve(size_t bytes)
    {
        if (bytes <= cap) return cudaSuccess;
        if (p) { cudaFree(p); p = nullptr; cap = 0; }
        cudaError_t e = cudaMalloc(&p, bytes);
        if (e == cudaSuccess) cap = bytes;
        return e;
    }
    template <class T> T *as() const { return static_cast<T *>(p); }
};

constexpr int64_t kCompactCap = 1 << 20;     // pairs in the top-k compact buffer (16 MB)

bool is_pow2(int64_t v) { return v > 0 && (v & (v - 1)) == 0; }

int64_t sat_mul(int64_t a, int64_t b)
{
    const __int128 r = (__int128)a * b;
    return r >= (__int128)kSat ? kSat : (int64_t)r;
}
int64_t sat_add(int64_t a, int64_t b)
{
    const __int128 r = (__int128)a + b;
    return r >= (__int128)kSat ? kSat : (int64_t)r;
}

}  // namespace

struct distsim_ctx {
    int device = 0;
    std::string err;
    bool table_loaded = false, space_set = false;
    int64_t launches = 0;

    // table
    TableConst tc{};
    std::vector<int32_t> class_mp, class_b;
    std::vector<int64_t> fwd, bwd, grad;
    std::vector<uint8_t> expert;
    DevBuf d_class_mp, d_class_b, d_fwd, d_bwd, d_expert, d_grad, d_next_grad, d_pe, d_jit_f, d_jit_b, d_jsum;
    RawTable raw{};

    // space
    SpaceConst sc{};
    std::vector<Row> rows;
    std::vector<Entry> entries;
    std::vector<int64_t> binom;
    int64_t time_bound = 0;
    int64_t op_words_per_cand = 0;
    int ilv_words = 0;                    // shared-memory words a warp needs for the interleaved rows
    int32_t stage_polls = 1 << 16;        // polls of the first wait for staged tables
    cudaEvent_t phase_ev[3] = {nullptr, nullptr, nullptr};   // timing of distsim_eval_select's phases (hook)
    bool phase_timing = false, phase_valid = false;
    DevBuf d_rows, d_entries, d_etf, d_etb, d_nb, d_tp, d_binom, d_dt, d_pfb32, d_dt32;
    bool have_dt = false, have_narrow = false;

    // scratch
    DevBuf d_status, d_sel, d_result, d_plans, d_plan_sums, d_op_start, d_totals, d_batch, d_topk;
    DevBuf d_order, d_order_before, d_order_off;          // item orders of the bidirectional schedule (see DeviceView)
    bool have_order = false;
    int two_way_words = 0;                // shared-memory words a warp needs for the bidirectional rows
    SideStream side;                      // extra streams of an evaluation (lock-step launches)
    cudaEvent_t planned = nullptr;        // recorded behind the emission-planning kernel
    EmitTotals last_plan{};               // totals of the most recent synchronising planning pass
    bool have_last_plan = false;
    int64_t *h_pinned = nullptr;          // 16 words of pinned host memory for small results:
                                          // [0..3] results, [4] status, [8..15] emission totals

    DeviceView view() const
    {
        DeviceView v{};
        v.tc = tc; v.sc = sc; v.raw = raw;
        v.rows = d_rows.as<Row>(); v.entries = d_entries.as<Entry>();
        v.etf = d_etf.as<int64_t>(); v.etb = d_etb.as<int64_t>();
        v.nb = d_nb.as<int64_t>(); v.tp = d_tp.as<int64_t>();
        v.binom = d_binom.as<int64_t>();
        v.dt = have_dt ? d_dt.as<int64_t>() : nullptr;
        v.tab_words = ((tc.n_layers + 1) * (tc.n_layers + 1) + 1) & ~1;
        v.tab_words32 = ((tc.n_layers + 1) * (tc.n_layers + 1) + 3) & ~3;
        v.pfb32 = have_narrow ? d_pfb32.as<uint2>() : nullptr;
        v.dt32 = have_narrow && have_dt ? d_dt32.as<uint32_t>() : nullptr;
        v.next_grad = d_next_grad.as<int32_t>(); v.pe = d_pe.as<int32_t>();
        v.jsum = tc.n_jitter > 0 ? d_jsum.as<int64_t>() : nullptr;
        v.order = have_order ? d_order.as<uint16_t>() : nullptr;
        v.order_off = have_order ? d_order_off.as<int64_t>() : nullptr;
        v.order_before = have_order ? d_order_before.as<uint32_t>() : nullptr;
        v.status = d_status.as<int32_t>();
        v.stage_polls = stage_polls;
        return v;
    }
    SelectScratch select_scratch() const
    {
        SelectScratch s{};
        unsigned long long *base = d_sel.as<unsigned long long>();
        s.key = base; s.hist = base + 8; s.sel_state = base + 8 + 2048;
        s.cand_time = reinterpret_cast<int64_t *>(base + 8 + 2048 + 16);
        s.cand_idx = s.cand_time + 4096;
        s.comp_time = s.cand_idx + 4096;
        s.comp_idx = s.comp_time + kCompactCap;
        s.comp_cap = kCompactCap;
        return s;
    }
};

namespace {

int fail(distsim_ctx *c, int code, const char *msg)
{
    if (c) c->err = msg;
    return code;
}
int cuda_fail(distsim_ctx *c, cudaError_t e, const char *what)
{
    if (c) c->err = std::string(what) + ": " + cudaGetErrorString(e);
    return DISTSIM_E_CUDA;
}

#define CU(call, what)                                               \
    do {                                                             \
        cudaError_t e__ = (call);                                    \
        if (e__ != cudaSuccess) return cuda_fail(ctx, e__, what);    \
    } while (0)

int set_device(distsim_ctx *ctx)
{
    CU(cudaSetDevice(ctx->device), "cudaSetDevice");
    return DISTSIM_OK;
}

template <class T>
int upload(distsim_ctx *ctx, DevBuf &b, const T *src, size_t n, const char *what)
{
    CU(b.reserve(n ? n * sizeof(T) : sizeof(T)), what);
    if (n) CU(cudaMemcpy(b.p, src, n * sizeof(T), cudaMemcpyHostToDevice), what);
    return DISTSIM_OK;
}

const char *const kTimeoutText =
    "a bounded device-side wait for a bulk copy gave up; the affected blocks read their tables from "
    "global memory instead, so the outputs are exact and have been written";

// Reads and clears the device status word; synchronises the stream.  A wait that gave up while
// the copy still completed before its block went on is advisory: *stalled is set and DISTSIM_OK
// returned, so that the caller can finish its work and report DISTSIM_E_TIMEOUT with valid outputs.
int take_status(distsim_ctx *ctx, cudaStream_t s, int32_t code, bool *stalled);
int read_status(distsim_ctx *ctx, cudaStream_t s, bool *stalled)
{
    int32_t *st = reinterpret_cast<int32_t *>(ctx->h_pinned + 4);
    CU(cudaMemcpyAsync(st, ctx->d_status.p, sizeof(int32_t), cudaMemcpyDeviceToHost, s), "status read");
    CU(cudaStreamSynchronize(s), "status sync");
    return take_status(ctx, s, *st, stalled);
}
// Acts on a status word read from the device (and clears the device's copy if it is set).
int take_status(distsim_ctx *ctx, cudaStream_t s, int32_t code, bool *stalled)
{
    if (code != 0) {
        cudaMemsetAsync(ctx->d_status.p, 0, sizeof(int32_t), s);
        if (code == DISTSIM_E_TIMEOUT) { *stalled = true; return DISTSIM_OK; }
        if (code == kStatusCopyPending)
            return fail(ctx, DISTSIM_E_TIMEOUT, "a bulk copy into shared memory never completed: results computed on this device since may be wrong");
        if (code == DISTSIM_E_RANGE) return fail(ctx, code, "candidate index out of range");
        if (code == DISTSIM_E_CAPACITY)
            return fail(ctx, code, "an asynchronous emission needed more than its shape or capacity allowed: it wrote no records");
        return fail(ctx, code, "device reported an error");
    }
    return DISTSIM_OK;
}

void destroy_side(SideStream &ss)
{
    if (ss.fork) cudaEventDestroy(ss.fork);
    for (int k = 0; k < 1; ++k) {
        if (ss.join[k]) cudaEventDestroy(ss.join[k]);
        if (ss.side[k]) cudaStreamDestroy(ss.side[k]);
    }
    ss = SideStream{};
}

int floor_log2(int64_t v) { int b = -1; while (v > 0) { ++b; v >>= 1; } return b; }

// Item orders of the bidirectional schedule for (pp, m), both even: pipeline 0 puts stage s on
// device s and takes the first m / 2 micro-batches, pipeline 1 puts it on device pp - 1 - s and
// takes the others; each keeps its 1F1B order, and a device merges its two orders the way they
// would interleave if every item took one time slot: slot by slot it runs the next item of either
// pipeline whose input is there from an earlier slot, the one earlier in its pipeline's sequence
// of micro-batches first.  out[d * (2 m + 1) + k] = pipeline << 15 | is-backward << 14 | micro-batch
// within its pipeline; *kept = the most items any device runs from the last backward item of its
// later stage on (its gradients are complete first).  Returns false if the merge does not end.
bool bidirectional_orders(int pp, int m, std::vector<uint16_t> &out, std::vector<uint32_t> &before, int *kept)
{
    const int half = m / 2;
    struct Item { bool bwd; int j; };
    auto stage_of = [&](int d, int u) { return u ? pp - 1 - d : d; };
    std::vector<std::vector<Item>> queue((size_t)2 * pp);          // [device * 2 + pipeline]
    for (int d = 0; d < pp; ++d)
        for (int u = 0; u < 2; ++u) {
            const int warm = std::min(pp - stage_of(d, u), half);
            std::vector<Item> &q = queue[(size_t)d * 2 + u];
            int nf = 0, nb = 0;
            for (; nf < warm; ++nf) q.push_back({false, nf});
            while (nb < half) {
                q.push_back({true, nb++});
                if (nf < half) q.push_back({false, nf++});
            }
        }
    // slot after which an item's result exists, [pipeline][stage][micro-batch]; 0: not yet
    std::vector<int> done_f((size_t)2 * pp * half, 0), done_b((size_t)2 * pp * half, 0);
    auto at = [&](int u, int s, int j) { return ((size_t)u * pp + s) * half + j; };
    std::vector<size_t> head((size_t)2 * pp, 0);
    std::vector<int> n_out(pp, 0), last_b_pos((size_t)2 * pp, 0);
    const size_t stride = (size_t)2 * m + 1;
    out.assign((size_t)pp * stride, 0);
    before.assign((size_t)pp * stride, 0);
    std::vector<uint32_t> so_far(pp, 0);            // counts packed as in DeviceView::order_before
    int left = pp * 2 * m;
    for (int slot = 1; left > 0; ++slot) {
        if (slot > 4 * (m + pp)) return false;
        std::vector<int> pick(pp, -1);
        for (int d = 0; d < pp; ++d) {
            int best = 0;
            for (int u = 0; u < 2; ++u) {
                const std::vector<Item> &q = queue[(size_t)d * 2 + u];
                if (head[(size_t)d * 2 + u] == q.size()) continue;
                const Item it = q[head[(size_t)d * 2 + u]];
                const int s = stage_of(d, u);
                int ready;                           // slot after which the input exists
                if (!it.bwd) ready = s == 0 ? -1 : done_f[at(u, s - 1, it.j)];
                else ready = s == pp - 1 ? done_f[at(u, s, it.j)] : done_b[at(u, s + 1, it.j)];
                if (ready == 0 || ready >= slot) continue;
                if (pick[d] < 0 || it.j < best) { pick[d] = u; best = it.j; }
            }
        }
        for (int d = 0; d < pp; ++d) {
            const int u = pick[d];
            if (u < 0) continue;
            const Item it = queue[(size_t)d * 2 + u][head[(size_t)d * 2 + u]++];
            const int s = stage_of(d, u);
            (it.bwd ? done_b : done_f)[at(u, s, it.j)] = slot;
            if (it.bwd && it.j == half - 1) last_b_pos[(size_t)d * 2 + u] = n_out[d];
            before[(size_t)d * stride + n_out[d]] = so_far[d];
            out[(size_t)d * stride + n_out[d]++] = (uint16_t)((u << 15) | ((it.bwd ? 1 : 0) << 14) | it.j);
            if (u == 0) so_far[d] += it.bwd ? (1u << 9) : 1u;
            else if (!it.bwd) so_far[d] += 1u << 18;
            --left;
        }
    }
    for (int d = 0; d < pp; ++d) before[(size_t)d * stride + 2 * m] = so_far[d];
    *kept = 2;
    for (int d = 0; d < pp; ++d) {
        const int u_first = stage_of(d, 0) > stage_of(d, 1) ? 0 : 1;      // the pipeline in which the device holds the later stage
        *kept = std::max(*kept, 2 * m - last_b_pos[(size_t)d * 2 + u_first]);
    }
    return true;
}

}  // namespace

extern "C" {

int distsim_create(distsim_ctx **out, int cuda_device)
{
    if (!out) return DISTSIM_E_ARG;
    *out = nullptr;
    int n = 0;
    if (cudaGetDeviceCount(&n) != cudaSuccess || cuda_device < 0 || cuda_device >= n) return DISTSIM_E_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, cuda_device) != cudaSuccess) return DISTSIM_E_CUDA;
    if (prop.major != 10) return DISTSIM_E_CUDA;           // built for sm_100a only
    distsim_ctx *ctx = new (std::nothrow) distsim_ctx;
    if (!ctx) return DISTSIM_E_ARG;
    ctx->device = cuda_device;
    if (cudaSetDevice(cuda_device) != cudaSuccess ||
        ctx->d_status.reserve(64) != cudaSuccess ||
        ctx->d_sel.reserve((8 + 2048 + 16 + 2 * 4096 + 2 * kCompactCap) * sizeof(int64_t)) != cudaSuccess ||
        ctx->d_result.reserve(64) != cudaSuccess || ctx->d_totals.reserve(64) != cudaSuccess ||
        cudaMemset(ctx->d_status.p, 0, 64) != cudaSuccess || cudaMemset(ctx->d_totals.p, 0, 64) != cudaSuccess ||
        cudaHostAlloc(&ctx->h_pinned, 16 * sizeof(int64_t), cudaHostAllocMapped) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->planned, cudaEventDisableTiming) != cudaSuccess) {
        distsim_destroy(ctx);
        return DISTSIM_E_CUDA;
    }
    // the side stream is an optimisation: without it evaluations run on the caller's stream alone
    int prio_lo = 0, prio_hi = 0;
    if (cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi) != cudaSuccess ||
        cudaStreamCreateWithPriority(&ctx->side.side[0], cudaStreamNonBlocking, prio_hi) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->side.fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->side.join[0], cudaEventDisableTiming) != cudaSuccess) {
        cudaGetLastError();
        destroy_side(ctx->side);
    }
    *out = ctx;
    return DISTSIM_OK;
}

void distsim_destroy(distsim_ctx *ctx)
{
    if (!ctx) return;
    cudaSetDevice(ctx->device);
    for (cudaEvent_t e : ctx->phase_ev) if (e) cudaEventDestroy(e);
    if (ctx->planned) cudaEventDestroy(ctx->planned);
    if (ctx->h_pinned) cudaFreeHost(ctx->h_pinned);
    destroy_side(ctx->side);
    delete ctx;
}

const char *distsim_last_error(const distsim_ctx *ctx) { return ctx ? ctx->err.c_str() : "null context"; }

int64_t distsim_testing_launch_count(const distsim_ctx *ctx) { return ctx ? ctx->launches : 0; }

int distsim_load_event_table(distsim_ctx *ctx, const distsim_event_table *t)
{
    if (!ctx) return DISTSIM_E_ARG;
    if (!t) return fail(ctx, DISTSIM_E_ARG, "null table");
    if (!t->class_mp || !t->class_b || !t->fwd_ns || !t->bwd_ns || !t->layer_is_expert || !t->grad_bytes)
        return fail(ctx, DISTSIM_E_ARG, "null array in table");
    if (t->n_layers < 1 || t->n_layers > DISTSIM_MAX_LAYERS) return fail(ctx, DISTSIM_E_ARG, "n_layers out of range");
    if (t->n_classes < 1) return fail(ctx, DISTSIM_E_ARG, "no event classes");
    if (!is_pow2(t->n_devices) || !is_pow2(t->gpus_per_node))
        return fail(ctx, DISTSIM_E_UNSUPPORTED, "n_devices and gpus_per_node must be powers of two");
    if (t->global_batch < 1 || t->seq < 0 || t->hidden < 0 || t->act_bytes_per_elem < 0)
        return fail(ctx, DISTSIM_E_ARG, "negative size");
    if (t->allreduce_profile_max < 0 || t->allreduce_profile_max == 1 || t->reserved != 0)
        return fail(ctx, DISTSIM_E_ARG, "bad allreduce_profile_max");
    if (t->n_jitter < 0 || t->n_jitter > 64 || (t->n_jitter & (t->n_jitter - 1)))
        return fail(ctx, DISTSIM_E_UNSUPPORTED, "n_jitter must be 0 or a power of two <= 64");
    if (t->n_jitter > 0) {
        if (!t->jitter_fwd_ns || !t->jitter_bwd_ns || t->jitter_stages < 1 || t->jitter_stages > DISTSIM_MAX_PP)
            return fail(ctx, DISTSIM_E_ARG, "bad jitter tables");
        for (int64_t i = 0; i < (int64_t)t->n_jitter * t->jitter_stages; ++i)
            if (t->jitter_fwd_ns[i] < 0 || t->jitter_bwd_ns[i] < 0 || t->jitter_fwd_ns[i] >= kSat / 8192 ||
                t->jitter_bwd_ns[i] >= kSat / 8192)
                return fail(ctx, DISTSIM_E_ARG, "jitter out of range");
    }
    if (t->alpha_intra_ns < 0 || t->alpha_inter_ns < 0 || t->beta_intra < 1 || t->beta_inter < 1 || t->dp_bucket_bytes < 0)
        return fail(ctx, DISTSIM_E_ARG, "bad link constants");
    const int64_t L = t->n_layers, K = t->n_classes;
    for (int64_t i = 0; i < K * L; ++i)
        if (t->fwd_ns[i] < 0 || t->bwd_ns[i] < 0) return fail(ctx, DISTSIM_E_ARG, "negative event time");
    for (int64_t k = 0; k < K; ++k)
        if (t->class_mp[k] < 1 || t->class_b[k] < 1) return fail(ctx, DISTSIM_E_ARG, "bad event class");
    int64_t gsum = 0;
    for (int64_t l = 0; l < L; ++l) {
        if (t->grad_bytes[l] < 0) return fail(ctx, DISTSIM_E_ARG, "negative gradient size");
        gsum = sat_add(gsum, t->grad_bytes[l]);
    }
    if (gsum >= kSat / (4 * (int64_t)t->n_devices)) return fail(ctx, DISTSIM_E_OVERFLOW, "gradient volume too large");
    if (int rc = set_device(ctx)) return rc;

    ctx->table_loaded = false; ctx->space_set = false;
    TableConst &tc = ctx->tc;
    tc.n_layers = t->n_layers; tc.n_classes = t->n_classes; tc.n_devices = t->n_devices;
    tc.gpus_per_node = t->gpus_per_node; tc.global_batch = t->global_batch; tc.seq = t->seq;
    tc.hidden = t->hidden; tc.alpha_intra = t->alpha_intra_ns; tc.beta_intra = t->beta_intra;
    tc.alpha_inter = t->alpha_inter_ns; tc.beta_inter = t->beta_inter; tc.bucket = t->dp_bucket_bytes;
    tc.overlap = t->dp_overlap ? 1 : 0; tc.elem_bytes = t->act_bytes_per_elem;
    tc.lp = (int32_t)((L + 1 + 1) & ~1); tc.ar_profile_max = t->allreduce_profile_max;
    tc.n_jitter = t->n_jitter; tc.jitter_stages = t->n_jitter > 0 ? t->jitter_stages : 0;
    ctx->class_mp.assign(t->class_mp, t->class_mp + K);
    ctx->class_b.assign(t->class_b, t->class_b + K);
    ctx->fwd.assign(t->fwd_ns, t->fwd_ns + K * L);
    ctx->bwd.assign(t->bwd_ns, t->bwd_ns + K * L);
    ctx->grad.assign(t->grad_bytes, t->grad_bytes + L);
    ctx->expert.assign(t->layer_is_expert, t->layer_is_expert + L);

    if (int rc = upload(ctx, ctx->d_class_mp, ctx->class_mp.data(), K, "upload class_mp")) return rc;
    if (int rc = upload(ctx, ctx->d_class_b, ctx->class_b.data(), K, "upload class_b")) return rc;
    if (int rc = upload(ctx, ctx->d_fwd, ctx->fwd.data(), K * L, "upload fwd")) return rc;
    if (int rc = upload(ctx, ctx->d_bwd, ctx->bwd.data(), K * L, "upload bwd")) return rc;
    if (int rc = upload(ctx, ctx->d_expert, ctx->expert.data(), L, "upload expert")) return rc;
    if (int rc = upload(ctx, ctx->d_grad, ctx->grad.data(), L, "upload grad")) return rc;
    CU(ctx->d_next_grad.reserve((L + 1) * sizeof(int32_t)), "alloc next_grad");
    CU(ctx->d_pe.reserve((L + 1) * sizeof(int32_t)), "alloc pe");
    ctx->raw.class_mp = ctx->d_class_mp.as<int32_t>(); ctx->raw.class_b = ctx->d_class_b.as<int32_t>();
    ctx->raw.fwd = ctx->d_fwd.as<int64_t>(); ctx->raw.bwd = ctx->d_bwd.as<int64_t>();
    ctx->raw.expert = ctx->d_expert.as<uint8_t>(); ctx->raw.grad = ctx->d_grad.as<int64_t>();
    ctx->raw.jit_f = ctx->raw.jit_b = nullptr;
    if (t->n_jitter > 0) {
        const size_t nj = (size_t)t->n_jitter * t->jitter_stages;
        if (int rc = upload(ctx, ctx->d_jit_f, t->jitter_fwd_ns, nj, "upload jitter")) return rc;
        if (int rc = upload(ctx, ctx->d_jit_b, t->jitter_bwd_ns, nj, "upload jitter")) return rc;
        ctx->raw.jit_f = ctx->d_jit_f.as<int64_t>(); ctx->raw.jit_b = ctx->d_jit_b.as<int64_t>();
    }
    launch_build_layer_tables(0, tc, ctx->raw, ctx->d_next_grad.as<int32_t>(), ctx->d_pe.as<int32_t>(), &ctx->launches);
    CU(cudaGetLastError(), "layer tables launch");
    ctx->table_loaded = true;
    return DISTSIM_OK;
}

int distsim_set_space(distsim_ctx *ctx, const distsim_space *sp, int64_t *n_candidates)
{
    if (!ctx) return DISTSIM_E_ARG;
    if (!sp || !n_candidates) return fail(ctx, DISTSIM_E_ARG, "null argument");
    if (!ctx->table_loaded) return fail(ctx, DISTSIM_E_STATE, "no event table loaded");
    if (sp->mp_max < 1 || sp->pp_max < 1 || sp->n_m < 1 || !sp->m_list) return fail(ctx, DISTSIM_E_ARG, "empty space");
    if (sp->pp_max > DISTSIM_MAX_PP) return fail(ctx, DISTSIM_E_ARG, "pp_max too large");
    if ((sp->sched_mask & 31) == 0 || (sp->sched_mask & ~31)) return fail(ctx, DISTSIM_E_ARG, "bad sched_mask");
    if ((sp->sched_mask & 16) && sp->pp_max > 32)
        return fail(ctx, DISTSIM_E_UNSUPPORTED, "the bidirectional schedule is evaluated for at most 32 stages");
    if ((sp->sched_mask & 16) && ctx->tc.n_jitter > 0)
        return fail(ctx, DISTSIM_E_UNSUPPORTED, "the bidirectional schedule does not combine with per-micro-batch jitter");
    if ((sp->sched_mask & 8) && (sp->v_max < 2 || sp->v_max > DISTSIM_MAX_PP / 2))
        return fail(ctx, DISTSIM_E_ARG, "interleaved schedule needs 2 <= v_max <= 32");
    if ((sp->sched_mask & 8) && ctx->tc.n_jitter > 0)
        return fail(ctx, DISTSIM_E_UNSUPPORTED, "the interleaved schedule does not combine with per-micro-batch jitter");
    if (sp->m_rule < 0 || sp->m_rule > 1 || sp->partition_mode < 0 || sp->partition_mode > 1)
        return fail(ctx, DISTSIM_E_ARG, "bad m_rule or partition_mode");
    for (int i = 0; i < sp->n_m; ++i) {
        if (sp->m_list[i] < 1 || sp->m_list[i] > DISTSIM_MAX_M) return fail(ctx, DISTSIM_E_ARG, "m out of range");
        if (i && sp->m_list[i] <= sp->m_list[i - 1]) return fail(ctx, DISTSIM_E_ARG, "m_list must ascend");
    }
    if (int rc = set_device(ctx)) return rc;
    ctx->space_set = false;
    ctx->have_narrow = false;
    const TableConst &tc = ctx->tc;
    const int L = tc.n_layers;
    const int64_t N = tc.n_devices, B = tc.global_batch;

    std::map<std::pair<int, int>, int> class_of;
    for (int k = 0; k < tc.n_classes; ++k) class_of.emplace(std::make_pair(ctx->class_mp[k], ctx->class_b[k]), k);

    // binomials C(n, k), n < L, k < binom_k, saturated
    int pp_cap = 1;
    while (pp_cap * 2 <= sp->pp_max && pp_cap * 2 <= L) pp_cap *= 2;
    int bk = pp_cap;                                // most (virtual) stages of any candidate
    if (sp->sched_mask & 8)
        for (int pp = 2; pp <= pp_cap; pp *= 2)
            for (int vc = 2; vc <= sp->v_max && pp * vc <= DISTSIM_MAX_PP && pp * vc <= L; vc *= 2)
                if (pp * vc > bk) bk = pp * vc;
    std::vector<int64_t> binom((size_t)L * bk, 0);
    for (int n = 0; n < L; ++n)
        for (int k = 0; k < bk; ++k) {
            int64_t v;
            if (k == 0) v = 1;
            else if (n == 0) v = 0;
            else v = sat_add(binom[(size_t)(n - 1) * bk + k - 1], binom[(size_t)(n - 1) * bk + k]);
            binom[(size_t)n * bk + k] = v;
        }

    std::vector<Row> rows;
    std::vector<Entry> entries;
    int64_t total = 0, op_words = 0;
    long double tb = 0;
    int n_sched = 0, sched_list = 0;
    for (int id = 0; id < 3; ++id)
        if (sp->sched_mask & (1 << id)) sched_list |= id << (2 * n_sched++);
    long double fg_max = 0;                       // largest per-class sum of layer times
    for (int k = 0; k < tc.n_classes; ++k) {
        long double s = 0;
        for (int l = 0; l < L; ++l) s += (long double)ctx->fwd[(size_t)k * L + l] + ctx->bwd[(size_t)k * L + l];
        if (s > fg_max) fg_max = s;
    }
    long double gsum = 0;
    for (int l = 0; l < L; ++l) gsum += ctx->grad[l];
    const long double a_max = (long double)(tc.alpha_inter > tc.alpha_intra ? tc.alpha_inter : tc.alpha_intra);
    const long double b_min = (long double)(tc.beta_inter < tc.beta_intra ? tc.beta_inter : tc.beta_intra);

    for (int64_t mp = 1; mp <= sp->mp_max; mp *= 2)
        for (int64_t pp = 1; pp <= sp->pp_max && pp <= L; pp *= 2) {
            if (N % (mp * pp)) continue;
            const int64_t dp = N / (mp * pp);
            if (B % dp) continue;
            const int64_t Bp = B / dp;
            // the row of the plain schedules, then one row of interleaved candidates per chunk
            // count, then the row of bidirectional-pipeline candidates
            std::vector<std::pair<int64_t, bool>> kinds;          // (chunks per device, two_way)
            if (n_sched > 0) kinds.emplace_back(1, false);
            if ((sp->sched_mask & 8) && pp >= 2)
                for (int64_t vc = 2; vc <= sp->v_max && pp * vc <= DISTSIM_MAX_PP && pp * vc <= L; vc *= 2) kinds.emplace_back(vc, false);
            if ((sp->sched_mask & 16) && pp >= 2) kinds.emplace_back(1, true);
            for (const auto &kind : kinds) {
                const int64_t vc = kind.first;
                const bool two_way = kind.second;
                const bool plain = vc == 1 && !two_way;
                const int64_t P = pp * vc;              // (virtual) stages
                Row r{};
                r.mp = (int32_t)mp; r.pp = (int32_t)pp; r.dp = (int32_t)dp; r.log2_mp = floor_log2(mp);
                r.v = (int32_t)vc; r.two_way = two_way ? 1 : 0;
                r.entry0 = (int32_t)entries.size(); r.n_entries = 0;
                r.n_sched = plain ? n_sched : 1; r.sched_list = plain ? sched_list : 3;
                r.p2p_period = mp >= tc.gpus_per_node ? 1 : (int32_t)(tc.gpus_per_node / mp);
                r.n_part = sp->partition_mode == 0 ? 1 : binom[(size_t)(L - 1) * bk + (P - 1)];
                for (int i = 0; i < sp->n_m; ++i) {
                    const int64_t m = sp->m_list[i];
                    if (m > Bp) continue;
                    if (sp->m_rule == 0 && Bp % m) continue;
                    if (vc > 1 && m % pp) continue;     // the interleaved order needs whole groups of pp micro-batches
                    if (two_way && m % 2) continue;     // half of the micro-batches go each way
                    const int64_t b = (Bp + m - 1) / m;
                    auto it = class_of.find(std::make_pair((int)mp, (int)b));
                    if (it == class_of.end()) {
                        char msg[128];
                        snprintf(msg, sizeof msg, "event class (mp=%lld, b=%lld) is not in the table", (long long)mp, (long long)b);
                        return fail(ctx, DISTSIM_E_ARG, msg);
                    }
                    Entry en{};
                    en.m = (int32_t)m; en.b = (int32_t)b; en.cls = it->second; en.row = (int32_t)rows.size();
                    entries.push_back(en);
                    ++r.n_entries;
                    if (2 * m * P > op_words) op_words = 2 * m * P;
                    // generous upper bound on any batch time of this entry: every item in sequence
                    const long double act = (long double)b * tc.seq * tc.hidden * tc.elem_bytes;
                    const long double comm = 2.0L * mp * a_max + 4.0L * act / b_min + 2 + dp * a_max + act / b_min + 2;
                    const long double p2p = a_max + act / b_min + 2;
                    // (a device of a two_way row sends two streams of buckets, each over 2 dp devices)
                    const long double nbk = ((tc.bucket > 0 ? gsum / tc.bucket + L + 1 : L + 1) + vc) * (two_way ? 2 : 1);
                    const long double bsz = tc.bucket > 0 ? (long double)tc.bucket : gsum;
                    const long double e_bound = (long double)m * (fg_max + 2.0L * L * comm + 2.0L * P * p2p) +
                                                nbk * (2.0L * (two_way ? 2 : 1) * dp * a_max + 2.0L * bsz / b_min + 2);
                    if (e_bound > tb) tb = e_bound;
                }
                if (r.n_entries == 0) continue;
                r.size = sat_mul(sat_mul(r.n_part, r.n_entries), r.n_sched);
                r.offset = total;
                r.row_tab_off = (int64_t)rows.size() * (((L + 1) * (L + 1) + 1) & ~1);   // even: 16-byte aligned tables
                total = sat_add(total, r.size);
                if (r.n_part >= kSat || total >= kSat) return fail(ctx, DISTSIM_E_OVERFLOW, "candidate count does not fit 62 bits");
                rows.push_back(r);
            }
        }
    if (rows.empty()) return fail(ctx, DISTSIM_E_ARG, "the space has no valid candidate");
    if (tc.n_jitter > 0)
        for (const Row &r : rows)
            if (r.pp > tc.jitter_stages) return fail(ctx, DISTSIM_E_ARG, "a strategy has more stages than the jitter tables have columns");
    if (tb >= (long double)kSat) return fail(ctx, DISTSIM_E_OVERFLOW, "batch-time bound does not fit 62 bits");

    ctx->rows = rows; ctx->entries = entries; ctx->binom = binom;
    ctx->time_bound = (int64_t)tb + 1;
    ctx->op_words_per_cand = op_words;
    ctx->ilv_words = 0;
    for (const Row &r : rows)
        if (r.v > 1 && interleaved_words_of(r.pp, r.v) > ctx->ilv_words) ctx->ilv_words = interleaved_words_of(r.pp, r.v);
    // item orders of the bidirectional rows: one per (pp, m), shared by the rows that differ in mp
    ctx->have_order = false;
    ctx->two_way_words = 0;
    {
        std::vector<uint16_t> all_orders;
        std::vector<uint32_t> all_before;
        std::vector<int64_t> order_off(entries.size(), 0);
        std::map<std::pair<int, int>, std::pair<int64_t, int>> made;       // (pp, m) -> (offset, kept items)
        for (const Row &r : rows) {
            if (!r.two_way) continue;
            for (int e = 0; e < r.n_entries; ++e) {
                const int m = entries[r.entry0 + e].m;
                auto it = made.find(std::make_pair((int)r.pp, m));
                if (it == made.end()) {
                    std::vector<uint16_t> one;
                    std::vector<uint32_t> one_before;
                    int kept = 0;
                    if (!bidirectional_orders(r.pp, m, one, one_before, &kept))
                        return fail(ctx, DISTSIM_E_STATE, "the bidirectional item order could not be built");
                    it = made.emplace(std::make_pair((int)r.pp, m), std::make_pair((int64_t)all_orders.size(), kept)).first;
                    all_orders.insert(all_orders.end(), one.begin(), one.end());
                    all_before.insert(all_before.end(), one_before.begin(), one_before.end());
                }
                order_off[r.entry0 + e] = it->second.first | ((int64_t)it->second.second << 48);
                if (it->second.second > bidirectional_kept_cap_of(r.pp))
                    return fail(ctx, DISTSIM_E_STATE, "the bidirectional item order keeps more items than the kernels allow for");
                const int words = bidirectional_words_of(r.pp, bidirectional_kept_cap_of(r.pp));
                if (words > ctx->two_way_words) ctx->two_way_words = words;
            }
        }
        if (!all_orders.empty()) {
            if (int rc = upload(ctx, ctx->d_order, all_orders.data(), all_orders.size(), "upload item orders")) return rc;
            if (int rc = upload(ctx, ctx->d_order_before, all_before.data(), all_before.size(), "upload item orders")) return rc;
            if (int rc = upload(ctx, ctx->d_order_off, order_off.data(), order_off.size(), "upload item orders")) return rc;
            ctx->have_order = true;
        }
    }
    SpaceConst &sc = ctx->sc;
    sc.n_rows = (int32_t)rows.size(); sc.n_entries = (int32_t)entries.size();
    sc.pp_max = sp->pp_max; sc.partition_mode = sp->partition_mode; sc.binom_k = bk; sc.pad = 0;
    sc.n_candidates = total;

    if (int rc = upload(ctx, ctx->d_rows, rows.data(), rows.size(), "upload rows")) return rc;
    if (int rc = upload(ctx, ctx->d_entries, entries.data(), entries.size(), "upload entries")) return rc;
    if (int rc = upload(ctx, ctx->d_binom, binom.data(), binom.size(), "upload binomials")) return rc;
    CU(ctx->d_etf.reserve(entries.size() * tc.lp * sizeof(int64_t)), "alloc prefix");
    CU(ctx->d_etb.reserve(entries.size() * tc.lp * sizeof(int64_t)), "alloc prefix");
    const size_t tab = rows.size() * (size_t)(((L + 1) * (L + 1) + 1) & ~1) * sizeof(int64_t);
    CU(ctx->d_nb.reserve(tab), "alloc bucket tables");
    CU(ctx->d_tp.reserve(tab), "alloc bucket tables");
    launch_fill_entries(0, tc, ctx->d_rows.as<Row>(), sc.n_rows, ctx->d_entries.as<Entry>(), sc.n_entries, &ctx->launches);
    launch_build_prefix(0, tc, ctx->raw, ctx->d_entries.as<Entry>(), sc.n_entries, ctx->d_etf.as<int64_t>(),
                        ctx->d_etb.as<int64_t>(), &ctx->launches);
    launch_build_bucket_tables(0, tc, ctx->raw, ctx->d_rows.as<Row>(), sc.n_rows, ctx->d_nb.as<int64_t>(),
                               ctx->d_tp.as<int64_t>(), &ctx->launches);
    // per-entry bucket-lane tables, when the search enumerates stage compositions and they fit
    const size_t dt_bytes = entries.size() * (size_t)(((L + 1) * (L + 1) + 1) & ~1) * sizeof(int64_t);
    ctx->have_dt = sp->partition_mode == 1 && dt_bytes <= ((size_t)256 << 20);
    if (ctx->have_dt) CU(ctx->d_dt.reserve(dt_bytes), "alloc bucket-lane tables");
    if (tc.n_jitter > 0) CU(ctx->d_jsum.reserve(entries.size() * DISTSIM_MAX_PP * sizeof(int64_t)), "alloc jitter sums");
    launch_build_entry_tables(0, ctx->view(), ctx->d_entries.as<Entry>(), ctx->have_dt ? ctx->d_dt.as<int64_t>() : nullptr,
                              tc.n_jitter > 0 ? ctx->d_jsum.as<int64_t>() : nullptr, &ctx->launches);
    // 32-bit copies for the entries that are evaluated in 32-bit arithmetic
    ctx->have_narrow = false;
    {
        const size_t t32 = (size_t)(((L + 1) * (L + 1) + 3) & ~3);
        CU(ctx->d_pfb32.reserve(entries.size() * tc.lp * sizeof(uint2)), "alloc 32-bit prefix rows");
        if (ctx->have_dt) CU(ctx->d_dt32.reserve(entries.size() * t32 * sizeof(uint32_t)), "alloc 32-bit bucket-lane tables");
        launch_build_narrow_tables(0, ctx->view(), ctx->d_pfb32.as<uint2>(),
                                   ctx->have_dt ? ctx->d_dt32.as<uint32_t>() : nullptr, &ctx->launches);
        ctx->have_narrow = true;
    }
    CU(cudaGetLastError(), "set-up launch");
    // the host copies take the device-filled fields; these copies also wait for set-up
    CU(cudaMemcpy(ctx->rows.data(), ctx->d_rows.p, rows.size() * sizeof(Row), cudaMemcpyDeviceToHost), "rows readback");
    CU(cudaMemcpy(ctx->entries.data(), ctx->d_entries.p, entries.size() * sizeof(Entry), cudaMemcpyDeviceToHost), "entries readback");
    // the device's per-entry bounds are tighter than the host's estimate
    int64_t bmax = 0;
    for (const Entry &en : ctx->entries) bmax = en.bound > bmax ? en.bound : bmax;
    if (bmax >= kSat) return fail(ctx, DISTSIM_E_OVERFLOW, "batch-time bound does not fit 62 bits");
    ctx->time_bound = bmax;
    ctx->space_set = true;
    *n_candidates = total;
    return DISTSIM_OK;
}

int distsim_decode(distsim_ctx *ctx, int64_t index, distsim_candidate *out)
{
    if (!ctx) return DISTSIM_E_ARG;
    if (!out) return fail(ctx, DISTSIM_E_ARG, "null output");
    if (!ctx->space_set) return fail(ctx, DISTSIM_E_STATE, "no search space set");
    if (index < 0 || index >= ctx->sc.n_candidates) return fail(ctx, DISTSIM_E_RANGE, "candidate index out of range");
    size_t r = 0;
    while (r + 1 < ctx->rows.size() && ctx->rows[r + 1].offset <= index) ++r;
    const Row &row = ctx->rows[r];
    const int64_t local = index - row.offset;
    const int64_t per_entry = row.n_part * row.n_sched;
    const int64_t e = local / per_entry, rem = local % per_entry;
    int64_t rank = rem / row.n_sched;
    const Entry &en = ctx->entries[row.entry0 + e];
    memset(out, 0, sizeof *out);
    out->mp = row.mp; out->pp = row.pp; out->dp = row.dp; out->m = en.m;
    out->sched = row_sched(row, (int)(rem % row.n_sched));
    out->micro_batch_size = en.b; out->class_index = en.cls;
    out->v = row.v;
    const int L = ctx->tc.n_layers, pp = row.pp * row.v /* (virtual) stages */, bk = ctx->sc.binom_k;
    out->bounds[0] = 0; out->bounds[pp] = L;
    if (ctx->sc.partition_mode == 0) {
        for (int j = 1; j < pp; ++j) out->bounds[j] = (int32_t)((int64_t)j * L / pp);
    } else {
        int c = 0;
        for (int i = 1; i < pp; ++i) {
            ++c;
            while (true) {
                const int64_t cnt = ctx->binom[(size_t)(L - 1 - c) * bk + (pp - 1 - i)];
                if (rank < cnt) break;
                rank -= cnt; ++c;
            }
            out->bounds[i] = c;
        }
    }
    return DISTSIM_OK;
}

int distsim_eval_strategies(distsim_ctx *ctx, void *stream, int64_t first, int64_t count,
                            int64_t *d_batch_ns, int64_t *d_stage_busy_ns)
{
    if (!ctx) return DISTSIM_E_ARG;
    if (!ctx->space_set) return fail(ctx, DISTSIM_E_STATE, "no search space set");
    if (!d_batch_ns) return fail(ctx, DISTSIM_E_ARG, "null output");
    if (first < 0 || count < 0 || first > ctx->sc.n_candidates || count > ctx->sc.n_candidates - first)
        return fail(ctx, DISTSIM_E_RANGE, "candidate range outside the space");
    if (count == 0) return DISTSIM_OK;
    if (int rc = set_device(ctx)) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const DeviceView v = ctx->view();
    launch_eval(s, ctx->side, v, ctx->rows.data(), (int)ctx->rows.size(), ctx->entries.data(), first, count,
                d_batch_ns, d_stage_busy_ns, &ctx->launches);
    CU(cudaGetLastError(), "evaluation launch");
    return DISTSIM_OK;
}

int distsim_eval_select(distsim_ctx *ctx, void *stream, int64_t first, int64_t count, int64_t *d_batch_ns,
                        int32_t k, int64_t *d_indices, int64_t *d_times, int64_t *d_best, int64_t *h_best_index,
                        int64_t *h_best_batch_ns)
{
    if (!ctx) return DISTSIM_E_ARG;
    if (!ctx->space_set) return fail(ctx, DISTSIM_E_STATE, "no search space set");
    if (!d_batch_ns || (!h_best_index != !h_best_batch_ns)) return fail(ctx, DISTSIM_E_ARG, "null argument");
    if (first < 0 || count < 1 || first > ctx->sc.n_candidates || count > ctx->sc.n_candidates - first)
        return fail(ctx, DISTSIM_E_RANGE, "candidate range outside the space");
    if (k < 0 || k > 4096 || k > count || (k > 0 && !d_indices))
        return fail(ctx, DISTSIM_E_ARG, "k must be in [0, min(count, 4096)] and d_indices non-null for k > 0");
    if (int rc = set_device(ctx)) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const DeviceView v = ctx->view();
    const SelectScratch sc = ctx->select_scratch();
    if (ctx->phase_timing) cudaEventRecord(ctx->phase_ev[0], s);
    launch_eval(s, ctx->side, v, ctx->rows.data(), (int)ctx->rows.size(), ctx->entries.data(), first, count,
                d_batch_ns, nullptr, &ctx->launches);
    CU(cudaGetLastError(), "evaluation launch");
    if (ctx->phase_timing) cudaEventRecord(ctx->phase_ev[1], s);
    const bool want_best = d_best || h_best_index;
    launch_select(s, d_batch_ns, first, count, k, ctx->time_bound, sc, want_best ? ctx->d_result.as<int64_t>() : nullptr,
                  d_indices, d_times, &ctx->launches);
    CU(cudaGetLastError(), "selection launch");
    if (d_best) {
        // (batch time, position) -> (batch time, candidate index)
        CU(cudaMemcpyAsync(d_best, ctx->d_result.p, 2 * sizeof(int64_t), cudaMemcpyDeviceToDevice, s), "best copy");
        launch_add_scalar(s, d_best + 1, first, &ctx->launches);
    }
    if (ctx->phase_timing) { cudaEventRecord(ctx->phase_ev[2], s); ctx->phase_valid = true; }
    if (!h_best_index) return DISTSIM_OK;              // nothing goes to the host: no synchronisation
    CU(cudaMemcpyAsync(ctx->h_pinned, ctx->d_result.p, 2 * sizeof(int64_t), cudaMemcpyDeviceToHost, s), "argmin readback");
    bool stalled = false;
    if (int rc = read_status(ctx, s, &stalled)) return rc;          // synchronises
    *h_best_batch_ns = ctx->h_pinned[0];
    *h_best_index = first + ctx->h_pinned[1];
    return stalled ? fail(ctx, DISTSIM_E_TIMEOUT, kTimeoutText) : DISTSIM_OK;
}

int distsim_argmin(distsim_ctx *ctx, void *stream, const int64_t *d_batch_ns, int64_t first,
                   int64_t count, int64_t *h_best_index, int64_t *h_best_batch_ns)
{
    if (!ctx) return DISTSIM_E_ARG;
    if (!ctx->space_set) return fail(ctx, DISTSIM_E_STATE, "no search space set");
    if (!d_batch_ns || !h_best_index || !h_best_batch_ns) return fail(ctx, DISTSIM_E_ARG, "null argument");
    if (count < 1 || first < 0) return fail(ctx, DISTSIM_E_RANGE, "empty range");
    if (int rc = set_device(ctx)) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    launch_argmin(s, d_batch_ns, count, ctx->time_bound, ctx->select_scratch(), ctx->d_result.as<int64_t>(), &ctx->launches);
    CU(cudaGetLastError(), "argmin launch");
    CU(cudaMemcpyAsync(ctx->h_pinned, ctx->d_result.p, 2 * sizeof(int64_t), cudaMemcpyDeviceToHost, s), "argmin readback");
    bool stalled = false;
    if (int rc = read_status(ctx, s, &stalled)) return rc;          // synchronises
    *h_best_batch_ns = ctx->h_pinned[0];
    *h_best_index = first + ctx->h_pinned[1];
    return stalled ? fail(ctx, DISTSIM_E_TIMEOUT, kTimeoutText) : DISTSIM_OK;
}

int distsim_topk(distsim_ctx *ctx, void *stream, const int64_t *d_batch_ns, int64_t first,
                 int64_t count, int32_t k, int64_t *d_indices, int64_t *d_times)
{
    if (!ctx) return DISTSIM_E_ARG;
    if (!ctx->space_set) return fail(ctx, DISTSIM_E_STATE, "no search space set");
    if (!d_batch_ns || !d_indices) return fail(ctx, DISTSIM_E_ARG, "null argument");
    if (count < 1 || first < 0) return fail(ctx, DISTSIM_E_RANGE, "empty range");
    if (k < 1 || k > 4096 || k > count) return fail(ctx, DISTSIM_E_ARG, "k must be in [1, min(count, 4096)]");
    if (int rc = set_device(ctx)) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    launch_topk(s, d_batch_ns, first, count, k, ctx->time_bound, ctx->select_scratch(), d_indices, d_times, &ctx->launches);
    CU(cudaGetLastError(), "top-k launch");
    return DISTSIM_OK;
}

int distsim_merge_topk(distsim_ctx *ctx, void *stream, const int64_t *d_times_in, const int64_t *d_indices_in,
                       int64_t n, int32_t k, int64_t *d_indices, int64_t *d_times)
{
    if (!ctx) return DISTSIM_E_ARG;
    if (!d_times_in || !d_indices_in || !d_indices) return fail(ctx, DISTSIM_E_ARG, "null argument");
    if (k < 1 || k > 4096 || k > n) return fail(ctx, DISTSIM_E_ARG, "k must be in [1, min(n, 4096)]");
    if (int rc = set_device(ctx)) return rc;
    launch_merge_pairs(static_cast<cudaStream_t>(stream), d_times_in, d_indices_in, n, k, ctx->select_scratch(),
                       d_indices, d_times, &ctx->launches);
    CU(cudaGetLastError(), "merge launch");
    return DISTSIM_OK;
}

int distsim_emit_timelines(distsim_ctx *ctx, void *stream, const int64_t *d_indices, int32_t n,
                           distsim_record *d_records, int64_t capacity_records, int64_t *d_offsets,
                           int64_t *d_busy_ns, double *d_util, int64_t *h_total_records)
{
    if (!ctx) return DISTSIM_E_ARG;
    if (!ctx->space_set) return fail(ctx, DISTSIM_E_STATE, "no search space set");
    if (!d_indices || !h_total_records) return fail(ctx, DISTSIM_E_ARG, "null argument");
    if (n < 1 || n > 65535) return fail(ctx, DISTSIM_E_ARG, "n must be in [1, 65535]");
    if (d_records && capacity_records < 0) return fail(ctx, DISTSIM_E_ARG, "negative capacity");
    if (int rc = set_device(ctx)) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CU(ctx->d_plans.reserve((size_t)n * sizeof(EmitPlan)), "alloc emission plans");
    CU(ctx->d_op_start.reserve((size_t)n * ctx->op_words_per_cand * sizeof(int64_t)), "alloc item start times");
    CU(ctx->d_plan_sums.reserve((size_t)n * kEmitSumWords * sizeof(int64_t)), "alloc plan summaries");
    const DeviceView v = ctx->view();
    launch_emit_plan(s, v, d_indices, n, ctx->d_plans.as<EmitPlan>(), ctx->d_op_start.as<int64_t>(),
                     ctx->op_words_per_cand, ctx->d_plan_sums.as<int64_t>(), d_offsets, d_busy_ns, d_util, ctx->d_totals.as<int64_t>(),
                     std::max(ctx->ilv_words, ctx->two_way_words),
                     ctx->h_pinned + 8, ctx->planned, &ctx->launches);
    CU(cudaGetLastError(), "emission planning launch");
    // The planning kernel's last block writes the totals and the status word straight into the
    // pinned words; the host waits for that kernel only, not for the per-device words behind it.
    static_assert(sizeof(EmitTotals) == 8 * sizeof(int64_t), "totals occupy the second half of the pinned words");
    const EmitTotals *totals = reinterpret_cast<const EmitTotals *>(ctx->h_pinned + 8);
    CU(cudaEventSynchronize(ctx->planned), "planning sync");
    bool stalled = false;
    if (int rc = take_status(ctx, s, (int32_t)ctx->h_pinned[8 + 7], &stalled)) return rc;
    *h_total_records = totals->records;
    ctx->last_plan = *totals; ctx->have_last_plan = true;
    if (d_records) {
        if (totals->records > capacity_records) return fail(ctx, DISTSIM_E_CAPACITY, "record buffer too small");
        launch_emit_records(s, ctx->side, v, n, ctx->d_plans.as<EmitPlan>(), ctx->d_op_start.as<int64_t>(),
                            ctx->op_words_per_cand, *totals, d_records, &ctx->launches);
        CU(cudaGetLastError(), "emission launch");
    }
    // the records are written in stream order
    return stalled ? fail(ctx, DISTSIM_E_TIMEOUT, kTimeoutText) : DISTSIM_OK;
}

int distsim_emit_shape_of_last_plan(distsim_ctx *ctx, distsim_emit_shape *h_shape)
{
    if (!ctx) return DISTSIM_E_ARG;
    if (!h_shape) return fail(ctx, DISTSIM_E_ARG, "null argument");
    if (!ctx->have_last_plan) return fail(ctx, DISTSIM_E_STATE, "no timelines have been planned yet");
    const EmitTotals &t = ctx->last_plan;
    h_shape->records = t.records; h_shape->item_tiles = t.item_tiles; h_shape->bucket_tiles = t.bucket_tiles;
    h_shape->tmpl_words = t.tmpl_words; h_shape->bucket_recs = t.bucket_recs; h_shape->run_words = t.run_words;
    return DISTSIM_OK;
}

int distsim_emit_timelines_async(distsim_ctx *ctx, void *stream, const int64_t *d_indices, int32_t n,
                                 distsim_record *d_records, int64_t capacity_records,
                                 const distsim_emit_shape *h_shape,
                                 int64_t *d_offsets, int64_t *d_busy_ns, double *d_util)
{
    if (!ctx) return DISTSIM_E_ARG;
    if (!ctx->space_set) return fail(ctx, DISTSIM_E_STATE, "no search space set");
    if (!d_indices || !d_records || !h_shape) return fail(ctx, DISTSIM_E_ARG, "null argument");
    if (n < 1 || n > 65535) return fail(ctx, DISTSIM_E_ARG, "n must be in [1, 65535]");
    if (capacity_records < 0) return fail(ctx, DISTSIM_E_ARG, "negative capacity");
    // what one launch can be given: the grids' first dimension, the item kernel's shared memory
    // (two images of a run and the templates) and the bucket kernel's
    const int64_t item_smem = (2 * ((h_shape->run_words + 1) & ~(int64_t)1) + 2 + h_shape->tmpl_words) * 8;
    if (h_shape->records < 0 || h_shape->item_tiles < 0 || h_shape->item_tiles > 0x7fffffff ||
        h_shape->bucket_tiles < 0 || h_shape->bucket_tiles > 0x7fffffff || h_shape->tmpl_words < 0 ||
        h_shape->bucket_recs < 0 || h_shape->run_words < 0 || item_smem > 227 * 1024)
        return fail(ctx, DISTSIM_E_ARG, "the shape asks for more than a launch can be given");
    if (int rc = set_device(ctx)) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CU(ctx->d_plans.reserve((size_t)n * sizeof(EmitPlan)), "alloc emission plans");
    CU(ctx->d_op_start.reserve((size_t)n * ctx->op_words_per_cand * sizeof(int64_t)), "alloc item start times");
    CU(ctx->d_plan_sums.reserve((size_t)n * kEmitSumWords * sizeof(int64_t)), "alloc plan summaries");
    const DeviceView v = ctx->view();
    EmitTotals lim{};
    lim.records = capacity_records;           // (shape.records is the sizing pass's count, for the caller's buffer)
    lim.item_tiles = h_shape->item_tiles; lim.bucket_tiles = h_shape->bucket_tiles; lim.tmpl_words = h_shape->tmpl_words;
    lim.bucket_recs = h_shape->bucket_recs; lim.run_words = h_shape->run_words;
    launch_emit_plan(s, v, d_indices, n, ctx->d_plans.as<EmitPlan>(), ctx->d_op_start.as<int64_t>(),
                     ctx->op_words_per_cand, ctx->d_plan_sums.as<int64_t>(), nullptr, nullptr, nullptr, ctx->d_totals.as<int64_t>(),
                     std::max(ctx->ilv_words, ctx->two_way_words), nullptr, nullptr, &ctx->launches, &lim);
    CU(cudaGetLastError(), "emission planning launch");
    // the record kernels are sized by the shape; they write only if the plans stay within it
    // (the per-device words are written beside them: nothing waits for those)
    const EmitDeviceWords words{d_offsets, d_busy_ns, d_util, ctx->d_totals.as<int64_t>()};
    launch_emit_records(s, ctx->side, v, n, ctx->d_plans.as<EmitPlan>(), ctx->d_op_start.as<int64_t>(),
                        ctx->op_words_per_cand, lim, d_records, &ctx->launches, ctx->d_totals.as<int64_t>(), &words);
    CU(cudaGetLastError(), "emission launch");
    return DISTSIM_OK;
}

int distsim_checksum_timelines(distsim_ctx *ctx, void *stream, const distsim_record *d_records,
                               const int64_t *d_offsets, int64_t n_lists, uint64_t *d_checksums)
{
    if (!ctx) return DISTSIM_E_ARG;
    if (!d_records || !d_offsets || !d_checksums) return fail(ctx, DISTSIM_E_ARG, "null argument");
    if (n_lists < 0) return fail(ctx, DISTSIM_E_ARG, "negative list count");
    if (int rc = set_device(ctx)) return rc;
    launch_checksum_lists(static_cast<cudaStream_t>(stream), d_records, d_offsets, n_lists, d_checksums, &ctx->launches);
    CU(cudaGetLastError(), "checksum launch");
    return DISTSIM_OK;
}

int distsim_search_host(distsim_ctx *ctx, const distsim_event_table *h_table, const distsim_space *h_space,
                        int32_t k, int64_t *h_n_candidates, int64_t *h_best_index,
                        int64_t *h_best_batch_ns, int64_t *h_topk_indices, int64_t *h_topk_times)
{
    if (!ctx) return DISTSIM_E_ARG;
    if (!h_n_candidates || !h_best_index || !h_best_batch_ns) return fail(ctx, DISTSIM_E_ARG, "null argument");
    if (k < 0 || (k > 0 && (!h_topk_indices || !h_topk_times))) return fail(ctx, DISTSIM_E_ARG, "bad top-k arguments");
    if (int rc = distsim_load_event_table(ctx, h_table)) return rc;
    int64_t n = 0;
    if (int rc = distsim_set_space(ctx, h_space, &n)) return rc;
    *h_n_candidates = n;
    CU(ctx->d_batch.reserve((size_t)n * sizeof(int64_t)), "alloc batch times");
    int64_t *d_batch = ctx->d_batch.as<int64_t>();
    if (k > n) k = (int32_t)n;
    if (k > 4096) k = 4096;
    int64_t *d_idx = nullptr;
    if (k > 0) {
        CU(ctx->d_topk.reserve((size_t)2 * k * sizeof(int64_t)), "alloc top-k");
        d_idx = ctx->d_topk.as<int64_t>();
    }
    const int rc = distsim_eval_select(ctx, nullptr, 0, n, d_batch, k, d_idx, d_idx ? d_idx + k : nullptr, nullptr,
                                       h_best_index, h_best_batch_ns);          // synchronises
    if (rc != DISTSIM_OK && rc != DISTSIM_E_TIMEOUT) return rc;
    if (k > 0) {
        CU(cudaMemcpy(h_topk_indices, d_idx, (size_t)k * sizeof(int64_t), cudaMemcpyDeviceToHost), "top-k readback");
        CU(cudaMemcpy(h_topk_times, d_idx + k, (size_t)k * sizeof(int64_t), cudaMemcpyDeviceToHost), "top-k readback");
    }
    return rc;
}

int distsim_testing_space_cells(distsim_ctx *ctx, int64_t *h_cells, int64_t *h_cells_32bit)
{
    if (!ctx) return DISTSIM_E_ARG;
    if (!h_cells || !h_cells_32bit) return fail(ctx, DISTSIM_E_ARG, "null argument");
    if (!ctx->space_set) return fail(ctx, DISTSIM_E_STATE, "no search space set");
    __int128 total = 0, narrow = 0;
    for (const Row &row : ctx->rows)
        for (int e = 0; e < row.n_entries; ++e) {
            const Entry &en = ctx->entries[row.entry0 + e];
            const __int128 c = (__int128)2 * en.m * row.pp * row.v * row.n_part * row.n_sched;
            total += c;
            // 32-bit arithmetic is used where the entry's time bound allows it and the row is
            // evaluated by the one-partition-per-thread kernel
            if (en.bound < ((int64_t)1 << 32) && row.pp <= 16 && row.v == 1 && !row.two_way) narrow += c;
        }
    *h_cells = total >= (__int128)kSat ? kSat : (int64_t)total;
    *h_cells_32bit = narrow >= (__int128)kSat ? kSat : (int64_t)narrow;
    return DISTSIM_OK;
}

int64_t distsim_testing_lockstep_pieces(int32_t pp, int64_t lo, int64_t hi, int64_t max_blocks, int64_t max_pieces,
                                        int64_t *h_lo, int64_t *h_hi, int32_t *h_blocks)
{
    if (pp < 1 || pp > DISTSIM_MAX_PP || (pp & (pp - 1)) || lo < 0 || hi < lo || max_blocks < 1 || max_pieces < 0 ||
        (max_pieces > 0 && (!h_lo || !h_hi || !h_blocks)))
        return DISTSIM_E_ARG;
    return lockstep_pieces(pp, lo, hi, max_blocks, max_pieces, h_lo, h_hi, h_blocks);
}

int distsim_testing_bidirectional_order(int32_t pp, int32_t m, uint16_t *h_order, int32_t *h_kept)
{
    if (pp < 2 || pp > 32 || (pp & 1) || m < 2 || m > DISTSIM_MAX_M || (m & 1) || !h_order || !h_kept) return DISTSIM_E_ARG;
    std::vector<uint16_t> order;
    std::vector<uint32_t> before;
    int kept = 0;
    if (!bidirectional_orders(pp, m, order, before, &kept)) return DISTSIM_E_ARG;
    for (int d = 0; d < pp; ++d)
        for (int k = 0; k < 2 * m; ++k) h_order[(size_t)d * 2 * m + k] = order[(size_t)d * (2 * m + 1) + k];
    *h_kept = kept;
    return DISTSIM_OK;
}

int distsim_testing_time_phases(distsim_ctx *ctx, int32_t enable)
{
    if (!ctx) return DISTSIM_E_ARG;
    if (int rc = set_device(ctx)) return rc;
    if (enable && !ctx->phase_ev[0])
        for (cudaEvent_t &e : ctx->phase_ev) CU(cudaEventCreate(&e), "event create");
    ctx->phase_timing = enable != 0;
    ctx->phase_valid = false;
    return DISTSIM_OK;
}

int distsim_testing_last_phase_ms(distsim_ctx *ctx, float *h_eval_ms, float *h_select_ms)
{
    if (!ctx) return DISTSIM_E_ARG;
    if (!h_eval_ms || !h_select_ms) return fail(ctx, DISTSIM_E_ARG, "null argument");
    if (!ctx->phase_valid) return fail(ctx, DISTSIM_E_STATE, "no timed distsim_eval_select call yet");
    CU(cudaEventElapsedTime(h_eval_ms, ctx->phase_ev[0], ctx->phase_ev[1]), "event time");
    CU(cudaEventElapsedTime(h_select_ms, ctx->phase_ev[1], ctx->phase_ev[2]), "event time");
    return DISTSIM_OK;
}

int distsim_testing_set_stage_wait_polls(distsim_ctx *ctx, int32_t polls)
{
    if (!ctx) return DISTSIM_E_ARG;
    if (polls < 0) return fail(ctx, DISTSIM_E_ARG, "negative poll count");
    ctx->stage_polls = polls;
    return DISTSIM_OK;
}

}  // extern "C"
