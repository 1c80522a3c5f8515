// Timeline emission: per-device event records (kind, layer, microbatch, start_ns, end_ns) of
// selected candidates, plus per-device activity time and utilisation.
//
//   emit_plan_kernel     one warp per selected candidate: decode it, run the lock-step recurrence
//                        while recording every item's start time into scratch, count records.
//   emit_scan_kernel     one block: exclusive scan of the per-candidate record totals.
//   emit_devices_kernel  per (candidate, device): record offset, activity time, utilisation.
//   emit_items_kernel    the bandwidth-bound part.  A block owns (candidate, stage, run of
//                        consecutive items, chunk of replicas).  It builds the stage's forward
//                        and backward item templates (records relative to the item's start) in
//                        shared memory once.  The run's records are contiguous in memory, so the
//                        block walks the run as one flat stream of int64 words: word x belongs to
//                        the item found by a search in the run's offset table, and its value is
//                        template word + {0, 0, microbatch, start, start}.  Consecutive threads
//                        write consecutive word pairs (16-byte stores, full-width warp stores
//                        whatever the item size) to each of the stage's mp*dp replicas, whose
//                        lists are identical.
//   emit_buckets_kernel  gradient-bucket records of every stage.
#include "recurrence.cuh"

namespace distsim {

namespace {

constexpr int kItemThreads = 256;
constexpr int kMaxTileItems = 128;  // most schedule items per block (a plan picks its own count)
constexpr int kTileWords = 16384;   // target size of a block's run, in int64 words per replica
constexpr int kTileReplicas = 8;    // replicas per block

__device__ __forceinline__ int find_row(const DeviceView &v, int64_t index)
{
    int lo = 0, hi = v.sc.n_rows - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (v.rows[mid].offset <= index) lo = mid; else hi = mid - 1;
    }
    return lo;
}

template <int S>
__device__ __forceinline__ void plan_candidate(const DeviceView &v, const Row &row, int row_index,
                                               int64_t index, EmitPlan *plan, int64_t *rec)
{
    const int lane = threadIdx.x & 31;
    const int wl = row.pp / S;
    const int seg_lane = lane % wl;
    const bool owner = lane < wl;          // the other segments of the warp shadow the same candidate
    const CandidateCoords cc = split_local(row, index - row.offset);
    const Entry en = v.entries[cc.entry];
    const int64_t *pf = v.etf + (int64_t)cc.entry * v.tc.lp;
    const int64_t *pb = v.etb + (int64_t)cc.entry * v.tc.lp;
    const int n_slots = 2 * (en.m + row.pp - 1);
    const StageResult<S> R = v.tc.n_jitter > 0
        ? lockstep_candidate<S, true, true>(v, row, en, cc.entry, pf, pb, cc.sched, cc.part_rank, seg_lane, wl,
                                            n_slots, owner ? rec : nullptr)
        : lockstep_candidate<S, true, false>(v, row, en, cc.entry, pf, pb, cc.sched, cc.part_rank, seg_lane, wl,
                                             n_slots, owner ? rec : nullptr);
    if (owner) {
        const int L1 = v.tc.n_layers + 1;
#pragma unroll
        for (int k = 0; k < S; ++k) {
            const int d = seg_lane * S + k;
            const int a = R.a[k], e = R.e[k];
            const int n_layers = e - a;
            const int n_exp = v.pe[e] - v.pe[a];
            const int64_t per_dir = (int64_t)n_layers * (row.mp > 1 ? 2 : 1) + (row.dp > 1 ? n_exp : 0) +
                                    (v.tc.n_jitter > 0 ? 1 : 0);      // an item starts with its jitter event
            const int64_t rf = per_dir + (d < row.pp - 1 ? 1 : 0);
            const int64_t rb = per_dir + (d > 0 ? 1 : 0);
            int64_t kb = 0;
            if (row.dp > 1) {
                const int64_t *nbt = v.nb + row.row_tab_off, *tpt = v.tp + row.row_tab_off;
                kb = nbt[(int64_t)e * L1 + a] + (tpt[(int64_t)e * L1 + a] > 0 ? 1 : 0);
            }
            plan->bounds[d] = a;
            if (d == row.pp - 1) plan->bounds[row.pp] = e;
            plan->rf[d] = (int32_t)rf; plan->rb[d] = (int32_t)rb;
            plan->n_buckets[d] = kb;
            plan->stage_recs[d] = (int64_t)en.m * (rf + rb) + kb;
            plan->busy[d] = R.busy[k];
            plan->main_end[d] = R.main_end[k];
            plan->last_b_start[d] = R.last_b_start[k];
        }
        if (lane == 0) {
            plan->index = index; plan->batch_ns = R.batch;
            plan->row = row_index; plan->entry = cc.entry; plan->m = en.m; plan->sched = cc.sched;
            plan->pp = row.pp; plan->mp = row.mp; plan->dp = row.dp; plan->ok = 1;
        }
    }
    __syncwarp();
    if (lane == 0) {
        int64_t acc = 0;
        for (int d = 0; d < row.pp; ++d) { plan->stage_rec_prefix[d] = acc; acc += plan->stage_recs[d]; }
        plan->stage_rec_prefix[row.pp] = acc;
        plan->rec_total = acc * row.mp * row.dp;
        int widest = 1;
        for (int d = 0; d < row.pp; ++d) widest = max(widest, plan->rf[d] + plan->rb[d]);
        const int per_tile = kTileWords / ((widest * 5 + 1) / 2);      // average item: (rf + rb) / 2 records
        plan->tile_items = max(8, min(kMaxTileItems, per_tile));
    }
}

__global__ void __launch_bounds__(128)
emit_plan_kernel(DeviceView v, const int64_t *__restrict__ indices, int n, EmitPlan *plans,
                 int64_t *op_start, int64_t op_words_per_cand)
{
    const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (i >= n) return;
    EmitPlan *plan = plans + i;
    const int64_t index = indices[i];
    if (index < 0 || index >= v.sc.n_candidates) {
        if ((threadIdx.x & 31) == 0) {
            plan->ok = 0; plan->rec_total = 0; plan->index = index; plan->pp = 0; plan->m = 0;
            plan->mp = 1; plan->dp = 1; plan->tile_items = 8;
            atomicCAS(v.status, 0, DISTSIM_E_RANGE);
        }
        return;
    }
    const int r = find_row(v, index);
    const Row row = v.rows[r];
    int64_t *rec = op_start + (int64_t)i * op_words_per_cand;
    if (row.pp > 32) plan_candidate<2>(v, row, r, index, plan, rec);
    else plan_candidate<1>(v, row, r, index, plan, rec);
}

// Exclusive scan of rec_total over the selections (n is small: one block, serial per chunk).
__global__ void emit_scan_kernel(EmitPlan *plans, int n, int64_t *totals /*[3]: records, max tiles, max bucket copies of a stage*/)
{
    __shared__ int64_t chunk_sum[1024];
    const int t = threadIdx.x, nt = blockDim.x;
    const int per = (n + nt - 1) / nt;
    const int b = min(n, t * per), e = min(n, b + per);
    int64_t s = 0, mt = 0, mb = 0;
    for (int i = b; i < e; ++i) s += plans[i].rec_total;
    chunk_sum[t] = s;
    __syncthreads();
    if (t == 0) {
        int64_t acc = 0;
        for (int k = 0; k < nt; ++k) { const int64_t x = chunk_sum[k]; chunk_sum[k] = acc; acc += x; }
        totals[0] = acc;
    }
    __syncthreads();
    int64_t acc = chunk_sum[t];
    for (int i = b; i < e; ++i) {
        plans[i].rec_base = acc; acc += plans[i].rec_total;
        if (plans[i].ok) {
            const int64_t reps = (int64_t)plans[i].mp * plans[i].dp;
            const int64_t tiles = (int64_t)plans[i].pp * ((2 * plans[i].m + plans[i].tile_items - 1) / plans[i].tile_items) *
                                  ((reps + kTileReplicas - 1) / kTileReplicas);
            mt = max64(mt, tiles);
            for (int d = 0; d < plans[i].pp; ++d) mb = max64(mb, plans[i].n_buckets[d] * reps);
        }
    }
    if (mt > 0) atomicMax((unsigned long long *)&totals[1], (unsigned long long)mt);
    if (mb > 0) atomicMax((unsigned long long *)&totals[2], (unsigned long long)mb);
}

__global__ void __launch_bounds__(256)
emit_devices_kernel(DeviceView v, const EmitPlan *__restrict__ plans, int n, int64_t *offsets,
                    int64_t *busy, double *util, const int64_t *totals)
{
    const int64_t N = v.tc.n_devices;
    const int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (g == 0 && offsets) offsets[(int64_t)n * N] = totals[0];
    if (g >= (int64_t)n * N) return;
    const int i = (int)(g / N);
    const int k = (int)(g - (int64_t)i * N);
    const EmitPlan &p = plans[i];
    if (!p.ok) {
        if (offsets) offsets[g] = p.rec_base;
        if (busy) busy[g] = 0;
        if (util) util[g] = 0.0;
        return;
    }
    const int q = k % p.mp, d = (k / p.mp) % p.pp, r = k / (p.mp * p.pp);
    if (offsets)
        offsets[g] = p.rec_base + (int64_t)r * p.mp * p.stage_rec_prefix[p.pp] +
                     (int64_t)p.mp * p.stage_rec_prefix[d] + (int64_t)q * p.stage_recs[d];
    if (busy) busy[g] = p.busy[d];
    if (util) util[g] = p.batch_ns > 0 ? (double)p.busy[d] / (double)p.batch_ns : 0.0;
}

// Position `s` in stage d's schedule order -> (is backward, micro-batch, items of each kind before it).
__device__ __forceinline__ void item_at(int sched, int pp, int m, int d, int s, bool &bwd, int &j, int &nf, int &nb)
{
    if (sched == 0) {
        if (s < m) { bwd = false; j = s; nf = s; nb = 0; }
        else { bwd = true; j = s - m; nf = m; nb = s - m; }
        return;
    }
    const int w = min(pp - d, m);
    if (s < w) { bwd = false; j = s; nf = s; nb = 0; }
    else if (s < 2 * m - w) {
        const int t = s - w;
        if (!(t & 1)) { bwd = true; j = t >> 1; nf = w + (t >> 1); nb = t >> 1; }
        else { bwd = false; j = w + (t >> 1); nf = w + (t >> 1); nb = (t >> 1) + 1; }
    } else { bwd = true; j = s - m; nf = m; nb = s - m; }
}

__global__ void __launch_bounds__(kItemThreads)
emit_items_kernel(DeviceView v, const EmitPlan *__restrict__ plans, const int64_t *__restrict__ op_start,
                  int64_t op_words_per_cand, int64_t *__restrict__ out /* records as flat words */)
{
    extern __shared__ __align__(16) int64_t tmpl[];     // [rf*5] forward, then [rb*5] backward
    __shared__ int64_t rep_off_s[kTileReplicas];
    __shared__ int64_t start_s[kMaxTileItems];          // start time of each item of the run
    __shared__ int32_t ioff[kMaxTileItems + 1];         // word offset of each item inside the run
    __shared__ int32_t meta_s[kMaxTileItems];           // micro-batch << 1 | is-backward
    __shared__ int64_t jit_s[kMaxTileItems];            // jitter at the start of each item
    const int i = blockIdx.y;
    const EmitPlan &p = plans[i];
    if (!p.ok) return;
    const int m = p.m, pp = p.pp, sched = p.sched, mp = p.mp;
    const int reps = mp * p.dp;
    const int tile_items = p.tile_items;
    const int item_chunks = (2 * m + tile_items - 1) / tile_items;
    const int rep_chunks = (reps + kTileReplicas - 1) / kTileReplicas;
    int tile = blockIdx.x;
    if (tile >= pp * item_chunks * rep_chunks) return;
    const int rc = tile % rep_chunks; tile /= rep_chunks;
    const int ic = tile % item_chunks;
    const int d = tile / item_chunks;

    const Row &row = v.rows[p.row];
    const Entry &en = v.entries[p.entry];
    const int a = p.bounds[d], e = p.bounds[d + 1];
    const int rf = p.rf[d], rb = p.rb[d];
    const int64_t *pf = v.etf + (int64_t)p.entry * v.tc.lp;
    const int64_t *pb = v.etb + (int64_t)p.entry * v.tc.lp;
    const int64_t *f = v.raw.fwd + (int64_t)en.cls * v.tc.n_layers;
    const int64_t *g = v.raw.bwd + (int64_t)en.cls * v.tc.n_layers;
    const int row_mp = row.mp, row_dp = row.dp;
    const int per_layer = row_mp > 1 ? 2 : 1;
    const int64_t ar = en.ar, a2a = en.a2a;
    int64_t *tf = tmpl, *tb = tmpl + (int64_t)rf * 5;
    const int jr = v.tc.n_jitter > 0 ? 1 : 0;           // record 0 of an item is its jitter event

    // ---- item templates: records relative to the end of the item's jitter event ----------
    if (jr && threadIdx.x == 32) {
        tf[0] = DISTSIM_JITTER_F; tf[1] = a; tf[2] = 0; tf[3] = 0; tf[4] = 0;
        tb[0] = DISTSIM_JITTER_B; tb[1] = e - 1; tb[2] = 0; tb[3] = 0; tb[4] = 0;
    }
    for (int l = a + threadIdx.x; l < e; l += blockDim.x) {
        const bool ex = row_dp > 1 && v.raw.expert[l];
        {   // forward: layers ascending
            const int r = jr + (l - a) * per_layer + (row_dp > 1 ? v.pe[l] - v.pe[a] : 0);
            int64_t t = pf[l] - pf[a];
            int64_t *w = tf + (int64_t)r * 5;
            w[0] = DISTSIM_COMPUTE_F; w[1] = l; w[2] = 0; w[3] = t; t += f[l]; w[4] = t; w += 5;
            if (row_mp > 1) { w[0] = DISTSIM_MP_AR_F; w[1] = l; w[2] = 0; w[3] = t; t += ar; w[4] = t; w += 5; }
            if (ex) { w[0] = DISTSIM_A2A_F; w[1] = l; w[2] = 0; w[3] = t; t += a2a; w[4] = t; }
        }
        {   // backward: layers descending
            const int r = jr + (e - 1 - l) * per_layer + (row_dp > 1 ? v.pe[e] - v.pe[l + 1] : 0);
            int64_t t = pb[e] - pb[l + 1];
            int64_t *w = tb + (int64_t)r * 5;
            w[0] = DISTSIM_COMPUTE_B; w[1] = l; w[2] = 0; w[3] = t; t += g[l]; w[4] = t; w += 5;
            if (row_mp > 1) { w[0] = DISTSIM_MP_AR_B; w[1] = l; w[2] = 0; w[3] = t; t += ar; w[4] = t; w += 5; }
            if (ex) { w[0] = DISTSIM_A2A_B; w[1] = l; w[2] = 0; w[3] = t; t += a2a; w[4] = t; }
        }
    }
    // ---- the run: its items' start times, kinds, micro-batches and word offsets ------------
    // an item's offset follows from how many forward / backward items precede it in the run
    const int s0 = ic * tile_items;
    const int n_items = min(2 * m, s0 + tile_items) - s0;
    bool bwd0; int j0, nf0, nb0;
    item_at(sched, pp, m, d, s0, bwd0, j0, nf0, nb0);
    if (threadIdx.x >= 64 && threadIdx.x < 64 + kMaxTileItems + 1) {
        const int k = threadIdx.x - 64;
        if (k <= n_items) {
            bool bwd; int j, nf, nb;
            item_at(sched, pp, m, d, s0 + k, bwd, j, nf, nb);       // k == n_items: one past the run
            ioff[k] = ((nf - nf0) * rf + (nb - nb0) * rb) * 5;
            if (k < n_items) {
                start_s[k] = op_start[(int64_t)i * op_words_per_cand + (int64_t)d * 2 * m + s0 + k];
                meta_s[k] = (j << 1) | (bwd ? 1 : 0);
                jit_s[k] = jitter_of(v, bwd ? v.raw.jit_b : v.raw.jit_f, j, d);
            }
        }
    }
    // word offset of every replica (r, q) of this tile relative to replica 0 of the stage
    const int rep0 = rc * kTileReplicas;
    const int n_rep = min(reps, rep0 + kTileReplicas) - rep0;
    if (threadIdx.x >= 32 && threadIdx.x < 32 + kTileReplicas) {
        const int k = threadIdx.x - 32;
        int64_t off = 0;
        if (k < n_rep) {
            const int rep = rep0 + k;
            const int r = rep / mp, q = rep - r * mp;
            off = (int64_t)r * mp * p.stage_rec_prefix[pp] * 5 + (int64_t)q * p.stage_recs[d] * 5;
        }
        rep_off_s[k] = off;
    }
    if (threadIdx.x == 0) {
        if (d < pp - 1) {
            int64_t *w = tf + (int64_t)(rf - 1) * 5;
            const int64_t t = pf[e] - pf[a];
            w[0] = DISTSIM_SEND_F; w[1] = e - 1; w[2] = 0; w[3] = t; w[4] = t + p2p_cost(row, en, d);
        }
        if (d > 0) {
            int64_t *w = tb + (int64_t)(rb - 1) * 5;
            const int64_t t = pb[e] - pb[a];
            w[0] = DISTSIM_SEND_B; w[1] = a; w[2] = 0; w[3] = t; w[4] = t + p2p_cost(row, en, d - 1);
        }
    }
    __syncthreads();

    // ---- stream the run as flat words ---------------------------------------------------------
    int64_t roff[kTileReplicas];                     // word offset of each replica of this tile
#pragma unroll
    for (int k = 0; k < kTileReplicas; ++k) roff[k] = rep_off_s[k];
    int64_t *run_out = out + (p.rec_base + (int64_t)mp * p.stage_rec_prefix[d]) * 5 +
                       ((int64_t)nf0 * rf + (int64_t)nb0 * rb) * 5;
    const int total = ioff[n_items];
    // Each pass covers 2 * blockDim.x consecutive words.  Records are 40 bytes, so a replica's
    // copy of the run starts on an even or an odd word; to write 16 bytes at a time to both
    // kinds, thread t prepares the words 2t-1, 2t and 2t+1 and stores the pair (2t, 2t+1) to
    // even-based replicas and the pair (2t-1, 2t) to odd-based ones (single words at the ends).
    unsigned odd_mask = 0;                           // bit k: replica k's copy starts on an odd word
#pragma unroll
    for (int k = 0; k < kTileReplicas; ++k)
        if (((reinterpret_cast<uintptr_t>(run_out + roff[k]) >> 3) & 1) != 0) odd_mask |= 1u << k;
    auto word = [&](int x, int it) -> int64_t {
        const int w = x - ioff[it];
        const int meta = meta_s[it];
        const int field = w - (w / 5) * 5;
        int64_t t = ((meta & 1) ? tb : tf)[w];
        // times: the jitter event runs [start, start + jitter); every later event is relative to its end
        if (field == 2) t += (int64_t)(meta >> 1);
        else if (field >= 3) t += start_s[it] + ((jr && w != 3) ? jit_s[it] : 0);
        return t;
    };
    // (x0 == total can occur: an odd-based replica's last word is then written by the thread at x == total)
    for (int x0 = 0; x0 <= total; x0 += 2 * kItemThreads) {
        const int x = x0 + 2 * threadIdx.x;          // the even word of this thread
        if (x - 1 >= total) break;
        int lo = 0, hi = n_items - 1;                // item holding word min(x, total-1)
        const int xs = min(x, total - 1);
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (ioff[mid] <= xs) lo = mid; else hi = mid - 1;
        }
        const bool has_m1 = x >= 1, has_0 = x < total, has_p1 = x + 1 < total;
        int64_t v_m1 = 0, v_0 = 0, v_p1 = 0;
        if (has_0) v_0 = word(x, lo);
        if (has_m1) v_m1 = word(x - 1, (has_0 && x == ioff[lo]) ? lo - 1 : lo);
        if (has_p1) v_p1 = word(x + 1, (x + 1 == ioff[lo + 1]) ? lo + 1 : lo);
#pragma unroll
        for (int k = 0; k < kTileReplicas; ++k) {
            if (k >= n_rep) continue;
            int64_t *dst = run_out + roff[k] + x;
            if (!((odd_mask >> k) & 1)) {            // (x, x+1) is 16-byte aligned
                if (has_p1) __stcs(reinterpret_cast<longlong2 *>(dst), make_longlong2(v_0, v_p1));
                else if (has_0) __stcs(dst, v_0);
            } else {                                 // (x-1, x) is 16-byte aligned
                if (has_m1 && has_0) __stcs(reinterpret_cast<longlong2 *>(dst - 1), make_longlong2(v_m1, v_0));
                else if (has_0) __stcs(dst, v_0);            // x == 0: the run's first word
                else if (has_m1) __stcs(dst - 1, v_m1);      // x == total: the run's last word
            }
        }
    }
}

// Gradient-bucket records: one warp per (selection, stage).  Buckets whose last byte lies in the
// same layer share a ready time, so once the first of them has started the rest follow back to
// back: per layer one serial step (lane 0), inside a layer a closed form (all lanes).
constexpr int kBucketWarps = 4;
__global__ void __launch_bounds__(kBucketWarps * 32)
emit_buckets_kernel(DeviceView v, const EmitPlan *__restrict__ plans, int n, int64_t *__restrict__ out)
{
    __shared__ int64_t g_start_s[kBucketWarps][DISTSIM_MAX_LAYERS + 1];   // start of the first bucket ending in layer a+i
    __shared__ int64_t g_first_s[kBucketWarps][DISTSIM_MAX_LAYERS + 1];   // number of that bucket
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t unit = (int64_t)blockIdx.x * kBucketWarps + warp;
    const int i = (int)(unit / v.sc.pp_max), d = (int)(unit % v.sc.pp_max);
    if (i >= n) return;
    const EmitPlan &p = plans[i];
    if (!p.ok || d >= p.pp || p.dp == 1) return;
    const int64_t kb = p.n_buckets[d];
    if (kb == 0) return;
    int64_t *g_start = g_start_s[warp], *g_first = g_first_s[warp];
    const Row &row = v.rows[p.row];
    const int a = p.bounds[d], e = p.bounds[d + 1];
    const int L1 = v.tc.n_layers + 1;
    const int64_t *nbe = v.nb + row.row_tab_off + (int64_t)e * L1;
    const int64_t part = v.tp[row.row_tab_off + (int64_t)e * L1 + a];
    const int64_t *pb = v.etb + (int64_t)p.entry * v.tc.lp;
    const int64_t n_full = nbe[a], t_full = row.t_full;
    int64_t part_start = 0;
    const int64_t tbs = p.last_b_start[d], main_end = p.main_end[d];
    // all lanes fetch the per-layer inputs (independent loads), then lane 0 runs the short chain
    for (int l = a + lane; l < e; l += 32) {
        g_first[l - a] = l + 1 < e ? nbe[l + 1] : 0;                       // buckets before layer l's group
        g_start[l - a] = v.tc.overlap ? tbs + (pb[e] - pb[l]) : main_end;    // ready time of the group
    }
    __syncwarp();
    if (lane == 0) {
        int64_t end = 0;
        for (int l = e - 1; l >= a; --l) {
            const int64_t nb_prev = g_first[l - a];
            const int64_t nb_l = l > a ? g_first[l - 1 - a] : n_full;       // nb[e][l]
            const int64_t start = max64(end, g_start[l - a]);
            g_start[l - a] = start;
            if (nb_l > nb_prev) end = start + (nb_l - nb_prev) * t_full;
        }
        if (part > 0) {
            const int ls = v.next_grad[a];
            const int64_t ready = v.tc.overlap ? tbs + (pb[e] - pb[ls]) : main_end;
            part_start = max64(end, ready);
        }
    }
    part_start = __shfl_sync(0xffffffffu, part_start, 0);
    __syncwarp();
    const int mp = p.mp, reps = mp * p.dp;
    // the stage's bucket words are cut into gridDim.y slices; a value is computed once and
    // written to every replica
    const int64_t per = ((kb * 5 + gridDim.y - 1) / gridDim.y + 31) & ~(int64_t)31;
    const int64_t w0 = (int64_t)blockIdx.y * per, w1 = min(kb * 5, w0 + per);
    const int64_t stage_words = p.stage_recs[d] * 5;
    const int64_t replica_words = (int64_t)mp * p.stage_rec_prefix[p.pp] * 5;
    int64_t *base = out + (p.rec_base + (int64_t)mp * p.stage_rec_prefix[d]) * 5 + (int64_t)p.m * (p.rf[d] + p.rb[d]) * 5;
    for (int64_t w = w0 + lane; w < w1; w += 32) {
        const int64_t k = w / 5;
        const int field = (int)(w - k * 5);
        int64_t val;
        if (field == 0) val = DISTSIM_DP_AR;
        else if (field == 1) val = k;
        else if (field == 2) val = -1;
        else {
            int64_t start, dur;
            if (k >= n_full) { start = part_start; dur = part; }
            else {
                // the layer whose group holds bucket k: the largest l with nb[e][l] > k
                // (nb[e][l] grows as l decreases, and nb[e][a] = n_full > k)
                int lo = a, hi = e - 1;
                while (lo < hi) {
                    const int mid = (lo + hi + 1) >> 1;
                    if (nbe[mid] > k) lo = mid; else hi = mid - 1;
                }
                start = g_start[lo - a] + (k - g_first[lo - a]) * t_full;
                dur = t_full;
            }
            val = field == 3 ? start : start + dur;
        }
        int r = 0, q = 0;
        int64_t *dst = base + w;
        for (int rep = 0; rep < reps; ++rep) {
            __stcs(dst, val);
            dst += stage_words;
            if (++q == mp) { q = 0; ++r; dst = base + w + (int64_t)r * replica_words; }
        }
    }
}

}  // namespace

void launch_emit_plan(cudaStream_t s, const DeviceView &v, const int64_t *d_indices, int n,
                      EmitPlan *plans, int64_t *op_start, int64_t op_words_per_cand,
                      int64_t *offsets, int64_t *busy, double *util, int64_t *d_totals,
                      int64_t *launches)
{
    cudaMemsetAsync(d_totals, 0, 3 * sizeof(int64_t), s);
    emit_plan_kernel<<<(n + 3) / 4, 128, 0, s>>>(v, d_indices, n, plans, op_start, op_words_per_cand);
    emit_scan_kernel<<<1, 1024, 0, s>>>(plans, n, d_totals);
    *launches += 2;
    if (offsets || busy || util) {
        const int64_t total = (int64_t)n * v.tc.n_devices + 1;
        emit_devices_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(v, plans, n, offsets, busy, util, d_totals);
        ++*launches;
    }
}

void launch_emit_records(cudaStream_t s, const DeviceView &v, int n, const EmitPlan *plans,
                         const int64_t *op_start, int64_t op_words_per_cand, int64_t max_tiles,
                         int64_t max_bucket_copies, distsim_record *records, int64_t *launches)
{
    if (n == 0 || max_tiles == 0) return;
    const size_t smem = (size_t)(2 * (3 * v.tc.n_layers + 1)) * 5 * sizeof(int64_t);
    static size_t smem_set = 0;
    if (smem > 48 * 1024 && smem > smem_set) {
        cudaFuncSetAttribute(emit_items_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        smem_set = smem;
    }
    int64_t *out = reinterpret_cast<int64_t *>(records);
    emit_items_kernel<<<dim3((unsigned)max_tiles, (unsigned)n), kItemThreads, smem, s>>>(
        v, plans, op_start, op_words_per_cand, out);
    ++*launches;
    if (v.tc.n_devices > 1) {
        const int64_t units = (int64_t)n * v.sc.pp_max;
        // stages with many bucket records times many replicas are cut into replica slices
        int64_t ny = (max_bucket_copies + 4095) / 4096;
        ny = ny < 1 ? 1 : (ny > 64 ? 64 : ny);
        emit_buckets_kernel<<<dim3((unsigned)((units + kBucketWarps - 1) / kBucketWarps), (unsigned)ny), kBucketWarps * 32, 0, s>>>(v, plans, n, out);
        ++*launches;
    }
}

}  // namespace distsim
