// Set-up kernels: turn the raw event table into the device tables the hot kernels read.
// They run once per (table, search space), so they favour clarity over speed; every
// division of the communication cost model happens here and none in the hot kernels.
#include "engine.h"
#include "costs.cuh"

namespace distsim {

namespace {

// One thread per entry: the communication-event costs that depend on (mp, dp, b).
// The first thread of each row also fills the row's full-bucket cost.
__global__ void fill_entries_kernel(TableConst tc, Row *rows, int n_rows, Entry *entries, int n_entries)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_entries) return;
    Entry en = entries[i];
    const Row row = rows[en.row];
    const int64_t act = (int64_t)en.b * tc.seq * tc.hidden * tc.elem_bytes;
    // a collective is intra-node iff all members share a node: for power-of-two degrees an MP
    // group of aligned consecutive ranks fits a node iff mp <= G; a DP group has stride mp*pp
    // and spans nodes whenever the cluster has more than one node
    const bool mp_inter = row.mp > tc.gpus_per_node;
    const bool dp_inter = tc.n_devices > tc.gpus_per_node;
    en.ar = 0;
    if (row.mp > 1)
        en.ar = allreduce_cost(tc, row.mp, 2 * act, mp_inter ? tc.alpha_inter : tc.alpha_intra,
                          mp_inter ? tc.beta_inter : tc.beta_intra);
    en.a2a = 0;
    if (row.dp > 1) {
        const int64_t a = dp_inter ? tc.alpha_inter : tc.alpha_intra;
        const int64_t be = dp_inter ? tc.beta_inter : tc.beta_intra;
        en.a2a = (row.dp - 1) * a + ceil_div((int64_t)(row.dp - 1) * act, (int64_t)row.dp * be);
    }
    en.p2p_intra = tc.alpha_intra + ceil_div(act, tc.beta_intra);
    en.p2p_inter = tc.alpha_inter + ceil_div(act, tc.beta_inter);
    entries[i] = en;
    if (i == row.entry0) {
        int64_t t_full = 0, t_full_near = 0;
        if (row.two_way) {
            // a stage's gradients are reduced over its 2 dp holders: across nodes, or inside one
            if (tc.bucket > 0) {
                t_full = allreduce_cost(tc, 2 * (int64_t)row.dp, tc.bucket, tc.alpha_inter, tc.beta_inter);
                t_full_near = allreduce_cost(tc, 2 * (int64_t)row.dp, tc.bucket, tc.alpha_intra, tc.beta_intra);
            }
        } else if (row.dp > 1 && tc.bucket > 0) {
            t_full = allreduce_cost(tc, row.dp, tc.bucket, dp_inter ? tc.alpha_inter : tc.alpha_intra,
                               dp_inter ? tc.beta_inter : tc.beta_intra);
        }
        rows[en.row].t_full = t_full;
        rows[en.row].t_full_near = t_full_near;
    }
}

// One thread per entry: exclusive prefix sums of the layer composites.
__global__ void build_prefix_kernel(TableConst tc, RawTable raw, const Entry *entries, int n_entries,
                                    int64_t *etf, int64_t *etb)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_entries) return;
    const Entry en = entries[i];
    const int64_t *f = raw.fwd + (int64_t)en.cls * tc.n_layers;
    const int64_t *g = raw.bwd + (int64_t)en.cls * tc.n_layers;
    int64_t *pf = etf + (int64_t)i * tc.lp;
    int64_t *pb = etb + (int64_t)i * tc.lp;
    int64_t sf = 0, sb = 0;
    for (int l = 0; l < tc.n_layers; ++l) {
        pf[l] = sf; pb[l] = sb;
        const int64_t comm = en.ar + (raw.expert[l] ? en.a2a : 0);
        sf += f[l] + comm;
        sb += g[l] + comm;
    }
    for (int l = tc.n_layers; l < tc.lp; ++l) { pf[l] = sf; pb[l] = sb; }
}

// One thread per (row, e): for a stage that ends at layer e (exclusive) and starts at layer l,
// the gradient stream is layers e-1, e-2, .., l with ceil(grad/mp) bytes each.
//   nb[e][l] = full buckets completed by the time layer l has produced its gradients
//   tp[e][l] = cost of the partial bucket left over for the stage [l, e)  (0 if none)
// With bucket size 0 the whole stage is one bucket: nb = 0 and tp = its cost.
__global__ void build_bucket_tables_kernel(TableConst tc, RawTable raw, const Row *rows, int n_rows,
                                           int64_t *nb, int64_t *tp)
{
    const int L1 = tc.n_layers + 1;
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_rows * L1) return;
    const int r = i / L1, e = i % L1;
    const Row row = rows[r];
    int64_t *nbr = nb + row.row_tab_off + (int64_t)e * L1;
    int64_t *tpr = tp + row.row_tab_off + (int64_t)e * L1;
    const bool dp_inter = tc.n_devices > tc.gpus_per_node;
    const int64_t a = dp_inter ? tc.alpha_inter : tc.alpha_intra;
    const int64_t be = dp_inter ? tc.beta_inter : tc.beta_intra;
    int64_t w = 0;
    for (int l = e; l >= 0; --l) {
        if (l < e) w += ceil_div(raw.grad[l], row.mp);
        int64_t full = 0, rem = w;
        if (tc.bucket > 0) { full = w / tc.bucket; rem = w - full * tc.bucket; }
        nbr[l] = full;
        // (a two_way row keeps the bytes of the trailing bucket: its cost depends on the device)
        tpr[l] = row.two_way ? rem : (rem > 0 && row.dp > 1) ? allreduce_cost(tc, row.dp, rem, a, be) : 0;
    }
    for (int l = e + 1; l < L1; ++l) { nbr[l] = 0; tpr[l] = 0; }
}

// next_grad[l] = smallest l' >= l whose gradient is non-empty (n_layers if none);
// pe[l] = number of expert layers before layer l.
__global__ void build_layer_tables_kernel(TableConst tc, RawTable raw, int32_t *next_grad, int32_t *pe)
{
    if (blockIdx.x != 0 || threadIdx.x != 0) return;
    int nxt = tc.n_layers;
    next_grad[tc.n_layers] = nxt;
    for (int l = tc.n_layers - 1; l >= 0; --l) {
        if (raw.grad[l] > 0) nxt = l;
        next_grad[l] = nxt;
    }
    int acc = 0;
    for (int l = 0; l < tc.n_layers; ++l) { pe[l] = acc; acc += raw.expert[l] ? 1 : 0; }
    pe[tc.n_layers] = acc;
}

// One thread per (entry, e): bucket-lane table row e of the entry.
//   overlap: DT[e][l] = max over the bucket groups of the stage [l, e) of (ready offset of the
//            group + cost of all buckets from that group on), offsets counted from the start of
//            the stage's last backward item; -1 when the stage has no buckets.
//   no overlap: total bucket cost of the stage.
__global__ void build_dt_kernel(DeviceView v, int64_t *dt)
{
    const int L1 = v.tc.n_layers + 1;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= v.sc.n_entries * L1) return;
    const int en_i = i / L1, e = i % L1;
    const Entry &en = v.entries[en_i];
    const Row &row = v.rows[en.row];
    int64_t *out = dt + (int64_t)en_i * v.tab_words + (int64_t)e * L1;
    const int64_t *nbe = v.nb + row.row_tab_off + (int64_t)e * L1;
    const int64_t *tpe = v.tp + row.row_tab_off + (int64_t)e * L1;
    const int64_t *pb = v.etb + (int64_t)en_i * v.tc.lp;
    for (int l = e; l < L1; ++l) out[l] = -1;
    if (row.dp == 1) { for (int l = 0; l < e; ++l) out[l] = v.tc.overlap ? -1 : 0; return; }
    for (int a = 0; a < e; ++a) {
        const int64_t n_full = nbe[a], partial = tpe[a];
        int64_t val;
        if (!v.tc.overlap) {
            val = n_full * row.t_full + partial;
        } else {
            val = -1;
            int64_t nb_prev = 0;
            for (int l = e - 1; l >= a; --l) {
                const int64_t nb_l = nbe[l];
                if (nb_l != nb_prev) {
                    const int64_t cand = (pb[e] - pb[l]) + (n_full - nb_prev) * row.t_full + partial;
                    val = cand > val ? cand : val;
                }
                nb_prev = nb_l;
            }
            if (partial > 0) {
                const int64_t cand = (pb[e] - pb[v.next_grad[a]]) + partial;
                val = cand > val ? cand : val;
            }
        }
        out[a] = val;
    }
}

// One thread per entry: an upper bound on every time any candidate of the entry can produce:
// all items of the pipeline in sequence plus the largest possible bucket-lane excess.
// rel_bound adds one more backward pass over all stages, the largest shift of the evaluation
// kernel's relative time frames.
__global__ void entry_bound_kernel(DeviceView v, Entry *entries, int64_t *jsum)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= v.sc.n_entries) return;
    Entry en = entries[i];
    const Row &row = v.rows[en.row];
    const int L = v.tc.n_layers, L1 = L + 1;
    const int64_t *pf = v.etf + (int64_t)i * v.tc.lp, *pb = v.etb + (int64_t)i * v.tc.lp;
    int64_t per_mb = pf[L] + pb[L], frame_shift = pb[L];
    for (int d = 0; d + 1 < row.pp; ++d) {
        const int64_t p2p = (((d + 1) & (row.p2p_period - 1)) == 0) ? en.p2p_inter : en.p2p_intra;
        per_mb += 2 * p2p * row.v;                  // once per model chunk
        frame_shift += p2p;
    }
    // interleaved candidates: the last device sends to the first between chunks
    if (row.v > 1) per_mb += 2 * (row.v - 1) * (en.p2p_inter > en.p2p_intra ? en.p2p_inter : en.p2p_intra);
    int64_t excess = 0;
    if (row.two_way) {
        // two streams of buckets per device, each at most the whole model's, priced across nodes
        const int64_t *nbL = v.nb + row.row_tab_off + (int64_t)L * L1;
        const int64_t *tpL = v.tp + row.row_tab_off + (int64_t)L * L1;
        const int64_t t_max = row.t_full > row.t_full_near ? row.t_full : row.t_full_near;
        const int64_t one = v.tc.bucket > 0 ? t_max
                                            : allreduce_cost(v.tc, 2 * (int64_t)row.dp, tpL[0], v.tc.alpha_inter, v.tc.beta_inter) +
                                              allreduce_cost(v.tc, 2 * (int64_t)row.dp, tpL[0], v.tc.alpha_intra, v.tc.beta_intra);
        excess = 2 * (nbL[0] * t_max + one);
    } else if (row.dp > 1) {
        const int64_t *nbL = v.nb + row.row_tab_off + (int64_t)L * L1;
        const int64_t *tpL = v.tp + row.row_tab_off + (int64_t)L * L1;
        // a device's buckets cost at most all full buckets of the model plus one more bucket per
        // model chunk it holds
        excess = nbL[0] * row.t_full + row.v * (v.tc.bucket > 0 ? row.t_full : tpL[0]);
    }
    // total jitter of a stage's items: whole cycles of the P slots plus the remainder
    __int128 jitter_total = 0;
    if (jsum) {
        const int P = v.tc.n_jitter, S = v.tc.jitter_stages;
        for (int d = 0; d < DISTSIM_MAX_PP; ++d) {
            int64_t sum = 0;
            if (d < row.pp) {
                int64_t cycle = 0, rest = 0;
                for (int p = 0; p < P; ++p) {
                    const int64_t x = v.raw.jit_f[p * S + d] + v.raw.jit_b[p * S + d];
                    cycle += x;
                    if (p < en.m % P) rest += x;
                }
                sum = (int64_t)(en.m / P) * cycle + rest;
            }
            jsum[(int64_t)i * DISTSIM_MAX_PP + d] = sum;
            jitter_total += sum;
        }
    }
    const __int128 b = (__int128)en.m * per_mb + excess + jitter_total;
    en.bound = b >= (__int128)kSat ? kSat : (int64_t)b;
    en.rel_bound = b + frame_shift >= (__int128)kSat ? kSat : (int64_t)(b + frame_shift);
    entries[i] = en;
}

// One thread per (entry, word): 32-bit copies of the entry's prefix rows and bucket-lane table.
// Every value of an entry is at most the entry's time bound, so for a bound below 2^32 the copy
// is exact; the table's "no buckets" marker (-1) becomes 0, which the evaluation treats alike.
__global__ void narrow_tables_kernel(DeviceView v, uint2 *pfb32, uint32_t *dt32)
{
    const int lp = v.tc.lp, t32 = v.tab_words32, n_tab = (v.tc.n_layers + 1) * (v.tc.n_layers + 1);
    const int per_entry = lp + (dt32 ? t32 : 0);
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (int64_t)v.sc.n_entries * per_entry) return;
    const int en = (int)(i / per_entry), k = (int)(i - (int64_t)en * per_entry);
    const bool narrow = v.entries[en].bound < ((int64_t)1 << 32);
    if (k < lp) {
        uint2 out = make_uint2(0u, 0u);
        if (narrow) out = make_uint2((uint32_t)v.etf[(int64_t)en * lp + k], (uint32_t)v.etb[(int64_t)en * lp + k]);
        pfb32[(int64_t)en * lp + k] = out;
    } else {
        const int w = k - lp;
        uint32_t out = 0;
        if (narrow && w < n_tab) {
            const int64_t val = v.dt[(int64_t)en * v.tab_words + w];
            out = val > 0 ? (uint32_t)val : 0u;
        }
        dt32[(int64_t)en * t32 + w] = out;
    }
}

}  // namespace

void launch_build_narrow_tables(cudaStream_t s, const DeviceView &v, uint2 *pfb32, uint32_t *dt32, int64_t *launches)
{
    if (v.sc.n_entries == 0 || !pfb32) return;
    const int64_t n = (int64_t)v.sc.n_entries * (v.tc.lp + (dt32 ? v.tab_words32 : 0));
    narrow_tables_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(v, pfb32, dt32);
    ++*launches;
}

void launch_build_entry_tables(cudaStream_t s, const DeviceView &v, Entry *entries, int64_t *dt,
                               int64_t *jsum, int64_t *launches)
{
    if (v.sc.n_entries == 0) return;
    if (dt) {
        const int n = v.sc.n_entries * (v.tc.n_layers + 1);
        build_dt_kernel<<<(n + 127) / 128, 128, 0, s>>>(v, dt);
        ++*launches;
    }
    entry_bound_kernel<<<(v.sc.n_entries + 127) / 128, 128, 0, s>>>(v, entries, jsum);
    ++*launches;
}

void launch_fill_entries(cudaStream_t s, const TableConst &tc, Row *rows, int n_rows,
                         Entry *entries, int n_entries, int64_t *launches)
{
    if (n_entries == 0) return;
    fill_entries_kernel<<<(n_entries + 127) / 128, 128, 0, s>>>(tc, rows, n_rows, entries, n_entries);
    ++*launches;
}

void launch_build_prefix(cudaStream_t s, const TableConst &tc, const RawTable &raw,
                         const Entry *entries, int n_entries, int64_t *etf, int64_t *etb,
                         int64_t *launches)
{
    if (n_entries == 0) return;
    build_prefix_kernel<<<(n_entries + 127) / 128, 128, 0, s>>>(tc, raw, entries, n_entries, etf, etb);
    ++*launches;
}

void launch_build_bucket_tables(cudaStream_t s, const TableConst &tc, const RawTable &raw,
                                const Row *rows, int n_rows, int64_t *nb, int64_t *tp,
                                int64_t *launches)
{
    const int n = n_rows * (tc.n_layers + 1);
    if (n == 0) return;
    build_bucket_tables_kernel<<<(n + 127) / 128, 128, 0, s>>>(tc, raw, rows, n_rows, nb, tp);
    ++*launches;
}

void launch_build_layer_tables(cudaStream_t s, const TableConst &tc, const RawTable &raw,
                               int32_t *next_grad, int32_t *pe, int64_t *launches)
{
    build_layer_tables_kernel<<<1, 32, 0, s>>>(tc, raw, next_grad, pe);
    ++*launches;
}

}  // namespace distsim
