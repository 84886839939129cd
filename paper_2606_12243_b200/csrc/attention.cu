// KV-append attention over a drafted block: each of the M query rows of a sequence attends to the
// committed cache rows 0..n-1 and to the block rows on its own root path (causal mask for a chain,
// ancestor mask for a tree).  Split-KV: a CTA handles one (sequence, kv head, key range, group of
// query rows), keeps an online softmax per query row and writes unnormalised partials; a second
// kernel merges the key ranges.
#include "common.cuh"
#include <string.h>
#include <stdlib.h>

namespace {

constexpr int TK = 32;          // keys per shared-memory tile
constexpr int QG = 16;          // query rows per CTA (2 per warp, 8 warps)
constexpr int ATT_WARPS = 8;

template <typename T, int HD>
__global__ void __launch_bounds__(ATT_WARPS * 32)
attention_split_kernel(float *__restrict__ part, const float *__restrict__ q, const T *__restrict__ kc,
                       const T *__restrict__ vc, const int *__restrict__ len_eff, const TreeInfo *__restrict__ tree,
                       int M, int H, int Hkv, int max_batch, int max_ctx, int layer_ord, int nsplit, float scale,
                       const int *run_flag) {
    RUN_FLAG_EXIT(run_flag);
    __shared__ float Qs[QG][HD];
    __shared__ float Ks[TK][HD + 1];
    __shared__ float Vs[TK][HD];
    constexpr int DPL = HD / 32;                     // output dims per lane
    PDL_TRIGGER();
    const int b = blockIdx.x / Hkv, g = blockIdx.x % Hkv, split = blockIdx.y, qg = blockIdx.z;
    const int grp = H / Hkv, QR = grp * M;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n = len_eff[b], Tk = n + M;
    int chunk = (Tk + nsplit - 1) / nsplit;
    chunk = (chunk + TK - 1) / TK * TK;
    const int k_begin = split * chunk, k_end = min(Tk, k_begin + chunk);

    // stage this CTA's query rows, pre-scaled
    for (int idx = threadIdx.x; idx < QG * HD; idx += blockDim.x) {
        int qq = idx / HD, dd = idx % HD;
        int qidx = qg * QG + qq;
        float v = 0.f;
        if (qidx < QR) {
            int h = g * grp + qidx / M, i = qidx % M;
            v = q[((size_t)(b * M + i) * H + h) * HD + dd] * scale;
        }
        Qs[qq][dd] = v;
    }
    float mrun[2] = {-INFINITY, -INFINITY}, lrun[2] = {0.f, 0.f}, o[2][DPL];
#pragma unroll
    for (int r = 0; r < 2; ++r)
#pragma unroll
        for (int c = 0; c < DPL; ++c) o[r][c] = 0.f;
    unsigned long long anc[2];
    int qrow[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        int qidx = qg * QG + warp * 2 + r;
        qrow[r] = qidx < QR ? qidx : -1;
        anc[r] = qidx < QR ? tree[b].anc[qidx % M] : 0ull;
    }
    const size_t cbase = (((size_t)layer_ord * max_batch + b) * Hkv + g) * (size_t)max_ctx * HD;

    for (int k0 = k_begin; k0 < k_end; k0 += TK) {
        __syncthreads();
        for (int idx = threadIdx.x; idx < TK * HD; idx += blockDim.x) {
            int j = idx / HD, dd = idx % HD;
            float kv = 0.f, vv = 0.f;
            if (k0 + j < k_end) {
                kv = to_f32<T>(kc[cbase + (size_t)(k0 + j) * HD + dd]);
                vv = to_f32<T>(vc[cbase + (size_t)(k0 + j) * HD + dd]);
            }
            Ks[j][dd] = kv;
            Vs[j][dd] = vv;
        }
        __syncthreads();
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            if (qrow[r] < 0) continue;
            const int j = k0 + lane;
            const bool valid = j < k_end && (j < n || ((anc[r] >> (j - n)) & 1ull));
            float s = 0.f;
            const float *qs = Qs[warp * 2 + r];
#pragma unroll 8
            for (int dd = 0; dd < HD; ++dd) s = fmaf(qs[dd], Ks[lane][dd], s);
            s = valid ? s : -INFINITY;
            float mnew = fmaxf(mrun[r], warp_max(s));
            if (mnew == -INFINITY) continue;                     // nothing visible yet
            float p = valid ? expf(s - mnew) : 0.f;
            float corr = expf(mrun[r] - mnew);                   // exp(-inf) = 0 on the first tile
            lrun[r] = lrun[r] * corr + warp_sum(p);
#pragma unroll
            for (int c = 0; c < DPL; ++c) o[r][c] *= corr;
#pragma unroll 8
            for (int jj = 0; jj < TK; ++jj) {
                float pj = __shfl_sync(0xffffffffu, p, jj);
#pragma unroll
                for (int c = 0; c < DPL; ++c) o[r][c] = fmaf(pj, Vs[jj][lane + 32 * c], o[r][c]);
            }
            mrun[r] = mnew;
        }
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        if (qrow[r] < 0) continue;
        int h = g * grp + qrow[r] / M, i = qrow[r] % M;
        float *dst = part + ((((size_t)b * H + h) * M + i) * nsplit + split) * (HD + 2);
#pragma unroll
        for (int c = 0; c < DPL; ++c) dst[lane + 32 * c] = o[r][c];
        if (lane == 0) { dst[HD] = mrun[r]; dst[HD + 1] = lrun[r]; }
    }
}

template <typename T, int HD>
__global__ void attention_combine_kernel(T *__restrict__ out, size_t plane, const float *__restrict__ part, int M, int H,
                                         int nsplit, const int *run_flag) {
    RUN_FLAG_EXIT(run_flag);
    const int r = blockIdx.x, h = blockIdx.y;        // r = b * M + i
    PDL_TRIGGER();
    const int b = r / M, i = r % M;
    const float *src = part + (((size_t)b * H + h) * M + i) * (size_t)nsplit * (HD + 2);
    float mmax = -INFINITY;
    for (int s = 0; s < nsplit; ++s) mmax = fmaxf(mmax, src[(size_t)s * (HD + 2) + HD]);
    for (int dd = threadIdx.x; dd < HD; dd += blockDim.x) {
        float num = 0.f, den = 0.f;
        for (int s = 0; s < nsplit; ++s) {
            const float *p = src + (size_t)s * (HD + 2);
            float ms = p[HD];
            if (ms == -INFINITY) continue;
            float w = expf(ms - mmax);
            num = fmaf(p[dd], w, num);
            den = fmaf(p[HD + 1], w, den);
        }
        store_act<T>(out, plane, ((size_t)r * H + h) * HD + dd, num / den);
    }
}

template <typename T, int HD>
int run(const viasd_model *m, const void *kc, const void *vc, int layer_ord, int batch, int M, int nsplit,
        cudaStream_t st) {
    const viasd_config &c = m->cfg;
    const int grp = c.n_heads / c.n_kv_heads;
    const int qgroups = (grp * M + QG - 1) / QG;
    dim3 grid(batch * c.n_kv_heads, nsplit, qgroups);
    attention_split_kernel<T, HD><<<grid, ATT_WARPS * 32, 0, st>>>(m->ws.part, m->ws.q, (const T *)kc,
        (const T *)vc, m->ws.len_eff, m->ws.tree, M, c.n_heads, c.n_kv_heads, c.max_batch, c.max_ctx, layer_ord, nsplit,
        1.0f / sqrtf((float)HD), m->run_flag);
    LAUNCH_CHECK();
    attention_combine_kernel<T, HD><<<dim3(batch * M, c.n_heads), HD < 128 ? HD : 128, 0, st>>>((T *)m->ws.attn,
        sizeof(T) == 2 ? m->ws.rows_alloc * (size_t)c.n_heads * HD : 0, m->ws.part, M, c.n_heads, nsplit, m->run_flag);
    LAUNCH_CHECK();
    return VIASD_OK;
}

}  // namespace

int attention_nsplit(const viasd_model *m, int batch, int M) {
    const viasd_config &c = m->cfg;
    const int grp = c.n_heads / c.n_kv_heads;
    const int qgroups = (grp * M + QG - 1) / QG;
    int ctas = batch * c.n_kv_heads * qgroups;
    int nsplit = (2 * m->sm_count + ctas - 1) / ctas;
    int by_len = (c.max_ctx + 127) / 128;            // at least 128 keys per split
    if (nsplit > by_len) nsplit = by_len;
    if (nsplit > 16) nsplit = 16;
    if (nsplit < 1) nsplit = 1;
    // never beyond what the partial buffer holds
    size_t per_split = (size_t)batch * c.n_heads * M * (c.head_dim + 2) * sizeof(float);
    while (nsplit > 1 && per_split * nsplit > m->ws.part_bytes) --nsplit;
    return nsplit;
}

// Key ranges per (sequence, kv head) for the tensor-core kernel, from a small cost model: items are dealt to
// CTAs in equal contiguous shares, each item costs a fixed part (query staging, merge, partial) plus its tiles,
// and every extra range adds merge work.  Depends on batch, heads and M only, so the one-stream and the two-stream
// launch cut the keys at the same places and produce the same bits.
static int mma_nsplit(const viasd_model *m, int batch, int M, int streams, bool tc, int reps, int subs, int tk_rows) {
    const viasd_config &c = m->cfg;
    const int base = batch * c.n_kv_heads * subs, sms = m->sm_count;      // subs: items per kv head (keys-on-lanes kernel)
    const int mt = ((c.n_heads / c.n_kv_heads) * M + 15) / 16;
    const int tiles = (c.max_ctx + 127) / 128;
    int max_s = tiles < 16 / reps ? tiles : 16 / reps;          // the partial buffer holds 16 ranges per (row, head)
    if (max_s < 1) max_s = 1;
    // microseconds, roughly: the tcgen05 kernel's tile does not depend on the number of query tiles
    // (keys-on-lanes kernel, measured: a tile costs its softmax chain, 1.1 - 1.8 us with 8 - 32 rows per item, an item
    // 5 - 10 us of query staging, result rows and merge)
    const double t_tile = tk_rows > 16 ? 1.8 : tk_rows > 8 ? 1.3 : tk_rows > 0 ? 1.1 : tc ? 0.7 : 0.5 + 0.8 * mt;
    const double t_item = tk_rows > 16 ? 8.0 : tk_rows > 0 ? 5.0 : tc ? 4.0 : 3.0;
    // One choice for the whole model, whichever call runs (the cuts must not depend on it): the routed layers are
    // charged as two-stream launches, as the verify step runs them, the others as one-stream launches.
    const int n_dual = m->n_routed, n_single = c.n_layers - m->n_routed;
    int best = 1;
    double best_cost = 1e30;
    for (int s = 1; s <= max_s; ++s) {
        const int tpi = ((tiles + s - 1) / s);
        double cost = 0.15 * s * reps * (n_dual + n_single);
        for (int st2 = 1; st2 <= 2; ++st2) {
            const int n = base * s * st2, ipc = (n + sms - 1) / sms;
            cost += (st2 == 2 ? n_dual : n_single) * ipc * (tpi * t_tile + t_item);
        }
        if (cost < best_cost - 1e-9) { best_cost = cost; best = s; }
    }
    if (m->opt.attn_splits >= 1 && m->opt.attn_splits <= max_s) best = m->opt.attn_splits;
    size_t per_split = (size_t)streams * batch * c.n_heads * M * (c.head_dim + 2) * sizeof(float) * reps;
    while (best > 1 && per_split * best > m->ws.part_bytes) --best;
    return best;
}

// merge of the key ranges: inside the attention kernel when there is little to merge, else its own kernel
static int mma_attention(viasd_model *m, const void *kc, const void *vc, bool slim, int layer_ord, const void *kc2,
                         const void *vc2, int layer_ord2, int streams, int batch, int M, cudaStream_t st) {
    const viasd_config &c = m->cfg;
    // Which kernel (VIASD_OPT_ATTENTION_KERNEL): the mma.sync kernel, tcgen05 with the query rows on the TMEM lanes, or
    // tcgen05 with the keys on the lanes (few query rows only).  Default: keys-on-lanes where it applies, else mma.sync.
    const int kind = m->opt.attn_kernel == 1 ? 0 : m->opt.attn_kernel == 2 ? 1 : m->opt.attn_kernel == 3 ? 2 : 3;   // 0 mma, 1 tc, 2 tk, 3 default
    const int QR = (c.n_heads / c.n_kv_heads) * M;
    // keys-on-lanes pays off when a CTA streams many tiles; with a handful per CTA (one short sequence) the
    // mma.sync kernel's shorter latency chain wins
    const long long tiles_total = (long long)streams * batch * c.n_kv_heads * ((c.max_ctx + 127) / 128);
    const int grp = c.n_heads / c.n_kv_heads, hpi = attention_tk_heads_per_item(grp, M);
    const int subs = hpi ? grp / hpi : 1, QRi = hpi * M;       // keys-on-lanes: items per kv head, query rows per item
    // (with more than 32 query rows per kv head the mma.sync kernel has one key group per query tile and is bound by
    // its MMA issue: there the keys-on-lanes kernel wins from two tiles per SM on)
    // (and with 17 - 32 query rows per kv head, two query tiles for the mma.sync kernel, from one tile per SM on: 32B
    // shape at batch 1, 264 tiles, attention 1.78 -> 1.61 ms per step)
    int use = kind == 3 ? (hpi && tiles_total * subs >= (subs > 1 ? 2LL : QRi > 16 ? 1LL : 8LL) * m->sm_count ? 2 : 0) : kind;
    if (use == 2 && !hpi) use = 0;
    const int reps = use == 1 ? attention_tc_replicas(QR) : 1;
    const int nsplit = mma_nsplit(m, batch, M, streams, use != 0, reps, use == 2 ? subs : 1, use == 2 ? QRi : 0);
    const int n_part = nsplit * reps;        // key ranges per (row, head) that have to be merged
    const bool fuse = n_part > 1 && n_part <= 32 && (use == 2 ? QRi : QR) * n_part <= 160;
    int rc;
    if (use == 2) {
        // The keys-on-lanes kernel deals tiles, not key ranges, evenly to the CTAs (nsplit 0) when the partial buffer
        // has its 16 slots per (row, head): whole (sequence, head) items leave SMs idle (320 items on 148 SMs: a
        // quarter of them).  Its merges are then always fused.  Not with more than 16 query rows per kv head: there an
        // item's fixed cost (staging 32 rows of queries, 32 rows of results) is worth a dozen tiles, and the extra
        // item per CTA cost more than the balance won (32B batch-16 step 36.5 -> 39.0 ms).  VIASD_OPT_TK_FLAT overrides.
        const size_t need = (size_t)streams * batch * c.n_heads * M * 16 * (c.head_dim + 2) * sizeof(float);
        if ((m->opt.tk_flat >= 0 ? m->opt.tk_flat != 0 : QR <= 16) && subs == 1 && need <= m->ws.part_bytes)
            return launch_attention_tk(m, kc, vc, slim, layer_ord, kc2, vc2, layer_ord2, streams, batch, M, 0, 1, st);
        rc = launch_attention_tk(m, kc, vc, slim, layer_ord, kc2, vc2, layer_ord2, streams, batch, M, nsplit, fuse ? 1 : 0, st);
    }
    else if (use == 1) rc = launch_attention_tc(m, kc, vc, slim, layer_ord, kc2, vc2, layer_ord2, streams, batch, M, nsplit, fuse ? 1 : 0, st);
    else rc = launch_attention_mma(m, kc, vc, slim, layer_ord, kc2, vc2, layer_ord2, streams, batch, M, nsplit, fuse ? 1 : 0, st);
    if (rc || n_part == 1 || fuse) return rc;
    attention_combine_kernel<__nv_bfloat16, 128><<<dim3(streams * batch * M, c.n_heads), 128, 0, st>>>(
        (__nv_bfloat16 *)m->ws.attn, m->ws.rows_alloc * (size_t)c.n_heads * 128, m->ws.part, M, c.n_heads, n_part, m->run_flag);
    LAUNCH_CHECK();
    return VIASD_OK;
}

int launch_attention(viasd_model *m, const void *kc, const void *vc, bool slim, int layer_ord, int batch, int M,
                     cudaStream_t st) {
    const viasd_config &c = m->cfg;
    if (attention_mma_supported(m, M)) {
        return mma_attention(m, kc, vc, slim, layer_ord, nullptr, nullptr, 0, 1, batch, M, st);
    }
    int nsplit = attention_nsplit(m, batch, M);
    if (c.dtype == 0) {
        if (c.head_dim == 64) return run<float, 64>(m, kc, vc, layer_ord, batch, M, nsplit, st);
        if (c.head_dim == 128) return run<float, 128>(m, kc, vc, layer_ord, batch, M, nsplit, st);
    } else {
        if (c.head_dim == 64) return run<__nv_bfloat16, 64>(m, kc, vc, layer_ord, batch, M, nsplit, st);
        if (c.head_dim == 128) return run<__nv_bfloat16, 128>(m, kc, vc, layer_ord, batch, M, nsplit, st);
    }
    return VIASD_EINVAL;
}

// Both verifiers in one launch: the full stream's rows against the full cache, the slim stream's rows against the
// slim cache (tensor-core kernel only).
int launch_attention_dual(viasd_model *m, const void *kf, const void *vf, int layer_full, const void *ks, const void *vs,
                          int ord_slim, int batch, int M, cudaStream_t st) {
    return mma_attention(m, kf, vf, false, layer_full, ks, vs, ord_slim, 2, batch, M, st);
}
