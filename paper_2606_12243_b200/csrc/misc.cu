// Small memory-bound kernels of the decoder block and the cache bookkeeping:
// rotary table, per-pass preparation (tree layout, row tokens, clamped lengths), embedding gather,
// RMSNorm, rotary embedding + KV append, KV commit.
#include "common.cuh"

// ---------------------------------------------------------------------------------------------
// rotary table: cos/sin(pos * theta^(-2p/hd)), computed in double once per handle
// ---------------------------------------------------------------------------------------------
__global__ void rope_table_kernel(float *cosv, float *sinv, int max_ctx, int half, double theta) {
    int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= max_ctx * half) return;
    int pos = idx / half, p = idx % half;
    double inv = pow(theta, -2.0 * (double)p / (double)(2 * half));
    double ang = (double)pos * inv;
    cosv[idx] = (float)cos(ang);
    sinv[idx] = (float)sin(ang);
}

int launch_rope_table(const viasd_model *m, cudaStream_t st) {
    int half = m->cfg.head_dim / 2;
    int n = m->cfg.max_ctx * half;
    rope_table_kernel<<<(n + 255) / 256, 256, 0, st>>>(m->ws.rope_cos, m->ws.rope_sin, m->cfg.max_ctx, half,
                                                       (double)m->cfg.rope_theta);
    LAUNCH_CHECK();
    return VIASD_OK;
}

// ---------------------------------------------------------------------------------------------
// per-pass preparation
// ---------------------------------------------------------------------------------------------
// parent: [N] shared by the batch, or [B, N] when per_seq
__global__ void prep_kernel(TreeInfo *tree, int *len_eff, int *row_tok, DeviceStats *stats, const int *len,
                            const int *pending, const int *draft_tok, const int *parent, int per_seq, int B, int N,
                            int max_ctx, int vocab, int full_pass) {
    const int M = N + 1;
    PDL_TRIGGER();
    if (threadIdx.x == 0 && full_pass) stats->full_ran = 1;     // the full verifier's cache receives this block's rows
    for (int b = threadIdx.x; b < B; b += blockDim.x) {
        build_tree(tree + b, parent + (per_seq ? (size_t)b * N : 0), N, stats);
        int l = len[b];
        int c = min(max(l, 0), max_ctx - M);
        if (c != l) stats->device_status = VIASD_ECAPACITY;
        len_eff[b] = c;
    }
    for (int r = threadIdx.x; r < B * M; r += blockDim.x) {
        int b = r / M, i = r % M;
        int t = (i == 0) ? pending[b] : draft_tok[b * N + i - 1];
        if (t < 0 || t >= vocab) { stats->device_status = VIASD_EDEVICE; t = 0; }
        row_tok[r] = t;
    }
}

int launch_prep(const viasd_model *m, const viasd_cache *c, const viasd_draft *d, bool full_pass, cudaStream_t st) {
    prep_kernel<<<1, 128, 0, st>>>(m->ws.tree, m->ws.len_eff, m->ws.row_tok, m->ws.stats, c->len, c->pending,
                                   d->draft_tok, d->parent, d->per_sequence, d->batch, d->n_nodes, m->cfg.max_ctx,
                                   m->cfg.vocab, full_pass ? 1 : 0);
    LAUNCH_CHECK();
    return VIASD_OK;
}

// Preparation of a replay pass (routed execution policy): the block of every sequence is extended, in front, by its
// last G committed tokens, so that the rows are
//     row 0 .. G-1 : tokens[len - G .. len - 1]  (a chain; row 0 plays the pending token's part)
//     row G        : the pending token
//     row G+1+n    : draft node n (its parent moved along)
// against a context of len - G rows.  The full verifier recomputes K/V of the G committed tokens (the same values
// where its cache had them, the missing ones where a skipped pass left a gap) on its way to the block's own rows.
__global__ void prep_replay_kernel(TreeInfo *tree, int *len_eff, int *row_tok, DeviceStats *stats, const int *len,
                                   const int *pending, const int *draft_tok, const int *parent, int per_seq,
                                   const int *tokens, int B, int N, int G, int max_ctx, int vocab, const int *run_flag) {
    RUN_FLAG_EXIT(run_flag);
    const int Mx = G + N + 1;
    if (threadIdx.x == 0) stats->full_ran = 1;
    for (int b = threadIdx.x; b < B; b += blockDim.x) {
        TreeInfo *t = tree + b;
        const int *par = parent + (per_seq ? (size_t)b * N : 0);
        t->anc[0] = 1ull;
        t->depth[0] = 0;
        for (int i = 0; i < Mx; ++i) { t->first_child[i] = -1; t->next_sibling[i] = -1; }
        for (int e = 0; e < G + N; ++e) {                       // extended node e is row e + 1
            int p = e < G ? e - 1 : par[e - G];
            const int i = e + 1;
            if (e >= G) {
                if (p == -2) { t->anc[i] = 1ull << i; t->depth[i] = 0; continue; }
                if (p < -1 || p >= e - G) { stats->device_status = VIASD_EDEVICE; p = -1; }
                p = p < 0 ? G - 1 : G + p;
            }
            const int pr = p + 1;
            t->anc[i] = t->anc[pr] | (1ull << i);
            t->depth[i] = t->depth[pr] + 1;
        }
        t->is_chain = 0;
        const int l = len[b] - G;
        const int c = min(max(l, 0), max_ctx - Mx);
        if (c != l) stats->device_status = VIASD_ECAPACITY;     // fewer than G committed tokens, or no room for the rows
        len_eff[b] = c;
    }
    for (int r = threadIdx.x; r < B * Mx; r += blockDim.x) {
        const int b = r / Mx, i = r % Mx;
        const int base = max(len[b] - G, 0);
        int t = i < G ? tokens[(size_t)b * max_ctx + min(base + i, max_ctx - 1)] : i == G ? pending[b] : draft_tok[b * N + i - G - 1];
        if (t < 0 || t >= vocab) { stats->device_status = VIASD_EDEVICE; t = 0; }
        row_tok[r] = t;
    }
}

int launch_prep_replay(const viasd_model *m, const viasd_cache *c, const viasd_draft *d, int G, cudaStream_t st) {
    prep_replay_kernel<<<1, 128, 0, st>>>(m->ws.tree, m->ws.len_eff, m->ws.row_tok, m->ws.stats, c->len, c->pending,
                                          d->draft_tok, d->parent, d->per_sequence, c->tokens, d->batch, d->n_nodes, G,
                                          m->cfg.max_ctx, m->cfg.vocab, m->run_flag);
    LAUNCH_CHECK();
    return VIASD_OK;
}

// The block's own rows (the last M of every sequence's G + M) of the head's input and of its row statistics, packed
// for the output head: row b * (G + M) + G + i -> row b * M + i.  One CTA per row.
__global__ void compact_head_rows_kernel(__nv_bfloat16 *dst, const __nv_bfloat16 *src, size_t plane, float *ssq_dst,
                                         const float *ssq_src, int ssq_stride, int ssq_n, int d, int M, int G,
                                         const int *run_flag) {
    RUN_FLAG_EXIT(run_flag);
    PDL_TRIGGER();
    const int r = blockIdx.x, b = r / M, i = r % M, from = b * (G + M) + G + i;
    const uint4 *s0 = reinterpret_cast<const uint4 *>(src + (size_t)from * d), *s1 = reinterpret_cast<const uint4 *>(src + plane + (size_t)from * d);
    uint4 *d0 = reinterpret_cast<uint4 *>(dst + (size_t)r * d), *d1 = reinterpret_cast<uint4 *>(dst + plane + (size_t)r * d);
    for (int c = threadIdx.x; c < d / 8; c += blockDim.x) { d0[c] = s0[c]; d1[c] = s1[c]; }
    for (int e = threadIdx.x; e < ssq_n; e += blockDim.x) ssq_dst[(size_t)e * ssq_stride + r] = ssq_src[(size_t)e * ssq_stride + from];
}

int launch_compact_head_rows(const viasd_model *m, int batch, int M, int G, cudaStream_t st) {
    const viasd_config &c = m->cfg;
    compact_head_rows_kernel<<<batch * M, 128, 0, st>>>((__nv_bfloat16 *)m->ws.a_head, (const __nv_bfloat16 *)m->ws.a,
        m->ws.rows_alloc * (size_t)c.d_model, m->ws.ssq_head, m->ws.ssq, (int)m->ws.rows_alloc, (c.d_model / 128) * 4,
        c.d_model, M, G, m->run_flag);
    LAUNCH_CHECK();
    return VIASD_OK;
}

// ---------------------------------------------------------------------------------------------
// embedding gather: h[r] = E[row_tok[r]]
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void embed_kernel(float *h, const T *E, const int *row_tok, int d) {
    int r = blockIdx.x;
    PDL_TRIGGER();
    const T *src = E + (size_t)row_tok[r] * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) h[(size_t)r * d + i] = to_f32<T>(src[i]);
}

// One embedding row by one CTA of 8 warps: h = E[tok], a = hi/lo(h * gain), sums of h^2 per 32 features.
// The row and the gains are loaded in batches of eight independent loads per thread: the embedding rows are cold in
// HBM, and one load per loop trip made this kernel a chain of memory round trips.
__device__ __forceinline__ void embed_row(float *h, __nv_bfloat16 *a, size_t plane, float *ssq, int ssq_stride,
                                          const __nv_bfloat16 *src, const float *gain, int r, int d, int warp, int lane) {
    for (int base0 = 0; base0 < d; base0 += 8 * 256) {
        float v[8], g[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int base = base0 + j * 256, i = base + warp * 32 + lane;   // d is a multiple of 128: whole warps stay in range
            const bool on = base + warp * 32 < d;
            v[j] = on ? __bfloat162float(src[i]) : 0.f;
            g[j] = on ? gain[i] : 0.f;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int base = base0 + j * 256, i = base + warp * 32 + lane;
            if (base + warp * 32 < d) {
                h[(size_t)r * d + i] = v[j];
                store_act<__nv_bfloat16>(a, plane, (size_t)r * d + i, v[j] * g[j]);
                const float sq = warp_sum(v[j] * v[j]);
                if (lane == 0) ssq[(size_t)(i >> 5) * ssq_stride + r] = sq;   // (tile * 4 + quarter) == feature / 32
            }
        }
    }
}

// Embedding gather fused with the preparation of the first RMSNorm of the pass (tensor-core path):
// h = E[tok]; a = hi/lo(h * gain); partial sums of h^2 per 32 features in the layout the GEMM epilogue reads.
__global__ void __launch_bounds__(256)
embed_norm_kernel(float *h, __nv_bfloat16 *a, size_t plane, float *ssq, int ssq_stride, const __nv_bfloat16 *E,
                  const float *gain, const int *row_tok, int d, const int *run_flag) {
    RUN_FLAG_EXIT(run_flag);
    const int r = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    PDL_TRIGGER();
    const __nv_bfloat16 *src = E + (size_t)row_tok[r] * d;
    embed_row(h, a, plane, ssq, ssq_stride, src, gain, r, d, warp, lane);
}

int launch_embed_norm(const viasd_model *m, const float *gain, int rows, cudaStream_t st) {
    embed_norm_kernel<<<rows, 256, 0, st>>>(m->ws.h, (__nv_bfloat16 *)m->ws.a, m->ws.rows_alloc * m->cfg.d_model, m->ws.ssq,
                                            (int)m->ws.rows_alloc, (const __nv_bfloat16 *)m->embed, gain, m->ws.row_tok,
                                            m->cfg.d_model, m->run_flag);
    LAUNCH_CHECK();
    return VIASD_OK;
}

// Two row streams from the same block rows: rows [0, rows) prepared for the full verifier's first layer,
// rows [rows, 2*rows) for the slim verifier's first routed layer (their first norms differ).
__global__ void __launch_bounds__(256)
embed_norm2_kernel(float *h, __nv_bfloat16 *a, size_t plane, float *ssq, int ssq_stride, const __nv_bfloat16 *E,
                   const float *gain_full, const float *gain_slim, const int *row_tok, int d, int rows) {
    const int r = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    PDL_TRIGGER();
    const float *gain = r < rows ? gain_full : gain_slim;
    const __nv_bfloat16 *src = E + (size_t)row_tok[r < rows ? r : r - rows] * d;
    embed_row(h, a, plane, ssq, ssq_stride, src, gain, r, d, warp, lane);
}

int launch_embed_norm2(const viasd_model *m, const float *gain_full, const float *gain_slim, int rows, cudaStream_t st) {
    embed_norm2_kernel<<<2 * rows, 256, 0, st>>>(m->ws.h, (__nv_bfloat16 *)m->ws.a, m->ws.rows_alloc * m->cfg.d_model,
                                                 m->ws.ssq, (int)m->ws.rows_alloc, (const __nv_bfloat16 *)m->embed, gain_full,
                                                 gain_slim, m->ws.row_tok, m->cfg.d_model, rows);
    LAUNCH_CHECK();
    return VIASD_OK;
}

int launch_embed(const viasd_model *m, int rows, cudaStream_t st) {
    if (m->cfg.dtype == 0)
        embed_kernel<float><<<rows, 256, 0, st>>>(m->ws.h, (const float *)m->embed, m->ws.row_tok, m->cfg.d_model);
    else
        embed_kernel<__nv_bfloat16><<<rows, 256, 0, st>>>(m->ws.h, (const __nv_bfloat16 *)m->embed,
                                                          m->ws.row_tok, m->cfg.d_model);
    LAUNCH_CHECK();
    return VIASD_OK;
}

// ---------------------------------------------------------------------------------------------
// RMSNorm: a[r] = h[r] / sqrt(mean(h[r]^2) + eps) * gain, written in the model dtype
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
rmsnorm_kernel(T *a, size_t plane, const float *h, const float *gain, int d, float eps) {
    __shared__ float red[8];
    PDL_TRIGGER();
    const int r = blockIdx.x;
    const float4 *x4 = reinterpret_cast<const float4 *>(h + (size_t)r * d);
    const float4 *g4 = reinterpret_cast<const float4 *>(gain);
    constexpr int MAXV = 8;                           // up to 8 float4 per thread: d <= 8192 stays in registers
    const int nv = d >> 2;
    float4 v[MAXV];
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < MAXV; ++j) {
        const int i = threadIdx.x + j * 256;
        if (i < nv) { v[j] = x4[i]; s += v[j].x * v[j].x + v[j].y * v[j].y + v[j].z * v[j].z + v[j].w * v[j].w; }
    }
    for (int i = threadIdx.x + MAXV * 256; i < nv; i += 256) { float4 t = x4[i]; s += t.x * t.x + t.y * t.y + t.z * t.z + t.w * t.w; }
    s = warp_sum(s);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += red[w];
    const float inv = rsqrtf(tot / (float)d + eps);
    auto emit = [&](int i, float4 t) {
        const float4 g = g4[i];
        const size_t o = (size_t)r * d + (size_t)i * 4;
        store_act<T>(a, plane, o, t.x * inv * g.x);
        store_act<T>(a, plane, o + 1, t.y * inv * g.y);
        store_act<T>(a, plane, o + 2, t.z * inv * g.z);
        store_act<T>(a, plane, o + 3, t.w * inv * g.w);
    };
#pragma unroll
    for (int j = 0; j < MAXV; ++j) {
        const int i = threadIdx.x + j * 256;
        if (i < nv) emit(i, v[j]);
    }
    for (int i = threadIdx.x + MAXV * 256; i < nv; i += 256) emit(i, x4[i]);
}

int launch_rmsnorm(const viasd_model *m, const float *gain, int rows, cudaStream_t st) {
    if (m->cfg.dtype == 0)
        rmsnorm_kernel<float><<<rows, 256, 0, st>>>((float *)m->ws.a, 0, m->ws.h, gain, m->cfg.d_model, m->cfg.rms_eps);
    else
        rmsnorm_kernel<__nv_bfloat16><<<rows, 256, 0, st>>>((__nv_bfloat16 *)m->ws.a, m->ws.rows_alloc * m->cfg.d_model,
                                                            m->ws.h, gain, m->cfg.d_model, m->cfg.rms_eps);
    LAUNCH_CHECK();
    return VIASD_OK;
}

// ---------------------------------------------------------------------------------------------
// rotary embedding of q and k, KV append at slot len + row
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void rope_append_kernel(float *q_out, T *kc, T *vc, const float *qkv, const float *cosv, const float *sinv,
                                   const int *len_eff, const TreeInfo *tree, int M, int H, int Hkv, int hd,
                                   int max_batch, int max_ctx, int layer_ord) {
    int r = blockIdx.x, head = blockIdx.y;
    PDL_TRIGGER();
    int b = r / M, i = r % M;
    int half = hd >> 1;
    int n = len_eff[b];
    int pos = n + tree[b].depth[i], slot = n + i;
    const float *src = qkv + (size_t)r * (H + 2 * Hkv) * hd + (size_t)head * hd;
    for (int p = threadIdx.x; p < half; p += blockDim.x) {
        float x1 = src[p], x2 = src[p + half];
        if (head < H + Hkv) {
            float c = cosv[(size_t)pos * half + p], s = sinv[(size_t)pos * half + p];
            float y1 = x1 * c - x2 * s, y2 = x2 * c + x1 * s;
            if (head < H) {
                float *dst = q_out + (size_t)r * H * hd + (size_t)head * hd;
                dst[p] = y1;
                dst[p + half] = y2;
            } else {
                int g = head - H;
                T *dst = kc + ((((size_t)layer_ord * max_batch + b) * Hkv + g) * max_ctx + slot) * hd;
                dst[p] = from_f32<T>(y1);
                dst[p + half] = from_f32<T>(y2);
            }
        } else {
            int g = head - H - Hkv;
            T *dst = vc + ((((size_t)layer_ord * max_batch + b) * Hkv + g) * max_ctx + slot) * hd;
            dst[p] = from_f32<T>(x1);
            dst[p + half] = from_f32<T>(x2);
        }
    }
}

int launch_rope_append(const viasd_model *m, void *kc, void *vc, int layer_ord, int batch, int M, cudaStream_t st) {
    const viasd_config &c = m->cfg;
    dim3 grid(batch * M, c.n_heads + 2 * c.n_kv_heads);
    int threads = c.head_dim / 2 < 32 ? 32 : c.head_dim / 2;
    if (c.dtype == 0)
        rope_append_kernel<float><<<grid, threads, 0, st>>>(m->ws.q, (float *)kc, (float *)vc, m->ws.qkv,
            m->ws.rope_cos, m->ws.rope_sin, m->ws.len_eff, m->ws.tree, M, c.n_heads, c.n_kv_heads, c.head_dim,
            c.max_batch, c.max_ctx, layer_ord);
    else
        rope_append_kernel<__nv_bfloat16><<<grid, threads, 0, st>>>(m->ws.q, (__nv_bfloat16 *)kc,
            (__nv_bfloat16 *)vc, m->ws.qkv, m->ws.rope_cos, m->ws.rope_sin, m->ws.len_eff, m->ws.tree, M, c.n_heads,
            c.n_kv_heads, c.head_dim, c.max_batch, c.max_ctx, layer_ord);
    LAUNCH_CHECK();
    return VIASD_OK;
}

// ---------------------------------------------------------------------------------------------
// KV commit: compact the accepted path, then advance len / pending / tokens
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void commit_move_kernel(T *kf, T *vf, T *ks, T *vs, const int *len_eff, const int *n_acc,
                                   const int *path, int N, int L, int Ls, int Hkv, int hd, int max_batch,
                                   int max_ctx, const DeviceStats *stats, int layer0) {
    int layer = layer0 + blockIdx.x, b = blockIdx.y, g = blockIdx.z;
    if (layer < L && !stats->full_ran) return;                  // the full verifier's cache did not receive this block
    T *kc = layer < L ? kf : ks;
    T *vc = layer < L ? vf : vs;
    int lo = layer < L ? layer : layer - L;
    size_t base = (((size_t)lo * max_batch + b) * Hkv + g) * (size_t)max_ctx * hd;
    int n = len_eff[b];
    int na = min(n_acc[b], N);
    // each thread owns fixed columns, so walking j in order is enough to keep sources intact
    for (int j = 0; j < na; ++j) {
        int node = path[b * N + j];
        if (node < j || node >= N) break;           // not a valid path entry: stop (never moves rows up)
        int src = n + node + 1, dst = n + 1 + j;
        if (src == dst) continue;
        for (int c = threadIdx.x; c < hd; c += blockDim.x) {
            kc[base + (size_t)dst * hd + c] = kc[base + (size_t)src * hd + c];
            vc[base + (size_t)dst * hd + c] = vc[base + (size_t)src * hd + c];
        }
    }
}

__global__ void commit_advance_kernel(int *len, int *len_full, int *pending, int *tokens, const int *len_eff,
                                      const int *n_emit, const int *out_tok, int B, int N, int max_ctx,
                                      DeviceStats *stats) {
    int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    int n = len_eff[b];
    int ne = min(max(n_emit[b], 0), N + 1);
    // the full verifier's cache is complete up to the new length exactly when its pass ran in this step
    if (len_full && stats->full_ran) len_full[b] = n + ne;
    if (b == 0 && !stats->full_ran) ++stats->full_skipped;
    if (ne == 0) return;
    if (tokens) {
        tokens[(size_t)b * max_ctx + n] = pending[b];
        for (int j = 0; j + 1 < ne; ++j) tokens[(size_t)b * max_ctx + n + 1 + j] = out_tok[b * (N + 1) + j];
    }
    len[b] = n + ne;
    pending[b] = out_tok[b * (N + 1) + ne - 1];
}

// slim_only: move the accepted rows in this handle's slim cache and nothing else (lengths, pending token and token
// list belong to the handle that commits last)
int launch_commit(const viasd_model *m, viasd_cache *c, const viasd_draft *d, const viasd_result *r, bool slim_only,
                  cudaStream_t st) {
    const viasd_config &cf = m->cfg;
    int rc = launch_prep(m, c, d, false, st);
    if (rc) return rc;
    const int layer0 = slim_only ? cf.n_layers : 0;
    dim3 grid(cf.n_layers + m->n_routed - layer0, d->batch, cf.n_kv_heads);
    int threads = cf.head_dim < 32 ? 32 : (cf.head_dim > 256 ? 256 : cf.head_dim);
    if (cf.dtype == 0)
        commit_move_kernel<float><<<grid, threads, 0, st>>>((float *)c->k_full, (float *)c->v_full, (float *)c->k_slim,
            (float *)c->v_slim, m->ws.len_eff, r->n_acc, r->path, d->n_nodes, cf.n_layers, m->n_routed, cf.n_kv_heads,
            cf.head_dim, cf.max_batch, cf.max_ctx, m->ws.stats, layer0);
    else
        commit_move_kernel<__nv_bfloat16><<<grid, threads, 0, st>>>((__nv_bfloat16 *)c->k_full,
            (__nv_bfloat16 *)c->v_full, (__nv_bfloat16 *)c->k_slim, (__nv_bfloat16 *)c->v_slim, m->ws.len_eff, r->n_acc,
            r->path, d->n_nodes, cf.n_layers, m->n_routed, cf.n_kv_heads, cf.head_dim, cf.max_batch, cf.max_ctx, m->ws.stats, layer0);
    LAUNCH_CHECK();
    if (slim_only) return VIASD_OK;
    commit_advance_kernel<<<(d->batch + 63) / 64, 64, 0, st>>>(c->len, c->len_full, c->pending, c->tokens, m->ws.len_eff,
                                                               r->n_emit, r->out_tok, d->batch, d->n_nodes, cf.max_ctx,
                                                               m->ws.stats);
    LAUNCH_CHECK();
    return VIASD_OK;
}
