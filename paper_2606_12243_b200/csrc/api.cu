// C ABI: argument checks, workspace carving, and the sequence of launches that makes up each call.
#include "common.cuh"
#include <new>
#include <string.h>
#include <stdlib.h>

int g_last_cuda_error = 0;
unsigned long long g_launch_count = 0;
int g_use_pdl = -1;

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
size_t elem_size(int dtype) { return dtype == 0 ? 4 : 2; }

struct Carver {
    char *base; size_t off;
    template <typename T> T *take(size_t bytes) {
        off = align_up(off, 256);
        T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
        off += bytes;
        return p;
    }
};

constexpr int MAX_SMS = 160;            // workspace is sized without asking the device
constexpr int MAX_GEMM_CTAS = 2 * MAX_SMS;

size_t part_bytes_for(const viasd_config &c) {
    const size_t R = (size_t)2 * c.max_batch * c.max_query;
    // attention split-KV partials: up to 16 key ranges of (head_dim + 2) floats per (row, head)
    size_t att = R * c.n_heads * 16 * (size_t)(c.head_dim + 2) * sizeof(float);
    const size_t cap = (size_t)256 << 20;
    return att < cap ? att : cap;
}

// One layout routine serves both the size query (base = null) and the real carve.
size_t carve(const viasd_config &c, char *base, Workspace *ws) {
    Carver cv{base, 0};
    const size_t R = (size_t)2 * c.max_batch * c.max_query, es = elem_size(c.dtype);   // two row streams
    const size_t qd = (size_t)c.n_heads * c.head_dim, kvd = (size_t)c.n_kv_heads * c.head_dim;
    Workspace w;
    w.rope_cos = cv.take<float>((size_t)c.max_ctx * (c.head_dim / 2) * 4);
    w.rope_sin = cv.take<float>((size_t)c.max_ctx * (c.head_dim / 2) * 4);
    w.h = cv.take<float>(R * c.d_model * 4);
    (void)es;
    w.rows_alloc = R;
    w.a = cv.take<void>(R * c.d_model * 4);            // fp32 plane, or bf16 hi + lo planes
    w.qkv = cv.take<float>(R * (qd + 2 * kvd) * 4);
    w.q = cv.take<float>(R * qd * 4);
    w.attn = cv.take<void>(R * qd * 4);
    w.act = cv.take<void>(R * c.d_ff * 4);
    w.part_bytes = part_bytes_for(c);
    w.part = cv.take<float>(w.part_bytes);
    w.len_eff = cv.take<int>((size_t)c.max_batch * 4);
    w.row_tok = cv.take<int>(R * 4);
    w.tree = cv.take<TreeInfo>(sizeof(TreeInfo) * (size_t)c.max_batch);
    w.stats = cv.take<DeviceStats>(sizeof(DeviceStats));
    w.accept_scratch = cv.take<float>(((size_t)c.max_batch * (VIASD_MAX_JUDGES + 1) * c.vocab +
                                       (size_t)c.max_batch * 3 * (VIASD_MAX_JUDGES + 1) * VIASD_MAX_ROWS_PER_SEQ) * 4);
    {
        const int nt = tc_pick_nt(R < 128 ? (int)R : 128, true);
        w.gemm_scratch = cv.take<float>(tc_scratch_floats(MAX_GEMM_CTAS, nt, true) * 4);
        size_t widest = (size_t)c.vocab;
        if (qd + 2 * kvd > widest) widest = qd + 2 * kvd;
        if ((size_t)c.d_ff > widest) widest = c.d_ff;
        w.ssq = cv.take<float>((size_t)(c.d_model / 128 + 1) * 4 * R * 4);
        w.a_head = cv.take<void>(R * c.d_model * 4);
        w.ssq_head = cv.take<float>((size_t)(c.d_model / 128 + 1) * 4 * R * 4);
        w.attn_counters = cv.take<int>(attn_counter_count(c.max_batch, c.n_kv_heads) * sizeof(int));
        w.n_counters = widest / 128 + 8;
        w.gemm_counters = cv.take<int>(w.n_counters * 4);
    }
    if (ws) *ws = w;
    return align_up(cv.off, 256);
}

// Runs one launcher, bracketed by events when timing is on.
template <typename F>
int timed(viasd_model *m, int cls, cudaStream_t st, F &&f) {
    KernelTimer &t = m->timer;
    if (!t.on) return f();
    if (t.open >= 0 && t.cls[t.open] == cls) { ++t.cnt[t.open]; return f(); }     // the run goes on
    if (t.open >= 0) { CUDA_TRY(cudaEventRecord(t.end[t.open], st)); t.open = -1; }
    if (t.n >= KernelTimer::CAP) { ++t.dropped; return f(); }
    const int i = t.n++;
    t.cls[i] = cls;
    t.cnt[i] = 1;
    CUDA_TRY(cudaEventRecord(t.beg[i], st));
    t.open = i;
    return f();
}

int env_int(const char *name, int dflt) { const char *e = getenv(name); return e && *e ? atoi(e) : dflt; }

// Initial option values: the defaults, or what the VIASD_* environment variables say (read here, once per model).
void default_options(ModelOptions &o) {
    o.attn_kernel = 0;
    if (const char *e = getenv("VIASD_ATTN")) o.attn_kernel = strcmp(e, "mma") == 0 ? 1 : strcmp(e, "tc") == 0 ? 2 : strcmp(e, "tk") == 0 ? 3 : 0;
    o.attn_splits = env_int("VIASD_ATTN_NSPLIT", 0);
    o.attn_lo = env_int("VIASD_ATTN_LO", 2);
    o.accept_team = env_int("VIASD_ACCEPT_TEAM", 0);
    o.dual_max_rows = env_int("VIASD_DUAL_MAX", 128);
    o.tk_grid = env_int("VIASD_TK_GRID", 0);
    o.tk_flat = env_int("VIASD_TK_FLAT", -1);
    o.ring_kb = env_int("VIASD_TC_RING_KB", 0);
    o.epi_groups = env_int("VIASD_TC_EPI_GROUPS", 0);
}

int check_config(const viasd_config *c) {
    if (!c) return VIASD_EINVAL;
    if (c->n_layers < 1 || c->n_layers > 512 || c->d_model < 8 || c->n_heads < 1 || c->n_kv_heads < 1) return VIASD_EINVAL;
    if (c->n_heads % c->n_kv_heads) return VIASD_EINVAL;
    if (c->head_dim != 64 && c->head_dim != 128) return VIASD_EINVAL;
    if (c->d_model % 8 || c->d_ff % 8 || c->d_ff < 8 || c->vocab < 2) return VIASD_EINVAL;
    if (c->dtype != 0 && c->dtype != 1) return VIASD_EINVAL;
    if (c->max_batch < 1 || c->max_query < 1 || c->max_query > VIASD_MAX_ROWS_PER_SEQ) return VIASD_EINVAL;
    if (c->max_ctx < c->max_query) return VIASD_EINVAL;
    if (!(c->rms_eps >= 0.f) || !(c->rope_theta > 0.f)) return VIASD_EINVAL;
    return VIASD_OK;
}

int check_draft(const viasd_model *m, const viasd_draft *d) {
    if (!m || !d) return VIASD_EINVAL;
    if (d->batch < 1 || d->batch > m->cfg.max_batch) return VIASD_EINVAL;
    if (d->n_nodes < 0 || d->n_nodes + 1 > m->cfg.max_query) return VIASD_EINVAL;
    if (!d->draft_tok && d->n_nodes) return VIASD_EINVAL;
    if (!d->parent && d->n_nodes) return VIASD_EINVAL;
    return VIASD_OK;
}

int check_cache(const viasd_cache *c) {
    if (!c || !c->k_full || !c->v_full || !c->k_slim || !c->v_slim || !c->len || !c->pending) return VIASD_EINVAL;
    return VIASD_OK;
}

// One projection.  bf16 models go to the tcgen05 kernel (activation hi/lo planes through TMA); fp32 models
// and anything that kernel does not take go to the CUDA-core kernel.
struct GemmCall {
    const void *x; size_t x_plane; const ActMaps *xmaps;      // input activation buffer
    const void *w[3]; const WMap *wmap[3]; int n[3]; int count;
    int k, epi;
    float *out_f32; void *out_act; size_t act_plane; int ld_out;
};

int run_gemm(viasd_model *m, const GemmCall &g, int rows, cudaStream_t st) {
    const viasd_config &c = m->cfg;
    if (!m->use_tc) {
        GemmSegs s{{g.w[0], g.w[1], g.w[2]}, {g.n[0], g.n[1], g.n[2]}, g.count};
        return launch_gemm_rowwarp(g.x, g.x_plane, s, rows, g.k, c.dtype, g.epi, g.out_f32, g.out_act, g.act_plane,
                                   g.ld_out, st);
    }
    for (int row0 = 0; row0 < rows; row0 += 128) {
        const int nr = rows - row0 < 128 ? rows - row0 : 128;
        const int nt = tc_pick_nt(nr, true);
        const int ni = nt / 8 - 1;
        TcLaunch L;
        memset(&L, 0, sizeof(L));
        for (int i = 0; i < g.count; ++i) { L.map_w[i] = &g.wmap[i]->map; L.seg_n[i] = g.n[i]; L.w_box_rows[i] = g.wmap[i]->box_rows; }
        L.n_seg = g.count;
        L.map_x = &g.xmaps->map[ni];
        L.x_box_rows = g.xmaps->box_rows[ni];
        L.has_lo = 1;
        L.lo_row_offset = (int)m->ws.rows_alloc;
        L.rows = nr; L.row0 = row0; L.k = g.k; L.nt = nt; L.epi = g.epi;
        L.out_f32 = g.out_f32; L.out_act = g.out_act; L.act_plane = g.act_plane; L.ld_out = g.ld_out;
        L.scratch = m->ws.gemm_scratch; L.counters = m->ws.gemm_counters; L.status = &m->ws.stats->device_status;
        L.sm_count = m->sm_count;
        L.ring_kb = m->opt.ring_kb; L.epi_groups = m->opt.epi_groups;
        int rc = launch_gemm_tc(L, st);
        if (rc) return rc;
    }
    return VIASD_OK;
}

// Tensor-core path with fused epilogues: per layer QKV (+RMS scale, rotary, KV append) -> attention ->
// O (+residual, next-norm preparation) -> gate/up (+RMS scale, SwiGLU) -> down (+residual, next-norm preparation).
// mode 0: full verifier q; mode 1: slim verifier q' (routed layers only); mode 2: both in one sweep over the
// layers.  In mode 2 the block rows exist twice, [full stream; slim stream]: a routed layer's weights are streamed
// once and applied to both streams, an unrouted layer runs on the full stream only.  Results are those of the two
// separate passes; only the weight traffic of the routed layers is shared.
// replay > 0 (mode 0 only, routed execution policy): every sequence's block is extended in front by its last `replay`
// committed tokens (see prep_replay_kernel); the logits written are those of the block's own rows.
int forward_sweep(viasd_model *m, const viasd_cache *cache, const viasd_draft *d, int mode, float *logits_full,
                  float *logits_slim, cudaStream_t st, int replay = 0) {
    const viasd_config &c = m->cfg;
    const int B = d->batch, M = d->n_nodes + 1 + replay, rows = B * M;
    const int qd = c.n_heads * c.head_dim, kvd = c.n_kv_heads * c.head_dim;
    const size_t R = m->ws.rows_alloc;
    const bool dual = mode == 2;
    int rc;
    // layers this sweep visits, and for each whether the slim stream takes part
    const int n_run = mode == 1 ? m->n_routed : c.n_layers;
    auto layer_id = [&](int it) { return mode == 1 ? m->routed[it] : it; };
    auto routed_ord = [&](int l) { for (int o = 0; o < m->n_routed; ++o) if (m->routed[o] == l) return o; return -1; };
    auto next_slim_gain = [&](int l) -> const float * {       // gain of the slim stream's next norm1 after layer l
        for (int o = 0; o < m->n_routed; ++o) if (m->routed[o] > l) return m->norm1[m->routed[o]];
        return m->final_norm;
    };
    auto gemm = [&](TcLaunch L, const ActMaps &xm, int nrows) -> int {
        return timed(m, VIASD_T_GEMM, st, [&]() -> int {
            for (int row0 = 0; row0 < nrows; row0 += 128) {
                const int nr = nrows - row0 < 128 ? nrows - row0 : 128, nt = tc_pick_nt(nr, true);
                const int ni = nt / 8 - 1;
                L.map_x = &xm.map[ni]; L.x_box_rows = xm.box_rows[ni];
                L.has_lo = 1; L.lo_row_offset = (int)R;
                L.rows = nr; L.row0 = row0; L.nt = nt;
                L.scratch = m->ws.gemm_scratch; L.counters = m->ws.gemm_counters; L.status = &m->ws.stats->device_status;
                L.sm_count = m->sm_count;
                L.ring_kb = m->opt.ring_kb; L.epi_groups = m->opt.epi_groups;
                L.run_flag = m->run_flag;
                L.ssq_stride = (int)R; L.inv_d = 1.0f / (float)c.d_model; L.eps = c.rms_eps;
                L.split_row = dual ? rows : 0;
                int r2 = launch_gemm_tc(L, st);
                if (r2) return r2;
            }
            return (int)VIASD_OK;
        });
    };
    auto wseg = [&](TcLaunch &L, int i, const WMap &w, int n) { L.map_w[i] = &w.map; L.seg_n[i] = n; L.w_box_rows[i] = w.box_rows; };
    const int ssq_n = (c.d_model / 128) * 4;

    if ((rc = timed(m, VIASD_T_EMBED, st, [&] { return replay ? launch_prep_replay(m, cache, d, replay, st)
                                                              : launch_prep(m, cache, d, mode != 1, st); }))) return rc;
    if (dual) {
        if ((rc = timed(m, VIASD_T_EMBED, st, [&] { return launch_embed_norm2(m, m->norm1[0], m->norm1[m->routed[0]], rows, st); })))
            return rc;
    } else {
        if ((rc = timed(m, VIASD_T_EMBED, st, [&] { return launch_embed_norm(m, m->norm1[layer_id(0)], rows, st); }))) return rc;
    }
    for (int it = 0; it < n_run; ++it) {
        const int l = layer_id(it);
        const int so = routed_ord(l);                          // slim ordinal of this layer, -1 if unrouted
        const bool both = dual && so >= 0;
        const int nrows = both ? 2 * rows : rows;
        const LayerMaps &lm = m->lmaps[l];
        // cache and layer ordinal of the first stream
        void *kc = mode == 1 ? cache->k_slim : cache->k_full, *vc = mode == 1 ? cache->v_slim : cache->v_full;
        const int ord = mode == 1 ? it : l;
        {   // QKV: scale by 1/rms, rotate q and k, append k and v to the cache
            TcLaunch L; memset(&L, 0, sizeof(L));
            wseg(L, 0, lm.wq, qd); wseg(L, 1, lm.wk, kvd); wseg(L, 2, lm.wv, kvd); L.n_seg = 3;
            L.k = c.d_model; L.epi = EPI_QKV_ROPE; L.ld_out = qd + 2 * kvd;
            L.ssq_in = m->ws.ssq; L.ssq_in_n = ssq_n;
            L.q_out = m->ws.q; L.kc = kc; L.vc = vc; L.cosv = m->ws.rope_cos; L.sinv = m->ws.rope_sin;
            L.len_eff = m->ws.len_eff; L.depth = m->ws.tree->depth; L.tree_stride = (int)(sizeof(TreeInfo) / sizeof(int)); L.rope_M = M; L.rope_H = c.n_heads; L.rope_Hkv = c.n_kv_heads;
            L.max_batch = c.max_batch; L.max_ctx = c.max_ctx; L.layer_ord = ord;
            L.kc2 = cache->k_slim; L.vc2 = cache->v_slim; L.layer_ord2 = so;
            L.kv_keep = replay ? cache->len_full : nullptr;
            if ((rc = gemm(L, m->maps_a, nrows))) return rc;
        }
        if (both) {
            if ((rc = timed(m, VIASD_T_ATTENTION, st, [&] { return launch_attention_dual(m, cache->k_full, cache->v_full, l,
                    cache->k_slim, cache->v_slim, so, B, M, st); }))) return rc;
        } else {
            if ((rc = timed(m, VIASD_T_ATTENTION, st, [&] { return launch_attention(m, kc, vc, mode == 1, ord, B, M, st); })))
                return rc;
        }
        {   // O projection into the residual; prepare the input of the post-attention norm
            TcLaunch L; memset(&L, 0, sizeof(L));
            wseg(L, 0, lm.wo, c.d_model); L.n_seg = 1;
            L.k = qd; L.epi = EPI_ADD_NORM; L.out_f32 = m->ws.h; L.ld_out = c.d_model;
            L.next_gain = m->norm2[l]; L.next_act = m->ws.a; L.next_plane = R * c.d_model; L.ssq_out = m->ws.ssq;
            if ((rc = gemm(L, m->maps_attn, nrows))) return rc;
        }
        {   // gate / up with SwiGLU
            TcLaunch L; memset(&L, 0, sizeof(L));
            wseg(L, 0, lm.wg, c.d_ff); wseg(L, 1, lm.wu, c.d_ff); L.n_seg = 2;
            L.k = c.d_model; L.epi = EPI_SWIGLU; L.out_act = m->ws.act; L.act_plane = R * c.d_ff; L.ld_out = c.d_ff;
            L.ssq_in = m->ws.ssq; L.ssq_in_n = ssq_n;
            if ((rc = gemm(L, m->maps_a, nrows))) return rc;
        }
        {   // down projection into the residual; prepare the input of each stream's next norm
            TcLaunch L; memset(&L, 0, sizeof(L));
            wseg(L, 0, lm.wd, c.d_model); L.n_seg = 1;
            L.k = c.d_ff; L.epi = EPI_ADD_NORM; L.out_f32 = m->ws.h; L.ld_out = c.d_model;
            L.next_gain = it + 1 < n_run ? m->norm1[layer_id(it + 1)] : m->final_norm;
            L.next_gain2 = both ? next_slim_gain(l) : nullptr;
            L.next_act = m->ws.a; L.next_plane = R * c.d_model; L.ssq_out = m->ws.ssq;
            if ((rc = gemm(L, m->maps_act, nrows))) return rc;
        }
    }
    TcLaunch L; memset(&L, 0, sizeof(L));
    wseg(L, 0, m->head_map, c.vocab); L.n_seg = 1;
    L.k = c.d_model; L.epi = EPI_STORE; L.out_f32 = mode == 1 ? logits_slim : logits_full; L.out_f32_2 = logits_slim;
    L.ld_out = c.vocab;
    L.ssq_in = m->ws.ssq; L.ssq_in_n = ssq_n;
    if (replay) {
        // the head runs on the block's own rows only, packed into a buffer of their own
        if ((rc = timed(m, VIASD_T_EMBED, st, [&] { return launch_compact_head_rows(m, B, M - replay, replay, st); }))) return rc;
        L.ssq_in = m->ws.ssq_head;
        return gemm(L, m->maps_head, B * (M - replay));
    }
    return gemm(L, m->maps_a, dual ? 2 * rows : rows);
}

// One pass of the sub-network made of `layers` (all of them for q, the routed ones for q').
int forward(viasd_model *m, const viasd_cache *cache, const viasd_draft *d, bool slim, float *logits,
            cudaStream_t st) {
    int rc;
    if ((rc = check_draft(m, d)) || (rc = check_cache(cache))) return rc;
    if (!logits) return VIASD_EINVAL;
    if (m->fused) return forward_sweep(m, cache, d, slim ? 1 : 0, slim ? nullptr : logits, slim ? logits : nullptr, st);
    const viasd_config &c = m->cfg;
    const int B = d->batch, M = d->n_nodes + 1, rows = B * M;
    const int qd = c.n_heads * c.head_dim, kvd = c.n_kv_heads * c.head_dim;
    void *kc = slim ? cache->k_slim : cache->k_full, *vc = slim ? cache->v_slim : cache->v_full;
    const int n_run = slim ? m->n_routed : c.n_layers;
    const size_t R = m->ws.rows_alloc;
    const size_t pa = c.dtype ? R * c.d_model : 0, pq = c.dtype ? R * qd : 0, pf = c.dtype ? R * c.d_ff : 0;

    if ((rc = timed(m, VIASD_T_EMBED, st, [&] { return launch_prep(m, cache, d, !slim, st); }))) return rc;
    if ((rc = timed(m, VIASD_T_EMBED, st, [&] { return launch_embed(m, rows, st); }))) return rc;
    for (int ord = 0; ord < n_run; ++ord) {
        const int l = slim ? m->routed[ord] : ord;
        const LayerMaps *lm = m->use_tc ? &m->lmaps[l] : nullptr;
        if ((rc = timed(m, VIASD_T_NORM, st, [&] { return launch_rmsnorm(m, m->norm1[l], rows, st); }))) return rc;
        GemmCall qkv{m->ws.a, pa, &m->maps_a, {m->wq[l], m->wk[l], m->wv[l]},
                     {lm ? &lm->wq : nullptr, lm ? &lm->wk : nullptr, lm ? &lm->wv : nullptr}, {qd, kvd, kvd}, 3,
                     c.d_model, EPI_STORE, m->ws.qkv, nullptr, 0, qd + 2 * kvd};
        if ((rc = timed(m, VIASD_T_GEMM, st, [&] { return run_gemm(m, qkv, rows, st); }))) return rc;
        if ((rc = timed(m, VIASD_T_ROPE, st, [&] { return launch_rope_append(m, kc, vc, ord, B, M, st); }))) return rc;
        if ((rc = timed(m, VIASD_T_ATTENTION, st, [&] { return launch_attention(m, kc, vc, slim, ord, B, M, st); }))) return rc;
        GemmCall wo{m->ws.attn, pq, &m->maps_attn, {m->wo[l], nullptr, nullptr}, {lm ? &lm->wo : nullptr, nullptr, nullptr},
                    {c.d_model, 0, 0}, 1, qd, EPI_ADD, m->ws.h, nullptr, 0, c.d_model};
        if ((rc = timed(m, VIASD_T_GEMM, st, [&] { return run_gemm(m, wo, rows, st); }))) return rc;
        if ((rc = timed(m, VIASD_T_NORM, st, [&] { return launch_rmsnorm(m, m->norm2[l], rows, st); }))) return rc;
        GemmCall gu{m->ws.a, pa, &m->maps_a, {m->wg[l], m->wu[l], nullptr}, {lm ? &lm->wg : nullptr, lm ? &lm->wu : nullptr, nullptr},
                    {c.d_ff, c.d_ff, 0}, 2, c.d_model, EPI_SWIGLU, nullptr, m->ws.act, pf, c.d_ff};
        if ((rc = timed(m, VIASD_T_GEMM, st, [&] { return run_gemm(m, gu, rows, st); }))) return rc;
        GemmCall wd{m->ws.act, pf, &m->maps_act, {m->wd[l], nullptr, nullptr}, {lm ? &lm->wd : nullptr, nullptr, nullptr},
                    {c.d_model, 0, 0}, 1, c.d_ff, EPI_ADD, m->ws.h, nullptr, 0, c.d_model};
        if ((rc = timed(m, VIASD_T_GEMM, st, [&] { return run_gemm(m, wd, rows, st); }))) return rc;
    }
    if ((rc = timed(m, VIASD_T_NORM, st, [&] { return launch_rmsnorm(m, m->final_norm, rows, st); }))) return rc;
    GemmCall head{m->ws.a, pa, &m->maps_a, {m->lm_head, nullptr, nullptr}, {m->use_tc ? &m->head_map : nullptr, nullptr, nullptr},
                  {c.vocab, 0, 0}, 1, c.d_model, EPI_STORE, logits, nullptr, 0, c.vocab};
    return timed(m, VIASD_T_GEMM, st, [&] { return run_gemm(m, head, rows, st); });
}

int check_params(const viasd_params *p) {
    if (!p) return VIASD_EINVAL;
    if (!(p->log_tau_lo <= p->log_tau_hi)) return VIASD_EINVAL;
    if (p->conf_source != 0 && p->conf_source != 1) return VIASD_EINVAL;
    if (p->mode != 0 && p->mode != 1) return VIASD_EINVAL;
    if (p->mode == 1 && !(p->temperature > 0.f)) return VIASD_EINVAL;
    if (!(p->alpha >= 0.f && p->alpha < 1.f) || !(p->beta > 0.f)) return VIASD_EINVAL;
    if (p->policy != 0 && p->policy != 1) return VIASD_EINVAL;
    return VIASD_OK;
}

int check_result(const viasd_result *r, int phase) {
    if (!r || !r->tier) return VIASD_EINVAL;
    if ((phase & 1) && !r->conf) return VIASD_EINVAL;
    if ((phase & 2) && (!r->n_acc || !r->path || !r->out_tok || !r->n_emit || !r->judge || !r->corr_src))
        return VIASD_EINVAL;
    return VIASD_OK;
}

}  // namespace

extern "C" {

size_t viasd_workspace_bytes(const viasd_config *cfg, int n_routed) {
    (void)n_routed;
    if (check_config(cfg)) return 0;
    return carve(*cfg, nullptr, nullptr);
}

int viasd_init_model(const viasd_config *cfg, const viasd_weights *w, const unsigned char *route_mask,
                     void *workspace, size_t workspace_bytes, viasd_model **out) {
    int rc = check_config(cfg);
    if (rc) return rc;
    if (!w || !route_mask || !workspace || !out) return VIASD_EINVAL;
    if (((uintptr_t)workspace & 255) != 0) return VIASD_EINVAL;
    if (!w->embed || !w->lm_head || !w->final_norm || !w->wq || !w->wk || !w->wv || !w->wo || !w->wg || !w->wu ||
        !w->wd || !w->norm1 || !w->norm2) return VIASD_EINVAL;
    if (workspace_bytes < carve(*cfg, nullptr, nullptr)) return VIASD_ECAPACITY;
    int dev = 0;
    cudaDeviceProp prop;
    CUDA_TRY(cudaGetDevice(&dev));
    CUDA_TRY(cudaGetDeviceProperties(&prop, dev));
    if (prop.major != 10) return VIASD_EUNSUPPORTED;

    if (g_use_pdl < 0) { const char *e = getenv("VIASD_PDL"); g_use_pdl = (e && e[0] == '0') ? 0 : 1; }
    viasd_model *m = new (std::nothrow) viasd_model();
    if (!m) return VIASD_EINVAL;
    memset(&m->timer, 0, sizeof(m->timer));
    default_options(m->opt);
    m->cfg = *cfg;
    m->sm_count = prop.multiProcessorCount;
    m->n_routed = 0;
    for (int l = 0; l < cfg->n_layers; ++l) if (route_mask[l]) m->routed[m->n_routed++] = l;
    if (m->n_routed == 0) { delete m; return VIASD_EINVAL; }
    const int L = cfg->n_layers;
    const void ***arrs[] = {&m->wq, &m->wk, &m->wv, &m->wo, &m->wg, &m->wu, &m->wd};
    const void *const *srcs[] = {w->wq, w->wk, w->wv, w->wo, w->wg, w->wu, w->wd};
    for (int i = 0; i < 7; ++i) {
        *arrs[i] = new const void *[L];
        for (int l = 0; l < L; ++l) {
            if (!srcs[i][l] || ((uintptr_t)srcs[i][l] & 15)) { viasd_free_model(m); return VIASD_EINVAL; }
            (*arrs[i])[l] = srcs[i][l];
        }
    }
    m->norm1 = new const float *[L];
    m->norm2 = new const float *[L];
    for (int l = 0; l < L; ++l) {
        if (!w->norm1[l] || !w->norm2[l]) { viasd_free_model(m); return VIASD_EINVAL; }
        m->norm1[l] = w->norm1[l];
        m->norm2[l] = w->norm2[l];
    }
    m->embed = w->embed; m->lm_head = w->lm_head; m->final_norm = w->final_norm;
    carve(*cfg, (char *)workspace, &m->ws);
    {
        const char *force = getenv("VIASD_GEMM");
        m->use_tc = cfg->dtype == 1 && m->sm_count <= MAX_SMS && !(force && strcmp(force, "rowwarp") == 0);
    }
    {
        const char *nf = getenv("VIASD_FUSED");
        m->fused = m->use_tc && cfg->head_dim == 128 && cfg->d_model % 128 == 0 && !(nf && nf[0] == '0');
    }
    if (m->use_tc) {
        const uint64_t d = cfg->d_model, qd = (uint64_t)cfg->n_heads * cfg->head_dim,
                       kvd = (uint64_t)cfg->n_kv_heads * cfg->head_dim, ff = cfg->d_ff, R = m->ws.rows_alloc;
        m->lmaps = new (std::nothrow) LayerMaps[L];
        auto wm = [&](WMap &o, const void *base, uint64_t n, uint64_t k) {
            o.box_rows = tc_box_rows(n, 128);
            return tc_make_map(&o.map, base, n, k, o.box_rows);
        };
        rc = m->lmaps ? VIASD_OK : VIASD_EINVAL;
        for (int l = 0; l < L && !rc; ++l) {
            LayerMaps &lm = m->lmaps[l];
            if ((rc = wm(lm.wq, m->wq[l], qd, d)) || (rc = wm(lm.wk, m->wk[l], kvd, d)) || (rc = wm(lm.wv, m->wv[l], kvd, d)) ||
                (rc = wm(lm.wo, m->wo[l], d, qd)) || (rc = wm(lm.wg, m->wg[l], ff, d)) || (rc = wm(lm.wu, m->wu[l], ff, d)) ||
                (rc = wm(lm.wd, m->wd[l], d, ff))) break;
        }
        if (!rc) rc = wm(m->head_map, m->lm_head, cfg->vocab, d);
        auto am = [&](ActMaps &o, const void *base, uint64_t k) {
            for (int i = 0; i < 16; ++i) {
                o.box_rows[i] = tc_box_rows(2 * R, 8 * (i + 1));
                int r2 = tc_make_map(&o.map[i], base, 2 * R, k, o.box_rows[i]);
                if (r2) return r2;
            }
            return (int)VIASD_OK;
        };
        if (!rc) rc = am(m->maps_a, m->ws.a, d);
        if (!rc) rc = am(m->maps_attn, m->ws.attn, qd);
        if (!rc) rc = am(m->maps_act, m->ws.act, ff);
        if (!rc) rc = am(m->maps_head, m->ws.a_head, d);
        if (rc) { viasd_free_model(m); return rc; }
    }
    m->run_flag = nullptr;
    cudaError_t e = cudaMemset(m->ws.stats, 0, sizeof(DeviceStats));
    if (e == cudaSuccess) { const int one = 1; e = cudaMemcpy(&m->ws.stats->full_ran, &one, sizeof(int), cudaMemcpyHostToDevice); }
    if (e == cudaSuccess) e = cudaMemset(m->ws.gemm_counters, 0, m->ws.n_counters * 4);
    if (e == cudaSuccess) e = cudaMemset(m->ws.attn_counters, 0, attn_counter_count(cfg->max_batch, cfg->n_kv_heads) * sizeof(int));
    if (e == cudaSuccess) { rc = launch_rope_table(m, 0); if (rc == VIASD_OK) e = cudaDeviceSynchronize(); }
    if (e != cudaSuccess) { g_last_cuda_error = (int)e; rc = VIASD_ECUDA; }
    if (rc) { viasd_free_model(m); return rc; }
    *out = m;
    return VIASD_OK;
}

void viasd_free_model(viasd_model *m) {
    if (!m) return;
    const void ***arrs[] = {&m->wq, &m->wk, &m->wv, &m->wo, &m->wg, &m->wu, &m->wd};
    for (int i = 0; i < 7; ++i) delete[] *arrs[i];
    delete[] m->norm1;
    delete[] m->norm2;
    delete[] m->lmaps;
    for (int i = 0; i < m->timer.created; ++i) { cudaEventDestroy(m->timer.beg[i]); cudaEventDestroy(m->timer.end[i]); }
    delete[] m->timer.beg;
    delete[] m->timer.end;
    delete[] m->timer.cls;
    delete[] m->timer.cnt;
    delete m;
}

int viasd_full_forward(viasd_model *m, const viasd_cache *cache, const viasd_draft *draft, float *logits, void *stream) {
    return forward(m, cache, draft, false, logits, (cudaStream_t)stream);
}

int viasd_slim_forward(viasd_model *m, const viasd_cache *cache, const viasd_draft *draft, float *logits, void *stream) {
    return forward(m, cache, draft, true, logits, (cudaStream_t)stream);
}

static int tier_accept_set(viasd_model *m, const viasd_draft *draft, const viasd_params *params, const JudgeSet &js,
                           int phase, viasd_result *result, bool tree_ready, void *stream) {
    int rc;
    if ((rc = check_draft(m, draft)) || (rc = check_params(params))) return rc;
    if (phase < 1 || phase > 3) return VIASD_EINVAL;
    if ((rc = check_result(result, phase))) return rc;
    if (draft->n_nodes < 1 || !draft->prow || !draft->drafter_logits || draft->n_prows < 1) return VIASD_EINVAL;
    for (int k = 1; k < js.n; ++k) if (!(js.log_tau[k] <= js.log_tau[k - 1])) return VIASD_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    if (phase & 1) {
        if ((rc = timed(m, VIASD_T_TIER_ACCEPT, st, [&] { return launch_tier(m, draft, params, js, result, st); }))) return rc;
    }
    if (phase & 2) {
        for (int k = 0; k < js.n; ++k) if (!js.logits[k]) return VIASD_EINVAL;
        if ((rc = timed(m, VIASD_T_TIER_ACCEPT, st, [&] { return launch_accept(m, draft, params, js, result, tree_ready, st); })))
            return rc;
    }
    return VIASD_OK;
}

static int tier_accept_impl(viasd_model *m, const viasd_draft *draft, const viasd_params *params, const float *slim_logits,
                           const float *full_logits, int phase, viasd_result *result, bool tree_ready, void *stream) {
    if (!params) return VIASD_EINVAL;
    JudgeSet js{2, {slim_logits, full_logits}, {params->log_tau_hi, params->log_tau_lo}};
    return tier_accept_set(m, draft, params, js, phase, result, tree_ready, stream);
}

int viasd_tier_accept(viasd_model *m, const viasd_draft *draft, const viasd_params *params, const float *slim_logits,
                      const float *full_logits, int phase, viasd_result *result, void *stream) {
    return tier_accept_impl(m, draft, params, slim_logits, full_logits, phase, result, false, stream);
}

int viasd_tier_accept_n(viasd_model *m, const viasd_draft *draft, const viasd_params *params, int n_judges,
                        const float *log_tau, const float *const *judge_logits, int phase, viasd_result *result,
                        void *stream) {
    if (!params || n_judges < 1 || n_judges > VIASD_MAX_JUDGES || !log_tau || !judge_logits) return VIASD_EINVAL;
    JudgeSet js;
    js.n = n_judges;
    for (int k = 0; k < VIASD_MAX_JUDGES; ++k) {
        js.logits[k] = k < n_judges ? judge_logits[k] : nullptr;
        js.log_tau[k] = k < n_judges ? log_tau[k] : 0.f;
    }
    // the thresholds of viasd_params play no part here, but its other fields are checked as usual
    viasd_params p = *params;
    p.log_tau_hi = js.log_tau[0];
    p.log_tau_lo = js.log_tau[n_judges - 1];
    return tier_accept_set(m, draft, &p, js, phase, result, false, stream);
}

int viasd_kv_commit(viasd_model *m, viasd_cache *cache, const viasd_draft *draft, const viasd_result *result,
                    void *stream) {
    int rc;
    if ((rc = check_draft(m, draft)) || (rc = check_cache(cache))) return rc;
    if (!result || !result->n_acc || !result->path || !result->out_tok || !result->n_emit) return VIASD_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    return timed(m, VIASD_T_COMMIT, st, [&] { return launch_commit(m, cache, draft, result, false, st); });
}

int viasd_kv_commit_slim(viasd_model *m, viasd_cache *cache, const viasd_draft *draft, const viasd_result *result,
                         void *stream) {
    int rc;
    if ((rc = check_draft(m, draft)) || (rc = check_cache(cache))) return rc;
    if (!result || !result->n_acc || !result->path) return VIASD_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    return timed(m, VIASD_T_COMMIT, st, [&] { return launch_commit(m, cache, draft, result, true, st); });
}

// Routed execution policy (policy 1): the full verifier is invoked only when the walk needs it.
//   tier -> slim pass -> probe (the accept walk on q' alone; raises the device flag when a tier-2 node is reached
//   before the first break, a bonus token is due, or the backlog would outgrow the replay window) -> full pass, every
//   kernel of which leaves at once when the flag is zero -> accept -> commit (len_full follows len only if q ran).
// The full pass is a replay pass: the block is extended in front by the last G = max_query - M committed tokens, which
// closes whatever gap skipped passes left in q's cache; q' keeps its cache current in every step.  No host decision,
// no device-to-host traffic.  Results are those of policy 0 (the passes compute the same distributions).
static int verify_step_routed(viasd_model *m, viasd_cache *cache, const viasd_draft *draft, const viasd_params *params,
                              float *slim_logits, float *full_logits, viasd_result *result, void *stream) {
    int rc;
    if ((rc = check_draft(m, draft)) || (rc = check_cache(cache))) return rc;
    if (!m->fused || !cache->len_full || !cache->tokens) return VIASD_EINVAL;
    const int M = draft->n_nodes + 1, G = m->cfg.max_query - M;
    if (G < 1) return VIASD_ECAPACITY;                        // no room for replayed rows: size max_query above M
    cudaStream_t st = (cudaStream_t)stream;
    int *flag = &m->ws.stats->full_ran;
    if (params->conf_source == 0) {
        if ((rc = viasd_tier_accept(m, draft, params, nullptr, nullptr, 1, result, stream))) return rc;
        if ((rc = forward_sweep(m, cache, draft, 1, nullptr, slim_logits, st))) return rc;
    } else {
        if ((rc = forward_sweep(m, cache, draft, 1, nullptr, slim_logits, st))) return rc;
        if ((rc = viasd_tier_accept(m, draft, params, slim_logits, nullptr, 1, result, stream))) return rc;
    }
    CUDA_TRY(cudaMemsetAsync(flag, 0, sizeof(int), st));
    AcceptProbe probe{G, flag, cache->len, cache->len_full};
    JudgeSet probe_set{2, {slim_logits, nullptr}, {params->log_tau_hi, params->log_tau_lo}};
    if ((rc = timed(m, VIASD_T_TIER_ACCEPT, st, [&] { return launch_accept(m, draft, params, probe_set, result, true, st,
                                                                      &probe); }))) return rc;
    m->run_flag = flag;
    rc = forward_sweep(m, cache, draft, 0, full_logits, nullptr, st, G);
    m->run_flag = nullptr;
    if (rc) return rc;
    if ((rc = tier_accept_impl(m, draft, params, slim_logits, full_logits, 2, result, false, stream))) return rc;
    return viasd_kv_commit(m, cache, draft, result, stream);
}

int viasd_verify_step(viasd_model *m, viasd_cache *cache, const viasd_draft *draft, const viasd_params *params,
                      float *slim_logits, float *full_logits, viasd_result *result, void *stream) {
    int rc;
    if (!slim_logits || !full_logits) return VIASD_EINVAL;
    if ((rc = check_params(params))) return rc;
    if (params->policy == 1) return verify_step_routed(m, cache, draft, params, slim_logits, full_logits, result, stream);
    // Both verifiers in one sweep over the layers (routed layers' weights are read once for both) while the two
    // row streams together fit one launch (128 token rows: an MMA of 256 columns with the hi/lo planes); beyond
    // that a sweep would stream every routed layer twice anyway, and the passes run one after the other.
    if (m && m->fused && draft && 2 * draft->batch * (draft->n_nodes + 1) <= m->opt.dual_max_rows) {
        if ((rc = check_draft(m, draft)) || (rc = check_cache(cache))) return rc;
        if ((rc = forward_sweep(m, cache, draft, 2, full_logits, slim_logits, (cudaStream_t)stream))) return rc;
        if ((rc = tier_accept_impl(m, draft, params, slim_logits, full_logits, 3, result, true, stream))) return rc;
        return viasd_kv_commit(m, cache, draft, result, stream);
    }
    if (params->conf_source == 0) {
        if ((rc = viasd_tier_accept(m, draft, params, nullptr, nullptr, 1, result, stream))) return rc;
        if ((rc = viasd_slim_forward(m, cache, draft, slim_logits, stream))) return rc;
    } else {
        if ((rc = viasd_slim_forward(m, cache, draft, slim_logits, stream))) return rc;
        if ((rc = viasd_tier_accept(m, draft, params, slim_logits, nullptr, 1, result, stream))) return rc;
    }
    if ((rc = viasd_full_forward(m, cache, draft, full_logits, stream))) return rc;
    if ((rc = tier_accept_impl(m, draft, params, slim_logits, full_logits, 2, result, true, stream))) return rc;
    return viasd_kv_commit(m, cache, draft, result, stream);
}

int viasd_get_stats(viasd_model *m, viasd_stats *host_out, void *stream) {
    if (!m || !host_out) return VIASD_EINVAL;
    DeviceStats s;
    CUDA_TRY(cudaMemcpyAsync(&s, m->ws.stats, sizeof(s), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    host_out->steps = s.steps;
    for (int i = 0; i < 3; ++i) host_out->tier_count[i] = s.tier_count[i];
    host_out->emitted = s.emitted;
    host_out->accepted = s.accepted;
    host_out->device_status = s.device_status;
    host_out->need_slim = s.need_slim;
    host_out->need_full = s.need_full;
    host_out->full_ran = s.full_ran;
    host_out->full_skipped = s.full_skipped;
    return VIASD_OK;
}

int viasd_set_option(viasd_model *m, int option, int value) {
    if (!m) return VIASD_EINVAL;
    ModelOptions &o = m->opt;
    switch (option) {
    case VIASD_OPT_ATTENTION_KERNEL: if (value < 0 || value > 3) return VIASD_EINVAL; o.attn_kernel = value; break;
    case VIASD_OPT_ATTENTION_SPLITS: if (value < 0 || value > 16) return VIASD_EINVAL; o.attn_splits = value; break;
    case VIASD_OPT_ATTENTION_LO: if (value < 0 || value > 2) return VIASD_EINVAL; o.attn_lo = value; break;
    case VIASD_OPT_ACCEPT_TEAM: if (value != 0 && value != 1 && value != 2 && value != 4 && value != 8) return VIASD_EINVAL; o.accept_team = value; break;
    case VIASD_OPT_DUAL_MAX_ROWS: if (value < 0 || value > 128) return VIASD_EINVAL; o.dual_max_rows = value; break;
    case VIASD_OPT_TK_GRID: if (value < 0) return VIASD_EINVAL; o.tk_grid = value; break;
    case VIASD_OPT_TK_FLAT: if (value < -1 || value > 1) return VIASD_EINVAL; o.tk_flat = value; break;
    case VIASD_OPT_GEMM_RING_KB: if (value != 0 && (value < 32 || value > 200)) return VIASD_EINVAL; o.ring_kb = value; break;
    case VIASD_OPT_GEMM_EPI_GROUPS: if (value < 0 || value > 2) return VIASD_EINVAL; o.epi_groups = value; break;
    default: return VIASD_EINVAL;
    }
    return VIASD_OK;
}

const char *viasd_strerror(int code) {
    switch (code) {
    case VIASD_OK: return "ok";
    case VIASD_EINVAL: return "invalid argument";
    case VIASD_ECAPACITY: return "capacity exceeded";
    case VIASD_ECUDA: return "CUDA runtime error";
    case VIASD_EDEVICE: return "device-side check failed";
    case VIASD_EUNSUPPORTED: return "unsupported device";
    default: return "unknown error";
    }
}

int viasd_last_cuda_error(void) { return g_last_cuda_error; }

unsigned long long viasd_launch_count(void) { return g_launch_count; }

int viasd_set_timing(viasd_model *m, int on) {
    if (!m) return VIASD_EINVAL;
    KernelTimer &t = m->timer;
    if (on && !t.beg) {
        t.beg = new cudaEvent_t[KernelTimer::CAP];
        t.end = new cudaEvent_t[KernelTimer::CAP];
        t.cls = new int[KernelTimer::CAP];
        t.cnt = new int[KernelTimer::CAP];
        for (t.created = 0; t.created < KernelTimer::CAP; ++t.created) {
            CUDA_TRY(cudaEventCreate(&t.beg[t.created]));
            CUDA_TRY(cudaEventCreate(&t.end[t.created]));
        }
    }
    t.on = on != 0;
    t.n = 0;
    t.open = -1;
    t.dropped = 0;
    return VIASD_OK;
}

int viasd_get_timing(viasd_model *m, viasd_timing *out, void *stream) {
    if (!m || !out) return VIASD_EINVAL;
    KernelTimer &t = m->timer;
    if (t.open >= 0) { CUDA_TRY(cudaEventRecord(t.end[t.open], (cudaStream_t)stream)); t.open = -1; }
    CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    memset(out, 0, sizeof(*out));
    for (int i = 0; i < t.n; ++i) {
        float ms = 0.f;
        CUDA_TRY(cudaEventElapsedTime(&ms, t.beg[i], t.end[i]));
        out->ms[t.cls[i]] += ms;
        out->launches[t.cls[i]] += t.cnt[i];
    }
    out->dropped = t.dropped;
    t.n = 0;
    t.dropped = 0;
    return VIASD_OK;
}

size_t viasd_gemm_scratch_bytes(int rows, int n, int k) {
    (void)k;
    if (rows < 1 || n < 1) return 256;
    const int nt = tc_pick_nt(rows < 128 ? rows : 128, false);
    // [tile counters | one status word] then the partial-tile slots
    return align_up((size_t)(tc_tiles(n) + 1) * 4, 256) + tc_scratch_floats(MAX_GEMM_CTAS, nt, false) * 4;
}

int viasd_gemm(const void *x, const void *w, float *y, int rows, int n, int k, int dtype, void *scratch,
               size_t scratch_bytes, void *stream) {
    if (!x || !w || !y || rows < 1 || rows > 256 || n < 1 || k < 8 || (k % 8) || (dtype != 0 && dtype != 1)) return VIASD_EINVAL;
    if (((uintptr_t)x & 15) || ((uintptr_t)w & 15)) return VIASD_EINVAL;
    if (!scratch || ((uintptr_t)scratch & 255)) return VIASD_EINVAL;
    if (scratch_bytes < viasd_gemm_scratch_bytes(rows, n, k)) return VIASD_ECAPACITY;
    cudaStream_t st = (cudaStream_t)stream;
    if (g_use_pdl < 0) { const char *e = getenv("VIASD_PDL"); g_use_pdl = (e && e[0] == '0') ? 0 : 1; }
    const char *force = getenv("VIASD_GEMM");
    if (dtype == 0 || (force && strcmp(force, "rowwarp") == 0)) {
        GemmSegs s{{w, nullptr, nullptr}, {n, 0, 0}, 1};
        return launch_gemm_rowwarp(x, 0, s, rows, k, dtype, EPI_STORE, y, nullptr, 0, n, st);
    }
    int dev = 0, sms = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    if (sms > MAX_SMS) sms = MAX_SMS;
    const size_t counter_bytes = align_up((size_t)(tc_tiles(n) + 1) * 4, 256);
    CUDA_TRY(cudaMemsetAsync(scratch, 0, counter_bytes, st));       // tile counters and the status word
    CUtensorMap mw, mx;
    int rc;
    const uint32_t wbox = tc_box_rows(n, 128);
    if ((rc = tc_make_map(&mw, w, n, k, wbox))) return rc;
    for (int row0 = 0; row0 < rows; row0 += 128) {
        const int nr = rows - row0 < 128 ? rows - row0 : 128;
        const int nt = tc_pick_nt(nr, false);
        const uint32_t xbox = tc_box_rows(rows, nt);
        if ((rc = tc_make_map(&mx, x, rows, k, xbox))) return rc;
        TcLaunch L;
        memset(&L, 0, sizeof(L));
        L.map_w[0] = &mw; L.seg_n[0] = n; L.w_box_rows[0] = wbox; L.n_seg = 1;
        L.map_x = &mx; L.x_box_rows = xbox; L.has_lo = 0; L.lo_row_offset = 0;
        L.rows = nr; L.row0 = row0; L.k = k; L.nt = nt; L.epi = EPI_STORE;
        L.out_f32 = y; L.ld_out = n;
        L.counters = (int *)scratch;
        L.scratch = (float *)((char *)scratch + counter_bytes);
        L.status = (int *)scratch + tc_tiles(n);                    // no handle here: an expired wait is recorded there
        L.sm_count = sms;
        if ((rc = launch_gemm_tc(L, st))) return rc;
    }
    return VIASD_OK;
}

// What the last viasd_gemm call that used this scratch recorded (n as in that call): VIASD_OK, or VIASD_EDEVICE when
// one of its bounded waits expired.  Synchronises `stream`.
int viasd_gemm_status(const void *scratch, int n, int *host_out, void *stream) {
    if (!scratch || !host_out || n < 1) return VIASD_EINVAL;
    CUDA_TRY(cudaMemcpyAsync(host_out, (const int *)scratch + tc_tiles(n), sizeof(int), cudaMemcpyDeviceToHost,
                             (cudaStream_t)stream));
    CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    return VIASD_OK;
}

}  // extern "C"
