// KV-append attention for bf16 caches on tensor cores, K/V tiles staged by TMA.
//
// One CTA serves one (sequence, kv head, key range): the query rows are the G = H / Hkv query heads
// of that kv head times the M block rows (G * M <= 128), so every K/V byte is read once for all of them.
// Keys are the committed cache rows 0..n-1 plus the M block rows at slots n..n+M-1, the latter masked
// per query row by its ancestor bit set (causal for a chain, tree mask otherwise).
//
// K and V tiles of 128 keys arrive through 2-D TMA boxes (64 dims x 128 keys, 128-byte swizzle) into a
// two-stage ring; scores S = Q K^T and the update O += P V run on mma.sync m16n8k16 with fp32
// accumulation.  Q and P are each used as bf16 hi + lo pairs so that only the cache itself is bf16.
// Work split inside the CTA: with at most two 16-row query tiles every warp takes 32 of the 128 keys of a
// tile and keeps its own online-softmax state (merged through shared memory at the end); with more
// query tiles the warps split the query tiles and walk all keys.
// The result is written normalised when one CTA covers all keys, else as (O, m, l) partials that
// attention_combine merges.  The only waits are on TMA arrival and are bounded.
#include "common.cuh"

namespace {

constexpr int HD = 128;
constexpr int TKEYS = 128;                 // keys per stage
constexpr int SUB = 32;                    // keys per warp step
constexpr int NSTAGE = 2;
constexpr int WARPS = 4;
constexpr uint32_t HALF_BYTES = TKEYS * 128;             // one 64-dim half of a K or V tile
constexpr uint32_t STAGE_BYTES = 4 * HALF_BYTES;         // K lo/hi halves + V lo/hi halves = 64 KB
constexpr long long WAIT_LIMIT = 4000000000ll;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int *status) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    int spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 255) == 0 && clock64() - t0 > WAIT_LIMIT) { atomicExch(status, VIASD_EDEVICE); return false; }
    }
    return true;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}
// hi = bf16(x), lo = bf16(x - hi), both packed for two values
__device__ __forceinline__ void split2(float x0, float x1, uint32_t &hi, uint32_t &lo) {
    __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
    hi = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
    lo = pack_bf16(x0 - __bfloat162float(h0), x1 - __bfloat162float(h1));
}

// byte offset of (row, 16-byte chunk) in a 128-byte-swizzled tile whose rows are 128 bytes
__device__ __forceinline__ uint32_t sw128(int row, int chunk) { return (uint32_t)row * 128u + (uint32_t)((chunk ^ (row & 7)) << 4); }
// Q tile: rows of 256 bytes (128 bf16), 16 chunks, swizzled on the low three chunk bits
__device__ __forceinline__ uint32_t qoff(int row, int chunk) { return (uint32_t)row * 256u + (uint32_t)((chunk ^ (row & 7)) << 4); }

struct AttnArgs {
    const float *q;             // [rows, H * HD] rotated queries
    float *part;                // [b][h][i][split][HD + 2]
    __nv_bfloat16 *out;         // attention output planes (nsplit == 1)
    size_t out_plane;
    const int *len_eff;
    const TreeInfo *tree;
    int *status;
    int M, H, Hkv, max_batch, max_ctx, layer_ord, nsplit, mt;   // mt = query tiles of 16 rows
    int batch, layer_ord2;      // second row stream (blockIdx.z = 1): rows batch*M.., its own cache and layer ordinal
    float scale;
};

// One warp, one 16-row query tile, 32 keys starting at key index kbase (tile-relative row r0 in the stage).
__device__ __forceinline__ void tile_step(uint32_t qhi, uint32_t qlo, int mrow0, uint32_t kst, uint32_t vst, int r0, int lane,
                                          int jbase, int n_ctx, int k_end, unsigned long long anc0, unsigned long long anc1,
                                          float (&mrun)[2], float (&lrun)[2], float (&o)[16][4]) {
    float s[4][4];
#pragma unroll
    for (int n = 0; n < 4; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) s[n][e] = 0.f;
    // S = Q K^T over the 128 dims: 8 k-steps, dims 0..63 in the first half tile, 64..127 in the second
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
        uint32_t ah[4], al[4];
        const int arow = mrow0 + (lane & 7) + ((lane >> 3) & 1) * 8, achunk = ks * 2 + (lane >> 4);
        ldsm_x4(qhi + qoff(arow, achunk), ah);
        ldsm_x4(qlo + qoff(arow, achunk), al);
        const uint32_t khalf = kst + (ks >> 2) * HALF_BYTES;
        const int kchunk = (ks & 3) * 2;
#pragma unroll
        for (int np = 0; np < 2; ++np) {        // two n-tiles (16 keys) per ldmatrix.x4
            uint32_t b[4];
            const int krow = r0 + np * 16 + (lane & 7) + ((lane >> 4) & 1) * 8, kc = kchunk + ((lane >> 3) & 1);
            ldsm_x4(khalf + sw128(krow, kc), b);
            mma16816(s[np * 2], ah, b[0], b[1]);
            mma16816(s[np * 2], al, b[0], b[1]);
            mma16816(s[np * 2 + 1], ah, b[2], b[3]);
            mma16816(s[np * 2 + 1], al, b[2], b[3]);
        }
    }
    // mask, online softmax (rows g and g + 8 of the tile; columns 8n + 2t, 8n + 2t + 1)
    const int t2 = (lane & 3) * 2;
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int n = 0; n < 4; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int j = jbase + n * 8 + t2 + (e & 1);
            const unsigned long long anc = (e < 2) ? anc0 : anc1;
            const bool ok = j < k_end && (j < n_ctx || ((anc >> (j - n_ctx)) & 1ull));
            s[n][e] = ok ? s[n][e] : -INFINITY;
            mx[e >> 1] = fmaxf(mx[e >> 1], s[n][e]);
        }
    float corr[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
        mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
        const float mnew = fmaxf(mrun[r], mx[r]);
        corr[r] = (mnew == -INFINITY) ? 1.f : expf(mrun[r] - mnew);
        mrun[r] = mnew;
    }
    float rs[2] = {0.f, 0.f};
#pragma unroll
    for (int n = 0; n < 4; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float m = mrun[e >> 1];
            const float p = (s[n][e] == -INFINITY) ? 0.f : expf(s[n][e] - m);
            s[n][e] = p;
            rs[e >> 1] += p;
        }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        rs[r] += __shfl_xor_sync(0xffffffffu, rs[r], 1);
        rs[r] += __shfl_xor_sync(0xffffffffu, rs[r], 2);
        lrun[r] = lrun[r] * corr[r] + rs[r];
    }
#pragma unroll
    for (int n = 0; n < 16; ++n) { o[n][0] *= corr[0]; o[n][1] *= corr[0]; o[n][2] *= corr[1]; o[n][3] *= corr[1]; }
    // O += P V: two k-steps of 16 keys, 16 n-tiles of 8 dims
#pragma unroll
    for (int ks = 0; ks < 2; ++ks) {
        uint32_t ph[4], pl[4];
        split2(s[2 * ks][0], s[2 * ks][1], ph[0], pl[0]);
        split2(s[2 * ks][2], s[2 * ks][3], ph[1], pl[1]);
        split2(s[2 * ks + 1][0], s[2 * ks + 1][1], ph[2], pl[2]);
        split2(s[2 * ks + 1][2], s[2 * ks + 1][3], ph[3], pl[3]);
#pragma unroll
        for (int np = 0; np < 8; ++np) {        // two n-tiles (16 dims) per ldmatrix.x4.trans
            uint32_t b[4];
            const int vrow = r0 + ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
            const int dchunk = np * 2 + (lane >> 4);                 // 16-byte chunk of the 128 dims
            const uint32_t vhalf = vst + (dchunk >> 3) * HALF_BYTES;
            ldsm_x4_t(vhalf + sw128(vrow, dchunk & 7), b);
            mma16816(o[np * 2], ph, b[0], b[1]);
            mma16816(o[np * 2], pl, b[0], b[1]);
            mma16816(o[np * 2 + 1], ph, b[2], b[3]);
            mma16816(o[np * 2 + 1], pl, b[2], b[3]);
        }
    }
}

// KEYSPLIT: warps split the keys of a stage (query tiles <= 2); else warps split the query tiles (<= 8)
template <bool KEYSPLIT>
__global__ void __launch_bounds__(WARPS * 32)
attention_mma_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                     const __grid_constant__ CUtensorMap map_k2, const __grid_constant__ CUtensorMap map_v2, const AttnArgs a) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) unsigned long long bars[NSTAGE];
    constexpr int MTW = 2;                                   // query tiles per warp at most
    PDL_TRIGGER();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.x / a.Hkv, g = blockIdx.x % a.Hkv, split = blockIdx.y, stream = blockIdx.z;
    const int be = stream * a.batch + b;                     // row block of this (stream, sequence)
    const CUtensorMap *mk = stream ? &map_k2 : &map_k, *mv = stream ? &map_v2 : &map_v;
    const int grp = a.H / a.Hkv, QR = grp * a.M, QRP = a.mt * 16;
    const int n_ctx = a.len_eff[b], Tk = n_ctx + a.M;
    int chunk = (Tk + a.nsplit - 1) / a.nsplit;
    chunk = (chunk + TKEYS - 1) / TKEYS * TKEYS;
    const int k_begin = split * chunk, k_end = min(Tk, k_begin + chunk);
    const int n_tiles = k_end > k_begin ? (k_end - k_begin + TKEYS - 1) / TKEYS : 0;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t qhi = base + NSTAGE * STAGE_BYTES, qlo = qhi + (uint32_t)QRP * 256u;
    uint8_t *gen_base = smem_raw + (base - smem_u32(smem_raw));

    if (threadIdx.x == 0) {
        for (int s = 0; s < NSTAGE; ++s) mbar_init(smem_u32(&bars[s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    // first rows of this (layer, sequence, kv head) in the cache viewed as a 2-D tensor [rows, HD]
    const int row_base = (((stream ? a.layer_ord2 : a.layer_ord) * a.max_batch + b) * a.Hkv + g) * a.max_ctx;
    auto issue = [&](int tile) {
        const int st = tile % NSTAGE;
        const uint32_t bar = smem_u32(&bars[st]), dst = base + st * STAGE_BYTES;
        const int y = row_base + k_begin + tile * TKEYS;
        mbar_expect_tx(bar, STAGE_BYTES);
        tma_load_2d(dst, mk, bar, 0, y);
        tma_load_2d(dst + HALF_BYTES, mk, bar, 64, y);
        tma_load_2d(dst + 2 * HALF_BYTES, mv, bar, 0, y);
        tma_load_2d(dst + 3 * HALF_BYTES, mv, bar, 64, y);
    };
    __syncthreads();
    if (threadIdx.x == 0) for (int t = 0; t < NSTAGE && t < n_tiles; ++t) issue(t);

    // stage the query rows as bf16 hi / lo, pre-scaled
    for (int idx = threadIdx.x; idx < QRP * (HD / 2); idx += blockDim.x) {
        const int row = idx / (HD / 2), d2 = (idx % (HD / 2)) * 2;
        float x0 = 0.f, x1 = 0.f;
        if (row < QR) {
            const int h = g * grp + row / a.M, i = row % a.M;
            const float2 v = *reinterpret_cast<const float2 *>(a.q + ((size_t)(be * a.M + i) * a.H + h) * HD + d2);
            x0 = v.x * a.scale; x1 = v.y * a.scale;
        }
        uint32_t hi, lo;
        split2(x0, x1, hi, lo);
        const uint32_t off = qoff(row, d2 >> 3) + (d2 & 7) * 2;
        *reinterpret_cast<uint32_t *>(gen_base + (qhi - base) + off) = hi;
        *reinterpret_cast<uint32_t *>(gen_base + (qlo - base) + off) = lo;
    }
    __syncthreads();

    // which query tiles this warp owns
    int my_mt[MTW];
    if (KEYSPLIT) { my_mt[0] = 0; my_mt[1] = a.mt > 1 ? 1 : -1; }
    else { my_mt[0] = warp < a.mt ? warp : -1; my_mt[1] = warp + WARPS < a.mt ? warp + WARPS : -1; }
    float mrun[MTW][2], lrun[MTW][2], o[MTW][16][4];
    unsigned long long anc[MTW][2];
#pragma unroll
    for (int m = 0; m < MTW; ++m) {
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            mrun[m][r] = -INFINITY; lrun[m][r] = 0.f;
            const int row = my_mt[m] * 16 + (lane >> 2) + r * 8;
            anc[m][r] = (my_mt[m] >= 0 && row < QR) ? a.tree->anc[row % a.M] : 0ull;
        }
#pragma unroll
        for (int n = 0; n < 16; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) o[m][n][e] = 0.f;
    }

    bool ok = true;
    for (int tile = 0; tile < n_tiles; ++tile) {
        const int st = tile % NSTAGE;
        ok = mbar_wait(smem_u32(&bars[st]), (tile / NSTAGE) & 1, a.status);
        if (!__syncthreads_and(ok)) { ok = false; break; }  // leave together if any thread gave up
        const uint32_t kst = base + st * STAGE_BYTES, vst = kst + 2 * HALF_BYTES;
        const int j0 = k_begin + tile * TKEYS;
#pragma unroll
        for (int m = 0; m < MTW; ++m) {
            if (my_mt[m] < 0) continue;
            if (KEYSPLIT) {
                if (j0 + warp * SUB < k_end)
                    tile_step(qhi, qlo, my_mt[m] * 16, kst, vst, warp * SUB, lane, j0 + warp * SUB, n_ctx, k_end, anc[m][0],
                              anc[m][1], mrun[m], lrun[m], o[m]);
            } else {
                for (int sub = 0; sub < TKEYS / SUB; ++sub)
                    if (j0 + sub * SUB < k_end)
                        tile_step(qhi, qlo, my_mt[m] * 16, kst, vst, sub * SUB, lane, j0 + sub * SUB, n_ctx, k_end, anc[m][0],
                                  anc[m][1], mrun[m], lrun[m], o[m]);
            }
        }
        __syncthreads();                                     // every warp is done with this stage
        if (threadIdx.x == 0 && tile + NSTAGE < n_tiles) issue(tile + NSTAGE);
    }
    __syncthreads();
    if (!ok) return;                                         // bounded wait expired: status is set, nothing is written

    // dump (O, m, l) per warp into shared memory (the stage ring is free now), then merge and write
    float *osm = reinterpret_cast<float *>(gen_base);       // [contributor][row][HD + 2]
    const int contributors = KEYSPLIT ? WARPS : 1;
    const int ROWF = HD + 2;
#pragma unroll
    for (int m = 0; m < MTW; ++m) {
        if (my_mt[m] < 0) continue;
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int row = my_mt[m] * 16 + (lane >> 2) + r * 8;
            float *dst = osm + ((size_t)(KEYSPLIT ? warp : 0) * QRP + row) * ROWF;
#pragma unroll
            for (int n = 0; n < 16; ++n) {
                dst[n * 8 + (lane & 3) * 2] = o[m][n][r * 2];
                dst[n * 8 + (lane & 3) * 2 + 1] = o[m][n][r * 2 + 1];
            }
            if ((lane & 3) == 0) { dst[HD] = mrun[m][r]; dst[HD + 1] = lrun[m][r]; }
        }
    }
    __syncthreads();
    for (int row = warp; row < QR; row += WARPS) {
        float mmax = -INFINITY;
        for (int c = 0; c < contributors; ++c) mmax = fmaxf(mmax, osm[((size_t)c * QRP + row) * ROWF + HD]);
        float l = 0.f, acc[HD / 32];
#pragma unroll
        for (int e = 0; e < HD / 32; ++e) acc[e] = 0.f;
        for (int c = 0; c < contributors; ++c) {
            const float *src = osm + ((size_t)c * QRP + row) * ROWF;
            const float mc = src[HD];
            if (mc == -INFINITY) continue;
            const float w = expf(mc - mmax);
            l += src[HD + 1] * w;
#pragma unroll
            for (int e = 0; e < HD / 32; ++e) acc[e] += src[lane + 32 * e] * w;
        }
        const int h = g * grp + row / a.M, i = row % a.M;
        if (a.nsplit == 1) {
            const float inv = 1.f / l;
#pragma unroll
            for (int e = 0; e < HD / 32; ++e)
                store_act<__nv_bfloat16>(a.out, a.out_plane, ((size_t)(be * a.M + i) * a.H + h) * HD + lane + 32 * e, acc[e] * inv);
        } else {
            float *dst = a.part + ((((size_t)be * a.H + h) * a.M + i) * a.nsplit + split) * (HD + 2);
#pragma unroll
            for (int e = 0; e < HD / 32; ++e) dst[lane + 32 * e] = acc[e];
            if (lane == 0) { dst[HD] = mmax; dst[HD + 1] = l; }
        }
    }
}

}  // namespace

// tensor maps over the caches are rebuilt only when the caller's pointers change
int attention_mma_supported(const viasd_model *m, int M) {
    const viasd_config &c = m->cfg;
    return c.dtype == 1 && c.head_dim == HD && (c.n_heads / c.n_kv_heads) * M <= 128 && m->use_tc;
}

static int cache_maps(viasd_model *m, CacheMaps &cm, const void *kc, const void *vc, int n_layers) {
    if (cm.k_ptr == kc && cm.v_ptr == vc) return VIASD_OK;
    const viasd_config &c = m->cfg;
    const uint64_t rows = (uint64_t)n_layers * c.max_batch * c.n_kv_heads * c.max_ctx;
    int rc;
    if ((rc = tc_make_map(&cm.k, kc, rows, HD, TKEYS))) return rc;
    if ((rc = tc_make_map(&cm.v, vc, rows, HD, TKEYS))) return rc;
    cm.k_ptr = kc; cm.v_ptr = vc;
    return VIASD_OK;
}

// streams = 1: one cache (full or slim).  streams = 2: rows [0, batch*M) against the full cache at layer_ord and
// rows [batch*M, 2*batch*M) against the slim cache at layer_ord2, in one launch.
int launch_attention_mma(viasd_model *m, const void *kc, const void *vc, bool slim, int layer_ord, const void *kc2,
                         const void *vc2, int layer_ord2, int streams, int batch, int M, int nsplit, cudaStream_t st) {
    const viasd_config &c = m->cfg;
    CacheMaps &cm = slim ? m->cmaps_slim : m->cmaps_full;
    int rc;
    if ((rc = cache_maps(m, cm, kc, vc, slim ? m->n_routed : c.n_layers))) return rc;
    CacheMaps *cm2 = &cm;
    if (streams == 2) {
        cm2 = &m->cmaps_slim;
        if ((rc = cache_maps(m, *cm2, kc2, vc2, m->n_routed))) return rc;
    }
    const int grp = c.n_heads / c.n_kv_heads, mt = (grp * M + 15) / 16;
    AttnArgs a;
    a.q = m->ws.q; a.part = m->ws.part; a.out = (__nv_bfloat16 *)m->ws.attn;
    a.out_plane = m->ws.rows_alloc * (size_t)c.n_heads * HD;
    a.len_eff = m->ws.len_eff; a.tree = m->ws.tree; a.status = &m->ws.stats->device_status;
    a.M = M; a.H = c.n_heads; a.Hkv = c.n_kv_heads; a.max_batch = c.max_batch; a.max_ctx = c.max_ctx;
    a.layer_ord = layer_ord; a.nsplit = nsplit; a.mt = mt; a.scale = 1.0f / sqrtf((float)HD);
    a.batch = batch; a.layer_ord2 = layer_ord2;
    const size_t q_bytes = (size_t)mt * 16 * 256 * 2;
    const size_t smem = 1024 + NSTAGE * STAGE_BYTES + q_bytes;
    static bool attr_done = false;
    if (!attr_done) {
        CUDA_TRY(cudaFuncSetAttribute(attention_mma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
        CUDA_TRY(cudaFuncSetAttribute(attention_mma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
        attr_done = true;
    }
    dim3 grid(batch * c.n_kv_heads, nsplit, streams);
    if (mt <= 2) attention_mma_kernel<true><<<grid, WARPS * 32, smem, st>>>(cm.k, cm.v, cm2->k, cm2->v, a);
    else attention_mma_kernel<false><<<grid, WARPS * 32, smem, st>>>(cm.k, cm.v, cm2->k, cm2->v, a);
    LAUNCH_CHECK();
    return VIASD_OK;
}
