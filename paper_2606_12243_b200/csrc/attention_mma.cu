// KV-append attention for bf16 caches on tensor cores, K/V tiles staged by TMA.
//
// One CTA serves one (sequence, kv head, key range): the query rows are the G = H / Hkv query heads
// of that kv head times the M block rows (G * M <= 128), so every K/V byte is read once for all of them.
// Keys are the committed cache rows 0..n-1 plus the M block rows at slots n..n+M-1, the latter masked
// per query row by its ancestor bit set (causal for a chain, tree mask otherwise).
//
// K and V tiles of 128 keys arrive through 2-D TMA boxes (64 dims x 128 keys, 128-byte swizzle) into a
// two-stage ring; scores S = Q K^T and the update O += P V run on mma.sync m16n8k16 with fp32
// accumulation.  Q is used as a bf16 hi + lo pair, and so is P when there are few query rows, so that only
// the cache itself is bf16.
// Work split inside the CTA (8 warps): a warp owns one 16-row query tile and one group of the 128 keys of a
// stage - 8 key groups of 16 keys when there is a single query tile, 4 x 32 for two, 2 x 64 for up to four,
// all 128 keys for up to eight - and keeps its own online-softmax state; the key groups of a query tile are
// merged pairwise in registers at the end of the key range.  Two warps per scheduler is what hides the
// latency of the dependent ldmatrix / mma / softmax chain.
// A CTA works through a contiguous list of (sequence, kv head, key range) items; the TMA ring runs across item
// boundaries, and tiles that lie wholly inside the committed context are requested before the kernel waits
// for its predecessor (programmatic dependent launch).  Key ranges of one (sequence, kv head) are merged by the
// last CTA to finish one of them (an atomic counter; nobody waits).  The only waits are on TMA arrival and are
// bounded.
#include "common.cuh"
#include <stdlib.h>
#include <stdio.h>

namespace {

constexpr int HD = 128;
constexpr int TKEYS = 128;                 // keys per stage
constexpr int MAX_NSTAGE = 3;
constexpr int WARPS = 8;
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
// K/V tiles are read once per layer: their lines are marked to leave L2 first (what the kernels around this one hand
// over to each other, and their instructions, stay)
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y, uint64_t pol) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "l"(pol) : "memory");
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
    const int *run_flag;        // null, or a device flag: the kernel leaves at once when it is zero
    int M, H, Hkv, max_batch, max_ctx, layer_ord, nsplit, mt;   // mt = query tiles of 16 rows
    int batch, layer_ord2;      // second row stream: rows batch*M.., its own cache and layer ordinal
    int streams, n_items, items_per_cta, fuse_merge, nstage, mt_eff;
    int *counters;              // [streams * batch * Hkv] arrivals per (sequence, kv head), zero between launches
    float scale;
};

__device__ __forceinline__ float ex2(float x) {            // 2^x, hardware approximation (2 ulp)
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// One warp, one 16-row query tile, SUBK (16 or 32) keys starting at key index jbase (tile-relative row r0).
// The query fragments live in registers; scores are in log2 units (the query was scaled by log2(e) / sqrt(hd)).
// MASKED: the keys reach past the committed context or past the end of the range.
template <int SUBK, bool PLO, bool QLO, bool MASKED>
__device__ __forceinline__ void tile_step(const uint32_t (&qh)[8][4], const uint32_t (&ql)[8][4], uint32_t kst, uint32_t vst,
                                          int r0, int lane, int jbase, int n_ctx, int k_end, unsigned long long anc0,
                                          unsigned long long anc1, float (&mrun)[2], float (&lrun)[2], float (&o)[16][4]) {
    constexpr int NS = SUBK / 8;                // score tiles of 8 keys
    float s[NS][4];
#pragma unroll
    for (int n = 0; n < NS; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) s[n][e] = 0.f;
    // S = Q K^T over the 128 dims: 8 k-steps, dims 0..63 in the first half tile, 64..127 in the second
    const int krow = r0 + (lane & 7) + ((lane >> 4) & 1) * 8;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
        const uint32_t khalf = kst + (ks >> 2) * HALF_BYTES;
        const int kc = (ks & 3) * 2 + ((lane >> 3) & 1);
        uint32_t b[NS / 2][4];
#pragma unroll
        for (int np = 0; np < NS / 2; ++np) ldsm_x4(khalf + sw128(krow + np * 16, kc), b[np]);
        // independent accumulators first with the hi part of Q, then with the lo part
#pragma unroll
        for (int np = 0; np < NS / 2; ++np) { mma16816(s[np * 2], qh[ks], b[np][0], b[np][1]); mma16816(s[np * 2 + 1], qh[ks], b[np][2], b[np][3]); }
        if (QLO) {
#pragma unroll
            for (int np = 0; np < NS / 2; ++np) { mma16816(s[np * 2], ql[ks], b[np][0], b[np][1]); mma16816(s[np * 2 + 1], ql[ks], b[np][2], b[np][3]); }
        }
    }
    // mask, online softmax (rows g and g + 8 of the tile; columns 8n + 2t, 8n + 2t + 1)
    float mx[2] = {-INFINITY, -INFINITY};
    if (MASKED) {
        const int t2 = (lane & 3) * 2;
#pragma unroll
        for (int n = 0; n < NS; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int j = jbase + n * 8 + t2 + (e & 1);
                const unsigned long long anc = (e < 2) ? anc0 : anc1;
                const bool ok = j < k_end && (j < n_ctx || ((anc >> (j - n_ctx)) & 1ull));
                s[n][e] = ok ? s[n][e] : -INFINITY;
            }
    }
#pragma unroll
    for (int n = 0; n < NS; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) mx[e >> 1] = fmaxf(mx[e >> 1], s[n][e]);
    float corr[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
        mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
        const float mnew = fmaxf(mrun[r], mx[r]);
        corr[r] = (mnew == -INFINITY) ? 1.f : ex2(mrun[r] - mnew);
        mrun[r] = mnew;
    }
    float rs[2] = {0.f, 0.f};
#pragma unroll
    for (int n = 0; n < NS; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float m = mrun[e >> 1];
            float p = (MASKED && s[n][e] == -INFINITY) ? 0.f : ex2(s[n][e] - m);
            // without the lo part the MMA sees bf16(p): normalise by the sum of those same rounded values, or the
            // rounding of near-equal weights would not cancel
            if (!PLO) p = __bfloat162float(__float2bfloat16_rn(p));
            s[n][e] = p;
            rs[e >> 1] += p;
        }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        rs[r] += __shfl_xor_sync(0xffffffffu, rs[r], 1);
        rs[r] += __shfl_xor_sync(0xffffffffu, rs[r], 2);
        lrun[r] = lrun[r] * corr[r] + rs[r];
    }
    if (__any_sync(0xffffffffu, corr[0] != 1.f || corr[1] != 1.f)) {    // the running maximum moved: rescale
#pragma unroll
        for (int n = 0; n < 16; ++n) { o[n][0] *= corr[0]; o[n][1] *= corr[0]; o[n][2] *= corr[1]; o[n][3] *= corr[1]; }
    }
    // O += P V: k-steps of 16 keys, 16 n-tiles of 8 dims; one pass with the hi part of P, one with the lo part
#pragma unroll
    for (int ks = 0; ks < SUBK / 16; ++ks) {
        uint32_t ph[4], pl[4];
        split2(s[2 * ks][0], s[2 * ks][1], ph[0], pl[0]);
        split2(s[2 * ks][2], s[2 * ks][3], ph[1], pl[1]);
        split2(s[2 * ks + 1][0], s[2 * ks + 1][1], ph[2], pl[2]);
        split2(s[2 * ks + 1][2], s[2 * ks + 1][3], ph[3], pl[3]);
        const int vrow = r0 + ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
        for (int pass = 0; pass < (PLO ? 2 : 1); ++pass) {
#pragma unroll
            for (int np = 0; np < 8; ++np) {    // two n-tiles (16 dims) per ldmatrix.x4.trans
                uint32_t b[4];
                const int dchunk = np * 2 + (lane >> 4);             // 16-byte chunk of the 128 dims
                const uint32_t vhalf = vst + (dchunk >> 3) * HALF_BYTES;
                ldsm_x4_t(vhalf + sw128(vrow, dchunk & 7), b);
                mma16816(o[np * 2], pass ? pl : ph, b[0], b[1]);
                mma16816(o[np * 2 + 1], pass ? pl : ph, b[2], b[3]);
            }
        }
    }
}

struct Item { int be, b, g, stream, split, n_ctx, k_begin, k_end, n_tiles, row_base; };

__device__ __forceinline__ Item decode_item(const AttnArgs &a, int item) {
    Item it;
    it.split = item % a.nsplit;
    const int bg = item / a.nsplit;
    it.g = bg % a.Hkv;
    it.be = bg / a.Hkv;
    it.stream = it.be / a.batch;
    it.b = it.be - it.stream * a.batch;
    it.n_ctx = a.len_eff[it.b];
    const int Tk = it.n_ctx + a.M;
    int chunk = (Tk + a.nsplit - 1) / a.nsplit;
    chunk = (chunk + TKEYS - 1) / TKEYS * TKEYS;
    it.k_begin = it.split * chunk;
    it.k_end = min(Tk, it.k_begin + chunk);
    it.n_tiles = it.k_end > it.k_begin ? (it.k_end - it.k_begin + TKEYS - 1) / TKEYS : 0;
    it.row_base = (((it.stream ? a.layer_ord2 : a.layer_ord) * a.max_batch + it.b) * a.Hkv + it.g) * a.max_ctx;
    return it;
}


// PLO / QLO: use the lo parts of the probabilities / of the query too
template <bool PLO, bool QLO>
__global__ void __launch_bounds__(WARPS * 32)
attention_mma_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                     const __grid_constant__ CUtensorMap map_k2, const __grid_constant__ CUtensorMap map_v2, const AttnArgs a) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) unsigned long long bars[MAX_NSTAGE];
    __shared__ int last_sh;
    constexpr int ROWF = HD + 2;
    RUN_FLAG_EXIT(a.run_flag);
    PDL_TRIGGER();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int NSTAGE = a.nstage;
    const int grp = a.H / a.Hkv, QR = grp * a.M, QRP = a.mt * 16;
    // this warp's query tile and key group (mt_eff = query tiles rounded up to a power of two, <= 8)
    const int mtile = warp & (a.mt_eff - 1), kgroup = warp / a.mt_eff, n_kg = WARPS / a.mt_eff, kg_keys = TKEYS / n_kg;
    const bool active = mtile < a.mt;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t qhi = base + NSTAGE * STAGE_BYTES, qlo = qhi + (uint32_t)QRP * 256u;
    uint8_t *gen_base = smem_raw + (base - smem_u32(smem_raw));
    float *osm = reinterpret_cast<float *>(gen_base + NSTAGE * STAGE_BYTES + (size_t)QRP * 512);   // merge exchange

    const int i0 = blockIdx.x * a.items_per_cta, i1 = min(a.n_items, i0 + a.items_per_cta);
    if (threadIdx.x == 0) {
        for (int s = 0; s < NSTAGE; ++s) mbar_init(smem_u32(&bars[s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    // producer cursor (thread 0 only): next tile to request, in the CTA's flattened (item, tile) order
    int p_item = i0, p_tile = 0, p_count = 0;
    const uint64_t kvpol = l2_evict_first_policy();
    Item pit = i0 < i1 ? decode_item(a, i0) : Item{};
    auto issue_next = [&](bool context_only) -> bool {      // false: nothing (more) to request under this condition
        while (p_item < i1 && p_tile >= pit.n_tiles) { ++p_item; p_tile = 0; if (p_item < i1) pit = decode_item(a, p_item); }
        if (p_item >= i1) return false;
        const int k0 = pit.k_begin + p_tile * TKEYS;
        if (context_only && k0 + TKEYS > pit.n_ctx) return false;     // this tile holds rows the previous kernel writes
        const int st = p_count % NSTAGE;
        const uint32_t bar = smem_u32(&bars[st]), dst = base + st * STAGE_BYTES;
        const CUtensorMap *mk = pit.stream ? &map_k2 : &map_k, *mv = pit.stream ? &map_v2 : &map_v;
        const int y = pit.row_base + k0;
        mbar_expect_tx(bar, STAGE_BYTES);
        tma_load_2d(dst, mk, bar, 0, y, kvpol);
        tma_load_2d(dst + HALF_BYTES, mk, bar, 64, y, kvpol);
        tma_load_2d(dst + 2 * HALF_BYTES, mv, bar, 0, y, kvpol);
        tma_load_2d(dst + 3 * HALF_BYTES, mv, bar, 64, y, kvpol);
        ++p_tile; ++p_count;
        return true;
    };
    if (threadIdx.x == 0) {
        // committed context does not change during the pass: ask for it before waiting for the previous kernel
        while (p_count < NSTAGE && issue_next(true)) { }
    }
    // the first item's description and its rows' ancestor sets come from the pass's preparation kernel, long done:
    // fetch them now, not after the dependency wait, where every dependent global load is a microsecond on the path
    const Item first_item = i0 < i1 ? decode_item(a, i0) : Item{};
    unsigned long long anc_first[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int row = (warp & (a.mt_eff - 1)) * 16 + (lane >> 2) + r * 8;
        anc_first[r] = row < (a.H / a.Hkv) * a.M ? a.tree[first_item.b].anc[row % a.M] : 0ull;
    }
    PDL_WAIT();
    if (threadIdx.x == 0) while (p_count < NSTAGE && issue_next(false)) { }

    uint32_t qh[8][4], ql[8][4];                             // this warp's query tile, hi and lo, as MMA A fragments
    int c_count = 0;                                         // tiles consumed so far (stage / parity bookkeeping)
    int q_be = -1, q_g = -1;
    bool ok = true;
    for (int item = i0; item < i1 && ok; ++item) {
        const Item it = item == i0 ? first_item : decode_item(a, item);
        if (it.be != q_be || it.g != q_g) {
            // stage the query rows of this (sequence, kv head) as bf16 hi / lo, pre-scaled
            __syncthreads();
            // four elements per thread at a time, loads first: the staging costs one memory round trip per batch
            for (int idx0 = threadIdx.x; idx0 < QRP * (HD / 2); idx0 += 4 * blockDim.x) {
                float2 v[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int idx = idx0 + q * blockDim.x, row = idx / (HD / 2), d2 = (idx % (HD / 2)) * 2;
                    v[q] = make_float2(0.f, 0.f);
                    if (idx < QRP * (HD / 2) && row < QR) {
                        const int h = it.g * grp + row / a.M, i = row % a.M;
                        v[q] = __ldcg(reinterpret_cast<const float2 *>(a.q + ((size_t)(it.be * a.M + i) * a.H + h) * HD + d2));
                    }
                }
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int idx = idx0 + q * blockDim.x, row = idx / (HD / 2), d2 = (idx % (HD / 2)) * 2;
                    if (idx >= QRP * (HD / 2)) continue;
                    uint32_t hi, lo;
                    split2(v[q].x * a.scale, v[q].y * a.scale, hi, lo);
                    const uint32_t off = qoff(row, d2 >> 3) + (d2 & 7) * 2;
                    *reinterpret_cast<uint32_t *>(gen_base + (qhi - base) + off) = hi;
                    *reinterpret_cast<uint32_t *>(gen_base + (qlo - base) + off) = lo;
                }
            }
            __syncthreads();
            q_be = it.be; q_g = it.g;
            if (active) {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const int arow = mtile * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, achunk = ks * 2 + (lane >> 4);
                    ldsm_x4(qhi + qoff(arow, achunk), qh[ks]);
                    ldsm_x4(qlo + qoff(arow, achunk), ql[ks]);
                }
            }
        }
        float mrun[2] = {-INFINITY, -INFINITY}, lrun[2] = {0.f, 0.f}, o[16][4];
        unsigned long long anc[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int row = mtile * 16 + (lane >> 2) + r * 8;
            anc[r] = !(active && row < QR) ? 0ull : item == i0 ? anc_first[r] : a.tree[it.b].anc[row % a.M];
        }
#pragma unroll
        for (int n = 0; n < 16; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) o[n][e] = 0.f;

        for (int tile = 0; tile < it.n_tiles; ++tile, ++c_count) {
            const int st = c_count % NSTAGE;
            ok = mbar_wait(smem_u32(&bars[st]), (c_count / NSTAGE) & 1, a.status);
            if (!__syncthreads_and(ok)) { ok = false; break; }   // leave together if any thread gave up
            const uint32_t kst = base + st * STAGE_BYTES, vst = kst + 2 * HALF_BYTES;
            const int j0 = it.k_begin + tile * TKEYS;
            if (active) {
                if (kg_keys == 16) {
                    const int r0 = kgroup * 16, jb = j0 + r0;
                    if (jb < it.k_end) {
                        if (jb + 16 <= it.n_ctx && jb + 16 <= it.k_end)
                            tile_step<16, PLO, QLO, false>(qh, ql, kst, vst, r0, lane, jb, it.n_ctx, it.k_end, anc[0], anc[1], mrun, lrun, o);
                        else
                            tile_step<16, PLO, QLO, true>(qh, ql, kst, vst, r0, lane, jb, it.n_ctx, it.k_end, anc[0], anc[1], mrun, lrun, o);
                    }
                } else {
                    for (int sub = 0; sub < kg_keys; sub += 32) {
                        const int r0 = kgroup * kg_keys + sub, jb = j0 + r0;
                        if (jb < it.k_end) {
                            if (jb + 32 <= it.n_ctx && jb + 32 <= it.k_end)
                                tile_step<32, PLO, QLO, false>(qh, ql, kst, vst, r0, lane, jb, it.n_ctx, it.k_end, anc[0], anc[1], mrun, lrun, o);
                            else
                                tile_step<32, PLO, QLO, true>(qh, ql, kst, vst, r0, lane, jb, it.n_ctx, it.k_end, anc[0], anc[1], mrun, lrun, o);
                        }
                    }
                }
            }
            __syncthreads();                                 // every warp is done with this stage
            if (threadIdx.x == 0) issue_next(false);
        }
        if (!ok) break;

        // ---- end of the item: merge the key groups of each query tile pairwise, in registers ----
        // (the fragment layouts match lane for lane, so the exchange buffer is just each lane's values)
        for (int stride = n_kg >> 1; stride >= 1; stride >>= 1) {
            // two exchange slots: a round with more than two giving warps goes in batches of two
            const int pairs = stride * a.mt_eff;
            for (int batch = 0; batch * 2 < pairs; ++batch) {
                const int give = (kgroup - stride) * a.mt_eff + mtile, take = kgroup * a.mt_eff + mtile;
                if (active && kgroup >= stride && kgroup < 2 * stride && (give >> 1) == batch) {
                    float *dst = osm + ((size_t)(give & 1) * 32 + lane) * 68;
#pragma unroll
                    for (int n = 0; n < 16; ++n)
#pragma unroll
                        for (int e = 0; e < 4; ++e) dst[n * 4 + e] = o[n][e];
#pragma unroll
                    for (int r = 0; r < 2; ++r) { dst[64 + r] = mrun[r]; dst[66 + r] = lrun[r]; }
                }
                __syncthreads();
                if (active && kgroup < stride && (take >> 1) == batch) {
                    const float *src = osm + ((size_t)(take & 1) * 32 + lane) * 68;
                    float wa[2], wb[2];
#pragma unroll
                    for (int r = 0; r < 2; ++r) {
                        const float mo = src[64 + r], lo2 = src[66 + r];
                        const float mn = fmaxf(mrun[r], mo);
                        wa[r] = (mn == -INFINITY) ? 1.f : ex2(mrun[r] - mn);
                        wb[r] = (mo == -INFINITY) ? 0.f : ex2(mo - mn);
                        lrun[r] = lrun[r] * wa[r] + lo2 * wb[r];
                        mrun[r] = mn;
                    }
#pragma unroll
                    for (int n = 0; n < 16; ++n)
#pragma unroll
                        for (int e = 0; e < 4; ++e) o[n][e] = o[n][e] * wa[e >> 1] + src[n * 4 + e] * wb[e >> 1];
                }
                __syncthreads();
            }
        }
        const bool single = a.nsplit == 1;
        if (active && kgroup == 0) {
            // this warp now holds its query tile for the whole key range: write it from registers
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const int row = mtile * 16 + (lane >> 2) + r * 8;
                if (row >= QR) continue;
                const int h = it.g * grp + row / a.M, i = row % a.M;
                const int c0 = (lane & 3) * 2;
                if (single) {
                    const float inv = 1.f / lrun[r];
                    const size_t o0 = ((size_t)(it.be * a.M + i) * a.H + h) * HD;
#pragma unroll
                    for (int n = 0; n < 16; ++n) {
                        store_act<__nv_bfloat16>(a.out, a.out_plane, o0 + n * 8 + c0, o[n][r * 2] * inv);
                        store_act<__nv_bfloat16>(a.out, a.out_plane, o0 + n * 8 + c0 + 1, o[n][r * 2 + 1] * inv);
                    }
                } else {
                    float *dst = a.part + ((((size_t)it.be * a.H + h) * a.M + i) * a.nsplit + it.split) * ROWF;
#pragma unroll
                    for (int n = 0; n < 16; ++n)
                        *reinterpret_cast<float2 *>(dst + n * 8 + c0) = make_float2(o[n][r * 2], o[n][r * 2 + 1]);
                    if ((lane & 3) == 0) { dst[HD] = mrun[r] * 0.6931471805599453f; dst[HD + 1] = lrun[r]; }   // natural-log units
                }
            }
        }
        if (!single && a.fuse_merge) {
            // last key range of this (sequence, kv head) to finish merges all of them, in range order
            // (one acquire-release atomic after the barrier instead of a fence per thread on both sides: the barrier
            // orders the CTA's stores before it, and the release is cumulative)
            __syncthreads();
            if (threadIdx.x == 0) {
                int old;
                asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(a.counters + it.be * a.Hkv + it.g) : "memory");
                last_sh = old == a.nsplit - 1;
                if (last_sh) a.counters[it.be * a.Hkv + it.g] = 0;
            }
            __syncthreads();
            if (last_sh) {
                // two rows per warp at a time, all loads of a round in flight before the first use (a row at a time is a
                // trip to L2 per row, one after the other; the kernel has no registers to spare for more)
                constexpr int MB = 2;
#pragma unroll 1
                for (int rb = warp; rb < QR; rb += MB * WARPS) {
                    const float *src[MB];
                    size_t odst[MB];
                    float ms[MB], ls[MB], w[MB], den[MB], num[MB][HD / 32];
#pragma unroll
                    for (int j = 0; j < MB; ++j) {
                        const int row = min(rb + j * WARPS, QR - 1);            // rows past the end repeat the last one, unstored
                        const int h = it.g * grp + row / a.M, i = row % a.M;
                        src[j] = a.part + (((size_t)it.be * a.H + h) * a.M + i) * (size_t)a.nsplit * ROWF;
                        odst[j] = ((size_t)(it.be * a.M + i) * a.H + h) * HD;
                        // lane s holds range s's (max, sum); the weights go round by shuffle (nsplit <= 32 when fused)
                        ms[j] = -INFINITY; ls[j] = 0.f;
                        if (lane < a.nsplit) { ms[j] = __ldcg(src[j] + (size_t)lane * ROWF + HD); ls[j] = __ldcg(src[j] + (size_t)lane * ROWF + HD + 1); }
#pragma unroll
                        for (int e = 0; e < HD / 32; ++e) num[j][e] = 0.f;
                    }
                    for (int s0 = 0; s0 < a.nsplit; s0 += 4) {
                        float v[MB][4][HD / 32];
#pragma unroll
                        for (int j = 0; j < MB; ++j)
#pragma unroll
                            for (int q = 0; q < 4; ++q)
#pragma unroll
                                for (int e = 0; e < HD / 32; ++e)
                                    v[j][q][e] = s0 + q < a.nsplit ? __ldcg(src[j] + (size_t)(s0 + q) * ROWF + lane + 32 * e) : 0.f;
                        if (s0 == 0) {
#pragma unroll
                            for (int j = 0; j < MB; ++j) {
                                const float mmax = warp_max(ms[j]);
                                w[j] = (ms[j] == -INFINITY) ? 0.f : expf(ms[j] - mmax);
                                den[j] = warp_sum(ls[j] * w[j]);
                            }
                        }
#pragma unroll
                        for (int j = 0; j < MB; ++j)
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const float wq = __shfl_sync(0xffffffffu, w[j], (s0 + q) & 31);
#pragma unroll
                                for (int e = 0; e < HD / 32; ++e) num[j][e] = fmaf(v[j][q][e], s0 + q < a.nsplit ? wq : 0.f, num[j][e]);
                            }
                    }
#pragma unroll
                    for (int j = 0; j < MB; ++j) {
                        if (rb + j * WARPS >= QR) continue;
                        const float inv = 1.f / den[j];
#pragma unroll
                        for (int e = 0; e < HD / 32; ++e)
                            store_act<__nv_bfloat16>(a.out, a.out_plane, odst[j] + lane + 32 * e, num[j][e] * inv);
                    }
                }
            }
            __syncthreads();
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
                         const void *vc2, int layer_ord2, int streams, int batch, int M, int nsplit, int fuse_merge,
                         cudaStream_t st) {
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
    const int mt_eff = mt <= 1 ? 1 : mt <= 2 ? 2 : mt <= 4 ? 4 : 8;
    AttnArgs a;
    a.q = m->ws.q; a.part = m->ws.part; a.out = (__nv_bfloat16 *)m->ws.attn;
    a.out_plane = m->ws.rows_alloc * (size_t)c.n_heads * HD;
    a.len_eff = m->ws.len_eff; a.tree = m->ws.tree; a.status = &m->ws.stats->device_status; a.run_flag = m->run_flag;
    a.M = M; a.H = c.n_heads; a.Hkv = c.n_kv_heads; a.max_batch = c.max_batch; a.max_ctx = c.max_ctx;
    a.layer_ord = layer_ord; a.nsplit = nsplit; a.mt = mt; a.scale = 1.4426950408889634f / sqrtf((float)HD);   // log2(e) / sqrt(hd)
    a.batch = batch; a.layer_ord2 = layer_ord2; a.streams = streams;
    a.counters = m->ws.attn_counters;
    a.fuse_merge = fuse_merge;
    a.mt_eff = mt_eff;
    a.n_items = streams * batch * c.n_kv_heads * nsplit;
    int grid = a.n_items < m->sm_count ? a.n_items : m->sm_count;
    a.items_per_cta = (a.n_items + grid - 1) / grid;
    grid = (a.n_items + a.items_per_cta - 1) / a.items_per_cta;
    const size_t q_bytes = (size_t)mt * 16 * 256 * 2;
    const size_t osm_bytes = mt_eff < 8 ? (size_t)2 * 32 * 68 * 4 : 0;        // two warps' states, lane by lane
    // three stages (two tiles in flight while one is consumed) when the rest of the CTA's shared memory allows
    a.nstage = 1024 + 3 * (size_t)STAGE_BYTES + q_bytes + osm_bytes <= 226 * 1024 ? 3 : 2;
    const size_t smem = 1024 + a.nstage * (size_t)STAGE_BYTES + q_bytes + osm_bytes;
    static bool attr_done[64];
    if (first_use_on_device(attr_done)) {
        CUDA_TRY(cudaFuncSetAttribute(attention_mma_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024));
        CUDA_TRY(cudaFuncSetAttribute(attention_mma_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024));
        CUDA_TRY(cudaFuncSetAttribute(attention_mma_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024));
    }
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    pdl_config(cfg, attr, dim3(grid), dim3(WARPS * 32), smem, st);
    const int lo_mode = m->opt.attn_lo;      // 2 = hi/lo for Q and P, 1 = hi/lo for Q only, 0 = plain bf16
    if (lo_mode >= 2) CUDA_TRY(cudaLaunchKernelEx(&cfg, attention_mma_kernel<true, true>, cm.k, cm.v, cm2->k, cm2->v, a));
    else if (lo_mode == 1) CUDA_TRY(cudaLaunchKernelEx(&cfg, attention_mma_kernel<false, true>, cm.k, cm.v, cm2->k, cm2->v, a));
    else CUDA_TRY(cudaLaunchKernelEx(&cfg, attention_mma_kernel<false, false>, cm.k, cm.v, cm2->k, cm2->v, a));
    LAUNCH_CHECK();
    return VIASD_OK;
}

