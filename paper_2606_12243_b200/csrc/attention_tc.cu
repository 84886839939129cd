// Block attention on the 5th-generation tensor cores (tcgen05 + TMEM), bf16 caches, head_dim 128.
//
// Same work as attention_mma.cu - the M block rows of a sequence (all query heads of one kv head packed into one
// query tile, at most 128 rows) against the committed context plus the block's own rows under the ancestor
// mask, split over key ranges - but with both contractions on tcgen05:
//
//   S[rows, 128 keys] = Q K^T      A = Q (shared memory, K-major, hi and lo planes: two MMAs into one S)
//                                  B = K tile exactly as its TMA box lands (K-major, 128-byte swizzle)
//   O[rows, 128 dims] += P V       A = P in TMEM (bf16 pairs, hi and lo planes: two MMAs into one O)
//                                  B = V tile as it lands, read MN-major (keys are the contraction)
//
// One TMEM lane is one query row, so a softmax thread owns a row: row maximum and row sum need no exchange
// between threads.  With few query rows (<= 32, or <= 64) the rows are staged 4 (or 2) times, once per block of
// 32 (64) lanes, and replica r looks only at keys [r * 128/R, (r + 1) * 128/R) of every tile: the four softmax
// warps then share a tile's exponentials instead of one warp doing them all, and each replica ends as a key
// range of its own (own maximum, sum and O rows) that the range merge adds to the others.  The running maximum is only raised when a tile exceeds it by more than 2^8 (the weights
// stay below 2^8 otherwise, harmless in fp32), which makes the rescaling of O in TMEM rare.
//
// Warp roles (192 threads): warp 0 requests K/V tiles by TMA into a ring that runs across the CTA's items,
// warp 1 owns TMEM and issues the MMAs, warps 2-5 stage Q, run the softmax and write the result.
// TMEM: two S buffers of 128 columns and O (128).  The softmax overwrites a tile's scores with its weights in
// place (per 16 keys: 8 columns of bf16 pairs hi, 8 columns lo), so P is double-buffered with S and a tile's
// softmax does not wait for the previous tile's P V.  MMAs run in issue order, which is what lets Q K^T of tile
// t + 2 reuse the buffer P V of tile t reads.
// Every wait is bounded: on expiry the CTA records VIASD_EDEVICE, lets its copies land and leaves.
#include "common.cuh"
#include "tc_ptx.cuh"
#include <stdlib.h>

namespace {

constexpr int HD = 128;                        // head dimension
constexpr int TKEYS = 128;                     // keys per tile
constexpr int HALF_BYTES = TKEYS * 128;        // 128 keys x 64 dims of bf16, as one TMA box lands
constexpr int STAGE_BYTES = 4 * HALF_BYTES;    // K dims 0..63, K dims 64..127, V dims 0..63, V dims 64..127
constexpr int AT_THREADS = 192;
constexpr int AT_MAX_STAGE = 3;
constexpr int ROWF = HD + 2;                   // partial row: 128 numerators, max (natural-log units), sum
constexpr float RESCALE_GAP = 8.f;             // log2 units

constexpr uint32_t TM_S = 0, TM_O = 256;       // TMEM column offsets: S / P buffers (2 x 128), O (128)

struct AttnTcArgs {
    const float *q;             // [rows, H * HD] rotated queries
    float *part;                // [b][h][i][split][HD + 2]
    __nv_bfloat16 *out;         // attention output planes (hi, lo)
    size_t out_plane;
    const int *len_eff;
    const TreeInfo *tree;
    int *status;
    const int *run_flag;        // null, or a device flag: the kernel leaves at once when it is zero
    int M, H, Hkv, max_batch, max_ctx, layer_ord, nsplit;
    int batch, layer_ord2;      // second row stream: rows batch*M.., its own cache and layer ordinal
    int streams, n_items, items_per_cta, fuse_merge, nstage;
    int qrows8;                 // query rows per kv head rounded up to 8
    int reps, rows_per_rep;     // R replicas of the query rows, 128 / R lanes each
    uint32_t qoff[4];           // byte offsets of the staged query regions: hi dims 0..63, hi 64..127, lo 0..63, lo 64..127
    uint32_t q_bytes;           // staged queries in all; the ring follows
    int *counters;              // arrivals per (stream, sequence, kv head), zero between launches
    float scale;                // log2(e) / sqrt(hd)
};

struct Item { int be, b, g, stream, split, n_ctx, k_begin, k_end, n_tiles, row_base; };

__device__ __forceinline__ Item decode_item(const AttnTcArgs &a, int item) {
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

__device__ __forceinline__ float ex2(float x) {            // 2^x, hardware approximation (2 ulp)
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// x0, x1 -> packed bf16 pairs hi = bf16(x), lo = bf16(x - hi); the low half word is the even element
__device__ __forceinline__ void split_pair(float x0, float x1, uint32_t &hi, uint32_t &lo) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
    hi = *reinterpret_cast<const uint32_t *>(&h);
    const __nv_bfloat162 l = __floats2bfloat162_rn(x0 - __uint_as_float(hi << 16), x1 - __uint_as_float(hi & 0xffff0000u));
    lo = *reinterpret_cast<const uint32_t *>(&l);
}

// MN-major operand tile with the 128-byte swizzle: 64 contiguous elements along MN per row of 128 bytes,
// 8 rows (8 steps of the contraction) per 1024-byte group; groups `sbo` bytes apart along the contraction,
// 64-element blocks `lbo` bytes apart along MN.
__device__ __forceinline__ uint64_t smem_desc_mn(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((addr >> 4) & 0x3FFF) | ((uint64_t)((lbo >> 4) & 0x3FFF) << 16) | ((uint64_t)((sbo >> 4) & 0x3FFF) << 32) |
           (1ull << 46) | (2ull << 61);
}

// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
          "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
          "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
          "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]),
          "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]),
          "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
          "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }


__global__ void __launch_bounds__(AT_THREADS, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                    const __grid_constant__ CUtensorMap map_k2, const __grid_constant__ CUtensorMap map_v2, const AttnTcArgs a) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) unsigned long long bars[2 * AT_MAX_STAGE + 9];
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh, last_sh;

    RUN_FLAG_EXIT(a.run_flag);
    PDL_TRIGGER();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int NSTAGE = a.nstage;
    const int grp = a.H / a.Hkv, QR = grp * a.M;
    // staged queries first (the MMA reads 128 rows from each chunk: what lies behind the live rows is the ring)
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t qsm = base, ring = base + a.q_bytes;
    uint8_t *q_gen = smem_raw + (base - smem_u32(smem_raw));
    auto full_bar = [&](int s) { return smem_u32(&bars[s]); };
    auto empty_bar = [&](int s) { return smem_u32(&bars[AT_MAX_STAGE + s]); };
    auto sfull_bar = [&](int b) { return smem_u32(&bars[2 * AT_MAX_STAGE + b]); };
    auto pfull_bar = [&](int b) { return smem_u32(&bars[2 * AT_MAX_STAGE + 2 + b]); };
    auto pvdone_bar = [&](int b) { return smem_u32(&bars[2 * AT_MAX_STAGE + 4 + b]); };
    const uint32_t ofree_bar = smem_u32(&bars[2 * AT_MAX_STAGE + 6]), qfull_bar = smem_u32(&bars[2 * AT_MAX_STAGE + 7]);
    const uint32_t wg_bar = smem_u32(&bars[2 * AT_MAX_STAGE + 8]);      // the softmax warps among themselves (bounded, unlike bar.sync)

    if (threadIdx.x == 0) {
        for (int s = 0; s < NSTAGE; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(sfull_bar(b), 1); mbar_init(pfull_bar(b), 4); mbar_init(pvdone_bar(b), 1); }
        mbar_init(ofree_bar, 4);
        mbar_init(qfull_bar, 4);
        mbar_init(wg_bar, 128);
        abort_sh = 0;
        last_sh = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_sh)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_sh;
    const int i0 = blockIdx.x * a.items_per_cta, i1 = min(a.n_items, i0 + a.items_per_cta);

    if (warp == 0) {
        // ---------------- TMA producer: the CTA's (item, tile) list, flattened ----------------
        if (lane == 0) {
            const uint64_t kvpol = l2_evict_first_policy();    // the cache passes through once per layer
            int p_item = i0, p_tile = 0, p_count = 0;
            bool ok = true;
            Item pit = i0 < i1 ? decode_item(a, i0) : Item{};
            auto issue_next = [&](bool context_only) -> bool {  // false: nothing (more) to request under this condition
                while (p_item < i1 && p_tile >= pit.n_tiles) { ++p_item; p_tile = 0; if (p_item < i1) pit = decode_item(a, p_item); }
                if (p_item >= i1) return false;
                const int k0 = pit.k_begin + p_tile * TKEYS;
                if (context_only && k0 + TKEYS > pit.n_ctx) return false;   // this tile holds rows the previous kernel writes
                const int st = p_count % NSTAGE;
                if (p_count >= NSTAGE && !(ok = mbar_wait(empty_bar(st), ((p_count / NSTAGE) & 1) ^ 1, &abort_sh, a.status))) return false;
                const uint32_t bar = full_bar(st), dst = ring + st * STAGE_BYTES;
                const CUtensorMap *mk = pit.stream ? &map_k2 : &map_k, *mv = pit.stream ? &map_v2 : &map_v;
                const int y = pit.row_base + k0;
                mbar_expect_tx(bar, STAGE_BYTES);
                tma_load_2d_hint(dst, mk, bar, 0, y, kvpol);
                tma_load_2d_hint(dst + HALF_BYTES, mk, bar, 64, y, kvpol);
                tma_load_2d_hint(dst + 2 * HALF_BYTES, mv, bar, 0, y, kvpol);
                tma_load_2d_hint(dst + 3 * HALF_BYTES, mv, bar, 64, y, kvpol);
                ++p_tile; ++p_count;
                return true;
            };
            // committed context does not change during the pass: ask for it before waiting for the previous kernel
            while (p_count < NSTAGE && issue_next(true)) { }
            PDL_WAIT();
            while (ok && issue_next(false)) { }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(TKEYS >> 3) << 17) | ((128u >> 4) << 24);
            const uint32_t idesc_pv = idesc | (1u << 16);                 // B (the V tile) is MN-major
            int c_tile = 0, n_q = 0, o_uses = 0, q_be = -1, q_g = -1;   // c_tile: tiles of earlier items (ring and buffer phase)
            bool ok = true;
            // tile g (counted over the whole CTA) uses stage g % NSTAGE and S / P buffer g & 1
            auto issue_qk = [&](int g) -> bool {
                const int st = g % NSTAGE, sb = g & 1;
                if (!mbar_wait(full_bar(st), (g / NSTAGE) & 1, &abort_sh, a.status)) return false;
                tc_fence_after();
                const uint32_t kst = ring + st * STAGE_BYTES, d = tmem + TM_S + sb * 128;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t kb = smem_desc(kst + (ks >> 2) * HALF_BYTES + (ks & 3) * 32);
                    tc_mma(d, smem_desc(qsm + a.qoff[ks >> 2] + (ks & 3) * 32), kb, idesc, ks > 0 ? 1u : 0u);
                    tc_mma(d, smem_desc(qsm + a.qoff[2 + (ks >> 2)] + (ks & 3) * 32), kb, idesc, 1u);   // lo plane of the queries
                }
                tc_commit(sfull_bar(sb));
                return true;
            };
            for (int item = i0; item < i1 && ok; ++item) {
                const Item it = decode_item(a, item);
                if (it.be != q_be || it.g != q_g) {
                    if (!(ok = mbar_wait(qfull_bar, n_q & 1, &abort_sh, a.status))) break;
                    ++n_q; q_be = it.be; q_g = it.g;
                }
                if (it.n_tiles == 0) continue;
                // issue order Q K^T(0), Q K^T(1), P V(0), Q K^T(2), P V(1), ...: Q K^T(t + 2) overwrites the buffer P V(t) reads
                if (!(ok = issue_qk(c_tile))) break;
                if (it.n_tiles > 1 && !(ok = issue_qk(c_tile + 1))) break;
                for (int t = 0; t < it.n_tiles; ++t) {
                    const int g = c_tile + t, sb = g & 1, st = g % NSTAGE;
                    if (t == 0 && o_uses > 0 && !(ok = mbar_wait(ofree_bar, (o_uses - 1) & 1, &abort_sh, a.status))) break;
                    if (!(ok = mbar_wait(pfull_bar(sb), (g >> 1) & 1, &abort_sh, a.status))) break;
                    tc_fence_after();
                    const uint32_t vst = ring + st * STAGE_BYTES + 2 * HALF_BYTES, pb = tmem + TM_S + sb * 128;
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {                      // 16 keys per step: two 8-key groups of 1024 bytes
                        const uint64_t vb = smem_desc_mn(vst + kk * 2048, HALF_BYTES, 1024);
                        const uint32_t pa = pb + kk * 16;                        // 16 keys: 8 columns hi, 8 columns lo
                        tc_mma_ts(tmem + TM_O, pa, vb, idesc_pv, (t > 0 || kk > 0) ? 1u : 0u);
                        tc_mma_ts(tmem + TM_O, pa + 8, vb, idesc_pv, 1u);         // lo plane of the weights
                    }
                    tc_commit(empty_bar(st));                             // the stage is free once these MMAs have read it
                    tc_commit(pvdone_bar(sb));
                    if (t + 2 < it.n_tiles && !(ok = issue_qk(g + 2))) break;
                }
                c_tile += it.n_tiles;
                ++o_uses;
            }
        }
    } else {
        // ---------------- softmax / epilogue (warps 2..5 <-> TMEM lane quarters 2,3,0,1): one thread, one query row ----------------
        const int quarter = warp & 3, trow = quarter * 32 + lane, et = threadIdx.x - 64;
        const int rep = trow / a.rows_per_rep, row = trow - rep * a.rows_per_rep;     // replica, query row
        const bool live = row < QR, warp_live = (quarter * 32) % a.rows_per_rep < QR;
        const int KR = TKEYS / a.reps, key0 = rep * KR;                                // this replica's keys of a tile
        const uint32_t tlane = tmem + ((uint32_t)(quarter * 32) << 16);
        PDL_WAIT();
        int s_cnt = 0, q_be = -1, q_g = -1, wg_phase = 0;        // s_cnt: tiles this CTA has finished (buffer phase)
        bool ok = true;
        auto wg_sync = [&]() -> bool {
            mbar_arrive(wg_bar);
            const bool done = mbar_wait(wg_bar, wg_phase & 1, &abort_sh, a.status);
            ++wg_phase;
            return done;
        };
        for (int item = i0; item < i1 && ok; ++item) {
            const Item it = decode_item(a, item);
            if (it.be != q_be || it.g != q_g) {
                // stage the query rows of this (sequence, kv head) as bf16 hi / lo planes, pre-scaled, in the K-major
                // 128-byte-swizzled layout the MMA reads; four elements per thread at a time, loads first
                const int n_el = a.qrows8 * (HD / 2);
                for (int idx0 = et; idx0 < n_el; idx0 += 4 * 128) {
                    float2 v[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int idx = idx0 + q * 128, r = idx / (HD / 2), d2 = (idx % (HD / 2)) * 2;
                        v[q] = make_float2(0.f, 0.f);
                        if (idx < n_el && r < QR) {
                            const int h = it.g * grp + r / a.M, i = r % a.M;
                            v[q] = __ldcg(reinterpret_cast<const float2 *>(a.q + ((size_t)(it.be * a.M + i) * a.H + h) * HD + d2));
                        }
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int idx = idx0 + q * 128, r = idx / (HD / 2), d2 = (idx % (HD / 2)) * 2;
                        if (idx >= n_el) continue;
                        uint32_t hi, lo;
                        split_pair(v[q].x * a.scale, v[q].y * a.scale, hi, lo);
                        const int dc = d2 & 63;                                    // dim inside its 64-dim chunk
                        for (int rp = 0; rp < a.reps; ++rp) {                      // one copy per replica's block of lanes
                            const uint32_t rr = (uint32_t)(rp * a.rows_per_rep + r);
                            const uint32_t off = rr * 128u + ((((uint32_t)dc >> 3) ^ (rr & 7u)) << 4) + ((uint32_t)dc & 7u) * 2u;
                            *reinterpret_cast<uint32_t *>(q_gen + a.qoff[d2 >> 6] + off) = hi;
                            *reinterpret_cast<uint32_t *>(q_gen + a.qoff[2 + (d2 >> 6)] + off) = lo;
                        }
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> the MMA's reads
                __syncwarp();
                if (lane == 0) mbar_arrive(qfull_bar);
                q_be = it.be; q_g = it.g;
            }
            const int h = it.g * grp + row / a.M, node = row % a.M;
            const unsigned long long anc = live ? a.tree[it.b].anc[node] : 0ull;
            float m_run = -INFINITY, l_run = 0.f;

            for (int t = 0; t < it.n_tiles; ++t, ++s_cnt) {
                const int sb = s_cnt & 1;
                if (!(ok = mbar_wait(sfull_bar(sb), (s_cnt >> 1) & 1, &abort_sh, a.status))) break;
                tc_fence_after();
                const int j0 = it.k_begin + t * TKEYS;
                const bool masked = j0 + TKEYS > it.n_ctx || j0 + TKEYS > it.k_end;
                const uint32_t tb = tlane + TM_S + sb * 128;               // this tile's S / P buffer, this warp's lanes
                const int jr = j0 + key0;                                  // first key of this replica's share
                // which of 16 keys from `base` on this row may see: inside the range, and committed context or an ancestor
                auto visible16 = [&](int base) -> uint32_t {
                    if (!masked) return 0xffffu;
                    const int nr = it.k_end - base, nc = it.n_ctx - base;
                    const uint32_t in_range = nr >= 16 ? 0xffffu : nr <= 0 ? 0u : (1u << nr) - 1u;
                    const uint32_t in_ctx = nc >= 16 ? 0xffffu : nc <= 0 ? 0u : (1u << nc) - 1u;
                    const uint32_t tree_bits = nc >= 16 ? 0u : nc > 0 ? (uint32_t)(anc << nc) : (nc > -64 ? (uint32_t)(anc >> -nc) : 0u);
                    return in_range & (in_ctx | tree_bits) & 0xffffu;
                };
                // pass 1: the row maximum over this replica's keys of the tile (16 keys at a time: the loop body stays
                // small enough to live in the instruction cache)
                float m_tile = -INFINITY;
                if (warp_live) {
#pragma unroll 1
                    for (int c = 0; c < KR / 16; ++c) {
                        uint32_t r[16];
                        tc_ld16(tb + key0 + c * 16, r);
                        const uint32_t vis = visible16(jr + c * 16);
#pragma unroll
                        for (int e = 0; e < 16; ++e) m_tile = fmaxf(m_tile, ((vis >> e) & 1u) ? __uint_as_float(r[e]) : -INFINITY);
                    }
                }
                float m_new = m_run, corr = 1.f;
                if (live && m_tile > m_run + RESCALE_GAP) {            // also the first tile with a visible key (m_run = -inf)
                    m_new = m_tile;
                    corr = (m_run == -INFINITY) ? 1.f : ex2(m_run - m_new);
                }
                if (warp_live && __any_sync(0xffffffffu, corr != 1.f)) {
                    // rare: the running maximum moved.  O is rescaled once the previous tile's P V has written it
                    // (the one before that finished earlier: MMAs complete in order).
                    if (s_cnt > 0 && !(ok = mbar_wait(pvdone_bar(sb ^ 1), ((s_cnt - 1) >> 1) & 1, &abort_sh, a.status))) break;
                    tc_fence_after();
#pragma unroll 1
                    for (int c = 0; c < 4; ++c) {
                        uint32_t r[32];
                        tc_ld32(tlane + TM_O + c * 32, r);
#pragma unroll
                        for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * corr);
                        tc_st32(tlane + TM_O + c * 32, r);
                    }
                }
                // pass 2: weights and their row sum; P replaces S in place, per 16 keys 8 columns of bf16 pairs hi and
                // 8 columns lo; the key columns of the other replicas are zeroed (their scores are not this row's business)
                float l_tile = 0.f;
                if (warp_live) {
                    const float m_use = m_new == -INFINITY ? 0.f : m_new;   // no visible key yet: every weight is masked to 0
#pragma unroll 1
                    for (int c = 0; c < TKEYS / 16; ++c) {
                        uint32_t w[16];
                        if (c * 16 < key0 || c * 16 >= key0 + KR) {
#pragma unroll
                            for (int e = 0; e < 16; ++e) w[e] = 0u;
                        } else {
                            uint32_t r[16];
                            tc_ld16(tb + c * 16, r);
                            const uint32_t vis = visible16(j0 + c * 16);
#pragma unroll
                            for (int e = 0; e < 16; e += 2) {
                                const float p0 = ((vis >> e) & 1u) ? ex2(__uint_as_float(r[e]) - m_use) : 0.f;
                                const float p1 = ((vis >> (e + 1)) & 1u) ? ex2(__uint_as_float(r[e + 1]) - m_use) : 0.f;
                                l_tile += p0 + p1;
                                split_pair(p0, p1, w[e >> 1], w[8 + (e >> 1)]);
                            }
                        }
                        tc_st16(tb + c * 16, w);
                    }
                }
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(pfull_bar(sb));             // P (and the rescaled O) are in place
                l_run = l_run * corr + l_tile;
                m_run = m_new;
            }
            if (!ok) break;
            // the last P V of the item (and with it all earlier ones) has written O
            if (it.n_tiles > 0 && !(ok = mbar_wait(pvdone_bar((s_cnt - 1) & 1), ((s_cnt - 1) >> 1) & 1, &abort_sh, a.status))) break;
            tc_fence_after();
            // ---- the item's result: O row from TMEM (zeros for an empty key range) ----
            const int n_part = a.nsplit * a.reps;                      // key ranges to merge: CTAs x replicas
            const bool single = n_part == 1;
            const size_t o0 = ((size_t)(it.be * a.M + node) * a.H + h) * HD;
            float *pdst = a.part + ((((size_t)it.be * a.H + h) * a.M + node) * n_part + it.split * a.reps + rep) * ROWF;
            const float inv = single ? 1.f / l_run : 1.f;
            if (warp_live) {
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    uint32_t r[32];
                    if (it.n_tiles > 0) {
                        tc_ld32(tlane + TM_O + c * 32, r);
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e) r[e] = 0u;
                    }
                    if (!live) continue;
                    if (single) {
#pragma unroll
                        for (int e = 0; e < 32; e += 8) {
                            uint4 hi, lo;
                            split_pair(__uint_as_float(r[e]) * inv, __uint_as_float(r[e + 1]) * inv, hi.x, lo.x);
                            split_pair(__uint_as_float(r[e + 2]) * inv, __uint_as_float(r[e + 3]) * inv, hi.y, lo.y);
                            split_pair(__uint_as_float(r[e + 4]) * inv, __uint_as_float(r[e + 5]) * inv, hi.z, lo.z);
                            split_pair(__uint_as_float(r[e + 6]) * inv, __uint_as_float(r[e + 7]) * inv, hi.w, lo.w);
                            *reinterpret_cast<uint4 *>(a.out + o0 + c * 32 + e) = hi;
                            *reinterpret_cast<uint4 *>(a.out + a.out_plane + o0 + c * 32 + e) = lo;
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; e += 2)
                            *reinterpret_cast<float2 *>(pdst + c * 32 + e) = make_float2(__uint_as_float(r[e]), __uint_as_float(r[e + 1]));
                    }
                }
                if (live && !single) { pdst[HD] = m_run * 0.6931471805599453f; pdst[HD + 1] = l_run; }   // natural-log units
            }
            if (it.n_tiles > 0) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(ofree_bar);                 // the next item may overwrite O
            }
            if (!single && a.fuse_merge) {
                // last key range of this (sequence, kv head) to finish merges all of them, in range order
                __threadfence();
                if (!(ok = wg_sync())) break;
                if (et == 0) {
                    const int old = atomicAdd(&a.counters[it.be * a.Hkv + it.g], 1);
                    last_sh = old == a.nsplit - 1;
                    if (last_sh) a.counters[it.be * a.Hkv + it.g] = 0;
                }
                if (!(ok = wg_sync())) break;
                if (last_sh) {
                    __threadfence();
                    for (int r = warp - 2; r < QR; r += 4) {
                        const int hh = it.g * grp + r / a.M, i = r % a.M;
                        const float *src = a.part + (((size_t)it.be * a.H + hh) * a.M + i) * (size_t)n_part * ROWF;
                        // lane s holds range s's (max, sum); the weights go round by shuffle (at most 32 ranges when fused)
                        float ms = -INFINITY, ls = 0.f;
                        if (lane < n_part) { ms = __ldcg(src + (size_t)lane * ROWF + HD); ls = __ldcg(src + (size_t)lane * ROWF + HD + 1); }
                        float num[HD / 32];
#pragma unroll
                        for (int e = 0; e < HD / 32; ++e) num[e] = 0.f;
                        const float mmax = warp_max(ms);
                        const float w = (ms == -INFINITY) ? 0.f : expf(ms - mmax);
                        const float den = warp_sum(ls * w);
                        for (int s0 = 0; s0 < n_part; s0 += 4) {
                            float v[4][HD / 32];
#pragma unroll
                            for (int q = 0; q < 4; ++q)
#pragma unroll
                                for (int e = 0; e < HD / 32; ++e)
                                    v[q][e] = s0 + q < n_part ? __ldcg(src + (size_t)(s0 + q) * ROWF + lane + 32 * e) : 0.f;
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const float wq = __shfl_sync(0xffffffffu, w, (s0 + q) & 31);
#pragma unroll
                                for (int e = 0; e < HD / 32; ++e) num[e] = fmaf(v[q][e], s0 + q < n_part ? wq : 0.f, num[e]);
                            }
                        }
                        const float invd = 1.f / den;
#pragma unroll
                        for (int e = 0; e < HD / 32; ++e)
                            store_act<__nv_bfloat16>(a.out, a.out_plane, ((size_t)(it.be * a.M + i) * a.H + hh) * HD + lane + 32 * e,
                                                     num[e] * invd);
                    }
                }
                if (!(ok = wg_sync())) break;                          // last_sh is reused by the next item
            }
        }
    }

    // ---------------- teardown ----------------
    __syncwarp();
    if (abort_sh && threadIdx.x == 0) {
        // give copies and MMAs that are still in flight time to land before shared memory and TMEM go away
        const long long t0 = clock64();
        while (clock64() - t0 < 400000) { }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
    }
}

}  // namespace

// Replicas of the query rows across the 128 TMEM lanes (each takes a share of every tile's keys)
int attention_tc_replicas(int query_rows) { return query_rows <= 32 ? 4 : query_rows <= 64 ? 2 : 1; }

// tensor maps over the caches are rebuilt only when the caller's pointers change
static int cache_maps_tc(viasd_model *m, CacheMaps &cm, const void *kc, const void *vc, int n_layers) {
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
int launch_attention_tc(viasd_model *m, const void *kc, const void *vc, bool slim, int layer_ord, const void *kc2,
                        const void *vc2, int layer_ord2, int streams, int batch, int M, int nsplit, int fuse_merge,
                        cudaStream_t st) {
    const viasd_config &c = m->cfg;
    CacheMaps &cm = slim ? m->cmaps_slim : m->cmaps_full;
    int rc;
    if ((rc = cache_maps_tc(m, cm, kc, vc, slim ? m->n_routed : c.n_layers))) return rc;
    CacheMaps *cm2 = &cm;
    if (streams == 2) {
        cm2 = &m->cmaps_slim;
        if ((rc = cache_maps_tc(m, *cm2, kc2, vc2, m->n_routed))) return rc;
    }
    const int grp = c.n_heads / c.n_kv_heads, QR = grp * M;
    if (QR > 128) return VIASD_EINVAL;
    AttnTcArgs a;
    a.q = m->ws.q; a.part = m->ws.part; a.out = (__nv_bfloat16 *)m->ws.attn;
    a.out_plane = m->ws.rows_alloc * (size_t)c.n_heads * HD;
    a.len_eff = m->ws.len_eff; a.tree = m->ws.tree; a.status = &m->ws.stats->device_status; a.run_flag = m->run_flag;
    a.M = M; a.H = c.n_heads; a.Hkv = c.n_kv_heads; a.max_batch = c.max_batch; a.max_ctx = c.max_ctx;
    a.layer_ord = layer_ord; a.nsplit = nsplit; a.scale = 1.4426950408889634f / sqrtf((float)HD);   // log2(e) / sqrt(hd)
    a.batch = batch; a.layer_ord2 = layer_ord2; a.streams = streams;
    a.counters = m->ws.attn_counters;
    a.fuse_merge = fuse_merge;
    a.qrows8 = (QR + 7) / 8 * 8;
    a.reps = attention_tc_replicas(QR);
    a.rows_per_rep = 128 / a.reps;
    {
        // staged query regions (hi / lo x two 64-dim chunks).  A region nominally spans 128 rows of 128 bytes, but
        // only qrows8 rows per replica block are live, so regions are interleaved in the dead rows where they fit.
        const uint32_t slot = (uint32_t)a.qrows8 * 128u, period = (uint32_t)a.rows_per_rep * 128u;
        const uint32_t per_period = a.reps == 1 ? 1u : period / slot;
        for (uint32_t k = 0; k < 4; ++k)
            a.qoff[k] = a.reps == 1 ? k * slot : (k / per_period) * 16384u + (k % per_period) * slot;
        a.q_bytes = a.qoff[3] + (uint32_t)(a.reps - 1) * period + slot;
    }
    a.n_items = streams * batch * c.n_kv_heads * nsplit;
    int grid = a.n_items < m->sm_count ? a.n_items : m->sm_count;
    a.items_per_cta = (a.n_items + grid - 1) / grid;
    grid = (a.n_items + a.items_per_cta - 1) / a.items_per_cta;
    const size_t q_bytes = a.q_bytes;
    a.nstage = 1024 + q_bytes + 3 * (size_t)STAGE_BYTES <= 220 * 1024 ? 3 : 2;
    const size_t smem = 1024 + q_bytes + a.nstage * (size_t)STAGE_BYTES;
    static bool attr_done[64];
    if (first_use_on_device(attr_done)) {
        CUDA_TRY(cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024));
    }
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    pdl_config(cfg, attr, dim3(grid), dim3(AT_THREADS), smem, st);
    CUDA_TRY(cudaLaunchKernelEx(&cfg, attention_tc_kernel, cm.k, cm.v, cm2->k, cm2->v, a));
    LAUNCH_CHECK();
    return VIASD_OK;
}

