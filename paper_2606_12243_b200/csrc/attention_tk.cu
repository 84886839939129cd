// Block attention on tcgen05 for few query rows (at most 32 per kv head): keys on the TMEM lanes.
//
// With 5-27 query rows an MMA whose M dimension is the query rows would be almost all padding.  Here the
// roles are swapped, as in the projection GEMMs: the 128 keys of a tile are the MMA's M dimension and the
// query rows its N dimension,
//
//   S^T[128 keys, rows] = K Q^T      A = K tile exactly as its TMA box lands (K-major, 128-byte swizzle)
//                                    B = Q, hi rows then lo rows (N = 2 x rows: x = hi + lo to ~16 bits)
//   O^T[128 dims, rows] += V^T P^T   A = V tile as it lands, read MN-major (the keys are the contraction)
//                                    B = P^T, hi rows then lo rows, written by the softmax threads into
//                                        shared memory in the swizzled K-major layout
//
// so a tile costs 16 MMAs of 128 x N x 16 with N = 16..64 instead of 32 of 128 x 128 x 16.
// A softmax thread owns a key (a TMEM lane) and sees all query rows of it.  Row maxima are exchanged once per
// tile (warp shuffles, then four values per row through shared memory and one barrier of the four warps); the
// running maximum only moves when a tile exceeds it by 2^8, so rescaling O^T in TMEM is rare, and every thread
// takes that decision from the same exchanged values.  Row sums stay per thread until the item ends.
//
// Warp roles (192 threads): warp 0 requests K/V tiles by TMA into a ring that runs across the CTA's items,
// warp 1 owns TMEM and issues the MMAs, warps 2-5 stage Q, run the softmax and write the result.
// TMEM: S^T double-buffered (2 x 64 columns), O^T (64 columns).
// Every wait is bounded: on expiry the CTA records VIASD_EDEVICE, lets its copies land and leaves.
#include "common.cuh"
#include "tc_ptx.cuh"
#include <stdlib.h>

namespace {

constexpr int HD = 128;                        // head dimension
constexpr int TKEYS = 128;                     // keys per tile
constexpr int HALF_BYTES = TKEYS * 128;        // 128 keys x 64 dims of bf16, as one TMA box lands
constexpr int SLOT_BYTES = 2 * HALF_BYTES;     // one tile of K or of V: dims 0..63, dims 64..127
constexpr int TK_THREADS = 192;                 // two service warps and four softmax warps (eight at 32 query rows)
constexpr int TK_MAX_STAGE = 3;
constexpr int ROWF = HD + 2;                   // partial row: 128 numerators, max (natural-log units), sum
constexpr float RESCALE_GAP = 8.f;             // log2 units
constexpr uint32_t TM_S = 0, TM_O = 128;       // TMEM column offsets: S^T buffers at 0 and 64, O^T at 128

struct AttnTkArgs {
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
    int streams, n_items, items_per_cta, fuse_merge, nk, nv;   // nk, nv: ring slots for K tiles and for V tiles
    int subs;                   // item groups per kv head: with more than 32 query rows per kv head, the query heads of a
                                // kv head are dealt to `subs` items (each streams the K/V tiles again, from L2)
    int flat, part_slots;       // flat: tiles (not key ranges) are dealt evenly to the CTAs; part_slots: partial slots per (row, head)
    int *counters;              // arrivals per (stream, sequence, kv head), zero between launches
    float scale;                // log2(e) / sqrt(hd)
};

struct Item { int be, b, g, stream, split, n_split, n_ctx, k_begin, k_end, n_tiles, row_base; };   // split of n_split key ranges of the pair

__device__ __forceinline__ Item decode_item(const AttnTkArgs &a, int item) {
    Item it;
    it.split = item % a.nsplit;
    it.n_split = a.nsplit;
    const int bg = item / a.nsplit;
    it.g = bg % (a.Hkv * a.subs);                  // group of query heads: kv head it.g / subs, part it.g % subs of its heads
    it.be = bg / (a.Hkv * a.subs);
    it.stream = it.be / a.batch;
    it.b = it.be - it.stream * a.batch;
    it.n_ctx = a.len_eff[it.b];
    const int Tk = it.n_ctx + a.M;
    int chunk = (Tk + a.nsplit - 1) / a.nsplit;
    chunk = (chunk + TKEYS - 1) / TKEYS * TKEYS;
    it.k_begin = it.split * chunk;
    it.k_end = min(Tk, it.k_begin + chunk);
    it.n_tiles = it.k_end > it.k_begin ? (it.k_end - it.k_begin + TKEYS - 1) / TKEYS : 0;
    it.row_base = (((it.stream ? a.layer_ord2 : a.layer_ord) * a.max_batch + it.b) * a.Hkv + it.g / a.subs) * a.max_ctx;
    return it;
}

// The CTA's work list, one item after the other.  Two ways of cutting the work:
//  - a.flat == 0: every (sequence, kv head) pair is cut into a.nsplit key ranges, and the ranges are dealt to the CTAs
//    in equal contiguous shares (whole items: 320 items on 148 SMs leave a quarter of the SMs idle);
//  - a.flat == 1: the tiles of all pairs of a row stream, laid end to end, are cut into one range of `per` tiles per
//    CTA; a pair that straddles a cut gets one key range per CTA it reaches.  The cuts depend on the lengths, the
//    number of kv heads and the grid only, so a one-stream launch and a two-stream launch (each CTA takes its
//    range of both streams) cut the same pairs at the same keys and produce the same bits.
struct ItemSrc { int item, i1, s, b, g, off; };
__device__ __forceinline__ void src_init(const AttnTkArgs &a, ItemSrc &c) {
    c.item = blockIdx.x * a.items_per_cta;
    c.i1 = min(a.n_items, c.item + a.items_per_cta);
    c.s = c.b = c.g = c.off = 0;
}
__device__ __forceinline__ bool next_item(const AttnTkArgs &a, int per, ItemSrc &c, Item &it) {
    if (!a.flat) {
        if (c.item >= c.i1) return false;
        it = decode_item(a, c.item++);
        return true;
    }
    const int lo = blockIdx.x * per, hi = lo + per, HkvV = a.Hkv * a.subs;
    while (c.s < a.streams) {
        if (c.b >= a.batch || c.off >= hi) { ++c.s; c.b = c.g = c.off = 0; continue; }   // done with this stream
        const int n_ctx = a.len_eff[c.b], Tk = n_ctx + a.M, tb = (Tk + TKEYS - 1) / TKEYS;
        if (c.off + HkvV * tb <= lo) { c.off += HkvV * tb; ++c.b; c.g = 0; continue; }      // this sequence ends before the range
        if (c.g == 0 && c.off < lo) c.g = (lo - c.off) / tb;                                // its first pair that reaches into the range
        const int p_lo = c.off + c.g * tb;
        if (c.g >= HkvV) { c.off += HkvV * tb; ++c.b; c.g = 0; continue; }
        if (p_lo >= hi) { ++c.s; c.b = c.g = c.off = 0; continue; }
        const int p_hi = p_lo + tb, t0 = max(lo, p_lo) - p_lo, t1 = min(hi, p_hi) - p_lo;
        const int first = p_lo / per, last = (p_hi - 1) / per;
        it.b = c.b; it.stream = c.s; it.be = c.s * a.batch + c.b; it.g = c.g;
        it.split = (int)blockIdx.x - first; it.n_split = last - first + 1;
        it.n_ctx = n_ctx; it.k_begin = t0 * TKEYS; it.k_end = min(Tk, t1 * TKEYS); it.n_tiles = t1 - t0;
        it.row_base = (((c.s ? a.layer_ord2 : a.layer_ord) * a.max_batch + c.b) * a.Hkv + c.g / a.subs) * a.max_ctx;
        ++c.g;
        return true;
    }
    return false;
}

__device__ __forceinline__ float ex2(float x) {            // 2^x, hardware approximation (2 ulp)
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// MN-major operand tile with the 128-byte swizzle: 64 contiguous elements along MN per row of 128 bytes,
// 8 rows (8 steps of the contraction) per 1024-byte group; groups `sbo` bytes apart along the contraction,
// 64-element blocks `lbo` bytes apart along MN.
__device__ __forceinline__ uint64_t smem_desc_mn(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((addr >> 4) & 0x3FFF) | ((uint64_t)((lbo >> 4) & 0x3FFF) << 16) | ((uint64_t)((sbo >> 4) & 0x3FFF) << 32) |
           (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
          "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// hi + lo columns of RG accumulator rows: v[i] = column row0 + i plus column NR + row0 + i
template <int NR, int RG>
__device__ __forceinline__ void load_rows(uint32_t taddr, int row0, float (&v)[RG]) {
    if constexpr (RG == 16 && NR == 32) {
        uint32_t hi[16], lo[16];
        tc_ld16(taddr + row0, hi);
        tc_ld16(taddr + NR + row0, lo);
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(hi[i]) + __uint_as_float(lo[i]);
        return;
    }
    float t[2 * NR];
#pragma unroll
    for (int c = 0; c < 2 * NR / 16; ++c) {
        uint32_t r[16];
        tc_ld16(taddr + c * 16, r);
#pragma unroll
        for (int e = 0; e < 16; ++e) t[c * 16 + e] = __uint_as_float(r[e]);
    }
#pragma unroll
    for (int r = 0; r < RG; ++r) v[r] = t[r] + t[NR + r];
}

// byte offset of element (row, col) in a K-major tile of 128-byte rows with the 128-byte swizzle; col in bf16 units < 64
__device__ __forceinline__ uint32_t sw_off(uint32_t row, uint32_t col) {
    return row * 128u + ((((col >> 3) ^ (row & 7u))) << 4) + (col & 7u) * 2u;
}


template <int NR>                                           // query rows per kv head rounded up to 8, 16 or 32
__global__ void __launch_bounds__(NR == 32 ? TK_THREADS + 128 : TK_THREADS, 1)
attention_tk_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                    const __grid_constant__ CUtensorMap map_k2, const __grid_constant__ CUtensorMap map_v2, const AttnTkArgs a) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) unsigned long long bars[4 * TK_MAX_STAGE + 10];
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh, last_sh, per_sh;
    constexpr int SG = NR == 32 ? 2 : 1;                    // groups of four softmax warps; a group takes RG of the query rows
    constexpr int RG = NR / SG, SW = 4 * SG, ST = 128 * SG; // rows per group, softmax warps, softmax threads
    __shared__ float wmax_sh[2][4][NR];                     // per tile parity, per lane quarter: row maxima of its 32 keys
    __shared__ float mref_sh[SW][RG];                        // per warp (each keeps its own copy): the rows' running maxima, 0 while none
    __shared__ float corr_sh[SW][RG];                        // per warp: rescale factors of a tile in which a maximum moved
    __shared__ float mraw_sh[NR];                           // the rows' running maxima at the end of an item (-inf: no visible key)
    __shared__ unsigned long long anc_sh[VIASD_MAX_ROWS_PER_SEQ];

    constexpr int NC = 2 * NR;                              // MMA N: hi rows then lo rows
    constexpr bool SPLIT = NR == 32;                        // K and V tiles in rings of their own (else a slot holds a tile's K and V)
    constexpr uint32_t QCH = (uint32_t)NC * 128u;           // one 64-wide chunk of an [NC rows] operand
    RUN_FLAG_EXIT(a.run_flag);
    PDL_TRIGGER();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int NK = a.nk, NV = a.nv;
    const int HkvV = a.Hkv * a.subs, grp = a.H / HkvV, QR = grp * a.M;   // query heads and rows per item group
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t qsm = base, psm = base + 2 * QCH, ring = base + 6 * QCH;   // Q (2 chunks), P^T (2 buffers x 2 chunks), ring
    uint8_t *gen = smem_raw + (base - smem_u32(smem_raw));
    // K tiles and V tiles have rings of their own: a K slot is free as soon as S^T = K Q^T has read it, long before the
    // tile's V, so the next K tiles are on their way while the softmax of the current one runs
    auto fullk_bar = [&](int s) { return smem_u32(&bars[s]); };
    auto emptyk_bar = [&](int s) { return smem_u32(&bars[TK_MAX_STAGE + s]); };
    auto fullv_bar = [&](int s) { return smem_u32(&bars[2 * TK_MAX_STAGE + s]); };
    auto emptyv_bar = [&](int s) { return smem_u32(&bars[3 * TK_MAX_STAGE + s]); };
    auto sfull_bar = [&](int b) { return smem_u32(&bars[4 * TK_MAX_STAGE + b]); };
    auto pfull_bar = [&](int b) { return smem_u32(&bars[4 * TK_MAX_STAGE + 2 + b]); };
    auto pvdone_bar = [&](int b) { return smem_u32(&bars[4 * TK_MAX_STAGE + 4 + b]); };
    const uint32_t ofree_bar = smem_u32(&bars[4 * TK_MAX_STAGE + 6]), qfull_bar = smem_u32(&bars[4 * TK_MAX_STAGE + 7]);
    const uint32_t wg_bar = smem_u32(&bars[4 * TK_MAX_STAGE + 8]);      // the softmax warps among themselves (bounded)

    if (threadIdx.x == 0) {
        for (int s = 0; s < TK_MAX_STAGE; ++s) { mbar_init(fullk_bar(s), 1); mbar_init(emptyk_bar(s), 1); mbar_init(fullv_bar(s), 1); mbar_init(emptyv_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(sfull_bar(b), 1); mbar_init(pfull_bar(b), SW); mbar_init(pvdone_bar(b), 1); }
        mbar_init(ofree_bar, SW);
        mbar_init(qfull_bar, SW);
        mbar_init(wg_bar, ST);
        abort_sh = 0;
        last_sh = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (threadIdx.x == 64) {
        // tiles per CTA when the tiles are dealt evenly: a pair may not be cut into more ranges than it has partial slots
        int per = 1;
        if (a.flat) {
            int T = 0, tmax = 1;
            for (int b = 0; b < a.batch; ++b) { const int tb = (a.len_eff[b] + a.M + TKEYS - 1) / TKEYS; T += a.Hkv * a.subs * tb; tmax = max(tmax, tb); }
            per = max(max((T + (int)gridDim.x - 1) / (int)gridDim.x, (tmax + a.part_slots - 2) / (a.part_slots - 1)), 1);
        }
        per_sh = per;
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_sh)), "r"(256) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_sh;
    const int per = per_sh;

    if (warp == 0) {
        // ---------------- TMA producer: the CTA's (item, tile) list, flattened ----------------
        if (lane == 0) {
            const uint64_t kvpol = l2_evict_first_policy();    // the cache passes through once per layer
            if constexpr (!SPLIT) {
                // few query rows: a tile's K and V share a ring slot and are requested together
                int p_tile = 0, p_count = 0;
                bool ok = true;
                ItemSrc src;
                src_init(a, src);
                Item pit;
                bool p_more = next_item(a, per, src, pit);
                auto issue_next = [&](bool context_only) -> bool {  // false: nothing (more) to request under this condition
                    while (p_more && p_tile >= pit.n_tiles) { p_tile = 0; p_more = next_item(a, per, src, pit); }
                    if (!p_more) return false;
                    const int k0 = pit.k_begin + p_tile * TKEYS;
                    if (context_only && k0 + TKEYS > pit.n_ctx) return false;   // this tile holds rows the previous kernel writes
                    const int st = p_count % NK;
                    if (p_count >= NK && !(ok = mbar_wait(emptyk_bar(st), ((p_count / NK) & 1) ^ 1, &abort_sh, a.status))) return false;
                    const uint32_t bar = fullk_bar(st), dst = ring + st * 2 * SLOT_BYTES;
                    const CUtensorMap *mk = pit.stream ? &map_k2 : &map_k, *mv = pit.stream ? &map_v2 : &map_v;
                    const int y = pit.row_base + k0;
                    mbar_expect_tx(bar, 2 * SLOT_BYTES);
                    tma_load_2d_hint(dst, mk, bar, 0, y, kvpol);
                    tma_load_2d_hint(dst + HALF_BYTES, mk, bar, 64, y, kvpol);
                    tma_load_2d_hint(dst + 2 * HALF_BYTES, mv, bar, 0, y, kvpol);
                    tma_load_2d_hint(dst + 3 * HALF_BYTES, mv, bar, 64, y, kvpol);
                    ++p_tile; ++p_count;
                    return true;
                };
                // committed context does not change during the pass: ask for it before waiting for the previous kernel
                while (p_count < NK && issue_next(true)) { }
                PDL_WAIT();
                while (ok && issue_next(false)) { }
            } else {
            struct Cursor { ItemSrc src; bool more; int tile, count; Item it; };
            Cursor ck;
            src_init(a, ck.src);
            ck.tile = ck.count = 0;
            ck.more = next_item(a, per, ck.src, ck.it);
            Cursor cv = ck;
            // 1: requested; 0: the slot is still being read; -1: nothing (more) to request under this condition
            auto request = [&](Cursor &c, bool is_v, bool context_only) -> int {
                while (c.more && c.tile >= c.it.n_tiles) { c.tile = 0; c.more = next_item(a, per, c.src, c.it); }
                if (!c.more) return -1;
                const int k0 = c.it.k_begin + c.tile * TKEYS;
                if (context_only && k0 + TKEYS > c.it.n_ctx) return -1;     // this tile holds rows the previous kernel writes
                const int n = is_v ? NV : NK, st = c.count % n;
                if (c.count >= n && !mbar_test(is_v ? emptyv_bar(st) : emptyk_bar(st), ((c.count / n) & 1) ^ 1)) return 0;
                const uint32_t bar = is_v ? fullv_bar(st) : fullk_bar(st), dst = ring + (uint32_t)(is_v ? NK + st : st) * SLOT_BYTES;
                const CUtensorMap *mp = is_v ? (c.it.stream ? &map_v2 : &map_v) : (c.it.stream ? &map_k2 : &map_k);
                const int y = c.it.row_base + k0;
                mbar_expect_tx(bar, SLOT_BYTES);
                tma_load_2d_hint(dst, mp, bar, 0, y, kvpol);
                tma_load_2d_hint(dst + HALF_BYTES, mp, bar, 64, y, kvpol);
                ++c.tile; ++c.count;
                return 1;
            };
            // committed context does not change during the pass: ask for it before waiting for the previous kernel
            while (ck.count < NK && request(ck, false, true) == 1) { }
            while (cv.count < NV && request(cv, true, true) == 1) { }
            PDL_WAIT();
            // K first, then V, whichever has a free slot; bounded like every wait: no request for too long ends the CTA
            long long t_last = clock64();
            int rk = 0, rv = 0;
            while (rk >= 0 || rv >= 0) {
                if (rk >= 0) rk = request(ck, false, false);
                if (rv >= 0) rv = request(cv, true, false);
                if (rk == 1 || rv == 1) { t_last = clock64(); continue; }
                if (*(volatile int *)&abort_sh) break;
                if (clock64() - t_last > WAIT_LIMIT_CYCLES) { abort_sh = 1; atomicExch(a.status, VIASD_EDEVICE); break; }
                // nothing to request right now: sleep on the slot that frees first (K's while K has tiles left); the
                // hardware wakes the thread when the phase completes or after its own short limit (a suspend-time
                // hint woke it late, not early: 0.25 us per tile)
                if (rk == 0) mbar_try_wait(emptyk_bar(ck.count % NK), ((ck.count / NK) & 1) ^ 1);
                else mbar_try_wait(emptyv_bar(cv.count % NV), ((cv.count / NV) & 1) ^ 1);
            }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NC >> 3) << 17) | ((128u >> 4) << 24);
            const uint32_t idesc_pv = idesc | (1u << 15);                 // A (the V tile) is MN-major
            int c_tile = 0, n_q = 0, o_uses = 0, q_be = -1, q_g = -1;   // c_tile: tiles of earlier items (ring and buffer phase)
            bool ok = true;
            // tile g (counted over the whole CTA) uses K slot g % NK, V slot g % NV, S^T buffer g & 1 and P^T buffer g & 1
            auto issue_qk = [&](int g) -> bool {
                const int st = g % NK, sb = g & 1;
                if (!mbar_wait(fullk_bar(st), (g / NK) & 1, &abort_sh, a.status)) return false;
                tc_fence_after();
                const uint32_t kst = ring + st * (SPLIT ? 1 : 2) * SLOT_BYTES, d = tmem + TM_S + sb * 64;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    tc_mma(d, smem_desc(kst + (ks >> 2) * HALF_BYTES + (ks & 3) * 32), smem_desc(qsm + (ks >> 2) * QCH + (ks & 3) * 32),
                           idesc, ks > 0 ? 1u : 0u);
                if (SPLIT) tc_commit(emptyk_bar(st));                     // the K slot is free once these MMAs have read it
                tc_commit(sfull_bar(sb));
                return true;
            };
            ItemSrc src;
            src_init(a, src);
            Item it;
            while (ok && next_item(a, per, src, it)) {
                if (it.be != q_be || it.g != q_g) {
                    if (!(ok = mbar_wait(qfull_bar, n_q & 1, &abort_sh, a.status))) break;
                    ++n_q; q_be = it.be; q_g = it.g;
                }
                if (it.n_tiles == 0) continue;
                // issue order S(0), S(1), O(0), S(2), O(1), ...: S(t + 2) is only issued once the softmax of tile t has
                // read its buffer (it arrived on p_full(t)), and its completion implies that O(t) has read P^T(t)
                if (!(ok = issue_qk(c_tile))) break;
                if (it.n_tiles > 1 && !(ok = issue_qk(c_tile + 1))) break;
                for (int t = 0; t < it.n_tiles; ++t) {
                    const int g = c_tile + t, sb = g & 1, st = g % NV;
                    if (t == 0 && o_uses > 0 && !(ok = mbar_wait(ofree_bar, (o_uses - 1) & 1, &abort_sh, a.status))) break;
                    if (SPLIT && !(ok = mbar_wait(fullv_bar(st), (g / NV) & 1, &abort_sh, a.status))) break;
                    if (!(ok = mbar_wait(pfull_bar(sb), (g >> 1) & 1, &abort_sh, a.status))) break;
                    tc_fence_after();
                    const uint32_t vst = SPLIT ? ring + (uint32_t)(NK + st) * SLOT_BYTES : ring + (uint32_t)(2 * st + 1) * SLOT_BYTES;
                    const uint32_t pb = psm + sb * 2 * QCH;
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)                        // 16 keys per step: two 8-key groups of 1024 bytes
                        tc_mma(tmem + TM_O, smem_desc_mn(vst + kk * 2048, HALF_BYTES, 1024),
                               smem_desc(pb + (kk >> 2) * QCH + (kk & 3) * 32), idesc_pv, (t > 0 || kk > 0) ? 1u : 0u);
                    tc_commit(SPLIT ? emptyv_bar(st) : emptyk_bar(st));   // the slot is free once these MMAs have read it
                    tc_commit(pvdone_bar(sb));
                    if (t + 2 < it.n_tiles && !(ok = issue_qk(g + 2))) break;
                }
                c_tile += it.n_tiles;
                ++o_uses;
            }
        }
    } else {
        // ---------------- softmax / epilogue (warps 2..5 <-> TMEM lane quarters 2,3,0,1): one thread, one key (later one dim) ----------------
        // With 32 query rows a second group of four warps (6..9, the same lane quarters) takes rows 16..31: the softmax
        // of a tile is then half as long per thread, and two warps per scheduler hide each other's latencies.
        const int quarter = warp & 3, kl = quarter * 32 + lane, et = threadIdx.x - 64;   // kl: key of the tile / dim of O^T
        const int sw = warp - 2, row0 = (sw >> 2) * RG;            // softmax warp number; first query row of its group
        const uint32_t tlane = tmem + ((uint32_t)(quarter * 32) << 16);
        int s_cnt = 0, q_be = -1, q_g = -1, wg_phase = 0;        // s_cnt: tiles this CTA has finished (buffer phase)
        int anc_b = -1;                                          // sequence whose ancestor sets anc_sh holds
        bool ok = true;
        auto wg_sync = [&]() -> bool {
            mbar_arrive(wg_bar);
            const bool done = mbar_wait(wg_bar, wg_phase & 1, &abort_sh, a.status);
            ++wg_phase;
            return done;
        };
        // (A dry first item, run on whatever TMEM holds before the dependency wait to warm the instruction cache, paid
        // while the streamed weights pushed the kernels' code out of L2 between launches; with the weights marked
        // evict-first the code stays in L2 and the dry item only delayed the first real one: removed.)
        ItemSrc src;
        src_init(a, src);
        for (int n_item = 0; ok; ++n_item) {
            Item it;
            if (!next_item(a, per, src, it)) break;
            if (n_item == 0) {
                PDL_WAIT();
            }
            if (it.b != anc_b) {
                // the ancestor sets of this sequence's draft tree (every sequence may have its own)
                if (n_item > 0 && !(ok = wg_sync())) break;           // nobody reads the previous sequence's sets any more
                if (et < a.M) anc_sh[et] = a.tree[it.b].anc[et];
                if (!(ok = wg_sync())) break;                         // anc_sh is visible
                anc_b = it.b;
            }
            if (it.be != q_be || it.g != q_g) {
                // stage the query rows of this (sequence, kv head): rows 0..NR-1 the hi parts, NR..2NR-1 the lo parts,
                // pre-scaled, in the K-major 128-byte-swizzled layout the MMA reads; loads first
                for (int idx0 = et; idx0 < NR * (HD / 2); idx0 += 4 * ST) {
                    float2 v[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int idx = idx0 + q * ST, r = idx / (HD / 2), d2 = (idx % (HD / 2)) * 2;
                        v[q] = make_float2(0.f, 0.f);
                        if (idx < NR * (HD / 2) && r < QR) {
                            const int h = it.g * grp + r / a.M, i = r % a.M;
                            v[q] = __ldcg(reinterpret_cast<const float2 *>(a.q + ((size_t)(it.be * a.M + i) * a.H + h) * HD + d2));
                        }
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int idx = idx0 + q * ST, r = idx / (HD / 2), d2 = (idx % (HD / 2)) * 2;
                        if (idx >= NR * (HD / 2)) continue;
                        const float x0 = v[q].x * a.scale, x1 = v[q].y * a.scale;
                        const __nv_bfloat162 hi = __floats2bfloat162_rn(x0, x1);
                        const __nv_bfloat162 lo = __floats2bfloat162_rn(x0 - __low2float(hi), x1 - __high2float(hi));
                        uint8_t *chunk = gen + (uint32_t)(d2 >> 6) * QCH;
                        *reinterpret_cast<__nv_bfloat162 *>(chunk + sw_off(r, d2 & 63)) = hi;
                        *reinterpret_cast<__nv_bfloat162 *>(chunk + sw_off(NR + r, d2 & 63)) = lo;
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> the MMA's reads
                __syncwarp();
                if (lane == 0) mbar_arrive(qfull_bar);
                q_be = it.be; q_g = it.g;
            }
            // Lane r of every warp keeps row r's running maximum (the four warps compute the same values); the other
            // lanes read it, as the exponent's reference, from the warp's copy in shared memory.
            float m_lane = -INFINITY, l_run[RG];
#pragma unroll
            for (int r = 0; r < RG; ++r) l_run[r] = 0.f;
            if (lane < RG) mref_sh[sw][lane] = 0.f;
            __syncwarp();

            for (int t = 0; t < it.n_tiles; ++t) {
                const int sb = s_cnt & 1;
                if (!(ok = mbar_wait(sfull_bar(sb), (s_cnt >> 1) & 1, &abort_sh, a.status))) break;
                tc_fence_after();
                float s[RG];
                load_rows<NR, RG>(tlane + TM_S + sb * 64, row0, s);
                // visibility: past the key range nothing; in the committed context everything; among the block's own
                // rows only the ancestors of the query's node
                const int j = it.k_begin + t * TKEYS + kl;
                if (j >= it.k_end) {
#pragma unroll
                    for (int r = 0; r < RG; ++r) s[r] = -INFINITY;
                } else if (j >= it.n_ctx) {
                    const int tb = j - it.n_ctx;
#pragma unroll
                    for (int r = 0; r < RG; ++r) if (!((anc_sh[(row0 + r) % a.M] >> tb) & 1ull)) s[r] = -INFINITY;
                }
                // row maxima: over the warp's 32 keys by one warp-wide reduction per row (lane r keeps row r's), over the
                // four warps through shared memory
                {
                    float mine = -INFINITY;
#pragma unroll
                    for (int r = 0; r < RG; ++r) {
                        float wm;
                        asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(wm) : "f"(s[r]));
                        if (lane == r) mine = wm;
                    }
                    if (lane < RG) wmax_sh[sb][quarter][row0 + lane] = mine;
                }
                if (!(ok = wg_sync())) break;
                bool moved_l = false;
                if (lane < RG) {
                    const int rr = row0 + lane;
                    const float mt = fmaxf(fmaxf(wmax_sh[sb][0][rr], wmax_sh[sb][1][rr]), fmaxf(wmax_sh[sb][2][rr], wmax_sh[sb][3][rr]));
                    float corr = 1.f;
                    if (mt > m_lane + RESCALE_GAP) {                   // also the first tile with a visible key (m_lane = -inf)
                        if (m_lane != -INFINITY) { corr = ex2(m_lane - mt); moved_l = true; }
                        m_lane = mt;
                        mref_sh[sw][lane] = mt;
                    }
                    corr_sh[sw][lane] = corr;
                }
                const bool moved = __any_sync(0xffffffffu, moved_l);
                __syncwarp();
                if (moved) {
                    // rare: a running maximum moved.  Every warp sees the same maxima, so all four come here
                    // together; O^T is rescaled once the previous tile's MMAs have written it.
#pragma unroll
                    for (int r = 0; r < RG; ++r) l_run[r] *= corr_sh[sw][r];
                    {
                        if (!(ok = mbar_wait(pvdone_bar(sb ^ 1), ((s_cnt - 1) >> 1) & 1, &abort_sh, a.status))) break;
                        tc_fence_after();
#pragma unroll
                        for (int c = 0; c < 2 * RG / 16; ++c) {             // this group's hi columns, then its lo columns
                            const uint32_t col = RG == 8 ? 0u : (uint32_t)(c * NR + row0);
                            uint32_t w[16];
                            tc_ld16(tlane + TM_O + col, w);
#pragma unroll
                            for (int e = 0; e < 16; ++e) w[e] = __float_as_uint(__uint_as_float(w[e]) * corr_sh[sw][(c * 16 + e) % RG]);
                            tc_st16(tlane + TM_O + col, w);
                        }
                        tc_wait_st();
                    }
                }
                // weights of this key for every row; P^T (hi rows, lo rows) into shared memory for the MMA
                uint8_t *pchunk = gen + 2 * QCH + (uint32_t)sb * 2 * QCH + (uint32_t)(kl >> 6) * QCH;
                float mref[RG];                                  // read before the stores below: they could alias, which would
#pragma unroll                                                   // put every one of these loads behind the previous row's stores
                for (int r = 0; r < RG; ++r) mref[r] = mref_sh[sw][r];
#pragma unroll
                for (int r = 0; r < RG; ++r) {
                    const float p = ex2(s[r] - mref[r]);                   // masked scores are -inf: weight 0
                    l_run[r] += p;
                    const __nv_bfloat16 hi = __float2bfloat16_rn(p), lo = __float2bfloat16_rn(p - __bfloat162float(hi));
                    *reinterpret_cast<__nv_bfloat16 *>(pchunk + sw_off(row0 + r, kl & 63)) = hi;
                    *reinterpret_cast<__nv_bfloat16 *>(pchunk + sw_off(NR + row0 + r, kl & 63)) = lo;
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> the MMA's reads
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(pfull_bar(sb));     // S^T is read, P^T (and the rescaled O^T) are in place
                ++s_cnt;
            }
            if (!ok) break;
            // ---- the item's result ----
            if (quarter == 0 && lane < RG) mraw_sh[row0 + lane] = m_lane;
            // the last MMA into O^T of the item (and with it all earlier ones) is complete
            if (it.n_tiles > 0 && !(ok = mbar_wait(pvdone_bar((s_cnt - 1) & 1), ((s_cnt - 1) >> 1) & 1, &abort_sh, a.status))) break;
            tc_fence_after();
            float o[RG];
            if (it.n_tiles > 0) {
                load_rows<NR, RG>(tlane + TM_O, row0, o);
            } else {
#pragma unroll
                for (int r = 0; r < RG; ++r) o[r] = 0.f;
            }
            const bool single = it.n_split == 1;
            // O^T and every thread's share of the row sums go through shared memory (the P^T buffers are idle: the item's
            // last MMA has read them) as [row][dim] and [row][key lane], and whole warps finish the rows in a rolled loop.
            // Unrolled over 32 rows, the sums and the stores were kilobytes of code run once per item: fetched cold, with
            // HBM saturated, they took 25 us.
            float *osm = reinterpret_cast<float *>(gen + 2 * QCH), *lsm = osm + NR * HD;
#pragma unroll
            for (int r = 0; r < RG; ++r) { osm[(row0 + r) * HD + kl] = o[r]; lsm[(row0 + r) * HD + kl] = l_run[r]; }
            if (!(ok = wg_sync())) break;
            const int rows_out = QR;
#pragma unroll 1
            for (int r = sw; r < rows_out; r += SW) {
                const float *lr = lsm + r * HD + lane;
                const float l = warp_sum((lr[0] + lr[32]) + (lr[64] + lr[96]));
                const float4 v = *reinterpret_cast<const float4 *>(osm + r * HD + lane * 4);
                const int hq = r / a.M, h = it.g * grp + hq, node = r - hq * a.M;
                if (single) {
                    const float x0 = v.x / l, x1 = v.y / l, x2 = v.z / l, x3 = v.w / l;
                    const __nv_bfloat162 h01 = __floats2bfloat162_rn(x0, x1), h23 = __floats2bfloat162_rn(x2, x3);
                    const __nv_bfloat162 l01 = __floats2bfloat162_rn(x0 - __low2float(h01), x1 - __high2float(h01));
                    const __nv_bfloat162 l23 = __floats2bfloat162_rn(x2 - __low2float(h23), x3 - __high2float(h23));
                    __nv_bfloat16 *dst = a.out + ((size_t)(it.be * a.M + node) * a.H + h) * HD + lane * 4;
                    {
                        *reinterpret_cast<uint2 *>(dst) = make_uint2(*reinterpret_cast<const uint32_t *>(&h01), *reinterpret_cast<const uint32_t *>(&h23));
                        if (a.out_plane)
                            *reinterpret_cast<uint2 *>(dst + a.out_plane) =
                                make_uint2(*reinterpret_cast<const uint32_t *>(&l01), *reinterpret_cast<const uint32_t *>(&l23));
                    }
                } else {
                    float *pdst = a.part + ((((size_t)it.be * a.H + h) * a.M + node) * a.part_slots + it.split) * ROWF;
                    *reinterpret_cast<float2 *>(pdst + lane * 4) = make_float2(v.x, v.y);       // rows are 8-byte aligned (HD + 2 floats)
                    *reinterpret_cast<float2 *>(pdst + lane * 4 + 2) = make_float2(v.z, v.w);
                    if (lane == 0) { pdst[HD] = mraw_sh[r] * 0.6931471805599453f; pdst[HD + 1] = l; }   // natural-log units
                }
            }
            if (it.n_tiles > 0) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(ofree_bar);                 // the next item may overwrite O^T
            }
            if (!single && a.fuse_merge) {
                // last key range of this (sequence, kv head) to finish merges all of them, in range order
                // (one acquire-release atomic after the barrier instead of a fence per thread on both sides)
                if (!(ok = wg_sync())) break;
                if (et == 0) {
                    int old;
                    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(a.counters + it.be * HkvV + it.g) : "memory");
                    last_sh = old == it.n_split - 1;
                    if (last_sh) a.counters[it.be * HkvV + it.g] = 0;
                }
                if (!(ok = wg_sync())) break;
                if (last_sh) {
                    // Four rows per warp at a time, every load of a round (the ranges' maxima and sums, four ranges'
                    // vectors) issued before the first use: a row at a time is a trip to L2 per row, one after the other.
                    constexpr int MB = 4;
#pragma unroll 1
                    for (int rb = sw; rb < QR; rb += MB * SW) {
                        const float *psrc[MB];
                        size_t odst[MB];
                        float ms[MB], ls[MB], w[MB], den[MB], num[MB][HD / 32];
#pragma unroll
                        for (int j = 0; j < MB; ++j) {
                            const int r = min(rb + j * SW, QR - 1);               // rows past the end repeat the last one, unstored
                            const int hh = it.g * grp + r / a.M, i = r % a.M;
                            psrc[j] = a.part + (((size_t)it.be * a.H + hh) * a.M + i) * (size_t)a.part_slots * ROWF;
                            odst[j] = ((size_t)(it.be * a.M + i) * a.H + hh) * HD;
                            // lane s holds range s's (max, sum); the weights go round by shuffle (at most 32 ranges when fused)
                            ms[j] = -INFINITY; ls[j] = 0.f;
                            if (lane < it.n_split) { ms[j] = __ldcg(psrc[j] + (size_t)lane * ROWF + HD); ls[j] = __ldcg(psrc[j] + (size_t)lane * ROWF + HD + 1); }
#pragma unroll
                            for (int e = 0; e < HD / 32; ++e) num[j][e] = 0.f;
                        }
                        for (int s0 = 0; s0 < it.n_split; s0 += 4) {
                            float v[MB][4][HD / 32];
#pragma unroll
                            for (int j = 0; j < MB; ++j)
#pragma unroll
                                for (int q = 0; q < 4; ++q)
#pragma unroll
                                    for (int e = 0; e < HD / 32; ++e)
                                        v[j][q][e] = s0 + q < it.n_split ? __ldcg(psrc[j] + (size_t)(s0 + q) * ROWF + lane + 32 * e) : 0.f;
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
                                    for (int e = 0; e < HD / 32; ++e) num[j][e] = fmaf(v[j][q][e], s0 + q < it.n_split ? wq : 0.f, num[j][e]);
                                }
                        }
#pragma unroll
                        for (int j = 0; j < MB; ++j) {
                            if (rb + j * SW >= QR) continue;
                            const float invd = 1.f / den[j];
#pragma unroll
                            for (int e = 0; e < HD / 32; ++e)
                                store_act<__nv_bfloat16>(a.out, a.out_plane, odst[j] + lane + 32 * e, num[j][e] * invd);
                        }
                    }
                }
                if (!(ok = wg_sync())) break;                          // last_sh and the staged rows are reused by the next item
            } else {
                if (!(ok = wg_sync())) break;                          // the staged rows are overwritten by the next item's P^T
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
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256) : "memory");
    }
}

}  // namespace

// Query heads of a kv head that one item takes: as many as fit 32 rows (a divisor of the group, at most 4 items per
// kv head: the arrival counters have four slots per (sequence, kv head)).  0: the kernel does not take this shape.
int attention_tk_heads_per_item(int group_heads, int M) {
    if (M > 32 || M < 1) return 0;
    for (int hpi = group_heads; hpi >= 1; --hpi)
        if (group_heads % hpi == 0 && hpi * M <= 32) return group_heads / hpi <= VIASD_ATTN_ITEMS_PER_KV_HEAD ? hpi : 0;
    return 0;
}
int attention_tk_supported(int group_heads, int M) { return attention_tk_heads_per_item(group_heads, M) > 0; }

// tensor maps over the caches are rebuilt only when the caller's pointers change
static int cache_maps_tk(viasd_model *m, CacheMaps &cm, const void *kc, const void *vc, int n_layers) {
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
int launch_attention_tk(viasd_model *m, const void *kc, const void *vc, bool slim, int layer_ord, const void *kc2,
                        const void *vc2, int layer_ord2, int streams, int batch, int M, int nsplit, int fuse_merge,
                        cudaStream_t st) {
    const viasd_config &c = m->cfg;
    CacheMaps &cm = slim ? m->cmaps_slim : m->cmaps_full;
    int rc;
    if ((rc = cache_maps_tk(m, cm, kc, vc, slim ? m->n_routed : c.n_layers))) return rc;
    CacheMaps *cm2 = &cm;
    if (streams == 2) {
        cm2 = &m->cmaps_slim;
        if ((rc = cache_maps_tk(m, *cm2, kc2, vc2, m->n_routed))) return rc;
    }
    const int grp = c.n_heads / c.n_kv_heads, hpi = attention_tk_heads_per_item(grp, M);
    if (hpi == 0) return VIASD_EINVAL;
    const int QR = hpi * M, subs = grp / hpi;                      // rows per item; items per kv head
    const int nr = QR <= 8 ? 8 : QR <= 16 ? 16 : 32;
    AttnTkArgs a;
    a.q = m->ws.q; a.part = m->ws.part; a.out = (__nv_bfloat16 *)m->ws.attn;
    a.out_plane = m->ws.rows_alloc * (size_t)c.n_heads * HD;
    a.len_eff = m->ws.len_eff; a.tree = m->ws.tree; a.status = &m->ws.stats->device_status; a.run_flag = m->run_flag;
    a.M = M; a.H = c.n_heads; a.Hkv = c.n_kv_heads; a.subs = subs; a.max_batch = c.max_batch; a.max_ctx = c.max_ctx;
    a.layer_ord = layer_ord; a.nsplit = nsplit; a.scale = 1.4426950408889634f / sqrtf((float)HD);   // log2(e) / sqrt(hd)
    a.batch = batch; a.layer_ord2 = layer_ord2; a.streams = streams;
    a.counters = m->ws.attn_counters;
    a.fuse_merge = fuse_merge;
    int grid;
    if (nsplit <= 0) {
        // tiles dealt evenly: one range per CTA and row stream, cut by the kernel from the lengths; merges are fused
        a.flat = 1; a.part_slots = 16; a.nsplit = 1; a.fuse_merge = 1; a.n_items = 0; a.items_per_cta = 0;
        grid = m->sm_count;
        if (m->opt.tk_grid >= 1 && m->opt.tk_grid < grid) grid = m->opt.tk_grid;     // tests: long ranges per CTA on small cases
    } else {
        a.flat = 0; a.part_slots = nsplit;
        a.n_items = streams * batch * c.n_kv_heads * subs * nsplit;
        grid = a.n_items < m->sm_count ? a.n_items : m->sm_count;
        a.items_per_cta = (a.n_items + grid - 1) / grid;
        grid = (a.n_items + a.items_per_cta - 1) / a.items_per_cta;
    }
    const size_t op_bytes = 6 * (size_t)(2 * nr) * 128;            // Q (2 chunks) and two P^T buffers (2 chunks each)
    // 32 query rows: the softmax of a tile is long, so K tiles get slots of their own, released by S^T = K Q^T, and the
    // tile after next is on its way meanwhile.  With fewer rows this measured slower than a slot per (K, V) pair.
    const size_t smem_max = 222 * 1024;
    size_t smem;
    if (nr == 32) {
        int slots = (int)((smem_max - 1024 - op_bytes) / SLOT_BYTES);
        if (slots > 2 * TK_MAX_STAGE) slots = 2 * TK_MAX_STAGE;
        a.nk = (slots + 1) / 2; a.nv = slots / 2;
        smem = 1024 + op_bytes + (size_t)slots * SLOT_BYTES;
    } else {
        a.nk = a.nv = 1024 + op_bytes + 3 * (size_t)(2 * SLOT_BYTES) <= 220 * 1024 ? 3 : 2;
        smem = 1024 + op_bytes + a.nk * (size_t)(2 * SLOT_BYTES);
    }
    static bool attr_done[64];
    if (first_use_on_device(attr_done)) {
        CUDA_TRY(cudaFuncSetAttribute(attention_tk_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 222 * 1024));
        CUDA_TRY(cudaFuncSetAttribute(attention_tk_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 222 * 1024));
        CUDA_TRY(cudaFuncSetAttribute(attention_tk_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, 222 * 1024));
    }
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    pdl_config(cfg, attr, dim3(grid), dim3(nr == 32 ? TK_THREADS + 128 : TK_THREADS), smem, st);
    if (nr == 8) CUDA_TRY(cudaLaunchKernelEx(&cfg, attention_tk_kernel<8>, cm.k, cm.v, cm2->k, cm2->v, a));
    else if (nr == 16) CUDA_TRY(cudaLaunchKernelEx(&cfg, attention_tk_kernel<16>, cm.k, cm.v, cm2->k, cm2->v, a));
    else CUDA_TRY(cudaLaunchKernelEx(&cfg, attention_tk_kernel<32>, cm.k, cm.v, cm2->k, cm2->v, a));
    LAUNCH_CHECK();
    return VIASD_OK;
}

