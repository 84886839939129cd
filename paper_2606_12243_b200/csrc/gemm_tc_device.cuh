// Device-side pieces of the tcgen05 GEMM kernel: tile constants, the unit-range walk of the stream-K
// schedule and the fused epilogues.
#pragma once
#include "common.cuh"
#include "gemm_tc.cuh"
#include "tc_ptx.cuh"

namespace {

constexpr int TILE_F = 128;          // output features per tile (MMA M)
constexpr int TILE_K = 64;           // bf16 per k-block: 128 bytes, one swizzle row
constexpr int MAX_STAGES = 12;

constexpr int CH = 8;                // token rows per epilogue chunk
__device__ __forceinline__ void tc_ld8(uint32_t taddr, float (&v)[CH]) {
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}

// two groups of columns with one wait (hi and lo columns of a chunk): the second load does not wait for the first
__device__ __forceinline__ void tc_ld8x2(uint32_t ta, uint32_t tb, float (&a)[CH], float (&b)[CH]) {
    uint32_t r[8], q[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(ta));
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(q[0]), "=r"(q[1]), "=r"(q[2]), "=r"(q[3]), "=r"(q[4]), "=r"(q[5]), "=r"(q[6]), "=r"(q[7])
                 : "r"(tb));
    // the wait names the registers: no use of them may be scheduled ahead of it
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                   "+r"(q[0]), "+r"(q[1]), "+r"(q[2]), "+r"(q[3]), "+r"(q[4]), "+r"(q[5]), "+r"(q[6]), "+r"(q[7])
                 :: "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) { a[i] = __uint_as_float(r[i]); b[i] = __uint_as_float(q[i]); }
}

struct Seg { int tile, ka, kb; };      // one contiguous piece of this CTA's unit range inside a tile

__device__ __forceinline__ bool next_seg(int &u, int u1, int k_tiles, Seg &s) {
    if (u >= u1) return false;
    s.tile = u / k_tiles;
    s.ka = u - s.tile * k_tiles;
    s.kb = min(k_tiles, s.ka + (u1 - u));
    u += s.kb - s.ka;
    return true;
}

// Epilogue for CH token rows r0..r0+CH-1 of one tile; thread f holds the full-K sums g (and u for the gate/up
// pair) of output feature f.  Called by all 128 epilogue threads together.  The epilogue kind is a template
// parameter so that each kernel carries one short epilogue: this code runs once per tile, straight from the
// instruction cache's cold side, and its size is what its latency is made of.
template <int EPI, int GROUPS>
__device__ __forceinline__ void finish_chunk(const TcParams &p, int tile, int f, int r0, float (&g)[CH], float (&uu)[CH],
                                             float *xch, const float *inv_sh, const int4 *rowmeta, int lane,
                                             const float *aux, int rows_live, bool have_gain, float2 gain, int group_bar) {
    // aux: null, or [rows][128] floats already in shared memory - the residual row of this tile (EPI_ADD_NORM),
    // or the row's 64 cosines followed by its 64 sines (EPI_QKV_ROPE) - so that no chunk waits for global memory.
    // rows_live: rows r0.. below it are written (p.rows, or 0 for the dry pass that only warms the instruction cache)
    // have_gain / gain: the next norm's gains of feature f, fetched by the caller long before (EPI_ADD_NORM)
    // group_bar: the named barrier of the calling group of 128 threads; xch is that group's exchange buffer
    constexpr bool DUAL = EPI == EPI_SWIGLU;
    if (EPI == EPI_STORE || EPI == EPI_SWIGLU || EPI == EPI_QKV_ROPE) {
        if (p.ssq_in) {                   // the input was h * gain without its RMS factor: apply it per row here
#pragma unroll
            for (int j = 0; j < CH; ++j) {
                const float sc = inv_sh[min(r0 + j, 127)];
                g[j] *= sc;
                if (DUAL) uu[j] *= sc;
            }
        }
    }
    const int nrow = min(CH, rows_live - r0);
    // dry pass: nothing is stored, but the lines (and pages) the real pass will write are asked for, so that its
    // first stores do not start with address-translation misses
    const bool touch = rows_live == 0 && (f & 31) == 0;
    auto want = [](const void *ptr) { asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr)); };
    if (DUAL) {
        const int n = tile * TILE_F + f;
        if (n >= p.seg_n[0]) return;
        __nv_bfloat16 *dst = p.out_act + (size_t)(p.row0 + r0) * p.ld_out + n;
        if (touch) { want(dst); want(dst + p.act_plane); }
#pragma unroll
        for (int j = 0; j < CH; ++j) {
            if (j < nrow) {
                const float sg = g[j] / (1.f + __expf(-g[j]));
                store_act<__nv_bfloat16>(dst, p.act_plane, (size_t)j * p.ld_out, sg * uu[j]);
            }
        }
        return;
    }
    int s = 0, t0 = 0, nbase = 0;
    while (s < 2 && tile >= p.seg_tile_end[s]) { t0 = p.seg_tile_end[s]; nbase += p.seg_n[s]; ++s; }
    const int nin = (tile - t0) * TILE_F + f;
    const bool valid = nin < p.seg_n[s];
    const int n = nbase + nin;
    if (EPI == EPI_STORE) {
        if (!valid) return;
        if (touch) want(p.out_f32 + (size_t)(p.row0 + r0) * p.ld_out + n);
#pragma unroll
        for (int j = 0; j < CH; ++j) {
            if (j < nrow) {
                const int row = p.row0 + r0 + j;          // the second stream's rows go to the second output
                float *dst = row < p.split_row ? p.out_f32 + (size_t)row * p.ld_out + n
                                               : p.out_f32_2 + (size_t)(row - p.split_row) * p.ld_out + n;
                if (p.epi == EPI_ADD) *dst += g[j]; else *dst = g[j];
            }
        }
    } else if (EPI == EPI_ADD_NORM) {
        // residual update, plus what the next RMSNorm needs: h * gain as hi/lo planes and partial sums of h^2.
        // Loads first, then arithmetic, then stores: the CH rows cost one memory round trip.
        // fetched here, the two gains are a round trip to L2 at the head of every chunk (the stores in between keep
        // the compiler from hoisting them): a microsecond on the launch's critical path
        const float gain_a = have_gain ? gain.x : (valid ? p.next_gain[n] : 0.f);
        const float gain_b = have_gain ? gain.y : ((valid && p.next_gain2) ? p.next_gain2[n] : gain_a);
        float *hp = p.out_f32 + (size_t)(p.row0 + r0) * p.ld_out + n;
        __nv_bfloat16 *ap = p.next_act + (size_t)(p.row0 + r0) * p.ld_out + n;
        if (touch) { want(hp); want(ap); want(ap + p.next_plane); want(p.ssq_out + ((size_t)tile * 4 + (f >> 5)) * p.ssq_stride + p.row0 + r0); }
        float v[CH];
        if (aux) {                                               // the residual rows are staged in shared memory
#pragma unroll
            for (int j = 0; j < CH; ++j) v[j] = (valid && j < nrow) ? aux[(r0 + j) * TILE_F + f] + g[j] : 0.f;
        } else {
#pragma unroll
            for (int j = 0; j < CH; ++j) v[j] = (valid && j < nrow) ? __ldcg(hp + (size_t)j * p.ld_out) + g[j] : 0.f;
        }
#pragma unroll
        for (int j = 0; j < CH; ++j) {
            if (valid && j < nrow) {
                hp[(size_t)j * p.ld_out] = v[j];
                store_act<__nv_bfloat16>(ap, p.next_plane, (size_t)j * p.ld_out,
                                         v[j] * (p.row0 + r0 + j < p.split_row ? gain_a : gain_b));
            }
            v[j] *= v[j];
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
#pragma unroll
            for (int j = 0; j < CH; ++j) v[j] += __shfl_xor_sync(0xffffffffu, v[j], o);
        if (lane < nrow) {
            float mine = v[0];
#pragma unroll
            for (int j = 1; j < CH; ++j) mine = lane == j ? v[j] : mine;
            p.ssq_out[((size_t)tile * 4 + (f >> 5)) * p.ssq_stride + p.row0 + r0 + lane] = mine;
        }
    } else {   // EPI_QKV_ROPE: one tile is one head of 128 dims; rotate pairs (p, p + 64), write q / K cache / V cache
#pragma unroll
        for (int j = 0; j < CH; ++j) xch[j * TILE_F + f] = g[j];
        if (GROUPS == 1) asm volatile("bar.sync 1, 128;" ::: "memory"); else asm volatile("bar.sync %0, 128;" ::"r"(group_bar) : "memory");
        const int head = tile - t0, pidx = f & 63;
        if (s < 2) {
            float c[CH], sn[CH];
            if (aux) {                                           // the rows' tables are staged in shared memory
#pragma unroll
                for (int j = 0; j < CH; ++j) {
                    const float *ar = aux + min(r0 + j, p.rows - 1) * TILE_F + pidx;
                    c[j] = ar[0];
                    sn[j] = ar[64];
                }
            } else {
#pragma unroll
                for (int j = 0; j < CH; ++j) {
                    const int pos = rowmeta[min(r0 + j, 127)].x;
                    c[j] = p.cosv[(size_t)pos * 64 + pidx];
                    sn[j] = p.sinv[(size_t)pos * 64 + pidx];
                }
            }
#pragma unroll
            for (int j = 0; j < CH; ++j) {
                const float other = xch[j * TILE_F + (f ^ 64)];
                g[j] = f < 64 ? g[j] * c[j] - other * sn[j] : g[j] * c[j] + other * sn[j];
            }
        }
        if (touch) {
            if (s == 0) want(p.q_out + ((size_t)(p.row0 + r0) * p.rope_H + head) * TILE_F + f);
            else want((s == 1 ? p.kc : p.vc) + ((((size_t)p.layer_ord * p.max_batch) * p.rope_Hkv + head) * p.max_ctx) * TILE_F + f);
        }
        if (s == 0) {
            float *dst = p.q_out + ((size_t)(p.row0 + r0) * p.rope_H + head) * TILE_F + f;
#pragma unroll
            for (int j = 0; j < CH; ++j) if (j < nrow) dst[(size_t)j * p.rope_H * TILE_F] = g[j];
        } else {
            __nv_bfloat16 *c0 = s == 1 ? p.kc : p.vc, *c1 = s == 1 ? p.kc2 : p.vc2;
            const size_t head_off = (size_t)head * p.max_ctx * TILE_F + f;
#pragma unroll
            for (int j = 0; j < CH; ++j) {
                const int4 rm = rowmeta[min(r0 + j, 127)];          // .z / .w: the row's offset in its cache (set with the table)
                if (j < nrow && rm.y >= 0) {
                    const size_t off = ((size_t)((unsigned)rm.w & 0x3fffffffu) << 32) | (unsigned)rm.z;
                    (((unsigned)rm.w >> 30) & 1u ? c1 : c0)[off + head_off] = __float2bfloat16_rn(g[j]);
                }
            }
        }
        if (GROUPS == 1) asm volatile("bar.sync 1, 128;" ::: "memory"); else asm volatile("bar.sync %0, 128;" ::"r"(group_bar) : "memory");
    }
}

}  // namespace
