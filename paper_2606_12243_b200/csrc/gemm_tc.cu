// Weight-streaming bf16 GEMM on the 5th-generation tensor cores (tcgen05 + TMEM), fed by TMA.
//
//   y[rows, n] = x[rows, k] * W[n, k]^T        rows <= 128 per launch, W streamed once from HBM
//
// The operands are swapped: a tile of 128 output features is the MMA's M dimension (A operand, the
// weights), the token rows are its N dimension (B operand, 16..128 wide).  Both are K-major in shared
// memory with the 128-byte swizzle, exactly as a 2-D TMA box of 64 bf16 x rows lands there.  The
// activation comes as two bf16 planes hi + lo (x = hi + lo to ~16 mantissa bits); each weight tile is
// multiplied with both, which costs tensor time the kernel has in abundance and no extra weight traffic.
//
// Persistent stream-K schedule: the (tile, k-block) units of the whole GEMM are cut into one contiguous
// range per CTA, so every SM streams the same number of bytes whatever the shape.  A CTA that holds all
// k-blocks of a tile finishes it from TMEM; otherwise it writes an fp32 partial and the last CTA to
// arrive at the tile (an atomic counter, no waiting) sums the partials in CTA order - bit-reproducible.
//
// Warp roles (192 threads): warp 0 issues TMA loads into a ring of stages, warp 1 allocates TMEM and
// issues tcgen05.mma, warps 2-5 read the accumulators (tcgen05.ld) and run the epilogue.  Accumulators
// are double-buffered in TMEM so the epilogue of one tile overlaps the main loop of the next.
// Every wait is bounded: on expiry the CTA records VIASD_EDEVICE, lets its copies land and leaves.
#include "common.cuh"
#include "gemm_tc.cuh"
#include <stdlib.h>

namespace {

constexpr int TILE_F = 128;          // output features per tile (MMA M)
constexpr int TILE_K = 64;           // bf16 per k-block: 128 bytes, one swizzle row
constexpr int MAX_STAGES = 12;
constexpr int THREADS = 192;
constexpr long long WAIT_LIMIT_CYCLES = 4000000000ll;   // about two seconds

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the limit expired or another role of this CTA already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    int spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 255) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
                *abort_flag = 1;
                atomicExch(status, VIASD_EDEVICE);
                return false;
            }
        }
    }
    return true;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
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

// K-major operand tile, 128-byte swizzle, rows 128 bytes apart, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
    return (uint64_t)((addr >> 4) & 0x3FFF) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

#ifdef VIASD_TC_TRACE
__device__ long long g_tc_trace[160 * 8];
#define TRACE(slot) do { if (p.trace_on) g_tc_trace[blockIdx.x * 8 + (slot)] = clock64(); } while (0)
#define DBG(p, bit) ((p).dbg & (bit))
__device__ unsigned long long g_tc_span[8192 * 2];       // per launch: earliest CTA start, latest CTA end (globaltimer ns)
__device__ __forceinline__ unsigned long long gtimer() { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
#define SPAN_BEGIN(p) do { if (threadIdx.x == 0) atomicMin(&g_tc_span[((p).launch_idx & 8191) * 2], gtimer()); } while (0)
#define SPAN_END(p) do { if (threadIdx.x == 0) atomicMax(&g_tc_span[((p).launch_idx & 8191) * 2 + 1], gtimer()); } while (0)
#else
#define SPAN_BEGIN(p) do { } while (0)
#define SPAN_END(p) do { } while (0)
#define DBG(p, bit) 0
#define TRACE(slot) do { } while (0)
#endif

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
template <int EPI>
__device__ __forceinline__ void finish_chunk(const TcParams &p, int tile, int f, int r0, float (&g)[CH], float (&uu)[CH],
                                             float *xch, const float *inv_sh, const int4 *rowmeta, int lane) {
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
    const int nrow = min(CH, p.rows - r0);
    if (DUAL) {
        const int n = tile * TILE_F + f;
        if (n >= p.seg_n[0]) return;
        __nv_bfloat16 *dst = p.out_act + (size_t)(p.row0 + r0) * p.ld_out + n;
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
        const float gain_a = valid ? p.next_gain[n] : 0.f;
        const float gain_b = (valid && p.next_gain2) ? p.next_gain2[n] : gain_a;
        float *hp = p.out_f32 + (size_t)(p.row0 + r0) * p.ld_out + n;
        __nv_bfloat16 *ap = p.next_act + (size_t)(p.row0 + r0) * p.ld_out + n;
        float v[CH];
#pragma unroll
        for (int j = 0; j < CH; ++j) v[j] = (valid && j < nrow) ? __ldcg(hp + (size_t)j * p.ld_out) + g[j] : 0.f;
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
        asm volatile("bar.sync 1, 128;" ::: "memory");
        const int head = tile - t0, pidx = f & 63;
        if (s < 2) {
            float c[CH], sn[CH];
#pragma unroll
            for (int j = 0; j < CH; ++j) {
                const int pos = rowmeta[min(r0 + j, 127)].x;
                c[j] = p.cosv[(size_t)pos * 64 + pidx];
                sn[j] = p.sinv[(size_t)pos * 64 + pidx];
            }
#pragma unroll
            for (int j = 0; j < CH; ++j) {
                const float other = xch[j * TILE_F + (f ^ 64)];
                g[j] = f < 64 ? g[j] * c[j] - other * sn[j] : g[j] * c[j] + other * sn[j];
            }
        }
        if (s == 0) {
            float *dst = p.q_out + ((size_t)(p.row0 + r0) * p.rope_H + head) * TILE_F + f;
#pragma unroll
            for (int j = 0; j < CH; ++j) if (j < nrow) dst[(size_t)j * p.rope_H * TILE_F] = g[j];
        } else {
#pragma unroll
            for (int j = 0; j < CH; ++j) {
                if (j < nrow) {
                    const int4 rm = rowmeta[r0 + j];
                    __nv_bfloat16 *cache = rm.w ? (s == 1 ? p.kc2 : p.vc2) : (s == 1 ? p.kc : p.vc);
                    const int lo = rm.w ? p.layer_ord2 : p.layer_ord;
                    cache[((((size_t)lo * p.max_batch + rm.z) * p.rope_Hkv + head) * p.max_ctx + rm.y) * TILE_F + f] =
                        __float2bfloat16_rn(g[j]);
                }
            }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
    }
}

template <int EPI>
__global__ void __launch_bounds__(THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_w0, const __grid_constant__ CUtensorMap map_w1,
               const __grid_constant__ CUtensorMap map_w2, const __grid_constant__ CUtensorMap map_x, const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) unsigned long long bars[2 * MAX_STAGES + 4];
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh, last_sh;
    __shared__ float inv_sh[128];                       // per-row 1/rms of the input (fused RMSNorm)
    __shared__ float xch[CH * TILE_F];                  // rotary partner exchange
    __shared__ int4 rowmeta[128];                       // per token row: rotary position, cache slot, sequence

    constexpr bool DUAL = EPI == EPI_SWIGLU;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel may start its prologue
    if (threadIdx.x == 0) TRACE(0);
    SPAN_BEGIN(p);
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int NT = p.nt, S = p.stages;
    constexpr int NACC = DUAL ? 2 : 1;
    const uint32_t a_bytes = TILE_F * TILE_K * 2, b_bytes = (uint32_t)NT * TILE_K * 2;
    const uint32_t stage_bytes = NACC * a_bytes + 2 * b_bytes;
    auto full_bar = [&](int s) { return smem_u32(&bars[s]); };
    auto empty_bar = [&](int s) { return smem_u32(&bars[MAX_STAGES + s]); };
    auto tfull_bar = [&](int b) { return smem_u32(&bars[2 * MAX_STAGES + b]); };
    auto tempty_bar = [&](int b) { return smem_u32(&bars[2 * MAX_STAGES + 2 + b]); };
    const int NB = p.has_lo ? 2 * NT : NT;                  // MMA N: hi and lo token columns side by side
    const uint32_t acc_cols = NACC * NB;                    // TMEM columns per accumulator buffer

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 4); }
        abort_sh = 0;
        last_sh = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_sh)),
                     "r"(p.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_sh;
    if (threadIdx.x == 0) TRACE(1);

    const int total_units = p.n_tiles * p.k_tiles;
    const int u_begin = blockIdx.x * p.units_per_cta;
    const int u_end = min(total_units, u_begin + p.units_per_cta);

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            const int n_it = u_end - u_begin;
            // unit -> weight matrix, its first row, k-block
            auto unit = [&](int it, const CUtensorMap *&mw, int &wrow, int &kt, int &sidx) {
                const int u = u_begin + it, tile = u / p.k_tiles;
                kt = u - tile * p.k_tiles;
                int s = 0, t0 = 0;
                if (!DUAL) while (s < 2 && tile >= p.seg_tile_end[s]) { t0 = p.seg_tile_end[s]; ++s; }
                mw = s == 0 ? &map_w0 : (s == 1 ? &map_w1 : &map_w2);
                wrow = (tile - t0) * TILE_F;
                sidx = s;
            };
            auto load_w = [&](int st, const CUtensorMap *mw, int wrow, int kt) {
                const uint32_t base = smem_base + st * stage_bytes;
                tma_load_2d(base, mw, full_bar(st), kt * TILE_K, wrow);
                if (DUAL) tma_load_2d(base + a_bytes, &map_w1, full_bar(st), kt * TILE_K, wrow);
            };
            auto load_x = [&](int st, int kt) {
                const uint32_t base = smem_base + st * stage_bytes + NACC * a_bytes;
                tma_load_2d(base, &map_x, full_bar(st), kt * TILE_K, p.row0);
                tma_load_2d(base + b_bytes, &map_x, full_bar(st), kt * TILE_K, p.row0 + p.lo_row_offset);
            };
            const CUtensorMap *mw; int wrow, kt, sidx;
            // Weights do not depend on the kernel before this one: fill the ring with them first, and only then
            // wait for that kernel (programmatic dependent launch) before touching the activations.
            const int pre = n_it < S ? n_it : S;
            for (int it = 0; it < pre; ++it) {
                unit(it, mw, wrow, kt, sidx);
                asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(full_bar(it)),
                             "r"(DUAL ? 2 * p.a_tx[0] : p.a_tx[sidx]) : "memory");
                load_w(it, mw, wrow, kt);
            }
            asm volatile("griddepcontrol.wait;" ::: "memory");
            for (int it = 0; it < pre; ++it) {
                unit(it, mw, wrow, kt, sidx);
                mbar_expect_tx(full_bar(it), 2 * p.b_tx);
                load_x(it, kt);
            }
            for (int it = pre; it < n_it; ++it) {
                const int st = it % S;
                if (!mbar_wait(empty_bar(st), ((it / S) & 1) ^ 1, &abort_sh, p.status)) break;
                unit(it, mw, wrow, kt, sidx);
                mbar_expect_tx(full_bar(st), (DUAL ? 2 * p.a_tx[0] : p.a_tx[sidx]) + 2 * p.b_tx);
                load_w(st, mw, wrow, kt);
                load_x(st, kt);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NB >> 3) << 17) | ((TILE_F >> 4) << 24);
            int it = 0, acc_it = 0, u = u_begin;
            Seg sg;
            bool ok = true;
            while (ok && next_seg(u, u_end, p.k_tiles, sg)) {
                const int buf = acc_it % p.acc_bufs;
                if (!(ok = mbar_wait(tempty_bar(buf), ((acc_it / p.acc_bufs) & 1) ^ 1, &abort_sh, p.status))) break;
                tc_fence_after();
                const uint32_t d0 = tmem_base + buf * acc_cols;
                for (int kt = sg.ka; kt < sg.kb; ++kt, ++it) {
                    const int st = it % S;
                    if (!(ok = mbar_wait(full_bar(st), (it / S) & 1, &abort_sh, p.status))) break;
                    tc_fence_after();
                    const uint32_t base = smem_base + st * stage_bytes;
                    // the hi tile is followed by the lo tile: together one K-major operand of NB rows
                    const uint32_t bh = base + NACC * a_bytes;
#pragma unroll
                    for (int k = 0; k < TILE_K / 16; ++k) {
                        const uint32_t acc = (kt > sg.ka || k > 0) ? 1u : 0u;
                        tc_mma(d0, smem_desc(base + k * 32), smem_desc(bh + k * 32), idesc, acc);
                        if (DUAL) tc_mma(d0 + NB, smem_desc(base + a_bytes + k * 32), smem_desc(bh + k * 32), idesc, acc);
                    }
                    tc_commit(empty_bar(st));              // the stage is free once these MMAs have read it
                }
                if (ok) tc_commit(tfull_bar(buf));          // accumulator complete
                ++acc_it;
            }
            TRACE(3);
        }
    } else {
        // ---------------- epilogue (warps 2..5 <-> TMEM lane quarters 2,3,0,1) ----------------
        asm volatile("griddepcontrol.wait;" ::: "memory");     // outputs, scratch and counters belong to the chain
        const int quarter = warp & 3;
        const int f = quarter * 32 + lane;                  // feature lane inside the tile
        const int et = threadIdx.x - 64;                    // 0..127 among epilogue threads
        const size_t slot_floats = (size_t)NACC * NT * TILE_F;
        // per-row tables (all 128 entries defined: chunks read a few rows past p.rows and discard them)
        inv_sh[et] = 0.f;
        rowmeta[et] = make_int4(0, 0, 0, 0);
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (p.ssq_in) {
            // 1/rms per input row: a warp sums the row's partial sums of squares (fixed order: reproducible)
            for (int r = (et >> 5); r < p.rows; r += 4) {
                float ss = 0.f;
                for (int j = lane; j < p.ssq_in_n; j += 32) ss += __ldcg(p.ssq_in + (size_t)j * p.ssq_stride + p.row0 + r);
                ss = warp_sum(ss);
                if (lane == 0) inv_sh[r] = rsqrtf(ss * p.inv_d + p.eps);
            }
        }
        if (EPI == EPI_QKV_ROPE) {
            if (et < p.rows) {
                // rows are laid out [stream][sequence][block row]; stream 1 (rows >= split_row) is the slim verifier
                const int row = p.row0 + et, stream = row >= p.split_row ? 1 : 0, rs = row - stream * p.split_row;
                const int b = rs / p.rope_M, i = rs - b * p.rope_M;
                const int n_ctx = p.len_eff[b];
                rowmeta[et] = make_int4(n_ctx + p.depth[i], n_ctx + i, b, stream);
            }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        int acc_it = 0, u = u_begin, seg_i = 0;
        Seg sg;
        bool ok = true;
        while (ok && next_seg(u, u_end, p.k_tiles, sg)) {
            const int buf = acc_it % p.acc_bufs;
            if (!(ok = mbar_wait(tfull_bar(buf), (acc_it / p.acc_bufs) & 1, &abort_sh, p.status))) break;
            tc_fence_after();
            const bool whole = sg.ka == 0 && sg.kb == p.k_tiles;
            const uint32_t t0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * acc_cols;
            // partial of a split tile: slot 0 if the tile is the first one this CTA touches, else slot 1
            float *slot = p.scratch + ((size_t)blockIdx.x * 2 + (seg_i == 0 ? 0 : 1)) * slot_floats;
            for (int c = 0; c < p.rows; c += CH) {           // padding rows beyond p.rows are never read
                float g[CH], uu[CH];
                tc_ld8(t0 + c, g);
                if (DUAL) tc_ld8(t0 + NB + c, uu);
                if (p.has_lo) {                              // add the product with the lo plane
                    float lo[CH];
                    tc_ld8(t0 + NT + c, lo);
#pragma unroll
                    for (int j = 0; j < CH; ++j) g[j] += lo[j];
                    if (DUAL) {
                        tc_ld8(t0 + NB + NT + c, lo);
#pragma unroll
                        for (int j = 0; j < CH; ++j) uu[j] += lo[j];
                    }
                }
                if (whole) {
                    finish_chunk<EPI>(p, sg.tile, f, c, g, uu, xch, inv_sh, rowmeta, lane);
                } else {
#pragma unroll
                    for (int j = 0; j < CH; ++j) {
                        slot[(size_t)(c + j) * TILE_F + f] = g[j];
                        if (DUAL) slot[(size_t)(NT + c + j) * TILE_F + f] = uu[j];
                    }
                }
            }
            if (et == 0) TRACE(2);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(buf));   // accumulator buffer may be overwritten
            if (!whole) {
                // publish the partial; the last contributor of the tile sums all of them in CTA order
                __threadfence();
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (et == 0) {
                    const int first_cta = (sg.tile * p.k_tiles) / p.units_per_cta;
                    const int last_cta = ((sg.tile + 1) * p.k_tiles - 1) / p.units_per_cta;
                    const int old = atomicAdd(&p.counters[sg.tile], 1);
                    last_sh = (old == last_cta - first_cta) ? 1 : 0;
                    if (last_sh) p.counters[sg.tile] = 0;   // ready for the next launch
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (et == 0) TRACE(5);
                if (last_sh) {
                    __threadfence();
                    const int first_cta = (sg.tile * p.k_tiles) / p.units_per_cta;
                    const int last_cta = ((sg.tile + 1) * p.k_tiles - 1) / p.units_per_cta;
                    for (int r0 = 0; r0 < p.rows; r0 += CH) {
                        float g[CH], uu[CH];
#pragma unroll
                        for (int j = 0; j < CH; ++j) { g[j] = 0.f; uu[j] = 0.f; }
                        // contributors four at a time: all their loads are in flight before the first add, and the
                        // sums still run in CTA order
                        for (int c0 = first_cta; c0 <= last_cta; c0 += 4) {
                            float pg[4][CH], pu[4][CH];
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const int c = c0 + q;
                                const bool on = c <= last_cta;
                                const int c_first_tile = (c * p.units_per_cta) / p.k_tiles;
                                const float *src = p.scratch + ((size_t)(on ? c : first_cta) * 2 + (c_first_tile == sg.tile ? 0 : 1)) *
                                                   slot_floats + (size_t)r0 * TILE_F + et;
#pragma unroll
                                for (int j = 0; j < CH; ++j) {     // slots are NT >= rows + CH - 1 rows deep: in bounds
                                    pg[q][j] = on ? __ldcg(src + (size_t)j * TILE_F) : 0.f;
                                    if (DUAL) pu[q][j] = on ? __ldcg(src + (size_t)(NT + j) * TILE_F) : 0.f;
                                }
                            }
#pragma unroll
                            for (int q = 0; q < 4; ++q)
#pragma unroll
                                for (int j = 0; j < CH; ++j) { g[j] += pg[q][j]; if (DUAL) uu[j] += pu[q][j]; }
                        }
                        if (et == 0) TRACE(6);
                        finish_chunk<EPI>(p, sg.tile, et, r0, g, uu, xch, inv_sh, rowmeta, lane);
                        if (et == 0) TRACE(1);
                    }
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");   // last_sh is reused by the next split tile
            }
            ++acc_it;
            ++seg_i;
            if (et == 0) TRACE(4);
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
    if (threadIdx.x == 0) TRACE(7);
    SPAN_END(p);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols) : "memory");
    }
}

typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                             const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeFn g_encode = nullptr;

}  // namespace

int tc_make_map(CUtensorMap *map, const void *base, uint64_t rows, uint64_t k, uint32_t box_rows) {
    if (!g_encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
        if (!fn || q != cudaDriverEntryPointSuccess) return VIASD_EUNSUPPORTED;
        g_encode = (EncodeFn)fn;
    }
    if (((uintptr_t)base & 15) || (k % 8) || rows == 0) return VIASD_EINVAL;
    cuuint64_t dims[2] = {k, rows};
    cuuint64_t strides[1] = {k * 2};
    cuuint32_t box[2] = {TILE_K, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { g_last_cuda_error = (int)r; return VIASD_ECUDA; }
    return VIASD_OK;
}

#ifdef VIASD_TC_TRACE
extern "C" int viasd_debug_trace(long long *host_out) {
    return (int)cudaMemcpyFromSymbol(host_out, g_tc_trace, sizeof(long long) * 160 * 8);
}
static int g_span_launches = 0;
extern "C" int viasd_debug_span_reset(void) {
    static unsigned long long init[8192 * 2];
    for (int i = 0; i < 8192; ++i) { init[2 * i] = ~0ull; init[2 * i + 1] = 0ull; }
    g_span_launches = 0;
    return (int)cudaMemcpyToSymbol(g_tc_span, init, sizeof(init));
}
extern "C" int viasd_debug_span_read(unsigned long long *host_out, int *n_launches, int *meta) {
    *n_launches = g_span_launches;
    (void)meta;
    return (int)cudaMemcpyFromSymbol(host_out, g_tc_span, sizeof(unsigned long long) * 8192 * 2);
}
#endif

int tc_pick_nt(int rows) { return rows <= 16 ? 16 : rows <= 32 ? 32 : rows <= 64 ? 64 : 128; }

uint32_t tc_box_rows(uint64_t tensor_rows, uint32_t want) { return tensor_rows < want ? (uint32_t)tensor_rows : want; }

size_t tc_scratch_floats(int sm_count, int nt, bool dual) { return (size_t)sm_count * 2 * (dual ? 2 : 1) * nt * TILE_F; }

int tc_tiles(int n) { return (n + TILE_F - 1) / TILE_F; }

int launch_gemm_tc(const TcLaunch &L, cudaStream_t st) {
    TcParams p;
    memset(&p, 0, sizeof(p));
    const bool dual = L.epi == EPI_SWIGLU;
    p.nt = L.nt;
    p.rows = L.rows;
    p.row0 = L.row0;
    p.k_tiles = (L.k + TILE_K - 1) / TILE_K;
    int tiles = 0;
    for (int s = 0; s < 3; ++s) {
        p.seg_n[s] = s < L.n_seg ? L.seg_n[s] : 0;
        if (!dual && s < L.n_seg) tiles += tc_tiles(L.seg_n[s]);
        p.seg_tile_end[s] = tiles;
        p.a_tx[s] = (s < L.n_seg ? L.w_box_rows[s] : 0) * TILE_K * 2;
    }
    if (dual) tiles = tc_tiles(L.seg_n[0]);
    p.n_tiles = tiles;
    p.b_tx = L.x_box_rows * TILE_K * 2;
    p.has_lo = L.has_lo;
    p.lo_row_offset = L.lo_row_offset;
    p.epi = L.epi;
    p.out_f32 = L.out_f32;
    p.out_act = (__nv_bfloat16 *)L.out_act;
    p.act_plane = L.act_plane;
    p.ld_out = L.ld_out;
    p.scratch = L.scratch;
    p.counters = L.counters;
    p.status = L.status;
    p.ssq_in = L.ssq_in; p.ssq_in_n = L.ssq_in_n; p.ssq_stride = L.ssq_stride; p.inv_d = L.inv_d; p.eps = L.eps;
    p.next_gain = L.next_gain; p.next_act = (__nv_bfloat16 *)L.next_act; p.next_plane = L.next_plane; p.ssq_out = L.ssq_out;
    p.q_out = L.q_out; p.kc = (__nv_bfloat16 *)L.kc; p.vc = (__nv_bfloat16 *)L.vc; p.cosv = L.cosv; p.sinv = L.sinv;
    p.len_eff = L.len_eff; p.depth = L.depth; p.rope_M = L.rope_M; p.rope_H = L.rope_H; p.rope_Hkv = L.rope_Hkv;
    p.max_batch = L.max_batch; p.max_ctx = L.max_ctx; p.layer_ord = L.layer_ord;
    p.split_row = L.split_row > 0 ? L.split_row : 0x7fffffff;
    p.out_f32_2 = L.out_f32_2; p.next_gain2 = L.next_gain2; p.kc2 = (__nv_bfloat16 *)L.kc2; p.vc2 = (__nv_bfloat16 *)L.vc2;
    p.layer_ord2 = L.layer_ord2;
    const int units = p.n_tiles * p.k_tiles;
    if (units <= 0) return VIASD_OK;
    int ctas_per_sm = 1;
#ifdef VIASD_TC_TRACE
    if (getenv("VIASD_TC_PER_SM")) ctas_per_sm = atoi(getenv("VIASD_TC_PER_SM"));
#endif
    int grid = L.sm_count * ctas_per_sm < units ? L.sm_count * ctas_per_sm : units;
    p.units_per_cta = (units + grid - 1) / grid;
    grid = (units + p.units_per_cta - 1) / p.units_per_cta;
    const int nacc = dual ? 2 : 1;
    const size_t stage = (size_t)nacc * TILE_F * TILE_K * 2 + 2 * (size_t)L.nt * TILE_K * 2;
    // a ring of about 100 KB keeps HBM busy (deeper rings measured no faster) and lets the CTA of the next
    // kernel in the stream become resident beside this one, so that its weight prefetch overlaps this tail
    int stages = (int)((size_t)104 * 1024 / stage);
    if (stages < 2) stages = 2;
    if (stages > MAX_STAGES) stages = MAX_STAGES;
#ifdef VIASD_TC_TRACE
    if (getenv("VIASD_TC_DBG")) p.dbg = atoi(getenv("VIASD_TC_DBG"));
    p.launch_idx = g_span_launches++;
    p.trace_on = getenv("VIASD_TC_TRACE_IDX") ? (atoi(getenv("VIASD_TC_TRACE_IDX")) == p.launch_idx) : 1;
    if (getenv("VIASD_TC_STAGES")) { int v = atoi(getenv("VIASD_TC_STAGES")); if (v >= 2 && v < stages) stages = v; }
#endif
    if (stages < 2) return VIASD_EINVAL;
    p.stages = stages;
    // accumulators are double-buffered when two of them fit in the 512 TMEM columns
    const int acc_cols = nacc * L.nt * (L.has_lo ? 2 : 1);
    p.acc_bufs = 2 * acc_cols <= 512 ? 2 : 1;
    int cols = p.acc_bufs * acc_cols;
    p.tmem_cols = cols <= 32 ? 32 : cols <= 64 ? 64 : cols <= 128 ? 128 : cols <= 256 ? 256 : 512;
    const size_t smem = stage * stages + 1024;
    const CUtensorMap &w0 = *L.map_w[0], &w1 = *L.map_w[L.n_seg > 1 ? 1 : 0], &w2 = *L.map_w[L.n_seg > 2 ? 2 : 0];
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    pdl_config(cfg, attr, dim3(grid), dim3(THREADS), smem, st);
    static bool attr_done[4] = {false, false, false, false};
#define TC_LAUNCH(IDX, KIND)                                                                                          \
    do {                                                                                                              \
        if (!attr_done[IDX]) {                                                                                        \
            CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel<KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize, 208 * 1024)); \
            attr_done[IDX] = true;                                                                                    \
        }                                                                                                             \
        CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_tc_kernel<KIND>, w0, w1, w2, *L.map_x, p));                            \
    } while (0)
    switch (L.epi) {
    case EPI_SWIGLU: TC_LAUNCH(0, EPI_SWIGLU); break;
    case EPI_ADD_NORM: TC_LAUNCH(1, EPI_ADD_NORM); break;
    case EPI_QKV_ROPE: TC_LAUNCH(2, EPI_QKV_ROPE); break;
    default: TC_LAUNCH(3, EPI_STORE); break;          // EPI_STORE and EPI_ADD share one kernel
    }
#undef TC_LAUNCH
    LAUNCH_CHECK();
    return VIASD_OK;
}
