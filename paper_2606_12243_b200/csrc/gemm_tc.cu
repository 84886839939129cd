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
// k-blocks of a tile finishes it from TMEM; otherwise it writes an fp32 partial and counts itself in.  The
// contributors that end their range inside the tile then share its finishing: each waits (bounded) for the
// count to be complete, pulls its slice of the token rows of every partial into the idle shared-memory ring
// with bulk copies and sums them in CTA order - bit-reproducible whoever does it.  A contributor that
// continues into the next tile never waits, so waits cannot chain.
//
// Warp roles (320 threads): warp 0 issues TMA loads into a ring of stages, warp 1 allocates TMEM and
// issues tcgen05.mma, warps 2-9 read the accumulators (tcgen05.ld) and run the epilogue.  Accumulators
// are double-buffered in TMEM so the epilogue of one tile overlaps the main loop of the next.
// Every wait is bounded: on expiry the CTA records VIASD_EDEVICE, lets its copies land and leaves.
#include "common.cuh"
#include "gemm_tc.cuh"
#include <stdlib.h>

#include "gemm_tc_device.cuh"

namespace {

template <int EPI, int GROUPS, int KBT>
__global__ void __launch_bounds__(64 + 128 * GROUPS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_w0, const __grid_constant__ CUtensorMap map_w1,
               const __grid_constant__ CUtensorMap map_w2, const __grid_constant__ CUtensorMap map_x, const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) unsigned long long bars[2 * MAX_STAGES + 5];
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;
    __shared__ float inv_sh[128];                       // per-row 1/rms of the input (fused RMSNorm)
    __shared__ float xch[GROUPS * CH * TILE_F];         // rotary partner exchange, one buffer per epilogue group
    __shared__ int4 rowmeta[128];                       // per token row: rotary position, cache slot, offset in its cache

    constexpr bool DUAL = EPI == EPI_SWIGLU;
    RUN_FLAG_EXIT(p.run_flag);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel may start its prologue
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int NT = p.nt, S = p.stages;
    constexpr int NACC = DUAL ? 2 : 1;
    // A stage holds KB boxes of 64 k-columns of every operand: two for the single-matrix launches (32 KB of weights per
    // stage, as the gate/up launch has with its two matrices).  With 16 KB per stage the bookkeeping of a stage - a
    // barrier wait, a fence and a commit in the MMA thread, a wait and the copies' issue in the TMA thread - took
    // longer than the stage's weights take to arrive: those launches streamed at 5.9 TB/s, not 6.5.
    constexpr int KB = DUAL ? 1 : KBT;                    // (the launch picks one box at wide token tiles: two would leave two stages)
    const uint32_t a_bytes = TILE_F * TILE_K * 2, b_bytes = (uint32_t)NT * TILE_K * 2;
    const uint32_t box_bytes = NACC * a_bytes + 2 * b_bytes;          // one k-box of every operand
    const uint32_t stage_bytes = KB * box_bytes;
    auto full_bar = [&](int s) { return smem_u32(&bars[s]); };
    auto empty_bar = [&](int s) { return smem_u32(&bars[MAX_STAGES + s]); };
    auto tfull_bar = [&](int b) { return smem_u32(&bars[2 * MAX_STAGES + b]); };
    auto tempty_bar = [&](int b) { return smem_u32(&bars[2 * MAX_STAGES + 2 + b]); };
    const uint32_t gather_bar = smem_u32(&bars[2 * MAX_STAGES + 4]);
    const int NB = p.has_lo ? 2 * NT : NT;                  // MMA N: hi and lo token columns side by side
    const uint32_t acc_cols = NACC * NB;                    // TMEM columns per accumulator buffer

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), GROUPS * 4); }
        mbar_init(gather_bar, GROUPS * 128);
        abort_sh = 0;
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

    const int total_units = p.n_tiles * p.k_tiles;
    const int u_begin = blockIdx.x * p.units_per_cta;
    const int u_end = min(total_units, u_begin + p.units_per_cta);

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            const int n_it = (u_end - u_begin) / KB;          // stages: ranges and tiles are whole numbers of KB boxes
            // unit -> weight matrix, its first row, k-block
            auto unit = [&](int it, const CUtensorMap *&mw, int &wrow, int &kt, int &sidx) {
                const int u = u_begin + it * KB, tile = u / p.k_tiles;
                kt = u - tile * p.k_tiles;
                int s = 0, t0 = 0;
                if (!DUAL) while (s < 2 && tile >= p.seg_tile_end[s]) { t0 = p.seg_tile_end[s]; ++s; }
                mw = s == 0 ? &map_w0 : (s == 1 ? &map_w1 : &map_w2);
                wrow = (tile - t0) * TILE_F;
                sidx = s;
            };
            const uint64_t wpol = l2_evict_first_policy();     // weights pass through once
            auto load_w = [&](int st, const CUtensorMap *mw, int wrow, int kt) {
                const uint32_t base = smem_base + st * stage_bytes;
#pragma unroll
                for (int kb = 0; kb < KB; ++kb)
                    tma_load_2d_hint(base + kb * box_bytes, mw, full_bar(st), (kt + kb) * TILE_K, wrow, wpol);
                if (DUAL) tma_load_2d_hint(base + a_bytes, &map_w1, full_bar(st), kt * TILE_K, wrow, wpol);
            };
            auto load_x = [&](int st, int kt) {
                const uint32_t base = smem_base + st * stage_bytes + NACC * a_bytes;
#pragma unroll
                for (int kb = 0; kb < KB; ++kb) {
                    tma_load_2d(base + kb * box_bytes, &map_x, full_bar(st), (kt + kb) * TILE_K, p.row0);
                    tma_load_2d(base + kb * box_bytes + b_bytes, &map_x, full_bar(st), (kt + kb) * TILE_K, p.row0 + p.lo_row_offset);
                }
            };
            const CUtensorMap *mw; int wrow, kt, sidx;
            // Weights do not depend on the kernel before this one: fill the ring with them first, and only then
            // wait for that kernel (programmatic dependent launch) before touching the activations.
            const int pre = n_it < S ? n_it : S;
            for (int it = 0; it < pre; ++it) {
                unit(it, mw, wrow, kt, sidx);
                asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(full_bar(it)),
                             "r"(DUAL ? 2 * p.a_tx[0] : KB * p.a_tx[sidx]) : "memory");
                load_w(it, mw, wrow, kt);
            }
            asm volatile("griddepcontrol.wait;" ::: "memory");
            for (int it = 0; it < pre; ++it) {
                unit(it, mw, wrow, kt, sidx);
                mbar_expect_tx(full_bar(it), KB * 2 * p.b_tx);
                load_x(it, kt);
            }
            for (int it = pre; it < n_it; ++it) {
                const int st = it % S;
                if (!mbar_wait(empty_bar(st), ((it / S) & 1) ^ 1, &abort_sh, p.status)) break;
                unit(it, mw, wrow, kt, sidx);
                mbar_expect_tx(full_bar(st), (DUAL ? 2 * p.a_tx[0] : KB * p.a_tx[sidx]) + KB * 2 * p.b_tx);
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
                for (int kt = sg.ka; kt < sg.kb; kt += KB, ++it) {
                    const int st = it % S;
                    if (!(ok = mbar_wait(full_bar(st), (it / S) & 1, &abort_sh, p.status))) break;
                    tc_fence_after();
                    const uint32_t base = smem_base + st * stage_bytes;
                    // the hi tile is followed by the lo tile: together one K-major operand of NB rows
                    const uint32_t bh = base + NACC * a_bytes;
                    // one descriptor per operand and stage; a k-step of 16 columns is 32 bytes further on, 2 in the
                    // descriptor's address field (the MMA-issuing thread is a single instruction stream that has about
                    // the arrival time of a stage to get through all this: every instruction here counts)
                    const uint64_t da2 = DUAL ? smem_desc(base + a_bytes) : 0ull;
#pragma unroll
                    for (int kb = 0; kb < KB; ++kb) {
                        const uint64_t da = smem_desc(base + kb * box_bytes), db = smem_desc(bh + kb * box_bytes);
#pragma unroll
                        for (int k = 0; k < TILE_K / 16; ++k) {
                            const uint32_t acc = (kt > sg.ka || kb > 0 || k > 0) ? 1u : 0u;
                            tc_mma(d0, da + 2 * k, db + 2 * k, idesc, acc);
                            if (DUAL) tc_mma(d0 + NB, da2 + 2 * k, db + 2 * k, idesc, acc);
                        }
                    }
                    tc_commit(empty_bar(st));              // the stage is free once these MMAs have read it
                }
                if (ok) tc_commit(tfull_bar(buf));          // accumulator complete
                ++acc_it;
            }
        }
    } else {
        // ---------------- epilogue (warps 2..5 and 6..9 <-> TMEM lane quarters 2,3,0,1) ----------------
        // One or two groups of 128 threads (the launch decides: the second group pays at wide token tiles, where the
        // finishing is many chunks long, and costs a little at narrow ones); wherever rows are handled chunk by
        // chunk, the groups take the chunks in turn.
        const int quarter = warp & 3;
        const int f = quarter * 32 + lane;                  // feature lane inside the tile, as TMEM lanes map to warps
        const int et_all = threadIdx.x - 64;                // 0..255 among epilogue threads
        const int group = GROUPS > 1 ? et_all >> 7 : 0, et = GROUPS > 1 ? (et_all & 127) : et_all;   // et: the thread's number in its group = its feature in staged tiles
        constexpr int epi_threads = GROUPS * 128, n_groups = GROUPS;
        const size_t slot_floats = (size_t)NACC * NT * TILE_F;
        // per-row tables (all 128 entries defined: chunks read a few rows past p.rows and discard them)
        inv_sh[et] = 0.f;
        rowmeta[et] = make_int4(0, 0, 0, 0);
        asm volatile("bar.sync 1, %0;" ::"n"(epi_threads) : "memory");
        // The tile this CTA's range ends in is the one it will help to finish: what that epilogue reads from
        // weights (not from the kernel before) is fetched now, off the critical path.
        const int last_tile = (u_end - 1) / p.k_tiles;
        float2 last_gain = make_float2(0.f, 0.f);
        if (EPI == EPI_ADD_NORM) {
            const int n = last_tile * TILE_F + et;
            if (n < p.seg_n[0]) {
                last_gain.x = __ldg(p.next_gain + n);
                last_gain.y = p.next_gain2 ? __ldg(p.next_gain2 + n) : last_gain.x;
            }
        }

        // A tile is finished from one of three sources: the accumulator in TMEM (this CTA held all of K), the
        // partials staged in shared memory, or the partials read straight from global memory.  All three feed ONE
        // copy of the epilogue code, and that copy runs once "dry" (no row is live, nothing is stored) before
        // the kernel waits for its predecessor: the epilogue otherwise runs exactly once per CTA, at the very end,
        // from a cold instruction cache while HBM is saturated, and those instruction misses were the tail.
        enum { SRC_DRY, SRC_TMEM, SRC_SMEM, SRC_GLOBAL };
        int acc_it = 0, u = u_begin, seg_i = 0;
        Seg sg;
        sg.tile = last_tile; sg.ka = 0; sg.kb = 0;                 // dry pass: the tile this CTA is most likely to finish
        bool ok = true, dry = true;
        while (ok) {
            int src = SRC_DRY, buf = 0, first_cta = 0, last_cta = 0;
            uint32_t t0 = 0;
            const float *parts = nullptr, *aux = nullptr;
            int stage_rows = 0, aux_kind = 0;                // staged gather: rows per round; 1: residual rows, 2: rotary tables
            int row_begin = 0, row_end = p.rows;             // the rows this CTA finishes
            if (dry) {
                // the dry pass sums one "contributor" out of whatever the ring holds, so that the staged path's code is warm too
                src = SRC_SMEM;
                parts = reinterpret_cast<const float *>(smem_raw + (smem_base - smem_u32(smem_raw)));
            } else {
                if (!next_seg(u, u_end, p.k_tiles, sg)) break;
                buf = acc_it % p.acc_bufs;
                if (!(ok = mbar_wait(tfull_bar(buf), (acc_it / p.acc_bufs) & 1, &abort_sh, p.status))) break;
                tc_fence_after();
                t0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * acc_cols;
                if (sg.ka == 0 && sg.kb == p.k_tiles) {
                    src = SRC_TMEM;
                } else {
                    // partial of a split tile: slot 0 if the tile is the first one this CTA touches, else slot 1
                    float *slot = p.scratch + ((size_t)blockIdx.x * 2 + (seg_i == 0 ? 0 : 1)) * slot_floats;
                    for (int c = group * CH; c < p.rows; c += n_groups * CH) {   // padding rows beyond p.rows are never read
                        float g[CH], uu[CH];
                        if (p.has_lo) {                          // add the product with the lo plane
                            float lo[CH];
                            tc_ld8x2(t0 + c, t0 + NT + c, g, lo);
#pragma unroll
                            for (int j = 0; j < CH; ++j) g[j] += lo[j];
                            if (DUAL) {
                                tc_ld8x2(t0 + NB + c, t0 + NB + NT + c, uu, lo);
#pragma unroll
                                for (int j = 0; j < CH; ++j) uu[j] += lo[j];
                            }
                        } else {
                            tc_ld8(t0 + c, g);
                            if (DUAL) tc_ld8(t0 + NB + c, uu);
                        }
#pragma unroll
                        for (int j = 0; j < CH; ++j) {
                            slot[(size_t)(c + j) * TILE_F + f] = g[j];
                            if (DUAL) slot[(size_t)(NT + c + j) * TILE_F + f] = uu[j];
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tempty_bar(buf));   // accumulator buffer may be overwritten
                    // Publish the partial.  The contributors for which this tile is the last piece of work then share
                    // its finishing: each waits (bounded) until every contributor has arrived and finishes its own
                    // slice of the token rows, summing the partials in CTA order.  A contributor that goes on into the
                    // next tile only arrives and never waits, so no wait depends on another wait.
                    // (release / acquire: the barrier orders the group's stores before its first thread's release, which
                    // is cumulative; a fence per thread on both sides was a microsecond of the launch's tail)
                    asm volatile("bar.sync 1, %0;" ::"n"(epi_threads) : "memory");
                    first_cta = (sg.tile * p.k_tiles) / p.units_per_cta;
                    last_cta = ((sg.tile + 1) * p.k_tiles - 1) / p.units_per_cta;
                    if (et_all == 0) asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(p.counters + sg.tile) : "memory");   // low half: arrivals
                    if (u < u_end) { ++acc_it; ++seg_i; continue; }
                    const int n_c = last_cta - first_cta + 1;
                    const int last_range_end = min(total_units, (last_cta + 1) * p.units_per_cta);
                    const int n_fin = n_c - (last_range_end > (sg.tile + 1) * p.k_tiles ? 1 : 0);
                    if (et_all == 0) {
                        const int *ctr = p.counters + sg.tile;
                        auto arrived = [&]() { int v; asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory"); return v & 0xffff; };
                        const long long w0 = clock64();
                        while (arrived() < n_c) {
                            if (abort_sh || clock64() - w0 > WAIT_LIMIT_CYCLES) { abort_sh = 1; atomicExch(p.status, VIASD_EDEVICE); break; }
                            __nanosleep(64);
                        }
                        // high half: finishers that have seen all arrivals; the last of them leaves the counter at zero
                        if (!abort_sh && (atomicAdd(&p.counters[sg.tile], 1 << 16) >> 16) == n_fin - 1) atomicExch(&p.counters[sg.tile], 0);
                    }
                    asm volatile("bar.sync 1, %0;" ::"n"(epi_threads) : "memory");
                    if (abort_sh) { ok = false; break; }
                    {
                        // this finisher's rows: whole chunks, dealt in order of CTA number
                        const int n_chunks = (p.rows + CH - 1) / CH, per = (n_chunks + n_fin - 1) / n_fin;
                        const int mine = blockIdx.x - first_cta;
                        row_begin = min(p.rows, mine * per * CH);
                        row_end = min(p.rows, (mine + 1) * per * CH);
                    }
                    src = SRC_GLOBAL;
                    // Staged gather: when this is the CTA's last piece of work the shared-memory ring is idle, so the
                    // partials (and the rows the epilogue would otherwise fetch chunk by chunk) come in by bulk copies,
                    // as many rows per round as the ring holds.  Same sums in the same order as the direct path.
                    const int fit = (int)(((uint32_t)S * stage_bytes) / ((uint32_t)(n_c * NACC + 1) * TILE_F * 4u)) / CH * CH;
                    if (fit >= CH && row_end > row_begin) {
                        const int my_rows = (row_end - row_begin + CH - 1) / CH * CH;
                        stage_rows = fit < my_rows ? fit : my_rows;
                        if (EPI == EPI_ADD_NORM && (sg.tile + 1) * TILE_F <= p.seg_n[0]) aux_kind = 1;
                        if (EPI == EPI_QKV_ROPE && sg.tile < p.seg_tile_end[1]) aux_kind = 2;
                        src = SRC_SMEM;
                    }
                }
            }

            // ---- the one finishing loop, over blocks of rows (one block unless the gather is staged in rounds)
            const int fe = src == SRC_TMEM ? f : et;
            const int rows_live = dry ? 0 : p.rows, rows_loop = dry ? CH : row_end;
            const int blk_rows = stage_rows ? stage_rows : (rows_loop > 0 ? rows_loop : 1);
            const int plane = stage_rows ? stage_rows * TILE_F : p.rows * TILE_F;     // floats between contributors in shared memory
            int round = 0;
#pragma unroll 1
            for (int blk0 = dry ? 0 : row_begin; blk0 < rows_loop && ok; blk0 += blk_rows, ++round) {
            const int blk_end = min(rows_loop, blk0 + blk_rows);
            if (stage_rows) {
                // rows blk0 .. blk_end-1 of every contributor (and of the epilogue's own inputs) into the ring
                const int nr = min(p.rows, blk_end) - blk0, n_c = last_cta - first_cta + 1;
                const uint32_t row_bytes = TILE_F * 4u, aux_sh = smem_base, part_sh = smem_base + (uint32_t)stage_rows * row_bytes;
                if (round > 0) asm volatile("bar.sync 1, %0;" ::"n"(epi_threads) : "memory");    // everyone is done with the previous round's rows
                const bool has_part = et_all < n_c * NACC, has_aux = aux_kind && et_all < nr;   // nr <= 128: first group
                asm volatile("fence.proxy.async.global;" ::: "memory");
                if (has_part || has_aux) {
                    mbar_expect_tx(gather_bar, (has_part ? (uint32_t)nr * row_bytes : 0u) + (has_aux ? row_bytes : 0u));
                    if (has_part) {
                        const int c = first_cta + et_all / NACC, half = et_all - (et_all / NACC) * NACC;
                        const int c_first_tile = (c * p.units_per_cta) / p.k_tiles;
                        const float *from = p.scratch + ((size_t)c * 2 + (c_first_tile == sg.tile ? 0 : 1)) * slot_floats +
                                            (size_t)half * NT * TILE_F + (size_t)blk0 * TILE_F;
                        bulk_load(part_sh + (uint32_t)et_all * (uint32_t)stage_rows * row_bytes, from, (uint32_t)nr * row_bytes, gather_bar);
                    }
                    if (has_aux) {
                        const uint32_t dst = aux_sh + (uint32_t)et * row_bytes;
                        if (aux_kind == 1) {
                            bulk_load(dst, p.out_f32 + (size_t)(p.row0 + blk0 + et) * p.ld_out + sg.tile * TILE_F, row_bytes, gather_bar);
                        } else {
                            const int pos = rowmeta[blk0 + et].x;
                            bulk_load(dst, p.cosv + (size_t)pos * 64, 256, gather_bar);
                            bulk_load(dst + 256, p.sinv + (size_t)pos * 64, 256, gather_bar);
                        }
                    }
                } else {
                    mbar_arrive(gather_bar);
                }
                if (!(ok = mbar_wait(gather_bar, round & 1, &abort_sh, p.status))) break;
                parts = reinterpret_cast<const float *>(smem_raw + (part_sh - smem_u32(smem_raw)));
                // finish_chunk indexes the epilogue's rows by their number in the launch: shift the base by the block start
                if (aux_kind) aux = reinterpret_cast<const float *>(smem_raw + (aux_sh - smem_u32(smem_raw))) - (size_t)blk0 * TILE_F;
            }
#pragma unroll 1
            for (int r0 = blk0 + group * CH; r0 < blk_end; r0 += n_groups * CH) {
                float g[CH], uu[CH];
#pragma unroll
                for (int j = 0; j < CH; ++j) { g[j] = 0.f; uu[j] = 0.f; }
                if (src == SRC_TMEM) {
                    tc_ld8(t0 + r0, g);
                    if (DUAL) tc_ld8(t0 + NB + r0, uu);
                    if (p.has_lo) {
                        float lo[CH];
                        tc_ld8(t0 + NT + r0, lo);
#pragma unroll
                        for (int j = 0; j < CH; ++j) g[j] += lo[j];
                        if (DUAL) {
                            tc_ld8(t0 + NB + NT + r0, lo);
#pragma unroll
                            for (int j = 0; j < CH; ++j) uu[j] += lo[j];
                        }
                    }
                } else if (src == SRC_SMEM) {
                    for (int c = 0; c <= last_cta - first_cta; ++c) {
#pragma unroll
                        for (int j = 0; j < CH; ++j) {
                            const int r = min(r0 + j, p.rows - 1) - blk0;  // row inside the staged block; rows past the end are discarded
                            g[j] += parts[(c * NACC) * plane + r * TILE_F + et];
                            if (DUAL) uu[j] += parts[(c * NACC + 1) * plane + r * TILE_F + et];
                        }
                    }
                } else if (src == SRC_GLOBAL) {
                    // rare (a tile shared by more CTAs than the ring can stage a chunk of): plain loads, contributor by
                    // contributor, kept small on purpose - the size of this loop's code is part of every launch's tail
#pragma unroll 1
                    for (int c = first_cta; c <= last_cta; ++c) {
                        const int c_first_tile = (c * p.units_per_cta) / p.k_tiles;
                        const float *from = p.scratch + ((size_t)c * 2 + (c_first_tile == sg.tile ? 0 : 1)) * slot_floats +
                                            (size_t)r0 * TILE_F + et;
#pragma unroll
                        for (int j = 0; j < CH; ++j) {         // slots are NT >= rows + CH - 1 rows deep: in bounds
                            g[j] += __ldcg(from + (size_t)j * TILE_F);
                            if (DUAL) uu[j] += __ldcg(from + (size_t)(NT + j) * TILE_F);
                        }
                    }
                }
                finish_chunk<EPI, GROUPS>(p, sg.tile, fe, r0, g, uu, xch + group * (CH * TILE_F), inv_sh, rowmeta, lane, aux, rows_live,
                                  src != SRC_TMEM && sg.tile == last_tile, last_gain, GROUPS > 1 ? 2 + group : 1);
            }
            }   // blocks of rows

            if (dry) {
                dry = false;
                asm volatile("griddepcontrol.wait;" ::: "memory");     // outputs, scratch and counters belong to the chain
                if (p.ssq_in) {
                    // 1/rms per input row from the row's partial sums of squares, always in one order: 32 lane-strided
                    // sub-sums, then the shuffle tree's pairing (16, 8, 4, 2, 1) - reproducible whatever the row count.
                    if (p.rows > 32) {
                      if (group == 0) {
                        // a thread per row: adjacent threads read adjacent floats, 32 independent loads at a time.  A
                        // warp per row (below) is a chain of dependent, uncoalesced loads, a microsecond per row, which
                        // at a hundred rows outlasted the streaming of the weights.
                        const float *from = p.ssq_in + p.row0 + min(et, p.rows - 1);
                        float acc[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) acc[i] = 0.f;
#pragma unroll 1
                        for (int j0 = 0; j0 < p.ssq_in_n; j0 += 32) {
                            float v[32];
#pragma unroll
                            for (int i = 0; i < 32; ++i) v[i] = j0 + i < p.ssq_in_n ? __ldcg(from + (size_t)(j0 + i) * p.ssq_stride) : 0.f;
#pragma unroll
                            for (int i = 0; i < 32; ++i) acc[i] += v[i];
                        }
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
                            for (int i = 0; i < o; ++i) acc[i] += acc[i + o];
                        }
                        if (et < p.rows) inv_sh[et] = rsqrtf(acc[0] * p.inv_d + p.eps);
                      }
                    } else {
                        for (int r = (et_all >> 5); r < p.rows; r += n_groups * 4) {
                            float ss = 0.f;
                            for (int j = lane; j < p.ssq_in_n; j += 32) ss += __ldcg(p.ssq_in + (size_t)j * p.ssq_stride + p.row0 + r);
                            ss = warp_sum(ss);
                            if (lane == 0) inv_sh[r] = rsqrtf(ss * p.inv_d + p.eps);
                        }
                    }
                }
                if (EPI == EPI_QKV_ROPE) {
                    if (et_all < p.rows) {
                        // rows are laid out [stream][sequence][block row]; stream 1 (rows >= split_row) is the slim verifier
                        const int row = p.row0 + et, stream = row >= p.split_row ? 1 : 0, rs = row - stream * p.split_row;
                        const int b = rs / p.rope_M, i = rs - b * p.rope_M;
                        const int n_ctx = p.len_eff[b];
                        // replay pass: rows that fall on slots the cache already holds are recomputed but not stored
                        const int slot = (p.kv_keep && n_ctx + i < p.kv_keep[b]) ? -1 : n_ctx + i;
                        // the row's place in its cache, without the head (element offset, 64 bits in .z / .w, the stream in
                        // bit 30 of .w): worked out once here, not per row and tile in the epilogue
                        const int lo = stream ? p.layer_ord2 : p.layer_ord;
                        const unsigned long long off = slot < 0 ? 0ull
                            : (((unsigned long long)lo * p.max_batch + b) * p.rope_Hkv * p.max_ctx + slot) * TILE_F;
                        rowmeta[et] = make_int4(n_ctx + p.depth[(size_t)b * p.tree_stride + i], slot, (int)(unsigned)(off & 0xffffffffull),
                                                (int)((unsigned)(off >> 32) | ((unsigned)stream << 30)));
                    }
                }
                asm volatile("bar.sync 1, %0;" ::"n"(epi_threads) : "memory");
                continue;
            }
            if (src == SRC_TMEM) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(tempty_bar(buf));   // accumulator buffer may be overwritten
            }
            ++acc_it;
            ++seg_i;
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


// token-tile width: the MMA's N (2 x NT with the hi / lo planes side by side, else NT) comes in multiples of 16
int tc_pick_nt(int rows, bool has_lo) {
    const int g = has_lo ? 8 : 16, nt = (rows + g - 1) / g * g;
    return nt < 16 ? 16 : nt > 128 ? 128 : nt;
}

uint32_t tc_box_rows(uint64_t tensor_rows, uint32_t want) { return tensor_rows < want ? (uint32_t)tensor_rows : want; }

size_t tc_scratch_floats(int sm_count, int nt, bool dual) { return (size_t)sm_count * 2 * (dual ? 2 : 1) * nt * TILE_F; }

int tc_tiles(int n) { return (n + TILE_F - 1) / TILE_F; }

// Groups of four epilogue warps: a second one above token tiles of 48 unless the caller says otherwise; the gate/up
// launch already from 17 rows on: its split tiles have two or three contributors, so a finisher has two chunks of 8 rows
// of two accumulators to finish, and the groups take one each (8B, 27 rows: finishing 7.5 -> 5.7 us; with 9 rows, or for
// the other epilogues, whose finishers have one chunk each, the second group only costs)
static int tc_groups(const TcLaunch &L) {
    return L.epi_groups == 1 || L.epi_groups == 2 ? L.epi_groups : (L.nt > 48 || (L.epi == EPI_SWIGLU && L.rows > 16) ? 2 : 1);
}
// k-boxes of 64 columns per ring stage (the kernel's KBT): two for the single-matrix launches up to token tiles of 96
// (32B batch 16, 96 rows: step 27.9 -> 27.1 ms with two stages of 80 KB; at 112 rows, two stages of 88 KB, no gain)
static int tc_boxes(const TcLaunch &L) { return L.epi == EPI_SWIGLU || L.nt > 96 ? 1 : 2; }

// TcLaunch (host description) -> TcParams (kernel argument block), schedule fields left to the caller
void tc_fill_params(const TcLaunch &L, TcParams &p) {
    memset(&p, 0, sizeof(p));
    const bool dual = L.epi == EPI_SWIGLU;
    p.nt = L.nt;
    p.rows = L.rows;
    p.row0 = L.row0;
    // k-boxes of 64 columns; an even number per tile for the single-matrix launches, whose narrow-tile instance takes
    // two boxes per stage (the columns past k read as zeros), so that both instances cut k at the same places
    p.k_tiles = dual ? (L.k + TILE_K - 1) / TILE_K : 2 * ((L.k + 2 * TILE_K - 1) / (2 * TILE_K));
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
    p.max_batch = L.max_batch; p.max_ctx = L.max_ctx; p.layer_ord = L.layer_ord; p.tree_stride = L.tree_stride;
    p.split_row = L.split_row > 0 ? L.split_row : 0x7fffffff;
    p.out_f32_2 = L.out_f32_2; p.next_gain2 = L.next_gain2; p.kc2 = (__nv_bfloat16 *)L.kc2; p.vc2 = (__nv_bfloat16 *)L.vc2;
    p.layer_ord2 = L.layer_ord2;
    p.run_flag = L.run_flag;
    p.kv_keep = L.kv_keep;
}

int launch_gemm_tc(const TcLaunch &L, cudaStream_t st) {
    TcParams p;
    tc_fill_params(L, p);
    const bool dual = L.epi == EPI_SWIGLU;
    const int units = p.n_tiles * p.k_tiles;
    if (units <= 0) return VIASD_OK;
    int ctas_per_sm = 1;
    int grid = L.sm_count * ctas_per_sm < units ? L.sm_count * ctas_per_sm : units;
    p.units_per_cta = (units + grid - 1) / grid;
    if (!dual) p.units_per_cta += p.units_per_cta & 1;        // whole stages of two boxes
    grid = (units + p.units_per_cta - 1) / p.units_per_cta;
    const int nacc = dual ? 2 : 1;
    const size_t stage = tc_boxes(L) * ((size_t)nacc * TILE_F * TILE_K * 2 + 2 * (size_t)L.nt * TILE_K * 2);
    // The depth of the ring bounds the streaming rate (bytes in flight per SM): 200 KB, one CTA per SM, measured
    // faster than 100 KB with the next kernel's CTA resident beside this one.
    const int ring_kb = L.ring_kb > 0 ? L.ring_kb : 200;
    int stages = (int)((size_t)ring_kb * 1024 / stage);
    if (stages < 2) stages = 2;
    if (stages > MAX_STAGES) stages = MAX_STAGES;
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
    const int groups = tc_groups(L);
    pdl_config(cfg, attr, dim3(grid), dim3(64 + 128 * groups), smem, st);
    static bool attr_done[64][16];           // the attribute belongs to a (kernel, device) pair
    const int boxes = tc_boxes(L);
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return VIASD_EUNSUPPORTED;
#define TC_LAUNCH_G(IDX, KIND, G, KBX)                                                                                     \
    do {                                                                                                              \
        if (!attr_done[dev][IDX]) {                                                                                   \
            CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel<KIND, G, KBX>, cudaFuncAttributeMaxDynamicSharedMemorySize, 208 * 1024)); \
            attr_done[dev][IDX] = true;                                                                               \
        }                                                                                                             \
        CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_tc_kernel<KIND, G, KBX>, w0, w1, w2, *L.map_x, p));                    \
    } while (0)
#define TC_LAUNCH(IDX, KIND) do { if (boxes == 2) { if (groups == 2) TC_LAUNCH_G(IDX + 12, KIND, 2, 2); else TC_LAUNCH_G(IDX + 8, KIND, 1, 2); } \
                                   else { if (groups == 2) TC_LAUNCH_G(IDX + 4, KIND, 2, 1); else TC_LAUNCH_G(IDX, KIND, 1, 1); } } while (0)
    switch (L.epi) {
    case EPI_SWIGLU: TC_LAUNCH(0, EPI_SWIGLU); break;
    case EPI_ADD_NORM: TC_LAUNCH(1, EPI_ADD_NORM); break;
    case EPI_QKV_ROPE: TC_LAUNCH(2, EPI_QKV_ROPE); break;
    default: TC_LAUNCH(3, EPI_STORE); break;          // EPI_STORE and EPI_ADD share one kernel
    }
#undef TC_LAUNCH
#undef TC_LAUNCH_G
    LAUNCH_CHECK();
    return VIASD_OK;
}
