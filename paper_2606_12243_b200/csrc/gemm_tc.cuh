// Interface of the tcgen05 weight-streaming GEMM (gemm_tc.cu).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <string.h>

struct TcParams {                       // kernel argument block
    int nt, stages, tmem_cols;          // token-tile width (MMA N), smem ring depth, TMEM columns to allocate
    int acc_bufs;                       // accumulator buffers in TMEM (2 when they fit, else 1)
    int rows, row0;                     // token rows of this launch and the first one
    int k_tiles, n_tiles, units_per_cta;
    int seg_n[3], seg_tile_end[3];      // output features per weight matrix; running tile count
    uint32_t a_tx[3], b_tx;             // bytes one TMA box of each operand delivers
    int has_lo, lo_row_offset;          // activation lo plane: present, and its row offset in the 2-D map
    int epi;                            // EPI_STORE / EPI_ADD / EPI_SWIGLU
    float *out_f32;
    __nv_bfloat16 *out_act;
    size_t act_plane;
    int ld_out;
    float *scratch;                     // [grid][2] partial-tile slots
    int *counters;                      // [n_tiles], zero between launches
    int *status;                        // device status word
    // fused RMSNorm on the input side: per-row partial sums of squares written by the producer
    const float *ssq_in; int ssq_in_n, ssq_stride; float inv_d, eps;
    // EPI_ADD_NORM: what the next RMSNorm needs
    const float *next_gain; __nv_bfloat16 * next_act; size_t next_plane; float *ssq_out;
    // EPI_QKV_ROPE
    float *q_out; __nv_bfloat16 *kc, *vc; const float *cosv, *sinv; const int *len_eff, *depth;
    int rope_M, rope_H, rope_Hkv, max_batch, max_ctx, layer_ord;
    int tree_stride;                    // ints between the depth tables of consecutive sequences
    // two row streams in one launch (full verifier rows first, slim verifier rows from split_row on)
    int split_row, layer_ord2; float *out_f32_2; const float *next_gain2; __nv_bfloat16 *kc2, *vc2;
    const int *run_flag;                // null, or a device flag: the kernel leaves at once when it is zero
    const int *kv_keep;                 // null, or [batch]: cache slots below kv_keep[b] are complete and are not rewritten
};

struct TcLaunch {                       // host-side description of one GEMM
    const CUtensorMap *map_w[3];
    int seg_n[3], n_seg;
    uint32_t w_box_rows[3];
    const CUtensorMap *map_x;
    uint32_t x_box_rows;
    int has_lo, lo_row_offset;
    int rows, row0, k, nt;
    int epi;
    float *out_f32;
    void *out_act;
    size_t act_plane;
    int ld_out;
    float *scratch;
    int *counters;
    int *status;
    int sm_count;
    // fused RMSNorm on the input side: per-row partial sums of squares written by the producer
    const float *ssq_in; int ssq_in_n, ssq_stride; float inv_d, eps;
    // EPI_ADD_NORM: what the next RMSNorm needs
    const float *next_gain; void * next_act; size_t next_plane; float *ssq_out;
    // EPI_QKV_ROPE
    float *q_out; void *kc, *vc; const float *cosv, *sinv; const int *len_eff, *depth;
    int rope_M, rope_H, rope_Hkv, max_batch, max_ctx, layer_ord, tree_stride;
    int split_row, layer_ord2; float *out_f32_2; const float *next_gain2; void *kc2, *vc2;
    const int *run_flag, *kv_keep;
    int ring_kb, epi_groups;            // stream-K kernel: ring size and epilogue groups; 0 = defaults (200 KB; by token tile)
};

// 2-D bf16 tensor [rows, k] row-major -> TMA map with a (64 x box_rows) box and the 128-byte swizzle
int tc_make_map(CUtensorMap *map, const void *base, uint64_t rows, uint64_t k, uint32_t box_rows);
int tc_pick_nt(int rows, bool has_lo);
uint32_t tc_box_rows(uint64_t tensor_rows, uint32_t want);
size_t tc_scratch_floats(int sm_count, int nt, bool dual);
int tc_tiles(int n);
int launch_gemm_tc(const TcLaunch &L, cudaStream_t st);

void tc_fill_params(const TcLaunch &L, TcParams &p);

