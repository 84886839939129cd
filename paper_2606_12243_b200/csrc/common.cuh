// Shared declarations of the CUDA side: model handle, workspace layout, launch prototypes.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include "../../include/viasd.h"
#include "gemm_tc.cuh"

#define VIASD_MAX_ROWS_PER_SEQ 64
// Arrival counters of the attention kernels: one per (stream, sequence, kv head, item of that kv head).  The
// keys-on-lanes kernel deals the query heads of a kv head to at most this many items.
#define VIASD_ATTN_ITEMS_PER_KV_HEAD 4
inline size_t attn_counter_count(int max_batch, int n_kv_heads) {
    return (size_t)2 * max_batch * n_kv_heads * VIASD_ATTN_ITEMS_PER_KV_HEAD;
}

// ---------------------------------------------------------------------------------------------
// device-side records kept in the workspace
// ---------------------------------------------------------------------------------------------
struct TreeInfo {                       // one per sequence, rebuilt from `parent` at the start of every pass
    unsigned long long anc[VIASD_MAX_ROWS_PER_SEQ];   // bit r set: row r is on the root path of row i
    int depth[VIASD_MAX_ROWS_PER_SEQ];
    int first_child[VIASD_MAX_ROWS_PER_SEQ];          // per row: first child node or -1
    int next_sibling[VIASD_MAX_ROWS_PER_SEQ];         // per node: next child of the same parent or -1
    int is_chain;
};

struct DeviceStats {
    unsigned long long steps;
    unsigned long long tier_count[3];
    unsigned long long emitted;
    unsigned long long accepted;
    int device_status;
    int need_slim, need_full;
    int full_ran;                       // the full verifier's pass of the current step ran (its cache holds the block's rows)
    unsigned long long full_skipped;    // steps whose full pass the routed execution policy skipped
};

struct Workspace {                      // pointers into the caller's workspace block
    float *rope_cos, *rope_sin;         // [max_ctx, hd/2]
    float *h;                           // [R, d] residual stream
    // GEMM input activations.  fp32 models: one fp32 plane [R, K].  bf16 models: two bf16 planes
    // [2][R, K], hi = bf16(x) and lo = bf16(x - hi), so that the tensor-core product with the (exact)
    // bf16 weights keeps ~16 mantissa bits of the activation; the planes are R * K elements apart.
    void *a;                            // normed activations, K = d
    float *qkv;                         // [R, (H + 2 Hkv) hd]
    float *q;                           // [R, H hd] rotated queries
    void *attn;                         // attention output, K = H hd
    void *act;                          // SwiGLU output, K = ff
    size_t rows_alloc;                  // R = max_batch * max_query
    float *part;                        // split partial sums (GEMM split-K / attention split-KV)
    size_t part_bytes;
    int *len_eff;                       // [B] committed length clamped to the cache capacity
    int *row_tok;                       // [R] token id per row
    TreeInfo *tree;                     // [max_batch]: every sequence has its own draft tree (copies when the call shares one)
    DeviceStats *stats;
    float *accept_scratch;              // [B, 3, V] sampling-mode distributions, then [3][B, 3, 64] row statistics
    float *gemm_scratch;                // partial tiles of split GEMM work (tcgen05 kernel)
    int *gemm_counters;                 // per-tile arrival counters, zero between launches
    size_t n_counters;
    int *attn_counters;                 // [attn_counter_count()] key-range arrivals per (stream, sequence, kv head, group of query heads)
    float *ssq;                         // [(d / 128) * 4][R] partial sums of h^2 for the fused RMSNorm
    void *a_head; float *ssq_head;      // the block's own rows of `a` and `ssq`, compacted for the output head after a replay pass
};

struct WMap { CUtensorMap map; uint32_t box_rows; };        // TMA view of one weight matrix
struct ActMaps { CUtensorMap map[16]; uint32_t box_rows[16]; }; // TMA views of an activation buffer, NT = 8, 16, ..., 128
struct LayerMaps { WMap wq, wk, wv, wo, wg, wu, wd; };
struct CacheMaps { CUtensorMap k, v; const void *k_ptr, *v_ptr; };   // TMA views of one model's KV cache

// Optional CUDA-event record (measurement only).  A run of consecutive launches of one class shares one pair of
// events, so that the launches inside it keep their programmatic overlap: an event between two kernels would
// serialise them, and what is timed then is not what runs.
struct KernelTimer {
    static constexpr int CAP = 8192;
    cudaEvent_t *beg, *end;
    int *cls, *cnt;                     // class and number of calls of each recorded run
    int n, created, open;               // open: index of the run that has no end event yet, or -1
    long long dropped;
    bool on;
};

// Tuning switches of one model (viasd_set_option; the VIASD_* environment variables give their initial values, read
// once in viasd_init_model).  The defaults are what is measured; tests use them to force every kernel onto every shape.
struct ModelOptions {
    int attn_kernel;        // VIASD_OPT_ATTENTION_KERNEL: 0 choose by shape, 1 mma.sync, 2 tcgen05 rows-on-lanes, 3 tcgen05 keys-on-lanes
    int attn_splits;        // VIASD_OPT_ATTENTION_SPLITS: key ranges per (sequence, kv head); 0 = cost model
    int attn_lo;            // VIASD_OPT_ATTENTION_LO: mma.sync kernel, hi/lo split of Q and P (2), of Q only (1), none (0)
    int accept_team;        // VIASD_OPT_ACCEPT_TEAM: CTAs per sequence in the accept walk; 0 = by mode and vocabulary
    int dual_max_rows;      // VIASD_OPT_DUAL_MAX_ROWS: most rows (both verifiers) the one-sweep schedule takes
    int tk_grid;            // VIASD_OPT_TK_GRID: CTAs of the keys-on-lanes kernel when tiles are dealt evenly; 0 = one per SM
    int tk_flat;            // VIASD_OPT_TK_FLAT: deal tiles (1) or key ranges (0); -1 = by shape
    int ring_kb;            // VIASD_OPT_GEMM_RING_KB: shared-memory ring of the stream-K GEMM
    int epi_groups;         // VIASD_OPT_GEMM_EPI_GROUPS: groups of four epilogue warps; 0 = by token tile
};

struct viasd_model {
    KernelTimer timer;
    ModelOptions opt;
    viasd_config cfg;
    int n_routed;
    int routed[512];                    // routed layer ids, increasing
    const void *embed, *lm_head;
    const float *final_norm;
    const void **wq, **wk, **wv, **wo, **wg, **wu, **wd;   // host arrays [L] of device pointers
    const float **norm1, **norm2;
    Workspace ws;
    int sm_count;
    // tcgen05 GEMM path (bf16 models)
    bool use_tc;
    bool fused;                         // RMSNorm and rotary/append folded into the GEMM epilogues
    LayerMaps *lmaps;                   // [L]
    WMap head_map;
    ActMaps maps_a, maps_attn, maps_act;
    CacheMaps cmaps_full, cmaps_slim;
    ActMaps maps_head;                  // TMA views of the compacted head input (routed execution policy)
    const int *run_flag;                // non-null while the launches of a conditional pass are being enqueued
};

#ifdef __CUDACC__
// Lays out one sequence's draft tree: ancestor sets, depths, child lists.  parent[n] = -1: child of the pending token;
// -2: the node is unused (a sequence with fewer nodes than the call's N): it is nobody's child and nothing attends to it.
__device__ inline void build_tree(TreeInfo *tree, const int *parent, int N, DeviceStats *stats) {
    const int M = N + 1;
    int last_child[VIASD_MAX_ROWS_PER_SEQ];
    for (int i = 0; i < M; ++i) { tree->first_child[i] = -1; tree->next_sibling[i] = -1; last_child[i] = -1; }
    tree->anc[0] = 1ull;
    tree->depth[0] = 0;
    int chain = 1;
    for (int n = 0; n < N; ++n) {
        int p = parent[n];
        const int i = n + 1;
        if (p == -2) { tree->anc[i] = 1ull << i; tree->depth[i] = 0; chain = 0; continue; }
        if (p < -1 || p >= n) { stats->device_status = VIASD_EDEVICE; p = -1; }
        if (p != n - 1) chain = 0;
        const int pr = p + 1;
        tree->anc[i] = tree->anc[pr] | (1ull << i);
        tree->depth[i] = tree->depth[pr] + 1;
        if (last_child[pr] < 0) tree->first_child[pr] = n; else tree->next_sibling[last_child[pr]] = n;
        last_child[pr] = n;
    }
    tree->is_chain = chain;
}

#endif

// error helpers -------------------------------------------------------------------------------
extern int g_last_cuda_error;
extern unsigned long long g_launch_count;
#define CUDA_TRY(expr)                                                     \
    do {                                                                   \
        cudaError_t e__ = (expr);                                          \
        if (e__ != cudaSuccess) { g_last_cuda_error = (int)e__; return VIASD_ECUDA; } \
    } while (0)
#define LAUNCH_CHECK() do { ++g_launch_count; CUDA_TRY(cudaGetLastError()); } while (0)

// cudaFuncSetAttribute applies to the current device only: remembers, per device, whether a launcher has set its
// kernels' attributes there.  Returns true the first time it is asked about (flags, current device).
inline bool first_use_on_device(bool (&flags)[64]) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return true;     // unknown: set them again, which is harmless
    const bool first = !flags[dev];
    flags[dev] = true;
    return first;
}

// Programmatic dependent launch: a kernel launched with this configuration may begin (prologue, weight
// prefetch) while the kernel before it in the stream is still finishing; it must execute griddepcontrol.wait
// before it touches anything that kernel reads or writes.  VIASD_PDL=0 turns the overlap off.
extern int g_use_pdl;
inline void pdl_config(cudaLaunchConfig_t &cfg, cudaLaunchAttribute *attr, dim3 grid, dim3 block, size_t smem,
                       cudaStream_t st) {
    cfg = cudaLaunchConfig_t{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = g_use_pdl ? 1 : 0;
}
// A pass that runs only when a device flag says so (the full verifier's pass under the routed execution policy): every
// kernel of it takes the flag's address and leaves at once when the flag is zero.  The flag is written by a kernel that
// has completed before the pass's first kernel starts (the pass opens with ordinary, fully ordered launches), so
// reading it ahead of the dependency wait is safe.
#define RUN_FLAG_EXIT(ptr) do { if ((ptr) != nullptr && *reinterpret_cast<const volatile int *>(ptr) == 0) return; } while (0)
#define PDL_WAIT() asm volatile("griddepcontrol.wait;" ::: "memory")
#define PDL_TRIGGER() asm volatile("griddepcontrol.launch_dependents;" ::: "memory")

// ---------------------------------------------------------------------------------------------
// kernel launchers (one .cu file each); all enqueue on `st` and return a VIASD_* code
// ---------------------------------------------------------------------------------------------
// misc.cu
int launch_rope_table(const viasd_model *m, cudaStream_t st);
int launch_prep(const viasd_model *m, const viasd_cache *c, const viasd_draft *d, bool full_pass, cudaStream_t st);
int launch_prep_replay(const viasd_model *m, const viasd_cache *c, const viasd_draft *d, int G, cudaStream_t st);
int launch_compact_head_rows(const viasd_model *m, int batch, int M, int G, cudaStream_t st);
int launch_embed(const viasd_model *m, int rows, cudaStream_t st);
int launch_embed_norm(const viasd_model *m, const float *gain, int rows, cudaStream_t st);
int launch_rmsnorm(const viasd_model *m, const float *gain, int rows, cudaStream_t st);
int launch_rope_append(const viasd_model *m, void *kc, void *vc, int layer_ord, int batch, int M,
                       cudaStream_t st);
int launch_commit(const viasd_model *m, viasd_cache *c, const viasd_draft *d, const viasd_result *r, bool slim_only,
                  cudaStream_t st);

// gemm_rowwarp.cu -- generic CUDA-core GEMM (fp32 models; shapes the tensor-core kernels do not take)
enum GemmEpilogue { EPI_STORE = 0, EPI_ADD = 1, EPI_SWIGLU = 2, EPI_ADD_NORM = 3, EPI_QKV_ROPE = 4 };
struct GemmSegs { const void *w[3]; int n[3]; int count; };
// x_plane / act_plane: element distance between the hi and lo planes (0: single plane)
int launch_gemm_rowwarp(const void *x, size_t x_plane, const GemmSegs &segs, int rows, int k, int dtype,
                        int epilogue, float *out_f32, void *out_act, size_t act_plane, int ld_out, cudaStream_t st);

// attention.cu
int launch_attention(viasd_model *m, const void *kc, const void *vc, bool slim, int layer_ord, int batch, int M,
                     cudaStream_t st);
// attention_mma.cu
int attention_mma_supported(const viasd_model *m, int M);
int launch_attention_mma(viasd_model *m, const void *kc, const void *vc, bool slim, int layer_ord, const void *kc2,
                         const void *vc2, int layer_ord2, int streams, int batch, int M, int nsplit, int fuse_merge,
                         cudaStream_t st);
int attention_tc_replicas(int query_rows);
int launch_attention_tc(viasd_model *m, const void *kc, const void *vc, bool slim, int layer_ord, const void *kc2,
                         const void *vc2, int layer_ord2, int streams, int batch, int M, int nsplit, int fuse_merge,
                         cudaStream_t st);
int attention_tk_heads_per_item(int group_heads, int M);
int attention_tk_supported(int group_heads, int M);
int launch_attention_tk(viasd_model *m, const void *kc, const void *vc, bool slim, int layer_ord, const void *kc2,
                         const void *vc2, int layer_ord2, int streams, int batch, int M, int nsplit, int fuse_merge,
                         cudaStream_t st);
int launch_attention_dual(viasd_model *m, const void *kf, const void *vf, int layer_full, const void *ks, const void *vs,
                          int ord_slim, int batch, int M, cudaStream_t st);
int launch_embed_norm2(const viasd_model *m, const float *gain_full, const float *gain_slim, int rows, cudaStream_t st);

// tier_accept.cu
// The verifiers that may judge a drafted token, weakest first, q last (two for the three-tier method), with the
// descending log thresholds that cut the confidence axis into n + 1 tiers.
struct JudgeSet { int n; const float *logits[VIASD_MAX_JUDGES]; float log_tau[VIASD_MAX_JUDGES]; };
int launch_tier(const viasd_model *m, const viasd_draft *d, const viasd_params *p, const JudgeSet &js, viasd_result *r,
                cudaStream_t st);
// probe != null: the walk on the slim verifier's logits alone, deciding whether the full verifier's pass is needed
struct AcceptProbe { int replay_rows; int *need_full; const int *len, *len_full; };
int launch_accept(const viasd_model *m, const viasd_draft *d, const viasd_params *p, const JudgeSet &js, viasd_result *r,
                  bool tree_ready, cudaStream_t st, const AcceptProbe *probe = nullptr);

// ---------------------------------------------------------------------------------------------
// small device helpers
// ---------------------------------------------------------------------------------------------
template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// activation store: fp32 plane, or bf16 hi/lo planes
template <typename T> __device__ __forceinline__ void store_act(T *buf, size_t plane, size_t idx, float v);
template <> __device__ __forceinline__ void store_act<float>(float *buf, size_t, size_t idx, float v) { buf[idx] = v; }
template <> __device__ __forceinline__ void store_act<__nv_bfloat16>(__nv_bfloat16 *buf, size_t plane, size_t idx, float v) {
    __nv_bfloat16 hi = __float2bfloat16_rn(v);
    buf[idx] = hi;
    if (plane) buf[plane + idx] = __float2bfloat16_rn(v - __bfloat162float(hi));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
