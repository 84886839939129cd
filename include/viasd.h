/*
 * viasd.h -- C ABI of the VIA-SD multi-tier verification step for NVIDIA B200 (sm_100a).
 *
 * One decoding cycle of hierarchical speculative verification (Algorithm 1, the body of the
 * while loop; Algorithm 2, lines "run q' in parallel on prefixes" to "append"; Sec. 3.5 steps 3-4):
 *   1. every drafted token is routed to one of three tiers by its confidence relative to the mode of
 *      the gating distribution (App. B, Eq. B.1-B.3): 0 = accept, 1 = slim verifier q', 2 = full
 *      verifier q;
 *   2. q' = Pi_z(q), the routed sub-network of q (Sec. 3.4: layers with z_l = 0 are bypassed; embeddings
 *      and output head are shared), runs on the block against its own KV cache;
 *   3. q runs on the block against its KV cache;
 *   4. the longest accepted prefix and the replacement token are resolved on the device (Sec. 3.5 step 4;
 *      App. A, Eq. A.2-A.3 for the sampling test and the residual distribution);
 *   5. the emitted tokens are committed to both caches; the rest of the block is discarded.
 *
 * Conventions
 *   - Every tensor argument is a DEVICE pointer owned by the caller unless marked "host".  The library
 *     allocates no device memory: scratch comes from the caller's workspace.  It keeps the pointers passed
 *     to viasd_init_model (weights, workspace); they must outlive the handle.
 *   - All work is enqueued on the caller's stream (a cudaStream_t passed as void*); no call synchronises
 *     except viasd_init_model and viasd_get_stats.
 *   - Every function returns 0 (VIASD_OK) or a negative error code; nothing throws, exits or traps.
 *     Conditions only the device can see (a sequence too long for the cache, a token id outside the
 *     vocabulary) are clamped to a safe value and recorded in a device status word that
 *     viasd_get_stats reports.
 *   - A block has N draft nodes and M = N + 1 rows per sequence: row 0 is the pending token (the last
 *     emitted token, whose K/V is not cached yet), row n + 1 is draft node n.  The logits of a row are
 *     the next-token distribution for that row's children.  M <= 64.
 *   - Matrices are row-major [out, in].  dtype 0 = fp32, 1 = bf16 applies to weights and KV caches;
 *     norm gains, logits and the residual stream are fp32.
 */
#ifndef VIASD_H
#define VIASD_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Verifiers that may judge a drafted token in one step: the slim verifiers, weakest first, and the full verifier
 * last.  The method as benchmarked has two (three tiers); Sec. 3.2 and Table 1 go up to five tiers. */
#define VIASD_MAX_JUDGES 4

enum {
    VIASD_OK = 0,
    VIASD_EINVAL = -1,        /* null or misaligned pointer, shape out of range */
    VIASD_ECAPACITY = -2,     /* workspace too small, or (device status) len + M > max_ctx */
    VIASD_ECUDA = -3,         /* a CUDA runtime call failed; see viasd_last_cuda_error() */
    VIASD_EDEVICE = -4,       /* device status word set: bad token id, bad tree, bounded wait expired */
    VIASD_EUNSUPPORTED = -5   /* no CUDA device of compute capability 10.x */
};

typedef struct viasd_model viasd_model; /* opaque */

typedef struct {
    int n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ff, vocab;
    int dtype;                 /* 0 fp32, 1 bf16 */
    float rms_eps;             /* RMSNorm epsilon */
    float rope_theta;          /* rotary base; pairs (p, p + head_dim/2), angle pos * theta^(-2p/head_dim) */
    int max_batch, max_ctx;    /* cache geometry */
    int max_query;             /* largest M the handle will see, <= 64 */
} viasd_config;

typedef struct {
    const void *embed;                 /* [vocab, d_model] */
    const void *lm_head;               /* [vocab, d_model] */
    const float *final_norm;           /* [d_model] */
    /* host arrays of n_layers device pointers */
    const void *const *wq, *const *wk, *const *wv, *const *wo;   /* [H*hd,d] [Hkv*hd,d] [Hkv*hd,d] [d,H*hd] */
    const void *const *wg, *const *wu, *const *wd;               /* [ff,d] [ff,d] [d,ff] */
    const float *const *norm1, *const *norm2;                    /* [d] */
} viasd_weights;

typedef struct {
    void *k_full, *v_full;     /* [n_layers, max_batch, n_kv_heads, max_ctx, head_dim]; K is stored rotated */
    void *k_slim, *v_slim;     /* [n_routed, ...] indexed by the routed layer's ordinal */
    int *len;                  /* [batch] committed length, shared by both caches */
    int *pending;              /* [batch] last emitted token */
    int *tokens;               /* [batch, max_ctx] committed token ids, or NULL */
    int *len_full;             /* [batch] how far the full verifier's cache is complete (<= len), or NULL.  Only the
                                  routed execution policy lets it fall behind len; viasd_kv_commit sets it to the new
                                  len whenever the full verifier's pass ran in the step it commits. */
} viasd_cache;

typedef struct {
    int batch, n_nodes;                /* B, N */
    const int *draft_tok;              /* [B, N] */
    const int *parent;                 /* [N] parent node, -1 = child of the pending token; parents first */
    const int *prow;                   /* [N] drafter-logit row the node was drafted from */
    int n_prows;                       /* R, 1..64 (one drafter row per distinct parent at most) */
    const float *drafter_logits;       /* [B, R, vocab] */
    int per_sequence;                  /* 0: one tree for the whole batch (parent and prow are [N]).  1: every sequence
                                          brings its own tree, which may change from call to call (dynamic drafts):
                                          parent and prow are [B, N]; a sequence that uses fewer than N nodes marks the
                                          others with parent -2 (they are nobody's children; their rows are computed and
                                          ignored).  Sequences are independent, so the result of each is the result of
                                          a batch-of-one call with its tree. */
} viasd_draft;

typedef struct {
    float log_tau_hi, log_tau_lo;      /* log of the relative-confidence thresholds, log_tau_lo <= log_tau_hi */
    int conf_source;                   /* 0: drafter confidence; 1: q' confidence at the parent row (Alg. 2) */
    int mode;                          /* 0 greedy, 1 sampling */
    float temperature;                 /* sampling only; divides verifier and drafter logits */
    float alpha, beta;                 /* Eq. A.2 / A.3; 0 and 1 give the lossless rule */
    float log_acc_rel[3];              /* greedy gate per tier: accept if l[v] - max l >= this; 0 = argmax */
    int strict_break;                  /* 1: an accepted tier-1 token still ends the block (Alg. 2 as printed) */
    int emit_bonus;                    /* 1: when the whole path is accepted, add a token from q at the leaf */
    int policy;                        /* 0: both passes run in every step.  1: routed execution (viasd_verify_step only;
                                          the point of the method, Sec. 1 and Eq. B.20): q' runs in every step, q only when
                                          the walk reaches a tier-2 node before the first break or a bonus token is due.  A
                                          skipped pass leaves q's cache short of the emitted tokens; the next pass of q
                                          replays the last G = max_query - (n_nodes + 1) committed tokens in front of the
                                          block, so a pass is skipped only while the backlog fits G, and every sequence
                                          must hold at least G committed tokens.  Needs cache.tokens and cache.len_full, a
                                          bf16 model with head_dim 128, and max_query > n_nodes + 1.  Emitted tokens are
                                          those of policy 0; full_logits is left untouched by a step that skips q. */
    unsigned long long seed, step;     /* counter-based random numbers for sampling mode */
} viasd_params;

typedef struct {
    unsigned char *tier;               /* [B, N] */
    float *conf;                       /* [B, N] log relative confidence d = l[v] - max l */
    int *n_acc;                        /* [B] kappa: accepted draft nodes */
    int *path;                         /* [B, N] accepted node ids, first n_acc valid */
    int *out_tok;                      /* [B, N+1] emitted tokens, first n_emit valid */
    int *n_emit;                       /* [B] */
    unsigned char *judge;              /* [B, N] 0 untouched, 1 accepted, 2 rejected, | judging tier << 4 */
    int *corr_src;                     /* [B] who emitted the last token: 0 nobody, 1 q', 2 q */
} viasd_result;

typedef struct {
    unsigned long long steps;          /* verify steps / tier passes since init */
    unsigned long long tier_count[3];  /* histogram of tiers: empirical region masses of Eq. B.4-B.6 */
    unsigned long long emitted;        /* tokens emitted by accept passes */
    unsigned long long accepted;       /* draft nodes accepted */
    int device_status;                 /* 0 or a VIASD_E* code recorded by a kernel */
    int need_slim, need_full;          /* last tier pass: any node in tier 1 / tier 2 */
    int full_ran;                      /* 1 if the full verifier's pass of the last step ran (always, under policy 0) */
    unsigned long long full_skipped;   /* committed steps whose full pass the routed execution policy skipped */
} viasd_stats;

/* Bytes of workspace viasd_init_model needs for this geometry. */
size_t viasd_workspace_bytes(const viasd_config *cfg, int n_routed);

/* Build a handle.  route_mask: host, [n_layers], the routing mask z (1 = layer kept by q').
 * workspace: device, 256-byte aligned, at least viasd_workspace_bytes().  Synchronises the device once
 * (it fills the rotary table).  Errors: EINVAL, ECAPACITY, ECUDA, EUNSUPPORTED. */
int viasd_init_model(const viasd_config *cfg, const viasd_weights *w, const unsigned char *route_mask,
                     void *workspace, size_t workspace_bytes, viasd_model **out);

/* Forward pass of q (all layers) / q' (routed layers) over the block: logits [B, M, vocab] fp32.
 * K/V of the M rows are written at slots len[b] .. len[b]+M-1 of the model's cache; len is not changed,
 * so the rows stay invisible until viasd_kv_commit.  (Algorithm 2, parallel block verification.) */
int viasd_full_forward(viasd_model *m, const viasd_cache *cache, const viasd_draft *draft, float *logits,
                       void *stream);
int viasd_slim_forward(viasd_model *m, const viasd_cache *cache, const viasd_draft *draft, float *logits,
                       void *stream);

/* phase 1: tier routing only (Eq. B.1-B.3) -> result.tier, result.conf.
 * phase 2: accept / resolve only (reads result.tier) -> n_acc, path, out_tok, n_emit, judge, corr_src.
 * phase 3: both.  slim_logits / full_logits [B, M, vocab]; phase 1 needs slim_logits only when
 * conf_source = 1. */
int viasd_tier_accept(viasd_model *m, const viasd_draft *draft, const viasd_params *params,
                      const float *slim_logits, const float *full_logits, int phase, viasd_result *result,
                      void *stream);

/* The tiered rule with more than one slim verifier (the n-tier remark of Sec. 3.2; Table 1): n_judges verifiers
 * u_1 ... u_n = q, each a routed sub-network of the next (its own handle with its own mask, workspace and slim cache
 * over the same weights; its logits come from viasd_slim_forward on that handle, q's from viasd_full_forward).
 * log_tau: host, [n_judges], descending: tier 0 (accepted outright) from log_tau[0] up, tier k (judged by verifier
 * k, counted from 1) between log_tau[k] and log_tau[k-1], tier n_judges (judged by q) below log_tau[n_judges-1].
 * judge_logits: host array of n_judges device pointers [B, M, vocab], weakest verifier first.  conf_source 1 gates
 * with the weakest verifier's confidence.  The walk is that of viasd_tier_accept: a tier-k child is judged by
 * verifier k (greedy: log_acc_rel[1] for the slim verifiers, [2] for q; sampling: Eq. A.2 / A.3 with that verifier as
 * the judge), the strongest judge that rejected emits the replacement; result.corr_src and the tier bits of
 * result.judge run from 1 to n_judges.  With n_judges = 2 this is viasd_tier_accept with log_tau = (hi, lo).
 * params.log_tau_hi / log_tau_lo are ignored.  Phases and errors as viasd_tier_accept.
 * Committing an n-tier step: viasd_kv_commit_slim on every slim verifier's handle but one, then viasd_kv_commit on
 * the remaining handle (it also moves q's rows and advances len, pending and tokens, which the handles share). */
int viasd_tier_accept_n(viasd_model *m, const viasd_draft *draft, const viasd_params *params, int n_judges,
                        const float *log_tau, const float *const *judge_logits, int phase, viasd_result *result,
                        void *stream);
/* Moves the accepted path's rows in this handle's slim cache only (no length changes): see viasd_tier_accept_n. */
int viasd_kv_commit_slim(viasd_model *m, viasd_cache *cache, const viasd_draft *draft, const viasd_result *result,
                         void *stream);

/* Commit (Algorithm 1, the lines after the prefix is chosen: append the accepted prefix and the regenerated
 * token, discard the remaining suffix, advance t; Sec. 3.5 step 4): move the accepted path's K/V rows to
 * slots len+1.., len += n_emit, pending = last emitted token, committed ids appended to cache.tokens.
 * Rejected rows are left beyond len: rollback is not keeping them. */
int viasd_kv_commit(viasd_model *m, viasd_cache *cache, const viasd_draft *draft, const viasd_result *result,
                    void *stream);

/* tier -> slim forward -> full forward -> accept -> commit, identical to calling the pieces (one decoding
 * cycle: Algorithm 1, body of the loop; Algorithm 2 from the parallel run of q' to the append).
 * slim_logits / full_logits: caller's buffers [B, M, vocab], filled as a side effect; both are required (the
 * workspace holds no logits: at the largest geometries they would be over a gigabyte). */
int viasd_verify_step(viasd_model *m, viasd_cache *cache, const viasd_draft *draft, const viasd_params *params,
                      float *slim_logits, float *full_logits, viasd_result *result, void *stream);

/* Copies the device counters out; synchronises `stream`. */
int viasd_get_stats(viasd_model *m, viasd_stats *host_out, void *stream);

/* Tuning switches of one handle (the paper has no counterpart).  The defaults are what the benchmark measures; the
 * tests use the switches to force every kernel onto every shape.  Takes effect from the next call on; results stay
 * within the stated tolerances under every setting, but their last bits may change with it.
 * Errors: EINVAL (null handle, unknown option, value out of range). */
enum {
    VIASD_OPT_ATTENTION_KERNEL = 0,    /* 0 choose by shape (default), 1 mma.sync, 2 tcgen05 with query rows on the
                                          TMEM lanes, 3 tcgen05 with keys on the lanes (where the shape allows) */
    VIASD_OPT_ATTENTION_SPLITS,        /* key ranges per (sequence, kv head), 1..16; 0 = cost model (default) */
    VIASD_OPT_ATTENTION_LO,            /* mma.sync kernel: hi/lo split of queries and probabilities 2 (default),
                                          queries only 1, neither 0 (fails the logit tolerance at full size) */
    VIASD_OPT_ACCEPT_TEAM,             /* CTAs per sequence in the accept walk: 1, 2, 4, 8; 0 = by mode and vocabulary (1 for
                                          greedy; sampling: 8 from 16384 tokens on, 16 from 65536 on where the device
                                          takes clusters of 16) */
    VIASD_OPT_DUAL_MAX_ROWS,           /* most token rows (both verifiers together) that viasd_verify_step runs as one
                                          sweep over the layers, 0..128 (default 128); above it the passes run in turn */
    VIASD_OPT_TK_GRID,                 /* keys-on-lanes attention with tiles dealt evenly: CTAs to use; 0 = one per SM */
    VIASD_OPT_TK_FLAT,                 /* keys-on-lanes attention: deal tiles 1, key ranges 0; -1 = by shape (default) */
    VIASD_OPT_GEMM_RING_KB,            /* stream-K GEMM: shared-memory ring in KB, 32..200; 0 = default (200) */
    VIASD_OPT_GEMM_EPI_GROUPS          /* stream-K GEMM: groups of four epilogue warps, 1 or 2; 0 = by token tile */
};
int viasd_set_option(viasd_model *m, int option, int value);

void viasd_free_model(viasd_model *m);
const char *viasd_strerror(int code);
int viasd_last_cuda_error(void);

/* One projection of the decoder block on its own: y[rows, n] = x[rows, k] * W[n, k]^T (the contraction
 * every layer of q and q' is made of, Sec. 3.4).  dtype as in viasd_config (x and W share it: fp32, or
 * bf16 with fp32 accumulation); y is fp32.  scratch: device, scratch_bytes >= viasd_gemm_scratch_bytes(),
 * used for split-K partial sums.  rows <= 256. */
size_t viasd_gemm_scratch_bytes(int rows, int n, int k);
int viasd_gemm(const void *x, const void *w, float *y, int rows, int n, int k, int dtype, void *scratch,
               size_t scratch_bytes, void *stream);
/* The calls above are asynchronous, so a device-side failure (a bounded wait of the kernel that expired) cannot come
 * back as their return value: it is recorded in a status word inside the scratch.  This reads it: *host_out =
 * VIASD_OK or VIASD_EDEVICE for the last viasd_gemm call that used `scratch` with this n (bf16 only; the fp32 kernel
 * has no waits).  Synchronises `stream`. */
int viasd_gemm_status(const void *scratch, int n, int *host_out, void *stream);

/* Same product as viasd_gemm for bf16 operands (y[rows, n] = x[rows, k] * W[n, k]^T, fp32 y) for callers that
 * cannot allocate device memory and therefore have no scratch to hand over: a serving process that gave all
 * of its HBM to weights and KV caches at start-up (a later cudaMalloc fails, or stalls every stream of the
 * device while it runs), or code running inside a host framework's callback where allocation calls are
 * forbidden.  The paper has no counterpart; this is plumbing.
 * The scratch (tile counters and partial tiles, about 2.6 MB) is a fixed array inside the library image: every
 * GPU that loads the library holds it until the process exits.  Limits: rows <= 16 and n <= 262144; larger
 * sizes return VIASD_ECAPACITY and launch nothing.  The call makes no cudaMalloc / cudaFree and uses no
 * allocating library routine.
 * The first call on each device looks up the array's device address (with that device current); make that
 * first call before starting any stream capture on the device.
 * All calls on a device share the one array: the counters are cleared at the start of every call, the rest
 * keeps the previous call's contents and is overwritten.  Two calls that overlap on the GPU (different
 * streams, or different host threads) race on it and give wrong results; serialise them.
 * Errors: EINVAL (null / misaligned pointer, k not a multiple of 8), ECAPACITY, ECUDA, EUNSUPPORTED. */
int viasd_gemm_static(const void *x, const void *w, float *y, int rows, int n, int k, void *stream);
/* Status of the last viasd_gemm_static call on the current device: *host_out = VIASD_OK, or VIASD_EDEVICE when a
 * bounded wait of its kernel expired (y is then incomplete).  Synchronises `stream`; allocates nothing. */
int viasd_gemm_static_status(int *host_out, void *stream);

/* KL-style verification cost of a judge distribution against a proposal, per row (Eq. 11), and its sum over the
 * rows given (block cost, Eq. 10).  With q = softmax(judge_logits / temperature), p = softmax(proposal_logits /
 * temperature), z1 = log(1 - alpha) + log p - log q, z2 = log(beta) + log p - log q:
 *     cost_rows[r] = sum_v p(v) phi(z1(v)) + sum_v q(v) phi(z2(v))
 * margin 0: phi(z) = max(0, z) (Eq. 11); margin 1: phi(z) = tau log(1 + exp(z / tau)) (App. F), which lies
 * between the margin-0 value and that value plus 2 tau log 2 (F.8).  The cost of a layer mask z over a window of
 * decoding steps (Eq. 12) is this call with the full verifier's logits as judge and the slim verifier's as
 * proposal; the gain of the routed path over the direct one (Sec. 2.2) is cost(q, p) - cost(u, p) - cost(q, u).
 * judge_logits, proposal_logits: device, fp32 [rows, vocab] row-major, read only.  cost_rows: device, [rows],
 * written.  cost_total: device, one float, written with the sum of cost_rows in row order; may be NULL.
 * Asynchronous on `stream`; allocates nothing.  Errors: EINVAL (null pointer, rows or vocab < 1, temperature <= 0,
 * alpha outside [0, 1), beta <= 0, unknown margin, tau <= 0 with margin 1), ECUDA. */
int viasd_kl_cost(const float *judge_logits, const float *proposal_logits, int rows, int vocab, float temperature,
                  float alpha, float beta, int margin, float tau, float *cost_rows, float *cost_total, void *stream);

/* Region masses (Eq. B.8-B.10; regions of Eq. B.1-B.3): per row, how much of the proposal distribution
 * p = softmax(proposal_logits / temperature) lies on the tokens that the gating row places in region A (accepted
 * outright), B (left to the slim verifier) and C (escalated to the full verifier):
 *     mass[r][0] = delta_p     = sum_u p(u) [d(u) >= log_tau_hi]
 *     mass[r][1] = delta_1-bar = sum_u p(u) [log_tau_lo <= d(u) < log_tau_hi]
 *     mass[r][2] = delta_2     = sum_u p(u) [d(u) < log_tau_lo],        d(u) = gate_logits[r][u] - max_w gate_logits[r][w]
 * with d taken in fp32 exactly as the tier step takes it for a drafted token, so these are the probabilities, under
 * v ~ p, of the three tiers (Eq. B.4-B.6) and the weights of the output mixture of Eq. B.7.
 * gate_logits, proposal_logits: device, fp32 [rows, vocab] row-major, read only.  mass: device, [rows, 3], written.
 * mean: device, 3 floats, written with the mean of the rows in row order; may be NULL.  Asynchronous on `stream`;
 * allocates nothing.  Errors: EINVAL (null pointer, rows or vocab < 1, temperature <= 0, log_tau_lo > log_tau_hi), ECUDA. */
int viasd_region_mass(const float *gate_logits, const float *proposal_logits, int rows, int vocab, float temperature,
                      float log_tau_hi, float log_tau_lo, float *mass, float *mean, void *stream);

/* Self-test of the failure path (the paper has no counterpart).  Every wait inside the kernels of this library - on a
 * TMA arrival, on a tensor-core commit, on another CTA's partial results - is bounded: when its limit expires the
 * waiting kernel records VIASD_EDEVICE in a status word and returns by itself, so that the context stays usable and
 * the next viasd_get_stats reports the failure.  Ordinary runs never take that path; this hook does, harmlessly: it
 * launches one CTA that waits, through the same routine with a limit of limit_us microseconds (1..100000), on a
 * barrier nothing arrives at.
 * status: device, one int, written with VIASD_EDEVICE when the wait has expired.  waited_cycles: device, one 64-bit
 * integer or NULL, written with the SM cycles the wait lasted (-1 if it did not expire).  Asynchronous on `stream`.
 * Errors: EINVAL, ECUDA. */
int viasd_selftest_wait_expiry(int *status, int limit_us, long long *waited_cycles, void *stream);

/* Measurement hooks (the paper has no counterpart; they exist so that a benchmark can attribute time).
 * viasd_launch_count: kernels launched by this library in this process so far.
 * viasd_set_timing(on): when on, every run of consecutive launches of one kernel class in the forward / tier /
 * accept / commit path is bracketed by one pair of CUDA events on the caller's stream (the launches inside a run
 * keep their programmatic overlap; a few thousand runs are kept, later ones are dropped).
 * viasd_get_timing: synchronises `stream`, sums the recorded intervals per kernel class into `out`
 * (VIASD_T_COUNT entries each) and clears the record. */
enum { VIASD_T_GEMM = 0, VIASD_T_ATTENTION, VIASD_T_NORM, VIASD_T_ROPE, VIASD_T_EMBED, VIASD_T_TIER_ACCEPT,
       VIASD_T_COMMIT, VIASD_T_COUNT };
typedef struct { double ms[VIASD_T_COUNT]; long long launches[VIASD_T_COUNT]; long long dropped; } viasd_timing;
unsigned long long viasd_launch_count(void);
int viasd_set_timing(viasd_model *m, int on);
int viasd_get_timing(viasd_model *m, viasd_timing *out, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* VIASD_H */
