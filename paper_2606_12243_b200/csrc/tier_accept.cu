// Fused confidence-tier kernel and accept / resolve kernel.
//
// Tier kernel (App. B, Eq. B.1-B.3): per drafted token v, d = l[v] - max_u l[u] on the gating logits;
// tier 0 if d >= log_tau_hi, 1 if d >= log_tau_lo, else 2.  One CTA per gating row scans the
// vocabulary once and serves every node gated by that row.
//
// Accept kernel (Algorithm 2, per-position loop; Algorithm 1, what is appended; App. A, Eq. A.2-A.3):
// one CTA per sequence (a cluster of eight when it samples over a large vocabulary) walks the draft from the pending token: children of the current row are tried in
// index order; tier-0 children are taken at once, tier-1 children are judged by q', tier-2 children by
// q.  The first row where no child passes ends the walk and the strongest judge that rejected there
// emits the replacement token.  The walk is sequential over depth, so everything that can be known before
// it is: a row-statistics kernel (one CTA per logits row, all rows at once) leaves each row's maximum,
// argmax and softmax denominator, which makes every first test at a position O(1).  Only a rejection in
// sampling mode (residual, Eq. A.3: two sweeps) and the final draw still sweep the vocabulary inside the walk;
// the CTAs of a cluster share each sweep and combine their block results through distributed shared memory in rank
// order, so all of them hold the same values and walk the same way.
#include "common.cuh"
#include <string.h>
#include <stdlib.h>

namespace {

constexpr int ACC_THREADS = 512;
constexpr int MAXJ = VIASD_MAX_JUDGES;    // verifiers that may judge a drafted token (the last one is q); 2 for three tiers
constexpr int KINDS = MAXJ + 1;           // distributions kept per position: the proposal and the judges
constexpr int ACC_TEAM = 8;               // CTAs per sequence in sampling mode (a portable cluster size)

// ---- counter-based uniforms -------------------------------------------------------------------
__device__ __forceinline__ unsigned long long mix64(unsigned long long z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
constexpr unsigned long long GAMMA = 0x9E3779B97F4A7C15ull;
__device__ __forceinline__ unsigned long long stream_key(unsigned long long seed, unsigned long long step, int b,
                                                         int stream) {
    unsigned long long k = mix64(seed + GAMMA);
    k = mix64(k + step * GAMMA + 1ull);
    return mix64(k + (unsigned long long)(b * 256 + stream) * GAMMA + 2ull);
}
// 23 random bits -> (k + 0.5) / 2^23: exact in fp32, strictly inside (0, 1)
__device__ __forceinline__ float unit_f32(unsigned long long key, unsigned long long idx) {
    unsigned long long w = mix64(key + idx * GAMMA + 3ull);
    return ((float)(w >> 41) + 0.5f) * 1.1920928955078125e-7f;
}

// ---- block reductions ---------------------------------------------------------------------------
struct MaxIdx { float v; int i; };
__device__ __forceinline__ MaxIdx better(MaxIdx a, MaxIdx b) {   // larger value, lowest index on ties
    if (b.v > a.v || (b.v == a.v && b.i < a.i)) return b;
    return a;
}
__device__ MaxIdx block_argmax(MaxIdx x, MaxIdx *sh) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        MaxIdx y;
        y.v = __shfl_xor_sync(0xffffffffu, x.v, o);
        y.i = __shfl_xor_sync(0xffffffffu, x.i, o);
        x = better(x, y);
    }
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = x;
    __syncthreads();
    MaxIdx r = sh[0];
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w) r = better(r, sh[w]);
    return r;
}
__device__ float block_sum(float x, float *sh) {
    x = warp_sum(x);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = x;
    __syncthreads();
    float r = 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) r += sh[w];
    return r;
}
__device__ float block_max(float x, float *sh) {
    x = warp_max(x);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = x;
    __syncthreads();
    float r = sh[0];
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w) r = fmaxf(r, sh[w]);
    return r;
}

// ---- tier kernel ------------------------------------------------------------------------------
// n thresholds in descending order cut the log-confidence axis into n + 1 tiers: tier 0 (accepted outright) from
// log_tau[0] up, tier k between log_tau[k] and log_tau[k - 1], tier n (the full verifier) below log_tau[n - 1].
struct TierCuts { int n; float log_tau[MAXJ]; };
// grid (gate rows per sequence, B).  conf_source 0: gate row of node n = prow[n], rows = drafter logits
// [B, R, V]; conf_source 1: gate row = parent[n] + 1, rows = slim logits [B, M, V].
__global__ void __launch_bounds__(1024)
tier_kernel(unsigned char *__restrict__ tier, float *__restrict__ conf, DeviceStats *stats,
            const float *__restrict__ gate_logits, const int *__restrict__ draft_tok, const int *__restrict__ prow,
            const int *__restrict__ parent, int per_seq, int conf_source, int rows_per_seq, int N, int V, TierCuts cuts) {
    __shared__ float sh[32];
    const int gr = blockIdx.x, b = blockIdx.y;
    if (per_seq) { prow += (size_t)b * N; parent += (size_t)b * N; }     // every sequence has its own tree
    const float *row = gate_logits + ((size_t)b * rows_per_seq + gr) * V;
    float mx = -INFINITY;
    if ((V & 3) == 0 && ((uintptr_t)row & 15) == 0) {
        const float4 *r4 = reinterpret_cast<const float4 *>(row);
        for (int i = threadIdx.x; i < V / 4; i += blockDim.x) {
            float4 v = r4[i];
            mx = fmaxf(mx, fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w)));
        }
    } else {
        for (int i = threadIdx.x; i < V; i += blockDim.x) mx = fmaxf(mx, row[i]);
    }
    mx = block_max(mx, sh);
    for (int n = threadIdx.x; n < N; n += blockDim.x) {
        if (parent[n] == -2) {                                   // unused node of this sequence's tree
            if (gr == 0) { tier[b * N + n] = 0; conf[b * N + n] = 0.f; }
            continue;
        }
        int g = conf_source == 0 ? prow[n] : parent[n] + 1;
        if (g != gr) continue;
        int t = draft_tok[b * N + n];
        t = min(max(t, 0), V - 1);
        float d = row[t] - mx;
        int tr = 0;                                              // thresholds descend: the first one d reaches names the tier
        while (tr < cuts.n && d < cuts.log_tau[tr]) ++tr;
        tier[b * N + n] = (unsigned char)tr;
        conf[b * N + n] = d;
        atomicAdd(&stats->tier_count[tr == 0 ? 0 : (tr == cuts.n ? 2 : 1)], 1ull);   // accepted / some slim verifier / q
        if (tr > 0 && tr < cuts.n) stats->need_slim = 1;
        if (tr == cuts.n) stats->need_full = 1;
    }
    if (gr == 0 && b == 0 && threadIdx.x == 0) atomicAdd(&stats->steps, 1ull);
}

// ---- row statistics ---------------------------------------------------------------------------
// grid (rows, B, 1 + judges): kind 0 = drafter rows [B, R, V], kind k = judge k's rows [B, M, V] (the last judge is q).
// Per row: max, argmax (lowest index on ties) and, when want_z, sum exp((l - max) / T).
constexpr int RS_STRIDE = VIASD_MAX_ROWS_PER_SEQ;
struct RowStats { float *mx; int *arg; float *z; };       // each [B, KINDS, RS_STRIDE]
struct RowPtrs { const float *p[KINDS]; };                // drafter logits, then each judge's

__global__ void __launch_bounds__(1024)
row_stats_kernel(RowStats rs, RowPtrs src, int R, int M, int V, float inv_temp, int want_z) {
    __shared__ float sh[32];
    __shared__ MaxIdx shm[32];
    const int kind = blockIdx.z, b = blockIdx.y, r = blockIdx.x;
    const float *base = src.p[kind];
    const int rows = kind == 0 ? R : M;
    if (!base || r >= rows) return;
    const float *row = base + ((size_t)b * rows + r) * V;
    const bool vec = (V & 3) == 0 && ((uintptr_t)row & 15) == 0;
    MaxIdx best; best.v = -INFINITY; best.i = 0x7fffffff;
    if (vec) {
        const float4 *r4 = reinterpret_cast<const float4 *>(row);
        for (int i = threadIdx.x; i < V / 4; i += blockDim.x) {
            const float4 v = r4[i];
            MaxIdx c;
            c.v = v.x; c.i = 4 * i; best = better(best, c);
            c.v = v.y; c.i = 4 * i + 1; best = better(best, c);
            c.v = v.z; c.i = 4 * i + 2; best = better(best, c);
            c.v = v.w; c.i = 4 * i + 3; best = better(best, c);
        }
    } else {
        for (int i = threadIdx.x; i < V; i += blockDim.x) { MaxIdx c; c.v = row[i]; c.i = i; best = better(best, c); }
    }
    best = block_argmax(best, shm);
    float z = 0.f;
    if (want_z) {
        const float mx = best.v;
        if (vec) {
            const float4 *r4 = reinterpret_cast<const float4 *>(row);
            for (int i = threadIdx.x; i < V / 4; i += blockDim.x) {
                const float4 v = r4[i];
                z += expf((v.x - mx) * inv_temp) + expf((v.y - mx) * inv_temp) + expf((v.z - mx) * inv_temp) +
                     expf((v.w - mx) * inv_temp);
            }
        } else {
            for (int i = threadIdx.x; i < V; i += blockDim.x) z += expf((row[i] - mx) * inv_temp);
        }
        z = block_sum(z, sh);
    }
    if (threadIdx.x == 0) {
        const size_t o = ((size_t)b * KINDS + kind) * RS_STRIDE + r;
        rs.mx[o] = best.v;
        rs.arg[o] = best.i == 0x7fffffff ? 0 : best.i;
        rs.z[o] = z;
    }
}

// ---- accept kernel ----------------------------------------------------------------------------
struct AcceptArgs {
    RowStats rs;
    const float *judges[KINDS];              // [1..n_judges]: each judge's logits [B, M, V], weakest first, q last
    const float *drafter;                    // [B, R, V]
    int n_judges;
    const int *draft_tok, *prow;             // [B, N], [N]
    const unsigned char *tier;               // [B, N]
    const TreeInfo *tree;
    float *scratch;                          // [B, KINDS, V]
    int *n_acc, *path, *out_tok, *n_emit, *corr_src;
    unsigned char *judge;
    DeviceStats *stats;
    int N, R, V;
    int mode, strict_break, emit_bonus;
    float inv_temp, log1m_alpha, inv_beta;
    float log_acc_rel[KINDS];                // greedy gate per judging tier
    unsigned long long seed, step;
    // Probe (routed execution policy): the same walk on the slim verifier's logits alone.  It stops where the full
    // verifier's judgment (a tier-2 node, or the bonus token at a leaf) would be needed and raises *need_full; it also
    // raises it when a sequence's backlog (len - len_full) plus this step's tokens would outgrow the replay window.
    // Writes no result.
    int per_seq;                             // prow is [B, N] and every sequence has its own tree
    int probe, replay_rows;
    int *need_full;
    const int *len, *len_full;
};

// ---- the CTAs of a sequence (a thread-block cluster in sampling mode, else one CTA) ---------------------
// Each CTA sweeps its share of the vocabulary (indices strided by CTAs x threads); block results are combined through
// distributed shared memory in rank order, so every CTA holds the same value and takes the same branches.
struct Team {
    unsigned rank, size;
    float *slot_f;              // [2] own slots, double-buffered by phase
    MaxIdx *slot_m;             // [2]
    int phase;
};
__device__ __forceinline__ void team_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t remote_addr(const void *own, unsigned rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"((uint32_t)__cvta_generic_to_shared(own)), "r"(rank));
    return r;
}
__device__ float team_sum(float x, float *sh, Team &tm) {
    x = block_sum(x, sh);
    if (tm.size == 1) return x;
    float *slot = tm.slot_f + (tm.phase & 1);
    if (threadIdx.x == 0) *slot = x;
    team_barrier();
    float r = 0.f;
    for (unsigned k = 0; k < tm.size; ++k) {
        float v;
        asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote_addr(slot, k)));
        r += v;
    }
    ++tm.phase;
    return r;
}
__device__ MaxIdx team_argmax(MaxIdx x, MaxIdx *shm, Team &tm) {
    x = block_argmax(x, shm);
    if (tm.size == 1) return x;
    MaxIdx *slot = tm.slot_m + (tm.phase & 1);
    if (threadIdx.x == 0) *slot = x;
    team_barrier();
    MaxIdx r; r.v = -INFINITY; r.i = 0x7fffffff;
    for (unsigned k = 0; k < tm.size; ++k) {
        MaxIdx y;
        const uint32_t ra = remote_addr(slot, k);
        asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(y.v) : "r"(ra));
        asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(y.i) : "r"(ra + 4));
        r = better(r, y);
    }
    ++tm.phase;
    return r;
}

// numerators of softmax(l / T) into dst (the row maximum comes from the row statistics); this CTA's share
__device__ void softmax_numerators(float *dst, const float *row, int V, float inv_temp, float mx, const Team &tm) {
    for (int i = tm.rank * blockDim.x + threadIdx.x; i < V; i += tm.size * blockDim.x) dst[i] = expf((row[i] - mx) * inv_temp);
    __syncthreads();
}

// argmax_v (log w[v] - log(-log u_v)): a draw from w / sum(w)
__device__ int gumbel_argmax(const float *w, int V, unsigned long long key, int row, MaxIdx *shm, Team &tm) {
    MaxIdx best; best.v = -INFINITY; best.i = 0x7fffffff;
    for (int i = tm.rank * blockDim.x + threadIdx.x; i < V; i += tm.size * blockDim.x) {
        float wi = w[i];
        if (wi > 0.f) {
            float u = unit_f32(key, ((unsigned long long)row << 32) + (unsigned long long)i);
            MaxIdx c; c.v = logf(wi) - logf(-logf(u)); c.i = i;
            best = better(best, c);
        }
    }
    best = team_argmax(best, shm, tm);
    return best.i == 0x7fffffff ? 0 : best.i;
}

__global__ void __launch_bounds__(ACC_THREADS)
accept_kernel(AcceptArgs a) {
    __shared__ MaxIdx shm[32];
    __shared__ float sh[32];
    __shared__ float slot_f[2];
    __shared__ MaxIdx slot_m[2];
    Team tm;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(tm.rank));
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(tm.size));
    tm.slot_f = slot_f; tm.slot_m = slot_m; tm.phase = 0;
    const bool lead = tm.rank == 0 && threadIdx.x == 0;       // the one thread that writes the results
    const int b = blockIdx.x / tm.size, N = a.N, M = N + 1, V = a.V;
    const TreeInfo *tree = a.tree + b;
    const int *prow = a.prow + (a.per_seq ? (size_t)b * N : 0);
    const bool sampling = a.mode == 1;
    const int J = a.n_judges;                                 // tier J is the full verifier's
    float *P[KINDS];
#pragma unroll
    for (int k = 0; k < KINDS; ++k) P[k] = a.scratch + ((size_t)b * KINDS + k) * V;
    const float *st_mx = a.rs.mx + (size_t)b * KINDS * RS_STRIDE, *st_z = a.rs.z + (size_t)b * KINDS * RS_STRIDE;
    const int *st_arg = a.rs.arg + (size_t)b * KINDS * RS_STRIDE;
    const unsigned long long k_acc = stream_key(a.seed, a.step, b, 0), k_gum = stream_key(a.seed, a.step, b, 1);
    if (tm.rank == 0 && !a.probe) for (int n = threadIdx.x; n < N; n += blockDim.x) a.judge[b * N + n] = 0;
    __syncthreads();

    int cur = 0, n_acc = 0, corr = -1, corr_src = 0;
    bool needs_q = false;
    while (true) {
        int c = tree->first_child[cur];
        if (c < 0) {                                             // leaf: whole path accepted
            if (a.emit_bonus && a.probe) { needs_q = true; break; }
            if (a.emit_bonus) {
                if (sampling) {
                    softmax_numerators(P[J], a.judges[J] + ((size_t)b * M + cur) * V, V, a.inv_temp, st_mx[J * RS_STRIDE + cur], tm);
                    corr = gumbel_argmax(P[J], V, k_gum, cur, shm, tm);
                } else {
                    corr = st_arg[J * RS_STRIDE + cur];
                }
                corr_src = J;
            }
            break;
        }
        // the distributions of this position: 0 = proposal (drafter row), k = judge k (the slim verifiers, then q).  Each
        // starts as "row + statistics" and is written out as numerators (mat) only once a residual has to be formed.
        const float *row[KINDS];
        float mx[KINDS], Z[KINDS];
        bool mat[KINDS];
        row[0] = nullptr; mx[0] = 0.f; Z[0] = 0.f; mat[0] = false;
#pragma unroll
        for (int k = 1; k < KINDS; ++k) {
            const bool on = k <= J && a.judges[k] != nullptr;
            row[k] = on ? a.judges[k] + ((size_t)b * M + cur) * V : nullptr;
            mx[k] = on ? st_mx[k * RS_STRIDE + cur] : 0.f;
            Z[k] = on ? st_z[k * RS_STRIDE + cur] : 0.f;
            mat[k] = false;
        }
        int failed = 0, taken = -1, taken_tier = 0;
        for (; c >= 0; c = tree->next_sibling[c]) {
            const int t = min((int)a.tier[b * N + c], J);
            int v = a.draft_tok[b * N + c];
            v = min(max(v, 0), V - 1);
            if (t == 0) {
                taken = c; taken_tier = 0;
                if (lead && !a.probe) a.judge[b * N + c] = 1;
                break;
            }
            if (t == J && a.probe) { needs_q = true; break; }     // from here on the walk depends on q
            bool pass;
            if (!sampling) {
                pass = (row[t][v] - mx[t]) >= a.log_acc_rel[t];
            } else {
                if (!row[0]) {
                    const int pr = prow[c];
                    row[0] = a.drafter + ((size_t)b * a.R + pr) * V;
                    mx[0] = st_mx[pr];
                    Z[0] = st_z[pr];
                }
                const float u = unit_f32(k_acc, (unsigned long long)c);
                const float pv = mat[0] ? __ldcg(&P[0][v]) : expf((row[0][v] - mx[0]) * a.inv_temp);
                const float jv = mat[t] ? __ldcg(&P[t][v]) : expf((row[t][v] - mx[t]) * a.inv_temp);
                const float lp = logf(pv / Z[0]);
                const float lj = logf(jv / Z[t]);
                pass = (logf(u) + a.log1m_alpha + lp) < lj;       // u < j(v) / ((1 - alpha) p(v)), Eq. A.2
            }
            if (pass) {
                taken = c; taken_tier = t;
                if (lead && !a.probe) a.judge[b * N + c] = (unsigned char)(1 | (t << 4));
                break;
            }
            if (lead && !a.probe) a.judge[b * N + c] = (unsigned char)(2 | (t << 4));
            failed = max(failed, t);
            if (sampling) {
                // Eq. A.3 round by round: the rejecting judge becomes its residual against the proposal (kept as is if
                // the residual vanishes); the rejected token leaves the proposal.  Two sweeps of the vocabulary: the
                // residual's mass, then both distributions written out (from the logits the first time at a position).
                __syncthreads();                                  // every thread has read P[.][v] above
                const float sj = a.inv_beta / Z[t], sp = 1.f / Z[0];
                const bool mt = mat[t], m0 = mat[0];
                const float *rt = row[t], *r0 = row[0];
                const float mxt = mx[t], mx0 = mx[0];
                float s = 0.f;
                for (int i = tm.rank * blockDim.x + threadIdx.x; i < V; i += tm.size * blockDim.x) {
                    const float jt = mt ? P[t][i] : expf((rt[i] - mxt) * a.inv_temp);
                    const float pr = m0 ? P[0][i] : expf((r0[i] - mx0) * a.inv_temp);
                    s += fmaxf(0.f, jt * sj - pr * sp);
                }
                s = team_sum(s, sh, tm);
                float z = 0.f;
                for (int i = tm.rank * blockDim.x + threadIdx.x; i < V; i += tm.size * blockDim.x) {
                    const float jt = mt ? P[t][i] : expf((rt[i] - mxt) * a.inv_temp);
                    const float pr = m0 ? P[0][i] : expf((r0[i] - mx0) * a.inv_temp);
                    P[t][i] = s > 0.f ? fmaxf(0.f, jt * sj - pr * sp) : jt;
                    const float keep = i == v ? 0.f : pr;
                    P[0][i] = keep;
                    z += keep;
                }
                z = team_sum(z, sh, tm);                          // (its barrier also publishes the arrays to the other CTAs)
                mat[t] = true; mat[0] = true;
                if (s > 0.f) Z[t] = s;
                if (z > 0.f) Z[0] = z;
                __syncthreads();
            }
        }
        if (needs_q) break;
        if (taken >= 0) {
            if (a.strict_break && taken_tier >= 1 && taken_tier < J) {
                corr = min(max(a.draft_tok[b * N + taken], 0), V - 1);
                corr_src = taken_tier;
                break;
            }
            if (lead && !a.probe) a.path[b * N + n_acc] = taken;
            ++n_acc;
            cur = taken + 1;
            continue;
        }
        corr_src = failed;
        if (sampling) {
            __syncthreads();
            corr = gumbel_argmax(P[failed], V, k_gum, cur, shm, tm);
        } else {
            corr = st_arg[failed * RS_STRIDE + cur];
        }
        break;
    }
    __syncthreads();
    if (a.probe) {
        if (lead) {
            // tokens this step emits if q is not asked: the accepted nodes and the replacement (or nothing at a leaf)
            const int ne = n_acc + (corr >= 0 ? 1 : 0);
            const bool room = a.len[b] - a.len_full[b] + ne <= a.replay_rows && a.len[b] >= a.replay_rows;
            if (needs_q || !room) atomicExch(a.need_full, 1);
        }
        if (tm.size > 1) team_barrier();
        return;
    }
    if (lead) {
        int ne = 0;
        for (int j = 0; j < n_acc; ++j) {
            int node = a.path[b * N + j];
            a.out_tok[b * (N + 1) + ne++] = min(max(a.draft_tok[b * N + node], 0), V - 1);
        }
        if (corr >= 0) a.out_tok[b * (N + 1) + ne++] = corr;
        a.n_acc[b] = n_acc;
        a.n_emit[b] = ne;
        a.corr_src[b] = corr_src;
        atomicAdd(&a.stats->emitted, (unsigned long long)ne);
        atomicAdd(&a.stats->accepted, (unsigned long long)n_acc);
    }
    if (tm.size > 1) team_barrier();          // no CTA leaves while another may still read its slots
}

// the accept kernel needs the tree layout but no cache: build it here when called on its own
__global__ void tree_only_kernel(TreeInfo *tree, DeviceStats *stats, const int *parent, int per_seq, int B, int N) {
    for (int b = threadIdx.x; b < B; b += blockDim.x) build_tree(tree + b, parent + (per_seq ? (size_t)b * N : 0), N, stats);
}

}  // namespace

int launch_tier(const viasd_model *m, const viasd_draft *d, const viasd_params *p, const JudgeSet &js, viasd_result *r,
                cudaStream_t st) {
    const int M = d->n_nodes + 1;
    if (js.n < 1 || js.n > MAXJ) return VIASD_EINVAL;
    CUDA_TRY(cudaMemsetAsync(&m->ws.stats->need_slim, 0, 2 * sizeof(int), st));
    const float *gate = p->conf_source == 0 ? d->drafter_logits : js.logits[0];   // Alg. 2 gates with the slim(mest) verifier
    const int rows = p->conf_source == 0 ? d->n_prows : M;
    if (!gate) return VIASD_EINVAL;
    TierCuts cuts;
    cuts.n = js.n;
    for (int k = 0; k < MAXJ; ++k) cuts.log_tau[k] = k < js.n ? js.log_tau[k] : 0.f;
    // (a CTA per gate row: with few rows the launch is bound by the loads each CTA has in flight, hence 1024 threads)
    tier_kernel<<<dim3(rows, d->batch), 1024, 0, st>>>(r->tier, r->conf, m->ws.stats, gate, d->draft_tok, d->prow,
        d->parent, d->per_sequence, p->conf_source, rows, d->n_nodes, m->cfg.vocab, cuts);
    LAUNCH_CHECK();
    return VIASD_OK;
}

// A cluster of 16 CTAs (beyond the portable 8) where the device takes it: asked once per device.
static bool accept_team16_ok() {
    static int state[64];                    // 0 unknown, 1 yes, -1 no
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    if (state[dev] == 0) {
        state[dev] = -1;
        if (cudaFuncSetAttribute(accept_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
            cudaLaunchConfig_t cfg;
            memset(&cfg, 0, sizeof(cfg));
            cfg.gridDim = dim3(16); cfg.blockDim = dim3(ACC_THREADS);
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = 16; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr; cfg.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, accept_kernel, &cfg) == cudaSuccess && n >= 1) state[dev] = 1;
        }
        (void)cudaGetLastError();
    }
    return state[dev] == 1;
}

int launch_accept(const viasd_model *m, const viasd_draft *d, const viasd_params *p, const JudgeSet &js, viasd_result *r,
                  bool tree_ready, cudaStream_t st, const AcceptProbe *probe) {
    if (js.n < 1 || js.n > MAXJ) return VIASD_EINVAL;
    if (!tree_ready) {                       // a forward pass of the same call has laid the tree out already
        tree_only_kernel<<<1, 64, 0, st>>>(m->ws.tree, m->ws.stats, d->parent, d->per_sequence, d->batch, d->n_nodes);
        LAUNCH_CHECK();
    }
    if (d->n_prows > RS_STRIDE) return VIASD_EINVAL;
    AcceptArgs a;
    {
        // row statistics live behind the distribution buffers
        float *base = m->ws.accept_scratch + (size_t)m->cfg.max_batch * KINDS * m->cfg.vocab;
        const size_t n = (size_t)m->cfg.max_batch * KINDS * RS_STRIDE;
        a.rs.mx = base; a.rs.arg = reinterpret_cast<int *>(base + n); a.rs.z = base + 2 * n;
        const int M = d->n_nodes + 1, rows = M > d->n_prows ? M : d->n_prows;
        RowPtrs src;
        src.p[0] = p->mode == 1 ? d->drafter_logits : nullptr;
        for (int k = 1; k < KINDS; ++k) src.p[k] = k <= js.n ? js.logits[k - 1] : nullptr;
        row_stats_kernel<<<dim3(rows, d->batch, js.n + 1), 1024, 0, st>>>(a.rs, src, d->n_prows, M, m->cfg.vocab,
                                                                         1.0f / p->temperature, p->mode == 1);
        LAUNCH_CHECK();
    }
    a.judges[0] = nullptr;
    for (int k = 1; k < KINDS; ++k) a.judges[k] = k <= js.n ? js.logits[k - 1] : nullptr;
    a.n_judges = js.n;
    a.drafter = d->drafter_logits;
    a.draft_tok = d->draft_tok; a.prow = d->prow; a.tier = r->tier; a.tree = m->ws.tree;
    a.scratch = m->ws.accept_scratch;
    a.n_acc = r->n_acc; a.path = r->path; a.out_tok = r->out_tok; a.n_emit = r->n_emit; a.corr_src = r->corr_src;
    a.judge = r->judge; a.stats = m->ws.stats;
    a.N = d->n_nodes; a.R = d->n_prows; a.V = m->cfg.vocab;
    a.mode = p->mode; a.strict_break = p->strict_break; a.emit_bonus = p->emit_bonus;
    a.inv_temp = 1.0f / p->temperature;
    a.log1m_alpha = log1pf(-p->alpha);
    a.inv_beta = 1.0f / p->beta;
    // greedy gates: log_acc_rel[1] for every slim verifier, log_acc_rel[2] for q
    for (int k = 0; k < KINDS; ++k) a.log_acc_rel[k] = k == 0 ? p->log_acc_rel[0] : k < js.n ? p->log_acc_rel[1] : p->log_acc_rel[2];
    a.seed = p->seed; a.step = p->step;
    a.per_seq = d->per_sequence;
    a.probe = probe ? 1 : 0;
    a.replay_rows = probe ? probe->replay_rows : 0;
    a.need_full = probe ? probe->need_full : nullptr;
    a.len = probe ? probe->len : nullptr;
    a.len_full = probe ? probe->len_full : nullptr;
    // sampling over a large vocabulary: a cluster of CTAs per sequence shares every sweep of the vocabulary
    int team = (p->mode == 1 && m->cfg.vocab >= 16384) ? ACC_TEAM : 1;
    if (team == ACC_TEAM && m->cfg.vocab >= 65536 && accept_team16_ok()) team = 16;     // every sweep of the vocabulary is shared
    { const int t = m->opt.accept_team; if (t == 1 || t == 2 || t == 4 || t == 8) team = t; }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(d->batch * team);
    cfg.blockDim = dim3(ACC_THREADS);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = team; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = team > 1 ? 1 : 0;
    CUDA_TRY(cudaLaunchKernelEx(&cfg, accept_kernel, a));
    LAUNCH_CHECK();
    return VIASD_OK;
}
