// KL-style verification cost of a judge against a proposal, per logits row (Eq. 11; smooth margin of App. F).
//
//   lp = log softmax(proposal / T), lq = log softmax(judge / T)
//   z1 = log(1 - alpha) + lp - lq,  z2 = log(beta) + lp - lq
//   R  = sum_v exp(lp) phi(z1) + sum_v exp(lq) phi(z2),   phi = max(0, .) or tau log(1 + exp(. / tau))
//
// HBM-bound: 2 rows of V floats in, one float out.  One CTA per row; the row pair is read three times (maxima, then
// the two denominators, then the sums), the second and third time from L2.  Reductions run in a fixed order, so the
// result is reproducible.  The block cost of Eq. 10 is the sum of the rows, added up by one thread in row order.
#include "common.cuh"

namespace {

constexpr int COST_THREADS = 512;

__device__ float block_sum_f(float x, float *sh) {
    x = warp_sum(x);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = x;
    __syncthreads();
    float r = 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) r += sh[w];
    return r;
}
__device__ float block_max_f(float x, float *sh) {
    x = warp_max(x);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = x;
    __syncthreads();
    float r = sh[0];
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w) r = fmaxf(r, sh[w]);
    return r;
}

// One sweep over a pair of rows: f(a[i], b[i]) for every i, each thread taking float4 pieces when the rows allow it
// (16-byte loads, four in flight per thread: with 4-byte loads a CTA pulled a tenth of its share of the bandwidth).
template <typename F>
__device__ __forceinline__ void sweep_pair(const float *a, const float *b, int V, F f) {
    if ((V & 3) == 0 && ((reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(b)) & 15) == 0) {
        const float4 *a4 = reinterpret_cast<const float4 *>(a), *b4 = reinterpret_cast<const float4 *>(b);
        const int n4 = V >> 2;
#pragma unroll 4
        for (int i = threadIdx.x; i < n4; i += blockDim.x) {
            const float4 x = a4[i], y = b4[i];
            f(x.x, y.x); f(x.y, y.y); f(x.z, y.z); f(x.w, y.w);
        }
    } else {
        for (int i = threadIdx.x; i < V; i += blockDim.x) f(a[i], b[i]);
    }
}

__device__ __forceinline__ float phi(float z, int smooth, float tau, float inv_tau) {
    if (!smooth) return fmaxf(z, 0.f);
    const float t = z * inv_tau;                              // tau log(1 + e^t), without overflow for large t
    return tau * (fmaxf(t, 0.f) + log1pf(expf(-fabsf(t))));
}

__global__ void __launch_bounds__(COST_THREADS)
kl_cost_kernel(float *__restrict__ cost_rows, const float *__restrict__ judge, const float *__restrict__ proposal, int V,
               float inv_temp, float log1m_alpha, float log_beta, int smooth, float tau) {
    __shared__ float sh[32];
    const float *jq = judge + (size_t)blockIdx.x * V, *pp = proposal + (size_t)blockIdx.x * V;
    float mq = -INFINITY, mp = -INFINITY;
    sweep_pair(jq, pp, V, [&](float q, float p) { mq = fmaxf(mq, q); mp = fmaxf(mp, p); });
    mq = block_max_f(mq, sh);
    mp = block_max_f(mp, sh);
    float sq = 0.f, sp = 0.f;
    sweep_pair(jq, pp, V, [&](float q, float p) { sq += expf((q - mq) * inv_temp); sp += expf((p - mp) * inv_temp); });
    sq = block_sum_f(sq, sh);
    sp = block_sum_f(sp, sh);
    const float lzq = logf(sq), lzp = logf(sp), inv_tau = smooth ? 1.f / tau : 0.f;
    float acc = 0.f;
    sweep_pair(jq, pp, V, [&](float q, float p) {
        const float lq = (q - mq) * inv_temp - lzq, lp = (p - mp) * inv_temp - lzp, d = lp - lq;
        acc += expf(lp) * phi(log1m_alpha + d, smooth, tau, inv_tau) + expf(lq) * phi(log_beta + d, smooth, tau, inv_tau);
    });
    acc = block_sum_f(acc, sh);
    if (threadIdx.x == 0) cost_rows[blockIdx.x] = acc;
}

__global__ void kl_cost_sum_kernel(float *total, const float *cost_rows, int rows) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    float s = 0.f;
    for (int r = 0; r < rows; ++r) s += cost_rows[r];
    *total = s;
}

// Region masses (Eq. B.8-B.10): per row, the mass of p = softmax(proposal / T) on the tokens the gating row places in
// region A (d >= log tau_hi), B (log tau_lo <= d < log tau_hi) and C (below), d = l[u] - max l in fp32 exactly as the
// tier kernel decides a drafted token.  HBM-bound: 2 rows of V floats in, 3 floats out; the rows are read twice
// (maxima, then the sums), the second time from L2.  Fixed reduction order.
__global__ void __launch_bounds__(COST_THREADS)
region_mass_kernel(float *__restrict__ mass, const float *__restrict__ gate, const float *__restrict__ proposal, int V,
                   float inv_temp, float log_tau_hi, float log_tau_lo) {
    __shared__ float sh[32];
    const float *gg = gate + (size_t)blockIdx.x * V, *pp = proposal + (size_t)blockIdx.x * V;
    float mg = -INFINITY, mp = -INFINITY;
    sweep_pair(gg, pp, V, [&](float g, float p) { mg = fmaxf(mg, g); mp = fmaxf(mp, p); });
    mg = block_max_f(mg, sh);
    mp = block_max_f(mp, sh);
    float sa = 0.f, sb = 0.f, sc = 0.f;
    sweep_pair(gg, pp, V, [&](float g, float p) {
        const float d = g - mg, e = expf((p - mp) * inv_temp);
        if (d >= log_tau_hi) sa += e; else if (d >= log_tau_lo) sb += e; else sc += e;
    });
    sa = block_sum_f(sa, sh);
    sb = block_sum_f(sb, sh);
    sc = block_sum_f(sc, sh);
    if (threadIdx.x == 0) {
        const float inv = 1.f / (sa + sb + sc);
        float *dst = mass + (size_t)blockIdx.x * 3;
        dst[0] = sa * inv; dst[1] = sb * inv; dst[2] = sc * inv;
    }
}

__global__ void region_mass_mean_kernel(float *mean, const float *mass, int rows) {
    if (blockIdx.x != 0 || threadIdx.x >= 3) return;
    float s = 0.f;
    for (int r = 0; r < rows; ++r) s += mass[(size_t)r * 3 + threadIdx.x];
    mean[threadIdx.x] = s / (float)rows;
}

}  // namespace

extern "C" int viasd_region_mass(const float *gate_logits, const float *proposal_logits, int rows, int vocab, float temperature,
                                 float log_tau_hi, float log_tau_lo, float *mass, float *mean, void *stream) {
    if (!gate_logits || !proposal_logits || !mass || rows < 1 || vocab < 1) return VIASD_EINVAL;
    if (!(temperature > 0.f) || !(log_tau_lo <= log_tau_hi)) return VIASD_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    region_mass_kernel<<<rows, COST_THREADS, 0, st>>>(mass, gate_logits, proposal_logits, vocab, 1.0f / temperature,
                                                      log_tau_hi, log_tau_lo);
    LAUNCH_CHECK();
    if (mean) {
        region_mass_mean_kernel<<<1, 32, 0, st>>>(mean, mass, rows);
        LAUNCH_CHECK();
    }
    return VIASD_OK;
}

extern "C" int viasd_kl_cost(const float *judge_logits, const float *proposal_logits, int rows, int vocab, float temperature,
                             float alpha, float beta, int margin, float tau, float *cost_rows, float *cost_total,
                             void *stream) {
    if (!judge_logits || !proposal_logits || !cost_rows || rows < 1 || vocab < 1) return VIASD_EINVAL;
    if (!(temperature > 0.f) || !(alpha >= 0.f) || !(alpha < 1.f) || !(beta > 0.f)) return VIASD_EINVAL;
    if (margin != 0 && margin != 1) return VIASD_EINVAL;
    if (margin == 1 && !(tau > 0.f)) return VIASD_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    kl_cost_kernel<<<rows, COST_THREADS, 0, st>>>(cost_rows, judge_logits, proposal_logits, vocab, 1.0f / temperature,
                                                  log1pf(-alpha), logf(beta), margin, tau);
    LAUNCH_CHECK();
    if (cost_total) {
        kl_cost_sum_kernel<<<1, 32, 0, st>>>(cost_total, cost_rows, rows);
        LAUNCH_CHECK();
    }
    return VIASD_OK;
}
