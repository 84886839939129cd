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
    for (int i = threadIdx.x; i < V; i += blockDim.x) { mq = fmaxf(mq, jq[i]); mp = fmaxf(mp, pp[i]); }
    mq = block_max_f(mq, sh);
    mp = block_max_f(mp, sh);
    float sq = 0.f, sp = 0.f;
    for (int i = threadIdx.x; i < V; i += blockDim.x) { sq += expf((jq[i] - mq) * inv_temp); sp += expf((pp[i] - mp) * inv_temp); }
    sq = block_sum_f(sq, sh);
    sp = block_sum_f(sp, sh);
    const float lzq = logf(sq), lzp = logf(sp), inv_tau = smooth ? 1.f / tau : 0.f;
    float acc = 0.f;
    for (int i = threadIdx.x; i < V; i += blockDim.x) {
        const float lq = (jq[i] - mq) * inv_temp - lzq, lp = (pp[i] - mp) * inv_temp - lzp, d = lp - lq;
        acc += expf(lp) * phi(log1m_alpha + d, smooth, tau, inv_tau) + expf(lq) * phi(log_beta + d, smooth, tau, inv_tau);
    }
    acc = block_sum_f(acc, sh);
    if (threadIdx.x == 0) cost_rows[blockIdx.x] = acc;
}

__global__ void kl_cost_sum_kernel(float *total, const float *cost_rows, int rows) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    float s = 0.f;
    for (int r = 0; r < rows; ++r) s += cost_rows[r];
    *total = s;
}

}  // namespace

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
