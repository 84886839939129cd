// Generic CUDA-core GEMM y[rows, n] = x[rows, k] * W[n, k]^T for a handful of rows.
// One warp owns FEAT output features and streams their weight rows once with 16-byte loads; the
// activation vector it multiplies with is reused across the FEAT features from registers.
// Serves the fp32 model configuration and any shape the tensor-core kernels do not take.
#include "common.cuh"

namespace {

template <typename T> struct Vec;                 // 16 bytes of T
template <> struct Vec<float> { static constexpr int N = 4; };
template <> struct Vec<__nv_bfloat16> { static constexpr int N = 8; };

template <typename T>
__device__ __forceinline__ void load16(const T *p, float (&out)[Vec<T>::N]);
template <>
__device__ __forceinline__ void load16<float>(const float *p, float (&out)[4]) {
    float4 v = *reinterpret_cast<const float4 *>(p);
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}
template <>
__device__ __forceinline__ void load16<__nv_bfloat16>(const __nv_bfloat16 *p, float (&out)[8]) {
    uint4 v = *reinterpret_cast<const uint4 *>(p);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        out[2 * i] = __uint_as_float(w[i] << 16);
        out[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

constexpr int FEAT = 4;
constexpr int WARPS = 8;

struct SegTable { const void *w[3]; int end[3]; int count; };

template <typename T>
__device__ __forceinline__ const T *weight_row(const SegTable &s, int n, int k) {
    int base = 0;
#pragma unroll
    for (int i = 0; i < 3; ++i) {
        if (i < s.count && n < s.end[i]) return reinterpret_cast<const T *>(s.w[i]) + (size_t)(n - base) * k;
        base = s.end[i];
    }
    return nullptr;
}

// RC rows are kept in registers at a time; more rows loop (weights then come from L2).
template <typename T, int RC, int EPI>
__global__ void __launch_bounds__(WARPS * 32)
gemm_rowwarp_kernel(const T *__restrict__ x, size_t x_plane, SegTable segs, int rows, int k, int n_total,
                    float *__restrict__ out_f32, T *__restrict__ out_act, size_t act_plane, int ld_out) {
    constexpr int VN = Vec<T>::N;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int group = blockIdx.x * WARPS + warp;
    const T *wrow[FEAT];
    int feat[FEAT];
    if (EPI == EPI_SWIGLU) {
        // features f0, f0+1 of the gate matrix and the same two of the up matrix
        const int ff = segs.end[0];
        const int f0 = group * 2;
        if (f0 >= ff) return;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            int f = f0 + j;
            feat[j] = f; feat[2 + j] = f;
            bool ok = f < ff;
            wrow[j] = ok ? reinterpret_cast<const T *>(segs.w[0]) + (size_t)f * k : nullptr;
            wrow[2 + j] = ok ? reinterpret_cast<const T *>(segs.w[1]) + (size_t)f * k : nullptr;
        }
    } else {
        const int n0 = group * FEAT;
        if (n0 >= n_total) return;
#pragma unroll
        for (int j = 0; j < FEAT; ++j) {
            feat[j] = n0 + j;
            wrow[j] = (n0 + j < n_total) ? weight_row<T>(segs, n0 + j, k) : nullptr;
        }
    }
    for (int r0 = 0; r0 < rows; r0 += RC) {
        float acc[RC][FEAT];
#pragma unroll
        for (int r = 0; r < RC; ++r)
#pragma unroll
            for (int j = 0; j < FEAT; ++j) acc[r][j] = 0.f;
        for (int k0 = lane * VN; k0 < k; k0 += 32 * VN) {
            float wv[FEAT][VN];
#pragma unroll
            for (int j = 0; j < FEAT; ++j) {
                if (wrow[j]) load16<T>(wrow[j] + k0, wv[j]);
                else {
#pragma unroll
                    for (int e = 0; e < VN; ++e) wv[j][e] = 0.f;
                }
            }
#pragma unroll
            for (int r = 0; r < RC; ++r) {
                if (r0 + r < rows) {
                    float xv[VN];
                    load16<T>(x + (size_t)(r0 + r) * k + k0, xv);
                    if (x_plane) {                      // bf16 activations come as hi + lo planes
                        float lo[VN];
                        load16<T>(x + x_plane + (size_t)(r0 + r) * k + k0, lo);
#pragma unroll
                        for (int e = 0; e < VN; ++e) xv[e] += lo[e];
                    }
#pragma unroll
                    for (int j = 0; j < FEAT; ++j)
#pragma unroll
                        for (int e = 0; e < VN; ++e) acc[r][j] = fmaf(xv[e], wv[j][e], acc[r][j]);
                }
            }
        }
#pragma unroll
        for (int r = 0; r < RC; ++r)
#pragma unroll
            for (int j = 0; j < FEAT; ++j) acc[r][j] = warp_sum(acc[r][j]);
        if (lane == 0) {
#pragma unroll
            for (int r = 0; r < RC; ++r) {
                if (r0 + r >= rows) break;
                if (EPI == EPI_SWIGLU) {
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        if (!wrow[j]) continue;
                        float g = acc[r][j], u = acc[r][2 + j];
                        float s = g / (1.f + expf(-g));
                        store_act<T>(out_act, act_plane, (size_t)(r0 + r) * ld_out + feat[j], s * u);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < FEAT; ++j) {
                        if (!wrow[j]) continue;
                        float *dst = out_f32 + (size_t)(r0 + r) * ld_out + feat[j];
                        if (EPI == EPI_ADD) *dst += acc[r][j]; else *dst = acc[r][j];
                    }
                }
            }
        }
    }
}

template <typename T, int RC>
int dispatch_epi(const T *x, size_t x_plane, const SegTable &s, int rows, int k, int n_total, int epi, float *out_f32,
                 T *out_act, size_t act_plane, int ld_out, cudaStream_t st) {
    int groups = epi == EPI_SWIGLU ? (s.end[0] + 1) / 2 : (n_total + FEAT - 1) / FEAT;
    int blocks = (groups + WARPS - 1) / WARPS;
    switch (epi) {
    case EPI_STORE:
        gemm_rowwarp_kernel<T, RC, EPI_STORE><<<blocks, WARPS * 32, 0, st>>>(x, x_plane, s, rows, k, n_total, out_f32, out_act, act_plane, ld_out);
        break;
    case EPI_ADD:
        gemm_rowwarp_kernel<T, RC, EPI_ADD><<<blocks, WARPS * 32, 0, st>>>(x, x_plane, s, rows, k, n_total, out_f32, out_act, act_plane, ld_out);
        break;
    case EPI_SWIGLU:
        gemm_rowwarp_kernel<T, RC, EPI_SWIGLU><<<blocks, WARPS * 32, 0, st>>>(x, x_plane, s, rows, k, n_total, out_f32, out_act, act_plane, ld_out);
        break;
    default:
        return VIASD_EINVAL;
    }
    LAUNCH_CHECK();
    return VIASD_OK;
}

template <typename T>
int dispatch_rows(const T *x, size_t x_plane, const SegTable &s, int rows, int k, int n_total, int epi, float *out_f32,
                  T *out_act, size_t act_plane, int ld_out, cudaStream_t st) {
    if (rows <= 4) return dispatch_epi<T, 4>(x, x_plane, s, rows, k, n_total, epi, out_f32, out_act, act_plane, ld_out, st);
    if (rows <= 8) return dispatch_epi<T, 8>(x, x_plane, s, rows, k, n_total, epi, out_f32, out_act, act_plane, ld_out, st);
    return dispatch_epi<T, 12>(x, x_plane, s, rows, k, n_total, epi, out_f32, out_act, act_plane, ld_out, st);
}

}  // namespace

int launch_gemm_rowwarp(const void *x, size_t x_plane, const GemmSegs &segs, int rows, int k, int dtype,
                        int epilogue, float *out_f32, void *out_act, size_t act_plane, int ld_out, cudaStream_t st) {
    if (rows <= 0) return VIASD_OK;
    if (k % 8 != 0) return VIASD_EINVAL;
    SegTable s;
    int total = 0;
    s.count = segs.count;
    for (int i = 0; i < 3; ++i) {
        s.w[i] = i < segs.count ? segs.w[i] : nullptr;
        if (i < segs.count) total += segs.n[i];
        s.end[i] = total;
    }
    if (epilogue == EPI_SWIGLU && (segs.count != 2 || segs.n[0] != segs.n[1])) return VIASD_EINVAL;
    if (dtype == 0)
        return dispatch_rows<float>((const float *)x, 0, s, rows, k, total, epilogue, out_f32, (float *)out_act, 0, ld_out, st);
    return dispatch_rows<__nv_bfloat16>((const __nv_bfloat16 *)x, x_plane, s, rows, k, total, epilogue, out_f32,
                                        (__nv_bfloat16 *)out_act, act_plane, ld_out, st);
}
