// viasd_gemm_static: the stand-alone projection GEMM for callers that cannot allocate device memory.
//
// The tensor-core GEMM splits work across CTAs and needs scratch for partial tiles and per-tile arrival
// counters.  viasd_gemm takes that scratch from the caller; this variant keeps it in a fixed array that is
// part of the library image, so the caller passes inputs and outputs only and no allocation call is made.
#include "common.cuh"

namespace {

constexpr int STATIC_MAX_ROWS = 16;                  // one 16-wide token tile
constexpr int STATIC_MAX_N = 262144;                 // 2048 output tiles of 128 features
constexpr int STATIC_CTAS = 160;                     // at most one CTA per SM is launched
constexpr size_t STATIC_COUNTER_BYTES = (size_t)(STATIC_MAX_N / 128 + 64) * 4;          // tile counters + status word
constexpr size_t STATIC_PARTIAL_BYTES = (size_t)STATIC_CTAS * 2 * 16 * 128 * 4;         // two partial-tile slots per CTA
constexpr size_t STATIC_BYTES = STATIC_COUNTER_BYTES + STATIC_PARTIAL_BYTES;            // about 2.6 MB per device
constexpr int STATIC_STATUS_WORD = STATIC_MAX_N / 128 + 63;                             // last word of the counter region

// Lives in every device's copy of the module from load to exit.  In host code this name is only a handle
// for the runtime's symbol lookup, not a device address.
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_BYTES];

constexpr int MAX_DEVICES = 64;
void *g_scratch_ptr[MAX_DEVICES];                    // device address of the array, looked up once per device

}  // namespace

extern "C" int viasd_gemm_static(const void *x, const void *w, float *y, int rows, int n, int k, void *stream) {
    if (!x || !w || !y) return VIASD_EINVAL;
    if (((uintptr_t)x & 15) || ((uintptr_t)w & 15)) return VIASD_EINVAL;
    if (rows < 1 || n < 1 || k < 8 || (k % 8)) return VIASD_EINVAL;
    if (rows > STATIC_MAX_ROWS || n > STATIC_MAX_N) return VIASD_ECAPACITY;     // beyond what the fixed array holds
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return VIASD_EUNSUPPORTED;
    if (!g_scratch_ptr[dev]) {
        // set-up, once per device, with that device current: ask the runtime where the array lives there
        cudaDeviceProp prop;
        CUDA_TRY(cudaGetDeviceProperties(&prop, dev));
        if (prop.major != 10) return VIASD_EUNSUPPORTED;
        void *ptr = nullptr;
        CUDA_TRY(cudaGetSymbolAddress((void **)&ptr, g_static_scratch));
        if (!ptr) return VIASD_ECUDA;
        g_scratch_ptr[dev] = ptr;
    }
    if (g_use_pdl < 0) g_use_pdl = 1;
    cudaStream_t st = (cudaStream_t)stream;
    int sms = 0;
    CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    if (sms > STATIC_CTAS) sms = STATIC_CTAS;
    char *base = (char *)g_scratch_ptr[dev];
    // the array keeps whatever the last call left: counters and the status word must start at zero
    CUDA_TRY(cudaMemsetAsync(base, 0, STATIC_COUNTER_BYTES, st));
    CUtensorMap mw, mx;
    int rc;
    const uint32_t wbox = tc_box_rows(n, 128), xbox = tc_box_rows(rows, 16);
    if ((rc = tc_make_map(&mw, w, n, k, wbox))) return rc;
    if ((rc = tc_make_map(&mx, x, rows, k, xbox))) return rc;
    TcLaunch L;
    memset(&L, 0, sizeof(L));
    L.map_w[0] = &mw; L.seg_n[0] = n; L.w_box_rows[0] = wbox; L.n_seg = 1;
    L.map_x = &mx; L.x_box_rows = xbox; L.has_lo = 0; L.lo_row_offset = 0;
    L.rows = rows; L.row0 = 0; L.k = k; L.nt = 16; L.epi = EPI_STORE;
    L.out_f32 = y; L.ld_out = n;
    L.counters = (int *)base;
    L.status = (int *)base + STATIC_STATUS_WORD;
    L.scratch = (float *)(base + STATIC_COUNTER_BYTES);
    L.sm_count = sms;
    return launch_gemm_tc(L, st);
}

// What the last viasd_gemm_static call on this device recorded: VIASD_OK, or VIASD_EDEVICE when one of its bounded
// waits expired (y is then incomplete).  Synchronises `stream`; allocates nothing.
extern "C" int viasd_gemm_static_status(int *host_out, void *stream) {
    if (!host_out) return VIASD_EINVAL;
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return VIASD_EUNSUPPORTED;
    *host_out = VIASD_OK;
    if (!g_scratch_ptr[dev]) return VIASD_OK;               // no call on this device yet
    CUDA_TRY(cudaMemcpyAsync(host_out, (int *)g_scratch_ptr[dev] + STATIC_STATUS_WORD, sizeof(int), cudaMemcpyDeviceToHost,
                             (cudaStream_t)stream));
    CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    return VIASD_OK;
}
