// Self-test hooks: code paths that ordinary runs never take, made reachable without faulting or hanging the device.
#include "common.cuh"
#include "tc_ptx.cuh"

namespace {

// One CTA waits, through the bounded wait every tcgen05 kernel of this library uses, on a barrier that nothing ever
// arrives at.  The wait gives up after limit_cycles, records VIASD_EDEVICE in *status and the kernel returns by itself.
__global__ void wait_expiry_kernel(int *status, long long limit_cycles, long long *waited_cycles) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_sh;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_sh = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const long long t0 = clock64();
    bool ok = true;
    if (threadIdx.x == 0) ok = mbar_wait(smem_u32(&bar), 0, &abort_sh, status, limit_cycles);
    __syncthreads();
    // the other roles of a kernel see the flag the expired wait raised and leave as well
    if (threadIdx.x == 32 && waited_cycles) *waited_cycles = abort_sh ? clock64() - t0 : -1;
    (void)ok;
}

}  // namespace

extern "C" int viasd_selftest_wait_expiry(int *status, int limit_us, long long *waited_cycles, void *stream) {
    if (!status || limit_us < 1 || limit_us > 100000) return VIASD_EINVAL;
    int dev = 0, khz = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    CUDA_TRY(cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev));
    const long long limit = (long long)limit_us * (khz > 0 ? khz : 1000000) / 1000;     // cycles at the nominal clock
    wait_expiry_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(status, limit, waited_cycles);
    LAUNCH_CHECK();
    return VIASD_OK;
}
