// Self-test of the bounded device-side wait that every barrier wait of the attention kernels goes through.
//
// One small CTA waits on an mbarrier that nobody ever arrives on, with nothing else in flight (no bulk copy,
// no MMA, no tensor memory).  The wait must run out of its budget, flag the give-up in the control words and
// return false; the kernel then reports LIBRA_ERR_TIMEOUT and leaves normally, so the context stays usable.
#include "common.h"
#include "ptx.cuh"

namespace libra {

__global__ void k_selftest_wait(uint32_t limit_ns, int* result /* [2]: status, nanoseconds waited */) {
    __shared__ uint64_t bar;
    __shared__ int ctl[2];
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        ctl[0] = 0;
        ctl[1] = (int)limit_ns;
        fence_mbar_init();
    }
    __syncthreads();
    const uint64_t t0 = globaltimer_ns();
    const bool done = mbar_wait(&bar, 0, ctl);          // phase 0 never completes
    const uint64_t waited = globaltimer_ns() - t0;
    __syncthreads();
    if (threadIdx.x == 0) {
        result[0] = done ? LIBRA_OK : (ctl[0] ? LIBRA_ERR_TIMEOUT : LIBRA_ERR_CUDA);
        result[1] = (int)(waited > 0x7fffffffull ? 0x7fffffffull : waited);
    }
}

}  // namespace libra

extern "C" int libra_selftest_wait_timeout(uint32_t limit_ns, int* status_host, int* waited_ns_host) {
    if (!status_host || limit_ns == 0 || limit_ns > 100000000u) return LIBRA_ERR_INVALID_ARG;   // at most 0.1 s
    int* d = nullptr;
    if (cudaMalloc((void**)&d, 2 * sizeof(int)) != cudaSuccess) return LIBRA_ERR_CUDA;
    int h[2] = {LIBRA_ERR_CUDA, 0};
    libra::k_selftest_wait<<<1, 64>>>(limit_ns, d);
    libra::count_launch();
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaMemcpy(h, d, sizeof(h), cudaMemcpyDeviceToHost);
    cudaFree(d);
    if (e != cudaSuccess) return LIBRA_ERR_CUDA;
    *status_host = h[0];
    if (waited_ns_host) *waited_ns_host = h[1];
    return LIBRA_OK;
}
