// Diagnostic for the bounded waits: a wait that can never be satisfied must end by itself and report
// DG4_ERR_TIMEOUT, leaving the context usable.  One CTA waits, with the library's own mbar_wait helper (the one
// every pipeline stage of the projection and levelised kernels uses), on an mbarrier nothing ever arrives on.

#include "dg4_internal.h"
#include "dg4_sm100.cuh"

namespace {

__global__ void bounded_wait_selftest_kernel(int32_t* status) {
    __shared__ uint64_t bar;
    const uint32_t b = sm100::smem_u32(&bar);
    if (threadIdx.x == 0) {
        sm100::mbar_init(b, 1);
        sm100::mbar_fence_init();
    }
    __syncthreads();
    const bool done = sm100::mbar_wait(b, 0);        // phase 0 never completes: nobody arrives
    if (threadIdx.x == 0) *status = done ? (int32_t)DG4_OK : (int32_t)DG4_ERR_TIMEOUT;
}

}  // namespace

extern "C" dg4_status dg4_selftest_bounded_wait(int32_t* device_status, void* stream) {
    if (!device_status) DG4_FAIL(DG4_ERR_INVALID_ARG, "device_status is null");
    bounded_wait_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(device_status);
    dg4i_count_launch();
    DG4_CUDA_TRY(cudaGetLastError());
    return DG4_OK;
}
