// Test hooks (include/fdkv_testing.h): reach the library's failure handling without a fault, a trap or a hang.
#include "../../include/fdkv_testing.h"
#include "fdkv_internal.h"
#include "mbar_wait.cuh"

namespace fdkv {
namespace {

// Thread 0 waits on a barrier nobody arrives at; the bounded wait gives up after `cap` polls and reports through the
// abort flag and the status word, as in the product kernels.  The other threads wait for it at the block barrier.
__global__ void __launch_bounds__(32) wait_expiry_kernel(int32_t* status, uint32_t cap, int32_t* polls_seen) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t abort_flag;
    const uint32_t b = (uint32_t)__cvta_generic_to_shared(&bar);
    if (threadIdx.x == 0) {
        abort_flag = 0;
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(b), "r"(1u));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        mbar_wait_bounded(b, 0u, &abort_flag, status, cap);
        // a second wait of the same block returns at once: the abort flag is up
        mbar_wait_bounded(b, 0u, &abort_flag, status, cap);
        if (polls_seen) *polls_seen = (int32_t)abort_flag;
    }
    __syncthreads();
}

}  // namespace
}  // namespace fdkv

extern "C" {

fdkv_status fdkv_test_wait_expiry(fdkv_ctx* c, int32_t poll_cap, void* stream) {
    if (!c || poll_cap < 1 || poll_cap > 65536) return FDKV_ERR_INVALID_ARG;
    int32_t* status = reinterpret_cast<int32_t*>(c->work + c->ws.status);
    fdkv::wait_expiry_kernel<<<1, 32, 0, reinterpret_cast<cudaStream_t>(stream)>>>(status, (uint32_t)poll_cap, status + 1);
    fdkv::count_launch(1);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? FDKV_OK : fdkv::record_cuda_error(e);
}

fdkv_status fdkv_test_clear_device_status(fdkv_ctx* c, void* stream) {
    if (!c) return FDKV_ERR_INVALID_ARG;
    const cudaError_t e = cudaMemsetAsync(c->work + c->ws.status, 0, 256, reinterpret_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? FDKV_OK : fdkv::record_cuda_error(e);
}

int32_t fdkv_test_per_device_visits(const int32_t* devs, int32_t n) {
    if (!devs || n < 0) return -1;
    return fdkv::per_device_first_visits(reinterpret_cast<const int*>(devs), n);
}

}  // extern "C"
