// Debug kernels: exercising the bounded-wait failure path without faulting or hanging the device.
#include "common.cuh"

namespace dyn {

// One warp waits, through the same bounded wait the FFN kernels use, on a barrier that nobody arrives at.  After
// `limit_ns` the wait gives up, records STATUS_TIMEOUT and the kernel returns normally: the context stays usable.
__global__ void __launch_bounds__(32) expire_wait_kernel(int32_t* status, unsigned long long limit_ns) {
    __shared__ uint64_t bar;
    __shared__ int poison;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        poison = 0;
        fence_barrier_init();
    }
    __syncwarp();
    if (threadIdx.x == 0) mbar_wait_bounded(&bar, 0, &poison, status, limit_ns);
}

cudaError_t launch_expire_wait(int32_t* status, unsigned long long limit_ns, cudaStream_t st) {
    expire_wait_kernel<<<1, 32, 0, st>>>(status, limit_ns);
    return cudaGetLastError();
}

}  // namespace dyn
