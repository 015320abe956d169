// Self-test of the bounded-wait mechanism of the tensor-core kernels: a wait that nothing will ever satisfy must
// run out, report SQAP_ERR_TIMEOUT through the device status word and let the kernel return normally.
#include "tc_common.cuh"

namespace sqap {

// One warp waits, with the same mbar_wait the GEMM kernels use, on a barrier that expects one arrival and gets
// none. No memory is touched beyond the barrier and the status word.
__global__ void __launch_bounds__(32) bounded_wait_selftest_kernel(long long limit_clocks, int* status) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        tc::mbar_init(tc::smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const bool done = tc::mbar_wait(tc::smem_u32(&bar), 0u, &abort_flag, limit_clocks);
    if (!__all_sync(0xffffffffu, done)) {
        if (threadIdx.x == 0) atomicOr(status, SQAP_ERR_TIMEOUT);
    }
}

}  // namespace sqap

extern "C" sqap_status sqap_selftest_bounded_wait(int64_t limit_clocks, void* stream) {
    using namespace sqap;
    // between a microsecond and about a tenth of a second at B200 clocks: the hook must never hold the GPU
    if (limit_clocks < 1000 || limit_clocks > 200000000) return SQAP_ERR_INVALID;
    if (!tc::device_is_sm100()) return SQAP_ERR_UNSUPPORTED;
    int* status = device_status_word();
    if (!status) return SQAP_ERR_CUDA;
    bounded_wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<long long>(limit_clocks), status);
    count_launch();
    return check_launch();
}
