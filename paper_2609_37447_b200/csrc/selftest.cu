// az_selftest_wait_timeout: exercises the bounded-wait path that every mbarrier wait of the
// tensor-core kernels goes through, without hanging anything: one warp waits on a barrier that
// nobody will ever arrive on, with a short poll limit, and must come back with the time-out status.
#include "common.cuh"
#include "ptx.cuh"

namespace az {
namespace {

__global__ void __launch_bounds__(64, 1) wait_timeout_kernel(uint32_t *status, uint32_t limit, int *reached_teardown) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_addr(&bar), 1);
        abort_flag = 0;
        ptx::fence_barrier_init();
    }
    __syncthreads();
    bool ok = true;
    if (threadIdx.x < 32) {
        // warp 0: the wait that runs out
        ok = bounded_wait(ptx::smem_addr(&bar), 0, &abort_flag, status, kStatusWaitTimeout, limit);
    } else {
        // warp 1: a second waiter on the same barrier; it must be released by the abort flag (or run out itself)
        ok = bounded_wait(ptx::smem_addr(&bar), 0, &abort_flag, status, kStatusWaitTimeout, limit * 4);
    }
    __syncthreads();                                   // the common teardown every role reaches
    if (threadIdx.x == 0) *reached_teardown = ok ? 2 : 1;
}

}  // namespace
}  // namespace az

extern "C" int az_selftest_wait_timeout(void *cuda_stream) {
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    uint32_t *status = nullptr;
    AZ_CUDA(cudaMalloc((void **)&status, 2 * sizeof(uint32_t)));
    cudaError_t e = cudaMemsetAsync(status, 0, 2 * sizeof(uint32_t), s);
    if (e == cudaSuccess) {
        az::wait_timeout_kernel<<<1, 64, 0, s>>>(status, 1u << 14, reinterpret_cast<int *>(status + 1));
        e = cudaGetLastError();
    }
    uint32_t host[2] = {0, 0};
    if (e == cudaSuccess) e = cudaMemcpyAsync(host, status, sizeof host, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    cudaFree(status);
    if (e != cudaSuccess) { az::set_cuda_error(e, "az_selftest_wait_timeout"); return AZ_ERR_CUDA; }
    if (host[1] != 1) return AZ_ERR_BAD_ARG;            // the kernel did not leave through its teardown with the wait failed
    return (host[0] & az::kStatusWaitTimeout) ? AZ_ERR_DEVICE_TIMEOUT : AZ_OK;
}
