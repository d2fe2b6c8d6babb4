// Self-test of the bounded wait every kernel of this library uses: a thread block waits on an
// mbarrier that nobody ever arrives on.  The wait must give up after the given number of cycles,
// record its code in the status word and let the kernel return normally - no trap, no hang.
#include <string>

#include <cuda_runtime.h>

#include "plan.h"
#include "sm100_ptx.cuh"

namespace tessera {
int32_t api_set_error(int32_t code, const std::string &msg);   // defined in api.cu
void count_launch();
}

namespace {

using namespace tessera::ptx;

__global__ void __launch_bounds__(64) bounded_wait_kernel(int *status, long long limit, long long *waited) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int s_abort;
    if (threadIdx.x == 0) {
        s_abort = 0;
        mbar_init(smem_u32(&bar), 1);
        fence_barrier_init();
    }
    __syncthreads();
    const long long t0 = clock64();
    const bool first = mbar_wait(smem_u32(&bar), 0, &s_abort, status, 42, limit);    // runs out
    const long long t1 = clock64();
    const bool second = mbar_wait(smem_u32(&bar), 0, &s_abort, status, 43, limit);   // returns at once: abort flag is up
    const long long t2 = clock64();
    if (threadIdx.x == 0 && waited) {
        waited[0] = t1 - t0;
        waited[1] = t2 - t1;
        waited[2] = (first ? 1 : 0) + (second ? 2 : 0);
    }
}

}  // namespace

extern "C" int32_t tessera_selftest_bounded_wait(int64_t max_cycles, int32_t *code_out, int64_t *cycles_out, void *stream) {
    using tessera::api_set_error;
    if (max_cycles <= 0 || max_cycles > 2000000000LL)
        return api_set_error(TESSERA_INVALID_ARG, "selftest_bounded_wait: max_cycles must be in (0, 2e9]");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int *d_status = nullptr;
    long long *d_waited = nullptr;
    cudaError_t e = cudaMalloc(&d_status, 4 * sizeof(int));
    if (e == cudaSuccess) e = cudaMalloc(&d_waited, 3 * sizeof(long long));
    if (e == cudaSuccess) e = cudaMemsetAsync(d_status, 0, 4 * sizeof(int), st);
    if (e == cudaSuccess) e = cudaMemsetAsync(d_waited, 0, 3 * sizeof(long long), st);
    int32_t code = 0;
    long long waited[3] = {0, 0, 0};
    if (e == cudaSuccess) {
        bounded_wait_kernel<<<1, 64, 0, st>>>(d_status, (long long)max_cycles, d_waited);
        tessera::count_launch();
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaMemcpyAsync(&code, d_status, sizeof code, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(waited, d_waited, sizeof waited, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (d_status) cudaFree(d_status);
    if (d_waited) cudaFree(d_waited);
    if (e != cudaSuccess)
        return api_set_error(TESSERA_CUDA_ERROR, std::string("selftest_bounded_wait: ") + cudaGetErrorString(e));
    if (code_out) *code_out = code;
    if (cycles_out) {
        cycles_out[0] = waited[0];
        cycles_out[1] = waited[1];
        cycles_out[2] = waited[2];
    }
    if (code != 0) return api_set_error(TESSERA_DEVICE_TIMEOUT, "selftest_bounded_wait: the wait gave up as intended, code " + std::to_string(code));
    return TESSERA_OK;
}
