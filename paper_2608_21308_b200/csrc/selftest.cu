// e2ttt_selftest_wait_timeout: exercises the device-side failure path without failing anything.  One CTA waits, with a
// short limit, on an mbarrier nobody ever arrives on; the bounded wait runs out, records its code in the status word
// and the kernel returns.  Nothing traps, faults or spins without a limit; the context stays usable.
#include <cuda_runtime.h>

#include "../../include/e2ttt.h"
#include "sm100.cuh"

namespace e2ttt {
namespace {

constexpr int kSelftestCode = 900;

__global__ void __launch_bounds__(64) selftest_wait_kernel(int* status, long long limit_cycles) {
    __shared__ uint64_t bar;
    __shared__ int dead;
    if (threadIdx.x == 0) {
        dead = 0;
        sm100::mbar_init(&bar, 1);
        sm100::fence_mbar_init();
    }
    __syncthreads();
    sm100::WaitCtx wc{&dead, status, limit_cycles};
    sm100::mbar_wait(&bar, 0u, wc, kSelftestCode);       // gives up after limit_cycles
    sm100::mbar_wait(&bar, 0u, wc, kSelftestCode + 1);   // the CTA-wide flag is up: returns at once
    __syncthreads();
}

}  // namespace
}  // namespace e2ttt

extern "C" E2TTT_API int e2ttt_selftest_wait_timeout(void* workspace, size_t workspace_bytes, long long limit_cycles,
                                                    void* stream) {
    if (!workspace) return E2TTT_ERR_NULL;
    if (workspace_bytes < 256) return E2TTT_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) % 256) != 0) return E2TTT_ERR_ALIGN;
    if (limit_cycles <= 0 || limit_cycles > e2ttt::sm100::kWaitCycles) return E2TTT_ERR_SHAPE;
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return E2TTT_ERR_ARCH;
    }
    if (major != 10) return E2TTT_ERR_ARCH;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(workspace, 0, sizeof(int), st) != cudaSuccess) { (void)cudaGetLastError(); return E2TTT_ERR_CUDA; }
    e2ttt::selftest_wait_kernel<<<1, 64, 0, st>>>(static_cast<int*>(workspace), limit_cycles);
    return cudaGetLastError() == cudaSuccess ? E2TTT_OK : E2TTT_ERR_CUDA;
}
