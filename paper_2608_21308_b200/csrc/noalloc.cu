// e2ttt_chunk_fwd_noalloc: the forward for callers that cannot obtain device memory themselves.
// The scratch the kernel needs lives in a fixed array inside this library's device image.
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/e2ttt.h"

namespace {

// Resident on every GPU that loads the library, for the life of the process.
static __device__ __align__(256) unsigned char g_static_scratch[E2TTT_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices];  // device address of g_static_scratch, per device ordinal
bool g_scratch_known[kMaxDevices];
std::mutex g_mu;

// In host code the array's name is only a handle: the address a kernel may use has to be asked for,
// once per device, while that device is current.
int scratch_for_current_device(void** out) {
    int dev = -1, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return E2TTT_ERR_ARCH; }
    if (dev < 0 || dev >= kMaxDevices) return E2TTT_ERR_ARCH;
    // the device image holds sm_100a code only: ask for the architecture before asking for a symbol of it
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) { (void)cudaGetLastError(); return E2TTT_ERR_ARCH; }
    if (major != 10) return E2TTT_ERR_ARCH;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_known[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) {
            (void)cudaGetLastError();
            return E2TTT_ERR_CUDA;
        }
        g_scratch_addr[dev] = p;
        g_scratch_known[dev] = true;
    }
    *out = g_scratch_addr[dev];
    return E2TTT_OK;
}

}  // namespace

namespace e2ttt {
// Device address of the scratch array on the current device, or nullptr before the first call there.  Its first
// word is the device status word of the calls that used it (read by e2ttt_device_status(NULL, ...)).
const void* noalloc_scratch_if_known() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
    if (dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_mu);
    return g_scratch_known[dev] ? g_scratch_addr[dev] : nullptr;
}
}  // namespace e2ttt

extern "C" E2TTT_API int e2ttt_chunk_fwd_noalloc(const e2ttt_params* p, const void* q, const void* k, const void* v,
                                                const float* eta, const float* beta, const float* gamma,
                                                const float* const* W_init, const float* const* M_init, void* o,
                                                float* const* W_final, float* const* M_final, void* stream) {
    size_t need = 0;
    int rc = e2ttt_workspace_bytes(p, 0, &need);
    if (rc != E2TTT_OK) return rc;
    if (need > (size_t)E2TTT_NOALLOC_SCRATCH_BYTES) return E2TTT_ERR_WORKSPACE;
    void* scratch = nullptr;
    rc = scratch_for_current_device(&scratch);
    if (rc != E2TTT_OK) return rc;
    return e2ttt_chunk_fwd(p, q, k, v, eta, beta, gamma, W_init, M_init, o, W_final, M_final, scratch,
                           (size_t)E2TTT_NOALLOC_SCRATCH_BYTES, 0, stream);
}
