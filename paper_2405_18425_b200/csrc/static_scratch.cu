// BiGLA forward for callers that must not allocate: the segment scratch lives in a fixed
// file-scope device array instead of memory obtained at call time.
#include <mutex>

#include "vig_internal.h"

namespace vig {
namespace {

// Scratch of the no-allocation entry point.  Every GPU whose context loads this library carries
// these bytes until the process exits, so the size is kept modest: it covers, for example,
// B*H = 32 sequences of 4096 tokens at dk = 24, dv = 48 (20.3 MiB).
static __device__ __align__(256) unsigned char g_static_scratch[VIG_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of g_static_scratch on the current device.  In host code the array's name is only a
// handle for the runtime, never an address a kernel may use; the address is looked up once per
// device, with that device current, and cached.
cudaError_t static_scratch_ptr(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        if (!p) return cudaErrorInvalidSymbol;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace
}  // namespace vig

extern "C" int vig_bigla_fwd_static_bf16(const void* q, const void* k, const void* v, const void* log_alpha_fwd,
                                         const void* log_alpha_bwd, void* out, int B, int H, int L, int dk, int dv,
                                         void* stream) {
    using namespace vig;
    using bf = __nv_bfloat16;
    if (!q || !k || !v || !log_alpha_fwd || !log_alpha_bwd || !out) return VIG_ERR_NULL_POINTER;
    if (B < 0 || H < 0 || L < 0 || dk < 1 || dv < 1) return VIG_ERR_BAD_DIM;
    const void* ptrs[6] = {q, k, v, log_alpha_fwd, log_alpha_bwd, out};
    for (const void* p : ptrs)
        if (reinterpret_cast<uintptr_t>(p) & 15u) return VIG_ERR_MISALIGNED;
    if (!tc_supported(dk, dv) || (long long)B * H > 0x7fffffffLL) return VIG_ERR_UNSUPPORTED;
    const long long units = (long long)B * H;
    const size_t need = tc_workspace_bytes(units, L, dk, dv);
    if (need > (size_t)VIG_STATIC_SCRATCH_BYTES) return VIG_ERR_WORKSPACE;   // beyond the fixed scratch: use the _ws form
    if (B == 0 || H == 0 || L == 0) return VIG_OK;
    void* scratch = nullptr;
    if (static_scratch_ptr(&scratch) != cudaSuccess) return VIG_ERR_CUDA;
    // Nothing in the scratch has to survive from call to call, and nothing in it has to start at zero: every word
    // a launch reads to form the result was written earlier in the same call.
    cudaError_t e = launch_bigla_tc((const bf*)q, (const bf*)k, (const bf*)v, (const bf*)log_alpha_fwd,
                                     (const bf*)log_alpha_bwd, (bf*)out, units, L, dk, dv, scratch,
                                     (cudaStream_t)stream);
    return e == cudaSuccess ? VIG_OK : VIG_ERR_CUDA;
}
