// placeholder until the tensor-core kernel lands
#include "vig_internal.h"
namespace vig {
bool mma_supported(int, int) { return false; }
size_t mma_workspace_bytes(long long, int, int, int) { return 0; }
cudaError_t launch_bigla_mma(const __nv_bfloat16*, const __nv_bfloat16*, const __nv_bfloat16*, const __nv_bfloat16*,
                             const __nv_bfloat16*, __nv_bfloat16*, long long, int, int, int, void*, cudaStream_t) {
    return cudaErrorNotSupported;
}
}  // namespace vig
