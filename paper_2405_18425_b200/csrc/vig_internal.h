// Internal declarations shared by the translation units of libvig_bigla (not part of the C ABI).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "vig_bigla.h"

namespace vig {

// Device status word: bit flags set by kernels whose bounded waits expire.
constexpr int kDevStatusTimeout = 1;
constexpr int kDevStatusInternal = 2;   // a kernel found its own set-up inconsistent (reported as VIG_ERR_CUDA)
int* device_status_ptr();            // device address of the status word of the current device (NULL on error);
                                     // one int behind it: the count of units handed to the in-kernel recurrence
int take_expire_next_wait();         // test hook: 1 once after vig_test_expire_next_wait(), else 0
void count_launch(unsigned n = 1);   // bumps the process-wide launch counter

// ---- fp32 SIMT recurrence (Eq. 6 evaluated step by step), any dk <= 128, dv <= 256 ----
bool recurrence_supported(int dk, int dv);
template <typename T>
cudaError_t launch_recurrence(const T* q, const T* k, const T* v, const T* la_f, const T* la_b, T* out,
                              long long units, int L, int dk, int dv, cudaStream_t stream);

// ---- gate preparation ----
template <typename T>
cudaError_t launch_gate_prep(const T* g_f, const T* g_b, T* la_f, T* la_b, long long n, float tau,
                             cudaStream_t stream);
// dg = dlog alpha * sigmoid(-g) / tau, both directions in one launch (the outputs may be the incoming gradients' buffers)
template <typename T>
cudaError_t launch_gate_prep_bwd(const T* g_f, const T* g_b, const T* d_f, const T* d_b, T* o_f, T* o_b, long long n, float tau,
                                 cudaStream_t stream);

// ---- bf16 tensor-core path: dispatch over the tcgen05 kernels (defined with the entry points) ----
bool tc_supported(int dk, int dv);
// Scratch bytes the tensor-core path needs for this shape; 0 if no launch of it uses scratch.
size_t tc_workspace_bytes(long long units, int L, int dk, int dv);
cudaError_t launch_bigla_tc(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                            const __nv_bfloat16* la_f, const __nv_bfloat16* la_b, __nv_bfloat16* out,
                            long long units, int L, int dk, int dv, void* ws, cudaStream_t stream);

// ---- bf16 tcgen05 / TMEM path (units of at most 256 tokens) ----
bool umma_supported(int dk, int dv, int L);
// gate_tau > 0: la_f / la_b hold the gate logits g and the kernel prepares log alpha = logsigmoid(g) / gate_tau itself.
cudaError_t launch_bigla_umma(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                              const __nv_bfloat16* la_f, const __nv_bfloat16* la_b, __nv_bfloat16* out,
                              long long units, int L, int dk, int dv, float gate_tau, cudaStream_t stream);

// ---- Eq. 7 around the mixer: depth-wise 3 x 3 convolution (channels last) and the 2-D gate blend ----
bool dwconv_supported(int C, size_t elem);
template <typename T>
cudaError_t launch_dwconv3x3(const T* x, const T* w, const T* bias, T* out, long long images, int Hh, int Ww, int C,
                             cudaStream_t stream);
template <typename T>
cudaError_t launch_gate_blend(const T* o_local, const T* z, const T* o_global, T* out, long long n, cudaStream_t stream);

// ---- the same kernel for sequences of up to 32 x 256 tokens: one block per 256-token segment, the blocks of a unit
// exchange their segment summaries through scratch memory inside one cooperative launch ----
bool umma_seg_supported(int dk, int dv, int L);
size_t umma_seg_workspace_bytes(long long units, int L);
cudaError_t launch_bigla_umma_seg(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                                  const __nv_bfloat16* la_f, const __nv_bfloat16* la_b, __nv_bfloat16* out,
                                  long long units, int L, int dk, int dv, void* ws, cudaStream_t stream);

// ---- bf16 tcgen05 / TMEM path for longer sequences: chunk tasks, states through scratch (three launches) ----
size_t umma_long_workspace_bytes(long long units, int L, int dk, int dv);
cudaError_t launch_bigla_umma_long(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                                   const __nv_bfloat16* la_f, const __nv_bfloat16* la_b, __nv_bfloat16* out,
                                   long long units, int L, int dk, int dv, void* ws, cudaStream_t stream);

// ---- gradient of the forward pass with respect to q, k and the log gates (fp32 recurrences on the CUDA cores); the
// gradient with respect to v is the forward pass on (k, q, d_out) with the gates from launch_shift_gates ----
bool bwd_supported(int dk, int dv);
size_t bwd_scratch_bytes(long long units, int L, int dk, int dv);   // 0: the device could not be queried
template <typename T>
cudaError_t launch_shift_gates(const T* la_f, const T* la_b, T* out_f, T* out_b, long long units, int L, int dk, cudaStream_t stream);
template <typename T>
cudaError_t launch_bigla_bwd(const T* q, const T* k, const T* v, const T* la_f, const T* la_b, const T* d_out, T* dq, T* dk_out, T* dla_f,
                             T* dla_b, float* scratch, long long units, int L, int dk, int dv, cudaStream_t stream);

// Launch with programmatic stream serialization: the kernel's prologue (everything before its pdl_wait) may overlap
// the tail of the kernel before it in the stream.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Kernel family the bf16 entry points use (a vig_test_kernel value; test_hooks.h): the default unless a test changed it.
int kernel_preference();

}  // namespace vig
