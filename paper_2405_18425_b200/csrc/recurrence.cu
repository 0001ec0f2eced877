// fp32 SIMT kernel: one thread block evaluates Eq. 6 step by step for one (batch, head) unit.
#include "recurrence.cuh"
#include "vig_internal.h"

namespace vig {

template <typename T>
__global__ void bigla_recurrence_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                                        const T* __restrict__ la_f, const T* __restrict__ la_b, T* __restrict__ out,
                                        int L, int dk, int dv) {
    extern __shared__ __align__(16) float rec_smem[];
    const size_t u = blockIdx.x;
    const size_t ok = u * (size_t)L * dk, ov = u * (size_t)L * dv;
    recurrence_unit<T>(q + ok, k + ok, v + ov, la_f + ok, la_b + ok, out + ov, L, dk, dv, rec_smem);
}

// Block size: dv columns times enough key-dim groups that a thread keeps at most 16 state rows
// (32 when that would exceed 1024 threads).
static int rec_threads(int dk, int dv) {
    int P = (dk + 15) / 16;
    if ((long long)dv * P > 1024) P = (dk + kRecR - 1) / kRecR;
    int nt = dv * P;
    nt = (nt + 31) / 32 * 32;
    return nt;
}

bool recurrence_supported(int dk, int dv) {
    if (dk < 1 || dv < 1 || dk > 128 || dv > 256) return false;
    const int nt = rec_threads(dk, dv);
    if (nt > 1024 || nt < dv) return false;
    const RecPlan pl = rec_plan(nt, dk, dv);
    return pl.Rn <= kRecR && (size_t)pl.smem_floats * 4 <= 200 * 1024;
}

template <typename T>
cudaError_t launch_recurrence(const T* q, const T* k, const T* v, const T* la_f, const T* la_b, T* out,
                              long long units, int L, int dk, int dv, cudaStream_t stream) {
    const int nt = rec_threads(dk, dv);
    const RecPlan pl = rec_plan(nt, dk, dv);
    const size_t smem = (size_t)pl.smem_floats * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(bigla_recurrence_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return e;
    bigla_recurrence_kernel<T><<<(unsigned)units, nt, smem, stream>>>(q, k, v, la_f, la_b, out, L, dk, dv);
    count_launch();
    return cudaGetLastError();
}

template cudaError_t launch_recurrence<float>(const float*, const float*, const float*, const float*, const float*,
                                              float*, long long, int, int, int, cudaStream_t);
template cudaError_t launch_recurrence<__nv_bfloat16>(const __nv_bfloat16*, const __nv_bfloat16*,
                                                      const __nv_bfloat16*, const __nv_bfloat16*,
                                                      const __nv_bfloat16*, __nv_bfloat16*, long long, int, int, int,
                                                      cudaStream_t);

}  // namespace vig
