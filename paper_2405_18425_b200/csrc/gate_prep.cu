// Gate preparation: log alpha = logsigmoid(g) / tau (paper Eq. 5 line 1), both directions in one launch.
#include "vig_internal.h"

namespace vig {

__device__ __forceinline__ float log_alpha_of(float g, float inv_tau) {
    // logsigmoid(g) = min(g, 0) - log1p(exp(-|g|)): no overflow for any finite g
    return (fminf(g, 0.f) - log1pf(expf(-fabsf(g)))) * inv_tau;
}

// 16-byte vector body (4 floats or 8 bf16 per thread) with a scalar tail; blockIdx.y picks the direction.
template <typename T>
__global__ void gate_prep_kernel(const T* g_f, const T* g_b, T* la_f, T* la_b, long long n, float inv_tau) {
    // no __restrict__: the output may alias the input (in-place call)
    const T* g = blockIdx.y == 0 ? g_f : g_b;
    T* la = blockIdx.y == 0 ? la_f : la_b;
    constexpr int V = 16 / sizeof(T);
    const long long nvec = n / V;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x; x < nvec; x += stride) {
        uint4 raw = reinterpret_cast<const uint4*>(g)[x];
        if constexpr (sizeof(T) == 4) {
            float* f = reinterpret_cast<float*>(&raw);
#pragma unroll
            for (int e = 0; e < 4; ++e) f[e] = log_alpha_of(f[e], inv_tau);
        } else {
            __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&raw);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float2 f = __bfloat1622float2(h[e]);
                f.x = log_alpha_of(f.x, inv_tau);
                f.y = log_alpha_of(f.y, inv_tau);
                h[e] = __floats2bfloat162_rn(f.x, f.y);
            }
        }
        reinterpret_cast<uint4*>(la)[x] = raw;
    }
    for (long long x = nvec * V + (long long)blockIdx.x * blockDim.x + threadIdx.x; x < n; x += stride) {
        if constexpr (sizeof(T) == 4) la[x] = log_alpha_of(g[x], inv_tau);
        else la[x] = __float2bfloat16_rn(log_alpha_of(__bfloat162float(g[x]), inv_tau));
    }
}

template <typename T>
cudaError_t launch_gate_prep(const T* g_f, const T* g_b, T* la_f, T* la_b, long long n, float tau,
                             cudaStream_t stream) {
    constexpr int V = 16 / sizeof(T);
    const int threads = 256;
    long long blocks = (n / V + threads - 1) / threads;
    if (blocks < 1) blocks = 1;
    if (blocks > 148 * 8) blocks = 148 * 8;
    gate_prep_kernel<T><<<dim3((unsigned)blocks, 2), threads, 0, stream>>>(g_f, g_b, la_f, la_b, n, 1.0f / tau);
    count_launch();
    return cudaGetLastError();
}

template cudaError_t launch_gate_prep<float>(const float*, const float*, float*, float*, long long, float,
                                             cudaStream_t);
template cudaError_t launch_gate_prep<__nv_bfloat16>(const __nv_bfloat16*, const __nv_bfloat16*, __nv_bfloat16*,
                                                     __nv_bfloat16*, long long, float, cudaStream_t);

}  // namespace vig
