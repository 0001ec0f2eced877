// Gate preparation: log alpha = logsigmoid(g) / tau (paper Eq. 5 line 1), both directions in one launch.
#include <atomic>

#include "ptx.cuh"
#include "vig_internal.h"

namespace vig {

__device__ __forceinline__ float log_alpha_of(float g, float inv_tau) {
    // logsigmoid(g) = min(g, 0) - log1p(exp(-|g|)): no overflow for any finite g
    return (fminf(g, 0.f) - log1pf(expf(-fabsf(g)))) * inv_tau;
}

// The same function for a result that is rounded to bf16 (8 significant bits): exp and log on the
// special-function unit.  With t = e^{-|g|} in (0, 1], log1p(t) is ln 2 * lg2(1 + t) for t >= 2^-6 (absolute
// error of lg2 about 2^-22 against a result of at least 0.022) and its cubic Taylor polynomial below that
// (relative error below t^3 / 4), so the relative error stays below 2e-5 for every finite g, far inside the
// bf16 rounding step.
__device__ __forceinline__ float log_alpha_fast(float g, float inv_tau) {
    float t, l;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(-fabsf(g) * 1.4426950408889634f));
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(l) : "f"(1.0f + t));
    const float big = l * 0.6931471805599453f;
    const float small = t * fmaf(t, fmaf(t, 0.33333334f, -0.5f), 1.0f);
    return (fminf(g, 0.f) - (t < 0.015625f ? small : big)) * inv_tau;
}

__device__ __forceinline__ uint4 log_alpha_bf16x8(uint4 raw, float inv_tau) {
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&raw);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const float2 f = __bfloat1622float2(h[e]);
        h[e] = __floats2bfloat162_rn(log_alpha_fast(f.x, inv_tau), log_alpha_fast(f.y, inv_tau));
    }
    return raw;
}

// 16-byte vector body (4 floats or 8 bf16 per thread) with a scalar tail; blockIdx.y picks the direction.
template <typename T>
__global__ void __launch_bounds__(256) gate_prep_kernel(const T* g_f, const T* g_b, T* la_f, T* la_b, long long n, float inv_tau) {
    // no __restrict__: the output may alias the input (in-place call)
    pdl_launch_dependents();
    pdl_wait();
    const T* g = blockIdx.y == 0 ? g_f : g_b;
    T* la = blockIdx.y == 0 ? la_f : la_b;
    constexpr int V = 16 / sizeof(T);
    const long long nvec = n / V;
    const long long stride = (long long)gridDim.x * blockDim.x;
    long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if constexpr (sizeof(T) == 2) {
        // four independent 16-byte loads in flight per thread
        for (; x + 3 * stride < nvec; x += 4 * stride) {
            uint4 r[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) r[u] = reinterpret_cast<const uint4*>(g)[x + u * stride];
#pragma unroll
            for (int u = 0; u < 4; ++u) reinterpret_cast<uint4*>(la)[x + u * stride] = log_alpha_bf16x8(r[u], inv_tau);
        }
        for (; x < nvec; x += stride) reinterpret_cast<uint4*>(la)[x] = log_alpha_bf16x8(reinterpret_cast<const uint4*>(g)[x], inv_tau);
    } else {
        for (; x < nvec; x += stride) {
            uint4 raw = reinterpret_cast<const uint4*>(g)[x];
            float* f = reinterpret_cast<float*>(&raw);
#pragma unroll
            for (int e = 0; e < 4; ++e) f[e] = log_alpha_of(f[e], inv_tau);
            reinterpret_cast<uint4*>(la)[x] = raw;
        }
    }
    for (x = nvec * V + (long long)blockIdx.x * blockDim.x + threadIdx.x; x < n; x += stride) {
        if constexpr (sizeof(T) == 4) la[x] = log_alpha_of(g[x], inv_tau);
        else la[x] = __float2bfloat16_rn(log_alpha_fast(__bfloat162float(g[x]), inv_tau));
    }
}

// Gradient through the gate preparation: dg = dlog alpha * sigmoid(-g) / tau (d/dg log sigmoid(g) = 1 - sigmoid(g)),
// in fp32; exp only of non-positive numbers.
__device__ __forceinline__ float gate_grad_of(float g, float d, float inv_tau) {
    const float e = __expf(-fabsf(g));
    return d * (g >= 0.f ? e : 1.f) / (1.f + e) * inv_tau;
}

// 16-byte vector body with a scalar tail; blockIdx.y picks the direction.
template <typename T>
__global__ void __launch_bounds__(256) gate_prep_bwd_kernel(const T* g_f, const T* g_b, const T* d_f, const T* d_b, T* o_f, T* o_b, long long n,
                                                            float inv_tau) {
    // no __restrict__: the output may be the incoming gradient's buffer
    pdl_launch_dependents();
    pdl_wait();
    const T* g = blockIdx.y == 0 ? g_f : g_b;
    const T* d = blockIdx.y == 0 ? d_f : d_b;
    T* o = blockIdx.y == 0 ? o_f : o_b;
    constexpr int V = 16 / sizeof(T);
    const long long nvec = n / V, stride = (long long)gridDim.x * blockDim.x;
    for (long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x; x < nvec; x += stride) {
        uint4 rg = reinterpret_cast<const uint4*>(g)[x], rd = reinterpret_cast<const uint4*>(d)[x];
        if constexpr (sizeof(T) == 4) {
            float *fg = reinterpret_cast<float*>(&rg), *fd = reinterpret_cast<float*>(&rd);
#pragma unroll
            for (int e = 0; e < 4; ++e) fd[e] = gate_grad_of(fg[e], fd[e], inv_tau);
        } else {
            __nv_bfloat162 *hg = reinterpret_cast<__nv_bfloat162*>(&rg), *hd = reinterpret_cast<__nv_bfloat162*>(&rd);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 a = __bfloat1622float2(hg[e]), b = __bfloat1622float2(hd[e]);
                hd[e] = __floats2bfloat162_rn(gate_grad_of(a.x, b.x, inv_tau), gate_grad_of(a.y, b.y, inv_tau));
            }
        }
        reinterpret_cast<uint4*>(o)[x] = rd;
    }
    for (long long x = nvec * V + (long long)blockIdx.x * blockDim.x + threadIdx.x; x < n; x += stride) {
        if constexpr (sizeof(T) == 4) o[x] = gate_grad_of(g[x], d[x], inv_tau);
        else o[x] = __float2bfloat16_rn(gate_grad_of(__bfloat162float(g[x]), __bfloat162float(d[x]), inv_tau));
    }
}

static cudaError_t gate_blocks(long long n, int vec, long long* blocks) {
    static std::atomic<int> sms_of[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    int sms = sms_of[dev].load(std::memory_order_relaxed);
    if (sms == 0) {
        const cudaError_t e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        sms_of[dev].store(sms, std::memory_order_relaxed);
    }
    long long b = (n / vec + 255) / 256;
    if (b < 1) b = 1;
    if (b > 4LL * sms) b = 4LL * sms;
    *blocks = b;
    return cudaSuccess;
}

template <typename T>
cudaError_t launch_gate_prep_bwd(const T* g_f, const T* g_b, const T* d_f, const T* d_b, T* o_f, T* o_b, long long n, float tau,
                                 cudaStream_t stream) {
    long long blocks = 1;
    const cudaError_t e = gate_blocks(n, 16 / (int)sizeof(T), &blocks);
    if (e != cudaSuccess) return e;
    const cudaError_t le = launch_pdl(gate_prep_bwd_kernel<T>, dim3((unsigned)blocks, 2), dim3(256), 0, stream, g_f, g_b, d_f, d_b, o_f, o_b, n,
                                      1.0f / tau);
    count_launch();
    return le != cudaSuccess ? le : cudaGetLastError();
}

template <typename T>
cudaError_t launch_gate_prep(const T* g_f, const T* g_b, T* la_f, T* la_b, long long n, float tau,
                             cudaStream_t stream) {
    constexpr int V = 16 / sizeof(T);
    const int threads = 256;
    long long blocks = (n / V + threads - 1) / threads;
    if (blocks < 1) blocks = 1;
    // both directions together: eight blocks per SM (the SM count of the current device, queried once per device)
    static std::atomic<int> sms_of[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    int sms = sms_of[dev].load(std::memory_order_relaxed);
    if (sms == 0) {
        const cudaError_t e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        sms_of[dev].store(sms, std::memory_order_relaxed);
    }
    if (blocks > 4LL * sms) blocks = 4LL * sms;
    const cudaError_t le = launch_pdl(gate_prep_kernel<T>, dim3((unsigned)blocks, 2), dim3(threads), 0, stream, g_f, g_b, la_f, la_b, n, 1.0f / tau);
    count_launch();
    return le != cudaSuccess ? le : cudaGetLastError();
}

template cudaError_t launch_gate_prep_bwd<float>(const float*, const float*, const float*, const float*, float*, float*, long long, float,
                                                 cudaStream_t);
template cudaError_t launch_gate_prep_bwd<__nv_bfloat16>(const __nv_bfloat16*, const __nv_bfloat16*, const __nv_bfloat16*,
                                                         const __nv_bfloat16*, __nv_bfloat16*, __nv_bfloat16*, long long, float, cudaStream_t);
template cudaError_t launch_gate_prep<float>(const float*, const float*, float*, float*, long long, float,
                                             cudaStream_t);
template cudaError_t launch_gate_prep<__nv_bfloat16>(const __nv_bfloat16*, const __nv_bfloat16*, __nv_bfloat16*,
                                                     __nv_bfloat16*, long long, float, cudaStream_t);

}  // namespace vig
