// The two element-wise neighbours of BiGLA in the 2-D gating locality injection (paper Eq. 7):
//   line 1     O_local = DWConv3x3(X): depth-wise 3 x 3 convolution over the patch grid (channels last)
//   lines 3-4  O = G * O_local + (1 - G) * O_global with G = sigmoid(z), z = O_local W + b given by the caller
// Both are bound by memory traffic; the blend also exists as the epilogue of the forward kernel (bigla_umma.cu).
#include <atomic>

#include "ptx.cuh"
#include "vig_internal.h"

namespace vig {

namespace {

template <typename T>
struct Vec;   // 16 bytes of T as fp32 lanes
template <>
struct Vec<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ void load(const float* p, float (&f)[4]) {
        const float4 v = *reinterpret_cast<const float4*>(p);
        f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
    }
    static __device__ __forceinline__ void store(float* p, const float (&f)[4]) {
        *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]);
    }
};
template <>
struct Vec<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&f)[8]) {
        const uint4 v = *reinterpret_cast<const uint4*>(p);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            const float2 t = unpack_bf16(w[x]);
            f[2 * x] = t.x;
            f[2 * x + 1] = t.y;
        }
    }
    static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&f)[8]) {
        *reinterpret_cast<uint4*>(p) = make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
    }
};

__device__ __forceinline__ float to_f(float x) { return x; }
__device__ __forceinline__ float to_f(__nv_bfloat16 x) { return __bfloat162float(x); }

// Thread = one pixel x one group of V channels (16 bytes).  The filters sit in shared memory as fp32, tap major
// ([9][C]), so that the V channels of a tap are one or two 16-byte reads; the nine neighbours come through L1 / L2 (each
// input line is used by the nine pixels around it).  fp32 accumulation, zero padding, cross-correlation:
//   out[n, i, j, c] = b[c] + sum_{di, dj} w[c, di + 1, dj + 1] x[n, i + di, j + dj, c].
template <typename T>
__global__ void __launch_bounds__(256) dwconv3x3_kernel(const T* __restrict__ x, const T* __restrict__ w, const T* __restrict__ bias,
                                                        T* __restrict__ out, long long pixels, int Hh, int Ww, int C) {
    constexpr int V = Vec<T>::N;
    extern __shared__ __align__(16) float wsm[];   // [9][C] then the bias [C]
    pdl_launch_dependents();
    pdl_wait();
    for (int e = threadIdx.x; e < 9 * C; e += blockDim.x) {
        const int c = e / 9, tap = e - 9 * c;
        wsm[tap * C + c] = to_f(w[e]);
    }
    for (int c = threadIdx.x; c < C; c += blockDim.x) wsm[9 * C + c] = bias ? to_f(bias[c]) : 0.f;
    __syncthreads();
    const int groups = C / V;
    const long long total = pixels * groups;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long long)gridDim.x * blockDim.x) {
        const long long pix = idx / groups;
        const int c0 = (int)(idx - pix * groups) * V;
        const int j = (int)(pix % Ww), i = (int)((pix / Ww) % Hh);
        float acc[V];
#pragma unroll
        for (int u = 0; u < V; ++u) acc[u] = wsm[9 * C + c0 + u];
#pragma unroll
        for (int di = -1; di <= 1; ++di) {
#pragma unroll
            for (int dj = -1; dj <= 1; ++dj) {
                if (i + di < 0 || i + di >= Hh || j + dj < 0 || j + dj >= Ww) continue;   // zero padding
                float xv[V];
                Vec<T>::load(x + ((pix + (long long)di * Ww + dj) * C + c0), xv);
                const float* wt = wsm + ((di + 1) * 3 + (dj + 1)) * C + c0;
#pragma unroll
                for (int u = 0; u < V; ++u) acc[u] = fmaf(wt[u], xv[u], acc[u]);
            }
        }
        Vec<T>::store(out + (pix * C + c0), acc);
    }
}

// O = G * O_local + (1 - G) * O_global, G = sigmoid(z) = 1 / (1 + e^{-z}) in fp32 (no overflow: e^{-|z|} <= 1).
__device__ __forceinline__ float blend_one(float ol, float z, float og) {
    const float e = __expf(-fabsf(z));
    const float g = (z >= 0.f ? 1.f : e) / (1.f + e);
    return fmaf(g, ol - og, og);
}

template <typename T>
__global__ void __launch_bounds__(256) gate_blend_kernel(const T* o_local, const T* z, const T* o_global, T* out, long long n) {
    // no __restrict__: out may be o_global (in-place call)
    constexpr int V = Vec<T>::N;
    pdl_launch_dependents();
    pdl_wait();
    const long long nvec = n / V, stride = (long long)gridDim.x * blockDim.x;
    for (long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x; x < nvec; x += stride) {
        float a[V], b[V], c[V];
        Vec<T>::load(o_local + x * V, a);
        Vec<T>::load(z + x * V, b);
        Vec<T>::load(o_global + x * V, c);
#pragma unroll
        for (int u = 0; u < V; ++u) a[u] = blend_one(a[u], b[u], c[u]);
        Vec<T>::store(out + x * V, a);
    }
    for (long long x = nvec * V + (long long)blockIdx.x * blockDim.x + threadIdx.x; x < n; x += stride) {
        const float r = blend_one(to_f(o_local[x]), to_f(z[x]), to_f(o_global[x]));
        if constexpr (sizeof(T) == 4) out[x] = r;
        else out[x] = __float2bfloat16_rn(r);
    }
}

cudaError_t sm_count(int* sms) {
    static std::atomic<int> sms_of[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    int s = sms_of[dev].load(std::memory_order_relaxed);
    if (s == 0) {
        const cudaError_t e = cudaDeviceGetAttribute(&s, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        sms_of[dev].store(s, std::memory_order_relaxed);
    }
    *sms = s;
    return cudaSuccess;
}

}  // namespace

bool dwconv_supported(int C, size_t elem) { return C >= 1 && C % (int)(16 / elem) == 0 && (size_t)10 * C * 4 <= 200 * 1024; }

template <typename T>
cudaError_t launch_dwconv3x3(const T* x, const T* w, const T* bias, T* out, long long images, int Hh, int Ww, int C, cudaStream_t stream) {
    int sms = 0;
    cudaError_t e = sm_count(&sms);
    if (e != cudaSuccess) return e;
    const size_t smem = (size_t)10 * C * sizeof(float);
    if (smem > 48 * 1024) {
        e = cudaFuncSetAttribute(dwconv3x3_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    const long long pixels = images * Hh * Ww, work = pixels * (C / (int)(16 / sizeof(T)));
    long long blocks = (work + 255) / 256;
    if (blocks > 8LL * sms) blocks = 8LL * sms;
    const cudaError_t le = launch_pdl(dwconv3x3_kernel<T>, dim3((unsigned)blocks), dim3(256), smem, stream, x, w, bias, out, pixels, Hh, Ww, C);
    count_launch();
    return le != cudaSuccess ? le : cudaGetLastError();
}

template <typename T>
cudaError_t launch_gate_blend(const T* o_local, const T* z, const T* o_global, T* out, long long n, cudaStream_t stream) {
    int sms = 0;
    cudaError_t e = sm_count(&sms);
    if (e != cudaSuccess) return e;
    long long blocks = (n / (long long)(16 / sizeof(T)) + 255) / 256;
    if (blocks < 1) blocks = 1;
    if (blocks > 8LL * sms) blocks = 8LL * sms;
    const cudaError_t le = launch_pdl(gate_blend_kernel<T>, dim3((unsigned)blocks), dim3(256), 0, stream, o_local, z, o_global, out, n);
    count_launch();
    return le != cudaSuccess ? le : cudaGetLastError();
}

template cudaError_t launch_dwconv3x3<float>(const float*, const float*, const float*, float*, long long, int, int, int, cudaStream_t);
template cudaError_t launch_dwconv3x3<__nv_bfloat16>(const __nv_bfloat16*, const __nv_bfloat16*, const __nv_bfloat16*, __nv_bfloat16*,
                                                     long long, int, int, int, cudaStream_t);
template cudaError_t launch_gate_blend<float>(const float*, const float*, const float*, float*, long long, cudaStream_t);
template cudaError_t launch_gate_blend<__nv_bfloat16>(const __nv_bfloat16*, const __nv_bfloat16*, const __nv_bfloat16*, __nv_bfloat16*,
                                                      long long, cudaStream_t);

}  // namespace vig
