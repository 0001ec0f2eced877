// The two element-wise neighbours of BiGLA in the 2-D gating locality injection (paper Eq. 7):
//   line 1     O_local = DWConv3x3(X): depth-wise 3 x 3 convolution over the patch grid (channels last)
//   lines 3-4  O = G * O_local + (1 - G) * O_global with G = sigmoid(z), z = O_local W + b given by the caller
// The blend is bound by memory traffic; the convolution reads every input once through tiled TMA loads and is then
// bound by its multiply-adds.
#include <atomic>

#include "ptx.cuh"
#include "tma_host.h"
#include "vig_internal.h"

namespace vig {

namespace {

template <typename T>
struct Vec;   // 16 bytes of T: Raw as loaded, N fp32 lanes unpacked
template <>
struct Vec<float> {
    static constexpr int N = 4;
    using Raw = float4;
    static __device__ __forceinline__ Raw zero() { return make_float4(0.f, 0.f, 0.f, 0.f); }
    static __device__ __forceinline__ void unpack(const Raw& v, float (&f)[4]) { f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w; }
    static __device__ __forceinline__ void unpack2x(const Raw& v, f32x2 (&f)[2]) { f[0] = pack2(v.x, v.y); f[1] = pack2(v.z, v.w); }
    static __device__ __forceinline__ void load(const float* p, float (&f)[4]) { unpack(*reinterpret_cast<const float4*>(p), f); }
    static __device__ __forceinline__ void store(float* p, const float (&f)[4]) {
        *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]);
    }
};
template <>
struct Vec<__nv_bfloat16> {
    static constexpr int N = 8;
    using Raw = uint4;
    static __device__ __forceinline__ Raw zero() { return make_uint4(0u, 0u, 0u, 0u); }
    static __device__ __forceinline__ void unpack(const Raw& v, float (&f)[8]) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            const float2 t = unpack_bf16(w[x]);
            f[2 * x] = t.x;
            f[2 * x + 1] = t.y;
        }
    }
    static __device__ __forceinline__ void unpack2x(const Raw& v, f32x2 (&f)[4]) {   // a bf16 is the upper half of its fp32
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int x = 0; x < 4; ++x) f[x] = pack2(__uint_as_float(w[x] << 16), __uint_as_float(w[x] & 0xffff0000u));
    }
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&f)[8]) { unpack(*reinterpret_cast<const uint4*>(p), f); }
    static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&f)[8]) {
        *reinterpret_cast<uint4*>(p) = make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
    }
};

__device__ __forceinline__ float to_f(float x) { return x; }
__device__ __forceinline__ float to_f(__nv_bfloat16 x) { return __bfloat162float(x); }

// Depth-wise 3 x 3 convolution, fp32 accumulation, zero padding, cross-correlation:
//   out[n, i, j, c] = b[c] + sum_{di, dj} w[c, di + 1, dj + 1] x[n, i + di, j + dj, c].
// Task = th output rows x tw columns of one image for one slab of gpb channel groups (a group = 16 bytes of channels).  Its
// input tile with the one-pixel halo, (th + 2) x (tw + 2) x gpb groups, comes by ONE tiled TMA load, which also supplies
// the zero padding (coordinates outside the image read as zero) - the bytes in flight occupy no registers, and an
// input element crosses L2 once per tile that needs it instead of nine times.  A block keeps its slab (blockIdx.y) and
// strides over tasks with two tile buffers: the next tile loads while this one is worked on.
// Thread = one channel group of one column: its V filters (nine taps each, 144 contiguous bytes of w) and biases sit
// in registers as fp32 pairs (two channels per packed multiply-add); walking down the tile it reads three 16-byte pieces per input row (left, centre, right) from
// shared memory and adds them into the three output rows they touch, which live in rolling accumulators.  Lanes run
// over channel groups first, so shared-memory reads and the 16-byte output stores are contiguous per warp.
template <typename T>
__global__ void __launch_bounds__(256) dwconv3x3_kernel(const __grid_constant__ CUtensorMap tm_x, const T* __restrict__ w,
                                                        const T* __restrict__ bias, T* __restrict__ out, int Hh, int Ww, int C, int gpb, int tw,
                                                        int th, int rowsegs, int coltiles, int tasks, int* dev_status) {
    constexpr int V = Vec<T>::N;
    using Raw = typename Vec<T>::Raw;
    extern __shared__ __align__(128) uint8_t dw_smem[];
    __shared__ __align__(8) unsigned long long dw_bar[2];
    const uint32_t tile_bytes = (uint32_t)(th + 2) * (tw + 2) * gpb * 16;
    const uint32_t buf_pitch = (tile_bytes + 127) / 128 * 128;
    const uint32_t bar0 = smem_u32(dw_bar);
    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        mbar_init(bar0, 1);
        mbar_init(bar0 + 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const int col = threadIdx.x / gpb, g = threadIdx.x % gpb;
    const int c_slab = blockIdx.y * gpb * V, c0 = c_slab + g * V;
    const bool chan_live = c0 < C;   // ragged last slab
    auto issue = [&](int task, int buf) {   // one thread: the tile of `task` into buffer `buf`
        const int j0 = (task % coltiles) * tw, i0 = ((task / coltiles) % rowsegs) * th, n = task / (coltiles * rowsegs);
        mbar_expect_tx(bar0 + 8 * buf, tile_bytes);
        tma_load_4d(smem_u32(dw_smem) + buf * buf_pitch, &tm_x, c_slab, j0 - 1, i0 - 1, n, bar0 + 8 * buf);
    };
    pdl_wait();   // x may be the output of the kernel before this one in the stream
    if (threadIdx.x == 0 && (int)blockIdx.x < tasks) issue(blockIdx.x, 0);
    f32x2 wr[9][V / 2], br[V / 2];   // filter taps and biases of the thread's channels as fp32 pairs
#pragma unroll
    for (int u = 0; u < V / 2; ++u) br[u] = 0ull;
    if (chan_live) {
        float t[9 * V];   // w[c0 .. c0 + V)[3][3]: 9 V contiguous elements = nine 16-byte pieces
#pragma unroll
        for (int x9 = 0; x9 < 9; ++x9) {
            float f[V];
            Vec<T>::load(w + (size_t)c0 * 9 + x9 * V, f);
#pragma unroll
            for (int u = 0; u < V; ++u) t[x9 * V + u] = f[u];
        }
#pragma unroll
        for (int tap = 0; tap < 9; ++tap)
#pragma unroll
            for (int u = 0; u < V / 2; ++u) wr[tap][u] = pack2(t[(2 * u) * 9 + tap], t[(2 * u + 1) * 9 + tap]);
        if (bias) {
            float f[V];
            Vec<T>::load(bias + c0, f);
#pragma unroll
            for (int u = 0; u < V / 2; ++u) br[u] = pack2(f[2 * u], f[2 * u + 1]);
        }
    }
    const uint32_t row_pitch_s = (uint32_t)(tw + 2) * gpb * 16;   // one tile row in shared memory
    const size_t row_pitch_g = (size_t)Ww * C;
    int it = 0;
    for (int task = blockIdx.x; task < tasks; task += gridDim.x, ++it) {
        const int buf = it & 1;
        // (every thread has left the other buffer: the barrier that ended the previous round)
        if (threadIdx.x == 0 && task + (int)gridDim.x < tasks) issue(task + gridDim.x, buf ^ 1);
        const bool arrived = mbar_wait_bounded(bar0 + 8 * buf, (it >> 1) & 1);
        if (!__syncthreads_and(arrived)) {   // a load that never lands: report it and leave, all threads together
            if (threadIdx.x == 0) atomicOr(dev_status, kDevStatusTimeout);
            break;
        }
        const int j0 = (task % coltiles) * tw, i0 = ((task / coltiles) % rowsegs) * th, n = task / (coltiles * rowsegs);
        const int j = j0 + col, rows = min(th, Hh - i0);   // output rows i0 .. i0 + rows - 1
        if (chan_live && j < Ww) {
            const uint8_t* tp = dw_smem + buf * buf_pitch + ((uint32_t)col * gpb + g) * 16;   // tile row 0, column j - 1
            T* op = out + (((size_t)n * Hh + i0) * Ww + j) * C + c0;
            // a_up: the output row above the input row at hand (complete with it), a_mid: the one at it, a_dn: the one below
            f32x2 a_up[V / 2], a_mid[V / 2];
#pragma unroll
            for (int u = 0; u < V / 2; ++u) a_up[u] = a_mid[u] = br[u];
            for (int r = 0; r < rows + 2; ++r) {   // tile row r = input row i0 - 1 + r (zeros outside the image)
                f32x2 in[3][V / 2];
#pragma unroll
                for (int d = 0; d < 3; ++d)
                    Vec<T>::unpack2x(*reinterpret_cast<const Raw*>(tp + (uint32_t)r * row_pitch_s + (uint32_t)d * gpb * 16), in[d]);
                f32x2 a_dn[V / 2];
#pragma unroll
                for (int u = 0; u < V / 2; ++u) {   // two channels per instruction (packed fp32 multiply-add)
                    a_dn[u] = br[u];
#pragma unroll
                    for (int d = 0; d < 3; ++d) {
                        a_up[u] = ffma2(wr[6 + d][u], in[d][u], a_up[u]);
                        a_mid[u] = ffma2(wr[3 + d][u], in[d][u], a_mid[u]);
                        a_dn[u] = ffma2(wr[d][u], in[d][u], a_dn[u]);
                    }
                }
                if (r >= 2) {
                    float o[V];
#pragma unroll
                    for (int u = 0; u < V / 2; ++u) unpack2(a_up[u], o[2 * u], o[2 * u + 1]);
                    Vec<T>::store(op + (size_t)(r - 2) * row_pitch_g, o);
                }
#pragma unroll
                for (int u = 0; u < V / 2; ++u) {
                    a_up[u] = a_mid[u];
                    a_mid[u] = a_dn[u];
                }
            }
        }
        __syncthreads();   // the tile may be overwritten by the load after next
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

bool dwconv_supported(int C, size_t elem) { return C >= 1 && C % (int)(16 / elem) == 0 && C <= (1 << 20); }

template <typename T>
cudaError_t launch_dwconv3x3(const T* x, const T* w, const T* bias, T* out, long long images, int Hh, int Ww, int C, cudaStream_t stream) {
    int sms = 0;
    cudaError_t e = sm_count(&sms);
    if (e != cudaSuccess) return e;
    constexpr int V = (int)(16 / sizeof(T));
    const int groups = C / V;
    const int slabs = (groups + 15) / 16, gpb = (groups + slabs - 1) / slabs;   // channel groups per block: at most 16
    const int tw_max = 256 / gpb < 254 ? 256 / gpb : 254;   // at most 256 threads; the tile with its halo at most 256 columns (a TMA box)
    const int coltiles = (Ww + tw_max - 1) / tw_max, tw = (Ww + coltiles - 1) / coltiles;
    const int rowsegs = (Hh + 7) / 8, th = (Hh + rowsegs - 1) / rowsegs;                            // at most 8 output rows per tile
    const long long tasks = images * rowsegs * coltiles;
    if (tasks > 0x7fffffffLL || slabs > 65535 || tw + 2 > 256) return cudaErrorInvalidValue;
    const size_t tile = (size_t)(th + 2) * (tw + 2) * gpb * 16, smem = 2 * ((tile + 127) / 128 * 128);
    if (smem > 200 * 1024) return cudaErrorInvalidValue;
    static std::atomic<bool> configured[64];
    int dev = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev].load(std::memory_order_acquire)) {
        if ((e = cudaFuncSetAttribute(dwconv3x3_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024)) != cudaSuccess) return e;
        configured[dev].store(true, std::memory_order_release);
    }
    CUtensorMap tm;
    if (!make_map_nhwc(&tm, x, images, Hh, Ww, C, (int)sizeof(T), gpb * V, tw + 2, th + 2)) return cudaErrorInvalidValue;
    int* status = device_status_ptr();
    if (!status) return cudaErrorInvalidValue;
    long long nb = 2LL * sms / slabs;   // two blocks per SM over all slabs
    if (nb < 1) nb = 1;
    if (nb > tasks) nb = tasks;
    const cudaError_t le = launch_pdl(dwconv3x3_kernel<T>, dim3((unsigned)nb, (unsigned)slabs), dim3((unsigned)(tw * gpb)), smem, stream, tm, w,
                                      bias, out, Hh, Ww, C, gpb, tw, th, rowsegs, coltiles, (int)tasks, status);
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
