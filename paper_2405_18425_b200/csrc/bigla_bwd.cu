// Gradient of the BiGLA forward pass (paper Eq. 6) with respect to q, k and the two log gates, by the reverse-mode
// adjoint of the two recurrences, in fp32 on the CUDA cores; the gradient with respect to v is a forward pass on swapped
// operands (see shift_gates below) and is launched by the caller of these kernels.
//
// With g = dLoss/d_out, a> = exp(log alpha>), a< = exp(log alpha<), per unit and token t:
//   S>_t = a>_t S>_{t-1} + k_t^T v_t            (Eq. 6)            dq>_t = S>_t g_t^T / 2
//   Z>_t = a>_{t+1} Z>_{t+1} + q_t^T g_t / 2    (adjoint of S>_t)   dk>_t = Z>_t v_t^T
//   S<_t = a<_t S<_{t+1} + k_t^T v_t            (Eq. 6)            dq<_t = S<_t g_t^T / 2
//   Z<_t = a<_{t-1} Z<_{t-1} + q_t^T g_t / 2    (adjoint of S<_t)   dk<_t = Z<_t v_t^T
//   dq = dq> + dq<,  dk = dk> + dk<
// The log gates enter only through sums of gates between a key and a query, so with E>_t = q_t * dq>_t - k_t * dk>_t
// (element-wise) and E<_t likewise:   dlog alpha>_t = sum_{m >= t} E>_m,   dlog alpha<_t = sum_{m <= t} E<_m
// = - sum_{m > t} E<_m  (each direction is unchanged by q -> q / c, k -> c k per key dimension, so sum_m E_m = 0).
//
// One block per unit walks the sequence twice.  The ascending walk carries S> and Z< and leaves dq>_t, dk<_t in fp32
// scratch; the descending walk carries S< and Z>, reads them back and finishes all four outputs, the gate gradients as
// running sums in walking order.  Thread (i, cg) keeps columns [cg CN, cg CN + CN) of row i of both dk x dv matrices in
// registers; the sums over the value dimension are finished over the four lanes of a row by shuffles.  Inputs and
// outputs pass through shared memory sixteen tokens at a time, so global memory sees whole rows.
#include <atomic>

#include "recurrence.cuh"
#include "vig_internal.h"

namespace vig {

namespace {

constexpr int kBwdTT = 16;   // tokens staged at once
constexpr int kBwdCG = 4;    // threads (lanes) per state row

template <typename T>
struct BwdArgs {
    const T *q, *k, *v, *la_f, *la_b, *g;
    T *dq, *dkey, *dla_f, *dla_b;
    float* scratch;   // [units][2][L][dk] fp32: dq>, dk< between the two walks
    long long units;
    int L, dk, dv;
};

// rows: state rows a block holds (threads / 4, >= dk); the padded rows and columns work on zeros.
__host__ __device__ inline size_t bwd_smem_floats(int rows, int cn) {
    return (size_t)kBwdTT * (10 * rows + 2 * kBwdCG * cn);
}

template <typename T, int CN>
__global__ void __launch_bounds__(512) bigla_bwd_kernel(BwdArgs<T> a) {
    extern __shared__ __align__(16) float bw_smem[];
    const int tid = threadIdx.x, nt = blockDim.x;
    const int rows = nt / kBwdCG, cols = kBwdCG * CN;
    const int i = tid / kBwdCG, cg = tid % kBwdCG;
    const int L = a.L, dk = a.dk, dv = a.dv;
    float* qs = bw_smem;                      // [TT][rows] each
    float* ks = qs + kBwdTT * rows;
    float* a1 = ks + kBwdTT * rows;           // decay of the S state at this token
    float* a2 = a1 + kBwdTT * rows;           // decay of the Z state: the gate of the token walked just before
    float* x1 = a2 + kBwdTT * rows;           // descending walk: dq>, dk< from scratch
    float* x2 = x1 + kBwdTT * rows;
    float* o1 = x2 + kBwdTT * rows;           // results of sixteen tokens
    float* o2 = o1 + kBwdTT * rows;
    float* o3 = o2 + kBwdTT * rows;
    float* o4 = o3 + kBwdTT * rows;
    float* vs = o4 + kBwdTT * rows;           // [TT][cols] each
    float* gs = vs + kBwdTT * cols;
    for (size_t x = tid; x < bwd_smem_floats(rows, CN); x += nt) bw_smem[x] = 0.f;   // the padding stays zero
    __syncthreads();
    const int nchunk = (L + kBwdTT - 1) / kBwdTT;

    for (long long unit = blockIdx.x; unit < a.units; unit += gridDim.x) {
        const size_t ok = (size_t)unit * L * dk, ov = (size_t)unit * L * dv;
        float* sc1 = a.scratch + (size_t)unit * 2 * L * dk;
        float* sc2 = sc1 + (size_t)L * dk;
        for (int walk = 0; walk < 2; ++walk) {
            const T* la_s = walk == 0 ? a.la_f : a.la_b;   // gates of the S state
            const T* la_z = walk == 0 ? a.la_b : a.la_f;   // gates of the Z state
            const int step = walk == 0 ? 1 : -1;
            float S[CN], Z[CN];
#pragma unroll
            for (int c = 0; c < CN; ++c) S[c] = Z[c] = 0.f;
            float run_f = 0.f, run_b = 0.f;   // running sums of E> and E< (descending walk)
            for (int cc = 0; cc < nchunk; ++cc) {
                const int t0 = (walk == 0 ? cc : nchunk - 1 - cc) * kBwdTT;
                const int nv = min(kBwdTT, L - t0);
                for (int x = tid; x < nv * dk; x += nt) {
                    const int tt = x / dk, r = x - tt * dk, t = t0 + tt;
                    const size_t gi = ok + (size_t)t * dk + r;
                    qs[tt * rows + r] = rec_to_float(a.q[gi]);
                    ks[tt * rows + r] = rec_to_float(a.k[gi]);
                    a1[tt * rows + r] = expf(rec_to_float(la_s[gi]));
                    const int tp = t - step;   // the token walked before t
                    a2[tt * rows + r] = (tp >= 0 && tp < L) ? expf(rec_to_float(la_z[ok + (size_t)tp * dk + r])) : 0.f;
                    if (walk == 1) {
                        x1[tt * rows + r] = sc1[(size_t)t * dk + r];
                        x2[tt * rows + r] = sc2[(size_t)t * dk + r];
                    }
                }
                for (int x = tid; x < nv * dv; x += nt) {
                    const int tt = x / dv, j = x - tt * dv;
                    vs[tt * cols + j] = rec_to_float(a.v[ov + (size_t)(t0 + tt) * dv + j]);
                    gs[tt * cols + j] = rec_to_float(a.g[ov + (size_t)(t0 + tt) * dv + j]);
                }
                __syncthreads();
                for (int n = 0; n < nv; ++n) {
                    const int tt = walk == 0 ? n : nv - 1 - n;
                    const float kq = ks[tt * rows + i], qv = qs[tt * rows + i], hq = 0.5f * qv;
                    const float ds = a1[tt * rows + i], dz = a2[tt * rows + i];
                    const float* vr = vs + tt * cols + cg * CN;
                    const float* gr = gs + tt * cols + cg * CN;
                    float accq = 0.f, acck = 0.f;
#pragma unroll
                    for (int c = 0; c < CN; ++c) {
                        const float vj = vr[c], gj = gr[c];
                        S[c] = fmaf(ds, S[c], kq * vj);
                        accq = fmaf(S[c], gj, accq);
                        Z[c] = fmaf(dz, Z[c], hq * gj);
                        acck = fmaf(Z[c], vj, acck);
                    }
                    accq += __shfl_xor_sync(0xffffffffu, accq, 1);
                    acck += __shfl_xor_sync(0xffffffffu, acck, 1);
                    accq += __shfl_xor_sync(0xffffffffu, accq, 2);
                    acck += __shfl_xor_sync(0xffffffffu, acck, 2);
                    accq *= 0.5f;
                    if (walk == 0) {
                        if (cg == 0) {
                            o1[tt * rows + i] = accq;   // dq>_t
                            o2[tt * rows + i] = acck;   // dk<_t
                        }
                    } else {
                        const float dqf = x1[tt * rows + i], dkb = x2[tt * rows + i];   // accq = dq<_t, acck = dk>_t
                        run_f += qv * dqf - kq * acck;
                        if (cg == 0) {
                            o1[tt * rows + i] = dqf + accq;
                            o2[tt * rows + i] = acck + dkb;
                            o3[tt * rows + i] = run_f;     // sum over m >= t of E>_m
                            o4[tt * rows + i] = -run_b;    // minus the sum over m > t of E<_m
                        }
                        run_b += qv * accq - kq * dkb;
                    }
                }
                __syncthreads();
                for (int x = tid; x < nv * dk; x += nt) {
                    const int tt = x / dk, r = x - tt * dk;
                    const size_t t = (size_t)(t0 + tt);
                    if (walk == 0) {
                        sc1[t * dk + r] = o1[tt * rows + r];
                        sc2[t * dk + r] = o2[tt * rows + r];
                    } else {
                        rec_store(a.dq + ok + t * dk + r, o1[tt * rows + r]);
                        rec_store(a.dkey + ok + t * dk + r, o2[tt * rows + r]);
                        rec_store(a.dla_f + ok + t * dk + r, o3[tt * rows + r]);
                        rec_store(a.dla_b + ok + t * dk + r, o4[tt * rows + r]);
                    }
                }
                // (the next chunk's staging writes other arrays; its results wait behind the barrier after staging)
            }
            __syncthreads();   // the scratch of the ascending walk is read back by other threads
        }
    }
}

// la_f'[t] = la_b[t - 1] (0 at t = 0), la_b'[t] = la_f[t + 1] (0 at t = L - 1): with these gates, d_out as the values and
// q, k swapped, the forward pass IS the gradient with respect to v:
//   dv_r = 1/2 sum_{t >= r} (k_r * prod_{m = r+1..t} alpha>_m . q_t) g_t + 1/2 sum_{t <= r} (k_r * prod_{m = t..r-1} alpha<_m . q_t) g_t,
// an anti-causal pass whose gate at "query" r .. "key" t - 1 is alpha>_{m+1}, and a causal one whose gate is alpha<_{m-1}.
template <typename T>
__global__ void __launch_bounds__(256) shift_gates_kernel(const T* __restrict__ la_f, const T* __restrict__ la_b, T* __restrict__ out_f,
                                                          T* __restrict__ out_b, long long n, int L, int dk) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x; x < n; x += stride) {
        const int t = (int)((x / dk) % L);
        T zero;
        rec_store(&zero, 0.f);
        out_f[x] = t > 0 ? la_b[x - dk] : zero;
        out_b[x] = t + 1 < L ? la_f[x + dk] : zero;
    }
}

template <typename T, int CN>
cudaError_t launch_bwd_t(const BwdArgs<T>& a, int threads, int sms, cudaStream_t stream) {
    const size_t smem = bwd_smem_floats(threads / kBwdCG, CN) * sizeof(float);
    static std::atomic<bool> configured[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev].load(std::memory_order_acquire)) {
        if ((e = cudaFuncSetAttribute(bigla_bwd_kernel<T, CN>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024)) != cudaSuccess) return e;
        configured[dev].store(true, std::memory_order_release);
    }
    long long grid = a.units < 32LL * sms ? a.units : 32LL * sms;
    bigla_bwd_kernel<T, CN><<<(unsigned)grid, threads, smem, stream>>>(a);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

bool bwd_supported(int dk, int dv) {
    if (dk < 1 || dv < 1 || dk > 128 || dv > 128) return false;   // at most 512 threads, 32 columns per thread
    const int threads = (kBwdCG * dk + 31) / 32 * 32, cn = (dv + kBwdCG - 1) / kBwdCG;
    return bwd_smem_floats(threads / kBwdCG, cn <= 8 ? 8 : (cn <= 12 ? 12 : (cn <= 16 ? 16 : 32))) * sizeof(float) <= 200 * 1024;
}

size_t bwd_scratch_bytes(long long units, int L, int dk) { return (size_t)units * 2 * L * dk * sizeof(float); }

template <typename T>
cudaError_t launch_shift_gates(const T* la_f, const T* la_b, T* out_f, T* out_b, long long units, int L, int dk, cudaStream_t stream) {
    const long long n = units * L * dk;
    long long blocks = (n + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    shift_gates_kernel<T><<<(unsigned)blocks, 256, 0, stream>>>(la_f, la_b, out_f, out_b, n, L, dk);
    count_launch();
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_bigla_bwd(const T* q, const T* k, const T* v, const T* la_f, const T* la_b, const T* d_out, T* dq, T* dk_out, T* dla_f,
                             T* dla_b, float* scratch, long long units, int L, int dk, int dv, cudaStream_t stream) {
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    BwdArgs<T> a{q, k, v, la_f, la_b, d_out, dq, dk_out, dla_f, dla_b, scratch, units, L, dk, dv};
    const int threads = (kBwdCG * dk + 31) / 32 * 32, cn = (dv + kBwdCG - 1) / kBwdCG;
    if (cn <= 8) return launch_bwd_t<T, 8>(a, threads, sms, stream);
    if (cn <= 12) return launch_bwd_t<T, 12>(a, threads, sms, stream);
    if (cn <= 16) return launch_bwd_t<T, 16>(a, threads, sms, stream);
    return launch_bwd_t<T, 32>(a, threads, sms, stream);
}

template cudaError_t launch_shift_gates<float>(const float*, const float*, float*, float*, long long, int, int, cudaStream_t);
template cudaError_t launch_shift_gates<__nv_bfloat16>(const __nv_bfloat16*, const __nv_bfloat16*, __nv_bfloat16*, __nv_bfloat16*, long long,
                                                       int, int, cudaStream_t);
template cudaError_t launch_bigla_bwd<float>(const float*, const float*, const float*, const float*, const float*, const float*, float*, float*,
                                             float*, float*, float*, long long, int, int, int, cudaStream_t);
template cudaError_t launch_bigla_bwd<__nv_bfloat16>(const __nv_bfloat16*, const __nv_bfloat16*, const __nv_bfloat16*, const __nv_bfloat16*,
                                                     const __nv_bfloat16*, const __nv_bfloat16*, __nv_bfloat16*, __nv_bfloat16*, __nv_bfloat16*,
                                                     __nv_bfloat16*, float*, long long, int, int, int, cudaStream_t);

}  // namespace vig
