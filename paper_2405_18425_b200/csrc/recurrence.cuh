// Step-by-step evaluation of the BiGLA recurrences (paper Eq. 6) by one thread block for one
// (batch, head) unit, in fp32 on the CUDA cores.  Used as the fp32 entry point's kernel, as the
// bf16 entry point's kernel for head sizes the tensor-core kernel does not cover, and inside the
// tensor-core kernel for units whose gates leave the range its factorised tiles can represent.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

namespace vig {

constexpr int kRecTT = 16;   // time steps staged in shared memory at once
constexpr int kRecR = 32;    // max state rows (key dims) held per thread

struct RecPlan {
    int P;    // thread groups along the key dimension
    int Rn;   // state rows per thread
    int smem_floats;
};

// Work split for a block of `nt` threads: thread (p, j) keeps rows [p*Rn, p*Rn + Rn) of column j
// of the dk x dv state in registers.  Valid iff nt >= dv and Rn <= kRecR.
__host__ __device__ inline RecPlan rec_plan(int nt, int dk, int dv) {
    RecPlan pl;
    int P = nt / dv;
    if (P < 1) P = 1;
    if (P > dk) P = dk;
    pl.Rn = (dk + P - 1) / P;
    pl.P = (dk + pl.Rn - 1) / pl.Rn;
    pl.smem_floats = kRecTT * (3 * dk + dv + pl.P * dv);
    return pl;
}

__device__ __forceinline__ float rec_to_float(float x) { return x; }
__device__ __forceinline__ float rec_to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void rec_store(float* p, float x) { *p = x; }
__device__ __forceinline__ void rec_store(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

// All threads of the block must call this (it uses __syncthreads).  q, k, la_f, la_b: [L, dk];
// v, out: [L, dv] of this unit (global or shared memory); ws: rec_plan(...).smem_floats floats of
// shared memory.  The forward pass stores o> in `out` (rounded to T), the backward pass turns it
// into (o> + o<)/2.  gate_inv_tau > 0: la_f / la_b hold gate logits g instead, and log alpha = logsigmoid(g) / tau
// (Eq. 5 line 1) is taken on the fly.
template <typename T>
__device__ void recurrence_unit(const T* q, const T* k, const T* v, const T* la_f, const T* la_b, T* out,
                                int L, int dk, int dv, float* ws, float gate_inv_tau = 0.f) {
    const int nt = blockDim.x, tid = threadIdx.x;
    const RecPlan pl = rec_plan(nt, dk, dv);
    float* qs = ws;
    float* ks = qs + kRecTT * dk;
    float* es = ks + kRecTT * dk;
    float* vs = es + kRecTT * dk;
    float* part = vs + kRecTT * dv;

    const int p = tid / dv, j = tid - p * dv;
    const bool active = p < pl.P;
    const int i0 = p * pl.Rn;
    const int rn = active ? min(pl.Rn, dk - i0) : 0;
    const int nchunk = (L + kRecTT - 1) / kRecTT;

    for (int dir = 0; dir < 2; ++dir) {
        const T* la = dir == 0 ? la_f : la_b;
        float S[kRecR];
#pragma unroll
        for (int r = 0; r < kRecR; ++r) S[r] = 0.f;
        for (int cc = 0; cc < nchunk; ++cc) {
            const int c = dir == 0 ? cc : nchunk - 1 - cc;
            const int t0 = c * kRecTT;
            const int nv = min(kRecTT, L - t0);
            for (int x = tid; x < nv * dk; x += nt) {
                const size_t g = (size_t)t0 * dk + x;
                qs[x] = rec_to_float(q[g]);
                ks[x] = rec_to_float(k[g]);
                float a = rec_to_float(la[g]);
                if (gate_inv_tau > 0.f) a = (fminf(a, 0.f) - log1pf(expf(-fabsf(a)))) * gate_inv_tau;
                es[x] = expf(a);   // alpha_t[i]
            }
            for (int x = tid; x < nv * dv; x += nt) vs[x] = rec_to_float(v[(size_t)t0 * dv + x]);
            __syncthreads();
            if (active) {
                for (int n = 0; n < nv; ++n) {
                    const int tt = dir == 0 ? n : nv - 1 - n;
                    const float vj = vs[tt * dv + j];
                    const float* er = es + tt * dk + i0;
                    const float* kr = ks + tt * dk + i0;
                    const float* qr = qs + tt * dk + i0;
                    float acc = 0.f;
#pragma unroll
                    for (int r = 0; r < kRecR; ++r) {
                        if (r < rn) {
                            S[r] = fmaf(er[r], S[r], kr[r] * vj);   // S_t = G_t . S_prev + k_t^T v_t
                            acc = fmaf(qr[r], S[r], acc);           // o_t = q_t S_t
                        }
                    }
                    part[(p * kRecTT + tt) * dv + j] = acc;
                }
            }
            __syncthreads();
            for (int x = tid; x < nv * dv; x += nt) {
                float o = 0.f;
                for (int pp = 0; pp < pl.P; ++pp) o += part[pp * kRecTT * dv + x];
                T* dst = out + (size_t)t0 * dv + x;
                if (dir == 0) rec_store(dst, o);
                else rec_store(dst, 0.5f * (rec_to_float(*dst) + o));
            }
            __syncthreads();
        }
    }
}

}  // namespace vig
