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
// registers; the sums over the value dimension are finished over the two or four lanes of a row by shuffles.  Inputs and
// outputs pass through shared memory sixteen tokens at a time: asynchronous copies (cp.async) bring the next sixteen
// tokens in while the block works on these, where a token's row is a whole number of 16-byte pieces.
#include <atomic>
#include <cstring>

#include "ptx.cuh"
#include "recurrence.cuh"
#include "vig_internal.h"

namespace vig {

namespace {

constexpr int kBwdTT = 16;   // tokens staged at once

template <typename T>
struct BwdArgs {
    const T *q, *k, *v, *la_f, *la_b, *g;
    T *dq, *dkey, *dla_f, *dla_b;
    float* scratch;   // [units][L][dk][2] fp32: (dq>, dk<) between the two walks (then the local gate sums of a segmented call)
    // Segmented call (few units, long sequences): a block walks one segment of seg_len tokens.  states: [units][nseg][4]
    // [dk][CG CN] fp32 - S>, Z<, S<, Z> of a segment run from zero, replaced by the states entering the segment; decay:
    // [units][nseg][4][dk] - the products of the gates over the segment; totals: [units][nseg][2][dk] - the segment's sums of
    // E> and E<.  All NULL / nseg = 1 for the call that walks whole units.
    float *states, *decay, *totals;
    long long units;
    int L, dk, dv, nseg, seg_len;
};

// Shared memory of a block.  rows: state rows it holds (threads / CG, >= dk; the padded rows and columns work on
// zeros).  fp32 staging: 16-byte row records [TT][rows], the partial results read back [TT][rows] pairs, v and d_out
// [TT][CG (cn + 4)] (+ 4: a lane group's columns start 16 bytes off the bank of the group before it); then the raw
// landing zone of the asynchronous copies of the next sixteen tokens: k, q, two gate rows, v, d_out in the call's type
// and the fp32 pairs.
__host__ __device__ inline size_t bwd_stage_floats(int rows, int cn, int cg) { return (size_t)kBwdTT * (6 * rows + 2 * cg * (cn + 4)); }
__host__ __device__ inline size_t bwd_smem_bytes(int rows, int cn, int cg, int dk, int dv, size_t elem) {
    return bwd_stage_floats(rows, cn, cg) * sizeof(float) + (size_t)kBwdTT * ((4 * dk + 2 * dv) * elem + dk * 8) + 64;
}

// Four consecutive elements of the call's type <-> fp32
__device__ __forceinline__ void load4(const float* p, float (&f)[4]) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
}
__device__ __forceinline__ void load4(const __nv_bfloat16* p, float (&f)[4]) {
    const uint2 v = *reinterpret_cast<const uint2*>(p);
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
}
__device__ __forceinline__ void store4(float* p, const float (&f)[4]) { *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]); }
__device__ __forceinline__ void store4(__nv_bfloat16* p, const float (&f)[4]) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(f[0], f[1]), hi = __floats2bfloat162_rn(f[2], f[3]);
    *reinterpret_cast<uint2*>(p) = make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
}

// 16-byte store to shared memory that the compiler does not take for a store to the C++ objects it tracks: the loads of
// the tokens after this one may move above it (they never read what it writes; whoever reads it does so behind a barrier).
__device__ __forceinline__ void sts128_untracked(void* p, float x, float y, float z, float w) {
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"((uint32_t)__cvta_generic_to_shared(p)), "f"(x), "f"(y), "f"(z), "f"(w));
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src) : "memory");
}

// Block shapes known at compile time are held to 85 registers (768 threads per SM: six blocks of 128).
constexpr int bwd_max_threads(int rows, int cg) { return rows > 0 ? rows * cg : 512; }
constexpr int bwd_min_blocks(int rows, int cg) { return rows > 0 ? 768 / (rows * cg) : 1; }

// CG: threads (adjacent lanes) per state row, 2 or 4.  CN: columns of the state per thread (a multiple of 4).  ROWS: state
// rows of the block (threads / CG) when known at compile time - every shared-memory offset is then an immediate - or 0
// for any block size.
// SUMMARY: the first launch of a segmented call - the four states of every segment run from zero and the products of their
// gates (state updates only, nothing else is read or written).
template <typename T, int CN, int ROWS, int CG, bool SUMMARY>
__global__ void __launch_bounds__(bwd_max_threads(ROWS, CG), bwd_min_blocks(ROWS, CG)) bigla_bwd_kernel(BwdArgs<T> a) {
    constexpr int kBwdCG = CG;
    static_assert(CN % 4 == 0, "columns per thread come in 16-byte pieces");
    extern __shared__ __align__(16) float bw_smem[];
    const int tid = threadIdx.x, nt = ROWS ? ROWS * kBwdCG : blockDim.x;
    const int rows = ROWS ? ROWS : nt / kBwdCG;
    constexpr int cols = kBwdCG * (CN + 4);   // a token's row of v / d_out: CG groups of CN (+ 4 unused) floats
    const int i = tid / kBwdCG, cg = tid % kBwdCG;
    const int L = a.L, dk = a.dk, dv = a.dv;
    float4* rowd = reinterpret_cast<float4*>(bw_smem);                  // [TT][rows]: k, q, decay of S, decay of Z; then the results
    float2* xd = reinterpret_cast<float2*>(rowd + kBwdTT * rows);       // [TT][rows]: dq>, dk< (descending walk)
    float* vs = reinterpret_cast<float*>(xd + kBwdTT * rows);           // [TT][cols]
    float* gs = vs + kBwdTT * cols;
    // raw landing zone (16-byte aligned pieces): k, q, gates of S, gates of Z, v, d_out as stored, then the fp32 pairs
    T* raw_k = reinterpret_cast<T*>(gs + kBwdTT * cols);
    T* raw_q = raw_k + kBwdTT * dk;
    T* raw_s = raw_q + kBwdTT * dk;
    T* raw_z = raw_s + kBwdTT * dk;
    T* raw_v = raw_z + kBwdTT * dk;
    T* raw_g = raw_v + kBwdTT * dv;
    float2* raw_x = reinterpret_cast<float2*>(raw_g + kBwdTT * dv);
    // The instances for the paper's head sizes (bf16, dv = CG CN exactly, whole 16-byte rows) read v and d_out in the walk
    // straight from the landing zone, as bf16: half the shared-memory traffic of the walk, which is what bounds it.  The
    // landing zone of v and d_out then has a second buffer (in place of the fp32 staging of the two).
    constexpr bool kVG16 = ROWS != 0 && sizeof(T) == 2;
    T* raw_v1 = reinterpret_cast<T*>(vs);
    T* raw_g1 = raw_v1 + kBwdTT * dv;
    // Rows of whole 16-byte pieces: the next sixteen tokens are copied asynchronously while these are worked on.
    const bool ahead = (dk * sizeof(T)) % 16 == 0 && (dv * sizeof(T)) % 16 == 0;
    for (size_t x = tid; x < bwd_stage_floats(rows, CN, CG); x += nt) bw_smem[x] = 0.f;   // the padding stays zero
    __syncthreads();
    const int st_r = tid % rows, st_t = tid / rows;   // staging: thread = one key dimension of every fourth token
    const bool segmented = a.states != nullptr;

    for (long long w = blockIdx.x; w < a.units * a.nseg; w += gridDim.x) {
        const long long unit = w / a.nseg;
        const int s0 = (int)(w % a.nseg) * a.seg_len, s1 = min(L, s0 + a.seg_len);   // this block's tokens [s0, s1)
        const int nchunk = (s1 - s0 + kBwdTT - 1) / kBwdTT;
        const size_t ok = (size_t)unit * L * dk, ov = (size_t)unit * L * dv;
        float2* sc = reinterpret_cast<float2*>(a.scratch) + ok;   // [L][dk] pairs (dq>, dk<)
        for (int walk = 0; walk < 2; ++walk) {
            const T* la_s = (walk == 0 ? a.la_f : a.la_b) + ok;   // gates of the S state
            const T* la_z = (walk == 0 ? a.la_b : a.la_f) + ok;   // gates of the Z state
            const int step = walk == 0 ? 1 : -1;
            f32x2 S[CN / 2], Z[CN / 2];
#pragma unroll
            for (int c = 0; c < CN / 2; ++c) S[c] = Z[c] = 0ull;   // (+0, +0)
            float run_f = 0.f, run_b = 0.f;   // running sums of E> and E< (descending walk)
            float prod_s = 1.f, prod_z = 1.f;   // SUMMARY: products of the gates of S and of Z over the segment
            const size_t st_base = ((size_t)w * 4 + (walk == 0 ? 0 : 2)) * dk;   // kinds: S> 0, Z< 1, S< 2, Z> 3
            if (!SUMMARY && segmented && i < dk) {   // the states that enter this segment
                const float* ps = a.states + (st_base + i) * (CG * CN) + cg * CN;
                const float* pz = ps + (size_t)dk * (CG * CN);
#pragma unroll
                for (int c = 0; c < CN / 2; ++c) {
                    S[c] = pack2(ps[2 * c], ps[2 * c + 1]);
                    Z[c] = pack2(pz[2 * c], pz[2 * c + 1]);
                }
            }
            // sixteen tokens of every input on their way into the landing zone (thread = 16-byte pieces)
            auto fetch = [&](int cc) {
                const int t0 = s0 + (walk == 0 ? cc : nchunk - 1 - cc) * kBwdTT;
                const int nv = min(kBwdTT, s1 - t0);
                const int pk = nv * dk * (int)sizeof(T) / 16, pv = nv * dv * (int)sizeof(T) / 16, row16 = dk * (int)sizeof(T) / 16;
                const char* gk = reinterpret_cast<const char*>(a.k + ok + (size_t)t0 * dk);
                const char* gq = reinterpret_cast<const char*>(a.q + ok + (size_t)t0 * dk);
                const char* gs_ = reinterpret_cast<const char*>(la_s + (size_t)t0 * dk);
                for (int x = tid; x < pk; x += nt) {
                    cp_async16(reinterpret_cast<char*>(raw_k) + 16 * x, gk + 16 * x);
                    cp_async16(reinterpret_cast<char*>(raw_q) + 16 * x, gq + 16 * x);
                    cp_async16(reinterpret_cast<char*>(raw_s) + 16 * x, gs_ + 16 * x);
                    const int tp = t0 + x / row16 - step;   // slot tt of the Z gates holds token t0 + tt - step, where it exists
                    if (tp >= 0 && tp < L)
                        cp_async16(reinterpret_cast<char*>(raw_z) + 16 * x, reinterpret_cast<const char*>(la_z + (size_t)tp * dk) + 16 * (x % row16));
                }
                const char* gv = reinterpret_cast<const char*>(a.v + ov + (size_t)t0 * dv);
                const char* gg = reinterpret_cast<const char*>(a.g + ov + (size_t)t0 * dv);
                char* dv_ = reinterpret_cast<char*>(kVG16 && (cc & 1) ? raw_v1 : raw_v);
                char* dg_ = reinterpret_cast<char*>(kVG16 && (cc & 1) ? raw_g1 : raw_g);
                for (int x = tid; x < pv; x += nt) {
                    cp_async16(dv_ + 16 * x, gv + 16 * x);
                    cp_async16(dg_ + 16 * x, gg + 16 * x);
                }
                if (walk == 1 && !SUMMARY) {
                    const char* gx = reinterpret_cast<const char*>(sc + (size_t)t0 * dk);
                    for (int x = tid; x < nv * dk / 2; x += nt) cp_async16(reinterpret_cast<char*>(raw_x) + 16 * x, gx + 16 * x);
                }
                asm volatile("cp.async.commit_group;" ::: "memory");
            };
            // sixteen tokens from `k_` ... (the landing zone, or global memory itself) into the fp32 staging
            auto convert = [&](const T* k_, const T* q_, const T* s_, const T* z_, const T* v_, const T* g_, const float2* x_, int t0, int nv) {
                if (st_r < dk) {
                    for (int tt = st_t; tt < nv; tt += kBwdCG) {
                        const int tp = t0 + tt - step;   // the token walked before this one
                        const int e = tt * dk + st_r;
                        float4 r4;
                        r4.x = rec_to_float(k_[e]);
                        r4.y = rec_to_float(q_[e]);
                        r4.z = expf(rec_to_float(s_[e]));
                        r4.w = (tp >= 0 && tp < L) ? expf(rec_to_float(z_[e])) : 0.f;
                        rowd[tt * rows + st_r] = r4;
                        if (walk == 1 && !SUMMARY) xd[tt * rows + st_r] = x_[e];
                    }
                }
                int tt = 0, j = tid;
                while (j >= dv) { j -= dv; ++tt; }
                while (tt < nv) {
                    const int at = tt * cols + (j / CN) * (CN + 4) + j % CN;
                    vs[at] = rec_to_float(v_[tt * dv + j]);
                    gs[at] = rec_to_float(g_[tt * dv + j]);
                    j += nt;
                    while (j >= dv) { j -= dv; ++tt; }
                }
            };
            // the same from the landing zone, four elements at a time (rows are whole 16-byte pieces there)
            auto convert4 = [&](int t0, int nv) {
                const int qk = dk / 4, qv = dv / 4;
                for (int x = tid; x < nv * qk; x += nt) {
                    const int tt = x / qk, r0 = (x - tt * qk) * 4, e = tt * dk + r0, tp = t0 + tt - step;
                    float kf[4], qf[4], sf[4], zf[4];
                    load4(raw_k + e, kf);
                    load4(raw_q + e, qf);
                    load4(raw_s + e, sf);
                    load4(raw_z + e, zf);
                    const bool zin = tp >= 0 && tp < L;
#pragma unroll
                    for (int u = 0; u < 4; ++u) rowd[tt * rows + r0 + u] = make_float4(kf[u], qf[u], expf(sf[u]), zin ? expf(zf[u]) : 0.f);
                    if (walk == 1 && !SUMMARY) {
                        const float4 xa = *reinterpret_cast<const float4*>(raw_x + e), xb = *reinterpret_cast<const float4*>(raw_x + e + 2);
                        float4* xo = reinterpret_cast<float4*>(xd + tt * rows + r0);
                        xo[0] = xa;
                        xo[1] = xb;
                    }
                }
                for (int x = tid; x < (kVG16 ? 0 : nv * qv); x += nt) {   // (kVG16: v and d_out stay where they landed)
                    const int tt = x / qv, j0 = (x - tt * qv) * 4;
                    const int at = tt * cols + (j0 / CN) * (CN + 4) + j0 % CN;
                    float f[4];
                    load4(raw_v + tt * dv + j0, f);
                    store4(vs + at, f);
                    load4(raw_g + tt * dv + j0, f);
                    store4(gs + at, f);
                }
            };
            if (ahead) fetch(0);
            for (int cc = 0; cc < nchunk; ++cc) {
                const int t0 = s0 + (walk == 0 ? cc : nchunk - 1 - cc) * kBwdTT;
                const int nv = min(kBwdTT, s1 - t0);
                if (ahead) {
                    asm volatile("cp.async.wait_group 0;" ::: "memory");
                    __syncthreads();   // everybody's pieces have landed (and the results of the chunk before are stored)
                    convert4(t0, nv);
                    __syncthreads();
                    if (cc + 1 < nchunk) fetch(cc + 1);
                } else {
                    __syncthreads();   // the results of the chunk before are stored
                    // (slot tt of the Z gates: token t0 + tt - step; the pointer is only followed where that token exists)
                    convert(a.k + ok + (size_t)t0 * dk, a.q + ok + (size_t)t0 * dk, la_s + (size_t)t0 * dk,
                            la_z + ((ptrdiff_t)t0 - step) * dk, a.v + ov + (size_t)t0 * dv, a.g + ov + (size_t)t0 * dv, sc + (size_t)t0 * dk, t0, nv);
                    __syncthreads();
                }
                {
                    const float4* rp = rowd + (walk == 0 ? 0 : nv - 1) * rows + i;
                    const float2* xp = xd + (walk == 0 ? 0 : nv - 1) * rows + i;
                    float4* op = rowd + (walk == 0 ? 0 : nv - 1) * rows + i;   // the record is replaced by the results (the lanes of a
                                                                                // row read it in the same instruction, before this lane writes)
                    const int first = walk == 0 ? 0 : nv - 1;
                    // this thread's columns of v and d_out, token by token: fp32 staging, or (kVG16) the bf16 rows as they landed
                    const char* vp = kVG16 ? reinterpret_cast<const char*>(((cc & 1) ? raw_v1 : raw_v) + first * dv + cg * CN)
                                           : reinterpret_cast<const char*>(vs + first * cols + cg * (CN + 4));
                    const char* gp = kVG16 ? reinterpret_cast<const char*>(((cc & 1) ? raw_g1 : raw_g) + first * dv + cg * CN)
                                           : reinterpret_cast<const char*>(gs + first * cols + cg * (CN + 4));
                    const int srow = step * rows, scol = step * (kVG16 ? dv * 2 : cols * 4);   // bytes per token
                    // four columns (two fp32 pairs) number c4 of the row at p
                    auto quad = [&](const char* p, int c4, f32x2& lo, f32x2& hi) {
                        if constexpr (kVG16) {
                            const uint2 wv = reinterpret_cast<const uint2*>(p)[c4];   // a bf16 is the upper half of its fp32
                            lo = pack2(__uint_as_float(wv.x << 16), __uint_as_float(wv.x & 0xffff0000u));
                            hi = pack2(__uint_as_float(wv.y << 16), __uint_as_float(wv.y & 0xffff0000u));
                        } else {
                            const ulonglong2 q2 = reinterpret_cast<const ulonglong2*>(p)[c4];
                            lo = q2.x;
                            hi = q2.y;
                        }
                    };
#pragma unroll 4
                    for (int n = 0; n < nv; ++n, rp += srow, xp += srow, op += srow, vp += scol, gp += scol) {
                        const float4 r4 = *rp;   // k, q, decay of S, decay of Z
                        const float hq = 0.5f * r4.y;
                        const f32x2 ds2 = pack2(r4.z, r4.z), dz2 = pack2(r4.w, r4.w), kq2 = pack2(r4.x, r4.x), hq2 = pack2(hq, hq);
                        if constexpr (SUMMARY) {
#pragma unroll
                            for (int c4 = 0; c4 < CN / 4; ++c4) {
                                f32x2 vq[2], gq[2];
                                quad(vp, c4, vq[0], vq[1]);
                                quad(gp, c4, gq[0], gq[1]);
#pragma unroll
                                for (int h = 0; h < 2; ++h) {
                                    const int c = 2 * c4 + h;
                                    S[c] = ffma2(ds2, S[c], fmul2(kq2, vq[h]));
                                    Z[c] = ffma2(dz2, Z[c], fmul2(hq2, gq[h]));
                                }
                            }
                            prod_s *= r4.z;
                            prod_z *= r4.w;
                            continue;
                        }
                        f32x2 aq[2] = {0ull, 0ull}, ak[2] = {0ull, 0ull};
#pragma unroll
                        for (int c4 = 0; c4 < CN / 4; ++c4) {
                            f32x2 vq[2], gq[2];
                            quad(vp, c4, vq[0], vq[1]);
                            quad(gp, c4, gq[0], gq[1]);
#pragma unroll
                            for (int h = 0; h < 2; ++h) {
                                const f32x2 vj = vq[h], gj = gq[h];
                                const int c = 2 * c4 + h;
                                S[c] = ffma2(ds2, S[c], fmul2(kq2, vj));   // S_t = a S + k^T v
                                aq[h] = ffma2(S[c], gj, aq[h]);            // S_t g^T
                                Z[c] = ffma2(dz2, Z[c], fmul2(hq2, gj));   // Z_t = a' Z + q^T g / 2
                                ak[h] = ffma2(Z[c], vj, ak[h]);            // Z_t v^T
                            }
                        }
                        float accq = sum2(aq[0]) + sum2(aq[1]), acck = sum2(ak[0]) + sum2(ak[1]);
                        accq += __shfl_xor_sync(0xffffffffu, accq, 1);
                        acck += __shfl_xor_sync(0xffffffffu, acck, 1);
                        if (CG == 4) {
                            accq += __shfl_xor_sync(0xffffffffu, accq, 2);
                            acck += __shfl_xor_sync(0xffffffffu, acck, 2);
                        }
                        accq *= 0.5f;
                        if (walk == 0) {
                            if (cg == 0) sts128_untracked(op, accq, acck, 0.f, 0.f);   // dq>_t, dk<_t
                        } else {
                            const float2 x2 = *xp;   // dq>_t, dk<_t;  accq = dq<_t, acck = dk>_t
                            run_f += r4.y * x2.x - r4.x * acck;
                            // dq, dk, the sum over m >= t of E>_m, minus the sum over m > t of E<_m (within the block's tokens)
                            if (cg == 0) sts128_untracked(op, x2.x + accq, acck + x2.y, run_f, -run_b);
                            run_b += r4.y * accq - r4.x * x2.y;
                        }
                    }
                }
                if constexpr (SUMMARY) continue;   // nothing to store per token (the barrier at the top of the loop orders the staging)
                __syncthreads();
                if (ahead) {   // four key dimensions of a token per thread: 8- or 16-byte stores
                    const int qk = dk / 4;
                    for (int x = tid; x < nv * qk; x += nt) {
                        const int tt = x / qk, r0 = (x - tt * qk) * 4;
                        const size_t gi = (size_t)(t0 + tt) * dk + r0;
                        float o[4][4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const float4 o4 = rowd[tt * rows + r0 + u];
                            o[0][u] = o4.x; o[1][u] = o4.y; o[2][u] = o4.z; o[3][u] = o4.w;
                        }
                        if (walk == 0) {
                            float4* so = reinterpret_cast<float4*>(sc + gi);
                            so[0] = make_float4(o[0][0], o[1][0], o[0][1], o[1][1]);
                            so[1] = make_float4(o[0][2], o[1][2], o[0][3], o[1][3]);
                        } else {
                            store4(a.dq + ok + gi, o[0]);
                            store4(a.dkey + ok + gi, o[1]);
                            if (segmented) {   // the gate sums of this segment alone, in fp32 over the consumed pairs
                                float4* so = reinterpret_cast<float4*>(sc + gi);
                                so[0] = make_float4(o[2][0], o[3][0], o[2][1], o[3][1]);
                                so[1] = make_float4(o[2][2], o[3][2], o[2][3], o[3][3]);
                            } else {
                                store4(a.dla_f + ok + gi, o[2]);
                                store4(a.dla_b + ok + gi, o[3]);
                            }
                        }
                    }
                } else if (st_r < dk) {
                    for (int tt = st_t; tt < nv; tt += kBwdCG) {
                        const size_t gi = (size_t)(t0 + tt) * dk + st_r;
                        const float4 o4 = rowd[tt * rows + st_r];
                        if (walk == 0) {
                            sc[gi] = make_float2(o4.x, o4.y);
                        } else {
                            rec_store(a.dq + ok + gi, o4.x);
                            rec_store(a.dkey + ok + gi, o4.y);
                            if (segmented) {
                                sc[gi] = make_float2(o4.z, o4.w);
                            } else {
                                rec_store(a.dla_f + ok + gi, o4.z);
                                rec_store(a.dla_b + ok + gi, o4.w);
                            }
                        }
                    }
                }
            }
            if (SUMMARY && i < dk) {   // what the segment adds to each state, and by how much it shrinks what enters it
                float* ps = a.states + (st_base + i) * (CG * CN) + cg * CN;
                float* pz = ps + (size_t)dk * (CG * CN);
#pragma unroll
                for (int c = 0; c < CN / 2; ++c) {
                    unpack2(S[c], ps[2 * c], ps[2 * c + 1]);
                    unpack2(Z[c], pz[2 * c], pz[2 * c + 1]);
                }
                if (cg == 0) {
                    a.decay[st_base + i] = prod_s;
                    a.decay[st_base + dk + i] = prod_z;
                }
            }
            if (!SUMMARY && segmented && walk == 1 && cg == 0 && i < dk) {
                a.totals[((size_t)w * 2) * dk + i] = run_f;
                a.totals[((size_t)w * 2 + 1) * dk + i] = run_b;
            }
            __syncthreads();   // the scratch of the ascending walk is read back by other threads
        }
    }
}

// Second launch of a segmented call: the states that enter each segment, X_in(s + 1) = D(s) X_in(s) + X(s) walking up for
// S> and Z<, X_in(s - 1) = D(s) X_in(s) + X(s) walking down for S< and Z>, written over the segments' own states.
// Thread = four columns of one state row of one unit.
__global__ void __launch_bounds__(256) bwd_fold_kernel(float* states, const float* decay, long long units, int nseg, int dk, int cols) {
    const int c4 = cols / 4;
    const long long n = units * dk * c4;
    for (long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x; x < n; x += (long long)gridDim.x * blockDim.x) {
        const int col = (int)(x % c4) * 4, i = (int)((x / c4) % dk);
        const long long unit = x / ((long long)c4 * dk);
#pragma unroll
        for (int kind = 0; kind < 4; ++kind) {
            float4 carry = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int n2 = 0; n2 < nseg; ++n2) {
                const int sg = kind < 2 ? n2 : nseg - 1 - n2;
                const size_t row = (((size_t)unit * nseg + sg) * 4 + kind) * dk + i;
                float4* p = reinterpret_cast<float4*>(states + row * cols + col);
                const float4 own = *p;
                const float d = decay[row];
                *p = carry;
                carry = make_float4(fmaf(d, carry.x, own.x), fmaf(d, carry.y, own.y), fmaf(d, carry.z, own.z), fmaf(d, carry.w, own.w));
            }
        }
    }
}

// Last launch of a segmented call: the gate gradients of a token are its segment's local sums plus what the segments
// walked before it (the later ones) add: dlog alpha>_t = local + sum_{s' > s} total>(s'), dlog alpha<_t = local - sum_{s' > s}
// total<(s').  Block = one segment of one unit.
template <typename T>
__global__ void __launch_bounds__(256) bwd_finish_kernel(const float2* local, const float* totals, T* dla_f, T* dla_b, int L, int dk, int nseg,
                                                         int seg_len) {
    extern __shared__ float off[];   // [2][dk]
    const long long w = blockIdx.x, unit = w / nseg;
    const int sg = (int)(w % nseg), s0 = sg * seg_len, s1 = min(L, s0 + seg_len);
    for (int x = threadIdx.x; x < 2 * dk; x += blockDim.x) {
        const int which = x / dk, i = x - which * dk;
        float acc = 0.f;
        for (int s2 = nseg - 1; s2 > sg; --s2) acc += totals[(((size_t)unit * nseg + s2) * 2 + which) * dk + i];   // in walking order
        off[x] = which == 0 ? acc : -acc;
    }
    __syncthreads();
    const size_t base = ((size_t)unit * L + s0) * dk;
    for (int x = threadIdx.x; x < (s1 - s0) * dk; x += blockDim.x) {
        const float2 l = local[base + x];
        const int i = x % dk;
        rec_store(dla_f + base + x, l.x + off[i]);
        rec_store(dla_b + base + x, l.y + off[dk + i]);
    }
}

// la_f'[t] = la_b[t - 1] (0 at t = 0), la_b'[t] = la_f[t + 1] (0 at t = L - 1): with these gates, d_out as the values and
// q, k swapped, the forward pass IS the gradient with respect to v:
//   dv_r = 1/2 sum_{t >= r} (k_r * prod_{m = r+1..t} alpha>_m . q_t) g_t + 1/2 sum_{t <= r} (k_r * prod_{m = t..r-1} alpha<_m . q_t) g_t,
// an anti-causal pass whose gate at "query" r .. "key" t - 1 is alpha>_{m+1}, and a causal one whose gate is alpha<_{m-1}.
template <typename T, typename V>   // V: the unit moved per thread (T itself, or 16 bytes of T when a token's row is a whole number of them)
__global__ void __launch_bounds__(256) shift_gates_kernel(const V* __restrict__ la_f, const V* __restrict__ la_b, V* __restrict__ out_f,
                                                          V* __restrict__ out_b, long long n, int L, int row) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x; x < n; x += stride) {
        const int t = (int)((x / row) % L);
        V zero;
        memset(&zero, 0, sizeof(V));   // +0 in either type
        out_f[x] = t > 0 ? la_b[x - row] : zero;
        out_b[x] = t + 1 < L ? la_f[x + row] : zero;
    }
}

template <typename T, int CN, int ROWS, int CG, bool SUMMARY>
cudaError_t launch_bwd_kernel(const BwdArgs<T>& a, int threads, int sms, cudaStream_t stream) {
    const size_t smem = bwd_smem_bytes(threads / CG, CN, CG, a.dk, a.dv, sizeof(T));
    static std::atomic<bool> configured[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev].load(std::memory_order_acquire)) {
        if ((e = cudaFuncSetAttribute(bigla_bwd_kernel<T, CN, ROWS, CG, SUMMARY>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024)) !=
            cudaSuccess)
            return e;
        configured[dev].store(true, std::memory_order_release);
    }
    const long long work = a.units * a.nseg;
    long long grid = work < 32LL * sms ? work : 32LL * sms;
    bigla_bwd_kernel<T, CN, ROWS, CG, SUMMARY><<<(unsigned)grid, threads, smem, stream>>>(a);
    count_launch();
    return cudaGetLastError();
}

// The walks of a call: one launch over whole units, or - segmented - the segments' own states, the fold that turns them
// into the states entering each segment, the walks proper from those states, and the gate gradients put together.
template <typename T, int CN, int ROWS, int CG>
cudaError_t launch_bwd_t(const BwdArgs<T>& a, int threads, int sms, cudaStream_t stream) {
    if (a.nseg == 1) return launch_bwd_kernel<T, CN, ROWS, CG, false>(a, threads, sms, stream);
    cudaError_t e = launch_bwd_kernel<T, CN, ROWS, CG, true>(a, threads, sms, stream);
    if (e != cudaSuccess) return e;
    const int cols = CG * CN;
    const long long n = a.units * a.dk * (cols / 4);
    long long blocks = (n + 255) / 256;
    if (blocks > 8LL * sms) blocks = 8LL * sms;
    bwd_fold_kernel<<<(unsigned)blocks, 256, 0, stream>>>(a.states, a.decay, a.units, a.nseg, a.dk, cols);
    count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if ((e = launch_bwd_kernel<T, CN, ROWS, CG, false>(a, threads, sms, stream)) != cudaSuccess) return e;
    bwd_finish_kernel<T><<<(unsigned)(a.units * a.nseg), 256, 2 * a.dk * sizeof(float), stream>>>(
        reinterpret_cast<const float2*>(a.scratch), a.totals, a.dla_f, a.dla_b, a.L, a.dk, a.nseg, a.seg_len);
    count_launch();
    return cudaGetLastError();
}

// Threads per key dimension.  Four: measured faster than two on the paper's shapes (768 units of 196 tokens: 411 us
// against 524 us - fewer instructions with two, but too few warps to hide the latency of a step); two only where four
// would leave a thread fewer than eight columns.
int bwd_cg(int dv) { return dv >= 32 ? 4 : 2; }
// ... in whole warps (the extra rows of the last warp work on zeros).
int bwd_threads(int dk, int cg) { return (cg * dk + 31) / 32 * 32; }
int bwd_cn(int dv, int cg) {   // columns per thread: the instantiated size that holds ceil(dv / cg)
    const int cn = (dv + cg - 1) / cg;
    return cn <= 8 ? 8 : (cn <= 12 ? 12 : (cn <= 16 ? 16 : (cn <= 24 ? 24 : 32)));
}

// Few units and long sequences: the sequence is cut into segments so that about five blocks per SM walk at once (a lone
// block per SM needs about 550 cycles per token).  Segments are multiples of the staging group and at least 64 tokens.
void bwd_plan(long long units, int L, int sms, int* nseg, int* seg_len) {
    *nseg = 1;
    *seg_len = L > 0 ? L : 1;
    if (units >= 2LL * sms || L < 128) return;
    long long want = (5LL * sms + units - 1) / units;
    if (want > L / 64) want = L / 64;
    if (want < 2) return;
    const int len = (int)(((L + want - 1) / want + kBwdTT - 1) / kBwdTT * kBwdTT);
    *seg_len = len;
    *nseg = (L + len - 1) / len;
}

cudaError_t sm_count_of_device(int* sms) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    return cudaDeviceGetAttribute(sms, cudaDevAttrMultiProcessorCount, dev);
}

}  // namespace

bool bwd_supported(int dk, int dv) {
    if (dk < 1 || dv < 1 || dk > 128 || dv > 128) return false;   // at most 512 threads, 32 columns per thread
    const int cg = bwd_cg(dv), threads = bwd_threads(dk, cg);
    return bwd_smem_bytes(threads / cg, bwd_cn(dv, cg), cg, dk, dv, 4) <= 200 * 1024;
}

// Scratch of the walks, in floats: the per-token pairs, then (segmented calls) the segment states, gate products and sums.
static void bwd_scratch_layout(long long units, int L, int dk, int dv, int nseg, size_t* pairs, size_t* states, size_t* decay, size_t* totals) {
    const int cg = bwd_cg(dv), cols = cg * bwd_cn(dv, cg);
    *pairs = ((size_t)units * 2 * L * dk + 63) / 64 * 64;
    *states = nseg > 1 ? (size_t)units * nseg * 4 * dk * cols : 0;
    *decay = nseg > 1 ? ((size_t)units * nseg * 4 * dk + 63) / 64 * 64 : 0;
    *totals = nseg > 1 ? (size_t)units * nseg * 2 * dk : 0;
}

size_t bwd_scratch_bytes(long long units, int L, int dk, int dv) {
    int sms = 0, nseg, seg_len;
    if (sm_count_of_device(&sms) != cudaSuccess) return 0;
    bwd_plan(units, L, sms, &nseg, &seg_len);
    size_t p, st, de, to;
    bwd_scratch_layout(units, L, dk, dv, nseg, &p, &st, &de, &to);
    return (p + st + de + to) * sizeof(float);
}

template <typename T>
cudaError_t launch_shift_gates(const T* la_f, const T* la_b, T* out_f, T* out_b, long long units, int L, int dk, cudaStream_t stream) {
    const bool wide = (dk * sizeof(T)) % 16 == 0;   // (all four pointers are 16-byte aligned)
    const int row = wide ? (int)(dk * sizeof(T) / 16) : dk;
    const long long n = units * L * row;
    long long blocks = (n + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (wide)
        shift_gates_kernel<T, uint4><<<(unsigned)blocks, 256, 0, stream>>>((const uint4*)la_f, (const uint4*)la_b, (uint4*)out_f, (uint4*)out_b, n, L, row);
    else
        shift_gates_kernel<T, T><<<(unsigned)blocks, 256, 0, stream>>>(la_f, la_b, out_f, out_b, n, L, row);
    count_launch();
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_bigla_bwd(const T* q, const T* k, const T* v, const T* la_f, const T* la_b, const T* d_out, T* dq, T* dk_out, T* dla_f,
                             T* dla_b, float* scratch, long long units, int L, int dk, int dv, cudaStream_t stream) {
    int sms = 0, nseg, seg_len;
    cudaError_t e = sm_count_of_device(&sms);
    if (e != cudaSuccess) return e;
    bwd_plan(units, L, sms, &nseg, &seg_len);
    size_t p, st, de, to;
    bwd_scratch_layout(units, L, dk, dv, nseg, &p, &st, &de, &to);
    BwdArgs<T> a{q, k, v, la_f, la_b, d_out, dq, dk_out, dla_f, dla_b, scratch,
                 nseg > 1 ? scratch + p : nullptr, nseg > 1 ? scratch + p + st : nullptr, nseg > 1 ? scratch + p + st + de : nullptr,
                 units, L, dk, dv, nseg, seg_len};
    const int cg = bwd_cg(dv), threads = bwd_threads(dk, cg), cn = bwd_cn(dv, cg), rows = threads / cg;
#define VIG_BWD_CASE(CN_, ROWS_, CG_) \
    if (cn == CN_ && cg == CG_ && (ROWS_ == 0 || (dk == ROWS_ && dv == CG_ * CN_))) return launch_bwd_t<T, CN_, ROWS_, CG_>(a, threads, sms, stream);
    if constexpr (sizeof(T) == 2) {   // the head sizes of the paper's models: block shape known at compile time
        VIG_BWD_CASE(8, 16, 4) VIG_BWD_CASE(8, 24, 4) VIG_BWD_CASE(8, 32, 4)        // dv = 32; dk = 16, 24, 32
        VIG_BWD_CASE(12, 16, 4) VIG_BWD_CASE(12, 24, 4) VIG_BWD_CASE(12, 32, 4)     // dv = 48
        VIG_BWD_CASE(16, 16, 4) VIG_BWD_CASE(16, 24, 4) VIG_BWD_CASE(16, 32, 4)     // dv = 64
    }
    VIG_BWD_CASE(8, 0, 2) VIG_BWD_CASE(12, 0, 2) VIG_BWD_CASE(16, 0, 2)             // dv < 32
    VIG_BWD_CASE(8, 0, 4) VIG_BWD_CASE(12, 0, 4) VIG_BWD_CASE(16, 0, 4) VIG_BWD_CASE(24, 0, 4) VIG_BWD_CASE(32, 0, 4)
#undef VIG_BWD_CASE
    return cudaErrorInvalidValue;
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
