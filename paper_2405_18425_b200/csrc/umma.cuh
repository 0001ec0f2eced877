// Pieces shared by the tcgen05 BiGLA kernels: tcgen05 / TMEM wrappers, shared-memory and instruction
// descriptors, the 0/1 tile of the prefix-sum products, masking and packing of the score tile.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>

#include "ptx.cuh"

namespace vig {
namespace umma {

constexpr int kChunk = 128;     // rows per MMA chunk
constexpr float kGateRange = 60.f;
constexpr float kLog2e = 1.4426950408889634f;
constexpr uint32_t kZRows = 240;                 // 112 constant rows, 16 triangle rows, 112 constant rows
constexpr uint32_t kZBytes = kZRows * 32;        // 16 bf16 per row

// ---- tcgen05 wrappers ------------------------------------------------------------------------
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Instruction descriptor of kind::f16: fp32 accumulate, bf16 A and B, majors, N >> 3, M >> 4.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, int a_mn_major, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// One thread of the (converged) warp.  Issued right at the branch it guards, so that the compiler sees an elected
// region: the MMA operands computed from warp-uniform values then stay in uniform registers.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n .reg .pred p;\n elect.sync _|p, 0xffffffff;\n selp.u32 %0, 1, 0, p;\n}\n" : "=r"(pred));
    return pred != 0;
}
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum)
        : "memory");
}
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n" ::"r"(d_tmem),
        "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accum)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t addr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(addr));
}
__device__ __forceinline__ void tmem_ld32(uint32_t addr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,"
        "%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(addr));
}
__device__ __forceinline__ void tmem_st16(uint32_t addr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(addr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ uint32_t mul_bf16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ float as_f(uint32_t u) { return __uint_as_float(u); }

// Masks of the diagonal 32 x 32 block of P, as packed bf16 pairs of 0 and 1.  For the row of lane t and the column
// pair (2e, 2e + 1) only d = t - 2e matters: the forward scores count for columns <= t (low half if d >= 0, high half if
// d >= 1), the backward scores for columns >= t (low half if d <= 0, high half if d <= 1).  The table holds, per parity
// of t, the 31 possible pairs (forward mask, backward mask) at index e - (t >> 1) + 15, so that a lane steps through
// consecutive entries as e grows.  kMaskBytes of shared memory; threads 0..61 of the block write it.
constexpr uint32_t kMaskBytes = 512;
__device__ __forceinline__ void build_diag_masks(uint8_t* tab, int tid) {
    if (tid < 62) {
        const int par = tid / 31, n = tid - par * 31, d = 2 * (15 - n) + par;
        const uint32_t fw = (d >= 0 ? 0x3F80u : 0u) | (d >= 1 ? 0x3F800000u : 0u);
        const uint32_t bw = (d <= 0 ? 0x3F80u : 0u) | (d <= 1 ? 0x3F800000u : 0u);
        *reinterpret_cast<uint2*>(tab + (par * 31 + n) * 8) = make_uint2(fw, bw);
    }
}
__device__ __forceinline__ uint32_t fma_bf16x2(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// Packed bf16 values of one 32-column block of P for this thread's row.  REL < 0: the block lies left
// of the diagonal block (forward scores only), REL > 0: right of it (backward only), REL == 0: the
// diagonal block: forward scores for s <= t plus backward scores for s >= t, taken as packed products with the 0 / 1
// masks above (exact off the diagonal; on it the two bf16 values are added and rounded once more).  The scores outside
// the masks are finite: the range check of the gates bounds the growing factors.
template <int REL>
__device__ __forceinline__ void combine_block(uint32_t fwd_addr, uint32_t bwd_addr, int lane, uint32_t masks, uint32_t (&pk)[16]) {
    if (REL != 0) {
        uint32_t r[32];
        tmem_ld32(REL < 0 ? fwd_addr : bwd_addr, r);
        tc_wait_ld();
#pragma unroll
        for (int e = 0; e < 16; ++e) pk[e] = pack_bf16(as_f(r[2 * e]), as_f(r[2 * e + 1]));
    } else if (masks == 0) {
        // no mask table (a kernel without the shared memory for it): the same block by selects in fp32
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t f[16], b[16];
            tmem_ld16(fwd_addr + 16 * h, f);
            tmem_ld16(bwd_addr + 16 * h, b);
            tc_wait_ld();
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int s0 = 16 * h + 2 * e, s1 = s0 + 1;
                const float f0 = as_f(f[2 * e]), b0 = as_f(b[2 * e]), f1 = as_f(f[2 * e + 1]), b1 = as_f(b[2 * e + 1]);
                const float lo = s0 < lane ? f0 : (s0 > lane ? b0 : f0 + b0);
                const float hi = s1 < lane ? f1 : (s1 > lane ? b1 : f1 + b1);
                pk[8 * h + e] = pack_bf16(lo, hi);
            }
        }
    } else {
        const uint32_t mrow = masks + (uint32_t)(((lane & 1) * 31 + 15 - (lane >> 1)) * 8);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint32_t f[16], b[16];
            tmem_ld16(fwd_addr + 16 * h, f);
            tmem_ld16(bwd_addr + 16 * h, b);
            tc_wait_ld();
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                uint32_t mf, mb;
                asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(mf), "=r"(mb) : "r"(mrow + (uint32_t)(8 * h + e) * 8));
                const uint32_t pf = pack_bf16(as_f(f[2 * e]), as_f(f[2 * e + 1])), pb = pack_bf16(as_f(b[2 * e]), as_f(b[2 * e + 1]));
                pk[8 * h + e] = fma_bf16x2(pf, mf, mul_bf16x2(pb, mb));
            }
        }
    }
}
__device__ __forceinline__ void combine_any(int cb, int wq, bool valid, uint32_t fwd_addr, uint32_t bwd_addr, int lane,
                                            uint32_t masks, uint32_t (&pk)[16]) {
    if (!valid) {
#pragma unroll
        for (int e = 0; e < 16; ++e) pk[e] = 0u;
    } else if (cb < wq) {
        combine_block<-1>(fwd_addr, bwd_addr, lane, masks, pk);
    } else if (cb == wq) {
        combine_block<0>(fwd_addr, bwd_addr, lane, masks, pk);
    } else {
        combine_block<1>(fwd_addr, bwd_addr, lane, masks, pk);
    }
}

// Shared-memory matrix descriptor, in halves.  Low word: start address and leading-dimension byte
// offset, both in 16-byte units (bits 0..13 and 16..29), so stepping an operand through shared memory is
// one 32-bit add.  High word: stride-dimension byte offset in 16-byte units (bits 32..45), descriptor
// version 1 (bit 46), swizzle mode in bits 61..63 (0 = none, 2 = 128B, 4 = 64B).
__device__ __forceinline__ uint32_t desc_lo(uint32_t addr, uint32_t lbo_bytes) {
    return ((addr >> 4) & 0x3FFFu) | ((lbo_bytes >> 4) << 16);
}
__host__ __device__ constexpr uint32_t desc_hi(uint32_t sbo_bytes, uint32_t swizzle) {
    return (sbo_bytes >> 4) | (1u << 14) | (swizzle << 29);
}
__device__ __forceinline__ uint64_t desc64(uint32_t lo, uint32_t hi) { return ((uint64_t)hi << 32) | lo; }

constexpr uint32_t kHiK64 = desc_hi(512, 4);     // K-major or MN-major tile with 64-byte rows, 64B swizzle
constexpr uint32_t kHiV128 = desc_hi(1024, 2);   // MN-major tile with 128-byte rows, 128B swizzle
constexpr uint32_t kHiZ = desc_hi(256, 0);       // 0/1 tile, no swizzle

// 1 / x for two packed positive, normal bf16 values without the special-function unit and without leaving the
// packed format: a bit-level first guess per half (one 32-bit subtraction: neither half borrows) and one Newton
// step r (2 - x r) in bf16x2 arithmetic.  Relative error at most 0.63 % (root mean square 0.27 %, the same as
// rounding an exact reciprocal to bf16 after a first guess of this kind); the result only scales bf16 operands,
// whose own rounding unit is 0.39 %, and it is the reciprocal of the very factor the other operand is scaled by.
__device__ __forceinline__ uint32_t rcp_bf16x2(uint32_t x) {
    const uint32_t r0 = 0x7EF27EF2u - x;
    const __nv_bfloat162 xb = *reinterpret_cast<const __nv_bfloat162*>(&x), rb = *reinterpret_cast<const __nv_bfloat162*>(&r0);
    const __nv_bfloat162 r1 = __hmul2(rb, __hfma2(__hneg2(xb), rb, __float2bfloat162_rn(2.0f)));
    return *reinterpret_cast<const uint32_t*>(&r1);
}

// Builds the 240-row 0/1 tile of the prefix sums (K-major without swizzle: 8-row groups of 256 bytes, each two
// 8x8 core matrices for K 0..7 and K 8..15).  Rows 0..111 are zeros, rows 112..127 the lower triangle (diagonal
// included), rows 128..239 ones.  The 128-row window starting at row 112 - 16 j is the operand of K step j.
// Threads 0..239 of the block write (pass tid + blockDim.x in a second call when the block has fewer).
__device__ __forceinline__ void build_zero_one_tile(uint8_t* zf, int tid) {
    if (tid < (int)kZRows) {
        uint32_t f[8];
#pragma unroll
        for (int p = 0; p < 8; ++p) {
            uint32_t wf = 0;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int kk = 2 * p + h, u = tid - 112;
                const bool one_f = tid >= 128 || (tid >= 112 && kk <= u);
                wf |= (one_f ? 0x3F80u : 0u) << (16 * h);
            }
            f[p] = wf;
        }
        const uint32_t off = (uint32_t)(tid >> 3) * 256 + (uint32_t)(tid & 7) * 16;
        *reinterpret_cast<uint4*>(zf + off) = make_uint4(f[0], f[1], f[2], f[3]);
        *reinterpret_cast<uint4*>(zf + off + 128) = make_uint4(f[4], f[5], f[6], f[7]);
    }
}

}  // namespace umma
}  // namespace vig
