// bf16 BiGLA forward on the 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM).
//
// One thread block owns one (batch, head) unit of up to 256 tokens, split into chunks of C = 128.
// With b_t the inclusive prefix sum of log alpha> from the start of the chunk (e_t the inclusive
// suffix sum of log alpha< to its end), Eq. 6 becomes, per chunk,
//     P    = tril(q~> k~>^T) + triu(q~< k~<^T)          q~> = q e^{b},  k~> = k e^{-b},  q~< = q e^{e},  k~< = k e^{-e}
//     out  = ( P v + q~> S>_in + q~< S<_in ) / 2
//     U    = [k~< | k~>]^T v                            (zero-input chunk summaries, both directions in one MMA)
//     S>_in(c+1) = (S>_in(c) + U>_c) * e^{b_last}       (rows scaled; mirrored for <)
// Every product is a tcgen05.mma with M = 128: P (N = 128, K = dk), U (A = the four operand tiles stacked
// along M, MN-major), P v (A = bf16 P read straight from TMEM), q~ S (B = the bf16 state tile).  The
// threads only do the element-wise work: operand scaling in place (phase 1), masking / packing P,
// scaling the chunk summaries, and the output epilogue.  TMEM use is 256 columns, shared memory
// 109 KB, so two blocks share an SM and one block's MMA round trips hide behind the other's
// element-wise phases.
#include <cuda.h>

#include "ptx.cuh"
#include "recurrence.cuh"
#include "tma_host.h"
#include "vig_internal.h"

namespace vig {
namespace {

constexpr int kBlk = 16;        // rows per prefix-sum block
constexpr int kChunk = 128;     // rows per MMA chunk
constexpr int kRows = 256;      // rows of every shared-memory tile (TMA zero-fills rows >= L)
constexpr int kThreads = 256;
constexpr float kGateRange = 60.f;
constexpr float kLog2e = 1.4426950408889634f;

// TMEM column map (256 columns allocated)
constexpr uint32_t kT1 = 0;      // P tile, fp32 [128 x 128]; later bf16 P in its first 64 columns
constexpr uint32_t kTO = 128;    // output accumulator [128 x 64]; before that, the summary U of chunk 1
constexpr uint32_t kTU = 192;    // summary U of chunk 0 [128 x 64]
constexpr uint32_t kTmemCols = 256;

// ---- tcgen05 wrappers ------------------------------------------------------------------------
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Shared-memory matrix descriptor (start address, leading / stride byte offsets in 16-byte units,
// descriptor version 1, swizzle mode in bits 61..63: 2 = 128B, 4 = 64B).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t swizzle) {
    return (uint64_t)((addr >> 4) & 0x3FFF) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32) | ((uint64_t)1 << 46) | ((uint64_t)swizzle << 61);
}
// Instruction descriptor of kind::f16: fp32 accumulate, bf16 A and B, majors, N >> 3, M >> 4.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, int a_mn_major, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
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
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

struct USmem {
    static constexpr uint32_t a0 = 0;                          // four q-type tiles, 16 KB each
    static constexpr uint32_t tile = kRows * 64;
    static constexpr uint32_t v = 4 * tile;                    // v tile, later the output tile (32 KB)
    static constexpr uint32_t s_fwd = v + kRows * 128;         // bf16 state entering chunk 1 from the left  [32 x 64]
    static constexpr uint32_t s_bwd = s_fwd + 32 * 128;        // bf16 state entering chunk 0 from the right [32 x 64]
    static constexpr uint32_t tot = s_bwd + 32 * 128;          // [2][16][32] fp32 block sums of log2 alpha
    static constexpr uint32_t misc = tot + 2 * 16 * 32 * 4;    // mbarriers, TMEM slot, flag
    static constexpr uint32_t total = misc + 64;
};

struct UArgs {
    const __nv_bfloat16 *q, *k, *v, *la_f, *la_b;
    __nv_bfloat16* out;
    int L;
    int* dev_status;
};

template <int DK, int DV>
__global__ void __launch_bounds__(kThreads, 2)
bigla_umma_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_f, const __grid_constant__ CUtensorMap tm_b,
                  const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o, const UArgs args) {
    static_assert((DK == 24 || DK == 32) && (DV == 48 || DV == 64), "unsupported head size");
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* bp = smem_raw + (base - smem_u32(smem_raw));

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int unit = blockIdx.x, L = args.L;
    const int nb = (L + kBlk - 1) / kBlk, nc = (L + kChunk - 1) / kChunk;
    const uint32_t bar_tma = base + USmem::misc, bar_mma = bar_tma + 8, slot = bar_tma + 16;
    volatile uint32_t* slot_p = reinterpret_cast<volatile uint32_t*>(bp + USmem::misc + 16);
    volatile int* slow_flag = reinterpret_cast<volatile int*>(bp + USmem::misc + 20);
    float* tot = reinterpret_cast<float*>(bp + USmem::tot);
    uint32_t mma_phase = 0;
    bool timed_out = false;

    if (tid == 0) {
        mbar_init(bar_tma, 1);
        mbar_init(bar_mma, 1);
        *slow_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"(kTmemCols));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *slot_p;

    if (tid == 0) {
        mbar_expect_tx(bar_tma, kRows * (4 * 64 + 128));
        tma_load_3d(base + USmem::a0 + 0 * USmem::tile, &tm_q, 0, 0, unit, bar_tma);
        tma_load_3d(base + USmem::a0 + 1 * USmem::tile, &tm_k, 0, 0, unit, bar_tma);
        tma_load_3d(base + USmem::a0 + 2 * USmem::tile, &tm_f, 0, 0, unit, bar_tma);
        tma_load_3d(base + USmem::a0 + 3 * USmem::tile, &tm_b, 0, 0, unit, bar_tma);
        tma_load_3d(base + USmem::v, &tm_v, 0, 0, unit, bar_tma);
    }
    if (__syncthreads_or(mbar_wait_bounded(bar_tma, 0) ? 0 : 1)) {
        mbar_wait_bounded(bar_tma, 0);   // a second bounded chance for copies still in flight
        timed_out = true;
    }

    if (!timed_out) {
        // ---- phase 1a: per-block sums of log2(alpha), both directions ------------------------------
        const int dir = lane >> 4, cp = lane & 15;
        const bool active = cp < DK / 2;
        const int chunk16 = cp >> 2, inchunk = (cp & 3) * 4;
        const uint32_t q_t = base + USmem::a0, k_t = q_t + USmem::tile, g_t = q_t + (2 + dir) * USmem::tile;
        const uint32_t kout_t = dir == 0 ? k_t : q_t;
        for (int n = warp; n < nb; n += kThreads / 32) {
            float sx = 0.f, sy = 0.f;
            if (active) {
#pragma unroll
                for (int m = 0; m < 16; ++m) {
                    const int r = dir == 0 ? m : 15 - m;
                    const float2 gf = unpack_bf16(lds32(g_t + sw_off<64>(n * kBlk + r, chunk16) + inchunk));
                    sx += gf.x;
                    sy += gf.y;
                }
            }
            *reinterpret_cast<float2*>(tot + (dir * 16 + n) * 32 + 2 * cp) = make_float2(sx * kLog2e, sy * kLog2e);
        }
        __syncthreads();

        // ---- phase 1b: scaled operands, in place; exponents run from the chunk boundary ----------------
        // Half-warp 0 walks a block downwards (forward gate, prefix sums), half-warp 1 upwards (backward
        // gate, suffix sums); q~ replaces the lane's gate values at once, k~ replaces k (forward) or q
        // (backward) from step 8 on, when both half-warps have read the row.
        for (int n = warp; n < nb; n += kThreads / 32) {
            const int first = n & ~7, last = min(first + 7, nb - 1);
            float accx = 0.f, accy = 0.f;
            if (dir == 0) {
                for (int m = first; m < n; ++m) {
                    const float2 t = *reinterpret_cast<const float2*>(tot + m * 32 + 2 * cp);
                    accx += t.x; accy += t.y;
                }
            } else {
                for (int m = last; m > n; --m) {
                    const float2 t = *reinterpret_cast<const float2*>(tot + (16 + m) * 32 + 2 * cp);
                    accx += t.x; accy += t.y;
                }
            }
            uint32_t held[8];
#pragma unroll
            for (int m = 0; m < 16; ++m) {
                const int r = dir == 0 ? m : 15 - m;
                const uint32_t off = sw_off<64>(n * kBlk + r, chunk16) + inchunk;
                uint32_t kt = 0;
                if (active) {
                    const float2 qf = unpack_bf16(lds32(q_t + off));
                    const float2 kf = unpack_bf16(lds32(k_t + off));
                    const float2 gf = unpack_bf16(lds32(g_t + off));
                    accx = fmaf(gf.x, kLog2e, accx);
                    accy = fmaf(gf.y, kLog2e, accy);
                    const float ex = ex2(accx), ey = ex2(accy), ix = ex2(-accx), iy = ex2(-accy);
                    sts32(g_t + off, pack_bf16(qf.x * ex, qf.y * ey));   // q~ = q e^{b}
                    kt = pack_bf16(kf.x * ix, kf.y * iy);                // k~ = k e^{-b}
                }
                if (m < 8) {
                    held[m] = kt;
                } else {
                    __syncwarp();
                    if (active) {
                        sts32(kout_t + off, kt);
                        const int r2 = dir == 0 ? 15 - m : m;
                        sts32(kout_t + sw_off<64>(n * kBlk + r2, chunk16) + inchunk, held[15 - m]);
                    }
                }
            }
            if (active && fminf(accx, accy) < -kGateRange * kLog2e) *slow_flag = 1;
        }
        fence_async_smem();   // operand tiles were written through the generic proxy, the MMAs read them through the async proxy
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    }

    const bool slow = !timed_out && *slow_flag != 0;
    if (!timed_out && !slow) {
        const int wq = warp & 3, half = warp >> 2;
        const uint32_t lane_base = (uint32_t)(wq * 32) << 16;
        constexpr uint32_t kIdP = instr_desc(128, 128, 0, 0);
        constexpr uint32_t kIdU = instr_desc(128, 64, 1, 1);
        constexpr uint32_t kIdO = instr_desc(128, 64, 0, 1);
        const uint32_t aT = base + USmem::a0, vT = base + USmem::v;

        // P of one direction for chunk c -> T1 (issued by one thread)
        auto issue_p = [&](int c, int d) {
            const uint32_t qa = aT + (2 + d) * USmem::tile + c * (kChunk * 64);
            const uint32_t ka = aT + (d == 0 ? 1 : 0) * USmem::tile + c * (kChunk * 64);
#pragma unroll
            for (int kk = 0; kk < 2; ++kk)
                umma_ss(tmem + kT1, smem_desc(qa + kk * 32, 16, 512, 4), smem_desc(ka + kk * 32, 16, 512, 4), kIdP, kk > 0);
        };
        auto issue_u = [&](int c, uint32_t dcol) {
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
                umma_ss(tmem + dcol, smem_desc(aT + c * (kChunk * 64) + kk * 1024, USmem::tile, 512, 4),
                        smem_desc(vT + c * (kChunk * 128) + kk * 2048, 16, 1024, 2), kIdU, kk > 0);
        };
        auto issue_o = [&](int c) {
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
                umma_ts(tmem + kTO, tmem + kT1 + kk * 8, smem_desc(vT + c * (kChunk * 128) + kk * 2048, 16, 1024, 2), kIdO,
                        kk > 0);
            if (nc == 2) {
                // inter-chunk term: chunk 1 gets the forward state of chunk 0, chunk 0 the backward state of chunk 1
                const uint32_t qa = aT + (c == 1 ? 2 : 3) * USmem::tile + c * (kChunk * 64);
                const uint32_t sa = base + (c == 1 ? USmem::s_fwd : USmem::s_bwd);
#pragma unroll
                for (int kk = 0; kk < 2; ++kk)
                    umma_ss(tmem + kTO, smem_desc(qa + kk * 32, 16, 512, 4), smem_desc(sa + kk * 2048, 16, 1024, 2), kIdO, 1);
            }
        };
        auto wait_mma = [&]() -> bool {
            const int bad = mbar_wait_bounded(bar_mma, mma_phase & 1) ? 0 : 1;
            ++mma_phase;
            const bool fail = __syncthreads_or(bad) != 0;
            tc_fence_after();
            return !fail;
        };

        if (tid == 0) {
            if (nc == 2) {
                issue_u(0, kTU);
                issue_u(1, kTO);
            }
            issue_p(0, 0);
            umma_commit(bar_mma);
        }

        for (int c = 0; c < nc && !timed_out; ++c) {
            const int rows_here = min(kChunk, L - c * kChunk);
            const bool rows_live = wq * 32 < rows_here;   // this warp's 32 rows hold at least one token
            uint32_t pk[2][16];
            float dg[32];
            if (!wait_mma()) { timed_out = true; break; }

            // forward part of P: column blocks below the diagonal, and the diagonal block masked to s <= t
            if (rows_live) {
#pragma unroll
                for (int bl = 0; bl < 2; ++bl) {
                    const int cb = 2 * half + bl;
                    if (cb < wq) {
                        uint32_t r[32];
                        tmem_ld32(tmem + kT1 + lane_base + cb * 32, r);
                        tc_wait_ld();
#pragma unroll
                        for (int e = 0; e < 16; ++e)
                            pk[bl][e] = pack_bf16(__uint_as_float(r[2 * e]), __uint_as_float(r[2 * e + 1]));
                    } else if (cb == wq) {
                        uint32_t r[32];
                        tmem_ld32(tmem + kT1 + lane_base + cb * 32, r);
                        tc_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) dg[e] = e <= lane ? __uint_as_float(r[e]) : 0.f;
                    }
                }
            }
            // chunk summaries -> bf16 state tiles (first chunk only; warps 4 and 5 have no forward P work)
            if (c == 0 && nc == 2 && (warp == 4 || warp == 5)) {
                const bool fwd = warp == 5;   // lanes 32..63 of U hold k~>^T v, lanes 0..31 hold k~<^T v
                const uint32_t ucol = fwd ? kTU : kTO;
                float dsum = 0.f;
                const int b0 = fwd ? 0 : 8, b1 = fwd ? 8 : nb;
                for (int m = b0; m < b1; ++m) dsum += tot[((fwd ? 0 : 16) + m) * 32 + lane];
                const float dec = ex2(dsum);   // decay of the whole chunk for key dim `lane`
                const uint32_t st = base + (fwd ? USmem::s_fwd : USmem::s_bwd);
#pragma unroll
                for (int hb = 0; hb < 2; ++hb) {
                    uint32_t r[32];
                    tmem_ld32(tmem + ucol + lane_base + hb * 32, r);
                    tc_wait_ld();
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
                        uint32_t o[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            o[e] = pack_bf16(__uint_as_float(r[ch * 8 + 2 * e]) * dec, __uint_as_float(r[ch * 8 + 2 * e + 1]) * dec);
                        sts128(st + sw_off<128>(lane, hb * 4 + ch), o[0], o[1], o[2], o[3]);
                    }
                }
                fence_async_smem();
            }
            tc_fence_before();
            __syncthreads();
            tc_fence_after();
            if (tid == 0) {
                issue_p(c, 1);
                umma_commit(bar_mma);
            }
            if (!wait_mma()) { timed_out = true; break; }

            // backward part of P, combine, pack, and put bf16 P where the P v MMA reads it
            if (rows_live) {
#pragma unroll
                for (int bl = 0; bl < 2; ++bl) {
                    const int cb = 2 * half + bl;
                    if (cb > wq) {
                        uint32_t r[32];
                        tmem_ld32(tmem + kT1 + lane_base + cb * 32, r);
                        tc_wait_ld();
#pragma unroll
                        for (int e = 0; e < 16; ++e)
                            pk[bl][e] = pack_bf16(__uint_as_float(r[2 * e]), __uint_as_float(r[2 * e + 1]));
                    } else if (cb == wq) {
                        uint32_t r[32];
                        tmem_ld32(tmem + kT1 + lane_base + cb * 32, r);
                        tc_wait_ld();
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            const float lo = (2 * e >= lane ? __uint_as_float(r[2 * e]) : 0.f) + dg[2 * e];
                            const float hi = (2 * e + 1 >= lane ? __uint_as_float(r[2 * e + 1]) : 0.f) + dg[2 * e + 1];
                            pk[bl][e] = pack_bf16(lo, hi);
                        }
                    }
                }
            }
            named_bar(1 + wq, 64);   // both warps of this row quadrant have finished reading fp32 P
            if (rows_live) {
#pragma unroll
                for (int bl = 0; bl < 2; ++bl) tmem_st16(tmem + kT1 + lane_base + (2 * half + bl) * 16, pk[bl]);
                tc_wait_st();
            }
            tc_fence_before();
            __syncthreads();
            tc_fence_after();
            if (tid == 0) {
                issue_o(c);
                umma_commit(bar_mma);
            }
            if (!wait_mma()) { timed_out = true; break; }
            if (tid == 0 && c + 1 < nc) {
                issue_p(c + 1, 0);   // next chunk's forward P runs while this chunk's output is written out
                umma_commit(bar_mma);
            }

            // epilogue: out = O / 2, bf16, into the dead v tile of this chunk (same swizzle as the TMA store expects)
            if (rows_live) {
                uint32_t r[32];
                tmem_ld32(tmem + kTO + lane_base + half * 32, r);
                tc_wait_ld();
                const int row = c * kChunk + wq * 32 + lane;
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    uint32_t o[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        o[e] = pack_bf16(0.5f * __uint_as_float(r[ch * 8 + 2 * e]), 0.5f * __uint_as_float(r[ch * 8 + 2 * e + 1]));
                    sts128(vT + sw_off<128>(row, half * 4 + ch), o[0], o[1], o[2], o[3]);
                }
            }
            tc_fence_before();   // the next chunk's O MMA overwrites the accumulator only after these loads
        }

        if (!timed_out) {
            fence_async_smem();
            __syncthreads();
            if (tid == 0) {
                tma_store_3d(&tm_o, 0, 0, unit, vT);   // rows >= L and columns >= dv are clipped
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            }
        }
    }

    // ---- release TMEM (every tcgen05 operation of this block has completed or was never issued) ----
    tc_fence_before();
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols));
    if (timed_out) {
        if (tid == 0) atomicOr(args.dev_status, kDevStatusTimeout);
        return;
    }
    if (slow) {
        // A gate left the range the factorised tiles can represent: evaluate this unit by the recurrence.
        const size_t ok = (size_t)unit * L * DK, ov = (size_t)unit * L * DV;
        recurrence_unit<__nv_bfloat16>(args.q + ok, args.k + ok, args.v + ov, args.la_f + ok, args.la_b + ok,
                                       args.out + ov, L, DK, DV, reinterpret_cast<float*>(bp));
    }
}

template <int DK, int DV>
cudaError_t launch_umma_t(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                          const __nv_bfloat16* la_f, const __nv_bfloat16* la_b, __nv_bfloat16* out, long long units, int L,
                          cudaStream_t stream) {
    CUtensorMap tq, tk, tf, tb, tv, to;
    if (!make_map(&tq, q, units, L, DK, 32, kRows) || !make_map(&tk, k, units, L, DK, 32, kRows) ||
        !make_map(&tf, la_f, units, L, DK, 32, kRows) || !make_map(&tb, la_b, units, L, DK, 32, kRows) ||
        !make_map(&tv, v, units, L, DV, 64, kRows) || !make_map(&to, out, units, L, DV, 64, kRows))
        return cudaErrorInvalidValue;
    UArgs a{};
    a.q = q; a.k = k; a.v = v; a.la_f = la_f; a.la_b = la_b; a.out = out; a.L = L;
    a.dev_status = device_status_ptr();
    if (!a.dev_status) return cudaErrorUnknown;
    size_t smem = USmem::total + 1024;
    const size_t rec = (size_t)rec_plan(kThreads, DK, DV).smem_floats * 4 + 1024;
    if (smem < rec) smem = rec;
    cudaError_t e = cudaFuncSetAttribute(bigla_umma_kernel<DK, DV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    bigla_umma_kernel<DK, DV><<<(unsigned)units, kThreads, smem, stream>>>(tq, tk, tf, tb, tv, to, a);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

bool umma_supported(int dk, int dv, int L) { return (dk == 24 || dk == 32) && (dv == 48 || dv == 64) && L <= kRows; }

cudaError_t launch_bigla_umma(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                              const __nv_bfloat16* la_f, const __nv_bfloat16* la_b, __nv_bfloat16* out, long long units,
                              int L, int dk, int dv, cudaStream_t stream) {
#define VIG_CASE(DK_, DV_) \
    if (dk == DK_ && dv == DV_) return launch_umma_t<DK_, DV_>(q, k, v, la_f, la_b, out, units, L, stream);
    VIG_CASE(24, 48) VIG_CASE(24, 64) VIG_CASE(32, 48) VIG_CASE(32, 64)
#undef VIG_CASE
    return cudaErrorNotSupported;
}

}  // namespace vig
