// bf16 tensor-core BiGLA forward for sm_100a.
//
// Chunkwise form of the two recurrences of Eq. 6 with 16-token blocks.  With b_t the inclusive
// prefix sum of log alpha> inside a block and S>_in the state entering the block,
//     o>_t  = (q_t * e^{b_t}) S>_in + sum_{s<=t} [ (q_t * e^{b_t}) . (k_s * e^{-b_s}) ] v_s
//     S>_out = ( S>_in + sum_s (k_s * e^{-b_s})^T v_s ) * e^{b_last}      (row i scaled by e^{b_last,i})
// and the mirror image for the backward direction with inclusive suffix sums.  All three products
// are bf16 mma.sync tiles with fp32 accumulators; both running states stay in registers.
//
// One thread block owns one segment (a whole unit when L <= 256) that five tiled TMA loads bring
// into swizzled shared memory once; TMA's out-of-bounds zero fill supplies the padding (dk -> 16k,
// rows -> 16n).  Phase 1 turns (q, k, log alpha>, log alpha<) in place into the scaled operands
// (q e^{b}, k e^{-b}) of both directions.  Phase 2 sweeps: one warp group walks the blocks left to
// right, the other right to left; the first direction to visit a block parks its partial output in
// shared memory, the second adds its own, halves, and writes the result over the dead v tile,
// which one TMA store sends to HBM.  Long sequences run as summary -> fold -> main launches whose
// segment boundary states travel through scratch memory.
#include <cuda.h>

#include "ptx.cuh"
#include "recurrence.cuh"
#include "tma_host.h"
#include "vig_internal.h"

namespace vig {
namespace {

constexpr int kBlk = 16;            // tokens per block
constexpr int kMaxSegBlocks = 16;   // TMA box rows <= 256
constexpr int kLongSegBlocks = 8;   // segment length of the multi-launch path: 128 tokens
constexpr float kGateRange = 60.f;  // |sum of log alpha over a block| above this -> exact recurrence
constexpr float kLog2e = 1.4426950408889634f;

enum Mode { kMain = 0, kSummary = 1 };

// ------------------------------------------------------------------------------------------------
// Compile-time geometry of one (dk, dv) instantiation
// ------------------------------------------------------------------------------------------------
template <int DK, int DV>
struct Geo {
    static constexpr int DKP = (DK + 15) / 16 * 16;   // key dim padded to the MMA k step
    static constexpr int DVP = DV <= 32 ? 32 : 64;    // value row length in shared memory
    static constexpr int RBK = DKP * 2;               // bytes per row of the q-type tiles
    static constexpr int RBV = DVP * 2;
    static constexpr int JW = DV == 48 ? 48 : 32;     // value columns per sweep warp
    static constexpr int NWD = DV / JW;               // sweep warps per direction
    static constexpr int NWARPS = 2 * NWD < 4 ? 4 : 2 * NWD;
    static constexpr int NT = NWARPS * 32;
    static constexpr int KT = DKP / 16, IT = DKP / 8, JT = JW / 8, MT = JW / 16;
    static_assert(DKP <= 32 && DV <= 64 && DV % 16 == 0 && DK % 8 == 0, "unsupported head size");
    static_assert(RBK == 32 || RBK == 64 || RBK == 128, "row bytes must equal a swizzle span");
};

struct SmemPlan {
    uint32_t a[4];      // q-type tiles: after phase 1 they hold  k~<, k~>, q~>, q~<
    uint32_t v;         // v tile, later the finished output tile
    uint32_t part;      // parked partial outputs
    uint32_t dfac;      // [2][nb][DKP] fp32 block decay factors
    uint32_t misc;      // mbarrier (8 B) + slow flag (4 B)
    uint32_t total;
};

template <int DK, int DV>
__host__ __device__ inline SmemPlan smem_plan(int box_blocks) {
    using G = Geo<DK, DV>;
    SmemPlan p;
    const uint32_t rows = box_blocks * kBlk;
    uint32_t off = 0;
    for (int i = 0; i < 4; ++i) { p.a[i] = off; off += rows * G::RBK; }
    off = (off + 1023) / 1024 * 1024;
    p.v = off; off += rows * G::RBV;
    p.part = off; off += rows * DV * 2;
    p.dfac = off; off += 2 * box_blocks * G::DKP * 4;
    p.misc = off; off += 16;
    p.total = off;
    return p;
}

struct KernelArgs {
    const __nv_bfloat16 *q, *k, *v, *la_f, *la_b;
    __nv_bfloat16* out;
    int L, nseg, box_blocks;
    float* ws_state;   // [units][nseg][2][DV][DKP]: segment summaries, folded in place into incoming states
    float* ws_decay;   // [units][nseg][2][DKP]: product of the block decay factors of a segment
    int* ws_flags;     // [units]: unit needs the exact recurrence
    int* dev_status;
};

// ------------------------------------------------------------------------------------------------
// The kernel
// ------------------------------------------------------------------------------------------------
template <int DK, int DV, int MODE>
__global__ void __launch_bounds__(Geo<DK, DV>::NT)
bigla_mma_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_f, const __grid_constant__ CUtensorMap tm_b,
                 const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                 const KernelArgs args) {
    using G = Geo<DK, DV>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const SmemPlan sp = smem_plan<DK, DV>(args.box_blocks);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int unit = blockIdx.x / args.nseg, seg = blockIdx.x - unit * args.nseg;
    const int row0 = seg * args.box_blocks * kBlk;                       // first token of this segment
    const int nb = min(args.box_blocks, (args.L - row0 + kBlk - 1) / kBlk);   // blocks with at least one token
    const uint32_t bar = base + sp.misc;
    volatile int* slow_flag = reinterpret_cast<volatile int*>(base_ptr + sp.misc + 8);

    if (MODE == kMain && args.nseg > 1 && args.ws_flags[unit] != 0) {
        // A gate of this unit left the factorised range somewhere: segment 0 evaluates the whole
        // unit by the recurrence, the other segments have nothing to do.
        if (seg == 0) {
            const size_t ok = (size_t)unit * args.L * DK, ov = (size_t)unit * args.L * DV;
            recurrence_unit<__nv_bfloat16>(args.q + ok, args.k + ok, args.v + ov, args.la_f + ok, args.la_b + ok,
                                           args.out + ov, args.L, DK, DV, reinterpret_cast<float*>(base_ptr));
        }
        return;
    }

    // ---- phase 0: bring the segment on chip --------------------------------------------------
    if (tid == 0) {
        mbar_init(bar, 1);
        *slow_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (tid == 0) {
        const uint32_t rows = args.box_blocks * kBlk;
        const uint32_t bytes = rows * ((MODE == kMain ? 4u : 3u) * G::RBK + G::RBV);
        mbar_expect_tx(bar, bytes);
        if (MODE == kMain) tma_load_3d(base + sp.a[0], &tm_q, 0, row0, unit, bar);
        tma_load_3d(base + sp.a[1], &tm_k, 0, row0, unit, bar);
        tma_load_3d(base + sp.a[2], &tm_f, 0, row0, unit, bar);
        tma_load_3d(base + sp.a[3], &tm_b, 0, row0, unit, bar);
        tma_load_3d(base + sp.v, &tm_v, 0, row0, unit, bar);
    }
    {
        const int timed_out = mbar_wait_bounded(bar, 0) ? 0 : 1;
        if (__syncthreads_or(timed_out)) {   // block-uniform decision
            if (tid == 0) atomicOr(args.dev_status, kDevStatusTimeout);
            mbar_wait_bounded(bar, 0);       // give copies still in flight a second bounded chance to land
            return;
        }
    }

    // ---- phase 1: scaled operands, in place ---------------------------------------------------
    // Half-warp 0 walks a block downwards with the forward gate (inclusive prefix sums), half-warp 1
    // upwards with the backward gate (inclusive suffix sums); lane = pair of key dims.  q~ replaces the
    // lane's own gate values at once.  k~ may replace k (forward) or q (backward) only after both
    // half-warps have read that row, i.e. from step 8 on; the first eight results wait in registers.
    {
        const int dir = lane >> 4, cp = lane & 15;
        const bool active = cp < DK / 2, padcol = !active && cp < G::DKP / 2;
        const int chunk = cp >> 2, inchunk = (cp & 3) * 4;
        const uint32_t q_t = base + sp.a[0], k_t = base + sp.a[1], g_t = base + sp.a[2 + dir];
        const uint32_t kout_t = dir == 0 ? k_t : q_t;
        float* dfac = reinterpret_cast<float*>(base_ptr + sp.dfac) + (size_t)dir * args.box_blocks * G::DKP;
        for (int n = warp; n < nb; n += G::NWARPS) {
            float accx = 0.f, accy = 0.f;   // running sum of log2(alpha)
            uint32_t held[8];
#pragma unroll
            for (int m = 0; m < 16; ++m) {
                const int r = dir == 0 ? m : 15 - m;
                const uint32_t off = sw_off<G::RBK>(n * kBlk + r, chunk) + inchunk;
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
                } else if (MODE == kSummary && padcol && dir == 1) {
                    sts32(kout_t + off, 0u);   // the q tile was not loaded: its padding columns hold no zeros yet
                }
                if (m < 8) {
                    held[m] = kt;
                } else {
                    __syncwarp();
                    if (active) {
                        sts32(kout_t + off, kt);
                        const int r2 = dir == 0 ? 15 - m : m;
                        sts32(kout_t + sw_off<G::RBK>(n * kBlk + r2, chunk) + inchunk, held[15 - m]);
                    }
                }
            }
            if (active) {
                *reinterpret_cast<float2*>(dfac + n * G::DKP + 2 * cp) = make_float2(ex2(accx), ex2(accy));
                if (fminf(accx, accy) < -kGateRange * kLog2e) *slow_flag = 1;
            } else if (padcol) {
                *reinterpret_cast<float2*>(dfac + n * G::DKP + 2 * cp) = make_float2(1.f, 1.f);
            }
        }
    }
    __syncthreads();

    if (*slow_flag != 0) {
        if (MODE == kSummary) {
            if (tid == 0) args.ws_flags[unit] = 1;
            return;
        }
        if (args.nseg == 1) {
            const size_t ok = (size_t)unit * args.L * DK, ov = (size_t)unit * args.L * DV;
            recurrence_unit<__nv_bfloat16>(args.q + ok, args.k + ok, args.v + ov, args.la_f + ok, args.la_b + ok,
                                           args.out + ov, args.L, DK, DV, reinterpret_cast<float*>(base_ptr));
            return;
        }
        // nseg > 1 and this flag set means the summary launch flagged the unit already (same data, same
        // arithmetic), which the check at the top of the kernel has handled.
    }

    // ---- phase 2: the two sweeps -----------------------------------------------------------------
    if (warp < 2 * G::NWD) {
        const int dir = warp / G::NWD, w = warp - dir * G::NWD;
        const int g = lane >> 2, tig = lane & 3, mi = lane >> 3, l7 = lane & 7;
        const uint32_t qt_t = base + sp.a[2 + dir];             // q~ of this direction
        const uint32_t kt_t = base + sp.a[dir == 0 ? 1 : 0];    // k~ of this direction
        const uint32_t v_t = base + sp.v, part_t = base + sp.part;
        const float* dfac = reinterpret_cast<const float*>(base_ptr + sp.dfac) + (size_t)dir * args.box_blocks * G::DKP;
        const int jchunk0 = w * G::JW / 8;

        float ST[G::MT][G::IT][4];   // state, transposed: rows = value dims of this warp, cols = key dims
        const size_t st_off = (((size_t)unit * args.nseg + seg) * 2 + dir) * DV * G::DKP;
        if (MODE == kMain && args.nseg > 1) {
            const float* sin = args.ws_state + st_off;
#pragma unroll
            for (int mt = 0; mt < G::MT; ++mt)
#pragma unroll
                for (int it = 0; it < G::IT; ++it) {
                    const int j = w * G::JW + mt * 16 + g, i = it * 8 + 2 * tig;
                    const float2 lo = *reinterpret_cast<const float2*>(sin + (size_t)j * G::DKP + i);
                    const float2 hi = *reinterpret_cast<const float2*>(sin + (size_t)(j + 8) * G::DKP + i);
                    ST[mt][it][0] = lo.x; ST[mt][it][1] = lo.y; ST[mt][it][2] = hi.x; ST[mt][it][3] = hi.y;
                }
        } else {
#pragma unroll
            for (int mt = 0; mt < G::MT; ++mt)
#pragma unroll
                for (int it = 0; it < G::IT; ++it)
#pragma unroll
                    for (int e = 0; e < 4; ++e) ST[mt][it][e] = 0.f;
        }
        float dprod[G::IT][2];   // summary mode: product of the block decay factors
#pragma unroll
        for (int it = 0; it < G::IT; ++it) dprod[it][0] = dprod[it][1] = 1.f;

        for (int m = 0; m < nb; ++m) {
            const int n = dir == 0 ? m : nb - 1 - m;
            const int rbase = n * kBlk;

            // v fragments: B operand of P.V and (regrouped) A operand of the state update
            uint32_t vf[G::JT][2];
#pragma unroll
            for (int jp = 0; jp < G::JT / 2; ++jp) {
                uint32_t r[4];
                ldsm_x4_t(v_t + sw_off<G::RBV>(rbase + (mi & 1) * 8 + l7, jchunk0 + 2 * jp + (mi >> 1)), r);
                vf[2 * jp][0] = r[0]; vf[2 * jp][1] = r[1]; vf[2 * jp + 1][0] = r[2]; vf[2 * jp + 1][1] = r[3];
            }

            if (MODE == kMain) {
                uint32_t qf[G::KT][4];
#pragma unroll
                for (int kt = 0; kt < G::KT; ++kt)
                    ldsm_x4(qt_t + sw_off<G::RBK>(rbase + (mi & 1) * 8 + l7, 2 * kt + (mi >> 1)), qf[kt]);

                // intra-block scores P[t][s] = q~_t . k~_s, masked to s <= t (forward) or s >= t (backward)
                float P[2][4];
#pragma unroll
                for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) P[nt][e] = 0.f;
#pragma unroll
                for (int kt = 0; kt < G::KT; ++kt) {
                    uint32_t kf[4];
                    ldsm_x4(kt_t + sw_off<G::RBK>(rbase + (mi >> 1) * 8 + l7, 2 * kt + (mi & 1)), kf);
                    mma16816(P[0], qf[kt][0], qf[kt][1], qf[kt][2], qf[kt][3], kf[0], kf[1]);
                    mma16816(P[1], qf[kt][0], qf[kt][1], qf[kt][2], qf[kt][3], kf[2], kf[3]);
                }
#pragma unroll
                for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int t = g + (e >> 1) * 8, s = nt * 8 + 2 * tig + (e & 1);
                        const bool keep = dir == 0 ? (s <= t) : (s >= t);
                        if (!keep) P[nt][e] = 0.f;
                    }
                const uint32_t pa0 = pack_bf16(P[0][0], P[0][1]), pa1 = pack_bf16(P[0][2], P[0][3]);
                const uint32_t pa2 = pack_bf16(P[1][0], P[1][1]), pa3 = pack_bf16(P[1][2], P[1][3]);

                // o = P v + q~ S_in
                float O[G::JT][4];
#pragma unroll
                for (int jt = 0; jt < G::JT; ++jt) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) O[jt][e] = 0.f;
                    mma16816(O[jt], pa0, pa1, pa2, pa3, vf[jt][0], vf[jt][1]);
                    const int mt = jt >> 1, h = (jt & 1) * 2;
#pragma unroll
                    for (int kt = 0; kt < G::KT; ++kt) {
                        const uint32_t b0 = pack_bf16(ST[mt][2 * kt][h], ST[mt][2 * kt][h + 1]);
                        const uint32_t b1 = pack_bf16(ST[mt][2 * kt + 1][h], ST[mt][2 * kt + 1][h + 1]);
                        mma16816(O[jt], qf[kt][0], qf[kt][1], qf[kt][2], qf[kt][3], b0, b1);
                    }
                }

                // hand-over between the two directions of this value slice
                const bool first_visit = dir == 0 ? (2 * m <= nb - 1) : (2 * m < nb - 1);
                const uint32_t part = part_t + (uint32_t)(((n * G::NWD + w) * (G::JT * 2)) * 32 + lane) * 4;
                if (first_visit) {
#pragma unroll
                    for (int jt = 0; jt < G::JT; ++jt) {
                        sts32(part + (2 * jt) * 128, pack_bf16(O[jt][0], O[jt][1]));
                        sts32(part + (2 * jt + 1) * 128, pack_bf16(O[jt][2], O[jt][3]));
                    }
                }
                named_bar(1 + w, 64);
                if (!first_visit) {
#pragma unroll
                    for (int jt = 0; jt < G::JT; ++jt) {
                        const float2 p0 = unpack_bf16(lds32(part + (2 * jt) * 128));
                        const float2 p1 = unpack_bf16(lds32(part + (2 * jt + 1) * 128));
                        const uint32_t o0 = pack_bf16(0.5f * (O[jt][0] + p0.x), 0.5f * (O[jt][1] + p0.y));
                        const uint32_t o1 = pack_bf16(0.5f * (O[jt][2] + p1.x), 0.5f * (O[jt][3] + p1.y));
                        sts32(v_t + sw_off<G::RBV>(rbase + g, jchunk0 + jt) + tig * 4, o0);
                        sts32(v_t + sw_off<G::RBV>(rbase + g + 8, jchunk0 + jt) + tig * 4, o1);
                    }
                }
            }

            // state update: S^T += v^T k~, then scale column i by the block decay e^{b_last,i}
#pragma unroll
            for (int ip = 0; ip < G::IT / 2; ++ip) {
                uint32_t kf[4];
                ldsm_x4_t(kt_t + sw_off<G::RBK>(rbase + (mi & 1) * 8 + l7, 2 * ip + (mi >> 1)), kf);
#pragma unroll
                for (int mt = 0; mt < G::MT; ++mt) {
                    mma16816(ST[mt][2 * ip], vf[2 * mt][0], vf[2 * mt + 1][0], vf[2 * mt][1], vf[2 * mt + 1][1], kf[0],
                             kf[1]);
                    mma16816(ST[mt][2 * ip + 1], vf[2 * mt][0], vf[2 * mt + 1][0], vf[2 * mt][1], vf[2 * mt + 1][1],
                             kf[2], kf[3]);
                }
            }
#pragma unroll
            for (int it = 0; it < G::IT; ++it) {
                const float2 d = *reinterpret_cast<const float2*>(dfac + n * G::DKP + it * 8 + 2 * tig);
#pragma unroll
                for (int mt = 0; mt < G::MT; ++mt) {
                    ST[mt][it][0] *= d.x; ST[mt][it][1] *= d.y; ST[mt][it][2] *= d.x; ST[mt][it][3] *= d.y;
                }
                if (MODE == kSummary) { dprod[it][0] *= d.x; dprod[it][1] *= d.y; }
            }
        }

        if (MODE == kSummary) {
            float* so = args.ws_state + st_off;
#pragma unroll
            for (int mt = 0; mt < G::MT; ++mt)
#pragma unroll
                for (int it = 0; it < G::IT; ++it) {
                    const int j = w * G::JW + mt * 16 + g, i = it * 8 + 2 * tig;
                    *reinterpret_cast<float2*>(so + (size_t)j * G::DKP + i) = make_float2(ST[mt][it][0], ST[mt][it][1]);
                    *reinterpret_cast<float2*>(so + (size_t)(j + 8) * G::DKP + i) =
                        make_float2(ST[mt][it][2], ST[mt][it][3]);
                }
            if (w == 0 && g == 0) {
                float* dd = args.ws_decay + (((size_t)unit * args.nseg + seg) * 2 + dir) * G::DKP;
#pragma unroll
                for (int it = 0; it < G::IT; ++it)
                    *reinterpret_cast<float2*>(dd + it * 8 + 2 * tig) = make_float2(dprod[it][0], dprod[it][1]);
            }
        }
    }

    // ---- phase 3: one TMA store of the finished tile (rows >= L and columns >= dv are clipped) ----
    if (MODE == kMain) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncthreads();
        if (tid == 0) {
            tma_store_3d(&tm_o, 0, row0, unit, base + sp.v);
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        }
    }
}

// Sequential fold of the segment summaries of one unit and direction, in place:
// slot m ends up holding the state that enters segment m (forward: from the left, backward: from the right).
__global__ void bigla_fold_kernel(float* ws_state, const float* ws_decay, const int* ws_flags, int nseg, int dv,
                                  int dkp) {
    const int unit = blockIdx.x, dir = blockIdx.y;
    if (ws_flags[unit] != 0) return;
    const int n = dv * dkp;
    for (int x = threadIdx.x; x < n; x += blockDim.x) {
        const int i = x % dkp;
        float carry = 0.f;
        for (int mm = 0; mm < nseg; ++mm) {
            const int m = dir == 0 ? mm : nseg - 1 - mm;
            const size_t slot = ((size_t)unit * nseg + m) * 2 + dir;
            float* s = ws_state + slot * n + x;
            const float u = *s, d = ws_decay[slot * dkp + i];
            *s = carry;
            carry = fmaf(carry, d, u);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------------
struct Plan {
    int nseg, box_blocks;
};
Plan make_plan(int L) {
    Plan p;
    const int nb = (L + kBlk - 1) / kBlk;
    if (nb <= kMaxSegBlocks) { p.nseg = 1; p.box_blocks = nb; }
    else { p.box_blocks = kLongSegBlocks; p.nseg = (nb + kLongSegBlocks - 1) / kLongSegBlocks; }
    return p;
}

struct WsLayout {
    size_t state, decay, flags, total;
};
WsLayout ws_layout(long long units, int nseg, int dv, int dkp) {
    WsLayout w;
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    w.state = 0;
    w.decay = up((size_t)units * nseg * 2 * dv * dkp * 4);
    w.flags = w.decay + up((size_t)units * nseg * 2 * dkp * 4);
    w.total = w.flags + up((size_t)units * 4);
    return w;
}

template <int DK, int DV>
cudaError_t launch_t(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v, const __nv_bfloat16* la_f,
                     const __nv_bfloat16* la_b, __nv_bfloat16* out, long long units, int L, void* ws,
                     cudaStream_t stream) {
    using G = Geo<DK, DV>;
    const Plan pl = make_plan(L);
    const int rows = pl.box_blocks * kBlk;
    CUtensorMap tq, tk, tf, tb, tv, to;
    if (!make_map(&tq, q, units, L, DK, G::DKP, rows) || !make_map(&tk, k, units, L, DK, G::DKP, rows) ||
        !make_map(&tf, la_f, units, L, DK, G::DKP, rows) || !make_map(&tb, la_b, units, L, DK, G::DKP, rows) ||
        !make_map(&tv, v, units, L, DV, G::DVP, rows) || !make_map(&to, out, units, L, DV, G::DVP, rows))
        return cudaErrorInvalidValue;

    KernelArgs a{};
    a.q = q; a.k = k; a.v = v; a.la_f = la_f; a.la_b = la_b; a.out = out;
    a.L = L; a.nseg = pl.nseg; a.box_blocks = pl.box_blocks;
    a.dev_status = device_status_ptr();
    if (!a.dev_status) return cudaErrorUnknown;

    const SmemPlan sp = smem_plan<DK, DV>(pl.box_blocks);
    size_t smem = sp.total + 1024;   // slack for the manual 1 KB alignment
    const size_t rec = (size_t)rec_plan(G::NT, DK, DV).smem_floats * 4 + 1024;
    if (smem < rec) smem = rec;
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(bigla_mma_kernel<DK, DV, kMain>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  (int)smem)) != cudaSuccess)
        return e;
    const unsigned grid = (unsigned)(units * pl.nseg);
    if (pl.nseg > 1) {
        const WsLayout wl = ws_layout(units, pl.nseg, DV, G::DKP);
        char* w8 = static_cast<char*>(ws);
        a.ws_state = reinterpret_cast<float*>(w8 + wl.state);
        a.ws_decay = reinterpret_cast<float*>(w8 + wl.decay);
        a.ws_flags = reinterpret_cast<int*>(w8 + wl.flags);
        if ((e = cudaMemsetAsync(a.ws_flags, 0, (size_t)units * 4, stream)) != cudaSuccess) return e;
        if ((e = cudaFuncSetAttribute(bigla_mma_kernel<DK, DV, kSummary>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)smem)) != cudaSuccess)
            return e;
        bigla_mma_kernel<DK, DV, kSummary><<<grid, G::NT, smem, stream>>>(tq, tk, tf, tb, tv, to, a);
        bigla_fold_kernel<<<dim3((unsigned)units, 2), 256, 0, stream>>>(a.ws_state, a.ws_decay, a.ws_flags, pl.nseg, DV,
                                                                        G::DKP);
        count_launch(2);
    }
    bigla_mma_kernel<DK, DV, kMain><<<grid, G::NT, smem, stream>>>(tq, tk, tf, tb, tv, to, a);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

bool mma_supported(int dk, int dv) {
    return (dk == 16 || dk == 24 || dk == 32) && (dv == 32 || dv == 48 || dv == 64);
}

size_t mma_workspace_bytes(long long units, int L, int dk, int dv) {
    const Plan pl = make_plan(L);
    if (pl.nseg == 1) return 0;
    if (kernel_preference() != VIG_KERNEL_MMA_SYNC) return umma_long_workspace_bytes(units, L, dk, dv);
    return ws_layout(units, pl.nseg, dv, (dk + 15) / 16 * 16).total;
}

cudaError_t launch_bigla_mma(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                             const __nv_bfloat16* la_f, const __nv_bfloat16* la_b, __nv_bfloat16* out, long long units,
                             int L, int dk, int dv, void* ws, cudaStream_t stream) {
    if (kernel_preference() != VIG_KERNEL_MMA_SYNC) {
        if (umma_supported(dk, dv, L)) return launch_bigla_umma(q, k, v, la_f, la_b, out, units, L, dk, dv, stream);
        return launch_bigla_umma_long(q, k, v, la_f, la_b, out, units, L, dk, dv, ws, stream);
    }
#define VIG_CASE(DK_, DV_) \
    if (dk == DK_ && dv == DV_) return launch_t<DK_, DV_>(q, k, v, la_f, la_b, out, units, L, ws, stream);
    VIG_CASE(16, 32) VIG_CASE(16, 48) VIG_CASE(16, 64)
    VIG_CASE(24, 32) VIG_CASE(24, 48) VIG_CASE(24, 64)
    VIG_CASE(32, 32) VIG_CASE(32, 48) VIG_CASE(32, 64)
#undef VIG_CASE
    return cudaErrorNotSupported;
}

}  // namespace vig
