// bf16 BiGLA forward for sequences longer than one thread block holds, on tcgen05 / TMEM.
//
// The sequence of every (batch, head) unit is cut into chunks of 128 tokens; a task is one chunk, and the
// running states of Eq. 6 that cross chunk boundaries travel through scratch memory in three launches:
//   1. summary: per chunk, the state a zero input would leave behind, U> = diag(e^{b_last}) (k~>)^T v and
//      U< = (k~<)^T v, and the chunk's decay d> = e^{b_last}, d< = e^{x_last}
//      (b: inclusive prefix sums of log alpha> inside the chunk, x: exclusive prefix sums of log alpha< - its tile
//      is loaded one row low, so chunk m's sums start with the gate of the token before it, the step across the
//      chunk boundary -, k~> = k e^{-b}, k~< = k e^{x}, as in the single-block kernel);
//   2. fold: S>_in(m + 1) = d>(m) S>_in(m) + U>(m) from the left; from the right R(m) = U<(m) + d<(m) R(m + 1) and
//      S<_in(m) = d<(m) R(m + 1) (q~< = q e^{-x} lacks the chunk's own decay), in fp32; every incoming state is
//      written out as the bf16 shared-memory image the next launch copies in with one bulk copy;
//   3. main: per chunk, out = ( P v + q~> S>_in + q~< S<_in ) / 2 with P = tril(q~> k~>^T) + triu(q~< k~<^T).
// Blocks are persistent (four per SM, 128 threads, 128 TMEM columns each) and walk over the tasks; thread r
// owns token r of the chunk in every element-wise phase.  All products are tcgen05.mma with M = 128.
#include <cuda.h>

#include <atomic>

#include "recurrence.cuh"
#include "tma_host.h"
#include "umma.cuh"
#include "vig_internal.h"

namespace vig {
namespace {

using namespace umma;

constexpr int kLThreads = 128;
constexpr uint32_t kLTmemCols = 128;
constexpr int kLBlocksPerSm = 4;          // main launch: blocks per SM (shared memory, registers and TMEM: 4 x 128 columns)
constexpr int kLSummaryBlocksPerSm = 4;   // summary launch (shared memory and TMEM: 4 x 128 columns)
constexpr int kMaxDevices = 64;
enum LongMode { kLMain = 0, kLSummary = 1 };

// ---- scratch ---------------------------------------------------------------------------------------------
// slot(unit, chunk, dir): 32 x DV fp32 (summary, key dim major);  image(unit, chunk, dir): the incoming state as a 4 KB
// bf16 tile [32][64] (128-byte rows, 128B swizzle), written by the fold;  decay(unit, chunk, dir): 32 fp32;
// flags(unit), chunk flags(unit, chunk): int.
// Every word is written before it is read within one call: nothing has to be cleared beforehand.
struct LongWs {
    size_t slot_bytes, img_off, decay_off, flags_off, cflags_off, total;
};
constexpr size_t kImgBytes = 4096;
LongWs long_ws_layout(long long units, int nch, int dv) {
    LongWs w;
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    w.slot_bytes = (size_t)32 * dv * 4;
    w.img_off = up((size_t)units * nch * 2 * w.slot_bytes);
    w.decay_off = w.img_off + up((size_t)units * nch * 2 * kImgBytes);
    w.flags_off = w.decay_off + up((size_t)units * nch * 2 * 32 * 4);
    w.cflags_off = w.flags_off + up((size_t)units * 4);
    w.total = w.cflags_off + up((size_t)units * nch * 4);
    return w;
}

// ---- shared memory -------------------------------------------------------------------------------------------
// Main mode holds four q-type tiles [128][32] bf16 (64B swizzle; loaded: q, k, log alpha>, log alpha<; scaled in
// place: k~<, k~>, q~>, q~<), the v tile (later the output tile) and the 0/1 tile; the two incoming states (4 KB
// each) land on the first 64 rows of the k~> and k~< tiles once the first score batch, their last reader, is done.
// Summary mode needs neither q nor states and writes k~< over the log alpha> tile once the prefix sums are taken,
// which keeps a block below a quarter of an SM's shared memory.
template <int MODE>
struct LLayout {
    static constexpr uint32_t tile = 128 * 64;
    static constexpr uint32_t k = MODE == kLMain ? tile : 0;             // k, then k~>
    static constexpr uint32_t f = k + tile;                               // log alpha>, then q~> (main) / k~< (summary)
    static constexpr uint32_t b = f + tile;                               // log alpha<, then q~< (main)
    static constexpr uint32_t q = 0;                                      // main only: q, then k~<
    static constexpr uint32_t kb = MODE == kLMain ? q : f;                // where k~< lives
    static constexpr uint32_t v = b + tile;                               // v tile [128][64] bf16 (128B swizzle)
    static constexpr uint32_t zf = v + 128 * 128;
    static constexpr uint32_t s_fwd = k;                                  // main only: incoming states, bf16 [32][64], 128B swizzle,
    static constexpr uint32_t s_bwd = q;                                  //   over rows 0..63 of k~> / k~< after the first score batch
    static constexpr uint32_t misc = zf + kZBytes;                        // mbarriers, TMEM slot, flags, totals
    static constexpr uint32_t total = misc + 64 + 256;
};

struct LArgs {
    const __nv_bfloat16 *q, *k, *v, *la_f, *la_b;
    __nv_bfloat16* out;
    int L, nch;
    long long tasks;
    uint8_t* ws_slots;    // [units][nch][2][slot_bytes]
    uint8_t* ws_img;      // [units][nch][2][4096]
    float* ws_decay;      // [units][nch][2][32]
    int* ws_flags;        // [units]: the unit needs the exact recurrence (written by the fold launch)
    int* ws_cflags;       // [units][nch]: per-chunk range check of the summary launch
    uint32_t slot_bytes;
    int* dev_status;
};

__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

template <int DK, int DV, int MODE>
__global__ void __launch_bounds__(kLThreads, MODE == kLSummary ? kLSummaryBlocksPerSm : kLBlocksPerSm)
bigla_long_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_f, const __grid_constant__ CUtensorMap tm_b,
                  const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o, const LArgs args) {
    static_assert((DK == 16 || DK == 24 || DK == 32) && (DV == 32 || DV == 48 || DV == 64), "unsupported head size");
    extern __shared__ __align__(1024) uint8_t smem_raw[];   // the swizzled tiles need the 1 KB alignment; no slack is allocated
    const uint32_t base = smem_u32(smem_raw);
    uint8_t* bp = smem_raw;
    using Y = LLayout<MODE>;
    if ((base & 1023u) != 0) {   // never expected: reported instead of computing on misplaced tiles
        if (threadIdx.x == 0) atomicOr(args.dev_status, kDevStatusInternal);
        return;
    }

    // warp index through a shuffle: uniform for the compiler, so MMA operands derived from it stay in uniform registers
    const int tid = threadIdx.x, lane = tid & 31, wq = __shfl_sync(0xffffffffu, tid >> 5, 0);
    const int L = args.L, nch = args.nch;
    // Warp 1 (not a range-check warp) issues the loads, the stores and the MMA batches, each through one elected thread
    // (always the same one: it owns the bulk-copy groups of the stores); its bookkeeping is warp-uniform.
    const bool ctl_warp = wq == 1;
    // mbarriers: log gates landed, q / k landed, v landed, incoming states landed, MMA batch done
    const uint32_t bar_g = base + Y::misc, bar_qk = bar_g + 8, bar_v = bar_g + 16, bar_s = bar_g + 24, bar_mma = bar_g + 32;
    const uint32_t slot = bar_g + 40;
    volatile uint32_t* slot_p = reinterpret_cast<volatile uint32_t*>(bp + Y::misc + 40);
    volatile int* time_flag = reinterpret_cast<volatile int*>(bp + Y::misc + 44);
    volatile int* slow_slot = reinterpret_cast<volatile int*>(bp + Y::misc + 48);   // range check of the chunk (summary mode)
    float* totals = reinterpret_cast<float*>(bp + Y::misc + 64);   // [2][32] chunk totals of the log gates: b and x at the last row
    uint32_t mma_phase = 0;

    const uint32_t t_kb = base + Y::kb, t_kf = base + Y::k, t_qf = base + Y::f, t_qb = base + Y::b, t_q = base + Y::q;
    const uint32_t t_v = base + Y::v;

    auto task_unit = [&](long long t) { return (int)(t / nch); };
    auto task_chunk = [&](long long t) { return (int)(t % nch); };
    auto load_operands = [&](long long t) {   // everything but v
        const int u = task_unit(t), r0 = task_chunk(t) * kChunk;
        mbar_expect_tx(bar_g, 2 * Y::tile);
        tma_load_3d(t_qf, &tm_f, 0, r0, u, bar_g);
        tma_load_3d(t_qb, &tm_b, 0, r0 - 1, u, bar_g);   // one row low (row -1 of the unit: the zero fill)
        if (MODE == kLMain) {
            mbar_expect_tx(bar_qk, 2 * Y::tile);
            tma_load_3d(t_q, &tm_q, 0, r0, u, bar_qk);
            tma_load_3d(t_kf, &tm_k, 0, r0, u, bar_qk);
        } else {
            mbar_expect_tx(bar_qk, Y::tile);
            tma_load_3d(t_kf, &tm_k, 0, r0, u, bar_qk);
        }
    };
    auto load_states = [&](long long t) {
        const uint8_t* im = args.ws_img + (size_t)t * 2 * kImgBytes;
        mbar_expect_tx(bar_s, 2 * 4096);
        bulk_load_1d(base + Y::s_fwd, im, 4096, bar_s);
        bulk_load_1d(base + Y::s_bwd, im + kImgBytes, 4096, bar_s);
    };
    auto load_v = [&](long long t) {
        mbar_expect_tx(bar_v, 128 * 128);
        tma_load_3d(t_v, &tm_v, 0, task_chunk(t) * kChunk, task_unit(t), bar_v);
    };

    pdl_launch_dependents();   // the next kernel's set-up may overlap this grid
    if (wq == 2 && blockIdx.x < args.tasks && elect_one()) {
        // Warm L2 with this block's first task while the kernel before this one in the stream still runs: a prefetch
        // consumes nothing, and L2 stays coherent with whatever that kernel is still writing.  The main launch only
        // asks for q: the summary launch has just read the other tiles, and every prefetch queues in front of the
        // loads proper in the TMA unit.
        const int pu = (int)(blockIdx.x / nch), pr = (int)(blockIdx.x % nch) * kChunk;
        if (MODE == kLMain) {
            tma_prefetch_3d(&tm_q, 0, pr, pu);
        } else {
            tma_prefetch_3d(&tm_k, 0, pr, pu);
            tma_prefetch_3d(&tm_v, 0, pr, pu);
            tma_prefetch_3d(&tm_f, 0, pr, pu);
            tma_prefetch_3d(&tm_b, 0, pr, pu);
        }
    }
    if (tid == 0) {
#pragma unroll
        for (int i = 0; i < 5; ++i) mbar_init(bar_g + 8 * i, 1);
        *time_flag = 0;
        slow_slot[0] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (wq == 0) {
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"(kLTmemCols));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    // the 240 rows of the 0/1 tile, two passes of 128 threads
    build_zero_one_tile(bp + Y::zf, tid);
    build_zero_one_tile(bp + Y::zf, tid + kLThreads);
    if (tid < 64) totals[tid] = 0.f;   // key dims a narrow head never writes
    pdl_wait();   // nothing above touches global memory: it may run while the previous kernel in the stream drains
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *slot_p;
    const uint32_t rc = tmem + ((uint32_t)(wq * 32) << 16);   // this thread's TMEM lane

    auto wait_bar = [&](uint32_t bar, uint32_t parity) {
        if (!mbar_wait_bounded(bar, parity)) *time_flag = 1;
    };
    auto wait_mma = [&]() {
        wait_bar(bar_mma, mma_phase & 1);
        ++mma_phase;
        tc_fence_after();
    };
    auto handover = [&]() {
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    };

    if (ctl_warp && blockIdx.x < args.tasks && elect_one()) {
        load_operands(blockIdx.x);
        load_v(blockIdx.x);
    }

    uint32_t it = 0;
    bool v_load_pending = false;   // control warp (uniform in it): the v tile of the current task has not been requested yet
    for (long long task = blockIdx.x; task < args.tasks; task += gridDim.x, ++it) {
        const uint32_t par = it & 1;
        const int unit = task_unit(task), m = task_chunk(task);
        const long long next = task + gridDim.x;
        const bool has_next = next < args.tasks;
        const int rows_here = min(kChunk, L - m * kChunk);
        const int ks = (rows_here + 15) >> 4, nkeys = ks * 16;
        const int row = wq * 32 + lane;
        const bool warp_live = wq * 32 < rows_here, row_live = row < rows_here;
        // a unit whose gates left the factorised range (found by the summary launch) is redone by the recurrence
        const bool unit_slow = MODE == kLMain && args.ws_flags[unit] != 0;

        // ---- prefix sums of both log-gate tiles (side by side along N) -> TMEM columns [0,32) / [32,64) ----------
        if (wq == 1 && elect_one()) {
            wait_bar(bar_g, par);
            constexpr uint32_t kIdS = instr_desc(128, 64, 0, 1);
            const uint32_t zf = desc_lo(base + Y::zf, 128);
            const uint32_t g = desc_lo(t_qf, Y::tile);   // second N block: the log alpha< tile
#pragma unroll 1   // issue loops stay rolled: less code for the instruction cache
            for (int j = 0; j < ks; ++j) {
                const uint32_t win = (uint32_t)(14 - 2 * j) * 16;   // window start row 112 - 16 j
                umma_ss(tmem + 0, desc64(zf + win, kHiZ), desc64(g + j * 64, kHiK64), kIdS, j > 0);
            }
            umma_commit(bar_mma);
        }
        wait_mma();
        wait_bar(bar_qk, par);

        // ---- scaled operands, in place: every thread rewrites its own row -----------------------------------------
        if (warp_live) {
            constexpr int kHalves = (DK + 15) / 16;
            const bool check_row = row == rows_here - 1;
#pragma unroll
            for (int hf = 0; hf < kHalves; ++hf) {
                uint32_t pf[16], pb[16];
                tmem_ld16(rc + 16 * hf, pf);
                tmem_ld16(rc + 32 + 16 * hf, pb);
                tc_wait_ld();
                if (check_row) {
                    // totals of the log gates over the chunk, b and x at its last row (range check after the hand-over,
                    // decay of the summary)
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        reinterpret_cast<uint4*>(totals + 16 * hf)[x] = make_uint4(pf[4 * x], pf[4 * x + 1], pf[4 * x + 2], pf[4 * x + 3]);
                        reinterpret_cast<uint4*>(totals + 32 + 16 * hf)[x] = make_uint4(pb[4 * x], pb[4 * x + 1], pb[4 * x + 2], pb[4 * x + 3]);
                    }
                }
                if (row_live) {
#pragma unroll
                    for (int c8 = 0; c8 < 2; ++c8) {
                        const int ch = 2 * hf + c8;   // 16-byte chunk of the row: key dims 8 ch .. 8 ch + 7
                        if (ch >= DK / 8) break;
                        const uint32_t off = sw_off<64>(row, ch);
                        const uint4 kv4 = *reinterpret_cast<const uint4*>(bp + Y::k + off);
                        const uint32_t kv[4] = {kv4.x, kv4.y, kv4.z, kv4.w};
                        uint32_t kf[4], kb[4];
                        if (MODE == kLMain) {
                            const uint4 qv4 = *reinterpret_cast<const uint4*>(bp + Y::q + off);
                            const uint32_t qv[4] = {qv4.x, qv4.y, qv4.z, qv4.w};
                            uint32_t qf[4], qb[4];
#pragma unroll
                            for (int mm = 0; mm < 4; ++mm) {
                                // the decaying factors on the special-function unit, the growing ones as their packed reciprocals
                                const int d0 = 8 * c8 + 2 * mm;
                                const float ex0 = ex2(as_f(pf[d0]) * kLog2e), ex1 = ex2(as_f(pf[d0 + 1]) * kLog2e);
                                const float ey0 = ex2(as_f(pb[d0]) * kLog2e), ey1 = ex2(as_f(pb[d0 + 1]) * kLog2e);
                                const uint32_t exp_f = pack_bf16(ex0, ex1), exp_b = pack_bf16(ey0, ey1);
                                qf[mm] = mul_bf16x2(qv[mm], exp_f);               // q~> = q e^{b}
                                kf[mm] = mul_bf16x2(kv[mm], rcp_bf16x2(exp_f));   // k~> = k e^{-b}
                                qb[mm] = mul_bf16x2(qv[mm], rcp_bf16x2(exp_b));   // q~< = q e^{-x}
                                kb[mm] = mul_bf16x2(kv[mm], exp_b);               // k~< = k e^{x}
                            }
                            *reinterpret_cast<uint4*>(bp + Y::f + off) = make_uint4(qf[0], qf[1], qf[2], qf[3]);
                            *reinterpret_cast<uint4*>(bp + Y::b + off) = make_uint4(qb[0], qb[1], qb[2], qb[3]);
                        } else {
#pragma unroll
                            for (int mm = 0; mm < 4; ++mm) {
                                const int d0 = 8 * c8 + 2 * mm;
                                kf[mm] = mul_bf16x2(kv[mm], pack_bf16(ex2(-as_f(pf[d0]) * kLog2e), ex2(-as_f(pf[d0 + 1]) * kLog2e)));
                                kb[mm] = mul_bf16x2(kv[mm], pack_bf16(ex2(as_f(pb[d0]) * kLog2e), ex2(as_f(pb[d0 + 1]) * kLog2e)));
                            }
                        }
                        *reinterpret_cast<uint4*>(bp + Y::k + off) = make_uint4(kf[0], kf[1], kf[2], kf[3]);
                        *reinterpret_cast<uint4*>(bp + Y::kb + off) = make_uint4(kb[0], kb[1], kb[2], kb[3]);
                    }
                }
            }
        }
        fence_async_smem();   // operand tiles were written through the generic proxy, the MMAs read them through the async proxy
        handover();
        if (wq == 2 && MODE == kLSummary) {
            // range check, one key dim per lane: b and x are smallest at the last row of the chunk
            const bool out_of_range = totals[lane] < -kGateRange || totals[32 + lane] < -kGateRange;
            const bool any = __any_sync(0xffffffffu, out_of_range);
            if (lane == 0) slow_slot[0] = any ? 1 : 0;
        }
        if (ctl_warp && v_load_pending) {
            // the store of the previous task has read the v tile by now; the tile is needed again only further down
            if (elect_one()) {
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                load_v(task);
            }
            v_load_pending = false;
        }

        if constexpr (MODE == kLSummary) {
            // ---- U = [k~> | k~<]^T v -> TMEM columns [64,128); rows 0..31: forward, rows 32..63: backward ----------
            if (wq == 1 && elect_one()) {
                wait_bar(bar_v, par);
                constexpr uint32_t kIdU = instr_desc(128, 64, 1, 1);
                const uint32_t ak = desc_lo(t_kf, Y::tile), bv = desc_lo(t_v, 16);   // M blocks: k~>, k~< (then two tiles of no interest)
#pragma unroll 1
                for (int kk = 0; kk < ks; ++kk) umma_ss(tmem + 64, desc64(ak + kk * 64, kHiK64), desc64(bv + kk * 128, kHiV128), kIdU, kk > 0);
                umma_commit(bar_mma);
            }
            wait_mma();
            if (ctl_warp && has_next) {   // the summary batch was the last reader of every tile
                // (the flag is read into one value for the whole warp first: elect.sync needs all of it)
                const bool go = __all_sync(0xffffffffu, *time_flag == 0);
                if (go && elect_one()) {
                    load_operands(next);
                    load_v(next);
                }
            }
            if (wq < 2) {
                // lane = key dim; warp 0: forward summary, warp 1: backward summary
                const int dir = wq;
                const float d = ex2(totals[(dir == 0 ? 0 : 32) + lane] * kLog2e);   // decay of the whole chunk for this key dim
                const float us = dir == 0 ? d : 1.f;   // the forward summary carries the chunk's decay, the backward one does not
                float* dst = reinterpret_cast<float*>(args.ws_slots + ((size_t)task * 2 + dir) * args.slot_bytes) + (size_t)lane * DV;
#pragma unroll
                for (int hb = 0; hb < 2; ++hb) {
                    if (hb * 32 >= DV) break;
                    uint32_t r[32];
                    tmem_ld32(rc + 64 + hb * 32, r);
                    tc_wait_ld();
#pragma unroll
                    for (int x = 0; x < 8; ++x) {
                        if (hb * 32 + 4 * x < DV)
                            reinterpret_cast<float4*>(dst + hb * 32)[x] =
                                make_float4(as_f(r[4 * x]) * us, as_f(r[4 * x + 1]) * us, as_f(r[4 * x + 2]) * us, as_f(r[4 * x + 3]) * us);
                    }
                }
                args.ws_decay[((size_t)task * 2 + dir) * 32 + lane] = d;
            }
            handover();
            if (tid == 0) args.ws_cflags[task] = slow_slot[0];
            if (*time_flag != 0) break;
        } else {
        // ---- main mode ---------------------------------------------------------------------------------------------
        // P, key columns [64 p, 64 p + 64): forward scores -> columns [0,64), backward -> [64,128)
        uint32_t hold[32];   // packed bf16 P of this row, key columns 0..63
#pragma unroll
        for (int p = 0; p < 2; ++p) {
            const int n = min(nkeys - 64 * p, 64);
            if (n <= 0) break;
            if (wq == 1 && elect_one()) {
                const uint32_t idp = instr_desc(128, n, 0, 0);
                const uint32_t aqf = desc_lo(t_qf, 16), aqb = desc_lo(t_qb, 16), bkf = desc_lo(t_kf, 16), bkb = desc_lo(t_kb, 16);
#pragma unroll
                for (int kk = 0; kk < 2; ++kk) {
                    umma_ss(tmem + 0, desc64(aqf + kk * 2, kHiK64), desc64(bkf + p * 256 + kk * 2, kHiK64), idp, kk > 0);
                    umma_ss(tmem + 64, desc64(aqb + kk * 2, kHiK64), desc64(bkb + p * 256 + kk * 2, kHiK64), idp, kk > 0);
                }
                umma_commit(bar_mma);
            }
            wait_mma();
            if (p == 0 && ctl_warp && elect_one()) load_states(task);   // rows 0..63 of k~> and k~< have been read for the last time
            if (warp_live) {
                uint32_t pk[16];
                combine_any(2 * p, wq, true, rc, rc + 64, lane, 0u, pk);   // (no room for the mask table at four blocks per SM: selects)
                if (p == 0) {
#pragma unroll
                    for (int e = 0; e < 16; ++e) hold[e] = pk[e];
                } else {
                    // key block 2 has been read: columns [0,32) are dead and take the packed first half
                    uint32_t h0[16], h1[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) { h0[e] = hold[e]; h1[e] = hold[16 + e]; }
                    tmem_st16(rc, h0);
                    tmem_st16(rc + 16, h1);
#pragma unroll
                    for (int e = 0; e < 16; ++e) hold[e] = pk[e];
                }
                combine_any(2 * p + 1, wq, 64 * p + 32 < nkeys, rc + 32, rc + 96, lane, 0u, pk);   // (no room for the mask table at four blocks per SM: selects)
                if (p == 0) {
#pragma unroll
                    for (int e = 0; e < 16; ++e) hold[16 + e] = pk[e];
                    if (nkeys <= 64) {   // no second half
                        uint32_t h0[16];
#pragma unroll
                        for (int e = 0; e < 16; ++e) h0[e] = hold[e];
                        tmem_st16(rc, h0);
                        tmem_st16(rc + 16, pk);
                    }
                } else {
                    uint32_t h0[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) h0[e] = hold[e];
                    tmem_st16(rc + 32, h0);
                    tmem_st16(rc + 48, pk);
                }
            }
            tc_wait_st();
            handover();
        }

        // out = (q~> S>_in + q~< S<_in + P v) / 2
        if (wq == 1 && elect_one()) {
            wait_bar(bar_v, par);
            wait_bar(bar_s, par);
            constexpr uint32_t kIdO = instr_desc(128, 64, 0, 1);
            const uint32_t qf = desc_lo(t_qf, 16), qb = desc_lo(t_qb, 16);
            const uint32_t sf = desc_lo(base + Y::s_fwd, 16), sb = desc_lo(base + Y::s_bwd, 16), bv = desc_lo(t_v, 16);
#pragma unroll
            for (int kk = 0; kk < 2; ++kk) umma_ss(tmem + 64, desc64(qf + kk * 2, kHiK64), desc64(sf + kk * 128, kHiV128), kIdO, kk > 0);
#pragma unroll
            for (int kk = 0; kk < 2; ++kk) umma_ss(tmem + 64, desc64(qb + kk * 2, kHiK64), desc64(sb + kk * 128, kHiV128), kIdO, 1);
#pragma unroll 1
            for (int kk = 0; kk < ks; ++kk) umma_ts(tmem + 64, tmem + kk * 8, desc64(bv + kk * 128, kHiV128), kIdO, 1);
            umma_commit(bar_mma);
        }
        wait_mma();
        const bool next_early = has_next && !unit_slow;
        if (ctl_warp && next_early) {   // every MMA that reads the operand tiles is done
            const bool go = __all_sync(0xffffffffu, *time_flag == 0);
            if (go && elect_one()) load_operands(next);
        }
        if (warp_live) {
            // epilogue: out = O / 2, bf16, into the dead v tile (same swizzle as the TMA store expects)
#pragma unroll
            for (int hb = 0; hb < DV / 32; ++hb) {
                uint32_t r[32];
                tmem_ld32(rc + 64 + hb * 32, r);
                tc_wait_ld();
                if (row_live) {
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
                        uint32_t o[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) o[e] = mul_bf16x2(pack_bf16(as_f(r[ch * 8 + 2 * e]), as_f(r[ch * 8 + 2 * e + 1])), 0x3F003F00u);   // x 1/2 after packing: exact
                        *reinterpret_cast<uint4*>(bp + Y::v + sw_off<128>(row, hb * 4 + ch)) = make_uint4(o[0], o[1], o[2], o[3]);
                    }
                }
            }
            if (DV == 48) {
                uint32_t r[16];
                tmem_ld16(rc + 64 + 32, r);
                tc_wait_ld();
                if (row_live) {
#pragma unroll
                    for (int ch = 0; ch < 2; ++ch) {
                        uint32_t o[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) o[e] = mul_bf16x2(pack_bf16(as_f(r[ch * 8 + 2 * e]), as_f(r[ch * 8 + 2 * e + 1])), 0x3F003F00u);   // x 1/2 after packing: exact
                        *reinterpret_cast<uint4*>(bp + Y::v + sw_off<128>(row, 4 + ch)) = make_uint4(o[0], o[1], o[2], o[3]);
                    }
                }
            }
        }
        fence_async_smem();
        handover();
        if (*time_flag != 0) break;
        if (!unit_slow) {
            if (ctl_warp) {
                if (elect_one()) {
                    tma_store_3d(&tm_o, 0, m * kChunk, unit, t_v);   // rows >= L and columns >= dv are clipped
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    if (has_next && !next_early) load_operands(next);
                }
                v_load_pending = has_next;   // the v tile only once the store has read it
            }
        } else {
            // the first chunk's task redoes the whole unit by the recurrence (its scratch overlays the tiles, so the
            // next loads wait until it is done); the other chunks of the unit store nothing
            if (m == 0) {
                if (tid == 0) atomicAdd(args.dev_status + 1, 1);   // units handed to the recurrence (read by the tests)
                const size_t ok = (size_t)unit * L * DK, ov = (size_t)unit * L * DV;
                recurrence_unit<__nv_bfloat16>(args.q + ok, args.k + ok, args.v + ov, args.la_f + ok, args.la_b + ok,
                                               args.out + ov, L, DK, DV, reinterpret_cast<float*>(bp));
                fence_async_smem();
                __syncthreads();
            }
            if (ctl_warp && has_next && elect_one()) {
                load_operands(next);
                load_v(next);
            }
        }
        }   // main mode
    }

    if (ctl_warp && elect_one()) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the last store still reads shared memory
    tc_fence_before();
    __syncthreads();
    if (wq == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kLTmemCols));
    if (tid == 0 && *time_flag != 0) atomicOr(args.dev_status, kDevStatusTimeout);
}

// Sequential fold of the chunk summaries of one unit and direction, eight key dims per block.  Thread (i, c) owns
// the four value dims 4 c .. 4 c + 3 of key dim i and takes the chunks in batches of 32, whose loads are all in
// flight together; the incoming states go out as bf16 tile images.  Every block also reduces the chunks' range
// flags to the unit's flag.
constexpr int kFoldRows = 8;
template <int DV>
__global__ void __launch_bounds__(kFoldRows * (DV / 4))
bigla_long_fold_kernel(const uint8_t* ws_slots, uint8_t* ws_img, const float* ws_decay, int* ws_flags, const int* ws_cflags, int nch,
                       uint32_t slot_bytes) {
    constexpr int C4 = DV / 4;   // float4 columns of live value dims
    constexpr int kBatch = 32;
    const int unit = blockIdx.x, dir = blockIdx.y;
    const int i = blockIdx.z * kFoldRows + threadIdx.x / C4, c = threadIdx.x % C4;
    pdl_launch_dependents();
    pdl_wait();
    int flagged = 0;
    for (int m = threadIdx.x; m < nch; m += blockDim.x) flagged |= ws_cflags[(size_t)unit * nch + m];
    float4 carry = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int mb = 0; mb < nch; mb += kBatch) {
        float4 u[kBatch];
        float d[kBatch];
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
            if (mb + b < nch) {
                const int m = dir == 0 ? mb + b : nch - 1 - (mb + b);
                const size_t s = ((size_t)unit * nch + m) * 2 + dir;
                u[b] = *(reinterpret_cast<const float4*>(ws_slots + s * slot_bytes) + ((size_t)i * DV + 4 * c) / 4);
                d[b] = ws_decay[s * 32 + i];
            }
        }
        if (mb == 0) {   // the flags arrive under the latency of the first batch
            flagged = __syncthreads_or(flagged);
            if (dir == 0 && blockIdx.z == 0 && threadIdx.x == 0) ws_flags[unit] = flagged;
        }
        if (flagged) return;   // the main launch redoes the unit by the recurrence
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
            if (mb + b < nch) {
                const int m = dir == 0 ? mb + b : nch - 1 - (mb + b);
                uint8_t* img = ws_img + (((size_t)unit * nch + m) * 2 + dir) * kImgBytes + i * 128;
                // forward: the state entering chunk m is the carry; backward: the carry times the chunk's own decay
                if (dir == 1) { carry.x *= d[b]; carry.y *= d[b]; carry.z *= d[b]; carry.w *= d[b]; }
                *reinterpret_cast<uint2*>(img + (((c >> 1) ^ (i & 7)) << 4) + (c & 1) * 8) =
                    make_uint2(pack_bf16(carry.x, carry.y), pack_bf16(carry.z, carry.w));
                if (c < 16 - C4)   // value dims beyond dv read as zero
                    *reinterpret_cast<uint2*>(img + ((((C4 + c) >> 1) ^ (i & 7)) << 4) + ((C4 + c) & 1) * 8) = make_uint2(0u, 0u);
                if (dir == 0) {
                    carry.x = fmaf(carry.x, d[b], u[b].x); carry.y = fmaf(carry.y, d[b], u[b].y);
                    carry.z = fmaf(carry.z, d[b], u[b].z); carry.w = fmaf(carry.w, d[b], u[b].w);
                } else {
                    carry.x += u[b].x; carry.y += u[b].y; carry.z += u[b].z; carry.w += u[b].w;
                }
            }
        }
    }
}

template <int DK, int DV>
cudaError_t launch_long_t(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v, const __nv_bfloat16* la_f,
                          const __nv_bfloat16* la_b, __nv_bfloat16* out, long long units, int L, void* ws,
                          cudaStream_t stream) {
    const int nch = (L + kChunk - 1) / kChunk;
    CUtensorMap tq, tk, tf, tb, tv, to;
    if (!make_map(&tq, q, units, L, DK, 32, kChunk) || !make_map(&tk, k, units, L, DK, 32, kChunk) ||
        !make_map(&tf, la_f, units, L, DK, 32, kChunk) || !make_map(&tb, la_b, units, L, DK, 32, kChunk) ||
        !make_map(&tv, v, units, L, DV, 64, kChunk) || !make_map(&to, out, units, L, DV, 64, kChunk))
        return cudaErrorInvalidValue;
    const LongWs wl = long_ws_layout(units, nch, DV);
    LArgs a{};
    a.q = q; a.k = k; a.v = v; a.la_f = la_f; a.la_b = la_b; a.out = out;
    a.L = L; a.nch = nch; a.tasks = units * nch;
    a.ws_slots = static_cast<uint8_t*>(ws);
    a.ws_img = static_cast<uint8_t*>(ws) + wl.img_off;
    a.ws_decay = reinterpret_cast<float*>(static_cast<uint8_t*>(ws) + wl.decay_off);
    a.ws_flags = reinterpret_cast<int*>(static_cast<uint8_t*>(ws) + wl.flags_off);
    a.ws_cflags = reinterpret_cast<int*>(static_cast<uint8_t*>(ws) + wl.cflags_off);
    a.slot_bytes = (uint32_t)wl.slot_bytes;
    a.dev_status = device_status_ptr();
    if (!a.dev_status) return cudaErrorUnknown;
    const size_t rec = (size_t)rec_plan(kLThreads, DK, DV).smem_floats * 4;   // scratch of the exact recurrence (main launch only)
    const size_t smem_sum = LLayout<kLSummary>::total;
    const size_t smem_main = LLayout<kLMain>::total > rec ? LLayout<kLMain>::total : rec;
    // once per device: shared-memory opt-in of the two kernels and the SM count
    static std::atomic<int> sms_of[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    int sms = sms_of[dev].load(std::memory_order_acquire);
    if (sms == 0) {
        cudaError_t e;
        if ((e = cudaFuncSetAttribute(bigla_long_kernel<DK, DV, kLSummary>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_sum)) != cudaSuccess) return e;
        if ((e = cudaFuncSetAttribute(bigla_long_kernel<DK, DV, kLMain>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_main)) != cudaSuccess) return e;
        if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        sms_of[dev].store(sms, std::memory_order_release);
    }
    // persistent blocks: block b takes tasks b, b + grid, ...
    const long long cap_sum = (long long)kLSummaryBlocksPerSm * sms, cap_main = (long long)kLBlocksPerSm * sms;
    const unsigned grid_sum = (unsigned)(a.tasks < cap_sum ? a.tasks : cap_sum), grid_main = (unsigned)(a.tasks < cap_main ? a.tasks : cap_main);
    cudaError_t le = launch_pdl(bigla_long_kernel<DK, DV, kLSummary>, dim3(grid_sum), dim3(kLThreads), smem_sum, stream, tq, tk, tf, tb, tv, to, a);
    if (le == cudaSuccess)
        le = launch_pdl(bigla_long_fold_kernel<DV>, dim3((unsigned)units, 2, 32 / kFoldRows), dim3(kFoldRows * (DV / 4)), 0, stream,
                        (const uint8_t*)a.ws_slots, a.ws_img, (const float*)a.ws_decay, a.ws_flags, (const int*)a.ws_cflags, nch, a.slot_bytes);
    if (le == cudaSuccess)
        le = launch_pdl(bigla_long_kernel<DK, DV, kLMain>, dim3(grid_main), dim3(kLThreads), smem_main, stream, tq, tk, tf, tb, tv, to, a);
    if (le != cudaSuccess) return le;
    count_launch(3);
    return cudaGetLastError();
}

}  // namespace

size_t umma_long_workspace_bytes(long long units, int L, int dk, int dv) {
    (void)dk;
    return long_ws_layout(units, (L + kChunk - 1) / kChunk, dv).total;
}

cudaError_t launch_bigla_umma_long(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                                   const __nv_bfloat16* la_f, const __nv_bfloat16* la_b, __nv_bfloat16* out, long long units,
                                   int L, int dk, int dv, void* ws, cudaStream_t stream) {
#define VIG_CASE(DK_, DV_) \
    if (dk == DK_ && dv == DV_) return launch_long_t<DK_, DV_>(q, k, v, la_f, la_b, out, units, L, ws, stream);
    VIG_CASE(16, 32) VIG_CASE(16, 48) VIG_CASE(16, 64)
    VIG_CASE(24, 32) VIG_CASE(24, 48) VIG_CASE(24, 64)
    VIG_CASE(32, 32) VIG_CASE(32, 48) VIG_CASE(32, 64)
#undef VIG_CASE
    return cudaErrorNotSupported;
}

}  // namespace vig
