// bf16 BiGLA forward on the 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM).
//
// One thread block owns one (batch, head) unit of up to 256 tokens, split into chunks of C = 128
// rows; thread r of the block owns token r (TMEM lane r mod 128 of chunk r / 128) in every
// element-wise phase.  With b_t the inclusive prefix sum of log alpha> from the start of the chunk
// and x_t the exclusive prefix sum of log alpha< (the backward decay from t to s > t is
// exp(x_s - x_t): the gates t .. s-1), Eq. 6 becomes, per chunk,
//     [b | x] = T [la> | la< shifted down one row]   prefix sums as one product with a 0/1 triangular matrix
//     q~> = q e^{b},  k~> = k e^{-b},  q~< = q e^{-x},  k~< = k e^{x}
//     P    = tril(q~> k~>^T) + triu(q~< k~<^T)
//     U    = [k~< | k~>]^T v                          zero-input chunk summaries, both directions in one product
//     out  = ( P v + q~> S>_in + q~< S<_in ) / 2      S>_in = U>(left chunk) e^{b_last(left chunk)},
//                                                     S<_in = U<(right chunk) e^{x_last(this chunk)}
// The log alpha< tile is loaded one row low (tile row r holds the gate of token r - 1, row 0 the
// zero fill), so its inclusive prefix sum is x; chunk 1's sums then start with the gate of token 127,
// which is the step from chunk 0's last token into chunk 1 that the state hand-over needs.
// Every product is a tcgen05.mma with M = 128:
//   - the prefix sums: A = a 128-row window of a 240-row 0/1 tile ([zeros; lower triangle; ones],
//     shifted by 16 rows per K step), B = both log-gate tiles of both chunks side by side along N
//     (128 columns, one batch of eight MMAs); fp32 accumulation of bf16 values times 0/1 is exact
//     up to fp32 addition;
//   - P in two column halves (fwd and bwd side by side in TMEM, so the mask and the sum of the
//     diagonal block happen in fp32), packed to bf16 and written back to TMEM as the A operand of P v;
//   - U with A = the four operand tiles stacked along M (MN-major), q~ S with B = the bf16 state tile.
// The threads only do element-wise work on their own row: operand scaling in place, masking and
// packing P, scaling the chunk summaries, the output epilogue.  TMEM use is 256 columns (128 per
// chunk: P, then bf16 P + U / out; the prefix sums of both chunks in chunk 0's), shared memory about 108 KB at L = 196, so
// two blocks share an SM and one block's MMA round trips hide behind the other's element-wise phases.
// Blocks are persistent: block b walks over units b, b + grid, ...; the two chunks of a unit run as
// separate pipelines (own issuing thread, own mbarrier) that meet at the prefix batch and at the
// exchange of the chunk summaries; the operand tiles of the next unit are requested as soon as their
// last reader of the current unit is done, and its prefix batch is issued while this unit is stored.
#include <cuda.h>

#include <atomic>

#include "ptx.cuh"
#include "recurrence.cuh"
#include "tma_host.h"
#include "umma.cuh"
#include "vig_internal.h"

namespace vig {
namespace {

using namespace umma;

constexpr int kMaxRows = 256;   // longest unit this kernel takes
constexpr int kThreads = 256;
constexpr uint32_t kTmemCols = 256;
constexpr int kMaxDevices = 64;

// ---- shared-memory plan (rows = tokens of the unit rounded up to 16) ---------------------------
struct ULayout {
    uint32_t tile;     // pitch of one q-type tile [rows][32] bf16 (64-byte rows, 64B swizzle); four of them from offset 0:
                       //   as loaded: q, k, log alpha>, log alpha< (one row low);  after scaling: k~<, k~>, q~>, q~<.
                       //   Two chunks: the pitch is 256 rows, so that chunk 0 and chunk 1 of both gate tiles are
                       //   four blocks at one stride, the N blocks of the prefix-sum product.
    uint32_t v;        // v tile [rows][64] bf16 (128B swizzle), later the output tile
    uint32_t s_fwd;    // bf16 state entering chunk 1 from the left  [32][64] (128B swizzle)
    uint32_t s_bwd;    // bf16 state entering chunk 0 from the right  (segmented sequences keep their states elsewhere)
    uint32_t zf;       // 0/1 tile of the prefix sums
    uint32_t dec;      // [2 chunks][2][32] fp32 totals of the log gates: b and x at the chunk's last row
    uint32_t masks;    // 0 / 1 masks of the diagonal score block (kMaskBytes)
    uint32_t misc;     // six mbarriers, TMEM slot, flags
    uint32_t total;
};
__host__ __device__ inline ULayout make_layout(int rows, bool seg) {
    ULayout l;
    l.tile = rows > kChunk ? 2u * kChunk * 64u : (uint32_t)rows * 64u;
    l.v = 4 * l.tile;
    l.s_fwd = (l.v + (uint32_t)rows * 128 + 1023u) & ~1023u;
    l.s_bwd = l.s_fwd + (seg ? 0 : 32 * 128);
    l.zf = l.s_bwd + (seg ? 0 : 32 * 128);
    l.dec = l.zf + kZBytes;
    l.masks = l.dec + 4 * 32 * 4;
    l.misc = l.masks + kMaskBytes;
    l.total = l.misc + 128;
    return l;
}

struct UArgs {
    const __nv_bfloat16 *q, *k, *v, *la_f, *la_b;
    __nv_bfloat16* out;
    int L, rows;          // tokens per unit; rows of the TMA boxes (tokens of a block rounded up to 16)
    long long units;
    int* dev_status;
    // segmented sequences only (SEG): a unit is cut into nseg segments of 256 tokens, one block each
    int nseg;
    uint8_t* ws;                  // exchange slots, [units][nseg][kSlotBytes]
    unsigned long long nonce;     // marks the flags of this call
    // fused gate preparation only (GATES): la_f / la_b hold the gate logits g, and log alpha = logsigmoid(g) / tau
    float inv_tau;
    int expire_wait;   // test hook: every block lets one bounded wait, on an mbarrier nothing completes, run out
};

// log2 alpha = logsigmoid(g) / (tau ln 2) (Eq. 5 line 1, in base 2 so that the operand scaling needs no further
// multiplication) for the eight bf16 gate logits of one 16-byte piece, evaluated in fp32 as
// (min(g, 0) log2(e) - log2(1 + e)) / tau with e = e^{-|g|} in (0, 1] from the special-function unit and
// log2(1 + e) = e p(e), p of degree three (absolute error 1e-4, i.e. 7e-5 / tau in log alpha: below the bf16 rounding
// that follows), on the FMA pipe: with the logarithm on the special-function unit too, that unit bounds the phase.
__device__ __forceinline__ float log2_1p_unit(float e) {
    float p = -0.08476800471544266f;
    p = fmaf(p, e, 0.3255951702594757f);
    p = fmaf(p, e, -0.6799444556236267f);
    p = fmaf(p, e, 1.4390150308609009f);
    return p * e;
}
__device__ __forceinline__ uint4 log2_alpha_piece(uint4 g, float inv_tau) {
    const float c_lin = kLog2e * inv_tau;
    uint32_t w[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const float2 z = unpack_bf16(w[x]);
        const float l0 = log2_1p_unit(ex2(-fabsf(z.x) * kLog2e)), l1 = log2_1p_unit(ex2(-fabsf(z.y) * kLog2e));
        w[x] = pack_bf16(fmaf(l0, -inv_tau, fminf(z.x, 0.f) * c_lin), fmaf(l1, -inv_tau, fminf(z.y, 0.f) * c_lin));
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// ---- exchange slot of one (unit, segment) in scratch memory (segmented sequences) -------------------------
// flag (8 bytes): (nonce << 16) | (out-of-range bit << 15) | number of readers that are done with the slot;
// then, from byte 256: D>[32], d<[32] (decay of the whole segment per key dim and direction, fp32), from byte 512:
// E>[32][64] (the forward state a zero input leaves behind the segment) and R[32][64] (what the segment adds to
// the backward state at its first token), bf16: they only ever feed states that are rounded to bf16 operands.
constexpr size_t kSlotDecay = 256, kSlotFwd = 512, kSlotBwd = 512 + 32 * 64 * 2, kSlotBytes = 512 + 2 * 32 * 64 * 2;
constexpr int kMaxSegments = 32;

__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

template <int DK, int DV, bool SEG, bool GATES>
__global__ void __launch_bounds__(kThreads, 2)
bigla_umma_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_f, const __grid_constant__ CUtensorMap tm_b,
                  const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o, const UArgs args) {
    static_assert((DK == 16 || DK == 24 || DK == 32) && (DV == 32 || DV == 48 || DV == 64), "unsupported head size");
    static_assert(!(SEG && GATES), "fused gate preparation is built for the single-block form only");
    extern __shared__ __align__(1024) uint8_t smem_raw[];   // the swizzled tiles need the 1 KB alignment; no slack is allocated
    const uint32_t base = smem_u32(smem_raw);
    uint8_t* bp = smem_raw;
    if ((base & 1023u) != 0) {   // never expected: reported instead of computing on misplaced tiles
        if (threadIdx.x == 0) atomicOr(args.dev_status, kDevStatusInternal);
        return;
    }
    const ULayout lay = make_layout(args.rows, SEG);

    // The warp index goes through a shuffle so that the compiler knows it, and every address and descriptor derived
    // from it, to be uniform across the warp: the operands of tcgen05.mma then stay in uniform registers instead of
    // being moved there one by one before every MMA (measured: -1 us per call).
    constexpr float kExp = GATES ? 1.f : kLog2e;   // prefix sums of log alpha -> exponent of two
    const int tid = threadIdx.x, lane = tid & 31, warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
    const int c = warp >> 2, wq = warp & 3;            // chunk and row quadrant of this warp
    // Segmented sequences: block b works on segment b % nseg of the units of group b / nseg; the blocks of a group
    // take the same units in the same order and exchange their segment summaries through scratch memory.
    const int nseg = SEG ? args.nseg : 1;
    const int seg = SEG ? (int)(blockIdx.x % (unsigned)nseg) : 0;
    const int group = SEG ? (int)(blockIdx.x / (unsigned)nseg) : (int)blockIdx.x;
    const int ngroups = SEG ? (int)(gridDim.x / (unsigned)nseg) : (int)gridDim.x;
    const int r0 = seg * kMaxRows;                     // first token of this block's segment
    const int L = SEG ? min(args.L - r0, kMaxRows) : args.L;   // tokens this block holds
    const int nc = (L + kChunk - 1) / kChunk;
    const int row = c * kChunk + wq * 32 + lane;       // token owned by this thread
    const bool warp_live = c * kChunk + wq * 32 < L;   // the warp holds at least one token
    const bool row_live = row < L;
    const bool chunk_on = c < nc;
    // One warp per chunk (warps 1 and 5, away from the warps whose first / last rows carry the range checks) issues that
    // chunk's MMAs, through one elected thread per batch; warp 1 also drives the loads and stores the same way.
    const bool issue_warp = wq == 1;   // one elected thread of it issues a batch and commits it
    const bool ctl_warp = warp == 1;   // one elected thread of it drives the loads and stores; the bookkeeping is warp-uniform
    const int ks = chunk_on ? (min(L - c * kChunk, kChunk) + 15) >> 4 : 0;   // 16-token K steps of this chunk
    const int nkeys = ks * 16;
    // mbarriers: log-gate tiles landed, q and k landed, v landed, MMA batches of chunk 0 / chunk 1, prefix sums done
    const uint32_t bar_g = base + lay.misc, bar_qk = bar_g + 8, bar_v = bar_g + 16, bar_mma = bar_g + 24 + 8 * c;
    const uint32_t bar_pfx = bar_g + 40, slot = bar_g + 48;
    volatile uint32_t* slot_p = reinterpret_cast<volatile uint32_t*>(bp + lay.misc + 48);
    volatile int* time_flag = reinterpret_cast<volatile int*>(bp + lay.misc + 52);
    volatile int* early_gates = reinterpret_cast<volatile int*>(bp + lay.misc + 72);   // (unit counter + 1) whose next log gates went out early
    volatile int* unit_slow_slot = reinterpret_cast<volatile int*>(bp + lay.misc + 76);   // SEG: some segment of the unit left the gate range
    volatile int* slow_slot = reinterpret_cast<volatile int*>(bp + lay.misc + 56);   // [4]: range check per chunk (two used)
    const int ks_c1 = nc == 2 ? (L - kChunk + 15) >> 4 : 0;                          // K steps of chunk 1
    const int npass_c1 = ks_c1 > 4 ? 2 : 1;
    const int ks_c0 = (min(L, kChunk) + 15) >> 4;                                     // K steps of chunk 0
    float* dec = reinterpret_cast<float*>(bp + lay.dec);
    uint32_t mma_phase = 0;

    const uint32_t t_v = base + lay.v;
    const uint32_t g_bytes = (uint32_t)args.rows * 128, v_bytes = (uint32_t)args.rows * 128;
    // The four q-type tiles form two pairs that swap roles from one unit to the next: the pair that held (q, k) - its
    // last reader is the chunk-summary MMA - receives the next unit's log gates while this unit is still being
    // finished, and the pair that held the log gates (then q~>, q~<) receives the next (q, k).
    auto load_gates = [&](int unit, uint32_t pair) {
        mbar_expect_tx(bar_g, g_bytes);
        tma_load_3d(base + pair, &tm_f, 0, r0, unit, bar_g);
        tma_load_3d(base + pair + lay.tile, &tm_b, 0, r0 - 1, unit, bar_g);   // one row low: row 0 takes the token before the
                                                                              // segment (the zero fill in front of the unit)
    };
    auto load_qk = [&](int unit, uint32_t pair) {
        mbar_expect_tx(bar_qk, g_bytes);
        tma_load_3d(base + pair, &tm_q, 0, r0, unit, bar_qk);
        tma_load_3d(base + pair + lay.tile, &tm_k, 0, r0, unit, bar_qk);
    };
    auto load_v = [&](int unit) {
        mbar_expect_tx(bar_v, v_bytes);
        tma_load_3d(t_v, &tm_v, 0, r0, unit, bar_v);
    };

    pdl_launch_dependents();   // the next kernel's set-up may overlap this grid
    if (warp == 2 && elect_one()) {
        // Warm L2 with this block's first unit while the kernel before this one in the stream still runs: a prefetch
        // consumes nothing, and L2 stays coherent with whatever that kernel is still writing.
        tma_prefetch_3d(&tm_q, 0, r0, group);
        tma_prefetch_3d(&tm_k, 0, r0, group);
        tma_prefetch_3d(&tm_v, 0, r0, group);
        tma_prefetch_3d(&tm_f, 0, r0, group);
        tma_prefetch_3d(&tm_b, 0, r0, group);
    }
    if (tid == 0) {
#pragma unroll
        for (int i = 0; i < 5; ++i) mbar_init(bar_g + 8 * i, 1);
        mbar_init(bar_pfx, 1);
        mbar_init(bar_g + 80, 1);   // never completed: only the test hook waits on it
        mbar_init(bar_g + 88, 2);   // both chunks' summary batches are done (one phase per unit)
        *time_flag = 0;
        *early_gates = -1;
        *unit_slow_slot = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) slow_slot[i] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"(kTmemCols));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    build_zero_one_tile(bp + lay.zf, tid);
    build_diag_masks(bp + lay.masks, tid);
    // Tile rows the loads never reach (from `rows` up to the 256-row pitch) are K rows of the prefix-sum product
    // of chunk 1: they must be finite, and nothing but the recurrence scratch ever writes them again.
    auto zero_tail_rows = [&]() {
        if (nc == 2) {
            const int tail16 = (2 * kChunk - args.rows) * 4;   // 16-byte pieces per tile
            for (int x = tid; x < 4 * tail16; x += kThreads)
                *reinterpret_cast<uint4*>(bp + (uint32_t)(x / tail16) * lay.tile + (uint32_t)args.rows * 64 + (uint32_t)(x % tail16) * 16) =
                    make_uint4(0u, 0u, 0u, 0u);
        }
    };
    zero_tail_rows();
    if (tid < 128) dec[tid] = 0.f;   // key dims a narrow head never writes
    pdl_wait();   // nothing above touches global memory: it may run while the previous kernel in the stream drains
    if (warp == 0 && elect_one()) {
        load_gates(group, 2 * lay.tile);
        load_qk(group, 0);
        load_v(group);
    }
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *slot_p;
    const uint32_t tc = tmem + (uint32_t)c * 128;                   // this chunk's 128 TMEM columns
    const uint32_t rc = tc + ((uint32_t)(wq * 32) << 16);           // ... at this thread's lane
    const uint32_t rl = tmem + ((uint32_t)(wq * 32) << 16);         // TMEM block 0 at this thread's lane

    // A bounded wait that expires raises the flag and lets the block finish the unit on whatever it has:
    // every later wait is bounded too, nothing more is stored, and the host sees the device status word.
    auto wait_bar = [&](uint32_t bar, uint32_t parity, uint32_t limit = 1u << 21) {
        if (!mbar_wait_bounded(bar, parity, limit)) *time_flag = 1;
    };
    auto wait_mma = [&]() {
        wait_bar(bar_mma, mma_phase & 1);
        ++mma_phase;
        tc_fence_after();
    };
    // the threads of this chunk have finished their TMEM / shared-memory accesses -> its issuing warp may go on
    auto chunk_handover = [&]() {
        tc_fence_before();
        named_bar(1 + c, kChunk);
        tc_fence_after();
    };
    const uint32_t row0_64 = (uint32_t)c * (kChunk * 64) >> 4, row0_128 = (uint32_t)c * (kChunk * 128) >> 4;   // in descriptor units
    // Prefix sums of both log-gate tiles of both chunks in one batch: B stacks, along N, the 32 key dims of
    // [la> chunk 0 | la> chunk 1 | la< chunk 0 | la< chunk 1] (one unit of 64 or more tokens: [la> | la<]), so the
    // sums land in TMEM block 0, columns 32 x that order - the columns the previous unit's packed scores and chunk 0's
    // output leave free.
    const uint32_t pfx_b_col = nc == 2 ? 64u : 32u;
    auto issue_prefix = [&](uint32_t gates_pair) {
        const uint32_t z = desc_lo(base + lay.zf, 128);
        const uint32_t g = desc_lo(base + gates_pair, nc == 2 ? kChunk * 64 : lay.tile);
        const uint32_t ids = instr_desc(128, nc == 2 ? 128 : 64, 0, 1);
#pragma unroll 1
        for (int j = 0; j < ks_c0; ++j) {
            const uint32_t win = (uint32_t)(14 - 2 * j) * 16;   // window start row 112 - 16 j
            umma_ss(tmem, desc64(z + win, kHiZ), desc64(g + j * 64, kHiK64), ids, j > 0);
        }
        umma_commit(bar_pfx);
    };
    const int npass_c0 = ks_c0 > 4 ? 2 : 1;
    // Fused gate preparation (GATES): the two gate tiles of a pair hold the logits g and are rewritten in place as
    // log2 alpha (the prefix sums, their totals and the range check are then in base 2 as well: kExp = 1), 16-byte pieces dealt out evenly to the threads of the block.  Rows and columns the loads filled with
    // zeros stay zero (log alpha = 0: no decay, and k = v = 0 there): the forward tile holds token r in row r, the
    // backward tile token r - 1 (rows 1 .. L).
    auto prepare_gates = [&](uint32_t pair) {
        const int per_tile = 4 * min(L + 1, args.rows);   // rows 0 .. L of a tile (as far as it reaches), four pieces each
#pragma unroll 1
        for (int x = tid; x < 2 * per_tile; x += kThreads) {
            const int tile = x >= per_tile, y = x - tile * per_tile, r = y >> 2, pc = y & 3;
            if ((pc ^ ((r >> 1) & 3)) * 8 >= DK) continue;   // this piece holds padding columns
            if (tile == 0 ? r >= L : r < 1) continue;
            uint4* gp = reinterpret_cast<uint4*>(bp + pair + (uint32_t)tile * lay.tile + (uint32_t)r * 64 + pc * 16);
            *gp = log2_alpha_piece(*gp, args.inv_tau);
        }
        fence_async_smem();   // written through the generic proxy, read by the prefix-sum MMAs through the async proxy
    };

    if (args.expire_wait && tid == 0) wait_bar(bar_g + 80, 0, 64);   // test hook: this wait cannot succeed
    // ---- the block walks over its units; the loads of the next one are issued while this one is stored ----
    uint32_t it = 0;
    bool v_load_pending = false;      // control warp (uniform in it): the v tile of the current unit has not been requested yet
    bool next_gates_issued = false;   // control warp: the log gates of the next unit are already on their way
    bool next_loads_issued = false;   // control warp: so are its q and k
    for (long long unit_ll = group; unit_ll < args.units; unit_ll += ngroups, ++it) {
        const int unit = (int)unit_ll;
        const uint32_t par = it & 1;
        const bool has_next = unit_ll + ngroups < args.units;
        const uint32_t pair_qk = (it & 1) ? 2 * lay.tile : 0, pair_g = (it & 1) ? 0 : 2 * lay.tile;   // byte offsets of this unit's tile pairs
        const uint32_t t_kb = base + pair_qk, t_kf = t_kb + lay.tile;   // q, k as loaded; k~<, k~> after scaling
        const uint32_t t_qf = base + pair_g, t_qb = t_qf + lay.tile;    // log alpha>, log alpha< as loaded; q~>, q~< after scaling
        if (warp == 7 && has_next && elect_one()) {
            // pull the tiles of this block's next unit into L2
            const int pu = unit + ngroups;
            tma_prefetch_3d(&tm_f, 0, r0, pu);
            tma_prefetch_3d(&tm_b, 0, r0, pu);
            tma_prefetch_3d(&tm_q, 0, r0, pu);
            tma_prefetch_3d(&tm_k, 0, r0, pu);
            tma_prefetch_3d(&tm_v, 0, r0, pu);
        }

        if constexpr (GATES) {
            // fused gate preparation, unless it was done (and the prefix sums were issued) under the previous unit's epilogue
            if (!(nc == 2 && *early_gates == (int)it)) {
                wait_bar(bar_g, par);
                prepare_gates(pair_g);
                __syncthreads();
            }
        }
        if (chunk_on) {
            // ---- prefix sums of the log gates (unless they were issued while the previous unit was finishing) ----
            if (issue_warp && c == 0 && !(nc == 2 && *early_gates == (int)it) && elect_one()) {
                wait_bar(bar_g, par);
                issue_prefix(pair_g);
            }
            wait_bar(bar_pfx, par);
            tc_fence_after();
            wait_bar(bar_qk, par);

            // ---- scaled operands, in place: every thread rewrites its own row ---------------------------------
            if (warp_live) {
                constexpr int kHalves = (DK + 15) / 16;
                const int last_row = min(L, (c + 1) * kChunk) - 1;
                const bool check_row = row == last_row;
                uint32_t pf[kHalves][16], pb[kHalves][16];
                tmem_ld16(rl + 32 * c, pf[0]);
                tmem_ld16(rl + pfx_b_col + 32 * c, pb[0]);
                tc_wait_ld();
                if (kHalves == 2) {   // the second half travels while the first is worked on
                    tmem_ld16(rl + 32 * c + 16, pf[kHalves - 1]);
                    tmem_ld16(rl + pfx_b_col + 32 * c + 16, pb[kHalves - 1]);
                }
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf) {
                    if (hf == 1) tc_wait_ld();
                    if (hf == kHalves - 1 && nc == 2 && c == 1) {
                        // chunk 0 may overwrite its TMEM block (where these sums live) from here on
                        tc_fence_before();
                        asm volatile("bar.arrive 3, 256;" ::: "memory");
                    }
                    if (check_row) {
                        // totals of the log gates over the chunk, b and x at its last row.  They feed the range check
                        // (done by a whole warp after the hand-over) and the decay of the chunk summaries.
#pragma unroll
                        for (int x = 0; x < 4; ++x) {
                            reinterpret_cast<uint4*>(dec + (2 * c) * 32 + 16 * hf)[x] = make_uint4(pf[hf][4 * x], pf[hf][4 * x + 1], pf[hf][4 * x + 2], pf[hf][4 * x + 3]);
                            reinterpret_cast<uint4*>(dec + (2 * c + 1) * 32 + 16 * hf)[x] = make_uint4(pb[hf][4 * x], pb[hf][4 * x + 1], pb[hf][4 * x + 2], pb[hf][4 * x + 3]);
                        }
                    }
                    if (row_live) {
#pragma unroll
                        for (int c8 = 0; c8 < 2; ++c8) {
                            const int ch = 2 * hf + c8;   // 16-byte chunk of the row: key dims 8 ch .. 8 ch + 7
                            if (ch >= DK / 8) break;
                            const uint32_t off = sw_off<64>(row, ch);
                            const uint4 qv4 = *reinterpret_cast<const uint4*>(bp + pair_qk + off);
                            const uint4 kv4 = *reinterpret_cast<const uint4*>(bp + pair_qk + lay.tile + off);
                            const uint32_t qv[4] = {qv4.x, qv4.y, qv4.z, qv4.w}, kv[4] = {kv4.x, kv4.y, kv4.z, kv4.w};
                            uint32_t qf[4], kf[4], qb[4], kb[4];
#pragma unroll
                            for (int m = 0; m < 4; ++m) {
                                // the decaying factors on the special-function unit, the growing ones as their packed reciprocals
                                const int d0 = 8 * c8 + 2 * m;
                                const float ex0 = ex2(as_f(pf[hf][d0]) * kExp), ex1 = ex2(as_f(pf[hf][d0 + 1]) * kExp);
                                const float ey0 = ex2(as_f(pb[hf][d0]) * kExp), ey1 = ex2(as_f(pb[hf][d0 + 1]) * kExp);
                                const uint32_t exp_f = pack_bf16(ex0, ex1), exp_b = pack_bf16(ey0, ey1);
                                qf[m] = mul_bf16x2(qv[m], exp_f);               // q~> = q e^{b}
                                kf[m] = mul_bf16x2(kv[m], rcp_bf16x2(exp_f));   // k~> = k e^{-b}
                                qb[m] = mul_bf16x2(qv[m], rcp_bf16x2(exp_b));   // q~< = q e^{-x}
                                kb[m] = mul_bf16x2(kv[m], exp_b);               // k~< = k e^{x}
                            }
                            *reinterpret_cast<uint4*>(bp + pair_g + off) = make_uint4(qf[0], qf[1], qf[2], qf[3]);
                            *reinterpret_cast<uint4*>(bp + pair_qk + lay.tile + off) = make_uint4(kf[0], kf[1], kf[2], kf[3]);
                            *reinterpret_cast<uint4*>(bp + pair_g + lay.tile + off) = make_uint4(qb[0], qb[1], qb[2], qb[3]);
                            *reinterpret_cast<uint4*>(bp + pair_qk + off) = make_uint4(kb[0], kb[1], kb[2], kb[3]);
                        }
                    }
                }
            }
            if (c == 1 && !warp_live) {   // warps of chunk 1 without tokens read no sums but still take part in the hand-over
                asm volatile("bar.arrive 3, 256;" ::: "memory");
            }
            fence_async_smem();   // operand tiles were written through the generic proxy, the MMAs read them through the async proxy
            if (nc == 2 && c == 0) {
                // the chunk's own hand-over, extended by the arrival of chunk 1's warps (they have read their sums)
                if (!SEG) asm volatile("bar.arrive 5, 160;" ::: "memory");   // chunk 0's totals are written: see the chunk summaries
                tc_fence_before();
                named_bar(3, 2 * kChunk);
                tc_fence_after();
            } else {
                chunk_handover();
            }
            if (wq == 2) {
                // range check, one key dim per lane: b and x are smallest at the last row of the chunk
                constexpr float kRange = GATES ? kGateRange * kLog2e : kGateRange;   // the same bound in the base the totals are in
                const bool out_of_range = dec[(2 * c) * 32 + lane] < -kRange || dec[(2 * c + 1) * 32 + lane] < -kRange;
                const bool any = __any_sync(0xffffffffu, out_of_range);
                if (lane == 0) slow_slot[c] = any ? 1 : 0;
            }
            if (ctl_warp && v_load_pending) {
                // The store of the previous unit was issued a phase ago and has read the v tile by now: this
                // wait is short, and the tile is only needed again when the chunk summaries are formed.
                if (elect_one()) {
                    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    load_v(unit);
                }
                v_load_pending = false;
            }

            // ---- P, key columns [64 p, 64 p + 64): forward scores -> columns [0,64), backward -> [64,128) ----
            uint32_t hold[32];   // packed bf16 P of this row, key columns 0..63
            const uint32_t aqf = desc_lo(t_qf, 16) + row0_64, aqb = desc_lo(t_qb, 16) + row0_64;
            const uint32_t bkf = desc_lo(t_kf, 16) + row0_64, bkb = desc_lo(t_kb, 16) + row0_64;
#pragma unroll
            for (int p = 0; p < 2; ++p) {
                const int n = min(nkeys - 64 * p, 64);   // key columns of this half
                if (n <= 0) break;
                if (issue_warp && elect_one()) {
                    const uint32_t idp = instr_desc(128, n, 0, 0);
#pragma unroll
                    for (int kk = 0; kk < 2; ++kk) {
                        umma_ss(tc + 0, desc64(aqf + kk * 2, kHiK64), desc64(bkf + p * 256 + kk * 2, kHiK64), idp, kk > 0);
                        umma_ss(tc + 64, desc64(aqb + kk * 2, kHiK64), desc64(bkb + p * 256 + kk * 2, kHiK64), idp, kk > 0);
                    }
                    umma_commit(bar_mma);
                }
                wait_mma();
                if (warp_live) {
                    uint32_t pk[16];
                    combine_any(2 * p, wq, true, rc, rc + 64, lane, base + lay.masks, pk);
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
                    combine_any(2 * p + 1, wq, 64 * p + 32 < nkeys, rc + 32, rc + 96, lane, base + lay.masks, pk);
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
                chunk_handover();
            }

            // ---- chunk summary -> bf16 state tile for the other chunk (two chunks only) ------------------------------
            if (nc == 2 || SEG) {
                if (issue_warp && elect_one()) {
                    wait_bar(bar_v, par);
                    constexpr uint32_t kIdU = instr_desc(128, 64, 1, 1);
                    const uint32_t ak = desc_lo(t_kb, lay.tile) + row0_64, bv = desc_lo(t_v, 16) + row0_128;
#pragma unroll 1   // issue loops stay rolled: less code for the instruction cache, and nothing is gained by unrolling them
                    for (int kk = 0; kk < ks; ++kk)
                        umma_ss(tc + 64, desc64(ak + kk * 64, kHiK64), desc64(bv + kk * 128, kHiV128), kIdU, kk > 0);
                    umma_commit(bar_mma);
                }
                wait_mma();
            }
            if (nc == 2 && !SEG) {
                if (warp == 1 || warp == 4) {
                    // rows (TMEM lanes) 0..31 of U hold k~<^T v, rows 32..63 hold k~>^T v; lane = key dim.
                    // warp 1 (chunk 0, lanes 32..63): forward state for chunk 1; warp 4 (chunk 1, lanes 0..31): backward state
                    // for chunk 0.  Both are scaled by chunk 0's total decay of their direction, for key dim `lane`.
                    if (warp == 4) named_bar(5, 160);   // chunk 0's threads arrived after writing their totals
                    const float d = ex2(dec[(warp == 1 ? 0 : 32) + lane] * kExp);
                    uint8_t* st = bp + (warp == 1 ? lay.s_fwd : lay.s_bwd);
#pragma unroll
                    for (int hb = 0; hb < 2; ++hb) {
                        uint32_t r[32];
                        tmem_ld32(rc + 64 + hb * 32, r);
                        tc_wait_ld();
#pragma unroll
                        for (int ch = 0; ch < 4; ++ch) {
                            uint32_t o[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) o[e] = pack_bf16(as_f(r[ch * 8 + 2 * e]) * d, as_f(r[ch * 8 + 2 * e + 1]) * d);
                            *reinterpret_cast<uint4*>(st + sw_off<128>(lane, hb * 4 + ch)) = make_uint4(o[0], o[1], o[2], o[3]);
                        }
                    }
                    fence_async_smem();
                }
                // Each chunk's issuing warp reports its summary batch done (its own wait above) on a barrier of its own: a
                // parity wait on the other chunk's batch barrier could not tell which of that chunk's batches it sees.
                if (issue_warp && elect_one()) mbar_arrive(bar_g + 88);
                if (warp == 5 && has_next && elect_one()) {
                    // The summaries were the last readers of the k~ pair: the next unit's log gates go there now, a good
                    // two microseconds before they are needed.  Issued from chunk 1's issuing warp, which has no share in
                    // the state hand-over that both chunks wait for.
                    wait_bar(bar_g + 88, par);
                    if ((slow_slot[0] | slow_slot[1] | slow_slot[2] | slow_slot[3]) == 0 && *time_flag == 0) {
                        load_gates(unit + ngroups, pair_qk);
                        *early_gates = (int)it + 1;   // seen by every warp after the exchange barrier
                    }
                }
            }
        }
        if (nc == 2 && !SEG) {   // the two chunks exchange their states
            tc_fence_before();
            __syncthreads();
            tc_fence_after();
        }
        if constexpr (SEG) {
            // ---- segmented sequences: summaries of this block's chunks -> segment summary -> exchange with the other
            // blocks of the unit through scratch memory -> the four incoming states of this block's chunks --------------
            // With T>(c) = (k~>)^T v and T<(c) = (k~<)^T v of chunk c, D>(c) = e^{b_last(c)}, d<(c) = e^{x_last(c)}:
            //   forward:  S>_in(c + 1) = D>(c) S>_in(c) + D>(c) T>(c)
            //   backward: R(c) = T<(c) + d<(c) R(c + 1),  S<_in(c) = d<(c) R(c + 1)   (q~< lacks the chunk's own decay)
            // and the same two recursions run over the segments with the segment summaries
            //   D> = D>(0) D>(1), E> = D>(1) D>(0) T>(0) + D>(1) T>(1);   d< = d<(0) d<(1), R = T<(0) + d<(0) T<(1).
            tc_fence_before();
            __syncthreads();   // every summary batch of the block is done: the k~ pair is dead
            tc_fence_after();
            float* su = reinterpret_cast<float*>(bp + pair_qk);   // [2 chunks][T>, T<][32 key dims][64], 16-byte pieces XORed with the key dim
            if (chunk_on && wq < 2) {
                // TMEM lanes 0..31 of the summary hold T<, lanes 32..63 hold T>; lane = key dim
                float* dst = su + (size_t)((c * 2 + (wq == 1 ? 0 : 1)) * 32 + lane) * 64;
#pragma unroll
                for (int hb = 0; hb < 2; ++hb) {
                    uint32_t r[32];
                    tmem_ld32(rc + 64 + hb * 32, r);
                    tc_wait_ld();
#pragma unroll
                    for (int x = 0; x < 8; ++x)
                        reinterpret_cast<uint4*>(dst)[(hb * 8 + x) ^ (lane & 15)] = make_uint4(r[4 * x], r[4 * x + 1], r[4 * x + 2], r[4 * x + 3]);
                }
            }
            __syncthreads();
            // thread (i, j8): key dim i, value dims 8 j8 .. 8 j8 + 7
            const int si = tid >> 3, sj = tid & 7;
            const bool two = nc == 2;
            const float Df0 = ex2(dec[si] * kLog2e), Db0 = ex2(dec[32 + si] * kLog2e);
            const float Df1 = two ? ex2(dec[64 + si] * kLog2e) : 1.f, Db1 = two ? ex2(dec[96 + si] * kLog2e) : 1.f;
            auto su_row = [&](int cc, int dir, float (&o)[8]) {
                const uint4* src = reinterpret_cast<const uint4*>(su + (size_t)((cc * 2 + dir) * 32 + si) * 64);
                const uint4 a = src[(2 * sj) ^ (si & 15)], b = src[(2 * sj + 1) ^ (si & 15)];
                o[0] = as_f(a.x); o[1] = as_f(a.y); o[2] = as_f(a.z); o[3] = as_f(a.w);
                o[4] = as_f(b.x); o[5] = as_f(b.y); o[6] = as_f(b.z); o[7] = as_f(b.w);
            };
            uint8_t* slot_u = args.ws + ((size_t)unit * nseg) * kSlotBytes;   // the unit's slots, one per segment
            {
                float tf0[8], tb0[8], tf1[8], tb1[8], e[8], r[8];
                su_row(0, 0, tf0);
                su_row(0, 1, tb0);
                if (two) { su_row(1, 0, tf1); su_row(1, 1, tb1); }
#pragma unroll
                for (int x = 0; x < 8; ++x) {
                    if (!two) { tf1[x] = 0.f; tb1[x] = 0.f; }
                    e[x] = Df1 * (Df0 * tf0[x] + tf1[x]);
                    r[x] = fmaf(Db0, tb1[x], tb0[x]);
                }
                uint8_t* mine = slot_u + (size_t)seg * kSlotBytes;
                const size_t eoff = (size_t)(si * 64 + sj * 8) * 2;
                __stcg(reinterpret_cast<uint4*>(mine + kSlotFwd + eoff),
                       make_uint4(pack_bf16(e[0], e[1]), pack_bf16(e[2], e[3]), pack_bf16(e[4], e[5]), pack_bf16(e[6], e[7])));
                __stcg(reinterpret_cast<uint4*>(mine + kSlotBwd + eoff),
                       make_uint4(pack_bf16(r[0], r[1]), pack_bf16(r[2], r[3]), pack_bf16(r[4], r[5]), pack_bf16(r[6], r[7])));
                if (sj == 0) {
                    float* dd = reinterpret_cast<float*>(mine + kSlotDecay);
                    __stcg(dd + si, Df0 * Df1);
                    __stcg(dd + 32 + si, Db0 * Db1);
                }
            }
            __syncthreads();   // the whole summary is written: the release below, by one thread, publishes all of it
            if (warp == 0) {
                const int local_slow = (slow_slot[0] | slow_slot[1] | slow_slot[2] | slow_slot[3]) != 0;
                if (lane == 0) {
                    __threadfence();
                    st_release_u64(reinterpret_cast<unsigned long long*>(slot_u + (size_t)seg * kSlotBytes),
                                   (args.nonce << 16) | ((unsigned long long)local_slow << 15));
                }
                // lane p waits for the summary of segment p (bounded: the blocks of a group are resident together)
                bool ok = true;
                int peer_slow = local_slow;
                if (lane < nseg && lane != seg) {
                    const unsigned long long* f = reinterpret_cast<const unsigned long long*>(slot_u + (size_t)lane * kSlotBytes);
                    ok = false;
#pragma unroll 1
                    for (uint32_t spin = 0; spin < (1u << 21); ++spin) {
                        const unsigned long long v = ld_acquire_u64(f);
                        if ((v >> 16) == args.nonce) { ok = true; peer_slow = (int)((v >> 15) & 1); break; }
                        if (spin > 64) __nanosleep(64);
                    }
                }
                const bool all_ok = __all_sync(0xffffffffu, ok);
                const bool any_slow = __any_sync(0xffffffffu, peer_slow != 0);
                if (lane == 0) {
                    if (!all_ok) *time_flag = 1;
                    *unit_slow_slot = any_slow ? 1 : 0;
                }
            }
            __syncthreads();
            {
                // fold the summaries of the segments to the left (forward state entering this segment, ascending) and to
                // the right (R at the first token of the next segment, descending); up to eight loads per direction are
                // issued before any of them is used
                float sin[8], rn[8];
#pragma unroll
                for (int x = 0; x < 8; ++x) sin[x] = rn[x] = 0.f;
                const bool usable = *time_flag == 0;   // after a time-out the slots may be incomplete: their values are not used
                constexpr int kB = 8;
                const size_t eoff = (size_t)(si * 64 + sj * 8) * 2;
                int pf = 0, pb = nseg - 1;   // next forward peer (ascending), next backward peer (descending)
                while (usable && (pf < seg || pb > seg)) {
                    uint4 ef[kB], rb[kB];
                    float df[kB], db[kB];
#pragma unroll
                    for (int b = 0; b < kB; ++b) {
                        if (pf + b < seg) {
                            const uint8_t* sl = slot_u + (size_t)(pf + b) * kSlotBytes;
                            ef[b] = __ldcg(reinterpret_cast<const uint4*>(sl + kSlotFwd + eoff));
                            df[b] = __ldcg(reinterpret_cast<const float*>(sl + kSlotDecay) + si);
                        }
                        if (pb - b > seg) {
                            const uint8_t* sl = slot_u + (size_t)(pb - b) * kSlotBytes;
                            rb[b] = __ldcg(reinterpret_cast<const uint4*>(sl + kSlotBwd + eoff));
                            db[b] = __ldcg(reinterpret_cast<const float*>(sl + kSlotDecay) + 32 + si);
                        }
                    }
#pragma unroll
                    for (int b = 0; b < kB; ++b) {
                        if (pf + b < seg) {
                            const uint32_t w[4] = {ef[b].x, ef[b].y, ef[b].z, ef[b].w};
#pragma unroll
                            for (int x = 0; x < 4; ++x) {
                                const float2 t = unpack_bf16(w[x]);
                                sin[2 * x] = fmaf(df[b], sin[2 * x], t.x);
                                sin[2 * x + 1] = fmaf(df[b], sin[2 * x + 1], t.y);
                            }
                        }
                        if (pb - b > seg) {
                            const uint32_t w[4] = {rb[b].x, rb[b].y, rb[b].z, rb[b].w};
#pragma unroll
                            for (int x = 0; x < 4; ++x) {
                                const float2 t = unpack_bf16(w[x]);
                                rn[2 * x] = fmaf(db[b], rn[2 * x], t.x);
                                rn[2 * x + 1] = fmaf(db[b], rn[2 * x + 1], t.y);
                            }
                        }
                    }
                    pf += kB;
                    pb -= kB;
                }
                // the four incoming states of this block's chunks, as bf16 tiles over the (now dead) summaries
                float tf0[8], tb1[8];
                su_row(0, 0, tf0);
                if (two) su_row(1, 1, tb1);
                __syncthreads();   // every thread has read what it needs of the summaries
                uint32_t sf0[4], sf1[4], sb0[4], sb1[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    float f1[2], b1[2], b0[2];
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int y = 2 * x + h;
                        f1[h] = Df0 * (sin[y] + tf0[y]);                    // S>_in(1) = D>(0) (S>_in(0) + T>(0))
                        const float r1 = two ? fmaf(Db1, rn[y], tb1[y]) : rn[y];   // R(1)
                        b1[h] = Db1 * rn[y];                                 // S<_in(1)
                        b0[h] = Db0 * r1;                                    // S<_in(0)
                    }
                    sf0[x] = pack_bf16(sin[2 * x], sin[2 * x + 1]);
                    sf1[x] = pack_bf16(f1[0], f1[1]);
                    sb0[x] = pack_bf16(b0[0], b0[1]);
                    sb1[x] = pack_bf16(b1[0], b1[1]);
                }
                uint8_t* st = bp + pair_qk;   // [chunk][S>_in, S<_in] tiles of [32][64] bf16, 128B swizzle
                const uint32_t so = sw_off<128>(si, sj);
                *reinterpret_cast<uint4*>(st + 0 * 4096 + so) = make_uint4(sf0[0], sf0[1], sf0[2], sf0[3]);
                *reinterpret_cast<uint4*>(st + 1 * 4096 + so) = make_uint4(sb0[0], sb0[1], sb0[2], sb0[3]);
                *reinterpret_cast<uint4*>(st + 2 * 4096 + so) = make_uint4(sf1[0], sf1[1], sf1[2], sf1[3]);
                *reinterpret_cast<uint4*>(st + 3 * 4096 + so) = make_uint4(sb1[0], sb1[1], sb1[2], sb1[3]);
                fence_async_smem();
            }
            tc_fence_before();
            __syncthreads();
            tc_fence_after();
        }

        if (chunk_on) {
            // ---- out = (P v + q~ S_in) / 2 ------------------------------------------------------------------------
            if (issue_warp && elect_one()) {
                wait_bar(bar_v, par);
                constexpr uint32_t kIdO = instr_desc(128, 64, 0, 1);
                uint32_t acc = 0;
                if constexpr (SEG) {
                    // both incoming states of this chunk: [chunk][S>_in, S<_in] tiles over the k~ pair
                    const uint32_t qf = desc_lo(t_qf, 16) + row0_64, qb = desc_lo(t_qb, 16) + row0_64;
                    const uint32_t sf = desc_lo(base + pair_qk + (uint32_t)c * 8192, 16), sb = sf + (4096 >> 4);
#pragma unroll
                    for (int kk = 0; kk < 2; ++kk) umma_ss(tc + 64, desc64(qf + kk * 2, kHiK64), desc64(sf + kk * 128, kHiV128), kIdO, kk > 0);
#pragma unroll
                    for (int kk = 0; kk < 2; ++kk) umma_ss(tc + 64, desc64(qb + kk * 2, kHiK64), desc64(sb + kk * 128, kHiV128), kIdO, 1);
                    acc = 1;
                } else if (nc == 2) {
                    // chunk 1 receives the forward state of chunk 0, chunk 0 the backward state of chunk 1
                    const uint32_t qa = desc_lo(c == 1 ? t_qf : t_qb, 16) + row0_64;
                    const uint32_t sa = desc_lo(base + (c == 1 ? lay.s_fwd : lay.s_bwd), 16);
#pragma unroll
                    for (int kk = 0; kk < 2; ++kk) umma_ss(tc + 64, desc64(qa + kk * 2, kHiK64), desc64(sa + kk * 128, kHiV128), kIdO, kk > 0);
                    acc = 1;
                }
                const uint32_t bv = desc_lo(t_v, 16) + row0_128;
#pragma unroll 1
                for (int kk = 0; kk < ks; ++kk) umma_ts(tc + 64, tc + kk * 8, desc64(bv + kk * 128, kHiV128), kIdO, kk > 0 ? 1u : acc);
                umma_commit(bar_mma);
            }
            wait_mma();
            if constexpr (GATES) {
                if (nc == 2) {
                    // The next unit's gate logits have been on their way since the chunk summaries: every thread prepares
                    // its share now, so that the prefix sums can be issued under this unit's epilogue as in the un-fused form.
                    if (*early_gates == (int)it + 1) {
                        wait_bar(bar_g, par ^ 1);
                        prepare_gates(pair_qk);
                    }
                    if (c == 1 && warp != 7) asm volatile("bar.arrive 6, 256;" ::: "memory");
                }
            }
            if (warp == 7 && nc == 2 && *early_gates == (int)it + 1 && elect_one()) {
                // The packed scores of both chunks have been consumed (this thread has waited for chunk 1's output batch,
                // now for chunk 0's): their TMEM columns take the next unit's prefix sums, whose log gates have been on
                // their way since the chunk summaries.  Warp 7 has the fewest rows to write out.
                wait_bar(bar_g + 24, ((it + 1) * (uint32_t)(npass_c0 + 2) - 1) & 1);
                wait_bar(bar_g, par ^ 1);
            }
            if (nc == 2 && warp == 7) {
                // ... and chunk 0's output has left TMEM block 0, which takes the sums of all four gate blocks
                named_bar(6, GATES ? 256 : 160);   // (fused gates: the other warps of chunk 1 have prepared their share too)
                tc_fence_after();
                if (*early_gates == (int)it + 1 && elect_one()) issue_prefix(pair_qk);
                __syncwarp();
            }
            if (ctl_warp && has_next) {
                // Every MMA that reads the q~ pair is done once chunk 1's last batch is: the next unit's q and k start
                // to load under the epilogue and the store (unless this unit must be redone by the recurrence,
                // whose scratch overlays the tiles).
                bool go = false;
                if (elect_one()) {
                    if (nc == 2) wait_bar(bar_mma + 8, ((it + 1) * (uint32_t)(npass_c1 + 2) - 1) & 1);
                    go = (SEG ? *unit_slow_slot : (slow_slot[0] | slow_slot[1] | slow_slot[2] | slow_slot[3])) == 0 && *time_flag == 0;
                    if (go) {
                        if (!(nc == 2 && !SEG && *early_gates == (int)it + 1)) load_gates(unit + ngroups, pair_qk);   // not on their way yet
                        load_qk(unit + ngroups, pair_g);
                    }
                }
                if (__any_sync(0xffffffffu, go)) next_gates_issued = next_loads_issued = true;
            }
            // epilogue: out = O / 2, bf16, into the dead v tile (same swizzle as the TMA store expects)
            if (warp_live) {
                uint32_t r[2][32];
                tmem_ld32(rc + 64, r[0]);
                if (DV == 64) tmem_ld32(rc + 96, r[1]);
                if (DV == 48) {
                    uint32_t t[16];
                    tmem_ld16(rc + 96, t);
#pragma unroll
                    for (int e = 0; e < 16; ++e) r[1][e] = t[e];
                }
                tc_wait_ld();
                if (nc == 2 && c == 0) {   // TMEM block 0 is free for the next unit's prefix sums
                    tc_fence_before();
                    if (GATES) asm volatile("bar.arrive 6, 256;" ::: "memory");
                    else asm volatile("bar.arrive 6, 160;" ::: "memory");
                }
                if (row_live) {
#pragma unroll
                    for (int ch = 0; ch < DV / 8; ++ch) {
                        uint32_t o[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e)   // halved after packing: exact (a power of two), one instruction per pair
                            o[e] = mul_bf16x2(pack_bf16(as_f(r[ch >> 2][(ch & 3) * 8 + 2 * e]), as_f(r[ch >> 2][(ch & 3) * 8 + 2 * e + 1])), 0x3F003F00u);
                        *reinterpret_cast<uint4*>(bp + lay.v + sw_off<128>(row, ch)) = make_uint4(o[0], o[1], o[2], o[3]);
                    }
                }
            }
        }
        fence_async_smem();
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        // every MMA of this unit has completed and every thread has left its tiles: block-uniform decisions
        const bool timed_out = *time_flag != 0;
        const bool slow = (SEG ? *unit_slow_slot : (slow_slot[0] | slow_slot[1] | slow_slot[2] | slow_slot[3])) != 0;   // SEG: any segment of the unit
        if (timed_out) break;
        if (SEG && warp == 7 && lane < nseg && lane != seg) {
            // This block is done with the other segments' slots of this unit: the last reader of a slot clears its flag, so
            // that a replay of the same call (a captured graph: same nonce) starts from flags that do not match.  Nothing
            // waits for this warp before the next unit's first barrier.
            unsigned long long* f = reinterpret_cast<unsigned long long*>(args.ws + ((size_t)unit * nseg + lane) * kSlotBytes);
            const unsigned long long old = atomicAdd(f, 1ull);
            if ((int)(old & 0x7fffull) == nseg - 2) st_release_u64(f, 0ull);
        }
        if (!slow) {
            if (ctl_warp) {
                if (elect_one()) {
                    tma_store_3d(&tm_o, 0, r0, unit, t_v);   // rows >= L and columns >= dv are clipped
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    if (has_next && !next_gates_issued && !(nc == 2 && !SEG && *early_gates == (int)it + 1)) load_gates(unit + ngroups, pair_qk);
                    if (has_next && !next_loads_issued) load_qk(unit + ngroups, pair_g);
                }
                next_gates_issued = next_loads_issued = false;
                v_load_pending = has_next;   // the v tile only once the store has read it: see above
            }
        } else {
            // A gate left the range the factorised tiles can represent: evaluate this unit by the recurrence
            // (its scratch overlays the tiles, so the next loads wait until it is done).
            // (segmented sequences: the block of the first segment redoes the whole unit, the others store nothing)
            if (seg == 0) {
                if (tid == 0) atomicAdd(args.dev_status + 1, 1);   // units handed to the recurrence (read by the tests)
                const size_t ok = (size_t)unit * args.L * DK, ov = (size_t)unit * args.L * DV;
                recurrence_unit<__nv_bfloat16>(args.q + ok, args.k + ok, args.v + ov, args.la_f + ok, args.la_b + ok,
                                               args.out + ov, args.L, DK, DV, reinterpret_cast<float*>(bp), GATES ? args.inv_tau : 0.f);
            }
            __syncthreads();
            zero_tail_rows();
            fence_async_smem();
            __syncthreads();
            if (ctl_warp && has_next && elect_one()) {
                load_gates(unit + ngroups, pair_qk);
                load_qk(unit + ngroups, pair_g);
                load_v(unit + ngroups);
            }
        }
    }

    // the last store still reads shared memory (the elected thread is the same every time: it owns the bulk groups)
    if (ctl_warp && elect_one()) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    // ---- release TMEM (every tcgen05 operation of this block has completed) ----
    tc_fence_before();
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols));
    if (tid == 0 && *time_flag != 0) atomicOr(args.dev_status, kDevStatusTimeout);
}

// Resident blocks per SM and SM count of the current device for one instantiation (queried once per device; also
// opts the kernel in to the shared memory of its longest unit).
struct DevPlan {
    int sms, per_sm;
};
template <int DK, int DV, bool SEG, bool GATES>
cudaError_t device_plan(size_t smem_max, DevPlan* out) {
    static std::atomic<int> sms_of[kMaxDevices], per_sm_of[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    int sms = sms_of[dev].load(std::memory_order_acquire);
    if (sms == 0) {
        cudaError_t e = cudaFuncSetAttribute(bigla_umma_kernel<DK, DV, SEG, GATES>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max);
        if (e != cudaSuccess) return e;
        // Blocks of this kernel an SM holds at once, from the resources themselves: two (2 x 256 of the 512 TMEM columns)
        // if shared memory (plus the kilobyte the system keeps per block) and the register file admit them.  The occupancy
        // calculator of the runtime reports one block for this kernel where the hardware runs two.
        cudaFuncAttributes fa;
        if ((e = cudaFuncGetAttributes(&fa, bigla_umma_kernel<DK, DV, SEG, GATES>)) != cudaSuccess) return e;
        int smem_sm = 0, regs_sm = 0;
        if ((e = cudaDeviceGetAttribute(&smem_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev)) != cudaSuccess) return e;
        if ((e = cudaDeviceGetAttribute(&regs_sm, cudaDevAttrMaxRegistersPerMultiprocessor, dev)) != cudaSuccess) return e;
        const int regs_block = (fa.numRegs + 7) / 8 * 8 * kThreads;
        const int per_sm = (2 * (smem_max + fa.sharedSizeBytes + 1024) <= (size_t)smem_sm && 2 * regs_block <= regs_sm) ? 2 : 1;
        if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        per_sm_of[dev].store(per_sm, std::memory_order_release);
        sms_of[dev].store(sms, std::memory_order_release);
    }
    out->sms = sms;
    out->per_sm = per_sm_of[dev].load(std::memory_order_acquire);
    return cudaSuccess;
}

// GATES: la_f / la_b are the gate logits and `tau` their temperature (fused gate preparation).
template <int DK, int DV, bool GATES>
cudaError_t launch_umma_t(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                          const __nv_bfloat16* la_f, const __nv_bfloat16* la_b, __nv_bfloat16* out, long long units, int L,
                          float tau, cudaStream_t stream) {
    const int rows = (L + 15) / 16 * 16;
    CUtensorMap tq, tk, tf, tb, tv, to;
    if (!make_map(&tq, q, units, L, DK, 32, rows) || !make_map(&tk, k, units, L, DK, 32, rows) ||
        !make_map(&tf, la_f, units, L, DK, 32, rows) || !make_map(&tb, la_b, units, L, DK, 32, rows) ||
        !make_map(&tv, v, units, L, DV, 64, rows) || !make_map(&to, out, units, L, DV, 64, rows))
        return cudaErrorInvalidValue;
    UArgs a{};
    a.q = q; a.k = k; a.v = v; a.la_f = la_f; a.la_b = la_b; a.out = out; a.L = L; a.rows = rows; a.units = units;
    a.nseg = 1;
    a.inv_tau = GATES ? 1.f / tau : 0.f;
    a.expire_wait = take_expire_next_wait();
    a.dev_status = device_status_ptr();
    if (!a.dev_status) return cudaErrorUnknown;
    // The MMAs of chunk 1 read 128 rows of the operand tiles from row 128 on, i.e. up to (256 - rows) * 64
    // bytes past the last q-type tile: that lands in the v tile, inside the allocation.
    size_t smem = make_layout(rows, false).total;
    const size_t rec = (size_t)rec_plan(kThreads, DK, DV).smem_floats * 4;
    if (smem < rec) smem = rec;
    size_t most = make_layout(kMaxRows, false).total;
    if (most < rec) most = rec;
    DevPlan dp;
    cudaError_t e = device_plan<DK, DV, false, GATES>(most, &dp);
    if (e != cudaSuccess) return e;
    // Persistent blocks, two per SM: block b takes units b, b + grid, b + 2 grid, ...  (Nothing waits for another block
    // here, so a grid larger than what is resident at once only costs time.)
    const long long cap = 2LL * dp.sms;
    const long long grid = units < cap ? units : cap;
    const cudaError_t le = launch_pdl(bigla_umma_kernel<DK, DV, false, GATES>, dim3((unsigned)grid), dim3(kThreads), smem, stream, tq, tk, tf, tb, tv, to, a);
    count_launch();
    return le != cudaSuccess ? le : cudaGetLastError();
}

// Segmented sequences: a unit of up to kMaxSegments x 256 tokens is cut into segments of 256 tokens, one block each.
// The blocks of a unit exchange their segment summaries through scratch memory and wait for each other, so the grid
// is a whole number of groups of nseg blocks and never larger than what the device holds at once: every block is then
// dispatched without any other block of the grid having to finish first.  (A cooperative launch would have the runtime
// enforce this, but its occupancy calculator admits only one block of this kernel per SM where the hardware runs two.)
// Every wait on another block is bounded and ends in VIG_ERR_DEVICE_TIMEOUT should the assumption ever fail.
std::atomic<unsigned long long> g_seg_calls{0};

template <int DK, int DV>
cudaError_t launch_umma_seg_t(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                              const __nv_bfloat16* la_f, const __nv_bfloat16* la_b, __nv_bfloat16* out, long long units,
                              int L, void* ws, cudaStream_t stream) {
    const int nseg = (L + kMaxRows - 1) / kMaxRows;
    CUtensorMap tq, tk, tf, tb, tv, to;
    if (!make_map(&tq, q, units, L, DK, 32, kMaxRows) || !make_map(&tk, k, units, L, DK, 32, kMaxRows) ||
        !make_map(&tf, la_f, units, L, DK, 32, kMaxRows) || !make_map(&tb, la_b, units, L, DK, 32, kMaxRows) ||
        !make_map(&tv, v, units, L, DV, 64, kMaxRows) || !make_map(&to, out, units, L, DV, 64, kMaxRows))
        return cudaErrorInvalidValue;
    UArgs a{};
    a.q = q; a.k = k; a.v = v; a.la_f = la_f; a.la_b = la_b; a.out = out; a.L = L; a.rows = kMaxRows; a.units = units;
    a.nseg = nseg;
    a.ws = static_cast<uint8_t*>(ws);
    // the flags of this call: a value no earlier call wrote and no uninitialised word holds by chance (48 bits)
    a.nonce = (0x5A17ull << 32) + (g_seg_calls.fetch_add(1, std::memory_order_relaxed) & 0xffffffffull) + 1;
    a.dev_status = device_status_ptr();
    if (!a.dev_status) return cudaErrorUnknown;
    size_t smem = make_layout(kMaxRows, true).total;
    const size_t rec = (size_t)rec_plan(kThreads, DK, DV).smem_floats * 4;
    if (smem < rec) smem = rec;
    DevPlan dp;
    cudaError_t e = device_plan<DK, DV, true, false>(smem, &dp);
    if (e != cudaSuccess) return e;
    const long long cap = (long long)dp.per_sm * dp.sms;
    long long groups = cap / nseg;
    if (groups < 1) return cudaErrorLaunchOutOfResources;
    if (groups > units) groups = units;
    const cudaError_t le = launch_pdl(bigla_umma_kernel<DK, DV, true, false>, dim3((unsigned)(groups * nseg)), dim3(kThreads), smem, stream, tq, tk, tf, tb, tv, to, a);
    count_launch();
    return le != cudaSuccess ? le : cudaGetLastError();
}

}  // namespace

bool umma_supported(int dk, int dv, int L) {
    return (dk == 16 || dk == 24 || dk == 32) && (dv == 32 || dv == 48 || dv == 64) && L <= kMaxRows;
}

bool umma_seg_supported(int dk, int dv, int L) {
    return (dk == 16 || dk == 24 || dk == 32) && (dv == 32 || dv == 48 || dv == 64) && L > kMaxRows &&
           L <= kMaxSegments * kMaxRows;
}

size_t umma_seg_workspace_bytes(long long units, int L) {
    return (size_t)units * (size_t)((L + kMaxRows - 1) / kMaxRows) * kSlotBytes;
}

cudaError_t launch_bigla_umma_seg(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                                  const __nv_bfloat16* la_f, const __nv_bfloat16* la_b, __nv_bfloat16* out, long long units,
                                  int L, int dk, int dv, void* ws, cudaStream_t stream) {
#define VIG_CASE(DK_, DV_) \
    if (dk == DK_ && dv == DV_) return launch_umma_seg_t<DK_, DV_>(q, k, v, la_f, la_b, out, units, L, ws, stream);
    VIG_CASE(16, 32) VIG_CASE(16, 48) VIG_CASE(16, 64)
    VIG_CASE(24, 32) VIG_CASE(24, 48) VIG_CASE(24, 64)
    VIG_CASE(32, 32) VIG_CASE(32, 48) VIG_CASE(32, 64)
#undef VIG_CASE
    return cudaErrorNotSupported;
}

cudaError_t launch_bigla_umma(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                              const __nv_bfloat16* la_f, const __nv_bfloat16* la_b, __nv_bfloat16* out, long long units,
                              int L, int dk, int dv, float gate_tau, cudaStream_t stream) {
#define VIG_CASE(DK_, DV_)                                                                                              \
    if (dk == DK_ && dv == DV_)                                                                                         \
        return gate_tau > 0.f ? launch_umma_t<DK_, DV_, true>(q, k, v, la_f, la_b, out, units, L, gate_tau, stream)     \
                              : launch_umma_t<DK_, DV_, false>(q, k, v, la_f, la_b, out, units, L, 0.f, stream);
    VIG_CASE(16, 32) VIG_CASE(16, 48) VIG_CASE(16, 64)
    VIG_CASE(24, 32) VIG_CASE(24, 48) VIG_CASE(24, 64)
    VIG_CASE(32, 32) VIG_CASE(32, 48) VIG_CASE(32, 64)
#undef VIG_CASE
    return cudaErrorNotSupported;
}

}  // namespace vig
