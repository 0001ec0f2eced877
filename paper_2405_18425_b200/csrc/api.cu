// C-ABI entry points of libvig_bigla: argument validation, dispatch, host-buffer path, diagnostics.
#include <atomic>
#include <cmath>
#include <mutex>

#include "test_hooks.h"
#include "vig_internal.h"

namespace vig {

// [0]: the device status word (bit flags, kDevStatus*);  [1]: units the tensor-core kernels handed to their in-kernel
// recurrence since the counter was last read (a test aid: kernels find it one word behind the status word).
__device__ int g_device_status[2] = {0, 0};
static std::atomic<int> g_expire_next_wait{0};   // test hook: the next single-block launch lets one bounded wait run out
int take_expire_next_wait() { return g_expire_next_wait.exchange(0, std::memory_order_relaxed); }

static std::atomic<unsigned long long> g_launches{0};
static std::atomic<int> g_kernel_pref{VIG_TEST_KERNEL_AUTO};   // changed by the test hook only
int kernel_preference() { return g_kernel_pref.load(std::memory_order_relaxed); }
void count_launch(unsigned n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

int* device_status_ptr() {
    int* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_device_status) != cudaSuccess) return nullptr;
    return p;
}

// ---- dispatch of the bf16 tensor-core path ----------------------------------------------------------------------
bool tc_supported(int dk, int dv) {
    return (dk == 16 || dk == 24 || dk == 32) && (dv == 32 || dv == 48 || dv == 64);
}

// Sequences of more than 256 tokens.  One launch with a block per 256-token segment reads every input once, but the
// blocks of a unit stall together while they exchange their summaries, and every block reads every other segment's
// summary: measured against the three chunk-task launches it wins for two segments, and for up to eight when all
// units are resident at once (one round); the chunk tasks take the rest.  Tests can force either.
static bool use_segments(long long units, int L, int dk, int dv) {
    if (!umma_seg_supported(dk, dv, L)) return false;
    const int pref = kernel_preference();
    if (pref == VIG_TEST_KERNEL_CHUNK_TASKS) return false;
    if (pref == VIG_TEST_KERNEL_SEGMENTS) return true;
    const int nseg = (L + 255) / 256;
    if (nseg <= 2) return true;
    if (nseg > 8) return false;
    static std::atomic<int> sms_cached{0};
    int sms = sms_cached.load(std::memory_order_relaxed);
    if (sms == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return false;
        sms_cached.store(sms, std::memory_order_relaxed);
    }
    return units * nseg <= 2LL * sms;
}

size_t tc_workspace_bytes(long long units, int L, int dk, int dv) {
    if (umma_supported(dk, dv, L)) return 0;   // one thread block covers a unit
    if (use_segments(units, L, dk, dv)) return umma_seg_workspace_bytes(units, L);
    return umma_long_workspace_bytes(units, L, dk, dv);
}

cudaError_t launch_bigla_tc(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                            const __nv_bfloat16* la_f, const __nv_bfloat16* la_b, __nv_bfloat16* out, long long units,
                            int L, int dk, int dv, void* ws, cudaStream_t stream) {
    if (umma_supported(dk, dv, L)) return launch_bigla_umma(q, k, v, la_f, la_b, out, units, L, dk, dv, 0.f, stream);
    if (use_segments(units, L, dk, dv)) return launch_bigla_umma_seg(q, k, v, la_f, la_b, out, units, L, dk, dv, ws, stream);
    return launch_bigla_umma_long(q, k, v, la_f, la_b, out, units, L, dk, dv, ws, stream);
}

// ---- scratch the library allocates itself -----------------------------------------------------------------------
// Stream-ordered allocations come from a memory pool of the library's own, one per device, whose release threshold
// keeps freed memory for the next call: with the default pool's threshold of zero every synchronisation hands the
// memory back to the driver and the next call maps it afresh (tens of microseconds per call, milliseconds for the
// buffers of the host path).  The application's default pool keeps whatever settings it was given.
static cudaMemPool_t device_pool() {
    static cudaMemPool_t pools[64] = {};
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!pools[dev]) {
        cudaMemPoolProps props = {};
        props.allocType = cudaMemAllocationTypePinned;
        props.handleTypes = cudaMemHandleTypeNone;
        props.location.type = cudaMemLocationTypeDevice;
        props.location.id = dev;
        cudaMemPool_t pool = nullptr;
        unsigned long long keep = ~0ull;
        if (cudaMemPoolCreate(&pool, &props) != cudaSuccess) return nullptr;
        if (cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &keep) != cudaSuccess) {
            cudaMemPoolDestroy(pool);
            return nullptr;
        }
        pools[dev] = pool;
    }
    return pools[dev];
}
static cudaError_t pool_alloc(void** p, size_t bytes, cudaStream_t stream) {
    cudaMemPool_t pool = device_pool();
    return pool ? cudaMallocFromPoolAsync(p, bytes, pool, stream) : cudaErrorMemoryAllocation;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Shared checks of the forward entry points.  Returns VIG_OK with *empty = true for B*H*L == 0.
static int check_fwd_args(const void* q, const void* k, const void* v, const void* la_f, const void* la_b,
                          const void* out, int B, int H, int L, int dk, int dv, bool* empty) {
    *empty = false;
    if (!q || !k || !v || !la_f || !la_b || !out) return VIG_ERR_NULL_POINTER;
    if (B < 0 || H < 0 || L < 0 || dk < 1 || dv < 1) return VIG_ERR_BAD_DIM;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(la_f) || !aligned16(la_b) || !aligned16(out))
        return VIG_ERR_MISALIGNED;
    if ((long long)B * H > 0x7fffffffLL) return VIG_ERR_UNSUPPORTED;
    if (B == 0 || H == 0 || L == 0) *empty = true;
    return VIG_OK;
}

static int fwd_bf16_impl(const void* q, const void* k, const void* v, const void* la_f, const void* la_b, void* out,
                         int B, int H, int L, int dk, int dv, void* ws, size_t ws_bytes, bool own_ws,
                         cudaStream_t stream) {
    bool empty;
    int st = check_fwd_args(q, k, v, la_f, la_b, out, B, H, L, dk, dv, &empty);
    if (st != VIG_OK) return st;
    const long long units = (long long)B * H;
    using bf = __nv_bfloat16;
    const bf *q_ = (const bf*)q, *k_ = (const bf*)k, *v_ = (const bf*)v, *f_ = (const bf*)la_f, *b_ = (const bf*)la_b;
    if (tc_supported(dk, dv) && kernel_preference() != VIG_TEST_KERNEL_SIMT) {
        const size_t need = tc_workspace_bytes(units, L, dk, dv);
        if (!own_ws && need > 0) {
            if (!ws || ws_bytes < need || (reinterpret_cast<uintptr_t>(ws) & 255u)) return VIG_ERR_WORKSPACE;
        }
        if (empty) return VIG_OK;
        void* scratch = ws;
        if (own_ws && need > 0) {
            if (pool_alloc(&scratch, need, stream) != cudaSuccess) return VIG_ERR_CUDA;
        }
        cudaError_t e = launch_bigla_tc(q_, k_, v_, f_, b_, (bf*)out, units, L, dk, dv, scratch, stream);
        if (own_ws && need > 0) {
            if (cudaFreeAsync(scratch, stream) != cudaSuccess) return VIG_ERR_CUDA;
        }
        return e == cudaSuccess ? VIG_OK : VIG_ERR_CUDA;
    }
    if (!recurrence_supported(dk, dv)) return VIG_ERR_UNSUPPORTED;
    if (empty) return VIG_OK;
    cudaError_t e = launch_recurrence<bf>(q_, k_, v_, f_, b_, (bf*)out, units, L, dk, dv, stream);
    return e == cudaSuccess ? VIG_OK : VIG_ERR_CUDA;
}

// Forward pass from the gate logits (Eq. 5 line 1 + Eq. 6).  Units of at most 256 tokens on the tensor-core shapes:
// one kernel that prepares log alpha on chip.  Everything else: gate preparation into scratch of the stream, then the
// ordinary forward pass.
// o_local != NULL: followed by the 2-D gate blend of Eq. 7 lines 3-4 as an element-wise launch over `out` (programmatic
// dependent launch: its set-up overlaps the forward kernel's tail, and it finds `out` in L2).  The blend inside the forward
// kernel's epilogue was built and measured slower than this chain: the forward kernel is bound by the dependent chain
// of a unit, two units per SM, and whatever the epilogue adds lengthens that chain.
static int fwd_gates_bf16_impl(const void* q, const void* k, const void* v, const void* g_f, const void* g_b, void* out,
                               int B, int H, int L, int dk, int dv, float tau, const void* o_local, const void* z2d,
                               cudaStream_t stream) {
    bool empty;
    int st = check_fwd_args(q, k, v, g_f, g_b, out, B, H, L, dk, dv, &empty);
    if (st != VIG_OK) return st;
    if ((o_local != nullptr) != (z2d != nullptr)) return VIG_ERR_NULL_POINTER;
    if (o_local && (!aligned16(o_local) || !aligned16(z2d))) return VIG_ERR_MISALIGNED;
    if (!(tau > 0.f) || !std::isfinite(tau)) return VIG_ERR_BAD_DIM;
    if (!tc_supported(dk, dv) && !recurrence_supported(dk, dv)) return VIG_ERR_UNSUPPORTED;
    if (empty) return VIG_OK;
    const long long units = (long long)B * H;
    using bf = __nv_bfloat16;
    if (tc_supported(dk, dv) && umma_supported(dk, dv, L) && kernel_preference() == VIG_TEST_KERNEL_AUTO) {
        cudaError_t e = launch_bigla_umma((const bf*)q, (const bf*)k, (const bf*)v, (const bf*)g_f, (const bf*)g_b, (bf*)out,
                                          units, L, dk, dv, tau, stream);
        if (e == cudaSuccess && o_local)
            e = launch_gate_blend<bf>((const bf*)o_local, (const bf*)z2d, (const bf*)out, (bf*)out, (long long)units * L * dv, stream);
        return e == cudaSuccess ? VIG_OK : VIG_ERR_CUDA;
    }
    const size_t n = (size_t)units * L * dk;
    const size_t gate_bytes = (n * sizeof(bf) + 255) / 256 * 256;
    char* la = nullptr;
    if (pool_alloc((void**)&la, 2 * gate_bytes, stream) != cudaSuccess) return VIG_ERR_CUDA;
    st = vig_gate_prep_bf16(g_f, g_b, la, la + gate_bytes, B, H, L, dk, tau, stream);
    if (st == VIG_OK) st = vig_bigla_fwd_bf16(q, k, v, la, la + gate_bytes, out, B, H, L, dk, dv, stream);
    if (cudaFreeAsync(la, stream) != cudaSuccess && st == VIG_OK) st = VIG_ERR_CUDA;
    if (st == VIG_OK && o_local &&
        launch_gate_blend<bf>((const bf*)o_local, (const bf*)z2d, (const bf*)out, (bf*)out, (long long)units * L * dv, stream) != cudaSuccess)
        st = VIG_ERR_CUDA;
    return st;
}

static int fwd_f32_impl(const void* q, const void* k, const void* v, const void* la_f, const void* la_b, void* out,
                        int B, int H, int L, int dk, int dv, cudaStream_t stream);

// Gradient of the forward pass (Eq. 6) for d_out = dLoss/d_out.  Three steps in the stream: the gates shifted by one
// token, the forward pass on (k, q, d_out) with them (= dv), the two recurrence walks for dq, dk and the gate gradients.
template <typename T>
static int bwd_impl(const void* q, const void* k, const void* v, const void* la_f, const void* la_b, const void* d_out, void* dq,
                    void* dk_out, void* dv_out, void* dla_f, void* dla_b, int B, int H, int L, int dk, int dv, cudaStream_t stream) {
    bool empty;
    int st = check_fwd_args(q, k, v, la_f, la_b, d_out, B, H, L, dk, dv, &empty);
    if (st != VIG_OK) return st;
    if (!dq || !dk_out || !dv_out || !dla_f || !dla_b) return VIG_ERR_NULL_POINTER;
    if (!aligned16(dq) || !aligned16(dk_out) || !aligned16(dv_out) || !aligned16(dla_f) || !aligned16(dla_b)) return VIG_ERR_MISALIGNED;
    if (!bwd_supported(dk, dv)) return VIG_ERR_UNSUPPORTED;
    if (sizeof(T) == 2 ? !(tc_supported(dk, dv) || recurrence_supported(dk, dv)) : !recurrence_supported(dk, dv)) return VIG_ERR_UNSUPPORTED;
    if (empty) return VIG_OK;
    const long long units = (long long)B * H;
    const size_t gate_bytes = ((size_t)units * L * dk * sizeof(T) + 255) / 256 * 256;
    char* scratch = nullptr;
    const size_t walk_bytes = bwd_scratch_bytes(units, L, dk, dv);
    if (walk_bytes == 0) return VIG_ERR_CUDA;
    if (pool_alloc((void**)&scratch, 2 * gate_bytes + walk_bytes, stream) != cudaSuccess) return VIG_ERR_CUDA;
    T *sf = (T*)scratch, *sb = (T*)(scratch + gate_bytes);
    if (launch_shift_gates<T>((const T*)la_f, (const T*)la_b, sf, sb, units, L, dk, stream) != cudaSuccess) st = VIG_ERR_CUDA;
    if (st == VIG_OK) {
        if constexpr (sizeof(T) == 2) st = fwd_bf16_impl(k, q, d_out, sf, sb, dv_out, B, H, L, dk, dv, nullptr, 0, true, stream);
        else st = fwd_f32_impl(k, q, d_out, sf, sb, dv_out, B, H, L, dk, dv, stream);
    }
    if (st == VIG_OK && launch_bigla_bwd<T>((const T*)q, (const T*)k, (const T*)v, (const T*)la_f, (const T*)la_b, (const T*)d_out, (T*)dq,
                                            (T*)dk_out, (T*)dla_f, (T*)dla_b, (float*)(scratch + 2 * gate_bytes), units, L, dk, dv,
                                            stream) != cudaSuccess)
        st = VIG_ERR_CUDA;
    if (cudaFreeAsync(scratch, stream) != cudaSuccess && st == VIG_OK) st = VIG_ERR_CUDA;
    return st;
}

template <typename T>
static int dwconv_impl(const void* x, const void* w, const void* bias, void* out, int B, int Hh, int Ww, int C, cudaStream_t stream) {
    if (!x || !w || !out) return VIG_ERR_NULL_POINTER;
    if (B < 0 || Hh < 0 || Ww < 0 || C < 1) return VIG_ERR_BAD_DIM;
    if (!aligned16(x) || !aligned16(out) || !aligned16(w) || (bias && !aligned16(bias))) return VIG_ERR_MISALIGNED;
    if (!dwconv_supported(C, sizeof(T)) || (long long)B * Hh * Ww > 0x7fffffffLL) return VIG_ERR_UNSUPPORTED;
    if (B == 0 || Hh == 0 || Ww == 0) return VIG_OK;
    return launch_dwconv3x3<T>((const T*)x, (const T*)w, (const T*)bias, (T*)out, B, Hh, Ww, C, stream) == cudaSuccess ? VIG_OK : VIG_ERR_CUDA;
}

template <typename T>
static int blend_impl(const void* o_local, const void* z, const void* o_global, void* out, long long n, cudaStream_t stream) {
    if (!o_local || !z || !o_global || !out) return VIG_ERR_NULL_POINTER;
    if (n < 0) return VIG_ERR_BAD_DIM;
    if (!aligned16(o_local) || !aligned16(z) || !aligned16(o_global) || !aligned16(out)) return VIG_ERR_MISALIGNED;
    if (n == 0) return VIG_OK;
    return launch_gate_blend<T>((const T*)o_local, (const T*)z, (const T*)o_global, (T*)out, n, stream) == cudaSuccess ? VIG_OK : VIG_ERR_CUDA;
}

static int fwd_f32_impl(const void* q, const void* k, const void* v, const void* la_f, const void* la_b, void* out,
                        int B, int H, int L, int dk, int dv, cudaStream_t stream) {
    bool empty;
    int st = check_fwd_args(q, k, v, la_f, la_b, out, B, H, L, dk, dv, &empty);
    if (st != VIG_OK) return st;
    if (!recurrence_supported(dk, dv)) return VIG_ERR_UNSUPPORTED;
    if (empty) return VIG_OK;
    cudaError_t e = launch_recurrence<float>((const float*)q, (const float*)k, (const float*)v, (const float*)la_f,
                                             (const float*)la_b, (float*)out, (long long)B * H, L, dk, dv, stream);
    return e == cudaSuccess ? VIG_OK : VIG_ERR_CUDA;
}

static int check_gate_args(const void* g_f, const void* g_b, const void* la_f, const void* la_b, int B, int H, int L,
                           int dk, float tau, bool* empty) {
    *empty = false;
    if (!g_f || !g_b || !la_f || !la_b) return VIG_ERR_NULL_POINTER;
    if (B < 0 || H < 0 || L < 0 || dk < 1 || !(tau > 0.f) || !std::isfinite(tau)) return VIG_ERR_BAD_DIM;
    if (!aligned16(g_f) || !aligned16(g_b) || !aligned16(la_f) || !aligned16(la_b)) return VIG_ERR_MISALIGNED;
    if (B == 0 || H == 0 || L == 0) *empty = true;
    return VIG_OK;
}

template <typename T>
static int gate_prep_impl(const void* g_f, const void* g_b, void* la_f, void* la_b, int B, int H, int L, int dk,
                          float tau, cudaStream_t stream) {
    bool empty;
    int st = check_gate_args(g_f, g_b, la_f, la_b, B, H, L, dk, tau, &empty);
    if (st != VIG_OK || empty) return st;
    const long long n = (long long)B * H * L * dk;
    cudaError_t e = launch_gate_prep<T>((const T*)g_f, (const T*)g_b, (T*)la_f, (T*)la_b, n, tau, stream);
    return e == cudaSuccess ? VIG_OK : VIG_ERR_CUDA;
}

template <typename T>
static int gate_prep_bwd_impl(const void* g_f, const void* g_b, const void* d_f, const void* d_b, void* o_f, void* o_b, int B, int H, int L,
                              int dk, float tau, cudaStream_t stream) {
    bool empty;
    int st = check_gate_args(g_f, g_b, o_f, o_b, B, H, L, dk, tau, &empty);
    if (st != VIG_OK) return st;
    if (!d_f || !d_b) return VIG_ERR_NULL_POINTER;
    if (!aligned16(d_f) || !aligned16(d_b)) return VIG_ERR_MISALIGNED;
    if (empty) return VIG_OK;
    const long long n = (long long)B * H * L * dk;
    cudaError_t e = launch_gate_prep_bwd<T>((const T*)g_f, (const T*)g_b, (const T*)d_f, (const T*)d_b, (T*)o_f, (T*)o_b, n, tau, stream);
    return e == cudaSuccess ? VIG_OK : VIG_ERR_CUDA;
}

// ---- host-buffer path: per device, two copy streams and the events that order them with the caller's stream -------
constexpr int kHostSlices = 4;
struct HostPath {
    std::mutex mu;
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t ev_start = nullptr, ev_done_in = nullptr, ev_done_out = nullptr, ev_in[kHostSlices] = {}, ev_k[kHostSlices] = {};
    bool ready = false;
};
static HostPath* host_path() {
    static HostPath per_device[64];
    static std::mutex init_mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    HostPath* hp = &per_device[dev];
    std::lock_guard<std::mutex> lock(init_mu);
    if (!hp->ready) {
        bool ok = cudaStreamCreateWithFlags(&hp->s_in, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&hp->s_out, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&hp->ev_start, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&hp->ev_done_in, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&hp->ev_done_out, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; ok && i < kHostSlices; ++i)
            ok = cudaEventCreateWithFlags(&hp->ev_in[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&hp->ev_k[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) return nullptr;
        hp->ready = true;
    }
    return hp;
}

}  // namespace vig

using namespace vig;

extern "C" {

int vig_bigla_fwd_bf16(const void* q, const void* k, const void* v, const void* log_alpha_fwd,
                       const void* log_alpha_bwd, void* out, int B, int H, int L, int dk, int dv, void* stream) {
    return fwd_bf16_impl(q, k, v, log_alpha_fwd, log_alpha_bwd, out, B, H, L, dk, dv, nullptr, 0, true,
                         (cudaStream_t)stream);
}

int vig_bigla_fwd(const void* q, const void* k, const void* v, const void* log_alpha_fwd, const void* log_alpha_bwd,
                  void* out, int B, int H, int L, int dk, int dv, void* stream) {
    return vig_bigla_fwd_bf16(q, k, v, log_alpha_fwd, log_alpha_bwd, out, B, H, L, dk, dv, stream);
}

int vig_bigla_fwd_f32(const void* q, const void* k, const void* v, const void* log_alpha_fwd,
                      const void* log_alpha_bwd, void* out, int B, int H, int L, int dk, int dv, void* stream) {
    return fwd_f32_impl(q, k, v, log_alpha_fwd, log_alpha_bwd, out, B, H, L, dk, dv, (cudaStream_t)stream);
}

int vig_bigla_fwd_gates_bf16(const void* q, const void* k, const void* v, const void* g_fwd, const void* g_bwd, void* out,
                             int B, int H, int L, int dk, int dv, float tau, void* stream) {
    return fwd_gates_bf16_impl(q, k, v, g_fwd, g_bwd, out, B, H, L, dk, dv, tau, nullptr, nullptr, (cudaStream_t)stream);
}

int vig_bigla_fwd_blend_bf16(const void* q, const void* k, const void* v, const void* g_fwd, const void* g_bwd,
                             const void* o_local, const void* gate2d_logits, void* out, int B, int H, int L, int dk, int dv,
                             float tau, void* stream) {
    if (!o_local || !gate2d_logits) return VIG_ERR_NULL_POINTER;
    return fwd_gates_bf16_impl(q, k, v, g_fwd, g_bwd, out, B, H, L, dk, dv, tau, o_local, gate2d_logits, (cudaStream_t)stream);
}

int vig_bigla_bwd_bf16(const void* q, const void* k, const void* v, const void* log_alpha_fwd, const void* log_alpha_bwd,
                       const void* d_out, void* dq, void* dk_out, void* dv_out, void* dlog_alpha_fwd, void* dlog_alpha_bwd, int B, int H,
                       int L, int dk, int dv, void* stream) {
    return bwd_impl<__nv_bfloat16>(q, k, v, log_alpha_fwd, log_alpha_bwd, d_out, dq, dk_out, dv_out, dlog_alpha_fwd, dlog_alpha_bwd, B, H, L,
                                   dk, dv, (cudaStream_t)stream);
}
int vig_bigla_bwd_f32(const void* q, const void* k, const void* v, const void* log_alpha_fwd, const void* log_alpha_bwd,
                      const void* d_out, void* dq, void* dk_out, void* dv_out, void* dlog_alpha_fwd, void* dlog_alpha_bwd, int B, int H,
                      int L, int dk, int dv, void* stream) {
    return bwd_impl<float>(q, k, v, log_alpha_fwd, log_alpha_bwd, d_out, dq, dk_out, dv_out, dlog_alpha_fwd, dlog_alpha_bwd, B, H, L, dk, dv,
                           (cudaStream_t)stream);
}

int vig_dwconv3x3_bf16(const void* x, const void* w, const void* bias, void* out, int B, int Hh, int Ww, int C, void* stream) {
    return dwconv_impl<__nv_bfloat16>(x, w, bias, out, B, Hh, Ww, C, (cudaStream_t)stream);
}
int vig_dwconv3x3_f32(const void* x, const void* w, const void* bias, void* out, int B, int Hh, int Ww, int C, void* stream) {
    return dwconv_impl<float>(x, w, bias, out, B, Hh, Ww, C, (cudaStream_t)stream);
}
int vig_gate_blend_bf16(const void* o_local, const void* gate2d_logits, const void* o_global, void* out, long long n, void* stream) {
    return blend_impl<__nv_bfloat16>(o_local, gate2d_logits, o_global, out, n, (cudaStream_t)stream);
}
int vig_gate_blend_f32(const void* o_local, const void* gate2d_logits, const void* o_global, void* out, long long n, void* stream) {
    return blend_impl<float>(o_local, gate2d_logits, o_global, out, n, (cudaStream_t)stream);
}

size_t vig_bigla_workspace_bytes(int B, int H, int L, int dk, int dv, int dtype) {
    if (B <= 0 || H <= 0 || L <= 0 || dk < 1 || dv < 1 || dtype != VIG_DTYPE_BF16) return 0;
    if (!tc_supported(dk, dv)) return 0;
    return tc_workspace_bytes((long long)B * H, L, dk, dv);
}

int vig_bigla_fwd_ws_bf16(const void* q, const void* k, const void* v, const void* log_alpha_fwd,
                          const void* log_alpha_bwd, void* out, int B, int H, int L, int dk, int dv, void* ws,
                          size_t ws_bytes, void* stream) {
    return fwd_bf16_impl(q, k, v, log_alpha_fwd, log_alpha_bwd, out, B, H, L, dk, dv, ws, ws_bytes, false,
                         (cudaStream_t)stream);
}

int vig_gate_prep_bf16(const void* g_fwd, const void* g_bwd, void* log_alpha_fwd, void* log_alpha_bwd, int B, int H,
                       int L, int dk, float tau, void* stream) {
    return gate_prep_impl<__nv_bfloat16>(g_fwd, g_bwd, log_alpha_fwd, log_alpha_bwd, B, H, L, dk, tau,
                                         (cudaStream_t)stream);
}

int vig_gate_prep_f32(const void* g_fwd, const void* g_bwd, void* log_alpha_fwd, void* log_alpha_bwd, int B, int H,
                      int L, int dk, float tau, void* stream) {
    return gate_prep_impl<float>(g_fwd, g_bwd, log_alpha_fwd, log_alpha_bwd, B, H, L, dk, tau, (cudaStream_t)stream);
}

int vig_gate_prep_bwd_bf16(const void* g_fwd, const void* g_bwd, const void* dlog_alpha_fwd, const void* dlog_alpha_bwd, void* dg_fwd,
                           void* dg_bwd, int B, int H, int L, int dk, float tau, void* stream) {
    return gate_prep_bwd_impl<__nv_bfloat16>(g_fwd, g_bwd, dlog_alpha_fwd, dlog_alpha_bwd, dg_fwd, dg_bwd, B, H, L, dk, tau, (cudaStream_t)stream);
}

int vig_gate_prep_bwd_f32(const void* g_fwd, const void* g_bwd, const void* dlog_alpha_fwd, const void* dlog_alpha_bwd, void* dg_fwd,
                          void* dg_bwd, int B, int H, int L, int dk, float tau, void* stream) {
    return gate_prep_bwd_impl<float>(g_fwd, g_bwd, dlog_alpha_fwd, dlog_alpha_bwd, dg_fwd, dg_bwd, B, H, L, dk, tau, (cudaStream_t)stream);
}

int vig_bigla_fwd_host(const void* q, const void* k, const void* v, const void* g_fwd, const void* g_bwd, void* out,
                       int B, int H, int L, int dk, int dv, float tau, int dtype, void* stream_) {
    cudaStream_t stream = (cudaStream_t)stream_;
    if (!q || !k || !v || !g_fwd || !g_bwd || !out) return VIG_ERR_NULL_POINTER;
    if (B < 0 || H < 0 || L < 0 || dk < 1 || dv < 1 || !(tau > 0.f) || !std::isfinite(tau)) return VIG_ERR_BAD_DIM;
    if (dtype != VIG_DTYPE_F32 && dtype != VIG_DTYPE_BF16) return VIG_ERR_UNSUPPORTED;
    if (dtype == VIG_DTYPE_F32 ? !recurrence_supported(dk, dv) : !(tc_supported(dk, dv) || recurrence_supported(dk, dv)))
        return VIG_ERR_UNSUPPORTED;
    if ((long long)B * H > 0x7fffffffLL) return VIG_ERR_UNSUPPORTED;
    if (B == 0 || H == 0 || L == 0) return VIG_OK;
    HostPath* hp = host_path();
    if (!hp) return VIG_ERR_CUDA;
    std::lock_guard<std::mutex> lock(hp->mu);   // the streams and events of the device serve one host call at a time
    const size_t es = dtype == VIG_DTYPE_F32 ? 4 : 2;
    const long long units = (long long)B * H;
    const size_t unit_k = (size_t)L * dk * es, unit_v = (size_t)L * dv * es;
    // every slab is rounded up to 256 bytes so that all device pointers stay aligned
    const size_t nk = (units * unit_k + 255) / 256 * 256, nv = (units * unit_v + 255) / 256 * 256;
    char* base = nullptr;
    if (pool_alloc((void**)&base, 4 * nk + 2 * nv, stream) != cudaSuccess) return VIG_ERR_CUDA;
    char *dq = base, *dk_ = base + nk, *dgf = base + 2 * nk, *dgb = base + 3 * nk, *dv_ = base + 4 * nk,
         *dout = base + 4 * nk + nv;
    // Slices of whole units: the copy of slice i + 1 to the device, the kernels of slice i and the copy of slice i - 1
    // back run at the same time (the host link carries both directions at once).  A slice offset must keep the 16-byte
    // alignment of the device pointers: unit sizes are multiples of 16 bytes whenever dk and dv are multiples of
    // 8 (bf16) or 4 (fp32); otherwise the call runs as one slice.
    int nsl = (unit_k % 16 == 0 && unit_v % 16 == 0 && units * (4 * unit_k + 2 * unit_v) >= (4u << 20)) ? kHostSlices : 1;
    if (nsl > units) nsl = (int)units;
    int st = VIG_OK;
    bool ok = cudaEventRecord(hp->ev_start, stream) == cudaSuccess &&
              cudaStreamWaitEvent(hp->s_in, hp->ev_start, 0) == cudaSuccess &&
              cudaStreamWaitEvent(hp->s_out, hp->ev_start, 0) == cudaSuccess;
    for (int i = 0; ok && i < nsl && st == VIG_OK; ++i) {
        const long long u0 = units * i / nsl, u1 = units * (i + 1) / nsl, nu = u1 - u0;
        const size_t ok_ = (size_t)u0 * unit_k, ov = (size_t)u0 * unit_v;
        ok = cudaMemcpyAsync(dgf + ok_, (const char*)g_fwd + ok_, nu * unit_k, cudaMemcpyHostToDevice, hp->s_in) == cudaSuccess &&
             cudaMemcpyAsync(dgb + ok_, (const char*)g_bwd + ok_, nu * unit_k, cudaMemcpyHostToDevice, hp->s_in) == cudaSuccess &&
             cudaMemcpyAsync(dq + ok_, (const char*)q + ok_, nu * unit_k, cudaMemcpyHostToDevice, hp->s_in) == cudaSuccess &&
             cudaMemcpyAsync(dk_ + ok_, (const char*)k + ok_, nu * unit_k, cudaMemcpyHostToDevice, hp->s_in) == cudaSuccess &&
             cudaMemcpyAsync(dv_ + ov, (const char*)v + ov, nu * unit_v, cudaMemcpyHostToDevice, hp->s_in) == cudaSuccess &&
             cudaEventRecord(hp->ev_in[i], hp->s_in) == cudaSuccess && cudaStreamWaitEvent(stream, hp->ev_in[i], 0) == cudaSuccess;
        if (!ok) break;
        if (dtype == VIG_DTYPE_F32) {
            st = vig_gate_prep_f32(dgf + ok_, dgb + ok_, dgf + ok_, dgb + ok_, (int)nu, 1, L, dk, tau, stream_);
            if (st == VIG_OK) st = vig_bigla_fwd_f32(dq + ok_, dk_ + ok_, dv_ + ov, dgf + ok_, dgb + ok_, dout + ov, (int)nu, 1, L, dk, dv, stream_);
        } else {
            st = vig_bigla_fwd_gates_bf16(dq + ok_, dk_ + ok_, dv_ + ov, dgf + ok_, dgb + ok_, dout + ov, (int)nu, 1, L, dk, dv, tau, stream_);
        }
        if (st != VIG_OK) break;
        ok = cudaEventRecord(hp->ev_k[i], stream) == cudaSuccess && cudaStreamWaitEvent(hp->s_out, hp->ev_k[i], 0) == cudaSuccess &&
             cudaMemcpyAsync((char*)out + ov, dout + ov, nu * unit_v, cudaMemcpyDeviceToHost, hp->s_out) == cudaSuccess;
    }
    // the caller's stream takes over again once both copy streams have drained (also after an error, so that the
    // buffer is not freed under a copy in flight)
    ok = (cudaEventRecord(hp->ev_done_in, hp->s_in) == cudaSuccess) & (cudaEventRecord(hp->ev_done_out, hp->s_out) == cudaSuccess) &
         (cudaStreamWaitEvent(stream, hp->ev_done_in, 0) == cudaSuccess) & (cudaStreamWaitEvent(stream, hp->ev_done_out, 0) == cudaSuccess) & ok;
    if (!ok && st == VIG_OK) st = VIG_ERR_CUDA;
    if (cudaFreeAsync(base, stream) != cudaSuccess && st == VIG_OK) st = VIG_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess && st == VIG_OK) st = VIG_ERR_CUDA;
    return st;
}

const char* vig_status_string(int status) {
    switch (status) {
        case VIG_OK: return "ok";
        case VIG_ERR_NULL_POINTER: return "a required pointer is NULL";
        case VIG_ERR_BAD_DIM: return "invalid size (negative dimension, dk or dv < 1, or tau not positive and finite)";
        case VIG_ERR_UNSUPPORTED: return "shape or dtype outside the supported set";
        case VIG_ERR_MISALIGNED: return "a pointer is not 16-byte aligned";
        case VIG_ERR_CUDA: return "a CUDA runtime call or kernel launch failed";
        case VIG_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case VIG_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
        default: return "unknown status";
    }
}

int vig_last_device_status(void* stream) {
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return VIG_ERR_CUDA;
    int word = 0;
    if (cudaMemcpyFromSymbol(&word, g_device_status, sizeof(int), 0) != cudaSuccess) return VIG_ERR_CUDA;
    if (word != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int), 0) != cudaSuccess) return VIG_ERR_CUDA;
    }
    if (word & kDevStatusInternal) return VIG_ERR_CUDA;
    return (word & kDevStatusTimeout) ? VIG_ERR_DEVICE_TIMEOUT : VIG_OK;
}

int vig_test_set_kernel_preference(int preference) {
    if (preference != VIG_TEST_KERNEL_AUTO && preference != VIG_TEST_KERNEL_SIMT && preference != VIG_TEST_KERNEL_CHUNK_TASKS &&
        preference != VIG_TEST_KERNEL_SEGMENTS)
        return VIG_ERR_UNSUPPORTED;
    g_kernel_pref.store(preference, std::memory_order_relaxed);
    return VIG_OK;
}

int vig_test_take_fallback_count(void* stream) {
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return VIG_ERR_CUDA;
    int n = 0;
    const int zero = 0;
    if (cudaMemcpyFromSymbol(&n, g_device_status, sizeof(int), sizeof(int)) != cudaSuccess ||
        cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int), sizeof(int)) != cudaSuccess)
        return VIG_ERR_CUDA;
    return n;
}

void vig_test_expire_next_wait(void) { g_expire_next_wait.store(1, std::memory_order_relaxed); }

unsigned long long vig_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
