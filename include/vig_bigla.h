/*
 * vig_bigla.h -- C ABI of the B200 (sm_100a) BiGLA forward library.
 *
 * BiGLA is the bidirectional gated-linear-attention token mixer of ViG
 * (arXiv 2405.18425, Sec. 4.2.1, Eq. 6).  For every (batch, head) unit, with
 * zero initial states,
 *
 *     S>_t = diag(alpha>_t) S>_{t-1} + k_t^T v_t        (t = 1 .. L)
 *     S<_t = diag(alpha<_t) S<_{t+1} + k_t^T v_t        (t = L .. 1)
 *     out_t = ( q_t S>_t + q_t S<_t ) / 2
 *
 * where S is dk x dv and the gate alpha_t in (0,1]^dk scales the rows of S
 * (G_t = alpha_t^T 1, Eq. 5).  Gates are passed as natural logarithms,
 * log alpha = logsigmoid(g) / tau (Eq. 5 line 1 / Eq. 6 line 1, tau = 16 in the
 * paper), which vig_gate_prep_* computes from the gate logits g.
 *
 * Conventions shared by every entry point
 *   - All tensors are dense, row-major [B, H, L, d] (d = dk for q, k, g and
 *     log alpha; d = dv for v and out): each (b, h) unit owns one contiguous
 *     [L, d] slab.  Flattening the H x W patch grid to L is the caller's job.
 *   - One element type per call for every tensor: bfloat16 (entry points named
 *     *_bf16) or float (entry points named *_f32).  Accumulation is fp32.
 *   - Unless a name says "host", every pointer is a DEVICE pointer, 16-byte
 *     aligned, owned by the caller.  Inputs are never written; `out` is fully
 *     overwritten.  q is used as given (no dk^-0.5 inside).
 *   - Domain of log alpha: finite and <= 0.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Device entry points enqueue work on it and return without
 *     synchronising.  The device of the current CUDA context must own the
 *     buffers.
 *   - Every entry point returns a vig_status.  Arguments are validated before
 *     anything is launched; an invalid call launches nothing.  B, H or L equal
 *     to 0 is a valid empty call (VIG_OK, nothing launched).
 *   - No entry point throws, prints, or falls back to the CPU.
 */
#ifndef VIG_BIGLA_H
#define VIG_BIGLA_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum vig_status {
    VIG_OK = 0,
    VIG_ERR_NULL_POINTER = -1,   /* a required pointer is NULL                                 */
    VIG_ERR_BAD_DIM = -2,        /* a negative size, dk or dv < 1, tau <= 0 or not finite      */
    VIG_ERR_UNSUPPORTED = -3,    /* dk / dv / size outside the supported set (see each call)   */
    VIG_ERR_MISALIGNED = -4,     /* a pointer is not 16-byte aligned                            */
    VIG_ERR_CUDA = -5,           /* a CUDA runtime call or launch failed                        */
    VIG_ERR_WORKSPACE = -6,      /* caller-provided workspace missing or too small              */
    VIG_ERR_DEVICE_TIMEOUT = -7  /* a bounded device-side wait gave up (see vig_last_device_status) */
} vig_status;

typedef enum vig_dtype { VIG_DTYPE_F32 = 0, VIG_DTYPE_BF16 = 1 } vig_dtype;

/* ---- BiGLA forward (Eq. 6), device buffers ---------------------------------------------------
 * q, k, log_alpha_fwd, log_alpha_bwd: [B,H,L,dk];  v, out: [B,H,L,dv].
 *
 * bf16: dk in {16, 24, 32} with dv in {32, 48, 64} run on the tensor-core kernels; any other
 *       dk <= 128, dv <= 256 runs on the fp32 SIMT recurrence kernel (slow, same result
 *       contract).  Tensor-core operands are bf16 with fp32 accumulation; states that cross
 *       a 128-token chunk are rounded to bf16 as tensor-core operands.  A unit whose gates decay
 *       by more than e^-60 inside one chunk of 128 tokens is computed by an in-kernel fp32
 *       recurrence (Eq. 6 step by step) instead of the factorised tiles.
 * f32:  dk <= 128, dv <= 256; fp32 SIMT recurrence, meant for validation-sized inputs.
 * Sequences of at most 256 tokens run in one launch with a unit per thread block and use no scratch.
 * Longer ones are cut into 256-token segments (one launch; the blocks of a unit exchange segment
 * summaries through scratch) or into 128-token chunk tasks (three launches; chunk summaries and
 * boundary states go through scratch), whichever suits the shape.  The library allocates and frees
 * that scratch on `stream` from a stream-ordered memory pool of its own (one per device, which keeps
 * freed memory for later calls instead of returning it to the driver); use the *_ws form to supply it.  The kernels are
 * launched with programmatic stream serialization: each waits for the work before it in `stream`
 * before it reads its inputs.
 * Errors: NULL_POINTER, BAD_DIM, UNSUPPORTED, MISALIGNED, CUDA. */
int vig_bigla_fwd_bf16(const void* q, const void* k, const void* v,
                       const void* log_alpha_fwd, const void* log_alpha_bwd, void* out,
                       int B, int H, int L, int dk, int dv, void* stream);
int vig_bigla_fwd_f32(const void* q, const void* k, const void* v,
                      const void* log_alpha_fwd, const void* log_alpha_bwd, void* out,
                      int B, int H, int L, int dk, int dv, void* stream);
/* Same call as vig_bigla_fwd_bf16 (bf16 in, fp32 accumulate, bf16 out). */
int vig_bigla_fwd(const void* q, const void* k, const void* v,
                  const void* log_alpha_fwd, const void* log_alpha_bwd, void* out,
                  int B, int H, int L, int dk, int dv, void* stream);

/* Bytes of device scratch a vig_bigla_fwd_* call of this shape needs (0 when the whole sequence
 * of a unit is handled by one thread block).  Returns 0 for invalid or unsupported shapes too. */
size_t vig_bigla_workspace_bytes(int B, int H, int L, int dk, int dv, int dtype);
/* vig_bigla_fwd_bf16 with caller-owned scratch: `ws` is a 256-byte aligned device buffer of at
 * least vig_bigla_workspace_bytes(...) bytes (may be NULL when that is 0).  Nothing is allocated.
 * Calls that share one `ws` must not overlap on the GPU.  Extra error: WORKSPACE. */
int vig_bigla_fwd_ws_bf16(const void* q, const void* k, const void* v,
                          const void* log_alpha_fwd, const void* log_alpha_bwd, void* out,
                          int B, int H, int L, int dk, int dv,
                          void* ws, size_t ws_bytes, void* stream);

/* vig_bigla_fwd_bf16 for callers that cannot allocate device memory (the paper has no counterpart;
 * this is a library convenience).  Some users of this code run where cudaMalloc is off limits at call
 * time: a serving loop whose memory budget was fixed at start-up, a process that shares the GPU under
 * a hard partition where a late allocation can fail or stall every stream, or an embedding
 * application that simply hands the library no allocator.  The other entry points either allocate
 * scratch on the stream or need a caller-made workspace; this one does neither.  Its scratch is a
 * fixed VIG_STATIC_SCRATCH_BYTES array inside the library's device image, which every GPU that loads
 * the library holds until the process exits.
 *   - Only the tensor-core shapes (dk in {16,24,32}, dv in {32,48,64}); otherwise UNSUPPORTED.
 *   - A problem whose scratch need (vig_bigla_workspace_bytes) exceeds VIG_STATIC_SCRATCH_BYTES is
 *     rejected with VIG_ERR_WORKSPACE and nothing is launched; use vig_bigla_fwd_ws_bf16 for it.
 *   - No cudaMalloc, cudaFree or other allocating call is made, by this entry point or beneath it.
 *   - The first call on each device looks up the array's device address (a one-time set-up step for
 *     that device, which also makes the runtime load the library's device image, the array included,
 *     if it has not yet); make that first call with the device current and before starting any stream
 *     capture.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left in it.
 *     Nothing in it has to start at zero: every word a call reads to form its result was written
 *     earlier in the same call.  Two calls that overlap on the GPU (different streams, no ordering
 *     between them) race on it and give undefined results: order them.
 * Same kernels and results as vig_bigla_fwd_ws_bf16 with a workspace of that size.  Errors: NULL_POINTER, BAD_DIM, MISALIGNED, UNSUPPORTED,
 * WORKSPACE, CUDA. */
#define VIG_STATIC_SCRATCH_BYTES (24u * 1024u * 1024u)
int vig_bigla_fwd_static_bf16(const void* q, const void* k, const void* v,
                              const void* log_alpha_fwd, const void* log_alpha_bwd, void* out,
                              int B, int H, int L, int dk, int dv, void* stream);

/* ---- Gate preparation (Eq. 5 line 1 / Eq. 6 lines 1-2 after the projection) ---------------------
 * log_alpha_x = logsigmoid(g_x) / tau for both directions, element-wise, evaluated in fp32 as
 * (min(g,0) - log1p(exp(-|g|))) / tau and rounded to the element type (the bf16 entry point takes exp
 * and log from the special-function unit: relative error below 2e-5 before the rounding).  g_*, log_alpha_*:
 * [B,H,L,dk]; any dk >= 1; tau > 0.  In-place (log_alpha_x == g_x) is allowed.
 * Errors: NULL_POINTER, BAD_DIM, MISALIGNED, CUDA. */
int vig_gate_prep_bf16(const void* g_fwd, const void* g_bwd,
                       void* log_alpha_fwd, void* log_alpha_bwd,
                       int B, int H, int L, int dk, float tau, void* stream);
int vig_gate_prep_f32(const void* g_fwd, const void* g_bwd,
                      void* log_alpha_fwd, void* log_alpha_bwd,
                      int B, int H, int L, int dk, float tau, void* stream);

/* ---- Gate preparation fused into the forward pass (Eq. 5 line 1 / Eq. 6 lines 1-2, then Eq. 6) ------------
 * out = BiGLA(q, k, v, logsigmoid(g_fwd) / tau, logsigmoid(g_bwd) / tau): the same result contract as
 * vig_gate_prep_bf16 followed by vig_bigla_fwd_bf16, without the round trip of log alpha through device
 * memory.  g_fwd, g_bwd: [B,H,L,dk] gate logits (read only); tau > 0.
 * Units of at most 256 tokens with dk in {16,24,32}, dv in {32,48,64} run in one kernel that turns each gate
 * tile into log alpha in shared memory (fp32 evaluation with exp and log from the special-function unit,
 * rounded to bf16 as the tensor-core operand of the prefix sums: the same rounding point as the un-fused
 * chain).  Longer sequences and other head sizes run gate preparation into scratch the library allocates and
 * frees on `stream` (its memory pool), then the ordinary forward pass.
 * Errors: NULL_POINTER, BAD_DIM (also tau), UNSUPPORTED, MISALIGNED, CUDA. */
int vig_bigla_fwd_gates_bf16(const void* q, const void* k, const void* v,
                             const void* g_fwd, const void* g_bwd, void* out,
                             int B, int H, int L, int dk, int dv, float tau, void* stream);

/* ---- 2-D gating locality injection around the mixer (Eq. 7) ------------------------------------------------
 * Eq. 7:  O_local = DWConv3x3(X);  O_global = BiGLA(O_local);  G_2D = sigmoid(O_local W + b);
 *         O = G_2D * O_local + (1 - G_2D) * O_global.
 * The dense projections (q, k, v, the gate logits, O_local W + b) are ordinary matrix products outside this
 * library; it provides line 1, the blend of lines 3-4 on its own, and the blend fused into the forward pass.
 *
 * vig_dwconv3x3_*: depth-wise 3 x 3 convolution over the patch grid (Eq. 7 line 1), stride 1, zero padding 1,
 * cross-correlation (the convention of deep-learning convolutions: w[c][0][1] weighs the pixel above).
 * x, out: [B, Hh, Ww, C] channels last (the mixer's sequence is the row-major Hh x Ww grid); w: [C, 3, 3];
 * bias: [C] or NULL; all of the call's element type and 16-byte aligned; fp32 accumulation.  C must be a multiple of
 * 8 (bf16) or 4 (fp32), at most 2^20.  x and out must not overlap.  The input tiles (with the padding, which reads
 * outside the image supply as zeros) come by tiled TMA loads; a load that never completes ends the kernel's bounded
 * wait and shows up as VIG_ERR_DEVICE_TIMEOUT in vig_last_device_status.
 * Errors: NULL_POINTER, BAD_DIM, MISALIGNED, UNSUPPORTED, CUDA. */
int vig_dwconv3x3_bf16(const void* x, const void* w, const void* bias, void* out,
                       int B, int Hh, int Ww, int C, void* stream);
int vig_dwconv3x3_f32(const void* x, const void* w, const void* bias, void* out,
                      int B, int Hh, int Ww, int C, void* stream);
/* vig_gate_blend_*: out = G * o_local + (1 - G) * o_global with G = sigmoid(gate2d_logits), element-wise over n
 * elements (Eq. 7 lines 3-4 with the logits O_local W + b given), evaluated in fp32.  out may be o_global.
 * Errors: NULL_POINTER, BAD_DIM, MISALIGNED, CUDA. */
int vig_gate_blend_bf16(const void* o_local, const void* gate2d_logits, const void* o_global, void* out,
                        long long n, void* stream);
int vig_gate_blend_f32(const void* o_local, const void* gate2d_logits, const void* o_global, void* out,
                       long long n, void* stream);
/* vig_bigla_fwd_blend_bf16: vig_bigla_fwd_gates_bf16 followed by the blend, in one call (Eq. 5 line 1, Eq. 6 and
 * Eq. 7 lines 3-4): out = G * o_local + (1 - G) * BiGLA(q, k, v, logsigmoid(g_fwd)/tau, logsigmoid(g_bwd)/tau).
 * o_local, gate2d_logits: [B,H,L,dv] like out (the caller lays the channels of O_local and of O_local W + b out per
 * head).  The blend runs as an element-wise launch over `out` behind the forward launch(es), in the same stream (it finds
 * `out` in L2; sigmoid in fp32).  Errors: as vig_bigla_fwd_gates_bf16. */
int vig_bigla_fwd_blend_bf16(const void* q, const void* k, const void* v,
                             const void* g_fwd, const void* g_bwd,
                             const void* o_local, const void* gate2d_logits, void* out,
                             int B, int H, int L, int dk, int dv, float tau, void* stream);

/* ---- Gradient of the forward pass ------------------------------------------------------------------------------
 * The paper trains with the layer of Eq. 6 (its Appendix C gives the recipe) without describing the gradient; this is
 * the reverse-mode adjoint of Eq. 6 as it stands.  For d_out = dLoss/d_out [B,H,L,dv] the call writes
 *   dq, dk_out [B,H,L,dk], dv_out [B,H,L,dv], dlog_alpha_fwd, dlog_alpha_bwd [B,H,L,dk]
 * (gradients with respect to the LOG gates as passed to the forward call; a caller that feeds gate logits g chains
 * them through vig_gate_prep_bwd_* below).  All device pointers of the call's element type, contiguous,
 * 16-byte aligned; inputs are not written; outputs must not overlap inputs or one another.
 * How: dv is the forward pass itself on (k, q, d_out) with the gates moved by one token (the tensor-core kernels for
 * the bf16 head sizes they cover); dq, dk and the gate gradients come from two fp32 walks over the sequence per unit
 * on the CUDA cores (states in registers), with the gate gradients as running sums of q * dq - k * dk per direction.
 * Calls with few units and long sequences (fewer than two units per SM, 128 tokens or more) cut every sequence into
 * segments that are walked in parallel: a first launch finds what each segment adds to the four states, a fold carries
 * the states across segments, the walks start from them, and a last launch adds the later segments' sums to the gate
 * gradients (vig_t-like 1024 x 1024 inputs, 32 units of 4096 tokens: 2.19 ms -> 0.55 ms).
 * Scratch (the moved gates, 8 L dk bytes per unit of partial results, the segments' states) comes from the library's
 * pool, stream-ordered.
 * Head sizes: dk <= 128, dv <= 128, and whatever the forward entry point of the same type takes.
 * Errors: NULL_POINTER, BAD_DIM, MISALIGNED, UNSUPPORTED, CUDA. */
int vig_bigla_bwd_bf16(const void* q, const void* k, const void* v,
                       const void* log_alpha_fwd, const void* log_alpha_bwd, const void* d_out,
                       void* dq, void* dk_out, void* dv_out, void* dlog_alpha_fwd, void* dlog_alpha_bwd,
                       int B, int H, int L, int dk, int dv, void* stream);
int vig_bigla_bwd_f32(const void* q, const void* k, const void* v,
                      const void* log_alpha_fwd, const void* log_alpha_bwd, const void* d_out,
                      void* dq, void* dk_out, void* dv_out, void* dlog_alpha_fwd, void* dlog_alpha_bwd,
                      int B, int H, int L, int dk, int dv, void* stream);

/* vig_gate_prep_bwd_*: the gradient through the gate preparation (Eq. 5 line 1), for callers whose parameters sit
 * behind the gate logits: dg = dlog_alpha * sigmoid(-g) / tau (d/dg log sigmoid(g) = 1 - sigmoid(g)), both directions
 * in one launch, fp32 arithmetic.  g_*, dlog_alpha_*, dg_*: [B,H,L,dk] of the call's element type, 16-byte aligned;
 * dg_* may be the dlog_alpha_* buffers (in place).  Errors: NULL_POINTER, BAD_DIM, MISALIGNED, CUDA. */
int vig_gate_prep_bwd_bf16(const void* g_fwd, const void* g_bwd, const void* dlog_alpha_fwd, const void* dlog_alpha_bwd,
                           void* dg_fwd, void* dg_bwd, int B, int H, int L, int dk, float tau, void* stream);
int vig_gate_prep_bwd_f32(const void* g_fwd, const void* g_bwd, const void* dlog_alpha_fwd, const void* dlog_alpha_bwd,
                          void* dg_fwd, void* dg_bwd, int B, int H, int L, int dk, float tau, void* stream);

/* ---- Whole path on HOST buffers -------------------------------------------------------------------
 * Gate preparation followed by the BiGLA forward (Eq. 5 line 1 + Eq. 6) for callers whose data
 * lives in host memory.  All seven pointers are HOST pointers (pinned memory makes the copies
 * asynchronous and faster; pageable memory works).  The call takes device buffers from the library's
 * memory pool on `stream`, cuts the batch into slices of whole units and runs, on two internal copy
 * streams ordered with `stream` by events, the copy of one slice to the device, the kernels of the
 * slice before it (vig_bigla_fwd_gates_bf16, or the two fp32 calls) and the copy of the slice before
 * that back to `out` at the same time; it returns the device memory to the pool and synchronises
 * `stream` before returning, so `out` is valid on return.  Results are those of the device entry
 * points, bit for bit.  Host calls on one device are serialised.
 * `dtype` is a vig_dtype.  Errors: as the device calls, plus CUDA for allocation failures. */
int vig_bigla_fwd_host(const void* q, const void* k, const void* v,
                       const void* g_fwd, const void* g_bwd, void* out,
                       int B, int H, int L, int dk, int dv, float tau, int dtype, void* stream);

/* ---- Diagnostics ---------------------------------------------------------------------------------- */
/* Static, NUL-terminated description of a vig_status value. */
const char* vig_status_string(int status);
/* Synchronises `stream`, then reads and clears the device status word of the current device.
 * Returns VIG_OK, VIG_ERR_DEVICE_TIMEOUT if a kernel's bounded wait on an asynchronous copy or on a
 * tensor-core batch expired (the output of that call is then undefined), or VIG_ERR_CUDA. */
int vig_last_device_status(void* stream);
/* Number of kernels this library has launched in this process so far (all devices, all streams). */
unsigned long long vig_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* VIG_BIGLA_H */
