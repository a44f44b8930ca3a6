/*
 * pq.h -- C ABI of the B200 (sm_100a) quantized linear layer: W8A8 and W4A8.
 *
 * The library implements the quantized linear operator of a decoder LLM as the
 * paper's "Unified low-bit inference framework" section states it: activations are
 * quantized per token to INT8, multiplied with INT8 (or packed INT4) weights in
 * integer arithmetic, and the INT32 result is dequantized to FP16.  The quantizer is
 * the paper's Eq. 1-2 with symmetric scaling (no zero point).
 *
 * Conventions for every call
 *   - All data pointers are DEVICE pointers owned by the caller, 16-byte aligned.
 *     The library allocates and frees no device memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Calls are asynchronous and stream-ordered; none synchronizes the device.
 *   - The kernels are launched with programmatic stream serialization: a call may begin its
 *     set-up while the kernel before it in the stream drains, and waits for that kernel's
 *     completion before it reads activations, codes or token scales and before it writes.
 *     Packed weights and weight scales are treated as constants of the model and may be
 *     read ahead of that wait: they must be complete before the operation that directly
 *     precedes the GEMM call in the stream begins.  pq_pack_w8 / pq_pack_w4 guarantee this
 *     for GEMM calls that follow them; a caller that writes weight buffers by other means
 *     puts any stream operation (or a synchronization) between that write and the GEMM.
 *   - Matrices are dense row-major: X/Q/Y have one token per row, W has one output
 *     channel per row (K contiguous).
 *   - The return value is a pq_status.  Argument errors are detected before anything
 *     is launched.  Nothing aborts, throws or traps; non-finite inputs are memory
 *     safe with unspecified results.
 *   - Every wait inside a kernel is bounded; if one expires the kernel records
 *     PQ_ERR_TIMEOUT in a device status word, waits (bounded) for the copies and MMAs it has
 *     in flight, and returns; the outputs of that call are then unspecified.
 *     pq_device_status() reads that word.
 *   - The library keeps no per-call state on the host: calls may be made from several host
 *     threads and on several streams at once.  The only memory a call shares with other calls
 *     is what the caller passes in (see `workspace` below).
 *   - Requires compute capability 10.0; anything else returns PQ_ERR_ARCH (there is
 *     no fallback path).
 */
#ifndef PQ_H_
#define PQ_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define PQ_API __attribute__((visibility("default")))
#else
#define PQ_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  PQ_OK = 0,
  PQ_ERR_NULL = 1,    /* a required pointer is NULL */
  PQ_ERR_SHAPE = 2,   /* a size is non-positive or violates a divisibility rule */
  PQ_ERR_ALIGN = 3,   /* a pointer is not 16-byte aligned */
  PQ_ERR_ARCH = 4,    /* the current device is not compute capability 10.0 */
  PQ_ERR_CUDA = 5,    /* a CUDA runtime/driver call or a launch failed */
  PQ_ERR_TIMEOUT = 6, /* a bounded wait inside a kernel expired (device status word) */
  PQ_ERR_LIMIT = 7    /* a size exceeds a stated maximum of the entry point */
} pq_status;

/* Static string for a status code. */
PQ_API const char* pq_status_str(int status);

/* Name of the CUDA error (e.g. "cudaErrorIllegalAddress") behind the most recent PQ_ERR_CUDA returned
 * to the calling host thread; "" if there was none.  Static string; diagnostic only. */
PQ_API const char* pq_last_cuda_error(void);

/* Shape rules shared by the calls below (else PQ_ERR_SHAPE):
 *   M >= 1, N >= 8 with N % 8 == 0, K >= 16 with K % 16 == 0, K < 131072 (so that
 *   K * 128 * 128 fits INT32); W4 additionally needs group == 128 and K % 128 == 0. */

/*
 * Per-token symmetric INT8 activation quantization (Eq. 1-2 with n = 8; one scale
 * per token over the feature dimension).  For each row m:
 *   a = max_k |X[m,k]|,  s_tok[m] = a / 127.5 (= 2a/255),
 *   Q[m,k] = clamp(rne(X[m,k] * (127.5 / a)), -128, 127),
 * evaluated in IEEE binary32 with round-half-to-even; an all-zero row gives scale 0
 * and codes 0.
 *   x_f16 [M,K] FP16 in;  q [M,K] INT8 out;  s_tok [M] FP32 out.
 */
PQ_API int pq_quantize_act(const void* x_f16, int64_t M, int64_t K, int8_t* q, float* s_tok,
                    void* stream);

/*
 * Offline per-output-channel INT8 weight quantization (Eq. 2 with n = 8, one scale
 * per output channel) into the layout the W8A8 GEMM reads.
 *   s_ch[n] = max_k |W[n,k]| / 127.5,  code = clamp(rne(W[n,k] / s_ch[n]), -128, 127).
 *   w_f16 [N,K] FP16 in;  wq: pq_packed_w8_bytes(N,K) bytes out (opaque);
 *   s_ch [N] FP32 out.
 */
PQ_API int pq_pack_w8(const void* w_f16, int64_t N, int64_t K, void* wq, float* s_ch, void* stream);

/*
 * Offline group-wise INT4 weight quantization (Eq. 2 with n = 4, one scale per output
 * channel and group of `group` consecutive k) into the packed layout the W4A8 GEMM
 * reads (two codes per byte along K).
 *   s = fp16(max_{k in g} |W[n,k]| / 7.5),  code = clamp(rne(W[n,k] / float(s)), -8, 7).
 *   w_f16 [N,K] FP16 in;  wp: pq_packed_w4_bytes(N,K) bytes out (opaque);
 *   s_grp_f16 [K/group, N] FP16 out (the scales of one K-group are contiguous over n).
 */
PQ_API int pq_pack_w4(const void* w_f16, int64_t N, int64_t K, int32_t group, void* wp,
               void* s_grp_f16, void* stream);

/*
 * SmoothQuant variant (Eq. 3: Y = (X S^-1)(S W), S = diag(s), s_j = max|X_j|^alpha / max|W_j|^(1-alpha),
 * alpha = 0.5 as in the paper's experiments).  The column factors are computed once, offline, from
 * calibration activations; at run time they cost one extra [K] FP32 vector read per call.
 *
 *   pq_col_absmax:     out[k] = max_r |A[r,k]| for A FP16 [R,K] row-major (R >= 1, K as for the
 *                      quantizer); out: [K] FP32.  Run it on calibration activations and on W.
 *   pq_smooth_scales:  s[k] = sqrt(x_absmax[k]) / sqrt(w_absmax[k]),  s_inv[k] = 1 / s[k]  (each a
 *                      correctly rounded FP32 operation); a channel with a zero maximum gets 1.
 *   pq_quantize_act_smooth: pq_quantize_act of X S^-1 -- every element is multiplied by s_inv[k] in
 *                      FP32 (not rounded to FP16) BEFORE the token maximum is taken.
 *   pq_pack_w8_smooth / pq_pack_w4_smooth: pq_pack_w8 / pq_pack_w4 of S W (W is [N,K], so s[k]
 *                      multiplies along K), same outputs and layouts.
 * s, s_inv: [K] FP32 device vectors, 16-byte aligned.  The GEMM calls are unchanged: codes and scales
 * produced by the smooth variants go into pq_gemm_w8a8 / pq_gemm_w4a8 as they are.
 */
PQ_API int pq_col_absmax(const void* a_f16, int64_t R, int64_t K, float* out, void* stream);
PQ_API int pq_smooth_scales(const float* x_absmax, const float* w_absmax, int64_t K, float* s, float* s_inv,
                            void* stream);
/* The same for a migration strength alpha = alpha_quarters / 4 (0 ... 4, else PQ_ERR_SHAPE):
 * s[k] = x_absmax[k]^alpha / w_absmax[k]^(1 - alpha), the quarter powers taken as square roots
 * (x^(1/4) = sqrt(sqrt(x)), x^(3/4) = sqrt(x) * sqrt(sqrt(x))) so that every step is a correctly rounded FP32
 * operation; alpha_quarters = 2 is pq_smooth_scales.  Any other factor vector a caller computes itself goes
 * into the quantizer and pack calls just the same. */
PQ_API int pq_smooth_scales_alpha(const float* x_absmax, const float* w_absmax, int64_t K, int32_t alpha_quarters,
                                  float* s, float* s_inv, void* stream);
PQ_API int pq_quantize_act_smooth(const void* x_f16, const float* s_inv, int64_t M, int64_t K, int8_t* q,
                                  float* s_tok, void* stream);
PQ_API int pq_pack_w8_smooth(const void* w_f16, const float* s, int64_t N, int64_t K, void* wq, float* s_ch,
                             void* stream);
PQ_API int pq_pack_w4_smooth(const void* w_f16, const float* s, int64_t N, int64_t K, int32_t group, void* wp,
                             void* s_grp_f16, void* stream);

/*
 * Static (calibrated) activation scale: the paper's accuracy runs quantize with "calibrated scales"
 * fixed ahead of time instead of the token's own maximum.  One scale for the whole tensor:
 *   code = clamp(rne(X[m,k] * (1 / s)), -128, 127)   (FP32; values beyond the range saturate),
 *   s_tok[m] = s for every token, so that the GEMM calls are used unchanged.
 * scale: DEVICE pointer to one FP32 value (it may be produced by a preceding kernel); s <= 0 gives
 * codes 0 and token scales 0.  No maximum pass: the kernel reads X once and is launched like
 * pq_quantize_act.
 */
PQ_API int pq_quantize_act_static(const void* x_f16, const float* scale, int64_t M, int64_t K, int8_t* q,
                                  float* s_tok, void* stream);

/*
 * The same with one calibrated scale per feature channel (the per-channel granularity the paper's
 * "Preliminary" section names), given as reciprocals:
 *   code = clamp(rne(X[m,k] * inv_s[k]), -128, 127)   (one FP32 product; inv_s[k] <= 0 gives code 0),
 *   s_tok[m] = 1: a scale that depends on k cannot be taken out of the sum over k, so the caller folds
 *   s[k] = 1 / inv_s[k] into the weights (pq_pack_w8_smooth / pq_pack_w4_smooth with that vector, as for
 *   Eq. 3) and uses the GEMM calls unchanged.
 * inv_s: [K] FP32 device vector, 16-byte aligned.
 */
PQ_API int pq_quantize_act_static_channel(const void* x_f16, const float* inv_s, int64_t M, int64_t K, int8_t* q,
                                          float* s_tok, void* stream);

/*
 * The MLP's gated activation fused with the down projection's activation quantizer.  The paper
 * quantizes all linear layers of a decoder and reports whole prefill passes (its latency table), but
 * does not define the activation between the gate/up linears and the down linear; the gated form
 * SwiGLU is taken:  h[m,i] = silu(gate[m,i]) * up[m,i],  silu(g) = g / (1 + e^-g).
 * h is evaluated in FP32 as a FIXED sequence of single correctly rounded operations (the argument of
 * the exponential clamped to [-87, 88]; the reduction t = n ln2 + r, the degree-7 Taylor polynomial p
 * of e^r in Horner form with fused multiply-adds, d = fma(p, 2^n, 1) = 1 + e^t; then the IEEE reciprocal
 * of d, the product g * (1 / d) and one product with `up`), because its value decides integer codes;
 * it is not rounded to FP16.  Then pq_quantize_act's rule (Eq. 1-2 per token) is applied to h.
 * One pass: 4 bytes read and 1 written per element, instead of an FP16 round trip of h plus a
 * separate quantizer pass.
 *   gate_f16, up_f16 [M,I] FP16 in (the outputs of the gate and up linears);  q [M,I] INT8 out;
 *   s_tok [M] FP32 out;  I as K of the quantizer, I <= 16384 (PQ_ERR_SHAPE beyond).
 */
PQ_API int pq_swiglu_quantize(const void* gate_f16, const void* up_f16, int64_t M, int64_t I, int8_t* q,
                              float* s_tok, void* stream);

/*
 * Hadamard variant (Eq. 4: Y = (X H)(H^T W), H a normalized Hadamard matrix).  With W stored [N,K]
 * both operands are rotated along K: (X H)(W H)^T = X W^T.  Where K is a power of two (up to 16384) H
 * is the Sylvester matrix of order K itself.  For other layer widths (11008 = 2^8 * 43) no construction
 * is at hand, and H = I (x) H_B / sqrt(B) is block diagonal, H_B the Sylvester matrix of order
 * B = the largest power of two dividing K, at most 256.  pq_hadamard_block(K) returns the order used
 * (K or B).  The rotation is the in-place butterfly (distances 1, 2, ..., B/2 in this order) in FP32
 * on the exact FP16 inputs, times 1/sqrt(B); the rotated values are quantized from FP32.
 *   pq_quantize_act_hadamard: pq_quantize_act of X H (on line, fused into the quantizer kernel);
 *   pq_pack_w8_hadamard / pq_pack_w4_hadamard: pq_pack_w8 / pq_pack_w4 of W H (off line).
 * Same arguments, outputs and layouts as the plain calls; K <= 16384 (PQ_ERR_SHAPE beyond).  The
 * GEMM calls are unchanged.  pq_hadamard_block is a host-only query (0 for a K the quantizer rejects).
 */
PQ_API int32_t pq_hadamard_block(int64_t K);
PQ_API int pq_quantize_act_hadamard(const void* x_f16, int64_t M, int64_t K, int8_t* q, float* s_tok,
                                    void* stream);
PQ_API int pq_pack_w8_hadamard(const void* w_f16, int64_t N, int64_t K, void* wq, float* s_ch, void* stream);
PQ_API int pq_pack_w4_hadamard(const void* w_f16, int64_t N, int64_t K, int32_t group, void* wp,
                               void* s_grp_f16, void* stream);

PQ_API size_t pq_packed_w8_bytes(int64_t N, int64_t K);
PQ_API size_t pq_packed_w4_bytes(int64_t N, int64_t K);

/* Recover the integer codes from the opaque layouts as row-major INT8 [N,K]
 * (W4 codes lie in [-8,7]).  For checking and interchange; not on the hot path. */
PQ_API int pq_unpack_w8(const void* wq, int64_t N, int64_t K, int8_t* codes, void* stream);
PQ_API int pq_unpack_w4(const void* wp, int64_t N, int64_t K, int8_t* codes, void* stream);

/*
 * W8A8 linear ("weight layout, dequantization logic and matrix multiplication" of the
 * framework section; weight-activation quantization runs the product itself in
 * integers):
 *   ACC[m,n] = sum_k Q[m,k] * Wq[n,k]                      exact, INT32
 *   Y[m,n]   = fp16( float(ACC[m,n]) * s_tok[m] * s_ch[n] )
 *   q [M,K] INT8, s_tok [M] FP32 (from pq_quantize_act);  wq, s_ch [N] (from pq_pack_w8);
 *   y_f16 [M,N] FP16 out.
 * Any M is accepted; small M (decode shapes) is routed to a weight-streaming schedule
 * that computes the same result.
 *
 * workspace / workspace_bytes: optional scratch of THIS call (NULL / 0 = none).  With few output
 * tiles and a long K (e.g. a 7B-class layer at M = 512) the GEMM cuts K into parts that run on
 * different SMs; the parts' INT32 partial accumulators pass through the workspace and are summed
 * exactly, so the result does not depend on it.  Without a workspace, or with one too small for the
 * shape, K is simply not split.  (The paper's "matrix multiplication ... within the operator
 * template library" leaves scheduling to the kernel; this is scheduling only.)
 *   - Device memory owned by the caller, 256-byte aligned (else PQ_ERR_ALIGN), of at least
 *     pq_workspace_bytes(...) bytes for the shape to be served in full.
 *   - Before its first use it is prepared once with pq_workspace_init (which zeroes its first
 *     64 KB, the arrival counters); every call that completes leaves it prepared for the next.
 *     After a PQ_ERR_TIMEOUT prepare it again.
 *   - Calls that may overlap on the GPU (different streams, parallel graph branches) must be
 *     given different workspaces; calls ordered in one stream may share one.
 */
PQ_API int pq_gemm_w8a8(const int8_t* q, const float* s_tok, const void* wq, const float* s_ch,
                 int64_t M, int64_t N, int64_t K, void* y_f16, void* workspace, size_t workspace_bytes,
                 void* stream);

/*
 * The whole path of one linear in one call: per-token quantization of the FP16 activations (Eq. 1-2,
 * exactly pq_quantize_act) followed by pq_gemm_w8a8 / pq_gemm_w4a8 on the result.  Y is bit for bit what
 * the two calls give.  For the smallest decode shapes (one to four tokens, where the CUDA-core row
 * kernel is the schedule) the GEMM kernel quantizes its tokens itself and nothing else is launched: a
 * decode step is a chain of dependent launches, and each launch costs microseconds whatever it does.
 *   x_f16 [M,K] device; q_tmp int8 [M,K] and s_tok_tmp float [M]: device buffers of the caller for the
 *   codes and scales (written when two kernels run; their contents are unspecified afterwards);
 *   everything else as in pq_gemm_w8a8 / pq_gemm_w4a8.  On an argument error nothing is launched.
 */
PQ_API int pq_linear_w8a8(const void* x_f16, const void* wq, const float* s_ch, int64_t M, int64_t N,
                          int64_t K, void* y_f16, int8_t* q_tmp, float* s_tok_tmp, void* workspace,
                          size_t workspace_bytes, void* stream);
PQ_API int pq_linear_w4a8(const void* x_f16, const void* wp, const void* s_grp_f16, int32_t group,
                          int64_t M, int64_t N, int64_t K, void* y_f16, int8_t* q_tmp, float* s_tok_tmp,
                          void* stream);

/*
 * W4A8 linear: INT4 codes are widened to INT8 inside the kernel, multiplied in
 * integers per K-group and dequantized per group into an FP32 running sum:
 *   ACC_g[m,n] = sum_{k in group g} Q[m,k] * C[n,k]        exact, INT32
 *   R[m,n]     = sum_g float(ACC_g[m,n]) * float(s_grp[g,n])   (FP32, g ascending)
 *   Y[m,n]     = fp16( R[m,n] * s_tok[m] )
 *   wp, s_grp_f16 [K/group, N] from pq_pack_w4;  group must be 128.
 */
PQ_API int pq_gemm_w4a8(const int8_t* q, const float* s_tok, const void* wp, const void* s_grp_f16,
                 int32_t group, int64_t M, int64_t N, int64_t K, void* y_f16, void* stream);

/*
 * The exact INT32 accumulators of the two linears, computed by the same tensor-core
 * main loops as the calls above and written out instead of the FP16 result (for
 * parity checking).   acc [M,N];   acc_g [K/group, M, N] (group-major).
 */
PQ_API int pq_acc_w8a8(const int8_t* q, const void* wq, int64_t M, int64_t N, int64_t K, int32_t* acc,
                void* stream);
PQ_API int pq_acc_w4a8(const int8_t* q, const void* wp, int32_t group, int64_t M, int64_t N, int64_t K,
                int32_t* acc_g, void* stream);

/*
 * Several W8A8 linears over the SAME quantized tokens (the q/k/v projections, or gate and up, of
 * the layers the paper quantizes) as one call.  Result: exactly what `count` calls of pq_gemm_w8a8
 * with (wq[g], s_ch[g], N[g], y_f16[g]) give, bit for bit.  The members' output tiles are scheduled
 * together in a single kernel launch (of the weight-streaming kernel up to 128 tokens, and up to 256
 * where the members' 128-channel tiles x 2 token blocks do not exceed the number of SMs; of the
 * prefill kernel otherwise), which fills the SMs' waves across the members and pays the per-launch fixed cost
 * once -- at decode-shaped token counts that fixed cost is most of a call.
 *   count: 1..PQ_MAX_GROUP.  wq, s_ch, N, y_f16: HOST arrays of `count` entries (device pointers
 *   and column counts; read during the call, not retained).  q, s_tok, M, K as in pq_gemm_w8a8.
 *   The outputs must not overlap each other.  On an argument error nothing is launched.
 *   workspace / workspace_bytes: as for pq_gemm_w8a8 (sized with pq_workspace_bytes for the group).
 */
#define PQ_MAX_GROUP 4
PQ_API int pq_gemm_w8a8_group(const int8_t* q, const float* s_tok, int32_t count, const void* const* wq,
                              const float* const* s_ch, const int64_t* N, void* const* y_f16, int64_t M,
                              int64_t K, void* workspace, size_t workspace_bytes, void* stream);

/* The same for W4A8 linears (pq_gemm_w4a8 per member; one launch for all of them, except at M <= 128 when
 * the members together hold more 128-channel tiles than the device has SMs).  For M <= 128, and for M <= 256
 * when the members' 128-channel tiles x 2 token blocks do not exceed the number of SMs, the FP32
 * group sums of the K parts are added in a fixed order, but the number of parts depends on how many tiles
 * the launch holds, so the grouped result may differ from the per-member call in the last FP32 bit. */
PQ_API int pq_gemm_w4a8_group(const int8_t* q, const float* s_tok, int32_t count, const void* const* wp,
                              const void* const* s_grp_f16, int32_t group, const int64_t* N,
                              void* const* y_f16, int64_t M, int64_t K, void* stream);

/*
 * Workspace of the W8A8 calls (see pq_gemm_w8a8).
 *   pq_workspace_bytes: host-only (touches no device).  The number of bytes with which
 *     pq_gemm_w8a8 (count = 1) or pq_gemm_w8a8_group over the column counts N[0..count) at these M
 *     and K runs the schedule it would pick with unlimited room, on a GPU with `sms`
 *     multiprocessors (148 on a B200); 0 when that schedule does not split K (then no workspace is
 *     of any use) or when an argument is invalid.  The maximum over the shapes a caller issues
 *     serves all of them.  pq_gemm_w4a8 and every call that the weight-streaming kernel serves (M <= 128, narrow
 *     linears up to M = 256) need none.
 *   pq_workspace_init: zeroes the first 64 KB of `workspace` on `stream` (bytes >= 65536, 256-byte
 *     aligned).  GEMM calls enqueued afterwards on that stream (or after a synchronization) may
 *     use the workspace.  A buffer the caller has zero-filled by other means is equally good.
 */
PQ_API size_t pq_workspace_bytes(int64_t M, const int64_t* N, int32_t count, int64_t K, int32_t sms);
PQ_API int pq_workspace_init(void* workspace, size_t bytes, void* stream);

/*
 * Host-only query (touches no device): the schedule of the prefill kernel (the one pq_gemm_w8a8 uses
 * beyond the token counts of the weight-streaming kernel) on a GPU with
 * `sms` multiprocessors and a workspace of `scratch_bytes` (0 = none): the output tile
 * width (*tile_n = 256 or 128 columns) and the number of parts K is cut into (*k_parts, 1 = no
 * split).  For capacity planning and tests; the result has no effect on later calls.
 */
PQ_API int pq_plan_w8a8(int64_t M, int64_t N, int64_t K, int32_t sms, size_t scratch_bytes, int32_t* tile_n,
                        int32_t* k_parts);

/*
 * W8A8 linear for callers that cannot allocate device memory (the paper has no counterpart to
 * this call; it exists for deployment constraints, not for the method).
 *
 * Same result as pq_gemm_w8a8, same arguments without the workspace.  The difference is where the
 * split-K scratch comes from: not from a workspace argument -- which somebody had to cudaMalloc --
 * but from a fixed 32 MiB + 64 KiB array inside the library, held by every GPU that loads the
 * library until the process exits.  Meant for hosts that hand a plug-in nothing but its inputs and
 * outputs, for serving loops and capture regions in which cudaMalloc (a synchronizing call) is
 * off limits, and for programs that fix their whole device-memory budget at start-up.  The call
 * itself invokes no allocation or free routine of any kind.
 *   - Limit: M and N each rounded up to a multiple of 256, multiplied, may not exceed 2,097,152
 *     (e.g. 512 x 4096, 1024 x 2048, 256 x 8192); beyond that the call returns PQ_ERR_LIMIT and
 *     launches nothing.  M <= 128 needs no scratch: such calls are forwarded to pq_gemm_w8a8
 *     whatever N is, and the limit does not apply to them.
 *   - The first call on each device looks up the array's device address; make that first call
 *     outside any stream capture.
 *   - All calls on a device share the one array, and it keeps whatever the last call left in it
 *     (a call that completes restores the few words that must read zero; after a call that ended
 *     in PQ_ERR_TIMEOUT, pq_device_status() -- the call that reports it -- clears them with a memset
 *     on the array, so read the status before going on).  Two calls that overlap on the GPU
 *     -- different streams, parallel graph branches -- would race on it: keep them ordered.
 */
PQ_API int pq_gemm_w8a8_noalloc(const int8_t* q, const float* s_tok, const void* wq, const float* s_ch,
                                int64_t M, int64_t N, int64_t K, void* y_f16, void* stream);

/*
 * Reads the device status word of the current device into *host_status (PQ_OK or
 * PQ_ERR_TIMEOUT) and clears it.  Synchronizes the device; call it outside timed
 * regions.
 */
PQ_API int pq_device_status(int* host_status);

/*
 * The poll bound of the waits inside the kernels launched from now on (process-wide; 0 restores
 * the default of 2^24 polls, about a second).  For tests of the give-up path: with PQ_WAIT_NONE no
 * wait polls at all, so every role of a kernel gives up at its first wait although nothing is
 * wrong; with a bound of a few polls some wait runs out somewhere in the middle.  Either way the
 * kernel reports PQ_ERR_TIMEOUT through the status word and returns with unspecified outputs.
 */
#define PQ_WAIT_NONE 0xFFFFFFFFu
PQ_API int pq_set_wait_limit(uint32_t polls);

#ifdef __cplusplus
}
#endif
#endif /* PQ_H_ */
