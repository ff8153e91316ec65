/*
 * xq -- expanded W4A4 linear layer for NVIDIA B200 (sm_100a).  C ABI.
 *
 * The layer (paper Sec. 3, "Post-Training Model Expansion via Online Incoherence
 * Processing"): an activation row x of K channels is zero-padded to K' channels and rotated by
 * a Hadamard matrix of order K' scaled by 1/sqrt(K') -- equivalently multiplied by the first K
 * rows of that matrix, the paper's truncated N x M matrix -- then quantized per token to 4 bits
 * (Sec. 4, "Quantization Details") and multiplied with weights that were expanded, rotated and
 * quantized per output channel offline; the product of the two quantized operands is what runs
 * at inference ("online incoherence processing", Sec. 3).
 *
 * Letters: M tokens, K input channels, Kp = K' expanded channels, N output channels.  Weights
 * are out x in: row n of W is output channel n, and the layer computes x W^T.
 *
 * Conventions for every call
 *  - Returns an xq_status; nothing throws, aborts or traps.  All argument, shape and alignment
 *    checks run on the host before anything is launched.
 *  - "dev" pointers are CUDA device pointers of the current device, "host" pointers are host
 *    memory.  The caller owns every buffer it passes (activations, outputs, workspace); the
 *    library owns only xq_weights objects, released with xq_weights_free.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls taking a
 *    stream only enqueue work; they do not synchronize unless stated.
 *  - bf16 tensors are raw 16-bit patterns.  Device pointers must be 16-byte aligned.
 *  - The device that was current when a weights object was made must be current in every call
 *    that takes the object (XQ_ERR_INVALID_ARG otherwise).
 *  - No global state, except in xq_expanded_linear_static (see there): calls on distinct streams
 *    with distinct workspaces may run concurrently.
 *  - One environment variable is read (once, at the first product of more than 32 tokens):
 *    XQ_PREFILL_KERNEL overrides the choice between the two forms of the tcgen05 tile kernel, for
 *    measurements and tests: "ss" keeps the first form (expanded weights in shared memory), "ts"
 *    or "ts:<tokens>" forces the second (expanded weights in tensor memory).  Results are the
 *    same bits either way.
 */
#ifndef XQ_H_
#define XQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  XQ_OK = 0,
  XQ_ERR_INVALID_ARG = 1,       /* null pointer, non-positive size, misaligned pointer, bad ld */
  XQ_ERR_UNSUPPORTED_ORDER = 2, /* K' has no Paley (prime field) x Sylvester factorisation the
                                   kernels support */
  XQ_ERR_WORKSPACE = 3,         /* workspace missing or smaller than xq_workspace_bytes */
  XQ_ERR_ALLOC = 4,             /* device or host allocation failed */
  XQ_ERR_CUDA = 5,              /* a CUDA runtime call or launch failed */
  XQ_ERR_TIMEOUT = 6,           /* a bounded device-side wait ran out (sticky, see xq_poll_status) */
  XQ_ERR_BOUNDS = 7             /* an index self check of a product kernel failed (sticky); raised only by the
                                   build made with -DXQ_DEBUG_BOUNDS, where the access is then skipped */
} xq_status;

/* Hadamard plan: Kp = p * 2^log2n and H = H_p (x) S_{2^log2n} (Kronecker product, the order-p
 * factor outermost: channel c = a * 2^log2n + b).  S is the Sylvester matrix
 * S[b][b'] = (-1)^popcount(b & b'); H_p is a Paley matrix over the prime field GF(q):
 * paley_kind 1 (q = p - 1 = 3 mod 4) or 2 (q = p/2 - 1 = 1 mod 4); paley_kind 0 means p = 1;
 * paley_kind 3 is the first construction over the field of q = 7^3 = 343 elements (p = 344: the
 * factor that the paper's Table 1 size 22016 = 344 * 64 needs).
 * The paper asks only for "an expanded M x M Hadamard matrix" (Sec. 3); this family is the
 * library's choice of one. */
typedef struct {
  int32_t K, Kp, p, log2n, paley_kind, q;
} xq_hadamard_plan_t;

/* Prepared (expanded, rotated, quantized, packed) weights of one linear layer.  Opaque; lives
 * in device memory owned by the library. */
typedef struct xq_weights xq_weights;

/* Factor Kp.  Host only, pure.  p is the smallest odd(Kp) * 2^j (j >= 2) that is a Paley order.
 * Errors: INVALID_ARG (out == NULL, K < 1, Kp < K, Kp odd and > 1), UNSUPPORTED_ORDER (no such
 * factor up to p = 8192; or p > 256, which only the general rotate kernel takes, with
 * 8 Kp + 3 q + 256 bytes above the 227 KiB of shared memory that kernel may use). */
xq_status xq_hadamard_plan(int32_t K, int32_t Kp, xq_hadamard_plan_t* out);

/* Offline step (Sec. 3: expanded weights = truncated-Hadamard^T times W; Sec. 4: per-channel
 * symmetric 4-bit).  Each of the N rows of W (bf16, HOST, row-major [N, K]) is zero-padded to
 * Kp, multiplied by H / sqrt(Kp), scaled by absmax / 7, rounded to nearest even, clamped to
 * [-8, 7] and packed into the device layout the GEMM kernels read.  Allocates device memory,
 * runs on `stream` and synchronizes it before returning.  *out receives the new object.
 * Kp must be a multiple of 8 (UNSUPPORTED_ORDER otherwise). */
xq_status xq_prepare_weights(const void* W_bf16_host, int32_t N, int32_t K, int32_t Kp,
                             void* stream, xq_weights** out);

/* Offline step with the weight quantizer of the paper's experiments (Sec. 4 "Quantization Details": GPTQ with
 * act-order on per-channel symmetric 4-bit weights; Sec. 3.1 Remark 2 bounds its error under expansion).  The rows of
 * W are expanded and rotated as in xq_prepare_weights; then, instead of rounding every value to the nearest grid
 * point, the channels are visited in descending order of diag(H) and the error of every quantized column is fed into
 * the columns still to come, so that tr((W~ - Q) H (W~ - Q)^T) is descended on.  H_host: HOST, double [Kp, Kp],
 * row-major, symmetric: the Hessian X_hat^T X_hat of the layer's expanded, rotated calibration activations (rows of
 * xq_rotate_quant's Y output).  damp times the mean of diag(H) is added to the diagonal first (0.01 is customary; the
 * Hessian of expanded activations has rank <= K < Kp, so some damping is needed); a channel with H[c][c] = 0 gets
 * zero codes.  Every row keeps the scale absmax / 7 of its rotated values; codes lie in [-8, 7].  fp64 on the device;
 * allocates about 8 (Kp^2 + 3 N Kp) bytes of device memory for the duration of the call; synchronizes `stream`.
 * Errors as xq_prepare_weights; INVALID_ARG also when H is not positive definite after damping.
 * xq_gptq_codes is the quantizer alone, on rows that are already rotated (HOST double [N, Kp]): codes int8 [N, Kp] and
 * scales float [N] to the HOST (what xq_weights_import takes). */
xq_status xq_prepare_weights_gptq(const void* W_bf16_host, int32_t N, int32_t K, int32_t Kp, const double* H_host,
                                  double damp, void* stream, xq_weights** out);
xq_status xq_gptq_codes(const double* Wt_host, const double* H_host, int32_t N, int32_t Kp, double damp,
                        int8_t* codes_host, float* s_w_host, void* stream);

/* Build a weights object from already quantized values (HOST): codes int8 [N, Kp] row-major with
 * values in -8..7 (INVALID_ARG otherwise), s_w float [N].  Synchronizes `stream`. */
xq_status xq_weights_import(const int8_t* codes_host, const float* s_w_host, int32_t N, int32_t K,
                            int32_t Kp, void* stream, xq_weights** out);

/* Canonical form back to the HOST: codes int8 [N, Kp], s_w float [N].  Synchronizes. */
xq_status xq_weights_export(const xq_weights* w, int8_t* codes_host, float* s_w_host);

/* Sizes and plan of a weights object. */
xq_status xq_weights_info(const xq_weights* w, int32_t* N, int32_t* K, int32_t* Kp,
                          xq_hadamard_plan_t* plan);

/* Releases the object and its device memory (NULL is allowed). */
void xq_weights_free(xq_weights* w);

/* Bytes of caller-provided device workspace that xq_w4a4_gemm / xq_expanded_linear(_host) need
 * for up to M_max tokens against `w`.  0 on bad arguments. */
size_t xq_workspace_bytes(int32_t M_max, const xq_weights* w);

/* Must be called once on a fresh workspace (zeroes its status word and counters -- the first
 * 1 KiB, or 256 bytes of a smaller workspace; enqueued on `stream`). */
xq_status xq_workspace_init(void* ws_dev, size_t ws_bytes, void* stream);

/* Online step (Sec. 3: expanded activations = X times the truncated Hadamard matrix; Sec. 4:
 * per-token 4-bit, symmetric in this library).  For each of the M rows of X (bf16, dev,
 * row-major, row pitch ldx elements, ldx >= K and a multiple of 8):
 *   y = [x, 0] H / sqrt(Kp);  s_x = max|y| / 7 (1 if the row is zero);
 *   code = clamp(round_half_even(y / s_x), -8, 7).
 * Outputs: Xq dev [M, Kp/2] bytes, byte j of a row = code 2j in bits 0-3 and code 2j+1 in bits
 * 4-7 (two's complement); s_x dev float [M]; if Y_f32_opt != NULL also the rotated values, dev
 * float [M, Kp] (for stage-wise checking).  M = 0 is a no-op. */
xq_status xq_rotate_quant(const void* X_bf16_dev, int32_t M, int64_t ldx,
                          const xq_hadamard_plan_t* plan, uint8_t* Xq_dev, float* s_x_dev,
                          float* Y_f32_opt_dev, void* stream);

/* Quantized product with dequantizing epilogue (Sec. 3: Q(XR) Q(W~)):
 *   acc[m][n] = sum_c qx[m][c] * qw[n][c]   (exact, int32)
 *   out[m][n] = bf16( acc * s_x[m] * s_w[n] ).
 * Xq, s_x in the xq_rotate_quant format (any nibble -8..7 is accepted).  out dev bf16 [M, N]
 * row-major.  If acc_opt != NULL the int32 accumulators are also written, dev [M, N].
 * ws: device workspace of at least xq_workspace_bytes(M, w), initialised once with
 * xq_workspace_init; concurrent calls need distinct workspaces. */
xq_status xq_w4a4_gemm(const uint8_t* Xq_dev, const float* s_x_dev, int32_t M, const xq_weights* w,
                       void* out_bf16_dev, int32_t* acc_opt_dev, void* ws_dev, size_t ws_bytes,
                       void* stream);

/* The whole layer on device buffers: xq_rotate_quant then xq_w4a4_gemm on `stream`, the
 * quantized activations staying in the workspace. */
xq_status xq_expanded_linear(const void* X_bf16_dev, int32_t M, int64_t ldx, const xq_weights* w,
                             void* out_bf16_dev, void* ws_dev, size_t ws_bytes, void* stream);

/* xq_expanded_linear for M <= 32 tokens as ONE kernel launch (Sec. 3: the rotation of the activations is an online
 * step of the layer; here it runs inside the product's launch).  Every CTA first requests its share of the weights,
 * which do not depend on the tokens; CTA r < M meanwhile pads, rotates and quantizes token row r, writes codes and
 * scale to the workspace and counts the row as published; every CTA waits, time-bounded, until M rows are counted
 * and goes on as xq_w4a4_gemm does.  asym != 0: asymmetric codes (as xq_expanded_linear_asym).  The output bits
 * are those of xq_expanded_linear.  Measured on B200 inside a captured, programmatically chained stream the two-kernel
 * form is the faster one (the chain already overlaps the next product's weight requests with the rotation); this
 * form halves the number of launches, which is what counts where the host's launch rate is the limit.
 * Limits: the plans of the tensor-core row routine (p > 1, 32 <= 2^k <= 256, K a multiple of 8, at most 64 input
 * rows of 2^k channels, at most 16 warps per row) on weights made by xq_prepare_weights / xq_weights_import with
 * p <= 256; otherwise UNSUPPORTED_ORDER (also M > 32).  The two counters it keeps in the workspace header are back at zero
 * when the launch ends; after a device-side time-out re-initialise the workspace. */
xq_status xq_expanded_linear_one_launch(const void* X_bf16_dev, int32_t M, int64_t ldx, const xq_weights* w, int32_t asym,
                                        void* out_bf16_dev, void* ws_dev, size_t ws_bytes, void* stream);

/* The same three calls with per-token ASYMMETRIC activation codes (Sec. 4: the setting of the
 * paper's experiments; weights stay symmetric per channel).  For each row, with y as above,
 * lo = min(0, min y), hi = max(0, max y):
 *   s_x = (hi - lo) / 15 (1 if hi = lo);  z = clamp(round_half_even(-lo / s_x), 0, 15);
 *   u = clamp(round_half_even(y / s_x) + z, 0, 15), which stands for s_x * (u - z).
 * Storage: codes and zero point are kept shifted by -8, so Xq holds the nibble c = u - 8
 * (two's complement, same packing as xq_rotate_quant) and zp_dev, dev int32 [M], receives
 * z - 8, in -8..7; a stored code stands for s_x * (c - zp).  The product is
 *   acc[m][n] = sum_c (qx[m][c] - zp[m]) * qw[n][c]      (exact, int32; this is what acc_opt gets)
 *   out[m][n] = bf16( acc * s_x[m] * s_w[n] ),
 * computed as the signed product minus zp[m] times the channel's code sum, which the weights
 * object holds.  xq_w4a4_gemm_asym accepts any nibbles and any zp in -8..7.  All other arguments,
 * layouts, workspace and error behaviour as in the symmetric calls. */
xq_status xq_rotate_quant_asym(const void* X_bf16_dev, int32_t M, int64_t ldx,
                               const xq_hadamard_plan_t* plan, uint8_t* Xq_dev, float* s_x_dev,
                               int32_t* zp_dev, float* Y_f32_opt_dev, void* stream);
xq_status xq_w4a4_gemm_asym(const uint8_t* Xq_dev, const float* s_x_dev, const int32_t* zp_dev, int32_t M,
                            const xq_weights* w, void* out_bf16_dev, int32_t* acc_opt_dev, void* ws_dev,
                            size_t ws_bytes, void* stream);
xq_status xq_expanded_linear_asym(const void* X_bf16_dev, int32_t M, int64_t ldx, const xq_weights* w,
                                  void* out_bf16_dev, void* ws_dev, size_t ws_bytes, void* stream);
/* xq_expanded_linear_host (below) with asymmetric activation codes. */
xq_status xq_expanded_linear_host_asym(const void* X_bf16_host, int32_t M, const xq_weights* w,
                                       void* out_bf16_host, void* ws_dev, size_t ws_bytes, void* stream);

/* Head-wise form (Sec. 4 "Compute Graph Details", Sec. 5 "Expanding R2 and R4": the rotation in
 * front of the attention output projection acts on every head separately, so expanding it grows
 * every head from head_dim to head_dim_p channels).  A row is `heads` blocks of head_dim channels;
 * every block is zero-padded to head_dim_p and multiplied by the Hadamard matrix of that order
 * scaled 1 / sqrt(head_dim_p) (plan = xq_hadamard_plan(head_dim, head_dim_p)); the blocks stay side
 * by side (row length heads * head_dim_p) and ONE quantizer runs over the whole row, symmetric, or
 * asymmetric when zp_opt_dev != NULL (formats as in xq_rotate_quant / xq_rotate_quant_asym).
 * Limits: 2 <= heads <= 128, head_dim <= 128 and a multiple of 8, head_dim_p <= 160 and a multiple
 * of 8, heads * head_dim_p a multiple of 32; otherwise UNSUPPORTED_ORDER.  ldx >= heads * head_dim.
 * xq_prepare_weights_heads is xq_prepare_weights with this map on the rows of W (host bf16
 * [N, heads * head_dim]); the object then reports K = heads * head_dim, Kp = heads * head_dim_p and
 * the plan of one head, and every xq_expanded_linear* call and xq_w4a4_gemm* call takes it as any
 * other weights object (the layer calls run the head-wise online step).  xq_weights_heads returns
 * the number of heads of an object (1 for xq_prepare_weights / xq_weights_import; 0 for NULL). */
xq_status xq_rotate_quant_heads(const void* X_bf16_dev, int32_t M, int64_t ldx, int32_t heads,
                                const xq_hadamard_plan_t* head_plan, uint8_t* Xq_dev, float* s_x_dev,
                                int32_t* zp_opt_dev, float* Y_f32_opt_dev, void* stream);
xq_status xq_prepare_weights_heads(const void* W_bf16_host, int32_t N, int32_t heads, int32_t head_dim,
                                   int32_t head_dim_p, void* stream, xq_weights** out);
int32_t xq_weights_heads(const xq_weights* w);

/* MXFP4 form (Sec. 4 "Quantization Details": weights and activations in the OCP microscaling
 * format -- an E8M0 scale for each group of 32 channels, 4-bit E2M1 elements; Sec. 5 "OCP MXFP4
 * Results").  The rotation is the same; the quantizer works per group of 32 consecutive channels of
 * the rotated row (K' a multiple of 32, at least 128):
 *   e = floor(log2(max |y|)) - 2 clamped to [-127, 127] (0 for a group of zeros); scale byte e + 127;
 *   element = the E2M1 value nearest to y / 2^e (0, 0.5, 1, 1.5, 2, 3, 4, 6 with a sign bit; ties to
 *   the even mantissa bit; larger magnitudes saturate at 6); code = sign << 3 | exponent << 1 | mantissa.
 * The product sums element products times 2^(e_x + e_w) per group in fp32 inside the tensor core
 * (tcgen05.mma kind::mxf4 with block scaling) and is rounded once to bf16.
 * Canonical formats at this boundary: codes dev [M, Kp/2] bytes (low nibble = even channel), scale
 * bytes dev [M, Kp/32].  xq_mx_weights is opaque (device memory owned by the library);
 * xq_mx_weights_import / _export take host arrays: import packed codes [N, Kp/2] and scales
 * [N, Kp/32]; export one code per byte [N, Kp] and scales [N, Kp/32].  N must be a multiple of 8.
 * xq_mx_rotate_quant needs Y_f32_dev, dev float [M, Kp]: it receives the rotated rows and is the
 * kernel's only scratch.  Workspace: xq_mx_workspace_bytes, initialised once with xq_workspace_init;
 * status through xq_poll_status.  Errors as for the INT4 calls. */
typedef struct xq_mx_weights xq_mx_weights;
xq_status xq_mx_prepare_weights(const void* W_bf16_host, int32_t N, int32_t K, int32_t Kp, void* stream,
                                xq_mx_weights** out);
/* MXFP4 weights behind the head-wise rotation (the paper's MXFP4 experiments expand the per-head rotation of the
 * attention output projection, Sec. 5): rows of W are rotated per head as in xq_prepare_weights_heads (same limits, and
 * heads * head_dim_p a multiple of 32, at least 128), then quantized in groups of 32 along the whole row; the layer calls
 * on such an object run the head-wise online step.  xq_mx_weights_heads: number of heads (1 otherwise; 0 for NULL). */
xq_status xq_mx_prepare_weights_heads(const void* W_bf16_host, int32_t N, int32_t heads, int32_t head_dim, int32_t head_dim_p,
                                      void* stream, xq_mx_weights** out);
int32_t xq_mx_weights_heads(const xq_mx_weights* w);
xq_status xq_mx_weights_import(const uint8_t* codes_packed_host, const uint8_t* scales_host, int32_t N, int32_t K,
                               int32_t Kp, void* stream, xq_mx_weights** out);
xq_status xq_mx_weights_export(const xq_mx_weights* w, uint8_t* codes_host, uint8_t* scales_host);
xq_status xq_mx_weights_info(const xq_mx_weights* w, int32_t* N, int32_t* K, int32_t* Kp, xq_hadamard_plan_t* plan);
void xq_mx_weights_free(xq_mx_weights* w);
size_t xq_mx_workspace_bytes(int32_t M_max, const xq_mx_weights* w);
xq_status xq_mx_rotate_quant(const void* X_bf16_dev, int32_t M, int64_t ldx, const xq_hadamard_plan_t* plan,
                             uint8_t* codes_dev, uint8_t* scales_dev, float* Y_f32_dev, void* stream);
xq_status xq_mx_gemm(const uint8_t* codes_dev, const uint8_t* scales_dev, int32_t M, const xq_mx_weights* w,
                     void* out_bf16_dev, void* ws_dev, size_t ws_bytes, void* stream);
xq_status xq_mx_expanded_linear(const void* X_bf16_dev, int32_t M, int64_t ldx, const xq_mx_weights* w,
                                void* out_bf16_dev, void* ws_dev, size_t ws_bytes, void* stream);
/* The two halves of xq_mx_expanded_linear, which is exactly these two calls in a row:
 * xq_mx_rotate_quant_staged quantizes M token rows into the workspace, in the GEMM kernel's own
 * input form (one kernel: pad, rotate, group exponents, codes); xq_mx_gemm_staged runs the product
 * on the tokens that the last staging (or xq_mx_gemm) call with the same M and the same weights
 * shape left there.  What a caller times separately, or re-runs against other weights of the same
 * shape. */
xq_status xq_mx_rotate_quant_staged(const void* X_bf16_dev, int32_t M, int64_t ldx, const xq_mx_weights* w, void* ws_dev,
                                    size_t ws_bytes, void* stream);
xq_status xq_mx_gemm_staged(int32_t M, const xq_mx_weights* w, void* out_bf16_dev, void* ws_dev, size_t ws_bytes,
                            void* stream);
/* Host buffers (X [M, K] contiguous, K a multiple of 8; out bf16 [M, N]): copies in, runs the layer, copies out,
 * synchronizes `stream`. */
xq_status xq_mx_expanded_linear_host(const void* X_bf16_host, int32_t M, const xq_mx_weights* w, void* out_bf16_host,
                                     void* ws_dev, size_t ws_bytes, void* stream);

/* The whole layer on HOST buffers: copies X (host, [M, K] contiguous; pinned memory makes the
 * copies asynchronous) into the workspace, runs the layer, copies out (host, bf16 [M, N]) back
 * and synchronizes `stream` before returning. */
xq_status xq_expanded_linear_host(const void* X_bf16_host, int32_t M, const xq_weights* w,
                                  void* out_bf16_host, void* ws_dev, size_t ws_bytes, void* stream);

/* xq_expanded_linear_host without the final synchronization: the two copies and the layer are only
 * enqueued on `stream` (pinned host memory; with pageable memory the runtime makes the copies
 * synchronous).  X_host must stay untouched and out_host is valid only after the caller has
 * synchronized the stream; several layers may be enqueued back to back and awaited once. */
xq_status xq_expanded_linear_host_enqueue(const void* X_bf16_host, int32_t M, const xq_weights* w,
                                          void* out_bf16_host, void* ws_dev, size_t ws_bytes, void* stream);

/* The whole layer for callers that cannot allocate device memory.  (No counterpart in the paper:
 * this is a deployment variant of xq_expanded_linear, same arithmetic, same kernels.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a plugin inside a host
 * application that owns the whole memory pool and hands out nothing at run time, a real-time
 * loop that may not take the allocator's locks or its implicit synchronization, a process
 * that already sits at its memory limit.  Such a caller has buffers for its inputs and outputs
 * but nowhere to put the workspace that xq_expanded_linear asks for.
 *
 * Here the intermediate results (packed INT4 codes of the M tokens, their M scales, the status
 * word) are kept in a fixed 4 MiB array that is part of the library image; every GPU on which
 * the library is used holds those 4 MiB until the process exits.  The call asks for no memory,
 * neither from the CUDA allocator nor from the host heap: it looks up the array, clears the status
 * word and enqueues the same two kernels as xq_expanded_linear on `stream`.  What the CUDA
 * runtime does by itself the first time a kernel of the library runs on a device (loading the
 * module, which is also when the 4 MiB array comes into being) happens in the first call; so do
 * an occupancy query and a driver entry-point lookup whose answers the library keeps (behind two
 * short host mutexes that every later call also takes for a table lookup).  From the second
 * call for a given token-count class on a device, the amount of free device memory no longer moves.
 *
 * Limit: 256 + roundup256(M * Kp / 2) + roundup256(4 * M) bytes, plus roundup256(M * Kp) when
 * M > 32, must fit in 4 MiB (about 1280 tokens at Kp = 2176, 180 at Kp = 15360); larger calls
 * return XQ_ERR_WORKSPACE and launch nothing.
 * First call on each device: it asks the runtime for the array's device address (with that
 * device current) and remembers it; make this first call outside any stream capture.
 * Sharing: all calls on one device use the same array, which keeps the previous call's
 * contents.  Calls that may overlap on the GPU (different streams, or the same stream with
 * programmatic overlap you arranged yourself) race on it: serialize them.  Calls issued one
 * after another on one stream are safe.
 * A device-side time-out of this path cannot be read with xq_poll_status (there is no
 * caller-visible workspace); X, out, w as in xq_expanded_linear.
 * Errors: INVALID_ARG (null or misaligned pointer, bad ldx, device index above 63), WORKSPACE
 * (does not fit the array), CUDA (a runtime call or launch failed). */
xq_status xq_expanded_linear_static(const void* X_bf16_dev, int32_t M, int64_t ldx, const xq_weights* w,
                                    void* out_bf16_dev, void* stream);

/* Diagnostic, host only, nothing is launched (no counterpart in the paper): which kernel the quantized
 * product of M tokens against w runs in, and its tile.  *kind = 0: the split-K weight-stream kernel
 * of M <= 32 tokens (tile_tokens = tokens padded to 8, 16 or 32; tile_channels = 16); 1: the
 * tcgen05 tile kernel in its first form (tile_tokens x tile_channels one of 128 x 256, 256 x 256, 256 x 128,
 * 256 x 224); 3: the tile kernel in its second form (tile_tokens a multiple of 32 up to 192, tile_channels = 256);
 * 2: the one-thread-per-output kernel (1 x 1).  Tests use it to name the tile shape a case exercised.
 * Errors: INVALID_ARG (null pointer, M < 1, wrong current device), CUDA. */
xq_status xq_gemm_kernel_info(int32_t M, const xq_weights* w, int32_t* kind, int32_t* tile_tokens,
                              int32_t* tile_channels);

/* Synchronizes `stream` and returns the sticky device status stored in the workspace (XQ_OK,
 * XQ_ERR_TIMEOUT or XQ_ERR_BOUNDS), or XQ_ERR_CUDA if the stream itself reports an error. */
xq_status xq_poll_status(const void* ws_dev, void* stream);

/* Self-test of the failure path (no counterpart in the paper): enqueues a one-warp kernel that
 * waits, with the same time-bounded wait every pipelined kernel uses, on a barrier that nothing
 * ever signals.  After about one second the wait gives up, the kernel records XQ_ERR_TIMEOUT in
 * the workspace status word and returns normally; xq_poll_status then reports XQ_ERR_TIMEOUT and
 * the CUDA context stays usable.  xq_workspace_init clears the status again. */
xq_status xq_selftest_wait_timeout(void* ws_dev, size_t ws_bytes, void* stream);

/* Measurement aid (no counterpart in the paper): enqueues one kernel in which every multiprocessor
 * issues iters * 4 tensor-core instructions of the kind the prefill product uses
 * (tcgen05.mma kind::i8, 128 x 256 x 32, operands resident in shared memory, no loads, no unpacking)
 * and returns in *ops_out (optional) the integer operations that launch performs, 2 per
 * multiply-add.  Timed with events by the caller, this gives the INT8 issue rate of the tensor pipe
 * on the device at hand: the ceiling the prefill kernel is measured against.  1 <= iters <= 2^22.
 * ws: any initialised workspace (status word for the bounded wait). */
xq_status xq_selftest_i8_mma_rate(int32_t iters, void* ws_dev, size_t ws_bytes, void* stream, double* ops_out);

const char* xq_status_string(xq_status s);

#ifdef __cplusplus
}
#endif
#endif /* XQ_H_ */
