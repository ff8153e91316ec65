// Internal declarations shared by the translation units of libxq (never installed, never
// included by the oracle).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>
#include <stdint.h>

#include "xq.h"

// ---------------------------------------------------------------------------------------------
// Prepared-weights device layout.
//
// Codes are packed two per byte exactly like the activation format (byte j of a row = code 2j in
// bits 0-3, code 2j+1 in bits 4-7, two's complement).  The smallest piece is 16 bytes: 32
// consecutive codes of one output channel.  Pieces are stored as
//     [block of 16 output channels][group of 32 codes][channel within the block][16 bytes]
// so that (a) the codes of 16 channels over any range of K that is a multiple of 32 are one
// contiguous run (the decode kernel streams such runs and cuts K between the CTAs of a cluster),
// (b) inside a 256-byte group lane 4g + t of a warp finds word t (8 codes) of channels g and g + 8
// at byte offsets 4 * lane and 128 + 4 * lane -- conflict-free 32-bit loads that become the A
// fragment of one m16n8k32 MMA after the nibble split -- and (c) 16 consecutive channel blocks at
// one 128-code block, fetched as 16 bulk copies of 1 KiB, form the 256-row tile the prefill
// kernel expands for tcgen05.mma.
// Rows are padded to a multiple of 256 and K' to a multiple of 128 with zero codes.
// ---------------------------------------------------------------------------------------------
constexpr int XQ_ROW_BLOCK = 16;
constexpr int XQ_K_GROUP = 32;                                   // codes per 16-byte piece
constexpr int XQ_GROUP_BYTES = XQ_ROW_BLOCK * XQ_K_GROUP / 2;    // 256: one group of one block
constexpr int XQ_K_BLOCK = 128;
constexpr int XQ_ROW_PAD = 256;

struct xq_weights {
  int32_t N, K, Kp;    // logical sizes (head-wise: K = heads * head_dim, Kp = heads * head_dim')
  int32_t heads;       // 1: one rotation over the whole row (plan is K -> Kp); > 1: the plan is that of one head
  int32_t Np, Kpp;     // padded sizes (multiples of 256 and 128)
  xq_hadamard_plan_t plan;
  uint8_t* packed;     // device, Np * Kpp / 2 bytes, block layout above
  float* s_w;          // device, Np floats (padding rows hold 0)
  int32_t* w_sum;      // device, Np ints: sum of the row's codes (the zero-point term of asymmetric tokens)
  uint16_t* head_signs;  // device, head-wise only: bf16 image of the truncated head matrix, [head_dim'][head_dim16 + 8]
  uint16_t* hp_signs;  // device, bf16 image of H_p^T for the rotate kernel ([P16][P16 + 8]); NULL when p == 1
  int device;
  int sms;             // multiprocessors of that device
};

// NVTX range around one entry point of the library (shows as a named span on the host timeline of a profiler; costs a
// pointer test when none is attached).
struct XqRange {
  explicit XqRange(const char* name) { nvtxRangePushA(name); }
  ~XqRange() { nvtxRangePop(); }
  XqRange(const XqRange&) = delete;
  XqRange& operator=(const XqRange&) = delete;
};
#define XQ_RANGE() XqRange xq_range_(__func__)

// True when `device` (the one a weights object lives on) is the current device: the kernels dereference the
// object's pointers, so a call made with another device current is refused on the host.
inline bool xq_on_device(int device) {
  int cur = -1;
  if (cudaGetDevice(&cur) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  return cur == device;
}

// Byte offset of the 32-bit word holding codes 8*kg .. 8*kg+7 of row n (k_groups = K'' / 32).
__host__ __device__ inline size_t xq_weight_word_offset(int n, int kg, int k_groups) {
  const int blk = n >> 4, r = n & 15, grp = kg >> 2, word = kg & 3;
  return ((size_t)blk * k_groups + grp) * XQ_GROUP_BYTES + (size_t)r * 16 + (size_t)word * 4;
}

// Workspace layout (all offsets multiples of 256 bytes).  The header is what xq_workspace_init
// clears: word 0 is the sticky status.
constexpr size_t XQ_WS_HEADER_BYTES = 256;
// MXFP4 workspaces: status word, then (from byte 256) one arrival counter per 128-channel tile of the split-K
// small-batch product; xq_workspace_init clears this much of a workspace that is at least this large.
constexpr size_t XQ_WS_COUNTER_BYTES = 1024;
struct xq_ws_layout {
  size_t header;   // XQ_WS_HEADER_BYTES
  size_t xq;       // M_max * Kp/2 bytes of packed activations
  size_t sx;       // M_max floats
  size_t zp;       // M_max ints: zero points of asymmetric activation codes
  size_t xstage;   // M_max * K bf16 (host entry point)
  size_t ostage;   // M_max * N bf16 (host entry point)
  size_t a8;       // M_max * K'' bytes: byte-per-code tokens for the tensor-core GEMM (only when M_max > 32)
  size_t total;
};
xq_ws_layout xq_ws_compute(int32_t M_max, const xq_weights* w);
// bf16 image of H_p^T (row a', column a; [P16][P16 + 8]) in device memory: a constant of the plan that the one-row
// rotate kernel reads.  *out stays null for plans without one.  False when the allocation or the copy fails.
bool xq_make_hp_signs(const xq_hadamard_plan_t& pl, uint16_t** out);
// bf16 image of the truncated matrix of one head (row c' = output channel, column c = input channel;
// [head_dim'][head_dim16 + 8]) for the head-wise rotate kernel.
bool xq_make_head_signs(const xq_hadamard_plan_t& pl, uint16_t** out);

// Size of the built-in scratch array of xq_expanded_linear_static.
constexpr size_t XQ_STATIC_SCRATCH_BYTES = 4u << 20;

constexpr int XQ_MAX_P = 8192;        // largest order-p factor (the general rotate kernel; its shared memory bounds K' too)
constexpr int XQ_MAX_P_IMAGE = 256;   // largest p with a sign-matrix image (the kernels that read it stop there)
constexpr int XQ_DECODE_MAX_M = 32;

// MXFP4 outputs of the online step in the layout the block-scaled GEMM reads: codes [rows][Kq / 2]
// bytes (Kq = K' rounded up to 256, padding zero), scale bytes in 512-byte blocks of 128 rows x 4
// groups: byte of (row m, group g) at xq_mx_sf_offset.
struct xq_mx_out {
  uint8_t* codes;
  uint8_t* sf_blocks;
  int32_t Kq;
};
__host__ __device__ inline size_t xq_mx_sf_offset(int m, int g, int Kq) {
  return ((size_t)(m >> 7) * (Kq >> 7) + (g >> 2)) * 512 + (size_t)(m & 31) * 16 + (size_t)((m >> 5) & 3) * 4 + (g & 3);
}
// True when xq_launch_rotate_mx can emit them directly (otherwise the caller quantizes the fp32 rows).
bool xq_rotate_mx_supported(const xq_hadamard_plan_t& pl);
cudaError_t xq_launch_rotate_mx(const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t& pl, const xq_mx_out& mx, int sms,
                                cudaStream_t st);
// The same from the one-row-per-CTA tensor-core kernel (few rows); cudaErrorNotSupported when the plan is not one of its.
cudaError_t xq_launch_rotate_tc_mx(const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t& pl, const xq_mx_out& mx,
                                   const void* Hsigns, int sms, cudaStream_t st);

// Launchers (each returns the CUDA error of its launch).
// A8opt (optional): byte-per-code copy of the codes in the operand format of the tcgen05 GEMM, [M, Kp].
// Hsigns (optional): device image of H_p^T as bf16, [P16][P16 + 8] with P16 = p rounded up to 16
// (xq_weights::hp_signs); without it the kernel derives the signs itself.
// zp (optional): when given, the rows are quantized asymmetrically (unsigned codes 0..15) and zp[m]
// receives the row's zero point; when null, symmetrically (signed codes -8..7).
cudaError_t xq_launch_rotate_quant(const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t& pl,
                                   uint8_t* Xq, float* sx, float* Yopt, uint8_t* A8opt, const void* Hsigns, int32_t* zp,
                                   int sms, cudaStream_t st);
// Throughput form for many rows (several independent row groups per CTA, double-buffered loads).
bool xq_rotate_rows_supported(const xq_hadamard_plan_t& pl);
cudaError_t xq_launch_rotate_rows(const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t& pl, uint8_t* Xq, float* sx,
                                  float* Yopt, uint8_t* A8opt, int32_t* zp, int sms, cudaStream_t st);
// Head-wise form (the row is `heads` blocks of pl.K channels, each rotated by the plan's matrix; one
// quantizer over the whole row).  Bimage (optional): xq_weights::head_signs.
bool xq_rotate_heads_supported(const xq_hadamard_plan_t& pl, int32_t heads);
size_t xq_head_image_elems(const xq_hadamard_plan_t& pl);
cudaError_t xq_launch_rotate_heads(const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t& pl, int32_t heads, uint8_t* Xq,
                                   float* sx, float* Yopt, uint8_t* A8opt, const void* Bimage, int32_t* zp, int sms,
                                   cudaStream_t st, const struct xq_mx_out* mx = nullptr);  // mx: MXFP4 outputs instead (Xq, sx, zp, A8opt unused)
// The online step of a layer, whichever form its weights were prepared with.
inline cudaError_t xq_launch_rotate_for(const xq_weights* w, const void* X, int32_t M, int64_t ldx, uint8_t* Xq, float* sx,
                                        uint8_t* A8opt, int32_t* zp, cudaStream_t st);
constexpr int XQ_ROTATE_ROWS_MIN_M = 48;  // below this the one-CTA-per-row kernel has the shorter latency
cudaError_t xq_launch_relayout_to_blocks(const uint8_t* canon, int32_t N, int32_t Kp, uint8_t* blocks,
                                         int32_t Np, int32_t Kpp, cudaStream_t st);
cudaError_t xq_launch_relayout_from_blocks(const uint8_t* blocks, int32_t Np, int32_t Kpp, uint8_t* canon,
                                           int32_t N, int32_t Kp, cudaStream_t st);
cudaError_t xq_launch_pack_codes(const int8_t* codes, int64_t count_pairs, uint8_t* packed, cudaStream_t st);
cudaError_t xq_launch_unpack_codes(const uint8_t* packed, int64_t count_pairs, int8_t* codes, cudaStream_t st);
// w_sum[n] = sum of the codes of row n of the block layout (0 for padding rows).
cudaError_t xq_launch_weight_sums(const uint8_t* blocks, int32_t Np, int32_t Kpp, int32_t* w_sum, cudaStream_t st);
// Decode path: returns cudaErrorNotSupported (nothing launched) when the shape does not fit it.
// zp (optional, here and below): per-token zero points; the epilogue then removes zp[m] * w_sum[n].
cudaError_t xq_launch_gemm_decode(const uint8_t* Xq, const float* sx, const int32_t* zp, int32_t M, const xq_weights* w,
                                  void* out, int32_t* acc_opt, int32_t* status, cudaStream_t st);
// The whole layer for M <= 32 tokens in one launch: the decode kernel with the online step (pad, rotate, quantize)
// inside.  Xq, sx, zp (zp null: symmetric codes) are workspace arrays the kernel fills and reads; header is the
// workspace header (status word, generation, exit count, row flags).  cudaErrorNotSupported (nothing launched) when
// the plan or the shape is not one it takes.
bool xq_linear_decode_supported(int32_t M, const xq_weights* w);
cudaError_t xq_launch_linear_decode(const void* X, int64_t ldx, uint8_t* Xq, float* sx, int32_t* zp, int32_t M, const xq_weights* w,
                                    void* out, int32_t* header, cudaStream_t st);
// True when M tokens against w run in the decode kernel; then also its padded token count and cluster size.
bool xq_decode_shape(int32_t M, const xq_weights* w, int* padded_tokens, int* cluster);
// Tile shape the tensor-core path picks: 0 = 128 tokens x 256 channels, 1 = 256 x 256, 2 = 256 x 128, 3 = 256 x 224
// (first form: expanded weights in shared memory); 4 = *ts_tokens tokens x 256 channels in the second form (expanded
// weights in tensor memory).
#define XQ_TS_MAX_TOKENS 192
int xq_prefill_tile_choice(int32_t M, const xq_weights* w, int sms, int* ts_tokens);
cudaError_t xq_launch_gemm_prefill_ts(const uint8_t* A8, const float* sx, const int32_t* zp, int32_t M, const xq_weights* w, void* out,
                                      int32_t* acc_opt, int32_t* status, int tile_tokens, int sms, cudaStream_t st);
// cuTensorMapEncodeTiled through the runtime's driver entry point lookup (null when the driver lacks it).
typedef CUresult (*XqEncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                    const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
XqEncodeTiledFn xq_encode_tiled_fn();
// Tensor-core path: takes the tokens one code per byte (16 x code, even codes of every word first),
// as written by the rotate kernels' optional output or by xq_launch_expand_tokens.
bool xq_prefill_supported(int32_t M, const xq_weights* w);
cudaError_t xq_launch_expand_tokens(const uint8_t* Xq, int32_t M, int32_t Kp, uint8_t* A8, cudaStream_t st);
cudaError_t xq_launch_gemm_prefill(const uint8_t* A8, const float* sx, const int32_t* zp, int32_t M, const xq_weights* w,
                                   void* out, int32_t* acc_opt, int32_t* status, int sms, cudaStream_t st);
// True when M tokens against w go down the tensor-core path (so that the caller lets the rotate
// kernel write the byte-per-code tokens).
cudaError_t xq_launch_selftest_wait_timeout(int32_t* status, cudaStream_t st);
bool xq_gemm_wants_a8(int32_t M, const xq_weights* w);
// Tensor-core issue-rate probe: one CTA per multiprocessor, iters * 4 MMAs of 128 x 256 x 32 (kind::i8) each.
cudaError_t xq_launch_i8_mma_rate(int iters, int32_t* status, int sms, cudaStream_t st);
// a8_ready: the a8 region of the workspace already holds the byte-per-code tokens.
cudaError_t xq_launch_gemm(const uint8_t* Xq, const float* sx, const int32_t* zp, int32_t M, const xq_weights* w, void* out,
                           int32_t* acc_opt, void* ws, const xq_ws_layout& L, bool a8_ready, cudaStream_t st);

inline cudaError_t xq_launch_rotate_for(const xq_weights* w, const void* X, int32_t M, int64_t ldx, uint8_t* Xq, float* sx,
                                        uint8_t* A8opt, int32_t* zp, cudaStream_t st) {
  if (w->heads > 1)
    return xq_launch_rotate_heads(X, M, ldx, w->plan, w->heads, Xq, sx, nullptr, A8opt, w->head_signs, zp, w->sms, st);
  return xq_launch_rotate_quant(X, M, ldx, w->plan, Xq, sx, nullptr, A8opt, w->hp_signs, zp, w->sms, st);
}
