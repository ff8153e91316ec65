// Quantized product of the expanded layer (paper Sec. 3: Q(XR) Q(W~), computed at inference)
// with the dequantizing epilogue: acc = sum_c (qx - z) qw (int32, exact; z = 0 for symmetric
// tokens, else sum_c qx qw - z sum_c qw), out = bf16(acc s_x s_w).
#include <cuda_bf16.h>

#include "xq_internal.h"
#include "xq_ptx.cuh"

using xqptx::split16;

namespace {

// General kernel: one thread per output, any M, N, K' (K' a multiple of 8).  Shape-agnostic
// path for sizes the tiled kernels do not take.
__global__ void __launch_bounds__(128) gemm_general_kernel(const uint32_t* __restrict__ Xq, const float* __restrict__ sx,
                                                           const int32_t* __restrict__ zp, const int32_t* __restrict__ wsum, int M,
                                                           const uint8_t* __restrict__ Wb, const float* __restrict__ sw, int N,
                                                           int Kp, int k_groups, __nv_bfloat16* __restrict__ out,
                                                           int32_t* __restrict__ acc_opt) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  const int m = blockIdx.y;
  if (n >= N || m >= M) return;
  const int words = Kp / 8;
  const uint32_t* xrow = Xq + (long long)m * words;
  int acc = 0;
  for (int kg = 0; kg < words; ++kg) {
    const uint32_t w = *reinterpret_cast<const uint32_t*>(Wb + xq_weight_word_offset(n, kg, k_groups));
    uint32_t we, wo, xe, xo;
    split16(w, we, wo);
    split16(xrow[kg], xe, xo);
    acc = __dp4a((int)we, (int)xe, acc);
    acc = __dp4a((int)wo, (int)xo, acc);
  }
  acc >>= 8;
  if (zp) acc -= zp[m] * wsum[n];
  if (acc_opt) acc_opt[(long long)m * N + n] = acc;
  out[(long long)m * N + n] = __float2bfloat16_rn((float)acc * sx[m] * sw[n]);
}

// One warp waits on a barrier that nobody arrives at: exercises the bounded wait and the status
// word without any fault, trap or endless loop.
__global__ void selftest_wait_timeout_kernel(int32_t* status) {
  __shared__ uint64_t bar;
  __shared__ int failed;
  if (threadIdx.x == 0) {
    xqptx::mbar_init(&bar, 1);
    failed = 0;
    xqptx::mbar_fence_init();
  }
  __syncwarp();
  xqptx::mbar_wait_bounded(&bar, 0, &failed, status, (int)XQ_ERR_TIMEOUT);
}

}  // namespace

cudaError_t xq_launch_selftest_wait_timeout(int32_t* status, cudaStream_t st) {
  selftest_wait_timeout_kernel<<<1, 32, 0, st>>>(status);
  return cudaGetLastError();
}

bool xq_gemm_wants_a8(int32_t M, const xq_weights* w) { return M > XQ_DECODE_MAX_M && xq_prefill_supported(M, w); }

cudaError_t xq_launch_gemm(const uint8_t* Xq, const float* sx, const int32_t* zp, int32_t M, const xq_weights* w, void* out,
                           int32_t* acc_opt, void* ws, const xq_ws_layout& L, bool a8_ready, cudaStream_t st) {
  if (w->Kp % 8 != 0) return cudaErrorInvalidValue;
  int32_t* header = (int32_t*)ws;
  if (M <= XQ_DECODE_MAX_M) {
    const cudaError_t e = xq_launch_gemm_decode(Xq, sx, zp, M, w, out, acc_opt, header, st);
    if (e != cudaErrorNotSupported) return e;
  }
  if (xq_prefill_supported(M, w) && L.a8 != 0) {
    uint8_t* A8 = (uint8_t*)ws + L.a8;
    if (!a8_ready) {
      const cudaError_t e = xq_launch_expand_tokens(Xq, M, w->Kp, A8, st);
      if (e != cudaSuccess) return e;
    }
    return xq_launch_gemm_prefill(A8, sx, zp, M, w, out, acc_opt, header, w->sms, st);
  }
  dim3 grid((w->N + 127) / 128, M);
  gemm_general_kernel<<<grid, 128, 0, st>>>((const uint32_t*)Xq, sx, zp, w->w_sum, M, w->packed, w->s_w, w->N, w->Kp,
                                            w->Kpp / XQ_K_GROUP, (__nv_bfloat16*)out, acc_opt);
  return cudaGetLastError();
}

// Which of the three product kernels xq_launch_gemm takes for M tokens against w (the same tests, nothing launched).
extern "C" xq_status xq_gemm_kernel_info(int32_t M, const xq_weights* w, int32_t* kind, int32_t* tile_tokens, int32_t* tile_channels) {
  if (!w || M < 1 || !kind || !tile_tokens || !tile_channels) return XQ_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  if (dev != w->device) return XQ_ERR_INVALID_ARG;
  int mt = 0, cluster = 0;
  if (M <= XQ_DECODE_MAX_M && xq_decode_shape(M, w, &mt, &cluster)) {
    *kind = 0;
    *tile_tokens = mt;
    *tile_channels = 16;
  } else if (xq_gemm_wants_a8(M, w)) {
    int ts_tokens = 0;
    const int c = xq_prefill_tile_choice(M, w, w->sms, &ts_tokens);
    *kind = c == 4 ? 3 : 1;
    *tile_tokens = c == 4 ? ts_tokens : (c == 0 ? 128 : 256);
    *tile_channels = c == 2 ? 128 : (c == 3 ? 224 : 256);
  } else {
    *kind = 2;
    *tile_tokens = 1;
    *tile_channels = 1;
  }
  return XQ_OK;
}
