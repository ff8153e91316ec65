// Online step of the expanded layer (paper Sec. 3: X_hat = X H_hat; Sec. 4: per-token 4-bit):
// fused zero-pad + Kronecker Hadamard (H_p (x) Sylvester) + per-row absmax + INT4 pack.
// The same kernels prepare weight rows offline.
#include <cuda_bf16.h>

#include "xq_internal.h"
#include "xq_hadamard.cuh"
#include "xq_ptx.cuh"
#include "xq_rotate_row.cuh"

using namespace xqhad;

namespace {

// Per-row symmetric INT4: scale = absmax / 7 (1 for a zero row); code = clamp(rne(y / s), -8, 7).
__device__ __forceinline__ int quant_code(float y, float s) {
  int q = __float2int_rn(__fdiv_rn(y, s));
  return max(-8, min(7, q));
}

// ---------------------------------------------------------------------------------------------
// General kernel: any plan, one CTA per row, everything in shared memory.  It is the fallback
// for orders without a specialised kernel and the shape-agnostic reference inside the library.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) rotate_quant_general_kernel(const __nv_bfloat16* __restrict__ X, int M,
                                                                   long long ldx, xq_hadamard_plan_t pl, float gamma,
                                                                   uint8_t* __restrict__ Xq, float* __restrict__ sx,
                                                                   float* __restrict__ Yopt, uint8_t* __restrict__ A8opt,
                                                                   int32_t* __restrict__ zp) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int K = pl.K, Kp = pl.Kp, p = pl.p, n = 1 << pl.log2n, q = pl.q;
  float* bufA = reinterpret_cast<float*>(smem_raw);
  float* bufB = bufA + Kp;
  float* red = bufB + Kp;
  int8_t* chi2 = reinterpret_cast<int8_t*>(red + 32);
  int8_t* sq = chi2 + 2 * q + 1;
  if (p > 1) build_chi(q, chi2, sq, pl.paley_kind);
  const int rows_a = (K + n - 1) / n;  // rows of the p x n view that can be non-zero

  for (int row = blockIdx.x; row < M; row += gridDim.x) {
    const __nv_bfloat16* x = X + (long long)row * ldx;
    for (int c = threadIdx.x; c < Kp; c += blockDim.x) bufA[c] = c < K ? __bfloat162float(x[c]) : 0.f;
    __syncthreads();
    float* y = bufA;
    if (p > 1) {
      // outer factor: t[a2][b] = sum_a H_p[a][a2] v[a][b]
      for (int o = threadIdx.x; o < Kp; o += blockDim.x) {
        const int a2 = o / n, b = o - a2 * n;
        float acc = 0.f;
        for (int a = 0; a < rows_a; ++a) {
          const float v = bufA[a * n + b];
          acc += paley_sign(pl.paley_kind, q, chi2, a, a2) > 0 ? v : -v;
        }
        bufB[o] = acc;
      }
      __syncthreads();
      y = bufB;
    }
    // inner factor: Walsh-Hadamard butterflies along b
    for (int h = 1; h < n; h <<= 1) {
      for (int i = threadIdx.x; i < Kp / 2; i += blockDim.x) {
        const int lo = i & (h - 1);
        const int j = ((i - lo) << 1) + lo;
        const float u = y[j], w = y[j + h];
        y[j] = u + w;
        y[j + h] = u - w;
      }
      __syncthreads();
    }
    float vmax = 0.f, vmin = 0.f;
    for (int c = threadIdx.x; c < Kp; c += blockDim.x) {
      const float v = y[c] * gamma;
      y[c] = v;
      vmax = fmaxf(vmax, v);
      vmin = fminf(vmin, v);
    }
    RowQuant rq;
    if (zp) {
      vmax = block_max(vmax, red);
      vmin = -block_max(-vmin, red);
      rq = row_quant_asym(vmin, vmax);
      if (threadIdx.x == 0) zp[row] = rq.z;
    } else {
      rq = row_quant_sym(block_max(fmaxf(vmax, -vmin), red));
    }
    if (threadIdx.x == 0) sx[row] = rq.s;
    uint8_t* out = Xq + (long long)row * (Kp / 2);
    for (int j = threadIdx.x; j < Kp / 2; j += blockDim.x) {
      const int lo = zp ? row_code(rq, y[2 * j]) : quant_code(y[2 * j], rq.s);
      const int hi = zp ? row_code(rq, y[2 * j + 1]) : quant_code(y[2 * j + 1], rq.s);
      out[j] = (uint8_t)((lo & 0xF) | ((hi & 0xF) << 4));
      if (A8opt) {
        // operand format of the tcgen05 GEMM: word kg of 8 codes -> 4 bytes of even codes x16, 4 of odd
        uint8_t* a8 = A8opt + (long long)row * Kp + (j >> 2) * 8 + (j & 3);
        a8[0] = (uint8_t)(lo << 4);
        a8[4] = (uint8_t)(hi << 4);
      }
    }
    if (Yopt)
      for (int c = threadIdx.x; c < Kp; c += blockDim.x) Yopt[(long long)row * Kp + c] = y[c];
    __syncthreads();
  }
}

// ---------------------------------------------------------------------------------------------
// Tensor-core kernel for p > 1, 32 <= n <= 256, ceil(K / n) <= 64: one CTA per row, all of its warps on
// that row (the row routine and its description: xq_rotate_row.cuh).
// ---------------------------------------------------------------------------------------------
template <int LOG2NB, int KS>
__global__ void __launch_bounds__(512) rotate_quant_tc_kernel(const __nv_bfloat16* __restrict__ X, int M, long long ldx,
                                                              xq_hadamard_plan_t pl, float gamma, uint8_t* __restrict__ Xq,
                                                              float* __restrict__ sx, float* __restrict__ Yopt,
                                                              uint8_t* __restrict__ A8opt, const __nv_bfloat16* __restrict__ Hsigns,
                                                              int32_t* __restrict__ zp, uint8_t* __restrict__ sfb, int Kq) {
  // sfb != null: MXFP4 instead of per-row INT4 -- a shared exponent per 32 channels, E2M1 codes; Xq then has the row
  // pitch Kq / 2 and the scale bytes go to sfb in the block layout of the block-scaled GEMM (sx, zp, A8opt unused).
  constexpr int NB = 1 << LOG2NB;  // columns per warp
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int K = pl.K, Kp = pl.Kp, p = pl.p, n = 1 << pl.log2n, q = pl.q;
  const int NC = n / NB;            // column chunks (1, 2 or 4)
  const int pitch = n + 8;          // bf16 elements per staged row (conflict-free ldmatrix)
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int mt = warp / NC;
  const int nthreads = blockDim.x;

  __nv_bfloat16* Xs = reinterpret_cast<__nv_bfloat16*>(smem_raw);
  uint32_t* outp = reinterpret_cast<uint32_t*>(Xs + KS * 16 * pitch);  // Kp / 8 words
  uint8_t* sfs = reinterpret_cast<uint8_t*>(outp + Kp / 8);           // Kp / 32 scale bytes of the row (MXFP4)
  float* red = reinterpret_cast<float*>(sfs + (Kp / 32 + 15) / 16 * 16);  // 32 floats
  int8_t* chi2 = reinterpret_cast<int8_t*>(red + 32);
  int8_t* sq = chi2 + 2 * q + 1;
  // shared image of H_p^T (only when the caller has one ready in global memory), then the exchange buffer
  const int P16 = (p + 15) / 16 * 16, hpitch = P16 + 8;
  __nv_bfloat16* Hs = reinterpret_cast<__nv_bfloat16*>(smem_raw + (((size_t)(sq + q - reinterpret_cast<int8_t*>(smem_raw)) + 15) & ~(size_t)15));
  float* exch = reinterpret_cast<float*>(Hs + (Hsigns ? P16 * hpitch : 0));

  xqptx::pdl_launch_dependents();
  // A = H_p^T, rows a' = 16 mt + {g, g+8}, k = a = 16 ks + {2t, 2t+1, 2t+8, 2t+9}
  uint32_t afrag[KS][4];
  if (Hsigns) {
    // the sign matrix was prepared with the weights (it is a constant of the plan): fetch the
    // image and read the fragments with ldmatrix -- a few hundred nanoseconds instead of the
    // table build and 8 KS sign evaluations per thread below
    for (int i = tid; i < P16 * hpitch / 8; i += nthreads) xqptx::cp_async16(Hs + 8 * i, Hsigns + 8 * i);
    xqptx::cp_async_wait_all();
    __syncthreads();
    xqrot::load_afrag<KS>(afrag, Hs, P16, hpitch, mt, lane);
  } else {
  build_chi(q, chi2, sq, pl.paley_kind);
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int a2 = 16 * mt + g + (r & 1) * 8;
      const int a = 16 * ks + 2 * t + (r >> 1) * 8;
      uint32_t lo = 0, hi = 0;
      if (a2 < p) {
        if (a < p) lo = sign_bf16(paley_sign(pl.paley_kind, q, chi2, a, a2));
        if (a + 1 < p) hi = sign_bf16(paley_sign(pl.paley_kind, q, chi2, a + 1, a2));
      }
      afrag[ks][r] = lo | (hi << 16);
    }
  }
  }
  // zero the staged rows once: rows past the data and the tail of a partial last row stay zero
  for (int i = tid; i < KS * 16 * pitch / 8; i += nthreads) reinterpret_cast<uint4*>(Xs)[i] = make_uint4(0, 0, 0, 0);
  xqptx::pdl_wait();
  __syncthreads();

  const xqrot::RowSmem sm = {Xs, outp, sfs, red, exch};
  const xqrot::RowOut out = {Xq, sx, Yopt, A8opt, zp, sfb, Kq};
  const int chunks = K / 8;  // 16-byte pieces of a row
  for (int row = blockIdx.x; row < M; row += gridDim.x) {
    const __nv_bfloat16* x = X + (long long)row * ldx;
    for (int i = tid; i < chunks; i += nthreads) {
      const int c = 8 * i, a = c >> pl.log2n, b = c & (n - 1);
      xqptx::cp_async16(Xs + a * pitch + b, x + c);
    }
    xqptx::cp_async_wait_all();
    __syncthreads();
    xqrot::rotate_row<LOG2NB, KS>(pl, gamma, afrag, sm, out, row, tid, nthreads, xqrot::CtaSync());
  }
}

template <int LOG2NB, int KS>
cudaError_t launch_tc(const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t& pl, float gamma, uint8_t* Xq, float* sx,
                      float* Yopt, uint8_t* A8opt, const void* Hsigns, int32_t* zp, int sms, cudaStream_t st,
                      const xq_mx_out* mx = nullptr) {
  const int n = 1 << pl.log2n, NB = 1 << LOG2NB, NC = n / NB, MT = (pl.p + 15) / 16;  // NC = xqrot::row_chunks(pl)
  size_t smem = (size_t)KS * 16 * (n + 8) * 2 + (size_t)pl.Kp / 2 + (size_t)pl.Kp / 32 + 16 + 128 + (size_t)(3 * pl.q + 1) + 32;
  if (mx) Xq = mx->codes;
  if (Hsigns) smem += (size_t)MT * 16 * (MT * 16 + 8) * 2;
  if (NC > 1) smem += (size_t)MT * 8 * (n + 8) * 4;
  auto kern = rotate_quant_tc_kernel<LOG2NB, KS>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int per_sm = smem > 100 * 1024 ? 1 : (smem > 48 * 1024 ? 2 : 4);
  const int grid = M < sms * per_sm ? M : sms * per_sm;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(32 * MT * NC);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, (const __nv_bfloat16*)X, (int)M, (long long)ldx, pl, gamma, Xq, sx, Yopt, A8opt,
                            (const __nv_bfloat16*)Hsigns, zp,
                            mx ? mx->sf_blocks : (uint8_t*)nullptr, mx ? (int)mx->Kq : 0);
}

template <int LOG2NB>
cudaError_t launch_tc_ks(int ks, const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t& pl, float gamma, uint8_t* Xq,
                         float* sx, float* Yopt, uint8_t* A8opt, const void* Hsigns, int32_t* zp, int sms, cudaStream_t st,
                         const xq_mx_out* mx = nullptr) {
  switch (ks) {
    case 1: return launch_tc<LOG2NB, 1>(X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, Hsigns, zp, sms, st, mx);
    case 2: return launch_tc<LOG2NB, 2>(X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, Hsigns, zp, sms, st, mx);
    case 3: return launch_tc<LOG2NB, 3>(X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, Hsigns, zp, sms, st, mx);
    default: return launch_tc<LOG2NB, 4>(X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, Hsigns, zp, sms, st, mx);
  }
}

// ---------------------------------------------------------------------------------------------
// Layout helpers (offline paths).
// ---------------------------------------------------------------------------------------------
__global__ void relayout_to_blocks_kernel(const uint8_t* __restrict__ canon, int N, int Kp, uint32_t* __restrict__ blocks,
                                          int Np, int Kpp) {
  const int k_groups = Kpp / XQ_K_GROUP, words_per_row = Kpp / 8, row_bytes = Kp / 2;
  const long long total = (long long)Np * words_per_row;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int n = (int)(i / words_per_row), kg = (int)(i % words_per_row);
    uint32_t w = 0;
    if (n < N) {
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int byte = 4 * kg + b;
        if (byte < row_bytes) w |= (uint32_t)canon[(long long)n * row_bytes + byte] << (8 * b);
      }
    }
    blocks[xq_weight_word_offset(n, kg, k_groups) / 4] = w;
  }
}

__global__ void relayout_from_blocks_kernel(const uint32_t* __restrict__ blocks, int Np, int Kpp, uint8_t* __restrict__ canon,
                                            int N, int Kp) {
  const int k_groups = Kpp / XQ_K_GROUP, row_bytes = Kp / 2;
  const long long total = (long long)N * row_bytes;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int n = (int)(i / row_bytes), byte = (int)(i % row_bytes);
    const uint32_t w = blocks[xq_weight_word_offset(n, byte >> 2, k_groups) / 4];
    canon[i] = (uint8_t)(w >> (8 * (byte & 3)));
  }
}

__global__ void pack_codes_kernel(const int8_t* __restrict__ codes, long long pairs, uint8_t* __restrict__ packed) {
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < pairs; i += (long long)gridDim.x * blockDim.x)
    packed[i] = (uint8_t)((codes[2 * i] & 0xF) | ((codes[2 * i + 1] & 0xF) << 4));
}

__global__ void unpack_codes_kernel(const uint8_t* __restrict__ packed, long long pairs, int8_t* __restrict__ codes) {
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < pairs; i += (long long)gridDim.x * blockDim.x) {
    const int b = packed[i];
    codes[2 * i] = (int8_t)(((b & 0xF) ^ 8) - 8);
    codes[2 * i + 1] = (int8_t)(((b >> 4) ^ 8) - 8);
  }
}

// One warp per row of the block layout: the sum of its K'' signed nibbles (padding holds zeros).
__global__ void weight_sums_kernel(const uint8_t* __restrict__ blocks, int Np, int Kpp, int32_t* __restrict__ w_sum) {
  const int n = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (n >= Np) return;
  const int k_groups = Kpp / XQ_K_GROUP;
  int acc = 0;
  for (int kg = lane; kg < Kpp / 8; kg += 32) {
    const uint32_t w = *reinterpret_cast<const uint32_t*>(blocks + xq_weight_word_offset(n, kg, k_groups));
#pragma unroll
    for (int i = 0; i < 8; ++i) acc += (int)(w << (28 - 4 * i)) >> 28;
  }
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) w_sum[n] = acc;
}

inline int grid_for(long long work, int threads) {
  long long g = (work + threads - 1) / threads;
  if (g < 1) g = 1;
  if (g > 148 * 32) g = 148 * 32;
  return (int)g;
}

}  // namespace

cudaError_t xq_launch_rotate_quant(const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t& pl, uint8_t* Xq,
                                   float* sx, float* Yopt, uint8_t* A8opt, const void* Hsigns, int32_t* zp, int sms, cudaStream_t st) {
  const float gamma = (float)(1.0 / sqrt((double)pl.Kp));
  const int n = 1 << pl.log2n;
  const int rows_a = (pl.K + n - 1) / n;
  const bool tc = xqrot::plan_supported(pl);
  // many rows, or an order that only the multi-row-group kernel and the general kernel take
  if ((M >= XQ_ROTATE_ROWS_MIN_M || !tc) && xq_rotate_rows_supported(pl))
    return xq_launch_rotate_rows(X, M, ldx, pl, Xq, sx, Yopt, A8opt, zp, sms, st);
  if (tc) {
    const int ks = (rows_a + 15) / 16;
    switch (pl.log2n) {
      case 5: return launch_tc_ks<5>(ks, X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, Hsigns, zp, sms, st);
      default: return launch_tc_ks<6>(ks, X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, Hsigns, zp, sms, st);
    }
  }
  const size_t smem = sizeof(float) * (2 * (size_t)pl.Kp + 32) + (size_t)(3 * pl.q + 1) + 16;
  cudaError_t e = cudaFuncSetAttribute(rotate_quant_general_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int grid = M < sms * 8 ? M : sms * 8;
  rotate_quant_general_kernel<<<grid, 256, smem, st>>>((const __nv_bfloat16*)X, M, (long long)ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp);
  return cudaGetLastError();
}

cudaError_t xq_launch_rotate_tc_mx(const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t& pl, const xq_mx_out& mx,
                                   const void* Hsigns, int sms, cudaStream_t st) {
  const float gamma = (float)(1.0 / sqrt((double)pl.Kp));
  const int n = 1 << pl.log2n;
  const int rows_a = (pl.K + n - 1) / n;
  const bool tc = xqrot::plan_supported(pl);
  if (!tc || pl.Kp % 32 != 0) return cudaErrorNotSupported;
  const int ks = (rows_a + 15) / 16;
  switch (pl.log2n) {
    case 5: return launch_tc_ks<5>(ks, X, M, ldx, pl, gamma, mx.codes, nullptr, nullptr, nullptr, Hsigns, nullptr, sms, st, &mx);
    default: return launch_tc_ks<6>(ks, X, M, ldx, pl, gamma, mx.codes, nullptr, nullptr, nullptr, Hsigns, nullptr, sms, st, &mx);
  }
}

cudaError_t xq_launch_relayout_to_blocks(const uint8_t* canon, int32_t N, int32_t Kp, uint8_t* blocks, int32_t Np,
                                         int32_t Kpp, cudaStream_t st) {
  const long long work = (long long)Np * (Kpp / 8);
  relayout_to_blocks_kernel<<<grid_for(work, 256), 256, 0, st>>>(canon, N, Kp, (uint32_t*)blocks, Np, Kpp);
  return cudaGetLastError();
}

cudaError_t xq_launch_relayout_from_blocks(const uint8_t* blocks, int32_t Np, int32_t Kpp, uint8_t* canon, int32_t N,
                                           int32_t Kp, cudaStream_t st) {
  const long long work = (long long)N * (Kp / 2);
  relayout_from_blocks_kernel<<<grid_for(work, 256), 256, 0, st>>>((const uint32_t*)blocks, Np, Kpp, canon, N, Kp);
  return cudaGetLastError();
}

cudaError_t xq_launch_weight_sums(const uint8_t* blocks, int32_t Np, int32_t Kpp, int32_t* w_sum, cudaStream_t st) {
  weight_sums_kernel<<<(Np + 3) / 4, 128, 0, st>>>(blocks, Np, Kpp, w_sum);
  return cudaGetLastError();
}

cudaError_t xq_launch_pack_codes(const int8_t* codes, int64_t pairs, uint8_t* packed, cudaStream_t st) {
  pack_codes_kernel<<<grid_for(pairs, 256), 256, 0, st>>>(codes, pairs, packed);
  return cudaGetLastError();
}

cudaError_t xq_launch_unpack_codes(const uint8_t* packed, int64_t pairs, int8_t* codes, cudaStream_t st) {
  unpack_codes_kernel<<<grid_for(pairs, 256), 256, 0, st>>>(packed, pairs, codes);
  return cudaGetLastError();
}
