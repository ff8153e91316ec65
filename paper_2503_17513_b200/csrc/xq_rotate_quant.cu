// Online step of the expanded layer (paper Sec. 3: X_hat = X H_hat; Sec. 4: per-token 4-bit):
// fused zero-pad + Kronecker Hadamard (H_p (x) Sylvester) + per-row absmax + INT4 pack.
// The same kernels prepare weight rows offline.
#include <cuda_bf16.h>

#include "xq_internal.h"

namespace {

// ---------------------------------------------------------------------------------------------
// Sign of entry (a, a2) of the order-p Paley factor from the quadratic-character table of GF(q).
// chi2 is indexed by d + q for d in (-q, q): chi2[d + q] = chi(d mod q), chi(0) = 0.
// Paley-I:  first row +1, first column -1 below it, core chi(i - j) + identity.
// Paley-II: symmetric S of order q + 1 (zero diagonal, border +1, core chi(i - j)); each entry s
//           becomes s * [[1, 1], [1, -1]], each diagonal zero becomes [[1, -1], [-1, -1]].
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ int paley_sign(int kind, int q, const int8_t* chi2, int a, int a2) {
  if (kind == 1) {
    if (a == 0) return 1;
    if (a2 == 0) return -1;
    const int d = a - a2;
    return d == 0 ? 1 : chi2[d + q];
  }
  const int i = a >> 1, u = a & 1, j = a2 >> 1, v = a2 & 1;
  if (i == j) return (u | v) ? -1 : 1;
  int s = (i == 0 || j == 0) ? 1 : chi2[i - j + q];
  return (u & v) ? -s : s;
}

// Fill chi2 (2q + 1 entries) cooperatively; `sq` is q scratch bytes.
__device__ void build_chi(int q, int8_t* chi2, int8_t* sq) {
  for (int i = threadIdx.x; i < q; i += blockDim.x) sq[i] = 0;
  __syncthreads();
  for (int i = 1 + threadIdx.x; i <= (q - 1) / 2; i += blockDim.x) sq[(i * i) % q] = 1;
  __syncthreads();
  for (int d = threadIdx.x; d < 2 * q + 1; d += blockDim.x) {
    int r = (d - q) % q;
    if (r < 0) r += q;
    chi2[d] = r == 0 ? 0 : (sq[r] ? 1 : -1);
  }
  __syncthreads();
}

__device__ __forceinline__ float block_max(float v, float* red) {
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float r = lane < nw ? red[lane] : 0.f;
  for (int o = 16; o > 0; o >>= 1) r = fmaxf(r, __shfl_xor_sync(0xffffffffu, r, o));
  __syncthreads();
  return r;
}

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
                                                                   float* __restrict__ Yopt) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int K = pl.K, Kp = pl.Kp, p = pl.p, n = 1 << pl.log2n, q = pl.q;
  float* bufA = reinterpret_cast<float*>(smem_raw);
  float* bufB = bufA + Kp;
  float* red = bufB + Kp;
  int8_t* chi2 = reinterpret_cast<int8_t*>(red + 32);
  int8_t* sq = chi2 + 2 * q + 1;
  if (p > 1) build_chi(q, chi2, sq);
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
    float amax = 0.f;
    for (int c = threadIdx.x; c < Kp; c += blockDim.x) {
      const float v = y[c] * gamma;
      y[c] = v;
      amax = fmaxf(amax, fabsf(v));
    }
    amax = block_max(amax, red);
    float s = amax > 0.f ? __fdiv_rn(amax, 7.f) : 1.f;
    if (!(s > 0.f)) s = 1.f;
    if (threadIdx.x == 0) sx[row] = s;
    uint8_t* out = Xq + (long long)row * (Kp / 2);
    for (int j = threadIdx.x; j < Kp / 2; j += blockDim.x) {
      const int lo = quant_code(y[2 * j], s), hi = quant_code(y[2 * j + 1], s);
      out[j] = (uint8_t)((lo & 0xF) | ((hi & 0xF) << 4));
    }
    if (Yopt)
      for (int c = threadIdx.x; c < Kp; c += blockDim.x) Yopt[(long long)row * Kp + c] = y[c];
    __syncthreads();
  }
}

// ---------------------------------------------------------------------------------------------
// Layout helpers (offline paths).
// ---------------------------------------------------------------------------------------------
__global__ void relayout_to_blocks_kernel(const uint8_t* __restrict__ canon, int N, int Kp, uint32_t* __restrict__ blocks,
                                          int Np, int Kpp) {
  const int k_blocks = Kpp / XQ_K_BLOCK, words_per_row = Kpp / 8, row_bytes = Kp / 2;
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
    blocks[xq_weight_word_offset(n, kg, k_blocks) / 4] = w;
  }
}

__global__ void relayout_from_blocks_kernel(const uint32_t* __restrict__ blocks, int Np, int Kpp, uint8_t* __restrict__ canon,
                                            int N, int Kp) {
  const int k_blocks = Kpp / XQ_K_BLOCK, row_bytes = Kp / 2;
  const long long total = (long long)N * row_bytes;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int n = (int)(i / row_bytes), byte = (int)(i % row_bytes);
    const uint32_t w = blocks[xq_weight_word_offset(n, byte >> 2, k_blocks) / 4];
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

inline int grid_for(long long work, int threads) {
  long long g = (work + threads - 1) / threads;
  if (g < 1) g = 1;
  if (g > 148 * 32) g = 148 * 32;
  return (int)g;
}

}  // namespace

cudaError_t xq_launch_rotate_quant(const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t& pl, uint8_t* Xq,
                                   float* sx, float* Yopt, cudaStream_t st) {
  const float gamma = (float)(1.0 / sqrt((double)pl.Kp));
  const size_t smem = sizeof(float) * (2 * (size_t)pl.Kp + 32) + (size_t)(3 * pl.q + 1) + 16;
  cudaError_t e = cudaFuncSetAttribute(rotate_quant_general_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int grid = M < 148 * 8 ? M : 148 * 8;
  rotate_quant_general_kernel<<<grid, 256, smem, st>>>((const __nv_bfloat16*)X, M, (long long)ldx, pl, gamma, Xq, sx, Yopt);
  return cudaGetLastError();
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

cudaError_t xq_launch_pack_codes(const int8_t* codes, int64_t pairs, uint8_t* packed, cudaStream_t st) {
  pack_codes_kernel<<<grid_for(pairs, 256), 256, 0, st>>>(codes, pairs, packed);
  return cudaGetLastError();
}

cudaError_t xq_launch_unpack_codes(const uint8_t* packed, int64_t pairs, int8_t* codes, cudaStream_t st) {
  unpack_codes_kernel<<<grid_for(pairs, 256), 256, 0, st>>>(packed, pairs, codes);
  return cudaGetLastError();
}
