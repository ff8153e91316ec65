// Device helpers shared by the rotate + quantize kernels: the order-p Paley factor from the
// quadratic-character table of GF(q), block-wide maximum, transposing matrix loads.
#pragma once

#include <cuda_fp4.h>
#include <stdint.h>

namespace xqhad {

// ---------------------------------------------------------------------------------------------
// Sign of entry (a, a2) of the order-p Paley factor from the quadratic-character table of GF(q).
// chi2 is indexed by d + q for d in (-q, q): chi2[d + q] = chi(d mod q), chi(0) = 0.
// Paley-I:  first row +1, first column -1 below it, core chi(i - j) + identity.
// Paley-II: symmetric S of order q + 1 (zero diagonal, border +1, core chi(i - j)); each entry s
//           becomes s * [[1, 1], [1, -1]], each diagonal zero becomes [[1, -1], [-1, -1]].
// ---------------------------------------------------------------------------------------------
// kind 3: Paley-I over the field of 7^3 = 343 elements (order 344), elements numbered a0 + 7 a1 + 49 a2 for the
// polynomial a0 + a1 x + a2 x^2 over GF(7) modulo x^3 - 5; chi2 then holds chi(element d) at index d, d < 343.
__device__ __forceinline__ int gf343_sub(int a, int b) {
  int d0 = a % 7 - b % 7, d1 = (a / 7) % 7 - (b / 7) % 7, d2 = a / 49 - b / 49;
  d0 += d0 < 0 ? 7 : 0;
  d1 += d1 < 0 ? 7 : 0;
  d2 += d2 < 0 ? 7 : 0;
  return d0 + 7 * d1 + 49 * d2;
}
__device__ __forceinline__ int gf343_square(int a) {
  const int a0 = a % 7, a1 = (a / 7) % 7, a2 = a / 49;
  // (a0 + a1 x + a2 x^2)^2 with x^3 = 5, x^4 = 5 x
  const int c0 = a0 * a0 + 10 * a1 * a2, c1 = 2 * a0 * a1 + 5 * a2 * a2, c2 = 2 * a0 * a2 + a1 * a1;
  return c0 % 7 + 7 * (c1 % 7) + 49 * (c2 % 7);
}

__device__ __forceinline__ int paley_sign(int kind, int q, const int8_t* chi2, int a, int a2) {
  if (kind == 3) {
    if (a == 0) return 1;
    if (a2 == 0) return -1;
    return a == a2 ? 1 : chi2[gf343_sub(a - 1, a2 - 1)];
  }
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

// Fill chi2 (2q + 1 entries; kind 3: the first q) cooperatively; `sq` is q scratch bytes.
__device__ __forceinline__ void build_chi(int q, int8_t* chi2, int8_t* sq, int kind = 1) {
  for (int i = threadIdx.x; i < q; i += blockDim.x) sq[i] = 0;
  __syncthreads();
  if (kind == 3) {
    for (int i = 1 + threadIdx.x; i < q; i += blockDim.x) sq[gf343_square(i)] = 1;
    __syncthreads();
    for (int d = threadIdx.x; d < q; d += blockDim.x) chi2[d] = d == 0 ? 0 : (sq[d] ? 1 : -1);
    __syncthreads();
    return;
  }
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

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* smem_ptr) {
  const uint32_t addr = (uint32_t)__cvta_generic_to_shared(smem_ptr);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* smem_ptr) {
  const uint32_t addr = (uint32_t)__cvta_generic_to_shared(smem_ptr);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}

// Quantizer constants of one row (paper Sec. 4: per-token activations, per-channel weights).
// Either way a stored code is c = clamp(rne(y / s) + z, -8, 7) and stands for s * (c - z).
// Symmetric: s = absmax / 7 (1 for a zero row), z = 0.
// Asymmetric (the range is forced to contain zero): s = (hi - lo) / 15 and the unsigned zero point
// clamp(rne(-lo / s), 0, 15); codes and zero point are kept shifted by -8, so that they are the same
// signed nibbles the symmetric path stores and the signed integer product serves both.
struct RowQuant {
  float s, inv;
  int z;
};
__device__ __forceinline__ RowQuant row_quant_sym(float amax) {
  RowQuant r;
  r.s = amax > 0.f ? __fdiv_rn(amax, 7.f) : 1.f;
  if (!(r.s > 0.f)) r.s = 1.f;
  r.inv = __frcp_rn(r.s);
  r.z = 0;
  return r;
}
__device__ __forceinline__ RowQuant row_quant_asym(float lo, float hi) {  // lo <= 0 <= hi
  RowQuant r;
  r.s = hi > lo ? __fdiv_rn(hi - lo, 15.f) : 1.f;
  if (!(r.s > 0.f)) r.s = 1.f;
  r.inv = __frcp_rn(r.s);
  r.z = max(0, min(15, __float2int_rn(__fdiv_rn(-lo, r.s)))) - 8;
  return r;
}
__device__ __forceinline__ int row_code(const RowQuant& r, float y) {
  return max(-8, min(7, __float2int_rn(y * r.inv) + r.z));
}

// MXFP4 element (paper Sec. 4: OCP microscaling): the E2M1 code nearest to v, ties to the even mantissa
// bit, magnitudes above 6 saturate; code = sign << 3 | magnitude index of {0, .5, 1, 1.5, 2, 3, 4, 6}.
// Below 1 the grid is the subnormal one (step 0.5): index = rne(2 a).  From 1 on, a is rounded to one
// mantissa bit in its bit pattern (round to nearest even on bit 22, carrying into the exponent) and
// the index is 2 (exponent - 127) + mantissa bit + 2 = (bits >> 22) - 252.
__device__ __forceinline__ uint32_t mx_e2m1_code(float v) {
  const float a = fabsf(v);
  uint32_t u = __float_as_uint(a);
  u += 0x1FFFFFu + ((u >> 22) & 1u);
  const uint32_t hi = min((u >> 22) - 252u, 7u);
  const uint32_t c = a < 1.f ? (uint32_t)__float2int_rn(a + a) : hi;
  return c | (v < 0.f ? 8u : 0u);  // a negative zero keeps the code of zero
}
// Two elements at once through the hardware conversion (round to nearest even, saturating): the byte holds the
// code of lo in bits 0-3 and of hi in bits 4-7.
__device__ __forceinline__ uint32_t mx_e2m1_pair(float lo, float hi) {
  return (uint32_t)__nv_cvt_float2_to_fp4x2(make_float2(lo, hi), __NV_E2M1, cudaRoundNearest);
}
// 2^-e as a float, e in [-127, 127] (2^-127 is a subnormal: it has no exponent field of its own).
__device__ __forceinline__ float mx_inv_scale(int e) { return e < 127 ? __uint_as_float((uint32_t)(127 - e) << 23) : 5.877471754111438e-39f; }
// Shared exponent of a group whose largest magnitude is a: floor(log2 a) - 2 in [-127, 127]; 0 for a = 0.
__device__ __forceinline__ int mx_shared_exp(float a) {
  if (!(a > 0.f)) return 0;
  const int field = (int)((__float_as_uint(a) >> 23) & 0xFF);
  return max(-127, min(127, (field == 0 ? -127 : field - 127) - 2));  // fp32 subnormals lie below 2^-126
}

__device__ __forceinline__ uint32_t sign_bf16(int s) { return s > 0 ? 0x3F80u : (s < 0 ? 0xBF80u : 0u); }

}  // namespace xqhad
