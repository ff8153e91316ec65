// One activation row through pad + Kronecker Hadamard + per-row quantizer on the warp-level tensor cores (paper
// Sec. 3: X_hat = X H_hat; Sec. 4: per-token 4-bit), as a device routine that a group of warps runs together.
// Two kernels call it: the one-row-per-CTA rotate + quantize kernel, and the decode product kernel, whose first
// CTAs rotate the token rows inside the product's own launch.
//
// For p > 1, 32 <= n <= 256, ceil(K / n) <= 64.  With the row viewed as V[a][b] (a < p, b < n) the layer needs
// Y = H_p^T V S_n.  The outer factor goes first, on the raw bf16 inputs: +-1 times bf16 is exact and the sums
// accumulate in fp32, so H_p^T V runs as m16n8k16 bf16 MMAs (A = H_p^T, B = V read from shared memory with a
// transposing ldmatrix).  Warp (mt, bc) owns 16 rows a' and a chunk of NB = min(n, 64) columns b, so the
// Sylvester butterflies over the low bits of b stay inside the warp: bit 0 inside a thread, bits 1-2 across the four
// lanes of a quad, higher bits across accumulator registers.  For n = 128 and 256 the last one or two butterflies
// cross the two or four column chunks through shared memory (short chunks keep the accumulators at 32 registers
// and put up to 16 warps on one row: the row's latency is what counts here).  absmax, scale, rounding and nibble packing follow in registers; the packed row leaves
// through shared memory as 128-bit stores (and, on request, as the byte-per-code operand format of the tcgen05
// GEMM).
#pragma once

#include <cuda_bf16.h>

#include "xq_hadamard.cuh"
#include "xq_internal.h"
#include "xq_ptx.cuh"

namespace xqrot {

using namespace xqhad;

// Synchronisation of the warps that work on a row: the whole CTA, or a named barrier among its first warps.
struct CtaSync {
  __device__ __forceinline__ void operator()() const { __syncthreads(); }
};
struct NamedSync {
  int id, threads;
  __device__ __forceinline__ void operator()() const { xqptx::bar_sync(id, threads); }
};

// Maximum over the group's threads (values are >= 0); `red` holds one float per warp.
template <class Sync>
__device__ __forceinline__ float group_max(float v, float* red, int tid, int nthreads, const Sync& sync) {
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  const int warp = tid >> 5, lane = tid & 31, nw = (nthreads + 31) >> 5;
  if (lane == 0) red[warp] = v;
  sync();
  float r = lane < nw ? red[lane] : 0.f;
  for (int o = 16; o > 0; o >>= 1) r = fmaxf(r, __shfl_xor_sync(0xffffffffu, r, o));
  sync();
  return r;
}

// Shared-memory regions of one row group.
struct RowSmem {
  __nv_bfloat16* Xs;   // [KS * 16][n + 8]: the staged input row (zero outside the data)
  uint32_t* outp;      // Kp / 8 words: the packed row
  uint8_t* sfs;        // Kp / 32 scale bytes (MXFP4)
  float* red;          // 32 floats
  float* exch;         // n > 64 only: [MT * 8][n + 8] floats
};

// Where a row's results go.
struct RowOut {
  uint8_t* Xq;         // packed codes, row pitch (sfb ? Kq : Kp) / 2
  float* sx;
  float* Yopt;
  uint8_t* A8opt;
  int32_t* zp;         // non-null: asymmetric codes
  uint8_t* sfb;        // non-null: MXFP4 (group exponents) instead of per-row INT4
  int Kq;
};

// The A fragments of H_p^T for this warp's 16 output rows, from the bf16 image in shared memory.
template <int KS>
__device__ __forceinline__ void load_afrag(uint32_t (&afrag)[KS][4], const __nv_bfloat16* Hs, int P16, int hpitch, int mt, int lane) {
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) {
    if (16 * ks < P16) ldmatrix_x4(afrag[ks], Hs + (16 * mt + (lane & 15)) * hpitch + 16 * ks + (lane >> 4) * 8);
    else afrag[ks][0] = afrag[ks][1] = afrag[ks][2] = afrag[ks][3] = 0u;
  }
}

// One row, staged in sm.Xs, by the group's `nthreads` threads (thread `tid` of the group; warp = (mt, bc)).
template <int LOG2NB, int KS, class Sync>
__device__ __forceinline__ void rotate_row(const xq_hadamard_plan_t& pl, float gamma, const uint32_t (&afrag)[KS][4], const RowSmem& sm,
                                           const RowOut& o, long long row, int tid, int nthreads, const Sync& sync) {
  constexpr int NB = 1 << LOG2NB;  // columns per warp
  constexpr int NT8 = NB / 8;      // n-tiles per warp
  const int Kp = pl.Kp, p = pl.p, n = 1 << pl.log2n;
  const int NC = n / NB;            // column chunks (1, 2 or 4)
  const int pitch = n + 8;          // bf16 elements per staged row (conflict-free ldmatrix)
  const int warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int mt = warp / NC, bc = warp - mt * NC;
  const __nv_bfloat16* Xs = sm.Xs;
  uint32_t* outp = sm.outp;
  uint8_t* sfs = sm.sfs;
  float* exch = sm.exch;
  uint8_t* const sfb = o.sfb;
  int32_t* const zp = o.zp;
  const int Kq = o.Kq;

  float acc[NT8][4];
#pragma unroll
  for (int j = 0; j < NT8; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f;
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) {
    const __nv_bfloat16* base = Xs + (16 * ks + (lane & 7) + ((lane >> 3) & 1) * 8) * pitch + bc * NB + ((lane >> 4) & 1) * 8;
#pragma unroll
    for (int jp = 0; jp < NT8 / 2; ++jp) {
      uint32_t bfr[4];
      ldmatrix_x4_trans(bfr, base + 16 * jp);
      xqptx::mma_bf16_16x8x16(acc[2 * jp], afrag[ks], bfr[0], bfr[1]);
      xqptx::mma_bf16_16x8x16(acc[2 * jp + 1], afrag[ks], bfr[2], bfr[3]);
    }
  }
  // Sylvester butterflies along b = 8 j + 2 t + e
#pragma unroll
  for (int j = 0; j < NT8; ++j) {
    const float u0 = acc[j][0], u1 = acc[j][1], u2 = acc[j][2], u3 = acc[j][3];
    acc[j][0] = u0 + u1; acc[j][1] = u0 - u1; acc[j][2] = u2 + u3; acc[j][3] = u2 - u3;
  }
#pragma unroll
  for (int bit = 1; bit <= 2; ++bit) {
    const float sgn = (t & bit) ? -1.f : 1.f;
#pragma unroll
    for (int j = 0; j < NT8; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float ov = __shfl_xor_sync(0xffffffffu, acc[j][e], bit);
        acc[j][e] = fmaf(sgn, acc[j][e], ov);
      }
  }
#pragma unroll
  for (int s = 1; s < NT8; s <<= 1)
#pragma unroll
    for (int j = 0; j < NT8; ++j)
      if (!(j & s)) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float u = acc[j][e], w = acc[j | s][e];
          acc[j][e] = u + w;
          acc[j | s][e] = u - w;
        }
      }
  if (NC > 1) {
    // the butterflies over the top bits of b run between the column chunks (warps), through shared memory: every warp
    // writes its chunk, reads the others and combines them level by level, exactly as the register levels do.  First
    // the rows g of every tile, then the rows g + 8 (half the buffer of doing both at once).
    const float s0 = (bc & 1) ? -1.f : 1.f, s1 = (bc & 2) ? -1.f : 1.f;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      float* rowp = exch + (size_t)(8 * mt + g) * (n + 8) + 2 * t;  // pitch n + 8: the eight rows of a store fall into distinct banks
#pragma unroll
      for (int j = 0; j < NT8; ++j) *reinterpret_cast<float2*>(rowp + bc * NB + 8 * j) = make_float2(acc[j][2 * h], acc[j][2 * h + 1]);
      sync();
      if (NC == 2) {
        const float* other = rowp + (bc ^ 1) * NB;
#pragma unroll
        for (int j = 0; j < NT8; ++j) {
          const float2 ov = *reinterpret_cast<const float2*>(other + 8 * j);
          acc[j][2 * h] = fmaf(s0, acc[j][2 * h], ov.x);
          acc[j][2 * h + 1] = fmaf(s0, acc[j][2 * h + 1], ov.y);
        }
      } else {  // NC == 4: v[c] = x[c & ~1] + (-1)^(c & 1) x[c | 1], then y[c] = v[c & ~2] + (-1)^(c >> 1 & 1) v[c | 2]
        const float* p1 = rowp + (bc ^ 1) * NB;
        const float* p2 = rowp + (bc ^ 2) * NB;
        const float* p3 = rowp + (bc ^ 3) * NB;
#pragma unroll
        for (int j = 0; j < NT8; ++j) {
          const float2 o1 = *reinterpret_cast<const float2*>(p1 + 8 * j);
          const float2 o2 = *reinterpret_cast<const float2*>(p2 + 8 * j);
          const float2 o3 = *reinterpret_cast<const float2*>(p3 + 8 * j);
          const float vx = fmaf(s0, acc[j][2 * h], o1.x), vy = fmaf(s0, acc[j][2 * h + 1], o1.y);  // level 1 of this chunk
          const float wx = fmaf(s0, o2.x, o3.x), wy = fmaf(s0, o2.y, o3.y);                        // level 1 of chunk bc ^ 2
          acc[j][2 * h] = fmaf(s1, vx, wx);
          acc[j][2 * h + 1] = fmaf(s1, vy, wy);
        }
      }
      if (h == 0) sync();  // the second half overwrites what the first half's readers read
    }
  }
  // scale by 1/sqrt(K'), per-token absmax
  // (rows of the tile padding hold zeros: harmless, the asymmetric range contains zero anyway)
  float vmax = 0.f, vmin = 0.f;
#pragma unroll
  for (int j = 0; j < NT8; ++j)
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      acc[j][e] *= gamma;
      vmax = fmaxf(vmax, acc[j][e]);
      vmin = fminf(vmin, acc[j][e]);
    }
  RowQuant rq = row_quant_sym(0.f);
  if (sfb) {
    // MXFP4: the group of 32 channels is four neighbouring column tiles of one row, spread over the quad
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const int a2 = 16 * mt + g + 8 * r;
#pragma unroll
      for (int gq = 0; gq < NT8 / 4; ++gq) {
        float gm = 0.f;
#pragma unroll
        for (int j = 4 * gq; j < 4 * gq + 4; ++j) gm = fmaxf(gm, fmaxf(fabsf(acc[j][2 * r]), fabsf(acc[j][2 * r + 1])));
        gm = fmaxf(gm, __shfl_xor_sync(0xffffffffu, gm, 1));
        gm = fmaxf(gm, __shfl_xor_sync(0xffffffffu, gm, 2));
        const int e = mx_shared_exp(gm);
        const float inv = mx_inv_scale(e);
#pragma unroll
        for (int j = 4 * gq; j < 4 * gq + 4; ++j) {
          uint32_t w = mx_e2m1_pair(acc[j][2 * r] * inv, acc[j][2 * r + 1] * inv) << (8 * t);
          w |= __shfl_xor_sync(0xffffffffu, w, 1);
          w |= __shfl_xor_sync(0xffffffffu, w, 2);
          if (t == 0 && a2 < p) outp[(a2 * n + bc * NB) / 8 + j] = w;
        }
        if (t == 0 && a2 < p) sfs[(a2 * n + bc * NB) / 32 + gq] = (uint8_t)(e + 127);
      }
    }
  } else if (zp) {
    vmax = group_max(vmax, sm.red, tid, nthreads, sync);
    vmin = -group_max(-vmin, sm.red, tid, nthreads, sync);
    rq = row_quant_asym(vmin, vmax);
  } else {
    rq = row_quant_sym(group_max(fmaxf(vmax, -vmin), sm.red, tid, nthreads, sync));
  }
  const float s = rq.s;
  // quantize, pack: the quad's four bytes of one (row, j) form one word of 8 codes
#pragma unroll
  for (int r = 0; r < 2 && !sfb; ++r) {
    const int a2 = 16 * mt + g + 8 * r;
#pragma unroll
    for (int j = 0; j < NT8; ++j) {
      const int lo = row_code(rq, acc[j][2 * r]);
      const int hi = row_code(rq, acc[j][2 * r + 1]);
      uint32_t w = (uint32_t)((lo & 0xF) | ((hi & 0xF) << 4)) << (8 * t);
      w |= __shfl_xor_sync(0xffffffffu, w, 1);
      w |= __shfl_xor_sync(0xffffffffu, w, 2);
      if (t == 0 && a2 < p) outp[(a2 * n + bc * NB) / 8 + j] = w;
    }
  }
  if (o.Yopt) {
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const int a2 = 16 * mt + g + 8 * r;
      if (a2 < p) {
        float* yrow = o.Yopt + row * Kp + a2 * n + bc * NB + 2 * t;
#pragma unroll
        for (int j = 0; j < NT8; ++j) *reinterpret_cast<float2*>(yrow + 8 * j) = make_float2(acc[j][2 * r], acc[j][2 * r + 1]);
      }
    }
  }
  sync();
  if (tid == 0 && !sfb) {
    o.sx[row] = s;
    if (zp) zp[row] = rq.z;
  }
  if (sfb) {
    // scale bytes into their blocks; padding up to Kq: unit scales and zero codes (never a NaN scale byte)
    for (int i = tid; i < Kq / 32; i += nthreads) sfb[xq_mx_sf_offset((int)row, i, Kq)] = i < Kp / 32 ? sfs[i] : (uint8_t)127;
    for (int i = tid; i < (Kq - Kp) / 8; i += nthreads) *reinterpret_cast<uint32_t*>(o.Xq + row * (Kq / 2) + Kp / 2 + 4 * i) = 0u;
  }
  uint4* dst = reinterpret_cast<uint4*>(o.Xq + row * ((sfb ? Kq : Kp) / 2));
  for (int i = tid; i < Kp / 32; i += nthreads) {
    const uint4 v = reinterpret_cast<const uint4*>(outp)[i];
    dst[i] = v;
    if (o.A8opt) {
      uint4 e0, e1;
      xqptx::split16(v.x, e0.x, e0.y);
      xqptx::split16(v.y, e0.z, e0.w);
      xqptx::split16(v.z, e1.x, e1.y);
      xqptx::split16(v.w, e1.z, e1.w);
      uint4* d8 = reinterpret_cast<uint4*>(o.A8opt + row * Kp);
      d8[2 * i] = e0;
      d8[2 * i + 1] = e1;
    }
  }
  sync();
}

// Column chunks (warps per tile of 16 output rows) of a row group: chunks of min(n, 64) columns.
__host__ __device__ inline int row_chunks(const xq_hadamard_plan_t& pl) { return pl.log2n > 6 ? 1 << (pl.log2n - 6) : 1; }
// log2 of the chunk length: the LOG2NB template argument of rotate_row for this plan.
__host__ __device__ inline int row_log2nb(const xq_hadamard_plan_t& pl) { return pl.log2n > 6 ? 6 : pl.log2n; }

// Shared memory of one row group in the order Xs | outp | red | Hs (image of H_p^T, [P16][P16 + 8] bf16) | exch.
struct RowLayout {
  size_t xs, outp, red, hs, exch, total;
};
__host__ __device__ inline RowLayout row_layout(const xq_hadamard_plan_t& pl) {
  const int n = 1 << pl.log2n, rows_a = (pl.K + n - 1) / n, ks = (rows_a + 15) / 16, P16 = (pl.p + 15) / 16 * 16;
  RowLayout L;
  size_t off = 0;
  L.xs = off;
  off += ((size_t)ks * 16 * (n + 8) * 2 + 15) / 16 * 16;
  L.outp = off;
  off += ((size_t)pl.Kp / 2 + 15) / 16 * 16;
  L.red = off;
  off += 128;
  L.hs = off;
  off += ((size_t)P16 * (P16 + 8) * 2 + 15) / 16 * 16;
  L.exch = off;
  if (n > 64) off += (size_t)(P16 / 2) * (n + 8) * 4;
  L.total = off;
  return L;
}

// True when the plan is one rotate_row takes (and the warp count of a row group fits 16 warps).
__host__ __device__ inline bool plan_supported(const xq_hadamard_plan_t& pl) {
  const int n = 1 << pl.log2n, rows_a = (pl.K + n - 1) / n, MT = (pl.p + 15) / 16;
  return pl.p > 1 && pl.log2n >= 5 && pl.log2n <= 8 && pl.K % 8 == 0 && rows_a <= 64 && MT * row_chunks(pl) <= 16;
}

}  // namespace xqrot
