// Online step of the expanded layer for many rows (paper Sec. 3: X_hat = X H_hat; Sec. 4:
// per-token 4-bit): the throughput form of the fused pad + Kronecker Hadamard + quantize kernel.
//
// One persistent CTA per SM holds H_p^T as a bf16 matrix in shared memory and runs G independent
// row groups of Wr warps each; a group streams its rows through a double-buffered cp.async stage
// (the next row lands while the current one is computed) and never meets the other groups: the
// only synchronisation is a named barrier inside the group (a warp-level one when Wr == 1).
// With the row viewed as V[a][b] (a < p, b < n = 2^k) the layer needs Y = H_p^T V S_n.  The outer
// factor goes first, on the raw bf16 inputs -- +-1 times bf16 is exact and the sums accumulate
// in fp32 -- as m16n8k16 MMAs: A fragments with ldmatrix from the shared H_p^T, B fragments with
// a transposing ldmatrix from the staged row.  A warp owns MTW tiles of 16 rows a' and all n
// columns, so the Sylvester butterflies along b stay inside the warp.  In the accumulator layout
// a thread holds columns b = 8j + 2t + e of its rows: bits 0 and 3.. of b are butterflied in
// registers; for bits 1-2 (the lane bits t) eight rows at a time pass through a small per-warp
// shared-memory tile and come back with all eight columns 8j..8j+7 of one row in one thread --
// the warp shuffle unit would otherwise be the bottleneck -- which is also exactly one packed
// word of eight codes.  Per-row absmax (five shuffles, then Wr values through shared memory),
// scale 1/sqrt(K') folded into the quantizer's multiplier, round-to-nearest-even by the
// magic-number add, nibble packing and coalesced 32-bit stores follow.
// Orders with n = 2^k > 128 run as n = 128 with the top f = k - 7 Sylvester bits folded into the
// outer factor: H_p (x) S_{2^k} = (H_p (x) S_{2^f}) (x) S_128, and channel a 2^k + b =
// (a 2^f + b_hi) 128 + b_lo, so the same code applies with a factor of order p 2^f whose signs
// carry one extra (-1)^popcount(b_hi & b_hi').  A pure Sylvester order (p = 1) is the case H_1 = [1].
#include <cuda_bf16.h>

#include "xq_internal.h"
#include "xq_hadamard.cuh"
#include "xq_ptx.cuh"

using namespace xqhad;

namespace {

constexpr int kMaxWarps = 16;

__device__ __forceinline__ void group_sync(int group, int Wr) {
  if (Wr == 1) __syncwarp();
  else xqptx::bar_sync(1 + group, 32 * Wr);
}

// QM: 0 symmetric per-row INT4, 1 asymmetric per-row INT4, 2 MXFP4 (a shared exponent per 32 channels; Xq then has
// the row pitch Kq / 2 and the scale bytes go to sfb in the block layout of the block-scaled GEMM).
template <int LOG2N, int KS, int MTW, int QM>
__global__ void __launch_bounds__(kMaxWarps * 32, 1)
    rotate_quant_rows_kernel(const __nv_bfloat16* __restrict__ X, int M, long long ldx, xq_hadamard_plan_t pl, float gamma,
                             uint8_t* __restrict__ Xq, float* __restrict__ sx, float* __restrict__ Yopt, uint8_t* __restrict__ A8opt,
                             int32_t* __restrict__ zp, uint8_t* __restrict__ sfb, int Kq, int Wr, int G, int fold, int nbuf) {
  constexpr bool ASYM = QM == 1;
  constexpr int n = 1 << LOG2N, NT8 = n / 8;
  constexpr int xpitch = n + 8;        // bf16 elements per staged row (conflict-free ldmatrix)
  constexpr int hpitch = KS * 16 + 8;  // bf16 elements per row of H_p^T
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int K = pl.K, Kp = pl.Kp, p = pl.p << fold, q = pl.q;  // p: order of the (folded) outer factor
  const int MT = (p + 15) / 16;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int group = warp / Wr, wg = warp - group * Wr, tg = tid - group * Wr * 32, gthreads = Wr * 32;

  __nv_bfloat16* Hs = reinterpret_cast<__nv_bfloat16*>(smem_raw);                       // [MT * 16][hpitch]
  __nv_bfloat16* Xs_all = Hs + MT * 16 * hpitch;                                        // [G][nbuf][KS * 16][xpitch]
  constexpr int tpitch = n + 8;        // floats per row of the transpose tile
  float* tr_all = reinterpret_cast<float*>(Xs_all + (size_t)G * nbuf * KS * 16 * xpitch);  // [warps][8][tpitch]
  float* red_all = tr_all + (size_t)G * Wr * 8 * tpitch;                                // [G][2 Wr] + 32 spare
  int8_t* chi2 = reinterpret_cast<int8_t*>(red_all + 2 * G * Wr + 32);
  int8_t* sq = chi2 + 2 * q + 1;

  if (pl.p > 1) build_chi(q, chi2, sq, pl.paley_kind);
  // H_p^T: row a' (output index), column a (input index); zero outside p x p
  for (int i = tid; i < MT * 16 * KS * 16; i += blockDim.x) {
    const int a2 = i / (KS * 16), a = i - a2 * (KS * 16);
    int s = 0;
    if (a2 < p && a < p) {
      s = pl.p > 1 ? paley_sign(pl.paley_kind, q, chi2, a >> fold, a2 >> fold) : 1;
      if (__popc(a & a2 & ((1 << fold) - 1)) & 1) s = -s;
    }
    Hs[a2 * hpitch + a] = __ushort_as_bfloat16((unsigned short)sign_bf16(s));
  }
  // zero the staged rows once: rows past the data and the tail of a partial last row stay zero
  for (int i = tid; i < G * nbuf * KS * 16 * xpitch / 8; i += blockDim.x) reinterpret_cast<uint4*>(Xs_all)[i] = make_uint4(0, 0, 0, 0);
  xqptx::pdl_wait();
  __syncthreads();
  // only now may the kernel after this one be scheduled (not before the wait: a chain in which every kernel releases its
  // successor before its own wait measured 2-5 % slower per layer)
  xqptx::pdl_launch_dependents();
  if (group >= G) return;

  __nv_bfloat16* Xs = Xs_all + (size_t)group * nbuf * KS * 16 * xpitch;
  float* tr = tr_all + (size_t)warp * 8 * tpitch;
  float* red = red_all + group * 2 * Wr;
  constexpr int TPL = NT8 / 4;  // (row, j) tuples of eight columns per lane and pass of eight rows
  const int chunks = K / 8;  // 16-byte pieces of a row
  const int stride = gridDim.x * G;
  auto issue_load = [&](int row, int buf) {
    const __nv_bfloat16* x = X + (long long)row * ldx;
    __nv_bfloat16* dst = Xs + (size_t)buf * KS * 16 * xpitch;
    for (int i = tg; i < chunks; i += gthreads) {
      const int c = 8 * i, a = c >> LOG2N, b = c & (n - 1);
      xqptx::cp_async16(dst + a * xpitch + b, x + c);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };

  // nbuf == 2: the next row lands while this one is computed; nbuf == 1 (long rows on a large order-p factor, whose
  // image leaves room for one stage only): the load of a row follows the last use of the stage by the row before
  int row = blockIdx.x * G + group, buf = 0;
  if (row < M && nbuf == 2) issue_load(row, 0);
  for (; row < M; row += stride, buf = nbuf == 2 ? buf ^ 1 : 0) {
    if (nbuf == 1) {
      issue_load(row, 0);
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    } else if (row + stride < M) {
      issue_load(row + stride, buf ^ 1);
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    group_sync(group, Wr);
    const __nv_bfloat16* xb = Xs + (size_t)buf * KS * 16 * xpitch;

    float acc[MTW][NT8][4];
#pragma unroll
    for (int m = 0; m < MTW; ++m)
#pragma unroll
      for (int j = 0; j < NT8; ++j) acc[m][j][0] = acc[m][j][1] = acc[m][j][2] = acc[m][j][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      uint32_t bfr[NT8][2];
      const __nv_bfloat16* base = xb + (16 * ks + (lane & 7) + ((lane >> 3) & 1) * 8) * xpitch + ((lane >> 4) & 1) * 8;
#pragma unroll
      for (int jp = 0; jp < NT8 / 2; ++jp) {
        uint32_t r4[4];
        ldmatrix_x4_trans(r4, base + 16 * jp);
        bfr[2 * jp][0] = r4[0];
        bfr[2 * jp][1] = r4[1];
        bfr[2 * jp + 1][0] = r4[2];
        bfr[2 * jp + 1][1] = r4[3];
      }
#pragma unroll
      for (int m = 0; m < MTW; ++m) {
        const int mt = wg * MTW + m;
        if (mt < MT) {
          uint32_t afr[4];
          ldmatrix_x4(afr, Hs + (16 * mt + (lane & 15)) * hpitch + 16 * ks + (lane >> 4) * 8);
#pragma unroll
          for (int j = 0; j < NT8; ++j) xqptx::mma_bf16_16x8x16(acc[m][j], afr, bfr[j][0], bfr[j][1]);
        }
      }
    }
    // Sylvester butterflies along b = 8 j + 2 t + e: bit 0 (e) and bits 3.. (j) in registers
#pragma unroll
    for (int m = 0; m < MTW; ++m) {
#pragma unroll
      for (int j = 0; j < NT8; ++j) {
        const float u0 = acc[m][j][0], u1 = acc[m][j][1], u2 = acc[m][j][2], u3 = acc[m][j][3];
        acc[m][j][0] = u0 + u1; acc[m][j][1] = u0 - u1; acc[m][j][2] = u2 + u3; acc[m][j][3] = u2 - u3;
      }
#pragma unroll
      for (int s = 1; s < NT8; s <<= 1)
#pragma unroll
        for (int j = 0; j < NT8; ++j)
          if (!(j & s)) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float u = acc[m][j][e], w = acc[m][j | s][e];
              acc[m][j][e] = u + w;
              acc[m][j | s][e] = u - w;
            }
          }
    }
    // bits 1-2 (t): eight rows at a time through the warp's tile; afterwards fin[m][h][k][0..7] are
    // the columns 8 jj .. 8 jj + 7 of row a' = 16 (wg MTW + m) + 8 h + r, (r, jj) = tuple lane + 32 k
    float fin[MTW][2][TPL][8];
    float amax = 0.f, amin = 0.f;  // symmetric: amax = max |y|; asymmetric: the row's extremes (both include 0)
#pragma unroll
    for (int m = 0; m < MTW; ++m)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
#pragma unroll
        for (int j = 0; j < NT8; ++j) *reinterpret_cast<float2*>(tr + g * tpitch + 8 * j + 2 * t) = make_float2(acc[m][j][2 * h], acc[m][j][2 * h + 1]);
        __syncwarp();
#pragma unroll
        for (int k = 0; k < TPL; ++k) {
          const int id = lane + 32 * k, r = id / NT8, jj = id % NT8;
          const float4 v0 = *reinterpret_cast<const float4*>(tr + r * tpitch + 8 * jj);
          const float4 v1 = *reinterpret_cast<const float4*>(tr + r * tpitch + 8 * jj + 4);
          // index i = 2 t + e inside the eight: bit 1 pairs (i, i ^ 2), bit 2 pairs (i, i ^ 4)
          const float a0 = v0.x + v0.z, a1 = v0.y + v0.w, a2 = v0.x - v0.z, a3 = v0.y - v0.w;
          const float a4 = v1.x + v1.z, a5 = v1.y + v1.w, a6 = v1.x - v1.z, a7 = v1.y - v1.w;
          float* f = fin[m][h][k];
          f[0] = a0 + a4; f[1] = a1 + a5; f[2] = a2 + a6; f[3] = a3 + a7;
          f[4] = a0 - a4; f[5] = a1 - a5; f[6] = a2 - a6; f[7] = a3 - a7;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            if (QM == 2) {
              // the groups of 32 are reduced where they are quantized
            } else if (ASYM) {
              amax = fmaxf(amax, f[i]);
              amin = fminf(amin, f[i]);
            } else {
              amax = fmaxf(amax, fabsf(f[i]));
            }
          }
        }
        __syncwarp();
      }
    if constexpr (QM == 2) {
      // MXFP4: a thread holds 8 consecutive channels, four neighbouring lanes one group of 32
      const long long cpitch = Kq / 2;
#pragma unroll
      for (int m = 0; m < MTW; ++m)
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int k = 0; k < TPL; ++k) {
            const int id = lane + 32 * k, r = id / NT8, jj = id % NT8;
            const int a2 = 16 * (wg * MTW + m) + 8 * h + r;
            float* f = fin[m][h][k];
            float gmax = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              f[i] *= gamma;
              gmax = fmaxf(gmax, fabsf(f[i]));
            }
            gmax = fmaxf(gmax, __shfl_xor_sync(0xffffffffu, gmax, 1));
            gmax = fmaxf(gmax, __shfl_xor_sync(0xffffffffu, gmax, 2));
            const int e = xqhad::mx_shared_exp(gmax);
            const float inv = xqhad::mx_inv_scale(e);  // a power of two: the products are exact
            uint32_t w = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) w |= xqhad::mx_e2m1_pair(f[2 * i] * inv, f[2 * i + 1] * inv) << (8 * i);
            if (a2 < p) {
              *reinterpret_cast<uint32_t*>(Xq + (long long)row * cpitch + 4ll * (a2 * NT8 + jj)) = w;
              if ((jj & 3) == 0) sfb[xq_mx_sf_offset(row, (a2 * n + 8 * jj) >> 5, Kq)] = (uint8_t)(e + 127);
            }
          }
      // padding up to Kq: zero codes, unit scales (never a NaN scale byte under the tensor core)
      for (int i = tg; i < (Kq - Kp) / 8; i += gthreads) *reinterpret_cast<uint32_t*>(Xq + (long long)row * cpitch + Kp / 2 + 4 * i) = 0u;
      for (int i = tg; i < (Kq - Kp) / 32; i += gthreads) sfb[xq_mx_sf_offset(row, Kp / 32 + i, Kq)] = (uint8_t)127;
    } else {
    for (int o = 16; o > 0; o >>= 1) {
      amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
      if (ASYM) amin = fminf(amin, __shfl_xor_sync(0xffffffffu, amin, o));
    }
    if (Wr > 1) {
      if (lane == 0) {
        red[wg] = amax;
        if (ASYM) red[Wr + wg] = amin;
      }
      group_sync(group, Wr);
      for (int i = 0; i < Wr; ++i) {
        amax = fmaxf(amax, red[i]);
        if (ASYM) amin = fminf(amin, red[Wr + i]);
      }
    }
    // the extremes of the scaled values: scaling is monotone
    const xqhad::RowQuant rq = ASYM ? xqhad::row_quant_asym(amin * gamma, amax * gamma) : xqhad::row_quant_sym(amax * gamma);
    const float mult = gamma * rq.inv;
    if (tg == 0) {
      sx[row] = rq.s;
      if (ASYM) zp[row] = rq.z;
    }
    // the rounding constant 1.5 * 2^23 also carries the zero point and an offset of 8 (offset
    // binary, undone below)
    const float magic = 12582920.f + (float)rq.z;
    // quantize (round to nearest even through the 1.5 * 2^23 add: the low mantissa bits are the
    // integer; symmetric |y / s| <= 7 needs no clamp), pack eight codes per word
    uint32_t* xq_row = reinterpret_cast<uint32_t*>(Xq + (long long)row * (Kp / 2));
#pragma unroll
    for (int m = 0; m < MTW; ++m)
#pragma unroll
      for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int k = 0; k < TPL; ++k) {
          const int id = lane + 32 * k, r = id / NT8, jj = id % NT8;
          const int a2 = 16 * (wg * MTW + m) + 8 * h + r;
          const float* f = fin[m][h][k];
          // Horner over the raw bit patterns 0x4B400008 + code (the add also biases the code by 8):
          // the constant parts sum to a fixed word that is removed once, and offset-binary
          // nibbles become two's complement by flipping their top bits.
          uint32_t w = 0;
#pragma unroll
          for (int i = 7; i >= 0; --i) {
            float v = fmaf(f[i], mult, magic);
            if (ASYM) v = fminf(fmaxf(v, 12582912.f), 12582927.f);  // rne(y / s) + z can leave the code range by one
            w = w * 16u + (uint32_t)__float_as_int(v);
          }
          w = (w - 0x4B400000u * 0x11111111u) ^ 0x88888888u;
          if (a2 < p) {
            xq_row[a2 * NT8 + jj] = w;
            if (A8opt) {
              uint2 e8;
              xqptx::split16(w, e8.x, e8.y);
              *reinterpret_cast<uint2*>(A8opt + (long long)row * Kp + (long long)a2 * n + 8 * jj) = e8;
            }
            if (Yopt) {
              float4* y = reinterpret_cast<float4*>(Yopt + (long long)row * Kp + (long long)a2 * n + 8 * jj);
              y[0] = make_float4(f[0] * gamma, f[1] * gamma, f[2] * gamma, f[3] * gamma);
              y[1] = make_float4(f[4] * gamma, f[5] * gamma, f[6] * gamma, f[7] * gamma);
            }
          }
        }
    }
    // every warp of the group is done with the stage before its reuse two loads from now
    group_sync(group, Wr);
  }
}

template <int LOG2N, int KS, int MTW>
cudaError_t launch_rows(const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t& pl, float gamma, uint8_t* Xq, float* sx,
                        float* Yopt, uint8_t* A8opt, int32_t* zp, int sms, cudaStream_t st, const xq_mx_out* mx = nullptr) {
  constexpr int n = 1 << LOG2N;
  const int fold = pl.log2n - LOG2N;  // Sylvester bits folded into the outer factor
  const int MT = ((pl.p << fold) + 15) / 16, Wr = (MT + MTW - 1) / MTW;
  int G = kMaxWarps / Wr, nbuf = 2;
  const size_t fixed = (size_t)MT * 16 * (KS * 16 + 8) * 2 + 32 * 4 + (size_t)(3 * pl.q + 1) + 64;
  size_t per_group = (size_t)2 * KS * 16 * (n + 8) * 2 + (size_t)Wr * 8 * (n + 8) * 4 + (size_t)Wr * 8;
  while (G > 1 && fixed + G * per_group > 224 * 1024) --G;
  // fewer row groups than multiprocessors: spread the rows over all of them instead (2048 rows in groups of 16 are 128
  // CTAs on 148 SMs; in groups of 14 they are 147)
  if (G > 1 && (M + G - 1) / G < sms) {
    const int g2 = (M + sms - 1) / sms;
    if (g2 >= 1 && g2 < G) G = g2;
  }
  if (fixed + G * per_group > 224 * 1024) {  // one row group and still too much: a single stage
    nbuf = 1;
    per_group -= (size_t)KS * 16 * (n + 8) * 2;
  }
  if (fixed + G * per_group > 224 * 1024 || Wr > kMaxWarps) return cudaErrorNotSupported;
  const size_t smem = fixed + G * per_group;
  auto kern = mx ? rotate_quant_rows_kernel<LOG2N, KS, MTW, 2>
                 : (zp ? rotate_quant_rows_kernel<LOG2N, KS, MTW, 1> : rotate_quant_rows_kernel<LOG2N, KS, MTW, 0>);
  uint8_t* sfb = mx ? mx->sf_blocks : nullptr;
  const int Kq = mx ? mx->Kq : 0;
  if (mx) Xq = mx->codes;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int want = (M + G - 1) / G;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(want < sms ? want : sms);
  cfg.blockDim = dim3(32 * Wr * G);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, (const __nv_bfloat16*)X, (int)M, (long long)ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sfb, Kq, Wr, G, fold, nbuf);
}

template <int LOG2N, int MTW>
cudaError_t launch_rows_ks(int ks, const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t& pl, float gamma, uint8_t* Xq,
                           float* sx, float* Yopt, uint8_t* A8opt, int32_t* zp, int sms, cudaStream_t st, const xq_mx_out* mx = nullptr) {
  switch (ks) {
    case 1: return launch_rows<LOG2N, 1, MTW>(X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
    case 2: return launch_rows<LOG2N, 2, MTW>(X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
    case 3: return launch_rows<LOG2N, 3, MTW>(X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
    default: return launch_rows<LOG2N, 4, MTW>(X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
  }
}

// n > 128 folded to 128: up to 128 staged rows
cudaError_t launch_rows_folded(int ks, const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t& pl, float gamma, uint8_t* Xq,
                               float* sx, float* Yopt, uint8_t* A8opt, int32_t* zp, int sms, cudaStream_t st, const xq_mx_out* mx = nullptr) {
  switch (ks) {
    case 5: return launch_rows<7, 5, 1>(X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
    case 6: return launch_rows<7, 6, 1>(X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
    case 7: return launch_rows<7, 7, 1>(X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
    case 8: return launch_rows<7, 8, 1>(X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
    default: return launch_rows_ks<7, 1>(ks, X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
  }
}

// n = 64 with 65..128 staged rows (long inputs on a short Sylvester factor, e.g. 8192 -> 8960 = 140 x 64)
cudaError_t launch_rows_64_long(int ks, const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t& pl, float gamma, uint8_t* Xq,
                                float* sx, float* Yopt, uint8_t* A8opt, int32_t* zp, int sms, cudaStream_t st, const xq_mx_out* mx = nullptr) {
  switch (ks) {
    case 5: return launch_rows<6, 5, 2>(X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
    case 6: return launch_rows<6, 6, 2>(X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
    case 7: return launch_rows<6, 7, 2>(X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
    case 8: return launch_rows<6, 8, 2>(X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
    case 9: case 10: return launch_rows<6, 10, 2>(X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
    case 11: case 12: return launch_rows<6, 12, 2>(X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
    case 13: case 14: return launch_rows<6, 14, 2>(X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
    default: return launch_rows_ks<6, 2>(ks, X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
  }
}

}  // namespace

bool xq_rotate_rows_supported(const xq_hadamard_plan_t& pl) {
  if (pl.log2n < 5 || pl.K % 8 != 0 || pl.Kp % 32 != 0) return false;
  if (pl.p == 1 && pl.log2n < 9) return false;  // small pure Sylvester orders: the general kernel
  const int log2n = pl.log2n > 7 ? 7 : pl.log2n, fold = pl.log2n - log2n;
  const int n = 1 << log2n, rows_a = (pl.K + n - 1) / n, MT = ((pl.p << fold) + 15) / 16;
  // n = 64 also takes long rows on a large order-p factor (the paper's 14336 -> 19968 = 312 x 64: 224 staged input rows,
  // 20 tiles of 16 output rows on 10 warps, a single load stage)
  const int max_rows = log2n == 6 && !fold ? 224 : (fold ? 128 : 64), max_mt = log2n == 6 && !fold ? 32 : 15;
  if (rows_a > max_rows || MT > max_mt) return false;
  if (rows_a > 64 || MT > 15) {  // the CTA must hold at least one row group, with one load stage if need be
    const int ks = (rows_a + 15) / 16 + ((rows_a > 128) ? ((rows_a + 15) / 16) % 2 : 0);  // long rows: KS comes in steps of 2
    const int wr = log2n == 6 ? (MT + 1) / 2 : MT;
    const size_t need = (size_t)MT * 16 * (ks * 16 + 8) * 2 + (size_t)ks * 16 * (n + 8) * 2 + (size_t)wr * 8 * (n + 8) * 4 + 4096;
    if (need > 224 * 1024 || wr > kMaxWarps) return false;
  }
  return true;
}

namespace {
cudaError_t rotate_rows_dispatch(const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t& pl, uint8_t* Xq, float* sx,
                                 float* Yopt, uint8_t* A8opt, int32_t* zp, int sms, cudaStream_t st, const xq_mx_out* mx) {
  const float gamma = (float)(1.0 / sqrt((double)pl.Kp));
  const int log2n = pl.log2n > 7 ? 7 : pl.log2n;
  const int n = 1 << log2n, rows_a = (pl.K + n - 1) / n, ks = (rows_a + 15) / 16;
  // tiles of 16 output rows per warp: 80 accumulator registers at n = 32, 64 at n = 64 and 128
  switch (pl.log2n) {
    case 5: return launch_rows_ks<5, 5>(ks, X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
    case 6: return launch_rows_64_long(ks, X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
    case 7: return launch_rows_ks<7, 1>(ks, X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
    default: return launch_rows_folded(ks, X, M, ldx, pl, gamma, Xq, sx, Yopt, A8opt, zp, sms, st, mx);
  }
}
}  // namespace

cudaError_t xq_launch_rotate_rows(const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t& pl, uint8_t* Xq, float* sx,
                                  float* Yopt, uint8_t* A8opt, int32_t* zp, int sms, cudaStream_t st) {
  return rotate_rows_dispatch(X, M, ldx, pl, Xq, sx, Yopt, A8opt, zp, sms, st, nullptr);
}

bool xq_rotate_mx_supported(const xq_hadamard_plan_t& pl) { return pl.Kp % 32 == 0 && xq_rotate_rows_supported(pl); }

cudaError_t xq_launch_rotate_mx(const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t& pl, const xq_mx_out& mx, int sms,
                                cudaStream_t st) {
  if (!xq_rotate_mx_supported(pl)) return cudaErrorNotSupported;
  return rotate_rows_dispatch(X, M, ldx, pl, mx.codes, nullptr, nullptr, nullptr, nullptr, sms, st, &mx);
}
