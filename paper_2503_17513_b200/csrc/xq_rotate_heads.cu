// Head-wise pad + rotate + quantize (paper Sec. 4 "Compute Graph Details", Sec. 5 "Expanding R2 and
// R4": the rotation in front of the attention output projection acts on every head separately, so
// its expansion grows each head from d to d' channels).
//
// A token row is `heads` blocks of d channels.  Every block is zero-padded to d' and multiplied
// by the same Hadamard matrix of order d' = p 2^k (scaled 1 / sqrt(d')); the quantizer then sees
// the whole row of heads * d' values, as after one long rotation.  With d' <= 160 the truncated
// matrix is small enough to keep whole in shared memory, so the step is the dense product
//     Y[heads, d'] = X[heads, d] . Hhat[d, d']
// per token: bf16 m16n8k16 MMAs (+-1 times bf16 is exact, fp32 accumulate) with the heads as the
// 16-row operand.  A CTA runs G independent token groups of HT = ceil(heads / 16) warps; a group
// streams its tokens through a double-buffered cp.async stage, warp ht owns heads 16 ht .. 16 ht + 15
// and all d' / 8 column tiles of them (its A fragments are read once per 16 input channels), so the
// accumulators of a token stay in registers through the per-token reduction (shuffles, then HT
// values through shared memory), the rounding and the nibble packing; the packed row leaves
// through the group's shared-memory row as 128-bit stores (and, on request, in the byte-per-code
// operand format of the tcgen05 GEMM).
#include <cuda_bf16.h>
#include <math.h>

#include "xq_hadamard.cuh"
#include "xq_internal.h"
#include "xq_ptx.cuh"

using namespace xqhad;

namespace {

constexpr int kWarps = 8;
constexpr int kMaxNT = 20;  // column tiles of 8 per warp (d' <= 160)

__device__ __forceinline__ void group_sync(int group, int HT) {
  if (HT == 1) __syncwarp();
  else xqptx::bar_sync(1 + group, 32 * HT);
}

template <bool MX>
__global__ void __launch_bounds__(kWarps * 32, MX ? 1 : 2) rotate_quant_heads_kernel(const __nv_bfloat16* __restrict__ X, int M, long long ldx,
                                                                         xq_hadamard_plan_t pl, int heads, float gamma,
                                                                         uint8_t* __restrict__ Xq, float* __restrict__ sx,
                                                                         float* __restrict__ Yopt, uint8_t* __restrict__ A8opt,
                                                                         const __nv_bfloat16* __restrict__ Bimage,
                                                                         int32_t* __restrict__ zp, uint8_t* __restrict__ sfb, int Kq,
                                                                         int G) {
  // MX: MXFP4 instead of per-row INT4 -- a shared exponent for every 32 consecutive channels of the whole row
  // (groups may cross head boundaries), E2M1 codes; Xq then has the row pitch Kq / 2 and the scale bytes go to sfb in
  // the block layout of the block-scaled GEMM (sx, zp, A8opt unused).
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int d = pl.K, dp = pl.Kp, q = pl.q, n = 1 << pl.log2n;
  const int d16 = (d + 15) / 16 * 16, pitch = d16 + 8;  // bf16 elements per row of both operands (conflict-free 32-bit reads)
  const int H16 = (heads + 15) / 16 * 16, HT = H16 / 16, NT = dp / 8;
  const int Kp = heads * dp;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int group = warp / HT, ht = warp - group * HT, gtid = tid - group * HT * 32, gthreads = HT * 32;

  __nv_bfloat16* Bs = reinterpret_cast<__nv_bfloat16*>(smem_raw);           // [dp][pitch]: row c' holds column c' of Hhat (k = c contiguous)
  __nv_bfloat16* Xs_all = Bs + (size_t)dp * pitch;                           // [G][2][H16][pitch]
  uint32_t* outp_all = reinterpret_cast<uint32_t*>(Xs_all + (size_t)G * 2 * H16 * pitch);  // [G][Kp / 8] words
  float* red_all = reinterpret_cast<float*>(outp_all + (size_t)G * (Kp / 8));              // [G][2 HT] + 32 spare
  float* tmax_all = red_all + 2 * kWarps + 32;                                             // [G][Kp / 8]: largest magnitude per 8-column tile
  uint8_t* sfs_all = reinterpret_cast<uint8_t*>(tmax_all + (size_t)G * (Kp / 8));            // [G][Kp / 32]: the row's scale bytes
  int8_t* chi2 = reinterpret_cast<int8_t*>(sfs_all + (size_t)G * (Kp / 32));
  int8_t* sq = chi2 + 2 * q + 1;

  xqptx::pdl_launch_dependents();
  if (Bimage) {
    // prepared with the weights (a constant of the plan)
    for (int i = tid; i < dp * pitch / 8; i += blockDim.x) xqptx::cp_async16(Bs + 8 * i, Bimage + 8 * i);
  } else {
    if (pl.p > 1) build_chi(q, chi2, sq, pl.paley_kind);
    for (int i = tid; i < dp * pitch; i += blockDim.x) {
      const int c2 = i / pitch, c = i - c2 * pitch;
      uint16_t bits = 0;
      if (c < d) {
        const int a = c >> pl.log2n, b = c & (n - 1), a2 = c2 >> pl.log2n, b2 = c2 & (n - 1);
        int s = (__popc(b & b2) & 1) ? -1 : 1;
        if (pl.p > 1) s *= paley_sign(pl.paley_kind, q, chi2, a, a2);
        bits = s > 0 ? 0x3F80 : 0xBF80;
      }
      reinterpret_cast<uint16_t*>(Bs)[i] = bits;
    }
  }
  // rows of absent heads and the columns past d stay zero in every stage
  for (int i = tid; i < G * 2 * H16 * pitch / 8; i += blockDim.x) reinterpret_cast<uint4*>(Xs_all)[i] = make_uint4(0, 0, 0, 0);
  xqptx::cp_async_wait_all();
  xqptx::pdl_wait();
  __syncthreads();
  if (group >= G) return;  // warps beyond the groups in use (few tokens: one group per CTA)

  __nv_bfloat16* Xs = Xs_all + (size_t)group * 2 * H16 * pitch;
  uint32_t* outp = outp_all + (size_t)group * (Kp / 8);
  float* red = red_all + group * 2 * HT;
  const int chunks = heads * d / 8;  // 16-byte pieces of a token row
  const int row0 = blockIdx.x * G + group, rstep = gridDim.x * G;

  auto load_row = [&](int row, int stage) {
    const __nv_bfloat16* x = X + (long long)row * ldx;
    __nv_bfloat16* dst = Xs + (size_t)stage * H16 * pitch;
    for (int i = gtid; i < chunks; i += gthreads) {
      const int c = 8 * i, h = c / d, k = c - h * d;
      xqptx::cp_async16(dst + h * pitch + k, x + c);
    }
  };
  if (row0 < M) load_row(row0, 0);
  xqptx::cp_async_commit();
  int stage = 0;
  for (int row = row0; row < M; row += rstep, stage ^= 1) {
    if (row + rstep < M) load_row(row + rstep, stage ^ 1);
    xqptx::cp_async_commit();
    xqptx::cp_async_wait_group<1>();
    group_sync(group, HT);

    float acc[kMaxNT][4];
#pragma unroll
    for (int j = 0; j < kMaxNT; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f;
    const __nv_bfloat16* ap = Xs + (size_t)stage * H16 * pitch + (16 * ht + g) * pitch + 2 * t;
    const __nv_bfloat16* bp = Bs + g * pitch + 2 * t;
    for (int k0 = 0; k0 < d16; k0 += 16) {
      uint32_t a[4];
      a[0] = *reinterpret_cast<const uint32_t*>(ap + k0);
      a[1] = *reinterpret_cast<const uint32_t*>(ap + 8 * pitch + k0);
      a[2] = *reinterpret_cast<const uint32_t*>(ap + k0 + 8);
      a[3] = *reinterpret_cast<const uint32_t*>(ap + 8 * pitch + k0 + 8);
#pragma unroll
      for (int j = 0; j < kMaxNT; ++j) {
        if (j < NT) {
          const uint32_t b0 = *reinterpret_cast<const uint32_t*>(bp + 8 * j * pitch + k0);
          const uint32_t b1 = *reinterpret_cast<const uint32_t*>(bp + 8 * j * pitch + k0 + 8);
          xqptx::mma_bf16_16x8x16(acc[j], a, b0, b1);
        }
      }
    }
    float vmax = 0.f, vmin = 0.f;
#pragma unroll
    for (int j = 0; j < kMaxNT; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        acc[j][e] *= gamma;  // tiles past NT hold zeros
        vmax = fmaxf(vmax, acc[j][e]);
        vmin = fminf(vmin, acc[j][e]);
      }
    for (int o = 16; o > 0 && !MX; o >>= 1) {
      vmax = fmaxf(vmax, __shfl_xor_sync(0xffffffffu, vmax, o));
      vmin = fminf(vmin, __shfl_xor_sync(0xffffffffu, vmin, o));
    }
    if (HT > 1 && !MX) {
      if (lane == 0) {
        red[ht] = vmax;
        red[HT + ht] = vmin;
      }
      group_sync(group, HT);
      for (int i = 0; i < HT; ++i) {
        vmax = fmaxf(vmax, red[i]);
        vmin = fminf(vmin, red[HT + i]);
      }
    }
    const RowQuant rq = zp ? row_quant_asym(vmin, vmax) : row_quant_sym(fmaxf(vmax, -vmin));
    if constexpr (MX) {
      // MXFP4: tile (head h, columns 8 j ..) is tile h NT + j of the row; four consecutive tiles are one group
      float* tmax = tmax_all + (size_t)group * (Kp / 8);
      uint8_t* sfs = sfs_all + (size_t)group * (Kp / 32);
#pragma unroll
      for (int j = 0; j < kMaxNT; ++j) {
        if (j < NT) {
#pragma unroll
          for (int r = 0; r < 2; ++r) {
            const int h = 16 * ht + g + 8 * r;
            float m = fmaxf(fabsf(acc[j][2 * r]), fabsf(acc[j][2 * r + 1]));
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
            if (t == 0 && h < heads) tmax[h * NT + j] = m;
          }
        }
      }
      group_sync(group, HT);
#pragma unroll
      for (int j = 0; j < kMaxNT; ++j) {
        if (j < NT) {
#pragma unroll
          for (int r = 0; r < 2; ++r) {
            const int h = 16 * ht + g + 8 * r;
            const int idx = (h < heads ? h : 0) * NT + j;
            const float4 q4 = *reinterpret_cast<const float4*>(tmax + (idx & ~3));
            const int e = mx_shared_exp(fmaxf(fmaxf(q4.x, q4.y), fmaxf(q4.z, q4.w)));
            const float inv = mx_inv_scale(e);
            uint32_t w = mx_e2m1_pair(acc[j][2 * r] * inv, acc[j][2 * r + 1] * inv) << (8 * t);
            w |= __shfl_xor_sync(0xffffffffu, w, 1);
            w |= __shfl_xor_sync(0xffffffffu, w, 2);
            if (t == 0 && h < heads) {
              outp[idx] = w;
              if ((idx & 3) == 0) sfs[idx >> 2] = (uint8_t)(e + 127);
            }
          }
          asm volatile("" ::: "memory");  // keeps the tile-maximum loads of later column tiles from being hoisted (registers)
        }
      }
    }
    // quantize, pack: the quad's four bytes of one (head, column tile) form one word of 8 codes
#pragma unroll
    for (int j = 0; j < kMaxNT; ++j) {
      if (j < NT && !MX) {
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          const int h = 16 * ht + g + 8 * r;
          const int lo = row_code(rq, acc[j][2 * r]);
          const int hi = row_code(rq, acc[j][2 * r + 1]);
          uint32_t w = (uint32_t)((lo & 0xF) | ((hi & 0xF) << 4)) << (8 * t);
          w |= __shfl_xor_sync(0xffffffffu, w, 1);
          w |= __shfl_xor_sync(0xffffffffu, w, 2);
          if (t == 0 && h < heads) outp[h * NT + j] = w;
          if (Yopt && h < heads)
            *reinterpret_cast<float2*>(Yopt + (long long)row * Kp + h * dp + 8 * j + 2 * t) = make_float2(acc[j][2 * r], acc[j][2 * r + 1]);
        }
      }
    }
    group_sync(group, HT);
    if (gtid == 0 && !MX) {
      sx[row] = rq.s;
      if (zp) zp[row] = rq.z;
    }
    if (MX) {  // scale bytes into their blocks; padding up to Kq: unit scales and zero codes (never a NaN scale byte)
      const uint8_t* sfs = sfs_all + (size_t)group * (Kp / 32);
      for (int i = gtid; i < Kq / 32; i += gthreads) sfb[xq_mx_sf_offset(row, i, Kq)] = i < Kp / 32 ? sfs[i] : (uint8_t)127;
      for (int i = gtid; i < (Kq - Kp) / 8; i += gthreads) *reinterpret_cast<uint32_t*>(Xq + (long long)row * (Kq / 2) + Kp / 2 + 4 * i) = 0u;
    }
    uint4* dst = reinterpret_cast<uint4*>(Xq + (long long)row * ((MX ? Kq : Kp) / 2));
    for (int i = gtid; i < Kp / 32; i += gthreads) {
      const uint4 v = reinterpret_cast<const uint4*>(outp)[i];
      dst[i] = v;
      if (A8opt) {
        uint4 e0, e1;
        xqptx::split16(v.x, e0.x, e0.y);
        xqptx::split16(v.y, e0.z, e0.w);
        xqptx::split16(v.z, e1.x, e1.y);
        xqptx::split16(v.w, e1.z, e1.w);
        uint4* d8 = reinterpret_cast<uint4*>(A8opt + (long long)row * Kp);
        d8[2 * i] = e0;
        d8[2 * i + 1] = e1;
      }
    }
    // the group is done with this stage, its packed row and the reduction slots
    group_sync(group, HT);
  }
  xqptx::cp_async_wait_all();
}

size_t heads_smem(const xq_hadamard_plan_t& pl, int heads, int G) {
  const int d16 = (pl.K + 15) / 16 * 16, pitch = d16 + 8, H16 = (heads + 15) / 16 * 16;
  return (size_t)pl.Kp * pitch * 2 + (size_t)G * 2 * H16 * pitch * 2 + (size_t)G * heads * pl.Kp + (size_t)G * heads * pl.Kp / 32 + (2 * kWarps + 32) * 4 +
         (size_t)(3 * pl.q + 1) + 32;
}

}  // namespace

bool xq_rotate_heads_supported(const xq_hadamard_plan_t& pl, int32_t heads) {
  if (heads < 1 || heads > 128 || pl.K % 8 != 0 || pl.K > 128 || pl.Kp % 8 != 0 || pl.Kp > 8 * kMaxNT) return false;
  if (((long long)heads * pl.Kp) % 32 != 0) return false;
  return heads_smem(pl, heads, 1) <= 200 * 1024;
}

size_t xq_head_image_elems(const xq_hadamard_plan_t& pl) {
  const int d16 = (pl.K + 15) / 16 * 16;
  return (size_t)pl.Kp * (d16 + 8);
}

cudaError_t xq_launch_rotate_heads(const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t& pl, int32_t heads, uint8_t* Xq,
                                   float* sx, float* Yopt, uint8_t* A8opt, const void* Bimage, int32_t* zp, int sms,
                                   cudaStream_t st, const xq_mx_out* mx) {
  if (!xq_rotate_heads_supported(pl, heads)) return cudaErrorNotSupported;
  if (mx) {
    if (((long long)heads * pl.Kp) % 32 != 0) return cudaErrorNotSupported;
    Xq = mx->codes;
  }
  const float gamma = (float)(1.0 / sqrt((double)pl.Kp));
  const int HT = (heads + 15) / 16;
  // token groups per CTA: as many as the warps allow once there are more tokens than multiprocessors
  int G = kWarps / HT;
  const int want = (M + sms - 1) / sms;
  if (G > want) G = want;
  while (G > 1 && heads_smem(pl, heads, G) > 200 * 1024) --G;
  const size_t smem = heads_smem(pl, heads, G);
  auto kern = mx ? rotate_quant_heads_kernel<true> : rotate_quant_heads_kernel<false>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int per_sm = (mx || smem > 100 * 1024) ? 1 : 2;  // two CTAs of the INT4 form fit the register file
  const int ctas = (M + G - 1) / G;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(ctas < sms * per_sm ? ctas : sms * per_sm);
  cfg.blockDim = dim3(kWarps * 32);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, (const __nv_bfloat16*)X, (int)M, (long long)ldx, pl, (int)heads, gamma,
                            Xq, sx, Yopt, A8opt, (const __nv_bfloat16*)Bimage, zp, mx ? mx->sf_blocks : (uint8_t*)nullptr,
                            mx ? (int)mx->Kq : 0, G);
}
