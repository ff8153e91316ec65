// MXFP4 form of the expanded layer (paper Sec. 4 "Quantization Details": weights and activations in
// the OCP microscaling format, an E8M0 scale for each group of 32 elements, E2M1 elements; Sec. 5
// "OCP MXFP4 Results": hardware that applies the group scales inside the matrix product).
//
// Online step: the pad + rotate kernels leave the rotated row in fp32, mx_quantize_kernel turns
// every group of 32 channels into a shared exponent and 32 four-bit codes.  Product: tcgen05.mma
// kind::mxf4 with block scaling -- both operands stay packed (two codes per byte) from HBM to the
// tensor core: TMA loads 128-byte rows (256 codes) into the 128-byte-swizzled K-major stage, the
// scale bytes travel as 512-byte blocks (32 rows x 16 bytes: the four scales of rows r, r + 32,
// r + 64, r + 96 for four consecutive groups) that tcgen05.cp broadcasts into tensor memory, and
// every MMA of 64 codes names the two scale bytes of each row it needs.  fp32 accumulators in
// tensor memory, bf16 epilogue.  No unpacking anywhere.
//
// Layouts in HBM (device, opaque): codes [rows][Kq / 2] bytes, Kq = K' rounded up to 256, low
// nibble = even channel; scale blocks [ceil(rows / 128)][Kq / 128][512 bytes] with the byte of
// (row m, group g) at (m % 32) * 16 + ((m / 32) % 4) * 4 + g % 4.
// All barrier waits are time-bounded as in the INT4 kernels.
#include <cuda.h>
#include <cuda_bf16.h>
#include <math.h>
#include <string.h>

#include <new>

#include "xq_hadamard.cuh"
#include "xq_internal.h"
#include "xq_ptx.cuh"

using namespace xqptx;

struct xq_mx_weights {
  int32_t N, K, Kp;  // logical sizes (head-wise: heads * head_dim, heads * head_dim')
  int32_t heads;     // 1: one rotation K -> Kp; > 1: the plan is that of one head
  uint16_t* head_signs;
  int32_t Np, Kq;    // rows padded to 256, K' padded to 256
  xq_hadamard_plan_t plan;
  uint8_t* codes;    // device, Np * Kq / 2
  uint8_t* sf;       // device, (Np / 128) * (Kq / 128) * 512
  uint8_t* sf_wide;  // device, the same bytes in the order of 224-channel tiles: ceil(N / 224) * (Kq / 128) * 1024
  uint16_t* hp_signs;
  int device, sms;
};

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

__host__ __device__ inline size_t sf_offset(int m, int g, int Kq) { return xq_mx_sf_offset(m, g, Kq); }
inline size_t sf_bytes(int rows, int Kq) { return (size_t)((rows + 127) / 128) * (Kq / 128) * 512; }

// ---------------------------------------------------------------------------------------------
// Quantizer: one warp per (row, group of 32); lane i holds channel 32 g + i.
//   e = floor(log2(max |v|)) - 2 clamped to [-127, 127] (0 for a group of zeros), scale byte e + 127,
//   element = nearest E2M1 value to v / 2^e, ties to the even mantissa bit, saturating at 6.
// Groups past K' (padding up to Kq) get zero codes.
// ---------------------------------------------------------------------------------------------

__global__ void __launch_bounds__(256) mx_quantize_kernel(const float* __restrict__ Y, int R, int Kp, int Kq, long long ldy,
                                                          uint8_t* __restrict__ codes, long long code_pitch,
                                                          uint8_t* __restrict__ sf_blocks, uint8_t* __restrict__ sf_rows) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int groups = Kq / 32, real = Kp / 32;
  const long long total = (long long)R * groups;
  for (long long wi = (blockIdx.x * (long long)blockDim.x + threadIdx.x) >> 5; wi < total; wi += ((long long)gridDim.x * blockDim.x) >> 5) {
    const int m = (int)(wi / groups), g = (int)(wi - (long long)m * groups);
    float v = 0.f;
    if (g < real) v = Y[(long long)m * ldy + 32 * g + lane];
    float a = fabsf(v);
    for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
    const int e = xqhad::mx_shared_exp(a);
    const uint32_t code = xqhad::mx_e2m1_code(v * xqhad::mx_inv_scale(e));  // exact scaling by a power of two
    uint32_t w = code << (4 * (lane & 7));
    w |= __shfl_xor_sync(0xffffffffu, w, 1);
    w |= __shfl_xor_sync(0xffffffffu, w, 2);
    w |= __shfl_xor_sync(0xffffffffu, w, 4);
    if ((lane & 7) == 0 && (code_pitch * 2 >= 32ll * (g + 1)))
      *reinterpret_cast<uint32_t*>(codes + (long long)m * code_pitch + 16 * g + 4 * (lane >> 3)) = w;
    if (lane == 0) {
      if (sf_blocks) sf_blocks[sf_offset(m, g, Kq)] = (uint8_t)(e + 127);
      if (sf_rows && g < real) sf_rows[(long long)m * real + g] = (uint8_t)(e + 127);
    }
  }
}

// Canonical form (codes [R][Kp / 2], scales [R][Kp / 32]) <-> device form.
__global__ void mx_to_device_form_kernel(const uint8_t* __restrict__ codes_rows, const uint8_t* __restrict__ sf_rows, int R, int Kp,
                                         int Kq, uint8_t* __restrict__ codes, uint8_t* __restrict__ sf_blocks) {
  pdl_launch_dependents();
  pdl_wait();
  const long long words = (long long)R * (Kq / 8);
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < words; i += (long long)gridDim.x * blockDim.x) {
    const int m = (int)(i / (Kq / 8)), wq = (int)(i % (Kq / 8));
    uint32_t w = 0;
    if (wq < Kp / 8) w = *reinterpret_cast<const uint32_t*>(codes_rows + (long long)m * (Kp / 2) + 4 * wq);
    *reinterpret_cast<uint32_t*>(codes + (long long)m * (Kq / 2) + 4 * wq) = w;
    if ((wq & 3) == 0) {
      const int g = wq >> 2;
      sf_blocks[sf_offset(m, g, Kq)] = g < Kp / 32 ? sf_rows[(long long)m * (Kp / 32) + g] : (uint8_t)127;
    }
  }
}

__global__ void mx_from_device_form_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ sf_blocks, int R, int Kp,
                                           int Kq, uint8_t* __restrict__ code_bytes, uint8_t* __restrict__ sf_rows) {
  const long long total = (long long)R * Kp;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int m = (int)(i / Kp), c = (int)(i % Kp);
    const uint8_t b = codes[(long long)m * (Kq / 2) + (c >> 1)];
    code_bytes[i] = (c & 1) ? (b >> 4) : (b & 0xF);
    if ((c & 31) == 0) sf_rows[(long long)m * (Kp / 32) + (c >> 5)] = sf_blocks[sf_offset(m, c >> 5, Kq)];
  }
}

// ---------------------------------------------------------------------------------------------
// Product.  Tile: 128 tokens x TN channels (TN = 224 or 256, see TileCfg), K in blocks of 256 codes
// (one 128-byte row piece).
//   warp 0   producer: per stage two TMA tiles (tokens 16 KiB, weights TN x 128 bytes) and the
//            scale blocks as bulk copies (tokens 1 KiB, weights 2 KiB)
//   warp 1   MMA issue: copies the scale blocks into tensor memory (tcgen05.cp), then four
//            tcgen05.mma kind::mxf4 of 128 x TN x 64; fp32 accumulators of TN columns
//   warps 2-5 epilogue: tcgen05.ld, fp32 -> bf16, 16-byte stores
// ---------------------------------------------------------------------------------------------
constexpr int BM = 128, BN = 256;
constexpr int kStages = 4;
constexpr int kABytes = BM * 128, kSfaBytes = 1024, kSfbBytes = 2048;
// TN = 256: one accumulator of 256 columns (the epilogue of a tile is not hidden).  TN = 224: two accumulators of 224
// columns, the epilogue of a tile runs under the main loop of the next; the weight scales then come in the
// 224-channel tile order (xq_mx_weights::sf_wide).  Tensor memory: 2 x 224 + 2 x 32 scale columns = 512.
template <int TN>
struct TileCfg {
  static constexpr int kBBytes = TN * 128;
  static constexpr int kStageBytes = kABytes + kBBytes + kSfaBytes + kSfbBytes;  // a multiple of 1024 for both
  static constexpr int kAccBufs = TN == 224 ? 2 : 1;
  static constexpr int kSfaCol = TN == 224 ? 448 : 256, kSfbCol = kSfaCol + (TN == 224 ? 8 : 16);  // + 32 per stage parity
  static constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + 256;
};
constexpr int kThreads = 6 * 32;
constexpr int kTmemCols = 512;

struct MxParams {
  const uint8_t* sfa;  // token scale blocks
  const uint8_t* sfb;  // weight scale blocks
  __nv_bfloat16* out;
  int32_t* status;
  int M, N, KB, Kq;    // KB = Kq / 256
  int tiles_m, tiles_n;
};

// E2M1 operands (format 1 of kind::mxf4) at bits 7-9 and 10-12, both K-major; N >> 3 at bits 17-22; E8M0 scales
// (bit 23); M >> 4 at bits 24-28; which bytes of the scale columns an instruction reads: bits 4-5 (B), 29-30 (A).
__device__ __forceinline__ uint32_t mx_idesc_n(uint32_t sf_id, int n) {
  return (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | (1u << 23) | ((uint32_t)(128 >> 4) << 24) | (sf_id << 4) | (sf_id << 29);
}
// 32 rows of 16 bytes, no swizzle: 8-row groups 128 bytes apart.
__device__ __forceinline__ uint64_t sf_desc(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | ((uint64_t)(128 >> 4) << 32) | (1ull << 46);
}
__device__ __forceinline__ void tmem_cp_32x128b_warpx4(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void umma_mxf4_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate,
                                             uint32_t sfa_tmem, uint32_t sfb_tmem) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.block32 [%0], %1, %2, %3, [%5], [%6], p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
      : "memory");
}

template <int TN>
__global__ void __launch_bounds__(kThreads, 1) gemm_mx_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                                                              const MxParams p) {
  using C = TileCfg<TN>;
  constexpr int kBBytes = C::kBBytes, kStageBytes = C::kStageBytes, kAccBufs = C::kAccBufs;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  unsigned char* base = smem_raw + (((raw + 1023u) & ~1023u) - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(base + (size_t)kStages * kStageBytes);
  uint64_t* full = bars;
  uint64_t* empty = full + kStages;
  uint64_t* acc_full = empty + kStages;
  uint64_t* acc_empty = acc_full + 2;
  uint64_t* drain = acc_empty + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
  volatile int* failed = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tiles = p.tiles_m * p.tiles_n;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&acc_full[b], 1);
      mbar_init(&acc_empty[b], 4);
    }
    mbar_init(drain, 1);
    *failed = 0;
    mbar_fence_init();
    tma_prefetch_desc(&mapA);
    tma_prefetch_desc(&mapB);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // the kernel after this one is let in late (by the MMA warp, below): released here, at the start, it cost 1-5 % of a
  // layer's step (measured)
  pdl_wait();  // tokens and their scales come from the kernel before this one

  if (warp == 0) {
    // ---------------- producer --------------------------------------------------------------------
    uint32_t it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
      const int tm = tile % p.tiles_m, tn = tile / p.tiles_m;
      for (int kb = 0; kb < p.KB; ++kb, ++it) {
        const int s = it % kStages;
        if (it >= (uint32_t)kStages) {
          ok = mbar_wait_bounded(&empty[s], ((it / kStages) - 1) & 1, failed, p.status, (int)XQ_ERR_TIMEOUT);
          if (!ok) break;
        }
        if (lane == 0) {
          unsigned char* st = base + (size_t)s * kStageBytes;
          mbar_expect_tx(&full[s], kStageBytes);
          tma_load_2d(st, &mapA, kb * 128, tm * BM, &full[s]);
          tma_load_2d(st + kABytes, &mapB, kb * 128, tn * TN, &full[s]);
          const size_t kblocks = (size_t)(p.Kq >> 7);  // scale blocks along K per 128 rows
          bulk_g2s(st + kABytes + kBBytes, p.sfa + ((size_t)tm * kblocks + 2 * kb) * 512, kSfaBytes, &full[s]);
          if (TN == 224) {  // tile order: [128-code block][channels 0..127 | 128..223]
            bulk_g2s(st + kABytes + kBBytes + kSfaBytes, p.sfb + (((size_t)tn * kblocks + 2 * kb) * 2) * 512, kSfbBytes, &full[s]);
          } else {          // blocks of 128 channels: [channels 0..127 | 128..255][128-code block]
            bulk_g2s(st + kABytes + kBBytes + kSfaBytes, p.sfb + ((size_t)(2 * tn) * kblocks + 2 * kb) * 512, 1024, &full[s]);
            bulk_g2s(st + kABytes + kBBytes + kSfaBytes + 1024, p.sfb + ((size_t)(2 * tn + 1) * kblocks + 2 * kb) * 512, 1024, &full[s]);
          }
        }
        __syncwarp();
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issue -------------------------------------------------------------------
    uint32_t it = 0, tcount = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tcount) {
      const uint32_t buf = kAccBufs == 2 ? (tcount & 1u) : 0u;
      const uint32_t use = kAccBufs == 2 ? (tcount >> 1) : tcount;  // earlier uses of this accumulator
      if (use >= 1u) {
        ok = mbar_wait_bounded(&acc_empty[buf], (use - 1) & 1, failed, p.status, (int)XQ_ERR_TIMEOUT);
        if (!ok) break;
      }
      tc_fence_after_sync();
      for (int kb = 0; kb < p.KB; ++kb, ++it) {
        const int s = it % kStages;
        ok = mbar_wait_bounded(&full[s], (it / kStages) & 1, failed, p.status, (int)XQ_ERR_TIMEOUT);
        if (!ok) break;
        tc_fence_after_sync();
        if (lane == 0) {
          const uint32_t a_addr = smem_u32(base + (size_t)s * kStageBytes);
          const uint32_t sfa_smem = a_addr + kABytes + kBBytes, sfb_smem = sfa_smem + kSfaBytes;
          // scale columns alternate between two sets so that a copy never lands under an MMA still in flight
          const uint32_t sfa_t = tmem_base + C::kSfaCol + 32 * (it & 1), sfb_t = tmem_base + C::kSfbCol + 32 * (it & 1);
#pragma unroll
          for (int j = 0; j < 2; ++j) {  // K halves of 128 codes: 4 token columns, 8 weight columns each
            tmem_cp_32x128b_warpx4(sfa_t + 4 * j, sf_desc(sfa_smem + 512 * j));
            // channels 0..127 of the tile, then the rest
            tmem_cp_32x128b_warpx4(sfb_t + 8 * j, sf_desc(sfb_smem + (TN == 224 ? 1024 * j : 512 * j)));
            tmem_cp_32x128b_warpx4(sfb_t + 8 * j + 4, sf_desc(sfb_smem + (TN == 224 ? 1024 * j + 512 : 1024 + 512 * j)));
          }
          const uint64_t adesc = umma_desc_k128(a_addr), bdesc = umma_desc_k128(a_addr + kABytes);
#pragma unroll
          for (int k = 0; k < 4; ++k)  // 64 codes = 32 bytes per instruction; its two scale bytes: 0-1 or 2-3 of the column
            umma_mxf4_ss(tmem_base + buf * TN, adesc + 2 * k, bdesc + 2 * k, mx_idesc_n(2u * (k & 1), TN), (kb | k) != 0 ? 1u : 0u,
                         sfa_t + 4 * (k >> 1), sfb_t + 8 * (k >> 1));
          umma_commit(&empty[s]);
        }
        __syncwarp();
      }
      if (ok && lane == 0) umma_commit(&acc_full[buf]);
      __syncwarp();
    }
    if (lane == 0) umma_commit(drain);
    pdl_launch_dependents();
    __syncwarp();
    mbar_wait_bounded(drain, 0, failed, p.status, (int)XQ_ERR_TIMEOUT);
  } else {
    // ---------------- epilogue --------------------------------------------------------------------
    const int q = warp & 3;  // tensor-memory lane quarter this warp may read
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tcount) {
      const int tm = tile % p.tiles_m, tn = tile / p.tiles_m;
      const int m = tm * BM + q * 32 + lane, n0 = tn * TN;
      const uint32_t buf = kAccBufs == 2 ? (tcount & 1u) : 0u;
      const uint32_t use = kAccBufs == 2 ? (tcount >> 1) : tcount;
      ok = mbar_wait_bounded(&acc_full[buf], use & 1, failed, p.status, (int)XQ_ERR_TIMEOUT);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * TN;
#pragma unroll 1
      for (int c = 0; c < TN / 32; ++c) {
        uint32_t v[32];
        tmem_ld_32x32(taddr + c * 32, v);
        tmem_ld_wait();
        const int nc = n0 + c * 32;
        if (m < p.M && nc < p.N) {
          const size_t o = (size_t)m * p.N + nc;
#pragma unroll
          for (int g8 = 0; g8 < 4; ++g8) {
            if (nc + 8 * g8 < p.N) {  // N is a multiple of 8
              uint32_t h[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const __nv_bfloat162 b2 = __halves2bfloat162(__float2bfloat16_rn(__uint_as_float(v[8 * g8 + 2 * e])),
                                                             __float2bfloat16_rn(__uint_as_float(v[8 * g8 + 2 * e + 1])));
                h[e] = *reinterpret_cast<const uint32_t*>(&b2);
              }
              *reinterpret_cast<uint4*>(p.out + o + 8 * g8) = make_uint4(h[0], h[1], h[2], h[3]);
            }
          }
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[buf]);
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0 && *failed) {
    // bounded drain of copies that may still be landing in this CTA's shared memory
    for (int s = 0; s < kStages; ++s) mbar_wait(&full[s], 0, 1u << 16), mbar_wait(&full[s], 1, 1u << 16);
  }
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---------------------------------------------------------------------------------------------
// Weight scales in the order of 224-channel tiles (what the 224-column tile kernel copies): per tile and 128-code
// block two blocks of 32 x 16 bytes, channels 0..127 and 128..223 of the tile.
// ---------------------------------------------------------------------------------------------
constexpr int WN = 224;

__host__ __device__ inline size_t sf_wide_offset(int n, int g, int Kq) {
  const int tile = n / WN, r = n - tile * WN, atom = r >> 7, ra = r & 127;
  return (((size_t)tile * (Kq >> 7) + (g >> 2)) * 2 + atom) * 512 + (size_t)(ra & 31) * 16 + (size_t)(ra >> 5) * 4 + (g & 3);
}

__global__ void mx_sf_to_wide_kernel(const uint8_t* __restrict__ sf_blocks, int N, int Kq, uint8_t* __restrict__ sf_wide) {
  const long long total = (long long)N * (Kq / 32);
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int n = (int)(i / (Kq / 32)), g = (int)(i % (Kq / 32));
    sf_wide[sf_wide_offset(n, g, Kq)] = sf_blocks[xq_mx_sf_offset(n, g, Kq)];
  }
}

// ---------------------------------------------------------------------------------------------
// Product for few tokens (M <= 32): the roles of the operands are swapped -- 128 output channels
// are the 128 rows of the MMA, the tokens its 32 columns -- so that a tile streams the weights of
// 128 channels, and K is cut into S slices over S CTAs so that every multiprocessor streams.  Each
// CTA leaves its 128 x 32 fp32 partial tile in the workspace and counts itself in; the CTA that
// arrives last adds the S partial tiles in slice order (the result does not depend on arrival
// order), writes bf16 and puts the counter back to zero.  Nobody waits for anybody.
// ---------------------------------------------------------------------------------------------
constexpr int DN = 32;                      // token columns of the MMA
constexpr int kDStages = 8;
constexpr int kDABytes = 128 * 128, kDBBytes = DN * 128, kDSfBytes = 1024;  // weights, tokens, scale blocks of each
constexpr int kDStageBytes = kDABytes + kDBBytes + 2 * kDSfBytes;           // 22 KiB
constexpr int kDTmemCols = 128;
constexpr int kDSfaCol = 32, kDSfbCol = 48;  // per stage parity: + 32 columns
constexpr size_t kDSmemBytes = 1024 + (size_t)kDStages * kDStageBytes + 256;

struct MxDecodeParams {
  const uint8_t* sfw;  // weight scale blocks
  const uint8_t* sfx;  // token scale blocks
  __nv_bfloat16* out;
  float* partial;      // [tiles][S][128][32] fp32
  int32_t* counters;   // [tiles]
  int32_t* status;
  int M, N, KB, Kq, S;
};

__global__ void __launch_bounds__(kThreads, 1) gemm_mx_decode_kernel(const __grid_constant__ CUtensorMap mapW,
                                                                     const __grid_constant__ CUtensorMap mapX, const MxDecodeParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  unsigned char* base = smem_raw + (((raw + 1023u) & ~1023u) - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(base + (size_t)kDStages * kDStageBytes);
  uint64_t* full = bars;
  uint64_t* empty = full + kDStages;
  uint64_t* acc_full = empty + kDStages;
  uint64_t* drain = acc_full + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
  volatile int* failed = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* last_flag = const_cast<int*>(reinterpret_cast<volatile int*>(tmem_slot + 2));

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tile = blockIdx.x / p.S, split = blockIdx.x - tile * p.S;
  const int kb_lo = (split * p.KB) / p.S, kb_hi = ((split + 1) * p.KB) / p.S;  // this CTA's 256-code blocks (at least one)

  if (tid == 0) {
    for (int s = 0; s < kDStages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    mbar_init(acc_full, 1);
    mbar_init(drain, 1);
    *failed = 0;
    *last_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&mapW);
    tma_prefetch_desc(&mapX);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kDTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  pdl_launch_dependents();

  if (warp == 0) {
    // ---------------- producer: weights first (they do not depend on the kernel before), then tokens ----------
    const size_t kblocks = (size_t)(p.Kq >> 7);
    bool ok = true;
    const int nk = kb_hi - kb_lo, pre = nk < kDStages ? nk : kDStages;
    if (lane == 0) {
      for (int i = 0; i < pre; ++i) {
        unsigned char* st = base + (size_t)i * kDStageBytes;
        mbar_expect_tx(&full[i], kDStageBytes);
        tma_load_2d(st, &mapW, (kb_lo + i) * 128, tile * 128, &full[i]);
        bulk_g2s(st + kDABytes + kDBBytes, p.sfw + ((size_t)tile * kblocks + 2 * (kb_lo + i)) * 512, kDSfBytes, &full[i]);
      }
    }
    __syncwarp();
    pdl_wait();  // the tokens and their scales come from the kernel before this one
    for (int i = 0; i < nk && ok; ++i) {
      const int s = i % kDStages, kb = kb_lo + i;
      if (i >= kDStages) {
        ok = mbar_wait_bounded(&empty[s], ((i / kDStages) - 1) & 1, failed, p.status, (int)XQ_ERR_TIMEOUT);
        if (!ok) break;
      }
      if (lane == 0) {
        unsigned char* st = base + (size_t)s * kDStageBytes;
        if (i >= kDStages) {
          mbar_expect_tx(&full[s], kDStageBytes);
          tma_load_2d(st, &mapW, kb * 128, tile * 128, &full[s]);
          bulk_g2s(st + kDABytes + kDBBytes, p.sfw + ((size_t)tile * kblocks + 2 * kb) * 512, kDSfBytes, &full[s]);
        }
        tma_load_2d(st + kDABytes, &mapX, kb * 128, 0, &full[s]);
        bulk_g2s(st + kDABytes + kDBBytes + kDSfBytes, p.sfx + (size_t)(2 * kb) * 512, kDSfBytes, &full[s]);
      }
      __syncwarp();
    }
  } else if (warp == 1) {
    // ---------------- MMA issue -------------------------------------------------------------------
    bool ok = true;
    const int nk = kb_hi - kb_lo;
    for (int i = 0; i < nk; ++i) {
      const int s = i % kDStages;
      ok = mbar_wait_bounded(&full[s], (i / kDStages) & 1, failed, p.status, (int)XQ_ERR_TIMEOUT);
      if (!ok) break;
      tc_fence_after_sync();
      if (lane == 0) {
        const uint32_t a_addr = smem_u32(base + (size_t)s * kDStageBytes);
        const uint32_t sfa_smem = a_addr + kDABytes + kDBBytes, sfb_smem = sfa_smem + kDSfBytes;
        const uint32_t sfa_t = tmem_base + kDSfaCol + 32 * (i & 1), sfb_t = tmem_base + kDSfbCol + 32 * (i & 1);
#pragma unroll
        for (int j = 0; j < 2; ++j) {  // K halves of 128 codes: 4 columns of channel scales, 4 of token scales (one used)
          tmem_cp_32x128b_warpx4(sfa_t + 4 * j, sf_desc(sfa_smem + 512 * j));
          tmem_cp_32x128b_warpx4(sfb_t + 4 * j, sf_desc(sfb_smem + 512 * j));
        }
        const uint64_t adesc = umma_desc_k128(a_addr), bdesc = umma_desc_k128(a_addr + kDABytes);
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_mxf4_ss(tmem_base, adesc + 2 * k, bdesc + 2 * k, mx_idesc_n(2u * (k & 1), DN), (i | k) != 0 ? 1u : 0u, sfa_t + 4 * (k >> 1),
                       sfb_t + 4 * (k >> 1));
        umma_commit(&empty[s]);
      }
      __syncwarp();
    }
    if (ok && lane == 0) umma_commit(acc_full);
    __syncwarp();
    if (lane == 0) umma_commit(drain);
    __syncwarp();
    mbar_wait_bounded(drain, 0, failed, p.status, (int)XQ_ERR_TIMEOUT);
  } else {
    // ---------------- epilogue: lane = one output channel, 32 token columns ---------------------------
    const int q = warp & 3, et = (warp - 2) * 32 + lane;  // thread index among the 128 epilogue threads
    const int c = q * 32 + lane, n = tile * 128 + c;
    bool ok = mbar_wait_bounded(acc_full, 0, failed, p.status, (int)XQ_ERR_TIMEOUT);
    float v[32];
    if (ok) {
      tc_fence_after_sync();
      uint32_t r[32];
      tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16), r);
      tmem_ld_wait();
#pragma unroll
      for (int m = 0; m < 32; ++m) v[m] = __uint_as_float(r[m]);
    }
    bool reduce = ok && p.S == 1;
    if (ok && p.S > 1) {
      float4* dst = reinterpret_cast<float4*>(p.partial + (((size_t)tile * p.S + split) * 128 + c) * 32);
#pragma unroll
      for (int m4 = 0; m4 < 8; ++m4) __stcg(dst + m4, make_float4(v[4 * m4], v[4 * m4 + 1], v[4 * m4 + 2], v[4 * m4 + 3]));
      __threadfence();
    }
    bar_sync(1, 128);
    if (p.S > 1) {
      if (et == 0) *last_flag = ok && atomicAdd(p.counters + tile, 1) == p.S - 1;
      bar_sync(1, 128);
      if (*last_flag) {
        __threadfence();
#pragma unroll
        for (int m = 0; m < 32; ++m) v[m] = 0.f;
        for (int s = 0; s < p.S; ++s) {  // slice order: the sum does not depend on who arrived when
          const float4* src = reinterpret_cast<const float4*>(p.partial + (((size_t)tile * p.S + s) * 128 + c) * 32);
#pragma unroll
          for (int m4 = 0; m4 < 8; ++m4) {
            const float4 t = __ldcg(src + m4);
            v[4 * m4] += t.x; v[4 * m4 + 1] += t.y; v[4 * m4 + 2] += t.z; v[4 * m4 + 3] += t.w;
          }
        }
        if (et == 0) p.counters[tile] = 0;  // ready for the next call on this workspace
        reduce = true;
      }
    }
    if (reduce && n < p.N) {
#pragma unroll
      for (int m = 0; m < 32; ++m)
        if (m < p.M) p.out[(size_t)m * p.N + n] = __float2bfloat16_rn(v[m]);
    }
    tc_fence_before_sync();
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0 && *failed) {
    for (int s = 0; s < kDStages; ++s) mbar_wait(&full[s], 0, 1u << 16), mbar_wait(&full[s], 1, 1u << 16);
  }
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kDTmemCols);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      f = nullptr;
    return (EncodeTiledFn)f;
  }();
  return fn;
}

bool make_map(CUtensorMap* map, const uint8_t* ptr, int rows, int Kq, int box_rows) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)(Kq / 2), (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)(Kq / 2)};
  const cuuint32_t box[2] = {128, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, (void*)ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

cudaLaunchConfig_t pdl_config(dim3 grid, dim3 block, size_t smem, cudaStream_t st, cudaLaunchAttribute* attr) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cfg;
}

cudaError_t launch_quantize(const float* Y, int R, int Kp, int Kq, int64_t ldy, uint8_t* codes, int64_t code_pitch, uint8_t* sf_blocks,
                            uint8_t* sf_rows, cudaStream_t st) {
  const long long warps = (long long)R * (Kq / 32);
  long long blocks = (warps + 7) / 8;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  cudaLaunchAttribute attr[1];
  cudaLaunchConfig_t cfg = pdl_config(dim3((unsigned)blocks), dim3(256), 0, st, attr);
  return cudaLaunchKernelEx(&cfg, mx_quantize_kernel, Y, R, Kp, Kq, (long long)ldy, codes, (long long)code_pitch, sf_blocks, sf_rows);
}

int mx_decode_splits(const xq_mx_weights* w);

cudaError_t launch_gemm_decode(const uint8_t* codes, const uint8_t* sfx, int M, const xq_mx_weights* w, void* out, uint8_t* ws,
                               size_t partial_off, cudaStream_t st) {
  CUtensorMap mapW, mapX;
  if (!make_map(&mapW, w->codes, w->Np, w->Kq, 128) || !make_map(&mapX, codes, M, w->Kq, DN)) return cudaErrorInvalidValue;
  MxDecodeParams p;
  p.sfw = w->sf;
  p.sfx = sfx;
  p.out = (__nv_bfloat16*)out;
  p.partial = (float*)(ws + partial_off);
  p.counters = (int32_t*)(ws + XQ_WS_HEADER_BYTES);
  p.status = (int32_t*)ws;
  p.M = M;
  p.N = w->N;
  p.Kq = w->Kq;
  p.KB = w->Kq / 256;
  p.S = mx_decode_splits(w);
  cudaError_t e = cudaFuncSetAttribute(gemm_mx_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDSmemBytes);
  if (e != cudaSuccess) return e;
  const int tiles = (w->N + 127) / 128;
  cudaLaunchAttribute attr[1];
  cudaLaunchConfig_t cfg = pdl_config(dim3(tiles * p.S), dim3(kThreads), kDSmemBytes, st, attr);
  return cudaLaunchKernelEx(&cfg, gemm_mx_decode_kernel, mapW, mapX, p);
}

template <int TN>
cudaError_t launch_gemm_tn(const uint8_t* codes, const uint8_t* sfa, int M, const xq_mx_weights* w, void* out, int32_t* status,
                           cudaStream_t st) {
  CUtensorMap mapA, mapB;
  if (!make_map(&mapA, codes, M, w->Kq, BM) || !make_map(&mapB, w->codes, w->Np, w->Kq, TN)) return cudaErrorInvalidValue;
  MxParams p;
  p.sfa = sfa;
  p.sfb = TN == 224 ? w->sf_wide : w->sf;
  p.out = (__nv_bfloat16*)out;
  p.status = status;
  p.M = M;
  p.N = w->N;
  p.Kq = w->Kq;
  p.KB = w->Kq / 256;
  p.tiles_m = (M + BM - 1) / BM;
  p.tiles_n = (w->N + TN - 1) / TN;
  constexpr size_t smem = TileCfg<TN>::kSmemBytes;
  cudaError_t e = cudaFuncSetAttribute(gemm_mx_kernel<TN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int tiles = p.tiles_m * p.tiles_n;
  cudaLaunchAttribute attr[1];
  cudaLaunchConfig_t cfg = pdl_config(dim3(tiles < w->sms ? tiles : w->sms), dim3(kThreads), smem, st, attr);
  return cudaLaunchKernelEx(&cfg, gemm_mx_kernel<TN>, mapA, mapB, p);
}

// codes / scale blocks of the tokens in device form -> out.  Two tile shapes; a simple cost model picks one: waves of
// tiles over the multiprocessors times the tensor-core cycles of a tile's main loop (128 per 128 x 256 x 64 MMA, scaled
// with the tile), plus the epilogue where it is not hidden behind the next tile (about 1500 cycles).
cudaError_t launch_gemm(const uint8_t* codes, const uint8_t* sfa, int M, const xq_mx_weights* w, void* out, int32_t* status,
                        cudaStream_t st) {
  const int KB = w->Kq / 256, sms = w->sms, N = w->N;
  auto waves = [&](int tiles) { return (double)((tiles + sms - 1) / sms); };
  const int tm = (M + 127) / 128;
  const double t256 = waves(tm * ((N + 255) / 256)) * (KB * 512.0 + 1500.0);
  const double t224 = waves(tm * ((N + 223) / 224)) * (KB * 448.0) + 1500.0;
  if (t224 <= t256) return launch_gemm_tn<224>(codes, sfa, M, w, out, status, st);
  return launch_gemm_tn<256>(codes, sfa, M, w, out, status, st);
}

// Workspace: header (status word) | rotated rows fp32 | codes | scale blocks | scratch outputs of the rotate kernel.
struct MxWs {
  size_t y, codes, sf, xq, sx, xstage, ostage, partial, total;
};
constexpr int kMxDecodeMaxM = DN;
// K slices of the small-batch product: every multiprocessor gets a CTA, a slice has at least one 256-code block.
int mx_decode_splits(const xq_mx_weights* w) {
  const int tiles = w->Np / 128, KB = w->Kq / 256;
  int S = w->sms / tiles;
  if (S < 1) S = 1;
  if (S > KB) S = KB;
  if (S > 3) S = 3;  // the last CTA of a tile adds S partial tiles one after the other: few, long slices
  if (KB <= kDStages + 1) S = 1;  // the whole K fits the stages requested before the tokens arrive: nothing to gain from slices
  if (tiles > (int)((XQ_WS_COUNTER_BYTES - XQ_WS_HEADER_BYTES) / 4)) S = 1;  // one counter per tile
  return S;
}
MxWs mx_ws(int M, const xq_mx_weights* w) {
  MxWs L;
  size_t off = XQ_WS_COUNTER_BYTES;
  L.y = off;
  off += align_up((size_t)M * w->Kp * 4, 256);
  L.codes = off;
  off += align_up((size_t)M * (w->Kq / 2), 256);
  L.sf = off;
  off += align_up(sf_bytes(M, w->Kq), 256);
  L.xq = off;
  off += align_up((size_t)M * (w->Kp / 2), 256);
  L.sx = off;
  off += align_up((size_t)M * 4, 256);
  L.xstage = off;  // host entry point: staged inputs and outputs
  off += align_up((size_t)M * w->K * 2, 256);
  L.ostage = off;
  off += align_up((size_t)M * w->N * 2, 256);
  L.partial = off;  // partial tiles of the split-K small-batch product
  off += (size_t)(w->Np / 128) * mx_decode_splits(w) * 128 * 32 * 4;
  L.total = off;
  return L;
}

struct DevBuf {
  void* p = nullptr;
  cudaError_t alloc(size_t bytes) { return cudaMalloc(&p, bytes ? bytes : 1); }
  ~DevBuf() {
    if (p) cudaFree(p);
  }
};

// heads > 1: K and Kp are the sizes of ONE head
xq_status make_mx_weights(int32_t N, int32_t K, int32_t Kp, xq_mx_weights** out, int32_t heads = 1) {
  if (N < 1 || K < 1 || Kp < K || heads < 1) return XQ_ERR_INVALID_ARG;
  xq_hadamard_plan_t pl;
  xq_status s = xq_hadamard_plan(K, Kp, &pl);
  if (s != XQ_OK) return s;
  if (heads > 1) {
    if (!xq_rotate_heads_supported(pl, heads)) return XQ_ERR_UNSUPPORTED_ORDER;
    K *= heads;
    Kp *= heads;
  }
  if (Kp % 32 != 0 || Kp < 128 || N % 8 != 0) return XQ_ERR_UNSUPPORTED_ORDER;  // whole groups; 16-byte output pieces
  xq_mx_weights* w = new (std::nothrow) xq_mx_weights();
  if (!w) return XQ_ERR_ALLOC;
  w->N = N;
  w->K = K;
  w->Kp = Kp;
  w->Np = (int32_t)align_up((size_t)N, 256);
  w->Kq = (int32_t)align_up((size_t)Kp, 256);
  w->plan = pl;
  w->heads = heads;
  w->head_signs = nullptr;
  w->codes = nullptr;
  w->sf = nullptr;
  w->sf_wide = nullptr;
  w->hp_signs = nullptr;
  if (cudaGetDevice(&w->device) != cudaSuccess ||
      cudaDeviceGetAttribute(&w->sms, cudaDevAttrMultiProcessorCount, w->device) != cudaSuccess) {
    delete w;
    return XQ_ERR_CUDA;
  }
  const size_t cb = (size_t)w->Np * (w->Kq / 2), sb = sf_bytes(w->Np, w->Kq);
  const size_t swb = (size_t)((N + WN - 1) / WN) * (w->Kq / 128) * 1024;
  if (cudaMalloc((void**)&w->codes, cb) != cudaSuccess || cudaMalloc((void**)&w->sf, sb) != cudaSuccess ||
      cudaMalloc((void**)&w->sf_wide, swb) != cudaSuccess || cudaMemset(w->sf_wide, 127, swb) != cudaSuccess ||
      cudaMemset(w->codes, 0, cb) != cudaSuccess || cudaMemset(w->sf, 127, sb) != cudaSuccess ||
      !(heads > 1 ? xq_make_head_signs(pl, &w->head_signs) : xq_make_hp_signs(pl, &w->hp_signs))) {
    cudaGetLastError();
    xq_mx_weights_free(w);
    return XQ_ERR_ALLOC;
  }
  *out = w;
  return XQ_OK;
}

}  // namespace

extern "C" {

void xq_mx_weights_free(xq_mx_weights* w) {
  if (!w) return;
  if (w->codes) cudaFree(w->codes);
  if (w->sf) cudaFree(w->sf);
  if (w->sf_wide) cudaFree(w->sf_wide);
  if (w->hp_signs) cudaFree(w->hp_signs);
  if (w->head_signs) cudaFree(w->head_signs);
  delete w;
}

xq_status xq_mx_weights_info(const xq_mx_weights* w, int32_t* N, int32_t* K, int32_t* Kp, xq_hadamard_plan_t* plan) {
  if (!w) return XQ_ERR_INVALID_ARG;
  if (N) *N = w->N;
  if (K) *K = w->K;
  if (Kp) *Kp = w->Kp;
  if (plan) *plan = w->plan;
  return XQ_OK;
}

}  // extern "C"

namespace {
// the fp32 rows of the online step, for the forms that have no fused quantizer
cudaError_t rotate_to_fp32(const xq_mx_weights* w, const void* X, int32_t M, int64_t ldx, uint8_t* xq_scratch, float* sx_scratch, float* Y,
                           cudaStream_t st) {
  if (w->heads > 1)
    return xq_launch_rotate_heads(X, M, ldx, w->plan, w->heads, xq_scratch, sx_scratch, Y, nullptr, w->head_signs, nullptr, w->sms, st);
  return xq_launch_rotate_quant(X, M, ldx, w->plan, xq_scratch, sx_scratch, Y, nullptr, w->hp_signs, nullptr, w->sms, st);
}

xq_status mx_prepare_impl(const void* W_host, int32_t N, int32_t heads, int32_t K, int32_t Kp, void* stream, xq_mx_weights** out) {
  if (!W_host || !out) return XQ_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  xq_mx_weights* w = nullptr;
  xq_status s = make_mx_weights(N, K, Kp, &w, heads);
  if (s != XQ_OK) return s;
  K = w->K;
  Kp = w->Kp;
  // rows of W go through the same pad + rotate kernels as token rows, in chunks of 2048 rows
  const int chunk = 2048;
  const int64_t ldw = (int64_t)align_up((size_t)K, 8);
  const int rows_max = N < chunk ? N : chunk;
  DevBuf dW, dY, dXq, dS;
  if (dW.alloc((size_t)rows_max * ldw * 2) != cudaSuccess || dY.alloc((size_t)rows_max * Kp * 4) != cudaSuccess ||
      dXq.alloc((size_t)rows_max * (Kp / 2)) != cudaSuccess || dS.alloc((size_t)rows_max * 4) != cudaSuccess) {
    cudaGetLastError();
    xq_mx_weights_free(w);
    return XQ_ERR_ALLOC;
  }
  cudaError_t e = cudaSuccess;
  for (int r0 = 0; r0 < N && e == cudaSuccess; r0 += chunk) {
    const int R = N - r0 < chunk ? N - r0 : chunk;
    e = cudaMemcpy2DAsync(dW.p, (size_t)ldw * 2, (const uint16_t*)W_host + (size_t)r0 * K, (size_t)K * 2, (size_t)K * 2, (size_t)R,
                          cudaMemcpyHostToDevice, st);
    // chunk starts are multiples of 128 rows: scale blocks of different chunks do not interleave
    uint8_t* ccodes = w->codes + (size_t)r0 * (w->Kq / 2);
    uint8_t* csf = w->sf + (size_t)(r0 / 128) * (w->Kq / 128) * 512;
    const xq_mx_out mxo = {ccodes, csf, w->Kq};
    if (e == cudaSuccess && w->heads > 1) {
      e = xq_launch_rotate_heads(dW.p, R, ldw, w->plan, w->heads, ccodes, nullptr, nullptr, nullptr, w->head_signs, nullptr, w->sms, st, &mxo);
    } else if (e == cudaSuccess && xq_rotate_mx_supported(w->plan)) {
      e = xq_launch_rotate_mx(dW.p, R, ldw, w->plan, mxo, w->sms, st);
    } else if (e == cudaSuccess) {
      e = rotate_to_fp32(w, dW.p, R, ldw, (uint8_t*)dXq.p, (float*)dS.p, (float*)dY.p, st);
      if (e == cudaSuccess) e = launch_quantize((const float*)dY.p, R, Kp, w->Kq, Kp, ccodes, w->Kq / 2, csf, nullptr, st);
    }
  }
  if (e == cudaSuccess) {
    mx_sf_to_wide_kernel<<<148 * 4, 256, 0, st>>>(w->sf, w->N, w->Kq, w->sf_wide);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) {
    cudaGetLastError();
    xq_mx_weights_free(w);
    return XQ_ERR_CUDA;
  }
  *out = w;
  return XQ_OK;
}

}  // namespace

extern "C" {

xq_status xq_mx_prepare_weights(const void* W_host, int32_t N, int32_t K, int32_t Kp, void* stream, xq_mx_weights** out) {
  XQ_RANGE();
  return mx_prepare_impl(W_host, N, 1, K, Kp, stream, out);
}

xq_status xq_mx_prepare_weights_heads(const void* W_host, int32_t N, int32_t heads, int32_t head_dim, int32_t head_dim_p, void* stream,
                                      xq_mx_weights** out) {
  XQ_RANGE();
  if (heads < 2) return XQ_ERR_INVALID_ARG;
  return mx_prepare_impl(W_host, N, heads, head_dim, head_dim_p, stream, out);
}

int32_t xq_mx_weights_heads(const xq_mx_weights* w) { return w ? w->heads : 0; }

xq_status xq_mx_weights_import(const uint8_t* codes_packed, const uint8_t* scales, int32_t N, int32_t K, int32_t Kp, void* stream,
                               xq_mx_weights** out) {
  XQ_RANGE();
  if (!codes_packed || !scales || !out) return XQ_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  xq_mx_weights* w = nullptr;
  xq_status s = make_mx_weights(N, K, Kp, &w);
  if (s != XQ_OK) return s;
  for (size_t i = 0; i < (size_t)N * (Kp / 32); ++i)
    if (scales[i] == 255) {  // the NaN scale
      xq_mx_weights_free(w);
      return XQ_ERR_INVALID_ARG;
    }
  DevBuf dC, dS;
  if (dC.alloc((size_t)N * (Kp / 2)) != cudaSuccess || dS.alloc((size_t)N * (Kp / 32)) != cudaSuccess) {
    cudaGetLastError();
    xq_mx_weights_free(w);
    return XQ_ERR_ALLOC;
  }
  cudaError_t e = cudaMemcpyAsync(dC.p, codes_packed, (size_t)N * (Kp / 2), cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(dS.p, scales, (size_t)N * (Kp / 32), cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) {
    mx_to_device_form_kernel<<<148 * 4, 256, 0, st>>>((const uint8_t*)dC.p, (const uint8_t*)dS.p, N, Kp, w->Kq, w->codes, w->sf);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) {
    mx_sf_to_wide_kernel<<<148 * 4, 256, 0, st>>>(w->sf, w->N, w->Kq, w->sf_wide);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) {
    cudaGetLastError();
    xq_mx_weights_free(w);
    return XQ_ERR_CUDA;
  }
  *out = w;
  return XQ_OK;
}

xq_status xq_mx_weights_export(const xq_mx_weights* w, uint8_t* codes, uint8_t* scales) {
  XQ_RANGE();
  if (!w || !codes || !scales || !xq_on_device(w->device)) return XQ_ERR_INVALID_ARG;
  DevBuf dC, dS;
  const size_t nc = (size_t)w->N * w->Kp, ns = (size_t)w->N * (w->Kp / 32);
  if (dC.alloc(nc) != cudaSuccess || dS.alloc(ns) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_ALLOC;
  }
  mx_from_device_form_kernel<<<148 * 4, 256>>>(w->codes, w->sf, w->N, w->Kp, w->Kq, (uint8_t*)dC.p, (uint8_t*)dS.p);
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) e = cudaMemcpy(codes, dC.p, nc, cudaMemcpyDeviceToHost);
  if (e == cudaSuccess) e = cudaMemcpy(scales, dS.p, ns, cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  return XQ_OK;
}

size_t xq_mx_workspace_bytes(int32_t M_max, const xq_mx_weights* w) {
  if (!w || M_max < 1) return 0;
  return mx_ws(M_max, w).total;
}

xq_status xq_mx_rotate_quant(const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t* plan, uint8_t* codes, uint8_t* scales,
                             float* Y, void* stream) {
  XQ_RANGE();
  if (!plan || M < 0) return XQ_ERR_INVALID_ARG;
  if (M == 0) return XQ_OK;
  if (!X || !codes || !scales || !Y) return XQ_ERR_INVALID_ARG;
  xq_hadamard_plan_t chk;
  xq_status s = xq_hadamard_plan(plan->K, plan->Kp, &chk);
  if (s != XQ_OK) return s;
  if (memcmp(&chk, plan, sizeof(chk)) != 0) return XQ_ERR_INVALID_ARG;
  if (plan->Kp % 32 != 0 || plan->Kp < 128) return XQ_ERR_UNSUPPORTED_ORDER;
  if (ldx < plan->K || (ldx % 8) != 0 || !aligned16(X) || !aligned16(codes) || !aligned16(scales) || !aligned16(Y)) return XQ_ERR_INVALID_ARG;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  cudaStream_t st = (cudaStream_t)stream;
  // The rotate kernel also emits INT4 codes and a scale per row; they land in the two output buffers (M K' / 2 bytes and, with
  // K' >= 128, at least 4 M bytes) and are overwritten by the quantizer that follows on the stream.
  if (xq_launch_rotate_quant(X, M, ldx, *plan, codes, (float*)scales, Y, nullptr, nullptr, nullptr, sms, st) != cudaSuccess ||
      launch_quantize(Y, M, plan->Kp, plan->Kp, plan->Kp, codes, plan->Kp / 2, nullptr, scales, st) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  return XQ_OK;
}

xq_status xq_mx_gemm(const uint8_t* codes, const uint8_t* scales, int32_t M, const xq_mx_weights* w, void* out, void* ws, size_t ws_bytes,
                     void* stream) {
  XQ_RANGE();
  if (!w || M < 0) return XQ_ERR_INVALID_ARG;
  if (M == 0) return XQ_OK;
  if (!codes || !scales || !out || !aligned16(codes) || !aligned16(out) || !xq_on_device(w->device)) return XQ_ERR_INVALID_ARG;
  const MxWs L = mx_ws(M, w);
  if (!ws || !aligned16(ws) || ws_bytes < L.total) return XQ_ERR_WORKSPACE;
  uint8_t* base = (uint8_t*)ws;
  cudaStream_t st = (cudaStream_t)stream;
  cudaLaunchAttribute attr[1];
  cudaLaunchConfig_t cfg = pdl_config(dim3(148 * 4), dim3(256), 0, st, attr);
  if (cudaLaunchKernelEx(&cfg, mx_to_device_form_kernel, codes, scales, (int)M, (int)w->Kp, (int)w->Kq, base + L.codes, base + L.sf) !=
          cudaSuccess ||
      (M <= kMxDecodeMaxM ? launch_gemm_decode(base + L.codes, base + L.sf, M, w, out, base, L.partial, st)
                          : launch_gemm(base + L.codes, base + L.sf, M, w, out, (int32_t*)ws, st)) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  return XQ_OK;
}

xq_status xq_mx_gemm_staged(int32_t M, const xq_mx_weights* w, void* out, void* ws, size_t ws_bytes, void* stream) {
  XQ_RANGE();
  if (!w || M < 0) return XQ_ERR_INVALID_ARG;
  if (M == 0) return XQ_OK;
  if (!out || !aligned16(out) || !xq_on_device(w->device)) return XQ_ERR_INVALID_ARG;
  const MxWs L = mx_ws(M, w);
  if (!ws || !aligned16(ws) || ws_bytes < L.total) return XQ_ERR_WORKSPACE;
  uint8_t* base = (uint8_t*)ws;
  cudaStream_t st = (cudaStream_t)stream;
  if ((M <= kMxDecodeMaxM ? launch_gemm_decode(base + L.codes, base + L.sf, M, w, out, base, L.partial, st)
                          : launch_gemm(base + L.codes, base + L.sf, M, w, out, (int32_t*)ws, st)) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  return XQ_OK;
}

xq_status xq_mx_rotate_quant_staged(const void* X, int32_t M, int64_t ldx, const xq_mx_weights* w, void* ws, size_t ws_bytes,
                                    void* stream) {
  XQ_RANGE();
  if (!w || M < 0) return XQ_ERR_INVALID_ARG;
  if (M == 0) return XQ_OK;
  if (!X || !xq_on_device(w->device)) return XQ_ERR_INVALID_ARG;
  if (ldx < w->K || (ldx % 8) != 0 || !aligned16(X)) return XQ_ERR_INVALID_ARG;
  const MxWs L = mx_ws(M, w);
  if (!ws || !aligned16(ws) || ws_bytes < L.total) return XQ_ERR_WORKSPACE;
  uint8_t* base = (uint8_t*)ws;
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = cudaErrorNotSupported;
  // one kernel: pad, rotate, group exponents, codes and scale blocks straight in the GEMM's layout
  const xq_mx_out mx = {base + L.codes, base + L.sf, w->Kq};
  if (w->heads > 1) {
    e = xq_launch_rotate_heads(X, M, ldx, w->plan, w->heads, mx.codes, nullptr, nullptr, nullptr, w->head_signs, nullptr, w->sms, st, &mx);
  } else if (M >= XQ_ROTATE_ROWS_MIN_M && xq_rotate_mx_supported(w->plan)) {
    e = xq_launch_rotate_mx(X, M, ldx, w->plan, mx, w->sms, st);
  } else if (M < XQ_ROTATE_ROWS_MIN_M) {
    e = xq_launch_rotate_tc_mx(X, M, ldx, w->plan, mx, w->hp_signs, w->sms, st);
  }
  if (e == cudaErrorNotSupported && w->heads == 1 && xq_rotate_mx_supported(w->plan)) e = xq_launch_rotate_mx(X, M, ldx, w->plan, mx, w->sms, st);
  if (e == cudaErrorNotSupported) {
    e = rotate_to_fp32(w, X, M, ldx, base + L.xq, (float*)(base + L.sx), (float*)(base + L.y), st);
    if (e == cudaSuccess)
      e = launch_quantize((const float*)(base + L.y), M, w->Kp, w->Kq, w->Kp, base + L.codes, w->Kq / 2, base + L.sf, nullptr, st);
  }
  if (e != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  return XQ_OK;
}

xq_status xq_mx_expanded_linear(const void* X, int32_t M, int64_t ldx, const xq_mx_weights* w, void* out, void* ws, size_t ws_bytes,
                                void* stream) {
  XQ_RANGE();
  if (M > 0 && (!out || !aligned16(out))) return XQ_ERR_INVALID_ARG;
  const xq_status s = xq_mx_rotate_quant_staged(X, M, ldx, w, ws, ws_bytes, stream);
  if (s != XQ_OK || M == 0) return s;
  return xq_mx_gemm_staged(M, w, out, ws, ws_bytes, stream);
}

xq_status xq_mx_expanded_linear_host(const void* X_host, int32_t M, const xq_mx_weights* w, void* out_host, void* ws, size_t ws_bytes,
                                     void* stream) {
  XQ_RANGE();
  if (!w || M < 0) return XQ_ERR_INVALID_ARG;
  if (M == 0) return XQ_OK;
  if (!X_host || !out_host || w->K % 8 != 0 || !xq_on_device(w->device)) return XQ_ERR_INVALID_ARG;
  const MxWs L = mx_ws(M, w);
  if (!ws || !aligned16(ws) || ws_bytes < L.total) return XQ_ERR_WORKSPACE;
  uint8_t* base = (uint8_t*)ws;
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = cudaMemcpyAsync(base + L.xstage, X_host, (size_t)M * w->K * 2, cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  xq_status s = xq_mx_expanded_linear(base + L.xstage, M, w->K, w, base + L.ostage, ws, ws_bytes, stream);
  if (s != XQ_OK) return s;
  e = cudaMemcpyAsync(out_host, base + L.ostage, (size_t)M * w->N * 2, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  return XQ_OK;
}

}  // extern "C"
