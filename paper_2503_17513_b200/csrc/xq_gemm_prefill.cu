// Prefill-shape W4A4 GEMM (many tokens): the quantized product Q(XR) Q(W~) of the paper's Sec. 3
// as a dense integer contraction on the fifth-generation tensor cores.
//
// Tile: MH x 128 tokens by 256 output channels (MH = 1 or 2), K in blocks of 128 codes.  A
// persistent CTA per SM walks its tiles with five kinds of warps:
//   weight producer (1 warp)  16 bulk copies of 1 KiB of packed weights per K block into a ring
//                             of packed stages;
//   token producer (1 warp)   TMA: the byte-per-code token tile (tensor map over the [M, K'] byte
//                             matrix, 128-byte swizzle, out-of-range rows and columns read as
//                             zero) straight into the operand stage that tcgen05.mma reads;
//   unpack   (8 warps)        expand the packed weight nibbles to signed bytes (16 x the code: the
//                             nibble moved to the top of its byte) and write them into the
//                             128-byte-swizzled K-major operand stage;
//   mma      (1 warp)         one thread issues tcgen05.mma kind::i8, 128 x 256 x 32 per
//                             instruction, int32 accumulators in tensor memory;
//   epilogue (4 MH warps)     tcgen05.ld the finished accumulator, remove the factor 256 exactly,
//                             multiply by the per-token and per-channel scales, write bf16.
// What bounds the kernel is shared-memory traffic per MMA cycle: the token operand therefore
// arrives already expanded (the rotate + quantize kernel, or a small expansion kernel, writes it
// once to global memory), and with MH = 2 one expanded weight tile feeds two accumulators.
// MH = 1 double-buffers its 256-column accumulator (the epilogue of a tile overlaps the main loop
// of the next); MH = 2 uses all 512 columns for one tile and is chosen when there are enough
// tiles for that to pay.
// Inside a word of eight codes the even positions come first after expansion (0,2,4,6,1,3,5,7);
// tokens and weights are expanded by the same rule, so the sum over K is unchanged.
// All barrier waits are time-bounded: on expiry the CTA records XQ_ERR_TIMEOUT in the workspace
// status word, every role leaves its loop, and tensor memory is released before exit.
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdlib.h>

#include <string>

#include "xq_internal.h"
#include "xq_ptx.cuh"

using namespace xqptx;

namespace {

constexpr int BMH = 128;                                     // rows of one accumulator
constexpr int kI8ABytes = BMH * 128;                         // expanded tokens: 16 KiB per 128 tokens
constexpr int kUnpackWarps = 8;
constexpr int kFirstEpiWarp = 4;
constexpr int kTmemCols = 512;

// MH accumulators of 128 tokens x BN channels per tile.  (1, 256) and (2, 128) use half of tensor memory per tile and
// double-buffer it (the epilogue of a tile overlaps the main loop of the next); (2, 256) uses all 512 columns.
template <int MH, int BN>
struct Cfg {
  static constexpr int kPkBBytes = BN * 64;    // packed weights of a K block
  static constexpr int kI8BBytes = BN * 128;   // expanded
  static constexpr int kI8StageBytes = MH * kI8ABytes + kI8BBytes;
  // stages: as many expanded ones as fit (a stage's hand-over chain -- commit, unpack wakes, expands, MMA wakes -- is
  // longer than its MMAs, so two stages leave the tensor pipe waiting); 256 x 256 has room for two only
  static constexpr int kI8Stages = kI8StageBytes <= 60 * 1024 ? 3 : 2;
  static constexpr int kPkStages = (BN == 224) ? 3 : 4;
  static constexpr int kEpiWarps = 4 * MH;
  static constexpr int kFirstUnpackWarp = kFirstEpiWarp + kEpiWarps;
  static constexpr int kThreads = (kFirstUnpackWarp + kUnpackWarps) * 32;
  static constexpr int kAccBufs = MH * BN <= 256 ? 2 : 1;
  static constexpr size_t kSmemBytes = 1024 /*alignment slack*/ + (size_t)kI8Stages * kI8StageBytes + (size_t)kPkStages * kPkBBytes +
                                       kEpiWarps * 64 * sizeof(float) /*scales, code sums of 32 channels per warp*/ + 256 /*barriers, flags*/;
};

struct PrefillParams {
  const uint8_t* W;    // block layout
  const float* sw;
  const float* sx;
  const int32_t* zp;   // per-token zero points of asymmetric activation codes, or null
  const int32_t* wsum; // per-channel sums of the weight codes
  __nv_bfloat16* out;
  int32_t* acc_opt;
  int32_t* status;
  size_t w_bytes;      // size of the weight image (read by the self checks of the debug build only)
  int M, N, KB;        // KB = K'' / 128 (k blocks of the padded weights)
  int row_blocks;      // blocks of 16 channels in the padded weights
  int tiles_m, tiles_n;
};

// Expand one 16-byte piece (32 codes of one row) and store it as two 16-byte pieces of the
// swizzled 128-byte row `r` (pieces 2j and 2j+1 before the XOR with r mod 8).
__device__ __forceinline__ void expand_store(const uint4 v, unsigned char* tile, int r, int j) {
  uint4 lo, hi;
  split16(v.x, lo.x, lo.y);
  split16(v.y, lo.z, lo.w);
  split16(v.z, hi.x, hi.y);
  split16(v.w, hi.z, hi.w);
  unsigned char* row = tile + r * 128;
  const int x = r & 7;
  *reinterpret_cast<uint4*>(row + (((2 * j) ^ x) << 4)) = lo;
  *reinterpret_cast<uint4*>(row + (((2 * j + 1) ^ x) << 4)) = hi;
}

template <int MH, int BN>
__global__ void __launch_bounds__(Cfg<MH, BN>::kThreads, 1) gemm_prefill_kernel(const __grid_constant__ CUtensorMap mapA, const PrefillParams p) {
  using C = Cfg<MH, BN>;
  constexpr int kI8Stages = C::kI8Stages, kI8StageBytes = C::kI8StageBytes, kAccBufs = C::kAccBufs, kPkBBytes = C::kPkBBytes;
  constexpr int kPkStages = C::kPkStages;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  unsigned char* base = smem_raw + (((raw + 1023u) & ~1023u) - raw);
  unsigned char* i8 = base;                                        // kI8Stages x [A (MH x 16 KiB) | B 32 KiB], 1024-aligned
  unsigned char* pk = i8 + (size_t)kI8Stages * kI8StageBytes;      // kPkStages x 16 KiB of packed weights
  float* sw_tile = reinterpret_cast<float*>(pk + (size_t)kPkStages * kPkBBytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(sw_tile + C::kEpiWarps * 64);
  uint64_t* pk_full = bars;
  uint64_t* pk_empty = pk_full + kPkStages;
  uint64_t* i8_full = pk_empty + kPkStages;
  uint64_t* i8_empty = i8_full + kI8Stages;
  uint64_t* acc_full = i8_empty + kI8Stages;
  uint64_t* acc_empty = acc_full + 2;
  uint64_t* drain = acc_empty + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
  volatile int* failed = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tiles = p.tiles_m * p.tiles_n;

  if (tid == 0) {
    for (int s = 0; s < kPkStages; ++s) {
      mbar_init(&pk_full[s], 1);
      mbar_init(&pk_empty[s], kUnpackWarps);
    }
    for (int s = 0; s < kI8Stages; ++s) {
      mbar_init(&i8_full[s], kUnpackWarps + 1);  // the unpack warps and the token producer's expect_tx
      mbar_init(&i8_empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&acc_full[b], 1);
      mbar_init(&acc_empty[b], C::kEpiWarps);
    }
    mbar_init(drain, 1);
    *failed = 0;
    mbar_fence_init();
    tma_prefetch_desc(&mapA);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // the kernel after this one is let in late (by the MMA warp, below): released here, at the start, it cost 2-5 % of a
  // layer's step (measured)
  pdl_wait();  // tokens and their scales may come from the kernel before this one

  if (warp == 0) {
    // ---------------- weight producer -----------------------------------------------------------
    uint32_t it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
      const int tn = tile / p.tiles_m;
      // lane l < BN / 16 fetches channel block l of the tile: 16 channels x 128 codes = 1 KiB contiguous; the last tile of
      // a 224-wide tiling may reach past the padded rows: those blocks are not fetched (their stage rows keep stale
      // bytes, which only feed accumulator columns the epilogue never stores)
      const int blk0 = tn * (BN / XQ_ROW_BLOCK);
      const int nblk = min(BN / XQ_ROW_BLOCK, p.row_blocks - blk0);
      const unsigned char* wsrc = p.W + ((size_t)(blk0 + (lane < nblk ? lane : 0)) * p.KB) * (4 * XQ_GROUP_BYTES);
      for (int kb = 0; kb < p.KB; ++kb, ++it) {
        const int s = it % kPkStages;
        if (it >= (uint32_t)kPkStages) {
          ok = mbar_wait_bounded(&pk_empty[s], ((it / kPkStages) - 1) & 1, failed, p.status, (int)XQ_ERR_TIMEOUT);
          if (!ok) break;
        }
        unsigned char* stage = pk + (size_t)s * kPkBBytes;
        if (lane == 0) mbar_expect_tx(&pk_full[s], (uint32_t)nblk * (4 * XQ_GROUP_BYTES));
        __syncwarp();
        if (lane < nblk) {
          const unsigned char* src = wsrc + (size_t)kb * (4 * XQ_GROUP_BYTES);
          if (XQ_IN_BOUNDS(src >= p.W && (size_t)(src - p.W) + 4 * XQ_GROUP_BYTES <= p.w_bytes && (lane + 1) * (4 * XQ_GROUP_BYTES) <= kPkBBytes, p.status))
            bulk_g2s(stage + lane * (4 * XQ_GROUP_BYTES), src, 4 * XQ_GROUP_BYTES, &pk_full[s]);
          else
            mbar_complete_tx(&pk_full[s], 4 * XQ_GROUP_BYTES);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issue -----------------------------------------------------------------
    constexpr uint32_t idesc = umma_idesc_s8(BMH, BN);
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
        const int u = it % kI8Stages;
        ok = mbar_wait_bounded(&i8_full[u], (it / kI8Stages) & 1, failed, p.status, (int)XQ_ERR_TIMEOUT);
        if (!ok) break;
        tc_fence_after_sync();
        if (lane == 0) {
          const uint32_t a_addr = smem_u32(i8 + (size_t)u * kI8StageBytes);
          const uint64_t bdesc = umma_desc_k128(a_addr + MH * kI8ABytes);
#pragma unroll
          for (int h = 0; h < MH; ++h) {
            const uint64_t adesc = umma_desc_k128(a_addr + h * kI8ABytes);
            const uint32_t d_tmem = tmem_base + (buf * MH + (uint32_t)h) * BN;
#pragma unroll
            for (int k = 0; k < 4; ++k) umma_i8_ss(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(&i8_empty[u]);
        }
        __syncwarp();
      }
      if (ok && lane == 0) umma_commit(&acc_full[buf]);
      __syncwarp();
    }
    // every MMA issued by this warp has completed before tensor memory is released
    if (lane == 0) umma_commit(drain);
    pdl_launch_dependents();
    __syncwarp();
    mbar_wait_bounded(drain, 0, failed, p.status, (int)XQ_ERR_TIMEOUT);
  } else if (warp == 2) {
    // ---------------- token producer ------------------------------------------------------------
    uint32_t it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
      const int tm = tile % p.tiles_m;
      for (int kb = 0; kb < p.KB; ++kb, ++it) {
        const int u = it % kI8Stages;
        if (it >= (uint32_t)kI8Stages) {
          ok = mbar_wait_bounded(&i8_empty[u], ((it / kI8Stages) - 1) & 1, failed, p.status, (int)XQ_ERR_TIMEOUT);
          if (!ok) break;
        }
        if (lane == 0) {
          unsigned char* stage = i8 + (size_t)u * kI8StageBytes;
          mbar_expect_tx(&i8_full[u], MH * kI8ABytes);
#pragma unroll
          for (int h = 0; h < MH; ++h) tma_load_2d(stage + h * kI8ABytes, &mapA, kb * 128, (tm * MH + h) * BMH, &i8_full[u]);
        }
        __syncwarp();
      }
    }
  } else if (warp == 3) {
    // idle: keeps the epilogue warps on tensor-memory lane quarters warp mod 4
  } else if (warp < C::kFirstUnpackWarp) {
    // ---------------- epilogue ------------------------------------------------------------------
    const int q = warp & 3;                        // tensor-memory lane quarter this warp may read
    const int eh = (warp - kFirstEpiWarp) >> 2;    // which 128-row half of the tile (MH = 2)
    // the scales and code sums of the 32 channels being stored, a private copy per warp (no cross-warp barrier); the
    // values of the next 32 travel in a register of each lane meanwhile
    float* sw_mine = sw_tile + (warp - kFirstEpiWarp) * 64;
    int* ws_mine = reinterpret_cast<int*>(sw_mine + 32);
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tcount) {
      const int tm = tile % p.tiles_m, tn = tile / p.tiles_m;
      const uint32_t buf = kAccBufs == 2 ? (tcount & 1u) : 0u;
      const uint32_t use = kAccBufs == 2 ? (tcount >> 1) : tcount;
      const int n0 = tn * BN;
      float sw_next = (n0 + lane < p.N) ? p.sw[n0 + lane] : 0.f;
      int ws_next = (p.zp && n0 + lane < p.N) ? p.wsum[n0 + lane] : 0;
      const int m = (tm * MH + eh) * BMH + q * 32 + lane;
      const float sxm = m < p.M ? p.sx[m] : 0.f;
      const int zpm = (p.zp && m < p.M) ? p.zp[m] : 0;
      ok = mbar_wait_bounded(&acc_full[buf], use & 1, failed, p.status, (int)XQ_ERR_TIMEOUT);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (buf * MH + (uint32_t)eh) * BN;
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        __syncwarp();
        sw_mine[lane] = sw_next;
        ws_mine[lane] = ws_next;
        __syncwarp();
        if (c + 1 < BN / 32) {
          const int nn = n0 + (c + 1) * 32 + lane;
          sw_next = nn < p.N ? p.sw[nn] : 0.f;
          ws_next = (p.zp && nn < p.N) ? p.wsum[nn] : 0;
        }
        uint32_t v[32];
        tmem_ld_32x32(taddr + c * 32, v);
        tmem_ld_wait();
        const int nc = n0 + c * 32;
        if (m < p.M && nc < p.N) {
          const size_t o = (size_t)m * p.N + nc;
#pragma unroll
          for (int g8 = 0; g8 < 4; ++g8) {
            if (nc + 8 * g8 < p.N &&  // N is a multiple of 8 on this path
                XQ_IN_BOUNDS(o + 8 * g8 + 8 <= (size_t)p.M * p.N && nc + 8 * g8 + 8 <= p.N, p.status)) {
              int a[8];
#pragma unroll
              for (int e = 0; e < 8; ++e)  // every product carries 16 x 16; sum (c - z) qw = sum c qw - z sum qw
                a[e] = ((int)v[8 * g8 + e] >> 8) - zpm * ws_mine[8 * g8 + e];
              if (p.acc_opt) {
                *reinterpret_cast<int4*>(p.acc_opt + o + 8 * g8) = make_int4(a[0], a[1], a[2], a[3]);
                *reinterpret_cast<int4*>(p.acc_opt + o + 8 * g8 + 4) = make_int4(a[4], a[5], a[6], a[7]);
              }
              uint32_t h[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float f0 = (float)a[2 * e] * sxm * sw_mine[8 * g8 + 2 * e];
                const float f1 = (float)a[2 * e + 1] * sxm * sw_mine[8 * g8 + 2 * e + 1];
                const __nv_bfloat162 b2 = __halves2bfloat162(__float2bfloat16_rn(f0), __float2bfloat16_rn(f1));
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
  } else {
    // ---------------- unpack --------------------------------------------------------------------
    const int ut = tid - C::kFirstUnpackWarp * 32;  // 0..255
    uint32_t it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
      for (int kb = 0; kb < p.KB; ++kb, ++it) {
        const int s = it % kPkStages, u = it % kI8Stages;
        ok = mbar_wait_bounded(&pk_full[s], (it / kPkStages) & 1, failed, p.status, (int)XQ_ERR_TIMEOUT);
        if (!ok) break;
        if (it >= (uint32_t)kI8Stages) {
          ok = mbar_wait_bounded(&i8_empty[u], ((it / kI8Stages) - 1) & 1, failed, p.status, (int)XQ_ERR_TIMEOUT);
          if (!ok) break;
        }
        // 16 channel blocks of 1 KiB, piece 16t + r of a block = codes 32t..32t+31 of channel r
        const unsigned char* src = pk + (size_t)s * kPkBBytes;
        unsigned char* dstB = i8 + (size_t)u * kI8StageBytes + MH * kI8ABytes;
        constexpr int kTotal = BN * 4;                                               // 16-byte pieces of the tile
        constexpr int kPieces = (kTotal + kUnpackWarps * 32 - 1) / (kUnpackWarps * 32);  // per thread (the last may be missing)
        uint4 v[kPieces];
#pragma unroll
        for (int i = 0; i < kPieces; ++i) {
          const int q = ut + i * kUnpackWarps * 32;
          if (kTotal % (kUnpackWarps * 32) == 0 || q < kTotal) v[i] = *reinterpret_cast<const uint4*>(src + (size_t)q * 16);
        }
#pragma unroll
        for (int i = 0; i < kPieces; ++i) {
          const int q = ut + i * kUnpackWarps * 32;
          if (kTotal % (kUnpackWarps * 32) == 0 || q < kTotal) expand_store(v[i], dstB, ((q >> 6) << 4) + (q & 15), (q >> 4) & 3);
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(&i8_full[u]);
          mbar_arrive(&pk_empty[s]);
        }
      }
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0 && *failed) {
    // bounded drain of copies that may still be landing in this CTA's shared memory
    for (int s = 0; s < kPkStages; ++s) mbar_wait(&pk_full[s], 0, 1u << 16), mbar_wait(&pk_full[s], 1, 1u << 16);
    for (int s = 0; s < kI8Stages; ++s) mbar_wait(&i8_full[s], 0, 1u << 16), mbar_wait(&i8_full[s], 1, 1u << 16);
  }
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// Packed tokens -> byte-per-code tokens in the operand order of the GEMM: a 16-byte piece (words
// w0..w3) becomes {even(w0), odd(w0), even(w1), odd(w1) | even(w2), odd(w2), even(w3), odd(w3)}.
__global__ void expand_tokens_kernel(const uint4* __restrict__ Xq, long long pieces, uint4* __restrict__ A8) {
  pdl_launch_dependents();
  pdl_wait();
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < pieces; i += (long long)gridDim.x * blockDim.x) {
    const uint4 v = Xq[i];
    uint4 lo, hi;
    split16(v.x, lo.x, lo.y);
    split16(v.y, lo.z, lo.w);
    split16(v.z, hi.x, hi.y);
    split16(v.w, hi.z, hi.w);
    A8[2 * i] = lo;
    A8[2 * i + 1] = hi;
  }
}

// Issue-rate probe of the tensor core for this kernel's MMA (measurement only): every CTA holds one operand stage
// of pseudo-random bytes in the layout the product kernel uses and one thread issues `iters` K blocks of four
// 128 x 256 x 32 kind::i8 MMAs each, alternating between two accumulators; nothing is loaded or unpacked meanwhile.
// Operations per CTA: iters * 4 * 2 * 128 * 256 * 32.
__global__ void __launch_bounds__(128, 1) i8_mma_rate_kernel(int iters, int32_t* status) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  unsigned char* base = smem_raw + (((raw + 1023u) & ~1023u) - raw);
  __shared__ uint64_t done;
  __shared__ uint32_t tmem_slot;
  __shared__ int failed;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int i = tid; i < (kI8ABytes + 256 * 128) / 4; i += blockDim.x)
    reinterpret_cast<uint32_t*>(base)[i] = (uint32_t)(i * 2654435761u + blockIdx.x * 40503u) & 0xF0F0F0F0u;
  if (tid == 0) {
    mbar_init(&done, 1);
    failed = 0;
    mbar_fence_init();
  }
  fence_proxy_async_smem();
  if (warp == 0) {
    tmem_alloc(&tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = tmem_slot;
  if (warp == 0) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_s8(BMH, 256);
      const uint32_t a_addr = smem_u32(base);
      const uint64_t adesc = umma_desc_k128(a_addr), bdesc = umma_desc_k128(a_addr + kI8ABytes);
      for (int it = 0; it < iters; ++it) {
        const uint32_t d_tmem = tmem_base + (uint32_t)(it & 1) * 256u;
#pragma unroll
        for (int k = 0; k < 4; ++k) umma_i8_ss(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (it >> 1 | k) != 0 ? 1u : 0u);
      }
      umma_commit(&done);
    }
    __syncwarp();
    mbar_wait_bounded(&done, 0, &failed, status, (int)XQ_ERR_TIMEOUT);
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
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

template <int MH, int BN>
cudaError_t launch_mh(const CUtensorMap& mapA, PrefillParams p, int sms, cudaStream_t st) {
  using C = Cfg<MH, BN>;
  p.tiles_m = (p.M + MH * BMH - 1) / (MH * BMH);
  p.tiles_n = (p.N + BN - 1) / BN;
  cudaError_t e = cudaFuncSetAttribute(gemm_prefill_kernel<MH, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::kSmemBytes);
  if (e != cudaSuccess) return e;
  const int tiles = p.tiles_m * p.tiles_n;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(tiles < sms ? tiles : sms);
  cfg.blockDim = dim3(C::kThreads);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, gemm_prefill_kernel<MH, BN>, mapA, p);
}

}  // namespace

XqEncodeTiledFn xq_encode_tiled_fn() { return (XqEncodeTiledFn)encode_tiled_fn(); }

bool xq_prefill_supported(int32_t M, const xq_weights* w) {
  return M >= 1 && w->Kp % 32 == 0 && w->N % 8 == 0 && w->Np % 256 == 0;
}

cudaError_t xq_launch_expand_tokens(const uint8_t* Xq, int32_t M, int32_t Kp, uint8_t* A8, cudaStream_t st) {
  const long long pieces = (long long)M * (Kp / 32);
  long long blocks = (pieces + 255) / 256;
  if (blocks > 148 * 8) blocks = 148 * 8;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)blocks);
  cfg.blockDim = dim3(256);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, expand_tokens_kernel, (const uint4*)Xq, pieces, (uint4*)A8);
}

// Two forms of the kernel and several tile shapes; a cost model picks one.  Costs are in units of about 1.5 ns,
// fitted to measured launches: waves of tiles over the multiprocessors times the cost of a tile.
// First form (expanded weights in shared memory): 69 units per 128 x 256 x 32 MMA; 128-token tiles expand every
// weight for half as many MMAs and run at about 0.62 of that rate; an epilogue that is not hidden costs about 2000.
// 256 tokens x 224 channels costs 7/8 of the 256 x 256 tile and exists for the wave count (14336 = 64 x 224).
// Second form (expanded weights in tensor memory, xq_gemm_prefill_ts.cu): tiles of NT tokens x 256 channels, NT in
// {192, 160, 128} or the token count rounded up to 32 when that is less; a K block costs 206 + 92 NT / 192 (the
// hand-over chain of the two staging stages bounds it, not the tensor pipe), a tile 2400 more (its epilogue is
// not hidden).  It is taken unless the best shape of the first form is clearly cheaper: measured inside a layer it is
// 5-10 % faster than the first form at the 1B and 8B prefill shapes and level with it at the smallest ones.
// Returns 0 for 128 tokens x 256 channels, 1 for 256 x 256, 2 for 256 x 128, 3 for 256 x 224 (first form), 4 for
// *ts_tokens x 256 in the second form.  XQ_PREFILL_KERNEL in the environment (read once) overrides the choice for
// measurements and tests: "ss" keeps the first form, "ts" or "ts:<tokens>" forces the second.
int xq_prefill_tile_choice(int32_t M, const xq_weights* w, int sms, int* ts_tokens) {
  static const std::string force = [] {
    const char* e = getenv("XQ_PREFILL_KERNEL");
    return std::string(e ? e : "");
  }();
  const int KB = w->Kpp / XQ_K_BLOCK, tm1 = (M + BMH - 1) / BMH, tm2 = (M + 2 * BMH - 1) / (2 * BMH);
  auto waves = [&](int tiles) { return (double)((tiles + sms - 1) / sms); };
  const int m32 = (M + 31) / 32 * 32;
  auto ts_cost = [&](int nt) { return waves(((M + nt - 1) / nt) * ((w->N + 255) / 256)) * (KB * (206.0 + 92.0 * nt / 192.0) + 2400.0); };
  int best_nt = m32 < 128 ? m32 : 128;
  double t_ts = ts_cost(best_nt);
  for (int nt = 160; nt <= XQ_TS_MAX_TOKENS && nt <= m32; nt += 32)
    if (ts_cost(nt) < t_ts) {
      t_ts = ts_cost(nt);
      best_nt = nt;
    }
  *ts_tokens = best_nt;
  if (force.rfind("ts", 0) == 0) {
    if (force.size() > 3) {
      const int nt = atoi(force.c_str() + 3) / 32 * 32;
      if (nt >= 32 && nt <= XQ_TS_MAX_TOKENS) *ts_tokens = nt < m32 ? nt : m32;
    }
    return 4;
  }
  const double t_1x256 = waves(tm1 * ((w->N + 255) / 256)) * (KB * 276.0 / 0.62);
  const double t_2x256 = waves(tm2 * ((w->N + 255) / 256)) * (KB * 552.0 + 2000.0);
  const double t_2x128 = waves(tm2 * ((w->N + 127) / 128)) * (KB * 276.0 / 0.80);  // N = 128 MMAs re-read the tokens twice as often
  const double t_2x224 = waves(tm2 * ((w->N + 223) / 224)) * (KB * 483.0 + 1750.0);
  int c = 0;
  double t_ss = t_1x256;
  if (t_2x224 < 0.97 * t_2x256 && t_2x224 < t_2x128 && t_2x224 < t_1x256) {  // only for a clear gain
    c = 3;
    t_ss = t_2x224;
  } else if (t_2x128 <= t_2x256 && t_2x128 <= t_1x256) {
    c = 2;
    t_ss = t_2x128;
  } else if (t_2x256 <= t_1x256) {
    c = 1;
    t_ss = t_2x256;
  }
  if (force != "ss" && t_ts <= 1.1 * t_ss) return 4;
  return c;
}

cudaError_t xq_launch_gemm_prefill(const uint8_t* A8, const float* sx, const int32_t* zp, int32_t M, const xq_weights* w,
                                   void* out, int32_t* acc_opt, int32_t* status, int sms, cudaStream_t st) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return cudaErrorNotSupported;
  CUtensorMap mapA;
  const cuuint64_t dims[2] = {(cuuint64_t)w->Kp, (cuuint64_t)M};
  const cuuint64_t strides[1] = {(cuuint64_t)w->Kp};
  const cuuint32_t box[2] = {128, (cuuint32_t)BMH};
  const cuuint32_t estr[2] = {1, 1};
  if (enc(&mapA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, (void*)A8, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  PrefillParams p;
  p.W = w->packed;
  p.sw = w->s_w;
  p.sx = sx;
  p.zp = zp;
  p.wsum = w->w_sum;
  p.out = (__nv_bfloat16*)out;
  p.acc_opt = acc_opt;
  p.status = status;
  p.w_bytes = (size_t)w->Np * w->Kpp / 2;
  p.M = M;
  p.N = w->N;
  p.KB = w->Kpp / XQ_K_BLOCK;
  p.row_blocks = w->Np / XQ_ROW_BLOCK;
  p.tiles_n = 0;
  p.tiles_m = 0;
  int ts_tokens = 0;
  switch (xq_prefill_tile_choice(M, w, sms, &ts_tokens)) {
    case 4: return xq_launch_gemm_prefill_ts(A8, sx, zp, M, w, out, acc_opt, status, ts_tokens, sms, st);
    case 3: return launch_mh<2, 224>(mapA, p, sms, st);
    case 2: return launch_mh<2, 128>(mapA, p, sms, st);
    case 1: return launch_mh<2, 256>(mapA, p, sms, st);
    default: return launch_mh<1, 256>(mapA, p, sms, st);
  }
}

cudaError_t xq_launch_i8_mma_rate(int iters, int32_t* status, int sms, cudaStream_t st) {
  const size_t smem = 1024 + kI8ABytes + 256 * 128;
  cudaError_t e = cudaFuncSetAttribute(i8_mma_rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  i8_mma_rate_kernel<<<sms, 128, smem, st>>>(iters, status);
  return cudaGetLastError();
}
