// Prefill-shape W4A4 GEMM, second form: the expanded weights go to tensor memory, not to shared memory.
//
// The quantized product Q(XR) Q(W~) of the paper's Sec. 3 again as tcgen05.mma kind::i8, but with the operands' roles
// swapped: the WEIGHTS are the A operand (128 channels per instruction, two accumulators side by side for a tile of
// 256 channels) and the TOKENS the B operand (NT tokens, NT a multiple of 32 up to 192, chosen per launch).  A may be
// read from tensor memory, so the unpack warps expand the packed nibbles in registers and store the bytes straight
// into a staging area of tensor memory (tcgen05.st): the 32 KiB write of expanded weights per K block into shared
// memory, and the tensor core's reads of them from there, are gone.  Shared-memory traffic per K block of 128 codes
// is then 16 KiB of packed weights in, 16 KiB out to registers, NT x 128 bytes of tokens in (TMA) and twice that out
// to the tensor core: 104 KiB at NT = 192 against 792 tensor-pipe cycles, where the first form moves 192 KiB per
// 1056 cycles of a 256 x 256 tile.
//
// Tensor memory (512 columns): accumulators of channel half h in columns [h NT, (h + 1) NT) (lane = channel, column =
// token), two staging stages of 64 columns from column 384 (32 columns per channel half and stage: a K block of 128
// bytes per lane).  What bounds the main loop is the hand-over chain of a staging stage (its MMAs complete, the unpack
// warps see it, store the next K block, the issuing threads see that, issue): about 0.9 us for two stages, i.e.
// 0.42-0.44 us per K block against 0.40 us of tensor-pipe time at NT = 192.
// The accumulator is transposed with respect to the output (a thread of the epilogue owns one channel and walks the
// tokens), so the epilogue turns it round in shared memory: 32 tokens x 32 channels of bf16 per warp and stage, written
// out by one tiled TMA store each (which also clips at M and N).  Every MMA accumulates; the epilogue leaves zeros behind.
//
// Warps: weight producer (one tiled TMA copy per K block gathers the tile's 16 channel blocks), token producer (TMA),
// two MMA issuers (one per channel half), 16 epilogue (the conversion is bound by instruction latency, not by
// issue slots: twice the warps halve it), 8 unpack.  Every wait is time-bounded as in the first form.
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdlib.h>

#include "xq_internal.h"
#include "xq_ptx.cuh"

using namespace xqptx;

namespace {

constexpr int kChannels = 256;                 // channels of a tile: two instructions of 128 rows
constexpr int kMaxTokens = XQ_TS_MAX_TOKENS;   // tokens of a tile, at most
constexpr int kTokStageBytes = kMaxTokens * 128;
constexpr int kPkStageBytes = kChannels * 64;  // packed weights of a K block
constexpr int kTokStages = 4, kPkStages = 4, kAStages = 2, kDoneRing = 4;
static_assert(kDoneRing >= kTokStages && kDoneRing >= kAStages, "a waiter must reach its barrier before the ring comes round again");
constexpr int kEpiWarps = 16, kUnpackWarps = 8, kFirstEpiWarp = 4, kFirstUnpackWarp = kFirstEpiWarp + kEpiWarps;
constexpr int kThreads = (kFirstUnpackWarp + kUnpackWarps) * 32;
constexpr int kTmemCols = 512, kStagingCol = 384;
constexpr int kEpiStageBytes = 32 * 32 * 2;  // output stage of an epilogue warp: 32 tokens x 32 channels of bf16
constexpr int kEpiStages = 2;
constexpr size_t kSmemBytes = 1024 + (size_t)kTokStages * kTokStageBytes + (size_t)kPkStages * kPkStageBytes +
                              (size_t)kEpiWarps * kEpiStages * kEpiStageBytes + 512;

struct TsParams {
  const float* sw;
  const float* sx;
  const int32_t* zp;    // per-token zero points of asymmetric activation codes, or null
  const int32_t* wsum;  // per-channel sums of the weight codes
  int32_t* acc_opt;     // int32 sums for the tests, or null (the bf16 output goes through the output tensor map)
  int32_t* status;
  int M, N, KB;         // KB = K'' / 128 (K blocks of the padded weights)
  int NT;               // tokens per tile
  int tiles_m, tiles_n;
  int tn_fast;          // order of the tiles: channel tiles fastest (the CTAs of a wave share few token tiles) or token tiles fastest
};

// Tile index -> (token tile, channel tile).  The tiles that run at the same time span all of the faster index and a few
// values of the slower one; the operand indexed by the slower one is fetched from DRAM once, the other once per wave
// unless it stays in L2: the launcher lets the larger operand be the one fetched once.
__device__ __forceinline__ void tile_coords(const TsParams& p, int tile, int& tm, int& tn) {
  if (p.tn_fast) {
    tn = tile % p.tiles_n;
    tm = tile / p.tiles_n;
  } else {
    tm = tile % p.tiles_m;
    tn = tile / p.tiles_m;
  }
}

// The epilogue of one tile for the channels of (lane quarter q, channel half h), the blocks of 32 tokens with index
// parity r: wait for the accumulator, then per chunk of 16 tokens read it, leave zero behind, scale, and put the bf16
// values into a small shared-memory stage in
// output order ([token][channel], 64 bytes per token, 32 tokens), which one tiled TMA store writes out (the store
// clips at M and N); kEpiStages stages per warp take turns.  At the end the accumulator is handed back.
__device__ __forceinline__ bool epilogue_part(const TsParams& p, const CUtensorMap* mapO, unsigned char* stages, uint32_t& blk, int tile, uint32_t tcount,
                                              uint32_t tmem_base, int q, int h, int r, int lane, uint64_t* acc_full, uint64_t* acc_empty,
                                              volatile int* failed) {
  const int NT = p.NT;
  int tm, tn;
  tile_coords(p, tile, tm, tn);
  const int nw = tn * kChannels + h * 128 + q * 32;  // first channel of this warp
  const int n = nw + lane;                           // this thread's channel
  const int m0 = tm * NT;
  const bool n_ok = n < p.N, asym = p.zp != nullptr;
  const float swn = n_ok ? p.sw[n] : 0.f;
  const int wsn = (asym && n_ok) ? p.wsum[n] : 0;
  // the tile's token scales (and zero points) wait in registers, lane l of register i holding token m0 + 32 i + l:
  // nothing is fetched from global memory between reading the accumulator and storing
  float sx_r[kMaxTokens / 32];
  int zp_r[kMaxTokens / 32];
#pragma unroll
  for (int i = 0; i < kMaxTokens / 32; ++i) {
    const int ml = m0 + 32 * i + lane;
    const bool m_ok = 32 * i < NT && ml < p.M;
    sx_r[i] = m_ok ? p.sx[ml] : 0.f;
    zp_r[i] = (asym && m_ok) ? p.zp[ml] : 0;
  }
  if (!mbar_wait_bounded(acc_full, tcount & 1, failed, p.status, (int)XQ_ERR_TIMEOUT)) return false;
  tc_fence_after_sync();
  const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(h * NT);
  const int c_end = min(NT, (p.M - m0 + 31) & ~31);  // blocks below the last token hold sums of zero rows
  const uint32_t zeros[16] = {};
#pragma unroll
  for (int i = 0; i < kMaxTokens / 32; ++i) {  // blocks of 32 tokens; unrolled: the scales stay in named registers
    const int c = 32 * i;
    if ((i & 1) == r && c < c_end) {  // the two warps of a (quarter, half) take the blocks in turn
      unsigned char* stg = stages + (blk++ % kEpiStages) * kEpiStageBytes;  // the stages take turns across tiles too
      if (lane == 0) bulk_wait_group_read<kEpiStages - 1>();  // the store that read this stage kEpiStages blocks ago has done so
      __syncwarp();
      __nv_bfloat16* col = reinterpret_cast<__nv_bfloat16*>(stg) + lane;  // [token][32 channels]
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        uint32_t v[16];
        tmem_ld_32x16(taddr + c + 16 * half, v);
        tmem_ld_wait();
        tmem_st_32x16(taddr + c + 16 * half, zeros);  // left at zero for the next tile
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          int a = (int)v[j] >> 8;  // every product carries 16 x 16
          if (asym) a -= __shfl_sync(0xffffffffu, zp_r[i], 16 * half + j) * wsn;  // sum (c - z) qw = sum c qw - z sum qw
          v[j] = (uint32_t)a;
          col[32 * (16 * half + j)] = __float2bfloat16_rn((float)a * __shfl_sync(0xffffffffu, sx_r[i], 16 * half + j) * swn);
        }
        if (p.acc_opt) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int m = m0 + c + 16 * half + j;
            if (m < p.M && n_ok && XQ_IN_BOUNDS((size_t)m * p.N + n < (size_t)p.M * p.N, p.status)) p.acc_opt[(size_t)m * p.N + n] = (int)v[j];
          }
        }
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        tma_store_2d(mapO, stg, nw, m0 + c);
        bulk_commit_group();
      }
    }
  }
  tmem_st_wait();
  tc_fence_before_sync();
  __syncwarp();
  if (lane == 0) mbar_arrive(acc_empty);
  return true;
}

__global__ void __launch_bounds__(kThreads, 1) gemm_prefill_ts_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapW,
                                                                      const __grid_constant__ CUtensorMap mapO, const TsParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  unsigned char* base = smem_raw + (((raw + 1023u) & ~1023u) - raw);
  unsigned char* tok = base;                                     // kTokStages x [NT tokens x 128 bytes], 1024-aligned
  unsigned char* pk = tok + (size_t)kTokStages * kTokStageBytes;  // kPkStages x 16 KiB of packed weights
  unsigned char* epi_stages = pk + (size_t)kPkStages * kPkStageBytes;  // two output stages per epilogue warp
  uint64_t* bars = reinterpret_cast<uint64_t*>(epi_stages + (size_t)kEpiWarps * kEpiStages * kEpiStageBytes);
  uint64_t* pk_full = bars;
  uint64_t* pk_empty = pk_full + kPkStages;
  uint64_t* tok_full = pk_empty + kPkStages;
  uint64_t* mma_done = tok_full + kTokStages;  // ring of kDoneRing: the MMAs of K block `it` have completed (both issuers)
  uint64_t* a_full = mma_done + kDoneRing;
  uint64_t* acc_full = a_full + kAStages;
  uint64_t* acc_empty = acc_full + 1;
  uint64_t* drain = acc_empty + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
  volatile int* failed = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tiles = p.tiles_m * p.tiles_n, NT = p.NT;

  if (tid == 0) {
    for (int s = 0; s < kPkStages; ++s) {
      mbar_init(&pk_full[s], 1);
      mbar_init(&pk_empty[s], kUnpackWarps);
    }
    for (int s = 0; s < kTokStages; ++s) mbar_init(&tok_full[s], 1);
    for (int s = 0; s < kDoneRing; ++s) mbar_init(&mma_done[s], 2);
    for (int s = 0; s < kAStages; ++s) mbar_init(&a_full[s], kUnpackWarps);
    mbar_init(acc_full, 2);
    mbar_init(acc_empty, kEpiWarps);
    mbar_init(drain, 2);
    *failed = 0;
    mbar_fence_init();
    tma_prefetch_desc(&mapX);
    tma_prefetch_desc(&mapW);
    tma_prefetch_desc(&mapO);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // The kernel after this one is let in late (by the issuing threads, below), not here: released here, it is resident
  // and waiting (and has released its own successor in turn) while this grid still has all its tiles ahead; measured
  // inside a layer (rotate, product, rotate, ...), the early release cost 2-5 % of the step.
  // What the kernel before this one writes are the tokens and their scales (and zero points): the token producer and the
  // epilogue warps wait for it (pdl_wait) before their first access; the weights are constants, so their copies, the
  // unpack warps and the staging of the first K blocks start at once.

  if (warp == 0) {
    // ---------------- weight producer -----------------------------------------------------------
    // one tiled copy per K block: the 1 KiB pieces (16 channels x 128 codes) of the tile's 16 channel blocks, which
    // lie KB KiB apart in the weight image, land side by side in the stage
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
        int tm, tn;
        tile_coords(p, tile, tm, tn);
        for (int kb = 0; kb < p.KB; ++kb, ++it) {
          const int s = it % kPkStages;
          if (it >= (uint32_t)kPkStages) {
            ok = mbar_wait_bounded(&pk_empty[s], ((it / kPkStages) - 1) & 1, failed, p.status, (int)XQ_ERR_TIMEOUT);
            if (!ok) break;
          }
          mbar_expect_tx(&pk_full[s], (uint32_t)kPkStageBytes);
          tma_load_3d(pk + (size_t)s * kPkStageBytes, &mapW, 0, kb, tn * (kChannels / XQ_ROW_BLOCK), &pk_full[s]);
        }
      }
    }
    __syncwarp();
  } else if (warp == 1 || warp == 3) {
    // ---------------- MMA issue -----------------------------------------------------------------
    // two issuing threads, one per channel half (one thread for both needs longer per K block than the tensor pipe;
    // two per half measured no better).  The two threads' instructions are not ordered among themselves and need not
    // be: they write different accumulators; every instruction accumulates, the epilogue leaves the accumulator zeroed.
    // The completion barriers count both.
    const int h = warp == 1 ? 0 : 1;
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_s8(128, NT);
      const uint32_t d_tmem = tmem_base + (uint32_t)(h * NT);
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tcount) {
        // the epilogue has read the previous tile out of the accumulator and zeroed it (first tile: zeroed it)
        ok = mbar_wait_bounded(acc_empty, tcount & 1, failed, p.status, (int)XQ_ERR_TIMEOUT);
        if (!ok) break;
        tc_fence_after_sync();
        for (int kb = 0; kb < p.KB; ++kb, ++it) {
          const int s = it % kTokStages, u = it % kAStages;
          ok = mbar_wait_bounded(&tok_full[s], (it / kTokStages) & 1, failed, p.status, (int)XQ_ERR_TIMEOUT) &&
               mbar_wait_bounded(&a_full[u], (it / kAStages) & 1, failed, p.status, (int)XQ_ERR_TIMEOUT);
          if (!ok) break;
          tc_fence_after_sync();
          const uint64_t bdesc = umma_desc_k128(smem_u32(tok + (size_t)s * kTokStageBytes));
          const uint32_t a_tmem = tmem_base + (uint32_t)(kStagingCol + u * 64 + h * 32);
#pragma unroll
          for (int k = 0; k < 4; ++k) umma_i8_ts(d_tmem, a_tmem + 8 * k, bdesc + 2 * k, idesc, 1u);
          umma_commit(&mma_done[it % kDoneRing]);
        }
        if (ok) umma_commit(acc_full);
      }
      // every MMA issued by this thread has completed before tensor memory is released
      umma_commit(drain);
      pdl_launch_dependents();  // the next kernel's CTAs may take the SMs as this grid's CTAs leave them
    }
    __syncwarp();
    if (warp == 1) mbar_wait_bounded(drain, 0, failed, p.status, (int)XQ_ERR_TIMEOUT);
  } else if (warp == 2) {
    // ---------------- token producer ------------------------------------------------------------
    pdl_wait();
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
        int tm, tn;
        tile_coords(p, tile, tm, tn);
        for (int kb = 0; kb < p.KB; ++kb, ++it) {
          const int s = it % kTokStages;
          if (it >= (uint32_t)kTokStages) {  // the MMAs of K block it - kTokStages, which read this stage, have completed
            const uint32_t j = it - kTokStages;
            ok = mbar_wait_bounded(&mma_done[j % kDoneRing], (j / kDoneRing) & 1, failed, p.status, (int)XQ_ERR_TIMEOUT);
            if (!ok) break;
          }
          mbar_expect_tx(&tok_full[s], (uint32_t)NT * 128u);
          tma_load_2d(tok + (size_t)s * kTokStageBytes, &mapX, kb * 128, tm * NT, &tok_full[s]);
        }
      }
    }
    __syncwarp();
  } else if (warp < kFirstUnpackWarp) {
    // ---------------- epilogue ------------------------------------------------------------------
    pdl_wait();  // before the first read of a token scale; also orders this kernel's completion after its predecessor's
    const int q = warp & 3;                            // tensor-memory lane quarter this warp may read
    const int h = ((warp - kFirstEpiWarp) >> 2) & 1;   // channel half of the tile
    const int r = (warp - kFirstEpiWarp) >> 3;         // which of the blocks of 32 tokens: even or odd
    {  // the accumulator starts at zero: every MMA accumulates
      const uint32_t zeros[16] = {};
      const uint32_t taddr0 = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(h * NT);
      for (int c = 32 * r; c < NT; c += 64) {
        tmem_st_32x16(taddr0 + c, zeros);
        tmem_st_32x16(taddr0 + c + 16, zeros);
      }
      tmem_st_wait();
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty);
    }
    uint32_t tcount = 0, blk = 0;
    for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x, ++tcount)
      if (!epilogue_part(p, &mapO, epi_stages + (size_t)(warp - kFirstEpiWarp) * kEpiStages * kEpiStageBytes, blk, tile, tcount, tmem_base, q, h, r, lane,
                         acc_full, acc_empty, failed))
        break;
    if (lane == 0) bulk_wait_group<0>();  // the output stores have completed before the shared memory goes away
    __syncwarp();
  } else {
    // ---------------- unpack --------------------------------------------------------------------
    // one thread per channel of the tile: its four 16-byte pieces of the K block (32 codes each) become 32 words of
    // bytes (16 x the code; inside a word of eight codes the even positions first, as in the token image) in its
    // lane of the staging area
    const int q = warp & 3, h = (warp - kFirstUnpackWarp) >> 2;
    const int ch = h * 128 + q * 32 + lane;  // channel inside the tile
    const int piece0 = (ch >> 4) * 64 + (ch & 15);  // piece 16 t + r of channel block ch / 16
    uint32_t it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
      for (int kb = 0; kb < p.KB; ++kb, ++it) {
        const int s = it % kPkStages, u = it % kAStages;
        ok = mbar_wait_bounded(&pk_full[s], (it / kPkStages) & 1, failed, p.status, (int)XQ_ERR_TIMEOUT);
        if (!ok) break;
        const uint4* src = reinterpret_cast<const uint4*>(pk + (size_t)s * kPkStageBytes) + piece0;
        uint4 v[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) v[t] = src[16 * t];
        uint32_t r[32];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          split16(v[t].x, r[8 * t + 0], r[8 * t + 1]);
          split16(v[t].y, r[8 * t + 2], r[8 * t + 3]);
          split16(v[t].z, r[8 * t + 4], r[8 * t + 5]);
          split16(v[t].w, r[8 * t + 6], r[8 * t + 7]);
        }
        if (it >= (uint32_t)kAStages) {  // the MMAs that read this staging stage kAStages K blocks ago have completed
          const uint32_t j = it - kAStages;
          ok = mbar_wait_bounded(&mma_done[j % kDoneRing], (j / kDoneRing) & 1, failed, p.status, (int)XQ_ERR_TIMEOUT);
          if (!ok) break;
        }
        tc_fence_after_sync();
        tmem_st_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(kStagingCol + u * 64 + h * 32), r);
        tmem_st_wait();
        tc_fence_before_sync();
        __syncwarp();
        // The packed stage goes back only here, after the expanded words have been used: every lane's loads from it
        // have then certainly returned.  (Handing it back right after issuing the loads let a copy into the stage
        // overtake a load still in flight about once in 10^5 tiles: eight channels of one K block read the wrong bytes.)
        if (lane == 0) {
          mbar_arrive(&a_full[u]);
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
    for (int s = 0; s < kTokStages; ++s) mbar_wait(&tok_full[s], 0, 1u << 16), mbar_wait(&tok_full[s], 1, 1u << 16);
  }
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace

cudaError_t xq_launch_gemm_prefill_ts(const uint8_t* A8, const float* sx, const int32_t* zp, int32_t M, const xq_weights* w, void* out,
                                      int32_t* acc_opt, int32_t* status, int tile_tokens, int sms, cudaStream_t st) {
  XqEncodeTiledFn enc = xq_encode_tiled_fn();
  if (!enc) return cudaErrorNotSupported;
  if (tile_tokens < 32 || tile_tokens > kMaxTokens || (tile_tokens & 31) || (w->N & 1) || w->Np % kChannels != 0) return cudaErrorInvalidValue;
  CUtensorMap mapX;
  const cuuint64_t dims[2] = {(cuuint64_t)w->Kp, (cuuint64_t)M};
  const cuuint64_t strides[1] = {(cuuint64_t)w->Kp};
  const cuuint32_t box[2] = {128, (cuuint32_t)tile_tokens};
  const cuuint32_t estr[2] = {1, 1};
  if (enc(&mapX, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, (void*)A8, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  // the weight image as [channel block][K block][256 words]: a box of 16 channel blocks x 1 K block x 1 KiB
  CUtensorMap mapW;
  const cuuint64_t wdims[3] = {256, (cuuint64_t)(w->Kpp / XQ_K_BLOCK), (cuuint64_t)(w->Np / XQ_ROW_BLOCK)};
  const cuuint64_t wstrides[2] = {1024, (cuuint64_t)(w->Kpp / XQ_K_BLOCK) * 1024};
  const cuuint32_t wbox[3] = {256, 1, (cuuint32_t)(kChannels / XQ_ROW_BLOCK)};
  const cuuint32_t westr[3] = {1, 1, 1};
  if (enc(&mapW, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, (void*)w->packed, wdims, wstrides, wbox, westr, CU_TENSOR_MAP_INTERLEAVE_NONE,
          CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  // the output as [M][N] bf16: a box of 32 tokens x 32 channels (rows beyond M and channels beyond N are dropped)
  CUtensorMap mapO;
  const cuuint64_t odims[2] = {(cuuint64_t)w->N, (cuuint64_t)M};
  const cuuint64_t ostrides[1] = {(cuuint64_t)w->N * 2};
  const cuuint32_t obox[2] = {32, 32};
  if ((w->N & 7) || enc(&mapO, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, out, odims, ostrides, obox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  TsParams p;
  p.sw = w->s_w;
  p.sx = sx;
  p.zp = zp;
  p.wsum = w->w_sum;
  p.acc_opt = acc_opt;
  p.status = status;
  p.M = M;
  p.N = w->N;
  p.KB = w->Kpp / XQ_K_BLOCK;
  p.NT = tile_tokens;
  p.tiles_m = (M + tile_tokens - 1) / tile_tokens;
  p.tiles_n = (w->N + kChannels - 1) / kChannels;
  p.tn_fast = (size_t)M * w->Kp > (size_t)w->N * w->Kp / 2 ? 1 : 0;  // bytes of the token image against bytes of the weights
  auto kernel = gemm_prefill_ts_kernel;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  if (e != cudaSuccess) return e;
  const int tiles = p.tiles_m * p.tiles_n;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(tiles < sms ? tiles : sms);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, mapX, mapW, mapO, p);
}

