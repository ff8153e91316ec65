// Decode-shape W4A4 GEMM (M <= 32 tokens): a memory-bound split-K kernel that streams the
// packed INT4 weights once from HBM (paper Sec. 3: the quantized product Q(XR) Q(W~) computed at
// inference; here the case where the weight stream, not the arithmetic, sets the time).
//
// Work is cut into 1 KiB units (16 output channels x 128 codes, contiguous in the weight layout,
// k fastest).  Each persistent CTA takes one contiguous range of units -- so its HBM stream is one
// linear run, fetched by a producer warp with bulk copies into a shared-memory ring of 8 KiB
// chunks, the first ring-full requested before the kernel waits for its predecessor in the
// stream.  Eight consumer warps take one unit of every chunk each: two 128-bit loads give a lane
// the codes of rows g and g+8, the nibble split turns them into the A fragments of four
// m16n8k32 integer MMAs (weights as the 16-row operand, 8 tokens as the columns).  The token
// operand is expanded once per CTA into shared memory in fragment order when it fits, else kept
// packed and split on the fly.  A warp adds its fragment into the CTA's per-row-block tile with
// shared-memory reductions whenever its unit crosses into another row block.  A row block that
// spans several CTAs is finished by the last CTA to arrive: contributors publish partial tiles in
// per-CTA slots and bump an arrival counter; nobody ever waits for another CTA.
#include <cuda_bf16.h>

#include "xq_internal.h"
#include "xq_ptx.cuh"

using namespace xqptx;

namespace {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;
constexpr int kChunkUnits = kConsumerWarps;                 // one unit per consumer warp
constexpr int kChunkBytes = kChunkUnits * XQ_BLOCK_BYTES;   // 8 KiB
constexpr int kMaxStages = 16;
constexpr int kSlotInts = 16 * 32;

struct DecodeParams {
  const uint8_t* W;
  const float* sw;
  const uint8_t* Xq;
  const float* sx;
  __nv_bfloat16* out;
  int32_t* acc_opt;
  int32_t* partial;   // [(row blocks + grid)] slots of 16 x 32 int32
  int32_t* counters;  // [row blocks], zero between launches
  int32_t* status;
  int U;              // units in total (fits 31 bits: checked on the host)
  int M, N, Kp, KB;   // KB = Kp / 128
  int stages;         // ring stages
  int act_pitch;      // bytes between token rows of the shared-memory token operand
  int max_tiles;      // row blocks a CTA's range can touch
};

template <int NT, bool PRESPLIT>  // token tiles of 8: M <= 8 * NT
__global__ void __launch_bounds__(kThreads, 1) gemm_decode_kernel(const DecodeParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = gridDim.x, cta = blockIdx.x;
  constexpr int MT = 8 * NT;   // padded token count
  constexpr int TP = MT + 8;   // pitch of a tile row (ints)

  unsigned char* ring = smem;
  unsigned char* act = ring + (size_t)p.stages * kChunkBytes;
  int* tiles = reinterpret_cast<int*>(act + (size_t)MT * p.act_pitch);
  uint64_t* full = reinterpret_cast<uint64_t*>(tiles + (size_t)p.max_tiles * 16 * TP);
  uint64_t* empty = full + p.stages;
  uint64_t* actbar = empty + p.stages;
  volatile int* flags = reinterpret_cast<volatile int*>(actbar + 1);  // [0] failed, [1] is_last

  const int u0 = (int)((long long)cta * p.U / G), u1 = (int)((long long)(cta + 1) * p.U / G);
  const int n_units = u1 - u0;
  const int rbA = u0 / p.KB;

  if (tid < p.stages) {
    mbar_init(&full[tid], 1);
    mbar_init(&empty[tid], kConsumerWarps);
  }
  if (tid == 32) {
    mbar_init(actbar, 1);
    flags[0] = 0;
    flags[1] = 0;
  }
  mbar_fence_init();
  __syncthreads();
  pdl_launch_dependents();

  if (warp == kConsumerWarps) {
    // ---------------- producer ------------------------------------------------------------------
    // The weights are constants: their first ring-full is requested at once.  The activations
    // may come from the kernel before this one, so they wait for the grid dependency.
    const long long bytes = (long long)n_units * XQ_BLOCK_BYTES;
    const unsigned char* src = p.W + (size_t)u0 * XQ_BLOCK_BYTES;
    const int chunks = (n_units + kChunkUnits - 1) / kChunkUnits;
    int s = 0;
    uint32_t wrap = 0;  // times the ring index wrapped
    auto issue = [&](int ci) -> bool {
      if (ci >= p.stages && !mbar_wait_bounded(&empty[s], (wrap - 1) & 1, flags, p.status, (int)XQ_ERR_TIMEOUT)) return false;
      const long long off = (long long)ci * kChunkBytes;
      const uint32_t n = (uint32_t)min((long long)kChunkBytes, bytes - off);
      mbar_expect_tx(&full[s], n);
      bulk_g2s(ring + (size_t)s * kChunkBytes, src + off, n, &full[s]);
      if (++s == p.stages) {
        s = 0;
        ++wrap;
      }
      return true;
    };
    const int first = min(chunks, p.stages);
    if (lane == 0)
      for (int ci = 0; ci < first; ++ci) issue(ci);
    pdl_wait();
    if (!PRESPLIT) {
      const uint32_t row_bytes = (uint32_t)(p.Kp / 2);
      if (lane == 0) mbar_expect_tx(actbar, row_bytes * (uint32_t)p.M);
      __syncwarp();
      if (lane < p.M) bulk_g2s(act + (size_t)lane * p.act_pitch, p.Xq + (size_t)lane * row_bytes, row_bytes, actbar);
    }
    if (lane == 0)
      for (int ci = first; ci < chunks; ++ci)
        if (!issue(ci)) break;
    return;
  }

  // ---------------- consumers ------------------------------------------------------------------
  for (int i = tid; i < p.max_tiles * 16 * TP; i += kConsumerThreads) tiles[i] = 0;
  if (PRESPLIT) {
    // token rows beyond M are zero
    for (int i = tid; i < (MT - p.M) * (p.act_pitch / 16); i += kConsumerThreads)
      reinterpret_cast<uint4*>(act + (size_t)p.M * p.act_pitch)[i] = make_uint4(0, 0, 0, 0);
    pdl_wait();
    // expand the packed tokens once: a 16-byte piece (words w0..w3) becomes 32 bytes
    // {even(w0), odd(w0), even(w1), odd(w1) | even(w2), odd(w2), even(w3), odd(w3)}
    const int pieces = p.Kp / 32;
    for (int m = warp; m < p.M; m += kConsumerWarps) {
      const uint4* srow = reinterpret_cast<const uint4*>(p.Xq + (size_t)m * (p.Kp / 2));
      uint4* drow = reinterpret_cast<uint4*>(act + (size_t)m * p.act_pitch);
      for (int c = lane; c < pieces; c += 32) {
        const uint4 v = __ldg(srow + c);
        uint4 lo, hi;
        split16(v.x, lo.x, lo.y);
        split16(v.y, lo.z, lo.w);
        split16(v.z, hi.x, hi.y);
        split16(v.w, hi.z, hi.w);
        drow[2 * c] = lo;
        drow[2 * c + 1] = hi;
      }
    }
  } else {
    pdl_wait();  // the workspace (partial slots, counters) may still be in use by the kernel before
    for (int i = tid; i < (MT - p.M) * (p.act_pitch / 16); i += kConsumerThreads)
      reinterpret_cast<uint4*>(act + (size_t)p.M * p.act_pitch)[i] = make_uint4(0, 0, 0, 0);
    mbar_wait_bounded(actbar, 0, flags, p.status, (int)XQ_ERR_TIMEOUT);
  }
  bar_sync(1, kConsumerThreads);

  const int g = lane >> 2, t = lane & 3;
  {
    int acc[NT][2][4];
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
      for (int c = 0; c < 2; ++c) acc[j][c][0] = acc[j][c][1] = acc[j][c][2] = acc[j][c][3] = 0;
    auto flush = [&](int tile_index) {
      int* tl = tiles + (size_t)tile_index * 16 * TP;
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        atomicAdd(&tl[g * TP + 8 * j + 2 * t], acc[j][0][0] + acc[j][1][0]);
        atomicAdd(&tl[g * TP + 8 * j + 2 * t + 1], acc[j][0][1] + acc[j][1][1]);
        atomicAdd(&tl[(g + 8) * TP + 8 * j + 2 * t], acc[j][0][2] + acc[j][1][2]);
        atomicAdd(&tl[(g + 8) * TP + 8 * j + 2 * t + 1], acc[j][0][3] + acc[j][1][3]);
#pragma unroll
        for (int c = 0; c < 2; ++c) acc[j][c][0] = acc[j][c][1] = acc[j][c][2] = acc[j][c][3] = 0;
      }
    };

    // this warp's units: local index warp, warp + 8, ...; (rb, kb) follow incrementally
    int kb = (u0 - rbA * p.KB) + warp, rb = rbA;
    while (kb >= p.KB) {
      kb -= p.KB;
      ++rb;
    }
    int cur_rb = rb, s = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int ul = warp; ul < n_units; ul += kChunkUnits) {
      if (rb != cur_rb) {
        flush(cur_rb - rbA);
        cur_rb = rb;
      }
      ok = mbar_wait_bounded(&full[s], phase, flags, p.status, (int)XQ_ERR_TIMEOUT);
      if (!ok) break;
      const unsigned char* unit = ring + (size_t)s * kChunkBytes + warp * XQ_BLOCK_BYTES;
      const uint4 w0 = *reinterpret_cast<const uint4*>(unit + g * 64 + t * 16);        // row g, codes 32t..32t+31
      const uint4 w1 = *reinterpret_cast<const uint4*>(unit + (g + 8) * 64 + t * 16);  // row g+8
      uint32_t a[4][4];
      split16(w0.x, a[0][0], a[0][2]);
      split16(w1.x, a[0][1], a[0][3]);
      split16(w0.y, a[1][0], a[1][2]);
      split16(w1.y, a[1][1], a[1][3]);
      split16(w0.z, a[2][0], a[2][2]);
      split16(w1.z, a[2][1], a[2][3]);
      split16(w0.w, a[3][0], a[3][2]);
      split16(w1.w, a[3][1], a[3][3]);
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        uint32_t b[4][2];
        if (PRESPLIT) {
          const uint4* xr = reinterpret_cast<const uint4*>(act + (size_t)(8 * j + g) * p.act_pitch + kb * 128 + t * 32);
          const uint4 x0 = xr[0], x1 = xr[1];
          b[0][0] = x0.x; b[0][1] = x0.y; b[1][0] = x0.z; b[1][1] = x0.w;
          b[2][0] = x1.x; b[2][1] = x1.y; b[3][0] = x1.z; b[3][1] = x1.w;
        } else {
          const uint4 x = *reinterpret_cast<const uint4*>(act + (size_t)(8 * j + g) * p.act_pitch + kb * 64 + t * 16);
          split16(x.x, b[0][0], b[0][1]);
          split16(x.y, b[1][0], b[1][1]);
          split16(x.z, b[2][0], b[2][1]);
          split16(x.w, b[3][0], b[3][1]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) mma_s8_16x8x32(acc[j][i & 1], a[i], b[i][0], b[i][1]);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[s]);
      if (++s == p.stages) {
        s = 0;
        phase ^= 1u;
      }
      kb += kChunkUnits;
      while (kb >= p.KB) {
        kb -= p.KB;
        ++rb;
      }
    }
    if (n_units > warp) flush(cur_rb - rbA);
  }
  bar_sync(1, kConsumerThreads);

  // ---------------- finish or hand over every row block of the range -----------------------------
  const int rbB = (u1 - 1) / p.KB;
  const bool active = tid < MT * 8;
  const int m = tid >> 3, np = tid & 7;  // token, pair of output channels
  for (int rb = rbA; rb <= rbB && n_units > 0; ++rb) {
    const int* tl = tiles + (size_t)(rb - rbA) * 16 * TP;
    int v0 = 0, v1 = 0;
    if (active) {
      v0 = tl[(2 * np) * TP + m];
      v1 = tl[(2 * np + 1) * TP + m];
    }
    const bool whole = (long long)rb * p.KB >= u0 && (long long)(rb + 1) * p.KB <= u1;
    bool finish = whole;
    if (!whole) {
      // contributors of this row block: CTAs c_first..c_last (c(u) = largest c with u0(c) <= u)
      const long long ua = (long long)rb * p.KB, ub = (long long)(rb + 1) * p.KB - 1;
      const int c_first = (int)(((ua + 1) * G - 1) / p.U), c_last = (int)(((ub + 1) * G - 1) / p.U);
      int32_t* slot = p.partial + ((size_t)rb + cta) * kSlotInts;
      if (active) *reinterpret_cast<int2*>(&slot[2 * tid]) = make_int2(v0, v1);
      bar_sync(1, kConsumerThreads);
      if (tid == 0) {
        __threadfence();  // cumulative: publishes the whole CTA's slot (ordered by the barrier)
        const int old = atomicAdd(&p.counters[rb], 1);
        __threadfence();
        flags[1] = (old == c_last - c_first) ? 1 : 0;
      }
      bar_sync(1, kConsumerThreads);
      finish = flags[1] != 0;
      if (finish) {
        if (active) {
          for (int c = c_first; c <= c_last; ++c) {
            if (c == cta) continue;
            const int2 o = __ldcg(reinterpret_cast<const int2*>(p.partial + ((size_t)rb + c) * kSlotInts + 2 * tid));
            v0 += o.x;
            v1 += o.y;
          }
        }
        if (tid == 0) p.counters[rb] = 0;  // ready for the next launch
      }
      bar_sync(1, kConsumerThreads);  // flags[1] is reused by the next partial row block
    }
    if (finish && active && m < p.M) {
      v0 >>= 8;  // every product carries 16 x 16
      v1 >>= 8;
      const int n0 = rb * 16 + 2 * np;
      const float sxm = p.sx[m];
      if (n0 < p.N) {
        const size_t o = (size_t)m * p.N + n0;
        if (p.acc_opt) p.acc_opt[o] = v0;
        const __nv_bfloat16 h0 = __float2bfloat16_rn((float)v0 * sxm * p.sw[n0]);
        if (n0 + 1 < p.N) {
          if (p.acc_opt) p.acc_opt[o + 1] = v1;
          const __nv_bfloat16 h1 = __float2bfloat16_rn((float)v1 * sxm * p.sw[n0 + 1]);
          if ((p.N & 1) == 0) {
            *reinterpret_cast<__nv_bfloat162*>(p.out + o) = __halves2bfloat162(h0, h1);
          } else {
            p.out[o] = h0;
            p.out[o + 1] = h1;
          }
        } else {
          p.out[o] = h0;
        }
      }
    }
  }
}

struct DecodePlan {
  int nt, stages, act_pitch, max_tiles, grid;
  bool presplit;
  size_t smem;
};

// Shared-memory plan for M tokens on `sms` multiprocessors; stages == 0 means it does not fit.
DecodePlan decode_plan(int M, const xq_weights* w, int sms) {
  DecodePlan d = {};
  d.nt = M <= 8 ? 1 : (M <= 16 ? 2 : 4);
  const int MT = 8 * d.nt, KB = w->Kp / 128;
  const long long U = (long long)(w->Np / 16) * KB;
  d.grid = (int)(U < sms ? U : sms);
  const long long per_cta = (U + d.grid - 1) / d.grid;
  d.max_tiles = (int)(per_cta / KB) + 2;
  const size_t tiles = (size_t)d.max_tiles * 16 * (MT + 8) * 4;
  const size_t misc = (2 * kMaxStages + 1) * 8 + 64 + 128;
  const size_t cap = 227 * 1024;
  const int want = (int)((per_cta + kChunkUnits - 1) / kChunkUnits);  // chunks of the longest range
  // row pitches that keep the 128-bit fragment reads of eight token rows on distinct banks
  const int pitch_split = w->Kp + 16, pitch_packed = w->Kp / 2 + ((w->Kp / 2) % 128 == 0 ? 64 : 0);
  const size_t act_split = (size_t)MT * pitch_split, act_packed = (size_t)MT * pitch_packed;
  const size_t min_ring = 4 * (size_t)kChunkBytes;
  d.presplit = act_split + tiles + misc + min_ring <= cap;
  const size_t actb = d.presplit ? act_split : act_packed;
  d.act_pitch = d.presplit ? pitch_split : pitch_packed;
  if (actb + tiles + misc + 2 * (size_t)kChunkBytes > cap) return d;  // stages == 0
  int s = (int)((cap - actb - tiles - misc) / kChunkBytes);
  if (s > kMaxStages) s = kMaxStages;
  if (s > want) s = want < 2 ? 2 : want;
  d.stages = s;
  d.smem = actb + tiles + misc + (size_t)s * kChunkBytes;
  return d;
}

template <int NT, bool PRESPLIT>
cudaError_t launch_nt(const DecodeParams& p, int grid, size_t smem, cudaStream_t st) {
  cudaError_t e = cudaFuncSetAttribute(gemm_decode_kernel<NT, PRESPLIT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, gemm_decode_kernel<NT, PRESPLIT>, p);
}

}  // namespace

bool xq_decode_supported(int32_t M, const xq_weights* w) {
  if (M < 1 || M > XQ_DECODE_MAX_M || w->Kp % 128 != 0) return false;
  if ((long long)(w->Np / 16) * (w->Kp / 128) > 0x7fffffffLL) return false;
  return decode_plan(M, w, w->sms).stages >= 2;
}

size_t xq_decode_ws_bytes(const xq_weights* w, int sms) {
  const size_t rbs = (size_t)w->Np / 16;
  return (rbs + sms) * kSlotInts * sizeof(int32_t);
}

cudaError_t xq_launch_gemm_decode(const uint8_t* Xq, const float* sx, int32_t M, const xq_weights* w, void* out,
                                  int32_t* acc_opt, int32_t* partial, int32_t* counters, int32_t* status, int sms,
                                  cudaStream_t st) {
  const DecodePlan d = decode_plan(M, w, sms);
  DecodeParams p;
  p.W = w->packed;
  p.sw = w->s_w;
  p.Xq = Xq;
  p.sx = sx;
  p.out = (__nv_bfloat16*)out;
  p.acc_opt = acc_opt;
  p.partial = partial;
  p.counters = counters;
  p.status = status;
  p.KB = w->Kp / 128;
  p.U = (w->Np / 16) * p.KB;
  p.M = M;
  p.N = w->N;
  p.Kp = w->Kp;
  p.stages = d.stages;
  p.act_pitch = d.act_pitch;
  p.max_tiles = d.max_tiles;
  if (d.presplit) {
    if (d.nt == 1) return launch_nt<1, true>(p, d.grid, d.smem, st);
    if (d.nt == 2) return launch_nt<2, true>(p, d.grid, d.smem, st);
    return launch_nt<4, true>(p, d.grid, d.smem, st);
  }
  if (d.nt == 1) return launch_nt<1, false>(p, d.grid, d.smem, st);
  if (d.nt == 2) return launch_nt<2, false>(p, d.grid, d.smem, st);
  return launch_nt<4, false>(p, d.grid, d.smem, st);
}
