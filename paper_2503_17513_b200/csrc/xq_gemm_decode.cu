// Decode-shape W4A4 GEMM (M <= 32 tokens): a memory-bound split-K kernel that streams the
// packed INT4 weights once from HBM (paper Sec. 3: the quantized product Q(XR) Q(W~) computed at
// inference; here the case where the weight stream, not the arithmetic, sets the time).
//
// Work is cut into 1 KiB units (16 output channels x 128 codes, contiguous in the weight layout,
// k fastest).  Each of the <= #SM persistent CTAs takes one contiguous range of units -- so the
// HBM stream of a CTA is one linear run, fetched by a producer warp with bulk copies into a
// shared-memory ring -- and eight consumer warps turn 512-byte half units into two
// m16n8k32 integer MMAs per 8 tokens (weights as the 16-row operand, tokens as the 8 columns).
// A range that ends inside a 16-channel row block leaves a partial sum; the CTAs sharing a row
// block meet through per-CTA partial slots and an arrival counter, the last one to arrive adds
// the others' slots and runs the epilogue.  No CTA ever waits for another.
#include <cuda_bf16.h>

#include "xq_internal.h"
#include "xq_ptx.cuh"

using namespace xqptx;

namespace {

constexpr int kConsumerWarps = 16;
constexpr int kThreads = (kConsumerWarps + 1) * 32;
constexpr int kChunkBytes = 8192;       // 8 units per ring stage
constexpr int kSubPerChunk = kChunkBytes / 512;

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
  int stages, pitch_words;
  int split_units;    // 1: ranges cut at any unit (balanced bytes, partial row blocks meet through the slots);
                      // 0: ranges cut at row blocks only (no partials)
};

__device__ __forceinline__ uint64_t globaltimer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// Wait on an mbarrier phase for at most about one second; on expiry record the time-out in the
// status word and in the CTA-wide flag so that every later wait returns at once.
__device__ __forceinline__ void wait_or_flag(uint64_t* bar, uint32_t parity, volatile int* failed, int32_t* status) {
  if (*failed) return;
  uint64_t t0 = 0;
  for (uint32_t i = 0;; ++i) {
    if (mbar_try_wait(bar, parity)) return;
    if ((i & 255u) == 255u) {
      const uint64_t now = globaltimer_ns();
      if (t0 == 0) t0 = now;
      if (now - t0 > 1000000000ull || *failed) break;
    }
  }
  *failed = 1;
  atomicExch(status, (int)XQ_ERR_TIMEOUT);
}

#ifdef XQ_DECODE_TIMING
#define TSTAMP(i) do { if (blockIdx.x == XQ_DECODE_TIMING && (threadIdx.x == 0)) ((long long*)(p.status + 16))[i] = clock64(); } while (0)
#else
#define TSTAMP(i) do { } while (0)
#endif

template <int NT>  // token tiles of 8: M <= 8 * NT
__global__ void __launch_bounds__(kThreads, 1) gemm_decode_kernel(const DecodeParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = gridDim.x, cta = blockIdx.x;
  constexpr int MT = 8 * NT;        // padded token count
  constexpr int RP = MT + 2;        // pitch of the reduction scratch (ints)

  unsigned char* ring = smem;
  uint32_t* act = reinterpret_cast<uint32_t*>(ring + (size_t)p.stages * kChunkBytes);
  int* red = reinterpret_cast<int*>(act + (size_t)MT * p.pitch_words);
  uint64_t* full = reinterpret_cast<uint64_t*>(red + kConsumerWarps * 16 * RP);
  uint64_t* empty = full + p.stages;
  uint64_t* actbar = empty + p.stages;
  volatile int* flags = reinterpret_cast<volatile int*>(actbar + 1);  // [0] failed, [1] is_last

  int u0, u1;
  if (p.split_units) {
    u0 = (int)((long long)cta * p.U / G);
    u1 = (int)((long long)(cta + 1) * p.U / G);
  } else {
    const int RB = p.U / p.KB;
    u0 = (int)((long long)cta * RB / G) * p.KB;
    u1 = (int)((long long)(cta + 1) * RB / G) * p.KB;
  }
  const int sb0 = 2 * u0, sb1 = 2 * u1;  // half units (512 B) of this CTA

  TSTAMP(0);
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
  TSTAMP(1);
  pdl_launch_dependents();

  if (warp == kConsumerWarps) {
    // ---------------- producer ------------------------------------------------------------------
    // The weights are constants: their first ring-full is requested at once.  The activations
    // may come from the kernel before this one, so they wait for the grid dependency.
    const long long bytes = (long long)(u1 - u0) * XQ_BLOCK_BYTES;
    const unsigned char* src = p.W + (size_t)u0 * XQ_BLOCK_BYTES;
    const int chunks = (int)((bytes + kChunkBytes - 1) / kChunkBytes);
    auto issue = [&](int ci) {
      const int s = ci % p.stages;
      if (ci >= p.stages) wait_or_flag(&empty[s], ((ci / p.stages) - 1) & 1, flags, p.status);
      const long long off = (long long)ci * kChunkBytes;
      const uint32_t n = (uint32_t)min((long long)kChunkBytes, bytes - off);
      mbar_expect_tx(&full[s], n);
      bulk_g2s(ring + (size_t)s * kChunkBytes, src + off, n, &full[s]);
    };
    const int first = min(chunks, p.stages);
    if (lane == 0)
      for (int ci = 0; ci < first; ++ci) issue(ci);
    pdl_wait();
    const uint32_t row_bytes = (uint32_t)(p.Kp / 2);
    if (lane == 0) mbar_expect_tx(actbar, row_bytes * (uint32_t)p.M);
    __syncwarp();
    if (lane < p.M) bulk_g2s(act + (size_t)lane * p.pitch_words, p.Xq + (size_t)lane * row_bytes, row_bytes, actbar);
    if (lane == 0)
      for (int ci = first; ci < chunks; ++ci) issue(ci);
    return;
  }

  // ---------------- consumers ------------------------------------------------------------------
  pdl_wait();  // the workspace (partial slots, counters) may still be in use by the kernel before
  for (int i = tid; i < (MT - p.M) * p.pitch_words; i += kConsumerWarps * 32)
    act[(size_t)p.M * p.pitch_words + i] = 0u;  // token rows beyond M
  TSTAMP(2);
  wait_or_flag(actbar, 0, flags, p.status);
  TSTAMP(3);
  bar_sync(1, kConsumerWarps * 32);
  TSTAMP(4);

  const int g = lane >> 2, t = lane & 3;
  int cur_chunk = -1;
  const int sbs_per_rb = 2 * p.KB;

  int seg_lo = sb0;
  while (seg_lo < sb1) {
    const int rb = seg_lo / sbs_per_rb;
    const int seg_hi = min(sb1, (rb + 1) * sbs_per_rb);
    int acc[NT][4], acc2[NT][4];  // two chains per token tile: the MMA latency is long
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0;
      acc2[j][0] = acc2[j][1] = acc2[j][2] = acc2[j][3] = 0;
    }

    // this warp's half units: global index congruent to the warp number modulo the warp count
    int sb = seg_lo + ((warp - (seg_lo & (kConsumerWarps - 1))) & (kConsumerWarps - 1));
    for (; sb < seg_hi; sb += kConsumerWarps) {
      const int ci = (sb - sb0) / kSubPerChunk;
      if (ci != cur_chunk) {
        if (cur_chunk >= 0) {
          __syncwarp();
          if (lane == 0) mbar_arrive(&empty[cur_chunk % p.stages]);
        }
        wait_or_flag(&full[ci % p.stages], (ci / p.stages) & 1, flags, p.status);
        cur_chunk = ci;
      }
#ifdef XQ_DECODE_TIMING
      const int it_ = (sb - sb0) / kConsumerWarps;
      if (it_ < 6) TSTAMP(9 + 2 * it_);
#endif
      const unsigned char* src = ring + (size_t)(ci % p.stages) * kChunkBytes + (size_t)((sb - sb0) % kSubPerChunk) * 512;
      const uint4 wv = *reinterpret_cast<const uint4*>(src + lane * 16);
      uint32_t a0[4], a1[4];
      split16(wv.x, a0[0], a0[2]);  // (row g   , word t)
      split16(wv.y, a0[1], a0[3]);  // (row g+8 , word t)
      split16(wv.z, a1[0], a1[2]);  // (row g   , word t+4)
      split16(wv.w, a1[1], a1[3]);  // (row g+8 , word t+4)
      const int kg0 = (sb - rb * sbs_per_rb) * 8;  // first 8-code word of this half unit
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        const uint32_t* xr = act + (size_t)(8 * j + g) * p.pitch_words + kg0 + t;
        uint32_t b0, b1, b2, b3;
        split16(xr[0], b0, b1);
        split16(xr[4], b2, b3);
        mma_s8_16x8x32(acc[j], a0, b0, b1);
        mma_s8_16x8x32(acc2[j], a1, b2, b3);
      }
#ifdef XQ_DECODE_TIMING
      if (it_ < 6) { if (acc[0][0] == 0x7fffffff) flags[1] = 5; TSTAMP(10 + 2 * it_); }
#endif
    }

    TSTAMP(5);
    // ---- fold the eight warps' fragments, then finish or hand over the row block ---------------
    int* my = red + warp * 16 * RP;
#pragma unroll
    for (int j = 0; j < NT; ++j) {
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[j][e] += acc2[j][e];
      *reinterpret_cast<int2*>(&my[g * RP + 8 * j + 2 * t]) = make_int2(acc[j][0], acc[j][1]);
      *reinterpret_cast<int2*>(&my[(g + 8) * RP + 8 * j + 2 * t]) = make_int2(acc[j][2], acc[j][3]);
    }
    bar_sync(1, kConsumerWarps * 32);
    const bool active = tid < MT * 8;
    const int m = tid >> 3, np = tid & 7;  // token, pair of output channels
    int v0 = 0, v1 = 0;
    if (active) {
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) {
        v0 += red[w * 16 * RP + (2 * np) * RP + m];
        v1 += red[w * 16 * RP + (2 * np + 1) * RP + m];
      }
    }
    TSTAMP(6);
    const bool whole = (seg_lo == rb * sbs_per_rb) && (seg_hi == (rb + 1) * sbs_per_rb);
    bool finish = whole;
    if (!whole) {
      // contributors of this row block: CTAs c_first..c_last (c(u) = largest c with u0(c) <= u)
      const long long ua = (long long)rb * p.KB, ub = (long long)(rb + 1) * p.KB - 1;
      const int c_first = (int)(((ua + 1) * G - 1) / p.U), c_last = (int)(((ub + 1) * G - 1) / p.U);
      int32_t* slot = p.partial + ((size_t)rb + cta) * (16 * 32);
      if (active) *reinterpret_cast<int2*>(&slot[2 * tid]) = make_int2(v0, v1);
      bar_sync(1, kConsumerWarps * 32);
      if (tid == 0) {
        __threadfence();  // cumulative: publishes the whole CTA's slot (ordered by the barrier)
        const int old = atomicAdd(&p.counters[rb], 1);
        __threadfence();
        flags[1] = (old == c_last - c_first) ? 1 : 0;
      }
      bar_sync(1, kConsumerWarps * 32);
      finish = flags[1] != 0;
      if (finish) {
        if (active) {
          for (int c = c_first; c <= c_last; ++c) {
            if (c == cta) continue;
            const int2 o = __ldcg(reinterpret_cast<const int2*>(p.partial + ((size_t)rb + c) * (16 * 32) + 2 * tid));
            v0 += o.x;
            v1 += o.y;
          }
        }
        if (tid == 0) p.counters[rb] = 0;  // ready for the next launch
      }
    }
    TSTAMP(7);
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
    bar_sync(1, kConsumerWarps * 32);  // scratch and flags are reused by the next segment
    TSTAMP(8);
    seg_lo = seg_hi;
  }
}

template <int NT>
cudaError_t launch_nt(const DecodeParams& p, int grid, size_t smem, cudaStream_t st) {
  cudaError_t e = cudaFuncSetAttribute(gemm_decode_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
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
  return cudaLaunchKernelEx(&cfg, gemm_decode_kernel<NT>, p);
}

}  // namespace

// Shared-memory plan of the decode kernel for M tokens; stages == 0 means it does not fit.
static void decode_smem_plan(int M, int Kp, int* stages, int* pitch_words, size_t* bytes) {
  const int MT = M <= 8 ? 8 : (M <= 16 ? 16 : 32);
  int pitch = Kp / 8;
  pitch += ((4 - pitch) % 32 + 32) % 32;  // pitch = 4 (mod 32): conflict-free fragment reads
  const size_t act = (size_t)MT * pitch * 4;
  const size_t red = (size_t)kConsumerWarps * 16 * (MT + 2) * 4;
  const size_t fixed = act + red + 8 /*act barrier*/ + 64 /*flags*/ + 128 /*alignment slack*/;
  const size_t cap = 227 * 1024;
  int s = 0;
  if (fixed + 2 * (kChunkBytes + 16) <= cap) {
    s = (int)((cap - fixed) / (kChunkBytes + 16));
    if (s > 24) s = 24;
  }
  *stages = s;
  *pitch_words = pitch;
  *bytes = fixed + (size_t)s * (kChunkBytes + 16);
}

bool xq_decode_supported(int32_t M, const xq_weights* w) {
  if (M < 1 || M > XQ_DECODE_MAX_M || w->Kp % 128 != 0) return false;
  int s, pw;
  size_t b;
  decode_smem_plan(M, w->Kp, &s, &pw, &b);
  return s >= 2;
}

size_t xq_decode_ws_bytes(const xq_weights* w, int sms) {
  const size_t rbs = (size_t)w->Np / 16;
  return (rbs + sms) * 16 * 32 * sizeof(int32_t);
}

cudaError_t xq_launch_gemm_decode(const uint8_t* Xq, const float* sx, int32_t M, const xq_weights* w, void* out,
                                  int32_t* acc_opt, int32_t* partial, int32_t* counters, int32_t* status, int sms,
                                  cudaStream_t st) {
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
  p.split_units = 0;
  p.M = M;
  p.N = w->N;
  p.Kp = w->Kp;
  size_t smem;
  decode_smem_plan(M, w->Kp, &p.stages, &p.pitch_words, &smem);
  const int RB = w->Np / 16;
  const int grid = RB < sms ? RB : sms;
  if (M <= 8) return launch_nt<1>(p, grid, smem, st);
  if (M <= 16) return launch_nt<2>(p, grid, smem, st);
  return launch_nt<4>(p, grid, smem, st);
}
