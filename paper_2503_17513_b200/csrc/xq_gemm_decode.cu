// Decode-shape W4A4 GEMM (M <= 32 tokens): a memory-bound split-K kernel that streams the
// packed INT4 weights once from HBM (paper Sec. 3: the quantized product Q(XR) Q(W~) computed at
// inference; here the case where the weight stream, not the arithmetic, sets the time).
//
// Decomposition.  Output channels are handled in blocks of 16; a thread-block cluster of C CTAs
// owns a contiguous range of blocks and cuts K between its CTAs in multiples of 32 codes, so a
// CTA needs only its K slice of the quantized tokens.  Inside a CTA the slice of a block is cut
// once more into S sub-slices so that there are about as many work items (block, sub-slice) as
// consumer warps; item t goes to warp t mod 16 and its partial sums stay in that warp's
// registers.  In the weight layout an item is one contiguous run of bytes; a producer warp
// fetches it in P pieces of at most 4 KiB with bulk copies into a shared-memory ring (lane l owns
// stage l), the first ring-full before the kernel waits for its predecessor in the stream.
//
// Arithmetic.  The weights are the 16-row A operand of m16n8k32 integer MMAs and eight tokens the
// B operand: shared-memory traffic per weight byte is what bounds this kernel after HBM, and this
// orientation reads the fewest token bytes.  MMA i of a chunk of four 32-code groups takes group
// i; lane (g, t) loads word t (eight codes) of channels g and g + 8 with two conflict-free 32-bit
// loads, the nibble split (16 x code in each byte) puts the even codes in K slots 4t.. and the odd
// codes in 16+4t..; the token fragments come from the token slice that the CTA expanded once into
// shared memory in exactly that order.  Block j is finished by CTA j mod C of the cluster: every
// warp stores the partial tile of its item into that CTA's shared memory (distributed shared
// memory), and after one cluster barrier the owner sums the C * S tiles and applies the epilogue
// (exact >> 8, scales, bf16, 16-byte stores).  No global scratch, no atomics, and no CTA waits on
// another outside the cluster barrier.
//
// Fused form (the whole layer in one launch, paper Sec. 3 "online": X_hat = X H_hat computed at inference, then
// the product).  The weights do not depend on the tokens, so every CTA requests its first ring-full before
// anything else; meanwhile CTA r (r < M) pads, rotates and quantizes token row r with the routine of
// xq_rotate_row.cuh (its scratch lies where the token slice and the partial tiles go later), writes the packed
// codes and the scale to the workspace and counts the row as published (release); every CTA then waits, time-bounded,
// until M rows are counted (acquire) and reads its K slice of the codes from L2.  Rotating CTAs never wait before they
// publish, so the launch makes progress whenever its first M CTAs run; a wait that runs out records
// XQ_ERR_TIMEOUT and the CTA leaves through the normal exits.  The last CTA to leave puts the two counters in the
// workspace header back to zero, so that replays of a captured launch need no host-side reset.
#include <cuda_bf16.h>

#include <mutex>

#include "xq_internal.h"
#include "xq_ptx.cuh"
#include "xq_rotate_row.cuh"

using namespace xqptx;

namespace {

constexpr int kConsumerWarps = 16;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;
constexpr int kChunkBytes = 4 * XQ_GROUP_BYTES;              // 1 KiB: 16 channels x 128 codes
constexpr int kPieceChunks = 4;                              // chunks per ring stage
constexpr int kStageBytes = kPieceChunks * kChunkBytes;      // 4 KiB
constexpr int kMaxStages = 48;

struct DecodeParams {
  const uint8_t* W;
  const float* sw;
  const uint8_t* Xq;
  const float* sx;
  __nv_bfloat16* out;
  int32_t* acc_opt;
  const int32_t* zp;    // per-token zero points of asymmetric activation codes, or null
  const int32_t* wsum;  // per-channel sums of the weight codes
  int32_t* status;
  size_t w_bytes;   // size of the weight image (read by the self checks of the debug build only)
  int M, N, Kp;
  int k_groups;     // groups of 32 codes per channel block in the weight layout (K'' / 32)
  int n_blocks;     // channel blocks holding real channels: ceil(N / 16)
  int stages;       // ring stages: 16, 32 or 48
  int act_pitch;    // bytes between token rows of the expanded token slice
  int max_blocks;   // blocks in the longest cluster range
  int log2S;        // sub-slices per block and CTA: S = 1 << log2S
  int P;            // ring pieces per work item
  int region_bytes; // token slice + partial tiles (fused form: or the rotation scratch, whichever is larger)
  // fused online step: the first M CTAs rotate and quantize the token rows into Xq / sx / zp (workspace)
  const __nv_bfloat16* X;
  long long ldx;
  xq_hadamard_plan_t plan;
  float gamma;
  const __nv_bfloat16* Hsigns;  // bf16 image of H_p^T
  uint8_t* Xq_w;
  float* sx_w;
  int32_t* zp_w;                // null: symmetric codes
  uint32_t* sync_words;         // workspace header words: [1] token rows published so far, [2] CTAs that have left
  int rot_threads;              // threads of a row group: 32 x tiles of 16 output rows x column chunks
};

// Workspace header words of the fused form: both are zero between launches (the last CTA to leave clears them).
constexpr int kRowsWord = 1, kExitWord = 2;

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void add_release_u32(uint32_t* p, uint32_t v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Rows blockIdx.x, blockIdx.x + gridDim.x, ... < M through pad + rotate + quantize by the first rot_threads threads
// of the CTA; each finished row is published by counting it (release).  `region` is this CTA's scratch.
template <int LOG2NB, int KS>
__device__ __noinline__ void fused_rotate_rows(const DecodeParams& p, unsigned char* region, int tid) {
  const xq_hadamard_plan_t& pl = p.plan;
  const int n = 1 << pl.log2n, pitch = n + 8, NB = 1 << LOG2NB, NC = n / NB;
  const int P16 = (pl.p + 15) / 16 * 16, hpitch = P16 + 8;
  const int nthreads = p.rot_threads, warp = tid >> 5, lane = tid & 31, mt = warp / NC;
  const xqrot::RowLayout L = xqrot::row_layout(pl);
  __nv_bfloat16* Xs = reinterpret_cast<__nv_bfloat16*>(region + L.xs);
  __nv_bfloat16* Hs = reinterpret_cast<__nv_bfloat16*>(region + L.hs);
  const xqrot::RowSmem sm = {Xs, reinterpret_cast<uint32_t*>(region + L.outp), nullptr, reinterpret_cast<float*>(region + L.red),
                             reinterpret_cast<float*>(region + L.exch)};
  const xqrot::NamedSync sync = {2, nthreads};
  // constants of the plan first: nothing here depends on the preceding kernel
  for (int i = tid; i < P16 * hpitch / 8; i += nthreads) cp_async16(Hs + 8 * i, p.Hsigns + 8 * i);
  for (int i = tid; i < KS * 16 * pitch / 8; i += nthreads) reinterpret_cast<uint4*>(Xs)[i] = make_uint4(0, 0, 0, 0);
  cp_async_wait_all();
  sync();
  uint32_t afrag[KS][4];
  xqrot::load_afrag<KS>(afrag, Hs, P16, hpitch, mt, lane);
  pdl_wait();
  const xqrot::RowOut out = {p.Xq_w, p.sx_w, nullptr, nullptr, p.zp_w, nullptr, 0};
  const int chunks = pl.K / 8;
  for (int row = blockIdx.x; row < p.M; row += gridDim.x) {
    const __nv_bfloat16* x = p.X + (long long)row * p.ldx;
    for (int i = tid; i < chunks; i += nthreads) {
      const int c = 8 * i, a = c >> pl.log2n, b = c & (n - 1);
      cp_async16(Xs + a * pitch + b, x + c);
    }
    cp_async_wait_all();
    sync();
    xqrot::rotate_row<LOG2NB, KS>(pl, p.gamma, afrag, sm, out, row, tid, nthreads, sync);
    // rotate_row ends with the group's barrier: every thread's stores of the row precede it
    if (tid == 0) add_release_u32(p.sync_words + kRowsWord, 1u);
  }
}

__device__ __forceinline__ void fused_rotate_dispatch(const DecodeParams& p, unsigned char* region, int tid) {
  const int n = 1 << p.plan.log2n, ks = ((p.plan.K + n - 1) / n + 15) / 16;
  if (p.plan.log2n == 5) {
    if (ks == 1) fused_rotate_rows<5, 1>(p, region, tid);
    else if (ks == 2) fused_rotate_rows<5, 2>(p, region, tid);
    else if (ks == 3) fused_rotate_rows<5, 3>(p, region, tid);
    else fused_rotate_rows<5, 4>(p, region, tid);
  } else {  // chunks of 64 columns
    if (ks == 1) fused_rotate_rows<6, 1>(p, region, tid);
    else if (ks == 2) fused_rotate_rows<6, 2>(p, region, tid);
    else if (ks == 3) fused_rotate_rows<6, 3>(p, region, tid);
    else fused_rotate_rows<6, 4>(p, region, tid);
  }
}

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_acquire() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// 8 bytes into the shared memory of CTA `rank` of the cluster, at the address that `local_ptr`
// has in this CTA.
__device__ __forceinline__ void st_cluster_v2(void* local_ptr, uint32_t rank, int2 v) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(local_ptr)), "r"(rank));
  asm volatile("st.shared::cluster.v2.s32 [%0], {%1, %2};" ::"r"(remote), "r"(v.x), "r"(v.y) : "memory");
}

template <int NT, int C, bool FUSED>  // NT token tiles of 8 (M <= 8 NT), clusters of C CTAs; FUSED: rotate + quantize inside
__global__ void __launch_bounds__(kThreads, 1) gemm_decode_kernel(const DecodeParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int MT = 8 * NT;  // padded token count
  const int rank = C == 1 ? 0 : (int)cluster_ctarank();
  const int cid = blockIdx.x / C, n_clusters = gridDim.x / C;

  unsigned char* ring = smem;
  unsigned char* act = ring + (size_t)p.stages * kStageBytes;
  // partial tiles of the blocks this CTA finishes: [owned block][source CTA, sub-slice][16 channels][MT tokens]
  const int S = 1 << p.log2S, srcs = C * S;
  int* tiles = reinterpret_cast<int*>(act + (size_t)MT * p.act_pitch);
  uint64_t* full = reinterpret_cast<uint64_t*>(act + p.region_bytes);
  uint64_t* empty = full + p.stages;
  volatile int* failed = reinterpret_cast<volatile int*>(empty + p.stages);

  // this cluster's channel blocks and this CTA's K slice (in groups of 32 codes)
  const int b0 = (int)((long long)cid * p.n_blocks / n_clusters), b1 = (int)((long long)(cid + 1) * p.n_blocks / n_clusters);
  const int n_blk = b1 - b0;
  const int groups = p.Kp / XQ_K_GROUP;
  const int g0 = rank * groups / C, g1 = (rank + 1) * groups / C;
  const int L = g1 - g0;               // groups in the slice
  const int n_chunks = (L + 3) >> 2;   // chunks of four groups
  const int n_items = n_blk << p.log2S, parts = p.P;
  const int rounds = (n_items + kConsumerWarps - 1) / kConsumerWarps;
  // item t = (block t >> log2S, sub-slice u = t & (S - 1)) covers chunks [u n_chunks / S, (u + 1) n_chunks / S);
  // its piece q covers chunks [lo + q len / P, lo + (q + 1) len / P)
  auto piece_range = [&](int u, int q, int& c_lo, int& c_hi) {
    const int lo = (u * n_chunks) >> p.log2S, len = (((u + 1) * n_chunks) >> p.log2S) - lo;
    if (parts == 1) {
      c_lo = lo;
      c_hi = lo + len;
    } else {
      c_lo = lo + q * len / parts;
      c_hi = lo + (q + 1) * len / parts;
    }
  };

  if (tid < p.stages) {
    mbar_init(&full[tid], 1);
    mbar_init(&empty[tid], 1);
    mbar_fence_init();  // only the initialising threads: a cluster-scope fence in every thread is costly
  }
  if (tid == 64) asm volatile("prefetch.global.L2 [%0];" ::"l"(p.sx));
  if (tid == 65) *failed = 0;
  __syncthreads();
  if (C > 1) cluster_arrive_relaxed();  // "this CTA runs": awaited before the first remote store
  pdl_launch_dependents();

  if (warp == kConsumerWarps) {
    // ---------------- producer ------------------------------------------------------------------
    // Warp w's n-th piece (n = round * P + part) goes to ring stage w + 16 (n mod slots), slots =
    // stages / 16.  Every stage is served by one lane, which issues that stage's pieces in order
    // and so sees every phase of its "empty" barrier in turn (a one-bit parity cannot tell phase
    // n from phase n + 2).  The lanes poll together with the
    // non-blocking probe: a lane suspended inside a blocking wait would hold up the lanes whose
    // stages are already free.  The weights are constants: nothing here waits for the preceding
    // kernel.
    // Lane l serves the stages l and (with 48 stages) l + 32, one after the other in piece order.
    const int w = lane & (kConsumerWarps - 1);
    const int per_round = p.stages / kConsumerWarps;   // ring slots per warp: 1, 2 or 3
    // this lane's k-th piece has slot index n(k) in its warp's sequence of (round, part) pairs:
    // slots with n mod per_round == lane / 16 (and == 2 for lanes 0..15 when per_round == 3)
    int n = lane >> 4;                                 // index into the warp's piece sequence
    uint32_t use_a = 0, use_b = 0;                     // fills so far of stage lane and stage lane + 32
    bool active = (lane >> 4) < per_round;
    const int total_n = rounds * parts;                // pieces of one warp, counting missing items
    auto exists = [&](int nn) { return nn < total_n && (nn / parts) * kConsumerWarps + w < n_items; };
    auto next_n = [&](int nn) {                        // the next slot this lane serves after nn
      if (per_round == 3 && lane < 16) return (nn % 3 == 0) ? nn + 2 : nn + 1;  // residues 0 and 2
      if (per_round == 3) return nn + 3;                                         // residue 1
      return nn + per_round;
    };
    if (active && !exists(n)) active = false;
    uint32_t idle = 0;
    uint64_t t_idle = 0;
    const uint64_t stream_policy = l2_policy_evict_first();  // the weights pass once: keep L2 for the tokens and scales
    while (__any_sync(0xffffffffu, active)) {
      bool ready = false;
      int stage = 0;
      if (active) {
        const bool second = (per_round == 3 && lane < 16 && n % 3 == 2);
        stage = second ? lane + 32 : lane;
        const uint32_t use = second ? use_b : use_a;
        ready = use == 0 || mbar_test(&empty[stage], (use - 1) & 1);
      }
      if (ready) {
        const int r = n / parts, q = n - r * parts;
        const int t = r * kConsumerWarps + w;
        int c_lo, c_hi;
        piece_range(t & (S - 1), q, c_lo, c_hi);
        const int ng = min(4 * c_hi, L) - 4 * c_lo;
        const uint32_t bytes = (uint32_t)ng * XQ_GROUP_BYTES;
        const unsigned char* src = p.W + ((size_t)(b0 + (t >> p.log2S)) * p.k_groups + g0 + 4 * c_lo) * XQ_GROUP_BYTES;
        mbar_expect_tx(&full[stage], bytes);
        if (XQ_IN_BOUNDS(ng > 0 && bytes <= (uint32_t)kStageBytes && stage < p.stages && src >= p.W && (size_t)(src - p.W) + bytes <= p.w_bytes,
                         p.status))
          bulk_g2s_hint(ring + (size_t)stage * kStageBytes, src, bytes, &full[stage], stream_policy);
        else
          mbar_complete_tx(&full[stage], bytes);
        if (stage == lane) ++use_a; else ++use_b;
        n = next_n(n);
        if (!exists(n)) active = false;
      }
      if (__any_sync(0xffffffffu, ready)) {
        idle = 0;
      } else {
        __nanosleep(40);
        if ((++idle & 255u) == 0u) {  // nothing moved for a while: bounded, like every other wait
          const uint64_t now = globaltimer_ns();
          if (idle == 256u) t_idle = now;
          if (*failed || now - t_idle > 1000000000ull) {
            if (lane == 0 && !*failed) {
              *failed = 1;
              atomicExch(p.status, (int)XQ_ERR_TIMEOUT);
            }
            break;
          }
        }
      }
    }
    __syncwarp();
    if (C > 1) cluster_wait_acquire();
  } else {
    // ---------------- consumers ----------------------------------------------------------------
    // the epilogue's channel scales: bring them into L2 now, they are constants
    for (int i = tid * 32; i < n_blk * 16; i += kConsumerThreads * 32)
      if (b0 * 16 + i < p.N) asm volatile("prefetch.global.L2 [%0];" ::"l"(p.sw + b0 * 16 + i));
    bool ok = true;
    if (FUSED) {
      // the online step of the layer, inside this launch: this CTA's token rows (if it has any), then the flags of all
      if (blockIdx.x < p.M && tid < p.rot_threads) fused_rotate_dispatch(p, act, tid);
      else pdl_wait();
      bar_sync(1, kConsumerThreads);  // the scratch of the rotation is free: the token slice goes there
      if (warp == 0) {
        // one lane per CTA watches the count of published rows, with a pause between looks: the word sits in one L2
        // slice that every weight stream also crosses
        bool seen = true;
        if (lane == 0) {
          uint64_t t0 = 0;
          for (uint32_t i = 1; ld_acquire_u32(p.sync_words + kRowsWord) < (uint32_t)p.M; ++i) {
            __nanosleep(100);
            if ((i & 31u) == 0u) {
              const uint64_t now = globaltimer_ns();
              if (t0 == 0) t0 = now;
              if (*failed || now - t0 > 1000000000ull) {
                seen = false;
                break;
              }
            }
          }
          if (!seen) {
            *failed = 1;
            atomicExch(p.status, (int)XQ_ERR_TIMEOUT);
          }
        }
        __syncwarp();
      }
    }
    // token rows beyond M are zero
    for (int i = tid; i < (MT - p.M) * (p.act_pitch / 16); i += kConsumerThreads)
      reinterpret_cast<uint4*>(act + (size_t)p.M * p.act_pitch)[i] = make_uint4(0, 0, 0, 0);
    if (FUSED) {
      bar_sync(1, kConsumerThreads);
      ok = !*failed;
    } else {
      pdl_wait();
    }
    // Expand this CTA's K slice of the packed tokens once, in fragment order: chunk c of four
    // groups takes 128 bytes per token, word t of group i (even codes, odd codes) at
    // c * 128 + t * 32 + i * 8.
    if (ok) {
      const int total = p.M * L;
      constexpr int kBatch = 6;
      for (int base = tid; base < total; base += kBatch * kConsumerThreads) {
        uint4 v[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
          const int i = base + u * kConsumerThreads;
          if (i < total) {
            const int m = i / L, l = i - m * L;
            const uint4* src = reinterpret_cast<const uint4*>(p.Xq + (size_t)m * (p.Kp / 2)) + g0 + l;
            v[u] = FUSED ? __ldcg(src) : __ldg(src);  // fused: written by other CTAs of this launch, read from L2
          }
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
          const int i = base + u * kConsumerThreads;
          if (i < total) {
            const int m = i / L, l = i - m * L;
            unsigned char* d = act + (size_t)m * p.act_pitch + (size_t)(l >> 2) * 128 + (size_t)(l & 3) * 8;
            if (!XQ_IN_BOUNDS(m < MT && (size_t)(l >> 2) * 128 + (size_t)(l & 3) * 8 + 104 <= (size_t)p.act_pitch, p.status)) continue;
            uint2 e;
            split16(v[u].x, e.x, e.y);
            *reinterpret_cast<uint2*>(d) = e;
            split16(v[u].y, e.x, e.y);
            *reinterpret_cast<uint2*>(d + 32) = e;
            split16(v[u].z, e.x, e.y);
            *reinterpret_cast<uint2*>(d + 64) = e;
            split16(v[u].w, e.x, e.y);
            *reinterpret_cast<uint2*>(d + 96) = e;
          }
        }
      }
    }
    bar_sync(1, kConsumerThreads);
    if (C > 1) cluster_wait_acquire();  // every CTA of the cluster has started: remote stores are legal

    const int ag = lane >> 2, at = lane & 3;  // MMA fragment coordinates: channel row / token column, word
    for (int r = 0; r < rounds && ok; ++r) {
      const int t = r * kConsumerWarps + warp;
      if (t >= n_items) break;
      const int j = t >> p.log2S, u = t & (S - 1);
      int acc[NT][4][4];  // one chain per MMA of a chunk: the integer MMA has a long latency
#pragma unroll
      for (int a = 0; a < NT; ++a)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[a][c][0] = acc[a][c][1] = acc[a][c][2] = acc[a][c][3] = 0;
      for (int q = 0; q < parts && ok; ++q) {
        // this warp's n-th piece sits in ring stage warp + 16 (n mod slots), in its (n / slots)-th use
        const int n = r * parts + q, per_round = p.stages / kConsumerWarps;
        const int s = warp + kConsumerWarps * (n % per_round);
        ok = mbar_wait_bounded(&full[s], (n / per_round) & 1, failed, p.status, (int)XQ_ERR_TIMEOUT);
        if (!ok) break;
        int c_lo, c_hi;
        piece_range(u, q, c_lo, c_hi);
        const int ng = min(4 * c_hi, L) - 4 * c_lo;
        const unsigned char* wp = ring + (size_t)s * kStageBytes + lane * 4;  // channel ag (and ag + 8 at +128), word at
        const unsigned char* ap = act + (size_t)ag * p.act_pitch + (size_t)c_lo * 128 + (size_t)at * 32;
#pragma unroll 1
        for (int gq = 0; gq < ng; gq += 4, wp += kChunkBytes, ap += 128) {
          const int nv = min(4, ng - gq);  // groups of this chunk that exist
          uint32_t a[4][4];
#pragma unroll
          for (int i4 = 0; i4 < 4; ++i4) {
            uint32_t lo = 0u, hi = 0u;
            if (i4 < nv) {
              lo = *reinterpret_cast<const uint32_t*>(wp + i4 * XQ_GROUP_BYTES);
              hi = *reinterpret_cast<const uint32_t*>(wp + i4 * XQ_GROUP_BYTES + 128);
            }
            split16(lo, a[i4][0], a[i4][2]);  // channel ag: even codes -> K slots 4 at.., odd -> 16 + 4 at..
            split16(hi, a[i4][1], a[i4][3]);  // channel ag + 8
          }
#pragma unroll
          for (int n = 0; n < NT; ++n) {
            const uint4* xp = reinterpret_cast<const uint4*>(ap + (size_t)(8 * n) * p.act_pitch);
            const uint4 x0 = xp[0], x1 = xp[1];  // token 8 n + ag: (even, odd) of word at of groups 0..3
            mma_s8_16x8x32(acc[n][0], a[0], x0.x, x0.y);
            mma_s8_16x8x32(acc[n][1], a[1], x0.z, x0.w);
            mma_s8_16x8x32(acc[n][2], a[2], x1.x, x1.y);
            mma_s8_16x8x32(acc[n][3], a[3], x1.z, x1.w);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[s]);
      }
      // D fragment: (channel ag, tokens 2 at, 2 at + 1), (channel ag + 8, same tokens) -> the
      // tile [j / C][rank * S + u] in the shared memory of CTA j mod C
      const int owner = j % C;
      int* tl = tiles + ((size_t)(j / C) * srcs + rank * S + u) * 16 * MT;
#pragma unroll
      for (int n = 0; n < NT; ++n) {
        const int2 v0 = make_int2(acc[n][0][0] + acc[n][1][0] + acc[n][2][0] + acc[n][3][0], acc[n][0][1] + acc[n][1][1] + acc[n][2][1] + acc[n][3][1]);
        const int2 v1 = make_int2(acc[n][0][2] + acc[n][1][2] + acc[n][2][2] + acc[n][3][2], acc[n][0][3] + acc[n][1][3] + acc[n][2][3] + acc[n][3][3]);
        int* d0 = &tl[ag * MT + 8 * n + 2 * at];
        int* d1 = &tl[(ag + 8) * MT + 8 * n + 2 * at];
        // the tile lies inside the partial-tile area of its owner (every CTA of the cluster has the same layout)
        if (!XQ_IN_BOUNDS(tl >= tiles && (size_t)(tl - tiles + 16 * MT) * sizeof(int) + (size_t)MT * p.act_pitch <= (size_t)p.region_bytes, p.status))
          continue;
        if (owner == rank) {
          *reinterpret_cast<int2*>(d0) = v0;
          *reinterpret_cast<int2*>(d1) = v1;
        } else {
          st_cluster_v2(d0, (uint32_t)owner, v0);
          st_cluster_v2(d1, (uint32_t)owner, v1);
        }
      }
    }
  }

  // ---------------- meet the other K slices and finish ------------------------------------------
  // this CTA finishes blocks j = rank, rank + C, ...: one thread per (block, token, half of the channels);
  // the scales of a thread's first output are fetched while the cluster barrier completes
  const int mine = (n_blk - rank + C - 1) / C;
  if (C > 1) cluster_arrive_release();
  float e_sx = 0.f;
  int e_z = 0;
  float4 e_s0 = make_float4(0.f, 0.f, 0.f, 0.f), e_s1 = e_s0;
  if (warp < kConsumerWarps && tid < mine * p.M * 2) {
    const int h = tid & 1, bm = tid >> 1, jj = bm / p.M, m = bm - jj * p.M;
    const int n0 = (b0 + rank + jj * C) * 16 + 8 * h;
    e_sx = FUSED ? __ldcg(p.sx + m) : p.sx[m];
    if (p.zp) e_z = FUSED ? __ldcg(p.zp + m) : p.zp[m];
    if (n0 + 8 <= p.N && (p.N & 7) == 0) {
      e_s0 = *reinterpret_cast<const float4*>(p.sw + n0);
      e_s1 = *reinterpret_cast<const float4*>(p.sw + n0 + 4);
    }
  }
  if (C > 1) cluster_wait_acquire();
  else __syncthreads();
  if (warp < kConsumerWarps && !*failed) {
    for (int idx = tid; idx < mine * p.M * 2; idx += kConsumerThreads) {
      const int h = idx & 1, bm = idx >> 1;
      const int jj = bm / p.M, m = bm - jj * p.M;
      const int j = rank + jj * C;
      const int n0 = (b0 + j) * 16 + 8 * h;
      const bool pre = idx == tid;  // scales already in registers
      int z = 0;
      int4 w0 = make_int4(0, 0, 0, 0), w1 = w0;
      if (p.zp) {  // issued ahead of the tile reads (w_sum covers the padded rows)
        z = pre ? e_z : (FUSED ? __ldcg(p.zp + m) : p.zp[m]);
        w0 = *reinterpret_cast<const int4*>(p.wsum + n0);
        w1 = *reinterpret_cast<const int4*>(p.wsum + n0 + 4);
      }
      const int* col = tiles + (size_t)jj * srcs * 16 * MT + (8 * h) * MT + m;
      if (!XQ_IN_BOUNDS(((size_t)(jj + 1) * srcs * 16 * MT) * sizeof(int) + (size_t)MT * p.act_pitch <= (size_t)p.region_bytes && m < p.M &&
                            n0 < p.n_blocks * 16,
                        p.status))
        continue;
      int v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = col[e * MT];
      for (int o = 1; o < srcs; ++o) {
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] += col[o * 16 * MT + e * MT];
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] >>= 8;  // every product carries 16 x 16
      if (p.zp) {  // sum (c - z) qw = sum c qw - z sum qw
        v[0] -= z * w0.x; v[1] -= z * w0.y; v[2] -= z * w0.z; v[3] -= z * w0.w;
        v[4] -= z * w1.x; v[5] -= z * w1.y; v[6] -= z * w1.z; v[7] -= z * w1.w;
      }
      const float sxm = pre ? e_sx : (FUSED ? __ldcg(p.sx + m) : p.sx[m]);
      const size_t o = (size_t)m * p.N + n0;
      if (n0 + 8 <= p.N && (p.N & 7) == 0) {
        const float4 s0 = pre ? e_s0 : *reinterpret_cast<const float4*>(p.sw + n0);
        const float4 s1 = pre ? e_s1 : *reinterpret_cast<const float4*>(p.sw + n0 + 4);
        const float sc[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
        uint32_t hw[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const __nv_bfloat162 b2 = __halves2bfloat162(__float2bfloat16_rn((float)v[2 * e] * sxm * sc[2 * e]),
                                                       __float2bfloat16_rn((float)v[2 * e + 1] * sxm * sc[2 * e + 1]));
          hw[e] = *reinterpret_cast<const uint32_t*>(&b2);
        }
        *reinterpret_cast<uint4*>(p.out + o) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
        if (p.acc_opt) {
          *reinterpret_cast<int4*>(p.acc_opt + o) = make_int4(v[0], v[1], v[2], v[3]);
          *reinterpret_cast<int4*>(p.acc_opt + o + 4) = make_int4(v[4], v[5], v[6], v[7]);
        }
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e)
          if (n0 + e < p.N) {
            p.out[o + e] = __float2bfloat16_rn((float)v[e] * sxm * p.sw[n0 + e]);
            if (p.acc_opt) p.acc_opt[o + e] = v[e];
          }
      }
    }
  }
  if (FUSED && tid == 0) {
    // this CTA is past the row count (its warp 0 waited for it): once every CTA has said so, both words go back to
    // zero for the next launch on this workspace (which looks at them only after this grid has completed)
    if (atomicAdd(p.sync_words + kExitWord, 1u) == gridDim.x - 1) {
      p.sync_words[kRowsWord] = 0u;
      p.sync_words[kExitWord] = 0u;
    }
  }
}

struct DecodePlan {
  int nt, C, stages, act_pitch, max_blocks, grid, log2S, P, region;
  size_t smem;
};

// Cached answers of cudaOccupancyMaxActiveClusters, keyed by (device, variant, shared memory).
struct ClusterCacheEntry {
  int device, nt, C, fused;
  size_t smem;
  int clusters;
};
std::mutex g_cache_mutex;
ClusterCacheEntry g_cache[128];
int g_cache_size = 0;

template <int NT, int C, bool FUSED>
cudaError_t launch_variant(const DecodeParams& p, int grid, size_t smem, cudaStream_t st, int* max_clusters) {
  auto kern = gemm_decode_kernel<NT, C, FUSED>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  if (max_clusters) {  // occupancy query only
    cfg.numAttrs = 1;
    cfg.gridDim = dim3(C);
    return cudaOccupancyMaxActiveClusters(max_clusters, kern, &cfg);
  }
  return cudaLaunchKernelEx(&cfg, kern, p);
}

template <bool FUSED>
cudaError_t dispatch_f(int nt, int C, const DecodeParams& p, int grid, size_t smem, cudaStream_t st, int* max_clusters) {
  if (C == 1) {
    if (nt == 1) return launch_variant<1, 1, FUSED>(p, grid, smem, st, max_clusters);
    if (nt == 2) return launch_variant<2, 1, FUSED>(p, grid, smem, st, max_clusters);
    return launch_variant<4, 1, FUSED>(p, grid, smem, st, max_clusters);
  }
  if (C == 2) {
    if (nt == 1) return launch_variant<1, 2, FUSED>(p, grid, smem, st, max_clusters);
    if (nt == 2) return launch_variant<2, 2, FUSED>(p, grid, smem, st, max_clusters);
    return launch_variant<4, 2, FUSED>(p, grid, smem, st, max_clusters);
  }
  if (nt == 1) return launch_variant<1, 4, FUSED>(p, grid, smem, st, max_clusters);
  if (nt == 2) return launch_variant<2, 4, FUSED>(p, grid, smem, st, max_clusters);
  return launch_variant<4, 4, FUSED>(p, grid, smem, st, max_clusters);
}

cudaError_t dispatch(bool fused, int nt, int C, const DecodeParams& p, int grid, size_t smem, cudaStream_t st, int* max_clusters) {
  return fused ? dispatch_f<true>(nt, C, p, grid, smem, st, max_clusters) : dispatch_f<false>(nt, C, p, grid, smem, st, max_clusters);
}

int max_active_clusters(int device, int nt, int C, bool fused, size_t smem) {
  std::lock_guard<std::mutex> lock(g_cache_mutex);
  for (int i = 0; i < g_cache_size; ++i)
    if (g_cache[i].device == device && g_cache[i].nt == nt && g_cache[i].C == C && g_cache[i].fused == (int)fused && g_cache[i].smem == smem)
      return g_cache[i].clusters;
  int n = 0;
  DecodeParams dummy = {};
  if (dispatch(fused, nt, C, dummy, C, smem, nullptr, &n) != cudaSuccess) {
    cudaGetLastError();
    n = 0;
  }
  if (g_cache_size < 128) g_cache[g_cache_size++] = {device, nt, C, (int)fused, smem, n};
  return n;
}

// Shared-memory plan for M tokens; stages == 0 means the shape does not fit this kernel.  rot_bytes > 0: the fused
// form, whose rotation scratch shares the region of the token slice and the partial tiles.
DecodePlan decode_plan(int M, const xq_weights* w, size_t rot_bytes = 0) {
  DecodePlan d = {};
  if (M < 1 || M > XQ_DECODE_MAX_M || w->Kp % XQ_K_GROUP != 0) return d;
  d.nt = M <= 8 ? 1 : (M <= 16 ? 2 : 4);
  const int MT = 8 * d.nt, groups = w->Kp / XQ_K_GROUP, n_blocks = (w->N + 15) / 16;
  const size_t cap = 227 * 1024;
  // Small layers are latency-bound: when a CTA would stream less than 64 KiB anyway, skip the K cut
  // between CTAs (no cluster barrier, no remote stores) if the whole token slice fits.
  const size_t weight_bytes = (size_t)n_blocks * 16 * (w->Kp / 2);
  const int c_first = (weight_bytes / (size_t)w->sms < 64 * 1024 && M * groups <= 1200) ? 1 : 2;  // and few tokens to expand
  // More than 8 tokens: every CTA reads its K slice of all tokens from L2, the same lines as every other cluster, and that
  // read is what the kernel waits for before its first MMA; clusters of four cut it to a quarter (measured: 4-12 % of
  // the step at 16 and 32 tokens).  The smaller cluster sizes follow as fall-backs.
  const int order_many[3] = {4, 2, 1}, order_few[3] = {c_first, 2 * c_first, c_first == 1 ? 4 : 0};
  for (int ci = 0; ci < 3; ++ci) {
    const int C = M > 8 ? order_many[ci] : order_few[ci];
    if (C == 0 || C > 4) break;
    if (M > 8 && C == 1 && c_first != 1) break;
    if (groups < 4 * C) {
      if (M > 8) continue;
      break;
    }
    const int Lmax = (groups + C - 1) / C, Lmin = groups / C;
    const int chunks = (Lmax + 3) / 4, chunks_min = (Lmin + 3) / 4;
    const int pitch = chunks * 128 + 16;  // 16 (mod 128): conflict-free 128-bit fragment reads
    const size_t act = (size_t)MT * pitch;
    // a first guess of the cluster count sizes the tiles; refined below with the occupancy answer
    for (int pass = 0, clusters = w->sms / C; pass < 2; ++pass) {
      if (clusters < 1) break;
      const int nc = clusters < n_blocks ? clusters : n_blocks;
      const int max_blocks = (n_blocks + nc - 1) / nc;
      // sub-slices: as few as give most consumer warps an item in the first round (long items keep
      // several ring pieces in flight per warp), each item at least one chunk long
      int log2S = 0;
      while ((max_blocks << log2S) < 12 && (2 << log2S) <= chunks_min && log2S < 4) ++log2S;
      const int S = 1 << log2S;
      const int item_chunks_max = (chunks + S - 1) / S, item_chunks_min = chunks_min / S;
      int P = (item_chunks_max + kPieceChunks - 1) / kPieceChunks;
      while (P <= item_chunks_min && (item_chunks_max + P - 1) / P > kPieceChunks) ++P;  // uneven cuts: keep pieces <= 4 KiB
      if (P < 1 || P > item_chunks_min) break;  // every piece holds at least one chunk
      const size_t tiles = (size_t)((max_blocks + C - 1) / C) * C * S * 16 * MT * 4;
      const size_t misc = 2 * kMaxStages * 8 + 64 + 128;
      const size_t region = ((act + tiles > rot_bytes ? act + tiles : rot_bytes) + 127) / 128 * 128;
      if (region + misc + 16 * (size_t)kStageBytes > cap) break;
      const int room = (int)((cap - region - misc) / kStageBytes);
      const int want = ((max_blocks << log2S) + kConsumerWarps - 1) / kConsumerWarps * P * kConsumerWarps;
      const int stg = (room >= 48 && want > 32) ? 48 : ((room >= 32 && want > 16) ? 32 : 16);
      const size_t smem = region + misc + (size_t)stg * kStageBytes;
      const int fit = max_active_clusters(w->device, d.nt, C, rot_bytes > 0, smem);
      if (fit < 1) break;
      if (pass == 1 || fit >= clusters) {
        d.C = C;
        d.stages = stg;
        d.act_pitch = pitch;
        d.max_blocks = max_blocks;
        d.grid = nc * C;
        d.smem = smem;
        d.log2S = log2S;
        d.P = P;
        d.region = (int)region;
        return d;
      }
      clusters = fit;
    }
  }
  return d;
}

}  // namespace

bool xq_decode_shape(int32_t M, const xq_weights* w, int* padded_tokens, int* cluster) {
  const DecodePlan d = decode_plan(M, w);
  if (d.stages < 16) return false;
  *padded_tokens = 8 * d.nt;
  *cluster = d.C;
  return true;
}

namespace {
void fill_params(DecodeParams& p, const DecodePlan& d, const uint8_t* Xq, const float* sx, const int32_t* zp, int32_t M, const xq_weights* w,
                 void* out, int32_t* acc_opt, int32_t* status) {
  p = {};
  p.W = w->packed;
  p.sw = w->s_w;
  p.Xq = Xq;
  p.sx = sx;
  p.out = (__nv_bfloat16*)out;
  p.acc_opt = acc_opt;
  p.zp = zp;
  p.wsum = w->w_sum;
  p.status = status;
  p.w_bytes = (size_t)w->Np * w->Kpp / 2;
  p.M = M;
  p.N = w->N;
  p.Kp = w->Kp;
  p.k_groups = w->Kpp / XQ_K_GROUP;
  p.n_blocks = (w->N + 15) / 16;
  p.stages = d.stages;
  p.act_pitch = d.act_pitch;
  p.max_blocks = d.max_blocks;
  p.log2S = d.log2S;
  p.P = d.P;
  p.region_bytes = d.region;
}
}  // namespace

cudaError_t xq_launch_gemm_decode(const uint8_t* Xq, const float* sx, const int32_t* zp, int32_t M, const xq_weights* w,
                                  void* out, int32_t* acc_opt, int32_t* status, cudaStream_t st) {
  const DecodePlan d = decode_plan(M, w);
  if (d.stages < 16) return cudaErrorNotSupported;
  DecodeParams p;
  fill_params(p, d, Xq, sx, zp, M, w, out, acc_opt, status);
  return dispatch(false, d.nt, d.C, p, d.grid, d.smem, st, nullptr);
}

bool xq_linear_decode_supported(int32_t M, const xq_weights* w) {
  if (M < 1 || M > XQ_DECODE_MAX_M || w->heads != 1 || !w->hp_signs || !xqrot::plan_supported(w->plan)) return false;
  return decode_plan(M, w, xqrot::row_layout(w->plan).total).stages >= 16;
}

cudaError_t xq_launch_linear_decode(const void* X, int64_t ldx, uint8_t* Xq, float* sx, int32_t* zp, int32_t M, const xq_weights* w,
                                    void* out, int32_t* header, cudaStream_t st) {
  if (M < 1 || M > XQ_DECODE_MAX_M || w->heads != 1 || !w->hp_signs || !xqrot::plan_supported(w->plan)) return cudaErrorNotSupported;
  const xq_hadamard_plan_t& pl = w->plan;
  const DecodePlan d = decode_plan(M, w, xqrot::row_layout(pl).total);
  if (d.stages < 16) return cudaErrorNotSupported;
  DecodeParams p;
  fill_params(p, d, Xq, sx, zp, M, w, out, nullptr, header);
  p.X = (const __nv_bfloat16*)X;
  p.ldx = ldx;
  p.plan = pl;
  p.gamma = (float)(1.0 / sqrt((double)pl.Kp));
  p.Hsigns = (const __nv_bfloat16*)w->hp_signs;
  p.Xq_w = Xq;
  p.sx_w = sx;
  p.zp_w = zp;
  p.sync_words = (uint32_t*)header;
  p.rot_threads = 32 * ((pl.p + 15) / 16) * xqrot::row_chunks(pl);
  return dispatch(true, d.nt, d.C, p, d.grid, d.smem, st, nullptr);
}
