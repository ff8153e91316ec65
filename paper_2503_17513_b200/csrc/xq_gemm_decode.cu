// Decode-shape W4A4 GEMM (M <= 32 tokens): a memory-bound split-K kernel that streams the
// packed INT4 weights once from HBM (paper Sec. 3: the quantized product Q(XR) Q(W~) computed at
// inference; here the case where the weight stream, not the arithmetic, sets the time).
//
// Decomposition.  Output channels are handled in blocks of 8; a thread-block cluster of C CTAs
// owns a contiguous range of blocks and cuts K between its CTAs in multiples of 32 codes, so a
// CTA needs only its K slice of the quantized tokens.  In the weight layout the K slice of one
// block is one contiguous run of bytes; a producer warp fetches runs with bulk copies (pieces of
// at most 4 KiB) into a shared-memory ring, the first ring-full before the kernel waits for its
// predecessor in the stream.  Each of the eight consumer warps owns whole blocks (block j of
// the range goes to warp j mod 8), so a block's partial sums stay in one warp's registers:
// MMA i of a chunk of four 32-code groups takes group i; lane (channel g, word t) loads its word
// of eight codes with one conflict-free 32-bit load, the nibble split turns it into the B
// fragment of an m16n8k32 integer MMA (even codes in K slots 4t.., odd codes in 16+4t..), and the
// A fragments (16 tokens) come from the token slice that the CTA expanded once into shared
// memory in exactly that fragment order.  Block j is finished by CTA j mod C
// of the cluster: every CTA stores its partial tile of the block into that CTA's shared memory
// (distributed shared memory), and after one cluster barrier the owner sums the C tiles and
// applies the epilogue (scales, bf16, 16-byte stores).  No global scratch, no atomics, and no
// CTA waits on another outside the cluster barrier.
#include <cuda_bf16.h>

#include <mutex>

#include "xq_internal.h"
#include "xq_ptx.cuh"

using namespace xqptx;

namespace {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;
constexpr int kPieceGroups = 32;                               // 32-code groups per ring stage
constexpr int kStageBytes = kPieceGroups * XQ_GROUP_BYTES;     // 4 KiB
constexpr int kMaxStages = 32;

struct DecodeParams {
  const uint8_t* W;
  const float* sw;
  const uint8_t* Xq;
  const float* sx;
  __nv_bfloat16* out;
  int32_t* acc_opt;
  int32_t* status;
  int M, N, Kp;
  int k_groups;     // groups of 32 codes per channel block in the weight layout (K'' / 32)
  int n_blocks;     // channel blocks holding real channels: ceil(N / 8)
  int stages;       // ring stages: 8, 16 or 32
  int act_pitch;    // bytes between token rows of the expanded token slice
  int max_blocks;   // blocks in the longest cluster range
};

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

template <int NT, int C>  // NT token tiles of 16 (M <= 16 NT), clusters of C CTAs
__global__ void __launch_bounds__(kThreads, 1) gemm_decode_kernel(const DecodeParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int MT = 16 * NT;  // padded token count
  const int rank = C == 1 ? 0 : (int)cluster_ctarank();
  const int cid = blockIdx.x / C, n_clusters = gridDim.x / C;

  unsigned char* ring = smem;
  unsigned char* act = ring + (size_t)p.stages * kStageBytes;
  // partial tiles of the blocks this CTA finishes: [owned block][source CTA][token][8 channels]
  int* tiles = reinterpret_cast<int*>(act + (size_t)MT * p.act_pitch);
  uint64_t* full = reinterpret_cast<uint64_t*>(tiles + (size_t)((p.max_blocks + C - 1) / C) * C * MT * 8);
  uint64_t* empty = full + p.stages;
  volatile int* failed = reinterpret_cast<volatile int*>(empty + p.stages);

  // this cluster's channel blocks and this CTA's K slice (in groups of 32 codes)
  const int b0 = (int)((long long)cid * p.n_blocks / n_clusters), b1 = (int)((long long)(cid + 1) * p.n_blocks / n_clusters);
  const int n_blk = b1 - b0;
  const int groups = p.Kp / XQ_K_GROUP;
  const int g0 = rank * groups / C, g1 = (rank + 1) * groups / C;
  const int L = g1 - g0;                                  // groups in the slice
  const int parts = (L + kPieceGroups - 1) / kPieceGroups;  // ring pieces per block
  const int rounds = (n_blk + kConsumerWarps - 1) / kConsumerWarps;

  if (tid < p.stages) {
    mbar_init(&full[tid], 1);
    mbar_init(&empty[tid], 1);
  }
  if (tid == 32) *failed = 0;
  mbar_fence_init();
  __syncthreads();
  if (C > 1) cluster_arrive_relaxed();  // "this CTA runs": awaited before the first remote store
  pdl_launch_dependents();
  const uint32_t smask = (uint32_t)p.stages - 1u;
  const int sshift = 31 - __clz(p.stages);

  if (warp == kConsumerWarps) {
    // ---------------- producer ------------------------------------------------------------------
    // Piece i = (round r, part q, warp w) -> ring stage i mod stages (a stage is always reused
    // by the same consumer warp).  Lane l owns ring stage l and issues its pieces l, l + stages,
    // ... in order, so it sees every phase of that stage's "empty" barrier in turn (a one-bit
    // parity cannot tell phase n from phase n + 2); one lane alone would be far too slow to feed
    // the copy engine.  The weights are constants: nothing here waits for the preceding kernel.
    const int total = rounds * parts * kConsumerWarps;
    for (int i = lane; i < total && lane < p.stages; i += p.stages) {
      const int w = i & (kConsumerWarps - 1), rq = i >> 3, r = rq / parts, q = rq - r * parts;
      const int j = r * kConsumerWarps + w;
      if (j >= n_blk) continue;
      const int s = i & smask;
      if (i >= p.stages && !mbar_wait_bounded(&empty[s], ((i >> sshift) - 1) & 1, failed, p.status, (int)XQ_ERR_TIMEOUT)) break;
      const int ng = min(kPieceGroups, L - q * kPieceGroups);
      const uint32_t bytes = (uint32_t)ng * XQ_GROUP_BYTES;
      const unsigned char* src = p.W + ((size_t)(b0 + j) * p.k_groups + g0 + q * kPieceGroups) * XQ_GROUP_BYTES;
      mbar_expect_tx(&full[s], bytes);
      bulk_g2s(ring + (size_t)s * kStageBytes, src, bytes, &full[s]);
    }
    __syncwarp();
    if (C > 1) cluster_wait_acquire();
  } else {
    // ---------------- consumers ----------------------------------------------------------------
    // token rows beyond M are zero
    for (int i = tid; i < (MT - p.M) * (p.act_pitch / 16); i += kConsumerThreads)
      reinterpret_cast<uint4*>(act + (size_t)p.M * p.act_pitch)[i] = make_uint4(0, 0, 0, 0);
    pdl_wait();
    // Expand this CTA's K slice of the packed tokens once, in fragment order: chunk c of four
    // groups takes 128 bytes per token, word t of group i (even codes, odd codes) at
    // c * 128 + t * 32 + i * 8.
    {
      const int total = p.M * L;
      constexpr int kBatch = 4;
      for (int base = tid; base < total; base += kBatch * kConsumerThreads) {
        uint4 v[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
          const int i = base + u * kConsumerThreads;
          if (i < total) {
            const int m = i / L, l = i - m * L;
            v[u] = __ldg(reinterpret_cast<const uint4*>(p.Xq + (size_t)m * (p.Kp / 2)) + g0 + l);
          }
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
          const int i = base + u * kConsumerThreads;
          if (i < total) {
            const int m = i / L, l = i - m * L;
            unsigned char* d = act + (size_t)m * p.act_pitch + (size_t)(l >> 2) * 128 + (size_t)(l & 3) * 8;
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

    const int ag = lane >> 2, at = lane & 3;  // MMA fragment coordinates: channel / token row, word
    bool ok = true;
    for (int r = 0; r < rounds && ok; ++r) {
      const int j = r * kConsumerWarps + warp;
      if (j >= n_blk) break;
      int acc[NT][2][4];
#pragma unroll
      for (int a = 0; a < NT; ++a)
#pragma unroll
        for (int c = 0; c < 2; ++c) acc[a][c][0] = acc[a][c][1] = acc[a][c][2] = acc[a][c][3] = 0;
      for (int q = 0; q < parts && ok; ++q) {
        const int i = (r * parts + q) * kConsumerWarps + warp;
        const int s = i & smask;
        ok = mbar_wait_bounded(&full[s], (i >> sshift) & 1, failed, p.status, (int)XQ_ERR_TIMEOUT);
        if (!ok) break;
        const int ng = min(kPieceGroups, L - q * kPieceGroups);
        const unsigned char* wp = ring + (size_t)s * kStageBytes + lane * 4;  // channel ag, word at of group 0
#pragma unroll 2
        for (int gq = 0; gq < ng; gq += 4, wp += 4 * XQ_GROUP_BYTES) {
          const int nv = min(4, ng - gq);  // groups of this chunk that exist
          uint32_t b[4][2];
#pragma unroll
          for (int i4 = 0; i4 < 4; ++i4) {
            const uint32_t wv = i4 < nv ? *reinterpret_cast<const uint32_t*>(wp + i4 * XQ_GROUP_BYTES) : 0u;
            split16(wv, b[i4][0], b[i4][1]);
          }
          const size_t coff = (size_t)(q * (kPieceGroups / 4) + (gq >> 2)) * 128 + (size_t)at * 32;
#pragma unroll
          for (int a = 0; a < NT; ++a) {
            const uint4* lo = reinterpret_cast<const uint4*>(act + (size_t)(16 * a + ag) * p.act_pitch + coff);
            const uint4* hi = reinterpret_cast<const uint4*>(act + (size_t)(16 * a + ag + 8) * p.act_pitch + coff);
            const uint4 x0 = lo[0], x1 = lo[1], y0 = hi[0], y1 = hi[1];
            const uint32_t a0[4] = {x0.x, y0.x, x0.y, y0.y};
            const uint32_t a1[4] = {x0.z, y0.z, x0.w, y0.w};
            const uint32_t a2[4] = {x1.x, y1.x, x1.y, y1.y};
            const uint32_t a3[4] = {x1.z, y1.z, x1.w, y1.w};
            mma_s8_16x8x32(acc[a][0], a0, b[0][0], b[0][1]);
            mma_s8_16x8x32(acc[a][1], a1, b[1][0], b[1][1]);
            mma_s8_16x8x32(acc[a][0], a2, b[2][0], b[2][1]);
            mma_s8_16x8x32(acc[a][1], a3, b[3][0], b[3][1]);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[s]);
      }
      // D fragment: (token ag, channels 2 at, 2 at + 1), (token ag + 8, same channels) -> the
      // tile [j / C][rank] in the shared memory of CTA j mod C
      const int owner = j % C;
      int* tl = tiles + ((size_t)(j / C) * C + rank) * MT * 8;
#pragma unroll
      for (int a = 0; a < NT; ++a) {
        const int2 v0 = make_int2(acc[a][0][0] + acc[a][1][0], acc[a][0][1] + acc[a][1][1]);
        const int2 v1 = make_int2(acc[a][0][2] + acc[a][1][2], acc[a][0][3] + acc[a][1][3]);
        int* d0 = &tl[(16 * a + ag) * 8 + 2 * at];
        int* d1 = &tl[(16 * a + ag + 8) * 8 + 2 * at];
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
  if (C > 1) {
    cluster_arrive_release();
    cluster_wait_acquire();
  } else {
    __syncthreads();
  }
  if (warp < kConsumerWarps && !*failed) {
    // this CTA finishes blocks j = rank, rank + C, ...: one thread per (block, token)
    const int mine = (n_blk - rank + C - 1) / C;
    for (int idx = tid; idx < mine * p.M; idx += kConsumerThreads) {
      const int jj = idx / p.M, m = idx - jj * p.M;
      const int j = rank + jj * C;
      const int* row = tiles + ((size_t)jj * C * MT + m) * 8;
      int4 lo = *reinterpret_cast<const int4*>(row), hi = *reinterpret_cast<const int4*>(row + 4);
#pragma unroll
      for (int o = 1; o < C; ++o) {
        const int4 l2 = *reinterpret_cast<const int4*>(row + o * MT * 8), h2 = *reinterpret_cast<const int4*>(row + o * MT * 8 + 4);
        lo.x += l2.x; lo.y += l2.y; lo.z += l2.z; lo.w += l2.w;
        hi.x += h2.x; hi.y += h2.y; hi.z += h2.z; hi.w += h2.w;
      }
      const int v[8] = {lo.x >> 8, lo.y >> 8, lo.z >> 8, lo.w >> 8, hi.x >> 8, hi.y >> 8, hi.z >> 8, hi.w >> 8};  // every product carries 16 x 16
      const int n0 = (b0 + j) * 8;
      const float sxm = p.sx[m];
      const size_t o = (size_t)m * p.N + n0;
      if (n0 + 8 <= p.N && (p.N & 7) == 0) {
        const float4 s0 = *reinterpret_cast<const float4*>(p.sw + n0), s1 = *reinterpret_cast<const float4*>(p.sw + n0 + 4);
        const float sc[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
        uint32_t h[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const __nv_bfloat162 b2 = __halves2bfloat162(__float2bfloat16_rn((float)v[2 * e] * sxm * sc[2 * e]),
                                                       __float2bfloat16_rn((float)v[2 * e + 1] * sxm * sc[2 * e + 1]));
          h[e] = *reinterpret_cast<const uint32_t*>(&b2);
        }
        *reinterpret_cast<uint4*>(p.out + o) = make_uint4(h[0], h[1], h[2], h[3]);
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
}

struct DecodePlan {
  int nt, C, stages, act_pitch, max_blocks, grid;
  size_t smem;
};

// Cached answers of cudaOccupancyMaxActiveClusters, keyed by (device, variant, shared memory).
struct ClusterCacheEntry {
  int device, nt, C;
  size_t smem;
  int clusters;
};
std::mutex g_cache_mutex;
ClusterCacheEntry g_cache[64];
int g_cache_size = 0;

template <int NT, int C>
cudaError_t launch_variant(const DecodeParams& p, int grid, size_t smem, cudaStream_t st, int* max_clusters) {
  auto kern = gemm_decode_kernel<NT, C>;
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

cudaError_t dispatch(int nt, int C, const DecodeParams& p, int grid, size_t smem, cudaStream_t st, int* max_clusters) {
  if (C == 2) {
    if (nt == 1) return launch_variant<1, 2>(p, grid, smem, st, max_clusters);
    return launch_variant<2, 2>(p, grid, smem, st, max_clusters);
  }
  if (nt == 1) return launch_variant<1, 4>(p, grid, smem, st, max_clusters);
  return launch_variant<2, 4>(p, grid, smem, st, max_clusters);
}

int max_active_clusters(int device, int nt, int C, size_t smem) {
  std::lock_guard<std::mutex> lock(g_cache_mutex);
  for (int i = 0; i < g_cache_size; ++i)
    if (g_cache[i].device == device && g_cache[i].nt == nt && g_cache[i].C == C && g_cache[i].smem == smem) return g_cache[i].clusters;
  int n = 0;
  DecodeParams dummy = {};
  if (dispatch(nt, C, dummy, C, smem, nullptr, &n) != cudaSuccess) {
    cudaGetLastError();
    n = 0;
  }
  if (g_cache_size < 64) g_cache[g_cache_size++] = {device, nt, C, smem, n};
  return n;
}

// Shared-memory plan for M tokens; stages == 0 means the shape does not fit this kernel.
DecodePlan decode_plan(int M, const xq_weights* w) {
  DecodePlan d = {};
  if (M < 1 || M > XQ_DECODE_MAX_M || w->Kp % XQ_K_GROUP != 0) return d;
  d.nt = M <= 16 ? 1 : 2;
  const int MT = 16 * d.nt, groups = w->Kp / XQ_K_GROUP, n_blocks = (w->N + 7) / 8;
  const size_t cap = 227 * 1024;
  for (int C = 2; C <= 4; C *= 2) {
    if (groups < C) break;
    const int Lmax = (groups + C - 1) / C;
    const int chunks = (Lmax + 3) / 4;
    const int pitch = chunks * 128 + 16;  // 16 (mod 128): conflict-free 128-bit fragment reads
    const size_t act = (size_t)MT * pitch;
    // a first guess of the cluster count sizes the tiles; refined below with the occupancy answer
    for (int pass = 0, clusters = w->sms / C; pass < 2; ++pass) {
      if (clusters < 1) break;
      const int nc = clusters < n_blocks ? clusters : n_blocks;
      const int max_blocks = (n_blocks + nc - 1) / nc;
      const size_t tiles = (size_t)((max_blocks + C - 1) / C) * C * MT * 8 * 4;
      const size_t misc = 2 * kMaxStages * 8 + 64 + 128;
      if (act + tiles + misc + 8 * (size_t)kStageBytes > cap) break;
      const int parts = (Lmax + kPieceGroups - 1) / kPieceGroups;
      const int rounds = (max_blocks + kConsumerWarps - 1) / kConsumerWarps;
      const int room = (int)((cap - act - tiles - misc) / kStageBytes);
      const int want = rounds * parts * kConsumerWarps;
      int s = 8;
      while (2 * s <= kMaxStages && 2 * s <= room && s < want) s *= 2;
      const size_t smem = act + tiles + misc + (size_t)s * kStageBytes;
      const int fit = max_active_clusters(w->device, d.nt, C, smem);
      if (fit < 1) break;
      if (pass == 1 || fit == clusters) {
        d.C = C;
        d.stages = s;
        d.act_pitch = pitch;
        d.max_blocks = max_blocks;
        d.grid = nc * C;
        d.smem = smem;
        return d;
      }
      clusters = fit < clusters ? fit : clusters;
    }
  }
  return d;
}

}  // namespace

cudaError_t xq_launch_gemm_decode(const uint8_t* Xq, const float* sx, int32_t M, const xq_weights* w, void* out,
                                  int32_t* acc_opt, int32_t* status, cudaStream_t st) {
  const DecodePlan d = decode_plan(M, w);
  if (d.stages < 8) return cudaErrorNotSupported;
  DecodeParams p;
  p.W = w->packed;
  p.sw = w->s_w;
  p.Xq = Xq;
  p.sx = sx;
  p.out = (__nv_bfloat16*)out;
  p.acc_opt = acc_opt;
  p.status = status;
  p.M = M;
  p.N = w->N;
  p.Kp = w->Kp;
  p.k_groups = w->Kpp / XQ_K_GROUP;
  p.n_blocks = (w->N + 7) / 8;
  p.stages = d.stages;
  p.act_pitch = d.act_pitch;
  p.max_blocks = d.max_blocks;
  return dispatch(d.nt, d.C, p, d.grid, d.smem, st, nullptr);
}
