// GPTQ with act-order for the expanded, rotated weights (paper Sec. 4 "Quantization Details": the weights of the
// experiments are quantized with GPTQ, act-order, per-channel symmetric 4-bit; Sec. 3.1 Remark 2 is about this
// quantizer under expansion).  Offline step, fp64 on the device.
//
// The published algorithm walks the channels in descending order of diag(H), quantizes one column at a time and
// feeds the error into the columns still to come through the upper Cholesky factor U of H^-1.  The same numbers come
// out of a form that needs no inverse: with H = R R^T, R upper triangular (a Cholesky factorisation started from the
// last channel), R = U^-1 and the value that column k is quantized from is
//     w'_k = w_k + sum_{j<k} (w_j - s q_j) R[j][k] / R[k][k],
// the deviations (w_j - s q_j) being those of the ORIGINAL weights.  Reversing the channel order turns R into an
// ordinary lower Cholesky factor L' of the reversed matrix, so the device work is: gather H in (reversed) visiting
// order with the damping on its diagonal, factorise it (blocked, right-looking), then sweep the columns from the
// last to the first in blocks of 64 -- one product of the deviations so far with a panel of L' per block, then the 64
// columns one after the other with the panel's triangle in shared memory, one thread per output channel.
#include <math.h>

#include <algorithm>
#include <numeric>
#include <vector>

#include "xq_internal.h"

namespace {

constexpr int kB = 64;  // block size of the factorisation and of the sweep
constexpr size_t kTwoBlocksSmem = 2 * (size_t)kB * (kB + 1) * sizeof(double);  // two kB x kB tiles of doubles

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct DevMem {
  void* p = nullptr;
  cudaError_t alloc(size_t bytes) { return cudaMalloc(&p, bytes ? bytes : 1); }
  ~DevMem() {
    if (p) cudaFree(p);
  }
  template <class T>
  T* as() const {
    return reinterpret_cast<T*>(p);
  }
};

// A[i][j] = H[src[i]][src[j]] (+ add on the diagonal; a dead channel, H[c][c] == 0, gets 1 there first).
__global__ void gather_hessian_kernel(const double* __restrict__ H, int n, const int* __restrict__ src, double add, double* __restrict__ A) {
  const long long total = (long long)n * n;
  for (long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x; t < total; t += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(t / n), j = (int)(t - (long long)i * n);
    double v = H[(size_t)src[i] * n + src[j]];
    if (i == j) v = (v == 0.0 ? 1.0 : v) + add;
    A[t] = v;
  }
}

// C[i][j] (i < m, j < nn) += alpha * sum_{k < kk} A[i * lda + k] * B[k * sbk + j * sbj]; lower_only: tiles above the
// diagonal of a square C are skipped.  64 x 64 tiles, 256 threads, 4 x 4 outputs each.
__global__ void __launch_bounds__(256) dgemm_tile_kernel(int m, int nn, int kk, double alpha, const double* __restrict__ A, size_t lda,
                                                         const double* __restrict__ B, size_t sbk, size_t sbj, double* __restrict__ C,
                                                         size_t ldc, int lower_only, const double* __restrict__ col_div, int assign) {
  if (lower_only && blockIdx.x > blockIdx.y) return;
  __shared__ double As[16][kB + 1];
  __shared__ double Bs[16][kB + 1];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int i0 = blockIdx.y * kB, j0 = blockIdx.x * kB;
  double acc[4][4] = {};
  for (int k0 = 0; k0 < kk; k0 += 16) {
    for (int t = threadIdx.x; t < 16 * kB; t += 256) {
      const int r = t >> 4, c = t & 15;  // A tile: row r of 64, k index c
      As[c][r] = (i0 + r < m && k0 + c < kk) ? A[(size_t)(i0 + r) * lda + k0 + c] : 0.0;
      const int kr = t / kB, jc = t - kr * kB;  // B tile: k index kr, column jc of 64
      Bs[kr][jc] = (k0 + kr < kk && j0 + jc < nn) ? B[(size_t)(k0 + kr) * sbk + (size_t)(j0 + jc) * sbj] : 0.0;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      double a[4], b[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        a[u] = As[k][ty + 16 * u];
        b[u] = Bs[k][tx + 16 * u];
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[u][v] = fma(a[u], b[v], acc[u][v]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int u = 0; u < 4; ++u)
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      const int i = i0 + ty + 16 * u, j = j0 + tx + 16 * v;
      if (i < m && j < nn) {
        double r = alpha * acc[u][v];
        if (col_div) r /= col_div[(size_t)j * (ldc + 1)];  // divide column j by the diagonal entry (j, j) of the factor
        double* c = C + (size_t)i * ldc + j;
        *c = assign ? r : *c + r;
      }
    }
}

// Lower Cholesky of the nb x nb block at (k0, k0), in place.  One CTA.
__global__ void __launch_bounds__(256) chol_diag_kernel(double* __restrict__ A, int n, int k0, int nb, int* __restrict__ fail) {
  __shared__ double a[kB][kB + 1];
  for (int t = threadIdx.x; t < nb * nb; t += blockDim.x) a[t / nb][t % nb] = A[(size_t)(k0 + t / nb) * n + k0 + t % nb];
  __syncthreads();
  for (int j = 0; j < nb; ++j) {
    const double d = a[j][j];
    if (!(d > 0.0)) {
      if (threadIdx.x == 0) *fail = 1;
      return;
    }
    const double r = sqrt(d);
    __syncthreads();
    for (int i = j + threadIdx.x; i < nb; i += blockDim.x) a[i][j] = i == j ? r : a[i][j] / r;
    __syncthreads();
    for (int t = threadIdx.x; t < (nb - j - 1) * (nb - j - 1); t += blockDim.x) {
      const int i = j + 1 + t / (nb - j - 1), k = j + 1 + t % (nb - j - 1);
      if (k <= i) a[i][k] -= a[i][j] * a[k][j];
    }
    __syncthreads();
  }
  for (int t = threadIdx.x; t < nb * nb; t += blockDim.x) {
    const int i = t / nb, j = t % nb;
    A[(size_t)(k0 + i) * n + k0 + j] = j <= i ? a[i][j] : 0.0;
  }
}

// Rows i >= k0 + nb of the panel: X L^T = A[i][k0 .. k0 + nb), L the factored diagonal block.  One thread per row.
__global__ void __launch_bounds__(kB) chol_panel_kernel(double* __restrict__ A, int n, int k0, int nb) {
  extern __shared__ double dyn_sm[];
  double(*L)[kB + 1] = reinterpret_cast<double(*)[kB + 1]>(dyn_sm);
  double(*X)[kB + 1] = L + kB;  // [column][row of this CTA]
  for (int t = threadIdx.x; t < nb * nb; t += blockDim.x) L[t / nb][t % nb] = A[(size_t)(k0 + t / nb) * n + k0 + t % nb];
  const int i = k0 + nb + blockIdx.x * kB + threadIdx.x;
  __syncthreads();
  if (i >= n) return;
  double* row = A + (size_t)i * n + k0;
  for (int c = 0; c < nb; ++c) {
    double v = row[c];
    for (int c2 = 0; c2 < c; ++c2) v -= X[c2][threadIdx.x] * L[c][c2];
    v /= L[c][c];
    X[c][threadIdx.x] = v;
    row[c] = v;
  }
}

// Per-row scale absmax / 7 (1 for a zero row) rounded to fp32, and the rows in reversed visiting order:
// V[r][c] = W[r][src[c]] (0 for a dead channel).
__global__ void gather_rows_kernel(const double* __restrict__ W, int N, int n, const int* __restrict__ src, const unsigned char* __restrict__ dead,
                                   double* __restrict__ V, float* __restrict__ s) {
  const int r = blockIdx.x;
  if (r >= N) return;
  __shared__ double red[32];
  double amax = 0.0;
  for (int c = threadIdx.x; c < n; c += blockDim.x) {
    const int sc = src[c];
    const double v = dead[sc] ? 0.0 : W[(size_t)r * n + sc];
    V[(size_t)r * n + c] = v;
    amax = fmax(amax, fabs(v));
  }
  for (int o = 16; o > 0; o >>= 1) amax = fmax(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 1; i < (int)(blockDim.x >> 5); ++i) amax = fmax(amax, red[i]);
    s[r] = amax > 0.0 ? (float)(amax / 7.0) : 1.f;
  }
}

// The columns [c0, c1) of one block from the last to the first.  Vc holds the block's columns already compensated
// for the deviations of every later block; L is the factor (row-major, n x n).  One thread per row r:
//   w' = Vc[r][c] + sum_{c < c2 < c1} D[r][c2] L[c2][c] / L[c][c];  q = clamp(rne(w' / s), -8, 7);  D[r][c] = V[r][c] - s q.
__global__ void __launch_bounds__(kB) gptq_block_kernel(const double* __restrict__ V, const double* __restrict__ Vc, double* __restrict__ D,
                                                        const double* __restrict__ L, const float* __restrict__ s, int N, int n, int c0,
                                                        int c1, int8_t* __restrict__ Q) {
  extern __shared__ double dyn_sm[];
  double(*Ls)[kB + 1] = reinterpret_cast<double(*)[kB + 1]>(dyn_sm);
  double(*Ds)[kB + 1] = Ls + kB;  // [column in block][row of this CTA]
  const int nb = c1 - c0;
  for (int t = threadIdx.x; t < nb * nb; t += blockDim.x) Ls[t / nb][t % nb] = L[(size_t)(c0 + t / nb) * n + c0 + t % nb];
  const int r = blockIdx.x * kB + threadIdx.x;
  __syncthreads();
  if (r >= N) return;
  const double sr = (double)s[r];
  for (int c = nb - 1; c >= 0; --c) {
    double acc = 0.0;
    for (int c2 = c + 1; c2 < nb; ++c2) acc = fma(Ds[c2][threadIdx.x], Ls[c2][c], acc);
    const double w = Vc[(size_t)r * n + c0 + c] + acc / Ls[c][c];
    double q = rint(w / sr);
    q = fmin(7.0, fmax(-8.0, q));
    const double d = V[(size_t)r * n + c0 + c] - sr * q;
    Ds[c][threadIdx.x] = d;
    D[(size_t)r * n + c0 + c] = d;
    Q[(size_t)r * n + c0 + c] = (int8_t)q;
  }
}

// codes[r][src[c]] = Q[r][c]
__global__ void scatter_codes_kernel(const int8_t* __restrict__ Q, int N, int n, const int* __restrict__ src, int8_t* __restrict__ codes) {
  const long long total = (long long)N * n;
  for (long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x; t < total; t += (long long)gridDim.x * blockDim.x) {
    const int r = (int)(t / n), c = (int)(t - (long long)r * n);
    codes[(size_t)r * n + src[c]] = Q[t];
  }
}

__global__ void f32_to_f64_kernel(const float* __restrict__ a, long long count, double* __restrict__ b) {
  for (long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x; t < count; t += (long long)gridDim.x * blockDim.x) b[t] = (double)a[t];
}

inline int grid_for(long long work, int threads) {
  long long g = (work + threads - 1) / threads;
  return (int)(g < 1 ? 1 : (g > 148 * 16 ? 148 * 16 : g));
}

cudaError_t dgemm(int m, int nn, int kk, double alpha, const double* A, size_t lda, const double* B, size_t sbk, size_t sbj, double* C,
                  size_t ldc, bool lower_only, const double* col_div, bool assign, cudaStream_t st) {
  if (m <= 0 || nn <= 0) return cudaSuccess;
  dim3 grid((nn + kB - 1) / kB, (m + kB - 1) / kB);
  dgemm_tile_kernel<<<grid, 256, 0, st>>>(m, nn, kk, alpha, A, lda, B, sbk, sbj, C, ldc, lower_only ? 1 : 0, col_div, assign ? 1 : 0);
  return cudaGetLastError();
}

// dW: device fp64 [N, n] rotated weights; dH: device fp64 [n, n] Hessian (read only); outputs dCodes int8 [N, n] in the
// original channel order and dS float [N].  Synchronizes `st`.
xq_status gptq_device(const double* dW, const double* dH, int N, int n, double damp, int8_t* dCodes, float* dS, cudaStream_t st) {
  // visiting order from the diagonal (host: n values)
  std::vector<double> diag((size_t)n);
  if (cudaMemcpy2DAsync(diag.data(), sizeof(double), dH, sizeof(double) * ((size_t)n + 1), sizeof(double), (size_t)n, cudaMemcpyDeviceToHost,
                        st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  std::vector<unsigned char> dead((size_t)n);
  double mean = 0.0;
  for (int i = 0; i < n; ++i) {
    dead[i] = diag[i] == 0.0;
    if (dead[i]) diag[i] = 1.0;
    mean += diag[i];
  }
  mean /= n;
  std::vector<int> perm((size_t)n), src((size_t)n);
  std::iota(perm.begin(), perm.end(), 0);
  std::stable_sort(perm.begin(), perm.end(), [&](int a, int b) { return diag[a] > diag[b]; });
  for (int c = 0; c < n; ++c) src[c] = perm[n - 1 - c];  // reversed visiting order: the sweep runs from the last column down

  DevMem mSrc, mDead, mA, mV, mVc, mD, mQ, mFail;
  if (mSrc.alloc(sizeof(int) * (size_t)n) != cudaSuccess || mDead.alloc((size_t)n) != cudaSuccess ||
      mA.alloc(sizeof(double) * (size_t)n * n) != cudaSuccess || mV.alloc(sizeof(double) * (size_t)N * n) != cudaSuccess ||
      mVc.alloc(sizeof(double) * (size_t)N * n) != cudaSuccess || mD.alloc(sizeof(double) * (size_t)N * n) != cudaSuccess ||
      mQ.alloc((size_t)N * n) != cudaSuccess || mFail.alloc(sizeof(int)) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_ALLOC;
  }
  double* A = mA.as<double>();
  if (cudaFuncSetAttribute(chol_panel_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTwoBlocksSmem) != cudaSuccess ||
      cudaFuncSetAttribute(gptq_block_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTwoBlocksSmem) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  cudaError_t e = cudaMemcpyAsync(mSrc.p, src.data(), sizeof(int) * (size_t)n, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(mDead.p, dead.data(), (size_t)n, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(mFail.p, 0, sizeof(int), st);
  if (e == cudaSuccess) {
    gather_hessian_kernel<<<grid_for((long long)n * n, 256), 256, 0, st>>>(dH, n, mSrc.as<int>(), damp * mean, A);
    e = cudaGetLastError();
  }
  // blocked right-looking Cholesky, lower, in place
  for (int k0 = 0; k0 < n && e == cudaSuccess; k0 += kB) {
    const int nb = std::min(kB, n - k0), rest = n - k0 - nb;
    chol_diag_kernel<<<1, 256, 0, st>>>(A, n, k0, nb, mFail.as<int>());
    if ((e = cudaGetLastError()) != cudaSuccess) break;
    if (rest > 0) {
      chol_panel_kernel<<<(rest + kB - 1) / kB, kB, kTwoBlocksSmem, st>>>(A, n, k0, nb);
      if ((e = cudaGetLastError()) != cudaSuccess) break;
      const double* P = A + (size_t)(k0 + nb) * n + k0;  // panel [rest, nb]
      e = dgemm(rest, rest, nb, -1.0, P, (size_t)n, P, 1, (size_t)n, A + (size_t)(k0 + nb) * n + k0 + nb, (size_t)n, true, nullptr, false, st);
    }
  }
  if (e == cudaSuccess) {
    gather_rows_kernel<<<N, 256, 0, st>>>(dW, N, n, mSrc.as<int>(), mDead.as<unsigned char>(), mV.as<double>(), dS);
    e = cudaGetLastError();
  }
  // the sweep, from the last block to the first
  const int n_blocks = (n + kB - 1) / kB;
  for (int b = n_blocks - 1; b >= 0 && e == cudaSuccess; --b) {
    const int c0 = b * kB, c1 = std::min(n, c0 + kB), later = n - c1;
    const double* Vc = mV.as<double>();
    if (later > 0) {
      // Vc[:, blk] = V[:, blk] + D[:, c1:] L[c1:, blk] / diag(L)[blk]
      e = cudaMemcpy2DAsync(mVc.as<double>() + c0, sizeof(double) * (size_t)n, mV.as<double>() + c0, sizeof(double) * (size_t)n,
                            sizeof(double) * (size_t)(c1 - c0), (size_t)N, cudaMemcpyDeviceToDevice, st);
      if (e != cudaSuccess) break;
      // every column of the product is divided by its diagonal entry of the factor before it is added
      e = dgemm(N, c1 - c0, later, 1.0, mD.as<double>() + c1, (size_t)n, A + (size_t)c1 * n + c0, (size_t)n, 1, mVc.as<double>() + c0, (size_t)n,
                false, A + (size_t)c0 * n + c0, false, st);
      if (e != cudaSuccess) break;
      Vc = mVc.as<double>();
    }
    gptq_block_kernel<<<(N + kB - 1) / kB, kB, kTwoBlocksSmem, st>>>(mV.as<double>(), Vc, mD.as<double>(), A, dS, N, n, c0, c1, mQ.as<int8_t>());
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) {
    scatter_codes_kernel<<<grid_for((long long)N * n, 256), 256, 0, st>>>(mQ.as<int8_t>(), N, n, mSrc.as<int>(), dCodes);
    e = cudaGetLastError();
  }
  int fail = 0;
  if (e == cudaSuccess) e = cudaMemcpyAsync(&fail, mFail.p, sizeof(int), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  return fail ? XQ_ERR_INVALID_ARG : XQ_OK;  // a Hessian that is not positive definite after damping
}

}  // namespace

extern "C" {

xq_status xq_gptq_codes(const double* Wt_host, const double* H_host, int32_t N, int32_t Kp, double damp, int8_t* codes_host, float* s_w_host,
                        void* stream) {
  XQ_RANGE();
  if (!Wt_host || !H_host || !codes_host || !s_w_host || N < 1 || Kp < 1 || !(damp >= 0.0)) return XQ_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  DevMem mW, mH, mC, mS;
  const size_t nw = (size_t)N * Kp, nh = (size_t)Kp * Kp;
  if (mW.alloc(sizeof(double) * nw) != cudaSuccess || mH.alloc(sizeof(double) * nh) != cudaSuccess || mC.alloc(nw) != cudaSuccess ||
      mS.alloc(sizeof(float) * (size_t)N) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_ALLOC;
  }
  if (cudaMemcpyAsync(mW.p, Wt_host, sizeof(double) * nw, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(mH.p, H_host, sizeof(double) * nh, cudaMemcpyHostToDevice, st) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  const xq_status s = gptq_device(mW.as<double>(), mH.as<double>(), N, Kp, damp, mC.as<int8_t>(), mS.as<float>(), st);
  if (s != XQ_OK) return s;
  if (cudaMemcpyAsync(codes_host, mC.p, nw, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaMemcpyAsync(s_w_host, mS.p, sizeof(float) * (size_t)N, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  return XQ_OK;
}

xq_status xq_prepare_weights_gptq(const void* W_host, int32_t N, int32_t K, int32_t Kp, const double* H_host, double damp, void* stream,
                                  xq_weights** out) {
  XQ_RANGE();
  if (!W_host || !H_host || !out || N < 1 || K < 1 || Kp < K || !(damp >= 0.0)) return XQ_ERR_INVALID_ARG;
  xq_hadamard_plan_t pl;
  xq_status s = xq_hadamard_plan(K, Kp, &pl);
  if (s != XQ_OK) return s;
  if (Kp % 8 != 0) return XQ_ERR_UNSUPPORTED_ORDER;
  cudaStream_t st = (cudaStream_t)stream;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  // the rows of W through the same pad + rotate kernel as the round-to-nearest path, keeping the rotated values
  const int64_t ldw = ((int64_t)K + 7) / 8 * 8;
  const size_t nw = (size_t)N * Kp;
  DevMem mW, mXq, mSx, mY, mYd, mH, mC, mS;
  if (mW.alloc((size_t)N * ldw * 2) != cudaSuccess || mXq.alloc(nw / 2) != cudaSuccess || mSx.alloc(sizeof(float) * (size_t)N) != cudaSuccess ||
      mY.alloc(sizeof(float) * nw) != cudaSuccess || mYd.alloc(sizeof(double) * nw) != cudaSuccess ||
      mH.alloc(sizeof(double) * (size_t)Kp * Kp) != cudaSuccess || mC.alloc(nw) != cudaSuccess || mS.alloc(sizeof(float) * (size_t)N) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_ALLOC;
  }
  cudaError_t e = cudaMemsetAsync(mW.p, 0, (size_t)N * ldw * 2, st);
  if (e == cudaSuccess) e = cudaMemcpy2DAsync(mW.p, (size_t)ldw * 2, W_host, (size_t)K * 2, (size_t)K * 2, (size_t)N, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(mH.p, H_host, sizeof(double) * (size_t)Kp * Kp, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess)
    e = xq_launch_rotate_quant(mW.p, N, ldw, pl, mXq.as<uint8_t>(), mSx.as<float>(), mY.as<float>(), nullptr, nullptr, nullptr, sms, st);
  if (e == cudaSuccess) {
    f32_to_f64_kernel<<<grid_for((long long)nw, 256), 256, 0, st>>>(mY.as<float>(), (long long)nw, mYd.as<double>());
    e = cudaGetLastError();
  }
  if (e != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  s = gptq_device(mYd.as<double>(), mH.as<double>(), N, Kp, damp, mC.as<int8_t>(), mS.as<float>(), st);
  if (s != XQ_OK) return s;
  // codes and scales into a weights object, exactly as xq_weights_import does from host arrays
  std::vector<int8_t> codes(nw);
  std::vector<float> sw((size_t)N);
  if (cudaMemcpyAsync(codes.data(), mC.p, nw, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaMemcpyAsync(sw.data(), mS.p, sizeof(float) * (size_t)N, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  return xq_weights_import(codes.data(), sw.data(), N, K, Kp, stream, out);
}

}  // extern "C"
