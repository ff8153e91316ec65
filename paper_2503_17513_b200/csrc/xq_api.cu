// C-ABI entry points of libxq: argument checks, the Hadamard plan, weight objects, workspace
// bookkeeping.  Every step of the layer itself runs in the kernels of the other files.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <vector>

#include "xq_internal.h"

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool prime(int v) {
  if (v < 2) return false;
  for (int d = 2; (long long)d * d <= v; ++d)
    if (v % d == 0) return false;
  return true;
}

// Quadratic character of GF(q), q prime: 0 for 0, +1 for non-zero squares, -1 otherwise.
int host_chi(int a, int q) {
  a %= q;
  if (a < 0) a += q;
  if (a == 0) return 0;
  for (int i = 1; i <= (q - 1) / 2; ++i)
    if ((i * i) % q == a) return 1;
  return -1;
}

// Entry (a, a2) of the order-p Paley factor (the construction the device kernels use: Paley-I has a
// first row of +1, a first column of -1 below it and the core chi(i - j) + identity; Paley-II
// expands the symmetric conference matrix of order q + 1 into 2 x 2 blocks).
// Quadratic character of the field of 7^3 elements (polynomials over GF(7) modulo x^3 - 5, numbered a0 + 7 a1 + 49 a2):
// the non-zero squares are collected once.
int host_chi343(int d) {
  static const std::vector<int8_t> table = [] {
    std::vector<int8_t> t(343, -1);
    t[0] = 0;
    for (int a = 1; a < 343; ++a) {
      const int a0 = a % 7, a1 = (a / 7) % 7, a2 = a / 49;
      const int c0 = a0 * a0 + 10 * a1 * a2, c1 = 2 * a0 * a1 + 5 * a2 * a2, c2 = 2 * a0 * a2 + a1 * a1;
      t[c0 % 7 + 7 * (c1 % 7) + 49 * (c2 % 7)] = 1;
    }
    return t;
  }();
  return table[d];
}

int host_paley_sign(const xq_hadamard_plan_t& pl, int a, int a2) {
  const int q = pl.q;
  if (pl.paley_kind == 3) {  // Paley-I over GF(7^3)
    if (a == 0) return 1;
    if (a2 == 0) return -1;
    if (a == a2) return 1;
    const int i = a - 1, j = a2 - 1;
    int d = 0, w = 1;
    for (int k = 0; k < 3; ++k, w *= 7) d += (((i / w) % 7 - (j / w) % 7 + 7) % 7) * w;
    return host_chi343(d);
  }
  if (pl.paley_kind == 1) {
    if (a == 0) return 1;
    if (a2 == 0) return -1;
    return a == a2 ? 1 : host_chi(a - a2, q);
  }
  const int i = a >> 1, u = a & 1, j = a2 >> 1, v = a2 & 1;
  if (i == j) return (u | v) ? -1 : 1;
  const int s = (i == 0 || j == 0) ? 1 : host_chi(i - j, q);
  return (u & v) ? -s : s;
}

struct DevBuf {  // scoped device allocation for the offline calls
  void* p = nullptr;
  cudaError_t alloc(size_t bytes) { return cudaMalloc(&p, bytes ? bytes : 1); }
  ~DevBuf() {
    if (p) cudaFree(p);
  }
};

// heads == 1: one rotation K -> Kp.  heads > 1: K and Kp are the sizes of ONE head.
xq_status make_weights(int32_t N, int32_t K, int32_t Kp, xq_weights** out, int32_t heads = 1) {
  xq_hadamard_plan_t pl;
  xq_status st = xq_hadamard_plan(K, Kp, &pl);
  if (st != XQ_OK) return st;
  if (heads > 1) {
    if (!xq_rotate_heads_supported(pl, heads)) return XQ_ERR_UNSUPPORTED_ORDER;
    K *= heads;
    Kp *= heads;
  }
  if (Kp % 8 != 0) return XQ_ERR_UNSUPPORTED_ORDER;  // the GEMM kernels read whole 8-code words
  xq_weights* w = new (std::nothrow) xq_weights();
  if (!w) return XQ_ERR_ALLOC;
  w->N = N;
  w->K = K;
  w->Kp = Kp;
  w->Np = (int32_t)align_up((size_t)N, XQ_ROW_PAD);
  w->Kpp = (int32_t)align_up((size_t)Kp, XQ_K_BLOCK);
  w->plan = pl;
  w->heads = heads;
  w->head_signs = nullptr;
  w->packed = nullptr;
  w->s_w = nullptr;
  w->w_sum = nullptr;
  w->hp_signs = nullptr;
  if (cudaGetDevice(&w->device) != cudaSuccess ||
      cudaDeviceGetAttribute(&w->sms, cudaDevAttrMultiProcessorCount, w->device) != cudaSuccess) {
    delete w;
    return XQ_ERR_CUDA;
  }
  const size_t bytes = (size_t)w->Np * w->Kpp / 2;
  if (cudaMalloc((void**)&w->packed, bytes) != cudaSuccess ||
      cudaMalloc((void**)&w->s_w, sizeof(float) * (size_t)w->Np) != cudaSuccess ||
      cudaMalloc((void**)&w->w_sum, sizeof(int32_t) * (size_t)w->Np) != cudaSuccess) {
    cudaGetLastError();
    xq_weights_free(w);
    return XQ_ERR_ALLOC;
  }
  if (heads > 1) {
    if (!xq_make_head_signs(pl, &w->head_signs)) {
      cudaGetLastError();
      xq_weights_free(w);
      return XQ_ERR_ALLOC;
    }
  } else if (!xq_make_hp_signs(pl, &w->hp_signs)) {
    cudaGetLastError();
    xq_weights_free(w);
    return XQ_ERR_ALLOC;
  }
  *out = w;
  return XQ_OK;
}

}  // namespace

bool xq_make_head_signs(const xq_hadamard_plan_t& pl, uint16_t** out) {
  *out = nullptr;
  const int d16 = (pl.K + 15) / 16 * 16, pitch = d16 + 8, n = 1 << pl.log2n;
  const size_t elems = xq_head_image_elems(pl);
  uint16_t* img = (uint16_t*)calloc(elems, sizeof(uint16_t));
  if (!img) return false;
  for (int c2 = 0; c2 < pl.Kp; ++c2)
    for (int c = 0; c < pl.K; ++c) {
      int s = (__builtin_popcount((c & (n - 1)) & (c2 & (n - 1))) & 1) ? -1 : 1;
      if (pl.p > 1) s *= host_paley_sign(pl, c >> pl.log2n, c2 >> pl.log2n);
      img[(size_t)c2 * pitch + c] = s > 0 ? 0x3F80 : 0xBF80;
    }
  const bool ok = cudaMalloc((void**)out, elems * sizeof(uint16_t)) == cudaSuccess &&
                  cudaMemcpy(*out, img, elems * sizeof(uint16_t), cudaMemcpyHostToDevice) == cudaSuccess;
  free(img);
  if (!ok && *out) {
    cudaFree(*out);
    *out = nullptr;
  }
  return ok;
}

bool xq_make_hp_signs(const xq_hadamard_plan_t& pl, uint16_t** out) {
  *out = nullptr;
  if (pl.p <= 1 || pl.p > XQ_MAX_P_IMAGE) return true;  // no image: the kernels that read one do not take this plan
  const int P16 = (pl.p + 15) / 16 * 16, pitch = P16 + 8;
  uint16_t* img = (uint16_t*)calloc((size_t)P16 * pitch, sizeof(uint16_t));
  if (!img) return false;
  for (int a2 = 0; a2 < pl.p; ++a2)
    for (int a = 0; a < pl.p; ++a) img[(size_t)a2 * pitch + a] = host_paley_sign(pl, a, a2) > 0 ? 0x3F80 : 0xBF80;
  const size_t img_bytes = (size_t)P16 * pitch * sizeof(uint16_t);
  const bool ok = cudaMalloc((void**)out, img_bytes) == cudaSuccess && cudaMemcpy(*out, img, img_bytes, cudaMemcpyHostToDevice) == cudaSuccess;
  free(img);
  if (!ok && *out) {
    cudaFree(*out);
    *out = nullptr;
  }
  return ok;
}

xq_ws_layout xq_ws_compute(int32_t M_max, const xq_weights* w) {
  xq_ws_layout L;
  size_t off = 0;
  L.header = off;
  off += XQ_WS_HEADER_BYTES;
  L.xq = off;
  off += align_up((size_t)M_max * (size_t)(w->Kpp / 2), 256);
  L.sx = off;
  off += align_up(sizeof(float) * (size_t)M_max, 256);
  L.zp = off;
  off += align_up(sizeof(int32_t) * (size_t)M_max, 256);
  L.xstage = off;
  off += align_up((size_t)M_max * (size_t)w->K * 2, 256);
  L.ostage = off;
  off += align_up((size_t)M_max * (size_t)w->N * 2, 256);
  L.a8 = 0;
  if (M_max > XQ_DECODE_MAX_M) {
    L.a8 = off;
    off += align_up((size_t)M_max * (size_t)w->Kp, 256);
  }
  L.total = off;
  return L;
}

extern "C" {

const char* xq_status_string(xq_status s) {
  switch (s) {
    case XQ_OK: return "ok";
    case XQ_ERR_INVALID_ARG: return "invalid argument";
    case XQ_ERR_UNSUPPORTED_ORDER: return "unsupported Hadamard order";
    case XQ_ERR_WORKSPACE: return "workspace missing or too small";
    case XQ_ERR_ALLOC: return "allocation failed";
    case XQ_ERR_CUDA: return "CUDA error";
    case XQ_ERR_TIMEOUT: return "device-side wait timed out";
    case XQ_ERR_BOUNDS: return "device-side bounds check failed";
  }
  return "unknown status";
}

xq_status xq_hadamard_plan(int32_t K, int32_t Kp, xq_hadamard_plan_t* out) {
  if (!out || K < 1 || Kp < K) return XQ_ERR_INVALID_ARG;
  if (Kp > 1 && (Kp & 1)) return XQ_ERR_INVALID_ARG;
  int odd = Kp, twos = 0;
  while (!(odd & 1)) {
    odd >>= 1;
    ++twos;
  }
  xq_hadamard_plan_t pl = {K, Kp, 1, twos, 0, 0};
  if (odd > 1) {
    bool found = false;
    for (int j = 2; j <= twos && !found; ++j) {
      const long long p = (long long)odd << j;
      if (p > XQ_MAX_P) break;
      const int q1 = (int)p - 1, q2 = (int)p / 2 - 1;
      if (prime(q1) && q1 % 4 == 3) {
        pl.p = (int)p; pl.log2n = twos - j; pl.paley_kind = 1; pl.q = q1;
        found = true;
      } else if (prime(q2) && q2 % 4 == 1) {
        pl.p = (int)p; pl.log2n = twos - j; pl.paley_kind = 2; pl.q = q2;
        found = true;
      } else if (q1 == 343) {  // 7^3 = 3 mod 4: Paley-I over the field of 343 elements
        pl.p = (int)p; pl.log2n = twos - j; pl.paley_kind = 3; pl.q = 343;
        found = true;
      }
    }
    if (!found) return XQ_ERR_UNSUPPORTED_ORDER;
    // orders beyond the specialised kernels run in the general one: a row and its image in shared memory
    if (pl.p > XQ_MAX_P_IMAGE && 8 * (size_t)Kp + 3 * (size_t)pl.q + 256 > 227 * 1024) return XQ_ERR_UNSUPPORTED_ORDER;
  }
  *out = pl;
  return XQ_OK;
}

void xq_weights_free(xq_weights* w) {
  if (!w) return;
  if (w->packed) cudaFree(w->packed);
  if (w->s_w) cudaFree(w->s_w);
  if (w->w_sum) cudaFree(w->w_sum);
  if (w->hp_signs) cudaFree(w->hp_signs);
  if (w->head_signs) cudaFree(w->head_signs);
  delete w;
}

xq_status xq_weights_info(const xq_weights* w, int32_t* N, int32_t* K, int32_t* Kp, xq_hadamard_plan_t* plan) {
  if (!w) return XQ_ERR_INVALID_ARG;
  if (N) *N = w->N;
  if (K) *K = w->K;
  if (Kp) *Kp = w->Kp;
  if (plan) *plan = w->plan;
  return XQ_OK;
}

}  // extern "C"

namespace {

// heads == 1: K -> Kp over the whole row; heads > 1: K, Kp are one head's sizes.
xq_status prepare_impl(const void* W_host, int32_t N, int32_t heads, int32_t K, int32_t Kp, void* stream, xq_weights** out) {
  if (!W_host || !out || N < 1 || K < 1 || Kp < K || heads < 1) return XQ_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  xq_weights* w = nullptr;
  xq_status s = make_weights(N, K, Kp, &w, heads);
  if (s != XQ_OK) return s;
  K = w->K;
  Kp = w->Kp;
  // Rows of W go through the same pad + rotate + quantize kernel as activation rows (both
  // operands receive the map v -> [v, 0] H / sqrt(K')), then into the block layout.
  const int64_t ldw = (int64_t)align_up((size_t)K, 8);
  DevBuf dW, dCanon;
  if (dW.alloc((size_t)N * ldw * 2) != cudaSuccess || dCanon.alloc((size_t)N * (Kp / 2)) != cudaSuccess) {
    cudaGetLastError();
    xq_weights_free(w);
    return XQ_ERR_ALLOC;
  }
  cudaError_t e = cudaMemcpy2DAsync(dW.p, (size_t)ldw * 2, W_host, (size_t)K * 2, (size_t)K * 2, (size_t)N,
                                    cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(w->s_w, 0, sizeof(float) * (size_t)w->Np, st);
  if (e == cudaSuccess) e = xq_launch_rotate_for(w, dW.p, N, ldw, (uint8_t*)dCanon.p, w->s_w, nullptr, nullptr, st);
  if (e == cudaSuccess)
    e = xq_launch_relayout_to_blocks((const uint8_t*)dCanon.p, N, Kp, w->packed, w->Np, w->Kpp, st);
  if (e == cudaSuccess) e = xq_launch_weight_sums(w->packed, w->Np, w->Kpp, w->w_sum, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) {
    cudaGetLastError();
    xq_weights_free(w);
    return XQ_ERR_CUDA;
  }
  *out = w;
  return XQ_OK;
}

}  // namespace

extern "C" {

xq_status xq_prepare_weights(const void* W_host, int32_t N, int32_t K, int32_t Kp, void* stream, xq_weights** out) {
  XQ_RANGE();
  return prepare_impl(W_host, N, 1, K, Kp, stream, out);
}

xq_status xq_prepare_weights_heads(const void* W_host, int32_t N, int32_t heads, int32_t head_dim, int32_t head_dim_p,
                                   void* stream, xq_weights** out) {
  XQ_RANGE();
  if (heads < 2) return XQ_ERR_INVALID_ARG;
  return prepare_impl(W_host, N, heads, head_dim, head_dim_p, stream, out);
}

int32_t xq_weights_heads(const xq_weights* w) { return w ? w->heads : 0; }

xq_status xq_weights_import(const int8_t* codes, const float* s_w, int32_t N, int32_t K, int32_t Kp,
                            void* stream, xq_weights** out) {
  XQ_RANGE();
  if (!codes || !s_w || !out || N < 1 || K < 1 || Kp < K) return XQ_ERR_INVALID_ARG;
  const size_t count = (size_t)N * Kp;
  for (size_t i = 0; i < count; ++i)
    if (codes[i] < -8 || codes[i] > 7) return XQ_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  xq_weights* w = nullptr;
  xq_status s = make_weights(N, K, Kp, &w);
  if (s != XQ_OK) return s;
  DevBuf dCodes, dCanon;
  if (dCodes.alloc(count) != cudaSuccess || dCanon.alloc(count / 2) != cudaSuccess) {
    cudaGetLastError();
    xq_weights_free(w);
    return XQ_ERR_ALLOC;
  }
  cudaError_t e = cudaMemcpyAsync(dCodes.p, codes, count, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(w->s_w, 0, sizeof(float) * (size_t)w->Np, st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(w->s_w, s_w, sizeof(float) * (size_t)N, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = xq_launch_pack_codes((const int8_t*)dCodes.p, (int64_t)(count / 2), (uint8_t*)dCanon.p, st);
  if (e == cudaSuccess)
    e = xq_launch_relayout_to_blocks((const uint8_t*)dCanon.p, N, Kp, w->packed, w->Np, w->Kpp, st);
  if (e == cudaSuccess) e = xq_launch_weight_sums(w->packed, w->Np, w->Kpp, w->w_sum, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) {
    cudaGetLastError();
    xq_weights_free(w);
    return XQ_ERR_CUDA;
  }
  *out = w;
  return XQ_OK;
}

xq_status xq_weights_export(const xq_weights* w, int8_t* codes, float* s_w) {
  XQ_RANGE();
  if (!w || !codes || !s_w || !xq_on_device(w->device)) return XQ_ERR_INVALID_ARG;
  const size_t count = (size_t)w->N * w->Kp;
  DevBuf dCodes, dCanon;
  if (dCodes.alloc(count) != cudaSuccess || dCanon.alloc(count / 2) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_ALLOC;
  }
  cudaStream_t st = nullptr;
  cudaError_t e = xq_launch_relayout_from_blocks(w->packed, w->Np, w->Kpp, (uint8_t*)dCanon.p, w->N, w->Kp, st);
  if (e == cudaSuccess) e = xq_launch_unpack_codes((const uint8_t*)dCanon.p, (int64_t)(count / 2), (int8_t*)dCodes.p, st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(codes, dCodes.p, count, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(s_w, w->s_w, sizeof(float) * (size_t)w->N, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  return XQ_OK;
}

size_t xq_workspace_bytes(int32_t M_max, const xq_weights* w) {
  if (!w || M_max < 1) return 0;
  return xq_ws_compute(M_max, w).total;
}

xq_status xq_workspace_init(void* ws, size_t ws_bytes, void* stream) {
  if (!ws || ws_bytes < XQ_WS_HEADER_BYTES || !aligned16(ws)) return XQ_ERR_WORKSPACE;
  // the status word, and the arrival counters that the MXFP4 workspaces keep behind it
  const size_t clear = ws_bytes < XQ_WS_COUNTER_BYTES ? XQ_WS_HEADER_BYTES : XQ_WS_COUNTER_BYTES;
  if (cudaMemsetAsync(ws, 0, clear, (cudaStream_t)stream) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  return XQ_OK;
}

}  // extern "C"

namespace {

// asym: zp is required and receives the zero points; otherwise zp must be null.
xq_status rotate_quant_impl(const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t* plan, uint8_t* Xq, float* s_x,
                            int32_t* zp, bool asym, float* Yopt, void* stream, int32_t heads = 1) {
  if (!plan || M < 0 || heads < 1) return XQ_ERR_INVALID_ARG;
  if (M == 0) return XQ_OK;
  if (!X || !Xq || !s_x || (asym && !zp)) return XQ_ERR_INVALID_ARG;
  if (zp && (reinterpret_cast<uintptr_t>(zp) & 3u)) return XQ_ERR_INVALID_ARG;
  // the plan must be one xq_hadamard_plan would return
  xq_hadamard_plan_t chk;
  xq_status s = xq_hadamard_plan(plan->K, plan->Kp, &chk);
  if (s != XQ_OK) return s;
  if (memcmp(&chk, plan, sizeof(chk)) != 0) return XQ_ERR_INVALID_ARG;
  if (ldx < (int64_t)heads * plan->K || (ldx % 8) != 0) return XQ_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(Xq) || (reinterpret_cast<uintptr_t>(s_x) & 3u) ||
      (Yopt && !aligned16(Yopt)))
    return XQ_ERR_INVALID_ARG;
  if (heads > 1 && !xq_rotate_heads_supported(*plan, heads)) return XQ_ERR_UNSUPPORTED_ORDER;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  const cudaError_t e =
      heads > 1 ? xq_launch_rotate_heads(X, M, ldx, *plan, heads, Xq, s_x, Yopt, nullptr, nullptr, zp, sms, (cudaStream_t)stream)
                : xq_launch_rotate_quant(X, M, ldx, *plan, Xq, s_x, Yopt, nullptr, nullptr, zp, sms, (cudaStream_t)stream);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  return XQ_OK;
}

xq_status gemm_impl(const uint8_t* Xq, const float* s_x, const int32_t* zp, bool asym, int32_t M, const xq_weights* w, void* out,
                    int32_t* acc_opt, void* ws, size_t ws_bytes, void* stream) {
  if (!w || M < 0) return XQ_ERR_INVALID_ARG;
  if (M == 0) return XQ_OK;
  if (!Xq || !s_x || !out || (asym && !zp) || !xq_on_device(w->device)) return XQ_ERR_INVALID_ARG;
  if (zp && (reinterpret_cast<uintptr_t>(zp) & 3u)) return XQ_ERR_INVALID_ARG;
  if (!aligned16(Xq) || !aligned16(out) || (reinterpret_cast<uintptr_t>(s_x) & 3u) ||
      (acc_opt && !aligned16(acc_opt)))
    return XQ_ERR_INVALID_ARG;
  const xq_ws_layout L = xq_ws_compute(M, w);
  if (!ws || !aligned16(ws) || ws_bytes < L.total) return XQ_ERR_WORKSPACE;
  if (xq_launch_gemm(Xq, s_x, zp, M, w, out, acc_opt, ws, L, false, (cudaStream_t)stream) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  return XQ_OK;
}

// one_launch: the form for M <= 32 tokens with the online step inside the product kernel (UNSUPPORTED_ORDER when the
// plan or the shape is not one it takes); otherwise the rotate + quantize kernel followed by the product kernel.
xq_status linear_impl(const void* X, int32_t M, int64_t ldx, const xq_weights* w, bool asym, void* out, void* ws,
                      size_t ws_bytes, void* stream, bool one_launch = false) {
  if (!w || M < 0) return XQ_ERR_INVALID_ARG;
  if (M == 0) return XQ_OK;
  if (!X || !out || !xq_on_device(w->device)) return XQ_ERR_INVALID_ARG;
  if (ldx < w->K || (ldx % 8) != 0 || !aligned16(X) || !aligned16(out)) return XQ_ERR_INVALID_ARG;
  const xq_ws_layout L = xq_ws_compute(M, w);
  if (!ws || !aligned16(ws) || ws_bytes < L.total) return XQ_ERR_WORKSPACE;
  uint8_t* base = (uint8_t*)ws;
  uint8_t* Xq = base + L.xq;
  float* sx = (float*)(base + L.sx);
  int32_t* zp = asym ? (int32_t*)(base + L.zp) : nullptr;
  cudaStream_t st = (cudaStream_t)stream;
  if (one_launch) {
    const cudaError_t e = xq_launch_linear_decode(X, ldx, Xq, sx, zp, M, w, out, (int32_t*)ws, st);
    if (e == cudaSuccess) return XQ_OK;
    cudaGetLastError();
    return e == cudaErrorNotSupported ? XQ_ERR_UNSUPPORTED_ORDER : XQ_ERR_CUDA;
  }
  uint8_t* A8 = xq_gemm_wants_a8(M, w) ? base + L.a8 : nullptr;
  if (xq_launch_rotate_for(w, X, M, ldx, Xq, sx, A8, zp, st) != cudaSuccess ||
      xq_launch_gemm(Xq, sx, zp, M, w, out, nullptr, ws, L, A8 != nullptr, st) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  return XQ_OK;
}

}  // namespace

extern "C" {

xq_status xq_rotate_quant(const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t* plan, uint8_t* Xq,
                          float* s_x, float* Yopt, void* stream) {
  XQ_RANGE();
  return rotate_quant_impl(X, M, ldx, plan, Xq, s_x, nullptr, false, Yopt, stream);
}

xq_status xq_rotate_quant_asym(const void* X, int32_t M, int64_t ldx, const xq_hadamard_plan_t* plan, uint8_t* Xq,
                               float* s_x, int32_t* zp, float* Yopt, void* stream) {
  XQ_RANGE();
  return rotate_quant_impl(X, M, ldx, plan, Xq, s_x, zp, true, Yopt, stream);
}

xq_status xq_rotate_quant_heads(const void* X, int32_t M, int64_t ldx, int32_t heads, const xq_hadamard_plan_t* head_plan,
                                uint8_t* Xq, float* s_x, int32_t* zp_opt, float* Yopt, void* stream) {
  XQ_RANGE();
  if (heads < 2) return XQ_ERR_INVALID_ARG;
  return rotate_quant_impl(X, M, ldx, head_plan, Xq, s_x, zp_opt, zp_opt != nullptr, Yopt, stream, heads);
}

xq_status xq_w4a4_gemm(const uint8_t* Xq, const float* s_x, int32_t M, const xq_weights* w, void* out,
                       int32_t* acc_opt, void* ws, size_t ws_bytes, void* stream) {
  XQ_RANGE();
  return gemm_impl(Xq, s_x, nullptr, false, M, w, out, acc_opt, ws, ws_bytes, stream);
}

xq_status xq_w4a4_gemm_asym(const uint8_t* Xq, const float* s_x, const int32_t* zp, int32_t M, const xq_weights* w,
                            void* out, int32_t* acc_opt, void* ws, size_t ws_bytes, void* stream) {
  XQ_RANGE();
  return gemm_impl(Xq, s_x, zp, true, M, w, out, acc_opt, ws, ws_bytes, stream);
}

xq_status xq_expanded_linear(const void* X, int32_t M, int64_t ldx, const xq_weights* w, void* out, void* ws,
                             size_t ws_bytes, void* stream) {
  XQ_RANGE();
  return linear_impl(X, M, ldx, w, false, out, ws, ws_bytes, stream);
}

xq_status xq_expanded_linear_asym(const void* X, int32_t M, int64_t ldx, const xq_weights* w, void* out, void* ws,
                                  size_t ws_bytes, void* stream) {
  XQ_RANGE();
  return linear_impl(X, M, ldx, w, true, out, ws, ws_bytes, stream);
}

xq_status xq_expanded_linear_one_launch(const void* X, int32_t M, int64_t ldx, const xq_weights* w, int32_t asym, void* out,
                                        void* ws, size_t ws_bytes, void* stream) {
  XQ_RANGE();
  return linear_impl(X, M, ldx, w, asym != 0, out, ws, ws_bytes, stream, true);
}

}  // extern "C"

namespace {

xq_status linear_host_impl(const void* X_host, int32_t M, const xq_weights* w, bool asym, void* out_host, void* ws,
                           size_t ws_bytes, void* stream, bool sync = true) {
  if (!w || M < 0) return XQ_ERR_INVALID_ARG;
  if (M == 0) return XQ_OK;
  if (!X_host || !out_host || !xq_on_device(w->device)) return XQ_ERR_INVALID_ARG;
  const xq_ws_layout L = xq_ws_compute(M, w);
  if (!ws || !aligned16(ws) || ws_bytes < L.total) return XQ_ERR_WORKSPACE;
  uint8_t* base = (uint8_t*)ws;
  cudaStream_t st = (cudaStream_t)stream;
  // staged rows must stay 16-byte aligned at pitch K
  if (w->K % 8 != 0) return XQ_ERR_INVALID_ARG;
  const int64_t ldx = w->K;
  cudaError_t e = cudaMemcpyAsync(base + L.xstage, X_host, (size_t)M * w->K * 2, cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  xq_status s = linear_impl(base + L.xstage, M, ldx, w, asym, base + L.ostage, ws, ws_bytes, stream);
  if (s != XQ_OK) return s;
  e = cudaMemcpyAsync(out_host, base + L.ostage, (size_t)M * w->N * 2, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess && sync) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  return XQ_OK;
}

}  // namespace

extern "C" {

xq_status xq_expanded_linear_host(const void* X_host, int32_t M, const xq_weights* w, void* out_host, void* ws,
                                  size_t ws_bytes, void* stream) {
  XQ_RANGE();
  return linear_host_impl(X_host, M, w, false, out_host, ws, ws_bytes, stream);
}

xq_status xq_expanded_linear_host_asym(const void* X_host, int32_t M, const xq_weights* w, void* out_host, void* ws,
                                       size_t ws_bytes, void* stream) {
  XQ_RANGE();
  return linear_host_impl(X_host, M, w, true, out_host, ws, ws_bytes, stream);
}

xq_status xq_expanded_linear_host_enqueue(const void* X_host, int32_t M, const xq_weights* w, void* out_host, void* ws,
                                          size_t ws_bytes, void* stream) {
  XQ_RANGE();
  return linear_host_impl(X_host, M, w, false, out_host, ws, ws_bytes, stream, false);
}

xq_status xq_selftest_wait_timeout(void* ws, size_t ws_bytes, void* stream) {
  if (!ws || ws_bytes < XQ_WS_HEADER_BYTES || !aligned16(ws)) return XQ_ERR_WORKSPACE;
  if (xq_launch_selftest_wait_timeout((int32_t*)ws, (cudaStream_t)stream) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  return XQ_OK;
}

xq_status xq_selftest_i8_mma_rate(int32_t iters, void* ws, size_t ws_bytes, void* stream, double* ops_out) {
  if (!ws || ws_bytes < XQ_WS_HEADER_BYTES || !aligned16(ws)) return XQ_ERR_WORKSPACE;
  if (iters < 1 || iters > (1 << 22)) return XQ_ERR_INVALID_ARG;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  if (xq_launch_i8_mma_rate(iters, (int32_t*)ws, sms, (cudaStream_t)stream) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  if (ops_out) *ops_out = (double)sms * iters * 4.0 * 2.0 * 128.0 * 256.0 * 32.0;
  return XQ_OK;
}

xq_status xq_poll_status(const void* ws, void* stream) {
  if (!ws) return XQ_ERR_WORKSPACE;
  int32_t word = 0;
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = cudaMemcpyAsync(&word, ws, sizeof(word), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  if (word == XQ_ERR_TIMEOUT) return XQ_ERR_TIMEOUT;
  if (word != 0) return XQ_ERR_BOUNDS;
  return XQ_OK;
}

}  // extern "C"
