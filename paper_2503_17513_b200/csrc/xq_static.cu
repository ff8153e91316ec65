// Allocation-free variant of the whole layer: the quantized activations, their scales and the
// status word -- what xq_expanded_linear keeps in the caller's workspace -- live in one fixed
// array in device memory that is part of the library image.
#include <mutex>

#include "xq_internal.h"

namespace {

constexpr size_t kStaticScratchBytes = XQ_STATIC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

// Every GPU that loads the library holds this array until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_addr_mutex;
unsigned char* g_scratch_addr[kMaxDevices] = {};

inline size_t round256(size_t v) { return (v + 255) / 256 * 256; }

// Device address of the array on the current device.  The symbol name itself is only a host-side
// handle, so the address is asked from the runtime, once per device, with that device current.
xq_status scratch_address(unsigned char** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  if (dev < 0 || dev >= kMaxDevices) return XQ_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_addr_mutex);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return XQ_ERR_CUDA;
    }
    g_scratch_addr[dev] = (unsigned char*)p;
  }
  *out = g_scratch_addr[dev];
  return XQ_OK;
}

}  // namespace

extern "C" xq_status xq_expanded_linear_static(const void* X, int32_t M, int64_t ldx, const xq_weights* w, void* out,
                                               void* stream) {
  XQ_RANGE();
  if (!w || M < 0) return XQ_ERR_INVALID_ARG;
  if (M == 0) return XQ_OK;
  if (!X || !out || !xq_on_device(w->device)) return XQ_ERR_INVALID_ARG;
  if (ldx < w->K || (ldx % 8) != 0 || (reinterpret_cast<uintptr_t>(X) & 15u) || (reinterpret_cast<uintptr_t>(out) & 15u))
    return XQ_ERR_INVALID_ARG;
  // [status header | packed codes M x K'/2 | scales M | byte-per-code tokens M x K' when M > 32]
  const size_t off_xq = XQ_WS_HEADER_BYTES;
  const size_t off_sx = off_xq + round256((size_t)M * (size_t)(w->Kp / 2));
  const size_t off_a8 = off_sx + round256(sizeof(float) * (size_t)M);
  const size_t need = off_a8 + (M > XQ_DECODE_MAX_M ? round256((size_t)M * (size_t)w->Kp) : 0);
  if (need > kStaticScratchBytes) return XQ_ERR_WORKSPACE;
  unsigned char* base = nullptr;
  const xq_status s = scratch_address(&base);
  if (s != XQ_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  // the array keeps whatever the last call left: the status word has to start at zero
  if (cudaMemsetAsync(base, 0, XQ_WS_HEADER_BYTES, st) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  uint8_t* Xq = base + off_xq;
  float* sx = (float*)(base + off_sx);
  xq_ws_layout L = {};
  L.xq = off_xq;
  L.sx = off_sx;
  L.a8 = M > XQ_DECODE_MAX_M ? off_a8 : 0;
  L.total = need;
  uint8_t* A8 = xq_gemm_wants_a8(M, w) ? base + off_a8 : nullptr;
  if (xq_launch_rotate_for(w, X, M, ldx, Xq, sx, A8, nullptr, st) != cudaSuccess ||
      xq_launch_gemm(Xq, sx, nullptr, M, w, out, nullptr, base, L, A8 != nullptr, st) != cudaSuccess) {
    cudaGetLastError();
    return XQ_ERR_CUDA;
  }
  return XQ_OK;
}
