"""Thin binding over the C-ABI library ``libxq.so``: argument marshalling only.

Function names match ``include/xq.h``.  Tensors are torch CUDA tensors used purely as device
memory (their ``data_ptr()`` is what crosses the boundary); bf16 data may be passed either as
``torch.bfloat16`` or as 16-bit integer bit patterns.  There is no fallback: a missing library
raises at first use.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# XQ_LIBRARY names another build of the same library (the self-checking one, see build.py) to load instead
LIB_PATH = os.environ.get("XQ_LIBRARY") or os.path.join(_PKG, "libxq.so")
_lib = None

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED_ORDER, ERR_WORKSPACE, ERR_ALLOC, ERR_CUDA, ERR_TIMEOUT, ERR_BOUNDS = range(8)


class XqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (xq_status {status})")


class HadamardPlan(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("K", "Kp", "p", "log2n", "paley_kind", "q")]

    def astuple(self):
        return (self.K, self.Kp, self.p, self.log2n, self.paley_kind, self.q)


EXPORTS = [
    "xq_status_string", "xq_hadamard_plan", "xq_prepare_weights", "xq_weights_import", "xq_weights_export",
    "xq_weights_info", "xq_weights_free", "xq_workspace_bytes", "xq_workspace_init", "xq_rotate_quant",
    "xq_w4a4_gemm", "xq_expanded_linear", "xq_expanded_linear_host", "xq_poll_status", "xq_expanded_linear_static",
    "xq_selftest_wait_timeout", "xq_rotate_quant_asym", "xq_w4a4_gemm_asym", "xq_expanded_linear_asym",
    "xq_expanded_linear_host_asym", "xq_rotate_quant_heads", "xq_prepare_weights_heads", "xq_weights_heads",
    "xq_mx_prepare_weights", "xq_mx_weights_import", "xq_mx_weights_export", "xq_mx_weights_info", "xq_mx_weights_free",
    "xq_mx_workspace_bytes", "xq_mx_rotate_quant", "xq_mx_gemm", "xq_mx_expanded_linear",
    "xq_mx_expanded_linear_host", "xq_mx_gemm_staged", "xq_mx_rotate_quant_staged",
    "xq_mx_prepare_weights_heads", "xq_mx_weights_heads", "xq_gemm_kernel_info", "xq_selftest_i8_mma_rate", "xq_expanded_linear_host_enqueue", "xq_expanded_linear_one_launch", "xq_prepare_weights_gptq", "xq_gptq_codes",
]


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2503_17513_b200.build` "
                "(there is no non-CUDA fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
        L.xq_status_string.restype = ctypes.c_char_p
        L.xq_status_string.argtypes = [ctypes.c_int]
        L.xq_hadamard_plan.argtypes = [i32, i32, ctypes.POINTER(HadamardPlan)]
        L.xq_prepare_weights.argtypes = [vp, i32, i32, i32, vp, ctypes.POINTER(vp)]
        L.xq_weights_import.argtypes = [vp, vp, i32, i32, i32, vp, ctypes.POINTER(vp)]
        L.xq_prepare_weights_gptq.argtypes = [vp, i32, i32, i32, vp, ctypes.c_double, vp, ctypes.POINTER(vp)]
        L.xq_gptq_codes.argtypes = [vp, vp, i32, i32, ctypes.c_double, vp, vp, vp]
        L.xq_weights_export.argtypes = [vp, vp, vp]
        L.xq_weights_info.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32),
                                      ctypes.POINTER(HadamardPlan)]
        L.xq_weights_free.argtypes = [vp]
        L.xq_weights_free.restype = None
        L.xq_workspace_bytes.argtypes = [i32, vp]
        L.xq_workspace_bytes.restype = sz
        L.xq_workspace_init.argtypes = [vp, sz, vp]
        L.xq_rotate_quant.argtypes = [vp, i32, i64, ctypes.POINTER(HadamardPlan), vp, vp, vp, vp]
        L.xq_w4a4_gemm.argtypes = [vp, vp, i32, vp, vp, vp, vp, sz, vp]
        L.xq_expanded_linear.argtypes = [vp, i32, i64, vp, vp, vp, sz, vp]
        L.xq_rotate_quant_asym.argtypes = [vp, i32, i64, ctypes.POINTER(HadamardPlan), vp, vp, vp, vp, vp]
        L.xq_w4a4_gemm_asym.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp, sz, vp]
        L.xq_expanded_linear_asym.argtypes = [vp, i32, i64, vp, vp, vp, sz, vp]
        L.xq_expanded_linear_one_launch.argtypes = [vp, i32, i64, vp, i32, vp, vp, sz, vp]
        L.xq_expanded_linear_host.argtypes = [vp, i32, vp, vp, vp, sz, vp]
        L.xq_expanded_linear_host_asym.argtypes = [vp, i32, vp, vp, vp, sz, vp]
        L.xq_expanded_linear_host_enqueue.argtypes = [vp, i32, vp, vp, vp, sz, vp]
        L.xq_rotate_quant_heads.argtypes = [vp, i32, i64, i32, ctypes.POINTER(HadamardPlan), vp, vp, vp, vp, vp]
        L.xq_prepare_weights_heads.argtypes = [vp, i32, i32, i32, i32, vp, ctypes.POINTER(vp)]
        L.xq_weights_heads.argtypes = [vp]
        L.xq_weights_heads.restype = i32
        L.xq_mx_prepare_weights.argtypes = [vp, i32, i32, i32, vp, ctypes.POINTER(vp)]
        L.xq_mx_weights_import.argtypes = [vp, vp, i32, i32, i32, vp, ctypes.POINTER(vp)]
        L.xq_mx_weights_export.argtypes = [vp, vp, vp]
        L.xq_mx_weights_info.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32),
                                         ctypes.POINTER(HadamardPlan)]
        L.xq_mx_weights_free.argtypes = [vp]
        L.xq_mx_weights_free.restype = None
        L.xq_mx_workspace_bytes.argtypes = [i32, vp]
        L.xq_mx_workspace_bytes.restype = sz
        L.xq_mx_rotate_quant.argtypes = [vp, i32, i64, ctypes.POINTER(HadamardPlan), vp, vp, vp, vp]
        L.xq_mx_gemm.argtypes = [vp, vp, i32, vp, vp, vp, sz, vp]
        L.xq_mx_expanded_linear.argtypes = [vp, i32, i64, vp, vp, vp, sz, vp]
        L.xq_mx_expanded_linear_host.argtypes = [vp, i32, vp, vp, vp, sz, vp]
        L.xq_mx_gemm_staged.argtypes = [i32, vp, vp, vp, sz, vp]
        L.xq_mx_rotate_quant_staged.argtypes = [vp, i32, i64, vp, vp, sz, vp]
        L.xq_mx_prepare_weights_heads.argtypes = [vp, i32, i32, i32, i32, vp, ctypes.POINTER(vp)]
        L.xq_mx_weights_heads.argtypes = [vp]
        L.xq_mx_weights_heads.restype = i32
        L.xq_poll_status.argtypes = [vp, vp]
        L.xq_expanded_linear_static.argtypes = [vp, i32, i64, vp, vp, vp]
        L.xq_selftest_wait_timeout.argtypes = [vp, sz, vp]
        L.xq_selftest_i8_mma_rate.argtypes = [i32, vp, sz, vp, ctypes.POINTER(ctypes.c_double)]
        L.xq_gemm_kernel_info.argtypes = [i32, vp, ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32)]
        for name in EXPORTS:
            if name not in ("xq_status_string", "xq_weights_free", "xq_workspace_bytes", "xq_weights_heads", "xq_mx_weights_free",
                            "xq_mx_workspace_bytes", "xq_mx_weights_heads"):
                getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().xq_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise XqError(status, where)


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _dp(t) -> ctypes.c_void_p:
    if t is None:
        return ctypes.c_void_p(0)
    assert t.is_cuda and t.is_contiguous()
    return ctypes.c_void_p(t.data_ptr())


def _hp(a: np.ndarray) -> ctypes.c_void_p:
    return a.ctypes.data_as(ctypes.c_void_p)


def xq_hadamard_plan(K: int, Kp: int) -> HadamardPlan:
    pl = HadamardPlan()
    _check(lib().xq_hadamard_plan(K, Kp, ctypes.byref(pl)), "xq_hadamard_plan")
    return pl


class Weights:
    """Owner of one ``xq_weights*`` (freed with the object)."""

    def __init__(self, handle: int):
        self.handle = ctypes.c_void_p(handle)
        n, k, kp, pl = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32(), HadamardPlan()
        _check(lib().xq_weights_info(self.handle, ctypes.byref(n), ctypes.byref(k), ctypes.byref(kp), ctypes.byref(pl)),
               "xq_weights_info")
        self.N, self.K, self.Kp, self.plan = n.value, k.value, kp.value, pl
        self.heads = int(lib().xq_weights_heads(self.handle))

    def free(self):
        if self.handle:
            lib().xq_weights_free(self.handle)
            self.handle = ctypes.c_void_p(0)

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def xq_prepare_weights(W_bf16_host: np.ndarray, Kp: int, stream=None) -> Weights:
    """W: host uint16 bf16 bit patterns [N, K] (out x in)."""
    W = np.ascontiguousarray(W_bf16_host, dtype=np.uint16)
    N, K = W.shape
    h = ctypes.c_void_p()
    _check(lib().xq_prepare_weights(_hp(W), N, K, Kp, _stream(stream), ctypes.byref(h)), "xq_prepare_weights")
    return Weights(h.value)


def xq_prepare_weights_gptq(W_bf16_host: np.ndarray, Kp: int, H_host: np.ndarray, damp: float = 0.01, stream=None) -> Weights:
    """W: host uint16 bf16 bit patterns [N, K]; H: host float64 [Kp, Kp], the Hessian of the rotated calibration activations."""
    W = np.ascontiguousarray(W_bf16_host, dtype=np.uint16)
    H = np.ascontiguousarray(H_host, dtype=np.float64)
    N, K = W.shape
    assert H.shape == (Kp, Kp)
    h = ctypes.c_void_p()
    _check(lib().xq_prepare_weights_gptq(_hp(W), N, K, Kp, _hp(H), float(damp), _stream(stream), ctypes.byref(h)), "xq_prepare_weights_gptq")
    return Weights(h.value)


def xq_gptq_codes(Wt_host: np.ndarray, H_host: np.ndarray, damp: float = 0.01, stream=None):
    """GPTQ with act-order on already rotated rows (host float64 [N, Kp]): returns (codes int8 [N, Kp], scales float32 [N])."""
    Wt = np.ascontiguousarray(Wt_host, dtype=np.float64)
    H = np.ascontiguousarray(H_host, dtype=np.float64)
    N, Kp = Wt.shape
    assert H.shape == (Kp, Kp)
    codes = np.empty((N, Kp), dtype=np.int8)
    s_w = np.empty((N,), dtype=np.float32)
    _check(lib().xq_gptq_codes(_hp(Wt), _hp(H), N, Kp, float(damp), _hp(codes), _hp(s_w), _stream(stream)), "xq_gptq_codes")
    return codes, s_w


def xq_prepare_weights_heads(W_bf16_host: np.ndarray, heads: int, head_dim_p: int, stream=None) -> Weights:
    """W: host uint16 bf16 bit patterns [N, heads * head_dim]; every head block is expanded to head_dim_p."""
    W = np.ascontiguousarray(W_bf16_host, dtype=np.uint16)
    N, K = W.shape
    assert K % heads == 0
    h = ctypes.c_void_p()
    _check(lib().xq_prepare_weights_heads(_hp(W), N, heads, K // heads, head_dim_p, _stream(stream), ctypes.byref(h)),
           "xq_prepare_weights_heads")
    return Weights(h.value)


def xq_rotate_quant_heads(X, heads: int, head_plan: HadamardPlan, Xq, s_x, zp=None, Y_f32=None, M=None, ldx=None, stream=None) -> None:
    M = X.shape[0] if M is None else M
    ldx = X.stride(0) if ldx is None else ldx
    _check(lib().xq_rotate_quant_heads(ctypes.c_void_p(X.data_ptr()), M, ldx, heads, ctypes.byref(head_plan), _dp(Xq), _dp(s_x),
                                       _dp(zp), _dp(Y_f32), _stream(stream)), "xq_rotate_quant_heads")


def xq_weights_import(codes_host: np.ndarray, s_w_host: np.ndarray, K: int, stream=None) -> Weights:
    codes = np.ascontiguousarray(codes_host, dtype=np.int8)
    s_w = np.ascontiguousarray(s_w_host, dtype=np.float32)
    N, Kp = codes.shape
    assert s_w.shape == (N,)
    h = ctypes.c_void_p()
    _check(lib().xq_weights_import(_hp(codes), _hp(s_w), N, K, Kp, _stream(stream), ctypes.byref(h)), "xq_weights_import")
    return Weights(h.value)


def xq_weights_export(w: Weights):
    codes = np.empty((w.N, w.Kp), dtype=np.int8)
    s_w = np.empty((w.N,), dtype=np.float32)
    _check(lib().xq_weights_export(w.handle, _hp(codes), _hp(s_w)), "xq_weights_export")
    return codes, s_w


def xq_workspace_bytes(M_max: int, w: Weights) -> int:
    return int(lib().xq_workspace_bytes(M_max, w.handle))


def xq_workspace_init(ws: torch.Tensor, stream=None) -> None:
    _check(lib().xq_workspace_init(_dp(ws), ws.numel() * ws.element_size(), _stream(stream)), "xq_workspace_init")


def new_workspace(M_max: int, w: Weights, device="cuda") -> torch.Tensor:
    """Allocate (with torch) and initialise a workspace for up to M_max tokens."""
    ws = torch.empty(xq_workspace_bytes(M_max, w), dtype=torch.uint8, device=device)
    xq_workspace_init(ws)
    return ws


def xq_rotate_quant(X, plan: HadamardPlan, Xq, s_x, Y_f32=None, M=None, ldx=None, stream=None) -> None:
    M = X.shape[0] if M is None else M
    ldx = X.stride(0) if ldx is None else ldx
    _check(lib().xq_rotate_quant(ctypes.c_void_p(X.data_ptr()), M, ldx, ctypes.byref(plan), _dp(Xq), _dp(s_x), _dp(Y_f32),
                                 _stream(stream)), "xq_rotate_quant")


def xq_w4a4_gemm(Xq, s_x, M: int, w: Weights, out, ws, acc=None, stream=None) -> None:
    _check(lib().xq_w4a4_gemm(_dp(Xq), _dp(s_x), M, w.handle, _dp(out), _dp(acc), _dp(ws), ws.numel() * ws.element_size(),
                              _stream(stream)), "xq_w4a4_gemm")


def xq_expanded_linear(X, w: Weights, out, ws, M=None, ldx=None, stream=None) -> None:
    M = X.shape[0] if M is None else M
    ldx = X.stride(0) if ldx is None else ldx
    _check(lib().xq_expanded_linear(ctypes.c_void_p(X.data_ptr()), M, ldx, w.handle, _dp(out), _dp(ws),
                                    ws.numel() * ws.element_size(), _stream(stream)), "xq_expanded_linear")


def xq_expanded_linear_one_launch(X, w: Weights, out, ws, asym=False, M=None, ldx=None, stream=None) -> None:
    M = X.shape[0] if M is None else M
    ldx = X.stride(0) if ldx is None else ldx
    _check(lib().xq_expanded_linear_one_launch(ctypes.c_void_p(X.data_ptr()), M, ldx, w.handle, int(bool(asym)), _dp(out), _dp(ws),
                                               ws.numel() * ws.element_size(), _stream(stream)), "xq_expanded_linear_one_launch")


def xq_rotate_quant_asym(X, plan: HadamardPlan, Xq, s_x, zp, Y_f32=None, M=None, ldx=None, stream=None) -> None:
    M = X.shape[0] if M is None else M
    ldx = X.stride(0) if ldx is None else ldx
    _check(lib().xq_rotate_quant_asym(ctypes.c_void_p(X.data_ptr()), M, ldx, ctypes.byref(plan), _dp(Xq), _dp(s_x), _dp(zp),
                                      _dp(Y_f32), _stream(stream)), "xq_rotate_quant_asym")


def xq_w4a4_gemm_asym(Xq, s_x, zp, M: int, w: Weights, out, ws, acc=None, stream=None) -> None:
    _check(lib().xq_w4a4_gemm_asym(_dp(Xq), _dp(s_x), _dp(zp), M, w.handle, _dp(out), _dp(acc), _dp(ws),
                                   ws.numel() * ws.element_size(), _stream(stream)), "xq_w4a4_gemm_asym")


def xq_expanded_linear_asym(X, w: Weights, out, ws, M=None, ldx=None, stream=None) -> None:
    M = X.shape[0] if M is None else M
    ldx = X.stride(0) if ldx is None else ldx
    _check(lib().xq_expanded_linear_asym(ctypes.c_void_p(X.data_ptr()), M, ldx, w.handle, _dp(out), _dp(ws),
                                         ws.numel() * ws.element_size(), _stream(stream)), "xq_expanded_linear_asym")


def xq_expanded_linear_host(X_host, w: Weights, out_host, ws, M=None, stream=None) -> None:
    """X_host / out_host: CPU tensors (pinned for asynchronous copies) of 16-bit elements."""
    M = X_host.shape[0] if M is None else M
    _check(lib().xq_expanded_linear_host(ctypes.c_void_p(X_host.data_ptr()), M, w.handle,
                                         ctypes.c_void_p(out_host.data_ptr()), _dp(ws), ws.numel() * ws.element_size(),
                                         _stream(stream)), "xq_expanded_linear_host")


def xq_expanded_linear_host_enqueue(X_host, w: Weights, out_host, ws, M=None, stream=None) -> None:
    """As xq_expanded_linear_host, but only enqueued: synchronize the stream before reading out_host."""
    M = X_host.shape[0] if M is None else M
    _check(lib().xq_expanded_linear_host_enqueue(ctypes.c_void_p(X_host.data_ptr()), M, w.handle,
                                                 ctypes.c_void_p(out_host.data_ptr()), _dp(ws), ws.numel() * ws.element_size(),
                                                 _stream(stream)), "xq_expanded_linear_host_enqueue")


def xq_expanded_linear_host_asym(X_host, w: Weights, out_host, ws, M=None, stream=None) -> None:
    M = X_host.shape[0] if M is None else M
    _check(lib().xq_expanded_linear_host_asym(ctypes.c_void_p(X_host.data_ptr()), M, w.handle,
                                              ctypes.c_void_p(out_host.data_ptr()), _dp(ws), ws.numel() * ws.element_size(),
                                              _stream(stream)), "xq_expanded_linear_host_asym")


def xq_expanded_linear_static(X, w: Weights, out, M=None, ldx=None, stream=None) -> None:
    """The layer without a caller workspace: intermediates live in the library's built-in 4 MiB
    device array (for callers that must not allocate).  Calls share that array: do not overlap them."""
    M = X.shape[0] if M is None else M
    ldx = X.stride(0) if ldx is None else ldx
    _check(lib().xq_expanded_linear_static(ctypes.c_void_p(X.data_ptr()), M, ldx, w.handle, _dp(out), _stream(stream)),
           "xq_expanded_linear_static")


def xq_selftest_wait_timeout(ws, stream=None) -> None:
    """Enqueue the self-test kernel whose bounded wait runs out after about a second."""
    _check(lib().xq_selftest_wait_timeout(_dp(ws), ws.numel() * ws.element_size(), _stream(stream)), "xq_selftest_wait_timeout")


def xq_gemm_kernel_info(M: int, w: Weights):
    """(kind, tile_tokens, tile_channels) of the product kernel that M tokens against w run in."""
    kind, tt, tc = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    _check(lib().xq_gemm_kernel_info(M, w.handle, ctypes.byref(kind), ctypes.byref(tt), ctypes.byref(tc)), "xq_gemm_kernel_info")
    return kind.value, tt.value, tc.value


def xq_selftest_i8_mma_rate(iters: int, ws, stream=None) -> float:
    """Enqueue the tensor-core issue-rate probe; returns the integer operations the launch performs."""
    ops = ctypes.c_double()
    _check(lib().xq_selftest_i8_mma_rate(iters, _dp(ws), ws.numel() * ws.element_size(), _stream(stream), ctypes.byref(ops)),
           "xq_selftest_i8_mma_rate")
    return ops.value


def xq_poll_status(ws, stream=None) -> int:
    return int(lib().xq_poll_status(_dp(ws), _stream(stream)))


# ---- MXFP4 form ------------------------------------------------------------------------------------

class MxWeights:
    """Owner of one ``xq_mx_weights*`` (freed with the object)."""

    def __init__(self, handle: int):
        self.handle = ctypes.c_void_p(handle)
        n, k, kp, pl = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32(), HadamardPlan()
        _check(lib().xq_mx_weights_info(self.handle, ctypes.byref(n), ctypes.byref(k), ctypes.byref(kp), ctypes.byref(pl)),
               "xq_mx_weights_info")
        self.N, self.K, self.Kp, self.plan = n.value, k.value, kp.value, pl
        self.heads = int(lib().xq_mx_weights_heads(self.handle))

    def free(self):
        if self.handle:
            lib().xq_mx_weights_free(self.handle)
            self.handle = ctypes.c_void_p(0)

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def xq_mx_prepare_weights(W_bf16_host: np.ndarray, Kp: int, stream=None) -> MxWeights:
    W = np.ascontiguousarray(W_bf16_host, dtype=np.uint16)
    N, K = W.shape
    h = ctypes.c_void_p()
    _check(lib().xq_mx_prepare_weights(_hp(W), N, K, Kp, _stream(stream), ctypes.byref(h)), "xq_mx_prepare_weights")
    return MxWeights(h.value)


def xq_mx_weights_import(codes_packed_host: np.ndarray, scales_host: np.ndarray, K: int, stream=None) -> MxWeights:
    codes = np.ascontiguousarray(codes_packed_host, dtype=np.uint8)
    sc = np.ascontiguousarray(scales_host, dtype=np.uint8)
    N, half = codes.shape
    assert sc.shape == (N, half // 16)
    h = ctypes.c_void_p()
    _check(lib().xq_mx_weights_import(_hp(codes), _hp(sc), N, K, 2 * half, _stream(stream), ctypes.byref(h)), "xq_mx_weights_import")
    return MxWeights(h.value)


def xq_mx_weights_export(w: MxWeights):
    codes = np.empty((w.N, w.Kp), dtype=np.uint8)
    sc = np.empty((w.N, w.Kp // 32), dtype=np.uint8)
    _check(lib().xq_mx_weights_export(w.handle, _hp(codes), _hp(sc)), "xq_mx_weights_export")
    return codes, sc


def new_mx_workspace(M_max: int, w: MxWeights, device="cuda") -> torch.Tensor:
    ws = torch.empty(int(lib().xq_mx_workspace_bytes(M_max, w.handle)), dtype=torch.uint8, device=device)
    xq_workspace_init(ws)
    return ws


def xq_mx_rotate_quant(X, plan: HadamardPlan, codes, scales, Y_f32, M=None, ldx=None, stream=None) -> None:
    M = X.shape[0] if M is None else M
    ldx = X.stride(0) if ldx is None else ldx
    _check(lib().xq_mx_rotate_quant(ctypes.c_void_p(X.data_ptr()), M, ldx, ctypes.byref(plan), _dp(codes), _dp(scales), _dp(Y_f32),
                                    _stream(stream)), "xq_mx_rotate_quant")


def xq_mx_gemm(codes, scales, M: int, w: MxWeights, out, ws, stream=None) -> None:
    _check(lib().xq_mx_gemm(_dp(codes), _dp(scales), M, w.handle, _dp(out), _dp(ws), ws.numel() * ws.element_size(), _stream(stream)),
           "xq_mx_gemm")


def xq_mx_expanded_linear(X, w: MxWeights, out, ws, M=None, ldx=None, stream=None) -> None:
    M = X.shape[0] if M is None else M
    ldx = X.stride(0) if ldx is None else ldx
    _check(lib().xq_mx_expanded_linear(ctypes.c_void_p(X.data_ptr()), M, ldx, w.handle, _dp(out), _dp(ws),
                                       ws.numel() * ws.element_size(), _stream(stream)), "xq_mx_expanded_linear")


def xq_mx_expanded_linear_host(X_host, w: MxWeights, out_host, ws, M=None, stream=None) -> None:
    M = X_host.shape[0] if M is None else M
    _check(lib().xq_mx_expanded_linear_host(ctypes.c_void_p(X_host.data_ptr()), M, w.handle, ctypes.c_void_p(out_host.data_ptr()),
                                            _dp(ws), ws.numel() * ws.element_size(), _stream(stream)), "xq_mx_expanded_linear_host")


def xq_mx_gemm_staged(M: int, w: MxWeights, out, ws, stream=None) -> None:
    _check(lib().xq_mx_gemm_staged(M, w.handle, _dp(out), _dp(ws), ws.numel() * ws.element_size(), _stream(stream)), "xq_mx_gemm_staged")


def xq_mx_rotate_quant_staged(X, w: MxWeights, ws, M=None, ldx=None, stream=None) -> None:
    M = X.shape[0] if M is None else M
    ldx = X.stride(0) if ldx is None else ldx
    _check(lib().xq_mx_rotate_quant_staged(ctypes.c_void_p(X.data_ptr()), M, ldx, w.handle, _dp(ws), ws.numel() * ws.element_size(),
                                           _stream(stream)), "xq_mx_rotate_quant_staged")


def xq_mx_prepare_weights_heads(W_bf16_host: np.ndarray, heads: int, head_dim_p: int, stream=None) -> MxWeights:
    W = np.ascontiguousarray(W_bf16_host, dtype=np.uint16)
    N, K = W.shape
    assert K % heads == 0
    h = ctypes.c_void_p()
    _check(lib().xq_mx_prepare_weights_heads(_hp(W), N, heads, K // heads, head_dim_p, _stream(stream), ctypes.byref(h)),
           "xq_mx_prepare_weights_heads")
    return MxWeights(h.value)
