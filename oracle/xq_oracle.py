"""numpy binding of the C oracle (``xq_oracle.c``).  Test infrastructure only.

Every function is argument marshalling around one C routine; the arithmetic lives in the C
file, which cites the passage of the paper each routine follows.  bf16 tensors travel as
``uint16`` arrays holding the raw bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "xq_oracle.c")
_LIB = os.path.join(_HERE, "libxq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, OpenMP over rows) into ``libxq_oracle.so``."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-Wall", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class _PlanC(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("K", "Kp", "p", "log2n", "paley_kind", "q")]


@dataclass(frozen=True)
class Plan:
    K: int
    Kp: int
    p: int
    log2n: int
    paley_kind: int
    q: int

    def _c(self) -> _PlanC:
        return _PlanC(self.K, self.Kp, self.p, self.log2n, self.paley_kind, self.q)


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.xqo_plan.restype = ctypes.c_int
        _lib.xqo_hadamard_entry.restype = ctypes.c_int
        _lib.xqo_num_threads.restype = ctypes.c_int
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _i64(v) -> ctypes.c_int64:
    return ctypes.c_int64(int(v))


def num_threads() -> int:
    return int(_load().xqo_num_threads())


def plan(K: int, Kp: int) -> Plan:
    """Factor Kp = p * 2^k.  Raises ValueError for bad sizes or an order with no Paley factor."""
    pc = _PlanC()
    rc = _load().xqo_plan(ctypes.c_int32(K), ctypes.c_int32(Kp), ctypes.byref(pc))
    if rc == 1:
        raise ValueError(f"invalid sizes K={K}, Kp={Kp}")
    if rc == 2:
        raise ValueError(f"no supported Hadamard order for Kp={Kp}")
    return Plan(pc.K, pc.Kp, pc.p, pc.log2n, pc.paley_kind, pc.q)


def hadamard_entry(pl: Plan, c: int, c2: int) -> int:
    pc = pl._c()
    return int(_load().xqo_hadamard_entry(ctypes.byref(pc), ctypes.c_int32(c), ctypes.c_int32(c2)))


def hadamard_dense(pl: Plan, rows: int | None = None) -> np.ndarray:
    """Rows [0, rows) of the +-1 matrix H (int8, [rows, Kp]); all Kp rows by default."""
    rows = pl.Kp if rows is None else rows
    out = np.empty((rows, pl.Kp), dtype=np.int8)
    pc = pl._c()
    _load().xqo_hadamard_dense(ctypes.byref(pc), ctypes.c_int32(rows), _p(out))
    return out


def bf16_to_f64(x_bits: np.ndarray) -> np.ndarray:
    x_bits = np.ascontiguousarray(x_bits, dtype=np.uint16)
    out = np.empty(x_bits.shape, dtype=np.float64)
    _load().xqo_bf16_to_f64(_p(x_bits), _i64(x_bits.size), _p(out))
    return out


def f64_to_bf16(v: np.ndarray) -> np.ndarray:
    v = np.ascontiguousarray(v, dtype=np.float64)
    out = np.empty(v.shape, dtype=np.uint16)
    _load().xqo_f64_to_bf16(_p(v), _i64(v.size), _p(out))
    return out


def _rot(fn, pl: Plan, x_bits: np.ndarray) -> np.ndarray:
    x_bits = np.ascontiguousarray(x_bits, dtype=np.uint16)
    assert x_bits.ndim == 2 and x_bits.shape[1] == pl.K
    rows = x_bits.shape[0]
    y = np.empty((rows, pl.Kp), dtype=np.float64)
    pc = pl._c()
    fn(ctypes.byref(pc), _p(x_bits), _i64(rows), _i64(pl.K), _p(y))
    return y


def rotate_dense(pl: Plan, x_bits: np.ndarray) -> np.ndarray:
    """[x, 0] H / sqrt(Kp) by the definition (O(K Kp) per row)."""
    return _rot(_load().xqo_rotate_dense, pl, x_bits)


def rotate_factored(pl: Plan, x_bits: np.ndarray) -> np.ndarray:
    """The same map through the Kronecker factors (held to rotate_dense by the tests)."""
    return _rot(_load().xqo_rotate_factored, pl, x_bits)


def rotate(pl: Plan, x_bits: np.ndarray) -> np.ndarray:
    """Dense definition while it is cheap, the factored form for large problems."""
    x_bits = np.asarray(x_bits)
    if x_bits.shape[0] * pl.K * pl.Kp <= 2_000_000_000:
        return rotate_dense(pl, x_bits)
    return rotate_factored(pl, x_bits)


def quantize(y: np.ndarray):
    """Per-row symmetric INT4: returns (codes int8 [rows, cols], scales float32 [rows])."""
    y = np.ascontiguousarray(y, dtype=np.float64)
    rows, cols = y.shape
    codes = np.empty((rows, cols), dtype=np.int8)
    scales = np.empty((rows,), dtype=np.float32)
    _load().xqo_quantize(_p(y), _i64(rows), _i64(cols), _p(codes), _p(scales))
    return codes, scales


def quantize_asym(y: np.ndarray):
    """Per-row asymmetric INT4 (range forced to contain zero): returns (codes uint8 [rows, cols] in 0..15,
    scales float32 [rows], zero points int32 [rows]); a code u stands for scale * (u - zero point)."""
    y = np.ascontiguousarray(y, dtype=np.float64)
    rows, cols = y.shape
    codes = np.empty((rows, cols), dtype=np.uint8)
    scales = np.empty((rows,), dtype=np.float32)
    zps = np.empty((rows,), dtype=np.int32)
    _load().xqo_quantize_asym(_p(y), _i64(rows), _i64(cols), _p(codes), _p(scales), _p(zps))
    return codes, scales, zps


def gemm_u_i64(ux: np.ndarray, qw: np.ndarray) -> np.ndarray:
    """acc[m, n] = sum_c ux[m, c] * qw[n, c] in int64 (unsigned activation codes)."""
    ux = np.ascontiguousarray(ux, dtype=np.uint8)
    qw = np.ascontiguousarray(qw, dtype=np.int8)
    M, Kp = ux.shape
    N, Kp2 = qw.shape
    assert Kp == Kp2
    acc = np.empty((M, N), dtype=np.int64)
    _load().xqo_gemm_u_i64(_p(ux), _p(qw), _i64(M), _i64(N), _i64(Kp), _p(acc))
    return acc


def epilogue_asym(acc: np.ndarray, s_x: np.ndarray, zp: np.ndarray, s_w: np.ndarray, qw: np.ndarray) -> np.ndarray:
    """bf16 bits of s_x[m] * s_w[n] * (acc - zp[m] * sum_c qw[n, c])."""
    acc = np.ascontiguousarray(acc, dtype=np.int64)
    s_x = np.ascontiguousarray(s_x, dtype=np.float32)
    zp = np.ascontiguousarray(zp, dtype=np.int32)
    s_w = np.ascontiguousarray(s_w, dtype=np.float32)
    qw = np.ascontiguousarray(qw, dtype=np.int8)
    M, N = acc.shape
    Kp = qw.shape[1]
    out = np.empty((M, N), dtype=np.uint16)
    _load().xqo_epilogue_asym(_p(acc), _p(s_x), _p(zp), _p(s_w), _p(qw), _i64(M), _i64(N), _i64(Kp), _p(out))
    return out


def pack_int4(codes: np.ndarray) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.int8)
    rows, cols = codes.shape
    assert cols % 2 == 0
    out = np.empty((rows, cols // 2), dtype=np.uint8)
    _load().xqo_pack_int4(_p(codes), _i64(rows), _i64(cols), _p(out))
    return out


def unpack_int4(packed: np.ndarray) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    rows, half = packed.shape
    out = np.empty((rows, 2 * half), dtype=np.int8)
    _load().xqo_unpack_int4(_p(packed), _i64(rows), _i64(2 * half), _p(out))
    return out


def gemm_i64(qx: np.ndarray, qw: np.ndarray) -> np.ndarray:
    """acc[m, n] = sum_c qx[m, c] * qw[n, c] in int64."""
    qx = np.ascontiguousarray(qx, dtype=np.int8)
    qw = np.ascontiguousarray(qw, dtype=np.int8)
    M, Kp = qx.shape
    N, Kp2 = qw.shape
    assert Kp == Kp2
    acc = np.empty((M, N), dtype=np.int64)
    _load().xqo_gemm_i64(_p(qx), _p(qw), _i64(M), _i64(N), _i64(Kp), _p(acc))
    return acc


def epilogue(acc: np.ndarray, s_x: np.ndarray, s_w: np.ndarray) -> np.ndarray:
    """bf16 bits of acc * s_x[m] * s_w[n]."""
    acc = np.ascontiguousarray(acc, dtype=np.int64)
    s_x = np.ascontiguousarray(s_x, dtype=np.float32)
    s_w = np.ascontiguousarray(s_w, dtype=np.float32)
    M, N = acc.shape
    assert s_x.shape == (M,) and s_w.shape == (N,)
    out = np.empty((M, N), dtype=np.uint16)
    _load().xqo_epilogue(_p(acc), _p(s_x), _p(s_w), _i64(M), _i64(N), _p(out))
    return out


def ref_product(x_bits: np.ndarray, w_bits: np.ndarray) -> np.ndarray:
    """fp64 product of the bf16 inputs, x W^T, no rotation and no quantization."""
    x_bits = np.ascontiguousarray(x_bits, dtype=np.uint16)
    w_bits = np.ascontiguousarray(w_bits, dtype=np.uint16)
    M, K = x_bits.shape
    N, K2 = w_bits.shape
    assert K == K2
    ref = np.empty((M, N), dtype=np.float64)
    _load().xqo_ref_product(_p(x_bits), _p(w_bits), _i64(M), _i64(N), _i64(K), _p(ref))
    return ref


# The three calls of the method, composed from the steps above in the paper's order.

def rotate_quant(pl: Plan, x_bits: np.ndarray):
    """Online step: pad, rotate, per-token INT4.  Returns (y fp64, codes int8, s_x float32)."""
    y = rotate(pl, x_bits)
    codes, s = quantize(y)
    return y, codes, s


def prepare_weights(pl: Plan, w_bits: np.ndarray):
    """Offline step on the out x in weight matrix: every row is padded, rotated and quantized
    per output channel.  Returns (codes int8 [N, Kp], s_w float32 [N])."""
    _, codes, s = rotate_quant(pl, w_bits)
    return codes, s


def rotate_quant_asym(pl: Plan, x_bits: np.ndarray):
    """Online step with the asymmetric activation quantizer: (y fp64, codes uint8, s_x float32, zero points int32)."""
    y = rotate(pl, x_bits)
    codes, s, z = quantize_asym(y)
    return y, codes, s, z


def expanded_linear_asym(pl: Plan, x_bits: np.ndarray, w_bits: np.ndarray):
    """Whole layer with asymmetric activations (weights unchanged: symmetric per channel)."""
    _, ux, s_x, z = rotate_quant_asym(pl, x_bits)
    qw, s_w = prepare_weights(pl, w_bits)
    acc = gemm_u_i64(ux, qw)
    return epilogue_asym(acc, s_x, z, s_w, qw), acc


def expanded_linear(pl: Plan, x_bits: np.ndarray, w_bits: np.ndarray):
    """Whole layer: returns (out bf16 bits [M, N], acc int64 [M, N])."""
    _, qx, s_x = rotate_quant(pl, x_bits)
    qw, s_w = prepare_weights(pl, w_bits)
    acc = gemm_i64(qx, qw)
    return epilogue(acc, s_x, s_w), acc


# Head-wise expansion (Sec. 4 "Compute Graph Details" and Sec. 5 "Expanding R2 and R4": the rotation in
# front of the attention output projection acts on every head separately, so expanding it grows each
# head from head_dim to head_dim' channels).  The row is cut into `heads` blocks of pl.K channels,
# each block goes through the rotation of the plan, the blocks are laid side by side again; the
# quantizers then see the whole row, exactly as for a single long rotation.

def rotate_heads(pl: Plan, heads: int, x_bits: np.ndarray) -> np.ndarray:
    """x_bits: bf16 bits [rows, heads * pl.K]  ->  fp64 [rows, heads * pl.Kp]."""
    x_bits = np.ascontiguousarray(x_bits, dtype=np.uint16)
    rows, cols = x_bits.shape
    assert cols == heads * pl.K
    y = np.empty((rows, heads * pl.Kp), dtype=np.float64)
    for h in range(heads):
        y[:, h * pl.Kp:(h + 1) * pl.Kp] = rotate(pl, x_bits[:, h * pl.K:(h + 1) * pl.K])
    return y


def rotate_quant_heads(pl: Plan, heads: int, x_bits: np.ndarray):
    """(y fp64, codes int8, scales float32): head-wise rotation, then the per-row symmetric quantizer."""
    y = rotate_heads(pl, heads, x_bits)
    codes, s = quantize(y)
    return y, codes, s


def rotate_quant_heads_asym(pl: Plan, heads: int, x_bits: np.ndarray):
    y = rotate_heads(pl, heads, x_bits)
    codes, s, z = quantize_asym(y)
    return y, codes, s, z


def expanded_linear_heads(pl: Plan, heads: int, x_bits: np.ndarray, w_bits: np.ndarray):
    """Whole layer with the head-wise rotation on both operands: (out bf16 bits [M, N], acc int64)."""
    _, qx, s_x = rotate_quant_heads(pl, heads, x_bits)
    _, qw, s_w = rotate_quant_heads(pl, heads, w_bits)
    acc = gemm_i64(qx, qw)
    return epilogue(acc, s_x, s_w), acc


# MXFP4 (Sec. 4 "Quantization Details": OCP microscaling, an E8M0 scale per group of 32, E2M1 elements).

def e2m1_value(codes: np.ndarray) -> np.ndarray:
    """fp64 values of E2M1 codes (0..15)."""
    lib = _load()
    lib.xqo_e2m1_value.restype = ctypes.c_double
    lib.xqo_e2m1_value.argtypes = [ctypes.c_uint8]
    flat = np.asarray(codes, dtype=np.uint8).ravel()
    return np.array([lib.xqo_e2m1_value(int(c)) for c in flat], dtype=np.float64).reshape(np.shape(codes))


def quantize_mx(y: np.ndarray):
    """Per group of 32 along the row: (codes uint8 [rows, cols] in 0..15, scale bytes uint8 [rows, cols / 32])."""
    y = np.ascontiguousarray(y, dtype=np.float64)
    rows, cols = y.shape
    assert cols % 32 == 0
    codes = np.empty((rows, cols), dtype=np.uint8)
    scales = np.empty((rows, cols // 32), dtype=np.uint8)
    _load().xqo_quantize_mx(_p(y), _i64(rows), _i64(cols), _p(codes), _p(scales))
    return codes, scales


def dequantize_mx(codes: np.ndarray, scales: np.ndarray) -> np.ndarray:
    lut = e2m1_value(np.arange(16, dtype=np.uint8))
    v = lut[np.asarray(codes, dtype=np.uint8)]
    return v * np.repeat(np.exp2(np.asarray(scales, dtype=np.float64) - 127.0), 32, axis=1)


def gemm_mx(cx: np.ndarray, sx: np.ndarray, cw: np.ndarray, sw: np.ndarray) -> np.ndarray:
    """fp64 product of two MXFP4 matrices (rows of cw are output channels)."""
    cx = np.ascontiguousarray(cx, dtype=np.uint8)
    cw = np.ascontiguousarray(cw, dtype=np.uint8)
    sx = np.ascontiguousarray(sx, dtype=np.uint8)
    sw = np.ascontiguousarray(sw, dtype=np.uint8)
    M, Kp = cx.shape
    N, Kp2 = cw.shape
    assert Kp == Kp2 and Kp % 32 == 0 and sx.shape == (M, Kp // 32) and sw.shape == (N, Kp // 32)
    ref = np.empty((M, N), dtype=np.float64)
    _load().xqo_gemm_mx(_p(cx), _p(sx), _p(cw), _p(sw), _i64(M), _i64(N), _i64(Kp), _p(ref))
    return ref


def rotate_quant_mx(pl: Plan, x_bits: np.ndarray, heads: int = 1):
    """(y fp64, codes, scale bytes): the online step with the MXFP4 quantizer (K' a multiple of 32)."""
    y = rotate_heads(pl, heads, x_bits) if heads > 1 else rotate(pl, x_bits)
    codes, s = quantize_mx(y)
    return y, codes, s


def expanded_linear_mx(pl: Plan, x_bits: np.ndarray, w_bits: np.ndarray, heads: int = 1):
    """Whole layer with MXFP4 weights and activations: (out bf16 bits [M, N], fp64 product)."""
    _, cx, sx = rotate_quant_mx(pl, x_bits, heads)
    _, cw, sw = rotate_quant_mx(pl, w_bits, heads)
    ref = gemm_mx(cx, sx, cw, sw)
    return f64_to_bf16(ref), ref
