"""Pins for the oracle's quantizer, integer product, epilogue and packing.

Hand-worked values, closed forms, invariants and brute force -- none of these re-derives the
oracle's result with the oracle's own formula.
"""
import numpy as np
import pytest
import torch

from paper_2503_17513_b200 import synth


def test_quantizer_worked_example_with_ties(oracle):
    # absmax 7 -> scale exactly 1; halves round to even; -0.5 -> 0
    y = np.array([[7.0, 3.5, 2.5, 1.5, -0.5, -2.5, -6.5, 0.49, -7.0, 6.5]])
    codes, s = oracle.quantize(y)
    assert s[0] == 1.0
    assert codes.tolist() == [[7, 4, 2, 2, 0, -2, -6, 0, -7, 6]]
    # scale is absmax / 7
    codes, s = oracle.quantize(np.array([[0.0, -14.0, 1.0, 3.0]]))
    assert s[0] == 2.0 and codes.tolist() == [[0, -7, 0, 2]]  # 0.5 -> 0, 1.5 -> 2


def test_quantizer_zero_row_and_shapes(oracle):
    y = np.zeros((3, 8))
    y[1, 2] = -3.0
    codes, s = oracle.quantize(y)
    assert s.dtype == np.float32 and codes.dtype == np.int8
    assert s[0] == 1.0 and s[2] == 1.0 and not codes[0].any() and not codes[2].any()
    assert codes[1, 2] == -7 and np.isclose(s[1], 3.0 / 7.0)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_quantizer_invariants(oracle, seed):
    g = np.random.default_rng(seed)
    y = g.standard_normal((16, 272)) * np.exp(g.uniform(-6, 6, size=(16, 1)))
    codes, s = oracle.quantize(y)
    s64 = s.astype(np.float64)[:, None]
    assert codes.min() >= -7 and codes.max() <= 7          # symmetric: -8 is never produced
    am = np.argmax(np.abs(y), axis=1)
    assert np.all(np.abs(codes[np.arange(16), am]) == 7)    # the absmax element maps to +-7
    assert np.all(np.abs(y - s64 * codes) <= 0.5 * s64 * (1 + 1e-6))
    assert np.allclose(s64[:, 0], np.abs(y).max(axis=1) / 7, rtol=1e-7)
    # a row already on the grid and containing a +-7 is a fixed point
    grid = codes.astype(np.float64) * s64
    codes2, s2 = oracle.quantize(grid)
    assert np.array_equal(codes2, codes) and np.array_equal(s2, s)


def test_pack_layout_and_round_trip(oracle):
    codes = np.array([[1, -1, 7, -8, 0, 3]], dtype=np.int8)
    packed = oracle.pack_int4(codes)
    # byte j: code 2j in bits 0-3, code 2j+1 in bits 4-7, two's complement nibbles
    assert packed.tolist() == [[0xF1, 0x87, 0x30]]
    allc = synth.int4_codes(5, 64, seed=9)
    assert np.array_equal(oracle.unpack_int4(oracle.pack_int4(allc)), allc)


def test_gemm_closed_forms(oracle):
    Kp = 40
    qx = np.full((3, Kp), -8, dtype=np.int8)
    qw = np.full((2, Kp), -8, dtype=np.int8)
    assert np.all(oracle.gemm_i64(qx, qw) == 64 * Kp)
    qw[1] = 7
    assert np.all(oracle.gemm_i64(qx, qw)[:, 1] == -56 * Kp)
    # single non-zero picks one element; operand roles are not interchangeable when M != N
    qx = np.zeros((2, Kp), dtype=np.int8)
    qx[1, 17] = 5
    qw = synth.int4_codes(4, Kp, seed=3)
    acc = oracle.gemm_i64(qx, qw)
    assert acc.shape == (2, 4)
    assert np.all(acc[0] == 0) and np.array_equal(acc[1], 5 * qw[:, 17].astype(np.int64))
    # largest order of the workloads stays far below 2^31
    qx = np.full((1, 15360), -8, dtype=np.int8)
    assert oracle.gemm_i64(qx, qx)[0, 0] == 64 * 15360 < 2**31


def test_gemm_brute_force_tiny(oracle):
    for (M, N, Kp) in [(1, 1, 2), (3, 5, 40), (8, 7, 72)]:
        qx = synth.int4_codes(M, Kp, seed=M)
        qw = synth.int4_codes(N, Kp, seed=N, tag="w")
        want = [[sum(int(qx[m, c]) * int(qw[n, c]) for c in range(Kp)) for n in range(N)] for m in range(M)]
        assert oracle.gemm_i64(qx, qw).tolist() == want


def test_bf16_rounding_against_library_and_ties(oracle):
    # hand-worked ties at 1.0 (bf16 ulp there is 2^-7)
    vals = np.array([1.0 + 2.0**-8, 1.0 + 3 * 2.0**-8, 1.0 + 2.0**-8 + 2.0**-30, -(1.0 + 2.0**-8),
                     0.0, 65280.0, 3.0e38, 3.4e38, 1e-40])
    got = oracle.f64_to_bf16(vals)
    want_f = [1.0, 1.0 + 2.0**-6, 1.0 + 2.0**-7, -1.0, 0.0, 65280.0]
    assert synth.bf16_bits_to_f32(got[:6]).tolist() == want_f
    # library conversion (binary32 -> bf16, round to nearest even) on values exact in binary32
    g = np.random.default_rng(0)
    f = (g.standard_normal(4096) * np.exp(g.uniform(-60, 60, 4096))).astype(np.float32)
    f = np.concatenate([f, np.array([3.0e38, 3.4e38, 1e-40, -1e-39, 2.0**-133, 2.0**-134], dtype=np.float32)])
    want = torch.from_numpy(f).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.f64_to_bf16(f.astype(np.float64)), want)
    # and back
    assert np.array_equal(oracle.bf16_to_f64(want[:4096]),
                          torch.from_numpy(want[:4096].view(np.int16)).view(torch.bfloat16).double().numpy())


def test_epilogue_closed_form(oracle):
    acc = np.array([[64 * 40, -3], [1, 0]], dtype=np.int64)
    s_x = np.array([0.5, 2.0], dtype=np.float32)
    s_w = np.array([0.25, 1.0], dtype=np.float32)
    out = synth.bf16_bits_to_f32(oracle.epilogue(acc, s_x, s_w))
    assert out.tolist() == [[320.0, -1.5], [0.5, 0.0]]
    # one rounding of the exact product: 257 * 1 * 1 -> tie between 256 and 258 -> 256
    out = oracle.epilogue(np.array([[257, 259]], dtype=np.int64), np.ones(1, np.float32), np.ones(2, np.float32))
    assert synth.bf16_bits_to_f32(out).tolist() == [[256.0, 260.0]]


def test_whole_layer_close_to_unquantized_product(oracle):
    """INT4 x INT4 with rotation tracks the fp64 product of the same inputs; the error shrinks
    when the quantizer is given more levels is not tested (4 bits fixed) -- only a sane bound."""
    K, Kp = 200, 240
    pl = oracle.plan(K, Kp)
    x = synth.activations(8, K, seed=0)
    w = synth.weights(12, K, seed=0)
    out, acc = oracle.expanded_linear(pl, x, w)
    ref = oracle.ref_product(x, w)
    rel = np.linalg.norm(synth.bf16_bits_to_f32(out) - ref) / np.linalg.norm(ref)
    assert rel < 0.3 and np.abs(acc).max() < 2**31
    # dequantized rotated operands reproduce the epilogue's pre-rounding value
    _, qx, sx = oracle.rotate_quant(pl, x)
    qw, sw = oracle.prepare_weights(pl, w)
    manual = (qx.astype(np.float64) * sx[:, None]) @ (qw.astype(np.float64) * sw[:, None]).T
    assert np.allclose(synth.bf16_bits_to_f32(out), manual, rtol=2.0**-8, atol=1e-30)
