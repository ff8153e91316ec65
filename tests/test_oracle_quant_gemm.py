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


# ---- asymmetric activation quantizer (the paper's setting, Sec. 4 "Quantization Details") --------

def test_asym_quantizer_range_endpoints_and_error_bound(oracle):
    g = np.random.default_rng(5)
    y = g.standard_normal((40, 333)) * g.uniform(0.01, 30.0, size=(40, 1)) + g.uniform(-5, 5, size=(40, 1))
    y[3] = 0.0                      # all-zero row
    y[4] = np.abs(y[4])             # no negative values: the range still starts at zero
    y[5] = -np.abs(y[5])            # no positive values
    u, s, z = oracle.quantize_asym(y)
    assert u.dtype == np.uint8 and u.min() >= 0 and u.max() <= 15
    assert s[3] == 1.0 and z[3] == 0 and not u[3].any()
    assert z[4] == 0 and z[5] == 15
    lo = np.minimum(y.min(axis=1), 0.0)
    hi = np.maximum(y.max(axis=1), 0.0)
    for r in range(y.shape[0]):
        if r == 3:
            continue
        assert np.isclose(s[r], (hi[r] - lo[r]) / 15.0, rtol=1e-6)
        # the extremes map to the ends of the code range
        if lo[r] < 0:
            assert u[r, np.argmin(y[r])] == 0
        if hi[r] > 0:
            assert u[r, np.argmax(y[r])] in (14, 15)  # 14 when rounding the zero point shifted the grid down
        # a code stands for s * (u - z); inside the range the error is at most half a step
        # (plus the half step by which rounding the zero point can shift the grid)
        err = np.abs(y[r] - s[r].astype(np.float64) * (u[r].astype(np.float64) - z[r]))
        assert err.max() <= s[r] * (1.0 + 1e-6)
        assert np.median(err) <= 0.5 * s[r]
    assert np.all((z >= 0) & (z <= 15))


def test_asym_quantizer_is_exact_on_an_integer_grid(oracle):
    """Values k * step with k in [-z, 15 - z] and both end points present come back exactly."""
    step = 0.375
    for z0 in (0, 3, 8, 15):
        k = np.arange(-z0, 16 - z0, dtype=np.float64)
        y = np.tile(k * step, (2, 3))
        u, s, z = oracle.quantize_asym(y)
        assert np.allclose(s, step, rtol=1e-7) and np.all(z == z0)
        assert np.array_equal(u[0, :16].astype(np.int64) - z0, k.astype(np.int64))


def test_asym_ties_round_to_even(oracle):
    # range [-2, 13] -> s = 1, z = 2; y = 0.5, 1.5, 2.5 are exact ties
    y = np.array([[-2.0, 13.0, 0.5, 1.5, 2.5, -0.5, -1.5]])
    u, s, z = oracle.quantize_asym(y)
    assert s[0] == 1.0 and z[0] == 2
    assert list(u[0].astype(int) - 2) == [-2, 13, 0, 2, 2, 0, -2]


def test_asym_epilogue_identity_against_float_product(oracle):
    """s_x s_w (acc - z wsum) equals the product of the dequantized operands (library matmul, fp64)."""
    g = np.random.default_rng(9)
    M, N, Kp = 7, 11, 96
    ux = g.integers(0, 16, size=(M, Kp), dtype=np.uint8)
    qw = g.integers(-8, 8, size=(N, Kp), dtype=np.int8)
    z = g.integers(0, 16, size=M, dtype=np.int32)
    s_x = synth.scales(M, seed=3, tag="ax")
    s_w = synth.scales(N, seed=3, tag="aw")
    acc = oracle.gemm_u_i64(ux, qw)
    assert np.array_equal(acc, ux.astype(np.int64) @ qw.astype(np.int64).T)
    out = synth.bf16_bits_to_f32(oracle.epilogue_asym(acc, s_x, z, s_w, qw)).astype(np.float64)
    xdq = s_x[:, None].astype(np.float64) * (ux.astype(np.float64) - z[:, None])
    wdq = s_w[:, None].astype(np.float64) * qw.astype(np.float64)
    want = xdq @ wdq.T
    assert np.all(np.abs(out - want) <= np.abs(want) * 2.0**-8 + 1e-30)
    # closed form: all codes 15, zero point 5, weights all -8: acc = -120 Kp, wsum = -8 Kp -> (acc - z wsum) = -80 Kp
    ux[:] = 15
    qw[:] = -8
    z[:] = 5
    out = synth.bf16_bits_to_f32(oracle.epilogue_asym(oracle.gemm_u_i64(ux, qw), np.ones(M, np.float32), z, np.ones(N, np.float32), qw))
    assert np.all(out == -80.0 * Kp)


def test_asym_layer_is_closer_to_the_unquantized_product_than_chance(oracle):
    """End to end on one-sided activations (where an asymmetric grid has twice the resolution): the
    asymmetric layer reproduces the fp64 product of the bf16 inputs at least as well as the symmetric one."""
    K, Kp, M, N = 200, 240, 12, 40
    pl = oracle.plan(K, Kp)
    x = synth.activations(M, K, seed=4, tag="asym")
    w = synth.weights(N, K, seed=4, tag="asym")
    ref = oracle.ref_product(x, w)
    out_a = synth.bf16_bits_to_f32(oracle.expanded_linear_asym(pl, x, w)[0]).astype(np.float64)
    out_s = synth.bf16_bits_to_f32(oracle.expanded_linear(pl, x, w)[0]).astype(np.float64)
    ea = np.linalg.norm(out_a - ref) / np.linalg.norm(ref)
    es = np.linalg.norm(out_s - ref) / np.linalg.norm(ref)
    assert ea < 0.5 and es < 0.5  # both are 4-bit approximations of the same product
    assert ea <= es * 1.25
