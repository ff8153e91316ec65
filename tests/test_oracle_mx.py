"""Pins for the oracle's MXFP4 quantizer and product (paper Sec. 4 "Quantization Details": the OCP
microscaling format, one E8M0 scale per group of 32 elements, E2M1 elements).

What is checked is fixed by the format itself: the sixteen E2M1 values from the bit fields, power-of-two
scales placing the group maximum in [4, 8), round-to-nearest-even on a one-bit mantissa (through
numpy's frexp / rint, not the oracle's table search), saturation at 6, exactness on the grid, and the
product against a library matmul of the dequantized matrices.
"""
import numpy as np
import pytest

from paper_2503_17513_b200 import synth


def test_e2m1_values_follow_the_bit_fields(oracle):
    """sign | 2 exponent bits (bias 1) | 1 mantissa bit; exponent field 0 is subnormal (0 or 0.5)."""
    codes = np.arange(16, dtype=np.uint8)
    want = []
    for c in codes:
        s, e, m = (c >> 3) & 1, (c >> 1) & 3, c & 1
        mag = 0.5 * m if e == 0 else (1.0 + 0.5 * m) * 2.0 ** (e - 1)
        want.append(-mag if s else mag)
    assert np.array_equal(oracle.e2m1_value(codes), np.array(want))
    assert sorted(set(np.abs(want))) == [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]


def one_bit_mantissa_rne(v):
    """Nearest E2M1 magnitude by the format's definition: subnormal step 0.5 below 1, else one mantissa bit;
    numpy's rint rounds half to even."""
    a = np.abs(v)
    out = np.empty_like(a)
    sub = a < 1.0
    out[sub] = np.rint(a[sub] * 2.0) / 2.0
    f, e = np.frexp(a[~sub])            # a = f 2^e, f in [0.5, 1)
    out[~sub] = np.ldexp(np.rint(f * 4.0) / 4.0, e)  # two significant bits: 1.m
    return np.sign(v) * np.minimum(out, 6.0)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_quantizer_matches_the_format_definition(oracle, seed):
    g = np.random.default_rng(seed)
    y = g.standard_normal((7, 96)) * np.exp2(g.integers(-20, 20, size=(7, 1)))
    y[2, 32:64] = 0.0
    codes, sc = oracle.quantize_mx(y)
    assert codes.shape == (7, 96) and sc.shape == (7, 3)
    amax = np.abs(y.reshape(7, 3, 32)).max(axis=2)
    e = sc.astype(np.int64) - 127
    nz = amax > 0
    assert np.all(e[~nz] == 0) and np.all(codes.reshape(7, 3, 32)[~nz] == 0)
    scaled_max = amax[nz] / np.exp2(e[nz])
    assert np.all((scaled_max >= 4.0) & (scaled_max < 8.0))          # e = floor(log2 amax) - 2
    X = np.repeat(np.exp2(e.astype(np.float64)), 32, axis=1)
    want = one_bit_mantissa_rne(y / X)
    got = oracle.e2m1_value(codes)
    assert np.array_equal(got, want)
    # every group's largest element lands on 4 or 6
    gmax = np.abs(got.reshape(7, 3, 32)).max(axis=2)
    assert set(np.unique(gmax[nz])) <= {4.0, 6.0}
    # error: half a step inside the range, at most 2 (scaled units) where 6 saturates values below 8
    err = np.abs(y / X - got)
    a = np.abs(y / X)
    bound = np.where(a < 2, 0.25, np.where(a < 4, 0.5, np.where(a <= 6, 1.0, 2.0)))
    assert np.all(err <= bound + 1e-12)


def test_ties_go_to_the_even_mantissa(oracle):
    row = np.zeros((1, 32))
    row[0, :9] = [4.0, 0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, -2.5]   # the 4.0 fixes the scale at 2^0
    codes, sc = oracle.quantize_mx(row)
    assert sc[0, 0] == 127
    assert list(oracle.e2m1_value(codes)[0, :9]) == [4.0, 0.0, 1.0, 1.0, 2.0, 2.0, 4.0, 4.0, -2.0]
    assert codes[0, 8] == 8 + 4  # sign bit set, magnitude code of 2.0


def test_grid_points_are_fixed_points(oracle):
    g = np.random.default_rng(5)
    codes = g.integers(0, 16, size=(6, 128)).astype(np.uint8)
    codes[:, ::32] = 6   # a 4.0 in every group: the shared exponent is recovered exactly
    sc = g.integers(100, 150, size=(6, 4)).astype(np.uint8)
    y = oracle.dequantize_mx(codes, sc)
    c2, s2 = oracle.quantize_mx(y)
    assert np.array_equal(s2, sc)
    assert np.array_equal(oracle.e2m1_value(c2), oracle.e2m1_value(codes))  # -0 and +0 are the same value


def test_scale_clamps_and_saturation(oracle):
    y = np.zeros((1, 64))
    y[0, 0] = 2.0 ** 200
    y[0, 1] = 2.0 ** 129
    y[0, 32] = 2.0 ** -140
    codes, sc = oracle.quantize_mx(y)
    assert sc[0, 0] == 254 and codes[0, 0] == 7 and oracle.e2m1_value(codes[0, 1:2])[0] == 4.0
    assert sc[0, 1] == 0 and codes[0, 32] == 0  # 2^-140 / 2^-127 rounds to zero


@pytest.mark.parametrize("M,N,Kp", [(3, 5, 64), (4, 7, 160)])
def test_product_is_the_matmul_of_the_dequantized_matrices(oracle, M, N, Kp):
    g = np.random.default_rng(9)
    cx = g.integers(0, 16, size=(M, Kp)).astype(np.uint8)
    cw = g.integers(0, 16, size=(N, Kp)).astype(np.uint8)
    sx = g.integers(117, 137, size=(M, Kp // 32)).astype(np.uint8)
    sw = g.integers(117, 137, size=(N, Kp // 32)).astype(np.uint8)
    ref = oracle.gemm_mx(cx, sx, cw, sw)
    want = oracle.dequantize_mx(cx, sx) @ oracle.dequantize_mx(cw, sw).T   # library matmul
    assert np.allclose(ref, want, rtol=1e-13, atol=0)
    # all-ones elements, unit scales: the dot product counts the channels
    one = np.full((1, Kp), 2, dtype=np.uint8)
    unit = np.full((1, Kp // 32), 127, dtype=np.uint8)
    assert oracle.gemm_mx(one, unit, one, unit)[0, 0] == Kp


def test_expanded_layer_with_mxfp4_stays_close_to_the_unquantized_product(oracle):
    K, Kp = 100, 160
    pl = oracle.plan(K, Kp)
    x = synth.activations(6, K, seed=21)
    w = synth.weights(9, K, seed=21)
    out, ref_mx = oracle.expanded_linear_mx(pl, x, w)
    ref = oracle.ref_product(x, w)
    assert np.linalg.norm(ref_mx - ref) < 0.3 * np.linalg.norm(ref)
    assert np.array_equal(out, oracle.f64_to_bf16(ref_mx))
