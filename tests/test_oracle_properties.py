"""Property pins for the oracle's three quantizers: facts that follow from their definitions and hold for
every input, checked on random rows (hypothesis).  A wrong rounding mode, a misplaced clamp or a scale taken
from the wrong extreme breaks at least one of them.
"""
import numpy as np
from hypothesis import given, settings
from hypothesis import strategies as st

rows = st.integers(min_value=0, max_value=2**31 - 1).map(
    lambda seed: np.random.default_rng(seed).standard_normal((3, 64)) * np.exp2(np.random.default_rng(seed + 1).integers(-12, 12)))
shifts = st.integers(min_value=-20, max_value=20)


@settings(max_examples=40, deadline=None)
@given(rows, shifts)
def test_power_of_two_scaling_moves_only_the_scale(oracle, y, k):
    """Multiplying a row by 2^k is exact in binary floating point: codes stay, scales move by 2^k."""
    c0, s0 = oracle.quantize(y)
    c1, s1 = oracle.quantize(np.ldexp(y, k))
    assert np.array_equal(c0, c1) and np.array_equal(s1, np.ldexp(s0, k).astype(np.float32))
    u0, t0, z0 = oracle.quantize_asym(y)
    u1, t1, z1 = oracle.quantize_asym(np.ldexp(y, k))
    assert np.array_equal(u0, u1) and np.array_equal(z0, z1) and np.array_equal(t1, np.ldexp(t0, k).astype(np.float32))
    m0, e0 = oracle.quantize_mx(y)
    m1, e1 = oracle.quantize_mx(np.ldexp(y, k))
    assert np.array_equal(m0, m1) and np.array_equal(e1.astype(int), e0.astype(int) + k)


@settings(max_examples=40, deadline=None)
@given(rows)
def test_negation(oracle, y):
    """Symmetric INT4 and MXFP4 are odd functions of the row (round half to even is symmetric; the symmetric scale and the
    shared exponents see magnitudes only); the asymmetric codes mirror around 15 with the zero point."""
    c0, s0 = oracle.quantize(y)
    c1, s1 = oracle.quantize(-y)
    assert np.array_equal(c1, -c0) and np.array_equal(s0, s1)
    m0, e0 = oracle.quantize_mx(y)
    m1, e1 = oracle.quantize_mx(-y)
    assert np.array_equal(oracle.e2m1_value(m1), -oracle.e2m1_value(m0)) and np.array_equal(e0, e1)
    u0, t0, z0 = oracle.quantize_asym(y)
    u1, t1, z1 = oracle.quantize_asym(-y)
    assert np.array_equal(t0, t1)
    # s (u - z) changes sign up to the rounding of the zero point: the represented values mirror within one step
    v0 = (u0.astype(np.int64) - z0[:, None]) * t0[:, None].astype(np.float64)
    v1 = (u1.astype(np.int64) - z1[:, None]) * t1[:, None].astype(np.float64)
    assert np.all(np.abs(v0 + v1) <= t0[:, None] * (1 + 1e-6))


@settings(max_examples=40, deadline=None)
@given(rows)
def test_reconstruction_error_bounds(oracle, y):
    c, s = oracle.quantize(y)
    assert np.all(np.abs(y - c * s[:, None].astype(np.float64)) <= 0.5 * s[:, None] * (1 + 1e-6))
    u, t, z = oracle.quantize_asym(y)
    assert np.all(np.abs(y - (u.astype(np.int64) - z[:, None]) * t[:, None].astype(np.float64)) <= 0.5 * t[:, None] * (1 + 1e-6) + 1e-300)
    assert np.all(t <= s * (14.0 / 15.0) * (1 + 1e-6))  # the asymmetric step never exceeds 14/15 of the symmetric one
    m, e = oracle.quantize_mx(y)
    err = np.abs(y - oracle.dequantize_mx(m, e))
    amax = np.abs(y.reshape(3, 2, 32)).max(axis=2)
    # 2^e lies in (amax / 8, amax / 4]: half of the widest step (2 x 2^e) is at most amax / 4, and a value saturated at
    # 6 x 2^e loses less than amax - 6 amax / 8 = amax / 4
    assert np.all(err.reshape(3, 2, 32) <= amax[:, :, None] / 4 + 1e-300)
