"""Pins for the oracle's Hadamard construction and rotation (paper Sec. 3, Remarks 1-2).

Each check is something the paper or the mathematics fixes, not a second copy of the oracle's
formula: orthogonality with +-1 entries, a library Walsh-Hadamard matrix for the power-of-two
case, a library Kronecker product for the index convention, the truncated-column norm, energy,
rank and the rotation invariance of the linear layer.
"""
import numpy as np
import pytest
import scipy.linalg

from paper_2503_17513_b200 import synth

# (K, Kp): every order-p factor used by the workloads (68, 60, 36, 20, 1) on a small Sylvester
# factor, plus further Paley orders (12, 28, 76, 140) from the paper's own Table 1 sizes.
SMALL = [(100, 136), (60, 68), (200, 240), (130, 144), (70, 80), (64, 64), (40, 48), (20, 24),
         (50, 56), (140, 152), (250, 280), (1, 2), (3, 4), (300, 344), (600, 688)]  # 344 = 7^3 + 1: Paley over GF(7^3)


@pytest.mark.parametrize("K,Kp", SMALL)
def test_entries_and_orthogonality(oracle, K, Kp):
    pl = oracle.plan(K, Kp)
    assert pl.p * (1 << pl.log2n) == Kp
    H = oracle.hadamard_dense(pl).astype(np.int64)
    assert set(np.unique(H)) <= {-1, 1}
    assert np.array_equal(H @ H.T, Kp * np.eye(Kp, dtype=np.int64))  # Sec. 3: H_hat H_hat^T = I with gamma = 1/sqrt(M)
    assert np.array_equal(H.T @ H, Kp * np.eye(Kp, dtype=np.int64))


@pytest.mark.parametrize("K,Kp", [(2048, 2176), (4096, 4608)])
def test_orthogonality_config_sizes(oracle, K, Kp):
    pl = oracle.plan(K, Kp)
    H = oracle.hadamard_dense(pl).astype(np.float64)  # +-1 sums below 2^53 are exact in fp64
    G = H @ H.T
    assert np.array_equal(G, Kp * np.eye(Kp))


@pytest.mark.parametrize("n", [1, 2, 16, 64, 256])
def test_power_of_two_is_the_library_walsh_hadamard(oracle, n):
    pl = oracle.plan(n, n)
    assert (pl.p, pl.paley_kind) == (1, 0)
    assert np.array_equal(oracle.hadamard_dense(pl), scipy.linalg.hadamard(n).astype(np.int8))


@pytest.mark.parametrize("K,Kp", [(100, 136), (200, 240), (130, 144), (70, 80), (40, 48)])
def test_kronecker_convention_outer_factor_is_order_p(oracle, K, Kp):
    """H = H_p (x) S_n with channel c = a * n + b.  H_p is read off H itself (rows/cols with
    b = 0, where the Sylvester factor is +1) and the whole matrix must equal the library
    Kronecker product of that block with the library Walsh-Hadamard matrix."""
    pl = oracle.plan(K, Kp)
    n = 1 << pl.log2n
    H = oracle.hadamard_dense(pl).astype(np.int64)
    Hp = H[::n, ::n]
    assert Hp.shape == (pl.p, pl.p)
    assert np.array_equal(Hp @ Hp.T, pl.p * np.eye(pl.p, dtype=np.int64))
    assert np.array_equal(H, np.kron(Hp, scipy.linalg.hadamard(n)))


def test_paley_structure(oracle):
    """Paley-I (q = 3 mod 4): H - I is skew-symmetric with a +1 first row; Paley-II
    (q = 1 mod 4): H is symmetric.  Both are textbook properties of the two constructions."""
    for Kp, kind, q in [(68, 1, 67), (60, 1, 59), (20, 1, 19), (12, 1, 11), (36, 2, 17), (76, 2, 37), (344, 3, 343)]:
        pl = oracle.plan(Kp, Kp)
        assert (pl.p, pl.paley_kind, pl.q, pl.log2n) == (Kp, kind, q, 0)
        H = oracle.hadamard_dense(pl).astype(np.int64)
        if kind in (1, 3):
            S = H - np.eye(Kp, dtype=np.int64)
            assert np.array_equal(S, -S.T)
            assert np.all(H[0] == 1)
        else:
            assert np.array_equal(H, H.T)


def test_gf343_character_is_a_character_with_as_many_squares_as_non_squares(oracle):
    """The order-344 factor rests on the quadratic character of GF(7^3).  Read off the matrix (row i + 1, column 1 is
    chi(e_i - e_0) = chi(e_i)): it is +1 on exactly (343 - 1) / 2 elements, and it is what squaring in an independent
    model of the field says -- polynomials over GF(7) modulo x^3 - 5, multiplied with numpy's polynomial routines."""
    pl = oracle.plan(344, 344)
    H = oracle.hadamard_dense(pl).astype(np.int64)
    chi = H[1:, 1].copy()
    chi[0] = 0  # the diagonal entry is the +1 of the identity, not a character value
    assert np.count_nonzero(chi == 1) == 171 and np.count_nonzero(chi == -1) == 171

    def square(idx):
        a = np.array([idx % 7, (idx // 7) % 7, idx // 49])
        prod = np.polymul(a[::-1], a[::-1])[::-1]  # coefficients, lowest degree first
        prod = np.concatenate([prod, np.zeros(5 - len(prod), dtype=prod.dtype)])
        c = [prod[0] + 5 * prod[3], prod[1] + 5 * prod[4], prod[2]]  # x^3 = 5
        return int(c[0] % 7 + 7 * (c[1] % 7) + 49 * (c[2] % 7))

    squares = {square(i) for i in range(1, 343)}
    assert len(squares) == 171
    for i in range(1, 343):
        assert chi[i] == (1 if i in squares else -1)


def test_plan_factors_the_workload_and_paper_sizes(oracle):
    # the workload sizes: K' = p * 2^k with the stated factors
    for (K, Kp), want in {
        (2048, 2176): (68, 5, 1, 67), (8192, 8704): (68, 7, 1, 67), (4096, 4352): (68, 6, 1, 67),
        (14336, 15360): (60, 8, 1, 59), (4096, 4608): (36, 7, 2, 17), (4096, 5120): (20, 8, 1, 19),
        (4096, 4096): (1, 12, 0, 0),
    }.items():
        pl = oracle.plan(K, Kp)
        assert (pl.p, pl.log2n, pl.paley_kind, pl.q) == want
    # Table 1's expanded down-projection sizes are all Hadamard orders that factor over a Paley matrix: over a prime
    # field, except 22016 = 344 x 64, whose order-344 factor is Paley's construction over GF(7^3).
    for K, Kp in [(8192, 8960), (8192, 9728), (8192, 10240), (8192, 12288), (14336, 15360),
                  (14336, 18432), (14336, 19968)]:
        pl = oracle.plan(K, Kp)
        assert pl.p * (1 << pl.log2n) == Kp and pl.paley_kind in (1, 2)
    pl = oracle.plan(14336, 22016)
    assert (pl.p, pl.log2n, pl.paley_kind, pl.q) == (344, 6, 3, 343)
    g = np.random.default_rng(0)
    rows = g.choice(22016, size=6, replace=False)
    R = np.array([[oracle.hadamard_entry(pl, int(r), c) for c in range(22016)] for r in rows], dtype=np.int64)
    assert np.array_equal(R @ R.T, 22016 * np.eye(6, dtype=np.int64))
    with pytest.raises(ValueError):
        oracle.plan(10, 8)
    with pytest.raises(ValueError):
        oracle.plan(4, 6)  # 6 = 3 * 2: no Hadamard matrix of order 6


def test_table1_layer_sizes_are_down_proj_in_channels(oracle):
    """Table 1 (values in tests/golden/table1_sizes.txt): the printed model sizes grow by exactly
    layers x hidden x (channels - base channels), so the 'layer size' column is the K' of the down
    projection, and every printed K' is an order the plan function can factor."""
    import os

    rows = []
    with open(os.path.join(os.path.dirname(__file__), "golden", "table1_sizes.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                m, layers, hidden, base, ch, size = line.split()
                rows.append((m, int(layers), int(hidden), int(base), int(ch), float(size)))
    assert len(rows) == 15
    base_size = {m: size for m, _, _, base, ch, size in rows if base == ch}
    for m, layers, hidden, base, ch, size in rows:
        predicted = base_size[m] + layers * hidden * (ch - base) / 1e9
        assert abs(predicted - size) < 1.5e-3, (m, ch, predicted, size)  # printed to three decimals
        pl = oracle.plan(base, ch)
        assert pl.p * (1 << pl.log2n) == ch


@pytest.mark.parametrize("K,Kp", [(100, 136), (200, 240), (130, 144), (64, 64), (2048, 2176)])
def test_truncated_column_norm_energy(oracle, K, Kp):
    pl = oracle.plan(K, Kp)
    Hhat = oracle.hadamard_dense(pl, rows=K).astype(np.float64) / np.sqrt(Kp)
    # Remark 2: every column of H_hat has norm sqrt(N / M)
    assert np.allclose(np.linalg.norm(Hhat, axis=0), np.sqrt(K / Kp), rtol=1e-13)
    # Sec. 3: H_hat H_hat^T = I_K
    assert np.allclose(Hhat @ Hhat.T, np.eye(K), atol=1e-12)
    x = synth.activations(5, K, seed=3)
    y = oracle.rotate_dense(pl, x)
    xf = oracle.bf16_to_f64(x)
    # the rotation is x @ H_hat (library matmul) and preserves energy (Remark 2)
    assert np.allclose(y, xf @ Hhat, rtol=0, atol=1e-12 * np.abs(xf).max() * np.sqrt(K))
    assert np.allclose(np.linalg.norm(y, axis=1), np.linalg.norm(xf, axis=1), rtol=1e-13)


def test_rank_preserved_nullity_grows(oracle):
    """Remark 1: rank(X H_hat) = rank(X), so the nullity grows by M - N."""
    K, Kp = 20, 24
    pl = oracle.plan(K, Kp)
    base = synth.bf16_bits_to_f32(synth.activations(3, K, seed=5))
    X = np.vstack([base, base[0] + base[1], 2 * base[2], base[0] - base[2]])  # rank 3, 6 rows
    xb = synth.f32_to_bf16_bits(X.astype(np.float32))
    Xf = oracle.bf16_to_f64(xb)
    r = np.linalg.matrix_rank(Xf)
    y = oracle.rotate_dense(pl, xb)
    assert np.linalg.matrix_rank(y) == r
    assert (Kp - np.linalg.matrix_rank(y)) - (K - r) == Kp - K


@pytest.mark.parametrize("K,Kp", [(100, 136), (200, 240), (130, 144), (70, 80), (64, 64), (2048, 2176)])
def test_rotation_invariance(oracle, K, Kp):
    """Sec. 3: X W = (X H_hat)(H_hat^T W); with out x in storage both operands get the same map."""
    pl = oracle.plan(K, Kp)
    x = synth.activations(4, K, seed=1)
    w = synth.weights(6, K, seed=1)
    ref = oracle.ref_product(x, w)
    got = oracle.rotate_dense(pl, x) @ oracle.rotate_dense(pl, w).T
    assert np.linalg.norm(got - ref) <= 1e-12 * np.linalg.norm(ref)


@pytest.mark.parametrize("K,Kp", [(100, 136), (200, 240), (130, 144), (70, 80), (64, 64),
                                  (2048, 2176), (4096, 4608), (4096, 5120)])
def test_factored_matches_dense(oracle, K, Kp):
    pl = oracle.plan(K, Kp)
    x = synth.activations(3, K, seed=2, heavy_tail=True)
    yd = oracle.rotate_dense(pl, x)
    yf = oracle.rotate_factored(pl, x)
    assert np.linalg.norm(yd - yf) <= 1e-12 * np.linalg.norm(yd)


def test_factored_large_shape_energy_and_invariance(oracle):
    """The largest workload order (15360 = 60 * 256) through the factored form only."""
    K, Kp = 14336, 15360
    pl = oracle.plan(K, Kp)
    x = synth.activations(2, K, seed=4)
    w = synth.weights(2, K, seed=4)
    yx, yw = oracle.rotate_factored(pl, x), oracle.rotate_factored(pl, w)
    xf = oracle.bf16_to_f64(x)
    assert np.allclose(np.linalg.norm(yx, axis=1), np.linalg.norm(xf, axis=1), rtol=1e-12)
    ref = oracle.ref_product(x, w)
    assert np.linalg.norm(yx @ yw.T - ref) <= 1e-11 * np.linalg.norm(ref)
    # one dense row of the definition as a spot check of the big index arithmetic
    yd = oracle.rotate_dense(pl, x[:1])
    assert np.linalg.norm(yd - yx[:1]) <= 1e-12 * np.linalg.norm(yd)


# Head-wise expansion (Sec. 5 "Expanding R2 and R4"): 64 -> 72 = H_72 (Paley-I, q = 71), 64 -> 80 = H_20 (x) S_4,
# 128 -> 144 = H_36 (x) S_4, 128 -> 160 = H_20 (x) S_8, and the unexpanded 64 -> 64.
HEAD_PLANS = [(4, 64, 72), (3, 64, 80), (2, 128, 144), (2, 128, 160), (4, 64, 64), (5, 8, 12)]


@pytest.mark.parametrize("heads,hd,hdp", HEAD_PLANS)
def test_headwise_rotation_is_the_block_diagonal_matrix(oracle, heads, hd, hdp):
    """The head-wise map is x @ kron(I_heads, H_hat): library Kronecker product and matmul."""
    pl = oracle.plan(hd, hdp)
    Hhat = oracle.hadamard_dense(pl, rows=hd).astype(np.float64) / np.sqrt(hdp)
    B = np.kron(np.eye(heads), Hhat)
    assert np.allclose(B @ B.T, np.eye(heads * hd), atol=1e-12)  # left inverse per block (Sec. 3)
    x = synth.activations(3, heads * hd, seed=8, tag="heads")
    xf = oracle.bf16_to_f64(x)
    y = oracle.rotate_heads(pl, heads, x)
    assert y.shape == (3, heads * hdp)
    assert np.allclose(y, xf @ B, rtol=0, atol=1e-12 * np.abs(xf).max() * np.sqrt(hd))
    # energy per head is preserved (Remark 2), so a head with a dominant channel stays inside its block
    for h in range(heads):
        assert np.allclose(np.linalg.norm(y[:, h * hdp:(h + 1) * hdp], axis=1),
                           np.linalg.norm(xf[:, h * hd:(h + 1) * hd], axis=1), rtol=1e-12)


@pytest.mark.parametrize("heads,hd,hdp", HEAD_PLANS)
def test_headwise_rotation_invariance(oracle, heads, hd, hdp):
    """Sec. 3 applied block by block: x W^T is unchanged when both operands get the head-wise map."""
    pl = oracle.plan(hd, hdp)
    x = synth.activations(4, heads * hd, seed=9, tag="hx")
    w = synth.weights(6, heads * hd, seed=9, tag="hw")
    ref = oracle.ref_product(x, w)
    got = oracle.rotate_heads(pl, heads, x) @ oracle.rotate_heads(pl, heads, w).T
    assert np.linalg.norm(got - ref) <= 1e-12 * np.linalg.norm(ref)


def test_headwise_with_one_head_is_the_plain_rotation(oracle):
    pl = oracle.plan(100, 136)
    x = synth.activations(3, 100, seed=10)
    assert np.array_equal(oracle.rotate_heads(pl, 1, x), oracle.rotate_dense(pl, x))
    y, codes, s = oracle.rotate_quant_heads(pl, 1, x)
    y2, codes2, s2 = oracle.rotate_quant(pl, x)
    assert np.array_equal(codes, codes2) and np.array_equal(s, s2)
