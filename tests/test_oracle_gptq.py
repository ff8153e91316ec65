"""Pins of the GPTQ oracle (oracle/gptq.py; paper Sec. 4 "Quantization Details": GPTQ with act-order) against what the
mathematics fixes, none of them a re-typing of its update formula:

* an identity Hessian couples no channels: the codes are those of round-to-nearest (the C oracle's quantizer);
* every decision is optimal given the earlier ones when the later weights are left free (the defining property of the
  method): checked by brute force over the 16 grid values with a least-squares solve for the free weights;
* two coupled channels: the textbook minimiser of a 2 x 2 quadratic form; all other channels stay round-to-nearest;
* relabelling the channels relabels the codes (the act-order bookkeeping round-trips);
* on random correlated Hessians the objective tr((W - Q) H (W - Q)^T) is never above round-to-nearest's;
* a channel that never fires (zero Hessian row) gets zero codes.
"""
import numpy as np
import pytest

from oracle import gptq


def rtn(oracle, W):
    return oracle.quantize(W)


def test_identity_hessian_is_round_to_nearest(oracle):
    rng = np.random.default_rng(0)
    W = rng.standard_normal((9, 40)) * 0.02
    for H in (np.eye(40), 3.5 * np.eye(40)):
        for damp in (0.0, 0.01):
            codes, s = gptq.gptq_quantize(W, H, damp=damp)
            c_ref, s_ref = rtn(oracle, W)
            assert np.array_equal(codes, c_ref) and np.array_equal(s, s_ref)


def test_each_decision_is_optimal_with_the_later_weights_free():
    rng = np.random.default_rng(1)
    n, N = 4, 6
    for trial in range(20):
        X = rng.standard_normal((7, n))
        H = X.T @ X + 0.05 * np.eye(n)
        W = rng.standard_normal((N, n))
        codes, s = gptq.gptq_quantize(W, H, damp=0.0, order=False)
        grid = np.arange(-8, 8)
        for r in range(N):
            w, sr = W[r], float(s[r])
            fixed = []
            for j in range(n):
                best, best_q = None, None
                for q in grid:
                    d_fixed = np.array([w[i] - sr * fixed[i] for i in range(j)] + [w[j] - sr * q])
                    # minimise over the free deviations d_free: [d_fixed, d_free] H [d_fixed, d_free]^T
                    if j + 1 < n:
                        Hff = H[j + 1:, j + 1:]
                        Hfx = H[j + 1:, :j + 1]
                        d_free = -np.linalg.solve(Hff, Hfx @ d_fixed)
                        d = np.concatenate([d_fixed, d_free])
                    else:
                        d = d_fixed
                    val = d @ H @ d
                    if best is None or val < best - 1e-12:
                        best, best_q = val, q
                assert codes[r, j] == best_q, (trial, r, j)
                fixed.append(int(codes[r, j]))


def test_two_coupled_channels_closed_form_and_visiting_order(oracle):
    rng = np.random.default_rng(2)
    n, N = 10, 8
    W = rng.standard_normal((N, n))
    d = np.linspace(1.0, 2.0, n)
    rng.shuffle(d)
    H = np.diag(d)
    i_first, i_second = np.argsort(-d)[:2]  # visited first and second under act-order
    b = 0.6 * np.sqrt(d[i_first] * d[i_second])
    H[i_first, i_second] = H[i_second, i_first] = b
    codes, s = gptq.gptq_quantize(W, H, damp=0.0)
    c_rtn, s_rtn = rtn(oracle, W)
    assert np.array_equal(s, s_rtn)
    others = [i for i in range(n) if i != i_second]
    assert np.array_equal(codes[:, others], c_rtn[:, others])  # uncoupled channels and the first visited one
    s64 = s.astype(np.float64)
    delta_first = W[:, i_first] - s64 * c_rtn[:, i_first]
    want = np.clip(np.rint((W[:, i_second] + delta_first * b / d[i_second]) / s64), -8, 7)
    assert np.array_equal(codes[:, i_second], want.astype(np.int8))
    # visiting the pair in the other order gives the mirrored result
    H2 = H.copy()
    H2[i_first, i_first], H2[i_second, i_second] = H[i_second, i_second], H[i_first, i_first]
    codes2, _ = gptq.gptq_quantize(W, H2, damp=0.0)
    delta_second = W[:, i_second] - s64 * c_rtn[:, i_second]
    want2 = np.clip(np.rint((W[:, i_first] + delta_second * b / H2[i_first, i_first]) / s64), -8, 7)
    assert np.array_equal(codes2[:, i_second], c_rtn[:, i_second]) and np.array_equal(codes2[:, i_first], want2.astype(np.int8))


def test_relabelling_the_channels_relabels_the_codes():
    rng = np.random.default_rng(3)
    n, N = 24, 5
    X = rng.standard_normal((30, n)) * rng.uniform(0.5, 2.0, size=n)
    H = X.T @ X
    W = rng.standard_normal((N, n))
    codes, s = gptq.gptq_quantize(W, H)
    pi = rng.permutation(n)
    codes_p, s_p = gptq.gptq_quantize(W[:, pi], H[np.ix_(pi, pi)])
    assert np.array_equal(s, s_p) and np.array_equal(codes_p, codes[:, pi])


@pytest.mark.parametrize("seed", range(8))
def test_objective_never_above_round_to_nearest(oracle, seed):
    rng = np.random.default_rng(100 + seed)
    n, N = 64, 16
    tokens = [16, 48, 200, 1000][seed % 4]            # rank-deficient and full-rank Hessians
    X = rng.standard_normal((tokens, n))
    X[:, rng.choice(n, 2, replace=False)] *= 20.0     # outlier channels
    X = X @ (np.eye(n) + 0.3 * rng.standard_normal((n, n)) / np.sqrt(n))  # correlated channels
    H = gptq.hessian(X)
    W = rng.standard_normal((N, n)) * 0.02
    codes, s = gptq.gptq_quantize(W, H)
    c_rtn, s_rtn = rtn(oracle, W)
    Hd, _ = gptq.damped(H, 0.01)
    assert gptq.objective(W, codes, s, Hd) <= gptq.objective(W, c_rtn, s_rtn, Hd) * (1 + 1e-12)
    assert gptq.objective(W, codes, s, H) <= gptq.objective(W, c_rtn, s_rtn, H) * (1 + 1e-9)
    assert codes.min() >= -8 and codes.max() <= 7


def test_dead_channel_gets_zero_codes():
    rng = np.random.default_rng(4)
    n, N = 12, 3
    X = rng.standard_normal((40, n))
    X[:, 5] = 0.0
    W = rng.standard_normal((N, n))
    codes, _ = gptq.gptq_quantize(W, gptq.hessian(X))
    assert not codes[:, 5].any()


def test_expanded_hessian_is_rank_deficient_and_the_objective_drops_with_expansion(oracle):
    """Under expansion the rotated activations X H_hat span only K of the K' channels (Sec. 3.1 Remark 1: the null
    space grows by K' - K), so the Hessian has rank <= K; the damping keeps the method defined.  Remark 2 bounds the
    error of this method by a factor sqrt(K / K'): on a synthetic layer the objective, relative to the same layer's energy
    tr(W H W^T), does not grow when the layer is expanded."""
    from paper_2503_17513_b200 import synth

    K, N, tokens = 64, 12, 96
    x = synth.activations(tokens, K, seed=3, tag="gptq-x")
    wb = synth.weights(N, K, seed=3, tag="gptq-w")
    rel = []
    for Kp in (64, 80, 96):   # 80 = 20 x 4, 96 = 12 x 8
        pl = oracle.plan(K, Kp)
        Y = oracle.rotate(pl, x)
        Wt = oracle.rotate(pl, wb)
        H = gptq.hessian(Y)
        assert np.linalg.matrix_rank(H, tol=1e-8 * np.trace(H)) <= K
        codes, s = gptq.gptq_quantize(Wt, H)
        rel.append(gptq.objective(Wt, codes, s, H) / np.einsum("ij,jk,ik->", Wt, H, Wt))
    assert rel[1] <= rel[0] * 1.05 and rel[2] <= rel[0] * 1.05
