"""GPTQ with act-order on the device (xq_gptq_codes, xq_prepare_weights_gptq) against the numpy oracle (oracle/gptq.py;
paper Sec. 4 "Quantization Details").

Both sides work in fp64 on the same rotated rows and the same Hessian, so the codes agree except where a value lies
within rounding noise of a grid midpoint; such a flip then changes what the later columns of that row are quantized
from, so rows are compared whole: at most a handful of rows may differ, and the objective tr((W - Q) H (W - Q)^T) --
what the method descends on -- agrees to 1e-3 relative either way.
"""
import numpy as np
import pytest
import torch

from oracle import gptq
from paper_2503_17513_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def xq():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2503_17513_b200 import xq as binding

    binding.lib()
    return binding


# (N, K, Kp, calibration tokens): several blocks of 64 with a ragged last one, rank-deficient Hessians (tokens < Kp and the
# expansion itself), one block only, the q_proj-like layer of the first workload
CASES = [(40, 100, 136, 64), (130, 200, 240, 400), (24, 48, 48, 20), (64, 250, 280, 1000), (256, 2048, 2176, 512)]


@pytest.mark.parametrize("N,K,Kp,tokens", CASES)
def test_gptq_codes_match_the_oracle(xq, oracle, N, K, Kp, tokens):
    pl = oracle.plan(K, Kp)
    Y = oracle.rotate(pl, synth.activations(tokens, K, seed=41, tag=f"gq{K}", heavy_tail=True))
    Wt = oracle.rotate(pl, synth.weights(N, K, seed=41, tag=f"gq{N}"))
    H = gptq.hessian(Y)
    c_ref, s_ref = gptq.gptq_quantize(Wt, H, damp=0.01)
    codes, s_w = xq.xq_gptq_codes(Wt, H, damp=0.01)
    assert np.array_equal(s_w, s_ref)
    assert codes.min() >= -8 and codes.max() <= 7
    rows_off = np.count_nonzero(np.any(codes != c_ref, axis=1))
    assert rows_off <= max(1, N // 50), f"{rows_off} of {N} rows differ"
    Hd, _ = gptq.damped(H, 0.01)
    o_dev, o_ref = gptq.objective(Wt, codes, s_w, Hd), gptq.objective(Wt, c_ref, s_ref, Hd)
    assert abs(o_dev - o_ref) <= 1e-3 * o_ref
    # and it is the descent it claims to be: never above round-to-nearest
    c_rtn, s_rtn = oracle.quantize(Wt)
    assert o_dev <= gptq.objective(Wt, c_rtn, s_rtn, Hd)


def test_identity_hessian_gives_round_to_nearest_on_the_device(xq, oracle):
    rng = np.random.default_rng(5)
    Wt = rng.standard_normal((70, 200)) * 0.02
    codes, s_w = xq.xq_gptq_codes(Wt, np.eye(200), damp=0.0)
    c_rtn, s_rtn = oracle.quantize(Wt)
    assert np.array_equal(codes, c_rtn) and np.array_equal(s_w, s_rtn)


def test_dead_channel_and_indefinite_hessian(xq):
    rng = np.random.default_rng(6)
    Wt = rng.standard_normal((16, 72))
    X = rng.standard_normal((100, 72))
    X[:, 9] = 0.0
    codes, _ = xq.xq_gptq_codes(Wt, gptq.hessian(X), damp=0.01)
    assert not codes[:, 9].any()
    bad = -np.eye(72)
    with pytest.raises(xq.XqError) as e:
        xq.xq_gptq_codes(Wt, bad, damp=0.0)
    assert e.value.status == xq.ERR_INVALID_ARG


def test_prepare_weights_gptq_end_to_end(xq, oracle):
    """The whole offline call from bf16 weights: the object it returns serves the layer, and on the calibration
    activations themselves the layer's output is closer to the unquantized product than with round-to-nearest
    weights (the Hessian is exactly those activations' second moment)."""
    N, K, Kp, tokens = 256, 2048, 2176, 256
    x = synth.activations(tokens, K, seed=42, tag="gqe", heavy_tail=True)
    wb = synth.weights(N, K, seed=42, tag="gqe")
    pl = oracle.plan(K, Kp)
    H = gptq.hessian(oracle.rotate(pl, x))
    w_gptq = xq.xq_prepare_weights_gptq(wb, Kp, H, damp=0.01)
    w_rtn = xq.xq_prepare_weights(wb, Kp)
    assert (w_gptq.N, w_gptq.K, w_gptq.Kp) == (N, K, Kp)
    codes, s_w = xq.xq_weights_export(w_gptq)
    # the codes against the oracle run on the oracle's own rotated rows: the device rotated in fp32, so values near a
    # grid midpoint may fall the other way and take the rest of their row with them; the objective still agrees
    Wt = oracle.rotate(pl, wb)
    c_ref, s_ref = gptq.gptq_quantize(Wt, H, damp=0.01)
    assert np.allclose(s_w, s_ref, rtol=2e-6)
    Hd, _ = gptq.damped(H, 0.01)
    o_dev, o_ref = gptq.objective(Wt, codes, s_w, Hd), gptq.objective(Wt, c_ref, s_ref, Hd)
    assert abs(o_dev - o_ref) <= 2e-2 * o_ref
    X = torch.from_numpy(x.view(np.int16)).cuda()
    ref = oracle.ref_product(x, wb)
    errs = []
    for w in (w_gptq, w_rtn):
        ws = xq.new_workspace(tokens, w)
        out = torch.empty((tokens, N), dtype=torch.int16, device="cuda")
        xq.xq_expanded_linear(X, w, out, ws)
        assert xq.xq_poll_status(ws) == xq.OK
        got = synth.bf16_bits_to_f32(out.cpu().numpy().view(np.uint16)).astype(np.float64)
        errs.append(np.linalg.norm(got - ref) / np.linalg.norm(ref))
    assert errs[0] < errs[1]
