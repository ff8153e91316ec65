"""The one-launch form of the layer for M <= 32 tokens (the online step inside the product kernel).

Its arithmetic is the same as that of the two separate calls, so xq_expanded_linear_one_launch must give the very bits that
xq_rotate_quant followed by xq_w4a4_gemm give -- and those two are held to the oracle stage by stage elsewhere
(test_gpu_parity.py); here the fused launch is also compared with the oracle directly.  What is new in the fused
launch is the hand-over of the quantized rows between CTAs (a count of published rows kept in the workspace header,
cleared by the last CTA to leave): the cases reuse one workspace across calls with changing token counts, replay a
captured launch, and mix in launches of the other kernels on the same workspace.
"""
import numpy as np
import pytest
import torch

from paper_2503_17513_b200 import synth

pytestmark = pytest.mark.gpu

E2E_REL_L2 = 2e-2


@pytest.fixture(scope="module")
def xq():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2503_17513_b200 import xq as binding

    binding.lib()
    return binding


def dev(a):
    return torch.from_numpy(a.view(np.int16)).cuda()


def f32(t):
    return synth.bf16_bits_to_f32(t.cpu().numpy().view(np.uint16)).astype(np.float64)


def two_calls(xq, X, w, ws, M, asym=False):
    """The layer as two launches: rotate + quantize into caller arrays, then the product."""
    Xq = torch.empty((M, w.Kp // 2), dtype=torch.uint8, device="cuda")
    sx = torch.empty((M,), dtype=torch.float32, device="cuda")
    out = torch.empty((M, w.N), dtype=torch.int16, device="cuda")
    if asym:
        zp = torch.empty((M,), dtype=torch.int32, device="cuda")
        xq.xq_rotate_quant_asym(X, w.plan, Xq, sx, zp)
        xq.xq_w4a4_gemm_asym(Xq, sx, zp, M, w, out, ws)
    else:
        xq.xq_rotate_quant(X, w.plan, Xq, sx)
        xq.xq_w4a4_gemm(Xq, sx, M, w, out, ws)
    return out


# (M, N, K, Kp): every order-p factor and Sylvester length of the workloads, one-CTA and clustered forms, ragged channels,
# more rows than CTAs (N = 16: a single channel block)
CASES = [
    (1, 2048, 2048, 2176), (8, 3072, 2048, 2176), (32, 2048, 2048, 2176), (17, 8192, 2048, 2176), (32, 2048, 8192, 8704),
    (1, 6144, 4096, 4352), (16, 14336, 4096, 4352), (16, 4096, 14336, 15360), (1, 4096, 14336, 15360), (5, 4096, 4096, 4608),
    (32, 4096, 4096, 5120), (3, 264, 1000, 1152), (32, 16, 2048, 2176),
]


@pytest.mark.parametrize("asym", [False, True], ids=["sym", "asym"])
@pytest.mark.parametrize("M,N,K,Kp", CASES)
def test_one_launch_equals_the_two_calls_and_the_oracle(xq, oracle, M, N, K, Kp, asym):
    x = synth.activations(M, K, seed=31, tag=f"fd{M}")
    wb = synth.weights(N, K, seed=31, tag=f"fd{N}")
    w = xq.xq_prepare_weights(wb, Kp)
    ws = xq.new_workspace(32, w)
    X = dev(x)
    out = torch.empty((M, N), dtype=torch.int16, device="cuda")
    for _ in range(3):  # the same workspace again and again: the row count of one launch must not satisfy the next
        out.fill_(0x7FC0)
        xq.xq_expanded_linear_one_launch(X, w, out, ws, asym=asym)
        assert xq.xq_poll_status(ws) == xq.OK
        assert torch.equal(out, two_calls(xq, X, w, ws, M, asym))
    # the default layer call gives the same bits
    out2 = torch.empty_like(out)
    (xq.xq_expanded_linear_asym if asym else xq.xq_expanded_linear)(X, w, out2, ws)
    assert torch.equal(out, out2)
    ref_bits, _ = (oracle.expanded_linear_asym if asym else oracle.expanded_linear)(oracle.plan(K, Kp), x, wb)
    got, want = f32(out), synth.bf16_bits_to_f32(ref_bits).astype(np.float64)
    assert np.linalg.norm(got - want) <= E2E_REL_L2 * np.linalg.norm(want)
    for m in range(M):
        assert np.linalg.norm(got[m] - want[m]) <= E2E_REL_L2 * np.linalg.norm(want[m])


def test_workspace_shared_by_changing_token_counts_and_other_kernels(xq):
    """One workspace, token counts going up and down, a tensor-core launch (M = 100) and a plain product call in
    between: every fused launch still sees only its own rows."""
    K, Kp, N = 2048, 2176, 1024
    w = xq.xq_prepare_weights(synth.weights(N, K, seed=32, tag="mix"), Kp)
    ws = xq.new_workspace(128, w)
    for i, M in enumerate([32, 1, 7, 100, 32, 2, 16, 1, 100, 31]):
        X = dev(synth.activations(M, K, seed=32, tag=f"mix{i}", heavy_tail=(M > 32)))
        out = torch.full((M, N), 0x7FC0, dtype=torch.int16, device="cuda")
        if M <= 32:
            xq.xq_expanded_linear_one_launch(X, w, out, ws)
        else:
            xq.xq_expanded_linear(X, w, out, ws)
        assert xq.xq_poll_status(ws) == xq.OK
        assert torch.equal(out, two_calls(xq, X, w, ws, M)), (i, M)


def test_replayed_capture_of_the_fused_launch(xq):
    """A captured chain of fused launches (two layers sharing one workspace, as the benchmark's steps do) replayed many
    times with new inputs each time: no host-side reset between replays."""
    K, Kp, N, M = 2048, 2176, 2048, 16
    w1 = xq.xq_prepare_weights(synth.weights(N, K, seed=33, tag="g1"), Kp)
    w2 = xq.xq_prepare_weights(synth.weights(N, K, seed=33, tag="g2"), Kp)
    ws = xq.new_workspace(M, w1)
    X = torch.zeros((M, K), dtype=torch.int16, device="cuda")
    o1 = torch.empty((M, N), dtype=torch.int16, device="cuda")
    o2 = torch.empty((M, N), dtype=torch.int16, device="cuda")
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        xq.xq_expanded_linear_one_launch(X, w1, o1, ws, stream=stream)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for _ in range(4):
                xq.xq_expanded_linear_one_launch(X, w1, o1, ws, stream=stream)
                xq.xq_expanded_linear_one_launch(X, w2, o2, ws, stream=stream)
        for i in range(5):
            X.copy_(dev(synth.activations(M, K, seed=33, tag=f"rep{i}")))
            g.replay()
            stream.synchronize()
            assert xq.xq_poll_status(ws, stream=stream) == xq.OK
            assert torch.equal(o1, two_calls(xq, X, w1, ws, M)) and torch.equal(o2, two_calls(xq, X, w2, ws, M)), i


def test_one_launch_refuses_what_it_does_not_take(xq):
    """Plans outside the tensor-core row routine, and more than 32 tokens, are refused with a status; nothing runs."""
    w = xq.xq_prepare_weights(synth.weights(40, 200, seed=34, tag="r"), 288)  # 288 = 36 x 8: the Sylvester factor is too short
    ws = xq.new_workspace(64, w)
    X = torch.zeros((64, 200), dtype=torch.int16, device="cuda")
    out = torch.zeros((64, 40), dtype=torch.int16, device="cuda")
    for M in (9, 64):
        with pytest.raises(xq.XqError) as e:
            xq.xq_expanded_linear_one_launch(X, w, out, ws, M=M)
        assert e.value.status == xq.ERR_UNSUPPORTED_ORDER
    assert xq.xq_poll_status(ws) == xq.OK
