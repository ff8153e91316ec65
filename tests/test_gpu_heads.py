"""GPU parity of the head-wise expanded rotation (paper Sec. 4 "Compute Graph Details", Sec. 5
"Expanding R2 and R4": the rotation in front of the attention output projection acts per head)
against the CPU oracle, through the C ABI.  Same bounds as the single-rotation path.
"""
import numpy as np
import pytest
import torch

from paper_2503_17513_b200 import synth

pytestmark = pytest.mark.gpu

ROT_REL_L2 = 1e-5
CODE_MISMATCH_FRAC = 1e-4
E2E_REL_L2 = 2e-2


@pytest.fixture(scope="module")
def xq():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2503_17513_b200 import xq as binding

    binding.lib()  # fails loudly if the CUDA library is missing
    return binding


def dev(a: np.ndarray) -> torch.Tensor:
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda()
    return torch.from_numpy(a).cuda()


def host_u16(t: torch.Tensor) -> np.ndarray:
    return t.cpu().view(torch.int16).numpy().view(np.uint16)


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    d = np.linalg.norm(b)
    return np.linalg.norm(a - b) / (d if d > 0 else 1.0)


# (M, heads, head_dim, head_dim'): Llama-3.2-1B-like (32 x 64) and Llama-3-8B-like (32 x 128) attention
# outputs at two expansions each, the unexpanded case, few heads, a ragged head tile (24 heads), many tokens.
HEAD_CASES = [
    (5, 4, 64, 72), (3, 32, 64, 72), (40, 32, 64, 80), (3, 32, 128, 144), (200, 32, 128, 160), (2, 8, 128, 128), (9, 128, 16, 16),
    (4, 8, 16, 24), (7, 24, 64, 72), (600, 32, 64, 72),
]


@pytest.mark.parametrize("M,heads,hd,hdp", HEAD_CASES)
@pytest.mark.parametrize("asym", [False, True], ids=["sym", "asym"])
def test_rotate_quant_heads_stage_parity(xq, oracle, M, heads, hd, hdp, asym):
    K, Kp = heads * hd, heads * hdp
    x = synth.activations(M, K, seed=12, tag=f"h{heads}x{hd}", heavy_tail=(M > 8))
    pl = xq.xq_hadamard_plan(hd, hdp)
    Xq = torch.empty((M, Kp // 2), dtype=torch.uint8, device="cuda")
    sx = torch.empty((M,), dtype=torch.float32, device="cuda")
    zp = torch.full((M,), 99, dtype=torch.int32, device="cuda") if asym else None
    Y = torch.empty((M, Kp), dtype=torch.float32, device="cuda")
    xq.xq_rotate_quant_heads(dev(x), heads, pl, Xq, sx, zp, Y)
    torch.cuda.synchronize()
    opl = oracle.plan(hd, hdp)
    if asym:
        y_ref, u_ref, s_ref, z_ref = oracle.rotate_quant_heads_asym(opl, heads, x)
        assert np.array_equal(zp.cpu().numpy() + 8, z_ref)
        want = u_ref.astype(np.int32) - 8
    else:
        y_ref, q_ref, s_ref = oracle.rotate_quant_heads(opl, heads, x)
        want = q_ref.astype(np.int32)
    assert rel_l2(Y.cpu().numpy(), y_ref) <= ROT_REL_L2
    assert np.allclose(sx.cpu().numpy(), s_ref, rtol=2e-6, atol=0)
    diff = oracle.unpack_int4(Xq.cpu().numpy()).astype(np.int32) - want
    assert np.abs(diff).max() <= 1, "codes may differ only by +-1"
    assert np.count_nonzero(diff) / diff.size <= CODE_MISMATCH_FRAC


def test_prepare_weights_heads_parity(xq, oracle):
    N, heads, hd, hdp = 48, 32, 64, 72
    wb = synth.weights(N, heads * hd, seed=13, tag="hw")
    w = xq.xq_prepare_weights_heads(wb, heads, hdp)
    assert (w.N, w.K, w.Kp, w.heads) == (N, heads * hd, heads * hdp, heads)
    assert w.plan.astuple() == xq.xq_hadamard_plan(hd, hdp).astuple()
    codes, s_w = xq.xq_weights_export(w)
    _, codes_ref, s_ref = oracle.rotate_quant_heads(oracle.plan(hd, hdp), heads, wb)
    assert np.allclose(s_w, s_ref, rtol=2e-6)
    diff = codes.astype(np.int32) - codes_ref.astype(np.int32)
    assert np.abs(diff).max() <= 1 and np.count_nonzero(diff) / diff.size <= CODE_MISMATCH_FRAC


E2E_CASES = [
    # (M, N, heads, head_dim, head_dim', heavy): the o_proj shapes of the 1B and 8B models, decode and prefill token counts
    (4, 64, 4, 64, 72, False), (16, 2048, 32, 64, 72, False), (1, 512, 32, 64, 80, False), (32, 256, 32, 128, 144, False),
    (200, 384, 32, 64, 72, True), (130, 256, 32, 128, 160, True),
]


@pytest.mark.parametrize("M,N,heads,hd,hdp,heavy", E2E_CASES)
def test_expanded_linear_heads_end_to_end(xq, oracle, M, N, heads, hd, hdp, heavy):
    K = heads * hd
    x = synth.activations(M, K, seed=14, tag=f"eh{M}", heavy_tail=heavy)
    wb = synth.weights(N, K, seed=14, tag=f"eh{N}")
    w = xq.xq_prepare_weights_heads(wb, heads, hdp)
    ws = xq.new_workspace(M, w)
    out = torch.empty((M, N), dtype=torch.int16, device="cuda")
    X = dev(x)
    xq.xq_expanded_linear(X, w, out, ws)
    assert xq.xq_poll_status(ws) == xq.OK
    out_ref, _ = oracle.expanded_linear_heads(oracle.plan(hd, hdp), heads, x, wb)
    got = synth.bf16_bits_to_f32(host_u16(out))
    want = synth.bf16_bits_to_f32(out_ref)
    assert rel_l2(got, want) <= E2E_REL_L2
    for m in range(M):
        assert rel_l2(got[m], want[m]) <= E2E_REL_L2
    # and both stay close to the unquantized product (the rotation itself changes nothing, Sec. 3)
    ref = oracle.ref_product(x, wb)
    assert rel_l2(got, ref) < 1.0
    # staged calls, the host-buffer entry point and the asymmetric form run on the same object
    Xq = torch.empty((M, w.Kp // 2), dtype=torch.uint8, device="cuda")
    sx = torch.empty((M,), dtype=torch.float32, device="cuda")
    xq.xq_rotate_quant_heads(X, heads, w.plan, Xq, sx)
    out2 = torch.empty_like(out)
    xq.xq_w4a4_gemm(Xq, sx, M, w, out2, ws)
    assert torch.equal(out, out2)
    xh = torch.from_numpy(x.view(np.int16)).pin_memory()
    oh = torch.empty((M, N), dtype=torch.int16).pin_memory()
    xq.xq_expanded_linear_host(xh, w, oh, ws)
    assert torch.equal(oh, out.cpu())
    out3 = torch.empty_like(out)
    xq.xq_expanded_linear_asym(X, w, out3, ws)
    assert rel_l2(synth.bf16_bits_to_f32(host_u16(out3)), ref) < 1.0


def test_heads_argument_errors(xq):
    pl = xq.xq_hadamard_plan(8, 12)
    X = torch.zeros((2, 24), dtype=torch.int16, device="cuda")
    Xq = torch.zeros((2, 18), dtype=torch.uint8, device="cuda")
    sx = torch.zeros((2,), dtype=torch.float32, device="cuda")
    with pytest.raises(xq.XqError) as e:  # 3 heads x 12 channels: the packed row is not a whole number of 16-byte pieces
        xq.xq_rotate_quant_heads(X, 3, pl, Xq, sx)
    assert e.value.status == xq.ERR_UNSUPPORTED_ORDER
    with pytest.raises(xq.XqError) as e:
        xq.xq_prepare_weights_heads(np.zeros((4, 24), np.uint16), 3, 12)
    assert e.value.status == xq.ERR_UNSUPPORTED_ORDER
