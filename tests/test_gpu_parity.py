"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle, stage by stage.

Bounds (from the benchmark spec): rotated fp32 values within relative L2 1e-5; at most 0.01 % of
INT4 codes differ and only by +-1; given identical codes and scales the int32 accumulators are
bit-exact; end-to-end bf16 outputs within relative L2 2e-2.
"""
import ctypes

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


def run_rotate_quant(xq, x_bits, K, Kp, want_y=True, ldx=None):
    M = x_bits.shape[0]
    pl = xq.xq_hadamard_plan(K, Kp)
    if ldx is None and K % 8:
        ldx = (K + 7) // 8 * 8  # row pitch must be a multiple of 8 elements
    if ldx is None:
        X = dev(x_bits)
    else:
        X = torch.zeros((M, ldx), dtype=torch.int16, device="cuda")
        X[:, :K] = dev(x_bits)
    Xq = torch.empty((M, Kp // 2), dtype=torch.uint8, device="cuda")
    sx = torch.empty((M,), dtype=torch.float32, device="cuda")
    Y = torch.empty((M, Kp), dtype=torch.float32, device="cuda") if want_y else None
    xq.xq_rotate_quant(X, pl, Xq, sx, Y, M=M, ldx=X.stride(0))
    torch.cuda.synchronize()
    return Xq.cpu().numpy(), sx.cpu().numpy(), (Y.cpu().numpy() if want_y else None)


def check_codes(oracle, got_packed, want_codes):
    got = oracle.unpack_int4(got_packed)
    diff = got.astype(np.int32) - want_codes.astype(np.int32)
    assert np.abs(diff).max() <= 1, "codes may differ only by +-1"
    frac = np.count_nonzero(diff) / diff.size
    assert frac <= CODE_MISMATCH_FRAC, f"{frac:.2e} of codes differ"
    return frac


# (M, K, Kp): small plans covering every order-p factor, then the workload orders.
ROTATE_CASES = [
    (5, 100, 136), (3, 200, 240), (4, 130, 144), (7, 70, 80), (2, 64, 64), (3, 40, 48), (3, 50, 56), (2, 250, 280),
    (2, 8, 8), (16, 2048, 2176), (3, 8192, 8704), (3, 4096, 4352), (2, 14336, 15360), (3, 4096, 4608),
    (3, 4096, 5120), (3, 4096, 4096), (33, 2048, 2176),
    # many rows: the multi-row-group kernel (several rows per CTA, ragged last pass), every n it takes
    (300, 2048, 2176), (333, 100, 160), (150, 4096, 4352), (100, 8192, 8704), (70, 1000, 1152), (49, 4096, 4608),
    (60, 14336, 15360), (100, 4096, 5120), (80, 5000, 5120),
    # n > 256 and pure Sylvester orders through the folded outer factor
    (50, 4096, 4096), (50, 8192, 12288), (64, 1000, 1024),
    # the expansion sizes of Table 1: 140 x 64 (128 staged input rows), 76 x 128, 20 x 512, 36 x 512, and the two
    # the two largest 8B sizes: 312 x 64 and 344 x 64 (Paley over GF(7^3)), long rows on a large outer factor; 344 and
    # 688 = 344 x 2 through the general kernel
    (3, 8192, 8960), (60, 8192, 8960), (3, 8192, 9728), (60, 8192, 9728), (3, 8192, 10240), (2, 14336, 18432),
    (60, 14336, 18432), (1, 14336, 19968), (170, 14336, 19968), (1, 14336, 22016), (155, 14336, 22016), (5, 300, 344), (70, 600, 688),
]


@pytest.mark.parametrize("M,K,Kp", ROTATE_CASES)
def test_rotate_quant_stage_parity(xq, oracle, M, K, Kp):
    x = synth.activations(M, K, seed=0, tag=f"rq{K}", heavy_tail=(M > 8))
    Xq, sx, Y = run_rotate_quant(xq, x, K, Kp)
    pl = oracle.plan(K, Kp)
    y_ref, codes_ref, s_ref = oracle.rotate_quant(pl, x)
    assert rel_l2(Y, y_ref) <= ROT_REL_L2
    for m in range(M):
        assert rel_l2(Y[m], y_ref[m]) <= ROT_REL_L2
    assert np.allclose(sx, s_ref, rtol=2e-6, atol=0)
    check_codes(oracle, Xq, codes_ref)


def test_rotate_quant_edge_rows(xq, oracle):
    """Zero row (scale 1, codes 0), a single spike, row pitch larger than K, no Y dump."""
    K, Kp = 2048, 2176
    x = synth.activations(6, K, seed=7)
    x[1] = 0
    x[2] = 0
    x[2, 5] = synth.f32_to_bf16_bits(np.array([3.0], dtype=np.float32))[0]
    Xq, sx, _ = run_rotate_quant(xq, x, K, Kp, want_y=False, ldx=K + 64)
    _, codes_ref, s_ref = oracle.rotate_quant(oracle.plan(K, Kp), x)
    assert sx[1] == 1.0 and not Xq[1].any()
    assert np.allclose(sx, s_ref, rtol=2e-6)
    check_codes(oracle, Xq, codes_ref)
    # a single non-zero input spreads to +-7 everywhere
    assert set(np.unique(np.abs(oracle.unpack_int4(Xq[2:3])))) == {7}


GEMM_CASES = [
    # (M, N, K, Kp)
    (1, 16, 100, 136), (3, 100, 200, 240), (8, 37, 130, 144), (5, 130, 70, 80), (33, 257, 64, 64),
    (1, 2048, 2048, 2176), (16, 2048, 2048, 2176), (8, 3072, 2048, 2176), (32, 2048, 8192, 8704),
    (17, 384, 4096, 4352), (160, 256, 2048, 2176), (300, 200, 4096, 4608),
    # tensor-core tiles: ragged token and channel tails, several tiles per CTA, a K tail inside a block
    (130, 264, 2048, 2176), (64, 2048, 8192, 8704), (1100, 4608, 250, 256), (129, 512, 90, 96), (2048, 2048, 2048, 2176),
]


@pytest.mark.parametrize("M,N,K,Kp", GEMM_CASES)
def test_gemm_bit_exact_given_codes(xq, oracle, M, N, K, Kp):
    """Any nibble -8..7 on both sides; accumulators bit-exact, outputs equal the one-rounding epilogue
    up to one bf16 ulp (fp32 vs fp64 product before the rounding)."""
    qx = synth.int4_codes(M, Kp, seed=1, tag=f"x{M}")
    qw = synth.int4_codes(N, Kp, seed=1, tag=f"w{N}")
    s_x = synth.scales(M, seed=1, tag="x")
    s_w = synth.scales(N, seed=1, tag="w")
    w = xq.xq_weights_import(qw, s_w, K)
    codes_back, s_back = xq.xq_weights_export(w)
    assert np.array_equal(codes_back, qw) and np.array_equal(s_back, s_w)
    ws = xq.new_workspace(M, w)
    Xq = dev(oracle.pack_int4(qx))
    out = torch.empty((M, N), dtype=torch.int16, device="cuda")
    acc = torch.empty((M, N), dtype=torch.int32, device="cuda")
    xq.xq_w4a4_gemm(Xq, dev(s_x), M, w, out, ws, acc=acc)
    assert xq.xq_poll_status(ws) == xq.OK
    acc_ref = oracle.gemm_i64(qx, qw)
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
    out_ref = oracle.epilogue(acc_ref, s_x, s_w)
    got = synth.bf16_bits_to_f32(host_u16(out)).astype(np.float64)
    want = synth.bf16_bits_to_f32(out_ref).astype(np.float64)
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0**-7 + 1e-30)
    assert np.mean(got == want) > 0.99
    # without the optional accumulator dump the output is the same
    out2 = torch.empty_like(out)
    xq.xq_w4a4_gemm(Xq, dev(s_x), M, w, out2, ws)
    assert torch.equal(out, out2)


def test_gemm_extreme_codes(xq, oracle):
    M, N, K, Kp = 4, 32, 2048, 2176
    qx = np.full((M, Kp), -8, dtype=np.int8)
    qw = np.full((N, Kp), -8, dtype=np.int8)
    qw[1] = 7
    w = xq.xq_weights_import(qw, np.ones(N, np.float32), K)
    ws = xq.new_workspace(M, w)
    out = torch.empty((M, N), dtype=torch.int16, device="cuda")
    acc = torch.empty((M, N), dtype=torch.int32, device="cuda")
    xq.xq_w4a4_gemm(dev(oracle.pack_int4(qx)), torch.ones(M, device="cuda"), M, w, out, ws, acc=acc)
    a = acc.cpu().numpy()
    assert np.all(a[:, 0] == 64 * Kp) and np.all(a[:, 1] == -56 * Kp)


PREP_CASES = [(24, 100, 136), (40, 200, 240), (130, 130, 144), (64, 2048, 2176), (16, 14336, 15360), (32, 4096, 4096)]


@pytest.mark.parametrize("N,K,Kp", PREP_CASES)
def test_prepare_weights_parity(xq, oracle, N, K, Kp):
    wb = synth.weights(N, K, seed=2, tag=f"p{K}")
    w = xq.xq_prepare_weights(wb, Kp)
    assert (w.N, w.K, w.Kp) == (N, K, Kp)
    codes, s_w = xq.xq_weights_export(w)
    codes_ref, s_ref = oracle.prepare_weights(oracle.plan(K, Kp), wb)
    assert np.allclose(s_w, s_ref, rtol=2e-6)
    diff = codes.astype(np.int32) - codes_ref.astype(np.int32)
    assert np.abs(diff).max() <= 1 and np.count_nonzero(diff) / diff.size <= CODE_MISMATCH_FRAC


E2E_CASES = [
    # (M, N, K, Kp, heavy_tail)
    (4, 24, 100, 136, False), (9, 100, 200, 240, False), (16, 2048, 2048, 2176, False),   # the q_proj-like config
    (1, 512, 2048, 2176, False), (8, 512, 8192, 8704, False), (32, 256, 2048, 2176, False),
    (200, 384, 2048, 2176, True), (130, 256, 4096, 4608, True), (16, 256, 4096, 5120, False),
    (16, 256, 4096, 4096, False),
    # Table 1 sizes
    (8, 256, 8192, 8960, False), (64, 256, 14336, 18432, True), (4, 64, 14336, 19968, False), (2, 32, 14336, 22016, False),
]


@pytest.mark.parametrize("M,N,K,Kp,heavy", E2E_CASES)
def test_expanded_linear_end_to_end(xq, oracle, M, N, K, Kp, heavy):
    x = synth.activations(M, K, seed=0, tag=f"e{M}", heavy_tail=heavy)
    wb = synth.weights(N, K, seed=0, tag=f"e{N}")
    w = xq.xq_prepare_weights(wb, Kp)
    ws = xq.new_workspace(M, w)
    out = torch.empty((M, N), dtype=torch.int16, device="cuda")
    ldx = (K + 7) // 8 * 8
    X = torch.zeros((M, ldx), dtype=torch.int16, device="cuda")
    X[:, :K] = dev(x)
    xq.xq_expanded_linear(X, w, out, ws, M=M, ldx=ldx)
    assert xq.xq_poll_status(ws) == xq.OK
    out_ref, _ = oracle.expanded_linear(oracle.plan(K, Kp), x, wb)
    got = synth.bf16_bits_to_f32(host_u16(out))
    want = synth.bf16_bits_to_f32(out_ref)
    r = rel_l2(got, want)
    assert r <= E2E_REL_L2
    for m in range(M):
        assert rel_l2(got[m], want[m]) <= E2E_REL_L2
    # the host-buffer entry point gives the same bits
    if K % 8 == 0:
        xh = torch.from_numpy(x.view(np.int16)).pin_memory()
        oh = torch.empty((M, N), dtype=torch.int16).pin_memory()
        xq.xq_expanded_linear_host(xh, w, oh, ws)
        assert torch.equal(oh, out.cpu())


def test_argument_errors_on_device(xq):
    K, Kp, N, M = 64, 64, 32, 4
    w = xq.xq_weights_import(synth.int4_codes(N, Kp), synth.scales(N), K)
    ws = xq.new_workspace(M, w)
    out = torch.empty((M, N), dtype=torch.int16, device="cuda")
    Xq = torch.zeros((M, Kp // 2), dtype=torch.uint8, device="cuda")
    sx = torch.ones(M, device="cuda")
    L = xq.lib()
    vp = ctypes.c_void_p
    # workspace too small
    assert L.xq_w4a4_gemm(vp(Xq.data_ptr()), vp(sx.data_ptr()), M, w.handle, vp(out.data_ptr()), vp(0), vp(ws.data_ptr()), 16,
                          vp(0)) == xq.ERR_WORKSPACE
    # misaligned output
    assert L.xq_w4a4_gemm(vp(Xq.data_ptr()), vp(sx.data_ptr()), M, w.handle, vp(out.data_ptr() + 2), vp(0), vp(ws.data_ptr()),
                          ws.numel(), vp(0)) == xq.ERR_INVALID_ARG
    # bad row pitch
    X = torch.zeros((M, K), dtype=torch.int16, device="cuda")
    assert L.xq_expanded_linear(vp(X.data_ptr()), M, K - 8, w.handle, vp(out.data_ptr()), vp(ws.data_ptr()), ws.numel(),
                                vp(0)) == xq.ERR_INVALID_ARG
    # codes outside the nibble range are refused at import
    bad = synth.int4_codes(N, Kp)
    bad[3, 3] = 9
    with pytest.raises(xq.XqError) as e:
        xq.xq_weights_import(bad, synth.scales(N), K)
    assert e.value.status == xq.ERR_INVALID_ARG
    # M = 0 is a no-op
    xq.xq_w4a4_gemm(Xq, sx, 0, w, out, ws)
    xq.xq_expanded_linear(X, w, out, ws, M=0)
    assert xq.xq_poll_status(ws) == xq.OK


def test_bounded_wait_times_out_cleanly(xq):
    """A wait on a barrier nobody signals gives up after about a second, records XQ_ERR_TIMEOUT in
    the workspace status word and leaves the context usable; re-initialising clears the status."""
    K, Kp, N, M = 64, 64, 32, 4
    w = xq.xq_weights_import(synth.int4_codes(N, Kp), synth.scales(N), K)
    ws = xq.new_workspace(M, w)
    assert xq.xq_poll_status(ws) == xq.OK
    xq.xq_selftest_wait_timeout(ws)
    assert xq.xq_poll_status(ws) == xq.ERR_TIMEOUT
    assert xq.xq_poll_status(ws) == xq.ERR_TIMEOUT  # sticky
    xq.xq_workspace_init(ws)
    assert xq.xq_poll_status(ws) == xq.OK
    # the context still works
    out = torch.empty((M, N), dtype=torch.int16, device="cuda")
    xq.xq_w4a4_gemm(torch.zeros((M, Kp // 2), dtype=torch.uint8, device="cuda"), torch.ones(M, device="cuda"), M, w, out, ws)
    assert xq.xq_poll_status(ws) == xq.OK
    assert not out.any()


# Full sizes of the benchmark workloads, in the launch configuration bench.py times (xq_expanded_linear,
# all N, all M): the oracle computes every output of a seeded sample of token rows.
FULL_CASES = [
    # (tag, M, N, K, Kp, heavy, sampled rows)
    ("1b-qkv-m32", 32, 3072, 2048, 2176, False, 32), ("1b-gate-m8", 8, 8192, 2048, 2176, False, 8),
    ("1b-down-m32", 32, 2048, 8192, 8704, False, 8), ("1b-o-m1", 1, 2048, 2048, 2176, False, 1),
    ("1b-up-m2048", 2048, 8192, 2048, 2176, True, 12), ("1b-down-m2048", 2048, 2048, 8192, 8704, True, 6),
    ("8b-qkv-m16", 16, 6144, 4096, 4352, False, 6), ("8b-down-m16", 16, 4096, 14336, 15360, False, 3),
    ("8b-gate-m4096", 4096, 14336, 4096, 4352, True, 4), ("sweep-kp5120-m8192", 8192, 4096, 4096, 5120, True, 6),
    ("sweep-kp4096-m1", 1, 4096, 4096, 4096, False, 1),
]


@pytest.mark.parametrize("tag,M,N,K,Kp,heavy,nsample", FULL_CASES, ids=[c[0] for c in FULL_CASES])
def test_full_size_sampled_rows(xq, oracle, tag, M, N, K, Kp, heavy, nsample):
    x = synth.activations(M, K, seed=0, tag=tag, heavy_tail=heavy)
    wb = synth.weights(N, K, seed=0, tag=tag)
    w = xq.xq_prepare_weights(wb, Kp)
    ws = xq.new_workspace(M, w)
    out = torch.empty((M, N), dtype=torch.int16, device="cuda")
    xq.xq_expanded_linear(dev(x), w, out, ws)
    assert xq.xq_poll_status(ws) == xq.OK
    rows = np.sort(np.random.default_rng(11).choice(M, size=min(nsample, M), replace=False))
    if M > 1:
        rows[-1] = M - 1  # the last (possibly ragged-tile) row is always checked
    pl = oracle.plan(K, Kp)
    qw, s_w = oracle.prepare_weights(pl, wb)
    _, qx, s_x = oracle.rotate_quant(pl, x[rows])
    want_bits = oracle.epilogue(oracle.gemm_i64(qx, qw), s_x, s_w)
    got = synth.bf16_bits_to_f32(host_u16(out[torch.from_numpy(rows).cuda()]))
    want = synth.bf16_bits_to_f32(want_bits)
    for i in range(len(rows)):
        assert rel_l2(got[i], want[i]) <= E2E_REL_L2, (tag, int(rows[i]))
    # weights as prepared on the GPU: the same +-1 / 0.01 % bound as the activations
    codes, s_back = xq.xq_weights_export(w)
    diff = codes.astype(np.int32) - qw.astype(np.int32)
    assert np.abs(diff).max() <= 1 and np.count_nonzero(diff) / diff.size <= CODE_MISMATCH_FRAC
    assert np.allclose(s_back, s_w, rtol=2e-6)
    # The product alone at full size, with no rounding-tie allowance in the way: the codes and scales that the GPU
    # itself made for these rows (the same rotate kernel the layer call ran) and the weights it prepared go through
    # the oracle's integer product and one-rounding epilogue; every output of the layer is within one bf16 ulp.
    Xq_g = torch.empty((M, Kp // 2), dtype=torch.uint8, device="cuda")
    sx_g = torch.empty((M,), dtype=torch.float32, device="cuda")
    xq.xq_rotate_quant(dev(x), w.plan, Xq_g, sx_g)
    ridx = torch.from_numpy(rows).cuda()
    qx_g = oracle.unpack_int4(Xq_g[ridx].cpu().numpy())
    want_g = synth.bf16_bits_to_f32(oracle.epilogue(oracle.gemm_i64(qx_g, codes), sx_g[ridx].cpu().numpy(), s_back)).astype(np.float64)
    got64 = got.astype(np.float64)
    assert np.all(np.abs(got64 - want_g) <= np.abs(want_g) * 2.0**-7 + 1e-30), tag
    assert np.mean(got64 == want_g) > 0.99
