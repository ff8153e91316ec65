"""GPU parity of the asymmetric-activation calls (paper Sec. 4: per-token asymmetric 4-bit
activations, symmetric per-channel weights) against the CPU oracle, through the C ABI.

The oracle works with the unsigned codes u in 0..15 and zero point z in 0..15; the library stores
both shifted by -8 (c = u - 8, zp = z - 8), which changes no represented value.  Bounds as for
the symmetric path: rotated values within relative L2 1e-5, at most 0.01 % of codes off and only
by +-1, zero points equal, integer accumulators bit-exact given the codes, end-to-end bf16
outputs within relative L2 2e-2.
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


def padded(x_bits, K):
    M = x_bits.shape[0]
    ldx = (K + 7) // 8 * 8
    X = torch.zeros((M, ldx), dtype=torch.int16, device="cuda")
    X[:, :K] = dev(x_bits)
    return X, ldx


def run_rotate_quant_asym(xq, x_bits, K, Kp, want_y=True):
    M = x_bits.shape[0]
    pl = xq.xq_hadamard_plan(K, Kp)
    X, ldx = padded(x_bits, K)
    Xq = torch.empty((M, Kp // 2), dtype=torch.uint8, device="cuda")
    sx = torch.empty((M,), dtype=torch.float32, device="cuda")
    zp = torch.full((M,), 99, dtype=torch.int32, device="cuda")
    Y = torch.empty((M, Kp), dtype=torch.float32, device="cuda") if want_y else None
    xq.xq_rotate_quant_asym(X, pl, Xq, sx, zp, Y, M=M, ldx=ldx)
    torch.cuda.synchronize()
    return Xq.cpu().numpy(), sx.cpu().numpy(), zp.cpu().numpy(), (Y.cpu().numpy() if want_y else None)


# (M, K, Kp): the one-row-per-CTA kernels (general and tensor-core form), the many-row kernel at
# every n it takes, folded and pure Sylvester orders.
ROTATE_CASES = [
    (5, 100, 136), (3, 200, 240), (7, 70, 80), (2, 64, 64), (2, 8, 8), (16, 2048, 2176), (3, 8192, 8704),
    (2, 14336, 15360), (3, 4096, 4608), (3, 4096, 5120), (3, 4096, 4096), (33, 2048, 2176),
    (300, 2048, 2176), (333, 100, 160), (150, 4096, 4352), (100, 8192, 8704), (60, 14336, 15360),
    (100, 4096, 5120), (50, 4096, 4096), (50, 8192, 12288), (64, 1000, 1024), (60, 8192, 8960), (1, 14336, 19968),
]


@pytest.mark.parametrize("M,K,Kp", ROTATE_CASES)
def test_rotate_quant_asym_stage_parity(xq, oracle, M, K, Kp):
    x = synth.activations(M, K, seed=3, tag=f"ra{K}", heavy_tail=(M > 8))
    Xq, sx, zp, Y = run_rotate_quant_asym(xq, x, K, Kp)
    y_ref, u_ref, s_ref, z_ref = oracle.rotate_quant_asym(oracle.plan(K, Kp), x)
    assert rel_l2(Y, y_ref) <= ROT_REL_L2
    assert np.allclose(sx, s_ref, rtol=2e-6, atol=0)
    assert np.array_equal(zp + 8, z_ref)
    u = oracle.unpack_int4(Xq).astype(np.int32) + 8
    assert u.min() >= 0 and u.max() <= 15
    diff = u - u_ref.astype(np.int32)
    assert np.abs(diff).max() <= 1, "codes may differ only by +-1"
    assert np.count_nonzero(diff) / diff.size <= CODE_MISMATCH_FRAC
    # the represented values reproduce the rotated row to within half a step (plus the clamp-free range)
    deq = (u - (zp[:, None] + 8)) * sx[:, None].astype(np.float64)
    assert np.all(np.abs(deq - y_ref) <= 0.5 * sx[:, None] * (1 + 1e-4) + 1e-30)


def test_rotate_quant_asym_edge_rows(xq, oracle):
    """A zero row has scale 1, zero point 0 (stored -8) and codes 0 (stored -8); a shifted row uses
    the range a symmetric quantizer would waste."""
    K, Kp = 2048, 2176
    x = synth.activations(40, K, seed=9)
    x[1] = 0
    x[17] = 0
    for M in (6, 40):  # one row per CTA / many rows per CTA
        Xq, sx, zp, _ = run_rotate_quant_asym(xq, x[:M], K, Kp, want_y=False)
        _, u_ref, s_ref, z_ref = oracle.rotate_quant_asym(oracle.plan(K, Kp), x[:M])
        assert sx[1] == 1.0 and zp[1] == -8 and np.all(oracle.unpack_int4(Xq[1:2]) == -8)
        assert np.allclose(sx, s_ref, rtol=2e-6) and np.array_equal(zp + 8, z_ref)
        u = oracle.unpack_int4(Xq).astype(np.int32) + 8
        assert np.abs(u - u_ref).max() <= 1


GEMM_CASES = [
    # (M, N, K, Kp): decode kernel (one-CTA and clustered forms, ragged channels), the general kernel,
    # tensor-core tiles (both accumulator shapes, ragged tails)
    (1, 16, 100, 136), (3, 100, 200, 240), (8, 37, 130, 144), (33, 257, 64, 64), (1, 2048, 2048, 2176),
    (16, 2048, 2048, 2176), (32, 2048, 8192, 8704), (17, 384, 4096, 4352), (160, 256, 2048, 2176),
    (300, 200, 4096, 4608), (130, 264, 2048, 2176), (1100, 4608, 250, 256), (2048, 2048, 2048, 2176),
]


@pytest.mark.parametrize("M,N,K,Kp", GEMM_CASES)
def test_gemm_asym_bit_exact_given_codes(xq, oracle, M, N, K, Kp):
    """Any unsigned code and any zero point: sum (u - z) qw is bit-exact, outputs equal the
    one-rounding epilogue up to one bf16 ulp."""
    ux = (synth.int4_codes(M, Kp, seed=4, tag=f"ux{M}").astype(np.int16) + 8).astype(np.uint8)
    z = (synth.int4_codes(M, 1, seed=4, tag=f"z{M}").astype(np.int32) + 8)[:, 0].copy()
    qw = synth.int4_codes(N, Kp, seed=4, tag=f"w{N}")
    s_x = synth.scales(M, seed=4, tag="x")
    s_w = synth.scales(N, seed=4, tag="w")
    w = xq.xq_weights_import(qw, s_w, K)
    ws = xq.new_workspace(M, w)
    Xq = dev(oracle.pack_int4((ux.astype(np.int16) - 8).astype(np.int8)))
    zp = dev((z - 8).astype(np.int32))
    out = torch.empty((M, N), dtype=torch.int16, device="cuda")
    acc = torch.empty((M, N), dtype=torch.int32, device="cuda")
    xq.xq_w4a4_gemm_asym(Xq, dev(s_x), zp, M, w, out, ws, acc=acc)
    assert xq.xq_poll_status(ws) == xq.OK
    acc_u = oracle.gemm_u_i64(ux, qw)
    acc_ref = acc_u - z[:, None].astype(np.int64) * qw.astype(np.int64).sum(axis=1)[None, :]
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
    out_ref = oracle.epilogue_asym(acc_u, s_x, z, s_w, qw)
    got = synth.bf16_bits_to_f32(host_u16(out)).astype(np.float64)
    want = synth.bf16_bits_to_f32(out_ref).astype(np.float64)
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0**-7 + 1e-30)
    assert np.mean(got == want) > 0.99
    out2 = torch.empty_like(out)
    xq.xq_w4a4_gemm_asym(Xq, dev(s_x), zp, M, w, out2, ws)
    assert torch.equal(out, out2)
    # a zero point of zero (stored 0, i.e. z = 8 for the oracle) is the symmetric product
    out3 = torch.empty_like(out)
    xq.xq_w4a4_gemm_asym(Xq, dev(s_x), torch.zeros(M, dtype=torch.int32, device="cuda"), M, w, out3, ws)
    xq.xq_w4a4_gemm(Xq, dev(s_x), M, w, out2, ws)
    assert torch.equal(out3, out2)


E2E_CASES = [
    # (M, N, K, Kp, heavy_tail)
    (4, 24, 100, 136, False), (16, 2048, 2048, 2176, False), (1, 512, 2048, 2176, False), (8, 512, 8192, 8704, False),
    (32, 256, 2048, 2176, True), (200, 384, 2048, 2176, True), (130, 256, 4096, 4608, True), (16, 256, 4096, 4096, False),
]


@pytest.mark.parametrize("M,N,K,Kp,heavy", E2E_CASES)
def test_expanded_linear_asym_end_to_end(xq, oracle, M, N, K, Kp, heavy):
    x = synth.activations(M, K, seed=5, tag=f"ea{M}", heavy_tail=heavy)
    wb = synth.weights(N, K, seed=5, tag=f"ea{N}")
    w = xq.xq_prepare_weights(wb, Kp)
    ws = xq.new_workspace(M, w)
    out = torch.empty((M, N), dtype=torch.int16, device="cuda")
    X, ldx = padded(x, K)
    xq.xq_expanded_linear_asym(X, w, out, ws, M=M, ldx=ldx)
    assert xq.xq_poll_status(ws) == xq.OK
    out_ref, _ = oracle.expanded_linear_asym(oracle.plan(K, Kp), x, wb)
    got = synth.bf16_bits_to_f32(host_u16(out))
    want = synth.bf16_bits_to_f32(out_ref)
    assert rel_l2(got, want) <= E2E_REL_L2
    for m in range(M):
        assert rel_l2(got[m], want[m]) <= E2E_REL_L2
    # the staged calls give the same bits as the fused entry point
    pl = xq.xq_hadamard_plan(K, Kp)
    Xq = torch.empty((M, Kp // 2), dtype=torch.uint8, device="cuda")
    sx = torch.empty((M,), dtype=torch.float32, device="cuda")
    zp = torch.empty((M,), dtype=torch.int32, device="cuda")
    xq.xq_rotate_quant_asym(X, pl, Xq, sx, zp, None, M=M, ldx=ldx)
    out2 = torch.empty_like(out)
    xq.xq_w4a4_gemm_asym(Xq, sx, zp, M, w, out2, ws)
    assert torch.equal(out, out2)
    # and so does the host-buffer entry point
    if K % 8 == 0:
        xh = torch.from_numpy(x.view(np.int16)).pin_memory()
        oh = torch.empty((M, N), dtype=torch.int16).pin_memory()
        xq.xq_expanded_linear_host_asym(xh, w, oh, ws)
        assert torch.equal(oh, out.cpu())


def test_asym_is_closer_to_the_unquantized_product_on_shifted_rows(xq, oracle):
    """Rows with a large common offset in the rotated domain (a dominant first input channel maps
    to a constant-sign column pattern only for b = 0, so the offset is built in the rotated domain:
    x = y0 H^T) lose less to the asymmetric quantizer; checked against the fp64 product."""
    M, N, K, Kp = 16, 128, 2048, 2048
    pl = oracle.plan(K, Kp)
    g = np.random.default_rng(11)
    y0 = g.normal(size=(M, Kp)) + 3.0                      # rotated-domain rows in about [0, 6]
    H = oracle.hadamard_dense(pl).astype(np.float64) / np.sqrt(Kp)
    x = synth.f32_to_bf16_bits((y0 @ H.T).astype(np.float32))
    wb = synth.weights(N, K, seed=6, tag="shift")
    w = xq.xq_prepare_weights(wb, Kp)
    ws = xq.new_workspace(M, w)
    X, ldx = padded(x, K)
    o_s = torch.empty((M, N), dtype=torch.int16, device="cuda")
    o_a = torch.empty_like(o_s)
    xq.xq_expanded_linear(X, w, o_s, ws, M=M, ldx=ldx)
    xq.xq_expanded_linear_asym(X, w, o_a, ws, M=M, ldx=ldx)
    ref = oracle.ref_product(x, wb)
    e_s = rel_l2(synth.bf16_bits_to_f32(host_u16(o_s)), ref)
    e_a = rel_l2(synth.bf16_bits_to_f32(host_u16(o_a)), ref)
    assert e_a < e_s


def test_asym_argument_errors(xq):
    K, Kp, N, M = 64, 64, 32, 4
    w = xq.xq_weights_import(synth.int4_codes(N, Kp), synth.scales(N), K)
    ws = xq.new_workspace(M, w)
    pl = xq.xq_hadamard_plan(K, Kp)
    X = torch.zeros((M, K), dtype=torch.int16, device="cuda")
    Xq = torch.zeros((M, Kp // 2), dtype=torch.uint8, device="cuda")
    sx = torch.ones((M,), dtype=torch.float32, device="cuda")
    zp = torch.zeros((M,), dtype=torch.int32, device="cuda")
    out = torch.empty((M, N), dtype=torch.int16, device="cuda")
    with pytest.raises(xq.XqError):
        xq.xq_rotate_quant_asym(X, pl, Xq, sx, None)
    with pytest.raises(xq.XqError):
        xq.xq_w4a4_gemm_asym(Xq, sx, None, M, w, out, ws)
    xq.xq_w4a4_gemm_asym(Xq, sx, zp, 0, w, out, ws)  # M = 0 is a no-op
    xq.xq_rotate_quant_asym(X, pl, Xq, sx, zp, M=0)


FULL_CASES = [
    # (tag, M, N, K, Kp, heavy, sampled rows): full workload sizes in the launch configuration the benchmark times
    ("1b-qkv-m32", 32, 3072, 2048, 2176, False, 8), ("1b-down-m32", 32, 2048, 8192, 8704, False, 4),
    ("1b-up-m2048", 2048, 8192, 2048, 2176, True, 6), ("8b-gate-m4096", 4096, 14336, 4096, 4352, True, 3),
]


@pytest.mark.parametrize("tag,M,N,K,Kp,heavy,nsample", FULL_CASES, ids=[c[0] for c in FULL_CASES])
def test_asym_full_size_sampled_rows(xq, oracle, tag, M, N, K, Kp, heavy, nsample):
    x = synth.activations(M, K, seed=0, tag=tag, heavy_tail=heavy)
    wb = synth.weights(N, K, seed=0, tag=tag)
    w = xq.xq_prepare_weights(wb, Kp)
    ws = xq.new_workspace(M, w)
    out = torch.empty((M, N), dtype=torch.int16, device="cuda")
    xq.xq_expanded_linear_asym(dev(x), w, out, ws)
    assert xq.xq_poll_status(ws) == xq.OK
    rows = np.sort(np.random.default_rng(11).choice(M, size=min(nsample, M), replace=False))
    if M > 1:
        rows[-1] = M - 1
    pl = oracle.plan(K, Kp)
    qw, s_w = oracle.prepare_weights(pl, wb)
    _, ux, s_x, z = oracle.rotate_quant_asym(pl, x[rows])
    want = synth.bf16_bits_to_f32(oracle.epilogue_asym(oracle.gemm_u_i64(ux, qw), s_x, z, s_w, qw))
    got = synth.bf16_bits_to_f32(host_u16(out[torch.from_numpy(rows).cuda()]))
    for i in range(len(rows)):
        assert rel_l2(got[i], want[i]) <= E2E_REL_L2, (tag, int(rows[i]))
