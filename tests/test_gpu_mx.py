"""GPU parity of the MXFP4 form (paper Sec. 4 "Quantization Details": OCP microscaling, an E8M0 scale
per group of 32 channels, E2M1 elements) against the CPU oracle, through the C ABI.

Bounds: rotated values rel-L2 <= 1e-5; scale bytes and codes equal to the oracle's except where the
fp32 rotation puts a value across a rounding or power-of-two boundary (<= 0.01 % of codes, then the
two dequantized values are neighbours on the group's grid); given identical codes and scales the
product equals the exact one up to fp32 accumulation (rel-L2 <= 1e-5 before the bf16 rounding, i.e.
bf16 outputs within one ulp); end to end rel-L2 <= 2e-2.
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


def unpack(packed):
    out = np.empty((packed.shape[0], packed.shape[1] * 2), dtype=np.uint8)
    out[:, 0::2] = packed & 0xF
    out[:, 1::2] = packed >> 4
    return out


def pack(codes):
    return (codes[:, 0::2] | (codes[:, 1::2] << 4)).astype(np.uint8)


def check_quantized(oracle, codes, sc, codes_ref, sc_ref):
    """Equal up to boundary effects: few differing entries, and those decode to neighbouring values."""
    assert np.count_nonzero(sc != sc_ref) / sc.size <= CODE_MISMATCH_FRAC
    same_scale = np.repeat(sc == sc_ref, 32, axis=1)
    differ = (codes != codes_ref) & same_scale
    assert np.count_nonzero(differ) / codes.size <= CODE_MISMATCH_FRAC
    lut = oracle.e2m1_value(np.arange(16, dtype=np.uint8))
    grid = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])
    a, b = np.abs(lut[codes[differ]]), np.abs(lut[codes_ref[differ]])
    ia, ib = np.searchsorted(grid, a), np.searchsorted(grid, b)
    assert np.all(np.abs(ia - ib) <= 1)


ROTATE_CASES = [(5, 100, 160), (3, 200, 256), (16, 2048, 2176), (3, 8192, 8704), (2, 14336, 15360), (3, 4096, 4096),
                (300, 2048, 2176), (100, 8192, 8704), (60, 4096, 5120)]


@pytest.mark.parametrize("M,K,Kp", ROTATE_CASES)
def test_mx_rotate_quant_stage_parity(xq, oracle, M, K, Kp):
    x = synth.activations(M, K, seed=15, tag=f"mx{K}", heavy_tail=(M > 8))
    pl = xq.xq_hadamard_plan(K, Kp)
    ldx = (K + 7) // 8 * 8
    X = torch.zeros((M, ldx), dtype=torch.int16, device="cuda")
    X[:, :K] = dev(x)
    codes = torch.empty((M, Kp // 2), dtype=torch.uint8, device="cuda")
    sc = torch.empty((M, Kp // 32), dtype=torch.uint8, device="cuda")
    Y = torch.empty((M, Kp), dtype=torch.float32, device="cuda")
    xq.xq_mx_rotate_quant(X, pl, codes, sc, Y, M=M, ldx=ldx)
    torch.cuda.synchronize()
    y_ref, codes_ref, sc_ref = oracle.rotate_quant_mx(oracle.plan(K, Kp), x)
    assert rel_l2(Y.cpu().numpy(), y_ref) <= ROT_REL_L2
    check_quantized(oracle, unpack(codes.cpu().numpy()), sc.cpu().numpy(), codes_ref, sc_ref)


GEMM_CASES = [
    # (M, N, K, Kp): one tile with a K tail inside the 256-code block, ragged token and channel tails, several tiles per CTA
    (5, 8, 100, 160), (33, 256, 64, 128), (1, 2048, 2048, 2176), (130, 264, 2048, 2176), (300, 512, 4096, 4608),
    (129, 1000, 200, 256), (2048, 2048, 2048, 2176), (16, 512, 8192, 8704), (32, 8192, 2048, 2176), (8, 3072, 2048, 2176),
    (32, 4096, 14336, 15360),
]


@pytest.mark.parametrize("M,N,K,Kp", GEMM_CASES)
def test_mx_gemm_given_codes(xq, oracle, M, N, K, Kp):
    """Random codes and a different random scale for every (row, group): any misplaced scale byte shows."""
    g = np.random.default_rng(1000 * M + N)
    cx = g.integers(0, 16, size=(M, Kp)).astype(np.uint8)
    cw = g.integers(0, 16, size=(N, Kp)).astype(np.uint8)
    sx = g.integers(115, 140, size=(M, Kp // 32)).astype(np.uint8)
    sw = g.integers(115, 140, size=(N, Kp // 32)).astype(np.uint8)
    w = xq.xq_mx_weights_import(pack(cw), sw, K)
    codes_back, sc_back = xq.xq_mx_weights_export(w)
    assert np.array_equal(codes_back, cw) and np.array_equal(sc_back, sw)
    ws = xq.new_mx_workspace(M, w)
    out = torch.empty((M, N), dtype=torch.int16, device="cuda")
    xq.xq_mx_gemm(dev(pack(cx)), dev(sx), M, w, out, ws)
    assert xq.xq_poll_status(ws) == xq.OK
    ref = oracle.gemm_mx(cx, sx, cw, sw)
    got = synth.bf16_bits_to_f32(host_u16(out)).astype(np.float64)
    want = synth.bf16_bits_to_f32(oracle.f64_to_bf16(ref)).astype(np.float64)
    assert rel_l2(got, ref) <= 3e-3            # bf16 rounding of the outputs
    assert rel_l2(got, want) <= 1e-3           # against the one-rounding result: fp32 accumulation only
    rms = np.sqrt(np.mean(ref**2))
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0**-7 + 1e-4 * rms)
    # a second call on the same workspace gives the same bits
    out2 = torch.empty_like(out)
    xq.xq_mx_gemm(dev(pack(cx)), dev(sx), M, w, out2, ws)
    assert torch.equal(out, out2)


def test_mx_prepare_weights_parity(xq, oracle):
    N, K, Kp = 264, 2048, 2176
    wb = synth.weights(N, K, seed=16, tag="mxw")
    w = xq.xq_mx_prepare_weights(wb, Kp)
    assert (w.N, w.K, w.Kp) == (N, K, Kp)
    codes, sc = xq.xq_mx_weights_export(w)
    _, codes_ref, sc_ref = oracle.rotate_quant_mx(oracle.plan(K, Kp), wb)
    check_quantized(oracle, codes, sc, codes_ref, sc_ref)


E2E_CASES = [
    # (M, N, K, Kp, heavy)
    (4, 24, 100, 160, False), (16, 2048, 2048, 2176, False), (1, 512, 2048, 2176, False), (8, 512, 8192, 8704, False),
    (200, 384, 2048, 2176, True), (130, 256, 4096, 4608, True), (300, 256, 14336, 15360, True),
]


@pytest.mark.parametrize("M,N,K,Kp,heavy", E2E_CASES)
def test_mx_expanded_linear_end_to_end(xq, oracle, M, N, K, Kp, heavy):
    x = synth.activations(M, K, seed=17, tag=f"me{M}", heavy_tail=heavy)
    wb = synth.weights(N, K, seed=17, tag=f"me{N}")
    w = xq.xq_mx_prepare_weights(wb, Kp)
    ws = xq.new_mx_workspace(M, w)
    out = torch.empty((M, N), dtype=torch.int16, device="cuda")
    ldx = (K + 7) // 8 * 8
    X = torch.zeros((M, ldx), dtype=torch.int16, device="cuda")
    X[:, :K] = dev(x)
    xq.xq_mx_expanded_linear(X, w, out, ws, M=M, ldx=ldx)
    assert xq.xq_poll_status(ws) == xq.OK
    out_ref, _ = oracle.expanded_linear_mx(oracle.plan(K, Kp), x, wb)
    got = synth.bf16_bits_to_f32(host_u16(out))
    want = synth.bf16_bits_to_f32(out_ref)
    assert rel_l2(got, want) <= E2E_REL_L2
    for m in range(M):
        assert rel_l2(got[m], want[m]) <= E2E_REL_L2
    out3 = torch.empty_like(out)  # the product alone, on the tokens the call above left in the workspace
    xq.xq_mx_gemm_staged(M, w, out3, ws)
    assert torch.equal(out3, out)
    if K % 8 == 0:  # the host-buffer entry point gives the same bits
        xh = torch.from_numpy(x.view(np.int16)).pin_memory()
        oh = torch.empty((M, N), dtype=torch.int16).pin_memory()
        xq.xq_mx_expanded_linear_host(xh, w, oh, ws)
        assert torch.equal(oh, out.cpu())


def test_mx_argument_errors(xq):
    with pytest.raises(xq.XqError) as e:  # K' = 136 is not a whole number of 32-channel groups
        xq.xq_mx_prepare_weights(np.zeros((8, 100), np.uint16), 136)
    assert e.value.status == xq.ERR_UNSUPPORTED_ORDER
    with pytest.raises(xq.XqError) as e:  # N must be a multiple of 8
        xq.xq_mx_prepare_weights(np.zeros((5, 100), np.uint16), 160)
    assert e.value.status == xq.ERR_UNSUPPORTED_ORDER


FULL_CASES = [
    # (tag, M, N, K, Kp, heavy, sampled rows): full workload sizes in the launch configuration the benchmark times
    ("1b-qkv-m32", 32, 3072, 2048, 2176, False, 8), ("1b-down-m32", 32, 2048, 8192, 8704, False, 4),
    ("1b-up-m2048", 2048, 8192, 2048, 2176, True, 6), ("8b-down-m16", 16, 4096, 14336, 15360, False, 2),
    ("8b-gate-m4096", 4096, 14336, 4096, 4352, True, 3),
]


@pytest.mark.parametrize("tag,M,N,K,Kp,heavy,nsample", FULL_CASES, ids=[c[0] for c in FULL_CASES])
def test_mx_full_size_sampled_rows(xq, oracle, tag, M, N, K, Kp, heavy, nsample):
    x = synth.activations(M, K, seed=0, tag=tag, heavy_tail=heavy)
    wb = synth.weights(N, K, seed=0, tag=tag)
    w = xq.xq_mx_prepare_weights(wb, Kp)
    ws = xq.new_mx_workspace(M, w)
    out = torch.empty((M, N), dtype=torch.int16, device="cuda")
    xq.xq_mx_expanded_linear(dev(x), w, out, ws)
    assert xq.xq_poll_status(ws) == xq.OK
    rows = np.sort(np.random.default_rng(11).choice(M, size=min(nsample, M), replace=False))
    if M > 1:
        rows[-1] = M - 1  # the last (possibly ragged-tile) row is always checked
    pl = oracle.plan(K, Kp)
    _, cw, sw = oracle.rotate_quant_mx(pl, wb)
    _, cx, sx = oracle.rotate_quant_mx(pl, x[rows])
    want = synth.bf16_bits_to_f32(oracle.f64_to_bf16(oracle.gemm_mx(cx, sx, cw, sw)))
    got = synth.bf16_bits_to_f32(host_u16(out[torch.from_numpy(rows).cuda()]))
    for i in range(len(rows)):
        assert rel_l2(got[i], want[i]) <= E2E_REL_L2, (tag, int(rows[i]))
    codes, sc = xq.xq_mx_weights_export(w)
    check_quantized(oracle, codes, sc, cw, sw)


HEADS_CASES = [
    # (M, N, heads, head_dim, head_dim'): the R2 + R4 setting of the paper's MXFP4 tables -- head-wise rotation, MXFP4 codes;
    # 72-channel heads make the groups of 32 straddle head boundaries
    (4, 64, 4, 64, 72), (16, 2048, 32, 64, 72), (200, 384, 32, 64, 80), (130, 256, 32, 128, 144),
]


@pytest.mark.parametrize("M,N,heads,hd,hdp", HEADS_CASES)
def test_mx_heads_end_to_end(xq, oracle, M, N, heads, hd, hdp):
    K = heads * hd
    x = synth.activations(M, K, seed=18, tag=f"mh{M}", heavy_tail=(M > 32))
    wb = synth.weights(N, K, seed=18, tag=f"mh{N}")
    w = xq.xq_mx_prepare_weights_heads(wb, heads, hdp)
    assert (w.N, w.K, w.Kp, w.heads) == (N, K, heads * hdp, heads)
    opl = oracle.plan(hd, hdp)
    codes, sc = xq.xq_mx_weights_export(w)
    _, cw, sw = oracle.rotate_quant_mx(opl, wb, heads)
    check_quantized(oracle, codes, sc, cw, sw)
    ws = xq.new_mx_workspace(M, w)
    out = torch.empty((M, N), dtype=torch.int16, device="cuda")
    xq.xq_mx_expanded_linear(dev(x), w, out, ws)
    assert xq.xq_poll_status(ws) == xq.OK
    out_ref, _ = oracle.expanded_linear_mx(opl, x, wb, heads)
    got = synth.bf16_bits_to_f32(host_u16(out))
    want = synth.bf16_bits_to_f32(out_ref)
    assert rel_l2(got, want) <= E2E_REL_L2
    for m in range(M):
        assert rel_l2(got[m], want[m]) <= E2E_REL_L2


def test_mx_edge_rows(xq, oracle):
    """A zero row (unit scale bytes, zero codes), a single spike (every rotated value has the same magnitude: all
    codes +-4 under one shared exponent), tiny and large magnitudes; few rows and many rows (both rotate kernels)."""
    K, Kp = 2048, 2176
    x = synth.activations(64, K, seed=19)
    x[1] = 0
    x[2] = 0
    x[2, 5] = synth.f32_to_bf16_bits(np.array([3.0], dtype=np.float32))[0]
    x[3] = synth.f32_to_bf16_bits((synth.bf16_bits_to_f32(x[3]) * 1e-30).astype(np.float32))
    x[4] = synth.f32_to_bf16_bits((synth.bf16_bits_to_f32(x[4]) * 1e30).astype(np.float32))
    pl = xq.xq_hadamard_plan(K, Kp)
    opl = oracle.plan(K, Kp)
    wb = synth.weights(64, K, seed=19, tag="edge")
    w = xq.xq_mx_prepare_weights(wb, Kp)
    for M in (6, 64):
        codes = torch.empty((M, Kp // 2), dtype=torch.uint8, device="cuda")
        sc = torch.empty((M, Kp // 32), dtype=torch.uint8, device="cuda")
        Y = torch.empty((M, Kp), dtype=torch.float32, device="cuda")
        xq.xq_mx_rotate_quant(dev(x[:M]), pl, codes, sc, Y)
        c, s = unpack(codes.cpu().numpy()), sc.cpu().numpy()
        _, c_ref, s_ref = oracle.rotate_quant_mx(opl, x[:M])
        assert np.all(s[1] == 127) and not c[1].any()
        assert len(set(s[2])) == 1 and set(np.unique(c[2] & 7)) == {6}   # |value| / 2^e = 4 everywhere
        check_quantized(oracle, c, s, c_ref, s_ref)
        # the fused kernels (layer call) see the same rows: outputs against the oracle, row by row
        ws = xq.new_mx_workspace(M, w)
        out = torch.empty((M, 64), dtype=torch.int16, device="cuda")
        xq.xq_mx_expanded_linear(dev(x[:M]), w, out, ws)
        got = synth.bf16_bits_to_f32(host_u16(out)).astype(np.float64)
        want = synth.bf16_bits_to_f32(oracle.expanded_linear_mx(opl, x[:M], wb)[0]).astype(np.float64)
        assert not got[1].any()
        for m in range(M):
            assert rel_l2(got[m], want[m]) <= E2E_REL_L2, m
