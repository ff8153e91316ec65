"""Bit-exact accumulators on every form and tile shape of the tcgen05 INT4 product kernel, each case naming
the shape it ran on (asked from the library with xq_gemm_kernel_info, nothing is assumed).

The quantized product Q(XR) Q(W~) of the paper's Sec. 3 is an integer sum, so given identical codes
the int32 accumulators must equal the oracle's int64 sums exactly, whatever form, tile shape, tile count
per CTA, K length or tail the launch has.  The kernel has two forms: the first keeps the expanded weights in
shared memory (tiles of 128 tokens x 256 channels, 256 x 256, 256 x 128, 256 x 224), the second in tensor memory
(tiles of 32 .. 192 tokens x 256 channels); the library picks per launch.  Cases here reach every shape at the layer
sizes the benchmark times, and the extreme codes (-8 against -8 and against 7) at the longest K' of the paper's
Table 1, where the 16 x 16 factor carried by the nibble expansion makes the partial sums largest.

Every case names two shapes: the one the library picks by itself and the one it picks when XQ_PREFILL_KERNEL=ss
keeps it to the first form; the last two tests run this file again in child processes, once with that setting and once
with XQ_PREFILL_KERNEL=ts (every case on the second form, whatever its size), so that both forms are held to the oracle
on all the cases.
"""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

from paper_2503_17513_b200 import synth

pytestmark = pytest.mark.gpu

FIRST, SECOND = 1, 3  # xq_gemm_kernel_info's kinds of the two forms
FORCED = os.environ.get("XQ_PREFILL_KERNEL", "")


def check_shape(info, case_default, case_first):
    """info = (kind, tile_tokens, tile_channels) as the library reports it for the case."""
    if FORCED == "ss":
        assert info == case_first
    elif FORCED == "ts":
        assert info[0] == SECOND and info[1] % 32 == 0 and 32 <= info[1] <= 192 and info[2] == 256
    else:
        assert info == case_default


@pytest.fixture(scope="module")
def xq():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2503_17513_b200 import xq as binding

    binding.lib()
    return binding


def dev(a: np.ndarray) -> torch.Tensor:
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda()
    return torch.from_numpy(a).cuda()


def host_u16(t: torch.Tensor) -> np.ndarray:
    return t.cpu().view(torch.int16).numpy().view(np.uint16)


def sample_rows(M, count, seed=13):
    rows = np.sort(np.random.default_rng(seed).choice(M, size=min(count, M), replace=False))
    rows[-1] = M - 1  # the last row of the last tile is always among them
    return rows


# (M, N, K, Kp, shape the library must report, shape with the first form forced, token rows compared: None = all)
TILE_CASES = [
    (384, 9728, 250, 256, (FIRST, 128, 256), (FIRST, 128, 256), None),
    (2048, 8192, 2048, 2176, (SECOND, 160, 256), (FIRST, 256, 224), None),    # gate / up of the 1B prefill workload: ragged last tiles
    (2048, 4096, 2048, 2176, (FIRST, 256, 256), (FIRST, 256, 256), None),
    (512, 14336, 4096, 4352, (FIRST, 256, 224), (FIRST, 256, 224), None),     # all channels of the 8B gate / up (64 x 224)
    (2048, 2048, 8192, 8704, (SECOND, 128, 256), (FIRST, 256, 128), None),    # down of the 1B prefill workload
    (2048, 3072, 2048, 2176, (SECOND, 192, 256), (FIRST, 256, 224), None),    # qkv of the 1B prefill workload: 2048 = 10 x 192 + 128
    (40, 520, 4096, 4352, (SECOND, 64, 256), (FIRST, 256, 128), None),        # one ragged token tile, ragged channels
    (4096, 14336, 4096, 4352, (SECOND, 192, 256), (FIRST, 256, 224), 64),     # the 8B prefill launches as the benchmark times them
    (4096, 6144, 4096, 4352, (SECOND, 192, 256), (FIRST, 256, 256), 64),
    (4096, 4096, 14336, 15360, (SECOND, 160, 256), (FIRST, 256, 256), 64),
    (8192, 4096, 4096, 4096, (SECOND, 192, 256), (FIRST, 256, 128), 64),      # the expansion sweep at its two ends
    (8192, 4096, 4096, 5120, (SECOND, 192, 256), (FIRST, 256, 256), 64),
]


def case_id(c):
    d, f = c[4], c[5]
    return f"M{c[0]}-N{c[1]}-Kp{c[3]}-{d[1]}x{d[2]}k{d[0]}-or-{f[1]}x{f[2]}"


IDS = [case_id(c) for c in TILE_CASES]


@pytest.mark.parametrize("M,N,K,Kp,tile,tile_first,nrows", TILE_CASES, ids=IDS)
def test_tile_shape_accumulators_bit_exact(xq, oracle, M, N, K, Kp, tile, tile_first, nrows):
    qx = synth.int4_codes(M, Kp, seed=21, tag=f"tx{M}")
    qw = synth.int4_codes(N, Kp, seed=21, tag=f"tw{N}")
    s_x = synth.scales(M, seed=21, tag="x")
    s_w = synth.scales(N, seed=21, tag="w")
    w = xq.xq_weights_import(qw, s_w, K)
    check_shape(xq.xq_gemm_kernel_info(M, w), tile, tile_first)
    ws = xq.new_workspace(M, w)
    out = torch.empty((M, N), dtype=torch.int16, device="cuda")
    acc = torch.empty((M, N), dtype=torch.int32, device="cuda")
    xq.xq_w4a4_gemm(dev(oracle.pack_int4(qx)), dev(s_x), M, w, out, ws, acc=acc)
    assert xq.xq_poll_status(ws) == xq.OK
    rows = np.arange(M) if nrows is None else sample_rows(M, nrows)
    ridx = torch.from_numpy(rows).cuda()
    acc_ref = oracle.gemm_i64(qx[rows], qw)
    assert np.array_equal(acc[ridx].cpu().numpy().astype(np.int64), acc_ref)
    want = synth.bf16_bits_to_f32(oracle.epilogue(acc_ref, s_x[rows], s_w)).astype(np.float64)
    got = synth.bf16_bits_to_f32(host_u16(out[ridx])).astype(np.float64)
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0**-7 + 1e-30)  # one bf16 ulp
    assert np.mean(got == want) > 0.99


ASYM_TILE_CASES = [
    (384, 9728, 250, 256, (FIRST, 128, 256), (FIRST, 128, 256), None),
    (2048, 8192, 2048, 2176, (SECOND, 160, 256), (FIRST, 256, 224), 256),
    (2048, 4096, 2048, 2176, (FIRST, 256, 256), (FIRST, 256, 256), 256),
    (2048, 2048, 8192, 8704, (SECOND, 128, 256), (FIRST, 256, 128), 256),
    (2048, 3072, 2048, 2176, (SECOND, 192, 256), (FIRST, 256, 224), 256),
    (4096, 4096, 14336, 15360, (SECOND, 160, 256), (FIRST, 256, 256), 64),
]


@pytest.mark.parametrize("M,N,K,Kp,tile,tile_first,nrows", ASYM_TILE_CASES, ids=[case_id(c) for c in ASYM_TILE_CASES])
def test_tile_shape_zero_point_epilogue_bit_exact(xq, oracle, M, N, K, Kp, tile, tile_first, nrows):
    """The zero-point term of asymmetric tokens (Sec. 4), sum (u - z) qw, on the same tile shapes."""
    ux = (synth.int4_codes(M, Kp, seed=22, tag=f"ux{M}").astype(np.int16) + 8).astype(np.uint8)
    z = (synth.int4_codes(M, 1, seed=22, tag=f"z{M}").astype(np.int32) + 8)[:, 0].copy()
    qw = synth.int4_codes(N, Kp, seed=22, tag=f"w{N}")
    s_x = synth.scales(M, seed=22, tag="x")
    s_w = synth.scales(N, seed=22, tag="w")
    w = xq.xq_weights_import(qw, s_w, K)
    check_shape(xq.xq_gemm_kernel_info(M, w), tile, tile_first)
    ws = xq.new_workspace(M, w)
    Xq = dev(oracle.pack_int4((ux.astype(np.int16) - 8).astype(np.int8)))
    out = torch.empty((M, N), dtype=torch.int16, device="cuda")
    acc = torch.empty((M, N), dtype=torch.int32, device="cuda")
    xq.xq_w4a4_gemm_asym(Xq, dev(s_x), dev((z - 8).astype(np.int32)), M, w, out, ws, acc=acc)
    assert xq.xq_poll_status(ws) == xq.OK
    rows = np.arange(M) if nrows is None else sample_rows(M, nrows)
    ridx = torch.from_numpy(rows).cuda()
    acc_u = oracle.gemm_u_i64(ux[rows], qw)
    acc_ref = acc_u - z[rows, None].astype(np.int64) * qw.astype(np.int64).sum(axis=1)[None, :]
    assert np.array_equal(acc[ridx].cpu().numpy().astype(np.int64), acc_ref)
    want = synth.bf16_bits_to_f32(oracle.epilogue_asym(acc_u, s_x[rows], z[rows], s_w, qw)).astype(np.float64)
    got = synth.bf16_bits_to_f32(host_u16(out[ridx])).astype(np.float64)
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0**-7 + 1e-30)


# (M, N, K, Kp, shape, shape with the first form forced): the largest partial sums the kernel can meet -- every product
# is (-8)(-8) = 64 or (-8)(7) = -56, times 256 inside the tensor core, over the two longest K' of Table 1.
EXTREME_CASES = [
    (64, 256, 14336, 18432, (SECOND, 64, 256), (FIRST, 256, 128)),
    (200, 256, 14336, 22016, (SECOND, 128, 256), (FIRST, 256, 128)),
    (1024, 9472, 14336, 18432, (SECOND, 128, 256), (FIRST, 256, 256)),
    (1024, 9472, 14336, 22016, (SECOND, 128, 256), (FIRST, 256, 256)),
    (384, 9728, 14336, 22016, (SECOND, 128, 256), (FIRST, 128, 256)),
    (512, 14336, 14336, 22016, (FIRST, 256, 224), (FIRST, 256, 224)),
    (4096, 4096, 14336, 22016, (SECOND, 160, 256), (FIRST, 256, 256)),
]


@pytest.mark.parametrize("M,N,K,Kp,tile,tile_first", EXTREME_CASES, ids=[case_id((*c, None)) for c in EXTREME_CASES])
def test_tile_shape_extreme_codes_closed_form(xq, oracle, M, N, K, Kp, tile, tile_first):
    qx = np.full((M, Kp), -8, dtype=np.int8)
    qw = np.full((N, Kp), -8, dtype=np.int8)
    qw[1::3] = 7
    w = xq.xq_weights_import(qw, np.ones(N, np.float32), K)
    check_shape(xq.xq_gemm_kernel_info(M, w), tile, tile_first)
    ws = xq.new_workspace(M, w)
    out = torch.empty((M, N), dtype=torch.int16, device="cuda")
    acc = torch.empty((M, N), dtype=torch.int32, device="cuda")
    xq.xq_w4a4_gemm(dev(oracle.pack_int4(qx)), torch.ones(M, device="cuda"), M, w, out, ws, acc=acc)
    assert xq.xq_poll_status(ws) == xq.OK
    want = np.full(N, 64 * Kp, dtype=np.int64)
    want[1::3] = -56 * Kp
    a = acc.cpu().numpy().astype(np.int64)
    assert np.array_equal(a, np.broadcast_to(want, (M, N)))
    # the outputs: bf16 of the closed form (scales are one)
    got = synth.bf16_bits_to_f32(host_u16(out)).astype(np.float64)
    ref = synth.bf16_bits_to_f32(oracle.epilogue(np.broadcast_to(want, (M, N)).copy(), np.ones(M, np.float32), np.ones(N, np.float32)))
    assert np.array_equal(got, ref.astype(np.float64))


def test_i8_mma_rate_probe_runs_and_reports_its_operations(xq):
    """The tensor-core issue-rate probe (the measured INT8 ceiling of the benchmark) completes, leaves the status
    word clean and counts 2 x 128 x 256 x 32 operations per instruction, four instructions per iteration and SM."""
    w = xq.xq_weights_import(synth.int4_codes(32, 64), synth.scales(32), 64)
    ws = xq.new_workspace(4, w)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    ops = xq.xq_selftest_i8_mma_rate(50, ws)
    assert xq.xq_poll_status(ws) == xq.OK
    assert ops == sms * 50 * 4 * 2 * 128 * 256 * 32


# (M, N, K'): small and odd products -- one K block, eight channels, token counts around the tile sizes of both forms.
# Whatever the library picks for them (the child runs force each form in turn), the sums are exact.
SMALL_CASES = [
    (33, 8, 32), (40, 16, 64), (64, 24, 96), (65, 64, 128), (96, 120, 160), (127, 248, 256), (128, 256, 288), (129, 264, 384),
    (191, 504, 1024), (192, 512, 1152), (193, 520, 2176), (200, 1000, 32), (255, 1032, 64), (256, 8, 2176), (257, 264, 96),
    (300, 120, 1152), (383, 520, 128), (385, 24, 1024), (500, 248, 160), (777, 64, 288), (1000, 16, 384),
]


@pytest.mark.parametrize("asym", [False, True], ids=["sym", "asym"])
@pytest.mark.parametrize("M,N,Kp", SMALL_CASES)
def test_small_and_odd_products_bit_exact(xq, oracle, M, N, Kp, asym):
    qx = synth.int4_codes(M, Kp, seed=23, tag=f"sx{M}_{Kp}")
    qw = synth.int4_codes(N, Kp, seed=23, tag=f"sw{N}_{Kp}")
    s_x = synth.scales(M, seed=23, tag="x")
    s_w = synth.scales(N, seed=23, tag="w")
    w = xq.xq_weights_import(qw, s_w, Kp)
    info = xq.xq_gemm_kernel_info(M, w)
    assert info[0] in (FIRST, SECOND) and (FORCED != "ss" or info[0] == FIRST) and (FORCED != "ts" or info[0] == SECOND)
    ws = xq.new_workspace(M, w)
    out = torch.empty((M, N), dtype=torch.int16, device="cuda")
    acc = torch.empty((M, N), dtype=torch.int32, device="cuda")
    Xq = dev(oracle.pack_int4(qx))
    if asym:
        z = (np.arange(M, dtype=np.int32) % 5) - 2  # zero points of the codes as stored (the unsigned code minus 8)
        xq.xq_w4a4_gemm_asym(Xq, dev(s_x), dev(z), M, w, out, ws, acc=acc)
        acc_ref = oracle.gemm_i64(qx, qw) - z[:, None].astype(np.int64) * qw.astype(np.int64).sum(axis=1)[None, :]
    else:
        xq.xq_w4a4_gemm(Xq, dev(s_x), M, w, out, ws, acc=acc)
        acc_ref = oracle.gemm_i64(qx, qw)
    assert xq.xq_poll_status(ws) == xq.OK
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
    want = synth.bf16_bits_to_f32(oracle.epilogue(acc_ref, s_x, s_w)).astype(np.float64)
    got = synth.bf16_bits_to_f32(host_u16(out)).astype(np.float64)
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0**-7 + 1e-30)  # one bf16 ulp


def test_repeated_launches_give_the_same_bits(xq, oracle):
    """The same product 300 times over (9 tiles per CTA, 34 K blocks per tile: about 3e5 tiles and 1e7 hand-overs of a
    shared-memory stage between the copy engine and the warps that read it): every launch gives the bits of the first,
    and the first agrees with the oracle on sampled rows.  A stage handed back to its producer a little too early shows
    up here as a handful of channels of one tile that differ in one launch out of tens."""
    M, N, K, Kp = 4096, 14336, 4096, 4352
    qx = synth.int4_codes(M, Kp, seed=24, tag="rx")
    qw = synth.int4_codes(N, Kp, seed=24, tag="rw")
    s_x = synth.scales(M, seed=24, tag="x")
    s_w = synth.scales(N, seed=24, tag="w")
    w = xq.xq_weights_import(qw, s_w, K)
    ws = xq.new_workspace(M, w)
    Xq, sx = dev(oracle.pack_int4(qx)), dev(s_x)
    first = torch.empty((M, N), dtype=torch.int16, device="cuda")
    xq.xq_w4a4_gemm(Xq, sx, M, w, first, ws)
    rows = sample_rows(M, 24)
    want = synth.bf16_bits_to_f32(oracle.epilogue(oracle.gemm_i64(qx[rows], qw), s_x[rows], s_w)).astype(np.float64)
    got = synth.bf16_bits_to_f32(host_u16(first[torch.from_numpy(rows).cuda()])).astype(np.float64)
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0**-7 + 1e-30)
    out = torch.empty_like(first)
    for i in range(300):
        out.fill_(0x7FC0)
        xq.xq_w4a4_gemm(Xq, sx, M, w, out, ws)
        assert torch.equal(out, first), i
    assert xq.xq_poll_status(ws) == xq.OK


def rerun_forced(setting):
    env = dict(os.environ, XQ_PREFILL_KERNEL=setting)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.abspath(__file__), "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider"],
                       env=env, cwd=root, capture_output=True, text=True, timeout=3000)
    assert r.returncode == 0, r.stdout[-4000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and "failed" not in r.stdout


@pytest.mark.skipif(FORCED != "", reason="this is a child run")
def test_the_same_cases_with_the_first_form_forced():
    """This file once more in a child process with XQ_PREFILL_KERNEL=ss: the cases that the library gives to the second
    form by default now run (and are compared with the oracle) on the first form's tile shapes."""
    rerun_forced("ss")


@pytest.mark.skipif(FORCED != "", reason="this is a child run")
def test_the_same_cases_with_the_second_form_forced():
    """And with XQ_PREFILL_KERNEL=ts: every case, the small and ragged ones included, on the second form."""
    rerun_forced("ts")
