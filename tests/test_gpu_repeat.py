"""The same launch many times over must give the same bits every time.

Every kernel of the path hands shared-memory stages between a copy engine and the warps that read them (and, in the
tile kernels, tensor-memory stages between warps and the tensor core).  A hand-over that is a little too early does not
show in a single comparison with the oracle: it shows as a few channels of one tile that differ in one launch out of
tens or hundreds.  Each case here runs one layer call (pad, rotate, quantize, product: Sec. 3 of the paper) a few
hundred times on the same inputs and requires the bits of the first launch every time; single launches of the same
shapes are held to the oracle in test_gpu_parity.py, test_gpu_tile_shapes.py and test_gpu_mx.py, and the tile kernel's two
forms have a repeated-launch test of their own in test_gpu_tile_shapes.py.
"""
import numpy as np
import pytest
import torch

from paper_2503_17513_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def xq():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2503_17513_b200 import xq as binding

    binding.lib()
    return binding


def dev(a):
    return torch.from_numpy(a.view(np.int16)).cuda()


# (M, N, K, Kp, launches): the decode stream in one-CTA and clustered forms, the tile kernel behind the many-row rotate kernel
INT4_CASES = [(1, 8192, 2048, 2176, 400), (32, 8192, 2048, 2176, 400), (16, 4096, 14336, 15360, 300), (2048, 8192, 2048, 2176, 200),
              (4096, 4096, 4096, 4352, 100)]


@pytest.mark.parametrize("M,N,K,Kp,launches", INT4_CASES)
def test_int4_layer_repeated(xq, M, N, K, Kp, launches):
    x = synth.activations(M, K, seed=51, tag=f"rp{M}", heavy_tail=(M > 32))
    wb = synth.weights(N, K, seed=51, tag=f"rp{N}")
    w = xq.xq_prepare_weights(wb, Kp)
    ws = xq.new_workspace(M, w)
    X = dev(x)
    first = torch.empty((M, N), dtype=torch.int16, device="cuda")
    xq.xq_expanded_linear(X, w, first, ws)
    out = torch.empty_like(first)
    for i in range(launches):
        out.fill_(0x7FC0)
        xq.xq_expanded_linear(X, w, out, ws)
        assert torch.equal(out, first), i
    assert xq.xq_poll_status(ws) == xq.OK


@pytest.mark.parametrize("M,N,K,Kp,launches", [(32, 8192, 2048, 2176, 300), (2048, 8192, 2048, 2176, 200)])
def test_mxfp4_layer_repeated(xq, M, N, K, Kp, launches):
    x = synth.activations(M, K, seed=52, tag=f"rm{M}", heavy_tail=(M > 32))
    w = xq.xq_mx_prepare_weights(synth.weights(N, K, seed=52, tag=f"rm{N}"), Kp)
    ws = xq.new_mx_workspace(M, w)
    X = dev(x)
    first = torch.empty((M, N), dtype=torch.int16, device="cuda")
    xq.xq_mx_expanded_linear(X, w, first, ws)
    out = torch.empty_like(first)
    for i in range(launches):
        out.fill_(0x7FC0)
        xq.xq_mx_expanded_linear(X, w, out, ws)
        assert torch.equal(out, first), i
    assert xq.xq_poll_status(ws) == xq.OK


def test_layers_on_distinct_streams_with_distinct_workspaces(xq):
    """The library's concurrency rule: calls on distinct streams with distinct workspaces may overlap.  Four layers of
    different shapes (tile kernel in both forms, decode stream, host-buffer entry) are issued round-robin on four streams
    without any synchronization between them, forty rounds; every output equals what the same call gives alone."""
    shapes = [(2048, 3072, 2048, 2176), (300, 2048, 2048, 2176), (16, 8192, 2048, 2176), (1024, 2048, 8192, 8704)]
    jobs = []
    for i, (M, N, K, Kp) in enumerate(shapes):
        x = synth.activations(M, K, seed=53, tag=f"cs{i}", heavy_tail=(M > 32))
        w = xq.xq_prepare_weights(synth.weights(N, K, seed=53, tag=f"cs{i}"), Kp)
        ws = xq.new_workspace(M, w)
        X = dev(x)
        alone = torch.empty((M, N), dtype=torch.int16, device="cuda")
        xq.xq_expanded_linear(X, w, alone, ws)
        Xh = torch.from_numpy(x.view(np.int16)).pin_memory()
        Oh = torch.empty((M, N), dtype=torch.int16).pin_memory()
        jobs.append((X, w, ws, alone, torch.empty_like(alone), torch.cuda.Stream(), Xh, Oh))
    torch.cuda.synchronize()
    for rnd in range(40):
        for j, (X, w, ws, alone, out, stream, Xh, Oh) in enumerate(jobs):
            if j == 3:  # the host-buffer entry, as the benchmark's end-to-end step uses it
                xq.xq_expanded_linear_host_enqueue(Xh, w, Oh, ws, stream=stream)
            else:
                xq.xq_expanded_linear(X, w, out, ws, stream=stream)
        if rnd % 8 == 7:
            torch.cuda.synchronize()
            for j, (X, w, ws, alone, out, stream, Xh, Oh) in enumerate(jobs):
                got = Oh.cuda() if j == 3 else out
                assert torch.equal(got, alone), (rnd, j)
                assert xq.xq_poll_status(ws, stream=stream) == xq.OK
