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
