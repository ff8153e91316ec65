"""The allocation-free entry point, xq_expanded_linear_static, against xq_expanded_linear.

Some users of this library run where device allocation is not allowed while the model is being
served (the host application owns the memory pool, or the serving loop may not touch the
allocator's locks).  For them the library carries its own 4 MiB scratch array.  Both entry points
run the same kernels, so on the same inputs the bf16 outputs must be identical bit for bit -- far
inside the 2e-2 relative-L2 bound the end-to-end tests use, which is checked as well.  The call is
made twice in a row with different inputs: the second call finds the first one's leftovers in the
shared array and must not be affected by them.  Oversized requests must be refused.

This file is collected last on purpose, so that a run that stops at the first failure has
already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2503_17513_b200 import synth

pytestmark = pytest.mark.gpu

E2E_REL_L2 = 2e-2


def _dev(a):
    return torch.from_numpy(a.view(np.int16)).cuda()


def _f32(t):
    return synth.bf16_bits_to_f32(t.cpu().numpy().view(np.uint16)).astype(np.float64)


def test_static_scratch_matches_workspace_path_twice_in_a_row(oracle):
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2503_17513_b200 import xq

    xq.lib()
    K, Kp, N = 2048, 2176, 512
    wb = synth.weights(N, K, seed=5, tag="na")
    w = xq.xq_prepare_weights(wb, Kp)
    # a decode-sized call, then a larger one that takes the tensor-core path, then the first again
    for M, tag in [(16, "a"), (160, "b"), (16, "c")]:
        x_bits = synth.activations(M, K, seed=5, tag=tag, heavy_tail=(M > 32))
        X = _dev(x_bits)
        want = torch.empty((M, N), dtype=torch.int16, device="cuda")
        ws = xq.new_workspace(M, w)
        xq.xq_expanded_linear(X, w, want, ws)
        assert xq.xq_poll_status(ws) == xq.OK
        got = torch.full((M, N), 0x7FC0, dtype=torch.int16, device="cuda")
        xq.xq_expanded_linear_static(X, w, got)
        torch.cuda.synchronize()
        a, b = _f32(got), _f32(want)
        assert np.linalg.norm(a - b) <= E2E_REL_L2 * np.linalg.norm(b)
        assert torch.equal(got, want), "same kernels, same inputs: the outputs are the same bits"
        # and directly against the CPU oracle, within the end-to-end bound of the other tests
        ref_bits, _ = oracle.expanded_linear(oracle.plan(K, Kp), x_bits, wb)
        ref = synth.bf16_bits_to_f32(ref_bits).astype(np.float64)
        assert np.linalg.norm(a - ref) <= E2E_REL_L2 * np.linalg.norm(ref)
        # a warm call takes no device memory: the free amount is the same before and after a second call
        free_before, _ = torch.cuda.mem_get_info()
        xq.xq_expanded_linear_static(X, w, got)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before
        assert torch.equal(got, want)


def test_static_scratch_refuses_what_does_not_fit():
    from paper_2503_17513_b200 import xq

    L = xq.lib()
    K, Kp, N = 2048, 2176, 64
    w = xq.xq_prepare_weights(synth.weights(N, K, seed=6, tag="nb"), Kp)
    M = 4096  # 4096 * 1088 bytes of codes alone exceed the 4 MiB array
    X = torch.zeros((M, K), dtype=torch.int16, device="cuda")
    out = torch.zeros((M, N), dtype=torch.int16, device="cuda")
    vp = ctypes.c_void_p
    assert L.xq_expanded_linear_static(vp(X.data_ptr()), M, K, w.handle, vp(out.data_ptr()), vp(0)) == xq.ERR_WORKSPACE
    assert L.xq_expanded_linear_static(vp(X.data_ptr()), 8, K - 8, w.handle, vp(out.data_ptr()), vp(0)) == xq.ERR_INVALID_ARG
    assert L.xq_expanded_linear_static(vp(0), 8, K, w.handle, vp(out.data_ptr()), vp(0)) == xq.ERR_INVALID_ARG
    assert L.xq_expanded_linear_static(vp(X.data_ptr()), 0, K, w.handle, vp(out.data_ptr()), vp(0)) == xq.OK
