"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, and its pure host entry points (plan, status strings, argument rejection that
happens before any CUDA call) behave as documented."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def xq():
    from paper_2503_17513_b200 import build, xq as binding

    build.build_library()
    return binding


def declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(xq_[a-z0-9_]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol(xq):
    names = declared_symbols()
    assert {"xq_prepare_weights", "xq_rotate_quant", "xq_w4a4_gemm", "xq_expanded_linear"} <= names
    L = ctypes.CDLL(xq.LIB_PATH)
    for n in sorted(names):
        assert hasattr(L, n), n
    assert names == set(xq.EXPORTS)  # the binding covers the same names


def test_plan_matches_oracle_plan(xq, oracle):
    for K, Kp in [(2048, 2176), (8192, 8704), (4096, 4352), (14336, 15360), (4096, 4608), (4096, 5120),
                  (4096, 4096), (8192, 8960), (8192, 9728), (8192, 10240), (8192, 12288), (14336, 18432), (14336, 19968),
                  (14336, 22016), (100, 136), (50, 56), (1, 2)]:
        assert xq.xq_hadamard_plan(K, Kp).astuple() == tuple(oracle.plan(K, Kp).__dict__.values())


def test_plan_errors(xq):
    for K, Kp, want in [(0, 8, xq.ERR_INVALID_ARG), (16, 8, xq.ERR_INVALID_ARG), (5, 7, xq.ERR_INVALID_ARG),
                        (4, 6, xq.ERR_UNSUPPORTED_ORDER),
                        # 39936 = 312 x 128: an order-312 factor goes to the general kernel, whose row buffers must fit shared memory
                        (20000, 39936, xq.ERR_UNSUPPORTED_ORDER)]:
        with pytest.raises(xq.XqError) as e:
            xq.xq_hadamard_plan(K, Kp)
        assert e.value.status == want
    assert xq.lib().xq_hadamard_plan(8, 8, None) == xq.ERR_INVALID_ARG


def test_status_strings(xq):
    seen = {xq.status_string(i) for i in range(8)}
    assert len(seen) == 8 and "ok" in seen


def test_null_arguments_rejected_before_any_cuda_call(xq):
    L = xq.lib()
    null = ctypes.c_void_p(0)
    out = ctypes.c_void_p()
    assert L.xq_prepare_weights(null, 4, 8, 8, null, ctypes.byref(out)) == xq.ERR_INVALID_ARG
    assert L.xq_weights_import(null, null, 4, 8, 8, null, ctypes.byref(out)) == xq.ERR_INVALID_ARG
    assert L.xq_weights_export(null, null, null) == xq.ERR_INVALID_ARG
    assert L.xq_weights_info(null, None, None, None, None) == xq.ERR_INVALID_ARG
    assert L.xq_workspace_bytes(4, null) == 0
    assert L.xq_workspace_init(null, 1024, null) == xq.ERR_WORKSPACE
    pl = xq.xq_hadamard_plan(8, 8)
    assert L.xq_rotate_quant(null, 4, 8, ctypes.byref(pl), null, null, null, null) == xq.ERR_INVALID_ARG
    assert L.xq_rotate_quant(null, 0, 8, ctypes.byref(pl), null, null, null, null) == xq.OK  # M = 0 is a no-op
    assert L.xq_w4a4_gemm(null, null, 4, null, null, null, null, 0, null) == xq.ERR_INVALID_ARG
    assert L.xq_expanded_linear(null, 4, 8, null, null, null, 0, null) == xq.ERR_INVALID_ARG
    assert L.xq_expanded_linear_host(null, 4, null, null, null, 0, null) == xq.ERR_INVALID_ARG
    assert L.xq_rotate_quant_asym(null, 4, 8, ctypes.byref(pl), null, null, null, null, null) == xq.ERR_INVALID_ARG
    assert L.xq_rotate_quant_asym(null, 0, 8, ctypes.byref(pl), null, null, null, null, null) == xq.OK
    assert L.xq_w4a4_gemm_asym(null, null, null, 4, null, null, null, null, 0, null) == xq.ERR_INVALID_ARG
    assert L.xq_expanded_linear_asym(null, 4, 8, null, null, null, 0, null) == xq.ERR_INVALID_ARG
    assert L.xq_expanded_linear_host_asym(null, 4, null, null, null, 0, null) == xq.ERR_INVALID_ARG
    hp = xq.xq_hadamard_plan(64, 72)
    assert L.xq_rotate_quant_heads(null, 4, 256, 4, ctypes.byref(hp), null, null, null, null, null) == xq.ERR_INVALID_ARG
    assert L.xq_rotate_quant_heads(null, 0, 256, 4, ctypes.byref(hp), null, null, null, null, null) == xq.OK
    assert L.xq_rotate_quant_heads(null, 0, 256, 1, ctypes.byref(hp), null, null, null, null, null) == xq.ERR_INVALID_ARG
    assert L.xq_prepare_weights_heads(null, 4, 4, 64, 72, null, ctypes.byref(out)) == xq.ERR_INVALID_ARG
    assert L.xq_weights_heads(null) == 0
    assert L.xq_mx_prepare_weights(null, 8, 100, 160, null, ctypes.byref(out)) == xq.ERR_INVALID_ARG
    assert L.xq_mx_weights_import(null, null, 8, 100, 160, null, ctypes.byref(out)) == xq.ERR_INVALID_ARG
    assert L.xq_mx_weights_export(null, null, null) == xq.ERR_INVALID_ARG
    assert L.xq_mx_weights_info(null, None, None, None, None) == xq.ERR_INVALID_ARG
    assert L.xq_mx_workspace_bytes(4, null) == 0
    assert L.xq_mx_rotate_quant(null, 4, 104, ctypes.byref(pl), null, null, null, null) == xq.ERR_INVALID_ARG
    assert L.xq_mx_gemm(null, null, 4, null, null, null, 0, null) == xq.ERR_INVALID_ARG
    assert L.xq_mx_expanded_linear(null, 4, 104, null, null, null, 0, null) == xq.ERR_INVALID_ARG
    assert L.xq_mx_expanded_linear_host(null, 4, null, null, null, 0, null) == xq.ERR_INVALID_ARG
    assert L.xq_mx_gemm_staged(4, null, null, null, 0, null) == xq.ERR_INVALID_ARG
    assert L.xq_mx_rotate_quant_staged(null, 4, 104, null, null, 0, null) == xq.ERR_INVALID_ARG
    assert L.xq_mx_prepare_weights_heads(null, 8, 4, 64, 72, null, ctypes.byref(out)) == xq.ERR_INVALID_ARG
    assert L.xq_mx_weights_heads(null) == 0
    L.xq_mx_weights_free(null)
    assert L.xq_poll_status(null, null) == xq.ERR_WORKSPACE
    L.xq_weights_free(null)  # allowed
