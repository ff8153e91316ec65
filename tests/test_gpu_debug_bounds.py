"""The self-checking build of the library (-DXQ_DEBUG_BOUNDS) over small and ragged shapes.

In that build the product kernels test every computed index before using it (the source range and ring stage of each
weight copy, the stores into the token slice and the partial tiles, the output offsets); a failing test writes
XQ_ERR_BOUNDS into the workspace status word and skips the access, nothing traps.  A memory checker cannot be run
where these tests run, so this build stands in for it: every kernel kind, both forms of the tile kernel and every tile shape are driven through shapes with
ragged tails, the status word must stay clean and the outputs must equal those of the normal build bit for bit.

The debug library is loaded in a child process (XQ_LIBRARY selects it), so that the normal one stays the library of
this process.
"""
import json
import os
import subprocess
import sys

import pytest
import torch

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

# (M, N, K, Kp): the decode stream in one-CTA and clustered forms, with 8, 16 and 32 padded tokens; the three-stage ring;
# every tile shape of the tensor-core kernel with ragged channels and tokens; the general kernel (N not a multiple of 8)
CASES = [
    (1, 16, 104, 136), (8, 37, 136, 144), (3, 2048, 2048, 2176), (12, 1024, 2048, 2176), (32, 2048, 2048, 2176), (17, 384, 4096, 4352),
    (32, 2048, 8192, 8704), (130, 264, 2048, 2176), (384, 9728, 248, 256), (300, 200, 4096, 4608),
    (2048, 4096, 2048, 2176), (2048, 3072, 2048, 2176), (2048, 2048, 8192, 8704), (2048, 8192, 2048, 2176), (33, 257, 64, 64),
]

CHILD = r"""
import json, sys
import numpy as np, torch
from paper_2503_17513_b200 import synth, xq
cases = json.loads(sys.argv[1])
xq.lib()
res = []
for (M, N, K, Kp) in cases:
    x = synth.activations(M, K, seed=41, tag=f"db{M}", heavy_tail=(M > 32))
    wb = synth.weights(N, K, seed=41, tag=f"db{N}")
    w = xq.xq_prepare_weights(wb, Kp)
    ws = xq.new_workspace(M, w)
    X = torch.from_numpy(x.view(np.int16)).cuda()
    rec = {"kind": list(xq.xq_gemm_kernel_info(M, w)), "status": [], "sums": [], "one_launch": []}
    for asym in (False, True):
        out = torch.zeros((M, N), dtype=torch.int16, device="cuda")
        (xq.xq_expanded_linear_asym if asym else xq.xq_expanded_linear)(X, w, out, ws)
        rec["status"].append(int(xq.xq_poll_status(ws)))
        rec["sums"].append(out.cpu().numpy().tobytes().hex() if M * N <= 4096 else
                           [int(v) for v in (out.to(torch.int64) & 0xFFFF).sum(dim=1)[:: max(1, M // 64)].cpu()])
        if M <= 32 and xq.xq_gemm_kernel_info(M, w)[0] == 0:
            try:
                out1 = torch.zeros_like(out)
                xq.xq_expanded_linear_one_launch(X, w, out1, ws, asym=asym)
                rec["status"].append(int(xq.xq_poll_status(ws)))
                rec["one_launch"].append(bool(torch.equal(out, out1)))
            except xq.XqError as e:
                rec["one_launch"].append(f"refused {e.status}")
    res.append(rec)
print("RESULT " + json.dumps(res))
"""


def run_child(library, tile_form):
    env = dict(os.environ)
    if library:
        env["XQ_LIBRARY"] = library
    else:
        env.pop("XQ_LIBRARY", None)
    if tile_form:
        env["XQ_PREFILL_KERNEL"] = tile_form
    else:
        env.pop("XQ_PREFILL_KERNEL", None)
    env["PYTHONPATH"] = ROOT + os.pathsep + env.get("PYTHONPATH", "")
    r = subprocess.run([sys.executable, "-c", CHILD, json.dumps(CASES)], env=env, capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    line = [ln for ln in r.stdout.splitlines() if ln.startswith("RESULT ")][-1]
    return json.loads(line[len("RESULT "):])


def test_debug_build_stays_clean_and_matches_the_normal_build():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2503_17513_b200 import build

    debug_lib = build.build_library(debug_bounds=True)  # no-op when the library is newer than its sources
    kinds = set()
    sums = []
    for tile_form in ("", "ss", "ts"):  # the library's own choice of tile kernel form, the first form only, the second only
        dbg = run_child(debug_lib, tile_form)
        ref = run_child(None, tile_form)
        for case, d, r in zip(CASES, dbg, ref):
            assert all(s == 0 for s in d["status"]), (case, d["status"])  # XQ_OK: neither XQ_ERR_BOUNDS nor a timeout
            assert d["kind"] == r["kind"] and d["sums"] == r["sums"] and d["one_launch"] == r["one_launch"], case
            assert False not in d["one_launch"], case  # the one-launch form, where the plan admits it, gives the same bits
            kinds.add(tuple(d["kind"]))
        sums.append([d["sums"] for d in dbg])
    assert sums[0] == sums[1] == sums[2]  # both forms of the tile kernel give the same bits
    # every kernel kind and every tile shape was reached
    assert {k[0] for k in kinds} == {0, 1, 2, 3}
    assert {(k[1], k[2]) for k in kinds if k[0] == 1} == {(128, 256), (256, 256), (256, 128), (256, 224)}
    assert len({k[1] for k in kinds if k[0] == 3}) >= 3 and all(k[2] == 256 for k in kinds if k[0] == 3)
    assert {k[1] for k in kinds if k[0] == 0} >= {8, 32}  # padded token counts of the decode stream
