#!/usr/bin/env python
"""Benchmark of the expanded W4A4 linear hot path (rotate+quantize, INT4 GEMM, bf16 epilogue).

One step = one pass of every decoder-layer linear of the workload (all layers, distinct prepared
weights per layer, so the weight stream is larger than L2) over one batch of M synthetic tokens,
each linear running xq_rotate_quant then xq_w4a4_gemm through the C ABI.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--workload 1b-decode|1b-prefill|8b-decode|8b-prefill|sweep] [--tokens M]

With --gpus N > 1 (under torchrun) every rank runs an independent replica (the path has no
exchange step); the value is the sum over ranks divided by the slowest rank's time.
--impl reference times the CPU oracle (tests' checker, as it stands) on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2503_17513_b200 import synth  # noqa: E402

WORKLOADS = {
    # name: (shape table, layers, default M, heavy-tailed activations)
    "1b-decode": (synth.LLAMA_1B, 16, 32, False),
    "1b-prefill": (synth.LLAMA_1B, 16, 2048, True),
    "8b-decode": (synth.LLAMA_8B, 8, 16, False),
    "8b-prefill": (synth.LLAMA_8B, 4, 4096, True),
    "sweep": (synth.SWEEP_4096, 4, 8192, True),
    "table1-1b-down": (synth.TABLE1_1B_DOWN, 8, 2048, True),
    "table1-8b-down": (synth.TABLE1_8B_DOWN, 4, 4096, True),
    "heads-1b-o": (synth.HEADS_1B_O, 32, 32, False),
    "heads-8b-o": (synth.HEADS_8B_O, 16, 16, False),
}
METRIC = "expanded W4A4 linear tokens/s"
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu capture summarised in
# profiles/gemm_decode_1b_decode_m32.txt (mean over the five linears of a layer); other workloads: not captured per launch.
NCU_TRAFFIC_BYTES_PER_LAUNCH = {("1b-decode", 32): 6.57e6}


def measured_peaks():
    """(HBM GB/s, dense INT8 tensor TOP/s, source).  The INT8 figure is the measured bf16 GEMM rate
    (the sustained one: the kernel is timed inside a long step) times the nominal 2:1 ratio."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), 2.0 * float(d.get("bf16_tflops_sustained", d.get("bf16_tflops", 0.0))), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, 2.0 * 1400.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def max_over_ranks(t_local: float, dist, device="cuda") -> float:
    """Slowest rank's time (the job is as slow as its slowest replica)."""
    if dist is None:
        return t_local
    import torch

    tt = torch.tensor([t_local], dtype=torch.float64, device=device)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return float(tt.item())


def whole_job_value(world: int, tokens_per_rank: int, t_step: float) -> float:
    """Tokens per second of the whole job: every rank pushes its own M tokens through the step."""
    return world * tokens_per_rank / t_step


def replica_tag(rank: int, world: int) -> str:
    return f"replica {rank} of {world}"


def host_inputs(table, layers, M, heavy):
    """Seeded host tensors: one activation batch per linear, one weight matrix per (layer, linear).
    Layers beyond the first reuse the first layer's draws rotated by whole rows (distinct memory, same
    distribution) to keep host-side generation short."""
    xs, ws = {}, {}
    for name, (K, Kp, N, *hh) in table.items():
        xs[name] = synth.activations(M, K, seed=0, tag=name, heavy_tail=heavy)
        base = synth.weights(N, K, seed=0, tag=name)
        ws[name] = [np.roll(base, 7 * layer, axis=0) if layer else base for layer in range(layers)]
    return xs, ws


def gemm_bytes(M, K, Kp, N):
    """Algorithmic HBM bytes of one GEMM launch: packed weights + scales, packed activations + scales, bf16 out."""
    return N * Kp // 2 + 4 * N + M * (Kp // 2 + 4) + 2 * M * N


def rotate_bytes(M, K, Kp):
    return M * (2 * K + Kp // 2 + 4)


def run_reference(args, table, layers, M, heavy):
    """CPU oracle on the host cores.  A step is a bounded sample of the workload -- the online path of
    ONE layer's linears for min(M, 32) tokens and min(N, 512) output channels per linear (weights prepared
    beforehand, as on the GPU) -- so that K steps end within minutes whatever K is; tokens/s is scaled
    linearly to all layers, all tokens and all channels (the path is independent per token and channel)."""
    import oracle

    oracle.build()
    Ms = min(M, 32)  # the same sample as the cpu_baseline leg: smaller ones let fixed call overheads dominate the scaled time
    prepared = {}
    xs = {}
    for name, (K, Kp, N, *hh) in table.items():
        Ns = min(N, 512)
        heads = hh[0] if hh else 1
        pl = oracle.plan(K // heads, Kp // heads)
        xs[name] = synth.activations(Ms, K, seed=0, tag=name, heavy_tail=heavy)
        wsample = synth.weights(Ns, K, seed=0, tag=name)
        if args.fmt == "mxfp4":
            _, qw, sw = oracle.rotate_quant_mx(pl, wsample, heads)
        else:
            _, qw, sw = oracle.rotate_quant_heads(pl, heads, wsample)
        prepared[name] = (pl, qw, sw, N / Ns, heads)

    def step():
        t_scaled = 0.0
        for name in table:
            pl, qw, sw, scale, heads = prepared[name]
            t0 = time.perf_counter()
            if args.fmt == "mxfp4":
                _, cx, sx = oracle.rotate_quant_mx(pl, xs[name], heads)
                t1 = time.perf_counter()
                oracle.f64_to_bf16(oracle.gemm_mx(cx, sx, qw, sw))
            elif args.act == "asym":
                _, ux, sx, z = oracle.rotate_quant_heads_asym(pl, heads, xs[name])
                t1 = time.perf_counter()
                oracle.epilogue_asym(oracle.gemm_u_i64(ux, qw), sx, z, sw, qw)
            else:
                _, qx, sx = oracle.rotate_quant_heads(pl, heads, xs[name])
                t1 = time.perf_counter()
                oracle.epilogue(oracle.gemm_i64(qx, qw), sx, sw)
            t2 = time.perf_counter()
            t_scaled += (t1 - t0) + (t2 - t1) * scale
        return t_scaled

    t_begin = time.perf_counter()
    for _ in range(args.warmup):
        step()
        if time.perf_counter() - t_begin > 30.0:
            break
    times = []
    for _ in range(args.steps):  # at most K steps, fewer when K of them would not end within minutes
        times.append(step())
        if time.perf_counter() - t_begin > 150.0:
            break
    t_layer = sum(times) / len(times)
    t_step = t_layer * layers * (M / Ms)
    value = M / t_step
    sample = (f"{len(times)} timed steps; per step: online path of one layer's linears for {Ms} tokens and up to 512 output channels per linear "
              f"(GEMM time scaled to full N), scaled to {layers} layers and M={M}")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus, "steps": len(times),
        "warmup": args.warmup, "ms_per_step": t_step * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64/int64 (oracle)", "data": "synthetic",
        "config": {"workload": f"{args.workload}: {','.join(table)} x {layers} layers, M={M}",
                   "activations": "mxfp4 groups of 32" if args.fmt == "mxfp4" else
                   ("asymmetric per token" if args.act == "asym" else "symmetric per token")},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="1b-decode", choices=sorted(WORKLOADS))
    ap.add_argument("--tokens", type=int, default=None)
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel directly instead of replaying a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--fmt", default="int4", choices=["int4", "mxfp4"],
                    help="number format of weights and activations: INT4 with per-row scales (default) or MXFP4")
    ap.add_argument("--act", default="sym", choices=["sym", "asym"],
                    help="per-token activation quantizer: symmetric (default) or asymmetric with a zero point")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    table, layers, M, heavy = WORKLOADS[args.workload]
    M = args.tokens or M
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        if rank == 0:
            run_reference(args, table, layers, M, heavy)
        return

    import torch

    from paper_2503_17513_b200 import xq

    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local_rank)
    xq.lib()
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    # ---- set-up (untimed): inputs, prepared weights, workspaces --------------------------------
    xs_h, ws_h = host_inputs(table, layers, M, heavy)
    names = list(table)
    X = {n: torch.from_numpy(xs_h[n].view(np.int16)).cuda() for n in names}
    heads_of = {n: (table[n][3] if len(table[n]) > 3 else 1) for n in names}

    mx = args.fmt == "mxfp4"
    if mx:
        assert args.act == "sym", "--fmt mxfp4 has its own quantizer: --act does not apply"

    def prepare(n, l):
        if mx and heads_of[n] > 1:
            return xq.xq_mx_prepare_weights_heads(ws_h[n][l], heads_of[n], table[n][1] // heads_of[n])
        if mx:
            return xq.xq_mx_prepare_weights(ws_h[n][l], table[n][1])
        if heads_of[n] > 1:
            return xq.xq_prepare_weights_heads(ws_h[n][l], heads_of[n], table[n][1] // heads_of[n])
        return xq.xq_prepare_weights(ws_h[n][l], table[n][1])

    Wt = {n: [prepare(n, l) for l in range(layers)] for n in names}
    out = {n: torch.empty((M, table[n][2]), dtype=torch.int16, device="cuda") for n in names}
    wsp = {n: (xq.new_mx_workspace(M, Wt[n][0]) if mx else xq.new_workspace(M, Wt[n][0])) for n in names}
    Xq = {n: torch.empty((M, table[n][1] // 2), dtype=torch.uint8, device="cuda") for n in names}
    sx = {n: torch.empty((M,), dtype=torch.float32, device="cuda") for n in names}
    zp = {n: torch.zeros((M,), dtype=torch.int32, device="cuda") for n in names}
    asym = args.act == "asym"
    weight_bytes = sum(layers * (table[n][2] * table[n][1] // 2) for n in names)
    stream = torch.cuda.Stream()

    def step_linear():
        for l in range(layers):
            for n in names:
                if mx:
                    xq.xq_mx_expanded_linear(X[n], Wt[n][l], out[n], wsp[n], stream=stream)
                elif asym:
                    xq.xq_expanded_linear_asym(X[n], Wt[n][l], out[n], wsp[n], stream=stream)
                else:
                    xq.xq_expanded_linear(X[n], Wt[n][l], out[n], wsp[n], stream=stream)

    def step_rotate_only():
        for l in range(layers):
            for n in names:
                if mx:  # the online step as the layer runs it: straight into the workspace, in the GEMM's input form
                    xq.xq_mx_rotate_quant_staged(X[n], Wt[n][l], wsp[n], stream=stream)
                elif heads_of[n] > 1:
                    xq.xq_rotate_quant_heads(X[n], heads_of[n], Wt[n][l].plan, Xq[n], sx[n], zp[n] if asym else None, stream=stream)
                elif asym:
                    xq.xq_rotate_quant_asym(X[n], Wt[n][l].plan, Xq[n], sx[n], zp[n], stream=stream)
                else:
                    xq.xq_rotate_quant(X[n], Wt[n][l].plan, Xq[n], sx[n], stream=stream)

    def step_gemm_only():
        for l in range(layers):
            for n in names:
                if mx:  # the GEMM kernel alone, on the tokens the full step left quantized in the workspace
                    xq.xq_mx_gemm_staged(M, Wt[n][l], out[n], wsp[n], stream=stream)
                elif asym:
                    xq.xq_w4a4_gemm_asym(Xq[n], sx[n], zp[n], M, Wt[n][l], out[n], wsp[n], stream=stream)
                else:
                    xq.xq_w4a4_gemm(Xq[n], sx[n], M, Wt[n][l], out[n], wsp[n], stream=stream)

    def make_runner(fn):
        with torch.cuda.stream(stream):
            fn()  # eager once (also sets function attributes outside capture)
            stream.synchronize()
            if args.no_graph:
                return fn
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                fn()
            return g.replay

    def timed(run, steps, warmup):
        with torch.cuda.stream(stream):
            for _ in range(warmup):
                run()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            stream.synchronize()
            if dist is not None:
                dist.barrier()
            torch.cuda.synchronize()
            e0.record(stream)
            for _ in range(steps):
                run()
            e1.record(stream)
            stream.synchronize()
            torch.cuda.synchronize()
            if dist is not None:
                dist.barrier()
            return e0.elapsed_time(e1) * 1e-3

    run_main = make_runner(step_linear)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    t_total = timed(run_main, args.steps, args.warmup)
    clocks = sampler.stop() if rank == 0 else None
    t_total = max_over_ranks(t_total, dist)
    t_step = t_total / args.steps
    value = whole_job_value(world, M, t_step)

    # ---- per-kernel timing for the roofline (same launch configuration, same stream) ------------
    n_sub = max(3, min(args.steps, 20))
    t_rot = timed(make_runner(step_rotate_only), n_sub, 3) / n_sub
    t_gemm = timed(make_runner(step_gemm_only), n_sub, 3) / n_sub
    launches_per_step = 2 * layers * len(names)
    hbm_peak, int8_peak, peak_kind = measured_peaks()
    tensor_peak, tensor_note = int8_peak, ": 2 x sustained bf16 GEMM"
    gemm_name = "xq_w4a4_gemm (gemm_prefill_kernel)"
    if mx:
        tensor_peak, tensor_note = 2.0 * int8_peak, ": 4 x sustained bf16 GEMM (FP4 : bf16 nominal ratio)"
        gemm_name = "xq_mx_gemm (gemm_mx_kernel, tcgen05.mma kind::mxf4)"
    gbytes = sum(layers * gemm_bytes(M, *table[n][:3]) for n in names)
    rbytes = sum(layers * rotate_bytes(M, table[n][0], table[n][1]) for n in names)
    ops = sum(layers * 2 * M * table[n][2] * table[n][1] for n in names)
    per_kernel = {"xq_w4a4_gemm": {"ms_per_step": t_gemm * 1e3, "GBps": gbytes / t_gemm / 1e9, "TOPS": ops / t_gemm / 1e12,
                                   "us_per_launch": t_gemm * 1e6 / (layers * len(names))},
                  "xq_rotate_quant": {"ms_per_step": t_rot * 1e3, "GBps": rbytes / t_rot / 1e9,
                                      "us_per_launch": t_rot * 1e6 / (layers * len(names))}}
    if M > 32 and t_gemm >= t_rot:
        # dense contraction: the tensor roofline of its own dtype
        achieved = ops / t_gemm / 1e12
        roofline = {"bound": "tensor", "kernel": gemm_name, "achieved": achieved, "peak": tensor_peak,
                    "unit": "TOP/s", "frac": achieved / tensor_peak, "peak_source": peak_kind + tensor_note,
                    "traffic": None, "per_kernel": per_kernel}
    else:
        if t_gemm >= t_rot:
            dom, dbytes, dt = ("xq_mx_gemm (gemm_mx_kernel)" if mx else "xq_w4a4_gemm (gemm_decode_kernel)"), gbytes, t_gemm
        else:
            dom, dbytes, dt = "xq_rotate_quant (rotate_quant_tc_kernel)", rbytes, t_rot
        achieved = dbytes / dt / 1e9
        traffic = NCU_TRAFFIC_BYTES_PER_LAUNCH.get((args.workload, M)) if dom.startswith("xq_w4a4_gemm") and not asym else None
        roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": hbm_peak, "unit": "GB/s", "frac": achieved / hbm_peak,
                    "peak_source": peak_kind, "traffic": traffic, "traffic_unit": "bytes per launch (ncu)",
                    "algorithmic_bytes_per_launch": dbytes / (layers * len(names)), "per_kernel": per_kernel}

    # ---- end to end through the host-buffer entry point -----------------------------------------
    Xh = {n: torch.from_numpy(xs_h[n].view(np.int16)).pin_memory() for n in names}
    Oh = {n: torch.empty((M, table[n][2]), dtype=torch.int16).pin_memory() for n in names}

    def step_host():
        for l in range(layers):
            for n in names:
                if mx:
                    xq.xq_mx_expanded_linear_host(Xh[n], Wt[n][l], Oh[n], wsp[n], stream=stream)
                elif asym:
                    xq.xq_expanded_linear_host_asym(Xh[n], Wt[n][l], Oh[n], wsp[n], stream=stream)
                else:
                    xq.xq_expanded_linear_host(Xh[n], Wt[n][l], Oh[n], wsp[n], stream=stream)

    e2e_steps = max(3, min(args.steps, 10))
    t_e2e = timed(step_host, e2e_steps, 3) / e2e_steps
    t_e2e = max_over_ranks(t_e2e, dist)
    e2e = {"value": whole_job_value(world, M, t_e2e), "unit": "tokens/s",
           "h2d_bytes_per_step": sum(layers * M * table[n][0] * 2 for n in names),
           "d2h_bytes_per_step": sum(layers * M * table[n][2] * 2 for n in names)}

    for n in names:
        assert xq.xq_poll_status(wsp[n]) == xq.OK

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    cpu_baseline = None
    if not args.no_cpu_baseline and world == 1:
        cpu_baseline = cpu_baseline_leg(table, layers, M, heavy, asym, mx)

    line = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": t_step * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "mxfp4 (e2m1 codes, e8m0 group scales), fp32 accumulate" if mx else "int4 codes, int32 accumulate",
        "data": "synthetic",
        "config": {"workload": f"{args.workload}: {','.join(names)} x {layers} layers, M={M}", "tokens": M, "layers": layers,
                   "activations": "mxfp4 groups of 32" if mx else ("asymmetric per token" if asym else "symmetric per token"),
                   "weight_bytes": weight_bytes, "l2": "weights of one step exceed L2 (126 MB)" if weight_bytes > 126e6 else
                   "weights fit in L2", "cuda_graph": not args.no_graph, "parallelism": "replicas" if world > 1 else "single"},
        "TOPS": ops / t_step / 1e12, "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
        "roofline": roofline, "cpu_baseline": cpu_baseline,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def cpu_baseline_leg(table, layers, M, heavy, asym=False, mx=False):
    """The oracle, as it stands, on the host cores: online path of one layer's linears for a bounded
    token and channel sample, scaled linearly (the path is independent per token and per channel)."""
    import oracle

    oracle.build()
    Ms = min(M, 32)
    t_layer = 0.0
    for name, (K, Kp, N, *hh) in table.items():
        Ns = min(N, 512)
        heads = hh[0] if hh else 1
        pl = oracle.plan(K // heads, Kp // heads)
        x = synth.activations(Ms, K, seed=0, tag=name, heavy_tail=heavy)
        wsample = synth.weights(Ns, K, seed=0, tag=name)
        if mx:
            _, cw, sw = oracle.rotate_quant_mx(pl, wsample, heads)
        else:
            _, qw, sw = oracle.rotate_quant_heads(pl, heads, wsample)
        t0 = time.perf_counter()
        if mx:
            _, cx, sx = oracle.rotate_quant_mx(pl, x, heads)
            t1 = time.perf_counter()
            oracle.f64_to_bf16(oracle.gemm_mx(cx, sx, cw, sw))
        elif asym:
            _, ux, sx, z = oracle.rotate_quant_heads_asym(pl, heads, x)
            t1 = time.perf_counter()
            oracle.epilogue_asym(oracle.gemm_u_i64(ux, qw), sx, z, sw, qw)
        else:
            _, qx, sx = oracle.rotate_quant_heads(pl, heads, x)
            t1 = time.perf_counter()
            oracle.epilogue(oracle.gemm_i64(qx, qw), sx, sw)
        t2 = time.perf_counter()
        t_layer += (t1 - t0) + (t2 - t1) * (N / Ns)
    t_step = t_layer * layers * (M / Ms)
    return {"value": M / t_step, "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"one layer, {Ms} tokens, up to 512 output channels per linear; scaled to {layers} layers, M={M}, full N"}


if __name__ == "__main__":
    main()
