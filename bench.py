#!/usr/bin/env python
"""Benchmark of the expanded W4A4 linear hot path (rotate+quantize, INT4 GEMM, bf16 epilogue).

One step = one pass of every decoder-layer linear of the workload (all layers, distinct prepared
weights per layer, so the weight stream is larger than L2) over one batch of M synthetic tokens,
each linear running xq_expanded_linear (rotate + quantize, then the quantized product) through the
C ABI.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--workload 8b-prefill|1b-prefill|8b-decode|1b-decode|sweep|...] [--tokens M]
                  [--only]

The headline (value, config, roofline, e2e, cpu_baseline) is the workload named by --workload
(default: the largest single-GPU configuration, the Llama-3-8B-shaped linears at M = 4096).  Unless
--only is given, the line also carries "per_workload": the other configurations the targets are
stated on (decode shapes against HBM, prefill shapes against the INT8 tensor peak), each with its own
step time and roofline, and for the expansion sweep the output error against the unquantized
product for every K'.

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
# The configurations reported beside the headline: (workload, tokens).
PER_WORKLOAD = [("1b-decode", 32), ("8b-decode", 1), ("8b-decode", 16), ("1b-prefill", 2048), ("sweep", 8192), ("sweep", 1)]
METRIC = "expanded W4A4 linear tokens/s"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = (1590.0, 1400.0)
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel (mean over the linears of a layer), from the
# ncu captures summarised in profiles/ (file named per entry); a workload that was not captured reports null.
NCU_TRAFFIC_BYTES_PER_LAUNCH = {
    ("1b-decode", 32): (6.58e6, "profiles/gemm_decode_1b_decode_m32.txt"),
    ("8b-decode", 16): ((13.47 + 31.32 + 31.32 + 31.49) * 1e6 / 4, "profiles/gemm_decode_8b_decode_m16.txt"),
    ("8b-prefill", 4096): ((31.332352 + 8.125440 + 49.274368 + 75.311360 + 49.238016 + 74.736640 + 106.173952 + 18.625792) * 1e6 / 4,
                           "profiles/gemm_prefill_8b_prefill_m4096.txt"),
    ("1b-prefill", 2048): ((7.913984 + 0.000000 + 6.732544 + 0.000000 + 13.496832 + 0.048640 + 13.496832 + 0.034816 + 26.833408 + 0.000000) * 1e6 / 5,
                           "profiles/gemm_prefill_1b_prefill_m2048.txt"),
}


def measured_peaks():
    """HBM GB/s and the dense INT8 tensor rates derived from the measured bf16 GEMM (burst and sustained, times the
    nominal 2 : 1 ratio of INT8 to bf16), with their source."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            d = json.load(f)
        burst = float(d["bf16_tflops"])
        return {"hbm": float(d["hbm_gbs"]), "int8_burst": 2.0 * burst, "int8_sustained": 2.0 * float(d.get("bf16_tflops_sustained", burst)),
                "source": "measured"}
    except Exception:
        return {"hbm": FALLBACK_HBM_GBS, "int8_burst": 2.0 * FALLBACK_BF16_TFLOPS[0], "int8_sustained": 2.0 * FALLBACK_BF16_TFLOPS[1],
                "source": "fallback"}


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


_BASE_WEIGHTS = {}


def base_weights(name, N, K):
    """One seeded draw per linear (cached: workloads that share a shape table share the draw)."""
    key = (name, N, K)
    if key not in _BASE_WEIGHTS:
        _BASE_WEIGHTS[key] = synth.weights(N, K, seed=0, tag=name)
    return _BASE_WEIGHTS[key]


def layer_weights(name, N, K, layer):
    """Layers beyond the first reuse the first layer's draw rotated by whole rows (distinct memory, same
    distribution) to keep host-side generation short."""
    base = base_weights(name, N, K)
    return np.roll(base, 7 * layer, axis=0) if layer else base


def gemm_bytes(M, K, Kp, N):
    """Algorithmic HBM bytes of one GEMM launch: packed weights + scales, packed activations + scales, bf16 out."""
    return N * Kp // 2 + 4 * N + M * (Kp // 2 + 4) + 2 * M * N


def rotate_bytes(M, K, Kp):
    return M * (2 * K + Kp // 2 + 4)


def reference_sample(args, table, M, heavy):
    """Prepared inputs of the oracle's bounded sample: the online path of ONE layer's linears for min(M, 32) tokens
    and min(N, 512) output channels per linear (weights prepared beforehand, as on the GPU)."""
    import oracle

    oracle.build()
    Ms = min(M, 32)
    prepared, xs = {}, {}
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
        """One pass over the sample; returns (wall seconds, seconds with the product scaled to all N channels)."""
        t_wall = t_scaled = 0.0
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
            t_wall += t2 - t0
            t_scaled += (t1 - t0) + (t2 - t1) * scale
        return t_wall, t_scaled

    return oracle, Ms, step


def run_reference(args, table, layers, M, heavy):
    """CPU oracle on the host cores.  A step is the bounded sample of reference_sample; `ms_per_step` and `steps`
    describe exactly what ran.  The metric is scaled linearly to all layers, all tokens and all channels (the path is
    independent per token and per channel); the factors are printed."""
    oracle, Ms, step = reference_sample(args, table, M, heavy)
    t_begin = time.perf_counter()
    for _ in range(args.warmup):
        step()
        if time.perf_counter() - t_begin > 30.0:
            break
    walls, scaled = [], []
    for _ in range(args.steps):  # at most K steps, fewer when K of them would not end within minutes
        a, b = step()
        walls.append(a)
        scaled.append(b)
        if time.perf_counter() - t_begin > 150.0:
            break
    t_wall = sum(walls) / len(walls)
    t_layer = sum(scaled) / len(scaled)
    t_full = t_layer * layers * (M / Ms)
    value = M / t_full
    sample = (f"per step: online path of one layer's linears for {Ms} tokens and up to 512 output channels per linear; "
              f"the metric scales that to {layers} layers, M={M} and all channels")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus, "steps": len(walls),
        "warmup": args.warmup, "ms_per_step": t_wall * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64/int64 (oracle)", "data": "synthetic",
        "config": workload_config(args, table, layers, M, sum(layers * (v[2] * v[1] // 2) for v in table.values()), args.gpus),
        "sample_scale": {"full_step_over_sample_step": t_full / t_wall, "ms_per_full_step_extrapolated": t_full * 1e3,
                         "tokens_in_sample": Ms, "layers_in_sample": 1},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def workload_config(args, table, layers, M, weight_bytes, world=1):
    """The `config` object; both arms print the same keys."""
    cfg = {"workload": f"{args.workload}: {','.join(table)} x {layers} layers, M={M}", "tokens": M, "layers": layers,
           "activations": "mxfp4 groups of 32" if args.fmt == "mxfp4" else
           ("asymmetric per token" if args.act == "asym" else "symmetric per token"),
           "l2": "inputs of one step exceed L2 (126 MB)", "cuda_graph": not args.no_graph,
           "parallelism": "replicas" if world > 1 else "single"}
    if weight_bytes is not None:
        cfg["weight_bytes"] = weight_bytes
    return cfg


class Bench:
    """Device-side state shared by the workloads of one run (prepared weights are cached per shape table)."""

    def __init__(self, args, rank, local_rank, world, dist):
        import torch

        from paper_2503_17513_b200 import xq

        self.torch, self.xq, self.args = torch, xq, args
        self.rank, self.local_rank, self.world, self.dist = rank, local_rank, world, dist
        self.stream = torch.cuda.Stream()
        self.mx = args.fmt == "mxfp4"
        self.asym = args.act == "asym"
        self.peaks = measured_peaks()
        self._weights = {}
        self.i8_probe = None

    # ---- set-up ---------------------------------------------------------------------------------
    def weights_for(self, table, layers):
        xq = self.xq
        out = {}
        for n, (K, Kp, N, *hh) in table.items():
            heads = hh[0] if hh else 1
            for l in range(layers):
                key = (n, K, Kp, N, heads, l, self.mx)
                if key not in self._weights:
                    wh = layer_weights(n, N, K, l)
                    if self.mx and heads > 1:
                        self._weights[key] = xq.xq_mx_prepare_weights_heads(wh, heads, Kp // heads)
                    elif self.mx:
                        self._weights[key] = xq.xq_mx_prepare_weights(wh, Kp)
                    elif heads > 1:
                        self._weights[key] = xq.xq_prepare_weights_heads(wh, heads, Kp // heads)
                    else:
                        self._weights[key] = xq.xq_prepare_weights(wh, Kp)
                out.setdefault(n, []).append(self._weights[key])
        return out

    def drop_weights(self):
        self._weights.clear()

    def timed(self, run, steps, warmup):
        torch, stream, dist = self.torch, self.stream, self.dist
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

    def make_runner(self, fn):
        torch, stream = self.torch, self.stream
        with torch.cuda.stream(stream):
            fn()  # eager once (also sets function attributes outside capture)
            stream.synchronize()
            if self.args.no_graph:
                return fn
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                fn()
            return g.replay

    def probe_i8_rate(self):
        """INT8 issue rate of the tensor pipe on this device (TOP/s): the library's probe kernel, timed with events."""
        if self.i8_probe is None:
            torch, xq = self.torch, self.xq
            w = xq.xq_weights_import(synth.int4_codes(32, 64), synth.scales(32), 64)
            ws = xq.new_workspace(4, w)
            ops = [0.0]

            def run():
                ops[0] = xq.xq_selftest_i8_mma_rate(20000, ws, stream=self.stream)

            t = self.timed(run, 3, 2) / 3
            assert xq.xq_poll_status(ws) == xq.OK
            self.i8_probe = ops[0] / t / 1e12
        return self.i8_probe

    # ---- one workload ---------------------------------------------------------------------------
    def run(self, workload, M, steps, warmup, headline):
        torch, xq, args, stream, mx, asym = self.torch, self.xq, self.args, self.stream, self.mx, self.asym
        table, layers, M_default, heavy = WORKLOADS[workload]
        M = M or M_default
        names = list(table)
        heads_of = {n: (table[n][3] if len(table[n]) > 3 else 1) for n in names}
        xs_h = {n: synth.activations(M, table[n][0], seed=0, tag=n, heavy_tail=heavy) for n in names}
        X = {n: torch.from_numpy(xs_h[n].view(np.int16)).cuda() for n in names}
        Wt = self.weights_for(table, layers)
        out = {n: torch.empty((M, table[n][2]), dtype=torch.int16, device="cuda") for n in names}
        wsp = {n: (xq.new_mx_workspace(M, Wt[n][0]) if mx else xq.new_workspace(M, Wt[n][0])) for n in names}
        Xq = {n: torch.empty((M, table[n][1] // 2), dtype=torch.uint8, device="cuda") for n in names}
        sx = {n: torch.empty((M,), dtype=torch.float32, device="cuda") for n in names}
        zp = {n: torch.zeros((M,), dtype=torch.int32, device="cuda") for n in names}
        weight_bytes = sum(layers * (table[n][2] * table[n][1] // 2) for n in names)

        def step_linear():
            for l in range(layers):
                for n in names:
                    if mx:
                        xq.xq_mx_expanded_linear(X[n], Wt[n][l], out[n], wsp[n], stream=stream)
                    elif asym:
                        xq.xq_expanded_linear_asym(X[n], Wt[n][l], out[n], wsp[n], stream=stream)
                    elif args.one_launch and M <= 32:
                        xq.xq_expanded_linear_one_launch(X[n], Wt[n][l], out[n], wsp[n], stream=stream)
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

        run_main = self.make_runner(step_linear)
        sampler = ClockSampler(self.local_rank)
        if self.rank == 0:
            sampler.start()
            time.sleep(0.3)
        t_total = self.timed(run_main, steps, warmup)
        clocks = sampler.stop() if self.rank == 0 else None
        t_step = max_over_ranks(t_total, self.dist) / steps
        value = whole_job_value(self.world, M, t_step)

        # ---- per-kernel timing for the roofline (same launch configuration, same stream) --------
        n_sub = max(3, min(steps, 20))
        t_rot = self.timed(self.make_runner(step_rotate_only), n_sub, 3) / n_sub
        t_gemm = self.timed(self.make_runner(step_gemm_only), n_sub, 3) / n_sub
        n_linears = layers * len(names)
        pk = self.peaks
        gbytes = sum(layers * gemm_bytes(M, *table[n][:3]) for n in names)
        rbytes = sum(layers * rotate_bytes(M, table[n][0], table[n][1]) for n in names)
        ops = sum(layers * 2 * M * table[n][2] * table[n][1] for n in names)
        per_kernel = {"xq_w4a4_gemm": {"ms_per_step": t_gemm * 1e3, "GBps": gbytes / t_gemm / 1e9, "TOPS": ops / t_gemm / 1e12,
                                       "us_per_launch": t_gemm * 1e6 / n_linears},
                      "xq_rotate_quant": {"ms_per_step": t_rot * 1e3, "GBps": rbytes / t_rot / 1e9,
                                          "us_per_launch": t_rot * 1e6 / n_linears, "frac_of_hbm": rbytes / t_rot / 1e9 / pk["hbm"]}}
        traffic, traffic_src = NCU_TRAFFIC_BYTES_PER_LAUNCH.get((workload, M), (None, None)) if not (mx or asym) else (None, None)
        if M > 32:
            # dense contraction: the tensor roofline of its own dtype.  `peak` is the measured bf16 burst rate (the product
            # kernel is timed alone, for tens of milliseconds) times the nominal ratio to bf16; the sustained-derived figure
            # and the issue rate the library's own probe kernel measures for this very instruction stand beside it.
            ratio = 4.0 if mx else 2.0
            achieved = ops / t_gemm / 1e12
            peak = pk["int8_burst"] * ratio / 2.0
            roofline = {"bound": "tensor",
                        "kernel": "xq_mx_gemm (gemm_mx_kernel, tcgen05.mma kind::mxf4)" if mx else "xq_w4a4_gemm (gemm_prefill_ts_kernel / gemm_prefill_kernel, tcgen05.mma kind::i8)",
                        "achieved": achieved, "peak": peak, "unit": "TOP/s", "frac": achieved / peak,
                        "peak_source": f"{pk['source']}: {ratio:g} x burst bf16 GEMM",
                        "peak_sustained": pk["int8_sustained"] * ratio / 2.0, "frac_of_sustained": achieved / (pk["int8_sustained"] * ratio / 2.0),
                        "traffic": traffic, "traffic_source": traffic_src}
            if not mx:
                probe = self.probe_i8_rate()
                roofline.update({"peak_probe": probe, "frac_of_probe": achieved / probe,
                                 "peak_probe_source": "tcgen05.mma kind::i8 128x256x32 issue loop on resident operands, timed here",
                                 "frac_of_nominal": achieved / 4500.0})
        else:
            if t_gemm >= t_rot:
                dom, dbytes, dt = ("xq_mx_gemm (gemm_mx_decode_kernel)" if mx else "xq_w4a4_gemm (gemm_decode_kernel)"), gbytes, t_gemm
            else:
                dom, dbytes, dt = "xq_rotate_quant (rotate_quant_tc_kernel)", rbytes, t_rot
                traffic = None
            achieved = dbytes / dt / 1e9
            roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": pk["hbm"], "unit": "GB/s", "frac": achieved / pk["hbm"],
                        "peak_source": pk["source"], "traffic": traffic, "traffic_source": traffic_src,
                        "traffic_unit": "bytes per launch (ncu)", "algorithmic_bytes_per_launch": dbytes / n_linears,
                        # the whole step (rotate + product of every linear) against the weight stream it has to move
                        "whole_step_weight_GBps": weight_bytes / t_step / 1e9, "whole_step_frac_of_hbm": weight_bytes / t_step / 1e9 / pk["hbm"]}
        roofline["per_kernel"] = per_kernel

        res = {"workload": workload, "tokens": M, "layers": layers, "linears": names, "ms_per_step": t_step * 1e3, "tokens_per_s": value,
               "us_per_linear": t_step * 1e6 / n_linears, "TOPS": ops / t_step / 1e12, "weight_bytes": weight_bytes, "gpu_launches_per_step": 2 * n_linears,
               "clocks": clocks, "roofline": roofline}

        if workload == "sweep" and not mx and self.rank == 0 and not args.no_cpu_baseline:
            res["error_vs_unquantized"] = self.sweep_error(table, names, xs_h, out, M)

        if headline:
            # ---- end to end through the host-buffer entry point: inputs from pinned host memory, outputs back to it ----
            Xh = {n: torch.from_numpy(xs_h[n].view(np.int16)).pin_memory() for n in names}
            Oh = {n: torch.empty((M, table[n][2]), dtype=torch.int16).pin_memory() for n in names}

            # One stream per linear of a layer (each with its own workspace and host buffers, as the library's concurrency
            # rule asks): the upload of one linear, the kernels of another and the download of a third overlap.  The streams
            # fork from and join the timing stream through events; one host synchronization per step.
            side = {n: torch.cuda.Stream() for n in names} if not (mx or asym) else {}
            fork, joins = torch.cuda.Event(), {n: torch.cuda.Event() for n in side}

            def step_host():
                if side:
                    fork.record(stream)
                    for n in names:
                        side[n].wait_event(fork)
                for l in range(layers):
                    for n in names:
                        if mx:
                            xq.xq_mx_expanded_linear_host(Xh[n], Wt[n][l], Oh[n], wsp[n], stream=stream)
                        elif asym:
                            xq.xq_expanded_linear_host_asym(Xh[n], Wt[n][l], Oh[n], wsp[n], stream=stream)
                        else:  # enqueued back to back; one synchronization per step (below) before the outputs count as read
                            xq.xq_expanded_linear_host_enqueue(Xh[n], Wt[n][l], Oh[n], wsp[n], stream=side[n])
                for n in side:
                    joins[n].record(side[n])
                    stream.wait_event(joins[n])
                stream.synchronize()

            e2e_steps = max(3, min(steps, 10))
            t_e2e = max_over_ranks(self.timed(step_host, e2e_steps, 3) / e2e_steps, self.dist)
            res["e2e"] = {"value": whole_job_value(self.world, M, t_e2e), "unit": "tokens/s", "ms_per_step": t_e2e * 1e3,
                          "h2d_bytes_per_step": sum(layers * M * table[n][0] * 2 for n in names),
                          "d2h_bytes_per_step": sum(layers * M * table[n][2] * 2 for n in names),
                          "streams": max(1, len(side))}
        for n in names:
            assert xq.xq_poll_status(wsp[n]) == xq.OK
        return res

    def sweep_error(self, table, names, xs_h, out, M):
        """Config 5's second axis: relative L2 error of the layer's INT4 output against the unquantized product of the
        same bf16 inputs (fp64, the oracle's plain x W^T) for every K' of the sweep, on a seeded sample of token rows."""
        import oracle

        oracle.build()
        torch = self.torch
        rows = np.sort(np.random.default_rng(5).choice(M, size=min(64, M), replace=False))
        ridx = torch.from_numpy(rows).cuda()
        res = {}
        for n in names:
            K, Kp, N = table[n][:3]
            # `out` holds the last layer's result of the timed step
            wb = layer_weights(n, N, K, WORKLOADS["sweep"][1] - 1)
            ref = oracle.ref_product(xs_h[n][rows], wb)
            got = synth.bf16_bits_to_f32(out[n][ridx].cpu().numpy().view(np.uint16)).astype(np.float64)
            res[str(Kp)] = {"rel_l2": float(np.linalg.norm(got - ref) / np.linalg.norm(ref)), "rows": int(len(rows)),
                            "sqrt_K_over_Kp": float(np.sqrt(K / Kp))}
        return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="8b-prefill", choices=sorted(WORKLOADS))
    ap.add_argument("--tokens", type=int, default=None)
    ap.add_argument("--only", action="store_true", help="time the named workload alone (no per_workload object)")
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel directly instead of replaying a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--gptq-report", action="store_true",
                    help="instead of timing: GPTQ (act-order) against round-to-nearest on the down projection at the paper's "
                         "Table 1 sizes of the 1B model, objective relative to the layer's energy per K' (one JSON line)")
    ap.add_argument("--one-launch", action="store_true",
                    help="M <= 32: run each linear as xq_expanded_linear_one_launch (the online step inside the product kernel)")
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
    if args.fmt == "mxfp4":
        assert args.act == "sym", "--fmt mxfp4 has its own quantizer: --act does not apply"

    if args.gptq_report:
        if rank == 0:
            gptq_report()
        return

    b = Bench(args, rank, local_rank, world, dist)
    head = b.run(args.workload, M, args.steps, args.warmup, headline=True)
    per_workload = {}
    if not args.only:
        for wl, m in PER_WORKLOAD:
            if (wl, m) == (args.workload, M):
                continue
            # decode-shaped steps are short: more replays for a stable figure; the timed work stays well under a second each
            r = b.run(wl, m, max(args.steps, 50) if m <= 32 else min(args.steps, 20), args.warmup, headline=False)
            per_workload[f"{wl} M={m}"] = r

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    cpu_baseline = None
    if not args.no_cpu_baseline and world == 1:
        cpu_baseline = cpu_baseline_leg(args, table, layers, M, heavy)

    launches = head["gpu_launches_per_step"] * args.steps
    line = {
        "metric": METRIC, "value": head["tokens_per_s"], "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "mxfp4 (e2m1 codes, e8m0 group scales), fp32 accumulate" if args.fmt == "mxfp4" else "int4 codes, int32 accumulate",
        "data": "synthetic",
        "config": workload_config(args, table, layers, M, head["weight_bytes"], world),
        "TOPS": head["TOPS"], "clocks": head["clocks"], "e2e": head["e2e"], "gpu_launches": launches,
        "roofline": head["roofline"], "cpu_baseline": cpu_baseline, "per_workload": per_workload,
    }
    if "error_vs_unquantized" in head:
        line["error_vs_unquantized"] = head["error_vs_unquantized"]
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def gptq_report(rows=256, tokens=2048):
    """Sec. 3.1 Remark 2 on synthetic data: the down projection of the 1B shape (K = 8192) at the expansion sizes of the
    paper's Table 1, `rows` output channels, Hessian from `tokens` synthetic calibration tokens.  Rotated activations and
    weights come from the library's rotate kernel (its fp32 dump), the Hessian and the objectives are plain fp64 matrix
    products (torch: bookkeeping of the report, not the path), the codes from xq_gptq_codes and from round-to-nearest."""
    import torch

    from paper_2503_17513_b200 import xq

    K = 8192
    x = synth.activations(tokens, K, seed=7, tag="gptq-cal", heavy_tail=True)
    wb = synth.weights(rows, K, seed=7, tag="gptq-down")
    X = torch.from_numpy(x.view(np.int16)).cuda()
    Wb = torch.from_numpy(wb.view(np.int16)).cuda()
    out = {}
    for Kp in (8192, 8960, 9728, 10240, 12288):
        pl = xq.xq_hadamard_plan(K, Kp)

        def rotated(T, n):
            Xq = torch.empty((n, Kp // 2), dtype=torch.uint8, device="cuda")
            sx = torch.empty((n,), dtype=torch.float32, device="cuda")
            Y = torch.empty((n, Kp), dtype=torch.float32, device="cuda")
            xq.xq_rotate_quant(T, pl, Xq, sx, Y)
            return Y.double()

        Y, Wt = rotated(X, tokens), rotated(Wb, rows)
        H = Y.T @ Y
        t0 = time.perf_counter()
        codes, s_w = xq.xq_gptq_codes(Wt.cpu().numpy(), H.cpu().numpy(), damp=0.01)
        t_gptq = time.perf_counter() - t0
        s_rtn = torch.clamp(Wt.abs().amax(dim=1) / 7.0, min=0).float().double()
        s_rtn[s_rtn == 0] = 1.0
        q_rtn = torch.clamp(torch.round(Wt / s_rtn[:, None]), -8, 7)

        def objective(Q, s):
            D = Wt - s[:, None] * Q
            return float(((D @ H) * D).sum())

        energy = float(((Wt @ H) * Wt).sum())
        o_g = objective(torch.from_numpy(codes.astype(np.float64)).cuda(), torch.from_numpy(s_w.astype(np.float64)).cuda())
        o_r = objective(q_rtn, s_rtn)
        out[str(Kp)] = {"gptq_rel_objective": o_g / energy, "rtn_rel_objective": o_r / energy, "sqrt_K_over_Kp": float(np.sqrt(K / Kp)),
                        "gptq_seconds": t_gptq}
    print(json.dumps({"report": "gptq objective vs K' (Remark 2), 1B down projection, synthetic Hessian", "K": K, "rows": rows,
                      "calibration_tokens": tokens, "damp": 0.01, "per_Kp": out}))


def cpu_baseline_leg(args, table, layers, M, heavy):
    """The oracle, as it stands, on the host cores: online path of one layer's linears for a bounded
    token and channel sample, scaled linearly (the path is independent per token and per channel)."""
    oracle, Ms, step = reference_sample(args, table, M, heavy)
    _, t_layer = step()
    t_step = t_layer * layers * (M / Ms)
    return {"value": M / t_step, "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"one layer, {Ms} tokens, up to 512 output channels per linear; scaled to {layers} layers, M={M}, full N"}


if __name__ == "__main__":
    main()
