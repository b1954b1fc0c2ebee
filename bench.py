#!/usr/bin/env python
"""Benchmark of the NVFP4 linear-layer hot path on B200.

One "step" = forward + dX + dW (six quantizers, three FP4 GEMMs each) of every linear of the workload, through the
C-ABI library. Default workload: every NVFP4 linear of a 24-layer ~370M LLaMA-style transformer (hidden 1024, FFN 2816),
tokens 16384 (BASELINE configuration 4), seeded synthetic BF16 inputs. Prints ONE JSON line (see the keys below); the
line also carries `large_shapes`: quantizer GB/s and GEMM TFLOP/s on the roofline-sweep shapes of configuration 5.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload attn|mlp|model370m]
                  [--gs tensor|row|block128] [--outliers p] [--rht] ...

N > 1: every rank runs the same workload on its own GPU (independent replicas, no collective on the data path); the
time is the max over ranks and the value the sum of all ranks' work. Under torchrun the ranks are given; a plain
`python bench.py --gpus N` starts the N ranks itself.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2510_27527_b200 import synth  # noqa: E402

WORKLOADS = {
    # name: (config id of the input recipe, tokens, [(linear name, D_in, C_out, swiglu input?)])
    "attn": (2, 8192, [("qkv", 1024, 3072, False), ("o", 1024, 1024, False)]),
    "mlp": (3, 8192, [("gate", 1024, 2816, False), ("up", 1024, 2816, False), ("down", 2816, 1024, True)]),
    "model370m": (4, 16384, [("qkv", 1024, 3072, False), ("o", 1024, 1024, False), ("gate", 1024, 2816, False),
                             ("up", 1024, 2816, False), ("down", 2816, 1024, True)]),
}
LAYERS = {"attn": 1, "mlp": 1, "model370m": 24}
GS = {"tensor": 0, "row": 1, "block128": 2}

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernels, from the ncu captures summarised under
# profiles/ (keyed by kernel label, linear and tokens; a capture on a smaller tensor of the same kernel is scaled by the
# number of elements, stated in the summary).
# Stochastic-rounding quantizer calls in TENSOR mode = amax pre-pass + quantizer. Captured on 8192 x 8192 (67.1 M elements):
# amax 138.0 MB, quantize_cols4 151.0 MB, quantize_rows4 157.3 MB per launch (profiles/quantizers_tensor_mode_8192x8192.txt,
# profiles/quantizers_block128_8192x8192.txt); both kernels stream, so traffic scales with the element count.
def _scaled_traffic(mb_per_67m, rows, cols):
    return sum(mb_per_67m) * 1e6 * (rows * cols) / (8192.0 * 8192.0)


PROFILED_TRAFFIC = {}
for _name, _d, _c in (("qkv", 1024, 3072), ("gate", 1024, 2816), ("up", 1024, 2816)):
    PROFILED_TRAFFIC[(f"quantize_cols_dY_SR(Q5) on {_name} {_d}->{_c}", "tensor")] = (
        _scaled_traffic((138.0, 151.0), 16384, _c), "ncu on 8192x8192 (amax_tensor_bf16 + quantize_cols4), scaled by the element count")
    PROFILED_TRAFFIC[(f"quantize_rows_dY_SR(Q3) on {_name} {_d}->{_c}", "tensor")] = (
        _scaled_traffic((138.0, 157.3), 16384, _c), "ncu on 8192x8192 (amax_tensor_bf16 + quantize_rows4), scaled by the element count")


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=d["hbm_gbs"], bf16=d["bf16_tflops"], bf16_sustained=d["bf16_tflops_sustained"], source="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


def flops_of(tokens, linears, layers):
    return layers * sum(6.0 * tokens * D * C for (_, D, C, _) in linears)


def workload_name(args):
    cfg_id, tokens, linears = WORKLOADS[args.workload]
    return (f"{args.workload}: tokens {tokens}, " + ", ".join(f"{n} {D}->{C}" for n, D, C, _ in linears) +
            (f", x{LAYERS[args.workload]} layers" if LAYERS[args.workload] > 1 else "") + ", fwd+dX+dW per linear")


def config_of(args):
    """The workload and how it is run: the same dictionary in the CUDA arm's and the oracle arm's line."""
    return {"workload": workload_name(args), "gs_mode": args.gs, "outcontrol_fraction": args.outliers, "rht": bool(args.rht),
            "sr_scale_up": bool(args.sr_scale_up), "outlier_fp8": bool(args.outlier_fp8),
            "weight_block": "16x16" if args.w16x16 else "1x16",
            "launch": "cuda_graph_replay" if args.graph else "stream",
            "l2": "256 MiB write + 256 MiB read flush before every timed step",
            "timing": "CUDA events per step on the launch stream, summed"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs (read-only queries)."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                                          "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._pump, daemon=True)
            self.t.start()
            time.sleep(0.3)  # let the first samples arrive before the timed region starts
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        for l in self.lines:
            f = [t.strip() for t in l.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
                pw.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "power_w_max": max(pw) if pw else None}


# ---------------------------------------------------------------------------------------------------------------
# the oracle arm (CPU): used for --impl reference and for the cpu_baseline leg of the default arm
# ---------------------------------------------------------------------------------------------------------------
def oracle_sample_step(workload: str, gs_mode: int, sample_tokens: int = 256, rht: bool = False, inputs=None):
    """One forward + dX + dW of every linear of one layer of the workload on a slab of `sample_tokens` tokens, through the
    oracle as it stands. Returns (seconds, flops of the sample, description, inputs)."""
    from oracle import nvfp4_oracle as orc

    cfg_id, tokens, linears = WORKLOADS[workload]
    c = synth.CONFIGS[cfg_id]
    if inputs is None:
        inputs = []
        for li, (name, D, C, swiglu) in enumerate(linears):
            inputs.append(synth.layer_inputs(cfg_id, sample_tokens, D, C, n_outlier=max(1, D // 100), factor=c["factor"],
                                             grad_scale=c["grad_scale"], swiglu=swiglu, weight_id=10 + li))
    orc.lib()
    t0 = time.perf_counter()
    ocfg = orc.LayerConfig(gs_mode=gs_mode, seed=0, rht=rht)
    for X, W, dY, _ in inputs:
        _, saved = orc.linear_fwd(X, W, ocfg)
        orc.linear_bwd_dx(dY, saved, ocfg)
        orc.linear_bwd_dw(dY, saved, ocfg)
    dt = time.perf_counter() - t0
    fl = sum(6.0 * sample_tokens * D * C for _, D, C, _ in linears)
    names = " + ".join(f"{name} {D}->{C}" for name, D, C, _ in linears)
    desc = (f"every linear of one layer ({names}), {sample_tokens}-token slab of the {tokens}-token workload, fwd+dX+dW; "
            f"value = the slab's GEMM flops / its time")
    return dt, fl, desc, inputs


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import nvfp4_oracle as orc

    gs_mode = GS[args.gs]
    inputs = None
    for _ in range(min(args.warmup, 1)):
        _, _, _, inputs = oracle_sample_step(args.workload, gs_mode, args.ref_tokens, args.rht, inputs)
    times, fl, desc = [], 0.0, ""
    for _ in range(args.steps):
        dt, fl, desc, inputs = oracle_sample_step(args.workload, gs_mode, args.ref_tokens, args.rht, inputs)
        times.append(dt)
    t = float(np.mean(times))
    val = fl / t / 1e12
    line = {
        "impl": "reference", "metric": "nvfp4_linear_fwd_bwd_tflops", "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config_of(args),
        "notes": "the oracle (CPU, as it stands) on a bounded sample of the same workload; the launch / l2 / timing entries of "
                 "config describe the CUDA arm",
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": orc.threads(), "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------------------------
# shared timing helper of the CUDA arm
# ---------------------------------------------------------------------------------------------------------------
class Timer:
    """CUDA-event timing with an L2 flush before every timed call: 256 MiB written (evicts everything), then another
    256 MiB read so that the lines left in L2 are clean (the timed kernels do not pay for writing the flush back)."""

    def __init__(self, dev):
        import torch

        self.torch = torch
        self.flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        self.flush_src = torch.zeros(256 << 20, dtype=torch.uint8, device=dev)

    def flush_l2(self):
        self.flush_buf.fill_(1)
        self.flush_src.max()

    def each(self, fn, n, warm=3):
        """Per-call milliseconds of n flushed calls (after `warm` untimed ones)."""
        torch = self.torch
        for _ in range(warm):
            fn()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        torch.cuda.synchronize()
        for i in range(n):
            self.flush_l2()
            ev[i][0].record()
            fn()
            ev[i][1].record()
        torch.cuda.synchronize()
        return [a.elapsed_time(bb) for a, bb in ev]

    def median_s(self, fn, n, warm=3):
        ms = sorted(self.each(fn, n, warm))
        return ms[len(ms) // 2] * 1e-3


def measure_large_shapes(b, dev, pk, timer, shapes, gs_names, n_iter):
    """Quantizers and GEMMs on the roofline-sweep shapes (BASELINE configuration 5): A [M, K], B [N, K] ~N(0,1) BF16 with
    0.5 % of the K channels x100, drawn with the seeded numpy recipe the parity tests use (seeds 5001 / 5002)."""
    import torch

    status = torch.zeros(1, dtype=torch.int32, device=dev)
    probe_flops = b.nvfp4_mma_issue_probe(2048, status)
    sec = timer.median_s(lambda: b.nvfp4_mma_issue_probe(2048, status), 10)
    issue_loop = probe_flops / sec / 1e12 if int(status.item()) == 0 else None
    # the same loop on hashed operand codes and scales (the arithmetic is the same, the power drawn is not): as a burst of
    # about the duration of one large GEMM, and held for about 12 ms (the clock the power cap settles at)
    rnd = {}
    for name, iters, reps in (("burst", 2048, 10), ("sustained", 32768, 4)):
        fl_r = b.nvfp4_mma_issue_probe(iters, status, 256, 0, 0, True)
        sec_r = timer.median_s(lambda: b.nvfp4_mma_issue_probe(iters, status, 256, 0, 0, True), reps)
        rnd[name] = fl_r / sec_r / 1e12 if int(status.item()) == 0 else None
    fp4_peak = 4.0 * pk["bf16"]
    out = {"mma_issue_loop_TFLOPs": issue_loop, "mma_issue_loop_random_data_TFLOPs": rnd, "fp4_peak_TFLOPs_4x_measured_bf16": fp4_peak,
           "hbm_peak_GBps": pk["hbm"], "shapes": []}
    cache = {}

    def operand_source(rows, K, tensor_id):
        key = (rows, K, tensor_id)
        if key not in cache:
            cache[key], _ = synth.activations(rows, K, synth.seed_of(5, tensor_id), n_outlier=max(1, int(K * 0.005)), factor=100.0)
        return b.upload_bf16(cache[key], dev)

    quantized_a = set()
    ws = b._workspace(1 << 20, dev)
    for (M, N, K) in shapes:
        r = {"M": M, "N": N, "K": K}
        A = operand_source(M, K, 1)
        Bm = operand_source(N, K, 2)
        fl = 2.0 * M * N * K
        for gname in gs_names:
            gs = GS[gname]
            qa, qb = b.alloc_operand(M, K, gs, device=dev), b.alloc_operand(N, K, gs, device=dev)
            C = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
            b.nvfp4_quantize(A, b.AXIS_ROW, b.ROUND_RTN, 0, 1, gs, out=qa, workspace=ws)
            b.nvfp4_quantize(Bm, b.AXIS_ROW, b.ROUND_RTN, 0, 2, gs, out=qb, workspace=ws)
            ms = sorted(timer.each(lambda: b.nvfp4_gemm(qa, qb, b.DT_BF16, out=C), n_iter))
            med = ms[len(ms) // 2] * 1e-3
            t_tensor, t_hbm = fl / (fp4_peak * 1e12), (0.5625 * (M + N) * K + 2.0 * M * N) / (pk["hbm"] * 1e9)
            r[f"gemm_{gname}"] = {"us": med * 1e6, "best_us": ms[0] * 1e3, "TFLOPs": fl / med / 1e12,
                                  "frac_of_4x_bf16_measured": fl / med / 1e12 / fp4_peak,
                                  "frac_of_9PF_nominal": fl / med / 1e12 / 9000.0,
                                  "frac_of_issue_loop": (fl / med / 1e12 / issue_loop) if issue_loop else None,
                                  "frac_of_issue_loop_random_data_burst": (fl / med / 1e12 / rnd["burst"]) if rnd["burst"] else None,
                                  "bound_us_max_tensor_hbm": max(t_tensor, t_hbm) * 1e6}

            def both():
                b.nvfp4_quantize(A, b.AXIS_ROW, b.ROUND_RTN, 0, 1, gs, out=qa, workspace=ws)
                b.nvfp4_quantize(Bm, b.AXIS_ROW, b.ROUND_RTN, 0, 2, gs, out=qb, workspace=ws)
                b.nvfp4_gemm(qa, qb, b.DT_BF16, out=C)

            med = timer.median_s(both, max(3, n_iter // 2))
            r[f"quantize_plus_gemm_{gname}"] = {"us": med * 1e6, "TFLOPs": fl / med / 1e12}
            if (M, K, gname) not in quantized_a:
                quantized_a.add((M, K, gname))
                qat = b.alloc_operand(K, M, gs, device=dev)
                n_el = M * K
                qbytes = n_el * (2 + 0.5 + 1.0 / 16) + (n_el / 128 * 4 if gs == 2 else 0.0)
                amax_read = 2.0 * n_el if gs != 2 else 0.0  # TENSOR / ROW read the source twice (amax pre-pass)
                for label, fn in (
                    ("quantize_rows_rtn", lambda: b.nvfp4_quantize(A, b.AXIS_ROW, b.ROUND_RTN, 0, 1, gs, out=qa, workspace=ws)),
                    ("quantize_rows_sr", lambda: b.nvfp4_quantize(A, b.AXIS_ROW, b.ROUND_SR, 0, 3, gs, out=qa, workspace=ws)),
                    ("quantize_cols_sr", lambda: b.nvfp4_quantize(A, b.AXIS_COL, b.ROUND_SR, 0, 5, gs, out=qat, workspace=ws)),
                ):
                    med = timer.median_s(fn, n_iter)
                    r[f"{label}_A_{gname}"] = {"us": med * 1e6, "GBps": (qbytes + amax_read) / med / 1e9,
                                               "frac_hbm_measured": (qbytes + amax_read) / med / 1e9 / pk["hbm"],
                                               "algorithmic_bytes": qbytes + amax_read}
                b.nvfp4_quantize(A, b.AXIS_ROW, b.ROUND_RTN, 0, 1, gs, out=qa, workspace=ws)
                med = timer.median_s(lambda: b.nvfp4_requantize_t(qa, b.ROUND_SR, 0, 6, out=qat, workspace=ws), n_iter)
                r[f"requantize_t_A_{gname}"] = {"us": med * 1e6, "GBps": n_el * 1.125 / med / 1e9, "Gelem_per_s": n_el / med / 1e9}
                del qat
            del qa, qb, C
        out["shapes"].append(r)
        del A, Bm
    return out


# ---------------------------------------------------------------------------------------------------------------
# the CUDA arm
# ---------------------------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2510_27527_b200 import binding as b
    from paper_2510_27527_b200 import multi

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl")
    dev = torch.device("cuda", local)
    gs_mode = GS[args.gs]
    cfg_id, tokens, linears = WORKLOADS[args.workload]
    layers = LAYERS[args.workload]
    c = synth.CONFIGS[cfg_id]

    # ---- inputs: activations / gradients per shape class, fresh weights per layer ------------------------------
    class Lin:
        pass

    lins = []
    for li, (name, D, C, swiglu) in enumerate(linears):
        X, W, dY, _ = synth.layer_inputs(cfg_id, tokens, D, C, n_outlier=max(1, D // 100), factor=c["factor"],
                                         grad_scale=c["grad_scale"], weight_id=10 + li, swiglu=swiglu)
        L = Lin()
        L.name, L.D, L.C = name, D, C
        L.Xh, L.dYh = X, dY
        L.X, L.dY = b.upload_bf16(X, dev), b.upload_bf16(dY, dev)
        L.W = [b.upload_bf16(W, dev)]
        for extra in range(1, layers):
            L.W.append(b.upload_bf16(synth.weights(C, D, synth.seed_of(cfg_id, 100 * extra + li)), dev))
        n_out = int(round(args.outliers * D))
        outl = synth.outlier_channels(D, n_out, synth.seed_of(cfg_id, 50 + li)) if n_out else None
        rounding = (b.ROUND_RTN, b.ROUND_RTN) + ((b.ROUND_SR_SCALE_UP,) * 4 if args.sr_scale_up else (b.ROUND_SR,) * 4)
        L.cfg = b.LayerConfig(gs_mode=gs_mode, seed=0, y_dtype=b.DT_BF16, dx_dtype=b.DT_BF16, dw_dtype=b.DT_F32, outliers=outl, rht=args.rht,
                              rounding=rounding, outlier_fp8=args.outlier_fp8, w_block16=args.w16x16, concurrent=not args.one_stream)
        L.cfg.prepare(D, dev)
        L.saved = b.alloc_saved(L.X, L.W[0], L.cfg)
        L.Y = torch.empty((tokens, C), dtype=torch.bfloat16, device=dev)
        L.dXo = torch.empty((tokens, D), dtype=torch.bfloat16, device=dev)
        L.dWo = torch.empty((C, D), dtype=torch.float32, device=dev)
        L.ws = [b.linear_workspace(k, tokens, D, C, L.cfg, dev) for k in (b.OP_FWD, b.OP_BWD_DX, b.OP_BWD_DW, b.OP_BWD)]
        lins.append(L)

    timer = Timer(dev)

    def step():
        for layer in range(layers):
            for L in lins:
                W = L.W[layer]
                b.nvfp4_linear_fwd(L.X, W, L.cfg, Y=L.Y, saved=L.saved, workspace=L.ws[0])
                b.nvfp4_linear_bwd(L.dY, L.saved, L.cfg, dX=L.dXo, dW=L.dWo, workspace=L.ws[3])

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def timed(fn, steps, flush=True):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        barrier()
        for s in range(steps):
            if flush:
                timer.flush_l2()
            ev[s][0].record()
            fn()
            ev[s][1].record()
        barrier()
        ms = [a.elapsed_time(bb) for a, bb in ev]
        return multi.max_over_ranks(sum(ms), dev) / steps, ms  # the job's time is the slowest rank's

    for _ in range(max(args.warmup, 3)):
        step()
    run_step, launches_per_step = step, None
    if args.graph:
        # The library neither allocates nor synchronises, so a whole step can be captured once and replayed: the timed
        # region then holds the same kernels in the same order without the host's per-call marshalling between them.
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        l0 = b.lib.nvfp4_launch_count()
        with torch.cuda.graph(graph):
            step()
        launches_per_step = b.lib.nvfp4_launch_count() - l0
        run_step = graph.replay
        for _ in range(3):
            run_step()
        torch.cuda.synchronize()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    l0 = b.lib.nvfp4_launch_count()
    ms_step, _ = timed(run_step, args.steps)
    launches = b.lib.nvfp4_launch_count() - l0 if launches_per_step is None else launches_per_step * args.steps
    clocks = sampler.stop() if rank == 0 else None
    fl = flops_of(tokens, linears, layers)
    value = world * fl / (ms_step * 1e-3) / 1e12

    if args.no_breakdown:
        if rank == 0:
            print(json.dumps({"metric": "nvfp4_linear_fwd_bwd_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": world,
                              "steps": args.steps, "ms_per_step": ms_step, "gpu_launches": int(launches), "clocks": clocks,
                              "config": config_of(args), "note": "--no-breakdown run"}))
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- end to end: host buffers in, results out, copies inside the timed region -------------------------------
    h2d, d2h = 0, 0
    for L in lins:
        xb = torch.from_numpy(synth.to_bf16_bits(L.Xh).view(np.int16)).view(torch.bfloat16).pin_memory()
        gb = torch.from_numpy(synth.to_bf16_bits(L.dYh).view(np.int16)).view(torch.bfloat16).pin_memory()
        L.pin = (xb, gb)
        L.out_pin = (torch.empty_like(L.Y, device="cpu").pin_memory(), torch.empty_like(L.dXo, device="cpu").pin_memory(),
                     torch.empty_like(L.dWo, device="cpu").pin_memory())
        h2d += layers * (xb.numel() + gb.numel()) * 2
        d2h += layers * (L.Y.numel() * 2 + L.dXo.numel() * 2 + L.dWo.numel() * 4)

    # Three streams: uploads, the library's kernels, downloads. A linear's inputs are uploaded while the previous one
    # computes and its results are downloaded while the next one computes (the two copy directions use separate engines).
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    for L in lins:
        L.ev_x, L.ev_dy, L.ev_fwd, L.ev_done, L.ev_drained = (torch.cuda.Event() for _ in range(5))
        L.used = False

    def step_e2e():
        cur = torch.cuda.current_stream()
        ev_begin = torch.cuda.Event()
        ev_begin.record(cur)
        s_in.wait_event(ev_begin)
        s_out.wait_event(ev_begin)
        for layer in range(layers):
            for L in lins:
                with torch.cuda.stream(s_in):
                    if L.used:
                        s_in.wait_event(L.ev_done)  # the kernels that read these input buffers have finished
                    L.X.copy_(L.pin[0], non_blocking=True)
                    L.ev_x.record(s_in)
                    L.dY.copy_(L.pin[1], non_blocking=True)  # arrives while forward runs and Y leaves
                    L.ev_dy.record(s_in)
                cur.wait_event(L.ev_x)
                if L.used:
                    cur.wait_event(L.ev_drained)  # the previous results have left the output buffers
                W = L.W[layer]
                b.nvfp4_linear_fwd(L.X, W, L.cfg, Y=L.Y, saved=L.saved, workspace=L.ws[0])
                L.ev_fwd.record(cur)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(L.ev_fwd)
                    L.out_pin[0].copy_(L.Y, non_blocking=True)
                cur.wait_event(L.ev_dy)
                b.nvfp4_linear_bwd(L.dY, L.saved, L.cfg, dX=L.dXo, dW=L.dWo, workspace=L.ws[3])
                L.ev_done.record(cur)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(L.ev_done)
                    L.out_pin[1].copy_(L.dXo, non_blocking=True)
                    L.out_pin[2].copy_(L.dWo, non_blocking=True)
                    L.ev_drained.record(s_out)
                L.used = True
        for L in lins:
            cur.wait_event(L.ev_drained)  # the step ends when its last result is in host memory

    e2e_steps = max(2, min(args.steps, 3 if layers > 1 else 5))
    step_e2e()
    ms_e2e, _ = timed(step_e2e, e2e_steps)
    e2e_value = world * fl / (ms_e2e * 1e-3) / 1e12

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- per-kernel breakdown over the linears of one layer (rank 0): which launch dominates, and its roofline -------
    pk = peaks()
    fp4_peak = pk["bf16"] * 4.0  # dense FP4 : dense BF16 nominal ratio 9 : 2.25
    ws_q = b._workspace(1 << 20, dev)
    qbytes = lambda n: n * (2 + 0.5 + 1.0 / 16) + (n / 128 * 4 if gs_mode == 2 else 0.0)
    rqbytes = lambda n: n * 2 * (0.5 + 1.0 / 16)
    amax_extra = 2.0 if gs_mode != 2 else 0.0  # TENSOR / ROW modes read the source twice (amax pre-pass)
    gemm_bytes = lambda M, N, K, ob: 0.5625 * (M + N) * K + ob * M * N
    parts = {}
    T = tokens
    n_break = 10
    for L in lins:
        D, C = L.D, L.C
        if L.cfg.n_out:
            continue  # the operand-level calls below have no OutControl form; the step numbers above cover it
        q3 = b.alloc_operand(T, C, gs_mode, device=dev)
        q4 = b.alloc_operand(D, C, gs_mode, device=dev)
        q5 = b.alloc_operand(C, T, gs_mode, device=dev)
        q6 = b.alloc_operand(D, T, gs_mode, device=dev)
        b.nvfp4_linear_fwd(L.X, L.W[0], L.cfg, Y=L.Y, saved=L.saved, workspace=L.ws[0])

        def add(name, fn, alg_bytes=None, flops=None):
            t = timer.median_s(fn, n_break)
            parts[f"{name} on {L.name} {D}->{C}"] = dict(seconds=t, GBps=(alg_bytes / t / 1e9 if alg_bytes else None),
                                                         TFLOPs=(flops / t / 1e12 if flops else None), bytes=alg_bytes, flops=flops)

        add("quantize_rows_X(Q1)", lambda: b.nvfp4_quantize(L.X, b.AXIS_ROW, b.ROUND_RTN, 0, 1, gs_mode, out=L.saved.qx, workspace=ws_q),
            qbytes(T * D) + amax_extra * T * D)
        add("quantize_rows_dY_SR(Q3)", lambda: b.nvfp4_quantize(L.dY, b.AXIS_ROW, b.ROUND_SR, 0, 3, gs_mode, out=q3, workspace=ws_q),
            qbytes(T * C) + amax_extra * T * C)
        add("quantize_cols_dY_SR(Q5)", lambda: b.nvfp4_quantize(L.dY, b.AXIS_COL, b.ROUND_SR, 0, 5, gs_mode, out=q5, workspace=ws_q),
            qbytes(T * C) + amax_extra * T * C)
        add("requantize_t_W(Q4)", lambda: b.nvfp4_requantize_t(L.saved.qw, b.ROUND_SR, 0, 4, out=q4, workspace=ws_q), rqbytes(C * D))
        add("requantize_t_X(Q6)", lambda: b.nvfp4_requantize_t(L.saved.qx, b.ROUND_SR, 0, 6, out=q6, workspace=ws_q), rqbytes(T * D))
        add("gemm_fwd", lambda: b.nvfp4_gemm(L.saved.qx, L.saved.qw, b.DT_BF16, out=L.Y), gemm_bytes(T, C, D, 2), 2.0 * T * C * D)
        add("gemm_dx", lambda: b.nvfp4_gemm(q3, q4, b.DT_BF16, out=L.dXo), gemm_bytes(T, D, C, 2), 2.0 * T * C * D)
        add("gemm_dw", lambda: b.nvfp4_gemm(q5, q6, b.DT_F32, out=L.dWo), gemm_bytes(C, D, T, 4), 2.0 * T * C * D)
        del q3, q4, q5, q6
    roof = None
    if parts:
        dom = max(parts, key=lambda k: parts[k]["seconds"])
        dp = parts[dom]
        if dom.startswith("gemm") and dp["flops"] / (fp4_peak * 1e12) >= dp["bytes"] / (pk["hbm"] * 1e9):
            roof = dict(bound="tensor", achieved=dp["TFLOPs"], peak=fp4_peak, unit="TFLOP/s", frac=dp["TFLOPs"] / fp4_peak)
        else:
            roof = dict(bound="hbm", achieved=dp["GBps"], peak=pk["hbm"], unit="GB/s", frac=dp["GBps"] / pk["hbm"])
        roof.update(kernel=f"{dom}, tokens {T}", peak_source=f"of {pk['source']}", traffic=None,
                    algorithmic_bytes_per_launch=dp["bytes"], seconds_per_launch=dp["seconds"],
                    note="the call that takes longest when every ABI call of one layer is timed alone (incl. its amax pre-pass)")
        key = (dom, args.gs)
        if key in PROFILED_TRAFFIC:
            roof["traffic"], roof["traffic_source"] = PROFILED_TRAFFIC[key]

    # ---- quantizers and GEMMs on the large sweep shapes (configuration 5) ----------------------------------------
    large = None
    if not args.no_large_shapes:
        sampler2 = ClockSampler(local)
        sampler2.start()
        shapes = synth.CONFIGS[5]["shapes"] if not args.shapes else [tuple(int(v) for v in t.split("x")) for t in args.shapes.split(",")]
        large = measure_large_shapes(b, dev, pk, timer, shapes, ("tensor", "block128"), 10)
        large["clocks"] = sampler2.stop()

    # ---- the oracle beside it ------------------------------------------------------------------------------------
    cpu = None
    if world == 1 and not args.no_cpu:
        from oracle import nvfp4_oracle as orc

        dt, sfl, desc, _ = oracle_sample_step(args.workload, gs_mode, args.cpu_tokens, args.rht)
        cpu = {"value": sfl / dt / 1e12, "unit": "TFLOP/s", "cores": orc.threads(), "kind": "oracle", "sample": desc,
               "seconds": dt}

    line = {
        "metric": "nvfp4_linear_fwd_bwd_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "fp4(e2m1)xfp4 with ue4m3 block scales, f32 accumulate", "data": "synthetic", "config": config_of(args),
        "e2e": {"value": e2e_value, "unit": "TFLOP/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e},
        "gpu_launches": int(launches), "clocks": clocks, "roofline": roof, "cpu_baseline": cpu,
        "kernels": {k: {kk: (round(vv, 9) if isinstance(vv, float) else vv) for kk, vv in v.items() if kk in ("seconds", "GBps", "TFLOPs")}
                    for k, v in parts.items()},
        "large_shapes": large,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_aux(args):
    """HBM roofline of the auxiliary kernels (OutControl calibration, OsciReset statistics / reset) on large matrices:
    one JSON line. Not the headline line."""
    import torch

    from paper_2510_27527_b200 import binding as b

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    pk = peaks()
    timer = Timer(dev)
    t_of = lambda fn, n: timer.median_s(fn, n)
    g = torch.Generator(device=dev)
    g.manual_seed(7)
    out = {}
    N, D = 16384, 8192
    X = torch.randn((N, D), device=dev, generator=g, dtype=torch.float32).to(torch.bfloat16)
    acc = torch.zeros(D, dtype=torch.float32, device=dev)
    ws = b._workspace(b.lib.nvfp4_outlier_accumulate_workspace_bytes(N, D), dev)
    sec = t_of(lambda: b.nvfp4_outlier_accumulate(X, acc, workspace=ws), args.steps)
    out["outlier_accumulate_16384x8192"] = {"us": sec * 1e6, "GBps": 2.0 * N * D / sec / 1e9, "frac_hbm_measured": 2.0 * N * D / sec / 1e9 / pk["hbm"]}
    sec = t_of(lambda: b.nvfp4_outlier_select(acc, D // 10), args.steps)
    out["outlier_select_8192_top10pct"] = {"us": sec * 1e6}
    del X
    C, D = 8192, 8192
    W = torch.randn((C, D), device=dev, generator=g, dtype=torch.float32) * 0.02
    W1 = W + torch.randn((C, D), device=dev, generator=g, dtype=torch.float32) * 4e-5
    st = b.alloc_osci_state(W)
    for name, gs in GS.items():
        wsp = b._workspace(b.lib.nvfp4_osci_workspace_bytes(C, gs), dev)
        b.nvfp4_osci_update(W, st, 0, gs, workspace=wsp)
        flip = [0]

        def upd():
            flip[0] ^= 1
            b.nvfp4_osci_update(W1 if flip[0] else W, st, 1, gs, workspace=wsp)

        sec = t_of(upd, args.steps)
        # algorithmic bytes: read W, W', D_M, D_Q and write W', D_M, D_Q (7 x 4 B); TENSOR / ROW re-read W and W' for amax
        alg = (28.0 + (8.0 if gs != 2 else 0.0)) * C * D
        out[f"osci_update_8192x8192_{name}"] = {"us": sec * 1e6, "GBps": alg / sec / 1e9, "frac_hbm_measured": alg / sec / 1e9 / pk["hbm"]}
        n = torch.zeros(1, dtype=torch.int64, device=dev)
        Wc = W1.clone()
        sec = t_of(lambda: b.nvfp4_osci_suppress(Wc, st, 8.0, gs, n_reset=n, workspace=wsp), args.steps)
        # read W, D_M, D_Q (12 B) (+4 B amax pre-pass); writes only the few reset blocks
        alg = (12.0 + (4.0 if gs != 2 else 0.0)) * C * D
        out[f"osci_suppress_8192x8192_{name}"] = {"us": sec * 1e6, "GBps": alg / sec / 1e9, "frac_hbm_measured": alg / sec / 1e9 / pk["hbm"]}
    # memory-efficient statistics: 5 % of the elements tracked
    n_track = C * D // 20
    for name, gs in GS.items():
        sp = b.alloc_osci_sparse_state(n_track, dev)
        ws0 = b._workspace(b.lib.nvfp4_osci_sparse_workspace_bytes(C, D, gs, n_track, 0), dev)
        ws1 = b._workspace(b.lib.nvfp4_osci_sparse_workspace_bytes(C, D, gs, n_track, 1), dev)
        sec = t_of(lambda: b.nvfp4_osci_sparse_update(W, sp, 0, gs, workspace=ws0), max(3, args.steps // 2))
        out[f"osci_sparse_select_8192x8192_{name}"] = {"us": sec * 1e6}
        flip = [0]

        def upd_s():
            flip[0] ^= 1
            b.nvfp4_osci_sparse_update(W1 if flip[0] else W, sp, 1, gs, workspace=ws1)

        sec = t_of(upd_s, args.steps)
        # bytes moved at most: W read once for the amax pre-pass (per tensor, row or 128-group) + per tracked element its
        # 64-byte block (blocks are shared between neighbours) and 36 B of state traffic
        alg = 4.0 * C * D + n_track * (64.0 + 36.0)
        out[f"osci_sparse_update_8192x8192_{name}"] = {"us": sec * 1e6, "state_bytes_per_param": 20.0 * n_track / (C * D),
                                                        "GBps_upper_bound_bytes": alg / sec / 1e9}
        del ws0
    # simulated FP6 x FP4 layer (Sec. 5.4) on the QKV linear of the 370M model, beside the FP4 layer on the same inputs
    T, D2, C2 = 16384, 1024, 3072
    Xs, Ws, dYs, _ = synth.layer_inputs(4, T, D2, C2, n_outlier=10, factor=30.0, grad_scale=1e-4, weight_id=10)
    Xd, Wd, dYd = b.upload_bf16(Xs, dev), b.upload_bf16(Ws, dev), b.upload_bf16(dYs, dev)

    def fp6_step():
        _, saved6 = b.fp6_linear_fwd(Xd, Wd, b.DT_BF16)
        b.fp6_linear_bwd(dYd, saved6, 0)

    cfg4 = b.LayerConfig(gs_mode=b.GS_TENSOR, seed=0)

    def fp4_step():
        _, saved4 = b.nvfp4_linear_fwd(Xd, Wd, cfg4)
        b.nvfp4_linear_bwd(dYd, saved4, cfg4)

    fl = 6.0 * T * D2 * C2
    for name, fn in (("fp6_sim_layer_qkv_tokens16384", fp6_step), ("fp4_layer_qkv_tokens16384_same_call_pattern", fp4_step)):
        sec = t_of(fn, max(3, args.steps // 2))
        out[name] = {"us": sec * 1e6, "TFLOPs": fl / sec / 1e12}
    print(json.dumps({"aux": out, "peaks": pk}))


def run_sweep(args):
    """Only the large-shape measurements (quantizers and GEMMs of configuration 5, or --shapes), one JSON line."""
    import torch

    from paper_2510_27527_b200 import binding as b

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    pk = peaks()
    shapes = synth.CONFIGS[5]["shapes"] if not args.shapes else [tuple(int(v) for v in t.split("x")) for t in args.shapes.split(",")]
    sampler = ClockSampler(0)
    sampler.start()
    out = measure_large_shapes(b, dev, pk, Timer(dev), shapes, (args.gs,), args.steps)
    out["clocks"] = sampler.stop()
    print(json.dumps({"sweep": out, "gs_mode": args.gs, "peaks": pk}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="model370m", choices=list(WORKLOADS))
    ap.add_argument("--gs", default="tensor", choices=list(GS))
    ap.add_argument("--ref-tokens", type=int, default=256, help="token slab of one oracle step (reference arm)")
    ap.add_argument("--cpu-tokens", type=int, default=2048, help="token slab of the cpu_baseline leg (every linear of one layer)")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--outliers", type=float, default=0.0,
                    help="OutControl: fraction of input channels kept in BF16 (0 = off; the paper uses 0.10)")
    ap.add_argument("--rht", action="store_true", help="random Hadamard transformation (block 16) in the four backward quantizers")
    ap.add_argument("--outlier-fp8", action="store_true", help="with --outliers: outlier channels on a power-of-two scaled E4M3 grid instead of BF16")
    ap.add_argument("--w16x16", action="store_true", help="weights in 16x16 scale squares (the recipe the paper compares with): no Q4 in backward")
    ap.add_argument("--sr-scale-up", action="store_true", help="backward quantizers round the block scale up (strictly unbiased variant)")
    ap.add_argument("--graph", action=argparse.BooleanOptionalAction, default=True,
                    help="capture one step in a CUDA graph and time its replays (default; --no-graph launches every kernel from the host)")
    ap.add_argument("--one-stream", action="store_true", help="no second stream: every chain of a layer call runs on the caller's stream")
    ap.add_argument("--no-breakdown", action="store_true", help="only warm-up + timed steps (used for ncu launch lists)")
    ap.add_argument("--no-large-shapes", action="store_true", help="skip the configuration-5 measurements of the default line")
    ap.add_argument("--sweep", action="store_true", help="only the large-shape measurements (configuration 5 or --shapes)")
    ap.add_argument("--aux", action="store_true", help="HBM roofline of the calibration and OsciReset kernels instead of the step benchmark")
    ap.add_argument("--shapes", default="", help="comma list of MxNxK for the large-shape measurements")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours" and not (args.sweep or args.aux):
        # not started by torchrun: start the N ranks here (one process per GPU), rank 0 prints the line
        from paper_2510_27527_b200 import multi

        sys.exit(multi.launch_ranks(args.gpus, os.path.abspath(__file__), sys.argv[1:]))
    if args.sweep:
        run_sweep(args)
    elif args.aux:
        run_aux(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
