#!/usr/bin/env python
"""Benchmark of the NVFP4 linear-layer hot path on B200.

One "step" = forward + dX + dW (six quantizers, three FP4 GEMMs each) of every linear of the workload, through the
C-ABI library. Default workload: LLaMA-style attention projections, hidden 1024, tokens 8192 (QKV 1024->3072 and
O 1024->1024), seeded synthetic BF16 inputs. Prints ONE JSON line (see the keys below).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload attn|mlp|model370m] [--gs tensor|row]

N > 1 (torchrun): every rank runs the same workload on its own GPU (independent replicas, no collective on the data
path); the time is the max over ranks and the value the sum of all ranks' work.
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


# dram__bytes_read.sum + dram__bytes_write.sum per launch, from the ncu captures summarised under profiles/
# (default workload, QKV linear, tokens 8192), keyed by the kernel labels of the per-kernel breakdown below.
# DRAM traffic (dram__bytes_read + dram__bytes_write) of one call = its quantize kernel (ncu capture of this workload) plus
# its amax pre-pass, which reads the source exactly once (268.4 MB for 134.2 M elements in the 16384 x 8192 capture, scaled
# to this tensor's 25.17 M elements: 50.33 MB)
PROFILED_TRAFFIC = {
    "quantize_cols_dY_SR(Q5)": (50355968 + 636416 + 50331648, "profiles/quantize_transpose_bf16_sr_attn_dY_8192x3072.txt"),
    "quantize_rows_dY_SR(Q3)": (50380800 + 246272 + 50331648, "profiles/quantize_rows_sr_attn_dY_8192x3072.txt"),
}


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=d["hbm_gbs"], bf16=d["bf16_tflops"], bf16_sustained=d["bf16_tflops_sustained"], source="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


def flops_of(tokens, linears, layers):
    return layers * sum(6.0 * tokens * D * C for (_, D, C, _) in linears)


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
        sm, mx, reasons = [], [], set()
        for l in self.lines:
            f = [t.strip() for t in l.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ---------------------------------------------------------------------------------------------------------------
# the oracle arm (CPU): used for --impl reference and for the cpu_baseline leg of the default arm
# ---------------------------------------------------------------------------------------------------------------
def oracle_sample_step(workload: str, gs_mode: int, sample_tokens: int = 256, rht: bool = False, all_linears: bool = False):
    """One forward + dX + dW on a slab of `sample_tokens` tokens, through the oracle as it stands: of the workload's first
    linear, or (all_linears) of every linear of one layer. Returns (seconds, flops of the sample, description)."""
    from oracle import nvfp4_oracle as orc

    cfg_id, tokens, linears = WORKLOADS[workload]
    c = synth.CONFIGS[cfg_id]
    chosen = linears if all_linears else linears[:1]
    inputs = []
    for li, (name, D, C, swiglu) in enumerate(chosen):
        inputs.append(synth.layer_inputs(cfg_id, sample_tokens, D, C, n_outlier=c["n_outlier"], factor=c["factor"],
                                         grad_scale=c["grad_scale"], swiglu=swiglu, weight_id=10 + li))
    orc.lib()
    t0 = time.perf_counter()
    ocfg = orc.LayerConfig(gs_mode=gs_mode, seed=0, rht=rht)
    for X, W, dY, _ in inputs:
        _, saved = orc.linear_fwd(X, W, ocfg)
        orc.linear_bwd_dx(dY, saved, ocfg)
        orc.linear_bwd_dw(dY, saved, ocfg)
    dt = time.perf_counter() - t0
    fl = sum(6.0 * sample_tokens * D * C for _, D, C, _ in chosen)
    names = " + ".join(f"{name} {D}->{C}" for name, D, C, _ in chosen)
    return dt, fl, f"linear(s) {names}, {sample_tokens}-token slab of the {tokens}-token workload, fwd+dX+dW"


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import nvfp4_oracle as orc

    gs_mode = GS[args.gs]
    cfg_id, tokens, linears = WORKLOADS[args.workload]
    for _ in range(min(args.warmup, 1)):
        oracle_sample_step(args.workload, gs_mode, 64, args.rht)
    times, fl, desc = [], 0.0, ""
    for _ in range(args.steps):
        dt, fl, desc = oracle_sample_step(args.workload, gs_mode, args.ref_tokens, args.rht)
        times.append(dt)
    t = float(np.mean(times))
    val = fl / t / 1e12
    line = {
        "impl": "reference", "metric": "nvfp4_linear_fwd_bwd_tflops", "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(args), "sample": desc, "gs_mode": args.gs},
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": orc.threads(), "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_name(args):
    cfg_id, tokens, linears = WORKLOADS[args.workload]
    return (f"{args.workload}: tokens {tokens}, " + ", ".join(f"{n} {D}->{C}" for n, D, C, _ in linears) +
            (f", x{LAYERS[args.workload]} layers" if LAYERS[args.workload] > 1 else "") + ", fwd+dX+dW per linear")


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
    host_inputs = {}
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
                              rounding=rounding, outlier_fp8=args.outlier_fp8, w_block16=args.w16x16)
        L.cfg.prepare(D, dev)
        L.saved = b.alloc_saved(L.X, L.W[0], L.cfg)
        L.Y = torch.empty((tokens, C), dtype=torch.bfloat16, device=dev)
        L.dXo = torch.empty((tokens, D), dtype=torch.bfloat16, device=dev)
        L.dWo = torch.empty((C, D), dtype=torch.float32, device=dev)
        L.ws = [b.linear_workspace(k, tokens, D, C, L.cfg, dev) for k in (b.OP_FWD, b.OP_BWD_DX, b.OP_BWD_DW, b.OP_BWD)]
        lins.append(L)

    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    flush_src = torch.zeros(256 << 20, dtype=torch.uint8, device=dev)

    def flush_l2():
        # write 256 MiB (evicts everything), then read another 256 MiB so that the lines left in L2 are clean:
        # otherwise the timed kernels would also pay for writing the flush's dirty lines back
        flush_buf.fill_(1)
        flush_src.max()

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
                flush_l2()
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
        if rank != 0:
            if world > 1:
                dist.destroy_process_group()
            return
        print(json.dumps({"metric": "nvfp4_linear_fwd_bwd_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": world,
                          "steps": args.steps, "ms_per_step": ms_step, "gpu_launches": int(launches), "note": "--no-breakdown run"}))
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- end to end: host buffers in, results out, copies inside the timed region -------------------------------
    pinned_in, h2d, d2h = [], 0, 0
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

    e2e_steps = max(2, min(args.steps, 5))
    step_e2e()
    ms_e2e, _ = timed(step_e2e, e2e_steps)
    e2e_value = world * fl / (ms_e2e * 1e-3) / 1e12

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- per-kernel breakdown on the largest linear (rank 0): which kernel dominates, and its roofline ----------
    pk = peaks()
    L = max(lins, key=lambda l: l.D * l.C)
    ws_q = b._workspace(1 << 20, dev)

    def t_of(fn, n=20):
        for _ in range(3):
            fn()
        t, _ = timed(fn, n)
        return t * 1e-3

    T, D, C = tokens, L.D, L.C
    q3 = b.alloc_operand(T, C, gs_mode, device=dev)
    q4 = b.alloc_operand(D, C, gs_mode, device=dev)
    q5 = b.alloc_operand(C, T, gs_mode, device=dev)
    q6 = b.alloc_operand(D, T, gs_mode, device=dev)
    b.nvfp4_linear_fwd(L.X, L.W[0], L.cfg, Y=L.Y, saved=L.saved, workspace=L.ws[0])
    parts = {}

    def add(name, fn, alg_bytes=None, flops=None):
        t = t_of(fn)
        parts[name] = dict(seconds=t, GBps=(alg_bytes / t / 1e9 if alg_bytes else None),
                           TFLOPs=(flops / t / 1e12 if flops else None), bytes=alg_bytes, flops=flops)

    qbytes = lambda n: n * (2 + 0.5 + 1.0 / 16)
    rqbytes = lambda n: n * 2 * (0.5 + 1.0 / 16)
    amax_extra = 2.0 if gs_mode != 2 else 0.0  # TENSOR / ROW modes read the source twice (amax pre-pass)
    add("quantize_rows_X(Q1)", lambda: b.nvfp4_quantize(L.X, b.AXIS_ROW, b.ROUND_RTN, 0, 1, gs_mode, out=L.saved.qx, workspace=ws_q),
        qbytes(T * D) + amax_extra * T * D)
    add("quantize_rows_dY_SR(Q3)", lambda: b.nvfp4_quantize(L.dY, b.AXIS_ROW, b.ROUND_SR, 0, 3, gs_mode, out=q3, workspace=ws_q),
        qbytes(T * C) + amax_extra * T * C)
    add("quantize_cols_dY_SR(Q5)", lambda: b.nvfp4_quantize(L.dY, b.AXIS_COL, b.ROUND_SR, 0, 5, gs_mode, out=q5, workspace=ws_q),
        qbytes(T * C) + amax_extra * T * C)
    add("requantize_t_W(Q4)", lambda: b.nvfp4_requantize_t(L.saved.qw, b.ROUND_SR, 0, 4, out=q4, workspace=ws_q), rqbytes(C * D))
    add("requantize_t_X(Q6)", lambda: b.nvfp4_requantize_t(L.saved.qx, b.ROUND_SR, 0, 6, out=q6, workspace=ws_q), rqbytes(T * D))
    gemm_bytes = lambda M, N, K, ob: 0.5625 * (M + N) * K + ob * M * N
    add("gemm_fwd", lambda: b.nvfp4_gemm(L.saved.qx, L.saved.qw, b.DT_BF16, out=L.Y), gemm_bytes(T, C, D, 2), 2.0 * T * C * D)
    add("gemm_dx", lambda: b.nvfp4_gemm(q3, q4, b.DT_BF16, out=L.dXo), gemm_bytes(T, D, C, 2), 2.0 * T * C * D)
    add("gemm_dw", lambda: b.nvfp4_gemm(q5, q6, b.DT_F32, out=L.dWo), gemm_bytes(C, D, T, 4), 2.0 * T * C * D)
    dom = max(parts, key=lambda k: parts[k]["seconds"])
    dp = parts[dom]
    fp4_peak = pk["bf16"] * 4.0  # dense FP4 : dense BF16 nominal ratio 9 : 2.25
    if dom.startswith("gemm"):
        t_tensor = dp["flops"] / (fp4_peak * 1e12)
        t_hbm = dp["bytes"] / (pk["hbm"] * 1e9)
        if t_tensor >= t_hbm:
            roof = dict(bound="tensor", achieved=dp["TFLOPs"], peak=fp4_peak, unit="TFLOP/s", frac=dp["TFLOPs"] / fp4_peak)
        else:
            roof = dict(bound="hbm", achieved=dp["GBps"], peak=pk["hbm"], unit="GB/s", frac=dp["GBps"] / pk["hbm"])
    else:
        roof = dict(bound="hbm", achieved=dp["GBps"], peak=pk["hbm"], unit="GB/s", frac=dp["GBps"] / pk["hbm"])
    roof.update(kernel=f"{dom} on {L.name} {D}->{C}, tokens {T}", peak_source=f"of {pk['source']}", traffic=None,
                algorithmic_bytes_per_launch=dp["bytes"], seconds_per_launch=dp["seconds"])
    if args.workload == "attn" and args.gs == "tensor" and dom in PROFILED_TRAFFIC:
        roof["traffic"], roof["traffic_source"] = PROFILED_TRAFFIC[dom]

    # ---- the oracle beside it ------------------------------------------------------------------------------------
    cpu = None
    if world == 1 and not args.no_cpu:
        from oracle import nvfp4_oracle as orc

        dt, sfl, desc = oracle_sample_step(args.workload, gs_mode, args.cpu_tokens, args.rht, all_linears=True)
        cpu = {"value": sfl / dt / 1e12, "unit": "TFLOP/s", "cores": orc.threads(), "kind": "oracle", "sample": desc,
               "seconds": dt}

    line = {
        "metric": "nvfp4_linear_fwd_bwd_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "fp4(e2m1)xfp4 with ue4m3 block scales, f32 accumulate", "data": "synthetic",
        "config": {"workload": workload_name(args), "gs_mode": args.gs, "outcontrol_fraction": args.outliers, "rht": bool(args.rht), "sr_scale_up": bool(args.sr_scale_up), "outlier_fp8": bool(args.outlier_fp8), "weight_block": "16x16" if args.w16x16 else "1x16", "launch": "cuda_graph_replay" if args.graph else "stream", "l2": "256 MiB write + 256 MiB read flush before every timed step",
                   "timing": "CUDA events per step on the launch stream, summed"},
        "e2e": {"value": e2e_value, "unit": "TFLOP/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e},
        "gpu_launches": int(launches), "clocks": clocks, "roofline": roof, "cpu_baseline": cpu,
        "kernels": {k: {kk: (round(vv, 9) if isinstance(vv, float) else vv) for kk, vv in v.items() if kk in ("seconds", "GBps", "TFLOPs")}
                    for k, v in parts.items()},
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
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    flush_src = torch.zeros(256 << 20, dtype=torch.uint8, device=dev)

    def t_of(fn, n):
        for _ in range(3):
            fn()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        torch.cuda.synchronize()
        for i in range(n):
            flush_buf.fill_(1)
            flush_src.max()
            ev[i][0].record()
            fn()
            ev[i][1].record()
        torch.cuda.synchronize()
        ms = sorted(a.elapsed_time(bb) for a, bb in ev)
        return ms[len(ms) // 2] * 1e-3

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
    print(json.dumps({"aux": out, "peaks": pk}))


def run_sweep(args):
    """Roofline sweep (square and skinny GEMMs with their quantizers), one JSON line with a list of shapes.
    Not the headline line: a measurement aid for the large-shape roofline fractions."""
    import torch

    from paper_2510_27527_b200 import binding as b

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    gs_mode = GS[args.gs]
    pk = peaks()
    shapes = synth.CONFIGS[5]["shapes"] if not args.shapes else [tuple(int(v) for v in t.split("x")) for t in args.shapes.split(",")]
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    flush_src = torch.zeros(256 << 20, dtype=torch.uint8, device=dev)
    out = []

    def t_of(fn, n):
        for _ in range(3):
            fn()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        torch.cuda.synchronize()
        for i in range(n):
            flush_buf.fill_(1)
            flush_src.max()  # leave clean lines in L2
            ev[i][0].record()
            fn()
            ev[i][1].record()
        torch.cuda.synchronize()
        ms = sorted(a.elapsed_time(bb) for a, bb in ev)
        return ms[len(ms) // 2] * 1e-3, ms[0] * 1e-3

    # tensor-core ceiling of this machine under load: the issue loop without memory traffic (4 MMAs of 128 x 256 x 64 per turn)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    probe_flops = b.nvfp4_mma_issue_probe(2048, status)
    sec, _ = t_of(lambda: b.nvfp4_mma_issue_probe(2048, status), 10)
    issue_loop_tflops = probe_flops / sec / 1e12 if int(status.item()) == 0 else None
    g = torch.Generator(device=dev)
    g.manual_seed(5)
    for (M, N, K) in shapes:
        A = torch.randn((M, K), device=dev, generator=g, dtype=torch.float32)
        nch = max(1, int(K * 0.005))
        A[:, torch.randperm(K, device=dev, generator=g)[:nch]] *= 100.0
        A = A.to(torch.bfloat16)
        Bm = torch.randn((N, K), device=dev, generator=g, dtype=torch.float32).to(torch.bfloat16)
        qa, qb = b.alloc_operand(M, K, gs_mode, device=dev), b.alloc_operand(N, K, gs_mode, device=dev)
        qat = b.alloc_operand(K, M, gs_mode, device=dev)
        ws = b._workspace(1 << 20, dev)
        C = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
        n = args.steps
        r = {"M": M, "N": N, "K": K}
        qbytes = lambda e: e * (2 + 0.5 + 1.0 / 16)
        amax_extra = 2.0 if gs_mode != 2 else 0.0
        for name, fn, nelem in (
            ("quantize_rows_rtn_A", lambda: b.nvfp4_quantize(A, b.AXIS_ROW, b.ROUND_RTN, 0, 1, gs_mode, out=qa, workspace=ws), M * K),
            ("quantize_rows_sr_A", lambda: b.nvfp4_quantize(A, b.AXIS_ROW, b.ROUND_SR, 0, 3, gs_mode, out=qa, workspace=ws), M * K),
            ("quantize_cols_sr_A", lambda: b.nvfp4_quantize(A, b.AXIS_COL, b.ROUND_SR, 0, 5, gs_mode, out=qat, workspace=ws), M * K),
        ):
            med, best = t_of(fn, n)
            r[name] = {"us": med * 1e6, "GBps": qbytes(nelem) / med / 1e9, "GBps_incl_amax_read": (qbytes(nelem) + amax_extra * nelem) / med / 1e9,
                       "frac_hbm_measured": (qbytes(nelem) + amax_extra * nelem) / med / 1e9 / pk["hbm"]}
        b.nvfp4_quantize(A, b.AXIS_ROW, b.ROUND_RTN, 0, 1, gs_mode, out=qa, workspace=ws)
        b.nvfp4_quantize(Bm, b.AXIS_ROW, b.ROUND_RTN, 0, 2, gs_mode, out=qb, workspace=ws)
        med, best = t_of(lambda: b.nvfp4_requantize_t(qa, b.ROUND_SR, 0, 6, out=qat, workspace=ws), n)
        r["requantize_t_A"] = {"us": med * 1e6, "GBps": M * K * 1.125 / med / 1e9, "Gelem_per_s": M * K / med / 1e9}
        med, best = t_of(lambda: b.nvfp4_gemm(qa, qb, b.DT_BF16, out=C), n)
        fl = 2.0 * M * N * K
        r["gemm"] = {"us": med * 1e6, "best_us": best * 1e6, "TFLOPs": fl / med / 1e12, "frac_of_4x_bf16_measured": fl / med / 1e12 / (4 * pk["bf16"]),
                     "frac_of_9PF_nominal": fl / med / 1e12 / 9000.0,
                     "frac_of_issue_loop": (fl / med / 1e12 / issue_loop_tflops) if issue_loop_tflops else None}

        def fused():
            b.nvfp4_quantize(A, b.AXIS_ROW, b.ROUND_RTN, 0, 1, gs_mode, out=qa, workspace=ws)
            b.nvfp4_quantize(Bm, b.AXIS_ROW, b.ROUND_RTN, 0, 2, gs_mode, out=qb, workspace=ws)
            b.nvfp4_gemm(qa, qb, b.DT_BF16, out=C)

        med, best = t_of(fused, n)
        r["quantize_plus_gemm"] = {"us": med * 1e6, "TFLOPs": fl / med / 1e12}
        out.append(r)
        del A, Bm, qa, qb, qat, C
    print(json.dumps({"sweep": out, "gs_mode": args.gs, "peaks": pk, "mma_issue_loop_TFLOPs": issue_loop_tflops}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="attn", choices=list(WORKLOADS))
    ap.add_argument("--gs", default="tensor", choices=list(GS))
    ap.add_argument("--ref-tokens", type=int, default=1024, help="token slab of one oracle step (reference arm)")
    ap.add_argument("--cpu-tokens", type=int, default=8192, help="token slab of the cpu_baseline leg (every linear of one layer)")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--outliers", type=float, default=0.0,
                    help="OutControl: fraction of input channels kept in BF16 (0 = off; the paper uses 0.10)")
    ap.add_argument("--rht", action="store_true", help="random Hadamard transformation (block 16) in the four backward quantizers")
    ap.add_argument("--outlier-fp8", action="store_true", help="with --outliers: outlier channels on a power-of-two scaled E4M3 grid instead of BF16")
    ap.add_argument("--w16x16", action="store_true", help="weights in 16x16 scale squares (the recipe the paper compares with): no Q4 in backward")
    ap.add_argument("--sr-scale-up", action="store_true", help="backward quantizers round the block scale up (strictly unbiased variant)")
    ap.add_argument("--graph", action=argparse.BooleanOptionalAction, default=True,
                    help="capture one step in a CUDA graph and time its replays (default; --no-graph launches every kernel from the host)")
    ap.add_argument("--no-breakdown", action="store_true", help="only warm-up + timed steps (used for ncu launch lists)")
    ap.add_argument("--sweep", action="store_true", help="roofline sweep of the large GEMM shapes instead of the step benchmark")
    ap.add_argument("--aux", action="store_true", help="HBM roofline of the calibration and OsciReset kernels instead of the step benchmark")
    ap.add_argument("--shapes", default="", help="with --sweep: comma list of MxNxK")
    args = ap.parse_args()
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
