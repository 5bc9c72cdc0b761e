#!/usr/bin/env python
"""Benchmark of the ConvAttn forward (ESC paper, Section 3.3, Eq. 4) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--layout nhwc|nchw]
    python bench.py --impl reference ...      # the CPU oracle on the host cores, same metric

A step is one whole forward pass (GAP + kernel estimator, then the fused stencil with its
copy-through) over one synthetic batch.  Prints ONE JSON line on rank 0.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "ConvAttn fwd Mpixel/s"
UNIT = "Mpixel/s"
DEFAULT_WORKLOAD = "cfg3_640x360_bf16"       # 640x360x64 bf16: the configuration the metric is quoted on
SM_COUNT_NOMINAL = 148
FMA_LANES_PER_SM = 128
L2_BYTES = 126 * 1024 * 1024
# dram__bytes_read.sum + dram__bytes_write.sum of one stencil-kernel launch from the ncu capture summarised under
# profiles/, keyed by (workload, layout, library version the capture was taken with).  Reported only while the
# library still has that version; otherwise the kernel has changed since and the figure is withheld.
# (Versions 109 to 111 added entry points and kernels for other variants; the kernel timed here is the one captured at 108.)
NCU_TRAFFIC_BYTES = {("cfg3_640x360_bf16", "nhwc", v): 29.56e6 + 0.47e6 for v in (108, 109, 110, 111)}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "sm_max_mhz": float(p.get("sm_max_mhz", 1965.0)),
                "bf16_tflops": float(p.get("bf16_tflops", 1590.0)), "source": "measured"}
    except Exception:
        return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0, "bf16_tflops": 1590.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []
        self.t_mark = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def mark(self):
        self.t_mark = time.time()

    def stop(self):
        t_end = time.time()
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        t0 = self.t_mark or 0.0
        rows = [l for (t, l) in self.lines if t0 <= t <= t_end + 0.2] or [l for (_, l) in self.lines[-3:]]
        mhz, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            parts = [q.strip() for q in r.split(",")]
            if len(parts) < 8:
                continue
            try:
                mhz.append(float(parts[0])); mx = float(parts[1])
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(mhz) if mhz else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(mhz)}


def rank_seed(wl, rank):
    """Each rank draws its own batch (weak scaling: the per-GPU workload is fixed as N grows)."""
    return wl.seed + 1000 * rank


def max_over_ranks(value, world, device=None):
    """Largest value over all ranks (the job is as slow as its slowest rank)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist

    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(pixels_per_rank, world, ms_per_step):
    """Whole-job throughput in Mpixel/s: every rank processes its own batch in the same step time."""
    return world * pixels_per_rank / (ms_per_step * 1e-3) / 1e6


def time_oracle(wl, layout_unused, budget_s=15.0, threads=None):
    """Oracle on the host cores over a bounded sample (a band of output rows of the same workload)."""
    import oracle
    from paper_2503_06671_b200 import synth

    d = synth.make_workload(wl)
    cores = threads or oracle.max_threads()
    oracle.set_threads(cores)
    g = oracle.gap(d["x"], wl.C_a)
    dk = oracle.dynkernel(g, d["w_dyn"], d["b_dyn"])
    rows = min(wl.H, 4)
    t0 = time.perf_counter()
    oracle.stencil(d["x"], wl.C_a, d["w_large"], dk, rows=(0, rows))
    t_probe = time.perf_counter() - t0
    rows = int(max(rows, min(wl.H, rows * budget_s / max(t_probe, 1e-4))))
    y0 = max(0, (wl.H - rows) // 2)
    reps = int(max(1, min(50, (0.7 * budget_s) / max(t_probe * rows / 4.0, 1e-3)))) if rows >= wl.H else 1
    t0 = time.perf_counter()
    for _ in range(reps):
        g = oracle.gap(d["x"], wl.C_a)
        dk = oracle.dynkernel(g, d["w_dyn"], d["b_dyn"])
        oracle.stencil(d["x"], wl.C_a, d["w_large"], dk, rows=(y0, y0 + rows))
    dt = (time.perf_counter() - t0) / reps
    px = wl.B * rows * wl.W
    return {"value": px / dt / 1e6, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"rows {y0}..{y0 + rows} of {wl.H} ({px} of {wl.pixels} pixels, all {wl.C} channels), "
                      f"{reps} repetition(s) of {dt:.2f} s, GAP over the whole map included"}, d


def run_reference(args, wl):
    """The oracle as the reference arm: each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle

    per_step = max(1.0, min(20.0, 90.0 / max(1, args.steps + args.warmup)))
    vals, last = [], None
    for i in range(args.warmup + args.steps):
        last, _ = time_oracle(wl, None, budget_s=per_step)
        if i >= args.warmup:
            vals.append(last["value"])
    v = sum(vals) / len(vals)
    ms = wl.pixels / (v * 1e6) * 1e3
    last["value"] = v
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": {"workload": wl.name, "B": wl.B, "C": wl.C, "C_a": wl.C_a,
                                                         "H": wl.H, "W": wl.W, "K": wl.K},
        "cpu_baseline": last, "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--layout", default="nhwc", choices=["nhwc", "nchw"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--launch", default="graph", choices=["graph", "eager"],
                    help="timed region: one CUDA graph holding the K steps (default) or K eager calls")
    args = ap.parse_args()

    from paper_2503_06671_b200 import synth

    wl = synth.WORKLOADS_BY_NAME[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
        return

    import numpy as np
    import torch
    import torch.distributed as dist

    import paper_2503_06671_b200 as pkg

    pkg.lib()   # raises if the CUDA library is missing: there is no fall-back
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    W_ = max(3, args.warmup)

    layout = synth.NHWC if args.layout == "nhwc" else synth.NCHW
    lay_code = pkg.ESC_NHWC if layout == synth.NHWC else pkg.ESC_NCHW
    tdt = torch.bfloat16 if wl.dtype == synth.BF16 else torch.float32
    es = 2 if wl.dtype == synth.BF16 else 4

    # ---- inputs: seeded, generated on the host, resident in HBM before the timed region -------
    d = synth.make_inputs(wl.B, wl.C, wl.C_a, wl.H, wl.W, wl.K, wl.dtype, rank_seed(wl, rank), wl.per_image_scale)
    x_host = torch.from_numpy(synth.to_layout(d["x"], layout)).to(tdt).pin_memory()
    w_host = [torch.from_numpy(d[k]).to(tdt) for k in ("w_large", "w_dyn", "b_dyn")]
    wl_d, wd_d, bd_d = (t.cuda() for t in w_host)
    tensor_bytes = x_host.numel() * es
    # rotate through enough (x, out) pairs that consecutive steps never find their data in L2
    n_rot = max(2, int(np.ceil(2.5 * L2_BYTES / (2 * tensor_bytes))))
    xs = [x_host.cuda() for _ in range(n_rot)]
    outs = [torch.empty_like(xs[0]) for _ in range(n_rot)]
    ws = pkg.new_workspace(wl.B, wl.C_a, wl.H, wl.W, wl.K)

    def step(i):
        pkg.esc_convattn_forward_ex(xs[i % n_rot], wl.C_a, wl.K, wl_d, wd_d, bd_d, outs[i % n_rot], lay_code, ws)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(W_):
        step(i)
    launches_per_step = pkg.esc_convattn_last_launches()
    path = pkg.esc_convattn_last_path()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    # extend very short runs so that the clock sampler sees the load (repeat the K-step region)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # The K steps are captured once into a CUDA graph (the library's calls are plain stream-ordered
    # launches) and the graph is launched once inside the timed region; --launch eager times K calls.
    launch_mode, graph, side = "eager", None, torch.cuda.Stream()
    if args.launch == "graph":
        try:
            with torch.cuda.stream(side):
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    for i in range(args.steps):
                        step(i)
                graph.replay()                      # one untimed launch: uploads the graph
            torch.cuda.synchronize()
            launch_mode = "graph"
        except Exception as exc:                    # capture refused: fall back to eager launches, and say so
            graph = None
            launch_mode = f"eager (graph capture failed: {type(exc).__name__})"
            torch.cuda.synchronize()
    barrier()
    sampler.mark()
    if graph is not None:
        with torch.cuda.stream(side):
            e0.record()
            graph.replay()
            e1.record()
    else:
        e0.record()
        for i in range(args.steps):
            step(i)
        e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    # keep the GPU under the same load a little longer for the clock record (not part of the number)
    t_end = time.time() + 0.4
    j = 0
    while time.time() < t_end:
        for _ in range(50):
            step(j); j += 1
        torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    assert pkg.esc_convattn_device_status(ws) == 0, "device-side wait timed out"
    ms_total = max_over_ranks(ms_total, world, "cuda")
    ms_step = ms_total / args.steps
    value = whole_job_value(wl.pixels, world, ms_step)

    # ---- dominant kernel alone: the fused stencil (stage 2), explicit dk, same rotation ------------
    dk = torch.empty(wl.B, wl.C_a, 3, 3, device="cuda")
    pkg.esc_convattn_dynkernel(xs[0], wl.C_a, wd_d, bd_d, dk, lay_code, ws)
    for i in range(W_):
        pkg.esc_convattn_stencil(xs[i % n_rot], wl.C_a, wl.K, wl_d, dk, outs[i % n_rot], lay_code, ws)
    stencil_launches = pkg.esc_convattn_last_launches()
    torch.cuda.synchronize()
    def timed(fn):
        """Average device time of one call of fn(i) over args.steps calls, launched like the timed region above."""
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if graph is not None:
            try:
                with torch.cuda.stream(side):
                    gk = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(gk, stream=side):
                        for i in range(args.steps):
                            fn(i)
                    gk.replay()
                    torch.cuda.synchronize()
                    a.record()
                    gk.replay()
                    b.record()
                torch.cuda.synchronize()
                return a.elapsed_time(b) / args.steps
            except Exception:
                torch.cuda.synchronize()
        a.record()
        for i in range(args.steps):
            fn(i)
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / args.steps

    ms_kernel = timed(lambda i: pkg.esc_convattn_stencil(xs[i % n_rot], wl.C_a, wl.K, wl_d, dk, outs[i % n_rot], lay_code, ws))
    ms_gap = timed(lambda i: pkg.esc_convattn_dynkernel(xs[i % n_rot], wl.C_a, wd_d, bd_d, dk, lay_code, ws))
    # the same stencil stage with its input resident in L2 (one buffer, no rotation): the case inside a network,
    # where the previous layer has just written x; reported beside the cold figure, never instead of it
    ms_kernel_hot = timed(lambda i: pkg.esc_convattn_stencil(xs[0], wl.C_a, wl.K, wl_d, dk, outs[0], lay_code, ws)) \
        if 2 * tensor_bytes < L2_BYTES else None
    # the whole step once more with the paper's two-layer estimator (hidden width 8, exact GELU), for comparison
    mlp_d = [torch.from_numpy(v).to(tdt).cuda() for v in synth.make_estimator_mlp(wl.C_a, 8, wl.dtype, wl.seed).values()]
    ms_step_mlp = timed(lambda i: pkg.esc_convattn_forward_mlp(xs[i % n_rot], wl.C_a, wl.K, wl_d, *mlp_d, outs[i % n_rot], lay_code, ws))
    # and with the decomposed large kernel of Eq. 5 (point-wise LK^c in front of the depth-wise stage)
    wp_d = torch.from_numpy(synth.make_pointwise(wl.C_a, wl.dtype, wl.seed)).to(tdt).cuda()
    ms_step_pw = timed(lambda i: pkg.esc_convattn_forward_pw(xs[i % n_rot], wl.C_a, wl.K, wl_d, wp_d, wd_d, bd_d, outs[i % n_rot], lay_code, ws))
    # and with the dense large kernel of the main model (Section 3.2): an implicit GEMM on the tensor cores
    dense = None
    if wl.C_a == 16 and wl.K == 13:
        wdn_d = torch.from_numpy(synth.make_dense_kernel(wl.C_a, wl.K, wl.dtype, wl.seed)).to(tdt).cuda()
        ms_dense = timed(lambda i: pkg.esc_convattn_forward_dense(xs[i % n_rot], wl.C_a, wl.K, wdn_d, wd_d, bd_d, outs[i % n_rot], lay_code, ws))
        fl = 2.0 * wl.C_a * wl.C_a * wl.K * wl.K * wl.pixels
        bf16_peak = peaks()["bf16_tflops"]
        dense = {"ms_per_step": ms_dense, "bound": "tensor", "achieved": fl / (ms_dense * 1e-3) / 1e12, "peak": bf16_peak,
                 "unit": "TFLOP/s", "frac": fl / (ms_dense * 1e-3) / 1e12 / bf16_peak,
                 "note": "whole step (GAP kernel + dense stencil kernel with copy blocks); warp-level mma.sync"}

    pk = peaks()
    flops = 2.0 * wl.K * wl.K * wl.C_a * wl.pixels                    # merged 169-tap form, Eq. 5
    alg_bytes = 2.0 * wl.C * es * wl.pixels                            # every byte read once, written once
    peak_tflops = SM_COUNT_NOMINAL * FMA_LANES_PER_SM * 2 * pk["sm_max_mhz"] * 1e6 / 1e12
    t_alu = flops / (peak_tflops * 1e12)
    t_hbm = alg_bytes / (pk["hbm_gbs"] * 1e9)
    if t_alu >= t_hbm:
        ach = flops / (ms_kernel * 1e-3) / 1e12
        roof = {"bound": "alu", "achieved": ach, "peak": peak_tflops, "unit": "TFLOP/s", "frac": ach / peak_tflops,
                "traffic": None,
                "peak_source": f"fp32 FMA pipe: {SM_COUNT_NOMINAL} SMs x {FMA_LANES_PER_SM} lanes x 2 flop x {pk['sm_max_mhz']:.0f} MHz "
                               f"({pk['source']} max SM clock)"}
    else:
        ach = alg_bytes / (ms_kernel * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": ach / pk["hbm_gbs"],
                "traffic": None, "peak_source": f"{pk['source']} copy bandwidth"}
    roof["traffic"] = NCU_TRAFFIC_BYTES.get((wl.name, args.layout, pkg.esc_version()))
    roof.update({"kernel": "stencil (stage 2)", "kernel_ms": ms_kernel, "gap_kernel_ms": ms_gap,
                 "kernel_ms_input_resident_in_l2": ms_kernel_hot,
                 "whole_step_frac": max(t_alu, t_hbm) / (ms_step * 1e-3),
                 "hbm_side": {"algorithmic_GBps": alg_bytes / (ms_kernel * 1e-3) / 1e9, "of_peak": alg_bytes / (ms_kernel * 1e-3) / 1e9 / pk["hbm_gbs"]}})

    # ---- end to end through the host-buffer entries (copies inside the timed region) ----------------
    # Every step uploads x and the weights from pinned host memory and downloads the whole result.  The
    # two-slot submit / wait pair lets the upload of step i overlap the download of step i - 1 (PCIe is
    # full duplex); the blocking single call is timed too.
    out_hosts = [torch.empty_like(x_host).pin_memory() for _ in range(2)]
    w_pinned = [t.pin_memory() for t in w_host]
    n_e2e = max(4, min(args.steps, 20))
    for _ in range(2):
        pkg.esc_convattn_forward_host(x_host, wl.C_a, wl.K, *w_pinned, out_hosts[0], lay_code)
    barrier()
    t0 = time.perf_counter()
    for _ in range(n_e2e):
        pkg.esc_convattn_forward_host(x_host, wl.C_a, wl.K, *w_pinned, out_hosts[0], lay_code)
    dt_block = time.perf_counter() - t0    # the call synchronises before it returns
    for i in range(2):
        pkg.esc_convattn_forward_host_submit(i, x_host, wl.C_a, wl.K, *w_pinned, out_hosts[i], lay_code)
    pkg.esc_convattn_forward_host_wait(0); pkg.esc_convattn_forward_host_wait(1)
    barrier()
    t0 = time.perf_counter()
    for i in range(n_e2e):
        pkg.esc_convattn_forward_host_submit(i % 2, x_host, wl.C_a, wl.K, *w_pinned, out_hosts[i % 2], lay_code)
        if i > 0:
            pkg.esc_convattn_forward_host_wait((i - 1) % 2)
    pkg.esc_convattn_forward_host_wait((n_e2e - 1) % 2)
    dt = time.perf_counter() - t0
    dt = max_over_ranks(dt, world, "cuda")
    dt_block = max_over_ranks(dt_block, world, "cuda")
    w_bytes = sum(t.numel() for t in w_host) * es
    e2e = {"value": whole_job_value(wl.pixels, world, dt / n_e2e * 1e3), "unit": UNIT, "h2d_bytes_per_step": tensor_bytes + w_bytes,
           "d2h_bytes_per_step": tensor_bytes, "steps": n_e2e,
           "api": "esc_convattn_forward_host_submit / _wait, two slots in turn (pinned host buffers)",
           "blocking_call_value": whole_job_value(wl.pixels, world, dt_block / n_e2e * 1e3)}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu, _ = time_oracle(wl, layout)

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": W_,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl.name, "B": wl.B, "C": wl.C, "C_a": wl.C_a, "H": wl.H, "W": wl.W, "K": wl.K,
                       "storage": wl.dtype, "layout": args.layout, "sharding": "replicas: one image batch per GPU, no collective",
                       "l2": f"inputs larger than L2: {n_rot} rotating (x,out) pairs, {n_rot * 2 * tensor_bytes / 1e6:.0f} MB",
                       "stencil_path": {1: "generic", 2: "tma"}.get(path, str(path)),
                       "launch": launch_mode, "estimator": "one linear layer", "large_kernel": "depth-wise LK^s"},
            "roofline": roof, "cpu_baseline": cpu, "e2e": e2e, "clocks": clocks,
            "gpu_launches": launches_per_step * args.steps,
            "launches_per_step": launches_per_step, "stencil_stage_launches": stencil_launches,
            "GB_per_s_whole_step": alg_bytes / (ms_step * 1e-3) / 1e9,
            "ms_per_step_two_layer_estimator_h8": ms_step_mlp,
            "ms_per_step_decomposed_large_kernel": ms_step_pw,
            "dense_large_kernel": dense,
        }))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
