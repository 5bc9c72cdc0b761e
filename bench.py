#!/usr/bin/env python
"""Benchmark of the ConvAttn forward (ESC paper, Section 3.3, Eq. 4) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--layout nhwc|nchw]
    python bench.py --impl reference ...      # the CPU oracle on the host cores, same metric

A step is one whole forward pass (GAP + kernel estimator, then the fused stencil with its
copy-through) over one synthetic batch.  Prints ONE JSON line on rank 0.

How a number is taken: the K steps are captured once into a CUDA graph; a sample is R replays of that
graph (R chosen so that a sample is at least 0.1 s of GPU work) between two CUDA events on the launch
stream; eleven samples, median reported with min and max beside it.  Inputs rotate through enough
(x, out) pairs to exceed the L2, so no step finds its data cached.
"""
from __future__ import annotations

import argparse
import ctypes
import hashlib
import json
import math
import os
import re
import shutil
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
FMA_LANES_PER_SM = 128
L2_BYTES = 126 * 1024 * 1024
SAMPLES = 11
MIN_SAMPLE_S = 0.1
PATH_NAMES = {1: "generic", 2: "tma-fp32", 3: "tensor-dense-mma.sync", 4: "tensor-toeplitz", 5: "tensor-dense-tcgen05", 6: "tensor-toeplitz-nchw"}
KERNEL_FILES = {1: "stencil_generic.cuh", 2: "stencil_tma.cuh", 3: "stencil_dense.cuh", 4: "stencil_toeplitz.cuh", 5: "stencil_dense_umma.cuh", 6: "stencil_toeplitz_nchw.cuh"}
TOEPLITZ_DENSITY = 13.0 / 32.0               # useful share of the multiply-adds the banded-Toeplitz kernel issues
PEAK_SRC = os.path.join(ROOT, "bench_fp32_peak.cu")
PEAK_LIB = os.path.join(ROOT, "paper_2503_06671_b200", "lib", "libbench_fp32_peak.so")


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "sm_max_mhz": float(p.get("sm_max_mhz", 1965.0)),
                "bf16_tflops": float(p.get("bf16_tflops", 1590.0)), "source": "measured"}
    except Exception:
        return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0, "bf16_tflops": 1590.0, "source": "fallback"}


def build_peak_probe(force=False):
    """Compile bench_fp32_peak.cu (the register-only FP32 multiply-add probe) into its own shared object."""
    if not force and os.path.exists(PEAK_LIB) and os.path.getmtime(PEAK_LIB) >= os.path.getmtime(PEAK_SRC):
        return PEAK_LIB
    nvcc = os.environ.get("NVCC") or shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    os.makedirs(os.path.dirname(PEAK_LIB), exist_ok=True)
    tmp = PEAK_LIB + ".tmp%d" % os.getpid()
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-shared",
                           "-Xcompiler", "-fPIC", "-o", tmp, PEAK_SRC])
    os.replace(tmp, PEAK_LIB)
    return PEAK_LIB


def measure_fp32_peak():
    """TFLOP/s of register-only fp32 multiply-adds on the current device, scalar and packed, or None."""
    try:
        lib = ctypes.CDLL(build_peak_probe())
        lib.fp32_peak_measure.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_double)]
        out = (ctypes.c_double * 4)()
        rc = lib.fp32_peak_measure(4096, 5, out)      # about 2 ms per launch
        if rc != 0:
            return {"error": f"cuda error {rc}"}
        return {"scalar_tflops": out[0], "packed_tflops": out[1], "sms": int(out[2]),
                "how": "bench_fp32_peak.cu: 16 independent chains per thread, 2 x 512 threads per SM, best of 5 launches of ~2 ms"}
    except Exception as exc:
        return {"error": f"{type(exc).__name__}: {exc}"}


def ncu_traffic(kernel_file, workload, layout):
    """dram bytes per launch of the dominant kernel from the ncu summary under profiles/, if that summary
    was taken from the kernel source as it stands now (it records the source file's hash), else None."""
    try:
        with open(os.path.join(ROOT, "paper_2503_06671_b200", "csrc", kernel_file), "rb") as f:
            digest = hashlib.sha256(f.read()).hexdigest()[:16]
        for name in sorted(os.listdir(os.path.join(ROOT, "profiles"))):
            text = open(os.path.join(ROOT, "profiles", name)).read()
            m = re.search(r"^traffic-record: workload=(\S+) layout=(\S+) source=(\S+) sha256=([0-9a-f]+) dram_bytes_per_launch=([0-9.eE+]+)",
                          text, flags=re.M)
            if m and m.group(1) == workload and m.group(2) == layout and m.group(3) == kernel_file and m.group(4) == digest:
                return float(m.group(5))
    except Exception:
        pass
    return None


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
        self.t_end = None

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

    def mark_end(self):
        self.t_end = time.time()

    def stop(self):
        t_end = self.t_end or time.time()
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.1)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        t0 = self.t_mark or 0.0
        rows = [l for (t, l) in self.lines if t0 <= t <= t_end + 0.05] or [l for (_, l) in self.lines[-3:]]
        mhz, mx, reasons, watts = [], None, set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            parts = [q.strip() for q in r.split(",")]
            if len(parts) < 8:
                continue
            try:
                mhz.append(float(parts[0])); mx = float(parts[1]); watts.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(mhz) if mhz else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(mhz), "power_w_max": max(watts) if watts else None}


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


def time_oracle(wl, budget_s=15.0, threads=None):
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
    oracle.set_threads(oracle.max_threads())
    return {"value": px / dt / 1e6, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"rows {y0}..{y0 + rows} of {wl.H} ({px} of {wl.pixels} pixels, all {wl.C} channels), "
                      f"{reps} repetition(s) of {dt:.2f} s, GAP over the whole map included"}


def run_reference(args, wl):
    """The oracle as the reference arm: each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    per_step = max(1.0, min(20.0, 90.0 / max(1, args.steps + args.warmup)))
    vals, last = [], None
    for i in range(args.warmup + args.steps):
        last = time_oracle(wl, budget_s=per_step)
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


class GraphTimer:
    """Times fn(i), i = 0..K-1, as a CUDA graph replayed R times per sample; medians over SAMPLES samples."""

    def __init__(self, torch, steps, launch="graph"):
        self.torch = torch
        self.steps = steps
        self.launch = launch
        self.side = torch.cuda.Stream()
        self.mode = launch

    def capture(self, fn):
        torch = self.torch
        if self.launch != "graph":
            return None
        try:
            with torch.cuda.stream(self.side):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=self.side):
                    for i in range(self.steps):
                        fn(i)
                g.replay()                              # one untimed launch: uploads the graph
            torch.cuda.synchronize()
            return g
        except Exception as exc:                        # capture refused: eager launches, and say so
            self.mode = f"eager (graph capture failed: {type(exc).__name__})"
            torch.cuda.synchronize()
            return None

    def _once(self, fn, g, reps):
        torch = self.torch
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if g is not None:
            with torch.cuda.stream(self.side):
                a.record()
                for _ in range(reps):
                    g.replay()
                b.record()
        else:
            a.record()
            for _ in range(reps):
                for i in range(self.steps):
                    fn(i)
            b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / (reps * self.steps)   # ms per step

    def measure(self, fn, samples=SAMPLES, min_sample_s=MIN_SAMPLE_S, graph=None, sync=None):
        """Returns (stats dict with ms per step, graph).  `sync` runs before every sample (rank barrier)."""
        g = graph if graph is not None else self.capture(fn)
        t1 = self._once(fn, g, 1)
        reps = max(1, min(2000, int(math.ceil(min_sample_s / max(t1 * self.steps * 1e-3, 1e-6)))))
        vals = []
        for _ in range(samples):
            if sync:
                sync()
            vals.append(self._once(fn, g, reps))
        vals.sort()
        return {"median_ms": statistics.median(vals), "min_ms": vals[0], "max_ms": vals[-1], "samples": samples,
                "replays_per_sample": reps, "steps_per_replay": self.steps}, g


def roofline_times(wl, es, pk, sms):
    flops = 2.0 * wl.K * wl.K * wl.C_a * wl.pixels                    # merged 169-tap form, Eq. 5
    alg_bytes = 2.0 * wl.C * es * wl.pixels                            # every byte read once, written once
    peak_tflops = sms * FMA_LANES_PER_SM * 2 * pk["sm_max_mhz"] * 1e6 / 1e12
    return flops, alg_bytes, peak_tflops, flops / (peak_tflops * 1e12), alg_bytes / (pk["hbm_gbs"] * 1e9)


def measure_config(pkg, torch, np, synth, wl, layout_name, steps, pk, sms, fp32_meas, launch, seed, full=False, sync=None, dense=False):
    """Whole step and stencil stage alone for one workload in one layout; returns (record, context)."""
    layout = synth.NHWC if layout_name == "nhwc" else synth.NCHW
    lay_code = pkg.ESC_NHWC if layout == synth.NHWC else pkg.ESC_NCHW
    tdt = torch.bfloat16 if wl.dtype == synth.BF16 else torch.float32
    es = 2 if wl.dtype == synth.BF16 else 4
    d = synth.make_inputs(wl.B, wl.C, wl.C_a, wl.H, wl.W, wl.K, wl.dtype, seed, wl.per_image_scale)
    x_host = torch.from_numpy(synth.to_layout(d["x"], layout)).to(tdt).pin_memory()
    w_host = [torch.from_numpy(d[k]).to(tdt) for k in ("w_large", "w_dyn", "b_dyn")]
    wl_d, wd_d, bd_d = (t.cuda() for t in w_host)
    tensor_bytes = x_host.numel() * es
    # rotate through enough (x, out) pairs that consecutive steps never find their data in L2
    n_rot = max(2, int(np.ceil(2.5 * L2_BYTES / (2 * tensor_bytes))))
    xs = [x_host.cuda() for _ in range(n_rot)]
    outs = [torch.empty_like(xs[0]) for _ in range(n_rot)]
    ws = pkg.new_workspace(wl.B, wl.C_a, wl.H, wl.W, wl.K)
    dk = torch.empty(wl.B, wl.C_a, 3, 3, device="cuda")

    if dense:                                   # the dense large kernel of Section 3.2 in place of the depth-wise one
        wdn_d = torch.from_numpy(synth.make_dense_kernel(wl.C_a, wl.K, wl.dtype, seed)).to(tdt).cuda()

        def step(i):
            pkg.esc_convattn_forward_dense(xs[i % n_rot], wl.C_a, wl.K, wdn_d, wd_d, bd_d, outs[i % n_rot], lay_code, ws)

        def stencil(i):
            pkg.esc_convattn_stencil_dense(xs[i % n_rot], wl.C_a, wl.K, wdn_d, dk, outs[i % n_rot], lay_code, ws)
    else:
        def step(i):
            pkg.esc_convattn_forward_ex(xs[i % n_rot], wl.C_a, wl.K, wl_d, wd_d, bd_d, outs[i % n_rot], lay_code, ws)

        def stencil(i):
            pkg.esc_convattn_stencil(xs[i % n_rot], wl.C_a, wl.K, wl_d, dk, outs[i % n_rot], lay_code, ws)

    for i in range(3):
        step(i)
    launches_per_step = pkg.esc_convattn_last_launches()
    path = pkg.esc_convattn_last_path()
    tile_w = pkg.esc_convattn_last_tile_width()
    pkg.esc_convattn_dynkernel(xs[0], wl.C_a, wd_d, bd_d, dk, lay_code, ws)
    for i in range(3):
        stencil(i)
    stencil_launches = pkg.esc_convattn_last_launches()
    torch.cuda.synchronize()

    timer = GraphTimer(torch, steps, launch)
    st_step, g_step = timer.measure(step, sync=sync)
    st_kernel, _ = timer.measure(stencil)
    assert pkg.esc_convattn_device_status(ws) == 0, "device-side wait timed out"

    flops, alg_bytes, peak_tflops, t_alu, t_hbm = roofline_times(wl, es, pk, sms)
    if dense:                                   # a real contraction: 16 x the multiply-adds, on the tensor cores
        flops = flops * wl.C_a
        peak_tflops = pk["bf16_tflops"]
        t_alu = flops / (peak_tflops * 1e12)
    bound = ("tensor" if dense else "alu") if t_alu >= t_hbm else "hbm"
    t_roof = max(t_alu, t_hbm)
    ms_step, ms_kernel = st_step["median_ms"], st_kernel["median_ms"]
    rec = {
        "workload": wl.name, "layout": layout_name, "storage": wl.dtype,
        "stencil_path": PATH_NAMES.get(path, str(path)), "tile_width": tile_w, "launches_per_step": launches_per_step,
        "step_us": ms_step * 1e3, "step_us_min": st_step["min_ms"] * 1e3, "step_us_max": st_step["max_ms"] * 1e3,
        "stencil_us": ms_kernel * 1e3, "stencil_us_min": st_kernel["min_ms"] * 1e3, "stencil_us_max": st_kernel["max_ms"] * 1e3,
        "samples": st_step["samples"], "replays_per_sample": st_step["replays_per_sample"],
        "Mpixel_per_s": wl.pixels / (ms_step * 1e-3) / 1e6,
        "algorithmic_GBps": alg_bytes / (ms_step * 1e-3) / 1e9,
        "TFMA_per_s": flops / 2 / (ms_step * 1e-3) / 1e12,
        "bound": bound, "t_roofline_us": t_roof * 1e6,
        "frac_step": t_roof / (ms_step * 1e-3), "frac_stencil": t_roof / (ms_kernel * 1e-3),
    }
    if bound == "alu" and fp32_meas and fp32_meas.get("packed_tflops"):
        t_meas = flops / (max(fp32_meas["packed_tflops"], fp32_meas["scalar_tflops"]) * 1e12)
        rec["frac_step_of_measured_fp32_peak"] = max(t_meas, t_hbm) / (ms_step * 1e-3)
    ctx = dict(d=d, x_host=x_host, w_host=w_host, wl_d=wl_d, wd_d=wd_d, bd_d=bd_d, xs=xs, outs=outs, ws=ws, dk=dk,
               n_rot=n_rot, lay_code=lay_code, tdt=tdt, es=es, tensor_bytes=tensor_bytes, timer=timer, step=step,
               stencil=stencil, g_step=g_step, launches_per_step=launches_per_step, stencil_launches=stencil_launches,
               path=path, st_step=st_step, st_kernel=st_kernel, flops=flops, alg_bytes=alg_bytes,
               peak_tflops=peak_tflops, t_alu=t_alu, t_hbm=t_hbm)
    return rec, ctx


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--layout", default="nhwc", choices=["nhwc", "nchw"])
    ap.add_argument("--large-kernel", default="depthwise", choices=["depthwise", "dense"],
                    help="depthwise: the headline path; dense: the 13x13x16x16 kernel of the paper's main models as the timed step")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--headline-only", action="store_true",
                    help="skip the per-workload table, the variants and the end-to-end leg (short runs under a profiler)")
    ap.add_argument("--launch", default="graph", choices=["graph", "eager"],
                    help="timed region: CUDA graphs holding the K steps (default) or K eager calls")
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
    pk = peaks()
    sms = torch.cuda.get_device_properties(local).multi_processor_count

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    fp32_meas = measure_fp32_peak() if rank == 0 else None

    # ---- headline: whole forward on the named workload; clocks sampled over its timed region ---------
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    # warm-up steps beyond those measure_config runs itself
    sampler.mark()
    rec, c = measure_config(pkg, torch, np, synth, wl, args.layout, args.steps, pk, sms, fp32_meas, args.launch,
                            rank_seed(wl, rank), sync=barrier, dense=args.large_kernel == "dense")
    sampler.mark_end()
    clocks = sampler.stop() if rank == 0 else None
    for i in range(max(0, W_ - 3)):
        c["step"](i)
    barrier()
    ms_step = max_over_ranks(c["st_step"]["median_ms"], world, "cuda")
    value = whole_job_value(wl.pixels, world, ms_step)
    ms_kernel = c["st_kernel"]["median_ms"]
    timer = c["timer"]
    launches_per_step, stencil_launches = c["launches_per_step"], c["stencil_launches"]
    xs, outs, ws, dk, n_rot, lay_code, tdt, es = (c[k] for k in ("xs", "outs", "ws", "dk", "n_rot", "lay_code", "tdt", "es"))
    wl_d, wd_d, bd_d, tensor_bytes = c["wl_d"], c["wd_d"], c["bd_d"], c["tensor_bytes"]

    flops, alg_bytes, peak_tflops, t_alu, t_hbm = (c[k] for k in ("flops", "alg_bytes", "peak_tflops", "t_alu", "t_hbm"))
    kernel_file = KERNEL_FILES.get(c["path"], "stencil_tma.cuh")
    if args.large_kernel == "dense":
        ach = flops / (ms_step * 1e-3) / 1e12
        roof = {"bound": "tensor", "achieved": ach, "peak": peak_tflops, "unit": "TFLOP/s", "frac": ach / peak_tflops,
                "peak_source": f"{pk['source']} bf16 GEMM throughput (burst)"}
    elif t_alu >= t_hbm:
        ach = flops / (ms_step * 1e-3) / 1e12
        roof = {"bound": "alu", "achieved": ach, "peak": peak_tflops, "unit": "TFLOP/s", "frac": ach / peak_tflops,
                "peak_source": f"fp32 FMA pipe: {sms} SMs x {FMA_LANES_PER_SM} lanes x 2 flop x {pk['sm_max_mhz']:.0f} MHz "
                               f"({pk['source']} max SM clock)"}
        if fp32_meas and fp32_meas.get("packed_tflops"):
            pm = max(fp32_meas["packed_tflops"], fp32_meas["scalar_tflops"])
            roof["peak_measured_this_run"] = pm
            roof["frac_of_measured_peak"] = ach / pm
            roof["stencil_stage_frac_of_measured_peak"] = flops / (ms_kernel * 1e-3) / 1e12 / pm
    else:
        ach = alg_bytes / (ms_step * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": ach / pk["hbm_gbs"],
                "peak_source": f"{pk['source']} copy bandwidth"}
    roof["traffic"] = ncu_traffic(kernel_file, wl.name, args.layout)
    if c["path"] == 4:
        # the depth-wise stage runs on the tensor cores as banded-Toeplitz products: the fraction above is still
        # the one of the FP32 roofline of the method's 169 multiply-adds per output (the contract's bound); beside
        # it, what the tensor pipe was asked to do
        issued = flops / TOEPLITZ_DENSITY
        roof["engine"] = "tensor cores: mma.sync m16n8k16 bf16 x bf16 -> fp32, 13 of 32 issued multiply-adds useful"
        roof["tensor_side"] = {"issued_TFLOPs_whole_step": issued / (ms_step * 1e-3) / 1e12,
                               "issued_TFLOPs_stencil_stage": issued / (ms_kernel * 1e-3) / 1e12,
                               "bf16_peak_TFLOPs": pk["bf16_tflops"],
                               "stencil_stage_of_bf16_peak": issued / (ms_kernel * 1e-3) / 1e12 / pk["bf16_tflops"]}
    roof.update({"frac_is": "whole step (all kernels of the forward), median", "kernel": "stencil (stage 2)",
                 "kernel_ms": ms_kernel, "stencil_stage_frac": max(t_alu, t_hbm) / (ms_kernel * 1e-3),
                 "whole_step_frac": max(t_alu, t_hbm) / (ms_step * 1e-3),
                 "fp32_peak_probe": fp32_meas,
                 "hbm_side": {"algorithmic_GBps": alg_bytes / (ms_step * 1e-3) / 1e9,
                              "of_peak": alg_bytes / (ms_step * 1e-3) / 1e9 / pk["hbm_gbs"]}})

    extras = {}
    per_workload = None
    e2e = None
    if args.large_kernel == "dense":
        args.headline_only = True               # the extras below describe the depth-wise path
    if not args.headline_only:
        st_gap, _ = timer.measure(lambda i: pkg.esc_convattn_dynkernel(xs[i % n_rot], wl.C_a, wd_d, bd_d, dk, lay_code, ws), samples=5)
        roof["gap_kernel_ms"] = st_gap["median_ms"]
        # the same stencil stage with its input resident in L2 (one buffer, no rotation): the case inside a network,
        # where the previous layer has just written x; reported beside the cold figure, never instead of it
        if 2 * c["tensor_bytes"] < L2_BYTES:
            st_hot, _ = timer.measure(lambda i: pkg.esc_convattn_stencil(xs[0], wl.C_a, wl.K, wl_d, dk, outs[0], lay_code, ws), samples=5)
            roof["kernel_ms_input_resident_in_l2"] = st_hot["median_ms"]
        # the same workload with the depth-wise stage pinned to the FP32 pipe (the register-tiled TMA kernel)
        if c["path"] == 4:
            pkg.esc_convattn_set_stencil_engine(pkg.ESC_ENGINE_FP32)
            try:
                st_f, _ = timer.measure(c["step"], samples=5)
                st_fk, _ = timer.measure(c["stencil"], samples=5)
            finally:
                pkg.esc_convattn_set_stencil_engine(pkg.ESC_ENGINE_AUTO)
            extras["fp32_engine"] = {"ms_per_step": st_f["median_ms"], "stencil_ms": st_fk["median_ms"],
                                     "whole_step_frac": max(t_alu, t_hbm) / (st_f["median_ms"] * 1e-3)}
            pkg.esc_convattn_set_fused_stage1(False)
            try:
                st_2, _ = timer.measure(c["step"], samples=5)
            finally:
                pkg.esc_convattn_set_fused_stage1(True)
            extras["two_launch_forward_ms_per_step"] = st_2["median_ms"]
        # the whole step with the paper's two-layer estimator (hidden width 8, exact GELU)
        mlp_d = [torch.from_numpy(v).to(tdt).cuda() for v in synth.make_estimator_mlp(wl.C_a, 8, wl.dtype, wl.seed).values()]
        st, _ = timer.measure(lambda i: pkg.esc_convattn_forward_mlp(xs[i % n_rot], wl.C_a, wl.K, wl_d, *mlp_d, outs[i % n_rot], lay_code, ws), samples=5)
        extras["ms_per_step_two_layer_estimator_h8"] = st["median_ms"]
        # with the decomposed large kernel of Eq. 5 (point-wise LK^c in front of the depth-wise stage)
        wp_d = torch.from_numpy(synth.make_pointwise(wl.C_a, wl.dtype, wl.seed)).to(tdt).cuda()
        st, _ = timer.measure(lambda i: pkg.esc_convattn_forward_pw(xs[i % n_rot], wl.C_a, wl.K, wl_d, wp_d, wd_d, bd_d, outs[i % n_rot], lay_code, ws), samples=5)
        extras["ms_per_step_decomposed_large_kernel"] = st["median_ms"]
        # the module with its closing 1x1 convolution and residual (Eq. 4 line 4, Eq. 3 line 3): one fused call against
        # the forward followed by a library 1x1 convolution and an add
        try:
            fz = synth.make_fuse(wl.C, wl.dtype, wl.seed)
            wf_d = torch.from_numpy(fz["w_fuse"]).to(tdt).cuda()
            bf_d = torch.from_numpy(fz["b_fuse"]).to(tdt).cuda()
            res_d = torch.randn_like(xs[0])
            st, _ = timer.measure(lambda i: pkg.esc_convattn_forward_fused(xs[i % n_rot], wl.C_a, wl.K, wl_d, wd_d, bd_d, wf_d, bf_d, res_d,
                                                                           outs[i % n_rot], lay_code, ws), samples=5)
            fused_ms, fused_launches = st["median_ms"], pkg.esc_convattn_last_launches()
            sep_ms = None
            if lay_code == pkg.ESC_NHWC:
                w4 = wf_d.view(wl.C, wl.C, 1, 1).contiguous(memory_format=torch.channels_last)
                views = [o.permute(0, 3, 1, 2) for o in outs]            # NHWC storage seen as [B,C,H,W] channels_last
                res_v = res_d.permute(0, 3, 1, 2)

                def separate(i):
                    pkg.esc_convattn_forward_ex(xs[i % n_rot], wl.C_a, wl.K, wl_d, wd_d, bd_d, outs[i % n_rot], lay_code, ws)
                    y = torch.nn.functional.conv2d(views[i % n_rot], w4, bf_d)
                    y.add_(res_v)

                with torch.cuda.stream(timer.side):
                    for i in range(3):
                        separate(i)
                torch.cuda.synchronize()
                st, _ = timer.measure(separate, samples=5)
                sep_ms = st["median_ms"]
            extras["module_with_conv_fuse"] = {
                "fused_call_ms": fused_ms, "fused_call_launches": fused_launches,
                "forward_then_library_conv1x1_and_add_ms": sep_ms,
                "algorithmic_bytes_per_pixel": {"fused_call": (wl.C_a * 2 + wl.C + wl.C + wl.C) * es,
                                                "separate": (2 * wl.C + 2 * wl.C + 3 * wl.C) * es},
                "note": "fused: stencil reads and writes the attention channels, the 1x1 kernel reads x's identity channels, the residual, "
                        "and writes out; separate: forward (read x, write cat), conv (read cat, write y), add (read y, residual, write y)"}
        except Exception as exc:                                          # never lose the headline over an extra
            extras["module_with_conv_fuse"] = {"error": f"{type(exc).__name__}: {exc}"}
        # the backward pass of the same module (gradients of x, LK, W_dyn, b_dyn): tap gradients and the stencil on
        # grad_out, 2 x K x K multiply-adds per attention pixel-channel
        try:
            go_d = torch.randn_like(xs[0])
            gx_d = torch.empty_like(xs[0])
            g_lk = torch.zeros(wl.C_a, wl.K, wl.K, device="cuda")
            g_w = torch.zeros(9 * wl.C_a, wl.C_a, device="cuda")
            g_b = torch.zeros(9 * wl.C_a, device="cuda")
            bws = pkg.new_backward_workspace(wl.B, wl.C_a, wl.H, wl.W, wl.K)
            st, _ = timer.measure(lambda i: pkg.esc_convattn_backward(xs[i % n_rot], go_d, wl.C_a, wl.K, wl_d, wd_d, bd_d, gx_d, g_lk, g_w, g_b,
                                                                      lay_code, bws), samples=5)
            t_fma = 2.0 * 2.0 * wl.K * wl.K * wl.C_a * wl.pixels / (sms * FMA_LANES_PER_SM * 2 * pk["sm_max_mhz"] * 1e6)
            extras["backward"] = {"ms_per_step": st["median_ms"], "launches": pkg.esc_convattn_last_launches(),
                                  "frac_of_fp32_roofline": t_fma / (st["median_ms"] * 1e-3),
                                  "note": "roofline: 2 x K x K multiply-adds per attention pixel-channel on the FP32 pipe"}
            if wl.C_a in (4, 8, 16, 32):
                # the same for the decomposed form of Eq. 5 (also the gradient of LK^c): two per-pixel kernels around it
                g_wp = torch.zeros(wl.C_a, wl.C_a, device="cuda")
                st, _ = timer.measure(lambda i: pkg.esc_convattn_backward_pw(xs[i % n_rot], go_d, wl.C_a, wl.K, wl_d, wp_d, wd_d, bd_d, gx_d, g_lk,
                                                                             g_wp, g_w, g_b, lay_code, bws), samples=5)
                extras["backward"]["decomposed_large_kernel_ms_per_step"] = st["median_ms"]
                extras["backward"]["decomposed_large_kernel_launches"] = pkg.esc_convattn_last_launches()
            if wl.C_a == 16:
                # the same with the dense large kernel (Section 3.2): 2 x 16 x 16 x K x K multiply-adds per pixel for the
                # kernel's gradient on the FP32 pipe, grad_x on the forward's tensor-core kernel
                wdn_b = torch.from_numpy(synth.make_dense_kernel(wl.C_a, wl.K, wl.dtype, wl.seed)).to(tdt).cuda()
                g_wdn = torch.zeros(wl.C_a, wl.C_a, wl.K, wl.K, device="cuda")
                dws = pkg.new_backward_dense_workspace(wl.B, wl.C_a, wl.H, wl.W, wl.K)
                st, _ = timer.measure(lambda i: pkg.esc_convattn_backward_dense(xs[i % n_rot], go_d, wl.C_a, wl.K, wdn_b, wd_d, bd_d, gx_d, g_wdn,
                                                                                g_w, g_b, lay_code, dws), samples=5)
                t_fma_d = 2.0 * wl.C_a * wl.C_a * wl.K * wl.K * wl.pixels / (sms * FMA_LANES_PER_SM * 2 * pk["sm_max_mhz"] * 1e6)
                extras["backward"]["dense_large_kernel_ms_per_step"] = st["median_ms"]
                extras["backward"]["dense_large_kernel_launches"] = pkg.esc_convattn_last_launches()
                extras["backward"]["dense_large_kernel_frac_of_fp32_roofline_of_its_weight_gradient"] = t_fma_d / (st["median_ms"] * 1e-3)
            if wl.C in (16, 32, 48, 64):
                # the closing 1x1 convolution's backward (grad_cat, grad W_fuse, grad b_fuse): 2 x 2 x C x C flops per pixel
                wfb = torch.from_numpy(synth.make_fuse(wl.C, wl.dtype, wl.seed)["w_fuse"]).to(tdt).cuda()
                g_wf = torch.zeros(wl.C, wl.C, device="cuda")
                g_bf = torch.zeros(wl.C, device="cuda")
                fws = torch.empty(pkg.esc_conv_fuse_backward_workspace_bytes(wl.B, wl.C, wl.H, wl.W), dtype=torch.uint8, device="cuda")
                st, _ = timer.measure(lambda i: pkg.esc_conv_fuse_backward(xs[i % n_rot], go_d, wfb, gx_d, g_wf, g_bf, lay_code, fws), samples=5)
                extras["backward"]["conv_fuse_ms_per_step"] = st["median_ms"]
                extras["backward"]["conv_fuse_launches"] = pkg.esc_convattn_last_launches()
        except Exception as exc:
            extras["backward"] = {"error": f"{type(exc).__name__}: {exc}"}
        # with the dense large kernel of the main model (Section 3.2): an implicit GEMM on the tensor cores
        if wl.C_a == 16 and wl.K == 13:
            wdn_d = torch.from_numpy(synth.make_dense_kernel(wl.C_a, wl.K, wl.dtype, wl.seed)).to(tdt).cuda()
            st, _ = timer.measure(lambda i: pkg.esc_convattn_forward_dense(xs[i % n_rot], wl.C_a, wl.K, wdn_d, wd_d, bd_d, outs[i % n_rot], lay_code, ws), samples=5)
            fl = 2.0 * wl.C_a * wl.C_a * wl.K * wl.K * wl.pixels
            ms_dense = st["median_ms"]
            extras["dense_large_kernel"] = {
                "ms_per_step": ms_dense, "bound": "tensor", "achieved": fl / (ms_dense * 1e-3) / 1e12, "peak": pk["bf16_tflops"],
                "unit": "TFLOP/s", "frac": fl / (ms_dense * 1e-3) / 1e12 / pk["bf16_tflops"],
                "path": PATH_NAMES.get(pkg.esc_convattn_last_path(), str(pkg.esc_convattn_last_path())),
                "note": "whole step (GAP kernel + dense stencil kernel with copy-through)"}

        # ---- end to end through the host-buffer entries (copies inside the timed region) ------------
        # Every step uploads x and the weights from pinned host memory and downloads the whole result.  The
        # two-slot submit / wait pair lets the upload of step i overlap the download of step i - 1 (PCIe is
        # full duplex); the blocking single call is timed too.
        x_host, w_host = c["x_host"], c["w_host"]
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
        e2e = {"value": whole_job_value(wl.pixels, world, dt / n_e2e * 1e3), "unit": UNIT,
               "h2d_bytes_per_step": c["tensor_bytes"] + w_bytes, "d2h_bytes_per_step": c["tensor_bytes"], "steps": n_e2e,
               "api": "esc_convattn_forward_host_submit / _wait, two slots in turn (pinned host buffers)",
               "blocking_call_value": whole_job_value(wl.pixels, world, dt_block / n_e2e * 1e3)}

    # ---- every evaluation workload, one GPU: whole step and stencil stage, medians --------------------
    cpu = None
    oracle_one_thread = None
    if rank == 0 and world == 1 and not args.headline_only:
        del xs, outs, c
        torch.cuda.empty_cache()
        per_workload = []
        plan = [("cfg1_64x64_f32", "nchw"), ("cfg2_320x180_f32", "nchw"), ("cfg3_640x360_bf16", "nhwc"),
                ("cfg3_640x360_bf16", "nchw"), ("cfg4_b64_64x64_bf16", "nhwc"), ("cfg4_b64_64x64_bf16", "nchw"),
                ("cfg5_1920x1080_ca32_bf16", "nhwc"), ("cfg5_1920x1080_ca32_bf16", "nchw")]
        for name, lay in plan:
            if name == wl.name and lay == args.layout:
                per_workload.append(rec)
                continue
            w2 = synth.WORKLOADS_BY_NAME[name]
            k2 = max(10, min(args.steps, int(0.05 / 30e-6)))          # enough steps per graph that a replay is not launch-bound
            r2, c2 = measure_config(pkg, torch, np, synth, w2, lay, k2, pk, sms, fp32_meas, args.launch, w2.seed)
            per_workload.append(r2)
            del c2
            torch.cuda.empty_cache()
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = time_oracle(wl)
        if not args.headline_only:
            oracle_one_thread = {}
            for name in ("cfg1_64x64_f32", "cfg2_320x180_f32", "cfg3_640x360_bf16"):
                r = time_oracle(synth.WORKLOADS_BY_NAME[name], budget_s=3.0, threads=1)
                oracle_one_thread[name] = {"Mpixel_per_s": r["value"], "sample": r["sample"]}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": W_,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl.name, "B": wl.B, "C": wl.C, "C_a": wl.C_a, "H": wl.H, "W": wl.W, "K": wl.K,
                       "storage": wl.dtype, "layout": args.layout, "sharding": "replicas: one image batch per GPU, no collective",
                       "l2": f"inputs larger than L2: {n_rot} rotating (x,out) pairs, {n_rot * 2 * tensor_bytes / 1e6:.0f} MB",
                       "stencil_path": rec["stencil_path"],
                       "launch": timer.mode, "estimator": "one linear layer",
                       "large_kernel": "dense 13x13x16x16 (Section 3.2)" if args.large_kernel == "dense" else "depth-wise LK^s"},
            "timing": {"ms_per_step_is": "median over samples", "samples": rec["samples"],
                       "replays_per_sample": rec["replays_per_sample"], "steps_per_replay": args.steps,
                       "min_ms": rec["step_us_min"] / 1e3, "max_ms": rec["step_us_max"] / 1e3,
                       "spread": (rec["step_us_max"] - rec["step_us_min"]) / rec["step_us"]},
            "roofline": roof, "cpu_baseline": cpu, "cpu_baseline_one_thread": oracle_one_thread, "e2e": e2e, "clocks": clocks,
            "gpu_launches": rec["samples"] * rec["replays_per_sample"] * args.steps * launches_per_step,
            "launches_per_step": launches_per_step, "stencil_stage_launches": stencil_launches,
            "GB_per_s_whole_step": alg_bytes / (ms_step * 1e-3) / 1e9,
            "per_workload": per_workload,
        }
        line.update(extras)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
