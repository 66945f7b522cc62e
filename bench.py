#!/usr/bin/env python
"""Benchmark of the block-sparse hot path: Gamma build -> compaction -> block-sparse conv with bias.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One step is one pass of the whole path over one batch of synthetic input: bsp_mask (block L2 scores and
selection to 50 % block sparsity), bsp_compact (block-CSR + packed tiles) and bsp_conv2d (implicit-GEMM
convolution with fused bias).  The default workload is the ResNet50-style 3x3 convolution (batch 32, 14x14,
256 -> 256 channels, bf16, 8x8 blocks at 50 %).  The metric is effective TFLOP/s counting only the FLOPs of
non-zero blocks.  Prints one JSON line (rank 0).

With --gpus N > 1 (launched under torch.distributed.run) every rank runs the same workload on its own batch
(no exchange on the path: output pixels are independent), the time is the maximum over ranks and the value
the sum of the work.  --impl reference times the CPU oracle on the host cores instead.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2407_09453_b200 import synth  # noqa: E402

METRIC = "effective TFLOP/s (non-zero blocks only)"
UNIT = "TFLOP/s"


def workload(name: str):
    """(layer, dtype, block shape, sparsity) of a named workload."""
    if name == "resnet50_conv3x3_256_b32":
        return synth.Layer(name, 256, 256, 3, 3, 32, 14, 14, 1, 1, 1, 1), "bf16", (8, 8), 0.5, 2
    if name == "gemm_4096_p8192":
        return synth.fc(name, 4096, 4096, 8192), "bf16", (8, 8), 0.5, 3
    if name == "vgg_conv3x3_256_56_i8":
        return synth.Layer(name, 256, 256, 3, 3, 32, 56, 56, 1, 1, 1, 1), "i8", (8, 8), 0.5, 5
    raise SystemExit(f"unknown workload {name}")


def useful_flops(layer, nnz, bo, bi):
    return 2.0 * layer.P * nnz * bo * bi * layer.H * layer.K


def algorithmic_bytes(layer, nnz, bo, bi, ex, ey):
    """Bytes the conv kernel must move: X once, Y once, the stored blocks, their indices, the bias."""
    NBo = layer.O // bo
    return (layer.N * layer.L * layer.J * layer.I * ex + layer.P * layer.O * ey
            + nnz * bo * bi * layer.H * layer.K * ex + 4 * (nnz + NBo + 1) + 4 * layer.O)


def measured_traffic(workload: str, kernel: str):
    """DRAM bytes per launch of the dominant kernel (conv_mma_kernel or conv_tc_kernel) from the committed ncu
    summary, or None when the kernel source has changed since the counters were taken (or no capture exists
    for this workload)."""
    import hashlib
    stem = kernel[:-len("_kernel")]
    path = os.path.join(ROOT, "profiles", f"traffic_{stem}_{workload}.json")
    src = os.path.join(ROOT, "paper_2407_09453_b200", "csrc", f"bsp_{stem}.cu")
    if not (os.path.exists(path) and os.path.exists(src)):
        return None
    d = json.load(open(path))
    if d.get("kernel_source_sha256") != hashlib.sha256(open(src, "rb").read()).hexdigest():
        return None
    return d.get("dram_bytes_per_launch")


def reduce_max(values, world: int, device):
    """Per-rank timings -> their maximum over all ranks (the job's time); identity for one rank."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(v) for v in values], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def job_tflops(flops_per_rank: float, world: int, ms: float) -> float:
    """Whole-job throughput: every rank does flops_per_rank of useful work in the job's ms (weak scaling)."""
    return world * flops_per_rank / (ms * 1e-3) / 1e12


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm = [float(r[0]) for r in self.rows if len(r) >= 6 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 6 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({n for r in self.rows if len(r) >= 6 for n, v in zip(names, r[2:6]) if v == "Active"})
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def time_oracle(layer, dtype, bo, bi, n_zero, W, X, b, min_seconds, max_reps):
    """The oracle as it stands on the host cores: scores -> Gamma -> compaction -> sparse conv (all pixels)."""
    from oracle import ref
    cores = ref.set_threads(0)
    times = []
    t_all = time.perf_counter()
    while len(times) < max_reps and (len(times) < 1 or time.perf_counter() - t_all < min_seconds):
        t0 = time.perf_counter()
        g = ref.mask(ref.scores(W, bo, bi), n_zero)
        rp, ci, pl = ref.compact(W, g, bo, bi)
        ref.conv2d(W.shape, bo, bi, rp, ci, pl, X, b, (layer.stride_h, layer.stride_w), (layer.pad_h, layer.pad_w))
        times.append(time.perf_counter() - t0)
    return float(np.mean(times)), cores, len(times)


def run_reference(args, layer, dtype, bo, bi, sparsity, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    W, X, b = synth.make_layer_tensors(layer, dtype, config=cfg)
    NB = (layer.O // bo) * (layer.I // bi)
    n_zero = int(sparsity * NB + 0.5)
    nnz = NB - n_zero
    for _ in range(min(args.warmup, 1)):
        time_oracle(layer, dtype, bo, bi, n_zero, W, X, b, 0, 1)
    t, cores, reps = time_oracle(layer, dtype, bo, bi, n_zero, W, X, b, float("inf"), max(args.steps, 1))   # exactly K passes
    val = useful_flops(layer, nnz, bo, bi) / t / 1e12
    sample = f"all {layer.P} output pixels of the workload, {reps} passes"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": reps,
        "warmup": min(args.warmup, 1), "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64" if dtype != "i8" else "int64", "data": "synthetic",
        "config": {"workload": layer.name, "block": f"{bo}x{bi}", "sparsity": sparsity, "timing": "host wall clock"},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet50_conv3x3_256_b32")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch the three calls of a step one by one instead of replaying a CUDA graph of them")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    layer, dtype, (bo, bi), sparsity, cfg = workload(args.workload)
    if args.impl == "reference":
        return run_reference(args, layer, dtype, bo, bi, sparsity, cfg)

    import torch
    import torch.distributed as dist
    from paper_2407_09453_b200 import bsp, build
    build.build()

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    tdt = {"bf16": torch.bfloat16, "f32": torch.float32, "i8": torch.int8}[dtype]
    ydt = torch.int32 if dtype == "i8" else torch.float32
    ex, ey = (1 if dtype == "i8" else 2 if dtype == "bf16" else 4), 4
    # every rank draws its own batch (weak scaling); weights are the same on all ranks
    W, X, b = synth.make_layer_tensors(layer, dtype, config=cfg, layer_id=0)
    if rank > 0:
        X = synth.make_layer_tensors(layer, dtype, config=cfg, layer_id=rank)[1]
    NB = (layer.O // bo) * (layer.I // bi)
    n_zero = int(sparsity * NB + 0.5)
    nnz = NB - n_zero

    stream = torch.cuda.current_stream()
    Wd = torch.from_numpy(W).cuda().to(tdt)
    Xd = torch.from_numpy(X).cuda().to(tdt)
    bd = torch.from_numpy(b).cuda()
    Y = torch.empty((layer.N, layer.M, layer.Nw, layer.O), dtype=ydt, device="cuda")
    lay = bsp.SparseLayer(layer.O, layer.I, layer.H, layer.K, bo, bi, tdt)
    dense = bsp.SparseLayer(layer.O, layer.I, layer.H, layer.K, bo, bi, tdt, canonical=False)
    flush = torch.empty(384 << 20, dtype=torch.uint8, device="cuda")       # larger than the 126 MB L2
    stride, pad = (layer.stride_h, layer.stride_w), (layer.pad_h, layer.pad_w)

    def step(events=None):
        if events:
            events[0].record(stream)
        lay.mask(Wd, n_zero)
        if events:
            events[1].record(stream)
        lay.compact(Wd)
        if events:
            events[2].record(stream)
        lay.conv2d(Xd, bd, Y, stride, pad)
        if events:
            events[3].record(stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        flush.zero_()
        step()
    lay.check()

    # ---- one step (the three calls) as a CUDA graph, captured on a side stream through the same C ABI
    graph, how = None, "three calls per step, launched one by one"
    if not args.no_graph:
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                step()
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                step()
            torch.cuda.synchronize()
            graph.replay()
            lay.check()
            how = "CUDA graph of the three calls, one replay per step"
        except Exception as e:          # capture not available: time the plain calls
            graph, how = None, f"three calls per step, launched one by one (graph capture failed: {type(e).__name__})"
            torch.cuda.synchronize()

    # ---- device-timed steps, inputs resident in HBM, L2 flushed between steps
    ev_step = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
    sampler = ClockSampler(local)
    sampler.start()
    barrier()
    for k in range(args.steps):
        flush.zero_()
        ev_step[k][0].record(stream)
        if graph is not None:
            graph.replay()
        else:
            step()
        ev_step[k][1].record(stream)
    barrier()
    clocks = sampler.stop()
    lay.check()
    t_step = np.array([e[0].elapsed_time(e[1]) for e in ev_step])
    ms_step = float(t_step.mean())

    # ---- the phases of a step, each call bracketed by events (launched one by one; the events and launch gaps make
    # their sum larger than a graph replay of the step)
    n_ph = max(10, min(args.steps, 50))
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(n_ph)]
    for k in range(n_ph):
        flush.zero_()
        step(evs[k])
    torch.cuda.synchronize()
    t_mask = np.array([e[0].elapsed_time(e[1]) for e in evs])
    t_comp = np.array([e[1].elapsed_time(e[2]) for e in evs])
    t_conv = np.array([e[2].elapsed_time(e[3]) for e in evs])

    # ---- the same layer dense (Gamma == 1) through the same kernel, for the speedup
    ones = torch.ones(NB, dtype=torch.uint8, device="cuda")
    dense.compact(Wd, ones)
    dense.nnz = NB
    t_dense = []
    for k in range(max(args.steps // 2, 5) + 3):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        dense.conv2d(Xd, bd, Y, stride, pad)
        e1.record(stream)
        torch.cuda.synchronize()
        if k >= 3:
            t_dense.append(e0.elapsed_time(e1))
    dense.check()
    ms_dense = float(np.mean(t_dense))

    # ---- end to end: host buffers in pinned memory, copies inside the timed region
    Wh = torch.from_numpy(W).to(tdt).pin_memory()
    Xh = torch.from_numpy(X).to(tdt).pin_memory()
    bh = torch.from_numpy(b).pin_memory()
    Yh = torch.empty(Y.shape, dtype=ydt).pin_memory()
    h2d = Wh.numel() * Wh.element_size() + Xh.numel() * Xh.element_size() + bh.numel() * bh.element_size()
    d2h = Yh.numel() * Yh.element_size()

    def e2e_step():
        Wd.copy_(Wh, non_blocking=True)
        Xd.copy_(Xh, non_blocking=True)
        bd.copy_(bh, non_blocking=True)
        step()
        Yh.copy_(Y, non_blocking=True)

    for _ in range(3):
        e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        e2e_step()
    e1.record(stream)
    barrier()
    ms_e2e = e0.elapsed_time(e1) / args.steps
    lay.check()

    # max over ranks
    ms_step, ms_e2e, ms_conv = reduce_max([ms_step, ms_e2e, float(t_conv.mean())], world, "cuda")

    fl = useful_flops(layer, nnz, bo, bi)
    pk = peaks()
    value = job_tflops(fl, world, ms_step)
    conv_tflops = fl / (ms_conv * 1e-3) / 1e12
    abytes = algorithmic_bytes(layer, nnz, bo, bi, ex, ey)
    # the tensor peak of the path's own input type: the measured bf16 peak times the nominal ratio of the dense peaks
    # (int8 4.5 : bf16 2.25 : tf32 1.1 PFLOP/s)
    ratio = {"bf16": 1.0, "i8": 2.0, "f32": 1.1 / 2.25}[dtype]
    tensor_peak = pk["bf16_tflops"] * ratio
    t_tensor = fl / (tensor_peak * 1e12)
    t_hbm = abytes / (pk["hbm_gbs"] * 1e9)
    if t_tensor >= t_hbm:
        roof = {"bound": "tensor", "achieved": conv_tflops, "peak": tensor_peak, "unit": "TFLOP/s",
                "frac": conv_tflops / tensor_peak, "traffic": None}
    else:
        gbs = abytes / (ms_conv * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": gbs, "peak": pk["hbm_gbs"], "unit": "GB/s",
                "frac": gbs / pk["hbm_gbs"], "traffic": None}
    kernel = bsp.conv_kernel_name(lay.wd, bsp.XDesc(layer.N, layer.L, layer.J, stride[0], stride[1], pad[0], pad[1]))
    roof["traffic"] = measured_traffic(layer.name, kernel)
    roof.update({"kernel": kernel, "algorithmic_bytes": abytes, "peak_source": pk["source"] + " (burst)" + ("" if dtype == "bf16" else f" bf16 x {ratio:.3g} nominal ratio"),
                 "kernel_ms": ms_conv, "roofline_ms": max(t_tensor, t_hbm) * 1e3})

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": {"bf16": "bf16", "f32": "tf32", "i8": "int8"}[dtype], "data": "synthetic",
        "config": {"workload": layer.name, "block": f"{bo}x{bi}", "sparsity": sparsity, "nnz_blocks": nnz,
                   "step": "bsp_mask + bsp_compact + bsp_conv2d", "launch": how,
                   "l2": "flushed between steps (384 MB write)",
                   "per_gpu_batch": layer.N},
        "phases_ms": {"mask": float(t_mask.mean()), "compact": float(t_comp.mean()), "conv": ms_conv,
                      "note": "each call between its own events, launched one by one"},
        "conv_only": {"tflops": conv_tflops, "ms": ms_conv, "ms_min": float(t_conv.min()),
                      "dense_ms": ms_dense, "speedup_vs_dense": ms_dense / ms_conv},
        "roofline": roof,
        "e2e": {"value": job_tflops(fl, world, ms_e2e), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e},
        "gpu_launches": args.steps * bsp.launches_per_step(lay.wd),
        "clocks": clocks,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        t, cores, reps = time_oracle(layer, dtype, bo, bi, n_zero, W, X, b, 8.0, 40)
        out["cpu_baseline"] = {"value": fl / t / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
                               "sample": f"all {layer.P} output pixels of the workload, {reps} passes, "
                                         f"{t * 1e3:.1f} ms each"}
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
