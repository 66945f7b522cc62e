#!/usr/bin/env python
"""Benchmark of the block-sparse hot path: Gamma build -> compaction -> block-sparse product with bias.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME] [--no-sweeps]

One step is one pass of the whole path over one batch of synthetic input: bsp_mask (block L2 scores and
selection to the target block sparsity), bsp_compact (block-CSR + packed forms) and bsp_gemm / bsp_conv2d
(tensor-core product with fused bias).  The default workload is the largest single-GPU configuration, the
matrix product O = I = 4096 over P = 8192 positions (bf16, 8x8 blocks at 50 %).  The metric is effective
TFLOP/s counting only the FLOPs of non-zero blocks.  Rank 0 prints one JSON line; besides the headline it carries
the block-shape / sparsity sweep of that product, a per-layer pass over the ResNet50-shaped layers (batch 64) and
one over the VGG16 / InceptionV3-shaped int8 layers (batch 32; Gamma build and compaction timed too).

With --gpus N > 1 (launched under torch.distributed.run) every rank runs the same workload on its own batch
(no exchange on the path: output positions are independent), the time is the maximum over ranks and the value
the sum of the work.  --impl reference times the CPU oracle on the host cores instead, on a bounded sample of
the same workload.
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
DEFAULT_WORKLOAD = "gemm_4096_p8192"


def workload(name: str):
    """(layer, dtype, block shape, sparsity, config number, sigma of the weights or None for He init)."""
    if name == "gemm_4096_p8192":
        return synth.fc(name, 4096, 4096, 8192), "bf16", (8, 8), 0.5, 3, 1.0 / 64.0
    if name == "resnet50_conv3x3_256_b32":
        return synth.Layer(name, 256, 256, 3, 3, 32, 14, 14, 1, 1, 1, 1), "bf16", (8, 8), 0.5, 2, None
    if name == "vgg_conv3x3_256_56_i8":
        return synth.Layer(name, 256, 256, 3, 3, 32, 56, 56, 1, 1, 1, 1), "i8", (8, 8), 0.5, 5, None
    raise SystemExit(f"unknown workload {name}")


def useful_flops(layer, nnz, bo, bi):
    return 2.0 * layer.P * nnz * bo * bi * layer.H * layer.K


def algorithmic_bytes(layer, nnz, bo, bi, ex, ey):
    """Bytes the product must move: X once, Y once, the stored blocks, their indices, the bias."""
    NBo = layer.O // bo
    return (layer.N * layer.L * layer.J * layer.I * ex + layer.P * layer.O * ey
            + nnz * bo * bi * layer.H * layer.K * ex + 4 * (nnz + NBo + 1) + 4 * layer.O)


def measured_traffic(workload: str, kernel: str):
    """DRAM bytes per launch of the dominant kernel from the committed ncu summary, or None when the kernel source
    has changed since the counters were taken (or no capture exists for this workload)."""
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


# tensor peak of a path's own input type: the measured bf16 peak times the nominal ratio of the dense peaks
# (int8 4.5 : bf16 2.25 : tf32 1.1 PFLOP/s)
PEAK_RATIO = {"bf16": 1.0, "i8": 2.0, "f32": 1.1 / 2.25}
ELEM = {"bf16": 2, "i8": 1, "f32": 4}


def roofline_of(layer, nnz, bo, bi, dtype, ey, ms, pk):
    """Roofline record of one product call: the slower of useful FLOPs at the tensor peak and algorithmic bytes at
    the HBM bandwidth, against the measured time."""
    fl = useful_flops(layer, nnz, bo, bi)
    ab = algorithmic_bytes(layer, nnz, bo, bi, ELEM[dtype], ey)
    tensor_peak = pk["bf16_tflops"] * PEAK_RATIO[dtype]
    t_tensor, t_hbm = fl / (tensor_peak * 1e12), ab / (pk["hbm_gbs"] * 1e9)
    if t_tensor >= t_hbm:
        ach = fl / (ms * 1e-3) / 1e12
        r = {"bound": "tensor", "achieved": ach, "peak": tensor_peak, "unit": "TFLOP/s", "frac": ach / tensor_peak}
    else:
        ach = ab / (ms * 1e-3) / 1e9
        r = {"bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": ach / pk["hbm_gbs"]}
    r.update({"algorithmic_bytes": ab, "useful_flops": fl, "roofline_ms": max(t_tensor, t_hbm) * 1e3})
    return r


class ClockSampler:
    """Samples SM clocks, utilisation and throttle reasons with nvidia-smi while the timed regions run."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap,utilization.gpu")

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
        ok = [r for r in self.rows if len(r) >= 7 and r[0].replace(".", "").isdigit()]
        busy = [r for r in ok if r[6].isdigit() and int(r[6]) > 0] or ok
        sm = [float(r[0]) for r in busy]
        mx = [float(r[1]) for r in ok if r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({n for r in ok for n, v in zip(names, r[2:6]) if v == "Active"})
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(ok), "samples_under_load": len(busy)}


# ---------------------------------------------------------------------------------------------------------------
# CPU oracle on the host cores (the --impl reference arm, and the cpu_baseline record of the GPU arm)

def oracle_sample(layer):
    """Output positions the oracle evaluates: all of them up to 8192, else a fixed strided subset of 256 (matrix
    product) or 2048 (convolution) positions; every position costs the same, so the full pass is n / len times it."""
    P = layer.P
    if P <= 8192 and layer.O * layer.I * layer.H * layer.K <= (1 << 21):
        return None, P
    n = 256 if layer.H * layer.K == 1 else 2048
    pix = (np.arange(n, dtype=np.int64) * P) // n
    return pix, n


def time_oracle(layer, dtype, bo, bi, n_zero, W, X, b, reps):
    """`reps` passes of the oracle as it stands: scores -> Gamma -> compaction in full, then the block-sparse product
    on the sample positions.  Returns (seconds of a full step, extrapolated; seconds measured per pass; cores;
    description of the sample)."""
    from oracle import ref
    cores = ref.set_threads(0)
    pix, n = oracle_sample(layer)
    t_setup, t_prod = [], []
    for _ in range(reps):
        t0 = time.perf_counter()
        g = ref.mask(ref.scores(W, bo, bi), n_zero)
        rp, ci, pl = ref.compact(W, g, bo, bi)
        t1 = time.perf_counter()
        if layer.H * layer.K == 1 and layer.L == 1 and layer.J == 1:
            ref.gemm(layer.O, layer.I, bo, bi, rp, ci, pl.reshape(-1, bo, bi), X.reshape(layer.P, layer.I), b, pix=pix)
        else:
            ref.conv2d(W.shape, bo, bi, rp, ci, pl, X, b, (layer.stride_h, layer.stride_w), (layer.pad_h, layer.pad_w), pix=pix)
        t2 = time.perf_counter()
        t_setup.append(t1 - t0)
        t_prod.append(t2 - t1)
    ts, tp = float(np.mean(t_setup)), float(np.mean(t_prod))
    full = ts + tp * layer.P / n
    if n == layer.P:
        what = f"all {layer.P} output positions, {reps} passes, {(ts + tp) * 1e3:.1f} ms each"
    else:
        what = (f"Gamma build and compaction in full ({ts * 1e3:.0f} ms) + the product on {n} of {layer.P} output positions "
                f"(fixed stride, {tp * 1e3:.0f} ms), {reps} passes; the step time is extrapolated to all positions")
    return full, ts + tp, cores, what


def make_host_tensors(layer, dtype, cfg, sigma, layer_id=0):
    return synth.make_layer_tensors(layer, dtype, config=cfg, layer_id=layer_id, w_sigma=sigma)


def run_reference(args, layer, dtype, bo, bi, sparsity, cfg, sigma):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    W, X, b = make_host_tensors(layer, dtype, cfg, sigma)
    NB = (layer.O // bo) * (layer.I // bi)
    n_zero = int(sparsity * NB + 0.5)
    nnz = NB - n_zero
    for _ in range(min(args.warmup, 1)):
        time_oracle(layer, dtype, bo, bi, n_zero, W, X, b, 1)
    full, measured, cores, what = time_oracle(layer, dtype, bo, bi, n_zero, W, X, b, max(args.steps, 1))
    val = useful_flops(layer, nnz, bo, bi) / full / 1e12
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": max(args.steps, 1),
        "warmup": min(args.warmup, 1), "ms_per_step": full * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64" if dtype != "i8" else "int64", "data": "synthetic",
        "config": {"workload": layer.name, "block": f"{bo}x{bi}", "sparsity": sparsity,
                   "timing": "host wall clock; ms_per_step is the full step" + ("" if measured == full else " (extrapolated)"),
                   "measured_ms_per_pass": measured * 1e3},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": what},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def cpu_baseline_subprocess(name: str):
    """The oracle timed in a fresh process (no torch thread pools beside its OpenMP threads), the way the reference
    arm times it: three passes after one warm-up."""
    try:
        out = subprocess.run([sys.executable, os.path.abspath(__file__), "--impl", "reference", "--workload", name,
                              "--steps", "3", "--warmup", "1"], capture_output=True, text=True, timeout=600,
                             env={k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")})
        line = [ln for ln in out.stdout.splitlines() if ln.startswith("{")][-1]
        return json.loads(line)["cpu_baseline"]
    except Exception as e:          # the baseline is a reported figure, not part of the timed path
        return {"value": None, "unit": UNIT, "cores": 0, "kind": "oracle", "sample": f"failed: {type(e).__name__}"}


# ---------------------------------------------------------------------------------------------------------------
# GPU arm

class Gpu:
    """Event timing on the current stream with the L2 flushed (a 384 MB write, larger than the 126 MB L2) before
    every timed call."""

    def __init__(self, torch):
        self.torch = torch
        self.stream = torch.cuda.current_stream()
        self.flush = torch.empty(384 << 20, dtype=torch.uint8, device="cuda")

    def timed(self, fn, reps, warm=2):
        t = self.torch
        out = []
        for k in range(warm + reps):
            self.flush.zero_()
            e0, e1 = t.cuda.Event(enable_timing=True), t.cuda.Event(enable_timing=True)
            e0.record(self.stream)
            fn()
            e1.record(self.stream)
            t.cuda.synchronize()
            if k >= warm:
                out.append(e0.elapsed_time(e1))
        return out


def stats(ms):
    a = np.asarray(ms, dtype=np.float64)
    return {"ms": float(np.median(a)), "ms_min": float(a.min()), "ms_mean": float(a.mean())}


def device_layer(torch, bsp, layer, dtype, seed, sigma=None, ydt=None):
    """Seeded synthetic tensors of one layer drawn on the device (the sweep passes only time the calls): weights
    N(0, sigma^2) (He init by default) and activations N(0, 1) rounded to bf16, or int8 uniform in [-127, 127]."""
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    wshape, xshape = (layer.O, layer.H, layer.K, layer.I), (layer.N, layer.L, layer.J, layer.I)
    if dtype == "i8":
        W = torch.randint(-127, 128, wshape, device="cuda", dtype=torch.int8, generator=g)
        X = torch.randint(-127, 128, xshape, device="cuda", dtype=torch.int8, generator=g)
        b = torch.randint(-(1 << 15), (1 << 15) + 1, (layer.O,), device="cuda", dtype=torch.int32, generator=g)
        ydt = torch.int32
    else:
        tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
        sigma = float(np.sqrt(2.0 / (layer.H * layer.K * layer.I))) if sigma is None else sigma
        W = (torch.randn(wshape, device="cuda", generator=g) * sigma).to(tdt)
        X = torch.randn(xshape, device="cuda", generator=g).to(tdt)
        b = torch.randn((layer.O,), device="cuda", generator=g) * 0.1
        ydt = ydt or torch.float32
    Y = torch.empty((layer.N, layer.M, layer.Nw, layer.O), dtype=ydt, device="cuda")
    return W, X, b, Y


def sweep_product(gpu, bsp, torch, layer, dtype, Wd, Xd, bd, Y, pk, reps=10):
    """Block shapes x sparsities on one layer: the product call alone, Gamma from bsp_mask (Gamma = 1 at sparsity 0)."""
    tdt = {"bf16": torch.bfloat16, "f32": torch.float32, "i8": torch.int8}[dtype]
    stride, pad = (layer.stride_h, layer.stride_w), (layer.pad_h, layer.pad_w)
    rows = []
    for bo, bi in ((8, 8), (4, 16), (16, 4)):
        lay = bsp.SparseLayer(layer.O, layer.I, layer.H, layer.K, bo, bi, tdt, canonical=False)
        NB = lay.NBo * lay.NBi
        dense_ms = None
        for s in (0.0, 0.25, 0.5, 0.75):
            n_zero = int(s * NB + 0.5)
            lay.mask(Wd, n_zero)
            lay.compact(Wd)
            st = stats(gpu.timed(lambda: lay.conv2d(Xd, bd, Y, stride, pad), reps))
            lay.check()
            nnz = NB - n_zero
            if s == 0.0:
                dense_ms = st["ms"]
            r = roofline_of(layer, nnz, bo, bi, dtype, Y.element_size(), st["ms"], pk)
            rows.append({"block": f"{bo}x{bi}", "sparsity": s, **st,
                         "effective_tflops": r["useful_flops"] / (st["ms"] * 1e-3) / 1e12,
                         "roofline_bound": r["bound"], "roofline_frac": r["frac"],
                         "speedup_vs_dense": dense_ms / st["ms"],
                         "executed_flops": float(layer.dense_flops()), "useful_flops": r["useful_flops"],
                         "stored_weight_bytes": layer.O * layer.I * layer.H * layer.K * ELEM[dtype],
                         "algorithmic_weight_bytes": nnz * bo * bi * layer.H * layer.K * ELEM[dtype]})
        del lay
    return rows


def pass_layers(gpu, bsp, torch, layers, dtype, sparsities, pk, ydt, with_setup, reps=5):
    """Every layer of a table at 8x8 blocks: the product call (and, with_setup, bsp_mask and bsp_compact) timed one by
    one with the L2 flushed; per layer its own roofline bound and fraction."""
    tdt = {"bf16": torch.bfloat16, "f32": torch.float32, "i8": torch.int8}[dtype]
    out = []
    for li, layer in enumerate(layers):
        Wd, Xd, bd, Y = device_layer(torch, bsp, layer, dtype, 4000 + li, ydt=ydt)
        lay = bsp.SparseLayer(layer.O, layer.I, layer.H, layer.K, 8, 8, tdt, canonical=False)
        NB = lay.NBo * lay.NBi
        stride, pad = (layer.stride_h, layer.stride_w), (layer.pad_h, layer.pad_w)
        kernel = bsp.conv_kernel_name(lay.wd, bsp.XDesc(layer.N, layer.L, layer.J, stride[0], stride[1], pad[0], pad[1]))
        for s in sparsities:
            n_zero = int(s * NB + 0.5)
            rec = {"layer": layer.name, "count": layer.count, "sparsity": s, "kernel": kernel}
            if with_setup:
                rec["mask_ms"] = stats(gpu.timed(lambda: lay.mask(Wd, n_zero), 3, 1))["ms"]
                rec["compact_ms"] = stats(gpu.timed(lambda: lay.compact(Wd), 3, 1))["ms"]
            else:
                lay.mask(Wd, n_zero)
                lay.compact(Wd)
            st = stats(gpu.timed(lambda: lay.conv2d(Xd, bd, Y, stride, pad), reps, 1))
            lay.check()
            r = roofline_of(layer, NB - n_zero, 8, 8, dtype, Y.element_size(), st["ms"], pk)
            rec.update({"conv_ms": st["ms"], "conv_ms_min": st["ms_min"], "bound": r["bound"], "frac": r["frac"],
                        "effective_tflops": r["useful_flops"] / (st["ms"] * 1e-3) / 1e12})
            if with_setup:
                rec["step_ms"] = rec["mask_ms"] + rec["compact_ms"] + rec["conv_ms"]
            if dtype == "i8" and layer.O % 16 == 0:
                # the same product with the requantised int8 output of the 8-bit pipeline (a quarter of the output bytes)
                Y8 = torch.empty(Y.shape, dtype=torch.int8, device="cuda")
                shift = torch.full((layer.O,), 10, dtype=torch.int32, device="cuda")
                s8 = stats(gpu.timed(lambda: lay.conv2d_q8(Xd, bd, shift, Y8, stride, pad), reps, 1))
                lay.check()
                r8 = roofline_of(layer, NB - n_zero, 8, 8, dtype, 1, s8["ms"], pk)
                rec.update({"conv_q8_ms": s8["ms"], "q8_bound": r8["bound"], "q8_frac": r8["frac"]})
                del Y8, shift
            out.append(rec)
        del Wd, Xd, bd, Y, lay
    return out


def pass_spgemm(gpu, bsp, torch, reps=5):
    """Block-sparse x block-sparse product C = (Gamma . A)(Omega . B)^t, 2048 x 4096 times (2048 x 4096)^t, bf16 8x8 blocks,
    magnitude masks at 50 % and 75 %: useful FLOPs are those of the block pairs that both masks keep.  The kernel runs on
    the general-purpose pipes (index look-ups, ballots; the 8 x 8 x 8 products of bf16 blocks go two at a time through one
    m16n8k16 tensor-core instruction of the warp), so its yardstick is the fp32 FMA rate: 148 SMs x 128 lanes x 2 x 1.965 GHz."""
    peak = 148 * 128 * 2 * 1.965e9 / 1e12
    out = []
    g = torch.Generator(device="cuda")
    g.manual_seed(77)
    O, I = 2048, 4096
    A = (torch.randn((O, 1, 1, I), device="cuda", generator=g) / 64).to(torch.bfloat16)
    B = (torch.randn((O, 1, 1, I), device="cuda", generator=g) / 64).to(torch.bfloat16)
    Cm = torch.empty((O, O), dtype=torch.float32, device="cuda")
    la = bsp.SparseLayer(O, I, 1, 1, 8, 8, torch.bfloat16)
    lb = bsp.SparseLayer(O, I, 1, 1, 8, 8, torch.bfloat16)
    NB = la.NBo * la.NBi
    for s in (0.5, 0.75):
        for lay, W in ((la, A), (lb, B)):
            lay.mask(W, int(s * NB + 0.5))
            lay.compact(W)
        st = stats(gpu.timed(lambda: bsp.bsp_spgemm(la.wd, la.handle(), lb.wd, lb.handle(), Cm, la.ws), reps, 1))
        la.check()
        ga = la.gamma.view(la.NBo, la.NBi).float()
        gb = lb.gamma.view(lb.NBo, lb.NBi).float()
        pairs = float((ga @ gb.t()).sum().item())             # block pairs that both masks keep
        fl = 2.0 * 512 * pairs
        out.append({"sparsity": s, **st, "useful_flops": fl, "tflops": fl / (st["ms"] * 1e-3) / 1e12,
                    "roofline": {"bound": "alu", "peak": peak, "unit": "TFLOP/s", "frac": fl / (st["ms"] * 1e-3) / 1e12 / peak}})
    return out


def pass_chain(gpu, bsp, torch, pk, reps=10):
    """Fused pairs of layers (bsp_conv2d_chain) against the two separate calls through a bfloat16 tensor in memory: the
    3x3 -> 1x1 tails of the ResNet50 bottlenecks, batch 64, bf16, 8x8 at 50 %, bf16 output.  The HBM roofline of the
    fused call counts X in and Y out only: the tensor between the layers never leaves the chip."""
    out = []
    g = torch.Generator(device="cuda")
    g.manual_seed(91)
    for name, L, I, O1, O2 in (("c2.3x3.64-64+1x1.64-256", 56, 64, 64, 256), ("c3.3x3.128-128+1x1.128-512", 28, 128, 128, 512),
                               ("c4.3x3.256-256+1x1.256-1024", 14, 256, 256, 1024)):
        N = 64
        W1 = (torch.randn((O1, 3, 3, I), device="cuda", generator=g) * (2.0 / (9 * I)) ** 0.5).to(torch.bfloat16)
        W2 = (torch.randn((O2, 1, 1, O1), device="cuda", generator=g) * (2.0 / O1) ** 0.5).to(torch.bfloat16)
        X = torch.randn((N, L, L, I), device="cuda", generator=g).to(torch.bfloat16)
        b1 = torch.randn((O1,), device="cuda", generator=g) * 0.1
        b2 = torch.randn((O2,), device="cuda", generator=g) * 0.1
        l1 = bsp.SparseLayer(O1, I, 3, 3, 8, 8, torch.bfloat16, canonical=False)
        l2 = bsp.SparseLayer(O2, O1, 1, 1, 8, 8, torch.bfloat16, canonical=False)
        for lay, W in ((l1, W1), (l2, W2)):
            lay.mask(W, lay.NBo * lay.NBi // 2)
            lay.compact(W)
        T = torch.empty((N, L, L, O1), dtype=torch.bfloat16, device="cuda")
        Ya = torch.empty((N, L, L, O2), dtype=torch.bfloat16, device="cuda")
        Yb = torch.empty_like(Ya)
        xd = bsp.XDesc(N, L, L, 1, 1, 1, 1)

        def separate():
            l1.conv2d(X, b1, T, (1, 1), (1, 1))
            l2.conv2d(T, b2, Ya)

        def fused():
            bsp.bsp_conv2d_chain(l1.wd, l1.handle(), l2.wd, l2.handle(), xd, X, b1, 0, b2, Yb, bsp.BF16, l1.ws)

        ts = stats(gpu.timed(separate, reps, 2))
        tf = stats(gpu.timed(fused, reps, 1))
        l1.check()
        l2.check()
        P = N * L * L
        useful = 2.0 * P * (l1.NBo * l1.NBi // 2) * 64 * 9 + 2.0 * P * (l2.NBo * l2.NBi // 2) * 64
        hbm = X.numel() * 2 + Yb.numel() * 2 + (W1.numel() + W2.numel())
        t_roof = max(useful / (pk["bf16_tflops"] * 1e12), hbm / (pk["hbm_gbs"] * 1e9)) * 1e3
        out.append({"pair": name, "separate_ms": ts["ms"], "fused_ms": tf["ms"], "speedup": ts["ms"] / tf["ms"],
                    "bit_identical": bool(torch.equal(Ya, Yb)), "effective_tflops": useful / (tf["ms"] * 1e-3) / 1e12,
                    "algorithmic_bytes": hbm, "bytes_saved_vs_separate": 2 * T.numel() * 2, "roofline_ms": t_roof,
                    "frac": t_roof / tf["ms"]})
    # the same tail on 8-bit tensors (int8 between the layers and out, power-of-two scales): exact, so the comparison is bit for bit
    N, L, I, O1, O2 = 64, 56, 64, 64, 256
    W1 = torch.randint(-127, 128, (O1, 3, 3, I), device="cuda", dtype=torch.int8, generator=g)
    W2 = torch.randint(-127, 128, (O2, 1, 1, O1), device="cuda", dtype=torch.int8, generator=g)
    X = torch.randint(-127, 128, (N, L, L, I), device="cuda", dtype=torch.int8, generator=g)
    b1 = torch.randint(-(1 << 15), 1 << 15, (O1,), device="cuda", dtype=torch.int32, generator=g)
    b2 = torch.randint(-(1 << 15), 1 << 15, (O2,), device="cuda", dtype=torch.int32, generator=g)
    s1 = torch.full((O1,), 11, device="cuda", dtype=torch.int32)
    s2 = torch.full((O2,), 9, device="cuda", dtype=torch.int32)
    l1 = bsp.SparseLayer(O1, I, 3, 3, 8, 8, torch.int8, canonical=False)
    l2 = bsp.SparseLayer(O2, O1, 1, 1, 8, 8, torch.int8, canonical=False)
    for lay, W in ((l1, W1), (l2, W2)):
        lay.mask(W, lay.NBo * lay.NBi // 2)
        lay.compact(W)
    T = torch.empty((N, L, L, O1), dtype=torch.int8, device="cuda")
    Ya = torch.empty((N, L, L, O2), dtype=torch.int8, device="cuda")
    Yb = torch.empty_like(Ya)
    xd = bsp.XDesc(N, L, L, 1, 1, 1, 1)

    def separate8():
        l1.conv2d_q8(X, b1, s1, T, (1, 1), (1, 1))
        l2.conv2d_q8(T, b2, s2, Ya)

    def fused8():
        bsp.bsp_conv2d_chain_q8(l1.wd, l1.handle(), l2.wd, l2.handle(), xd, X, b1, s1, 0, b2, s2, Yb, l1.ws)

    ts = stats(gpu.timed(separate8, reps, 2))
    tf = stats(gpu.timed(fused8, reps, 1))
    l1.check()
    l2.check()
    hbm = X.numel() + Yb.numel() + (W1.numel() + W2.numel()) // 2
    out.append({"pair": "c2.3x3.64-64+1x1.64-256 int8 -> int8", "separate_ms": ts["ms"], "fused_ms": tf["ms"], "speedup": ts["ms"] / tf["ms"],
                "bit_identical": bool(torch.equal(Ya, Yb)), "algorithmic_bytes": hbm, "bytes_saved_vs_separate": 2 * T.numel(),
                "roofline_ms": hbm / (pk["hbm_gbs"] * 1e9) * 1e3, "frac": hbm / (pk["hbm_gbs"] * 1e9) * 1e3 / tf["ms"]})
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweeps", action="store_true", help="headline only: skip the block-shape sweep and the layer-table passes")
    ap.add_argument("--only-chain", action="store_true", help="of the extra passes run the fused pairs of layers only (for profiling)")
    ap.add_argument("--no-graph", action="store_true", help="launch the three calls of a step one by one instead of replaying a CUDA graph of them")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    layer, dtype, (bo, bi), sparsity, cfg, sigma = workload(args.workload)
    if args.impl == "reference":
        return run_reference(args, layer, dtype, bo, bi, sparsity, cfg, sigma)

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
    ex, ey = ELEM[dtype], 4
    # every rank draws its own batch (weak scaling); weights are the same on all ranks
    W, X, b = make_host_tensors(layer, dtype, cfg, sigma, 0)
    if rank > 0:
        X = make_host_tensors(layer, dtype, cfg, sigma, rank)[1]
    NB = (layer.O // bo) * (layer.I // bi)
    n_zero = int(sparsity * NB + 0.5)
    nnz = NB - n_zero

    gpu = Gpu(torch)
    stream = gpu.stream
    Wd = torch.from_numpy(W).cuda().to(tdt)
    Xd = torch.from_numpy(X).cuda().to(tdt)
    bd = torch.from_numpy(b).cuda()
    Y = torch.empty((layer.N, layer.M, layer.Nw, layer.O), dtype=ydt, device="cuda")
    lay = bsp.SparseLayer(layer.O, layer.I, layer.H, layer.K, bo, bi, tdt, canonical=False)
    stride, pad = (layer.stride_h, layer.stride_w), (layer.pad_h, layer.pad_w)
    pk = peaks()

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
        gpu.flush.zero_()
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
        gpu.flush.zero_()
        ev_step[k][0].record(stream)
        if graph is not None:
            graph.replay()
        else:
            step()
        ev_step[k][1].record(stream)
    barrier()
    lay.check()
    t_step = np.array([e[0].elapsed_time(e[1]) for e in ev_step])
    ms_step = float(t_step.mean())

    # ---- the phases of a step, each call bracketed by events (launched one by one; the events and launch gaps make
    # their sum larger than a graph replay of the step)
    n_ph = max(10, min(args.steps, 50))
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(n_ph)]
    for k in range(n_ph):
        gpu.flush.zero_()
        step(evs[k])
    torch.cuda.synchronize()
    t_mask = np.array([e[0].elapsed_time(e[1]) for e in evs])
    t_comp = np.array([e[1].elapsed_time(e[2]) for e in evs])
    t_conv = np.array([e[2].elapsed_time(e[3]) for e in evs])

    # ---- the same layer dense (Gamma == 1) through the same kernel, for the speedup
    dense = bsp.SparseLayer(layer.O, layer.I, layer.H, layer.K, bo, bi, tdt, canonical=False)
    dense.compact(Wd, torch.ones(NB, dtype=torch.uint8, device="cuda"))
    dense.nnz = NB
    t_dense = gpu.timed(lambda: dense.conv2d(Xd, bd, Y, stride, pad), max(args.steps // 2, 5), 3)
    dense.check()
    ms_dense = float(np.median(t_dense))
    del dense

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

    n_e2e = max(3, min(args.steps, 20))
    for _ in range(3):
        e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(n_e2e):
        e2e_step()
    e1.record(stream)
    barrier()
    ms_e2e = e0.elapsed_time(e1) / n_e2e
    lay.check()

    # ---- the sweeps (rank 0 of a single-GPU run): block shapes x sparsities on the headline layer, then the layer tables
    sweeps = {}
    if rank == 0 and world == 1 and args.only_chain:
        del Xd, Y, Wh, Xh, Yh
        torch.cuda.empty_cache()
        sweeps["chain_resnet50_tails_b64_bf16_8x8_50"] = pass_chain(gpu, bsp, torch, pk, reps=2)
    elif rank == 0 and world == 1 and not args.no_sweeps:
        gemm_layer, gdt, _, _, _, gsig = workload("gemm_4096_p8192")
        if layer.name == gemm_layer.name:
            sweeps["sweep_gemm_4096_p8192"] = sweep_product(gpu, bsp, torch, layer, dtype, Wd, Xd, bd, Y, pk)
        del Xd, Y, Wh, Xh, Yh
        torch.cuda.empty_cache()
        if layer.name != gemm_layer.name:
            gW, gX, gb, gY = device_layer(torch, bsp, gemm_layer, gdt, 3000, gsig)
            sweeps["sweep_gemm_4096_p8192"] = sweep_product(gpu, bsp, torch, gemm_layer, gdt, gW, gX, gb, gY, pk)
            del gW, gX, gb, gY
        r50 = pass_layers(gpu, bsp, torch, synth.resnet50_layers(64), "bf16", (0.5,), pk, torch.bfloat16, False)
        sweeps["resnet50_b64_bf16_8x8_50"] = {
            "layers": r50, "sparse_layers_ms": float(sum(r["conv_ms"] * r["count"] for r in r50)),
            "note": "every sparse-eligible conv / FC layer once (x count in the sum), bf16 in and out, product call only"}
        i8 = pass_layers(gpu, bsp, torch, synth.vgg16_layers(32) + synth.inception_v3_layers(32), "i8", (0.5, 0.75), pk,
                         torch.int32, True, reps=3)
        sweeps["vgg16_inceptionv3_b32_int8_8x8"] = {
            "layers": i8, "note": "int8 -> int32, bsp_mask, bsp_compact and the product each timed on their own",
            "sum_ms": {str(s): {k: float(sum(r.get(k, r["conv_ms"]) * r["count"] for r in i8 if r["sparsity"] == s))
                                for k in ("mask_ms", "compact_ms", "conv_ms", "step_ms", "conv_q8_ms")} for s in (0.5, 0.75)}}
        sweeps["spgemm_2048x4096_bf16_8x8"] = pass_spgemm(gpu, bsp, torch)
        sweeps["chain_resnet50_tails_b64_bf16_8x8_50"] = pass_chain(gpu, bsp, torch, pk)
    clocks = sampler.stop()

    # max over ranks
    ms_step, ms_e2e, ms_conv = reduce_max([ms_step, ms_e2e, float(t_conv.mean())], world, "cuda")

    fl = useful_flops(layer, nnz, bo, bi)
    value = job_tflops(fl, world, ms_step)
    roof = roofline_of(layer, nnz, bo, bi, dtype, ey, ms_conv, pk)
    kernel = bsp.conv_kernel_name(lay.wd, bsp.XDesc(layer.N, layer.L, layer.J, stride[0], stride[1], pad[0], pad[1]))
    roof.pop("useful_flops")
    roof.update({"traffic": measured_traffic(layer.name, kernel), "kernel": kernel, "kernel_ms": ms_conv,
                 "peak_source": pk["source"] + " (burst)" + ("" if dtype == "bf16" else f" bf16 x {PEAK_RATIO[dtype]:.3g} nominal ratio")})

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": {"bf16": "bf16", "f32": "tf32", "i8": "int8"}[dtype], "data": "synthetic",
        "config": {"workload": layer.name, "block": f"{bo}x{bi}", "sparsity": sparsity, "nnz_blocks": nnz,
                   "step": "bsp_mask + bsp_compact + " + ("bsp_gemm" if layer.H * layer.K == 1 else "bsp_conv2d"), "launch": how,
                   "l2": "flushed between steps (384 MB write)", "per_gpu_batch": layer.N},
        "ms_per_step_median": float(np.median(t_step)), "ms_per_step_min": float(t_step.min()),
        "phases_ms": {"mask": float(t_mask.mean()), "compact": float(t_comp.mean()), "product": ms_conv,
                      "note": "each call between its own events, launched one by one"},
        "product_only": {"tflops": fl / (ms_conv * 1e-3) / 1e12, "ms": ms_conv, "ms_median": float(np.median(t_conv)),
                         "ms_min": float(t_conv.min()), "dense_ms": ms_dense, "speedup_vs_dense": ms_dense / ms_conv,
                         "useful_flops": fl, "executed_flops": float(layer.dense_flops()),
                         "algorithmic_weight_bytes": nnz * bo * bi * layer.H * layer.K * ex,
                         "stored_weight_bytes": layer.O * layer.I * layer.H * layer.K * ex if kernel == "gemm_tc_kernel" else None},
        "roofline": roof,
        "e2e": {"value": job_tflops(fl, world, ms_e2e), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e, "steps": n_e2e},
        "gpu_launches": args.steps * bsp.launches_per_step(lay.wd),
        "clocks": clocks,
    }
    out.update(sweeps)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline_subprocess(layer.name)
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
