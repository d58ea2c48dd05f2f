"""Benchmark of the group-wise mixed-precision weight-only linear layer on B200.

Default workload: the LLaMA-7B decode layer set at M = 1, average 2 bits (bit-widths {1,2,3} per
group of 128 input columns): q/k/v/o 4096x4096, gate/up 11008x4096, down 4096x11008 for all 32
blocks, 224 distinct layers (1.83 GB of packed weights, scales and zeros, far larger than L2).
One step = one pass over all 224 layers, replayed from a CUDA graph.  The metric is achieved
GB/s over the algorithmic bytes (packed codes + fp16 scales and zeros + bit map + x + y).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints one JSON line (rank 0).  With N > 1 every rank runs an independent replica of the
workload on its own GPU (no data-path collective); the value is the sum over ranks divided by
the slowest rank's time.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2405_14917_b200 import workloads as wl  # noqa: E402

METRIC = "mixed-precision dequant GEMV GB/s at M=1 (LLaMA-7B layer set, avg 2-bit, g=128)"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_TENSOR_TFLOPS = 1400.0

# DRAM traffic of the GEMV kernel per launch from one ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum), keyed by the sha256 of the kernel source it was taken from.  A kernel
# that has changed since reports null.
NCU_TRAFFIC = {
    # layer-set kernel, 4 blocks of the LLaMA-7B sweep (28 layers, avg 2-bit, M = 1): 228,629,760 B read +
    # 4,367,360 B written per launch (algorithmic 228,297,816 B); scaled to the full sweep by the algorithmic bytes
    "e25960915e353f61dfff3a350b7b271bfc027a892e28cdcf869cb410ab6b1a0e": {"layer": "4 blocks", "traffic_bytes": 232997120, "algorithmic_bytes": 228297816},
    # 4096x4096 layer, avg 2-bit, M = 1: 4,755,200 B read + 0 written per launch (algorithmic 4,735,008 B);
    # scaled to the sweep's average launch by the algorithmic bytes (traffic grows with the layer size)
    "4b06a5d5b512621bbe525cb3d0c66822ff452c130a671af895469c10fb834593": {"layer": "4096x4096", "traffic_bytes": 4755200, "algorithmic_bytes": 4735008},
}


# DRAM bytes (read + written) of the 14 gemm_kernel launches of one step of llama13b-prefill-avg3-m2048, from one ncu
# capture of dram__bytes_read.sum and dram__bytes_write.sum; keyed by the SHA-256 of slim_gemm.cu at capture time
NCU_TRAFFIC_GEMM = {
    "1a98f6bdbcf5c7c1c57790e2a1ed836e1474feb538dcafefdc70f951cd97623b": {"workload": "llama13b-prefill-avg3-m2048", "launches": 14, "traffic_bytes": 1119355392 + 232290560},
}


def workload_spec(name: str):
    if name == "llama7b-decode-avg2":
        return dict(model="llama-7b", avg_bits=2, M=1, n_blocks=wl.N_BLOCKS["llama-7b"])
    if name == "llama7b-decode-avg3":
        return dict(model="llama-7b", avg_bits=3, M=1, n_blocks=wl.N_BLOCKS["llama-7b"])
    if name == "llama7b-block-avg2":      # four blocks only (small case for profiling)
        return dict(model="llama-7b", avg_bits=2, M=1, n_blocks=4)
    if name.startswith("llama13b-prefill-avg3-m"):    # batched tensor-core path, two blocks (14 layers)
        return dict(model="llama-13b", avg_bits=3, M=int(name.rsplit("m", 1)[1]), n_blocks=2)
    # other decode configurations: <model>-decode-avg<bits>-m<M>[-blocks<n>], model in llama7b / llama70b
    import re
    m = re.fullmatch(r"(llama7b|llama70b)-decode-avg([23])-m(\d+)(?:-blocks(\d+))?", name)
    if m:
        model = {"llama7b": "llama-7b", "llama70b": "llama-2-70b"}[m.group(1)]
        blocks = int(m.group(4)) if m.group(4) else (wl.N_BLOCKS[model] if model == "llama-7b" else 8)
        return dict(model=model, avg_bits=int(m.group(2)), M=int(m.group(3)), n_blocks=blocks)
    raise SystemExit(f"unknown workload {name}")


# ------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
            time.sleep(0.3)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [t.strip() for t in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1]))
                    mx.append(float(f[2]))
                except ValueError:
                    continue
                for nm, v in zip(names, f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(nm)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def measured_tensor_peak():
    """Dense fp16 peak = the measured bf16 figure (same nominal rate), sustained: the kernel is
    timed inside a long step."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["bf16_tflops_sustained"]), "measured (sustained bf16, same nominal rate as fp16)"
    except Exception:
        return FALLBACK_TENSOR_TFLOPS, "fallback"


# ------------------------------------------------------------------------------------------ CPU oracle legs
def _oracle_layers(spec, n_layers):
    """First n_layers layers of the sweep, generated and quantised on the host by the oracle."""
    from oracle import slim_oracle as orc
    out = []
    for (name, blk, N, K, seed) in wl.model_layers(spec["model"], spec["n_blocks"]):
        if len(out) >= n_layers:
            break
        W = wl.make_weight(seed, N, K)
        a = wl.make_act_norms(seed, K)
        bits, codes, scales, zeros = orc.make_layer(W, a, spec["avg_bits"])
        out.append(dict(name=name, N=N, K=K, bits=bits, codes=codes, scales=scales, zeros=zeros,
                        x=wl.make_x(seed, spec["M"], K)))
    return out


def _time_oracle(layers, rows_of_first=None):
    """Runs the plain-C oracle once over `layers` (optionally only the first rows of the first
    layer).  Returns (seconds, algorithmic bytes, threads)."""
    from oracle import slim_oracle_c as oc
    total_bytes, threads = 0, 1
    t0 = time.perf_counter()
    for L in layers:
        codes, scales, zeros, N = L["codes"], L["scales"], L["zeros"], L["N"]
        if rows_of_first is not None:
            N = rows_of_first
            codes, scales, zeros = codes[:N], np.ascontiguousarray(scales[:, :N]), np.ascontiguousarray(zeros[:, :N])
        _, threads = oc.linear_f64(L["x"], codes, scales, zeros)
        total_bytes += wl.algorithmic_bytes(L["x"].shape[0], N, L["K"], L["bits"])
    return time.perf_counter() - t0, total_bytes, threads


def cpu_baseline(spec, budget_s=12.0):
    """The oracle as it stands on the host cores, over the first block's layers (bounded)."""
    from oracle import slim_oracle_c as oc
    oc.build()
    layers = _oracle_layers(spec, 7)
    _time_oracle(layers[:1], rows_of_first=256)   # load the library, touch the code
    secs, nbytes, reps, threads = 0.0, 0, 0, 1
    while secs < budget_s and reps < 8:
        s, b, threads = _time_oracle(layers)
        secs, nbytes, reps = secs + s, nbytes + b, reps + 1
    return {"value": nbytes / secs / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"block 0 of the sweep (7 layers, {nbytes // reps / 1e6:.1f} MB algorithmic) x {reps} passes, "
                      f"plain-C fp64 dequantise-then-dot, OpenMP over rows, {secs:.1f} s"}


def run_reference(args, spec):
    """--impl reference: the CPU oracle, each step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import slim_oracle_c as oc
    oc.build()
    steps = args.steps if args.steps is not None else 5
    warmup = args.warmup if args.warmup is not None else 1
    layers = _oracle_layers(spec, 7)
    # calibrate on 256 rows of the first layer, then size the per-step sample for ~100 s in total
    t_cal, _, threads = _time_oracle(layers[:1], rows_of_first=256)
    t_cal, _, threads = _time_oracle(layers[:1], rows_of_first=256)
    per_row = t_cal / 256
    budget = 100.0 / max(steps + warmup, 1)
    block_rows = sum(L["N"] * L["K"] for L in layers) / layers[0]["K"]
    if per_row * block_rows <= budget:
        sample, rows, what = layers, None, "block 0 of the sweep (7 layers)"
    else:
        rows = int(min(layers[0]["N"], max(16, budget / per_row))) // 16 * 16
        rows = max(rows, 16)
        sample, what = layers[:1], f"first {rows} output rows of layer q, block 0"
    for _ in range(warmup):
        _time_oracle(sample, rows)
    secs, nbytes = 0.0, 0
    for _ in range(steps):
        s, b, threads = _time_oracle(sample, rows)
        secs, nbytes = secs + s, nbytes + b
    value = nbytes / secs / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": warmup, "ms_per_step": 1e3 * secs / steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "M": spec["M"], "avg_bits": spec["avg_bits"], "g": wl.GROUP},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": what + "; plain-C fp64 dequantise-then-dot, OpenMP over rows"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------ GPU arm
def build_layers(spec, device, rank):
    """Quantises the whole sweep on the device through the library: salience, bit allocation,
    Eq. 1 quantizer, packing.  Returns the resident layers."""
    import torch
    from paper_2405_14917_b200 import binding as slim
    layers = []
    for (name, blk, N, K, seed) in wl.model_layers(spec["model"], spec["n_blocks"]):
        W, a = wl.make_weight_and_norms_device(seed + (rank,), N, K, device)
        layers.append(slim.QuantLinear.from_weight(W, a, spec["avg_bits"]))
        del W, a
    torch.cuda.synchronize()
    return layers


def run_sba(args):
    """--workload sba-llama7b-block: the SBA search (func SBA of Algorithm 2) on the seven layers of one
    LLaMA-7B block, avg 2-bit, 128 synthetic calibration tokens; G/2 + 1 candidate bit maps per layer, each
    quantised (Eq. 1), packed and evaluated by the hot path, error = softmax-KL against x W^T."""
    import torch
    from paper_2405_14917_b200 import binding as slim
    steps = args.steps if args.steps is not None else 5
    warmup = max(args.warmup if args.warmup is not None else 3, 3)
    M = 128
    torch.cuda.set_device(0)
    slim.lib()
    layers = []
    for (name, blk, N, K, seed) in wl.model_layers("llama-7b", 1):
        W, a = wl.make_weight_and_norms_device(seed, N, K, "cuda")
        x = torch.from_numpy(wl.make_x(seed, M, K)).cuda()
        ws = torch.empty(slim.sba_workspace_bytes(M, N, K, 2), dtype=torch.uint8, device="cuda")
        layers.append((W, x, a, ws, W.cpu().pin_memory(), x.cpu().pin_memory()))
    candidates = sum(W.shape[1] // 128 // 2 + 1 for W, *_ in layers)
    weight_visits = sum((W.shape[1] // 128 // 2 + 1) * W.numel() for W, *_ in layers)

    def step_device():
        for W, x, a, ws, _, _ in layers:
            slim.sba_search(W, x, a, 2, workspace=ws)

    def step_e2e():
        for W, x, a, ws, Wh, xh in layers:
            W.copy_(Wh, non_blocking=True)
            x.copy_(xh, non_blocking=True)
            slim.sba_search(W, x, a, 2, workspace=ws)       # p*, the bit map and the error curve come back to the host

    def timed(fn, k):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(k):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    for _ in range(warmup):
        step_device()
    sampler = ClockSampler(0)
    sampler.start()
    ms = timed(step_device, steps)
    clocks = sampler.stop()
    for _ in range(3):
        step_e2e()
    e2e_steps = max(steps // 2, 3)
    ms_e2e = timed(step_e2e, e2e_steps)
    value = candidates * steps / (ms * 1e-3)
    # dominant kernel (31 % of the device time in the ncu launch list): gemm_kernel<128>, the hot path evaluating a
    # candidate on the 128 calibration tokens, 2 M N K FLOPs each; charged with the whole step (quantizer, packing,
    # KL and the host loop included)
    flops = 2.0 * M * weight_visits
    achieved = flops * steps / (ms * 1e-3) / 1e12
    peak, peak_kind = measured_tensor_peak()
    line = {"metric": "SBA search: candidate bit maps evaluated per second (LLaMA-7B block, avg 2-bit, 128 tokens)",
            "value": value, "unit": "candidates/s", "n_gpus": 1, "steps": steps, "warmup": warmup, "ms_per_step": ms / steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64 quantizer and KL, f16 tensor-core layer calls", "data": "synthetic",
            "config": {"workload": args.workload, "layers": len(layers), "candidates_per_step": candidates, "tokens": M,
                       "l2": "404 MB of fp16 weights per step > L2"},
            "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                         "peak_kind": peak_kind, "kernel": "gemm_kernel",
                         "avg_launch_us": 1e3 * ms / steps / candidates, "flops_per_launch": flops / candidates,
                         "traffic": None},
            "e2e": {"value": candidates * e2e_steps / (ms_e2e * 1e-3), "unit": "candidates/s",
                    "h2d_bytes_per_step": int(sum(2 * W.numel() + 2 * x.numel() for W, x, *_ in layers)),
                    "d2h_bytes_per_step": int(sum(8 * (W.shape[1] // 128) + 8 * (W.shape[1] // 256 + 1) * (M + 1) for W, *_ in layers)),
                    "steps": e2e_steps, "ms_per_step": ms_e2e / e2e_steps},
            "gpu_launches": steps * (candidates * 4 + 2 * len(layers)), "clocks": clocks}
    print(json.dumps(line), flush=True)


def run_sqc(args):
    """--workload sqc-llama7b-block: Salience-Weighted Quantizer Calibration (Algorithm 2) of the seven
    layers of one LLaMA-7B block (202 M weights, avg 2-bit map, lambda = 0.1, n = 50) per step."""
    import torch
    from paper_2405_14917_b200 import binding as slim
    steps = args.steps if args.steps is not None else 20
    warmup = max(args.warmup if args.warmup is not None else 3, 3)
    torch.cuda.set_device(0)
    slim.lib()
    layers = []
    for (name, blk, N, K, seed) in wl.model_layers("llama-7b", 1):
        W, a = wl.make_weight_and_norms_device(seed, N, K, "cuda")
        bits = slim.allocate_bits(slim.group_salience(W, a).cpu().numpy(), 2)
        layers.append((W, bits, W.cpu().pin_memory()))
    weights = sum(W.numel() for W, _, _ in layers)

    def step_device():
        for W, bits, _ in layers:
            slim.quantize_sqc(W, bits)

    outs_host = [(torch.empty(W.shape, dtype=torch.uint8).pin_memory(),
                  torch.empty((W.shape[1] // 128, W.shape[0]), dtype=torch.float16).pin_memory(),
                  torch.empty((W.shape[1] // 128, W.shape[0]), dtype=torch.float16).pin_memory()) for W, _, _ in layers]

    def step_e2e():
        for (W, bits, Wh), (ch, sh, zh) in zip(layers, outs_host):
            W.copy_(Wh, non_blocking=True)
            codes, scales, zeros, _ = slim.quantize_sqc(W, bits)
            ch.copy_(codes, non_blocking=True); sh.copy_(scales, non_blocking=True); zh.copy_(zeros, non_blocking=True)
        torch.cuda.current_stream().synchronize()

    def timed(fn, k):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(k):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    for _ in range(warmup):
        step_device()
    sampler = ClockSampler(0)
    sampler.start()
    ms = timed(step_device, steps)
    clocks = sampler.stop()
    for _ in range(3):
        step_e2e()
    e2e_steps = max(steps // 4, 3)
    ms_e2e = timed(step_e2e, e2e_steps)
    value = weights * steps / (ms * 1e-3) / 1e9
    # fp64 work: 2n = 100 candidates per weight, 10 fp64 operations each (divide, round, add, min, max,
    # subtract, multiply, subtract, multiply, add); peak = 148 SMs x 64 fp64 lanes x 1.965 GHz
    ops = 100 * 10 * weights
    achieved = ops * steps / (ms * 1e-3) / 1e12
    peak = 148 * 64 * 1.965e9 / 1e12
    line = {"metric": "SQC calibration throughput (LLaMA-7B block, 2n = 100 candidates, g=128)", "value": value,
            "unit": "Gweight/s", "n_gpus": 1, "steps": steps, "warmup": warmup, "ms_per_step": ms / steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "layers": len(layers), "weights_per_step": weights, "lambda": 0.1, "n": 50,
                       "l2": "404 MB of fp16 weights per step > L2"},
            "roofline": {"bound": "alu", "achieved": achieved, "peak": peak, "unit": "Tinstr/s (fp64 lanes)", "frac": achieved / peak,
                         "peak_kind": "derived: 148 SMs x 64 fp64 lanes x 1.965 GHz", "kernel": "quantize_sqc_kernel",
                         "avg_launch_us": 1e3 * ms / steps / len(layers), "traffic": None},
            "e2e": {"value": weights * e2e_steps / (ms_e2e * 1e-3) / 1e9, "unit": "Gweight/s",
                    "h2d_bytes_per_step": 2 * weights, "d2h_bytes_per_step": weights + 4 * weights // 128 * 1,
                    "steps": e2e_steps, "ms_per_step": ms_e2e / e2e_steps},
            "gpu_launches": steps * len(layers), "clocks": clocks}
    print(json.dumps(line), flush=True)


def run_gptq(args):
    """--workload gptq-llama7b-layer: Algorithm 1 on one LLaMA-7B attention projection (4096 x 4096, avg 2-bit
    map, SQC quantizer, 2048 synthetic calibration tokens with correlated channels) per step: Hessian, Cholesky
    factor of the damped inverse, 32 groups of quantise-and-push."""
    import torch
    from paper_2405_14917_b200 import binding as slim
    steps = args.steps if args.steps is not None else 5
    warmup = max(args.warmup if args.warmup is not None else 3, 3)
    N = K = 4096
    T = 2048
    torch.cuda.set_device(0)
    slim.lib()
    seed = wl.layer_seed("llama-7b", "q_proj", 0)
    W_h = wl.make_weight(seed, N, K)
    x_h = wl.make_calibration_x(seed, T, K)
    W, x = torch.from_numpy(W_h).cuda(), torch.from_numpy(x_h).cuda()
    a = torch.from_numpy(wl.make_act_norms(seed, K)).cuda()
    bits = slim.allocate_bits(slim.group_salience(W, a).cpu().numpy(), 2)
    ws = torch.empty(slim.gptq_workspace_bytes(T, N, K), dtype=torch.uint8, device="cuda")
    Wp, xp = torch.from_numpy(W_h).pin_memory(), torch.from_numpy(x_h).pin_memory()
    G, nb = K // 128, K // 64
    outs = (torch.empty((N, K), dtype=torch.uint8).pin_memory(), torch.empty((G, N), dtype=torch.float16).pin_memory(),
            torch.empty((G, N), dtype=torch.float16).pin_memory())

    def step_device():
        return slim.gptq_quantize(W, x, bits, 0.01, "sqc", workspace=ws)

    def step_e2e():
        W.copy_(Wp, non_blocking=True)
        x.copy_(xp, non_blocking=True)
        res = slim.gptq_quantize(W, x, bits, 0.01, "sqc", workspace=ws)
        for h, d in zip(outs, res):
            h.copy_(d, non_blocking=True)
        torch.cuda.current_stream().synchronize()

    def timed(fn, k):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(k):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    for _ in range(warmup):
        step_device()
    sampler = ClockSampler(0)
    sampler.start()
    ms = timed(step_device, steps)
    clocks = sampler.stop()
    for _ in range(3):
        step_e2e()
    e2e_steps = max(steps // 2, 3)
    ms_e2e = timed(step_e2e, e2e_steps)
    weights = N * K
    value = weights * steps / (ms * 1e-3) / 1e6
    # fp64 operations the GEMM-shaped kernels execute (2 per multiply-add): Hessian tiles on and above the diagonal,
    # trailing updates of the factorisation, block rows of the triangular inverse, pushes of the group errors
    tile = 2.0 * 64 * 64
    flops = (nb * (nb + 1) // 2) * tile * T
    flops += sum(b * (b + 1) // 2 + b for b in range(1, nb)) * tile * 64      # trailing tiles and panel tiles
    seg = 64
    while seg < K:                                        # triangular inverse by doubling: T = B C^-1, then -A^-1 T
        for o in range(0, K, 2 * seg):
            s2 = min(seg, K - o - seg)
            if s2 > 0:
                flops += (seg // 64) * sum(tile * 64 * (tj + 1) for tj in range(s2 // 64))
                flops += (s2 // 64) * sum(tile * (seg - 64 * ti) for ti in range(seg // 64))
        seg *= 2
    flops += sum(2.0 * N * 128 * (K - 128 * (j + 1)) for j in range(G))
    achieved = flops * steps / (ms * 1e-3) / 1e12
    peak = 148 * 64 * 2 * 1.965e9 / 1e12
    levels = (nb - 1).bit_length()
    launches = 2 + nb + 2 * (nb - 1) + 2 * levels + 1 + 1 + 4 * G - 1
    line = {"metric": "GPTQ error compensation with SQC (Algorithm 1): weights quantised per second (LLaMA-7B 4096x4096 layer, avg 2-bit, g=128)",
            "value": value, "unit": "Mweight/s", "n_gpus": 1, "steps": steps, "warmup": warmup, "ms_per_step": ms / steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "N": N, "K": K, "calibration_tokens": T, "lambda": 0.01, "quantizer": "sqc",
                       "l2": "268 MB of fp64 factors and 134 MB of running weights per step > L2"},
            "roofline": {"bound": "alu", "achieved": achieved, "peak": peak, "unit": "TFLOP/s (fp64)", "frac": achieved / peak,
                         "peak_kind": "derived: 148 SMs x 64 fp64 FMA lanes x 2 x 1.965 GHz", "kernel": "gptq_update_kernel",
                         "flops_per_step": flops, "traffic": None},
            "e2e": {"value": weights * e2e_steps / (ms_e2e * 1e-3) / 1e6, "unit": "Mweight/s",
                    "h2d_bytes_per_step": 2 * weights + 2 * T * K, "d2h_bytes_per_step": weights + 4 * G * N,
                    "steps": e2e_steps, "ms_per_step": ms_e2e / e2e_steps},
            "gpu_launches": steps * launches, "clocks": clocks}
    if not args.no_cpu_baseline:
        from oracle import slim_oracle as orc
        rows = 128
        t0 = time.perf_counter()
        orc.gptq_quantize(W_h[:rows], x_h, np.asarray(bits), 0.01, "sqc")
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": rows * K / dt / 1e6, "unit": "Mweight/s", "cores": len(os.sched_getaffinity(0)), "kind": "oracle",
                                "sample": f"{rows} of {N} rows (rows are independent given the factor); the whole Hessian and factor are included"}
    print(json.dumps(line), flush=True)


def finish_gemm_line(args, spec, layers, world, steps, warmup, ms, e2e_steps, ms_e2e, x_host, y_host, clocks):
    """JSON line of a batched (M > 16) workload: TFLOP/s against the dense fp16 tensor peak."""
    M = spec["M"]
    flops = sum(2.0 * M * L.N * L.K for L in layers)
    value = world * flops * steps / (ms * 1e-3) / 1e12
    e2e_value = world * flops * e2e_steps / (ms_e2e * 1e-3) / 1e12
    peak, peak_kind = measured_tensor_peak()
    n_launch = len(layers)
    per_launch_us = 1e3 * ms / steps / n_launch
    achieved = flops / n_launch / (per_launch_us * 1e-6) / 1e12
    sha = hashlib.sha256(open(os.path.join(ROOT, "paper_2405_14917_b200", "csrc", "slim_gemm.cu"), "rb").read()).hexdigest()
    cap = NCU_TRAFFIC_GEMM.get(sha)
    traffic = cap["traffic_bytes"] / cap["launches"] if cap and cap["workload"] == args.workload and cap["launches"] == n_launch else None
    line = {
        "metric": f"mixed-precision dequant GEMM TFLOP/s at M={M} (LLaMA-13B layer shapes, avg 3-bit, g=128)",
        "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16 (tcgen05 kind::f16, f32 accumulate)", "data": "synthetic",
        "config": {"workload": args.workload, "layers": n_launch, "M": M, "avg_bits": spec["avg_bits"], "g": wl.GROUP,
                   "flops_per_step": flops, "l2": "14 distinct layers, 258 MB of weights per step > L2",
                   "launch": "CUDA graph of one launch per layer", "parallelism": f"replicas x{world}"},
        "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                     "peak_kind": peak_kind, "kernel": "gemm_kernel", "avg_launch_us": per_launch_us,
                     "flops_per_launch": flops / n_launch, "traffic": traffic, "frac_of_nominal_2250": achieved / 2250.0},
        "e2e": {"value": e2e_value, "unit": "TFLOP/s", "h2d_bytes_per_step": int(x_host.numel() * 2),
                "d2h_bytes_per_step": int(y_host.numel() * 2), "steps": e2e_steps, "ms_per_step": ms_e2e / e2e_steps},
        "gpu_launches": steps * n_launch,
        "clocks": clocks,
    }
    print(json.dumps(line), flush=True)


def run_ours(args, spec):
    import torch
    import torch.distributed as dist
    from paper_2405_14917_b200 import binding as slim
    from paper_2405_14917_b200 import replicas

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    steps = args.steps if args.steps is not None else (2000 if spec["M"] <= 16 else 300)
    warmup = max(args.warmup if args.warmup is not None else 20, 3)
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    slim.lib()   # fails loudly if the CUDA library is missing

    layers = build_layers(spec, device, rank)
    M = spec["M"]
    alg_bytes = sum(L.algorithmic_bytes(M) for L in layers)

    # all activations of the sweep in one buffer, all outputs in another
    x_off = np.cumsum([0] + [M * L.K for L in layers])
    y_off = np.cumsum([0] + [M * L.N for L in layers])
    gen = torch.Generator(device="cpu")
    gen.manual_seed(1234 + rank)
    x_host = torch.randn(int(x_off[-1]), generator=gen, dtype=torch.float32).to(torch.float16).pin_memory()
    y_host = torch.empty(int(y_off[-1]), dtype=torch.float16).pin_memory()
    x_dev = x_host.to(device)
    y_dev = torch.zeros(int(y_off[-1]), dtype=torch.float16, device=device)
    ws = torch.zeros(max(L.workspace_bytes(M) for L in layers), dtype=torch.uint8, device=device)
    slim.workspace_init(ws)
    xs = [x_dev[x_off[i]:x_off[i + 1]].view(M, L.K) for i, L in enumerate(layers)]
    ys = [y_dev[y_off[i]:y_off[i + 1]].view(M, L.N) for i, L in enumerate(layers)]

    use_set = M <= slim.GEMV_MAX_M and args.launch == "set"
    layer_set = slim.LayerSet(list(zip(layers, xs, ys))) if use_set else None

    def sweep():
        if use_set:
            layer_set.run()
            return
        for L, x, y in zip(layers, xs, ys):
            L.forward(x, ws, out=y)

    # capture one sweep in a CUDA graph (launch-bound otherwise: ~1.4 us of HBM time per layer)
    side = torch.cuda.Stream(device)
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        sweep()
        sweep()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        sweep()
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(step_fn, n):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for _ in range(n):
            step_fn()
        e1.record()
        barrier()
        return replicas.max_over_ranks(e0.elapsed_time(e1), device)

    def step_device():
        graph.replay()

    def step_e2e():
        x_dev.copy_(x_host, non_blocking=True)
        graph.replay()
        y_host.copy_(y_dev, non_blocking=True)
        torch.cuda.current_stream().synchronize()

    for _ in range(warmup):
        step_device()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ms = timed(step_device, steps)
    clocks = sampler.stop() if rank == 0 else None
    slim.workspace_status(ws)
    if use_set:
        layer_set.check()

    e2e_steps = max(steps // 4, 3)
    for _ in range(3):
        step_e2e()
    ms_e2e = timed(step_e2e, e2e_steps)
    slim.workspace_status(ws)
    if use_set:
        layer_set.check()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # launches of the dominant kernel per step: the persistent kernel once, or one kernel per layer
    n_launch = 1 if use_set else len(layers)
    per_launch_us = 1e3 * ms / steps / n_launch
    if M > slim.GEMV_MAX_M:
        finish_gemm_line(args, spec, layers, world, steps, warmup, ms, e2e_steps, ms_e2e, x_host, y_host, clocks)
        if world > 1:
            dist.destroy_process_group()
        return
    value = world * alg_bytes * steps / (ms * 1e-3) / 1e9
    e2e_value = world * alg_bytes * e2e_steps / (ms_e2e * 1e-3) / 1e9
    peak, peak_kind = measured_hbm_peak()
    achieved = alg_bytes / n_launch / (per_launch_us * 1e-6) / 1e9
    kernel_file = "slim_gemv_set.cu" if use_set else "slim_gemv.cu"
    sha = hashlib.sha256(open(os.path.join(ROOT, "paper_2405_14917_b200", "csrc", kernel_file), "rb").read()).hexdigest()
    traffic = NCU_TRAFFIC.get(sha)
    # the set launch also runs the small kernel that puts x into fragment order; its time is inside avg_launch_us
    kernels_per_step = 2 if use_set else len(layers) * (2 if M >= 4 else 1)
    line = {
        "metric": METRIC if args.workload == "llama7b-decode-avg2" else
                  f"mixed-precision dequant GEMV GB/s at M={M} ({spec['model']} layer set, avg {spec['avg_bits']}-bit, g=128)",
        "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": ("s32 (mma.sync m16n8k32 u8 x s8: byte-masked code words against base-256 digits of fixed-point x; f32 fold)"
                  if use_set and M == 1 else "f16 (mma.sync m16n8k16 on raw code fields, f32 accumulate)"), "data": "synthetic",
        "config": {"workload": args.workload, "layers": len(layers), "M": M, "avg_bits": spec["avg_bits"], "g": wl.GROUP,
                   "algorithmic_bytes_per_step": alg_bytes, "l2": f"distinct layers, {alg_bytes / 1e9:.2f} GB per step >> L2",
                   "launch": ("CUDA graph of the layer-set launch: one persistent kernel for the whole sweep "
                              "(plus one kernel that stages x)") if use_set else
                             "CUDA graph of one launch per layer, programmatic dependent launch",
                   "grouped_launch": bool(use_set),
                   "parallelism": f"replicas x{world}"},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": peak_kind, "kernel": "gemv_set_kernel" if use_set else "gemv_kernel", "avg_launch_us": per_launch_us,
                     "algorithmic_bytes_per_launch": alg_bytes / n_launch,
                     "traffic": (traffic["traffic_bytes"] / traffic["algorithmic_bytes"] * alg_bytes / n_launch) if traffic else None,
                     "frac_of_nominal_8000": achieved / 8000.0},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(x_host.numel() * 2),
                "d2h_bytes_per_step": int(y_host.numel() * 2), "steps": e2e_steps, "ms_per_step": ms_e2e / e2e_steps},
        "gpu_launches": steps * kernels_per_step,
        "clocks": clocks,
    }
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(spec)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama7b-decode-avg2")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--launch", default="set", choices=["set", "per-layer"],
                    help="decode workloads (M <= 16): the layer-set launch (one persistent kernel for the sweep) or one launch per layer")
    args = ap.parse_args()
    if args.workload == "sqc-llama7b-block" and args.impl != "reference":
        run_sqc(args)
        return
    if args.workload == "sba-llama7b-block" and args.impl != "reference":
        run_sba(args)
        return
    if args.workload == "gptq-llama7b-layer" and args.impl != "reference":
        run_gptq(args)
        return
    spec = workload_spec(args.workload)
    if args.impl == "reference":
        run_reference(args, spec)
    else:
        run_ours(args, spec)


if __name__ == "__main__":
    main()
