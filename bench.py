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
# dram__bytes_write.sum), keyed by the sha256 of the kernel's sources (slim_gemv_set.cu and the two device headers
# it includes, concatenated in that order) at the time of the capture.  A kernel that has changed since reports null.
SET_KERNEL_SOURCES = ("slim_gemv_set.cu", "slim_gemv_i8.cuh", "slim_gemv_dev.cuh")


def set_kernel_hash():
    h = hashlib.sha256()
    for name in SET_KERNEL_SOURCES:
        h.update(open(os.path.join(ROOT, "paper_2405_14917_b200", "csrc", name), "rb").read())
    return h.hexdigest()


NCU_TRAFFIC = {
    # layer-set kernel, 4 blocks of the LLaMA-7B sweep (28 layers, avg 2-bit, M = 1): 228,638,976 B read +
    # 4,520,192 B written per launch (algorithmic 228,297,816 B); scaled to the full sweep by the algorithmic bytes
    # (the traffic is the packed data read once, so it grows in proportion)
    "29183f24d4a3808dbf387c86522c99263ccdf08449605d2c7dfbcb28876d928c": {"layer": "4 blocks", "traffic_bytes": 233159168, "algorithmic_bytes": 228297816},
}


# DRAM bytes (read + written) of the 14 gemm_kernel launches of one step of llama13b-prefill-avg3-m2048, from one ncu
# capture of dram__bytes_read.sum and dram__bytes_write.sum; keyed by the SHA-256 of slim_gemm.cu at capture time
NCU_TRAFFIC_GEMM = {
    "a9b998b7a42c63bfc7bf8985dc1e3ee6b8be9ec1e3e35774be2538fadf174e9b": {"workload": "llama13b-prefill-avg3-m2048", "launches": 14, "traffic_bytes": 1049365760 + 218744064},
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


NOMINAL_HBM_GBS = 8000.0
NOMINAL_TENSOR_TFLOPS = 2250.0


def measured_tensor_burst():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops"])
    except Exception:
        return 1590.0


def _graph_of(fn, device):
    """Captures fn() (already run twice on a side stream) in a CUDA graph."""
    import torch
    side = torch.cuda.Stream(device)
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        fn()
        fn()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        fn()
    torch.cuda.synchronize()
    return graph


class Timer:
    """Device timing of blocks of exactly `steps` steps: barrier + synchronize on both sides, CUDA events on the
    current stream, largest time over the ranks.  Blocks are repeated until `min_total_s` of timed work has run (a
    handful of steps says little on a GPU whose clocks settle under its power limit after a few hundred ms)."""

    def __init__(self, device, world):
        self.device, self.world = device, world

    def barrier(self):
        import torch
        import torch.distributed as dist
        if self.world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def block(self, step_fn, steps, join=None):
        """`join`, if given, runs after the last step and before the closing event: a step function that works on
        other streams makes the current stream wait for them there."""
        import torch
        from paper_2405_14917_b200 import replicas
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.barrier()
        e0.record()
        for _ in range(steps):
            step_fn()
        if join is not None:
            join()
        e1.record()
        self.barrier()
        return replicas.max_over_ranks(e0.elapsed_time(e1), self.device)

    def blocks(self, step_fn, steps, min_total_s=1.0, min_blocks=1, max_blocks=400, join=None):
        ms = [self.block(step_fn, steps, join)]
        n = int(min(max_blocks, max(min_blocks, np.ceil(min_total_s * 1e3 / max(ms[0], 1e-3)))))
        for _ in range(n - 1):                     # n follows from a number every rank has: the ranks agree on it
            ms.append(self.block(step_fn, steps, join))
        return ms


def _timing_summary(ms_blocks, steps):
    per = np.asarray(ms_blocks) / steps
    return {"blocks": len(ms_blocks), "steps_per_block": steps, "ms_per_step_median": float(np.median(per)),
            "ms_per_step_min": float(per.min()), "ms_per_step_max": float(per.max()), "timed_ms_total": float(np.sum(ms_blocks))}


def decode_buffers(layers, M, device, seed):
    """All activations of a sweep in one pinned host buffer and one device buffer, all outputs in another pair."""
    import torch
    x_off = np.cumsum([0] + [M * L.K for L in layers])
    y_off = np.cumsum([0] + [M * L.N for L in layers])
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    x_host = torch.randn(int(x_off[-1]), generator=gen, dtype=torch.float32).to(torch.float16).pin_memory()
    y_host = torch.empty(int(y_off[-1]), dtype=torch.float16).pin_memory()
    x_dev = x_host.to(device)
    y_dev = torch.zeros(int(y_off[-1]), dtype=torch.float16, device=device)
    xs = [x_dev[x_off[i]:x_off[i + 1]].view(M, L.K) for i, L in enumerate(layers)]
    ys = [y_dev[y_off[i]:y_off[i + 1]].view(M, L.N) for i, L in enumerate(layers)]
    return x_host, y_host, x_dev, y_dev, xs, ys


def decode_sweep(layers, M, device, launch, seed=1234):
    """One pass over `layers` at M tokens as a CUDA graph.  launch: 'set' (one layer-set launch for everything),
    'per-layer' (slim_mpq_gemv per layer) or 'decoder-order' (what a decoder can issue: per block the q/k/v
    projections as a set of three on one x, o alone, gate/up as a set of two, down alone, in that order).
    Returns (graph, objects to keep alive, launches of the dominant kernel per step, kernels per step, buffers)."""
    import torch
    from paper_2405_14917_b200 import binding as slim
    bufs = decode_buffers(layers, M, device, seed)
    x_host, y_host, x_dev, y_dev, xs, ys = bufs
    ws = torch.zeros(max(L.workspace_bytes(M) for L in layers), dtype=torch.uint8, device=device)
    slim.workspace_init(ws)
    keep = [ws]
    if launch == "set":
        layer_set = slim.LayerSet(list(zip(layers, xs, ys)))
        keep.append(layer_set)
        run, checks, n_dom, n_kern = layer_set.run, [layer_set.check], 1, (1 if layer_set.info["resident_pairs"] > 0 else 2)
    elif launch == "per-layer":
        def run():
            for L, x, y in zip(layers, xs, ys):
                L.forward(x, ws, out=y)
        checks, n_dom, n_kern = [], len(layers), len(layers) * (2 if M >= 4 else 1)
    else:
        assert len(layers) % 7 == 0
        calls, checks, n_kern = [], [], 0
        for b0 in range(0, len(layers), 7):
            q, k, v, o, gate, up, down = range(b0, b0 + 7)
            qkv = slim.LayerSet([(layers[i], xs[q], ys[i]) for i in (q, k, v)])          # one input, three outputs
            gu = slim.LayerSet([(layers[i], xs[gate], ys[i]) for i in (gate, up)])
            keep += [qkv, gu]
            checks += [qkv.check, gu.check]
            calls += [qkv.run, (lambda i=o: layers[i].forward(xs[i], ws, out=ys[i])), gu.run,
                      (lambda i=down: layers[i].forward(xs[i], ws, out=ys[i]))]
            one = 1 if M < 4 else 2                                  # slim_mpq_gemv: from four tokens on a kernel stages x first
            n_kern += sum(1 if st.info["resident_pairs"] > 0 else 2 for st in (qkv, gu)) + 2 * one

        def run():
            for c in calls:
                c()
        n_dom = len(calls)
    graph = _graph_of(run, device)

    def check():
        slim.workspace_status(ws)
        for c in checks:
            c()
    return graph, keep, n_dom, n_kern, bufs, check


def decode_entry(name, layers, spec, device, timer, launch, steps, min_total_s, with_e2e=False, clock_gpu=None, warmup=5):
    """Measures one decode configuration; returns the dict that goes into the JSON line."""
    import torch
    M = spec["M"]
    graph, keep, n_dom, n_kern, bufs, check = decode_sweep(layers, M, device, launch)
    x_host, y_host, x_dev, y_dev, _, _ = bufs
    alg_bytes = sum(L.algorithmic_bytes(M) for L in layers)
    for _ in range(max(warmup, 3)):
        graph.replay()
    sampler = ClockSampler(clock_gpu) if clock_gpu is not None else None
    if sampler:
        sampler.start()
    ms_blocks = timer.blocks(graph.replay, steps, min_total_s)
    clocks = sampler.stop() if sampler else None
    check()
    tm = _timing_summary(ms_blocks, steps)
    ms = tm["ms_per_step_median"]
    value = timer.world * alg_bytes / (ms * 1e-3) / 1e9
    peak, peak_kind = measured_hbm_peak()
    per_launch_us = 1e3 * ms / n_dom
    achieved = alg_bytes / n_dom / (per_launch_us * 1e-6) / 1e9
    one = "gemv_one_kernel" if M == 1 else "gemv_kernel"      # slim_mpq_gemv's single-token kernel, or the general one
    kernel = {"set": "gemv_set_kernel", "per-layer": one, "decoder-order": "gemv_set_kernel + " + one}[launch]
    integer_form = M == 1
    out = {"name": name, "metric": f"mixed-precision dequant GEMV GB/s at M={M} ({spec['model']} layers, avg {spec['avg_bits']}-bit, g=128)",
           "value": value, "unit": UNIT, "ms_per_step": ms, "timing": tm,
           "dtype": ("s32 (mma.sync m16n8k32 u8 x s8: byte-masked code words against base-256 digits of fixed-point x; f32 fold)"
                     if integer_form and launch == "set" else
                     "s32 (mma.sync m16n8k32 u8 x s8 on byte-masked code words, f32 fold) in every call" if integer_form else
                     "f16 (mma.sync m16n8k16 on raw code fields, f32 accumulate)"),
           "config": {"workload": name, "layers": len(layers), "M": M, "avg_bits": spec["avg_bits"], "g": wl.GROUP,
                      "algorithmic_bytes_per_step": alg_bytes, "l2": f"distinct layers, {alg_bytes / 1e9:.2f} GB per step > L2",
                      "launch": {"set": "CUDA graph of the layer-set launch: one persistent kernel for the whole sweep (plus one kernel that stages x)",
                                 "per-layer": "CUDA graph of one slim_mpq_gemv launch per layer (the launch mode of App. B.2), programmatic dependent launch",
                                 "decoder-order": "CUDA graph; per block: set(q, k, v) on one x, o, set(gate, up) on one x, down: the calls a decoder can issue, in its order (at one token the q/k/v set is one resident launch, gate/up the ring)"}[launch],
                      "grouped_launch": launch != "per-layer"},
           "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_kind": peak_kind,
                        "kernel": kernel, "avg_launch_us": per_launch_us, "algorithmic_bytes_per_launch": alg_bytes / n_dom,
                        "frac_of_nominal_8000": achieved / NOMINAL_HBM_GBS},
           "gpu_launches_per_step": n_kern, "clocks": clocks}
    if with_e2e:
        def step_e2e():
            x_dev.copy_(x_host, non_blocking=True)
            graph.replay()
            y_host.copy_(y_dev, non_blocking=True)
            torch.cuda.current_stream().synchronize()
        for _ in range(3):
            step_e2e()
        e2e_steps = max(steps // 4, 3)
        ms_serial = float(np.median(timer.blocks(step_e2e, e2e_steps, min_total_s / 4))) / e2e_steps
        check()
        # The same steps as a pipeline, which is how a serving loop feeds the GPU: two sets of buffers (x, y, plan,
        # workspace) on two streams, step i on stream i mod 2, so the copies of one step run under the kernels of
        # the other.  Every step still copies its x from pinned host memory and its y back inside the timed region.
        graph2, keep2, _, _, bufs2, check2 = decode_sweep(layers, M, device, launch)
        lanes = [(torch.cuda.Stream(device), graph, x_dev, y_dev, y_host),
                 (torch.cuda.Stream(device), graph2, bufs2[2], bufs2[3], bufs2[1])]
        main = torch.cuda.current_stream()
        count = [0]

        def step_piped():
            side, g, xd, yd, yh = lanes[count[0] & 1]
            if count[0] < 2:
                side.wait_stream(main)              # not before the block's opening event
            count[0] += 1
            with torch.cuda.stream(side):
                xd.copy_(x_host, non_blocking=True)
                g.replay()
                yh.copy_(yd, non_blocking=True)

        def join():
            for lane in lanes:
                main.wait_stream(lane[0])
            count[0] = 0
        for _ in range(4):
            step_piped()
        join()
        torch.cuda.synchronize()
        ms_e2e = float(np.median(timer.blocks(step_piped, e2e_steps, min_total_s / 4, join=join))) / e2e_steps
        check()
        check2()
        assert torch.equal(y_host, bufs2[1]), "the two buffer sets of the pipeline disagree"
        out["e2e"] = {"value": timer.world * alg_bytes / (ms_e2e * 1e-3) / 1e9, "unit": UNIT, "h2d_bytes_per_step": int(x_host.numel() * 2),
                      "d2h_bytes_per_step": int(y_host.numel() * 2), "steps": e2e_steps, "ms_per_step": ms_e2e,
                      "how": "two buffer sets on two streams, step i on stream i mod 2: copies overlap the other step's kernels",
                      "one_step_at_a_time": {"value": timer.world * alg_bytes / (ms_serial * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": ms_serial,
                                             "how": "copy x in, run, copy y out, synchronise, every step"}}
        del graph2, keep2
    del graph, keep
    return out


def gemm_entry(name, layers, spec, device, timer, steps, min_total_s, with_e2e=False, clock_gpu=None, warmup=3):
    """Measures one batched (M > 16) configuration: TFLOP/s against the dense fp16 tensor peak."""
    import torch
    from paper_2405_14917_b200 import binding as slim
    M = spec["M"]
    x_host, y_host, x_dev, y_dev, xs, ys = decode_buffers(layers, M, device, 4321)
    ws = torch.zeros(max(L.workspace_bytes(M) for L in layers), dtype=torch.uint8, device=device)
    slim.workspace_init(ws)

    def run():
        for L, x, y in zip(layers, xs, ys):
            L.forward(x, ws, out=y)
    graph = _graph_of(run, device)
    for _ in range(max(warmup, 3)):
        graph.replay()
    sampler = ClockSampler(clock_gpu) if clock_gpu is not None else None
    if sampler:
        sampler.start()
    ms_blocks = timer.blocks(graph.replay, steps, min_total_s)
    clocks = sampler.stop() if sampler else None
    slim.workspace_status(ws)
    tm = _timing_summary(ms_blocks, steps)
    ms = tm["ms_per_step_median"]
    flops = sum(2.0 * M * L.N * L.K for L in layers)
    value = timer.world * flops / (ms * 1e-3) / 1e12
    peak, peak_kind = measured_tensor_peak()
    n_launch = len(layers)
    per_launch_us = 1e3 * ms / n_launch
    achieved = flops / n_launch / (per_launch_us * 1e-6) / 1e12
    sha = hashlib.sha256(open(os.path.join(ROOT, "paper_2405_14917_b200", "csrc", "slim_gemm.cu"), "rb").read()).hexdigest()
    cap = NCU_TRAFFIC_GEMM.get(sha)
    traffic = cap["traffic_bytes"] / cap["launches"] if cap and cap["workload"] == name and cap["launches"] == n_launch else None
    out = {"name": name, "metric": f"mixed-precision dequant GEMM TFLOP/s at M={M} (LLaMA-13B layer shapes, avg 3-bit, g=128)",
           "value": value, "unit": "TFLOP/s", "ms_per_step": ms, "timing": tm, "dtype": "f16 (tcgen05 kind::f16, f32 accumulate)",
           "config": {"workload": name, "layers": n_launch, "M": M, "avg_bits": spec["avg_bits"], "g": wl.GROUP, "flops_per_step": flops,
                      "l2": "14 distinct layers, 258 MB of weights per step > L2", "launch": "CUDA graph of one launch per layer"},
           "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak, "peak_kind": peak_kind,
                        "frac_of_burst": achieved / measured_tensor_burst(), "frac_of_nominal_2250": achieved / NOMINAL_TENSOR_TFLOPS,
                        "kernel": "gemm_kernel", "avg_launch_us": per_launch_us, "flops_per_launch": flops / n_launch, "traffic": traffic},
           "gpu_launches_per_step": n_launch, "clocks": clocks}
    if with_e2e:
        def step_e2e():
            x_dev.copy_(x_host, non_blocking=True)
            graph.replay()
            y_host.copy_(y_dev, non_blocking=True)
            torch.cuda.current_stream().synchronize()
        for _ in range(3):
            step_e2e()
        e2e_steps = max(steps // 4, 3)
        ms_e2e = float(np.median(timer.blocks(step_e2e, e2e_steps, min_total_s / 4))) / e2e_steps
        slim.workspace_status(ws)
        out["e2e"] = {"value": timer.world * flops / (ms_e2e * 1e-3) / 1e12, "unit": "TFLOP/s", "h2d_bytes_per_step": int(x_host.numel() * 2),
                      "d2h_bytes_per_step": int(y_host.numel() * 2), "steps": e2e_steps, "ms_per_step": ms_e2e}
    return out


def single_layer_entry(layer, device, timer, copies=64):
    """Config 1: one 4096 x 4096 layer at M = 1 through slim_mpq_gemv.  (a) latency of an isolated launch with a cold
    L2 (a 256 MB buffer is overwritten before every call); (b) throughput over `copies` distinct copies of the layer
    (303 MB > L2), one launch each, replayed from a CUDA graph; (c) the same copies as one layer-set launch."""
    import torch
    from paper_2405_14917_b200 import binding as slim
    M = 1
    clones = [slim.QuantLinear(layer.packed.clone(), layer.bits, layer.scales.clone(), layer.zeros.clone(), layer.N, layer.K) for _ in range(copies)]
    alg = layer.algorithmic_bytes(M)
    # (a)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
    ws = slim.new_workspace(M, layer.N, layer.K, layer.bits)
    x = torch.randn(M, layer.K, device=device).half()
    y = torch.empty(M, layer.N, dtype=torch.float16, device=device)
    lat = []
    for i in range(40):
        flush.fill_(i & 1)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        clones[i % copies].forward(x, ws, out=y)
        e1.record()
        torch.cuda.synchronize()
        lat.append(e0.elapsed_time(e1) * 1e3)
    slim.workspace_status(ws)
    del flush
    spec = dict(model="llama-7b", avg_bits=2, M=1)
    per_layer = decode_entry("single-4096x4096-avg2-m1-rotating-per-layer", clones, spec, device, timer, "per-layer", 20, 0.3)
    as_set = decode_entry("single-4096x4096-avg2-m1-rotating-set", clones, spec, device, timer, "set", 20, 0.3)
    peak, _ = measured_hbm_peak()
    return {"name": "single-4096x4096-avg2-m1", "metric": "one 4096 x 4096 layer, avg 2-bit, M = 1 (slim_mpq_gemv)",
            "isolated_launch_us": {"median": float(np.median(lat[5:])), "min": float(np.min(lat[5:])), "max": float(np.max(lat[5:])),
                                   "what": "one call timed with CUDA events around it, L2 flushed before every call, includes launch latency"},
            "isolated_launch_gbs": alg / (float(np.median(lat[5:])) * 1e-6) / 1e9,
            "ideal_us_at_measured_peak": alg / (peak * 1e9) * 1e6, "algorithmic_bytes": alg,
            "rotating_copies": copies, "rotating_per_layer": per_layer, "rotating_set": as_set}


def group_size_entries(device, timer):
    """One 4096 x 4096 layer, avg 2-bit, M = 1, at the group sizes of the paper's group-size ablation: 64 distinct copies
    (> L2) per step through slim_mpq_gemv, each made on the device from a seeded weight at that group size (salience ->
    bit allocation -> Eq. 1 -> packing)."""
    import torch
    from paper_2405_14917_b200 import binding as slim
    N = K = 4096
    copies = 64
    out = []
    gen = torch.Generator(device=device)
    gen.manual_seed(32)
    for g in (32, 64, 128, 256, 512):
        layers = []
        for i in range(copies):
            W, a = wl.make_weight_and_norms_device((32, g, i), N, K, device)
            layers.append(slim.QuantLinear.from_weight(W, a, 2, g=g))
            del W, a
        M = 1
        x = torch.randn(M, K, generator=gen, device=device).half()
        ys = [torch.empty(M, N, dtype=torch.float16, device=device) for _ in layers]
        ws = torch.zeros(max(L.workspace_bytes(M) for L in layers), dtype=torch.uint8, device=device)
        slim.workspace_init(ws)

        def run():
            for L, y in zip(layers, ys):
                L.forward(x, ws, out=y)
        graph = _graph_of(run, device)
        for _ in range(3):
            graph.replay()
        tm = _timing_summary(timer.blocks(graph.replay, 10, 0.3), 10)
        slim.workspace_status(ws)
        alg = sum(L.algorithmic_bytes(M) for L in layers)
        ms = tm["ms_per_step_median"]
        peak, peak_kind = measured_hbm_peak()
        achieved = alg / (ms * 1e-3) / 1e9
        out.append({"name": f"single-4096x4096-avg2-m1-g{g}", "metric": f"one 4096 x 4096 layer per launch, avg 2-bit, M = 1, group size {g} (slim_mpq_gemv, 64 rotating copies)",
                    "value": achieved, "unit": UNIT, "ms_per_step": ms, "timing": tm,
                    "kernel": "gemv_small_kernel (CUDA cores)" if g < 128 else "gemv_one_kernel (tensor cores)",
                    "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_kind": peak_kind,
                                 "avg_launch_us": 1e3 * ms / copies, "algorithmic_bytes_per_launch": alg / copies},
                    "config": {"workload": f"single-4096x4096-avg2-m1-g{g}", "g": g, "layers": copies, "algorithmic_bytes_per_step": alg,
                               "data": "synthetic weights quantised on the device at this group size"}})
        del layers, graph
        torch.cuda.empty_cache()
    return out


def cpu_baseline_legs(spec):
    """The oracle as it stands on the host cores: all cores (the reported baseline) and one core."""
    base = cpu_baseline(spec, budget_s=10.0)
    from oracle import slim_oracle_c as oc
    layers = _oracle_layers(spec, 1)
    L = layers[0]
    rows = 512
    codes, scales, zeros = L["codes"][:rows], np.ascontiguousarray(L["scales"][:, :rows]), np.ascontiguousarray(L["zeros"][:, :rows])
    oc.linear_f64(L["x"], codes, scales, zeros, threads=1)
    t0 = time.perf_counter()
    reps = 0
    while time.perf_counter() - t0 < 4.0:
        oc.linear_f64(L["x"], codes, scales, zeros, threads=1)
        reps += 1
    dt = time.perf_counter() - t0
    nbytes = wl.algorithmic_bytes(L["x"].shape[0], rows, L["K"], L["bits"]) * reps
    oc.linear_f64(L["x"], codes, scales, zeros, threads=base["cores"])          # back to all cores
    base["single_thread"] = {"value": nbytes / dt / 1e9, "unit": UNIT, "cores": 1,
                             "sample": f"first {rows} output rows of layer q, block 0, x {reps} passes, {dt:.1f} s"}
    return base


def secondary_entries(args, device, timer, primary_layers, clock_gpu):
    """The rest of the metric and of the configurations, each timed for about a second, for the same JSON line."""
    import torch
    out = []

    def guarded(fn):
        try:
            out.append(fn())
        except Exception as e:               # a secondary entry never takes the primary line down
            out.append({"name": getattr(fn, "__name__", "entry"), "error": f"{type(e).__name__}: {e}"})
        torch.cuda.empty_cache()

    spec7 = workload_spec("llama7b-decode-avg2")
    guarded(lambda: decode_entry("llama7b-decode-avg2-m1-per-layer", primary_layers, spec7, device, timer, "per-layer", 50, 0.5, clock_gpu=clock_gpu))
    guarded(lambda: decode_entry("llama7b-decode-avg2-m1-decoder-order", primary_layers, spec7, device, timer, "decoder-order", 50, 0.5, clock_gpu=clock_gpu))
    guarded(lambda: single_layer_entry(primary_layers[0], device, timer))
    try:
        out.extend(group_size_entries(device, timer))
    except Exception as e:
        out.append({"name": "group sizes", "error": f"{type(e).__name__}: {e}"})
    torch.cuda.empty_cache()
    for wname in ("llama13b-prefill-avg3-m2048", "llama13b-prefill-avg3-m512", "llama13b-prefill-avg3-m128"):
        spec = workload_spec(wname)
        layers13 = build_layers(spec, device, 0) if wname.endswith("m2048") else layers13
        guarded(lambda: gemm_entry(wname, layers13, spec, device, timer, 20, 1.0 if spec["M"] >= 512 else 0.5, clock_gpu=clock_gpu))
    del layers13
    torch.cuda.empty_cache()
    spec3 = workload_spec("llama7b-decode-avg3-m1-blocks8")
    layers3 = build_layers(spec3, device, 0)
    for M in (1, 4, 8, 16, 32, 64):
        sp = dict(spec3, M=M)
        guarded(lambda: decode_entry(f"llama7b-decode-avg3-m{M}-blocks8", layers3, sp, device, timer, "set", 50, 0.6, clock_gpu=clock_gpu))
    del layers3
    torch.cuda.empty_cache()
    spec70 = workload_spec("llama70b-decode-avg2-m1")
    layers70 = build_layers(spec70, device, 0)
    for M in (1, 16):
        sp = dict(spec70, M=M)
        guarded(lambda: decode_entry(f"llama70b-decode-avg2-m{M}-blocks8", layers70, sp, device, timer, "set", 20, 0.6, clock_gpu=clock_gpu))
    guarded(lambda: decode_entry("llama70b-decode-avg2-m1-blocks8-per-layer", layers70, dict(spec70, M=1), device, timer, "per-layer", 20, 0.5, clock_gpu=clock_gpu))
    del layers70
    torch.cuda.empty_cache()
    return out


def run_ours(args, spec):
    import torch
    import torch.distributed as dist
    from paper_2405_14917_b200 import binding as slim

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    steps = args.steps if args.steps is not None else (200 if spec["M"] <= 16 else 50)
    warmup = max(args.warmup if args.warmup is not None else 20, 3)
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    slim.lib()   # fails loudly if the CUDA library is missing
    timer = Timer(device, world)
    layers = build_layers(spec, device, rank)
    M = spec["M"]
    clock_gpu = local_rank if rank == 0 else None
    launch = "set" if (M <= slim.GEMV_MAX_M and args.launch == "set") else "per-layer"
    if M > slim.GEMV_MAX_M:
        entry = gemm_entry(args.workload, layers, spec, device, timer, steps, args.min_seconds, with_e2e=True, clock_gpu=clock_gpu, warmup=warmup)
    else:
        entry = decode_entry(args.workload, layers, spec, device, timer, launch if args.launch != "decoder-order" else "decoder-order",
                             steps, args.min_seconds, with_e2e=True, clock_gpu=clock_gpu, warmup=warmup)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    tm = entry["timing"]
    line = {"metric": METRIC if args.workload == "llama7b-decode-avg2" else entry["metric"],
            "value": entry["value"], "unit": entry["unit"], "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": entry["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": entry["dtype"], "data": "synthetic",
            "config": dict(entry["config"], parallelism=f"replicas x{world}",
                           timing=f"median of {tm['blocks']} blocks of exactly {steps} steps each (barrier + synchronize around every block)"),
            "timing": tm, "roofline": entry["roofline"], "e2e": entry["e2e"],
            "gpu_launches": steps * tm["blocks"] * entry["gpu_launches_per_step"], "clocks": entry["clocks"]}
    if M <= slim.GEMV_MAX_M and launch == "set":
        traffic = NCU_TRAFFIC.get(set_kernel_hash())
        line["roofline"]["traffic"] = (traffic["traffic_bytes"] / traffic["algorithmic_bytes"] * entry["roofline"]["algorithmic_bytes_per_launch"]) if traffic else None
    elif "traffic" not in line["roofline"]:
        line["roofline"]["traffic"] = None
    if world == 1 and args.workload == "llama7b-decode-avg2" and not args.no_secondary:
        line["secondary"] = secondary_entries(args, device, timer, layers, clock_gpu)
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline_legs(spec) if M <= slim.GEMV_MAX_M else cpu_baseline(spec)
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
    ap.add_argument("--launch", default="set", choices=["set", "per-layer", "decoder-order"],
                    help="decode workloads (M <= 16): the layer-set launch (one persistent kernel for the sweep), one launch per layer, "
                         "or the calls a decoder can issue (per block: q/k/v as a set, o, gate/up as a set, down)")
    ap.add_argument("--min-seconds", type=float, default=1.0,
                    help="blocks of --steps steps are repeated until this much timed work has run; the median block is reported")
    ap.add_argument("--no-secondary", action="store_true", help="default workload only: skip the other configurations of the same JSON line")
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
