#!/usr/bin/env python
"""Benchmark of the gradient evaluation (forward products, fused epilogues, delta products, weight-gradient
products with their fixed-order reduction, then the plain step W -= lr*grad) on synthetic data shaped like
the paper's 400-480-3203 character-recognition network.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--math 3xtf32|tf32|simt|bf16] [--workload config3|config1|config4|config5]
    python bench.py --workload scale_small|scale_jocr|scale_worker [--scaling weak|strong]    # Section 6.3's three cases
    python bench.py --workload sgemm | peaks
    python bench.py --impl reference ...      # times the CPU checker on the host cores instead

One "step" = one error-and-gradient evaluation of one batch plus the parameter step.  Flops are counted with the
paper's formula n_p*(4*n_i*n_h + 6*n_h*n_o) (Section 6.2), 2 per multiply-add, nothing else counted.
Prints ONE JSON line on rank 0.
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

WORKLOADS = {
    # name: (sizes, patterns per GPU, seed)
    "config1": ([256, 128, 64], 4096, 0),
    "config3": ([400, 480, 3203], 65536, 2),
    "config5": ([1024, 4096, 4096, 3203], 131072, 4),
    # one step = one pass over 9,000,000 resident patterns in 131072-pattern chunks accumulated in a fixed order
    # (Section 4.3), then the parameter step; use --steps 5 or so (a step takes about half a second)
    "config4": ([400, 480, 3203], 9_000_000, 3),
    # the three workloads of the processor-scaling experiment (Section 6.3): a small network on 40,960 patterns and the
    # character network on 163,480 patterns, both with the total fixed while workers are added, and the character
    # network with 32,000 patterns per worker
    "scale_small": ([400, 80, 200], 40_960, 5),
    "scale_jocr": ([400, 480, 3203], 163_480, 6),
    "scale_worker": ([400, 480, 3203], 32_000, 7),
}
DEFAULT_SCALING = {"scale_small": "strong", "scale_jocr": "strong"}       # everything else: patterns per GPU fixed
CHUNK = {"config4": 131072}
MATH = {"3xtf32": 0, "tf32": 1, "simt": 2, "bf16": 3}
NOMINAL_TF32_OVER_BF16 = 0.5        # dense TF32 tensor rate is half the BF16 rate
# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture) of the products that can be the
# dominant kernel, captured on a smaller batch and scaled by the pattern count, to which these products' traffic is
# proportional.  Reported only while the library still is the version the counters were taken on; null otherwise.
NCU_TRAFFIC = {
    "library_version": 109,
    # captured at 16384 patterns (x4); in 16-bit mode at 32768 patterns (x2)
    ("config3", "3xtf32", (3203, 481, 65536)): 4 * (302.14912e6 + 22.673664e6),
    ("config3", "3xtf32", (65536, 480, 3203)): 4 * (310.02726e6 + 23.085568e6),
    ("config3", "3xtf32", (65536, 3203, 480)): 4 * (77.086720e6 + 166.95372e6),
    ("config3", "tf32", (65536, 3203, 480)): 4 * (39.002112e6 + 162.37900e6),
    ("config3", "tf32", (65536, 480, 3203)): 4 * (256.99609e6 + 22.658560e6),
    ("config3", "tf32", (3203, 481, 65536)): 4 * (250.86515e6 + 21.920000e6),
    ("config3", "bf16", (65536, 3203, 480)): 2 * (38.447872e6 + 175.91628e6),
    ("config3", "bf16", (65536, 480, 3203)): 2 * (249.72902e6 + 20.953344e6),
    ("config3", "bf16", (3203, 481, 65536)): 2 * (253.34092e6 + 21.497088e6),
}
# cuBLAS through torch.matmul, 8192^3, on this machine's B200s (`--workload peaks`): TF32 allowed, best of 10 isolated
# calls and 4 s back to back under the power cap (SM clock 1042 MHz of 1965).  Printed beside the peak the fractions use.
TF32_CUBLAS_MEASURED = {"burst_tflops": 719.2, "sustained_tflops": 600.9}
NOMINAL_TFLOPS = {"tf32": 1100.0, "bf16": 2250.0}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) >= 7:
                self.rows.append(parts)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        if self.thread:
            self.thread.join(timeout=2)
        sm, mx, reasons = [], None, set()
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx = float(r[1])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def cpu_baseline(sizes, seed, n_sample, head="softmax", offset=0):
    """The CPU checker, as it stands, on n_sample patterns of the workload starting at `offset`.  Returns the record
    and the checker's (loss, dW, db)."""
    import oracle
    import synth_inputs as si
    from paper_1911_05181_b200 import flops
    Ws, bs = si.mlp_params(seed, sizes)
    X, y = si.mlp_batch(seed, sizes, n_sample, offset=offset)
    T = si.mlp_targets(seed, sizes, n_sample, offset) if head == "sse" else None
    t0 = time.perf_counter()
    if head == "sse":
        ref = oracle.mlp_sse_gradient(Ws, bs, X, T)
    else:
        ref = oracle.mlp_gradient(Ws, bs, X, y)
    dt = time.perf_counter() - t0
    rec = {"value": flops.gradient_flops(sizes, n_sample) / dt / 1e9, "unit": "GFLOP/s", "cores": oracle.num_threads(),
           "kind": "oracle", "sample": "first %d patterns of the batch, one gradient evaluation, %.1f s" % (n_sample, dt),
           "patterns_per_s": n_sample / dt}
    return rec, ref


def run_reference(args):
    """--impl reference: the CPU checker on the host cores, same metric and config, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    import synth_inputs as si
    from paper_1911_05181_b200 import flops
    sizes, batch, seed = WORKLOADS[args.workload]
    if args.patterns > 0:
        batch = args.patterns
    n_sample = min(batch, 1024 if args.workload != "config5" else 128)
    Ws, bs = si.mlp_params(seed, sizes)
    X, y = si.mlp_batch(seed, sizes, n_sample)
    for _ in range(args.warmup):
        oracle.mlp_gradient(Ws, bs, X, y)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        loss, dW, db = oracle.mlp_gradient(Ws, bs, X, y)
        for w, g in zip(Ws + bs, dW + db):          # the parameter step, on a copy, so that every step sees the same weights
            oracle.sgd_step(w.ravel(), g.astype("float32").ravel(), 1e-3 / n_sample)
    dt = (time.perf_counter() - t0) / args.steps
    val = flops.gradient_flops(sizes, n_sample) / dt / 1e9
    sample = "%d of %d patterns per step (work is additive over patterns)" % (n_sample, batch)
    line = {
        "impl": "reference", "metric": "gradient_eval_gflops", "value": val, "unit": "GFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "%s: %s MLP, %d patterns, seed %d" % (args.workload, "-".join(map(str, sizes)), batch, seed),
                   "sample": sample},
        "patterns_per_s": n_sample / dt,
        "cpu_baseline": {"value": val, "unit": "GFLOP/s", "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "GFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


SGEMM_SWEEP = [  # (transA, transB, M, N, K): the standalone-SGEMM configuration (Section 3.4's experiment, restaged)
    ("N", "N", 256, 256, 256), ("N", "N", 1024, 1024, 1024), ("N", "N", 4096, 4096, 4096), ("N", "N", 8192, 8192, 8192),
    ("N", "T", 4096, 4096, 4096), ("T", "N", 4096, 4096, 4096), ("T", "T", 4096, 4096, 4096),
    ("N", "T", 65536, 480, 400), ("N", "T", 65536, 3203, 480), ("N", "N", 65536, 3203, 480), ("T", "N", 480, 3203, 65536),
]


def run_sgemm_sweep(args):
    """--workload sgemm: C = A*B (alpha 1, beta 0) over the sweep, device-resident operands uniform [-1,1), seed 1.
    Leading dimensions are packed, so the operands with rows of 3203 floats cannot be addressed by TMA: the library
    re-buffers them into the workspace first (Section 3.3), inside the timed call.  Calls are isolated (a buffer larger
    than L2 is overwritten between them), so the fractions are of the burst peak.  Prints one JSON line; `value` is the
    8192^3 rate."""
    import torch
    import synth_inputs as si
    from paper_1911_05181_b200 import binding as ul
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    if int(os.environ.get("RANK", "0")) != 0:
        return 0
    math_mode = MATH[args.math]
    peaks = load_peaks()
    tp = tensor_peaks(peaks, args.math == "bf16")
    mult = 3.0 if args.math == "3xtf32" else 1.0
    stream = torch.cuda.current_stream()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")          # > L2: written between timed calls
    rows = []
    for ta, tb, M, N, K in SGEMM_SWEEP:
        ra, ca = (K, M) if ta == "T" else (M, K)
        rb, cb = (N, K) if tb == "T" else (K, N)
        A = torch.empty(ra, ca, device="cuda"); B = torch.empty(rb, cb, device="cuda"); C = torch.empty(M, N, device="cuda")
        ul.fill_uniform(A, A.numel(), 1, si.TID_GEMM_A, 0, 1); ul.fill_uniform(B, B.numel(), 1, si.TID_GEMM_B, 0, 1)
        nbytes = ul.sgemm_workspace_bytes_for(ta, tb, M, N, K, A, ca, B, cb, math_mode)
        ws = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
        wp = (ws.data_ptr() + 255) // 256 * 256

        def call():
            ul.sgemm_ex(ta, tb, M, N, K, 1.0, A, ca, B, cb, 0.0, C, N, math_mode, wp if nbytes else None, nbytes)

        for _ in range(3):
            call()
        torch.cuda.synchronize()
        time.sleep(0.5)           # isolated calls: the clocks recover from the previous shape's load (a 3xTF32 8192^3
                                  # product pulls the GPU to its power cap and the next shape would run ~15 % slower)
        reps = 20 if M * N * K < (1 << 34) else 8
        times = []
        for _ in range(reps):
            time.sleep(0.02)
            flush.fill_(1)                                                     # cold L2, as the paper flushed its caches
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record(stream); call(); e1.record(stream)
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        ms = statistics.median(times)
        tf = 2.0 * M * N * K / (ms * 1e-3) / 1e12
        rows.append({"form": ta + tb, "M": M, "N": N, "K": K, "ms": round(ms, 4), "logical_tflops": round(tf, 2),
                     "workspace_mb": round(nbytes / 1e6, 1),
                     "tensor_pipe_frac_of_burst": round(mult * tf / tp["burst"], 3) if args.math != "simt" else None,
                     "tensor_pipe_frac_of_sustained": round(mult * tf / tp["sustained"], 3) if args.math != "simt" else None})
        del A, B, C, ws
    big = [r for r in rows if r["M"] == 8192][0]
    line = {"metric": "sgemm_gflops", "value": big["logical_tflops"] * 1e3, "unit": "GFLOP/s", "n_gpus": 1, "steps": 8,
            "warmup": 3, "ms_per_step": big["ms"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if args.math == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": "sgemm sweep (alpha 1, beta 0, uniform [-1,1), seed 1); value = NN 8192^3", "math": args.math,
                       "l2": "a 256 MB buffer is overwritten between timed calls"},
            "sweep": rows, "peak_burst_tflops": tp["burst"], "peak_sustained_tflops": tp["sustained"], "peak_source": tp["source"],
            "tf32_cublas_measured": None if args.math == "bf16" else TF32_CUBLAS_MEASURED,
            "gpu_launches": int(sum(ul.launch_counts().values()))}
    print(json.dumps(line))
    return 0


def run_peaks(args):
    """--workload peaks: the denominators measured directly on this GPU with library routines (never on the library's
    own path): torch.matmul 8192^3 with TF32 allowed and in bf16, each as the best of 10 isolated calls (burst) and
    back to back for 4 s (sustained, under the power cap), with the SM clock sampled during the sustained loop."""
    import torch
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    if int(os.environ.get("RANK", "0")) != 0:
        return 0
    n = 8192
    out = {"workload": "peaks", "n": n, "nominal_tf32_tflops": 1100.0, "nominal_bf16_tflops": 2250.0}
    for name, dtype, tf32 in (("tf32", torch.float32, True), ("bf16", torch.bfloat16, False)):
        torch.backends.cuda.matmul.allow_tf32 = tf32
        a = torch.randn(n, n, device="cuda", dtype=dtype); b = torch.randn(n, n, device="cuda", dtype=dtype)
        c = torch.empty(n, n, device="cuda", dtype=dtype)
        for _ in range(3):
            torch.matmul(a, b, out=c)
        torch.cuda.synchronize()
        best = float("inf")
        for _ in range(10):
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record(); torch.matmul(a, b, out=c); e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
            time.sleep(0.05)
        sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")))
        sampler.start()
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        reps = 0
        t0 = time.perf_counter()
        e0.record()
        while time.perf_counter() - t0 < 4.0:
            for _ in range(20):
                torch.matmul(a, b, out=c)
            reps += 20
            torch.cuda.synchronize()
        e1.record()
        torch.cuda.synchronize()
        clocks = sampler.stop()
        out[name] = {"burst_tflops": 2.0 * n ** 3 / (best * 1e-3) / 1e12,
                     "sustained_tflops": 2.0 * n ** 3 * reps / (e0.elapsed_time(e1) * 1e-3) / 1e12,
                     "sustained_clocks": clocks}
        time.sleep(1.0)
    torch.backends.cuda.matmul.allow_tf32 = False
    print(json.dumps(out))
    return 0


def tensor_peaks(peaks, half):
    """Tensor peaks of the mode's operand type from the measured bf16 cuBLAS rates: as measured for the 16-bit mode,
    halved (the nominal TF32 : BF16 ratio) for the TF32 modes.  burst: isolated calls at the full SM clock;
    sustained: seconds of back-to-back calls under the power cap."""
    f = 1.0 if half else NOMINAL_TF32_OVER_BF16
    mx = float(peaks.get("sm_max_mhz") or 1965.0)
    under_load = float((peaks.get("clocks_under_load") or {}).get("sm_mhz_median") or 1357.0)
    return {"burst": peaks["bf16_tflops"] * f, "sustained": peaks["bf16_tflops_sustained"] * f,
            "burst_clock_mhz": mx, "sustained_clock_mhz": under_load,
            "source": "%s cuBLAS bf16%s" % (peaks["_source"], "" if half else " x 0.5 (nominal TF32:BF16)")}


def fractions(achieved, tp, timed_region_ms, sm_mhz):
    """The fraction the run is held to: of the burst peak when the timed region is shorter than a second (the clocks
    have not come down under the power cap yet), of the sustained peak otherwise; both are printed.  The clock-normalised
    fraction divides by the peak scaled to the median SM clock sampled during the run."""
    which = "burst" if timed_region_ms < 1000.0 else "sustained"
    out = {"peak": tp[which], "peak_kind": which, "frac": achieved / tp[which],
           "peak_burst": tp["burst"], "frac_of_burst": achieved / tp["burst"],
           "peak_sustained": tp["sustained"], "frac_of_sustained": achieved / tp["sustained"],
           "peak_source": tp["source"]}
    if sm_mhz:
        scaled = tp[which] * float(sm_mhz) / tp[which + "_clock_mhz"]
        out["frac_clock_normalised"] = achieved / scaled
        out["clock_normalised_how"] = "peak x %.0f MHz (median SM clock of this run) / %.0f MHz (clock of the peak's measurement)" % (
            float(sm_mhz), tp[which + "_clock_mhz"])
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--math", default="3xtf32", choices=sorted(MATH))
    ap.add_argument("--workload", default="config3", choices=sorted(WORKLOADS) + ["sgemm", "peaks"])
    ap.add_argument("--head", default="softmax", choices=["softmax", "sse"],
                    help="softmax + cross-entropy on labels (the benchmark's workload) or the paper's tanh outputs with "
                         "summed squared error on a dense target matrix")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--scaling", default=None, choices=["weak", "strong"],
                    help="several GPUs: weak = the workload's pattern count per GPU, strong = that count in total, divided "
                         "over the GPUs (default: strong for scale_small and scale_jocr, weak otherwise)")
    ap.add_argument("--total-patterns", type=int, default=0, help="strong scaling: total pattern count instead of the workload's")
    ap.add_argument("--exchange", default="allreduce", choices=["allreduce", "ordered"],
                    help="gradient exchange over several GPUs: NCCL all-reduce, or all-gather + sum in rank order")
    ap.add_argument("--overlap", default="on", choices=["on", "off"],
                    help="several GPUs: start the exchange of a layer's gradient as soon as it is final, on a second stream, "
                         "while the products of the layers below still run (Section 5.2), or exchange after the last product")
    ap.add_argument("--e2e-gradient", action="store_true",
                    help="end-to-end leg: copy the gradient (not only the loss) back to the host every step")
    ap.add_argument("--patterns", type=int, default=0,
                    help="patterns per GPU instead of the workload's own count (for profiler captures of a smaller case)")
    args = ap.parse_args()
    if args.workload == "peaks":
        return run_peaks(args) if args.impl == "ours" else 0
    if args.workload == "sgemm":
        return run_sgemm_sweep(args) if args.impl == "ours" else 0
    if args.impl == "reference":
        return run_reference(args)

    import numpy as np
    import torch
    import synth_inputs as si
    from paper_1911_05181_b200 import binding as ul, dp, flops

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    ul.lib()                                       # raises if the CUDA library is not built: there is no other path

    sizes, count, seed = WORKLOADS[args.workload]
    if args.patterns > 0:
        count = args.patterns
    scaling = args.scaling or DEFAULT_SCALING.get(args.workload, "weak")
    math_mode = MATH[args.math]
    L = len(sizes) - 1
    # Section 4.3: the patterns are partitioned, the parameters replicated.  Weak scaling: every rank evaluates `count`
    # patterns, slice [rank*count, (rank+1)*count) of one seeded stream.  Strong scaling: a fixed set of patterns is
    # divided as evenly as possible (the first ranks get one more when it does not divide).
    if scaling == "strong":
        total = args.total_patterns if args.total_patterns > 0 else count
        first, last = dp.split_range(total, world, rank)
    else:
        total = count * world
        first, last = dp.shard_range(rank, world, count)
    batch = last - first
    per_rank = [(lambda fl: fl[1] - fl[0])(dp.split_range(total, world, r) if scaling == "strong" else dp.shard_range(r, world, count))
                for r in range(world)]
    Ws, bs = si.mlp_params(seed, sizes)
    W = [torch.from_numpy(w).cuda() for w in Ws]
    b = [torch.from_numpy(v).cuda() for v in bs]
    W0 = [w.clone() for w in W]; b0 = [v.clone() for v in b]
    dW = [torch.empty_like(w) for w in W]; db = [torch.empty_like(v) for v in b]
    loss = torch.zeros(1, dtype=torch.float64, device="cuda")
    X = torch.empty(batch, sizes[0], device="cuda"); y = torch.empty(batch, dtype=torch.int32, device="cuda")
    ul.fill_uniform(X, X.numel(), seed, si.TID_X, first * sizes[0], 0)
    ul.fill_labels(y, batch, seed, si.TID_LABELS, first, sizes[-1])
    if args.head == "sse":       # dense targets uniform [-1, 1) in place of the labels
        y = torch.empty(batch, sizes[-1], device="cuda")
        ul.fill_uniform(y, y.numel(), seed, si.TID_TARGETS, first * sizes[-1], 1)
    Xh = torch.empty(batch, sizes[0], pin_memory=True); yh = torch.empty(y.shape, dtype=y.dtype, pin_memory=True)
    Xh.copy_(X); yh.copy_(y)
    loss_h = torch.zeros(1, dtype=torch.float64, pin_memory=True)
    grad_h = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in dW + db] if args.e2e_gradient else []
    chunk = min(batch, CHUNK.get(args.workload, batch))
    starts = list(range(0, batch, chunk))
    net = ul.Mlp(sizes, math_mode, chunk)
    lr = 1e-3 / total
    stream = torch.cuda.current_stream()
    # The exchange of the method (Section 4.3): the per-rank gradients and losses are summed.  With --overlap on, the
    # library records an event per layer when that layer's gradient is final (the top layer's first), and the
    # exchange of that layer starts on a second stream while the products below it still run.
    overlap = world > 1 and args.overlap == "on" and len(starts) == 1
    exchange = dp.GradientExchange(dW + db, dist, ordered=args.exchange == "ordered",
                                   groups=dp.layer_groups(L) if overlap else None)
    xstream = torch.cuda.Stream() if overlap else None
    layer_events = None
    if overlap:
        layer_events = [torch.cuda.Event() for _ in range(L)]
        for e in layer_events:
            e.record(stream)                        # an event exists once it has been recorded
        net.set_gradient_events(layer_events)

    def gradient(Xd, yd, lo, hi, acc):
        if args.head == "sse":
            net.gradient_sse(W, b, Xd[lo:hi], sizes[0], yd[lo:hi], sizes[-1], hi - lo, acc, dW, db, loss)
        else:
            net.gradient(W, b, Xd[lo:hi], sizes[0], yd[lo:hi], hi - lo, acc, dW, db, loss)

    def step(Xd, yd, host=None):
        for i, lo in enumerate(starts):
            hi = min(batch, lo + chunk)
            if host is not None:            # end-to-end leg: this chunk's patterns come from pinned host memory
                Xd[lo:hi].copy_(host[0][lo:hi], non_blocking=True); yd[lo:hi].copy_(host[1][lo:hi], non_blocking=True)
            gradient(Xd, yd, lo, hi, i > 0)
        if overlap:
            with torch.cuda.stream(xstream):
                for g in range(L):                  # group g = layer L-1-g, in the order the library finishes them
                    xstream.wait_event(layer_events[L - 1 - g])
                    exchange.start(g, dW + db)
                exchange.finish(dW + db, loss)
            stream.wait_stream(xstream)
        else:
            exchange.all_reduce(dW + db, loss)
        net.sgd_step(W, b, dW, db, lr)

    def reset_params():
        for w, w0 in zip(W + b, W0 + b0):
            w.copy_(w0)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        barrier()
        ms = e0.elapsed_time(e1)
        if world > 1:
            t = torch.tensor([ms], device="cuda"); dist.all_reduce(t, op=dist.ReduceOp.MAX); ms = float(t.item())
        return ms / steps

    # ---- device-resident throughput (inputs already in HBM; X 105 MB, logits 840 MB: far larger than the 126 MB L2)
    for _ in range(max(args.warmup, 3)):
        step(X, y)
    reset_params()
    net.enable_timing(True)
    c0 = ul.launch_counts()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.start()
    ms_step = timed(lambda: step(X, y), args.steps)
    clocks = sampler.stop() if sampler else None
    c1 = ul.launch_counts()
    phases = net.phase_times()
    net.enable_timing(False)
    status = net.last_device_status()
    launches = sum(c1[k] - c0[k] for k in c1)

    # ---- the same evaluation twice from the same parameters: every bit of the loss and of the gradient must repeat
    reset_params()
    bitwise = True
    first_run = None
    for _ in range(2):
        for i, lo in enumerate(starts):
            gradient(X, y, lo, min(batch, lo + chunk), i > 0)
        torch.cuda.synchronize()
        cur = [loss.clone()] + [t.clone() for t in dW + db]
        if first_run is None:
            first_run = cur
        else:
            bitwise = all(torch.equal(u.view(torch.uint8), v.view(torch.uint8)) for u, v in zip(first_run, cur))
    del first_run

    # ---- end to end through the public call: inputs from pinned host memory every step, loss read back every step
    reset_params()

    def read_back():
        loss_h.copy_(loss, non_blocking=True)
        for hbuf, t in zip(grad_h, dW + db):
            hbuf.copy_(t, non_blocking=True)

    def e2e_step():
        step(X, y, host=(Xh, yh))
        read_back()

    if len(starts) == 1:
        # Double-buffered: while step i computes on one device buffer, a copy stream brings step i+1's batch from
        # pinned host memory into the other.  Every step still pays for its own host-to-device copy and reads its
        # loss back; the timed region starts before the first copy and ends after the last read-back.
        copy_stream = torch.cuda.Stream()
        bufs = [(X, y), (torch.empty_like(X), torch.empty_like(y))]
        copied = [torch.cuda.Event() for _ in range(2)]
        freed = [torch.cuda.Event() for _ in range(2)]

        def prefetch(i):
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(freed[i % 2])
                bufs[i % 2][0].copy_(Xh, non_blocking=True); bufs[i % 2][1].copy_(yh, non_blocking=True)
                copied[i % 2].record(copy_stream)

        def run_e2e(steps):
            for ev in freed:
                ev.record(stream)
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            barrier()
            e0.record(stream)
            copy_stream.wait_event(e0)
            prefetch(0)
            for i in range(steps):
                stream.wait_event(copied[i % 2])
                if i + 1 < steps:
                    prefetch(i + 1)
                step(*bufs[i % 2])
                freed[i % 2].record(stream)
                read_back()
            e1.record(stream)
            barrier()
            ms = e0.elapsed_time(e1)
            if world > 1:
                t = torch.tensor([ms], device="cuda"); dist.all_reduce(t, op=dist.ReduceOp.MAX); ms = float(t.item())
            return ms / steps

        run_e2e(2)
        reset_params()
        ms_e2e = run_e2e(args.steps)
        e2e_mode = "double-buffered host-to-device copies on a second stream"
    else:
        for _ in range(2):
            e2e_step()
        reset_params()
        ms_e2e = timed(e2e_step, args.steps)
        e2e_mode = "each chunk copied from pinned host memory right before it is evaluated"

    gflop_step = flops.gradient_flops(sizes, total) / 1e9
    value = gflop_step / (ms_step * 1e-3)
    e2e_value = gflop_step / (ms_e2e * 1e-3)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    # ---- roofline of the dominant product (largest share of the step)
    peaks = load_peaks()
    half = args.math == "bf16"
    tp = tensor_peaks(peaks, half)
    sm_mhz = (clocks or {}).get("sm_mhz")
    region_ms = ms_step * args.steps
    dom = max(range(len(phases)), key=lambda i: phases[i][0]) if phases else None
    roofline = None
    if dom is not None:
        ms_k, M, N, K = phases[dom]
        logical = 2.0 * M * N * K
        counts = ul.launch_counts()
        on_tensor = args.math != "simt" and counts["tc_gemm"] > 0
        if on_tensor:
            mult = 3.0 if args.math == "3xtf32" else 1.0
            esize = 2.0 if half else 4.0
            achieved = mult * logical / (ms_k * 1e-3) / 1e12
            # What the product must move, as the path lays its operands out: both operands once, the output once
            # (split-K partials for a weight-gradient product, whose K is the pattern count), and for a delta product
            # (phases L .. 2L-2) the hidden activations its tanh' epilogue reads; operands kept as TF32 (hi, lo) pairs in
            # 3xTF32 mode (weights, hidden activations) count twice.
            pair = 2.0 if args.math == "3xtf32" else 1.0
            is_delta = L <= dom < 2 * L - 1
            is_wgrad = dom >= 2 * L - 1
            if dom < L:                 # forward: A = batch or activations (pair from the second layer on), B = weights (pair)
                alg = esize * (M * K * (pair if dom >= 1 else 1.0) + K * N * pair) + esize * M * N * (pair if dom < L - 1 else 1.0)
            elif is_delta:              # A = stored exponentials / deltas, B = weights (pair), epilogue reads H (pair), writes delta
                alg = esize * (M * K + K * N * pair) + esize * M * N * pair + esize * M * N
            else:                       # A = exponentials / deltas, B = activations (pair) or the batch; output: the slices' partial products
                w = L - 1 - (dom - (2 * L - 1))
                splits = max(1, -(-K // 4096)) if not half else max(1, -(-K // 8192))
                alg = esize * (M * K + K * N * (pair if w >= 1 else 1.0)) + 4.0 * M * N * splits
            roofline = {"bound": "tensor", "achieved": achieved, "unit": "TFLOP/s"}
            roofline.update(fractions(achieved, tp, region_ms, sm_mhz))
            roofline.update({
                "traffic": (NCU_TRAFFIC.get((args.workload, args.math, (M, N, K)))
                            if ul.version() == NCU_TRAFFIC["library_version"] and args.patterns <= 0 else None),
                "algorithmic_bytes": alg,
                "kernel": "%s M=%d N=%d K=%d" % ("bf16_gemm" if half else "tc_gemm", M, N, K), "ms": ms_k,
                "flops_counted": "%gx 2MNK" % mult, "logical_tflops": logical / (ms_k * 1e-3) / 1e12,
                "nominal_peak": NOMINAL_TFLOPS["bf16" if half else "tf32"],
                "frac_of_nominal": achieved / NOMINAL_TFLOPS["bf16" if half else "tf32"],
                "tf32_cublas_measured": None if half else TF32_CUBLAS_MEASURED})
        else:
            mhz = sm_mhz or peaks.get("sm_max_mhz", 1965.0)
            peak = 148 * 128 * 2 * mhz * 1e6 / 1e12      # FFMA lanes x 2 flops x clock seen during the run
            achieved = logical / (ms_k * 1e-3) / 1e12
            roofline = {"bound": "alu", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                        "traffic": None, "kernel": "simt_gemm M=%d N=%d K=%d" % (M, N, K), "ms": ms_k,
                        "peak_source": "148 SMs x 128 FFMA lanes x 2 x %.0f MHz (median SM clock of this run)" % mhz}
    gemm_ms = sum(p[0] for p in phases)

    # ---- the CPU checker on a sample of the same workload: its rate, and the GPU's error against it on that sample
    cpu = None
    accuracy = {"bitwise_repeat": bool(bitwise), "rel_l2": None}
    if not args.no_cpu_baseline:
        n_sample = min(batch, {"config1": 4096, "config5": 1024}.get(args.workload, 16384))
        cpu, ref = cpu_baseline(sizes, seed, n_sample, args.head, first)
        reset_params()
        gradient(X, y, 0, n_sample, False)
        torch.cuda.synchronize()
        import oracle
        names = ["dW%d" % l for l in range(L)] + ["db%d" % l for l in range(L)]
        errs = {nm: oracle.rel_l2(t.cpu().numpy(), r) for nm, t, r in zip(names, dW + db, ref[1] + ref[2])}
        errs["loss"] = abs(float(loss.item()) - ref[0]) / abs(ref[0])
        accuracy.update({"rel_l2": errs, "worst": max(errs.values()),
                         "tolerance": {"3xtf32": 1e-5, "simt": 1e-5, "tf32": 5e-3, "bf16": 2e-2}[args.math],
                         "sample": "first %d patterns of rank 0's batch against the CPU checker in float64" % n_sample})

    mult = 3.0 if args.math == "3xtf32" else 1.0
    step_pipe = mult * value / world / 1e3          # tensor-pipe TFLOP/s per GPU over the whole step
    line = {
        "metric": "gradient_eval_gflops", "value": value, "unit": "GFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": scaling,
        "vs_baseline": None, "dtype": "bf16" if half else "f32", "data": "synthetic",
        "config": {"workload": "%s: %s MLP, %d patterns %s, seed %d" % (
                       args.workload, "-".join(map(str, sizes)), count if scaling == "weak" else total,
                       "per GPU" if scaling == "weak" else "in total", seed),
                   "math": args.math, "head": args.head, "global_batch": total, "patterns_per_rank": per_rank,
                   "parallelism": "dp%d" % world, "exchange": args.exchange if world > 1 else None,
                   "exchange_overlap": ("per layer on a second stream" if overlap else "after the last product") if world > 1 else None,
                   "l2": "no flush: inputs and intermediates of a step (X %.0f MB, logits %.0f MB) exceed the 126 MB L2"
                         % (batch * sizes[0] * 4 / 1e6, batch * sizes[-1] * 4 / 1e6),
                   "step": "gradient evaluation + W -= lr*grad, lr = 1e-3 / global_batch"},
        "patterns_per_s": total / (ms_step * 1e-3),
        "e2e": {"value": e2e_value, "unit": "GFLOP/s", "ms_per_step": ms_e2e, "how": e2e_mode,
                "h2d_bytes_per_step": Xh.numel() * 4 + yh.numel() * 4,
                "d2h_bytes_per_step": 8 + sum(t.numel() * 4 for t in grad_h),
                "read_back": ("the loss and the whole gradient" if args.e2e_gradient else
                              "the loss only (8 bytes): the gradient stays on the device, where the parameter step uses it; "
                              "--e2e-gradient copies it back as well")},
        "gpu_launches": int(launches),
        "launch_kinds": {k: int(c1[k] - c0[k]) for k in c1},
        "roofline": roofline,
        "phases_ms": [{"ms": round(p[0], 4), "M": p[1], "N": p[2], "K": p[3]} for p in phases],
        "gemm_share_of_step": gemm_ms / ms_step if ms_step and len(starts) == 1 else None,
        "accuracy": accuracy,
        "cpu_baseline": cpu,
        "clocks": clocks,
        "device_status": status,
        "peaks": {k: peaks.get(k) for k in ("hbm_gbs", "bf16_tflops", "bf16_tflops_sustained", "_source")},
    }
    if args.math != "simt":
        # the whole step (products, reductions, parameter step) as a tensor-pipe rate, against the same peaks
        whole = {"tensor_pipe_tflops_per_gpu": step_pipe, "logical_tflops_per_gpu": value / world / 1e3,
                 "peak_dtype": "bf16" if half else "tf32"}
        whole.update(fractions(step_pipe, tp, region_ms, sm_mhz))
        whole["frac_of_nominal"] = step_pipe / NOMINAL_TFLOPS["bf16" if half else "tf32"]
        line["step_vs_tensor_peak"] = whole
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
