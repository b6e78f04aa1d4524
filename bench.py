#!/usr/bin/env python
"""Benchmark of the gradient evaluation (forward products, fused epilogues, delta products, weight-gradient
products with their fixed-order reduction, then the plain step W -= lr*grad) on synthetic data shaped like
the paper's 400-480-3203 character-recognition network.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--math 3xtf32|tf32|simt|bf16] [--workload config3|config1|config5]
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
}
CHUNK = {"config4": 131072}
MATH = {"3xtf32": 0, "tf32": 1, "simt": 2, "bf16": 3}
NOMINAL_TF32_OVER_BF16 = 0.5        # dense TF32 tensor rate is half the BF16 rate
# DRAM bytes per launch of the products that can be the dominant kernel, from ncu captures on a smaller batch scaled by
# the pattern count (profiles/tc_gemm_3xtf32_config3.md, profiles/bf16_gemm_config3.md).  Only reported while the
# library still is the version the counters were taken on.
NCU_TRAFFIC = {
    "library_version": 108,
    # dram__bytes_read.sum + dram__bytes_write.sum per launch, captured at 16384 patterns (x4) / 32768 patterns (x2)
    ("config3", "3xtf32", (3203, 481, 65536)): 4 * (301.98144e6 + 22.541824e6),
    ("config3", "3xtf32", (65536, 480, 3203)): 4 * (309.94867e6 + 23.211520e6),
    ("config3", "3xtf32", (65536, 3203, 480)): 4 * (77.123840e6 + 166.81395e6),
    ("config3", "bf16", (65536, 3203, 480)): 2 * (38.540544e6 + 172.197632e6),
    ("config3", "bf16", (3203, 481, 65536)): 2 * (253.675520e6 + 17.889792e6),
    ("config3", "bf16", (65536, 480, 3203)): 2 * (250.972416e6 + 18.076160e6),
}
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


def cpu_baseline(sizes, seed, n_sample, head="softmax"):
    """The CPU checker, as it stands, on the first n_sample patterns of the workload."""
    import oracle
    import synth_inputs as si
    from paper_1911_05181_b200 import flops
    Ws, bs = si.mlp_params(seed, sizes)
    X, y = si.mlp_batch(seed, sizes, n_sample)
    T = si.mlp_targets(seed, sizes, n_sample) if head == "sse" else None
    t0 = time.perf_counter()
    if head == "sse":
        oracle.mlp_sse_gradient(Ws, bs, X, T)
    else:
        oracle.mlp_gradient(Ws, bs, X, y)
    dt = time.perf_counter() - t0
    return {"value": flops.gradient_flops(sizes, n_sample) / dt / 1e9, "unit": "GFLOP/s", "cores": oracle.num_threads(),
            "kind": "oracle", "sample": "first %d patterns of the batch, one gradient evaluation, %.1f s" % (n_sample, dt),
            "patterns_per_s": n_sample / dt}


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
    ("N", "T", 65536, 480, 400), ("N", "T", 65536, 3204, 480), ("T", "N", 480, 3204, 65536),
]


def run_sgemm_sweep(args):
    """--workload sgemm: C = A*B (alpha 1, beta 0) over the sweep, device-resident operands uniform [-1,1), seed 1.
    N = 3204 stands in for 3203 (a packed leading dimension of 3203 floats cannot be addressed by TMA and goes to
    the FFMA engine).  Prints one JSON line; `value` is the 8192^3 rate."""
    import torch
    import synth_inputs as si
    from paper_1911_05181_b200 import binding as ul
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    if int(os.environ.get("RANK", "0")) != 0:
        return 0
    math_mode = MATH[args.math]
    peaks = load_peaks()
    # tensor peak of the mode's operand type: the measured bf16 rate, halved for TF32 (nominal ratio)
    tf32_peak = peaks["bf16_tflops_sustained"] * (1.0 if args.math == "bf16" else NOMINAL_TF32_OVER_BF16)
    mult = 3.0 if args.math == "3xtf32" else 1.0
    stream = torch.cuda.current_stream()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")          # > L2: written between timed calls
    rows = []
    for ta, tb, M, N, K in SGEMM_SWEEP:
        ra, ca = (K, M) if ta == "T" else (M, K)
        rb, cb = (N, K) if tb == "T" else (K, N)
        A = torch.empty(ra, ca, device="cuda"); B = torch.empty(rb, cb, device="cuda"); C = torch.empty(M, N, device="cuda")
        ul.fill_uniform(A, A.numel(), 1, si.TID_GEMM_A, 0, 1); ul.fill_uniform(B, B.numel(), 1, si.TID_GEMM_B, 0, 1)
        nbytes = ul.sgemm_workspace_bytes(ta, tb, M, N, K, math_mode)
        ws = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
        wp = (ws.data_ptr() + 255) // 256 * 256

        def call():
            ul.sgemm_ex(ta, tb, M, N, K, 1.0, A, ca, B, cb, 0.0, C, N, math_mode, wp if nbytes else None, nbytes)

        for _ in range(3):
            call()
        reps = 20 if M * N * K < (1 << 34) else 8
        times = []
        for _ in range(reps):
            flush.fill_(1)                                                     # cold L2, as the paper flushed its caches
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record(stream); call(); e1.record(stream)
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        ms = statistics.median(times)
        tf = 2.0 * M * N * K / (ms * 1e-3) / 1e12
        rows.append({"form": ta + tb, "M": M, "N": N, "K": K, "ms": round(ms, 4), "logical_tflops": round(tf, 2),
                     "tensor_pipe_frac_of_measured": round(mult * tf / tf32_peak, 3) if args.math != "simt" else None})
    big = [r for r in rows if r["M"] == 8192][0]
    line = {"metric": "sgemm_gflops", "value": big["logical_tflops"] * 1e3, "unit": "GFLOP/s", "n_gpus": 1, "steps": 8,
            "warmup": 3, "ms_per_step": big["ms"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if args.math == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": "sgemm sweep (alpha 1, beta 0, uniform [-1,1), seed 1); value = NN 8192^3", "math": args.math,
                       "l2": "a 256 MB buffer is overwritten between timed calls"},
            "sweep": rows, "peak_tflops": tf32_peak, "gpu_launches": int(sum(ul.launch_counts().values()))}
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
    ap.add_argument("--exchange", default="allreduce", choices=["allreduce", "ordered"],
                    help="gradient exchange over several GPUs: NCCL all-reduce, or all-gather + sum in rank order")
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

    sizes, batch, seed = WORKLOADS[args.workload]
    if args.patterns > 0:
        batch = args.patterns
    math_mode = MATH[args.math]
    L = len(sizes) - 1
    # Weak scaling (Section 4.3: patterns are partitioned, parameters replicated): every rank evaluates its own
    # `batch` patterns, slice [rank*batch, (rank+1)*batch) of one seeded stream, and the gradients are summed.
    Ws, bs = si.mlp_params(seed, sizes)
    W = [torch.from_numpy(w).cuda() for w in Ws]
    b = [torch.from_numpy(v).cuda() for v in bs]
    W0 = [w.clone() for w in W]; b0 = [v.clone() for v in b]
    dW = [torch.empty_like(w) for w in W]; db = [torch.empty_like(v) for v in b]
    loss = torch.zeros(1, dtype=torch.float64, device="cuda")
    X = torch.empty(batch, sizes[0], device="cuda"); y = torch.empty(batch, dtype=torch.int32, device="cuda")
    first, _ = dp.shard_range(rank, world, batch)
    ul.fill_uniform(X, X.numel(), seed, si.TID_X, first * sizes[0], 0)
    ul.fill_labels(y, batch, seed, si.TID_LABELS, first, sizes[-1])
    if args.head == "sse":       # dense targets uniform [-1, 1) in place of the labels
        y = torch.empty(batch, sizes[-1], device="cuda")
        ul.fill_uniform(y, y.numel(), seed, si.TID_TARGETS, first * sizes[-1], 1)
    Xh = torch.empty(batch, sizes[0], pin_memory=True); yh = torch.empty(y.shape, dtype=y.dtype, pin_memory=True)
    Xh.copy_(X); yh.copy_(y)
    loss_h = torch.zeros(1, dtype=torch.float64, pin_memory=True)
    chunk = min(batch, CHUNK.get(args.workload, batch))
    starts = list(range(0, batch, chunk))
    net = ul.Mlp(sizes, math_mode, chunk)
    lr = 1e-3 / (batch * world)
    stream = torch.cuda.current_stream()
    exchange = dp.GradientExchange(dW + db, dist, ordered=args.exchange == "ordered")

    def step(Xd, yd, host=None):
        for i, lo in enumerate(starts):
            hi = min(batch, lo + chunk)
            if host is not None:            # end-to-end leg: this chunk's patterns come from pinned host memory
                Xd[lo:hi].copy_(host[0][lo:hi], non_blocking=True); yd[lo:hi].copy_(host[1][lo:hi], non_blocking=True)
            if args.head == "sse":
                net.gradient_sse(W, b, Xd[lo:hi], sizes[0], yd[lo:hi], sizes[-1], hi - lo, i > 0, dW, db, loss)
            else:
                net.gradient(W, b, Xd[lo:hi], sizes[0], yd[lo:hi], hi - lo, i > 0, dW, db, loss)
        # the one exchange step of the method: sum of the per-rank gradients and losses (Section 4.3), NCCL
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

    # ---- end to end through the public call: inputs from pinned host memory every step, loss read back every step
    reset_params()

    def e2e_step():
        step(X, y, host=(Xh, yh))
        loss_h.copy_(loss, non_blocking=True)

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
                loss_h.copy_(loss, non_blocking=True)
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

    gflop_step = flops.gradient_flops(sizes, batch) * world / 1e9
    value = gflop_step / (ms_step * 1e-3)
    e2e_value = gflop_step / (ms_e2e * 1e-3)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    # ---- roofline of the dominant product (largest share of the step)
    peaks = load_peaks()
    dom = max(range(len(phases)), key=lambda i: phases[i][0]) if phases else None
    roofline = None
    if dom is not None:
        ms_k, M, N, K = phases[dom]
        logical = 2.0 * M * N * K
        counts = ul.launch_counts()
        on_tensor = args.math != "simt" and counts["tc_gemm"] > 0
        if on_tensor:
            mult = 3.0 if args.math == "3xtf32" else 1.0
            half = args.math == "bf16"
            peak = peaks["bf16_tflops_sustained"] * (1.0 if half else NOMINAL_TF32_OVER_BF16)
            esize = 2.0 if half else 4.0
            achieved = mult * logical / (ms_k * 1e-3) / 1e12
            roofline = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                        "traffic": (NCU_TRAFFIC.get((args.workload, args.math, (M, N, K)))
                                    if ul.version() == NCU_TRAFFIC["library_version"] and args.patterns <= 0 else None),
                        "algorithmic_bytes": esize * (M * K + K * N) + (esize * M * N if K <= 8192 else 0.0),
                        "kernel": "%s M=%d N=%d K=%d" % ("bf16_gemm" if half else "tc_gemm", M, N, K), "ms": ms_k,
                        "flops_counted": "%gx 2MNK" % mult, "logical_tflops": logical / (ms_k * 1e-3) / 1e12,
                        "peak_source": ("%s cuBLAS bf16 sustained" if half else
                                        "%s cuBLAS bf16 sustained x 0.5 (nominal TF32:BF16)") % peaks["_source"]}
        else:
            sm_mhz = (clocks or {}).get("sm_mhz") or peaks.get("sm_max_mhz", 1965.0)
            peak = 148 * 128 * 2 * sm_mhz * 1e6 / 1e12      # FFMA lanes x 2 flops x clock seen during the run
            achieved = logical / (ms_k * 1e-3) / 1e12
            roofline = {"bound": "alu", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                        "traffic": None, "kernel": "simt_gemm M=%d N=%d K=%d" % (M, N, K), "ms": ms_k,
                        "peak_source": "148 SMs x 128 FFMA lanes x 2 x %.0f MHz (median SM clock of this run)" % sm_mhz}
    gemm_ms = sum(p[0] for p in phases)

    cpu = None
    if not args.no_cpu_baseline:
        n_sample = {"config1": 4096, "config3": 16384, "config5": 1024, "config4": 16384}[args.workload]
        cpu = cpu_baseline(sizes, seed, min(batch, n_sample), args.head)

    line = {
        "metric": "gradient_eval_gflops", "value": value, "unit": "GFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if args.math == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": "%s: %s MLP, %d patterns per GPU, seed %d" % (args.workload, "-".join(map(str, sizes)), batch, seed),
                   "math": args.math, "head": args.head, "global_batch": batch * world, "parallelism": "dp%d" % world, "exchange": args.exchange if world > 1 else None,
                   "l2": "no flush: inputs and intermediates of a step (X %.0f MB, logits %.0f MB) exceed the 126 MB L2"
                         % (batch * sizes[0] * 4 / 1e6, batch * sizes[-1] * 4 / 1e6),
                   "step": "gradient evaluation + W -= lr*grad, lr = 1e-3 / global_batch"},
        "patterns_per_s": batch * world / (ms_step * 1e-3),
        "pct_of_tf32_peak": None,
        "e2e": {"value": e2e_value, "unit": "GFLOP/s", "ms_per_step": ms_e2e, "how": e2e_mode,
                "h2d_bytes_per_step": Xh.numel() * 4 + yh.numel() * 4, "d2h_bytes_per_step": 8},
        "gpu_launches": int(launches),
        "launch_kinds": {k: int(c1[k] - c0[k]) for k in c1},
        "roofline": roofline,
        "phases_ms": [{"ms": round(p[0], 4), "M": p[1], "N": p[2], "K": p[3]} for p in phases],
        "gemm_share_of_step": gemm_ms / ms_step if ms_step and len(starts) == 1 else None,
        "cpu_baseline": cpu,
        "clocks": clocks,
        "device_status": status,
        "peaks": {k: peaks.get(k) for k in ("hbm_gbs", "bf16_tflops", "bf16_tflops_sustained", "_source")},
    }
    # tensor peak of the mode's operand type: the measured bf16 rate, halved (nominal ratio) for the TF32 modes
    half = args.math == "bf16"
    tf32_peak = peaks["bf16_tflops_sustained"] * (1.0 if half else NOMINAL_TF32_OVER_BF16) * 1e3   # GFLOP/s
    mult = 3.0 if args.math == "3xtf32" else 1.0
    line["pct_of_tf32_peak"] = {"logical": 100.0 * value / world / tf32_peak,
                                "tensor_pipe": 100.0 * mult * value / world / tf32_peak if args.math != "simt" else None,
                                "peak_gflops": tf32_peak, "peak_dtype": "bf16" if half else "tf32"}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
