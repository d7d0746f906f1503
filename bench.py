#!/usr/bin/env python
"""Benchmark of the BlockDialect quantized linear layer on B200.

One step = one pass of the whole hot path (online two-stage activation
quantisation + block-scaled DialectFP4 x DialectFP4 product, bf16 output) over
the four LLaMA3-8B-shaped linear layers at M = 2048 tokens:
(K, N) = (4096, 4096), (4096, 1024), (4096, 14336), (14336, 4096).
Weights are quantised offline (two-stage rule) before timing.  Inputs are
seeded synthetic tensors (Student-t activations with 1 % outlier channels,
N(0, 0.02) weights).

The JSON line carries:
  value / ms_per_step  device-timed (CUDA events), inputs resident in HBM
  e2e                  the same step through the C ABI with the activations coming from
                       pinned host memory and the outputs copied back, inside the timed region
  roofline             the dominant kernel (tensor-core product of the largest layer)
  act_quantizer        the standalone activation quantizer on bf16 [8192, 4096] against HBM
  cpu_baseline         the CPU oracle timed on a bounded sample of the same workload

`--impl reference` times the CPU oracle alone (same metric and unit).
With --gpus N > 1 (under torchrun) every rank runs the same per-GPU workload on
its own tokens (no collective: token batches are independent); value is the sum.
"""
import argparse
import datetime
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

LAYERS = [("qo_proj", 4096, 4096), ("kv_proj", 4096, 1024), ("gate_up", 4096, 14336), ("down", 14336, 4096)]
M_TOKENS = 2048
QUANT_SHAPE = (8192, 4096)
BYTES_PER_ELEM_QUANT = 2 + 0.5 + 1.5 / 32           # bf16 read + 4-bit code + (4-bit id + 8-bit scale) / 32
# dram__bytes_read.sum + dram__bytes_write.sum per launch, from the ncu captures summarised under profiles/
QUANT_DRAM_BYTES = 67.13e6 + 4.82e6                 # quantize_bf16_kernel on bf16 [8192, 4096]
GEMM_GATE_UP_DRAM_BYTES = 40.84e6 + 20.82e6         # tc::gemm_wtmem_kernel on the gate/up layer
QUANT_WARP_INSTRUCTIONS = 12.9e6                    # smsp__inst_executed.sum of the same quantizer launch
SM_COUNT, ISSUE_PER_SM_CLK = 148, 4                 # warp instructions per clock an SM can issue (4 schedulers)
MLP_SWEEP = [(4096, 11008), (11008, 4096)]
MLP_SWEEP_M = [1, 16, 128, 1024, 8192]


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clock samples taken while the timed region runs."""
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "25",
                 "-i", str(self.gpu_index)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self, t_begin=None, t_end=None):
        """Median SM clock and the throttle reasons seen between the wall-clock times t_begin and t_end
        (the timed region); with no sample inside, the samples nearest to it are used."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.05)
        self.proc.terminate()
        self.proc.wait()
        rows, smax = [], None
        for line in open(self.path):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                stamp = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                mhz = float(f[1])
                smax = float(f[2])
                watts = float(f[3])
            except ValueError:
                continue
            active = [name for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                                 "sw_power_cap"), f[5:9]) if val.lower().startswith("active")]
            rows.append((stamp, mhz, watts, active))
        os.unlink(self.path)
        inside = [r for r in rows if t_begin is not None and t_begin <= r[0] <= t_end]
        where = "timed region"
        if not inside and rows and t_begin is not None:
            mid = 0.5 * (t_begin + t_end)
            inside = sorted(rows, key=lambda r: abs(r[0] - mid))[:3]
            where = "nearest samples (region shorter than the sampling period)"
        elif not inside:
            inside, where = rows, "whole run"
        reasons = sorted({a for r in inside for a in r[3]})
        return {"sm_mhz": float(np.median([r[1] for r in inside])) if inside else None, "sm_max_mhz": smax,
                "power_w": float(np.median([r[2] for r in inside])) if inside else None, "reasons": reasons,
                "samples": len(inside), "window": where}


# ---------------------------------------------------------------------------
# CPU oracle leg (cpu_baseline and --impl reference)
# ---------------------------------------------------------------------------
_ORACLE_WEIGHTS = {}


def oracle_step_sample(rows=16):
    """One oracle pass over a bounded sample: `rows` tokens of each of the four layers
    (quantise the activations, dequantise, fp64 product against the dequantised weights).
    Returns (flops_done, seconds, threads)."""
    import oracle
    from paper_2501_01144_b200 import inputs
    flops, secs = 0.0, 0.0
    for i, (_, K, N) in enumerate(LAYERS):
        xb = inputs.act_student_t(rows, K, seed=2 + i)
        if i not in _ORACLE_WEIGHTS:                         # offline weight quantisation, not timed
            wq = oracle.quantize(inputs.weights_normal(N, K, seed=2 + i), dtype=oracle.BF16)
            _ORACLE_WEIGHTS[i] = oracle.dequantize(*wq)
        wdq = _ORACLE_WEIGHTS[i]
        t0 = time.perf_counter()
        xq = oracle.quantize(xb, dtype=oracle.BF16)
        xdq = oracle.dequantize(*xq)
        oracle.gemm(xdq, wdq)
        secs += time.perf_counter() - t0
        flops += 2.0 * rows * N * K
    return flops, secs, oracle.threads()


def run_reference(args, rank):
    if rank != 0:
        return
    import oracle
    oracle.build()
    rows = 16
    for _ in range(max(1, min(args.warmup, 1))):
        oracle_step_sample(rows)
    flops = secs = 0.0
    for _ in range(args.steps):
        f, s, threads = oracle_step_sample(rows)
        flops += f
        secs += s
    value = flops / secs / 1e12
    full_flops = sum(2.0 * M_TOKENS * N * K for _, K, N in LAYERS)
    line = {
        "impl": "reference", "metric": "bd_linear_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": full_flops / (value * 1e12) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "llama3-8b linear layers, M=2048 (oracle on a 16-token sample per layer, "
                               "ms_per_step extrapolated to 2048 tokens)"},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": threads, "kind": "oracle",
                         "sample": f"{rows} tokens x 4 layers per step"},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def fp8_dense_probe(dev, n=8192, reps=10):
    """A dense FP8 yardstick measured in this run: the library GEMM torch._scaled_mm (E4M3 x E4M3 -> bf16,
    n^3) timed alone, best of `reps`.  It is never on the product path; it only gives the tensor roofline a
    measured FP8 denominator beside the figure derived from the bf16 peak.  None when the call is unavailable."""
    import torch
    try:
        a = (torch.randn(n, n, device=dev) * 0.5).to(torch.float8_e4m3fn)
        b = (torch.randn(n, n, device=dev) * 0.5).to(torch.float8_e4m3fn).t()       # column-major second operand
        one = torch.ones((), device=dev)
        for _ in range(3):
            torch._scaled_mm(a, b, scale_a=one, scale_b=one, out_dtype=torch.bfloat16)
        best = None
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            torch._scaled_mm(a, b, scale_a=one, scale_b=one, out_dtype=torch.bfloat16)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1)
            best = ms if best is None else min(best, ms)
        return {"tflops": 2.0 * n ** 3 / (best * 1e-3) / 1e12, "ms": best,
                "how": f"torch._scaled_mm e4m3 x e4m3 -> bf16, {n}^3, best of {reps}, timed alone (burst)"}
    except Exception as e:                                  # noqa: BLE001 - a yardstick, not part of the product
        return {"tflops": None, "how": f"unavailable: {type(e).__name__}: {str(e)[:120]}"}


def oracle_quantizer_baseline():
    """The CPU oracle's two-stage quantizer on the full activation-quantizer workload (bf16 [8192, 4096]),
    on all host threads and on one, as GB/s of the same algorithmic bytes the GPU figure counts."""
    import ctypes

    import oracle
    from paper_2501_01144_b200 import inputs
    qm, qk = QUANT_SHAPE
    x = inputs.act_normal_outliers(qm, qk, seed=1)
    nbytes = qm * qk * BYTES_PER_ELEM_QUANT
    out = {"workload": "bf16 [8192, 4096], whole tensor", "unit": "GB/s", "kind": "oracle"}
    threads = oracle.threads()
    t0 = time.perf_counter()
    oracle.quantize(x, dtype=oracle.BF16)
    out["all_threads"] = {"value": nbytes / (time.perf_counter() - t0) / 1e9, "cores": threads}
    try:
        gomp = ctypes.CDLL("libgomp.so.1")
        gomp.omp_set_num_threads(1)
        t0 = time.perf_counter()
        oracle.quantize(x, dtype=oracle.BF16)
        out["one_thread"] = {"value": nbytes / (time.perf_counter() - t0) / 1e9, "cores": 1}
        gomp.omp_set_num_threads(threads)
    except OSError:
        out["one_thread"] = None
    return out


# ---------------------------------------------------------------------------
# GPU leg
# ---------------------------------------------------------------------------
def run_gpu(args, rank, world, local_rank):
    import torch

    import paper_2501_01144_b200 as bd
    from paper_2501_01144_b200 import inputs, replicas

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    replicas.init("nccl", dev)
    bd.load()
    peaks = measured_peaks()

    def dev_bf16(bits):
        return torch.from_numpy(bits.view(np.int16)).to(dev).view(torch.bfloat16)

    # resident state: offline-quantised weights, device activations, outputs, workspaces
    layers = []
    for i, (name, K, N) in enumerate(LAYERS):
        xb = inputs.act_student_t(M_TOKENS, K, seed=replicas.rank_seed(2 + i, rank))
        wq = bd.quantize_weights(dev_bf16(inputs.weights_normal(N, K, seed=2 + i)), bd.SELECT_TWO_STAGE)
        x_host = torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).pin_memory()
        layers.append({
            "name": name, "K": K, "N": N, "Wq": wq, "X": x_host.to(dev), "X_host": x_host,
            "X_stage": torch.empty_like(x_host, device=dev),
            "Y": torch.empty(M_TOKENS, N, dtype=torch.bfloat16, device=dev),
            "Y_host": torch.empty(M_TOKENS, N, dtype=torch.bfloat16).pin_memory(),
            "ws": torch.empty(bd.linear_workspace_size(M_TOKENS, N, K), dtype=torch.uint8, device=dev),
            "flops": 2.0 * M_TOKENS * N * K,
        })
    bd.poll_status()
    step_flops = sum(l["flops"] for l in layers)
    footprint = sum(l["Wq"].nbytes() + l["X"].numel() * 2 + l["Y"].numel() * 2 + l["ws"].numel() for l in layers)

    def step():
        for l in layers:
            bd.linear(l["X"], l["Wq"], out=l["Y"], workspace=l["ws"])

    # end to end: every step copies each layer's activations from pinned host memory and its result back.
    # Three streams (host->device, compute, device->host) with events per layer, so that the copies of one layer
    # run under the kernels of another; a staging buffer is refilled only after the kernels that read it.
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    for l in layers:
        l["x_ready"], l["x_free"], l["y_ready"], l["y_free"] = (torch.cuda.Event() for _ in range(4))
        l["x_free"].record()
        l["y_free"].record()

    def step_e2e():
        compute = torch.cuda.current_stream()
        for l in layers:
            with torch.cuda.stream(s_in):
                s_in.wait_event(l["x_free"])
                l["X_stage"].copy_(l["X_host"], non_blocking=True)
                l["x_ready"].record(s_in)
            compute.wait_event(l["x_ready"])
            compute.wait_event(l["y_free"])
            bd.linear(l["X_stage"], l["Wq"], out=l["Y"], workspace=l["ws"])
            l["x_free"].record(compute)
            l["y_ready"].record(compute)
            with torch.cuda.stream(s_out):
                s_out.wait_event(l["y_ready"])
                l["Y_host"].copy_(l["Y"], non_blocking=True)
                l["y_free"].record(s_out)

    def finish_e2e():
        compute = torch.cuda.current_stream()
        for l in layers:                                   # the last results must be on the host before the clock stops
            compute.wait_event(l["y_free"])

    def barrier():
        replicas.barrier(torch.cuda.synchronize)

    per_step = []                                        # device time of each step of the last timed() call

    def timed(fn, steps, warmup, finish=None, head_start=False):
        for _ in range(warmup):
            fn()
        barrier()
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        e0, e1 = marks[0], marks[-1]
        if head_start:
            # the GPU spins for a few milliseconds while the host queues the first steps behind it, so that a
            # host hiccup (interpreter, sampler thread) does not starve the GPU inside the timed region
            torch.cuda._sleep(10_000_000)
        e0.record()
        for i in range(steps):
            fn()
            if i + 1 < steps:
                marks[i + 1].record()                      # a marker in the stream; the host does not wait on it
        if finish:
            finish()
        e1.record()
        barrier()
        per_step[:] = [marks[i].elapsed_time(marks[i + 1]) for i in range(steps)]
        return replicas.max_over_ranks(e0.elapsed_time(e1), dev)   # the job's time is the slowest rank's

    sampler = ClockSampler(local_rank)
    sampler.start()                                        # runs through warm-up and the timed region
    time.sleep(0.05)
    for _ in range(args.warmup):
        step()
    barrier()
    launches_warm = bd.launch_count()
    t_begin = time.time()
    total_ms = timed(step, args.steps, 0, head_start=True)
    t_end = time.time()
    clocks = sampler.stop(t_begin, t_end)
    launches = bd.launch_count() - launches_warm
    ms_per_step = total_ms / args.steps
    step_median, step_best = float(np.median(per_step)), float(np.min(per_step))
    value = replicas.whole_job_rate(step_flops, ms_per_step * 1e-3, world) / 1e12

    # the same step over about half a second: after some 50 ms under load the power cap settles the clock lower
    # (the measured bf16 reference shows the same drop between its burst and sustained figures)
    sustained_steps = 1600
    sustained_ms = timed(step, sustained_steps, 0, head_start=True) / sustained_steps
    sustained_value = replicas.whole_job_rate(step_flops, sustained_ms * 1e-3, world) / 1e12
    time.sleep(1.0)                                        # let the clock recover before the other sections

    e2e_ms = timed(step_e2e, args.steps, min(args.warmup, 3), finish_e2e) / args.steps
    e2e_value = replicas.whole_job_rate(step_flops, e2e_ms * 1e-3, world) / 1e12
    h2d = sum(l["X_host"].numel() * 2 for l in layers)
    d2h = sum(l["Y_host"].numel() * 2 for l in layers)

    # ---- dominant kernel: the product of the largest layer, one event pair per launch ----
    big = max(layers, key=lambda l: l["flops"])
    others = [l for l in layers if l is not big]
    xq = bd.quantize_act(big["X"])
    gws = torch.empty(max(1, bd.gemm_workspace_size(M_TOKENS, big["N"], big["K"])), dtype=torch.uint8, device=dev)
    reps = max(3, min(args.steps, 10))
    durations = []
    for it in range(reps + 2):
        for l in others:                                  # evicts the big layer's operands from L2
            bd.linear(l["X"], l["Wq"], out=l["Y"], workspace=l["ws"])
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        bd.gemm(xq, big["Wq"], out=big["Y"], workspace=gws)
        b.record()
        torch.cuda.synchronize()
        if it >= 2:
            durations.append(a.elapsed_time(b))
    gemm_ms = float(np.mean(durations))
    achieved_tf = big["flops"] / (gemm_ms * 1e-3) / 1e12
    fp8_peak = 2.0 * peaks["bf16_tflops"]                 # dense FP8 = 2 x dense bf16 (nominal ratio), burst: kernel timed alone
    time.sleep(0.5)
    fp8_probe = fp8_dense_probe(dev) if rank == 0 else None
    time.sleep(0.5)                                       # let the clock recover before the other sections
    # DRAM traffic of this launch from the committed ncu capture (profiles/gemm_wtmem_kernel_llama3_gate_up.md)
    roofline = {"bound": "tensor", "kernel": "bd_gemm " + big["name"] + " (decode_e4m3 of the activations + tc::gemm_wtmem_kernel)",
                "achieved": achieved_tf, "peak": fp8_peak,
                "unit": "TFLOP/s", "frac": achieved_tf / fp8_peak, "traffic": GEMM_GATE_UP_DRAM_BYTES,
                "peak_source": f"2 x {peaks['source']} bf16 burst", "ms_per_launch": gemm_ms,
                "frac_of_nominal_4500": achieved_tf / 4500.0,
                # the same launch against a dense FP8 library GEMM timed in this run (a yardstick only)
                "fp8_probe": fp8_probe,
                "frac_of_fp8_probe": (achieved_tf / fp8_probe["tflops"]) if fp8_probe and fp8_probe.get("tflops") else None}

    # ---- standalone activation quantizer on bf16 [8192, 4096] (HBM-bound) ----
    qm, qk = QUANT_SHAPE
    n_sets = 4                                            # 4 x (64 MiB in + 20 MiB out) > 2 x L2
    xs = [dev_bf16(inputs.act_normal_outliers(qm, qk, seed=1 + s)) for s in range(n_sets)]
    qs = [bd.QTensor(qm, qk, dev) for _ in range(n_sets)]
    for i in range(3 * n_sets):
        bd.quantize_act(xs[i % n_sets], out=qs[i % n_sets])
    torch.cuda.synchronize()
    q_reps = 40
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda._sleep(4_000_000)                          # ~2 ms of GPU head start: the host queues all launches
    e0.record()                                           # behind it, so the events see kernel time, not launch rate
    for i in range(q_reps):
        bd.quantize_act(xs[i % n_sets], out=qs[i % n_sets])
    e1.record()
    torch.cuda.synchronize()
    q_ms = e0.elapsed_time(e1) / q_reps
    q_bytes = qm * qk * BYTES_PER_ELEM_QUANT
    q_gbs = q_bytes / (q_ms * 1e-3) / 1e9
    act_quantizer = {"workload": "bf16 [8192, 4096] N(0,1), 1% outlier channels, 4 rotating buffer sets (L2-cold)",
                     "bound": "hbm", "achieved": q_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": q_gbs / peaks["hbm_gbs"], "frac_of_nominal_8000": q_gbs / 8000.0,
                     "us_per_launch": q_ms * 1e3, "algorithmic_bytes": q_bytes, "traffic": QUANT_DRAM_BYTES,
                     "peak_source": peaks["source"],
                     # the kernel is held by instruction issue, not by HBM: its warp instructions per second against
                     # what 148 SMs x 4 schedulers issue at the maximum SM clock
                     "alu": {"bound": "alu", "achieved": QUANT_WARP_INSTRUCTIONS / (q_ms * 1e-3) / 1e9,
                             "peak": SM_COUNT * ISSUE_PER_SM_CLK * 1.965, "unit": "G warp-instructions/s",
                             "frac": QUANT_WARP_INSTRUCTIONS / (q_ms * 1e-3) / 1e9 / (SM_COUNT * ISSUE_PER_SM_CLK * 1.965)}}
    bd.poll_status()

    # ---- LLaMA2-7B MLP shapes, decode to prefill (reported per M; not part of the timed step).  Inputs are
    # the seeded generators the parity tests use (|N| * N products with 1 % outlier channels).  The decode-sized
    # calls are bound by the weight stream, so the weights rotate over six copies (6 x 24.7 MB > the 126 MB L2):
    # no call finds its weights in L2. ----
    sweep = []
    if rank == 0:
        n_wsets = 6
        for K, N in MLP_SWEEP:
            wsrc = dev_bf16(inputs.weights_normal(N, K, seed=3))
            wqs = [bd.quantize_weights(wsrc, bd.SELECT_TWO_STAGE) for _ in range(n_wsets)]
            del wsrc
            for M in MLP_SWEEP_M:
                x = dev_bf16(inputs.act_post_silu(M, K, seed=3))
                y = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
                ws = torch.empty(bd.linear_workspace_size(M, N, K), dtype=torch.uint8, device=dev)
                for i in range(n_wsets):
                    bd.linear(x, wqs[i], out=y, workspace=ws)
                l0 = bd.launch_count()
                bd.linear(x, wqs[0], out=y, workspace=ws)
                launches_per_call = bd.launch_count() - l0          # 2: quantizer + product (warp-level kernel for up to 8
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)   # tokens); 3: + the K split's sum
                n_rep = 24 if M <= 1024 else 6
                torch.cuda._sleep(2_000_000)                  # GPU head start: the events see kernel time, not launch rate
                a.record()
                for i in range(n_rep):
                    bd.linear(x, wqs[i % n_wsets], out=y, workspace=ws)
                b.record()
                torch.cuda.synchronize()
                us = a.elapsed_time(b) / n_rep * 1e3
                # host time of one call (argument checks, tensor-map encoding, launches), GPU idle
                t0 = time.perf_counter()
                for i in range(n_rep):
                    bd.linear(x, wqs[i % n_wsets], out=y, workspace=ws)
                host_us = (time.perf_counter() - t0) / n_rep * 1e6
                torch.cuda.synchronize()
                flops = 2.0 * M * N * K
                nbytes = N * K * 0.546875 + M * K * 2 + M * N * 2
                bound_tf = min(2.0 * peaks["bf16_tflops"], flops / nbytes * peaks["hbm_gbs"] / 1e3)
                sweep.append({"K": K, "N": N, "M": M, "us": us, "host_us_per_call": host_us, "tflops": flops / us / 1e6,
                              "gbs": nbytes / us / 1e3, "floor_us": flops / bound_tf / 1e6,
                              "frac_of_roofline": flops / us / 1e6 / bound_tf, "launches_per_call": launches_per_call})
            del wqs
        bd.poll_status()

    # ---- one token through the four linear layers of a LLaMA3-8B block (the benchmark's shapes at M = 1): called one by
    # one, and the same four calls replayed from a CUDA graph.  Weights of two blocks in rotation (152 MB > L2). ----
    decode_block = None
    if rank == 0:
        blocks = []
        for seed in (21, 22):
            blocks.append([bd.quantize_weights(dev_bf16(inputs.weights_normal(N, K, seed=seed + 10 * i)), bd.SELECT_TWO_STAGE)
                           for i, (_, K, N) in enumerate(LAYERS)])
        xs1 = [dev_bf16(inputs.act_post_silu(1, K, seed=5)) for _, K, _ in LAYERS]
        ys1 = [torch.empty(1, N, dtype=torch.bfloat16, device=dev) for _, _, N in LAYERS]
        wss = [torch.empty(bd.linear_workspace_size(1, N, K), dtype=torch.uint8, device=dev) for _, K, N in LAYERS]

        def one_token(b):
            for i in range(len(LAYERS)):
                bd.linear(xs1[i], blocks[b][i], out=ys1[i], workspace=wss[i])

        for i in range(4):
            one_token(i % 2)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda._sleep(4_000_000)
        e0.record()
        for i in range(20):
            one_token(i % 2)
        e1.record()
        torch.cuda.synchronize()
        eager_us = e0.elapsed_time(e1) / 20 * 1e3
        gs = torch.cuda.Stream(device=dev)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(gs):
            with torch.cuda.graph(graph, stream=gs):
                one_token(0)
                one_token(1)
        for _ in range(3):
            graph.replay()
        e0.record()
        for _ in range(10):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        graph_us = e0.elapsed_time(e1) / 20 * 1e3
        del graph
        wbytes = sum(N * K for _, K, N in LAYERS) * 0.546875
        decode_block = {"workload": "llama3-8b linear layers (q/o, k/v, gate/up, down) at M = 1, one after the other",
                        "us_per_token": eager_us, "us_per_token_graph_replay": graph_us, "weight_bytes": wbytes,
                        "floor_us": wbytes / peaks["hbm_gbs"] / 1e3, "frac_of_roofline": wbytes / peaks["hbm_gbs"] / 1e3 / graph_us}
        del blocks
        bd.poll_status()

    # ---- two chained layers (gate/up then down, M = 2048) with and without the requantising epilogue (Sec. 3.3,
    # last paragraph).  Without: the first layer writes bf16, the second layer's quantizer reads it back.  With: the
    # first product's epilogue writes the DialectFP4 operand and the second product takes it (its operand bytes are
    # expanded by a small kernel).  Three copies of both weight matrices in rotation (186 MB > L2). ----
    chained = None
    if rank == 0:
        d0, d1, d2 = 4096, 14336, 4096
        xs = dev_bf16(inputs.act_student_t(M_TOKENS, d0, seed=2))
        w1 = dev_bf16(inputs.weights_normal(d1, d0, seed=4))
        w2 = dev_bf16(inputs.weights_normal(d2, d1, seed=5))
        sets = [(bd.quantize_weights(w1, bd.SELECT_TWO_STAGE), bd.quantize_weights(w2, bd.SELECT_TWO_STAGE)) for _ in range(3)]
        del w1, w2
        h16 = torch.empty(M_TOKENS, d1, dtype=torch.bfloat16, device=dev)
        hq = bd.QTensor(M_TOKENS, d1, dev)
        yo = torch.empty(M_TOKENS, d2, dtype=torch.bfloat16, device=dev)
        ws1 = torch.empty(max(bd.linear_workspace_size(M_TOKENS, d1, d0), bd.linear_requant_workspace_size(M_TOKENS, d1, d0)),
                          dtype=torch.uint8, device=dev)
        ws2 = torch.empty(max(bd.linear_workspace_size(M_TOKENS, d2, d1), bd.gemm_workspace_size(M_TOKENS, d2, d1), 1),
                          dtype=torch.uint8, device=dev)

        def plain(i):
            a, b = sets[i % 3]
            bd.linear(xs, a, out=h16, workspace=ws1)
            bd.linear(h16, b, out=yo, workspace=ws2)

        def fused(i):
            a, b = sets[i % 3]
            bd.linear_requant(xs, a, out=hq, workspace=ws1)
            bd.gemm(hq, b, out=yo, workspace=ws2)

        def time_chain(fn, n_rep=30):
            for i in range(3):
                fn(i)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda._sleep(4_000_000)
            e0.record()
            for i in range(n_rep):
                fn(i)
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / n_rep * 1e3

        plain_us = time_chain(plain)
        time.sleep(0.3)
        fused_us = time_chain(fused)
        chain_flops = 2.0 * M_TOKENS * (d0 * d1 + d1 * d2)
        chained = {"workload": "gate/up (4096 -> 14336) then down (14336 -> 4096), M = 2048, bf16 final result",
                   "bf16_between_us": plain_us, "requantised_between_us": fused_us,
                   "bf16_between_tflops": chain_flops / plain_us / 1e6, "requantised_between_tflops": chain_flops / fused_us / 1e6,
                   "speedup": plain_us / fused_us}
        del sets, h16, hq, yo, ws1, ws2
        bd.poll_status()
        time.sleep(0.5)

    # ---- block sizes 16 / 32 / 64 (Sec. 4.2, Table 3; e.g. block 16 for the down projection): the quantizer on the
    # activation-quantizer workload and the down projection at M = 2048.  Block 64 is stored as pairs of 32-blocks
    # (same product kernel, same time); block 16 is stored zero-padded to 32-blocks: twice the code bytes and MMA work ----
    block_sizes = None
    if rank == 0:
        block_sizes = []
        xq_src = dev_bf16(inputs.act_normal_outliers(qm, qk, seed=1))
        Kd, Nd = 14336, 4096
        xd_src = dev_bf16(inputs.act_student_t(M_TOKENS, Kd, seed=5))
        wd_src = dev_bf16(inputs.weights_normal(Nd, Kd, seed=5))
        yd = torch.empty(M_TOKENS, Nd, dtype=torch.bfloat16, device=dev)
        for block in (16, 32, 64):
            qo = bd.QTensor(qm, bd.physical_k(qk, block), dev)
            for _ in range(3):
                bd.quantize_bs(xq_src, block, out=qo)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(10):
                bd.quantize_bs(xq_src, block, out=qo)
            e1.record()
            torch.cuda.synchronize()
            q_us = e0.elapsed_time(e1) / 10 * 1e3
            q_bytes_b = qm * qk * (2 + 0.5 + 1.5 / block)
            wq_b = bd.quantize_bs(wd_src, block)
            ws_b = torch.empty(bd.linear_bs_workspace_size(M_TOKENS, Nd, Kd, block), dtype=torch.uint8, device=dev)
            for _ in range(3):
                bd.linear_bs(xd_src, wq_b, block, out=yd, workspace=ws_b)
            e0.record()
            for _ in range(10):
                bd.linear_bs(xd_src, wq_b, block, out=yd, workspace=ws_b)
            e1.record()
            torch.cuda.synchronize()
            l_us = e0.elapsed_time(e1) / 10 * 1e3
            block_sizes.append({"block": block, "quantizer_us": q_us, "quantizer_gbs_algorithmic": q_bytes_b / q_us / 1e3,
                                "bits_per_element_paper_accounting": 4 + 9 / block, "bits_per_element_stored": 8.75 if block == 16 else 4.375,
                                "linear_down_proj_us": l_us, "linear_down_proj_tflops": 2.0 * M_TOKENS * Nd * Kd / l_us / 1e6})
            del qo, wq_b, ws_b
        del xq_src, xd_src, wd_src, yd
        bd.poll_status()
        time.sleep(0.3)

    # ---- KV cache (appendix "Quantization Dimension", Fig. 9b), Mistral-7B shape: 8 KV heads of head_dim 128 with 4113
    # tokens each (128 stored chunks + 17 recent tokens in high precision); one decode step = append one token per head,
    # then scores and P V for the 4 query heads of each KV head.  One cache object per KV head, so a step is dozens of
    # small launches: the time is launch-bound, far from the 4.6 MB of cache bytes it reads ----
    kv_cache = None
    if rank == 0:
        kvh, grp, hd, n_tok, cap = 8, 4, 128, 4113, 4224
        rng_kv = np.random.default_rng(6)
        caches = []
        for g in range(kvh):
            cch = bd.KVCache(cap, hd, device=dev)
            cch.append(dev_bf16(inputs.to_bf16_bits(rng_kv.standard_normal((n_tok, hd)).astype(np.float32))),
                       dev_bf16(inputs.to_bf16_bits(rng_kv.standard_normal((n_tok, hd)).astype(np.float32))))
            caches.append(cch)
        q_rows = [bd.quantize_act(dev_bf16(inputs.to_bf16_bits(rng_kv.standard_normal((grp, hd)).astype(np.float32)))) for _ in range(kvh)]
        pitch = (n_tok + 3) // 4 * 4
        probs = torch.softmax(torch.randn(kvh, grp, pitch, device=dev), -1)[:, :, :n_tok]
        s_out = torch.empty(kvh, grp, n_tok, dtype=torch.float32, device=dev)
        o_out = torch.empty(kvh, grp, hd, dtype=torch.bfloat16, device=dev)

        def attend_per_head():
            for g in range(kvh):
                caches[g].scores(q_rows[g], out=s_out[g])
                caches[g].pv(probs[g], out=o_out[g])

        def attend():                                         # all KV heads of the layer per call
            bd.kvcache_scores_batched(caches, q_rows, out=s_out)
            bd.kvcache_pv_batched(caches, probs, out=o_out)

        for _ in range(3):
            attend_per_head()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(10):
            attend_per_head()
        e1.record()
        torch.cuda.synchronize()
        per_head_us = e0.elapsed_time(e1) / 10 * 1e3

        for _ in range(3):
            attend()
        launches0 = bd.launch_count()
        attend()
        attend_launches = bd.launch_count() - launches0
        e0.record()
        for _ in range(10):
            attend()
        e1.record()
        torch.cuda.synchronize()
        attend_us = e0.elapsed_time(e1) / 10 * 1e3
        o32 = torch.empty(kvh, grp, hd, dtype=torch.bfloat16, device=dev)
        for _ in range(3):
            bd.kvcache_attention(caches, q_rows, 1.0 / np.sqrt(hd), out=o32)
        launches0 = bd.launch_count()
        bd.kvcache_attention(caches, q_rows, 1.0 / np.sqrt(hd), out=o32)
        step_launches = bd.launch_count() - launches0
        e0.record()
        for _ in range(10):                                   # scores, fp32 softmax and P x V of all heads in one call
            bd.kvcache_attention(caches, q_rows, 1.0 / np.sqrt(hd), out=o32)
        e1.record()
        torch.cuda.synchronize()
        step_us = e0.elapsed_time(e1) / 10 * 1e3
        # the same call replayed from a CUDA graph: the six launches without the host's share
        gstream = torch.cuda.Stream(device=dev)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(gstream):
            with torch.cuda.graph(graph, stream=gstream):
                bd.kvcache_attention(caches, q_rows, 1.0 / np.sqrt(hd), out=o32)
        for _ in range(3):
            graph.replay()
        e0.record()
        for _ in range(20):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        step_graph_us = e0.elapsed_time(e1) / 20 * 1e3
        del graph
        new_k = dev_bf16(inputs.to_bf16_bits(rng_kv.standard_normal((1, hd)).astype(np.float32)))
        new_kv = new_k.expand(kvh, 1, hd).contiguous()
        e0.record()
        for _ in range(5):                                    # five tokens per head, one call per head
            for g in range(kvh):
                caches[g].append(new_k, new_k)
        e1.record()
        torch.cuda.synchronize()
        append_per_head_us = e0.elapsed_time(e1) / 5 * 1e3
        e0.record()
        for _ in range(5):                                    # five more tokens, all heads per call (27 recent tokens at the end)
            bd.kvcache_append_batched(caches, new_kv, new_kv)
        e1.record()
        torch.cuda.synchronize()
        append_us = e0.elapsed_time(e1) / 5 * 1e3
        cache_bytes = kvh * 2 * n_tok * hd * 0.546875
        kv_cache = {"workload": "8 KV heads x 4113 tokens x head_dim 128, 4 query heads per KV head, one object per KV head, scores and P x V of all heads per call",
                    "attention_us_per_step": step_us, "attention_launches_per_step": step_launches, "attention_us_per_step_graph_replay": step_graph_us,
                    "scores_and_pv_us_per_step": attend_us, "launches_per_step": attend_launches, "scores_and_pv_us_per_step_head_by_head": per_head_us,
                    "append_one_token_us_per_step": append_us, "append_one_token_us_per_step_head_by_head": append_per_head_us,
                    "cache_bytes_read_per_step": cache_bytes, "cache_read_gbs": cache_bytes / attend_us / 1e3,
                    "stored_bits_per_value": 4.375, "recent_tokens_in_high_precision": n_tok % 32}
        del caches, probs
        bd.poll_status()

    # ---- attention products with both operands quantised online (Mistral-7B shapes: 32 heads, 8 KV heads,
    # 4096 tokens, head_dim 128; reported, not part of the timed step).  QK^T is bound by the write of the
    # scores, PV by the read of the fp32 probabilities. ----
    attention = None
    if rank == 0:
        heads, kvh, S, hd = 32, 8, 4096, 128
        grp = heads // kvh
        n_pheads = 3 * grp                                    # probabilities for three KV groups (each head 64 MiB)
        # the seeded generator of the parity tests: Q/K with head-dim outlier channels, Dirichlet(0.1) rows of P
        Qb, Kb, Pn, Vb = inputs.attention_case(heads, kvh, S, hd, seed=4, p_heads=n_pheads)
        Aq = [bd.quantize_act(dev_bf16(Qb[h])) for h in range(heads)]
        Bk = [bd.quantize_act(dev_bf16(Kb[g])) for g in range(kvh)]
        scores = torch.empty(heads, S, S, dtype=torch.bfloat16, device=dev)          # 1 GiB: L2-cold by size
        gws = torch.empty(max(1, bd.gemm_batched_workspace_size(S, S, hd, heads // kvh)), dtype=torch.uint8, device=dev)

        def time_us(fn, n_rep):
            fn()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(n_rep):
                fn()
            b.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b) / n_rep * 1e3

        qk_us = time_us(lambda: bd.gemm_batched(Aq, Bk, b_group=heads // kvh, out=scores, workspace=gws), 3)
        # context for the write-bound product: what a plain write-only stream reaches on this GPU (the measured
        # peak is a copy, half reads and half writes)
        fill_us = time_us(lambda: scores.fill_(0), 5)
        write_stream_gbs = scores.numel() * 2.0 / fill_us / 1e3
        del scores
        # the four query heads of a KV group share V, so their probabilities go through one call as one
        # [4 * 4096, 4096] matrix (contiguous heads): one quantizer launch and one product per group
        P = [torch.from_numpy(Pn[g * grp:(g + 1) * grp].reshape(grp * S, S)).to(dev) for g in range(3)]   # 3 x 256 MiB > L2
        del Pn
        Bv = bd.quantize_act(dev_bf16(Vb[0]), axis=bd.AXIS_STRIDED)
        O = torch.empty(grp * S, hd, dtype=torch.bfloat16, device=dev)
        lws = torch.empty(bd.linear_workspace_size(grp * S, hd, S), dtype=torch.uint8, device=dev)
        turn = [0]

        def pv():
            bd.linear(P[turn[0] % 3], Bv, out=O, workspace=lws)
            turn[0] += 1

        pv_us = time_us(pv, 6) / grp
        # the KV groups are independent problems: on two streams the quantizer of one group's probabilities (HBM)
        # runs beside the product of the previous group's (tensor cores)
        side = [torch.cuda.Stream(), torch.cuda.Stream()]
        O2 = [O, torch.empty_like(O)]
        lws2 = [lws, torch.empty_like(lws)]

        def pv_two_streams(n_rep):
            cur = torch.cuda.current_stream()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for st in side:
                st.wait_event(a)
            for i in range(n_rep):
                bd.linear(P[i % 3], Bv, out=O2[i % 2], workspace=lws2[i % 2], stream=side[i % 2])
            for st in side:
                cur.wait_stream(st)
            b.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b) / n_rep * 1e3

        pv_two_streams(2)
        pv2_us = pv_two_streams(8) / grp
        # the fused kernel: scores, softmax, quantisation of the probabilities and P V without S or P in memory
        Vall = [bd.quantize_act(dev_bf16(Vb[g]), axis=bd.AXIS_STRIDED) for g in range(kvh)]
        Aq2 = [bd.quantize_act(dev_bf16(Qb[h])) for h in range(heads)]
        Bk2 = [bd.quantize_act(dev_bf16(Kb[g])) for g in range(kvh)]
        o_fused = torch.empty(heads, S, hd, dtype=torch.bfloat16, device=dev)
        fused_us = time_us(lambda: bd.attention(Aq2, Bk2, Vall, group=grp, out=o_fused), 3)
        del Vall, Aq2, Bk2
        qk_bytes, pv_bytes = heads * S * S * 2.0, S * S * 4.0
        attention = {"workload": "QK^T: 32 heads x [4096,128] x [4096,128]^T (head-dim outlier channels), bf16 scores; "
                                 "PV: fp32 Dirichlet(0.1) rows P [4096,4096] per head quantised online x V (token-axis "
                                 "blocks) [128,4096]^T, the 4 heads of a KV group per call; seeded generator, seed 4",
                     "qk_us_32_heads": qk_us, "qk_write_gbs": qk_bytes / qk_us / 1e3,
                     "qk_frac_of_hbm": qk_bytes / qk_us / 1e3 / peaks["hbm_gbs"],
                     "write_only_stream_gbs": write_stream_gbs,
                     "qk_frac_of_write_only_stream": qk_bytes / qk_us / 1e3 / write_stream_gbs,
                     "pv_us_per_head": pv_us, "pv_read_gbs": pv_bytes / pv_us / 1e3,
                     "pv_frac_of_hbm": pv_bytes / pv_us / 1e3 / peaks["hbm_gbs"],
                     "pv_two_streams_us_per_head": pv2_us, "pv_two_streams_read_gbs": pv_bytes / pv2_us / 1e3,
                     "pv_two_streams_frac_of_hbm": pv_bytes / pv2_us / 1e3 / peaks["hbm_gbs"],
                     # fused: all 32 heads in one call; the materialised route beside it is QK^T + P V of all heads
                     # and does not even include the softmax between them
                     "fused_us_32_heads": fused_us, "materialised_products_us_32_heads": qk_us + pv_us * heads,
                     "fused_tflops": 3 * 2.0 * heads * S * S * hd / fused_us / 1e6,
                     "fused_note": "flops counted: Q K^T twice (two walks over the keys) + P V; warp-level bf16 MMA"}
        del P, Aq, Bk
        bd.poll_status()

    if rank != 0:
        return
    cpu = None
    if world == 1 or True:
        import oracle
        oracle.build()
        f = s = 0.0
        t_end = time.perf_counter() + 12.0
        n = 0
        while n < 1 or (time.perf_counter() < t_end and n < 8):
            ff, ss, threads = oracle_step_sample(16)
            f += ff
            s += ss
            n += 1
        cpu = {"value": f / s / 1e12, "unit": "TFLOP/s", "cores": threads, "kind": "oracle",
               "sample": f"{n} passes over 16 tokens x 4 layers (quantise + dequantise + fp64 product)",
               "act_quantizer": oracle_quantizer_baseline()}

    line = {
        "metric": "bd_linear_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "ms_per_step_median": step_median,
        "ms_per_step_best": step_best, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "e4m3 x e4m3 (exact DialectFP4 decode), fp32 accumulate", "data": "synthetic",
        "config": {"workload": "llama3-8b linear layers (q/o, k/v, gate/up, down), M=2048 tokens per GPU, "
                               "online two-stage quantise kernel + W4A4 tensor-core product kernel per layer "
                               "(linked by programmatic dependent launch), bf16 out",
                   "l2": f"working set {footprint / 2**20:.0f} MiB per step cycles through 4 layers (> 126 MB L2)",
                   "weights": "offline two-stage rule", "block": 32},
        "clocks": clocks,
        # the whole step (quantizers included, per GPU) against dense-FP8 figures derived from the bf16 peaks:
        # twice the burst and twice the sustained (seconds-long, power-capped) measured bf16 rate, and the nominal 4500
        "step_vs_fp8_peaks": {"of_2x_bf16_burst": value / world / (2.0 * peaks["bf16_tflops"]),
                              "of_2x_bf16_sustained": value / world / (2.0 * peaks["bf16_tflops_sustained"]),
                              "of_nominal_4500": value / world / 4500.0, "peak_source": peaks["source"]},
        "sustained": {"steps": sustained_steps, "ms_per_step": sustained_ms, "value": sustained_value, "unit": "TFLOP/s",
                      "of_2x_bf16_sustained": sustained_value / world / (2.0 * peaks["bf16_tflops_sustained"])},
        "e2e": {"value": e2e_value, "unit": "TFLOP/s", "ms_per_step": e2e_ms, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "act_quantizer": act_quantizer,
        "cpu_baseline": cpu,
        "per_layer_gflop": {l["name"]: l["flops"] / 1e9 for l in layers},
        "llama2_mlp_m_sweep": sweep,
        "decode_block": decode_block,
        "chained_layers": chained,
        "block_sizes": block_sizes,
        "kv_cache": kv_cache,
        "attention_mistral7b": attention,
    }
    print(json.dumps(line))
    replicas.shutdown()


def _lib_override():
    """BDLIB=<path>: load another build of the library (A/B timing of work-in-progress kernels)."""
    if os.environ.get("BDLIB"):
        from paper_2501_01144_b200 import binding
        binding._LIB_PATH = os.environ["BDLIB"]


def run_case(args):
    """A few launches of one kernel family on a small, fixed case (for ncu captures).
    quantizer: bd_quantize_act on bf16 [8192, 4096] (168 MiB of buffers in rotation).
    quantizer_f32: bd_quantize_act on fp32 [4096, 4096] (three buffer sets in rotation).
    linear_<layer>: bd_linear of one LLaMA3-8B layer at M = 2048 (layer in qo_proj, kv_proj, gate_up, down).
    decode: bd_linear of 16 tokens against K = 11008, N = 4096.  quantizer_strided: the token-axis quantizer on V [4096, 128].
    requant_gate_up: bd_linear_requant of the gate/up layer.  attention: bd_attention on four heads of 4096 tokens."""
    import torch

    import paper_2501_01144_b200 as bd
    from paper_2501_01144_b200 import inputs

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)

    def dev_bf16(bits):
        return torch.from_numpy(bits.view(np.int16)).to(dev).view(torch.bfloat16)

    reps = args.steps
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if args.case == "quantizer":
        qm, qk = QUANT_SHAPE
        xs = [dev_bf16(inputs.act_normal_outliers(qm, qk, seed=1 + s)) for s in range(2)]
        qs = [bd.QTensor(qm, qk, dev) for _ in range(2)]
        for i in range(args.warmup):
            bd.quantize_act(xs[i % 2], out=qs[i % 2])
        torch.cuda._sleep(4_000_000)                      # GPU head start: events see kernel time, not launch rate
        e0.record()
        for i in range(reps):
            bd.quantize_act(xs[i % 2], out=qs[i % 2])
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) / reps * 1e3
        print(json.dumps({"case": args.case, "us_per_launch": us,
                          "GB/s": qm * qk * BYTES_PER_ELEM_QUANT / us / 1e3}))
        return
    if args.case == "quantizer_f32":
        # fp32 source (the attention probabilities of the PV product): [4096, 4096], three buffer sets in rotation
        g = torch.Generator(device=dev)
        g.manual_seed(1)
        xs = [torch.rand(4096, 4096, device=dev, generator=g) for _ in range(3)]
        qs = [bd.QTensor(4096, 4096, dev) for _ in range(3)]
        for i in range(args.warmup):
            bd.quantize_act(xs[i % 3], out=qs[i % 3])
        torch.cuda._sleep(4_000_000)
        e0.record()
        for i in range(reps):
            bd.quantize_act(xs[i % 3], out=qs[i % 3])
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) / reps * 1e3
        print(json.dumps({"case": args.case, "us_per_launch": us, "GB/s": 4096 * 4096 * 4.546875 / us / 1e3}))
        return
    if args.case == "step":
        # the benchmark step alone: the four layers through bd_linear, nothing else on the GPU
        ls = []
        for i, (_, K, N) in enumerate(LAYERS):
            ls.append((dev_bf16(inputs.act_student_t(M_TOKENS, K, seed=2 + i)),
                       bd.quantize_weights(dev_bf16(inputs.weights_normal(N, K, seed=2 + i)), bd.SELECT_TWO_STAGE),
                       torch.empty(M_TOKENS, N, dtype=torch.bfloat16, device=dev),
                       torch.empty(bd.linear_workspace_size(M_TOKENS, N, K), dtype=torch.uint8, device=dev)))
        for it in range(args.warmup + reps):
            if it == args.warmup:
                e0.record()
            for x, wq, y, ws in ls:
                bd.linear(x, wq, out=y, workspace=ws)
        e1.record()
        torch.cuda.synchronize()
        print(json.dumps({"case": args.case, "us_per_step": e0.elapsed_time(e1) / reps * 1e3}))
        return
    if args.case in ("decode", "decode8"):
        # a decode-sized call of the LLaMA2 MLP sweep, six weight copies in rotation.  decode: 16 tokens against
        # K = 11008, N = 4096 (tensor-core path with a K split); decode8: 8 tokens against K = 4096, N = 11008 (the
        # warp-level kernel)
        K, N, M = (11008, 4096, 16) if args.case == "decode" else (4096, 11008, 8)
        wsrc = dev_bf16(inputs.weights_normal(N, K, seed=3))
        wqs = [bd.quantize_weights(wsrc, bd.SELECT_TWO_STAGE) for _ in range(6)]
        x = dev_bf16(inputs.act_post_silu(M, K, seed=3))
        y = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
        ws = torch.empty(bd.linear_workspace_size(M, N, K), dtype=torch.uint8, device=dev)
        for i in range(args.warmup):
            bd.linear(x, wqs[i % 6], out=y, workspace=ws)
        e0.record()
        for i in range(reps):
            bd.linear(x, wqs[i % 6], out=y, workspace=ws)
        e1.record()
        torch.cuda.synchronize()
        print(json.dumps({"case": args.case, "us_per_call": e0.elapsed_time(e1) / reps * 1e3}))
        return
    if args.case == "kv_attention":
        # the attention of one decode step over 8 cached KV heads x 4113 tokens x 128, 4 query rows per head
        rng = np.random.default_rng(6)
        kvh, grp, hd, n_tok, cap = 8, 4, 128, 4113, 4224
        caches = []
        for g in range(kvh):
            c = bd.KVCache(cap, hd, device=dev)
            c.append(dev_bf16(inputs.to_bf16_bits(rng.standard_normal((n_tok, hd)).astype(np.float32))),
                     dev_bf16(inputs.to_bf16_bits(rng.standard_normal((n_tok, hd)).astype(np.float32))))
            caches.append(c)
        qs = [bd.quantize_act(dev_bf16(inputs.to_bf16_bits(rng.standard_normal((grp, hd)).astype(np.float32)))) for _ in range(kvh)]
        o = torch.empty(kvh, grp, hd, dtype=torch.bfloat16, device=dev)
        for _ in range(args.warmup):
            bd.kvcache_attention(caches, qs, hd ** -0.5, out=o)
        e0.record()
        for _ in range(reps):
            bd.kvcache_attention(caches, qs, hd ** -0.5, out=o)
        e1.record()
        torch.cuda.synchronize()
        print(json.dumps({"case": args.case, "us_per_call": e0.elapsed_time(e1) / reps * 1e3}))
        return
    if args.case == "quantizer_strided":
        # the value matrix of one KV head, blocks along the token axis: V [4096 tokens, 128] bf16 -> operand [128, 4096]
        vs = [dev_bf16(inputs.to_bf16_bits(np.random.default_rng(s).standard_normal((4096, 128)).astype(np.float32))) for s in range(2)]
        qs = [bd.QTensor(128, 4096, dev) for _ in range(2)]
        for i in range(args.warmup):
            bd.quantize_act(vs[i % 2], axis=bd.AXIS_STRIDED, out=qs[i % 2])
        e0.record()
        for i in range(reps):
            bd.quantize_act(vs[i % 2], axis=bd.AXIS_STRIDED, out=qs[i % 2])
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) / reps * 1e3
        print(json.dumps({"case": args.case, "us_per_launch": us, "GB/s": 4096 * 128 * BYTES_PER_ELEM_QUANT / us / 1e3}))
        return
    if args.case == "requant_gate_up":
        # the gate/up layer at M = 2048 with the requantising epilogue
        K, N = 4096, 14336
        x = dev_bf16(inputs.act_student_t(M_TOKENS, K, seed=2))
        wq = bd.quantize_weights(dev_bf16(inputs.weights_normal(N, K, seed=2)), bd.SELECT_TWO_STAGE)
        hq = bd.QTensor(M_TOKENS, N, dev)
        ws = torch.empty(bd.linear_requant_workspace_size(M_TOKENS, N, K), dtype=torch.uint8, device=dev)
        for _ in range(args.warmup):
            bd.linear_requant(x, wq, out=hq, workspace=ws)
        e0.record()
        for _ in range(reps):
            bd.linear_requant(x, wq, out=hq, workspace=ws)
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) / reps * 1e3
        print(json.dumps({"case": args.case, "us_per_call": us, "TFLOP/s": 2.0 * M_TOKENS * N * K / us / 1e6}))
        return
    if args.case == "attention":
        # the fused attention kernel on four query heads of one KV head, 4096 tokens, head_dim 128
        rng = np.random.default_rng(0)
        mk = lambda n: inputs.to_bf16_bits(rng.standard_normal((n, 4096, 128)).astype(np.float32))
        Qb, Kb, Vb = mk(4), mk(1), mk(1)
        Qs = [bd.quantize_act(dev_bf16(Qb[h])) for h in range(4)]
        Ks = [bd.quantize_act(dev_bf16(Kb[0]))]
        Vs = [bd.quantize_act(dev_bf16(Vb[0]), axis=bd.AXIS_STRIDED)]
        o = torch.empty(4, 4096, 128, dtype=torch.bfloat16, device=dev)
        for _ in range(args.warmup):
            bd.attention(Qs, Ks, Vs, group=4, out=o)
        e0.record()
        for _ in range(reps):
            bd.attention(Qs, Ks, Vs, group=4, out=o)
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) / reps * 1e3
        print(json.dumps({"case": args.case, "us_per_call": us, "TFLOP/s": 3 * 2.0 * 4 * 4096 * 4096 * 128 / us / 1e6}))
        return
    name = args.case[len("linear_"):]
    K, N = {n: (k, nn) for n, k, nn in LAYERS}[name]
    x = dev_bf16(inputs.act_student_t(M_TOKENS, K, seed=2))
    wq = bd.quantize_weights(dev_bf16(inputs.weights_normal(N, K, seed=2)), bd.SELECT_TWO_STAGE)
    y = torch.empty(M_TOKENS, N, dtype=torch.bfloat16, device=dev)
    ws = torch.empty(bd.linear_workspace_size(M_TOKENS, N, K), dtype=torch.uint8, device=dev)
    for _ in range(args.warmup):
        bd.linear(x, wq, out=y, workspace=ws)
    e0.record()
    for _ in range(reps):
        bd.linear(x, wq, out=y, workspace=ws)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) / reps * 1e3
    print(json.dumps({"case": args.case, "us_per_call": us, "TFLOP/s": 2.0 * M_TOKENS * N * K / us / 1e6}))


def spawn_ranks(args):
    """`python bench.py --gpus N` outside torchrun: re-run this file as N ranks of one node (one process per
    GPU, rendezvous on 127.0.0.1 at a free port).  Rank 0 prints the JSON line; the exit code is the job's."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__),
           "--gpus", str(args.gpus), "--steps", str(args.steps), "--warmup", str(args.warmup), "--impl", args.impl]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--case", default=None,
                    choices=["quantizer", "quantizer_f32", "step", "decode", "decode8", "kv_attention", "quantizer_strided", "requant_gate_up", "attention"]
                    + ["linear_" + n for n, _, _ in LAYERS],
                    help="run a few launches of one small case (for profiler captures) instead of the benchmark")
    args = ap.parse_args()
    _lib_override()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.case:
        # started as a plain process: start the N ranks here, one per GPU, the way torchrun would
        sys.exit(spawn_ranks(args))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.case:
        run_case(args)
        return
    run_gpu(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
