#!/usr/bin/env python
"""Benchmark of the HiF4 W4A4 linear-layer hot path (hif4_quantize + hif4_gemm) on B200.

One "step" is one pass over the Llama-3-8B-shaped linears (K=4096 -> N in {4096, 1024, 14336} and
K=14336 -> N=4096) for M in {1, 16, 4096} tokens: for each (M, K, N) the BF16 activations are
quantized to HiF4 (Algorithm 1) and multiplied with the pre-quantized HiF4 weights (Eq. 3, FP32
accumulation).  All inputs are seeded synthetic tensors (Student-t activations with outlier
channels, Gaussian weights); the model name only lends the layer shapes.

Prints ONE JSON line: metric, value (whole-job TFLOP/s with inputs resident), ms_per_step, gpu_launches, clocks,
roofline (the prefill GEMM kernel against the measured BF16 peak), per_shape, roofline_quantize, reference_points,
e2e (through host buffers) and cpu_baseline.  `--impl reference` times the CPU oracle
on a bounded sample of the same workload instead.
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

import torch  # noqa: E402

import hif4_workloads as wl  # noqa: E402

METRIC = "hif4_gemm TFLOP/s + hif4_quantize GB/s at LLM shapes, % of roofline (1 B200)"
WORKLOAD = "llama3_8b_linears: K=4096 N in {4096,1024,14336} + K=14336 N=4096, M in {1,16,4096}"
SHAPES = [(M, K, N, name) for M in wl.LLAMA3_8B_M for (name, K, N) in wl.LLAMA3_8B_LINEARS]
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under
# profiles/ (None until a capture exists for that kernel).
NCU_DRAM_BYTES_PER_LAUNCH = {"gemm_tc2_kernel": 264.1e6,      # captured on M=4096 N=14336 K=4096 (algorithmic 277.3e6)
                             "quantize_bf16_kernel@2^28": 659.0e6}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"]))}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self, t0: float = 0.0, t1: float = float("inf")) -> dict:
        """Summary of the samples taken between host times t0 and t1 (the timed region)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        if self.thread:
            self.thread.join(timeout=2)
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for (ts, r) in self.rows:
            if len(r) < 7 or ts < t0 or ts > t1 + 0.05:
                continue
            try:
                sm.append(float(r[0])); smax.append(float(r[1]))
            except ValueError:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def flops(M, K, N):
    return 2.0 * M * N * K


def quant_bytes(M, K):
    return M * K * 2.5625          # 2 B read + 36/64 B written per BF16 element


def gemm_min_bytes(M, K, N):
    return 0.5625 * (M + N) * K + 4.0 * M * N


# --------------------------------------------------------------------------------------- own arm
def run_cuda(args):
    import paper_2602_11287_b200 as hif4

    from paper_2602_11287_b200 import dp
    rank, local_rank, world = dp.rank_info()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the HiF4 path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    peaks, peak_kind = load_peaks()

    # ---- resident inputs: every rank holds its own batch of tokens (data parallel, no exchange)
    weights = {}
    for (name, K, N) in wl.LLAMA3_8B_LINEARS:
        w = wl.gaussian(N, K, 0.02, seed=2000 + N + K, device=dev)
        weights[(K, N)] = hif4.hif4_quantize(w)
        del w
    acts, xq, cs = {}, {}, {}
    for (M, K, N, name) in SHAPES:
        if (M, K) not in acts:
            acts[(M, K)] = wl.llama_activations(M, K, seed=dp.rank_seed(1002 + M + K, rank), device=dev)
        xq[(M, K, N)] = torch.empty(M, K // 64, 36, dtype=torch.uint8, device=dev)
        cs[(M, K, N)] = torch.empty(M, N, dtype=torch.float32, device=dev)
    # one scratch buffer for the GEMM workspaces (stream-ordered reuse)
    ws = torch.empty(max(max(max(hif4.hif4_gemm_workspace(M, N, K), hif4.hif4_linear_workspace(M, N, K) if M <= 16 else 0)
                             for (M, K, N, _) in SHAPES), 256), dtype=torch.uint8, device=dev)
    torch.cuda.synchronize()

    stream = torch.cuda.current_stream()
    # Step order: M=1 linears, two prefill linears, M=16 linears, two prefill linears -- more than the
    # 126 MB of L2 is touched between two uses of any weight matrix (M=1 and M=16 share theirs).
    big = [sh for sh in SHAPES if sh[0] >= 4096]
    groups = [[sh for sh in SHAPES if sh[0] == 1], big[:2], [sh for sh in SHAPES if sh[0] == 16], big[2:]]
    small = groups[0] + groups[2]                       # decode-shaped: microseconds per kernel, launch-bound
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def run_shapes(shapes, events=None):
        for (M, K, N, name) in shapes:
            if events is not None:
                e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
                e0.record(stream)
            hif4.hif4_quantize(acts[(M, K)], out=xq[(M, K, N)])
            if events is not None:
                e1.record(stream)
            hif4.hif4_gemm(xq[(M, K, N)], weights[(K, N)], out=cs[(M, K, N)], workspace=ws)
            if events is not None:
                e2.record(stream)
                events.append(((M, K, N), e0, e1, e2))

    def run_linears(shapes):
        """The same work through the one-call linear layer (quantize + GEMM): for M <= 16 the activations are
        quantized inside the token preparation of the weight-streaming kernel, one launch fewer per linear."""
        for (M, K, N, name) in shapes:
            hif4.hif4_linear(acts[(M, K)], weights[(K, N)], out=cs[(M, K, N)], workspace=ws)

    def barrier():
        dp.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(max(args.warmup, 3)):
        run_shapes(SHAPES)
    run_linears(small)
    barrier()

    # The launches of the decode-shaped linears are captured once into two CUDA graphs (M=1, M=16) and
    # replayed every step (their kernels run a few microseconds each, so launch gaps would dominate);
    # the four prefill linears are launched directly, with events around them for the roofline.
    graphs, graph_launches = {}, 0
    if not args.no_graph:
        for gi in (0, 2):
            n0 = hif4.launch_count()
            graphs[gi] = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graphs[gi]):
                run_linears(groups[gi])
            graph_launches += hif4.launch_count() - n0
        torch.cuda.synchronize()

    def step(events=None):
        for gi, shapes in enumerate(groups):
            if gi in graphs:
                graphs[gi].replay()
            elif gi in (0, 2):
                run_linears(shapes)
            else:
                run_shapes(shapes, events)

    step()
    barrier()
    events = []
    launches0 = hif4.launch_count()
    barrier()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    host_t0 = time.time()
    t_start.record(stream)
    for _ in range(args.steps):
        step(events)
    t_end.record(stream)
    barrier()
    host_t1 = time.time()
    launches = hif4.launch_count() - launches0 + graph_launches * args.steps
    clocks = sampler.stop(host_t0, host_t1)
    elapsed_ms = dp.max_over_ranks(t_start.elapsed_time(t_end), dev)
    status = hif4.hif4_last_device_status()
    if status != 0:
        raise SystemExit(f"device status {status}: {hif4.status_string(status)}")

    # per-kernel times of the decode-shaped linears: a separate pass with events around every call and
    # L2 flushed (a 256 MB write) before each linear
    small_events = []
    for _ in range(20):
        for sh in small:
            flush.zero_()
            run_shapes([sh], small_events)
    torch.cuda.synchronize()
    events += small_events

    step_flops = sum(flops(M, K, N) for (M, K, N, _) in SHAPES)
    ms_per_step = elapsed_ms / args.steps
    value = dp.job_throughput(step_flops, world, ms_per_step * 1e-3) / 1e12

    # ---- per-kernel times (prefill shapes: inside the timed region; decode shapes: the pass above)
    per_shape = {}
    for (shape, e0, e1, e2) in events:
        d = per_shape.setdefault(shape, [0.0, 0.0, 0])
        d[0] += e0.elapsed_time(e1); d[1] += e1.elapsed_time(e2); d[2] += 1
    table = []
    tc_flops = tc_ms = 0.0
    for (M, K, N, name) in SHAPES:
        q_ms, g_ms, n = per_shape[(M, K, N)]
        q_ms /= n; g_ms /= n
        row = {"M": M, "K": K, "N": N, "quantize_us": round(q_ms * 1e3, 2), "gemm_us": round(g_ms * 1e3, 2),
               "gemm_tflops": round(flops(M, K, N) / g_ms / 1e9, 2),
               "gemm_min_traffic_gbs": round(gemm_min_bytes(M, K, N) / g_ms / 1e6, 1)}
        if M >= 4096:
            tc_flops += flops(M, K, N); tc_ms += g_ms
            row["frac_of_bf16_peak"] = round(flops(M, K, N) / g_ms / 1e9 / peaks["bf16_tflops_sustained"], 3)
        else:
            row["frac_of_hbm_peak"] = round(gemm_min_bytes(M, K, N) / g_ms / 1e6 / peaks["hbm_gbs"], 3)
        table.append(row)
    achieved = tc_flops / tc_ms / 1e9
    roofline = {"bound": "tensor", "kernel": "gemm_tc2_kernel (M=4096 launches)", "achieved": round(achieved, 1),
                "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                "frac": round(achieved / peaks["bf16_tflops_sustained"], 4),
                "frac_of_burst_peak": round(achieved / peaks["bf16_tflops"], 4), "peak_kind": f"of {peak_kind} (sustained)",
                "traffic": NCU_DRAM_BYTES_PER_LAUNCH["gemm_tc2_kernel"],
                "traffic_note": "dram bytes of the M=4096 N=14336 K=4096 launch (profiles/gemm_tc2_kernel_4096x14336x4096.md)"}

    out = {
        "metric": METRIC, "value": round(value, 2), "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": round(ms_per_step, 4), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16 x bf16 -> f32 (HiF4 decoded exactly to bf16)",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "weights": "pre-quantized to HiF4, resident",
                   "l2": "no flush: the step order (M=1 linears, two prefill linears, M=16 linears, two prefill linears) "
                         "touches > 126 MB (L2) between two uses of any tensor; per_shape rows with M <= 16 come from "
                         "a separate pass that writes 256 MB before each linear",
                   "launch": ("decode-shaped linears (hif4_linear, two kernels each) replayed from two CUDA graphs per step, "
                              "prefill linears (hif4_quantize + hif4_gemm) launched directly"
                              if graphs else "every kernel launched directly (hif4_linear for M <= 16, hif4_quantize + hif4_gemm for M = 4096)"),
                   "parallelism": f"dp{world} (independent token batches, no collective)"},
        "gpu_launches": int(launches), "clocks": clocks, "roofline": roofline, "per_shape": table,
    }

    if rank == 0 and world == 1:
        out["roofline_quantize"] = measure_quantize_roofline(hif4, dev, peaks, peak_kind)
        out["reference_points"] = measure_reference_points(dev)
    out["e2e"] = measure_e2e(hif4, dev, weights, world, args)
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline_sample()
        print(json.dumps(out))
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


def measure_quantize_roofline(hif4, dev, peaks, peak_kind):
    """hif4_quantize alone on the config-3 tensor (2^28 BF16 elements, 512 MiB in: larger than L2)."""
    n = 2 ** 28
    x = wl.quantize_sweep(n, device=dev)
    out = torch.empty(n // 4096, 64, 36, dtype=torch.uint8, device=dev)
    for _ in range(3):
        hif4.hif4_quantize(x, out=out)
    torch.cuda.synchronize()
    reps = 20
    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s.record()
    for _ in range(reps):
        hif4.hif4_quantize(x, out=out)
    e.record()
    torch.cuda.synchronize()
    ms = s.elapsed_time(e) / reps
    gbs = n * 2.5625 / ms / 1e6
    del x, out
    return {"bound": "hbm", "kernel": "quantize_bf16_kernel, 2^28 elements (config 3 mix)", "achieved": round(gbs, 1),
            "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": round(gbs / peaks["hbm_gbs"], 4),
            "peak_kind": f"of {peak_kind}", "frac_of_nominal_8tbs": round(gbs / 8000.0, 4),
            "traffic": NCU_DRAM_BYTES_PER_LAUNCH["quantize_bf16_kernel@2^28"], "us_per_launch": round(ms * 1e3, 1)}


def measure_reference_points(dev):
    """Context only: the same (M, N, K) through the box's library GEMMs -- native NVFP4 block-scaled
    (torch._scaled_mm on packed FP4 with one E4M3 scale per 16 values, random bits: time only) and BF16
    (torch.matmul).  Neither is part of the HiF4 path."""
    M, N, K = 4096, 14336, 4096
    out = {"shape": [M, N, K]}

    def timed(fn):
        fn(); torch.cuda.synchronize()
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        for _ in range(20):
            fn()
        e.record(); torch.cuda.synchronize()
        us = s.elapsed_time(e) / 20 * 1e3
        return {"us": round(us, 1), "tflops": round(flops(M, K, N) / us / 1e6, 1)}

    try:
        a = torch.randint(0, 255, (M, K // 2), dtype=torch.uint8, device=dev).view(torch.float4_e2m1fn_x2)
        b = torch.randint(0, 255, (N, K // 2), dtype=torch.uint8, device=dev).view(torch.float4_e2m1fn_x2)
        cols = (K // 16 + 3) // 4 * 4
        sa = torch.ones(((M + 127) // 128 * 128) * cols, device=dev).to(torch.float8_e4m3fn)
        sb = torch.ones(((N + 127) // 128 * 128) * cols, device=dev).to(torch.float8_e4m3fn)
        out["nvfp4_scaled_mm"] = timed(lambda: torch._scaled_mm(a, b.t(), sa, sb, out_dtype=torch.bfloat16))
    except Exception as ex:                                   # noqa: BLE001 - any failure means "not on this box"
        out["nvfp4_scaled_mm"] = {"unavailable": f"{type(ex).__name__}: {str(ex)[:120]}"}
    try:
        a = torch.randn(M, K, device=dev, dtype=torch.bfloat16)
        b = torch.randn(N, K, device=dev, dtype=torch.bfloat16)
        out["bf16_matmul"] = timed(lambda: torch.matmul(a, b.t()))
    except Exception as ex:                                   # noqa: BLE001
        out["bf16_matmul"] = {"unavailable": f"{type(ex).__name__}: {str(ex)[:120]}"}
    return out


def measure_e2e(hif4, dev, weights, world, args):
    """Same step through the public API with HOST buffers: pinned BF16 activations copied in, FP32
    results copied out, every step; copies and kernels overlap on three streams."""
    host_x, dev_x, host_c, dev_c, dev_q = {}, {}, {}, {}, {}
    for (M, K, N, name) in SHAPES:
        if (M, K) not in host_x:
            host_x[(M, K)] = wl.llama_activations(M, K, seed=77 + M + K).pin_memory()
            dev_x[(M, K)] = torch.empty(M, K, dtype=torch.bfloat16, device=dev)
        host_c[(M, K, N)] = torch.empty(M, N, dtype=torch.float32).pin_memory()
        dev_c[(M, K, N)] = torch.empty(M, N, dtype=torch.float32, device=dev)
        dev_q[(M, K, N)] = torch.empty(M, K // 64, 36, dtype=torch.uint8, device=dev)
    ws = torch.empty(max(max(hif4.hif4_gemm_workspace(M, N, K) for (M, K, N, _) in SHAPES), 256), dtype=torch.uint8, device=dev)
    h2d = sum(t.numel() * 2 for t in host_x.values())
    d2h = sum(t.numel() * 4 for t in host_c.values())

    # Three streams: pinned activations in, kernels, results out.  Events order each buffer's reuse: the
    # kernels of a shape wait for its activations, the copy-out waits for its GEMM, the next step's GEMM
    # waits until the previous result has left, the next step's copy-in until the quantizers have read.
    compute = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    in_ready = {k: torch.cuda.Event() for k in host_x}
    x_consumed = {k: torch.cuda.Event() for k in host_x}
    c_ready = {k: torch.cuda.Event() for k in host_c}
    c_left = {k: torch.cuda.Event() for k in host_c}
    last_user = {}
    for (M, K, N, name) in SHAPES:
        last_user[(M, K)] = (M, K, N)
    state = {"first": True}

    def step():
        with torch.cuda.stream(s_in):
            for key, t in host_x.items():
                if not state["first"]:
                    s_in.wait_event(x_consumed[key])
                dev_x[key].copy_(t, non_blocking=True)
                in_ready[key].record(s_in)
        for (M, K, N, name) in SHAPES:
            compute.wait_event(in_ready[(M, K)])
            hif4.hif4_quantize(dev_x[(M, K)], out=dev_q[(M, K, N)])
            if last_user[(M, K)] == (M, K, N):
                x_consumed[(M, K)].record(compute)
            if not state["first"]:
                compute.wait_event(c_left[(M, K, N)])
            hif4.hif4_gemm(dev_q[(M, K, N)], weights[(K, N)], out=dev_c[(M, K, N)], workspace=ws)
            c_ready[(M, K, N)].record(compute)
            with torch.cuda.stream(s_out):
                s_out.wait_event(c_ready[(M, K, N)])
                host_c[(M, K, N)].copy_(dev_c[(M, K, N)], non_blocking=True)
                c_left[(M, K, N)].record(s_out)
        state["first"] = False

    def join():
        for ev in c_left.values():
            compute.wait_event(ev)

    steps = max(3, min(args.steps, 10))
    for _ in range(2):
        step()
    join()
    torch.cuda.synchronize()
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s.record()
    for _ in range(steps):
        step()
    join()                                   # the step is over when its last result has reached the host
    e.record()
    torch.cuda.synchronize()
    ms = s.elapsed_time(e) / steps
    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    step_flops = sum(flops(M, K, N) for (M, K, N, _) in SHAPES)
    return {"value": round(world * step_flops / (ms * 1e-3) / 1e12, 2), "unit": "TFLOP/s", "ms_per_step": round(ms, 3),
            "steps": steps, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h)}


# ------------------------------------------------------------------------------ CPU oracle legs
ORACLE_SAMPLE_ROWS, ORACLE_SAMPLE_COLS = 16, 128


def _oracle_sample_inputs():
    """For every linear of the workload: 16 activation rows and 128 weight rows at full K."""
    items = []
    for (name, K, N) in wl.LLAMA3_8B_LINEARS:
        x = wl.bf16_to_u16_numpy(wl.llama_activations(ORACLE_SAMPLE_ROWS, K, seed=1002 + K))
        w = wl.bf16_to_u16_numpy(wl.gaussian(ORACLE_SAMPLE_COLS, K, 0.02, seed=2000 + N + K))
        items.append((K, x, w))
    return items


def _oracle_step(oracle, items, threads):
    fl = 0.0
    for (K, x, w) in items:
        xq = oracle.quantize(x, nthreads=threads)
        wq = oracle.quantize(w, nthreads=threads)
        oracle.gemm_f64(xq, wq, nthreads=threads, want_abs=False)
        fl += flops(x.shape[0], K, w.shape[0])
    return fl


def cpu_baseline_sample():
    import oracle
    threads = oracle.hardware_threads()
    items = _oracle_sample_inputs()
    _oracle_step(oracle, items, threads)
    t0 = time.perf_counter()
    reps, fl = 0, 0.0
    while time.perf_counter() - t0 < 10.0:
        fl += _oracle_step(oracle, items, threads)
        reps += 1
    dt = time.perf_counter() - t0
    return {"value": round(fl / dt / 1e12, 6), "unit": "TFLOP/s", "cores": threads, "kind": "oracle",
            "sample": f"{reps} passes over a slab of each linear: quantize {ORACLE_SAMPLE_ROWS} activation rows and "
                      f"{ORACLE_SAMPLE_COLS} weight rows at full K, FP64 GEMM of the slab ({dt:.1f} s of CPU work)"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    threads = oracle.hardware_threads()
    items = _oracle_sample_inputs()
    warm = max(args.warmup, 1)
    for _ in range(warm):
        _oracle_step(oracle, items, threads)
    t0 = time.perf_counter()
    fl = 0.0
    for _ in range(args.steps):
        fl += _oracle_step(oracle, items, threads)
    dt = time.perf_counter() - t0
    value = round(fl / dt / 1e12, 6)
    sample = (f"per step: for each of the 4 linears quantize {ORACLE_SAMPLE_ROWS} activation rows and "
              f"{ORACLE_SAMPLE_COLS} weight rows at full K and multiply the slab in FP64")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s",
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": warm,
        "ms_per_step": round(dt / args.steps * 1e3, 3), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64 (CPU oracle)", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_case(spec: str):
    """Small single-kernel cases: what the ncu summaries under profiles/ were captured from."""
    import paper_2602_11287_b200 as hif4
    kind, _, rest = spec.partition(":")
    nums = [int(v) for v in rest.split(",") if v]
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    reps = 20
    if kind == "gemm":
        M, N, K = nums
        a = hif4.hif4_quantize(wl.llama_activations(M, K, device=dev))
        b = hif4.hif4_quantize(wl.gaussian(N, K, 0.02, seed=5, device=dev))
        c = torch.empty(M, N, dtype=torch.float32, device=dev)
        ws = torch.empty(max(hif4.hif4_gemm_workspace(M, N, K), 256), dtype=torch.uint8, device=dev)
        fn = lambda: hif4.hif4_gemm(a, b, out=c, workspace=ws)
        work = f"{flops(M, K, N) / 1e9:.1f} GFLOP, min traffic {gemm_min_bytes(M, K, N) / 1e6:.1f} MB"
    elif kind in ("quantize32", "dequantize32"):
        n = 2 ** nums[0]
        x = wl.quantize_sweep(n, device=dev, dtype=torch.float32)
        q = torch.empty(n // 4096, 64, 36, dtype=torch.uint8, device=dev)
        hif4.hif4_quantize(x, out=q)
        fn = (lambda: hif4.hif4_quantize(x, out=q)) if kind == "quantize32" else (lambda: hif4.hif4_dequantize(q, out=x))
        work = f"{n * 4.5625 / 1e6:.1f} MB"
    elif kind == "quantizeT":                       # units down the columns of a [4096, n / 4096] matrix
        n = 2 ** nums[0]
        x = wl.quantize_sweep(n, device=dev).view(4096, n // 4096)
        q = torch.empty(n // 4096, 64, 36, dtype=torch.uint8, device=dev)
        fn = lambda: hif4.hif4_quantize_transposed(x, out=q)
        work = f"{n * 2.5625 / 1e6:.1f} MB"
    elif kind == "quantizeT32":                     # the same from an FP32 source
        n = 2 ** nums[0]
        x = wl.quantize_sweep(n, device=dev, dtype=torch.float32).view(4096, n // 4096)
        q = torch.empty(n // 4096, 64, 36, dtype=torch.uint8, device=dev)
        fn = lambda: hif4.hif4_quantize_transposed(x, out=q)
        work = f"{n * 4.5625 / 1e6:.1f} MB"
    elif kind == "quantize16":                      # FP16 source (widened to FP32 inside the kernel)
        n = 2 ** nums[0]
        x = wl.quantize_sweep(n, device=dev).to(torch.float16)
        q = torch.empty(n // 4096, 64, 36, dtype=torch.uint8, device=dev)
        fn = lambda: hif4.hif4_quantize(x, out=q)
        work = f"{n * 2.5625 / 1e6:.1f} MB"
    elif kind in ("quantize", "dequantize"):
        n = 2 ** nums[0]
        x = wl.quantize_sweep(n, device=dev)
        q = torch.empty(n // 4096, 64, 36, dtype=torch.uint8, device=dev)
        hif4.hif4_quantize(x, out=q)
        fn = (lambda: hif4.hif4_quantize(x, out=q)) if kind == "quantize" else (lambda: hif4.hif4_dequantize(q, out=x))
        work = f"{n * 2.5625 / 1e6:.1f} MB"
    elif kind == "grouped":
        tokens, experts, N, K = nums
        r = wl.moe_routing(tokens=tokens, experts=experts, topk=min(8, experts), device=dev)
        total = int(r["offsets"][-1])
        a = hif4.hif4_quantize(wl.outlier_channel_activations(total, K, seed=3, device=dev))
        b = torch.empty(experts, N, K // 64, 36, dtype=torch.uint8, device=dev)
        for e0 in range(0, experts, 16):                    # BF16 sources are drawn 16 experts at a time
            n_e = min(16, experts - e0)
            hif4.hif4_quantize(wl.gaussian(n_e * N, K, 0.02, seed=4 + e0, device=dev), out=b[e0:e0 + n_e].view(n_e * N, K // 64, 36))
        c = torch.empty(total, N, dtype=torch.float32, device=dev)
        ws = torch.empty(max(hif4.hif4_grouped_gemm_workspace(experts, total, N, K), 1), dtype=torch.uint8, device=dev)
        fn = lambda: hif4.hif4_grouped_gemm(a, b, r["offsets"], out=c, workspace=ws)
        work = f"{flops(total, K, N) / 1e9:.1f} GFLOP"
    else:
        raise SystemExit(f"unknown case {spec}")
    fn()
    torch.cuda.synchronize()
    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda._sleep(4_000_000)          # keeps the GPU busy while the host queues the launches below
    s.record()
    for _ in range(reps):
        fn()
    e.record()
    torch.cuda.synchronize()
    status = hif4.hif4_last_device_status()
    print(json.dumps({"case": spec, "work_per_launch": work, "us_per_launch": round(s.elapsed_time(e) / reps * 1e3, 2),
                      "device_status": status}))
    if status != 0:
        raise SystemExit(1)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch the decode-shaped linears directly instead of replaying a CUDA graph")
    ap.add_argument("--gemm-path", type=int, default=0, help="with --case: kernel selection, see hif4_debug_set_gemm_path")
    ap.add_argument("--case", default=None,
                    help="run one kernel a few times instead of the benchmark (for ncu captures): "
                         "gemm:M,N,K | quantize:LOG2_ELEMS | dequantize:LOG2_ELEMS | quantize32 / dequantize32 (FP32 side) | quantize16 (FP16 source) | quantizeT / quantizeT32 (column-wise units, BF16 / FP32 source) | "
                         "grouped:TOKENS,EXPERTS,N,K")
    args = ap.parse_args()
    if args.case:
        if args.gemm_path:
            import paper_2602_11287_b200 as hif4
            hif4.hif4_debug_set_gemm_path(args.gemm_path)
        run_case(args.case)
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
