#!/usr/bin/env python
"""Benchmark of the dual-basis PoT linear path on B200.

Default arm: the CUDA path through the C ABI. A "step" is one batch-1 decode pass over every
linear of a LLaMA-2-7B-shaped stack (32 layers x 7 linears = 224 W3/A16 GEMVs, group 128): about
3.2 GB of packed weights per step, far larger than L2, so every step streams from HBM.
`value` = algorithmic weight+activation bytes per step / device time (GB/s), summed over ranks.

`--impl reference`: the CPU oracle timed as it stands on a bounded sample of the same workload.

Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import synth_inputs as si  # noqa: E402

GROUP = 128
WBITS = 3
# what the timed kernel computes in: bf16 activations become 16-bit block fixed point (two int8 slices per value), the PoT
# weights small integers; sums are exact in int32, the coefficient multiply and the sum over macro-blocks are fp32
DTYPE = "int8 x int8 -> int32 (bf16 activations as 16-bit block fixed point), f32 coefficient stage"
METRIC = "w3a16_gemv_hbm_gbs"
UNIT = "GB/s"
WORKLOAD = "llama2-7b-shaped linear stack (32 layers x 7 linears), W3 dual-basis PoT, group 128, batch-1 decode GEMV"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        measured_peaks.sustained = float(p.get("bf16_tflops_sustained", 1400.0))
        return float(p["hbm_gbs"]), float(p.get("bf16_tflops", 1590.0)), "measured (MEASURED_PEAKS.json)"
    measured_peaks.sustained = 1400.0
    return 6650.0, 1590.0, "fallback (earlier measurement on this pool)"


def algorithmic_bytes(n, k, batch, y_bytes=4):
    """Weights (codes + 0.75-bit records + fp16 coefficient pairs) + activations in + outputs."""
    return n * k * (4 * WBITS + 3) // 32 + n * (k // GROUP) * 4 + batch * k * 2 + batch * n * y_bytes


# ---------------------------------------------------------------------------------------------
# clock sampling during the timed region (NVML, read-only)
# ---------------------------------------------------------------------------------------------
class ClockSampler:
    def __init__(self, device_index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "hw_power_brake": getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80),
        }
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons", None)
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                if get_reasons:
                    r = get_reasons(self.h)
                    for k, bit in names.items():
                        if r & bit:
                            self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.004)

    def __enter__(self):
        if self.nv:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ---------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and --impl reference)
# ---------------------------------------------------------------------------------------------
def oracle_sample(rows_per_linear=2048, seed=0):
    """One layer's seven linears restricted to `rows_per_linear` output rows each, batch 1."""
    items = []
    for i, (name, n, k) in enumerate(si.LLAMA2_7B_LINEARS):
        r = min(rows_per_linear, n)
        codes, meta, coef = si.random_quantized(r, k, GROUP, WBITS, seed=seed * 7 + i)
        x = si.bf16_bits_to_f64(si.bf16_activations(1, k, seed=100 + i))
        items.append((codes, meta, coef, x, algorithmic_bytes(r, k, 1)))
    return items


def time_oracle(items, repeats=1):
    from oracle import goq_oracle as O
    best = float("inf")
    for _ in range(repeats):
        t0 = time.perf_counter()
        for codes, meta, coef, x, _ in items:
            O.linear_f64(codes, meta, coef, x, GROUP, WBITS)
        best = min(best, time.perf_counter() - t0)
    nbytes = sum(it[4] for it in items)
    return nbytes / best / 1e9, best


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max((p.get("num_threads", 1) for p in threadpool_info()), default=1)
        return int(n)
    except Exception:
        return len(os.sched_getaffinity(0))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    items = oracle_sample()
    for _ in range(args.warmup):
        time_oracle(items)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time_oracle(items)
    dt = (time.perf_counter() - t0) / args.steps
    nbytes = sum(it[4] for it in items)
    val = nbytes / dt / 1e9
    sample = "one layer's 7 linears x 2048 output rows each, batch 1, per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------
# CUDA arm
# ---------------------------------------------------------------------------------------------
def build_stack(goq, torch, layers, seed0, batch):
    """Random W3 records generated on the device (seeded), packed by goq_pack."""
    gen = torch.Generator(device="cuda")
    stack = []
    for layer in range(layers):
        for idx, (name, n, k) in enumerate(si.LLAMA2_7B_LINEARS):
            gen.manual_seed(seed0 + layer * 7 + idx)
            d = goq.desc(n, k, GROUP, WBITS)
            codes = torch.randint(0, 1 << WBITS, (n, k), dtype=torch.uint8, device="cuda", generator=gen)
            meta = torch.randint(0, 64, (n, k // 8), dtype=torch.uint8, device="cuda", generator=gen)
            # coefficient scale for unit gain: with uniform codes E[b^2] = 0.33 per basis, so |W x| ~ |x| when the two
            # coefficients have standard deviation 1 / sqrt(0.66 k); a chain fed its own outputs then neither dies out nor overflows
            coef = (torch.randn((n, k // GROUP, 2), device="cuda", generator=gen) * (0.66 * k) ** -0.5).to(torch.float16)
            packed = torch.empty(goq.packed_bytes(d), dtype=torch.uint8, device="cuda")
            goq.pack(d, codes, meta, coef, packed)
            x = torch.randn((batch, k), device="cuda", generator=gen).to(torch.bfloat16)
            y = torch.empty((batch, n), dtype=torch.float32, device="cuda")
            stack.append({"d": d, "packed": packed, "x": x, "y": y, "n": n, "k": k,
                          "yb": torch.zeros((batch, n), dtype=torch.bfloat16, device="cuda")})
            build_stack.ws_bytes = max(getattr(build_stack, "ws_bytes", 256), goq.workspace_bytes(d, goq.OP_GEMV, 16))
            del codes, meta, coef
    torch.cuda.synchronize()
    return stack


def flow_items(goq, stack, x0=None, outs=None):
    """The decode step as a true chain: linear j reads the first k_j channels of linear j-1's bf16 output (the first one
    reads x0). No item is flagged: the library finds the dependencies from the address ranges."""
    items = []
    for j, s in enumerate(stack):
        y = outs[j] if outs is not None else s["yb"]
        if j == 0:
            x = x0 if x0 is not None else s["x"]
        else:
            prev = outs[j - 1] if outs is not None else stack[j - 1]["yb"]
            x = prev[:, :s["k"]]
        items.append((s["d"], s["packed"], x, 1, y, goq.BF16, False))
    return items


def capture(torch, fn):
    """Capture fn() (a sequence of library calls on the current stream) into a CUDA graph."""
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        fn()  # warm-up outside capture
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        fn()
    return g


def time_graph(torch, graph, steps, warmup):
    for _ in range(warmup):
        graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps  # ms per step


def time_loop_with_clocks(torch, fn, device_index, min_seconds=0.5, warmup=3):
    """Run fn() back to back for at least min_seconds with the clock sampler around the timed region.
    Returns (ms per call, clock summary)."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(); fn(); e1.record(); torch.cuda.synchronize()
    reps = max(3, int(min_seconds * 1e3 / max(e0.elapsed_time(e1), 1e-3)) + 1)
    sampler = ClockSampler(device_index)
    with sampler:
        torch.cuda.synchronize()
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps, sampler.summary()


def clock_fractions(value, clocks, peaks):
    """value against each peak, as measured and rescaled to the maximum SM clock (value * max MHz / median MHz)."""
    out = {"clocks": clocks}
    mhz, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    scaled = value * mx / mhz if mhz and mx else None
    out["at_max_clock"] = scaled
    for name, pk in peaks.items():
        out["frac_of_" + name] = value / pk
    return out


def replica_seed(rank):
    """Each rank is an independent replica of the decode step with its own weights and activations."""
    return 1000 * rank


def aggregate_replicas(ms_local, step_bytes, world, device):
    """Whole-job throughput of `world` replicas: every rank moves step_bytes per step and the step
    takes as long as the slowest rank (max over ranks). Returns (ms_max, GB/s)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms_local], device=device, dtype=torch.float64)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_max = float(t.item())
    return ms_max, world * step_bytes / (ms_max * 1e-3) / 1e9


def run_cuda(args):
    import torch
    import torch.distributed as dist
    from paper_2605_26092_b200 import build
    build.build()
    from paper_2605_26092_b200 import goq

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    hbm_peak, tf_peak, peak_src = measured_peaks()

    if args.gemv_variant:
        goq.set_gemv_variant(args.gemv_variant)
    layers = args.layers
    stack = build_stack(goq, torch, layers, seed0=replica_seed(rank), batch=1)
    n_lin = len(stack)
    step_bytes = sum(algorithmic_bytes(s["n"], s["k"], 1) for s in stack)
    # one scratch buffer shared by all calls: launches on one stream run in order
    ws = torch.empty(build_stack.ws_bytes, dtype=torch.uint8, device="cuda")
    goq.workspace_init(ws)

    if args.launch == "sequence":
        # the whole step is one persistent kernel and a true chain: every linear reads the previous linear's output
        seq = goq.make_sequence(flow_items(goq, stack))
        ws_seq = torch.empty(goq.sequence_workspace_bytes(n_lin), dtype=torch.uint8, device="cuda")
        goq.workspace_init(ws_seq)
        kernels_per_step = (n_lin + 255) // 256
        try:   # a device that refuses the cooperative launch still gets a number, from the per-linear launches
            goq.gemv_sequence(seq, ws_seq)
            torch.cuda.synchronize()
        except goq.GoqError as e:
            print("goq_gemv_sequence unavailable (%s): timing per-linear launches instead" % e, file=sys.stderr)
            args.launch = "graph"
    if args.launch == "sequence":

        def step():
            goq.gemv_sequence(seq, ws_seq)
    else:
        kernels_per_step = n_lin

        def step():
            for s in stack:
                goq.gemv(s["d"], s["packed"], s["x"], 1, s["y"], goq.F32, ws=ws)

    graph = capture(torch, step)

    # ---- timed region: warm-up, then exactly K steps between barriers ---------------------------
    for _ in range(max(args.warmup, 3)):
        graph.replay()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    sampler = ClockSampler(local)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with sampler:
        torch.cuda.synchronize()
        e0.record()
        for _ in range(args.steps):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    ms = e0.elapsed_time(e1) / args.steps
    ms_max, value = aggregate_replicas(ms, step_bytes, world, "cuda")

    # ---- end to end: host buffers in, host buffers out, through the C ABI's host entry points ---------
    if args.launch == "sequence":
        # one pinned host block with the step's input activations, one with every linear's output; goq_gemv_sequence_host
        # copies the first in, runs the sequence kernel on views of the device blocks, copies the second out
        y_off, yo = [], 0
        for s in stack:
            y_off.append(yo); yo += (s["n"] * 2 + 255) // 256 * 256
        xo = (stack[0]["k"] * 2 + 255) // 256 * 256
        x_stage = torch.zeros(xo, dtype=torch.uint8, device="cuda")
        y_stage = torch.zeros(yo, dtype=torch.uint8, device="cuda")
        x_host = torch.zeros(xo, dtype=torch.uint8).pin_memory()
        y_host = torch.zeros(yo, dtype=torch.uint8).pin_memory()
        x_host[:stack[0]["k"] * 2] = stack[0]["x"].view(torch.uint8).flatten().cpu()
        x0v = x_stage[:stack[0]["k"] * 2].view(torch.bfloat16).view(1, stack[0]["k"])
        outs = [y_stage[b:b + s["n"] * 2].view(torch.bfloat16).view(1, s["n"]) for s, b in zip(stack, y_off)]
        seq_e2e = goq.make_sequence(flow_items(goq, stack, x0v, outs))
        e2e_desc = "one CUDA graph holding one goq_gemv_sequence_host call (one pinned H2D block, the sequence kernel, one D2H block)"

        def step_e2e():
            goq.gemv_sequence_host(seq_e2e, x_host, x_stage, y_host, y_stage, ws_seq)
    else:
        host = []
        for s in stack:
            xh = s["x"].cpu().pin_memory()
            yh = torch.empty((1, s["n"]), dtype=torch.float32).pin_memory()
            host.append((xh, yh))
        e2e_desc = "one CUDA graph of goq_gemv_host calls (pinned H2D, kernel, D2H per linear)"

        def step_e2e():
            for s, (xh, yh) in zip(stack, host):
                goq.gemv_host(s["d"], s["packed"], xh, 1, yh, goq.F32, s["x"], s["y"], ws=ws)

    g2 = capture(torch, step_e2e)
    e2e_steps = max(3, args.steps // 4)
    ms_e2e = time_graph(torch, g2, e2e_steps, 3)
    _, e2e_val = aggregate_replicas(ms_e2e, step_bytes, world, "cuda")
    if args.launch == "sequence":
        h2d, d2h = x_stage.numel(), y_stage.numel()   # the blocks as copied (each linear's slice padded to 256 bytes)
    else:
        h2d = sum(s["k"] * 2 for s in stack)
        d2h = sum(s["n"] * 4 for s in stack)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- rank 0 only: extras (other batch sizes, per-shape times, GEMM, integer path) and CPU baseline
    extras = {}
    if not args.no_extras:
        extras = run_extras(torch, goq, stack, layers, tf_peak, ws)
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        items = oracle_sample()
        gbs, secs = time_oracle(items, repeats=3)
        cpu = {"value": gbs, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
               "sample": "one layer's 7 linears x 2048 output rows each, batch 1 (%.2f s per pass, best of 3)" % secs}

    launch_bytes = step_bytes / kernels_per_step
    launch_ms = ms / kernels_per_step
    achieved = launch_bytes / (launch_ms * 1e-3) / 1e9
    if args.launch == "sequence":
        kernel_name = "gemv_chain_kernel<3,4,1>"
        launch_desc = ("one CUDA graph holding one goq_gemv_sequence call: %d linears in a true chain, each reads the previous "
                       "one's bf16 output (its first k channels)" % n_lin)
        ratio, ratio_src = NCU_TRAFFIC_RATIO_SEQ, "ncu dram bytes of a 14-linear chain launch (profiles/gemv_chain_llama7b_2layers_batch1.md) scaled by algorithmic bytes"
        if int(goq.workspace_status(ws_seq)) != 0:
            raise RuntimeError("sequence kernel reported a device-side timeout")
    else:
        kernel_name = {2: "linear_mma_kernel<3,1>", 1: "gemv_scalar_kernel"}.get(
            args.gemv_variant, "gemv_stream_kernel<3,1,4,true>")
        launch_desc = "one CUDA graph of %d goq_gemv nodes per step" % n_lin
        # one ncu capture of the 4096x4096 launch read 8.96 MB of DRAM for 8.39 MB of algorithmic bytes;
        # the packed image grows in proportion to n*k, so the ratio is applied to the average launch
        ratio, ratio_src = NCU_TRAFFIC_RATIO, "ncu dram bytes of the 4096x4096 launch (8.96 MB) scaled by algorithmic bytes"
    if args.traffic_bytes is not None:
        traffic, traffic_src = args.traffic_bytes, "--traffic-bytes"
    else:
        traffic, traffic_src = (launch_bytes * ratio, ratio_src) if ratio else (None, "not captured")
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_max, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": DTYPE,
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "layers": layers, "linears_per_step": n_lin, "batch": 1,
                   "bytes_per_step": step_bytes, "l2": "weights per step %.2f GB >> 126 MB L2, no flush needed" % (step_bytes / 1e9),
                   "launch": launch_desc,
                   "parallelism": "replicas" if world > 1 else "single"},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": hbm_peak, "unit": "GB/s", "frac": achieved / hbm_peak,
                     "traffic": traffic, "traffic_source": traffic_src, "peak_source": peak_src, "frac_of_8000_nominal": achieved / 8000.0,
                     "kernel": kernel_name, "bytes_per_launch_avg": launch_bytes, "us_per_launch_avg": launch_ms * 1e3},
        "cpu_baseline": cpu,
        "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "launch": e2e_desc},
        "gpu_launches": args.steps * kernels_per_step,
        "clocks": sampler.summary(),
        "extras": extras,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_extras(torch, goq, stack, layers, tf_peak, ws):
    out = {}
    n_lin = len(stack)
    # decode at batch 4 and 16 over the same stack
    for batch in (4, 16):
        xs = [torch.randn((batch, s["k"]), device="cuda").to(torch.bfloat16) for s in stack]
        ys = [torch.empty((batch, s["n"]), dtype=torch.float32, device="cuda") for s in stack]

        def step():
            for s, x, y in zip(stack, xs, ys):
                goq.gemv(s["d"], s["packed"], x, batch, y, goq.F32, ws=ws)

        g = capture(torch, step)
        ms = time_graph(torch, g, 20, 3)
        nbytes = sum(algorithmic_bytes(s["n"], s["k"], batch) for s in stack)
        out["gemv_batch%d_gbs" % batch] = nbytes / (ms * 1e-3) / 1e9
        del g
        if batch <= 4:   # the same step as one dependent sequence (the integer-operand form takes up to 4 tokens)
            try:
                seq_b = goq.make_sequence([(s["d"], s["packed"], x, batch, y, goq.F32, j > 0)
                                           for j, (s, x, y) in enumerate(zip(stack, xs, ys))])
                ws_b = torch.empty(goq.sequence_workspace_bytes(len(stack)), dtype=torch.uint8, device="cuda")
                goq.workspace_init(ws_b)
                g = capture(torch, lambda: goq.gemv_sequence(seq_b, ws_b))
                ms = time_graph(torch, g, 20, 3)
                out["gemv_sequence_batch%d_gbs" % batch] = nbytes / (ms * 1e-3) / 1e9
                del g
            except goq.GoqError as e:
                out["gemv_sequence_batch%d_gbs" % batch] = "unavailable: %s" % e
        del xs, ys
    # the same decode step issued the other way (per-linear launches in a CUDA graph)
    def step_graph():
        for s in stack:
            goq.gemv(s["d"], s["packed"], s["x"], 1, s["y"], goq.F32, ws=ws)

    g = capture(torch, step_graph)
    ms = time_graph(torch, g, 20, 3)
    out["gemv_graph_of_launches_gbs"] = sum(algorithmic_bytes(s["n"], s["k"], 1) for s in stack) / (ms * 1e-3) / 1e9
    del g
    # ... as a sequence of flagged items over independent buffers: every linear waits until all SMs have finished the previous
    # one (the completion-counter barrier; the timed path orders by data flow instead)
    seq = goq.make_sequence([(s["d"], s["packed"], s["x"], 1, s["y"], goq.F32, j > 0) for j, s in enumerate(stack)])
    ws_seq = torch.empty(goq.sequence_workspace_bytes(len(stack)), dtype=torch.uint8, device="cuda")
    goq.workspace_init(ws_seq)
    g = capture(torch, lambda: goq.gemv_sequence(seq, ws_seq))
    ms = time_graph(torch, g, 20, 3)
    out["gemv_sequence_barrier_chain_gbs"] = sum(algorithmic_bytes(s["n"], s["k"], 1) for s in stack) / (ms * 1e-3) / 1e9
    del g
    # ... and with the data flow of a transformer layer: q, k and v read the previous layer's down output, o reads v's,
    # gate and up read o's, down reads up's (bf16 outputs, dependencies found from the address ranges)
    src = {"q_proj": ("down_proj", -1), "k_proj": ("down_proj", -1), "v_proj": ("down_proj", -1), "o_proj": ("v_proj", 0),
           "gate_proj": ("o_proj", 0), "up_proj": ("o_proj", 0), "down_proj": ("up_proj", 0)}
    names = [nm for nm, _, _ in si.LLAMA2_7B_LINEARS]
    items = []
    for j, s in enumerate(stack):
        layer, nm = divmod(j, 7)[0], names[j % 7]
        pn, dl = src[nm]
        pj = (layer + dl) * 7 + names.index(pn)
        x = s["x"] if pj < 0 else stack[pj]["yb"][:, :s["k"]]
        items.append((s["d"], s["packed"], x, 1, s["yb"], goq.BF16, False))
    seq = goq.make_sequence(items)
    goq.workspace_init(ws_seq)
    g = capture(torch, lambda: goq.gemv_sequence(seq, ws_seq))
    ms = time_graph(torch, g, 20, 3)
    out["gemv_sequence_layer_groups_gbs"] = sum(algorithmic_bytes(s["n"], s["k"], 1) for s in stack) / (ms * 1e-3) / 1e9
    del g, items
    # ... and with the usual serving fusions: q, k, v share their input and become one 12288 x 4096 linear, gate and up
    # one 22016 x 4096 (row-wise quantization groups make the concatenation exact): 4 dependent linears per layer, same bytes
    fused_shapes = [(3 * 4096, 4096), (4096, 4096), (2 * 11008, 4096), (4096, 11008)]
    gen = torch.Generator(device="cuda")
    fused = []
    for layer in range(layers):
        for idx, (n, k) in enumerate(fused_shapes):
            gen.manual_seed(9000 + layer * 4 + idx)
            d = goq.desc(n, k, GROUP, WBITS)
            codes = torch.randint(0, 1 << WBITS, (n, k), dtype=torch.uint8, device="cuda", generator=gen)
            meta = torch.randint(0, 64, (n, k // 8), dtype=torch.uint8, device="cuda", generator=gen)
            coef = (torch.randn((n, k // GROUP, 2), device="cuda", generator=gen) * (0.66 * k) ** -0.5).to(torch.float16)
            packed = torch.empty(goq.packed_bytes(d), dtype=torch.uint8, device="cuda")
            goq.pack(d, codes, meta, coef, packed)
            x = torch.randn((1, k), device="cuda", generator=gen).to(torch.bfloat16)
            y = torch.zeros((1, n), dtype=torch.bfloat16, device="cuda")
            fused.append({"d": d, "packed": packed, "x": x, "y": y, "n": n, "k": k})
            del codes, meta, coef
    # data flow: o reads the v third of q|k|v, gate|up reads o, down reads the up half of gate|up, the next q|k|v reads down
    items = []
    for j, s in enumerate(fused):
        if j == 0:
            x = s["x"]
        else:
            prev = fused[j - 1]
            x = prev["y"][:, prev["n"] - s["k"]:]
        items.append((s["d"], s["packed"], x, 1, s["y"], goq.BF16, False))
    seq_f = goq.make_sequence(items)
    ws_f = torch.empty(goq.sequence_workspace_bytes(len(fused)), dtype=torch.uint8, device="cuda")
    goq.workspace_init(ws_f)
    g = capture(torch, lambda: goq.gemv_sequence(seq_f, ws_f))
    ms = time_graph(torch, g, 20, 3)
    out["gemv_sequence_fused_qkv_gateup_gbs"] = sum(algorithmic_bytes(s["n"], s["k"], 1) for s in fused) / (ms * 1e-3) / 1e9
    del g, fused, seq_f, items
    # per-shape batch-1 time (rotating over the layers' copies of that shape, so each launch reads cold weights)
    shapes = {}
    for idx, (name, n, k) in enumerate(si.LLAMA2_7B_LINEARS):
        if (n, k) in shapes:
            continue
        sel = [s for s in stack if (s["n"], s["k"]) == (n, k)]

        def step():
            for s in sel:
                goq.gemv(s["d"], s["packed"], s["x"], 1, s["y"], goq.F32, ws=ws)

        g = capture(torch, step)
        ms = time_graph(torch, g, 20, 3)
        us = ms * 1e3 / len(sel)
        shapes[(n, k)] = {"us": us, "gbs": algorithmic_bytes(n, k, 1) / (us * 1e-6) / 1e9}
        del g
    out["gemv_batch1_per_shape"] = {"%dx%d" % k: v for k, v in shapes.items()}
    # prefill GEMM, M = 2048, over every linear of the stack (32 layers x 7: the packed weights are resident), repeated
    # for at least half a second with the clock sampler around exactly that region. Inputs per shape are shared (a linear
    # stack with independent inputs), outputs per shape are reused.
    m = 2048
    dev_index = torch.cuda.current_device()
    xs_k = {k: torch.randn((m, k), device="cuda").to(torch.bfloat16) for k in sorted({s["k"] for s in stack})}
    ys_n = {n: torch.empty((m, n), dtype=torch.float32, device="cuda") for n in sorted({s["n"] for s in stack})}
    ws_gemm = torch.empty(max(goq.workspace_bytes(s["d"], goq.OP_GEMM, m) for s in stack[:7]), dtype=torch.uint8, device="cuda")
    goq.workspace_init(ws_gemm)

    def step_gemm_stack():
        for s in stack:
            goq.gemm(s["d"], s["packed"], xs_k[s["k"]], m, goq.BF16, y=ys_n[s["n"]], y_dtype=goq.F32, ws=ws_gemm)

    ms, clk = time_loop_with_clocks(torch, step_gemm_stack, dev_index)
    flops = sum(2.0 * m * s["n"] * s["k"] for s in stack)
    tf = flops / (ms * 1e-3) / 1e12
    out["gemm_m2048_stack_tflops"] = tf
    out["gemm_m2048_stack_ms"] = ms
    out["gemm_m2048_stack"] = clock_fractions(tf, clk, {"bf16_burst_peak": tf_peak, "bf16_sustained_peak": measured_peaks.sustained})
    out["gemm_m2048_frac_of_bf16_peak"] = tf / tf_peak
    yb_n = {n: torch.empty((m, n), dtype=torch.bfloat16, device="cuda") for n in ys_n}

    def step_gemm_bf16_out():
        for s in stack[:7]:
            goq.gemm(s["d"], s["packed"], xs_k[s["k"]], m, goq.BF16, y=yb_n[s["n"]], y_dtype=goq.BF16, ws=ws_gemm)

    ms_l, _ = time_loop_with_clocks(torch, step_gemm_bf16_out, dev_index, min_seconds=0.1)
    out["gemm_m2048_layer_tflops_bf16_out"] = sum(2.0 * m * s["n"] * s["k"] for s in stack[:7]) / (ms_l * 1e-3) / 1e12
    del xs_k, ys_n, yb_n, ws_gemm
    # batch-size crossover on one 70B-shaped linear (8192 x 8192, g128) at W3, W2 and W4: goq_gemv up to batch 16,
    # goq_gemm from there on; eight copies of the weights are rotated so every call reads cold weights
    n = k = 8192
    for wb in (3, 2, 4):
        d70 = goq.desc(n, k, GROUP, wb)
        gen = torch.Generator(device="cuda")
        copies = []
        for c in range(8):
            gen.manual_seed(7000 + c)
            codes = torch.randint(0, 1 << wb, (n, k), dtype=torch.uint8, device="cuda", generator=gen)
            meta = torch.randint(0, 64, (n, k // 8), dtype=torch.uint8, device="cuda", generator=gen)
            coef = (torch.randn((n, k // GROUP, 2), device="cuda", generator=gen) * 0.03).to(torch.float16)
            pk = torch.empty(goq.packed_bytes(d70), dtype=torch.uint8, device="cuda")
            goq.pack(d70, codes, meta, coef, pk)
            copies.append(pk)
            del codes, meta, coef
        cross = {}
        for batch in (1, 4, 16, 32, 33, 64, 256):
            x = torch.randn((batch, k), device="cuda").to(torch.bfloat16)
            y = torch.empty((batch, n), dtype=torch.float32, device="cuda")
            paths = (["gemv"] if batch <= 16 else []) + (["gemm"] if batch >= 16 else [])
            for path in paths:
                wsx = goq.new_workspace(d70, goq.OP_GEMV if path == "gemv" else goq.OP_GEMM, batch)

                def step_x():
                    for pk in copies:
                        if path == "gemv":
                            goq.gemv(d70, pk, x, batch, y, goq.F32, ws=wsx)
                        else:
                            goq.gemm(d70, pk, x, batch, goq.BF16, y=y, y_dtype=goq.F32, ws=wsx)

                g = capture(torch, step_x)
                us = time_graph(torch, g, 10, 3) * 1e3 / len(copies)
                cross["batch%d_%s_us" % (batch, path)] = us
                del g
        out["crossover_8192x8192_w%d" % wb] = cross
        del copies
    # integer path: ViT-B/16-shaped linears, 197 x 64 tokens, W3 group 64, int8 activations and coefficients
    mt = si.VIT_B16_TOKENS
    vit = []
    gen = torch.Generator(device="cuda")
    for idx, (name, n, k) in enumerate(si.VIT_B16_LINEARS):
        gen.manual_seed(5000 + idx)
        d = goq.desc(n, k, 64, WBITS)
        codes = torch.randint(0, 1 << WBITS, (n, k), dtype=torch.uint8, device="cuda", generator=gen)
        meta = torch.randint(0, 64, (n, k // 8), dtype=torch.uint8, device="cuda", generator=gen)
        coef = (torch.randn((n, k // 64, 2), device="cuda", generator=gen) * 0.03).to(torch.float16)
        packed = torch.empty(goq.packed_bytes(d), dtype=torch.uint8, device="cuda")
        goq.pack(d, codes, meta, coef, packed)
        vit.append({
            "d": d, "packed": packed, "n": n, "k": k,
            "x": torch.randint(-127, 128, (mt, k), dtype=torch.int8, device="cuda", generator=gen),
            "sx": torch.rand((mt,), device="cuda", generator=gen) * 0.01 + 0.001,
            "cq": torch.randint(-127, 128, (n, k // 64, 2), dtype=torch.int8, device="cuda", generator=gen),
            "sc": torch.rand((n, 2), device="cuda", generator=gen) * 1e-3 + 1e-4,
            "acc": torch.empty((2, mt, n), dtype=torch.int32, device="cuda"),
        })

    def step_a8():
        for v in vit:
            goq.gemm(v["d"], v["packed"], v["x"], mt, goq.I8, sx=v["sx"], cq=v["cq"], sc=v["sc"], acc=v["acc"])

    ms, clk = time_loop_with_clocks(torch, step_a8, dev_index)
    ops = sum(2.0 * 2.0 * mt * v["n"] * v["k"] for v in vit)  # two bases, multiply-add = 2 ops
    tops = ops / (ms * 1e-3) / 1e12
    out["w3a8_vit_b16_int_tops"] = tops
    out["w3a8_vit_b16_ms"] = ms
    # int8 peak taken as twice the measured bf16 figures (the nominal ratio of the dense rates)
    out["w3a8_vit_b16"] = clock_fractions(tops, clk, {"int8_burst_peak_2x_bf16": 2 * tf_peak, "int8_sustained_peak_2x_bf16": 2 * measured_peaks.sustained})
    # the same linears with the scaled bf16 output instead of the two int32 accumulator planes (2 against 8 bytes per output)
    ys_a8 = [torch.empty((mt, v["n"]), dtype=torch.bfloat16, device="cuda") for v in vit]

    def step_a8_y():
        for v, yv in zip(vit, ys_a8):
            goq.gemm(v["d"], v["packed"], v["x"], mt, goq.I8, sx=v["sx"], cq=v["cq"], sc=v["sc"], y=yv, y_dtype=goq.BF16)

    ms_y, _ = time_loop_with_clocks(torch, step_a8_y, dev_index, min_seconds=0.1)
    out["w3a8_vit_b16_int_tops_bf16_out"] = ops / (ms_y * 1e-3) / 1e12
    del ys_a8
    del vit
    # steady state of the decode GEMV: one 70B-shaped 28672 x 8192 linear (117 MB of weights), eight copies rotated so
    # that every call streams from HBM; as single goq_gemv calls and as one chain of eight independent linears
    big = []
    for c in range(8):
        gen.manual_seed(8000 + c)
        n, k = 28672, 8192
        d = goq.desc(n, k, GROUP, WBITS)
        codes = torch.randint(0, 1 << WBITS, (n, k), dtype=torch.uint8, device="cuda", generator=gen)
        meta = torch.randint(0, 64, (n, k // 8), dtype=torch.uint8, device="cuda", generator=gen)
        coef = (torch.randn((n, k // GROUP, 2), device="cuda", generator=gen) * 0.03).to(torch.float16)
        pk = torch.empty(goq.packed_bytes(d), dtype=torch.uint8, device="cuda")
        goq.pack(d, codes, meta, coef, pk)
        big.append({"d": d, "packed": pk, "n": n, "k": k, "x": torch.randn((1, k), device="cuda", generator=gen).to(torch.bfloat16),
                    "y": torch.empty((1, n), dtype=torch.float32, device="cuda")})
        del codes, meta, coef
    nbytes = sum(algorithmic_bytes(s["n"], s["k"], 1) for s in big)
    ws_big = goq.new_workspace(big[0]["d"], goq.OP_GEMV, 1)
    g = capture(torch, lambda: [goq.gemv(s["d"], s["packed"], s["x"], 1, s["y"], goq.F32, ws=ws_big) for s in big])
    out["gemv_batch1_steady_gbs"] = nbytes / (time_graph(torch, g, 10, 3) * 1e-3) / 1e9
    del g
    seq_big = goq.make_sequence([(s["d"], s["packed"], s["x"], 1, s["y"], goq.F32, False) for s in big])
    ws_sb = torch.empty(goq.sequence_workspace_bytes(len(big)), dtype=torch.uint8, device="cuda")
    goq.workspace_init(ws_sb)
    g = capture(torch, lambda: goq.gemv_sequence(seq_big, ws_sb))
    out["gemv_batch1_steady_chain_gbs"] = nbytes / (time_graph(torch, g, 10, 3) * 1e-3) / 1e9
    del g, big, seq_big
    # the same decode step with bf16 operands (exponent shift of the bf16 activation in the tensor core: the streaming kernel)
    prev = goq.set_gemv_variant(3)
    try:
        g = capture(torch, step_graph)
        out["gemv_bf16_operand_form_gbs"] = sum(algorithmic_bytes(s["n"], s["k"], 1) for s in stack) / (time_graph(torch, g, 10, 3) * 1e-3) / 1e9
        del g
    finally:
        goq.set_gemv_variant(prev)
    # GEO quantizer on the device: the 7B stack's shapes, fp32 weights in, codes + records + fp16 pairs out
    # (algorithmic bytes per weight: 4 read, 1 + 1/8 + 4/group written)
    qt = {}
    total_s = 0.0
    for (n, k), count in (((4096, 4096), 4), ((11008, 4096), 2), ((4096, 11008), 1)):
        d = goq.desc(n, k, GROUP, WBITS)
        w = torch.randn((n, k), device="cuda") * 0.02
        codes = torch.empty((n, k), dtype=torch.uint8, device="cuda")
        meta = torch.empty((n, k // 8), dtype=torch.uint8, device="cuda")
        coef = torch.empty((n, k // GROUP, 2), dtype=torch.float16, device="cuda")
        ms_q, _ = time_loop_with_clocks(torch, lambda: goq.quantize_geo(d, w, codes, meta, coef), dev_index, min_seconds=0.05)
        qbytes = n * k * (4 + 1 + 0.125) + n * (k // GROUP) * 4
        qt["%dx%d" % (n, k)] = {"us": ms_q * 1e3, "gbs": qbytes / (ms_q * 1e-3) / 1e9}
        total_s += ms_q * 1e-3 * count * layers
        del w, codes, meta, coef
    out["quantize_geo_per_shape"] = qt
    out["quantize_geo_7b_stack_seconds"] = total_s   # context: the paper reports 0.47 min for LLaMA-2-7B on its own hardware
    return out


NCU_TRAFFIC_RATIO = 8.96 / 8.39
NCU_TRAFFIC_RATIO_SEQ = (215.8 + 4.4) / 202.9   # ncu: 215.2 MB read + 4.2 MB written for the 202.9 MB (algorithmic) of a 14-linear launch


def run_probe_steady(args):
    """`--probe steady`: only the steady-state case of the decode GEMV - a chain of `--copies` independent 28672 x 8192
    linears (117 MB each) - a few times. Small enough for a profiler capture of one launch; prints one JSON line."""
    import torch
    from paper_2605_26092_b200 import build
    build.build()
    from paper_2605_26092_b200 import goq
    gen = torch.Generator(device="cuda")
    n, k = 28672, 8192
    d = goq.desc(n, k, GROUP, WBITS)
    items, keep = [], []
    for c in range(args.copies):
        gen.manual_seed(8000 + c)
        codes = torch.randint(0, 1 << WBITS, (n, k), dtype=torch.uint8, device="cuda", generator=gen)
        meta = torch.randint(0, 64, (n, k // 8), dtype=torch.uint8, device="cuda", generator=gen)
        coef = (torch.randn((n, k // GROUP, 2), device="cuda", generator=gen) * 0.03).to(torch.float16)
        pk = torch.empty(goq.packed_bytes(d), dtype=torch.uint8, device="cuda")
        goq.pack(d, codes, meta, coef, pk)
        x = torch.randn((1, k), device="cuda", generator=gen).to(torch.bfloat16)
        y = torch.empty((1, n), dtype=torch.float32, device="cuda")
        keep += [pk, x, y]
        items.append((d, pk, x, 1, y, goq.F32, False))
        del codes, meta, coef
    seq = goq.make_sequence(items)
    ws = torch.empty(goq.sequence_workspace_bytes(len(items)), dtype=torch.uint8, device="cuda")
    goq.workspace_init(ws)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    best = float("inf")
    for _ in range(max(args.steps, 1) + max(args.warmup, 1)):
        e0.record(); goq.gemv_sequence(seq, ws); e1.record(); torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1))
    nbytes = args.copies * algorithmic_bytes(n, k, 1)
    print(json.dumps({"probe": "steady", "copies": args.copies, "algorithmic_bytes": nbytes, "best_ms": best,
                      "gbs": nbytes / (best * 1e-3) / 1e9, "status": int(goq.workspace_status(ws))}))


def run_probe_gemm(args):
    """`--probe gemm`: one 4096 x 4096 W3 g128 linear at M = 2048 tokens through goq_gemm (activation pre-pass + tcgen05
    GEMM), a few times. Small enough for a profiler capture of one launch; prints one JSON line."""
    import torch
    from paper_2605_26092_b200 import build
    build.build()
    from paper_2605_26092_b200 import goq
    gen = torch.Generator(device="cuda")
    gen.manual_seed(8100)
    n, k, m = 4096, 4096, 2048
    d = goq.desc(n, k, GROUP, WBITS)
    codes = torch.randint(0, 1 << WBITS, (n, k), dtype=torch.uint8, device="cuda", generator=gen)
    meta = torch.randint(0, 64, (n, k // 8), dtype=torch.uint8, device="cuda", generator=gen)
    coef = (torch.randn((n, k // GROUP, 2), device="cuda", generator=gen) * 0.02).to(torch.float16)
    pk = torch.empty(goq.packed_bytes(d), dtype=torch.uint8, device="cuda")
    goq.pack(d, codes, meta, coef, pk)
    x = torch.randn((m, k), device="cuda", generator=gen).to(torch.bfloat16)
    y = torch.empty((m, n), dtype=torch.float32, device="cuda")
    ws = goq.new_workspace(d, goq.OP_GEMM, m)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    best = float("inf")
    for _ in range(max(args.steps, 1) + max(args.warmup, 1)):
        e0.record(); goq.gemm(d, pk, x, m, goq.BF16, y=y, y_dtype=goq.F32, ws=ws); e1.record(); torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1))
    print(json.dumps({"probe": "gemm", "shape": [n, k], "tokens": m, "best_ms": best,
                      "tflops": 2.0 * m * n * k / (best * 1e-3) / 1e12, "status": int(goq.workspace_status(ws))}))


def launch_command(n_gpus, argv, port=None):
    """The command that starts one rank per GPU on this node for `bench.py --gpus N` (N > 1) when no launcher has."""
    port = port or (29500 + os.getpid() % 2000)
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n_gpus),
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--layers", type=int, default=si.LLAMA2_7B_LAYERS)
    ap.add_argument("--no-extras", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--launch", choices=("sequence", "graph"), default="sequence",
                    help="how a step is issued: one goq_gemv_sequence call, or a CUDA graph of per-linear goq_gemv launches")
    ap.add_argument("--gemv-variant", type=int, default=0,
                    help="force a kernel variant (goq_set_gemv_variant): 0 automatic, 3 streaming, 4 tcgen05 tensor-memory GEMV, ...")
    ap.add_argument("--traffic-bytes", type=float, default=None,
                    help="dram bytes per launch of the dominant kernel from an ncu capture (reported as-is)")
    ap.add_argument("--probe", choices=("steady", "gemm"), default=None, help="run one small case only (for profiler captures)")
    ap.add_argument("--copies", type=int, default=2, help="--probe steady: number of 28672 x 8192 linears in the chain")
    args = ap.parse_args()
    if args.probe == "steady":
        if args.steps == 200:
            args.steps = 3
        return run_probe_steady(args)
    if args.probe == "gemm":
        if args.steps == 200:
            args.steps = 3
        return run_probe_gemm(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # asked for N GPUs without a launcher: start the N ranks (replicas, one per GPU) ourselves
        os.execv(sys.executable, launch_command(args.gpus, sys.argv[1:]))
    if args.impl == "reference":
        if args.steps == 200:
            args.steps = 5
        if args.warmup == 5:
            args.warmup = 1
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
