#!/usr/bin/env python
"""Benchmark of the RaZeR matmul path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--no-extras]

One "step" is one pass of the decode hot path over one batch: the three Llama-7B-shaped
GEMVs (M = 1; N x K = 4096x4096, 11008x4096, 4096x11008) against packed RaZeR weights.
The headline value is the effective HBM bandwidth of that step: algorithmic bytes
(N*K*0.5625 weight bytes + 2K activation + 2N output bytes per GEMV) over device time.
Weights rotate over several distinct packed copies (> 500 MB in total, four times the L2)
so every step streams from HBM.  Further lines of the same JSON object give the skinny
(M = 4..64), prefill (M = 2048) and weight-activation results, the roofline fraction and
the CPU oracle timed on the host cores.

With --gpus N > 1 (launched by torchrun, one rank per GPU) every rank runs an independent
replica of the same workload: the path has no exchange step, so there is no collective in
the data path; the value is the sum over ranks over the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

DECODE_SHAPES = [(4096, 4096), (11008, 4096), (4096, 11008)]
SKINNY_SHAPES = [(8192, 8192), (28672, 8192), (8192, 28672)]
PREFILL_SHAPES = [(14336, 4096), (4096, 14336)]
# DRAM bytes of one step (its three launches) read from the ncu capture of the kernel as committed:
# 9,506,304 + 25,430,272 + 25,445,120 read, 0 written.  Set to None whenever the kernel changes until re-captured.
NCU_DRAM_BYTES_PER_STEP = 60381696
METRIC = "razer_gemv_effective_hbm_bandwidth"


def algo_bytes(M, N, K):
    return N * K * 0.5625 + 2 * M * K + 2 * M * N


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=float(d["hbm_gbs"]), bf16=float(d["bf16_tflops"]),
                    bf16_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "20"], stdout=f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if not self.proc:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        try:
            for ln in open(self.path):
                c = [v.strip() for v in ln.split(",")]
                if len(c) < 9:
                    continue
                try:
                    sm.append(float(c[1])); smax.append(float(c[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            sm.sort()
            out.update(sm_mhz=sm[len(sm) // 2], sm_max_mhz=max(smax), reasons=sorted(reasons), samples=len(sm))
        return out


def host_threads():
    """Threads the numpy oracle can use: the BLAS pool behind numpy's matmul, bounded by the cores this process may
    run on (the element-wise decode steps of the oracle run on one thread)."""
    cores = len(os.sched_getaffinity(0))
    try:
        from threadpoolctl import threadpool_info
        blas = [int(i["num_threads"]) for i in threadpool_info() if i.get("user_api") == "blas"]
        if blas:
            return min(cores, max(blas))
    except Exception:
        pass
    return cores


def time_cuda(fn, iters, torch):
    """Device time of `iters` calls of fn(i), CUDA events on the current stream, ms per call."""
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    start.record()
    for i in range(iters):
        fn(i)
    end.record()
    torch.cuda.synchronize()
    return start.elapsed_time(end) / iters


def make_sets(b, torch, inputs, N, K, n_sets, seed):
    """n_sets distinct packed copies of an N x K random RaZeR tensor (rows rolled per copy)."""
    codes, scales = inputs.random_codes(N, K, seed)
    codes, scales = codes.cuda(), scales.cuda()
    desc = b.make_desc(N, K, 0.002)
    sets = []
    for s in range(n_sets):
        c = torch.roll(codes, shifts=37 * s, dims=0).contiguous() if s else codes
        sc = torch.roll(scales, shifts=37 * s, dims=0).contiguous() if s else scales
        sets.append(b.razer_pack_layout(desc, c, sc))
    torch.cuda.synchronize()
    return desc, sets, (codes, scales)


def max_over_ranks(ms, dist, device):
    """Slowest rank's time: the replicas are independent, so the job is as slow as its slowest GPU."""
    if dist is None:
        return float(ms)
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbps(world, step_bytes, ms):
    """Aggregate over all replicas: every rank moves step_bytes per step in (at most) ms."""
    return world * step_bytes / (ms * 1e-3) / 1e9


def run_reference(args):
    """The CPU oracle as it stands, timed on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    import torch
    from oracle import razer_oracle as ro
    from paper_2501_04052_b200 import inputs
    N, K = DECODE_SHAPES[0]
    codes, scales = inputs.random_codes(N, K, 1000)
    codes, scales = codes.numpy(), scales.numpy()
    x = inputs.bf16_to_bits(inputs.activations(1, K, 1000))
    times = []
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        ro.matmul_w4a16(x, codes, scales, np.float32(0.002))
        if i >= args.warmup:
            times.append(time.perf_counter() - t0)
    ms = 1e3 * sum(times) / len(times)
    gbs = algo_bytes(1, N, K) / (ms * 1e-3) / 1e9
    cores = host_threads()
    sample = f"each step = one {N}x{K} M=1 GEMV (first of the three decode shapes): oracle decode + FP64 matmul"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "decode GEMV, Llama-7B-shaped layers, M=1 (config 2)", "sample": sample},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_shape(args):
    """One matmul shape alone: `warmup` launches, then `steps` launches timed with CUDA events, two packed copies
    of the weights in turn.  M <= 64 goes through razer_gemv, larger M through razer_gemm."""
    import torch
    from paper_2501_04052_b200 import build
    build.build()
    from paper_2501_04052_b200 import binding as b
    from paper_2501_04052_b200 import inputs
    M, N, K = (int(v) for v in args.shape.lower().split("x"))
    desc, sets, _ = make_sets(b, torch, inputs, N, K, 2, 7)
    x = inputs.activations(M, K, 3).cuda()
    y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    if args.op == "auto":
        fn, op = (b.razer_gemv, b.OP_GEMV) if M <= 64 else (b.razer_gemm, b.OP_GEMM)
        name = "razer_gemv" if M <= 64 else "razer_gemm"
        ws = b.alloc_workspace(desc, M, op, "cuda")
        call = lambda i: fn(desc, sets[i % 2], x, y, ws)
    elif args.op == "w4a4-fp4-prepared":
        name = "razer_gemm_w4a4_fp4 (two-pass block-scaled FP4, prepared operand)"
        ws = b.alloc_workspace(desc, M, b.OP_GEMM_W4A4, "cuda")
        act4, ats4 = b.razer_quant_act_fp4(x)
        call = lambda i: b.razer_gemm_w4a4_fp4(desc, sets[i % 2], act4, ats4, M, y=y, workspace=ws)
    else:
        native = args.op == "w4a4-fp4"
        name = "razer_gemm_w4a4 (two-pass block-scaled FP4)" if native else "razer_gemm_w4a4"
        ws = b.alloc_workspace(desc, M, b.OP_GEMM_W4A4, "cuda")
        ac, as_, ats = b.razer_quant_act(x, sv_mag=0.0 if native else 5.0)
        call = lambda i: b.razer_gemm_w4a4(desc, sets[i % 2], ac, as_, ats, y=y, workspace=ws, use_native_fp4=native)
    for i in range(args.warmup):
        call(i)
    ms = time_cuda(call, args.steps, torch)
    b.razer_workspace_status(ws)
    print(json.dumps({"shape": [M, N, K], "op": name, "us_per_launch_stream": ms * 1e3,
                      "launches": args.warmup + args.steps, "algorithmic_bytes": algo_bytes(M, N, K),
                      "flops": 2.0 * M * N * K}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--no-extras", action="store_true", help="skip the skinny / prefill / W4A4 lines")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline")
    ap.add_argument("--windows", type=int, default=7, help="timed windows (the median is reported)")
    ap.add_argument("--window-ms", type=float, default=200.0, help="length of a timed window (0: one graph replay)")
    ap.add_argument("--shape", default="", help="MxNxK: time that one matmul alone (a small, single-kernel run for "
                                                "profiler captures); prints its own short JSON line, not the bench line")
    ap.add_argument("--op", default="auto", help="with --shape: auto (razer_gemv / razer_gemm by M), w4a4, w4a4-fp4 "
                                                 "(interchange-format activations) or w4a4-fp4-prepared")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.shape:
        return run_shape(args)

    import torch
    from paper_2501_04052_b200 import build
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank == 0:
        build.build()
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    from paper_2501_04052_b200 import binding as b
    from paper_2501_04052_b200 import inputs
    pk = peaks()

    # ---------------- decode step (config 2): resident inputs
    n_sets = 9
    layers = []
    for i, (N, K) in enumerate(DECODE_SHAPES):
        desc, sets, raw = make_sets(b, torch, inputs, N, K, n_sets, 1000 + i)
        x = inputs.activations(1, K, 1000 + i).cuda()
        y = torch.empty((1, N), dtype=torch.bfloat16, device="cuda")
        ws = b.alloc_workspace(desc, 1, b.OP_GEMV, "cuda")
        layers.append(dict(N=N, K=K, desc=desc, sets=sets, raw=raw if i == 0 else None, x=x, y=y, ws=ws))
    step_bytes = sum(algo_bytes(1, l["N"], l["K"]) for l in layers)
    packed_total = sum(s.numel() for l in layers for s in l["sets"])

    def step(i):
        for l in layers:
            b.razer_gemv(l["desc"], l["sets"][i % n_sets], l["x"], l["y"], l["ws"])

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    # The timed region replays a CUDA graph of the K steps (3 K kernel launches): the kernels run 10-25 us
    # each, shorter than a Python-driven launch, and the metric is the device path.  The same steps launched
    # one by one from the host are timed as well and reported as "stream_launch".
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    launches0 = b.razer_kernel_launches()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for i in range(args.steps):
                step(i)
    launches = b.razer_kernel_launches() - launches0      # kernels one replay executes
    torch.cuda.synchronize()
    graph.replay()
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    # One replay of the graph is short (K steps of ~20 us), so a timed window replays it until the window lasts
    # about 200 ms, and the reported time per step is the median over 7 such windows (spread reported too); the
    # clock sampler runs across all of them.
    probe = time_cuda(lambda i: graph.replay(), 3, torch)                     # ms per replay
    replays = max(1, int(args.window_ms / max(probe, 1e-3) + 0.5))
    sampler = ClockSampler(local_rank)
    sampler.start()
    windows = [time_cuda(lambda i: graph.replay(), replays, torch) / args.steps for _ in range(max(1, args.windows))]
    ms_stream = time_cuda(step, args.steps, torch)
    clocks = sampler.stop()
    windows.sort()
    ms = windows[len(windows) // 2]
    window_stats = {"windows": len(windows), "replays_per_window": replays, "window_ms": ms * args.steps * replays,
                    "ms_per_step_min": windows[0], "ms_per_step_max": windows[-1]}
    launches_timed = launches * replays * len(windows)
    ms = max_over_ranks(ms, dist, "cuda")
    value = whole_job_gbps(world, step_bytes, ms)

    # ---------------- end to end: host buffers, copies inside the timed region
    for l in layers:
        l["xh"] = l["x"].cpu().pin_memory()
        l["yh"] = torch.empty((1, l["N"]), dtype=torch.bfloat16).pin_memory()

    def step_host(i):
        for l in layers:
            b.razer_gemv_host(l["desc"], l["sets"][i % n_sets], l["xh"], l["yh"], l["x"], l["y"], l["ws"])

    for i in range(3):
        step_host(i)
    e2e_steps = max(20, args.steps // 4)
    ms_e2e = time_cuda(step_host, e2e_steps, torch)
    ms_e2e = max_over_ranks(ms_e2e, dist, "cuda")
    e2e = {"value": whole_job_gbps(world, step_bytes, ms_e2e), "unit": "GB/s",
           "h2d_bytes_per_step": sum(2 * l["K"] for l in layers), "d2h_bytes_per_step": sum(2 * l["N"] for l in layers),
           "ms_per_step": ms_e2e}

    def graph_time(fn, reps):
        """ms per call of fn(i), i = 0..reps-1, replayed from a CUDA graph."""
        g = torch.cuda.CUDAGraph()
        s2 = torch.cuda.Stream()
        s2.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s2):
            with torch.cuda.graph(g, stream=s2):
                for i in range(reps):
                    fn(i)
        torch.cuda.synchronize()
        g.replay()
        return time_cuda(lambda i: g.replay(), 3, torch) / reps

    per_shape = []
    for l in layers:
        t = graph_time(lambda i, l=l: b.razer_gemv(l["desc"], l["sets"][i % n_sets], l["x"], l["y"], l["ws"]), 4 * n_sets)
        gbs = algo_bytes(1, l["N"], l["K"]) / (t * 1e-3) / 1e9
        per_shape.append({"M": 1, "N": l["N"], "K": l["K"], "us": t * 1e3, "GBps": gbs, "frac_hbm": gbs / pk["hbm"]})

    result = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "decode GEMV, Llama-7B-shaped layers, M=1 (config 2): N x K = 4096x4096, 11008x4096, "
                               "4096x11008; random RaZeR codes, bf16 N(0,1) activations",
                   "l2": f"inputs larger than L2: weights rotate over {n_sets} packed copies, {packed_total / 1e6:.0f} MB",
                   "parallelism": "replicas" if world > 1 else "single GPU"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches_timed),
        "timing": "CUDA events around windows of repeated replays of a CUDA graph holding the K steps; median window",
        "timing_windows": window_stats, "gpu_launches_per_step": int(launches // max(args.steps, 1)),
        "stream_launch": {"value": world * step_bytes / (ms_stream * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": ms_stream},
        "roofline": {"bound": "hbm", "achieved": value / world, "peak": pk["hbm"], "unit": "GB/s",
                     "frac": value / world / pk["hbm"], "traffic": NCU_DRAM_BYTES_PER_STEP, "peak_source": pk["source"],
                     "traffic_source": "ncu dram__bytes_read.sum + dram__bytes_write.sum of the step's three launches "
                                       "(profiles/razer_stream_kernel_gemv_config2.md)",
                     "kernel": "razer_stream_kernel via razer_gemv (3 launches per step)", "algorithmic_bytes_per_step": step_bytes,
                     "frac_of_nominal_8TBps": value / world / 8000.0},
        "decode_per_shape": per_shape,
    }

    if rank == 0 and not args.no_extras:
        extras = []
        del layers[1:]
        torch.cuda.empty_cache()
        for (N, K) in SKINNY_SHAPES:
            ns = 6 if N * K < 100e6 else 3
            desc, sets, _ = make_sets(b, torch, inputs, N, K, ns, 2000)
            for M in (4, 16, 64):
                x = inputs.activations(M, K, 2000 + M).cuda()
                y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
                ws = b.alloc_workspace(desc, M, b.OP_GEMV, "cuda")
                f = lambda i: b.razer_gemv(desc, sets[i % ns], x, y, ws)
                for i in range(3):
                    f(i)
                t = graph_time(f, 4 * ns)
                gbs = algo_bytes(M, N, K) / (t * 1e-3) / 1e9
                extras.append({"config": 3, "op": "razer_gemv", "M": M, "N": N, "K": K, "us": t * 1e3, "GBps": gbs,
                               "frac_hbm": gbs / pk["hbm"], "TFLOPs": 2.0 * M * N * K / (t * 1e-3) / 1e12})
            del sets
            torch.cuda.empty_cache()
        for (N, K) in PREFILL_SHAPES:
            M = 2048
            desc, sets, _ = make_sets(b, torch, inputs, N, K, 2, 3000)
            x = inputs.activations(M, K, 3000, outlier_channel_frac=0.01).cuda()
            y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
            ws = b.alloc_workspace(desc, M, b.OP_GEMM, "cuda")
            f = lambda i: b.razer_gemm(desc, sets[i % 2], x, y, ws)
            for i in range(3):
                f(i)
            t = graph_time(f, 8)
            tf = 2.0 * M * N * K / (t * 1e-3) / 1e12
            extras.append({"config": 4, "op": "razer_gemm", "M": M, "N": N, "K": K, "us": t * 1e3, "TFLOPs": tf,
                           "frac_bf16": tf / pk["bf16"]})
            del sets
            torch.cuda.empty_cache()
        M, N, K = 256, 8192, 8192
        desc, sets, _ = make_sets(b, torch, inputs, N, K, 4, 4000)
        x = inputs.activations(M, K, 4000, outlier_channel_frac=0.01).cuda()
        y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        ws = b.alloc_workspace(desc, M, b.OP_GEMM_W4A4, "cuda")
        ac, as_, ats = b.razer_quant_act(x)
        tq = graph_time(lambda i: b.razer_quant_act(x), 8)
        f = lambda i: b.razer_gemm_w4a4(desc, sets[i % 4], ac, as_, ats, y=y, workspace=ws)
        for i in range(3):
            f(i)
        t = graph_time(f, 8)
        extras.append({"config": 5, "op": "razer_quant_act", "M": M, "K": K, "us": tq * 1e3,
                       "GBps": (M * K * 2 + M * K * 0.5625) / (tq * 1e-3) / 1e9})
        tf = 2.0 * M * N * K / (t * 1e-3) / 1e12
        extras.append({"config": 5, "op": "razer_gemm_w4a4", "M": M, "N": N, "K": K, "us": t * 1e3, "TFLOPs": tf,
                       "frac_bf16": tf / pk["bf16"]})
        # the two-pass block-scaled FP4 realization (RaZeR weights x plain-NVFP4 activations); operations counted
        # as 2MNK although two passes execute; the FP4 peak is the measured bf16 peak x the nominal ratio of 4
        ac0, as0, ats0 = b.razer_quant_act(x, sv_mag=0.0)
        ws4 = b.alloc_workspace(desc, M, b.OP_GEMM_W4A4, "cuda")       # a workspace serves one of the two paths
        f4 = lambda i: b.razer_gemm_w4a4(desc, sets[i % 4], ac0, as0, ats0, y=y, workspace=ws4, use_native_fp4=True)
        for i in range(3):
            f4(i)
        t4 = graph_time(f4, 8)
        tf4 = 2.0 * M * N * K / (t4 * 1e-3) / 1e12
        extras.append({"config": 5, "op": "razer_gemm_w4a4 (two-pass block-scaled FP4)", "M": M, "N": N, "K": K,
                       "us": t4 * 1e3, "TFLOPs_effective": tf4, "frac_fp4_two_pass": 2.0 * tf4 / (4.0 * pk["bf16"]),
                       "GBps": algo_bytes(M, N, K) / (t4 * 1e-3) / 1e9, "frac_hbm": algo_bytes(M, N, K) / (t4 * 1e-3) / 1e9 / pk["hbm"]})
        # the same with the quantizer writing the tensor core's operand layout itself (no re-layout kernel)
        act4, ats4 = b.razer_quant_act_fp4(x)
        tq4 = graph_time(lambda i: b.razer_quant_act_fp4(x, act_fp4=act4), 8)
        f5 = lambda i: b.razer_gemm_w4a4_fp4(desc, sets[i % 4], act4, ats4, M, y=y, workspace=ws4)
        for i in range(3):
            f5(i)
        t5 = graph_time(f5, 8)
        tf5 = 2.0 * M * N * K / (t5 * 1e-3) / 1e12
        extras.append({"config": 5, "op": "razer_quant_act_fp4", "M": M, "K": K, "us": tq4 * 1e3,
                       "GBps": (M * K * 2 + M * K * 0.5625) / (tq4 * 1e-3) / 1e9})
        extras.append({"config": 5, "op": "razer_gemm_w4a4_fp4 (two-pass block-scaled FP4, prepared operand)", "M": M, "N": N,
                       "K": K, "us": t5 * 1e3, "TFLOPs_effective": tf5, "frac_fp4_two_pass": 2.0 * tf5 / (4.0 * pk["bf16"]),
                       "frac_bf16_effective": tf5 / pk["bf16"], "GBps": algo_bytes(M, N, K) / (t5 * 1e-3) / 1e9,
                       "frac_hbm": algo_bytes(M, N, K) / (t5 * 1e-3) / 1e9 / pk["hbm"]})
        # GPU weight quantizer (offline step; FP32 in, interchange format out), 4096 x 4096
        wq = inputs.student_t_weights(4096, 4096, 5000, outlier_frac=0.001).cuda()
        b.razer_quant_weight(wq)
        tw = graph_time(lambda i: b.razer_quant_weight(wq), 8)
        extras.append({"config": "offline", "op": "razer_quant_weight", "N": 4096, "K": 4096, "us": tw * 1e3,
                       "GBps": 4096 * 4096 * (4 + 0.5625) / (tw * 1e-3) / 1e9,
                       "note": "bytes = one FP32 read + the 4.5-bit output; the kernel reads the input twice (maximum, then quantize)"})
        result["extras"] = extras

    if rank == 0 and not args.no_cpu:
        import numpy as np
        from oracle import razer_oracle as ro
        l = layers[0]
        codes, scales = l["raw"][0].cpu().numpy(), l["raw"][1].cpu().numpy()
        xb = inputs.bf16_to_bits(l["x"].cpu())
        t0 = time.perf_counter()
        reps = 0
        while reps < 2 or (time.perf_counter() - t0 < 10.0 and reps < 20):
            yref = ro.matmul_w4a16(xb, codes, scales, np.float32(0.002))
            reps += 1
        dt = (time.perf_counter() - t0) / reps
        b.razer_gemv(l["desc"], l["sets"][0], l["x"], l["y"], l["ws"])
        torch.cuda.synchronize()
        err = ro.rel_frobenius(inputs.bf16_to_bits(l["y"].cpu()), yref)
        result["cpu_baseline"] = {"value": algo_bytes(1, l["N"], l["K"]) / dt / 1e9, "unit": "GB/s",
                                  "cores": host_threads(), "kind": "oracle",
                                  "sample": f"{reps} x the {l['N']}x{l['K']} M=1 GEMV of the step "
                                            "(oracle decode + FP64 matmul); the other two shapes scale with N*K",
                                  "parity_rel_frobenius_vs_gpu": err}
    if rank == 0:
        print(json.dumps(result))
    if dist:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
