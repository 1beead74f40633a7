#!/usr/bin/env python
"""Benchmark of the STWQ quantized linear hot path on B200.

A step is one pass of the whole hot path (activation quantize -> int8 GEMM -> dequantize
epilogue, i.e. one `qlinear` call) over each of the four block linears of the VAR-d16-shaped
workload (batch 16 x 680 tokens, hidden 1024: qkv, proj, fc1+GELU, fc2; W8A8, bf16 output),
on seeded synthetic inputs already resident in HBM. The metric is int8 TOPS of the whole step
(2*M*N*K per layer over the step time, quantize kernels included).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--config 2]

Prints one JSON line (rank 0). With N > 1 (torchrun) every rank runs the same per-GPU batch on
its own rows (weak scaling, no collective on the data path); time is the max over ranks.
`--impl reference` times the CPU oracle on the host cores instead (a deliberately plain program).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

PCT = 999900
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
INT8_OVER_BF16 = 2.0          # nominal dense tensor ratio (4.5 vs 2.25 PFLOP/s)
# DRAM bytes (read + write) per launch of the dominant kernel, mean over the four layer shapes, from
# the ncu capture summarised in profiles/qgemm2_kernel_config2.md (24.7, 12.3, 46.4, 51.5 MB).
NCU_TRAFFIC_BYTES_PER_LAUNCH = 33.7e6


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


def stand_in_channel_scales(layer: wl.Layer) -> np.ndarray:
    """Seeded stand-in for the GPS vector in the CPU reference arm, where only the time matters
    (Algorithm 1 in the oracle over a full calibration set would take longer than the arm's
    budget): larger on the outlier channels, log-normal jitter elsewhere."""
    z = wl.normals(layer.seed, 8, 0, layer.K)
    return (np.sqrt(wl.outlier_factors(layer)) * np.exp(0.25 * z)).astype(np.float32)


def rank_step(rank: int, step: int = 0, world: int = 1) -> int:
    """Which seeded batch a rank draws: the job's global batch is `world` per-GPU batches, rank r
    takes the r-th one (weak scaling: rows are independent, parameters are replicated, so no
    collective touches the data path)."""
    return step * world + rank


def max_over_ranks(ms: float, world: int, device) -> float:
    """Slowest rank's time (all-reduce MAX of one scalar; the only collective of the benchmark)."""
    if world == 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tops(world: int, ops_per_rank_step: float, ms_step: float) -> float:
    """Aggregate int8 TOPS of the job: every rank performs ops_per_rank_step in the slowest rank's time."""
    return world * ops_per_rank_step / (ms_step * 1e-3) / 1e12


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.idx}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, smax, reasons, power = [], [], set(), []
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
                power.append(float(f[3]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                               f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------ GPU arm
def setup_layers(ctx, torch, dev, layers, calib_samples, rank=0, world=1):
    """Offline part, on the GPU: fold + quantize weights, calibrate per-position scales; then the
    step's activations (drawn on the device)."""
    T = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    out = []
    for L in layers:
        W = T(wl.weights(L))
        Xc, pc = wl.calibration(L, calib_samples)
        Xc_d, pc_d = T(Xc), T(pc)
        s_ch = None
        if L.use_gps:                                      # Algorithm 1 on the calibration set
            s_ch = torch.empty(L.K, device=dev)
            ctx.gps_scales(Xc_d, W, L.bits, PCT, 0, s_ch)
        Wq = torch.empty((L.N, L.K), dtype=torch.int8, device=dev)
        s_w = torch.empty(L.N, device=dev)
        ctx.gps_fold(W, s_ch, L.bits, Wq, s_w)
        s_tok = torch.empty(L.P, device=dev)
        ctx.stwq_calibrate(Xc_d, pc_d, L.P, s_ch, L.bits, PCT, s_tok)
        X, pos = wl.activations_device(L, dev, step=rank_step(rank, 0, world))
        ydt = {"bf16": torch.bfloat16, "fp32": torch.float32}[L.out_dtype]
        Y = torch.empty((L.M, L.N), dtype=ydt, device=dev)
        Xq = torch.empty((L.M, L.K), dtype=torch.int8, device=dev)
        torch.cuda.synchronize()
        del W, Xc_d, pc_d
        out.append(dict(L=L, Wq=Wq, s_w=s_w, s_ch=s_ch, s_tok=s_tok, bias=T(wl.bias(L)), X=X, pos=pos, Y=Y,
                        Xq=Xq, out_code=1 if L.out_dtype == "bf16" else 0))
    ctx.check_device_status()
    return out


def run_step(ctx, S):
    for s in S:
        L = s["L"]
        ctx.qlinear(s["X"], s["pos"], s["Wq"], s["s_w"], s["s_tok"], s["s_ch"], s["bias"], L.bits, L.act,
                    s["out_code"], s["Y"])


def gpu_arm(args):
    import torch
    import torch.distributed as dist

    import paper_2601_21238_b200 as pk
    from paper_2601_21238_b200 import build as pkbuild

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path for the product arm")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        pkbuild.build()
    if world > 1:
        dist.barrier()
    ctx = pk.Context(local)
    layers = wl.config_layers(args.config)
    S = setup_layers(ctx, torch, dev, layers, args.calib_samples, rank, world)
    ops_step = sum(L.ops for L in layers)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing: K whole steps --------------------------------------------
    # The step (4 qlinear calls = 8 kernels) is captured once into a CUDA graph through the same
    # C-ABI calls and replayed K times, the way a serving loop would issue it; --no-graph issues
    # the calls one by one instead (then the host's launch rate adds ~10 % to the step).
    for _ in range(args.warmup):
        run_step(ctx, S)
    torch.cuda.synchronize()
    main = torch.cuda.Stream()
    graph = None
    if not args.no_graph:
        with torch.cuda.stream(main):
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=main):
                run_step(ctx, S)
            for _ in range(args.warmup):
                graph.replay()
        torch.cuda.synchronize()
    launches_per_step = 2 * len(S)
    sampler = ClockSampler(local)
    barrier()
    if rank == 0:
        sampler.start()
    launches0 = ctx.stwq_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    with torch.cuda.stream(main):
        e0.record()
        for _ in range(args.steps):
            if graph is not None:
                graph.replay()
            else:
                run_step(ctx, S)
        e1.record()
    barrier()
    launches = (ctx.stwq_launch_count() - launches0) if graph is None else launches_per_step * args.steps
    ms_total = max_over_ranks(e0.elapsed_time(e1), world, dev)
    clocks = sampler.stop() if rank == 0 else None
    ctx.check_device_status()
    ms_step = ms_total / args.steps
    value = whole_job_tops(world, ops_step, ms_step)

    # ---- per-kernel timing: quantize and GEMM+epilogue separately ------------------------------
    # Each kernel is captured a few times into a CUDA graph and the replays are timed with events
    # on the replay stream, so that the figure is device time, not the host's launch rate. The
    # quantize kernel reads a different copy of X on every launch (working set > L2, as in the
    # step, where the four layers' inputs evict one another); the GEMM reads the codes that the
    # quantize kernel has just written, as in the step.
    side = torch.cuda.Stream()

    def graph_time(calls, replays=5):
        with torch.cuda.stream(side):
            for c in calls:
                c()
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                for c in calls:
                    c()
            g.replay()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(replays):
                g.replay()
            b.record()
            torch.cuda.synchronize()
        return a.elapsed_time(b) / (replays * len(calls))

    tq, tg = {}, {}
    l2_bytes = 2 * 126e6
    for s in S:
        L = s["L"]
        ncopy = max(2, int(l2_bytes // (5.0 * L.M * L.K)) + 1)
        Xc = [s["X"]] + [s["X"].clone() for _ in range(ncopy - 1)]
        tq[L.name] = graph_time([(lambda x=x: ctx.stwq_quantize(x, s["pos"], s["s_ch"], s["s_tok"], L.bits, s["Xq"]))
                                 for x in Xc] * 2)
        del Xc
        tg[L.name] = graph_time([lambda: ctx.qlinear_q(s["Xq"], s["pos"], s["Wq"], s["s_w"], s["s_tok"], s["bias"],
                                                       L.act, s["out_code"], s["Y"])] * 10)
    peaks = measured_peaks()
    per_layer = []
    for s in S:
        L = s["L"]
        qbytes = 5.0 * L.M * L.K
        per_layer.append({"layer": L.name, "M": L.M, "K": L.K, "N": L.N,
                          "gemm_ms": round(tg[L.name], 5), "gemm_tops": round(L.ops / tg[L.name] / 1e9, 1),
                          "quantize_ms": round(tq[L.name], 5),
                          "quantize_gbs": round(qbytes / tq[L.name] / 1e6, 1)})
    gemm_ms = sum(tg.values())
    achieved = ops_step / (gemm_ms * 1e-3) / 1e12
    peak = peaks["bf16_tflops"] * INT8_OVER_BF16
    roofline = {"kernel": "qgemm2_kernel (CTA-pair tcgen05 kind::i8 GEMM + dequant epilogue), mean over the 4 layer shapes", "bound": "tensor",
                "achieved": round(achieved, 1), "peak": round(peak, 1), "unit": "TOP/s",
                "frac": round(achieved / peak, 4),
                "peak_source": f"2 x bf16_tflops of {peaks['_source']} peaks (burst)",
                "avg_launch_ms": round(gemm_ms / len(S), 5), "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH,
                "quantize": {"bound": "hbm", "achieved": round(sum(5.0 * s["L"].M * s["L"].K for s in S)
                                                                / (sum(tq.values()) * 1e-3) / 1e9, 1),
                             "peak": peaks["hbm_gbs"], "unit": "GB/s",
                             "frac": round(sum(5.0 * s["L"].M * s["L"].K for s in S)
                                           / (sum(tq.values()) * 1e-3) / 1e9 / peaks["hbm_gbs"], 4)}}

    if all(s["L"].decode for s in S):
        # few-row layers: the GEMM is the weight-streaming kernel, bound by bytes, not by the pipe
        byts = sum(float(s["L"].N) * s["L"].K + float(s["L"].M) * s["L"].K + 2.0 * s["L"].M * s["L"].N for s in S)
        gbs = byts / (gemm_ms * 1e-3) / 1e9
        roofline.update({"kernel": "decode_kernel (few-row CTA-pair GEMM, weights streamed once), mean over the layer shapes",
                         "bound": "hbm", "achieved": round(gbs, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": round(gbs / peaks["hbm_gbs"], 4),
                         "peak_source": f"hbm_gbs of {peaks['_source']} peaks; weights stay in L2 between replays",
                         "traffic": None})

    # ---- end to end: pinned host X -> device -> qlinear -> device -> pinned host Y ------------
    hX = [torch.empty((s["L"].M, s["L"].K), dtype=torch.float32).pin_memory() for s in S]
    hY = [torch.empty_like(s["Y"], device="cpu").pin_memory() for s in S]
    for h, s in zip(hX, S):
        h.copy_(s["X"])
    torch.cuda.synchronize()
    h2d = sum(h.numel() * h.element_size() for h in hX)
    d2h = sum(h.numel() * h.element_size() for h in hY)

    # Three streams, as a user streaming batches through the layer would do it: copies in, the
    # calls, copies out. A layer's X buffer is refilled only after the call that read it, and its
    # Y buffer rewritten only after the copy that read it (events), so steps overlap but every
    # byte of every step is still copied in and out inside the timed region.
    main = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in S]       # X_i is on the device
    ev_used = [torch.cuda.Event() for _ in S]     # the call has consumed X_i and written Y_i
    ev_out = [torch.cuda.Event() for _ in S]      # Y_i is on the host
    for e in ev_used + ev_out:
        e.record(main)

    def e2e_step():
        for i, (s, hx, hy) in enumerate(zip(S, hX, hY)):
            L = s["L"]
            s_in.wait_event(ev_used[i])
            with torch.cuda.stream(s_in):
                s["X"].copy_(hx, non_blocking=True)
                ev_in[i].record(s_in)
            main.wait_event(ev_in[i])
            main.wait_event(ev_out[i])
            ctx.qlinear(s["X"], s["pos"], s["Wq"], s["s_w"], s["s_tok"], s["s_ch"], s["bias"], L.bits, L.act,
                        s["out_code"], s["Y"])
            ev_used[i].record(main)
            s_out.wait_event(ev_used[i])
            with torch.cuda.stream(s_out):
                hy.copy_(s["Y"], non_blocking=True)
                ev_out[i].record(s_out)

    def e2e_drain():
        main.wait_stream(s_in)
        main.wait_stream(s_out)

    for _ in range(min(args.warmup, 3)):
        e2e_step()
    e2e_drain()
    barrier()
    e0.record()
    for _ in range(args.steps):
        e2e_step()
    e2e_drain()
    e1.record()
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), world, dev) / args.steps
    e2e = {"value": round(whole_job_tops(world, ops_step, e2e_ms), 3), "unit": "TOPS",
           "ms_per_step": round(e2e_ms, 4), "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}
    ctx.check_device_status()

    line = {"metric": "qlinear int8 TOPS (quantize + int8 GEMM + dequant epilogue, whole step)",
            "value": round(value, 2), "unit": "TOPS", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": round(ms_step, 5), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": {"workload": f"config {args.config}: " + ", ".join(
                           f"{L.name} {L.K}->{L.N}" for L in layers) + f"; M={layers[0].M} per GPU, W8A8, "
                           f"{layers[0].out_dtype} out",
                       "l2": "inputs larger than L2 (one step touches ~0.6 GB per GPU)",
                       "launch": "CUDA graph of the step's 4 qlinear calls" if graph is not None else "one C-ABI call at a time",
                       "s_ch": "GPS (Algorithm 1) on the calibration set, computed on the GPU, for qkv/fc1", "calib_samples": args.calib_samples},
            "roofline": roofline, "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
            "layers": per_layer,
            "pct_of_nominal_int8_peak": round(100 * achieved / 4500.0, 2)}
    if not args.no_extras:
        line["other_configs"] = other_configs(ctx, pk, torch, dev, peaks)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(S, layers, torch, rows=args.cpu_rows)
    if rank == 0:
        print(json.dumps(line), flush=True)
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def other_configs(ctx, pk, torch, dev, peaks):
    """Timing-only figures for the workload shapes that are not the benchmark's step (random codes
    and scales of the right shapes; parity of these shapes is the tests' business): the GEMM and
    quantize kernels of the VAR-d30 and MAR-Huge layers, and the decode-step qlinear measured in a
    CUDA graph that rotates through more weight copies than fit in L2."""
    out = {}
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def burst(fn, n=20, warm=3):
        for _ in range(warm):
            fn()
        a, b = ev(), ev()
        a.record()
        for _ in range(n):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / n

    for cfg in (3, 5):
        rows = []
        for L in wl.config_layers(cfg):
            X = torch.randn(L.M, L.K, device=dev)
            Xq = torch.empty((L.M, L.K), dtype=torch.int8, device=dev)
            Wq = torch.randint(-128, 128, (L.N, L.K), dtype=torch.int8, device=dev)
            pos = torch.from_numpy(wl.positions(L)).to(dev)
            s_w = torch.rand(L.N, device=dev) * 1e-3 + 1e-4
            s_tok = torch.rand(L.P, device=dev) * 0.05 + 0.01
            s_ch = (torch.rand(L.K, device=dev) + 0.5) if L.use_gps else None
            b = torch.randn(L.N, device=dev) * 0.02
            Y = torch.empty((L.M, L.N), dtype=torch.bfloat16, device=dev)
            tq = burst(lambda: ctx.stwq_quantize(X, pos, s_ch, s_tok, 8, Xq))
            tg = burst(lambda: ctx.qlinear_q(Xq, pos, Wq, s_w, s_tok, b, L.act, pk.OUT_BF16, Y))
            rows.append({"layer": L.name, "M": L.M, "K": L.K, "N": L.N, "act": L.act,
                         "gemm_tops": round(L.ops / tg / 1e9, 1), "gemm_ms": round(tg, 4),
                         "quantize_gbs": round(5.0 * L.M * L.K / tq / 1e6, 1), "quantize_ms": round(tq, 4)})
            del X, Xq, Wq, Y
        out[f"config{cfg}"] = rows
    # decode step: X fp32 + Wq + Y bf16 per call, weights rotated so that they come from HBM
    rows = []
    copies = 12
    for L in wl.config_layers(4):
        Xs = [torch.randn(L.M, L.K, device=dev) for _ in range(copies)]
        Ws = [torch.randint(-128, 128, (L.N, L.K), dtype=torch.int8, device=dev) for _ in range(copies)]
        Ys = [torch.empty((L.M, L.N), dtype=torch.bfloat16, device=dev) for _ in range(copies)]
        pos = torch.full((L.M,), 17, dtype=torch.int32, device=dev)
        s_w = torch.rand(L.N, device=dev) * 1e-3 + 1e-4
        s_tok = torch.rand(L.P, device=dev) * 0.05 + 0.01
        s_ch = (torch.rand(L.K, device=dev) + 0.5) if L.use_gps else None
        b = torch.randn(L.N, device=dev) * 0.02

        def rot():
            for i in range(copies):
                ctx.qlinear(Xs[i], pos, Ws[i], s_w, s_tok, s_ch, b, 8, 0, pk.OUT_BF16, Ys[i])
        rot()
        torch.cuda.synchronize()
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            rot()
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                rot()
        torch.cuda.synchronize()
        us = burst(g.replay, n=20) / copies * 1e3
        byts = 4.0 * L.M * L.K + L.N * L.K + 2.0 * L.M * L.N
        rows.append({"layer": L.name, "M": L.M, "K": L.K, "N": L.N, "qlinear_us": round(us, 2),
                     "gbs": round(byts / us / 1e3, 1), "frac_of_hbm": round(byts / us / 1e3 / peaks["hbm_gbs"], 4),
                     "tops": round(L.ops / us / 1e6, 1), "timing": f"CUDA graph, {copies} weight copies rotated (HBM-cold)"})
        del Xs, Ws, Ys, g
    out["config4"] = rows
    # static versus dynamic token-wise quantization (Table 5 of the paper prices the dynamic
    # min-max pass at 473.9 ms against 397.9 ms for whole-model latency on its GPU): the two
    # quantize kernels and the two whole calls on the benchmark's layer shapes, inputs rotated
    rows = []
    for L in wl.config_layers(2):
        ncopy = max(2, int(2 * 126e6 // (5.0 * L.M * L.K)) + 1)
        Xs = [torch.randn(L.M, L.K, device=dev) for _ in range(ncopy)]
        Xq = torch.empty((L.M, L.K), dtype=torch.int8, device=dev)
        Wq = torch.randint(-128, 128, (L.N, L.K), dtype=torch.int8, device=dev)
        pos = torch.from_numpy(wl.positions(L)).to(dev)
        s_w = torch.rand(L.N, device=dev) * 1e-3 + 1e-4
        s_tok = torch.rand(L.P, device=dev) * 0.05 + 0.01
        s_row = torch.empty(L.M, device=dev)
        s_ch = (torch.rand(L.K, device=dev) + 0.5) if L.use_gps else None
        b = torch.randn(L.N, device=dev) * 0.02
        Y = torch.empty((L.M, L.N), dtype=torch.bfloat16, device=dev)

        def graph_ms(fn):
            for x in Xs:
                fn(x)
            torch.cuda.synchronize()
            side = torch.cuda.Stream()
            with torch.cuda.stream(side):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    for x in Xs:
                        fn(x)
                g.replay()
                a, e = ev(), ev()
                a.record()
                for _ in range(5):
                    g.replay()
                e.record()
                torch.cuda.synchronize()
            return a.elapsed_time(e) / (5 * len(Xs))
        t_sq = graph_ms(lambda x: ctx.stwq_quantize(x, pos, s_ch, s_tok, 8, Xq))
        t_dq = graph_ms(lambda x: ctx.dtwq_quantize(x, s_ch, 8, Xq, s_row))
        t_sl = graph_ms(lambda x: ctx.qlinear(x, pos, Wq, s_w, s_tok, s_ch, b, 8, L.act, pk.OUT_BF16, Y))
        t_dl = graph_ms(lambda x: ctx.qlinear_dtwq(x, Wq, s_w, s_ch, b, 8, L.act, pk.OUT_BF16, Y))
        rows.append({"layer": L.name, "K": L.K, "N": L.N, "stwq_quantize_us": round(t_sq * 1e3, 2),
                     "dtwq_quantize_us": round(t_dq * 1e3, 2), "stwq_qlinear_us": round(t_sl * 1e3, 2),
                     "dtwq_qlinear_us": round(t_dl * 1e3, 2), "dtwq_over_stwq_qlinear": round(t_dl / t_sl, 3)})
        del Xs, Xq, Wq, Y
    out["static_vs_dynamic_config2"] = rows
    # fc1 -> fc2 of a block, unfused (fc1 writes fp32 activations, fc2's call quantizes them) and
    # chained (fc1's epilogue emits fc2's codes; fc2 runs from codes)
    rows = []
    for cfg in (2, 5):
        fc1, fc2 = [L for L in wl.config_layers(cfg) if L.name in ("fc1", "fc2")]
        X = torch.randn(fc1.M, fc1.K, device=dev)
        pos = torch.from_numpy(wl.positions(fc1)).to(dev)
        W1 = torch.randint(-128, 128, (fc1.N, fc1.K), dtype=torch.int8, device=dev)
        W2 = torch.randint(-128, 128, (fc2.N, fc2.K), dtype=torch.int8, device=dev)
        sw1 = torch.rand(fc1.N, device=dev) * 1e-4 + 1e-5
        sw2 = torch.rand(fc2.N, device=dev) * 1e-3 + 1e-4
        st1 = torch.rand(fc1.P, device=dev) * 0.05 + 0.01
        st2 = torch.rand(fc1.P, device=dev) * 0.05 + 0.01
        sc1 = torch.rand(fc1.K, device=dev) + 0.5
        b1 = torch.randn(fc1.N, device=dev) * 0.02
        b2 = torch.randn(fc2.N, device=dev) * 0.02
        H = torch.empty((fc1.M, fc1.N), dtype=torch.float32, device=dev)
        Hq = torch.empty((fc1.M, fc1.N), dtype=torch.int8, device=dev)
        Y = torch.empty((fc2.M, fc2.N), dtype=torch.bfloat16, device=dev)

        def unfused():
            ctx.qlinear(X, pos, W1, sw1, st1, sc1, b1, 8, fc1.act, pk.OUT_F32, H)
            ctx.qlinear(H, pos, W2, sw2, st2, None, b2, 8, 0, pk.OUT_BF16, Y)

        def chained():
            ctx.qlinear_chain(X, pos, W1, sw1, st1, sc1, b1, 8, fc1.act, None, st2, 8, Hq)
            ctx.qlinear_q(Hq, pos, W2, sw2, st2, b2, 0, pk.OUT_BF16, Y)
        res = {}
        for name, fn in (("unfused", unfused), ("chained", chained)):
            fn()
            torch.cuda.synchronize()
            side = torch.cuda.Stream()
            with torch.cuda.stream(side):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    fn()
                g.replay()
                a, e = ev(), ev()
                a.record()
                for _ in range(10):
                    g.replay()
                e.record()
                torch.cuda.synchronize()
            res[name] = a.elapsed_time(e) / 10
        ops = fc1.ops + fc2.ops
        rows.append({"config": cfg, "M": fc1.M, "hidden": fc1.K, "ffn": fc1.N,
                     "unfused_us": round(res["unfused"] * 1e3, 1), "chained_us": round(res["chained"] * 1e3, 1),
                     "unfused_tops": round(ops / res["unfused"] / 1e9, 1), "chained_tops": round(ops / res["chained"] / 1e9, 1)})
        del X, W1, W2, H, Hq, Y
    out["ffn_fc1_fc2_chained"] = rows
    # the asymmetric quantizer (Eq. 1 with zero points) beside the symmetric one, whole calls
    rows = []
    for L in wl.config_layers(2):
        X = torch.randn(L.M, L.K, device=dev) + 0.5
        Wq = torch.randint(-128, 128, (L.N, L.K), dtype=torch.int8, device=dev)
        pos = torch.from_numpy(wl.positions(L)).to(dev)
        s_w = torch.rand(L.N, device=dev) * 1e-3 + 1e-4
        z_w = torch.randint(-40, 40, (L.N,), dtype=torch.int32, device=dev)
        cs = Wq.to(torch.int32).sum(dim=1).to(torch.int32)
        s_tok = torch.rand(L.P, device=dev) * 0.05 + 0.01
        z_tok = torch.randint(-40, 40, (L.P,), dtype=torch.int32, device=dev)
        s_ch = (torch.rand(L.K, device=dev) + 0.5) if L.use_gps else None
        b = torch.randn(L.N, device=dev) * 0.02
        Y = torch.empty((L.M, L.N), dtype=torch.bfloat16, device=dev)
        res = {}
        for name, fn in (("sym", lambda: ctx.qlinear(X, pos, Wq, s_w, s_tok, s_ch, b, 8, L.act, pk.OUT_BF16, Y)),
                         ("asym", lambda: ctx.qlinear_asym(X, pos, Wq, s_w, z_w, cs, s_tok, z_tok, s_ch, b, 8, L.act,
                                                           pk.OUT_BF16, Y))):
            fn()
            torch.cuda.synchronize()
            side = torch.cuda.Stream()
            with torch.cuda.stream(side):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    for _ in range(4):
                        fn()
                g.replay()
                a, e = ev(), ev()
                a.record()
                for _ in range(5):
                    g.replay()
                e.record()
                torch.cuda.synchronize()
            res[name] = a.elapsed_time(e) / 20
        rows.append({"layer": L.name, "K": L.K, "N": L.N, "sym_qlinear_us": round(res["sym"] * 1e3, 2),
                     "asym_qlinear_us": round(res["asym"] * 1e3, 2), "asym_tops": round(L.ops / res["asym"] / 1e9, 1)})
        del X, Wq, Y
    out["asymmetric_config2"] = rows
    # activations handed over in bf16 (2 bytes read per element instead of 4): qlinear_bf16 beside qlinear
    rows = []
    for L in wl.config_layers(2):
        ncopy = max(2, int(2 * 126e6 // (5.0 * L.M * L.K)) + 1)
        Xs = [torch.randn(L.M, L.K, device=dev) for _ in range(ncopy)]
        Xb = [x.to(torch.bfloat16) for x in Xs]
        Wq = torch.randint(-128, 128, (L.N, L.K), dtype=torch.int8, device=dev)
        pos = torch.from_numpy(wl.positions(L)).to(dev)
        s_w = torch.rand(L.N, device=dev) * 1e-3 + 1e-4
        s_tok = torch.rand(L.P, device=dev) * 0.05 + 0.01
        s_ch = (torch.rand(L.K, device=dev) + 0.5) if L.use_gps else None
        b = torch.randn(L.N, device=dev) * 0.02
        Y = torch.empty((L.M, L.N), dtype=torch.bfloat16, device=dev)
        res = {}
        for name, xs, fn in (("fp32", Xs, ctx.qlinear), ("bf16", Xb, ctx.qlinear_bf16)):
            call = lambda x: fn(x, pos, Wq, s_w, s_tok, s_ch, b, 8, L.act, pk.OUT_BF16, Y)
            for x in xs:
                call(x)
            torch.cuda.synchronize()
            side = torch.cuda.Stream()
            with torch.cuda.stream(side):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    for x in xs:
                        call(x)
                g.replay()
                a, e = ev(), ev()
                a.record()
                for _ in range(5):
                    g.replay()
                e.record()
                torch.cuda.synchronize()
            res[name] = a.elapsed_time(e) / (5 * len(xs))
        rows.append({"layer": L.name, "K": L.K, "N": L.N, "fp32_in_qlinear_us": round(res["fp32"] * 1e3, 2),
                     "bf16_in_qlinear_us": round(res["bf16"] * 1e3, 2), "bf16_in_tops": round(L.ops / res["bf16"] / 1e9, 1)})
        del Xs, Xb, Wq, Y
    out["bf16_input_config2"] = rows
    ctx.check_device_status()
    return out


# ------------------------------------------------------------------------------------------ CPU oracle
def cpu_baseline(S, layers, torch, rows):
    """The oracle's qlinear on the host cores over the first `rows` rows of every layer."""
    import oracle
    total_ops, total_s = 0.0, 0.0
    for s in S:
        L = s["L"]
        r = min(rows, L.M)
        X = s["X"][:r].cpu().numpy()
        pos = s["pos"][:r].cpu().numpy()
        args = (X, pos, s["Wq"].cpu().numpy(), s["s_w"].cpu().numpy(), s["s_tok"].cpu().numpy(),
                None if s["s_ch"] is None else s["s_ch"].cpu().numpy(), s["bias"].cpu().numpy(), L.bits, L.act)
        t0 = time.perf_counter()
        oracle.qlinear(*args)
        total_s += time.perf_counter() - t0
        total_ops += 2.0 * r * L.N * L.K
    return {"value": round(total_ops / total_s / 1e12, 5), "unit": "TOPS", "cores": oracle.num_threads(),
            "kind": "oracle", "seconds": round(total_s, 2),
            "sample": f"first {rows} rows of each of the {len(S)} layers, all output columns"}


def reference_arm(args):
    """The CPU oracle as the reference implementation: same metric, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    layers = wl.config_layers(args.config)

    def prepare(rows):
        prepared = []
        for L in layers:
            W = wl.weights(L)
            s_ch = stand_in_channel_scales(L) if L.use_gps else None
            Wq, s_w = oracle.gps_fold(W, s_ch, L.bits)
            Xc, pc = wl.calibration(L, 2)
            s_tok = oracle.stwq_calibrate(Xc, pc, L.P, s_ch, L.bits, PCT)
            X = wl.activations(L, rows=slice(0, rows))
            pos = wl.positions(L)[:rows]
            prepared.append((L, X, pos, Wq, s_w, s_tok, s_ch, wl.bias(L)))
        return prepared

    def run(prepared):
        for L, X, pos, Wq, s_w, s_tok, s_ch, b in prepared:
            oracle.qlinear(X, pos, Wq, s_w, s_tok, s_ch, b, L.bits, L.act)

    # The sample per step is sized so that warm-up + steps stay within about two minutes: a probe
    # at --ref-rows rows gives the oracle's rate on this host, the rows per step follow from it.
    probe = prepare(args.ref_rows)
    run(probe)
    t0 = time.perf_counter()
    run(probe)
    t_probe = time.perf_counter() - t0
    budget_s = 120.0
    rows = int(args.ref_rows * budget_s / max(1, args.steps + args.warmup) / max(t_probe, 1e-6))
    rows = max(4, min(rows, args.ref_rows * 8, min(L.M for L in layers)))
    prepared = probe if rows == args.ref_rows else prepare(rows)
    ops = sum(2.0 * rows * L.N * L.K for L in layers)

    def step():
        run(prepared)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / args.steps
    v = round(ops / dt / 1e12, 5)
    sample = f"first {rows} rows of each layer per step, all output columns"
    line = {"impl": "reference", "metric": "qlinear int8 TOPS (quantize + int8 GEMM + dequant epilogue, whole step)",
            "value": v, "unit": "TOPS", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": round(dt * 1e3, 3), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": {"workload": f"config {args.config} (CPU oracle, {sample})"},
            "cpu_baseline": {"value": v, "unit": "TOPS", "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": v, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, help="workload family 1..5 (default: VAR-d16 block)")
    ap.add_argument("--calib-samples", type=int, default=32)
    ap.add_argument("--cpu-rows", type=int, default=10880)
    ap.add_argument("--ref-rows", type=int, default=256)
    ap.add_argument("--no-graph", action="store_true", help="issue the step's calls one by one instead of replaying a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the timing-only figures of configs 3, 4, 5")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        reference_arm(args)
    else:
        gpu_arm(args)


if __name__ == "__main__":
    main()
