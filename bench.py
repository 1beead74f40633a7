#!/usr/bin/env python
"""Benchmark of the STWQ quantized linear hot path on B200.

Workload (default): the VAR-d30-shaped block of linears, the largest single-GPU workload of the
method: batch 32 x 680 tokens (M = 21760), hidden 1920: qkv 1920->5760, proj 1920->1920,
fc1 1920->7680, fc2 7680->1920; W8A8, bf16 output; seeded synthetic inputs resident in HBM.

A step is one pass of the whole hot path (activation quantize -> int8 GEMM -> dequantize epilogue,
i.e. one `qlinear` call per layer) over one batch of `--inner` micro-batches of 32 sequences each.
The calls of two micro-batches (two distinct input sets) are captured once into a CUDA graph
through the C ABI and replayed; with the default --inner the timed region of 20 steps lasts more
than half a second, so the clocks are the ones the GPU holds under this load, not a burst. The
metric is int8 TOPS of the whole step (2*M*N*K per layer over the step time, quantize kernels
included).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--config 3] [--inner R]
    python bench.py --ncu-raw-csv FILE --profile-key qgemm2_kernel/config3     # ncu counters -> profiles/

Prints one JSON line (rank 0). With N > 1 (torchrun) every rank runs the same per-GPU batch on
its own rows (weak scaling, no collective on the data path); time is the max over ranks.
`--impl reference` times the CPU oracle on the host cores instead (a deliberately plain program).
"""
from __future__ import annotations

import argparse
import csv
import hashlib
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
NOMINAL_INT8_TOPS = 4500.0
OPS_PER_CLK_PER_SM = 16384.0  # int8 operations one SM's tensor pipe retires per clock
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "roofline_traffic.json")
CSRC = os.path.join(ROOT, "paper_2601_21238_b200", "csrc")
KERNEL_SOURCES = {"qgemm2_kernel": ["stwq_qgemm2.cu", "stwq_ptx.cuh"], "decode_kernel": ["stwq_decode.cu", "stwq_ptx.cuh"],
                  "quantize_kernel": ["stwq_quantize.cu"]}


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


# ------------------------------------------------------------------------------------------ ncu traffic
def source_digest(kernel: str) -> str:
    h = hashlib.sha256()
    for name in KERNEL_SOURCES[kernel]:
        with open(os.path.join(CSRC, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def recorded_traffic(kernel: str, key: str):
    """DRAM bytes (read + write) per launch of `kernel` on workload `key`, from the ncu capture
    recorded in profiles/roofline_traffic.json; None once the kernel's source has changed since."""
    try:
        with open(TRAFFIC_FILE) as f:
            rec = json.load(f)[kernel][key]
    except (OSError, KeyError, ValueError):
        return None, "no ncu capture recorded for this kernel and workload"
    if rec.get("source_digest") != source_digest(kernel):
        return None, "the kernel's source changed after the ncu capture; counters not valid any more"
    return rec["traffic_bytes_per_launch"], rec.get("note", "")


def summarise_ncu(args):
    """Turn `ncu -i REP --page raw --csv --print-units base` output into the per-launch DRAM traffic
    of one kernel and store it, with the digest of the kernel's source, in profiles/roofline_traffic.json."""
    kernel, key = args.profile_key.split("/")
    rows = []
    with open(args.ncu_raw_csv, newline="") as f:
        lines = [ln for ln in f if not ln.startswith("==")]
    rd = csv.reader(lines)
    header = next(rd)
    units = next(rd)
    col = {n: i for i, n in enumerate(header)}
    for r in rd:
        if len(r) != len(header) or kernel.split("_kernel")[0] not in r[col["Kernel Name"]]:
            continue
        def val(name):
            v = float(r[col[name]].replace(",", ""))
            u = units[col[name]].lower()
            return v * {"byte": 1.0, "kbyte": 1e3, "mbyte": 1e6, "gbyte": 1e9, "": 1.0}.get(u, 1.0)
        rows.append({"kernel": r[col["Kernel Name"]][:60], "grid": r[col["Grid Size"]],
                     "dram_read": val("dram__bytes_read.sum"), "dram_write": val("dram__bytes_write.sum"),
                     "ns": float(r[col["gpu__time_duration.sum"]].replace(",", "")) if "gpu__time_duration.sum" in col else None})
    if args.profile_launches:
        rows = [rows[int(i)] for i in args.profile_launches.split(",")]
    if not rows:
        raise SystemExit("no launch of that kernel in the csv")
    rec = {}
    if os.path.exists(TRAFFIC_FILE):
        with open(TRAFFIC_FILE) as f:
            rec = json.load(f)
    mean = sum(r["dram_read"] + r["dram_write"] for r in rows) / len(rows)
    rec.setdefault(kernel, {})[key] = {"traffic_bytes_per_launch": round(mean), "launches": rows,
                                      "source_digest": source_digest(kernel), "note": args.profile_note}
    with open(TRAFFIC_FILE, "w") as f:
        json.dump(rec, f, indent=1)
    print(json.dumps(rec[kernel][key], indent=1))


# ------------------------------------------------------------------------------------------ helpers
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
    """nvidia-smi clocks and throttle reasons sampled while a timed region runs."""
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
        return self

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.1)
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
        # under load = the samples drawing clearly more than idle power
        busy = [c for c, p in zip(sm, power) if power and p > 0.5 * max(power)] or sm
        return {"sm_mhz": statistics.median(busy) if busy else None, "sm_mhz_min": min(busy) if busy else None,
                "sm_max_mhz": max(smax) if smax else None, "power_w_max": max(power) if power else None,
                "samples": len(sm), "samples_under_load": len(busy), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------ GPU arm
def setup_layers(ctx, torch, dev, layers, calib_samples, rank=0, world=1, input_sets=1):
    """Offline part, on the GPU: GPS scales, fold + quantize weights, calibrate per-position scales;
    then the step's activations (drawn on the device), `input_sets` distinct batches per layer."""
    T = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    out = []
    for L in layers:
        W = T(wl.weights(L))
        Xc, pc = wl.calibration(L, calib_samples)
        Xc_d, pc_d = T(Xc), T(pc)
        del Xc
        s_ch = None
        if L.use_gps:                                      # Algorithm 1 on the calibration set
            s_ch = torch.empty(L.K, device=dev)
            ctx.gps_scales(Xc_d, W, L.bits, PCT, 0, s_ch)
        Wq = torch.empty((L.N, L.K), dtype=torch.int8, device=dev)
        s_w = torch.empty(L.N, device=dev)
        ctx.gps_fold(W, s_ch, L.bits, Wq, s_w)
        s_tok = torch.empty(L.P, device=dev)
        ctx.stwq_calibrate(Xc_d, pc_d, L.P, s_ch, L.bits, PCT, s_tok)
        ydt = {"bf16": torch.bfloat16, "fp32": torch.float32}[L.out_dtype]
        Xs, Ys, pos = [], [], None
        for i in range(input_sets):
            X, pos = wl.activations_device(L, dev, step=rank_step(rank, i, world))
            Xs.append(X)
            Ys.append(torch.empty((L.M, L.N), dtype=ydt, device=dev))
        Xq = torch.empty((L.M, L.K), dtype=torch.int8, device=dev)
        torch.cuda.synchronize()
        del W, Xc_d, pc_d
        ctx.stwq_reserve_layer(L.M, L.K, L.N, L.P)        # nothing is allocated inside a capture
        out.append(dict(L=L, Wq=Wq, s_w=s_w, s_ch=s_ch, s_tok=s_tok, bias=T(wl.bias(L)), Xs=Xs, Ys=Ys, X=Xs[0],
                        Y=Ys[0], pos=pos, Xq=Xq, out_code=1 if L.out_dtype == "bf16" else 0))
    ctx.check_device_status()
    return out


def run_block(ctx, S, which=0):
    """One micro-batch: one qlinear call per layer on input set `which`."""
    for s in S:
        L = s["L"]
        ctx.qlinear(s["Xs"][which], s["pos"], s["Wq"], s["s_w"], s["s_tok"], s["s_ch"], s["bias"], L.bits, L.act,
                    s["out_code"], s["Ys"][which])


def capture(torch, stream, fn):
    """Run fn once eagerly (first-use set-up happens outside the capture), then capture it."""
    with torch.cuda.stream(stream):
        fn()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            fn()
        g.replay()
        torch.cuda.synchronize()
    return g


def timed_replays(torch, stream, g, min_seconds, min_replays=3):
    """Mean device time of one replay (ms): events on the replay stream, replays repeated until the
    timed region has lasted min_seconds."""
    with torch.cuda.stream(stream):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        g.replay()
        b.record()
        torch.cuda.synchronize()
        one = max(a.elapsed_time(b), 1e-3)
        n = max(min_replays, int(min_seconds * 1e3 / one) + 1)
        a.record()
        for _ in range(n):
            g.replay()
        b.record()
        torch.cuda.synchronize()
    return a.elapsed_time(b) / n


def kernel_times(ctx, torch, S, seconds):
    """Device time of each layer's quantize kernel and GEMM kernel on their own (ms per launch): each
    is captured several times into a CUDA graph whose replays are timed with events on the replay
    stream for `seconds`. The quantize kernel reads a different copy of X on every launch (working
    set beyond L2); the GEMM reads the codes the quantize kernel wrote, as in the step."""
    side = torch.cuda.Stream()
    tq, tg = {}, {}
    for s in S:
        L = s["L"]
        ncopy = max(2, int(2 * 126e6 // (5.0 * L.M * L.K)) + 1)
        Xc = list(s["Xs"]) + [s["X"].clone() for _ in range(max(0, ncopy - len(s["Xs"])))]

        def qcalls():
            for _ in range(2):
                for x in Xc:
                    ctx.stwq_quantize(x, s["pos"], s["s_ch"], s["s_tok"], L.bits, s["Xq"])
        g = capture(torch, side, qcalls)
        tq[L.name] = timed_replays(torch, side, g, seconds) / (2 * len(Xc))
        del g, Xc

        def gcalls():
            for _ in range(8):
                ctx.qlinear_q(s["Xq"], s["pos"], s["Wq"], s["s_w"], s["s_tok"], s["bias"], L.act, s["out_code"], s["Y"])
        g = capture(torch, side, gcalls)
        tg[L.name] = timed_replays(torch, side, g, seconds) / 8
        del g
    return tq, tg


def probe_peak(ctx, torch, seconds):
    """The int8 tensor pipe on its own (resident operands, no memory traffic): TOPS of a short burst
    after an idle pause and of a loop of `seconds`."""
    side = torch.cuda.Stream()
    out = {}
    with torch.cuda.stream(side):
        ops = ctx.stwq_probe_int8_peak(256)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        best = 0.0
        for _ in range(5):                                   # best of five short launches, an idle pause before each
            time.sleep(0.2)
            a.record()
            ops = ctx.stwq_probe_int8_peak(2048)
            b.record()
            torch.cuda.synchronize()
            best = max(best, ops / a.elapsed_time(b) / 1e9)
        out["burst_tops"] = round(best, 1)
        kb = 8192
        ops = ctx.stwq_probe_int8_peak(kb)
        torch.cuda.synchronize()
        n = max(3, int(seconds / (ops / (out["burst_tops"] * 1e12))) + 1)
        a.record()
        for _ in range(n):
            ctx.stwq_probe_int8_peak(kb)
        b.record()
        torch.cuda.synchronize()
        out["sustained_tops"] = round(n * ops / a.elapsed_time(b) / 1e9, 1)
        out["sustained_seconds"] = round(a.elapsed_time(b) / 1e3, 3)
    ctx.check_device_status()
    return out


def tensor_roofline(S, tg, tq, peaks, clocks, probe, traffic_key):
    ops = sum(s["L"].ops for s in S)
    gemm_ms = sum(tg.values())
    achieved = ops / (gemm_ms * 1e-3) / 1e12
    peak_s = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]) * INT8_OVER_BF16
    peak_b = peaks["bf16_tflops"] * INT8_OVER_BF16
    traffic, note = recorded_traffic("qgemm2_kernel", traffic_key)
    qbytes = sum(5.0 * s["L"].M * s["L"].K for s in S)
    qgbs = qbytes / (sum(tq.values()) * 1e-3) / 1e9
    mhz = clocks.get("sm_mhz") if clocks else None
    r = {"kernel": f"qgemm2_kernel (CTA-pair tcgen05 kind::i8 GEMM + dequant epilogue), over the {len(S)} layer shapes",
         "bound": "tensor", "achieved": round(achieved, 1), "peak": round(peak_s, 1), "unit": "TOP/s",
         "frac": round(achieved / peak_s, 4),
         "peak_source": f"2 x bf16_tflops_sustained of {peaks['_source']} peaks (the kernel is timed in loops of the "
                        f"length of the step, under the power cap); burst figure beside it",
         "peak_burst": round(peak_b, 1), "frac_of_burst_peak": round(achieved / peak_b, 4),
         "frac_of_nominal_int8_4500": round(achieved / NOMINAL_INT8_TOPS, 4),
         "avg_launch_ms": round(gemm_ms / len(S), 5),
         "algorithmic_ops_per_launch": round(ops / len(S)), "traffic": traffic, "traffic_note": note,
         "quantize": {"kernel": "quantize_kernel", "bound": "hbm", "achieved": round(qgbs, 1), "peak": peaks["hbm_gbs"],
                      "unit": "GB/s", "frac": round(qgbs / peaks["hbm_gbs"], 4)}}
    if probe:
        r["peak_probe_tops"] = probe
        r["frac_of_probe_sustained"] = round(achieved / probe["sustained_tops"], 4)
    if mhz:
        clock_peak = OPS_PER_CLK_PER_SM * 148 * mhz * 1e6 / 1e12
        r["clock_peak"] = {"sm_mhz_median": mhz, "tops": round(clock_peak, 1), "frac": round(achieved / clock_peak, 4),
                           "how": "16384 int8 ops per clock per SM x 148 SMs x the median SM clock sampled while the kernels ran"}
    return r


def layer_table(S, tg, tq):
    rows = []
    for s in S:
        L = s["L"]
        rows.append({"layer": L.name, "M": L.M, "K": L.K, "N": L.N, "act": L.act,
                     "gemm_ms": round(tg[L.name], 5), "gemm_tops": round(L.ops / tg[L.name] / 1e9, 1),
                     "quantize_ms": round(tq[L.name], 5), "quantize_gbs": round(5.0 * L.M * L.K / tq[L.name] / 1e6, 1)})
    return rows


def decode_rows(ctx, pk, torch, dev, peaks, seconds):
    """The decode-step shapes (256 rows at one position): whole qlinear calls in a CUDA graph that
    rotates through more weight copies than fit in L2, so that Wq comes from HBM as in a model with
    many layers. Algorithmic bytes per call: X fp32 + Wq + Y bf16."""
    rows = []
    copies = 12
    side = torch.cuda.Stream()
    for L in wl.config_layers(4):
        Xs = [torch.randn(L.M, L.K, device=dev) for _ in range(copies)]
        Ws = [torch.randint(-128, 128, (L.N, L.K), dtype=torch.int8, device=dev) for _ in range(copies)]
        Ys = [torch.empty((L.M, L.N), dtype=torch.bfloat16, device=dev) for _ in range(copies)]
        pos = torch.full((L.M,), 17, dtype=torch.int32, device=dev)
        s_w = torch.rand(L.N, device=dev) * 1e-3 + 1e-4
        s_tok = torch.rand(L.P, device=dev) * 0.05 + 0.01
        s_ch = (torch.rand(L.K, device=dev) + 0.5) if L.use_gps else None
        b = torch.randn(L.N, device=dev) * 0.02
        ctx.stwq_reserve_layer(L.M, L.K, L.N, L.P)

        def rot():
            for i in range(copies):
                ctx.qlinear(Xs[i], pos, Ws[i], s_w, s_tok, s_ch, b, 8, 0, pk.OUT_BF16, Ys[i])
        g = capture(torch, side, rot)
        us = timed_replays(torch, side, g, seconds) / copies * 1e3
        # the same calls from codes a producer layer has already emitted (no quantize step in the chain)
        Xqs = [torch.randint(-128, 128, (L.M, L.K), dtype=torch.int8, device=dev) for _ in range(copies)]

        def rot_q():
            for i in range(copies):
                ctx.qlinear_q(Xqs[i], pos, Ws[i], s_w, s_tok, b, 0, pk.OUT_BF16, Ys[i])
        gq = capture(torch, side, rot_q)
        us_q = timed_replays(torch, side, gq, seconds) / copies * 1e3
        byts_q = 1.0 * L.M * L.K + L.N * L.K + 2.0 * L.M * L.N
        del gq, Xqs
        byts = 4.0 * L.M * L.K + L.N * L.K + 2.0 * L.M * L.N
        traffic, note = recorded_traffic("decode_kernel", L.name)
        rows.append({"layer": L.name, "M": L.M, "K": L.K, "N": L.N, "qlinear_us": round(us, 2),
                     "tops": round(L.ops / us / 1e6, 1), "timing": f"CUDA graph, {copies} weight copies rotated (HBM-cold)",
                     "from_codes": {"qlinear_q_us": round(us_q, 2), "gbs": round(byts_q / us_q / 1e3, 1),
                                    "frac_of_hbm": round(byts_q / us_q / 1e3 / peaks["hbm_gbs"], 4),
                                    "note": "qlinear_q on int8 codes (what a chained producer layer emits): the few-row "
                                            "kernel alone, algorithmic bytes Xq + Wq + Y"},
                     "roofline": {"kernel": "quantize_kernel + decode_kernel (one qlinear call)", "bound": "hbm",
                                  "achieved": round(byts / us / 1e3, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                  "frac": round(byts / us / 1e3 / peaks["hbm_gbs"], 4),
                                  "algorithmic_bytes_per_launch": byts, "traffic": traffic, "traffic_note": note}})
        del Xs, Ws, Ys, g
    return rows


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
    inner = max(2, args.inner + (args.inner & 1))           # micro-batches per step, two per graph replay
    S = setup_layers(ctx, torch, dev, layers, args.calib_samples, rank, world, input_sets=2)
    ops_block = sum(L.ops for L in layers)
    ops_step = ops_block * inner

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing: K whole steps --------------------------------------------
    def two_blocks():
        run_block(ctx, S, 0)
        run_block(ctx, S, 1)

    main = torch.cuda.Stream()
    graph = None if args.no_graph else capture(torch, main, two_blocks)

    def one_step():
        for _ in range(inner // 2):
            if graph is not None:
                graph.replay()
            else:
                two_blocks()

    with torch.cuda.stream(main):
        for _ in range(args.warmup):
            one_step()
    torch.cuda.synchronize()
    launches_per_step = 2 * len(S) * inner
    sampler = ClockSampler(local)
    barrier()
    if rank == 0:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    with torch.cuda.stream(main):
        e0.record()
        for _ in range(args.steps):
            one_step()
        e1.record()
    barrier()
    launches = launches_per_step * args.steps
    ms_total = max_over_ranks(e0.elapsed_time(e1), world, dev)
    clocks = sampler.stop() if rank == 0 else None
    ctx.check_device_status()
    ms_step = ms_total / args.steps
    value = whole_job_tops(world, ops_step, ms_step)

    # ---- per-kernel timing, the pipe's own peak, the roofline -----------------------------------
    ksampler = ClockSampler(local).start() if rank == 0 else None
    tq, tg = kernel_times(ctx, torch, S, args.kernel_seconds)
    kclocks = ksampler.stop() if ksampler else None
    probe = None
    if rank == 0 and not args.no_probe:
        psampler = ClockSampler(local).start()
        probe = probe_peak(ctx, torch, args.probe_seconds)
        probe["clocks"] = psampler.stop()
    peaks = measured_peaks()
    decode = all(s["L"].decode for s in S)
    if decode:
        byts = sum(float(s["L"].N) * s["L"].K + float(s["L"].M) * s["L"].K + 2.0 * s["L"].M * s["L"].N for s in S)
        gbs = byts / (sum(tg.values()) * 1e-3) / 1e9
        roofline = {"kernel": "decode_kernel (few-row CTA-pair GEMM, weights streamed once), over the layer shapes",
                    "bound": "hbm", "achieved": round(gbs, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": round(gbs / peaks["hbm_gbs"], 4),
                    "peak_source": f"hbm_gbs of {peaks['_source']} peaks; weights stay in L2 between replays here, "
                                   f"the HBM-cold figure is under other_configs.config4",
                    "traffic": None}
    else:
        roofline = tensor_roofline(S, tg, tq, peaks, kclocks, probe, f"config{args.config}")
    roofline["clocks_while_timed"] = kclocks

    # ---- end to end: pinned host X -> device -> qlinear -> device -> pinned host Y ------------
    e2e_inner = 2
    hX = [torch.empty((s["L"].M, s["L"].K), dtype=torch.float32).pin_memory() for s in S]
    hY = [torch.empty_like(s["Y"], device="cpu").pin_memory() for s in S]
    for h, s in zip(hX, S):
        h.copy_(s["X"])
    torch.cuda.synchronize()
    h2d = sum(h.numel() * h.element_size() for h in hX) * e2e_inner
    d2h = sum(h.numel() * h.element_size() for h in hY) * e2e_inner

    # Three streams, as a user streaming batches through the layer would do it: copies in, the
    # calls, copies out. A layer's X buffer is refilled only after the call that read it, and its
    # Y buffer rewritten only after the copy that read it (events), so micro-batches overlap but
    # every byte of every micro-batch is still copied in and out inside the timed region.
    cur = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in S]       # X_i is on the device
    ev_used = [torch.cuda.Event() for _ in S]     # the call has consumed X_i and written Y_i
    ev_out = [torch.cuda.Event() for _ in S]      # Y_i is on the host
    for e in ev_used + ev_out:
        e.record(cur)

    def e2e_block():
        for i, (s, hx, hy) in enumerate(zip(S, hX, hY)):
            L = s["L"]
            s_in.wait_event(ev_used[i])
            with torch.cuda.stream(s_in):
                s["X"].copy_(hx, non_blocking=True)
                ev_in[i].record(s_in)
            cur.wait_event(ev_in[i])
            cur.wait_event(ev_out[i])
            ctx.qlinear(s["X"], s["pos"], s["Wq"], s["s_w"], s["s_tok"], s["s_ch"], s["bias"], L.bits, L.act,
                        s["out_code"], s["Y"])
            ev_used[i].record(cur)
            s_out.wait_event(ev_used[i])
            with torch.cuda.stream(s_out):
                hy.copy_(s["Y"], non_blocking=True)
                ev_out[i].record(s_out)

    def e2e_drain():
        cur.wait_stream(s_in)
        cur.wait_stream(s_out)

    for _ in range(2):
        e2e_block()
    e2e_drain()
    barrier()
    e0.record()
    for _ in range(args.steps * e2e_inner):
        e2e_block()
    e2e_drain()
    e1.record()
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), world, dev) / args.steps
    e2e = {"value": round(whole_job_tops(world, ops_block * e2e_inner, e2e_ms), 3), "unit": "TOPS",
           "ms_per_step": round(e2e_ms, 4), "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
           "micro_batches_per_step": e2e_inner,
           "note": "the same metric through the C-ABI call with pinned host buffers: every micro-batch's X is copied "
                   "in and its Y copied out inside the timed region; a rate, so the step here is "
                   f"{e2e_inner} micro-batches instead of {inner} to keep the run short"}
    ctx.check_device_status()

    L0 = layers[0]
    line = {"metric": "qlinear int8 TOPS (quantize + int8 GEMM + dequant epilogue, whole step)",
            "value": round(value, 2), "unit": "TOPS", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": round(ms_step, 5), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": {"workload": f"config {args.config}: " + ", ".join(f"{L.name} {L.K}->{L.N}" for L in layers)
                                   + f"; M={L0.M} rows per micro-batch, {inner} micro-batches per step per GPU, "
                                     f"W{L0.bits}A{L0.bits}, {L0.out_dtype} out",
                       "timed_region_s": round(ms_total / 1e3, 3),
                       "l2": f"inputs larger than L2 (one micro-batch touches "
                             f"{sum(4.0 * L.M * L.K + L.N * L.K + 2.0 * L.M * L.N for L in layers) / 1e9:.2f} GB per GPU; "
                             f"two input sets alternate)",
                       "launch": "CUDA graph of two micro-batches (8 qlinear calls), replayed" if graph is not None
                                 else "one C-ABI call at a time",
                       "s_ch": "GPS (Algorithm 1) on the calibration set, computed on the GPU, for qkv/fc1",
                       "calib_samples": args.calib_samples},
            "roofline": roofline, "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
            "layers": layer_table(S, tg, tq),
            "kernel_sum_check": {"sum_kernel_ms_per_micro_batch": round(sum(tg.values()) + sum(tq.values()), 5),
                                 "step_ms_per_micro_batch": round(ms_step / inner, 5)}}
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(S, torch, rows=args.cpu_rows)
    del hX, hY, graph
    for s in S:
        s.clear()
    del S
    torch.cuda.empty_cache()
    if not args.no_extras and rank == 0:
        line["other_configs"] = other_configs(ctx, pk, torch, dev, peaks, args)
    if rank == 0:
        print(json.dumps(line), flush=True)
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def whole_config(ctx, torch, dev, cfg, peaks, args):
    """Another workload family measured the way the headline is: seeded layers, offline calls on the
    GPU, a CUDA graph of real qlinear calls, whole-step value, per-kernel times."""
    layers = wl.config_layers(cfg)
    S = setup_layers(ctx, torch, dev, layers, args.calib_samples, input_sets=2)
    side = torch.cuda.Stream()

    def two_blocks():
        run_block(ctx, S, 0)
        run_block(ctx, S, 1)
    g = capture(torch, side, two_blocks)
    ms = timed_replays(torch, side, g, args.extra_seconds) / 2
    ops = sum(L.ops for L in layers)
    tq, tg = kernel_times(ctx, torch, S, args.kernel_seconds / 2)
    out = {"workload": ", ".join(f"{L.name} {L.K}->{L.N}" for L in layers) + f"; M={layers[0].M}, W8A8, bf16 out",
           "ms_per_micro_batch": round(ms, 5), "value_tops": round(ops / ms / 1e9, 1),
           "roofline": tensor_roofline(S, tg, tq, peaks, None, None, f"config{cfg}"), "layers": layer_table(S, tg, tq)}
    ctx.check_device_status()
    del g
    for s in S:
        s.clear()
    torch.cuda.empty_cache()
    return out


def attention_rows(ctx, pk, torch, dev, peaks, graph_us):
    """Quantized attention of a VAR-d16-shaped layer (batch 16 x 16 heads, 680 positions, head dimension
    64): filling the quantized KV cache, then the attention head on int8 codes, as one kernel and as
    three separate stages (block-causal masks of the real model are replaced by a plain causal one)."""
    out = {}
    G, T, d, Tmax = 256, 680, 64, 688
    Q = torch.randn(G, T, d, device=dev)
    Kn = torch.randn(G, T, d, device=dev)
    Vn = torch.randn(G, T, d, device=dev)
    pos_q = torch.arange(T, dtype=torch.int32, device=dev)
    s_q = torch.full((T,), 4.0 * 2 / 255, device=dev)
    s_k = torch.full((T,), 4.0 * 2 / 255, device=dev)
    s_kcol = s_k * (1.0 / d ** 0.5)
    s_v = torch.full((d,), 4.0 * 2 / 255, device=dev)
    Kc = torch.zeros((G, Tmax, d), dtype=torch.int8, device=dev)
    Vt = torch.zeros((G, d, Tmax), dtype=torch.int8, device=dev)
    O = torch.empty((G, T, d), dtype=torch.bfloat16, device=dev)
    ctx.stwq_reserve_attention(G, T, T, d)
    t_app = graph_us(lambda: ctx.kv_append(Kn, Vn, 0, s_k, s_v, 8, Kc, Vt), 1)
    t_att = graph_us(lambda: ctx.qattention(Q, pos_q, T, Kc, Vt, s_q, s_kcol, s_v, 8, True, pk.OUT_BF16, O), 1)
    # a decode step: one new query per head against the whole cache
    Q1 = torch.randn(G, 1, d, device=dev)
    O1 = torch.empty((G, 1, d), dtype=torch.bfloat16, device=dev)
    pos_1 = torch.full((1,), T - 1, dtype=torch.int32, device=dev)
    t_dec = graph_us(lambda: ctx.qattention(Q1, pos_1, T, Kc, Vt, s_q, s_kcol, s_v, 8, False, pk.OUT_BF16, O1), 1)
    ctx.stwq_set_option(pk.OPT_VARIANT, 9)
    try:
        ctx.stwq_reserve_attention(G, T, T, d)
        t_staged = graph_us(lambda: ctx.qattention(Q, pos_q, T, Kc, Vt, s_q, s_kcol, s_v, 8, True, pk.OUT_BF16, O), 1)
    finally:
        ctx.stwq_set_option(pk.OPT_VARIANT, 0)
    # what a head must move: Q fp32, both code caches once, O
    att_bytes = G * T * d * (4 + 2) + 2 * G * T * d
    app_bytes = 2 * G * T * d * (4 + 1)
    # what bounds the one-kernel head is the exponential: one ex2 per score and walk, 16 per clock per SM.
    # Scores are processed in blocks of 32 rows x 32 keys; a block is skipped when the causal mask hides
    # all of it.
    blocks = 0
    for q0 in range(0, T, 32):
        last_visible = min(T - 1, q0 + 31)                   # Tq = Tk: the last row of the block of rows sees this key
        blocks += last_visible // 32 + 1
    ex2 = 2.0 * G * blocks * 32 * 32
    xu_peak = 16.0 * 148 * 1.965e9
    # the kernel alone (the key scales are padded by a tiny kernel in the same call)
    out["attention_var_d16"] = {"heads": G, "positions": T, "head_dim": d, "kv_append_us": round(t_app, 1),
                                "kv_append_frac_of_hbm": round(app_bytes / t_app / 1e3 / peaks["hbm_gbs"], 3),
                                "qattention_us": round(t_att, 1),
                                "qattention_three_stages_us": round(t_staged, 1),
                                "qattention_one_query_per_head_us": round(t_dec, 1),
                                "matmul_tops": round(2 * 2.0 * G * T * T * d / t_att / 1e6, 1),
                                "min_bytes_frac_of_hbm": round(att_bytes / t_att / 1e3 / peaks["hbm_gbs"], 3),
                                "roofline": {"kernel": "qattn_fused_kernel", "bound": "alu", "unit": "G ex2/s",
                                             "achieved": round(ex2 / t_att / 1e3, 1), "peak": round(xu_peak / 1e9, 1),
                                             "frac": round(ex2 / (t_att * 1e-6) / xu_peak, 3),
                                             "peak_source": "16 ex2 per clock per SM x 148 SMs x 1965 MHz (the special-function "
                                                            "unit; a loop of nothing but ex2 measures 16.3 per clock per SM)"},
                                "note": "one kernel per 128 queries of a head: Q quantized, Q K^T, softmax, probability codes "
                                        "and P V on the SM (keys walked twice); three_stages = batched int8 GEMMs with scores "
                                        "and codes in workspace; one_query_per_head = a decode step (one CTA per head reads the "
                                        "cache once, dp4a, caches L2-resident here); ops counted for the full T x T matrices, "
                                        "bytes = Q fp32 + both code caches + O bf16"}
    del Q, Kn, Vn, Kc, Vt, O, Q1, O1
    return out["attention_var_d16"]


def other_configs(ctx, pk, torch, dev, peaks, args):
    """The other workload families: whole-step figures of the VAR-d16 and MAR-Huge blocks (and of
    VAR-d30 when it is not the headline), the decode-step calls with their own roofline, and a few
    comparisons on the VAR-d16 layer shapes (static against dynamic token-wise quantization,
    chained against unfused fc1 -> fc2 with the exact and the short GELU, asymmetric against
    symmetric, bf16 against fp32 input)."""
    out = {}
    ev = lambda: torch.cuda.Event(enable_timing=True)
    for cfg in (2, 3, 5):
        if cfg != args.config:
            out[f"config{cfg}"] = whole_config(ctx, torch, dev, cfg, peaks, args)
    out["config4"] = decode_rows(ctx, pk, torch, dev, peaks, args.extra_seconds)
    side = torch.cuda.Stream()

    def graph_us(fn, calls_per_graph, seconds=0.05):
        g = capture(torch, side, fn)
        return timed_replays(torch, side, g, seconds) / calls_per_graph * 1e3

    # static versus dynamic token-wise quantization (Table 5 of the paper prices the dynamic
    # min-max pass at 473.9 ms against 397.9 ms for whole-model latency on its GPU): the two
    # quantize kernels and the two whole calls on the VAR-d16 layer shapes, inputs rotated
    rows = []
    for L in wl.config_layers(2):
        ncopy = max(2, int(2 * 126e6 // (5.0 * L.M * L.K)) + 1)
        Xs = [torch.randn(L.M, L.K, device=dev) for _ in range(ncopy)]
        Xb = [x.to(torch.bfloat16) for x in Xs]
        Xq = torch.empty((L.M, L.K), dtype=torch.int8, device=dev)
        Wq = torch.randint(-128, 128, (L.N, L.K), dtype=torch.int8, device=dev)
        pos = torch.from_numpy(wl.positions(L)).to(dev)
        s_w = torch.rand(L.N, device=dev) * 1e-3 + 1e-4
        s_tok = torch.rand(L.P, device=dev) * 0.05 + 0.01
        s_row = torch.empty(L.M, device=dev)
        s_ch = (torch.rand(L.K, device=dev) + 0.5) if L.use_gps else None
        b = torch.randn(L.N, device=dev) * 0.02
        Y = torch.empty((L.M, L.N), dtype=torch.bfloat16, device=dev)
        z_w = torch.randint(-40, 40, (L.N,), dtype=torch.int32, device=dev)
        cs = Wq.to(torch.int32).sum(dim=1).to(torch.int32)
        z_tok = torch.randint(-40, 40, (L.P,), dtype=torch.int32, device=dev)
        ctx.stwq_reserve_layer(L.M, L.K, L.N, L.P)

        def over(fn, xs=Xs):
            def run():
                for x in xs:
                    fn(x)
            return graph_us(run, len(xs))
        rows.append({"layer": L.name, "K": L.K, "N": L.N,
                     "stwq_quantize_us": round(over(lambda x: ctx.stwq_quantize(x, pos, s_ch, s_tok, 8, Xq)), 2),
                     "dtwq_quantize_us": round(over(lambda x: ctx.dtwq_quantize(x, s_ch, 8, Xq, s_row)), 2),
                     "stwq_qlinear_us": round(over(lambda x: ctx.qlinear(x, pos, Wq, s_w, s_tok, s_ch, b, 8, L.act, pk.OUT_BF16, Y)), 2),
                     "dtwq_qlinear_us": round(over(lambda x: ctx.qlinear_dtwq(x, Wq, s_w, s_ch, b, 8, L.act, pk.OUT_BF16, Y)), 2),
                     "asym_qlinear_us": round(over(lambda x: ctx.qlinear_asym(x, pos, Wq, s_w, z_w, cs, s_tok, z_tok, s_ch, b, 8,
                                                                             L.act, pk.OUT_BF16, Y)), 2),
                     "bf16_in_qlinear_us": round(over(lambda x: ctx.qlinear_bf16(x, pos, Wq, s_w, s_tok, s_ch, b, 8, L.act,
                                                                                 pk.OUT_BF16, Y), Xb), 2)})
        del Xs, Xb, Xq, Wq, Y
    out["var_d16_layers_static_dynamic_asym_bf16in"] = rows
    # fc1 -> fc2 of a block, unfused (fc1 writes fp32 activations, fc2's call quantizes them) and
    # chained (fc1's epilogue emits fc2's codes; fc2 runs from codes), with the GELU of the model
    # (erf form, fp32-accurate) and with the short form a caller may ask for
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
        ctx.stwq_reserve_layer(fc2.M, fc2.K, fc2.N, fc2.P)
        row = {"config": cfg, "M": fc1.M, "hidden": fc1.K, "ffn": fc1.N}
        for tag, act in (("gelu_erf", pk.ACT_GELU_ERF), ("gelu_fast", pk.ACT_GELU_FAST)):
            def unfused():
                ctx.qlinear(X, pos, W1, sw1, st1, sc1, b1, 8, act, pk.OUT_F32, H)
                ctx.qlinear(H, pos, W2, sw2, st2, None, b2, 8, 0, pk.OUT_BF16, Y)

            def chained():
                ctx.qlinear_chain(X, pos, W1, sw1, st1, sc1, b1, 8, act, None, st2, 8, Hq)
                ctx.qlinear_q(Hq, pos, W2, sw2, st2, b2, 0, pk.OUT_BF16, Y)
            row[f"unfused_{tag}_us"] = round(graph_us(unfused, 1), 1)
            row[f"chained_{tag}_us"] = round(graph_us(chained, 1), 1)
        row["chained_gelu_erf_tops"] = round((fc1.ops + fc2.ops) / row["chained_gelu_erf_us"] / 1e6, 1)
        rows.append(row)
        del X, W1, W2, H, Hq, Y
    out["ffn_fc1_fc2_chained"] = rows
    out["attention_var_d16"] = attention_rows(ctx, pk, torch, dev, peaks, graph_us)
    ctx.check_device_status()
    return out


# ------------------------------------------------------------------------------------------ CPU oracle
def cpu_baseline(S, torch, rows):
    """The oracle's qlinear on the host cores over the first `rows` rows of every layer."""
    import oracle
    total_ops, total_s = 0.0, 0.0
    for s in S:
        L = s["L"]
        r = min(rows, L.M)
        X = s["X"][:r].cpu().numpy()
        pos = s["pos"][:r].cpu().numpy()
        a = (X, pos, s["Wq"].cpu().numpy(), s["s_w"].cpu().numpy(), s["s_tok"].cpu().numpy(),
             None if s["s_ch"] is None else s["s_ch"].cpu().numpy(), s["bias"].cpu().numpy(), L.bits, L.act)
        t0 = time.perf_counter()
        oracle.qlinear(*a)
        total_s += time.perf_counter() - t0
        total_ops += 2.0 * r * L.N * L.K
    return {"value": round(total_ops / total_s / 1e12, 5), "unit": "TOPS", "cores": oracle.num_threads(),
            "kind": "oracle", "seconds": round(total_s, 2),
            "sample": f"first {rows} rows of each of the {len(S)} layers of the same workload, all output columns; "
                      f"rows are independent, so the rate carries over to the full batch (extrapolated)",
            "threads_note": "the oracle's integer GEMM loop runs on all `cores` threads; its quantize and "
                            "dequantize loops are serial (a few per cent of its time)"}


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


def attention_arm(args):
    """Only the attention layer of other_configs(), for a profiler capture of its kernels."""
    import torch

    import paper_2601_21238_b200 as pk
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path for the product arm")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    ctx = pk.Context(0)
    side = torch.cuda.Stream()

    def graph_us(fn, calls_per_graph, seconds=args.extra_seconds):
        g = capture(torch, side, fn)
        return timed_replays(torch, side, g, seconds) / calls_per_graph * 1e3

    row = attention_rows(ctx, pk, torch, dev, measured_peaks(), graph_us)
    ctx.check_device_status()
    print(json.dumps({"attention_var_d16": row}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=3, help="workload family 2..5 (default: the VAR-d30 block)")
    ap.add_argument("--inner", type=int, default=32, help="micro-batches per step (even)")
    ap.add_argument("--calib-samples", type=int, default=32)
    ap.add_argument("--cpu-rows", type=int, default=16384)
    ap.add_argument("--ref-rows", type=int, default=128)
    ap.add_argument("--kernel-seconds", type=float, default=0.2, help="timed seconds per kernel in the per-kernel section")
    ap.add_argument("--probe-seconds", type=float, default=0.5)
    ap.add_argument("--extra-seconds", type=float, default=0.2)
    ap.add_argument("--no-graph", action="store_true", help="issue the step's calls one by one instead of replaying a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-probe", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the other workload families")
    ap.add_argument("--only-attention", action="store_true", help="time only the quantized attention layer (profiling aid)")
    ap.add_argument("--ncu-raw-csv", help="raw ncu csv export to summarise into profiles/roofline_traffic.json")
    ap.add_argument("--profile-key", default="qgemm2_kernel/config3", help="kernel/workload the csv belongs to")
    ap.add_argument("--profile-note", default="")
    ap.add_argument("--profile-launches", default="", help="comma-separated indices of the launches (of that kernel) to use")
    args = ap.parse_args()
    if args.ncu_raw_csv:
        summarise_ncu(args)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        reference_arm(args)
    elif args.only_attention:
        attention_arm(args)
    else:
        gpu_arm(args)


if __name__ == "__main__":
    main()
