#!/usr/bin/env python
"""Benchmark of the low-bit / routed decoder linear path on B200.

One step = one pass of the decode sweep over a 7B-class decoder layer's four linears
(fused QKV 4096->12288, O 4096->4096, fused gate/up 4096->22016, down 11008->4096) at
M in {1, 8, 16}, INT4 group 128: twelve dmr_lowbit_linear calls.  The headline value is the
weight bytes those calls stream divided by the time they take (GB/s), to be read against the
HBM copy bandwidth.  Further sections of the same JSON line report prefill TFLOP/s, the routed
batch, quantization and the dense bf16 linear.

Timing: CUDA events on the launching stream around CUDA-graph replays; several independent
copies of the layer are visited in rotation so that no call finds its weights in L2.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--sections a,b,...]
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "low-bit linear: decode weight GB/s vs HBM peak; prefill TFLOP/s vs bf16 peak"
WORKLOAD = "decode sweep, 7B-class layer (qkv, o, gate_up, down), M in {1,8,16}, INT4 g=128"
DECODE_MS = (1, 8, 16)
BITS, GROUP = 4, 128
# dram__bytes_read.sum + dram__bytes_write.sum per launch of decode_stream_kernel, mean of the four 7B-class
# linears at M = 1 (ncu capture summarised in profiles/decode_stream_kernel_int4_g128_7b_M1.txt)
DECODE_TRAFFIC_BYTES_PER_LAUNCH = 26.56e6
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


# ----------------------------------------------------------------------------------------------
# clocks sampler
# ----------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while a region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.samples = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 7:
                self.samples.append(parts)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            try:
                sm.append(float(s[0]))
                mx.append(float(s[1]))
                power.append(float(s[2]))
            except ValueError:
                continue
            for name, v in zip(names, s[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------------------------
# reference arm: the CPU oracle on a bounded sample of the same workload
# ----------------------------------------------------------------------------------------------
class OracleDecode:
    """The CPU oracle on the decode sweep: the same twelve calls as one GPU step, optionally on the
    first `frac` of each linear's output features so that a step stays bounded."""

    def __init__(self):
        import oracle
        from paper_2602_02711_b200 import inputs
        self.oracle = oracle
        self.cores = oracle.num_threads()
        self.layers = {}
        for i, (name, (N, K)) in enumerate(inputs.LAYER_7B.items()):
            W = inputs.weights(N, K, seed=0, index=i)
            self.layers[name] = (N, K, oracle.quantize(W, bits=BITS, group=GROUP))
        self.X = {(name, M): inputs.activations(M, K, seed=0, index=M)
                  for name, (N, K, _) in self.layers.items() for M in DECODE_MS}

    def step(self, frac: float = 1.0):
        """Runs the sweep; returns (weight bytes streamed, seconds)."""
        nbytes, t0 = 0.0, time.perf_counter()
        for M in DECODE_MS:
            for name, (N, K, (qw, sc, zp)) in self.layers.items():
                n = max(16, int(N * frac))
                self.oracle.lowbit_linear(self.X[(name, M)], qw[:n], sc[:n], zp[:n], bits=BITS, group=GROUP)
                nbytes += qw[:n].nbytes + sc[:n].nbytes + zp[:n].nbytes
        return nbytes, time.perf_counter() - t0

    def describe(self, frac):
        part = "all output features" if frac >= 1.0 else f"first {frac:.3%} of each linear's output features"
        return f"oracle lowbit_linear (fp64, OpenMP), 7B decode sweep M in {{1,8,16}}, {part}"


def oracle_cpu_baseline(target_seconds: float = 12.0):
    od = OracleDecode()
    nb, sec, n = 0.0, 0.0, 0
    while sec < target_seconds and n < 8:
        b, t = od.step(1.0)
        nb += b
        sec += t
        n += 1
    return nb / sec / 1e9, od.cores, od.describe(1.0) + f", {n} passes, {sec:.1f} s"


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    od = OracleDecode()
    b, t = od.step(0.02)                       # calibration pass
    rate = b / t
    budget = min(3.0, 150.0 / (args.steps + args.warmup))
    full_bytes, _ = 0, 0
    full_bytes = sum(qw.nbytes + sc.nbytes + zp.nbytes for (_, _, (qw, sc, zp)) in od.layers.values()) * len(DECODE_MS)
    frac = min(1.0, rate * budget / full_bytes)
    for _ in range(args.warmup):
        od.step(frac)
    nb, sec = 0.0, 0.0
    for _ in range(args.steps):
        b, t = od.step(frac)
        nb += b
        sec += t
    value = nb / sec / 1e9
    sample = od.describe(frac)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": od.cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
# GPU arm
# ----------------------------------------------------------------------------------------------
def time_graph_replays(graphs, steps, warmup, torch, flush=None):
    """Replays graphs[s % len] for warmup + steps steps; returns seconds for the timed steps."""
    stream = torch.cuda.current_stream()
    for s in range(warmup):
        graphs[s % len(graphs)].replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for s in range(steps):
        graphs[(warmup + s) % len(graphs)].replay()
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e-3


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2602_02711_b200 as dmr
    from paper_2602_02711_b200 import inputs, sharding, QFormat, OUT_BF16

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    peaks = load_peaks()
    fmt = QFormat(BITS, GROUP)
    l2_bytes = torch.cuda.get_device_properties(dev).L2_cache_size
    sections = set(args.sections.split(",")) if args.sections else {"decode", "e2e", "cpu", "prefill", "routed", "dense", "quantize", "layer_cost", "kl"}

    def bf16_dev(bits_np):
        return torch.from_numpy(bits_np.view(np.int16)).view(torch.bfloat16).to(dev)

    # ---- weights: `copies` independent layers so that rotation defeats the L2 ----
    shapes = inputs.LAYER_7B
    names = list(shapes)
    layer_bytes = sum(N * K // 2 + 3 * N * (K // GROUP) for N, K in shapes.values())
    copies = max(4, int(np.ceil(3.0 * l2_bytes / layer_bytes)))
    layers = []
    for c in range(copies):
        qs = {}
        for i, name in enumerate(names):
            N, K = shapes[name]
            g = torch.Generator(device=dev)
            g.manual_seed(1000 * c + i + 17 * rank)
            W = (torch.randn((N, K), generator=g, device=dev, dtype=torch.float32) * inputs.WEIGHT_SIGMA).to(torch.bfloat16)
            qs[name] = dmr.dmr_quantize(W, fmt)
            del W
        layers.append(qs)
    assert sum(q.weight_bytes() for q in layers[0].values()) == layer_bytes
    X = {(name, M): bf16_dev(inputs.activations(M, shapes[name][1], seed=0, index=M)) for name in names for M in DECODE_MS}
    Y = {(name, M): torch.empty((M, shapes[name][0]), dtype=torch.bfloat16, device=dev) for name in names for M in DECODE_MS}
    ws = dmr.new_workspace(0, 16, 22016, 11008, fmt, dev)

    def decode_step(step_index: int):
        for mi, M in enumerate(DECODE_MS):
            layer = layers[(step_index * len(DECODE_MS) + mi) % copies]
            for name in names:
                dmr.dmr_lowbit_linear(X[(name, M)], layer[name], OUT_BF16, Y=Y[(name, M)], workspace=ws)

    result = {}
    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        # warm-up outside capture (sets kernel attributes), then capture one graph per rotation phase
        for s in range(copies):
            decode_step(s)
        torch.cuda.synchronize()
        period = copies  # step s and s + copies use the same layer copies
        graphs, launches_per_step = [], 0
        for s in range(period):
            g = torch.cuda.CUDAGraph()
            n0 = dmr.dmr_launch_count()
            with torch.cuda.graph(g, stream=stream):
                decode_step(s)
            launches_per_step = dmr.dmr_launch_count() - n0
            graphs.append(g)
        torch.cuda.synchronize()

        sampler = ClockSampler(local)
        sampler.start()
        # keep the GPU under the same load while nvidia-smi starts sampling (not timed)
        t_load = time.perf_counter()
        while time.perf_counter() - t_load < 1.5:
            for s in range(period):
                graphs[s].replay()
            torch.cuda.synchronize()
        sharding.barrier()
        torch.cuda.synchronize()
        seconds = time_graph_replays(graphs, args.steps, args.warmup, torch)
        sharding.barrier()
        clocks = sampler.stop()

        step_bytes = layer_bytes * len(DECODE_MS)
        t_max = sharding.max_over_ranks(seconds, dev)
        value = sharding.sum_over_ranks(step_bytes * args.steps, dev) / t_max / 1e9
        per_gpu = step_bytes * args.steps / seconds / 1e9
        n_launch = launches_per_step * args.steps
        result.update({
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": t_max / args.steps * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "format": "asymmetric INT4, group 128, bf16 scale, u8 zero",
                       "weight_bytes_per_step": step_bytes, "layer_copies": copies,
                       "l2": f"{copies} layer copies ({copies * layer_bytes / 1e6:.0f} MB) visited in rotation; "
                             f"L2 is {l2_bytes / 1e6:.0f} MB, so inputs exceed L2 between reuses",
                       "timing": "CUDA events around CUDA-graph replays, max over ranks",
                       "parallelism": f"replicas x{world}" if world > 1 else "single GPU"},
            "clocks": dict(clocks, window="sampled from 1.5 s before the timed region (same load) to its end"),
            "gpu_launches": n_launch,
            "roofline": {"bound": "hbm", "achieved": per_gpu, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": per_gpu / peaks["hbm_gbs"], "traffic": DECODE_TRAFFIC_BYTES_PER_LAUNCH,
                         "kernel": "decode_stream_kernel", "peak_source": peaks["_source"],
                         "us_per_launch": seconds / n_launch * 1e6,
                         "algorithmic_bytes_per_launch": step_bytes / launches_per_step},
        })

        # per-shape decode numbers (same rotation, one shape at a time)
        if "decode" in sections and rank == 0:
            per = {}
            for name in names:
                for M in DECODE_MS:
                    gs = []
                    for c in range(copies):
                        g = torch.cuda.CUDAGraph()
                        with torch.cuda.graph(g, stream=stream):
                            dmr.dmr_lowbit_linear(X[(name, M)], layers[c][name], OUT_BF16, Y=Y[(name, M)], workspace=ws)
                        gs.append(g)
                    reps = 40 * copies
                    sec = time_graph_replays(gs, reps, copies, torch)
                    b = layers[0][name].weight_bytes()
                    per[f"{name}_M{M}"] = {"us": sec / reps * 1e6, "gbs": b * reps / sec / 1e9,
                                          "frac_hbm": b * reps / sec / 1e9 / peaks["hbm_gbs"]}
            result["decode_per_shape"] = per

        # end-to-end: host activations in, host outputs back, through the host-buffer entry point
        if "e2e" in sections:
            Xh = {k: v.cpu().pin_memory() for k, v in X.items()}
            Yh = {k: torch.empty_like(v, device="cpu").pin_memory() for k, v in Y.items()}
            L = dmr.lib()
            staging = torch.empty(L.dmr_host_staging_bytes(16, 22016, 11008, OUT_BF16), dtype=torch.uint8, device=dev)

            def e2e_step(s):
                for mi, M in enumerate(DECODE_MS):
                    layer = layers[(s * len(DECODE_MS) + mi) % copies]
                    for name in names:
                        dmr.dmr_lowbit_linear_host(Xh[(name, M)], layer[name], Yh[(name, M)], OUT_BF16,
                                                   staging=staging, workspace=ws, stream=stream)
                stream.synchronize()  # the step's result is read on the host

            for s in range(3):
                e2e_step(s)
            sharding.barrier()
            e_steps = max(3, min(args.steps, 50))
            t0 = time.perf_counter()
            for s in range(e_steps):
                e2e_step(s)
            e_sec = time.perf_counter() - t0
            e_max = sharding.max_over_ranks(e_sec, dev)
            h2d = sum(v.numel() * 2 for v in Xh.values())
            d2h = sum(v.numel() * 2 for v in Yh.values())
            result["e2e"] = {"value": sharding.sum_over_ranks(step_bytes * e_steps, dev) / e_max / 1e9, "unit": "GB/s",
                             "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e_steps,
                             "note": "weights resident on the device; activations copied in and outputs copied "
                                     "back every call through dmr_lowbit_linear_host"}

        extra = run_extra_sections(sections, rank, dev, torch, dmr, inputs, fmt, peaks, copies, stream)
        result.update(extra)

    if rank == 0:
        if "cpu" in sections and world >= 1:
            v, cores, sample = oracle_cpu_baseline()
            result["cpu_baseline"] = {"value": v, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample}
        print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


def run_extra_sections(sections, rank, dev, torch, dmr, inputs, fmt, peaks, copies, stream):
    """Prefill, routed, dense and quantize numbers (rank 0 only; not part of the timed headline)."""
    from paper_2602_02711_b200 import OUT_BF16
    out = {}
    if rank != 0:
        return out

    def randw(N, K, seed):
        g = torch.Generator(device=dev)
        g.manual_seed(seed)
        return (torch.randn((N, K), generator=g, device=dev, dtype=torch.float32) * inputs.WEIGHT_SIGMA).to(torch.bfloat16)

    def randx(M, K, seed):
        g = torch.Generator(device=dev)
        g.manual_seed(seed)
        return torch.randn((M, K), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)

    def timeit(fn, reps, warm=3):
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e-3 / reps

    if "prefill" in sections:
        pre = {}
        for name, (N, K) in inputs.LAYER_7B.items():
            W = randw(N, K, 5)
            q = dmr.dmr_quantize(W, fmt)
            del W
            for M in (512, 2048, 8192):
                X = randx(M, K, M)
                Y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
                ws = dmr.new_workspace(0, M, N, K, fmt, dev)
                t = timeit(lambda: dmr.dmr_lowbit_linear(X, q, OUT_BF16, Y=Y, workspace=ws), reps=5, warm=2)
                tf = 2.0 * M * N * K / t / 1e12
                pre[f"{name}_M{M}"] = {"us": t * 1e6, "tflops": tf, "frac_bf16_burst": tf / peaks["bf16_tflops"],
                                       "frac_bf16_sustained": tf / peaks["bf16_tflops_sustained"]}
                del X, Y
            del q
        out["prefill"] = pre
        # all four linears at M = 8192 as one figure for the tensor-core roofline
        fl = sum(2.0 * 8192 * N * K for N, K in inputs.LAYER_7B.values())
        tt = sum(pre[f"{name}_M8192"]["us"] for name in inputs.LAYER_7B) * 1e-6
        out["roofline_prefill"] = {"bound": "tensor", "achieved": fl / tt / 1e12, "peak": peaks["bf16_tflops"],
                                   "unit": "TFLOP/s", "frac": fl / tt / 1e12 / peaks["bf16_tflops"], "traffic": None,
                                   "kernel": "prefill_kernel", "peak_source": peaks["_source"] + " (burst)",
                                   "workload": "7B-class layer, four linears, M=8192, INT4 g=128, bf16 out"}

    if "routed" in sections:
        M = 64
        tot_t, tot_b, per = 0.0, 0.0, {}
        for name, (N, K) in inputs.LAYER_14B.items():
            # rotate over copies so that neither weight set is served from L2
            nc = 3
            Ws = [randw(N, K, 31 + c) for c in range(nc)]
            qs = [dmr.dmr_quantize(w, fmt) for w in Ws]
            X = randx(M, K, 7)
            mask = torch.from_numpy(inputs.precision_mask(M, 0.3, seed=0)).to(dev)
            Y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
            ws = dmr.new_workspace(2, M, N, K, fmt, dev)
            # one CUDA graph per weight copy (a routed call is several launches: partition, gathers, the two
            # halves), replayed in rotation, so that the figure is device time and not Python launch overhead
            for c in range(nc):
                dmr.dmr_routed_linear(X, mask, Ws[c], qs[c], OUT_BF16, Y=Y, workspace=ws)
            torch.cuda.synchronize()
            graphs = []
            for c in range(nc):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    dmr.dmr_routed_linear(X, mask, Ws[c], qs[c], OUT_BF16, Y=Y, workspace=ws)
                graphs.append(g)
            state = {"i": 0}

            def call():
                state["i"] += 1
                graphs[state["i"] % nc].replay()

            t = timeit(call, reps=30, warm=3)
            b = N * K * 2 + qs[0].weight_bytes()
            per[name] = {"us": t * 1e6, "gbs": b / t / 1e9, "frac_hbm": b / t / 1e9 / peaks["hbm_gbs"]}
            tot_t += t
            tot_b += b
            del Ws, qs
        out["routed"] = {"layer_us": tot_t * 1e6, "gbs": tot_b / tot_t / 1e9, "frac_hbm": tot_b / tot_t / 1e9 / peaks["hbm_gbs"],
                         "workload": "14B-class layer, 7 linears, M=64, mask~Bernoulli(0.3)", "per_linear": per}

    if "dense" in sections:
        den = {}
        for name, (N, K) in inputs.LAYER_7B.items():
            Ws = [randw(N, K, 41 + c) for c in range(3)]
            for M in (1, 16):
                X = randx(M, K, 3)
                Y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
                ws = dmr.new_workspace(1, M, N, K, fmt, dev)
                state = {"i": 0}

                def call():
                    state["i"] += 1
                    dmr.dmr_dense_linear(X, Ws[state["i"] % 3], OUT_BF16, Y=Y, workspace=ws)

                t = timeit(call, reps=30)
                den[f"{name}_M{M}"] = {"us": t * 1e6, "gbs": N * K * 2 / t / 1e9, "frac_hbm": N * K * 2 / t / 1e9 / peaks["hbm_gbs"]}
            del Ws
        out["dense_decode"] = den

    if "layer_cost" in sections:
        # Per-token decode cost of one 7B-class layer at bf16 (T_high) and at INT4 g=128 (T_low): the four
        # linears chained in one CUDA graph, weights rotated over copies so that they come from HBM.  The
        # latency-based cost of the paper (Sec. 4.3, cost C = T_router N_steps + T_high N_high + T_low N_low)
        # then gives the relative cost of a routed run at high-precision budget rho, router cost aside:
        # C(rho) / C(all bf16) = rho + (1 - rho) T_low / T_high.
        lc = {}
        ncopy = 3
        Ws = [{n: randw(N, K, 71 + 7 * c + i) for i, (n, (N, K)) in enumerate(inputs.LAYER_7B.items())} for c in range(ncopy)]
        Qs = [{n: dmr.dmr_quantize(w, fmt) for n, w in layer.items()} for layer in Ws]
        for M in (1, 16):
            Xs = {n: randx(M, K, 3) for n, (N, K) in inputs.LAYER_7B.items()}
            Ys = {n: torch.empty((M, N), dtype=torch.bfloat16, device=dev) for n, (N, K) in inputs.LAYER_7B.items()}
            wsd = dmr.new_workspace(1, M, 22016, 11008, fmt, dev)
            wsl = dmr.new_workspace(0, M, 22016, 11008, fmt, dev)
            times = {}
            for kind in ("bf16", "int4"):
                graphs = []
                for c in range(ncopy):
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=stream):
                        for n in inputs.LAYER_7B:
                            if kind == "bf16":
                                dmr.dmr_dense_linear(Xs[n], Ws[c][n], OUT_BF16, Y=Ys[n], workspace=wsd)
                            else:
                                dmr.dmr_lowbit_linear(Xs[n], Qs[c][n], OUT_BF16, Y=Ys[n], workspace=wsl)
                    graphs.append(g)
                state = {"i": 0}

                def call():
                    state["i"] += 1
                    graphs[state["i"] % ncopy].replay()

                times[kind] = timeit(call, reps=60)
            ratio = times["int4"] / times["bf16"]
            lc[f"M{M}"] = {"t_high_us_per_layer": times["bf16"] * 1e6, "t_low_us_per_layer": times["int4"] * 1e6,
                           "t_high_over_t_low": 1.0 / ratio,
                           "relative_cost_at_budget": {f"rho={r}": r + (1 - r) * ratio for r in (0.2, 0.4, 0.7)}}
        del Ws, Qs
        out["layer_cost_7b"] = lc

    if "crossover" in sections:
        # 32B-class gate and down linears, INT4 g=64 and INT8 per-channel, M = 1 .. 256, 1 % outlier channels x20:
        # where the library's dispatch (streaming kernel up to 32 rows, tensor-core kernels above) stands.
        # The streaming family at larger M is timed by separate runs with DMR_DECODE_MAX_M=256.
        from paper_2602_02711_b200 import QFormat as QF
        cx = {"dispatch": f"DMR_DECODE_MAX_M={os.environ.get('DMR_DECODE_MAX_M', '32')}"}
        for lname, (N, K) in inputs.LAYER_32B.items():
            for fname, f5 in (("int4_g64", QF(4, 64)), ("int8_pc", QF(8, 0))):
                Ws = [randw(N, K, 61 + c) for c in range(2)]
                qs = [dmr.dmr_quantize(w, f5) for w in Ws]
                del Ws
                for M in (1, 2, 4, 8, 16, 32, 64, 128, 256):
                    X = torch.from_numpy(inputs.activations(M, K, seed=5, index=M, outlier_frac=0.01).view(np.int16)).view(torch.bfloat16).to(dev)
                    Y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
                    ws = dmr.new_workspace(0, M, N, K, f5, dev)
                    state = {"i": 0}

                    def call():
                        state["i"] += 1
                        dmr.dmr_lowbit_linear(X, qs[state["i"] % 2], OUT_BF16, Y=Y, workspace=ws)

                    t = timeit(call, reps=20)
                    b = qs[0].weight_bytes()
                    cx[f"{lname}_{fname}_M{M}"] = {"us": t * 1e6, "gbs": b / t / 1e9, "tflops": 2.0 * M * N * K / t / 1e12}
                del qs
        out["crossover_32b"] = cx

    if "kl" in sections:
        # Step-wise KL divergence: two [T][V] bf16 logit tensors (1.24 GB, far beyond the L2) read once.
        T, V = 2048, 151936
        g = torch.Generator(device=dev)
        g.manual_seed(97)
        hi = (torch.randn((T, V), generator=g, device=dev, dtype=torch.float32) * 2.5).to(torch.bfloat16)
        lo = (hi.float() + torch.randn((T, V), generator=g, device=dev, dtype=torch.float32) * 0.1).to(torch.bfloat16)
        offs = torch.from_numpy(inputs.step_offsets(T, 12, seed=3)).to(dev)
        t = timeit(lambda: dmr.dmr_stepwise_kl(hi, lo, offs), reps=10, warm=3)
        b = 2.0 * T * V * 2
        out["stepwise_kl"] = {"us": t * 1e6, "gbs": b / t / 1e9, "frac_hbm": b / t / 1e9 / peaks["hbm_gbs"],
                              "tokens_per_s": T / t,
                              "workload": f"{T} action tokens x {V} logits, bf16, two models, {int(offs.numel()) - 1} steps"}
        del hi, lo

    if "quantize" in sections:
        qz = {}
        for name, (N, K) in inputs.LAYER_7B.items():
            W = randw(N, K, 51)
            t = timeit(lambda: dmr.dmr_quantize(W, fmt, check=False), reps=5, warm=2)
            qz[name] = {"us": t * 1e6, "gweights_per_s": N * K / t / 1e9}
            del W
        out["quantize"] = qz
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sections", default="", help="comma list: decode,e2e,cpu,prefill,routed,dense,quantize,crossover,layer_cost,kl")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
