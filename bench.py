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
# dram__bytes_read.sum + dram__bytes_write.sum per launch of decode_w4_kernel, mean of the four 7B-class
# linears at M = 1 (ncu capture summarised in profiles/decode_w4_kernel_int4_g128_7b_M1.txt)
DECODE_TRAFFIC_BYTES_PER_LAUNCH = 26.54e6
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def emit_section(name, obj):
    """Full per-section results go out as a line of their own (and are appended to the file DMR_BENCH_SECTIONS names, if
    set); the final line of the run only carries short summaries."""
    line = json.dumps({"section": name, "results": obj})
    print(line, flush=True)
    path = os.environ.get("DMR_BENCH_SECTIONS")
    if path:
        try:
            with open(path, "a") as f:
                f.write(line + "\n")
        except OSError:
            pass


def copies_beyond_l2(nbytes, l2_bytes, least=3):
    """How many independent copies of a tensor set to rotate over so that more than 3 x L2 lies between two uses."""
    return max(least, int(np.ceil(3.0 * l2_bytes / max(nbytes, 1))) + 1)


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
    sections = set(args.sections.split(",")) if args.sections else {"decode", "e2e", "cpu", "prefill", "routed", "dense", "quantize", "layer_cost", "w3", "router", "kl", "crossover"}

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
                         "kernel": "decode_w4_kernel", "peak_source": peaks["_source"],
                         "us_per_launch": seconds / n_launch * 1e6,
                         "algorithmic_bytes_per_launch": step_bytes / launches_per_step},
        })

        # per-shape decode numbers: each shape alone, over enough copies of its own that 3 x L2 lies between two uses
        # of a copy; one CUDA graph holds one round over the copies (a chain of launches, as in a decoder)
        if "decode" in sections and rank == 0:
            per = {}
            for i, name in enumerate(names):
                N, K = shapes[name]
                b = layers[0][name].weight_bytes()
                nc = copies_beyond_l2(b, l2_bytes)
                qs = [layers[c][name] for c in range(min(nc, copies))]
                for c in range(len(qs), nc):
                    g = torch.Generator(device=dev)
                    g.manual_seed(5000 + 100 * i + c)
                    W = (torch.randn((N, K), generator=g, device=dev, dtype=torch.float32) * inputs.WEIGHT_SIGMA).to(torch.bfloat16)
                    qs.append(dmr.dmr_quantize(W, fmt))
                    del W
                for M in DECODE_MS:
                    for c in range(nc):
                        dmr.dmr_lowbit_linear(X[(name, M)], qs[c], OUT_BF16, Y=Y[(name, M)], workspace=ws)
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=stream):
                        for c in range(nc):
                            dmr.dmr_lowbit_linear(X[(name, M)], qs[c], OUT_BF16, Y=Y[(name, M)], workspace=ws)
                    rounds = max(3, 160 // nc)
                    sec = time_graph_replays([g], rounds, 2, torch) / (rounds * nc)
                    per[f"{name}_M{M}"] = {"us": sec * 1e6, "gbs": b / sec / 1e9, "frac_hbm": b / sec / 1e9 / peaks["hbm_gbs"], "copies": nc}
                del qs
            emit_section("decode_per_shape", per)
            result["decode_frac_hbm"] = {k: round(v["frac_hbm"], 3) for k, v in per.items()}

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

        extra = run_extra_sections(sections, rank, dev, torch, dmr, inputs, fmt, peaks, l2_bytes, stream)
        result.update(extra)

    if rank == 0:
        if "cpu" in sections and world >= 1:
            v, cores, sample = oracle_cpu_baseline()
            result["cpu_baseline"] = {"value": v, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample}
        # the run's records keep the end of the output: a short summary of every section goes last
        summary = {}
        if "roofline_prefill" in result:
            rp = result["roofline_prefill"]
            summary["prefill_frac_bf16_burst_by_M"] = rp["frac_by_M"]
            summary["prefill_M8192"] = {"tflops": round(rp["achieved"], 1), "us": round(rp["us"], 1)}
        if "routed" in result:
            summary["routed_14b_M64"] = {"layer_us": round(result["routed"]["layer_us"], 1), "frac_hbm": round(result["routed"]["frac_hbm"], 3)}
        if "w3_vs_w4_decode_7b" in result:
            w = result.pop("w3_vs_w4_decode_7b")
            summary["t_w4_over_t_w3"] = {k: v["ratio"] for k, v in w.items()}
            if "w3_prefill_M2048_tflops" in result:
                summary["w3_prefill_M2048_tflops"] = result.pop("w3_prefill_M2048_tflops")
        if "router_forward" in result:
            summary["router_forward_ms"] = {k: v["ms"] for k, v in result.pop("router_forward").items()}
        for key in ("crossover_32b", "dense_decode_frac_hbm", "layer_cost_7b", "stepwise_kl"):
            if key in result:
                summary[key] = result.pop(key)
        result["summary"] = summary
        print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


def run_extra_sections(sections, rank, dev, torch, dmr, inputs, fmt, peaks, l2_bytes, stream):
    """Prefill, routed, dense, crossover, cost-model, KL and quantize numbers (rank 0 only; not part of the timed
    headline).  Every section prints its full table as a line of its own and returns a short summary."""
    from paper_2602_02711_b200 import OUT_BF16, QFormat as QF, cost
    from paper_2602_02711_b200.binding import OP_LOWBIT, OP_DENSE
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

    def time_rotating(call, ncopy, reps):
        """Seconds per call of call(c), c = 0 .. ncopy - 1 visited in rotation: one CUDA graph holds one round over
        all copies, so the figure is device time and every call meets weights that left the L2 long ago."""
        for c in range(ncopy):
            call(c)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for c in range(ncopy):
                call(c)
        rounds = max(2, int(np.ceil(reps / ncopy)))
        return timeit(g.replay, reps=rounds, warm=2) / ncopy

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
                t = timeit(lambda: dmr.dmr_lowbit_linear(X, q, OUT_BF16, Y=Y, workspace=ws), reps=20, warm=3)
                tf = 2.0 * M * N * K / t / 1e12
                pre[f"{name}_M{M}"] = {"us": t * 1e6, "tflops": tf, "frac_bf16_burst": tf / peaks["bf16_tflops"],
                                       "frac_bf16_sustained": tf / peaks["bf16_tflops_sustained"],
                                       "kernel": dmr.dmr_describe_dispatch(OP_LOWBIT, M, N, K, fmt)}
                del X, Y
            del q
        emit_section("prefill", pre)
        per_m = {}
        for M in (512, 2048, 8192):
            fl = sum(2.0 * M * N * K for N, K in inputs.LAYER_7B.values())
            tt = sum(pre[f"{name}_M{M}"]["us"] for name in inputs.LAYER_7B) * 1e-6
            per_m[M] = {"tflops": fl / tt / 1e12, "us": tt * 1e6}
        # all four linears at M = 8192 as one figure for the tensor-core roofline
        out["roofline_prefill"] = {"bound": "tensor", "achieved": per_m[8192]["tflops"], "peak": peaks["bf16_tflops"],
                                   "unit": "TFLOP/s", "frac": per_m[8192]["tflops"] / peaks["bf16_tflops"], "traffic": None,
                                   "us": per_m[8192]["us"], "kernel": "prefill_kernel", "peak_source": peaks["_source"] + " (burst)",
                                   "frac_by_M": {str(M): round(v["tflops"] / peaks["bf16_tflops"], 3) for M, v in per_m.items()},
                                   "workload": "7B-class layer, four linears, INT4 g=128, bf16 out; headline figure at M=8192"}

    if "routed" in sections:
        M = 64
        tot_t, tot_b, per = 0.0, 0.0, {}
        for name, (N, K) in inputs.LAYER_14B.items():
            # enough copies of both weight sets that neither is served from the L2
            nc = copies_beyond_l2(N * K * 2.5234, l2_bytes)
            Ws = [randw(N, K, 31 + c) for c in range(nc)]
            qs = [dmr.dmr_quantize(w, fmt) for w in Ws]
            X = randx(M, K, 7)
            mask = torch.from_numpy(inputs.precision_mask(M, 0.3, seed=0)).to(dev)
            Y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
            ws = dmr.new_workspace(2, M, N, K, fmt, dev)
            t = time_rotating(lambda c: dmr.dmr_routed_linear(X, mask, Ws[c], qs[c], OUT_BF16, Y=Y, workspace=ws), nc, reps=30)
            b = N * K * 2 + qs[0].weight_bytes()
            per[name] = {"us": t * 1e6, "gbs": b / t / 1e9, "frac_hbm": b / t / 1e9 / peaks["hbm_gbs"], "copies": nc}
            tot_t += t
            tot_b += b
            del Ws, qs
        emit_section("routed", per)
        out["routed"] = {"layer_us": tot_t * 1e6, "gbs": tot_b / tot_t / 1e9, "frac_hbm": tot_b / tot_t / 1e9 / peaks["hbm_gbs"],
                         "workload": "14B-class layer, 7 linears, M=64, mask~Bernoulli(0.3)",
                         "us": {k: round(v["us"], 1) for k, v in per.items()}}

    if "dense" in sections:
        den = {}
        for name, (N, K) in inputs.LAYER_7B.items():
            nc = copies_beyond_l2(N * K * 2, l2_bytes)
            Ws = [randw(N, K, 41 + c) for c in range(nc)]
            for M in (1, 16):
                X = randx(M, K, 3)
                Y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
                ws = dmr.new_workspace(1, M, N, K, fmt, dev)
                t = time_rotating(lambda c: dmr.dmr_dense_linear(X, Ws[c], OUT_BF16, Y=Y, workspace=ws), nc, reps=40)
                den[f"{name}_M{M}"] = {"us": t * 1e6, "gbs": N * K * 2 / t / 1e9, "frac_hbm": N * K * 2 / t / 1e9 / peaks["hbm_gbs"],
                                       "copies": nc}
            del Ws
        emit_section("dense_decode", den)
        out["dense_decode_frac_hbm"] = {k: round(v["frac_hbm"], 3) for k, v in den.items()}

    if "layer_cost" in sections:
        # Per-token decode cost of one 7B-class layer at bf16 (T_high) and at INT4 g=128 (T_low): the four
        # linears chained in one CUDA graph, weights rotated over copies so that they come from HBM.  The
        # latency-based cost of the paper (Sec. 4.3, C = T_router N_steps + T_high N_high + T_low N_low) then
        # gives the relative cost of a routed run at high-precision budget rho; the router's own time is left
        # out (no router is built here), which the output says.
        lc = {}
        layer_bf16 = sum(N * K * 2 for N, K in inputs.LAYER_7B.values())
        ncopy = copies_beyond_l2(layer_bf16, l2_bytes)
        Ws = [{n: randw(N, K, 71 + 7 * c + i) for i, (n, (N, K)) in enumerate(inputs.LAYER_7B.items())} for c in range(ncopy)]
        Qs = [{n: dmr.dmr_quantize(w, fmt) for n, w in layer.items()} for layer in Ws]
        for M in (1, 16):
            Xs = {n: randx(M, K, 3) for n, (N, K) in inputs.LAYER_7B.items()}
            Ys = {n: torch.empty((M, N), dtype=torch.bfloat16, device=dev) for n, (N, K) in inputs.LAYER_7B.items()}
            wsd = dmr.new_workspace(1, M, 22016, 11008, fmt, dev)
            wsl = dmr.new_workspace(0, M, 22016, 11008, fmt, dev)

            def layer_call(kind):
                def call(c):
                    for n in inputs.LAYER_7B:
                        if kind == "bf16":
                            dmr.dmr_dense_linear(Xs[n], Ws[c][n], OUT_BF16, Y=Ys[n], workspace=wsd)
                        else:
                            dmr.dmr_lowbit_linear(Xs[n], Qs[c][n], OUT_BF16, Y=Ys[n], workspace=wsl)
                return call

            t_high = time_rotating(layer_call("bf16"), ncopy, reps=60)
            t_low = time_rotating(layer_call("int4"), ncopy, reps=60)
            lc[f"M{M}"] = {"t_high_us_per_layer": t_high * 1e6, "t_low_us_per_layer": t_low * 1e6,
                           "t_high_over_t_low": t_high / t_low, "t_router": "excluded (no router in this library)",
                           "relative_cost_at_budget": {f"rho={r}": cost.relative_cost_at_budget(r, t_high, t_low) for r in (0.2, 0.4, 0.7)}}
        del Ws, Qs
        emit_section("layer_cost_7b", lc)
        out["layer_cost_7b"] = {k: {"t_high_us": round(v["t_high_us_per_layer"], 1), "t_low_us": round(v["t_low_us_per_layer"], 1),
                                    "ratio": round(v["t_high_over_t_low"], 2)} for k, v in lc.items()}

    if "w3" in sections:
        # The 3-bit variant (W3A16 g=128, Sec. 5 / App. "Quantization Detail") against the 4-bit one on the same 7B-class
        # layer: per-token decode time of the four linears chained in one CUDA graph, weights rotated over copies larger
        # than the L2.  The paper has no 3-bit kernel and projects T_W3 = T_W4 / 1.15 (App. "Latency calibration");
        # this is the measured ratio for this library's kernels.
        w3 = {}
        f3, f4 = QF(3, 128), QF(4, 128)
        layer_w4 = sum(N * K // 2 for N, K in inputs.LAYER_7B.values())
        layer_w3 = sum(N * K * 3 // 8 for N, K in inputs.LAYER_7B.values())
        ncopy = copies_beyond_l2(layer_w3, l2_bytes)
        Q3s, Q4s = [], []
        for c in range(ncopy):
            l3, l4 = {}, {}
            for i, (n, (N, K)) in enumerate(inputs.LAYER_7B.items()):
                W = randw(N, K, 171 + 7 * c + i)
                l3[n] = dmr.dmr_quantize(W, f3)
                l4[n] = dmr.dmr_quantize(W, f4)
                del W
            Q3s.append(l3)
            Q4s.append(l4)
        for M in (1, 8, 16):
            Xs = {n: randx(M, K, 3) for n, (N, K) in inputs.LAYER_7B.items()}
            Ys = {n: torch.empty((M, N), dtype=torch.bfloat16, device=dev) for n, (N, K) in inputs.LAYER_7B.items()}
            ws3 = dmr.new_workspace(0, M, 22016, 11008, f3, dev)
            ws4 = dmr.new_workspace(0, M, 22016, 11008, f4, dev)

            def layer_call(Qs, ws):
                def call(c):
                    for n in inputs.LAYER_7B:
                        dmr.dmr_lowbit_linear(Xs[n], Qs[c][n], OUT_BF16, Y=Ys[n], workspace=ws)
                return call

            t4 = time_rotating(layer_call(Q4s, ws4), ncopy, reps=60)
            t3 = time_rotating(layer_call(Q3s, ws3), ncopy, reps=60)
            w3[f"M{M}"] = {"t_w4_us_per_layer": t4 * 1e6, "t_w3_us_per_layer": t3 * 1e6, "t_w4_over_t_w3": t4 / t3,
                           "w4_weight_gbs": layer_w4 / t4 / 1e9, "w3_weight_gbs": layer_w3 / t3 / 1e9,
                           "w3_frac_hbm": layer_w3 / t3 / 1e9 / peaks["hbm_gbs"],
                           "paper_projection_t_w4_over_t_w3": 1.15}
        # prefill-sized batches: the same tensor-core kernel with the 3-bit unpack (codes read from global memory by the
        # unpack threads) against the 4-bit one, four linears, M = 2048
        t3p = t4p = flops = 0.0
        for n, (N, K) in inputs.LAYER_7B.items():
            Xp = randx(2048, K, 9)
            Yp = torch.empty((2048, N), dtype=torch.bfloat16, device=dev)
            for fq, Qs in ((f3, Q3s), (f4, Q4s)):
                wsp = dmr.new_workspace(0, 2048, N, K, fq, dev)
                t = timeit(lambda: dmr.dmr_lowbit_linear(Xp, Qs[0][n], OUT_BF16, Y=Yp, workspace=wsp), reps=10, warm=3)
                if fq is f3:
                    t3p += t
                else:
                    t4p += t
            flops += 2.0 * 2048 * N * K
        w3["prefill_M2048"] = {"t_w4_us": t4p * 1e6, "t_w3_us": t3p * 1e6, "w4_tflops": flops / t4p / 1e12, "w3_tflops": flops / t3p / 1e12,
                               "w3_frac_bf16_burst": flops / t3p / 1e12 / peaks["bf16_tflops"]}
        del Q3s, Q4s
        emit_section("w3_vs_w4_decode_7b", w3)
        out["w3_vs_w4_decode_7b"] = {k: {"t_w4_us": round(v["t_w4_us_per_layer"], 1), "t_w3_us": round(v["t_w3_us_per_layer"], 1),
                                         "ratio": round(v["t_w4_over_t_w3"], 3)} for k, v in w3.items() if k.startswith("M")}
        out["w3_prefill_M2048_tflops"] = round(w3["prefill_M2048"]["w3_tflops"], 1)

    if "router" in sections:
        # The step-level router's forward pass (Sec. 4.1) at the default depth of 8 layers on sentence-encoder-sized
        # embeddings (width 384, 6 heads, feed-forward 1536, 2 precision choices; the paper prints none of these sizes),
        # random-init weights as in the paper's own timing (App. "Per-call router coefficient"), sequences of 1 .. 32
        # entries.  One call decides B concurrent agent steps.  fp32 CUDA-core arithmetic: the roofline is the fp32
        # FMA peak, 148 SMs x 128 lanes x 2 flop x 1.965 GHz = 74.5 TFLOP/s.
        from paper_2602_02711_b200 import RouterCfg
        kw = dict(d=384, heads=6, ffn=1536, layers=8, l_max=32, classes=2)
        cfg = RouterCfg(**kw)
        params = dmr.pack_router_params(inputs.router_params(**kw, seed=0), cfg, dev)
        L = 32
        rt = {}
        for B in (1, 64):
            Z = torch.from_numpy(inputs.router_embeddings(B, L, kw["d"], seed=0)).to(dev)
            n = torch.from_numpy(inputs.router_lengths(B, L, seed=0)).to(dev)
            wsr = torch.empty(dmr.lib().dmr_router_workspace_bytes(cfg, B, L), dtype=torch.uint8, device=dev)
            g = torch.cuda.CUDAGraph()
            dmr.dmr_router_forward(params, cfg, Z, n, 1, workspace=wsr)
            torch.cuda.synchronize()
            with torch.cuda.graph(g, stream=stream):
                dmr.dmr_router_forward(params, cfg, Z, n, 1, workspace=wsr)
            t = timeit(g.replay, reps=20, warm=3)
            T = B * L
            flops = 2.0 * T * kw["layers"] * (4 * kw["d"] * kw["d"] + 2 * kw["d"] * kw["ffn"])
            rt[f"B{B}"] = {"ms_per_call": t * 1e3, "tokens": T, "tflops_fp32": flops / t / 1e12,
                           "frac_fp32_fma_peak": flops / t / 1e12 / 74.5, "launches_per_call": 2 + 7 * kw["layers"]}
        rt["config"] = dict(kw, note="sizes are this library's reading; the paper prints none")
        rt["paper_t_router_ms_per_call"] = "17.13-29.15 (A6000, router plus frozen sentence encoder)"
        emit_section("router_forward", rt)
        out["router_forward"] = {k: {"ms": round(v["ms_per_call"], 3), "frac_fp32": round(v["frac_fp32_fma_peak"], 3)} for k, v in rt.items() if k.startswith("B")}

    if "crossover" in sections:
        # 32B-class gate and down linears, INT4 g=64 and INT8 per-channel, M = 1 .. 256, 1 % outlier channels x20,
        # with the library's default dispatch (decode kernels up to 32 rows, tensor-core kernels above): where
        # the bandwidth-bound family hands over to the compute-bound one.  Two weight copies exceed 3 x L2 for INT8
        # (141 MB each) and come close for INT4 g64 (77 MB each; three copies are used).
        cx = {"dispatch": f"DMR_DECODE_MAX_M={os.environ.get('DMR_DECODE_MAX_M', '32')}"}
        summary = {}
        for lname, (N, K) in inputs.LAYER_32B.items():
            for fname, f5 in (("int4_g64", QF(4, 64)), ("int8_pc", QF(8, 0))):
                wb = N * K * f5.bits // 8
                nc = copies_beyond_l2(wb, l2_bytes, least=2)
                qs = []
                for c in range(nc):
                    w = randw(N, K, 61 + c)
                    qs.append(dmr.dmr_quantize(w, f5))
                    del w
                best = None
                for M in (1, 2, 4, 8, 16, 32, 64, 128, 256):
                    X = torch.from_numpy(inputs.activations(M, K, seed=5, index=M, outlier_frac=0.01).view(np.int16)).view(torch.bfloat16).to(dev)
                    Y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
                    ws = dmr.new_workspace(0, M, N, K, f5, dev)
                    t = time_rotating(lambda c: dmr.dmr_lowbit_linear(X, qs[c], OUT_BF16, Y=Y, workspace=ws), nc, reps=12)
                    b = qs[0].weight_bytes()
                    kern = dmr.dmr_describe_dispatch(OP_LOWBIT, M, N, K, f5)["kernel"]
                    cx[f"{lname}_{fname}_M{M}"] = {"us": t * 1e6, "gbs": b / t / 1e9, "tflops": 2.0 * M * N * K / t / 1e12, "kernel": kern}
                    if kern in ("decode_w4", "stream"):
                        best = M
                summary[f"{lname}_{fname}"] = {
                    "M1_frac_hbm": round(cx[f"{lname}_{fname}_M1"]["gbs"] / peaks["hbm_gbs"], 3),
                    "M16_frac_hbm": round(cx[f"{lname}_{fname}_M16"]["gbs"] / peaks["hbm_gbs"], 3),
                    "M256_tflops": round(cx[f"{lname}_{fname}_M256"]["tflops"], 1),
                    "last_M_on_decode_kernels": best}
                del qs
        emit_section("crossover_32b", cx)
        out["crossover_32b"] = summary

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
        kl = {"us": t * 1e6, "gbs": b / t / 1e9, "frac_hbm": b / t / 1e9 / peaks["hbm_gbs"], "tokens_per_s": T / t,
              "workload": f"{T} action tokens x {V} logits, bf16, two models, {int(offs.numel()) - 1} steps"}
        emit_section("stepwise_kl", kl)
        out["stepwise_kl"] = {"us": round(kl["us"], 1), "frac_hbm": round(kl["frac_hbm"], 3)}
        del hi, lo

    if "quantize" in sections:
        qz = {}
        for name, (N, K) in inputs.LAYER_7B.items():
            W = randw(N, K, 51)
            t = timeit(lambda: dmr.dmr_quantize(W, fmt, check=False), reps=5, warm=2)
            qz[name] = {"us": t * 1e6, "gweights_per_s": N * K / t / 1e9}
            del W
        emit_section("quantize", qz)
        out["quantize_us"] = {k: round(v["us"], 1) for k, v in qz.items()}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sections", default="", help="comma list: decode,e2e,cpu,prefill,routed,dense,quantize,crossover,layer_cost,w3,router,kl (default: all; none = headline only)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
