#!/usr/bin/env python
"""Benchmark of the LUT-linear hot path (input transformation -> table lookup -> accumulation) on B200.

One "step" is one pass of the whole hot path over one decoder layer's projections: for every matrix,
`lcd_smooth_quantize_act` on its input tokens followed by `lcd_lut_linear`.  The default workload is the
LLaMA-7B-shaped layer at M = 1 with 2-bit weights; the metric is microseconds per layer (lower is better)
with the matching HBM GB/s on index + codebook + activation bytes.  Weights rotate over several device copies
(> 256 MB in total) so that L2 cannot serve them.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

With --impl reference the CPU oracle is timed instead (a deliberately slow double-precision program).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from synth import gen  # noqa: E402

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum, bytes per launch) of the dominant kernel of a workload,
# from one ncu capture each, with the hash of the kernel source the capture was taken from: a kernel that has changed
# since reports traffic = null.  Keys: (kernel source, configuration, M).
NCU_TRAFFIC = {
    # one launch (input transformation + lookup) of the LLaMA-7B-shaped 2-bit layer at M = 1
    ("lut_smem.cu", 1, 1): {"sha256": "f14795184ea2befb46a489352d144b95f89ea0e2f26f8c36bad69d4a05436a55", "bytes_per_launch": 51871232 + 122368},
    # the seven launches of the LLaMA-13B-shaped layer at M = 2048: q captured (17.11 + 0.44 MB, taken four times for
    # q/k/v/o), gate captured (28.37 + 56.32 MB, twice for gate/up), down scaled from q by its 2.7 times longer rows
    # (same tiles, traffic in proportion to K)
    ("dense_tc.cu", 3, 2048): {"sha256": "c29890f9ab90dad858f8486d69f2bb16e902631e75ef856b650a66523b6d474b",
                               "bytes_per_launch": int(4 * 17.55e6 + 2 * 84.70e6 + 17.55e6 * 13824 / 5120)},
}
L2_BYTES = 126e6
ROTATE_BYTES = 300e6          # total size of the weight copies the timed loop rotates over


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", type=int, default=1, help="index of the workload configuration (default 1: LLaMA-7B-shaped layer, 2 bit, M = 1)")
    ap.add_argument("--M", type=int, default=None, help="token count (default: first M of the config)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-secondary", action="store_true", help="default workload only: skip the M = 2048 and other workloads of the line")
    ap.add_argument("--act-bits", type=int, default=4, choices=[4, 8],
                    help="activation levels: 4 bit (the benchmark configurations) or 8 bit (the paper's b = 8)")
    ap.add_argument("--aux", default=None, choices=["smoothing", "reclassify", "dbci"],
                    help="time an offline piece instead of the hot path: 'smoothing' = the Section 3.4 grid search, "
                         "'reclassify' = the Section 3.2 reclassification and centroid offsets, 'dbci' = the Section 3.1 "
                         "centroid initialisation")
    ap.add_argument("--two-call", action="store_true",
                    help="quantise and look up in separate calls instead of the fused one")
    ap.add_argument("--algo", default="auto", choices=["auto", "register", "bucket", "tensor", "shared"],
                    help="lookup kernel for M <= 16 (default: the library's choice)")
    return ap.parse_args()


def algorithmic_bytes(N, K, bits, M, act_bits=4):
    """index + codebook + activation-index bytes the method must read for one matrix (no padding, no output)."""
    return N * K * bits / 8 + N * (1 << bits) * 2 + M * (K * act_bits / 8 + 4)


def build_layers(cfg_id, M):
    cfg = gen.CONFIGS[cfg_id]
    layers = []
    for mi, (name, N, K) in enumerate(cfg["shapes"]):
        L = gen.make_layer(cfg_id, mi, N, K, cfg["bits"], M, C=cfg.get("C"), outlier_frac=cfg["frac"],
                           outlier_scale=cfg["scale"])
        layers.append((name, L))
    return cfg, layers


# ----------------------------------------------------------------------------------------------- oracle
def oracle_layer_pass(layers):
    from oracle import lcd_oracle as O
    outs = []
    for _, L in layers:
        q, s = O.smooth_quantize(L.x, L.inv_s)
        outs.append(O.lut_linear_dequant(L.idx, L.codebook, q, s))
    return outs


def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
        return int(n)
    except Exception:
        return 1


def oracle_sample(cfg_id, layers, M):
    """Bounded sample for the CPU legs: whole layer at small M; at large M the first matrix restricted to
    256 output rows and 64 tokens, scaled to the layer by multiply-accumulate count."""
    total_macs = sum(L.N * L.K * M for _, L in layers)
    if M * sum(L.N * L.K for _, L in layers) <= 4e9:
        return layers, 1.0, f"all {len(layers)} matrices of one layer, M={M}, dequant form"
    name, L = layers[0]
    rows, toks = min(256, L.N), min(64, M)
    import copy
    S = copy.copy(L)
    S.idx, S.codebook, S.x, S.N, S.M = L.idx[:rows], L.codebook[:rows], L.x[:toks], rows, toks
    scale = total_macs / (rows * L.K * toks)
    return [(name, S)], scale, f"{name}: {rows} output rows x {toks} tokens, scaled x{scale:.0f} by MAC count"


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = gen.CONFIGS[args.config]
    M = args.M or cfg["Ms"][0]
    _, layers = build_layers(args.config, M)
    sample, scale, desc = oracle_sample(args.config, layers, M)
    for _ in range(min(args.warmup, 1)):
        oracle_layer_pass(sample)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_layer_pass(sample)
    dt = (time.perf_counter() - t0) / args.steps * scale
    us = dt * 1e6
    cores = oracle_threads()
    line = {"impl": "reference", "metric": metric_name(M), "value": us, "unit": "us/layer", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(args.config, M, 1),
            "cpu_baseline": {"value": us, "unit": "us/layer", "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": us, "unit": "us/layer", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def metric_name(M):
    return "lut_linear_us_per_layer_m%d" % M


def workload_config(cfg_id, M, copies, act_bits=4):
    cfg = gen.CONFIGS[cfg_id]
    return {"workload": f"configuration {cfg_id} ({cfg['name']}): " +
                        ", ".join(f"{n} {N}x{K}" for n, N, K in cfg["shapes"]),
            "bits": cfg["bits"], "M": M, "act_bits": act_bits, "outliers": f"{cfg['frac'] * 100:g}% x{cfg['scale']:g}",
            "l2": f"weights rotate over {copies} device copies (> {int(L2_BYTES / 1e6)} MB L2)"}


# ----------------------------------------------------------------------------------------------- clocks
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in out.strip().splitlines():
            f = [v.strip() for v in ln.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------------------------- ranks
def max_over_ranks(ms, device):
    """The slowest rank's time (every rank runs its own replica of the layer; no data-path collective)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def per_layer_us(ms_step, world):
    """Whole-job metric for replicas: `world` replicas each finish one layer per step."""
    return ms_step * 1e3 / world


# ----------------------------------------------------------------------------------------------- ours
def run_ours(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    cfg = gen.CONFIGS[args.config]
    M = args.M or cfg["Ms"][0]
    line = measure_config(args, args.config, M, dev, world, local, primary=True)
    if rank == 0 and line is not None:
        if world == 1 and not args.no_secondary and args.config == 1 and args.M is None and args.act_bits == 4 \
                and args.algo == "auto" and not args.two_call:
            # the rest of the metric in the same line: the prefill half (M = 2048) and the other single-token workloads
            line["secondary"] = []
            for cid, m in ((3, 2048), (4, 1), (0, 1)):
                sec = measure_config(args, cid, m, dev, 1, local, primary=False)
                line["secondary"].append({k: sec[k] for k in ("metric", "value", "unit", "ms_per_step", "timing", "config",
                                                              "TFLOPs_equiv", "layer_GBps", "roofline", "parity",
                                                              "gpu_launches") if k in sec})
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def measure_config(args, cfg_id, M, dev, world, local, primary):
    """One workload: builds its layer, times the step (median over repeats of exactly --steps steps, at least 0.2 s in
    all), the dominant kernel and (primary only) the end-to-end path, compares the timed path's outputs with the
    oracle and returns the JSON line as a dict (None on ranks other than 0)."""
    import torch
    import torch.distributed as dist
    import paper_2506_12038_b200 as lcd

    rank = int(os.environ.get("RANK", "0"))
    cfg = gen.CONFIGS[cfg_id]
    bits = cfg["bits"]
    steps = args.steps if primary else max(10, min(args.steps, 40))
    _, layers = build_layers(cfg_id, M)            # every rank: its own replica of the layer (weak scaling)
    layer_bytes = sum(lcd.packed_weights_bytes(L.N, L.K, bits) for _, L in layers)
    copies = max(2, int(np.ceil(ROTATE_BYTES / layer_bytes)))
    if not primary:
        steps = max(steps, 2 * copies)       # whole rounds of the back-to-back graph, as in a long run

    mats = []
    for name, L in layers:
        blob = lcd.pack_weights(L.idx, L.codebook, bits, L.C)
        ws = [lcd.PackedWeights(blob, dev) for _ in range(copies)]
        x = torch.from_numpy(L.x).to(dev)
        inv_s = torch.from_numpy(L.inv_s).to(dev)
        K_pad = ws[0].K_pad
        a = (torch.empty((M, K_pad // 2), dtype=torch.uint8, device=dev) if args.act_bits == 4 else
             torch.empty((M, K_pad), dtype=torch.int8, device=dev))
        s = torch.empty((M,), dtype=torch.float32, device=dev)
        y = torch.empty((M, L.N), dtype=torch.float32, device=dev)
        wsb = lcd.lut_linear_workspace_bytes(ws[0], M)
        work = torch.zeros(max(wsb, 256), dtype=torch.uint8, device=dev)
        mats.append(dict(name=name, L=L, w=ws, x=x, inv_s=inv_s, a=a, s=s, y=y, work=work,
                         bytes=algorithmic_bytes(L.N, L.K, bits, M, args.act_bits), flop=2.0 * M * L.N * L.K))

    grouped = M <= 16 and len(mats) <= lcd.MAX_BATCH
    algo = {"auto": lcd.ALGO_AUTO, "register": lcd.ALGO_REGISTER_LUT, "bucket": lcd.ALGO_BUCKET_LUT,
            "tensor": lcd.ALGO_TC_LUT, "shared": lcd.ALGO_SHARED_BUCKET}[args.algo]
    # which lookup kernel the library runs for this launch shape (its own answer, not a guess made here)
    shared_bucket = grouped and lcd.resolve_batch_algo([(mt["w"][0], M) for mt in mats], algo) == lcd.ALGO_SHARED_BUCKET \
        and args.act_bits == 4
    lookup_kernel = "lut_smem_kernel" if shared_bucket else "lut_gemv_kernel"
    # every kernel that can give up on a bounded wait reports it here; a non-zero word voids the run
    status = torch.zeros((1,), dtype=torch.int32, device=dev)
    if grouped:
        # one launch quantises every matrix's tokens, one launch runs every matrix's lookup: the inputs are
        # independent, so the whole layer is a single grouped problem
        qbatch = lcd.ActBatch([(mt["x"], mt["inv_s"], mt["a"], mt["s"]) for mt in mats])
        lbatch = [lcd.LinearBatch([(mt["w"][c], mt["a"], mt["s"], mt["y"]) for mt in mats], algo=algo, status_word=status)
                  for c in range(copies)]
        single = [[lcd.LinearBatch([(mt["w"][c], mt["a"], mt["s"], mt["y"])], algo=algo, status_word=status)
                   for c in range(copies)] for mt in mats]

        # default: ONE launch per layer, the lookup kernel does the input transformation itself (4-bit levels, the
        # register or bucket kernel); --two-call, 8-bit levels and the tensor-memory kernel: quantise, then look up
        # (M = 1 only: with more tokens every CTA would repeat the transformation of all tokens, measured slower)
        fused = (not args.two_call) and args.act_bits == 4 and args.algo != "tensor" and M == 1
        if fused:
            fbatch = [lcd.FusedBatch([(mt["w"][c], mt["x"], mt["inv_s"], mt["y"]) for mt in mats], algo=algo,
                                     status_word=status) for c in range(copies)]
            qbatch.run()          # the per-matrix lookup-only timings below use the stored levels

        def step(c):
            if fused:
                fbatch[c].run()
            else:
                qbatch.run()
                lbatch[c].run()

        def lookup_only(mi, c):
            single[mi][c].run()
    else:
        # many tokens, 4-bit levels: the library's one-call form, which transforms the inputs of all matrices in one
        # launch straight into the tensor-core kernel's operand bytes and then runs that kernel per matrix;
        # --two-call, 8-bit levels and 17..32 tokens: per matrix quantise, (expand,) lookup
        fused = (not args.two_call) and args.act_bits == 4 and args.algo == "auto" and M > 32 and len(mats) <= lcd.MAX_BATCH
        if fused:
            fbatch = [lcd.FusedBatch([(mt["w"][c], mt["x"], mt["inv_s"], mt["y"]) for mt in mats], status_word=status)
                      for c in range(copies)]
            for mt in mats:       # the stored levels of the per-matrix timings and of the parity check
                lcd.smooth_quantize_act(mt["x"], mt["inv_s"], act_idx=mt["a"], act_scale=mt["s"])

        def step(c):
            if fused:
                fbatch[c].run()
                return
            for mt in mats:
                lcd.smooth_quantize_act(mt["x"], mt["inv_s"], act_idx=mt["a"], act_scale=mt["s"],
                                        act_bits=args.act_bits)
                lcd.lut_linear(mt["w"][c], mt["a"], mt["s"], y=mt["y"], workspace=mt["work"], status_word=status)

        def lookup_only(mi, c):
            mt = mats[mi]
            lcd.lut_linear(mt["w"][c], mt["a"], mt["s"], y=mt["y"], workspace=mt["work"], status_word=status)

    # kernels per step: grouped 1 (fused) or 2; many tokens 1 + one per matrix (fused) or quantise, expand, lookup per matrix
    launches_per_step = (1 if fused else 2) if grouped else (1 + len(mats) if fused else 3 * len(mats))
    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        for c in range(copies):
            step(c)
        torch.cuda.synchronize()
        # one CUDA graph per weight copy: the layer's launches back to back, no host gaps
        graphs = []
        for c in range(copies):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                step(c)
            graphs.append(g)
        # and one graph of `copies` consecutive steps (a model runs its layers back to back): the timed loop replays
        # it for every full round of copies and finishes the remainder with the single-step graphs
        round_graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(round_graph, stream=stream):
            for c in range(copies):
                step(c)
        for i in range(max(args.warmup, 3) if primary else 3):
            graphs[i % copies].replay()
        round_graph.replay()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        sampler = ClockSampler(local)
        sampler.start()
        # Every repeat times exactly `steps` steps between two events; repeats go on until at least 5 were taken and
        # 0.2 s were timed in all (a short --steps run would otherwise be a fraction of a millisecond and one clock
        # sample).  The reported step time is the median over the repeats, the minimum is given beside it.
        rep_ms = []
        torch.cuda.synchronize()
        while len(rep_ms) < 5 or (sum(rep_ms) < 200.0 and len(rep_ms) < 2000):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(steps // copies):
                round_graph.replay()
            for i in range(steps % copies):
                graphs[i].replay()
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1)
            if world > 1:
                ms = max_over_ranks(ms, dev)          # the same number of repeats on every rank: the maxima decide
            rep_ms.append(ms)
        ms_total = statistics.median(rep_ms)
        if world > 1:
            dist.barrier()

        # dominant kernel: the lookup+accumulate launches alone, back to back inside a graph, every launch on
        # another weight copy.  Grouped: one launch per layer; the per-matrix table times single-matrix launches.
        def time_graph(fn, n_launch):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                fn()
            g.replay()
            torch.cuda.synchronize()
            k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            n_rep = max(3, min(steps, 20))
            k0.record()
            for _ in range(n_rep):
                g.replay()
            k1.record()
            torch.cuda.synchronize()
            return k0.elapsed_time(k1) / (n_rep * n_launch)

        reps = 4
        per_matrix, sum_ms = [], 0.0
        for mi, mt in enumerate(mats):
            ms = time_graph(lambda: [lookup_only(mi, c) for _ in range(reps) for c in range(copies)], reps * copies)
            sum_ms += ms
            per_matrix.append({"matrix": mt["name"], "N": mt["L"].N, "K": mt["L"].K, "us": ms * 1e3,
                               "GBps": mt["bytes"] / ms / 1e6, "TFLOPs_equiv": mt["flop"] / ms / 1e9})
        kern_bytes = sum(mt["bytes"] for mt in mats)
        kern_flop = sum(mt["flop"] for mt in mats)
        if grouped and fused:
            kern_ms = time_graph(lambda: [fbatch[c].run() for _ in range(reps) for c in range(copies)], reps * copies)
            kern_name = lookup_kernel + ", one launch per layer: input transformation + lookup of all its matrices"
            # the launch reads x (fp16) and the smoothing factors instead of stored levels and scales
            kern_bytes += sum(M * mt["L"].K * 2 + mt["L"].K * 4 - M * (mt["L"].K / 2 + 4) for mt in mats)
        elif grouped:
            kern_ms = time_graph(lambda: [lbatch[c].run() for _ in range(reps) for c in range(copies)], reps * copies)
            kern_name = lookup_kernel + ", one grouped launch over the layer's matrices"
        else:
            kern_ms = sum_ms
            kern_name = "lcd_lut_linear launches of one layer (sum of bytes / sum of durations)"
        clocks = sampler.stop()

        # end to end through the host-buffer entry points: pinned host x -> device -> kernels -> pinned host y.
        # Grouped (M <= 16): one copy in, two launches, one copy out per layer; else per matrix.
        e2e_ms, h2d, d2h = None, 0, 0
        if not primary:
            pass
        elif grouped and args.act_bits == 4:
            hbatch = [lcd.HostBatch([(mt["w"][c], mt["inv_s"], M) for mt in mats], dev) for c in range(copies)]
            for hb in hbatch:
                for i, mt in enumerate(mats):
                    hb.x_view(i).copy_(torch.from_numpy(mt["L"].x))
                hb.capture()       # copy in, launches, copy out recorded once; every step replays them and waits
            h2d, d2h = hbatch[0].x_host.numel(), hbatch[0].y_host.numel()

            def e2e_step(c):
                hbatch[c].run()
                torch.cuda.current_stream().synchronize()
        else:
            host = []
            for mt in mats:
                L = mt["L"]
                xh = torch.from_numpy(L.x).pin_memory()
                yh = torch.empty((M, L.N), dtype=torch.float32).pin_memory()
                sc = torch.zeros(lcd.linear_host_scratch_bytes(mt["w"][0], M), dtype=torch.uint8, device=dev)
                host.append((xh, yh, sc))
                h2d += xh.numel() * 2
                d2h += yh.numel() * 4

            def e2e_step(c):
                if args.act_bits == 4:
                    for mt, (xh, yh, sc) in zip(mats, host):
                        lcd.linear_host(mt["w"][c], xh, mt["inv_s"], yh, sc)
                else:          # no host-buffer entry point for 8-bit levels: the copies are made here
                    for mt, (xh, yh, sc) in zip(mats, host):
                        mt["x"].copy_(xh, non_blocking=True)
                    step(c)
                    for mt, (xh, yh, sc) in zip(mats, host):
                        yh.copy_(mt["y"], non_blocking=True)
                torch.cuda.current_stream().synchronize()

        if primary:
            n_e2e = max(3, min(steps, 50))
            for c in range(min(copies, 3)):
                e2e_step(c)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            g0.record()
            for i in range(n_e2e):
                e2e_step(i % copies)
            g1.record()
            torch.cuda.synchronize()
            e2e_ms = max(g0.elapsed_time(g1), (time.perf_counter() - t0) * 1e3) / n_e2e
            if world > 1:
                e2e_ms = max_over_ranks(e2e_ms, dev)
        # the outputs and stored levels of the timed path, for the comparison with the oracle below
        step(0)
        torch.cuda.synchronize()

    ms_step = ms_total / steps
    us_per_layer = per_layer_us(ms_step, world)
    layer_alg_bytes = sum(mt["bytes"] for mt in mats)
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    tensor_bound = M > 16
    if tensor_bound:
        peak = peaks.get("bf16_tflops", 1590.0)
        achieved = kern_flop / kern_ms / 1e9
        roof = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                "traffic": None, "peak_source": "measured (cuBLAS bf16 burst)" if peaks else "fallback",
                "frac_of_sustained": achieved / peaks.get("bf16_tflops_sustained", 1400.0),
                "frac_of_2250_nominal": achieved / 2250.0}
    else:
        peak = peaks.get("hbm_gbs", 6650.0)
        achieved = kern_bytes / kern_ms / 1e6
        roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": None, "peak_source": "measured (copy)" if peaks else "fallback",
                "frac_of_8TBps_nominal": achieved / 8000.0}
    src = "dense_tc.cu" if tensor_bound else ("lut_smem.cu" if shared_bucket else "lut_gemv.cu")
    rec = NCU_TRAFFIC.get((src, cfg_id, M))
    if rec and rec["bytes_per_launch"] is not None:
        import hashlib
        with open(os.path.join(ROOT, "paper_2506_12038_b200", "csrc", src), "rb") as fh:
            if hashlib.sha256(fh.read()).hexdigest() == rec["sha256"]:
                roof["traffic"] = rec["bytes_per_launch"]
    torch.cuda.synchronize()
    if int(status.item()) != 0:
        raise RuntimeError(f"a kernel reported status {int(status.item())} (bounded wait expired): timings are void")
    roof["kernel"] = kern_name
    roof["us_per_launch"] = kern_ms * 1e3
    roof["per_matrix"] = per_matrix

    if rank != 0:
        return None
    line = {"metric": metric_name(M), "value": us_per_layer, "unit": "us/layer", "n_gpus": world, "steps": steps,
            "warmup": max(args.warmup, 3) if primary else 3, "ms_per_step": ms_step, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None,
            "dtype": ("s8 table bytes x s8 levels -> s32 (tcgen05 kind::i8), f32 epilogue" if tensor_bound else
                      "u8 bucket-table bytes -> s32 (int8 MMA), f32 sums and epilogue" if shared_bucket else
                      "s8 table bytes x s8 levels -> s32 (int8 MMA), f32 epilogue"),
            "data": "synthetic", "config": dict(workload_config(cfg_id, M, copies, args.act_bits),
                                                graphs=f"steps replayed as CUDA graphs of {copies} consecutive steps",
                                                launches=("1 launch per layer: quantise + lookup fused" if grouped and fused
                                                          else "1 grouped quantise + 1 grouped lookup per layer" if grouped
                                                          else "1 quantise launch for the layer + 1 tensor-core launch per matrix (one library call)" if fused
                                                          else "per matrix: quantise + lookup")),
            "timing": {"repeats": len(rep_ms), "steps_per_repeat": steps, "timed_ms_total": sum(rep_ms),
                       "us_per_step_median": statistics.median(rep_ms) / steps * 1e3 / world,
                       "us_per_step_min": min(rep_ms) / steps * 1e3 / world},
            "layer_GBps": layer_alg_bytes * world / (ms_step * 1e-3) / 1e9,
            "layer_algorithmic_bytes": layer_alg_bytes,
            "TFLOPs_equiv": sum(mt["flop"] for mt in mats) * world / (ms_step * 1e-3) / 1e12,
            "clocks": clocks, "gpu_launches": launches_per_step * steps * len(rep_ms),
            "roofline": roof}
    if e2e_ms is not None:
        line["e2e"] = {"value": e2e_ms * 1e3 / world, "unit": "us/layer", "h2d_bytes_per_step": h2d,
                       "d2h_bytes_per_step": d2h}
    if world == 1 and not args.no_cpu_baseline:
        # The oracle on the same inputs: its outputs judge the timed path (every output at small M, the sample at
        # M = 2048), its running time is the CPU baseline (primary workload only).
        sample, scale, desc = oracle_sample(cfg_id, layers, M)
        t0 = time.perf_counter()
        n = 0
        while True:
            outs = oracle_layer_pass(sample)
            n += 1
            if not primary or time.perf_counter() - t0 > 10.0 or n >= 5:
                break
        us = (time.perf_counter() - t0) / n * scale * 1e6
        if primary:
            line["cpu_baseline"] = {"value": us, "unit": "us/layer", "cores": oracle_threads(), "kind": "oracle",
                                    "sample": desc + f", mean of {n} passes"}
        line["parity"] = parity_verdict(sample, outs, mats, args.act_bits)
        if not line["parity"]["ok"]:
            print(json.dumps(line))
            raise SystemExit("parity with the oracle lost: " + json.dumps(line["parity"]))
    return line


def parity_verdict(sample, oracle_outs, mats, act_bits):
    """The timed path's outputs against the oracle's on the same inputs: per matrix relative L2 error and
    max-abs error over the largest reference magnitude (stated tolerance 2e-3 and 1e-2), and the stored activation
    levels and scales bit for bit.  `sample` is the whole layer, or (large M) the leading rows and tokens of its first
    matrix: the corresponding corner of the device output is compared."""
    from oracle import lcd_oracle as O
    rel_max, abs_max, exact = 0.0, 0.0, True
    by_name = {mt["name"]: mt for mt in mats}
    for (name, S), y_ref in zip(sample, oracle_outs):
        mt = by_name[name]
        y = mt["y"][:S.M, :S.N].detach().cpu().numpy().astype(np.float64)
        if not np.all(np.isfinite(y)):
            return {"ok": False, "reason": f"{name}: non-finite output"}
        d = np.linalg.norm(y_ref)
        rel_max = max(rel_max, float(np.linalg.norm(y - y_ref) / (d if d > 0 else 1.0)))
        ninf = np.abs(y_ref).max()
        abs_max = max(abs_max, float(np.abs(y - y_ref).max() / (ninf if ninf > 0 else 1.0)))
        q, sq = O.smooth_quantize(S.x, S.inv_s, act_bits=act_bits)
        packed = O.pack_act(q) if act_bits == 4 else O.pad_act8(q)
        exact = exact and np.array_equal(mt["a"][:S.M].cpu().numpy(), packed) and np.array_equal(mt["s"][:S.M].cpu().numpy(), sq)
    return {"ok": bool(rel_max <= 2e-3 and abs_max <= 1e-2 and exact), "rel_l2_max": rel_max,
            "max_abs_over_inf": abs_max, "indices_bit_exact": bool(exact),
            "compared": f"{len(sample)} matrices, " + ("every output" if len(sample) == len(mats) else "the sampled corner (see cpu_baseline.sample)")}


def run_aux_smoothing(args):
    """Section 3.4 grid search on a 128-token synthetic calibration batch per matrix of the configuration
    (same outlier recipe as the test tokens): 21 candidates, CUDA events, printed as one JSON line."""
    import torch
    import paper_2506_12038_b200 as lcd
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    cfg = gen.CONFIGS[args.config]
    alphas = [i / 20 for i in range(21)]
    rows, total_ms = [], 0.0
    for mi, (name, N, K) in enumerate(cfg["shapes"]):
        ch = gen.outlier_channels(1000 + mi, K, cfg["frac"])
        x = torch.from_numpy(gen.activations(2000 + mi, 128, K, ch, cfg["scale"])).to(dev)
        wmax = torch.from_numpy((np.abs(gen.normal(3000 + mi, K)) * 0.05 + 0.01).astype(np.float32)).to(dev)
        for _ in range(3):
            lcd.smoothing_search(x, wmax, alphas)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(10):
            best, mse, inv = lcd.smoothing_search(x, wmax, alphas)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / 10
        total_ms += ms
        rows.append({"matrix": name, "K": K, "us": ms * 1e3, "best_alpha": alphas[int(best.item())]})
    print(json.dumps({"aux": "smoothing_search", "config": {"workload": f"configuration {args.config} ({cfg['name']})",
                                                            "calibration_tokens": 128, "candidates": len(alphas)},
                      "us_per_layer": total_ms * 1e3, "per_matrix": rows, "data": "synthetic"}))


def run_aux_reclassify(args):
    """Section 3.2 bookkeeping on every matrix of the configuration: random clusters, sorted random codebooks and
    N(0, 0.4) updates; 6 bytes per weight (index and update read, index written); CUDA events, one JSON line."""
    import torch
    import paper_2506_12038_b200 as lcd
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    cfg = gen.CONFIGS[args.config]
    C = 1 << cfg["bits"]
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    peak = peaks.get("hbm_gbs", 6650.0)
    rows, tot_ms, tot_bytes = [], 0.0, 0.0
    g = torch.Generator(device=dev)
    g.manual_seed(1234)
    for name, N, K in cfg["shapes"]:
        idx = torch.randint(0, C, (N, K), dtype=torch.uint8, device=dev, generator=g)
        cb = torch.sort(torch.randn((N, C), device=dev, generator=g), dim=1).values.to(torch.float16)
        dw = torch.randn((N, K), device=dev, generator=g) * 0.4
        out = lcd.reclassify(idx, cb, dw)
        stream = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(stream):
            for _ in range(3):
                lcd.reclassify(idx, cb, dw, out=out)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()              # ten launches back to back, no host gaps
            with torch.cuda.graph(graph, stream=stream):
                for _ in range(10):
                    lcd.reclassify(idx, cb, dw, out=out)
            graph.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            graph.replay()
            e1.record()
            torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / 10
        b = 6.0 * N * K
        tot_ms += ms
        tot_bytes += b
        rows.append({"matrix": name, "N": N, "K": K, "us": ms * 1e3, "GBps": b / ms / 1e6})
    print(json.dumps({"aux": "reclassify", "config": {"workload": f"configuration {args.config} ({cfg['name']})", "C": C},
                      "us_per_layer": tot_ms * 1e3, "per_matrix": rows, "data": "synthetic",
                      "roofline": {"bound": "hbm", "achieved": tot_bytes / tot_ms / 1e6, "peak": peak, "unit": "GB/s",
                                   "frac": tot_bytes / tot_ms / 1e6 / peak,
                                   "peak_source": "measured (copy)" if peaks else "fallback"}}))


def run_aux_dbci(args):
    """Section 3.1 on every matrix of the configuration taken as one flat array: N(0, 0.02) weights with ten
    12-sigma outliers; CUDA events around three calls after a warm-up; one JSON line."""
    import torch
    import paper_2506_12038_b200 as lcd
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    cfg = gen.CONFIGS[args.config]
    g = torch.Generator(device=dev)
    g.manual_seed(4321)
    rows, tot_ms = [], 0.0
    for name, N, K in cfg["shapes"]:
        w = torch.randn((N * K,), device=dev, generator=g) * 0.02
        w[:: max(N * K // 10, 1)] *= 12
        r = lcd.dbci(w, want_labels=False)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(3):
            r = lcd.dbci(w, want_labels=False)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / 3
        tot_ms += ms
        rows.append({"matrix": name, "weights": N * K, "ms": ms, "Gweights_per_s": N * K / ms / 1e6,
                     "centroids": int(r["centroids"].numel()), "sigma": r["sigma"], "min_pts": r["min_pts"]})
    print(json.dumps({"aux": "dbci", "config": {"workload": f"configuration {args.config} ({cfg['name']})"},
                      "ms_per_layer": tot_ms, "per_matrix": rows, "data": "synthetic"}))


def main():
    args = parse_args()
    if args.aux == "smoothing":
        run_aux_smoothing(args)
        return
    if args.aux == "dbci":
        run_aux_dbci(args)
        return
    if args.aux == "reclassify":
        run_aux_reclassify(args)
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
