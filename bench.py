#!/usr/bin/env python
"""Benchmark of the Rollout-ResQ FP4 linear path (Eq. (5)) on B200.

A "step" is one pass of the whole hot path -- quantize X, residual, re-quantize, select, two-term
GEMM against packed HiF4 weights -- over the four linears of one transformer block of the
workload (default: the Qwen2.5-3B decode-shaped configuration, M = 256 tokens, S_2:4).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--pattern P] [--format F]
    python bench.py --impl reference ...        # times the CPU oracle on a bounded sample

Prints ONE JSON line on stdout (rank 0); `--verbose` adds a per-layer table on stderr.
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

from workloads import CONFIGS, make_activation, make_weight  # noqa: E402

METRIC = "hif4_resq_linear TFLOP/s & GB/s at 1 B200; % of FP4-tensor/HBM roofline"
L2_BYTES = 126 * 1024 * 1024
PATTERN_IDS = {"none": 0, "dense": 1, "2:4": 2, "row50": 3, "chan50": 4, "block": 5}
# sparsity sweep: the selecting patterns with 1/4 or 3/4 kept (RESQ_KEEP_QUARTERS)
for _name, _base in (("{}:4", 2), ("row{}", 3), ("chan{}", 4), ("block{}", 5)):
    for _q in (1, 3):
        PATTERN_IDS[_name.format(_q if _base == 2 else 25 * _q)] = _base | (_q << 8)
PATTERN_IDS["block-strip"] = 5 | (1 << 12)  # block selection inside every strip of 32 rows (RESQ_BLOCK_PER_STRIP)
RHO = {0: 0.0, 1: 1.0, 2: 0.5, 3: 0.5, 4: 0.5, 5: 0.5}
RHO.update({p: ((p >> 8) & 0xF) / 4.0 if (p >> 8) & 0xF else 0.5 for p in PATTERN_IDS.values() if p >> 8})
# mean DRAM bytes per GEMM launch from an ncu capture of the default workload (see profiles/)
NCU_TRAFFIC_BYTES_PER_LAUNCH = {(1, 2, "hif4"): 15.3e6}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ----------------------------------------------------------------------------- algorithmic work

def layer_flops(M, N, K, pattern):
    """2 M N K (1 + rho): the dense term plus the kept half (or all) of the residual term (Section 5.4)."""
    return 2.0 * M * N * K * (1.0 + RHO[pattern])


def layer_bytes(M, N, K, pattern, fmt):
    """Bytes the method must move per call: bf16 X in, packed W in, bf16 Y out."""
    w_bits = 4.5 if fmt == "hif4" else 4.25
    return 2.0 * M * K + w_bits / 8.0 * N * K + 2.0 * M * N


# ----------------------------------------------------------------------------- clocks sampler

class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.QUERY, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._reader, daemon=True)
        self.thread.start()

    def _reader(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        rows = [r for (t, r) in self.rows if t0 - 0.05 <= t <= t1 + 0.15 and len(r) >= 9] or \
               [r for (_, r) in self.rows if len(r) >= 9]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm = [float(r[1]) for r in rows]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({n for r in rows for n, v in zip(names, r[5:9]) if v.lower().startswith("active")})
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": float(rows[0][2]), "reasons": reasons,
                "samples": len(rows), "power_w_max": max(float(r[3]) for r in rows)}


# ----------------------------------------------------------------------------- CPU oracle timing

def time_oracle(cfg, pattern, fmt, budget_s=20.0):
    """Times the oracle, as it stands, on a bounded sample of the workload: every layer of the config, on
    the first rows of X (all of them if that fits the budget).  Returns (TFLOP/s, cores, description, s)."""
    import oracle
    from workloads import bf16_bits_to_f32
    threads = oracle.num_threads()
    macs_per_row = sum(2.0 * l.K * l.N for l in cfg.layers)          # two fp64 sweeps per output element
    rate = 0.6e9 * threads                                            # rough fp64 MAC/s of the plain triple loop
    rows = int(max(32, min(cfg.M, budget_s * rate / macs_per_row)))
    rows -= rows % 32
    flops, dt = 0.0, 0.0
    for li, spec in enumerate(cfg.layers):
        x = bf16_bits_to_f32(make_activation(cfg, li, M=rows))
        w = bf16_bits_to_f32(make_weight(cfg, li))
        t0 = time.perf_counter()
        oracle.resq_linear(x, w, pattern, fmt, want_abs=False)
        dt += time.perf_counter() - t0
        flops += layer_flops(rows, spec.N, spec.K, pattern)
    sample = (f"{cfg.name}: all {len(cfg.layers)} layers, first {rows} of {cfg.M} token rows "
              f"(weight packing, quantizer, masks and fp64 product all timed)")
    return flops / dt / 1e12, threads, sample, dt


# ----------------------------------------------------------------------------- main

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=1, help="index into the workload configs (default 1: 3B decode)")
    ap.add_argument("--pattern", default=None,
                    help="none|dense|2:4|row50|chan50|block (default: the config's); sparsity sweep: 1:4|3:4|row25|row75|"
                         "chan25|chan75|block25|block75|block-strip")
    ap.add_argument("--format", default="hif4", choices=["hif4", "mxfp4"])
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--out-dtype", default="bf16", choices=["bf16", "f32"])
    ap.add_argument("--layers", default=None, help="comma-separated subset of the config's layers (profiling aid)")
    ap.add_argument("--tokens", type=int, default=None, help="override M (profiling aid; not the benchmark workload)")
    ap.add_argument("--skip-e2e", action="store_true", help="skip the end-to-end and per-kernel passes (profiling aid)")
    ap.add_argument("--quantizer-sweep", action="store_true",
                    help="bandwidth sweep of *_quantize_act over M x K (prints a table on stderr and one JSON line)")
    ap.add_argument("--accuracy-contrast", action="store_true",
                    help="relative error of plain FP4, the rotation baseline and the residual variants against the exact "
                         "bf16 product on the config's synthetic outlier tensors (no timing)")
    ap.add_argument("--no-graph", action="store_true", help="launch eagerly instead of replaying a CUDA graph per step")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--verbose", action="store_true")
    args = ap.parse_args()

    cfg = CONFIGS[args.config]
    if args.layers or args.tokens:
        import dataclasses
        keep = args.layers.split(",") if args.layers else [l.name for l in cfg.layers]
        cfg = dataclasses.replace(cfg, layers=tuple(l for l in cfg.layers if l.name in keep),
                                  M=args.tokens or cfg.M, name=cfg.name + " (subset)")
    pattern = PATTERN_IDS[args.pattern] if args.pattern else cfg.patterns[0]
    pattern_name = {v: k for k, v in PATTERN_IDS.items()}[pattern]
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    config_desc = {
        "workload": f"{cfg.name}: M={cfg.M}, layers " + ", ".join(f"{l.name} {l.K}->{l.N}" for l in cfg.layers),
        "pattern": pattern_name, "format": args.format, "out_dtype": args.out_dtype,
        "parallelism": "replicas only (one independent copy of the step per GPU)",
    }

    if args.impl == "reference":
        if rank != 0:
            return
        vals = []
        for _ in range(max(1, min(args.warmup, 1))):
            time_oracle(cfg, pattern, args.format, budget_s=3.0)
        info = None
        for _ in range(max(1, min(args.steps, 3))):
            info = time_oracle(cfg, pattern, args.format, budget_s=8.0)
            vals.append(info[0])
        v = statistics.median(vals)
        line = {"impl": "reference", "metric": METRIC, "value": v, "unit": "TFLOP/s", "n_gpus": args.gpus,
                "steps": len(vals), "warmup": 1, "ms_per_step": info[3] * 1e3, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config_desc,
                "cpu_baseline": {"value": v, "unit": "TFLOP/s", "cores": info[1], "kind": "oracle", "sample": info[2]},
                "e2e": {"value": v, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return

    import torch
    import paper_2607_26515_b200 as rq
    from paper_2607_26515_b200.replicas import max_over_ranks

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    rq.lib()  # fail loudly if the CUDA library is missing
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    out_dtype = torch.bfloat16 if args.out_dtype == "bf16" else torch.float32
    fmt = args.format

    if args.quantizer_sweep:
        # hif4_quantize_act / mxfp4_quantize_act alone: read bf16 X, write packed codes + metadata.
        peaks, peak_kind = load_peaks()
        bpe = 2.0 + (0.5625 if fmt == "hif4" else 0.53125)
        rows = []
        for K in (2048, 18944):
            for M in (256, 512, 1024, 2048, 4096, 8192, 16384, 32768):
                nbuf = max(2, int(np.ceil(1.5 * L2_BYTES / (M * K * 2))))
                nbuf = min(nbuf, 64)
                xs = [torch.randn((M, K), device=dev, dtype=torch.float32).to(torch.bfloat16) for _ in range(nbuf)]
                for i in range(3):
                    rq.quantize_act(xs[i % nbuf], fmt)
                torch.cuda.synchronize()
                reps = max(10, min(200, int(2e9 / (M * K * bpe))))
                codes = torch.empty((M, K // 2), dtype=torch.uint8, device=dev)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for i in range(reps):
                    rq.quantize_act(xs[i % nbuf], fmt)
                e1.record()
                torch.cuda.synchronize()
                us = e0.elapsed_time(e1) * 1e3 / reps
                gbs = M * K * bpe / (us * 1e-6) / 1e9
                rows.append({"M": M, "K": K, "us": us, "GB/s": gbs, "frac_of_hbm": gbs / peaks["hbm_gbs"]})
                print(f"[quantize_act {fmt}] M={M:6d} K={K:6d}  {us:9.1f} us  {gbs:8.1f} GB/s  "
                      f"{100 * gbs / peaks['hbm_gbs']:5.1f} % of {peak_kind} copy rate", file=sys.stderr)
                del xs, codes
        best = max(rows, key=lambda r: r["GB/s"])
        print(json.dumps({"metric": f"{fmt}_quantize_act GB/s (algorithmic {bpe} B/element)", "value": best["GB/s"],
                          "unit": "GB/s", "roofline": {"bound": "hbm", "achieved": best["GB/s"], "peak": peaks["hbm_gbs"],
                                                       "unit": "GB/s", "frac": best["frac_of_hbm"]},
                          "sweep": rows, "data": "synthetic", "note": "includes launch overhead at small M"}))
        return

    if args.accuracy_contrast:
        # What the residual correction buys against the rotation baseline on this workload's synthetic tensors
        # (outlier channels as in the paper's Figure 1): relative Frobenius error of Y against the exact product of
        # the bf16 operands (fp64 on the device; plumbing, not part of the path).
        signs = 0x9E3779B97F4A7C15
        table = {}
        for li, spec in enumerate(cfg.layers):
            rows = min(cfg.M, 256)
            x = torch.from_numpy(make_activation(cfg, li)[:rows].view(np.int16)).view(torch.bfloat16).to(dev)
            w = torch.from_numpy(make_weight(cfg, li).view(np.int16)).view(torch.bfloat16).to(dev)
            exact = x.double() @ w.double().t()
            norm = exact.norm().item()
            wc, ws = rq.pack_weight(w, fmt)
            wcr, wsr = rq.rht_pack_weight(w, signs, fmt)
            err = {}
            for name, pat in (("plain", rq.S_NONE), ("resq_1:4", rq.keep_quarters(rq.S_2_4, 1)), ("resq_2:4", rq.S_2_4),
                              ("resq_3:4", rq.keep_quarters(rq.S_2_4, 3)), ("resq_chan50", rq.S_CHAN50),
                              ("resq_block", rq.S_BLOCK), ("resq_dense", rq.S_DENSE)):
                if (pat & 0xFF) == rq.S_BLOCK and rows % 32:
                    continue
                y = rq.resq_linear(x, wc, ws, pat, fmt, out_dtype=torch.float32)
                err[name] = ((y.double() - exact).norm().item() / norm)
            y = rq.rht_resq_linear(x, signs, wcr, wsr, rq.S_NONE, fmt, out_dtype=torch.float32)
            err["rotation"] = ((y.double() - exact).norm().item() / norm)
            y = rq.rht_resq_linear(x, signs, wcr, wsr, rq.S_2_4, fmt, out_dtype=torch.float32)
            err["rotation+resq_2:4"] = ((y.double() - exact).norm().item() / norm)
            y = rq.w16a4_linear(x, w, rq.S_NONE, fmt, out_dtype=torch.float32)
            err["w16a4"] = ((y.double() - exact).norm().item() / norm)
            y = rq.w4a8_linear(x, wc, ws, fmt, out_dtype=torch.float32)
            err["w4a8"] = ((y.double() - exact).norm().item() / norm)
            y = rq.w4a16_linear(x, wc, ws, fmt, out_dtype=torch.float32)
            err["w4a16"] = ((y.double() - exact).norm().item() / norm)
            table[spec.name] = err
            print(f"[contrast {fmt}] {spec.name:8s} " + "  ".join(f"{k} {v:.4f}" for k, v in err.items()), file=sys.stderr)
        print(json.dumps({"metric": f"relative Frobenius error of Y against the exact bf16 product ({fmt})", "contrast": table,
                          "data": "synthetic", "config": config_desc}))
        return

    # ---- inputs: generated once on the host, packed once (weights are packed per policy update, not per call)
    layers = []
    w_bytes_total = 0
    for li, spec in enumerate(cfg.layers):
        xb = make_activation(cfg, li)
        wb = make_weight(cfg, li)
        x_host = torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).pin_memory()
        w_dev = torch.from_numpy(wb.view(np.int16)).view(torch.bfloat16).to(dev)
        wc, ws = rq.pack_weight(w_dev, fmt)
        del w_dev
        w_bytes_total += wc.numel() + ws.numel() * ws.element_size()
        layers.append({"spec": spec, "x_host": x_host, "wc": wc, "ws": ws})
    # rotate over enough copies of the packed weights that a step never finds them in L2
    n_sets = max(2, int(np.ceil(1.5 * L2_BYTES / max(1, w_bytes_total))))
    n_sets = min(n_sets, 16)
    for L in layers:
        spec = L["spec"]
        L["w_sets"] = [(L["wc"], L["ws"])] + [(L["wc"].clone(), L["ws"].clone()) for _ in range(n_sets - 1)]
        L["x_sets"] = [L["x_host"].to(dev) for _ in range(n_sets)]
        L["y"] = torch.empty((cfg.M, spec.N), dtype=out_dtype, device=dev)
        L["y_host"] = torch.empty((cfg.M, spec.N), dtype=out_dtype).pin_memory()
        L["x_stage"] = torch.empty_like(L["x_sets"][0])
        L["work"] = rq.alloc_workspace(rq.resq_workspace_bytes(cfg.M, spec.N, spec.K, pattern, fmt), dev)
    config_desc["l2"] = (f"rotating {n_sets} copies of weights and activations "
                         f"({n_sets * w_bytes_total / 1e6:.0f} MB of packed weights > 126 MB L2)")

    def step(i):
        k = i % n_sets
        for L in layers:
            wc, ws = L["w_sets"][k]
            rq.resq_linear(L["x_sets"][k], wc, ws, pattern, fmt, Y=L["y"], workspace=L["work"])

    # One CUDA graph per rotation set: at decode sizes the step is a dozen short kernels and the host
    # (tensor-map encoding, launches) would otherwise be the bottleneck.  Everything the library enqueues
    # (memsets, kernels, cluster launches) is capturable; attributes were set during warm-up.
    graphs = []

    def build_graphs():
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for k in range(n_sets):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    step(k)
                graphs.append(g)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()

    def step_graph(i):
        graphs[i % n_sets].replay()

    # End to end: every step copies each layer's activations from pinned host memory, runs the layer through the
    # public call and reads its output back.  The layers of a step are independent calls, so their copies run on
    # two copy streams beside the compute stream (input of the next layer and output of the previous one overlap
    # the current layer's kernels); the layer with the largest output goes first.  A step ends when every output
    # is in host memory.
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    e2e_order = sorted(layers, key=lambda L: -L["y"].numel())

    def step_e2e(i, capturing=False):
        k = i % n_sets
        main = torch.cuda.current_stream()
        s_in.wait_stream(main)    # earlier work on the inputs' staging buffers is done (previous steps were synchronized)
        for L in e2e_order:
            with torch.cuda.stream(s_in):
                L["x_stage"].copy_(L["x_host"], non_blocking=True)       # host -> device, pinned
                L["ev_in"] = s_in.record_event()
        for L in e2e_order:
            wc, ws = L["w_sets"][k]
            main.wait_event(L["ev_in"])
            rq.resq_linear(L["x_stage"], wc, ws, pattern, fmt, Y=L["y"], workspace=L["work"])
            ev = main.record_event()
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev)
                L["y_host"].copy_(L["y"], non_blocking=True)             # device -> host
        if capturing:
            main.wait_stream(s_out)   # join the copy branches into the captured stream
        else:
            s_out.synchronize()
            main.synchronize()

    e2e_graphs = []

    def build_e2e_graphs():
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for k in range(n_sets):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    step_e2e(k, capturing=True)
                e2e_graphs.append(g)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()

    def step_e2e_graph(i):
        e2e_graphs[i % n_sets].replay()       # copies in, kernels and copies out: one graph launch per step
        torch.cuda.current_stream().synchronize()

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.time()
        e0.record()
        for i in range(steps):
            fn(i)
        e1.record()
        barrier()
        t1 = time.time()
        ms = max_over_ranks(e0.elapsed_time(e1), dev)
        return ms, t0, t1

    def per_layer_table():
        rq.profile_enable(True)
        for L in layers:
            spec = L["spec"]
            rq.profile_read()
            for i in range(10):
                wc, ws = L["w_sets"][i % n_sets]
                rq.resq_linear(L["x_sets"][i % n_sets], wc, ws, pattern, fmt, Y=L["y"], workspace=L["work"])
            torch.cuda.synchronize()
            pr = rq.profile_read()
            f = layer_flops(cfg.M, spec.N, spec.K, pattern)
            g_us = pr["gemm"][0] * 100.0
            print(f"[layer {spec.name:8s}] K={spec.K:6d} N={spec.N:6d}  quant {pr['quantize'][0]*100:8.1f} us  "
                  f"select {pr['select'][0]*100:7.1f} us  gemm {g_us:8.1f} us  reduce {pr['splitk_reduce'][0]*100:6.1f} us  "
                  f"gemm {f / (g_us * 1e-6) / 1e12:7.1f} TFLOP/s", file=sys.stderr)
        rq.profile_enable(False)

    warmup = max(3, args.warmup)
    for i in range(warmup):
        step(i)
    for L in layers:
        if rq.check(L["work"]) != 0:
            raise SystemExit("device status: " + rq.last_error())

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    launches0 = rq.kernel_launches()
    step(0)
    launches_per_step = rq.kernel_launches() - launches0
    use_graph = not args.no_graph
    if use_graph:
        build_graphs()
        for i in range(3):
            step_graph(i)
    run_step = step_graph if use_graph else step
    config_desc["launch"] = "one CUDA graph replay per step" if use_graph else "eager launches"
    ms, t0, t1 = timed(run_step, args.steps)
    launches = launches_per_step * args.steps
    # keep the GPU busy a little longer so that the 100 ms sampler certainly sees the loaded state
    t_load0 = time.time()
    reps = 0
    while time.time() - t_load0 < 0.6:
        for i in range(20):
            run_step(i)
        torch.cuda.synchronize()
        reps += 1
    t_load1 = time.time()
    clocks = sampler.stop(t0, t_load1) if rank == 0 else None

    flops_step = sum(layer_flops(cfg.M, L["spec"].N, L["spec"].K, pattern) for L in layers)
    bytes_step = sum(layer_bytes(cfg.M, L["spec"].N, L["spec"].K, pattern, fmt) for L in layers)
    ms_per_step = ms / args.steps
    tflops = world * flops_step / (ms_per_step * 1e-3) / 1e12
    gbs = world * bytes_step / (ms_per_step * 1e-3) / 1e9

    if args.verbose and rank == 0:
        per_layer_table()
    if args.skip_e2e:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": tflops, "unit": "TFLOP/s", "ms_per_step": ms_per_step,
                              "config": config_desc, "note": "profiling aid run: no e2e / roofline passes"}))
        return
    # ---- end-to-end: host buffers, copies inside the timed region
    for i in range(3):
        step_e2e(i)
    run_e2e = step_e2e
    if use_graph:
        build_e2e_graphs()
        run_e2e = step_e2e_graph
        for i in range(3):
            run_e2e(i)
    for L in layers:  # the pipelined copies delivered what the device holds
        if not torch.equal(L["y_host"], L["y"].cpu()) or not torch.equal(L["x_stage"].cpu(), L["x_host"]):
            raise RuntimeError(f"end-to-end step: host copy of layer {L['spec'].name} differs from the device tensor")
    ms_e2e, _, _ = timed(run_e2e, args.steps)
    if os.environ.get("RESQ_BENCH_E2E_BOTH"):  # aid: the eager-launch figure beside the graph one
        ms_eager, _, _ = timed(step_e2e, args.steps)
        print(f"e2e eager {ms_eager / args.steps:.4f} ms  graph {ms_e2e / args.steps:.4f} ms", file=sys.stderr)
    e2e_tflops = world * flops_step / (ms_e2e / args.steps * 1e-3) / 1e12
    h2d = sum(L["x_host"].numel() * 2 for L in layers)
    d2h = sum(L["y_host"].numel() * L["y_host"].element_size() for L in layers)

    # ---- per-kernel device time (CUDA events around every launch, on the launching stream)
    rq.profile_enable(True)
    rq.profile_read()
    barrier()
    for i in range(args.steps):
        step(i)
    torch.cuda.synchronize()
    prof = rq.profile_read()
    rq.profile_enable(False)
    gemm_ms, gemm_n = prof["gemm"]
    quant_ms, quant_n = prof["quantize"]
    peaks, peak_kind = load_peaks()
    gemm_tflops = flops_step * args.steps / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else None
    if fmt == "mxfp4":
        # block-scaled FP4 pipe: the measured bf16 peak times the nominal FP4 : bf16 ratio (9 : 2.25 PFLOP/s)
        kernel_name = "gemm_mxfp4_native_kernel (tcgen05.mma kind::mxf4.block_scale on packed E2M1 codes; bf16 route for some layers)"
        tensor_peak, peak_src = peaks["bf16_tflops"] * 4.0, f"bf16 burst ({peak_kind}) x 4 (nominal FP4 : bf16 ratio)"
    else:
        kernel_name = "gemm_pair_kernel (tcgen05.mma cta_group::2 kind::f16 on in-kernel bf16-expanded 4-bit weights)"
        tensor_peak, peak_src = peaks["bf16_tflops"], f"bf16 burst, {peak_kind}"
    roofline = {
        "kernel": kernel_name,
        "bound": "tensor",
        "achieved": gemm_tflops, "peak": tensor_peak, "unit": "TFLOP/s",
        "frac": (gemm_tflops / tensor_peak) if gemm_tflops else None,
        "peak_source": peak_src, "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH.get((args.config, pattern, fmt)),
        "traffic_source": "ncu dram__bytes_read.sum + dram__bytes_write.sum, mean over the step's GEMM launches "
                          "(profiles/gemm_pair_kernel_3b-decode_2to4.md); null for workloads not captured",
        "avg_launch_us": gemm_ms * 1e3 / max(1, gemm_n), "launches": gemm_n,
        "quantizer_avg_launch_us": quant_ms * 1e3 / max(1, quant_n),
        "quantizer_share_of_kernel_time": quant_ms / max(1e-9, sum(v[0] for v in prof.values())),
        "hbm_frac_of_step": gbs / world / peaks["hbm_gbs"],
        "frac_of_fp8_nominal": (gemm_tflops / 4500.0) if gemm_tflops else None,
        "frac_of_fp4_nominal": (gemm_tflops / 9000.0) if gemm_tflops else None,
    }

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, cores, sample, dt = time_oracle(cfg, pattern, fmt)
        cpu_baseline = {"value": v, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample,
                        "seconds": dt}

    if rank == 0:
        line = {
            "metric": METRIC, "value": tflops, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if fmt == "hif4" else "fp4 (e2m1, ue8m0 block scales) / bf16",
            "data": "synthetic", "config": config_desc,
            "gb_per_s": gbs, "clocks": clocks,
            "e2e": {"value": e2e_tflops, "unit": "TFLOP/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": ms_e2e / args.steps},
            "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu_baseline,
        }
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
