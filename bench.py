#!/usr/bin/env python
"""Benchmark of the Rollout-ResQ FP4 linear path (Eq. (5)) on B200.

A "step" is one pass of the whole hot path -- quantize X, residual, re-quantize, select, two-term
GEMM against packed HiF4 weights -- over the four linears of one transformer block of the workload.
The headline workload is the largest single-GPU configuration, the Qwen2.5-Math-7B prefill-shaped
block (M = 16384 tokens) with the S_2:4 residual; the same JSON line carries the other
configurations (`per_config`), the residual patterns and the MXFP4 twin on the headline workload
(`per_pattern`), a true decode sweep M = 16 ... 128 with its HBM fraction (`decode_sweep`) and the
quantizer-only bandwidth sweep (`quantizer_sweep`).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--pattern P] [--format F]
    python bench.py --impl reference ...        # times the CPU oracle on a bounded sample

Prints ONE JSON line on stdout (rank 0); `--verbose` adds a per-layer table on stderr.
"""
from __future__ import annotations

import argparse
import dataclasses
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

from workloads import CONFIGS  # noqa: E402
from workloads import make_activation as _make_activation, make_weight as _make_weight  # noqa: E402

_HOST_TENSORS = {}


def make_activation(cfg, li, M=None):
    """The seeded activation of a layer, generated once per process (the 7B prefill tensors take seconds to draw)."""
    key = ("x", cfg.index, cfg.layers[li].name, cfg.M if M is None else M)
    if key not in _HOST_TENSORS:
        base = CONFIGS[cfg.index]  # (cfg may be a subset of its layers or carry another M: seeds follow the base config)
        _HOST_TENSORS[key] = _make_activation(base, [l.name for l in base.layers].index(cfg.layers[li].name),
                                              cfg.M if M is None else M)
    return _HOST_TENSORS[key]


def make_weight(cfg, li):
    key = ("w", cfg.index, cfg.layers[li].name)
    if key not in _HOST_TENSORS:
        _HOST_TENSORS[key] = _make_weight(CONFIGS[cfg.index], [l.name for l in CONFIGS[cfg.index].layers].index(cfg.layers[li].name))
    return _HOST_TENSORS[key]


METRIC = "hif4_resq_linear TFLOP/s & GB/s at 1 B200; % of FP4-tensor/HBM roofline"
HEADLINE_CONFIG = 4       # the largest single-GPU configuration (7B prefill, M = 16384)
HEADLINE_PATTERN = "2:4"  # the paper's main variant, Rollout-ResQ-S_2:4
L2_BYTES = 126 * 1024 * 1024
PATTERN_IDS = {"none": 0, "dense": 1, "2:4": 2, "row50": 3, "chan50": 4, "block": 5}
# sparsity sweep: the selecting patterns with 1/4 or 3/4 kept (RESQ_KEEP_QUARTERS)
for _name, _base in (("{}:4", 2), ("row{}", 3), ("chan{}", 4), ("block{}", 5)):
    for _q in (1, 3):
        PATTERN_IDS[_name.format(_q if _base == 2 else 25 * _q)] = _base | (_q << 8)
PATTERN_IDS["block-strip"] = 5 | (1 << 12)  # block selection inside every strip of 32 rows (RESQ_BLOCK_PER_STRIP)
PATTERN_NAMES = {v: k for k, v in PATTERN_IDS.items()}
RHO = {0: 0.0, 1: 1.0, 2: 0.5, 3: 0.5, 4: 0.5, 5: 0.5}
RHO.update({p: ((p >> 8) & 0xF) / 4.0 if (p >> 8) & 0xF else 0.5 for p in PATTERN_IDS.values() if p >> 8})
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of ONE launch of the dominant GEMM kernel from ncu captures
# of single layers (summaries with their commands under profiles/), keyed by (config, layer, pattern id, format)
NCU_TRAFFIC = {
    (4, "gate_up", 2, "hif4"): {"bytes": 3.53e9, "source": "profiles/gemm_pair_kernel_7b-prefill-gate_up_dram.md"},
    (4, "qkv", 2, "hif4"): {"bytes": 3.21e8, "source": "profiles/gemm_pair_kernel_7b-prefill-qkv_2to4.md"},
}
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


def gemm_bytes(M, N, K, pattern, fmt):
    """Algorithmic bytes of the GEMM launch alone: packed W, packed Q(X), the packed (2:4: compressed) residual, bf16 Y."""
    side = 0.5625 if fmt == "hif4" else 0.53125
    res = {0: 0.0, 1: side, 2: side - 0.125}.get(pattern & 0xFF, side - 0.125)
    return side * N * K + (side + res) * M * K + 2.0 * M * N


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

    def window(self, t0: float, t1: float):
        """Summary of the samples taken between two wall-clock instants (the sampler keeps running)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        rows = [r for (t, r) in list(self.rows) if t0 - 0.05 <= t <= t1 + 0.15 and len(r) >= 9]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm = [float(r[1]) for r in rows]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({n for r in rows for n, v in zip(names, r[5:9]) if v.lower().startswith("active")})
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": float(rows[0][2]), "reasons": reasons,
                "samples": len(rows), "power_w_max": max(float(r[3]) for r in rows)}

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass


# ----------------------------------------------------------------------------- CPU oracle timing

def oracle_sample(cfg, budget_s):
    """A bounded sample of the workload for the CPU oracle: every layer of the config, the first rows of X (all of
    them if that fits the budget).  Returns (rows, [(X f32, W f32, spec)])."""
    import oracle
    from workloads import bf16_bits_to_f32
    threads = oracle.num_threads()
    macs_per_row = sum(2.0 * l.K * l.N for l in cfg.layers)          # two fp64 sweeps per output element
    rate = 0.6e9 * threads                                            # rough fp64 MAC/s of the plain triple loop
    rows = int(max(32, min(cfg.M, budget_s * rate / macs_per_row)))
    rows -= rows % 32
    tensors = [(bf16_bits_to_f32(make_activation(cfg, li, M=rows)), bf16_bits_to_f32(make_weight(cfg, li)), spec)
               for li, spec in enumerate(cfg.layers)]
    return rows, tensors


def time_oracle(cfg, pattern, fmt, rows, tensors):
    """Times the oracle, as it stands, on the sample.  Returns (TFLOP/s, cores, description, seconds)."""
    import oracle
    flops, dt = 0.0, 0.0
    for x, w, spec in tensors:
        t0 = time.perf_counter()
        oracle.resq_linear(x, w, pattern, fmt, want_abs=False)
        dt += time.perf_counter() - t0
        flops += layer_flops(rows, spec.N, spec.K, pattern)
    sample = (f"{cfg.name}: all {len(cfg.layers)} layers, first {rows} of {cfg.M} token rows "
              f"(weight packing, quantizer, masks and fp64 product all timed)")
    return flops / dt / 1e12, oracle.num_threads(), sample, dt


# ----------------------------------------------------------------------------- one workload on the device

class Workload:
    """The tensors of one configuration on the device, and the step over its layers."""

    def __init__(self, rq, torch, dev, cfg, pattern, fmt, out_dtype, host_copies=False, group=False):
        self.rq, self.torch, self.dev, self.cfg, self.pattern, self.fmt = rq, torch, dev, cfg, pattern, fmt
        self.group = group
        self.layers = []
        w_bytes_total = 0
        for li, spec in enumerate(cfg.layers):
            xb = make_activation(cfg, li)
            wb = make_weight(cfg, li)
            x_host = torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16)
            if host_copies:
                x_host = x_host.pin_memory()
            w_dev = torch.from_numpy(wb.view(np.int16)).view(torch.bfloat16).to(dev)
            wc, ws = rq.pack_weight(w_dev, fmt)
            del w_dev
            w_bytes_total += wc.numel() + ws.numel() * ws.element_size()
            self.layers.append({"spec": spec, "x_host": x_host, "wc": wc, "ws": ws})
        # rotate over enough copies of the packed weights that a step never finds them in L2
        act_bytes = sum(cfg.M * l.K * 2 for l in cfg.layers)
        n_sets = max(2, int(np.ceil(1.5 * L2_BYTES / max(1, w_bytes_total + act_bytes))))
        self.n_sets = n_sets = min(n_sets, 16)
        for L in self.layers:
            spec = L["spec"]
            L["w_sets"] = [(L["wc"], L["ws"])] + [(L["wc"].clone(), L["ws"].clone()) for _ in range(n_sets - 1)]
            L["x_sets"] = [L["x_host"].to(dev) for _ in range(n_sets)]
            L["y"] = torch.empty((cfg.M, spec.N), dtype=out_dtype, device=dev)
            L["work"] = rq.alloc_workspace(rq.resq_workspace_bytes(cfg.M, spec.N, spec.K, pattern, fmt), dev)
            if host_copies:
                L["y_host"] = torch.empty((cfg.M, spec.N), dtype=out_dtype).pin_memory()
                L["x_stage"] = torch.empty_like(L["x_sets"][0])
        if group:  # the layers of a step as one *_resq_linear_group call (one quantizer launch, one GEMM launch)
            self.group_problems = [[(L["x_sets"][k], L["w_sets"][k][0], L["w_sets"][k][1], L["y"]) for L in self.layers]
                                   for k in range(n_sets)]
            self.group_work = rq.alloc_workspace(rq.resq_group_workspace_bytes(self.group_problems[0], pattern, fmt, out_dtype), dev)
        self.out_dtype = out_dtype
        self.l2_note = (f"rotating {n_sets} copies of weights and activations "
                        f"({n_sets * (w_bytes_total + act_bytes) / 1e6:.0f} MB > 126 MB L2)")
        self.w_bytes_total = w_bytes_total
        self.graphs = []
        self.flops_step = sum(layer_flops(cfg.M, L["spec"].N, L["spec"].K, pattern) for L in self.layers)
        self.bytes_step = sum(layer_bytes(cfg.M, L["spec"].N, L["spec"].K, pattern, fmt) for L in self.layers)

    def step(self, i):
        k = i % self.n_sets
        if self.group:
            self.rq.resq_linear_group(self.group_problems[k], self.pattern, self.fmt, out_dtype=self.out_dtype,
                                      workspace=self.group_work)
            return
        for L in self.layers:
            wc, ws = L["w_sets"][k]
            self.rq.resq_linear(L["x_sets"][k], wc, ws, self.pattern, self.fmt, Y=L["y"], workspace=L["work"])

    def check(self):
        if self.group:
            if self.rq.check(self.group_work) != 0:
                raise SystemExit("device status: " + self.rq.last_error())
            return
        for L in self.layers:
            if self.rq.check(L["work"]) != 0:
                raise SystemExit("device status: " + self.rq.last_error())

    # One CUDA graph per rotation set: at decode sizes the step is a handful of short kernels and the host
    # (tensor-map encoding, launches) would otherwise be the bottleneck.  Everything the library enqueues
    # is capturable; attributes were set during warm-up.
    def build_graphs(self, fn=None, into=None):
        torch = self.torch
        into = self.graphs if into is None else into
        fn = fn or self.step
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for k in range(self.n_sets):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    fn(k)
                into.append(g)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()

    def step_graph(self, i):
        self.graphs[i % self.n_sets].replay()

    def profile(self, steps):
        """Per-kernel device time: CUDA events around every launch on the launching stream (a separate pass: the event
        records serialize the kernels and switch the programmatic dependent launch off, so these are upper bounds)."""
        rq, torch = self.rq, self.torch
        rq.profile_enable(True)
        rq.profile_read()
        torch.cuda.synchronize()
        per_layer = []
        for L in self.layers:
            for i in range(steps):
                wc, ws = L["w_sets"][i % self.n_sets]
                rq.resq_linear(L["x_sets"][i % self.n_sets], wc, ws, self.pattern, self.fmt, Y=L["y"], workspace=L["work"])
            torch.cuda.synchronize()
            pr = rq.profile_read()
            per_layer.append({k: (v[0] / steps, v[1] // steps) for k, v in pr.items()})
        rq.profile_enable(False)
        return per_layer

    def free(self):
        self.graphs.clear()
        self.layers.clear()
        self.torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=HEADLINE_CONFIG,
                    help="index into the workload configs (default 4: 7B prefill, the largest single-GPU configuration)")
    ap.add_argument("--pattern", default=None,
                    help="none|dense|2:4|row50|chan50|block (default: 2:4 on config 4, else the config's); sparsity sweep: "
                         "1:4|3:4|row25|row75|chan25|chan75|block25|block75|block-strip")
    ap.add_argument("--format", default="hif4", choices=["hif4", "mxfp4"])
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--out-dtype", default="bf16", choices=["bf16", "f32"])
    ap.add_argument("--layers", default=None, help="comma-separated subset of the config's layers (profiling aid)")
    ap.add_argument("--tokens", type=int, default=None, help="override M (profiling aid; not the benchmark workload)")
    ap.add_argument("--skip-e2e", action="store_true", help="skip the end-to-end and per-kernel passes (profiling aid)")
    ap.add_argument("--headline-only", action="store_true", help="skip per_config / per_pattern / sweeps")
    ap.add_argument("--group", action="store_true",
                    help="run the step's layers as one *_resq_linear_group call (row-local selections only)")
    ap.add_argument("--quantizer-sweep", action="store_true",
                    help="only the bandwidth sweep of *_quantize_act over M x K (table on stderr and one JSON line)")
    ap.add_argument("--accuracy-contrast", action="store_true",
                    help="relative error of plain FP4, the rotation baseline and the residual variants against the exact "
                         "bf16 product on the config's synthetic outlier tensors (no timing)")
    ap.add_argument("--no-graph", action="store_true", help="launch eagerly instead of replaying a CUDA graph per step")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--verbose", action="store_true")
    args = ap.parse_args()

    cfg = CONFIGS[args.config]
    subset = bool(args.layers or args.tokens)
    if subset:
        keep = args.layers.split(",") if args.layers else [l.name for l in cfg.layers]
        cfg = dataclasses.replace(cfg, layers=tuple(l for l in cfg.layers if l.name in keep),
                                  M=args.tokens or cfg.M, name=cfg.name + " (subset)")
    if args.pattern:
        pattern = PATTERN_IDS[args.pattern]
    else:
        pattern = PATTERN_IDS[HEADLINE_PATTERN] if args.config == HEADLINE_CONFIG else cfg.patterns[0]
    pattern_name = PATTERN_NAMES[pattern]
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    config_desc = {
        "workload": f"config {args.config} ({cfg.name}): M={cfg.M}, layers " + ", ".join(f"{l.name} {l.K}->{l.N}" for l in cfg.layers),
        "pattern": pattern_name, "format": args.format, "out_dtype": args.out_dtype,
        "parallelism": "replicas only (one independent copy of the step per GPU)",
    }

    if args.impl == "reference":
        if rank != 0:
            return
        rows, tensors = oracle_sample(cfg, budget_s=8.0)
        vals, info = [], None
        for _ in range(max(1, min(args.warmup, 1))):
            time_oracle(cfg, pattern, args.format, rows, tensors)
        for _ in range(max(1, min(args.steps, 3))):
            info = time_oracle(cfg, pattern, args.format, rows, tensors)
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
    peaks, peak_kind = load_peaks()

    def quantizer_sweep(fmt, Ms, verbose):
        """*_quantize_act alone: read bf16 X, write packed codes + metadata; rotating inputs larger than L2."""
        bpe = 2.0 + (0.5625 if fmt == "hif4" else 0.53125)
        rows = []
        for K in (2048, 18944):
            for M in Ms:
                nbuf = min(64, max(2, int(np.ceil(1.5 * L2_BYTES / (M * K * 2)))))
                xs = [torch.randn((M, K), device=dev, dtype=torch.float32).to(torch.bfloat16) for _ in range(nbuf)]
                for i in range(3):
                    rq.quantize_act(xs[i % nbuf], fmt)
                torch.cuda.synchronize()
                reps = max(10, min(200, int(2e9 / (M * K * bpe))))
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for i in range(reps):
                    rq.quantize_act(xs[i % nbuf], fmt)
                e1.record()
                torch.cuda.synchronize()
                us = e0.elapsed_time(e1) * 1e3 / reps
                gbs = M * K * bpe / (us * 1e-6) / 1e9
                rows.append({"M": M, "K": K, "us": round(us, 2), "GB/s": round(gbs, 1), "frac_of_hbm": round(gbs / peaks["hbm_gbs"], 4)})
                if verbose:
                    print(f"[quantize_act {fmt}] M={M:6d} K={K:6d}  {us:9.1f} us  {gbs:8.1f} GB/s  "
                          f"{100 * gbs / peaks['hbm_gbs']:5.1f} % of {peak_kind} copy rate", file=sys.stderr)
                del xs
        return bpe, rows

    if args.quantizer_sweep:
        bpe, rows = quantizer_sweep(fmt, (256, 512, 1024, 2048, 4096, 8192, 16384, 32768), True)
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

    use_graph = not args.no_graph
    warmup = max(3, args.warmup)

    def tensor_peak_for(fmt_, clocks):
        """Denominator of the GEMM roofline: the measured bf16 peak -- the sustained figure when the clock record of
        the timed region shows the power-capped regime (sw_power_cap active or SM clock well below its maximum), the
        burst figure otherwise; the block-scaled FP4 route takes it times the nominal FP4 : bf16 ratio (9 : 2.25)."""
        capped = bool(clocks) and clocks.get("sm_mhz") and (
            "sw_power_cap" in clocks.get("reasons", []) or clocks["sm_mhz"] < 0.85 * clocks["sm_max_mhz"])
        key = "bf16_tflops_sustained" if capped and peaks.get("bf16_tflops_sustained") else "bf16_tflops"
        p = float(peaks[key])
        src = f"bf16 {'sustained' if key.endswith('sustained') else 'burst'}, of {peak_kind}"
        if fmt_ == "mxfp4":
            return p * 4.0, src + " x 4 (nominal FP4 : bf16 ratio)"
        return p, src

    def measure(cfg_, pattern_, fmt_, steps, sampler=None, e2e=False, verbose=False, group=False):
        """Times `steps` steps of one workload (value), then the per-kernel pass; optionally the end-to-end pass."""
        wl = Workload(rq, torch, dev, cfg_, pattern_, fmt_, out_dtype, host_copies=e2e, group=group)
        for i in range(warmup):
            wl.step(i)
        wl.check()
        launches0 = rq.kernel_launches()
        wl.step(0)
        launches_per_step = rq.kernel_launches() - launches0
        run_step = wl.step
        if use_graph:
            wl.build_graphs()
            for i in range(3):
                wl.step_graph(i)
            run_step = wl.step_graph
        ms, t0, t1 = timed(run_step, steps)
        # keep the GPU busy a little longer so that the 100 ms sampler certainly sees the loaded state
        clocks = None
        if sampler is not None:
            t_load0 = time.time()
            while time.time() - t_load0 < 0.6:
                for i in range(max(1, min(20, int(20.0 / max(ms / steps, 1e-3))))):
                    run_step(i)
                torch.cuda.synchronize()
            clocks = sampler.window(t0, time.time())
        wl.check()
        ms_per_step = ms / steps
        res = {
            "ms_per_step": ms_per_step, "launches_per_step": int(launches_per_step),
            "tflops": world * wl.flops_step / (ms_per_step * 1e-3) / 1e12,
            "gbs": world * wl.bytes_step / (ms_per_step * 1e-3) / 1e9,
            "clocks": clocks, "l2": wl.l2_note, "flops_step": wl.flops_step, "bytes_step": wl.bytes_step,
        }
        if not args.skip_e2e and not group:
            per_layer = wl.profile(min(steps, 10))
            kinds = ("quantize", "select", "gemm", "splitk_reduce")
            tot = {k: sum(pl[k][0] for pl in per_layer) for k in kinds}
            n = {k: sum(pl[k][1] for pl in per_layer) for k in kinds}
            kernel_ms = sum(tot.values())
            res.update({"gemm_ms": tot["gemm"], "gemm_launches": n["gemm"], "quant_ms": tot["quantize"], "quant_launches": n["quantize"],
                        "select_ms": tot["select"], "reduce_ms": tot["splitk_reduce"], "kernel_ms": kernel_ms,
                        "per_layer": [{"layer": L["spec"].name, "K": L["spec"].K, "N": L["spec"].N,
                                       "quant_us": round(pl["quantize"][0] * 1e3, 1), "select_us": round(pl["select"][0] * 1e3, 1),
                                       "gemm_us": round((pl["gemm"][0] + pl["splitk_reduce"][0]) * 1e3, 1),
                                       "gemm_tflops": round(layer_flops(cfg_.M, L["spec"].N, L["spec"].K, pattern_) /
                                                            max(1e-9, (pl["gemm"][0] + pl["splitk_reduce"][0]) * 1e-3) / 1e12, 1)}
                                      for L, pl in zip(wl.layers, per_layer)]})
            if verbose:
                for row in res["per_layer"]:
                    print(f"[layer {row['layer']:8s}] K={row['K']:6d} N={row['N']:6d}  quant {row['quant_us']:8.1f} us  "
                          f"select {row['select_us']:7.1f} us  gemm {row['gemm_us']:8.1f} us  {row['gemm_tflops']:7.1f} TFLOP/s",
                          file=sys.stderr)
        if e2e:
            res["e2e"] = measure_e2e(wl, steps)
        wl.free()
        del wl
        return res

    def measure_e2e(wl, steps):
        # End to end: every step copies each layer's activations from pinned host memory, runs the layer through the
        # public call and reads its output back.  The layers of a step are independent calls, so their copies run on
        # two copy streams beside the compute stream (input of the next layer and output of the previous one overlap
        # the current layer's kernels); the layer with the largest output goes first.  A step ends when every output
        # is in host memory.  With a selection that is local to a token row, a large layer is called on row chunks (the
        # public call on sub-matrices of X and Y), so that the read-back of a chunk's output overlaps the next chunk's
        # kernels instead of starting after the whole layer: the step is bound by the outputs crossing PCIe.
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        order = sorted(wl.layers, key=lambda L: -L["y"].numel())
        row_local = (wl.pattern & 0xFF) in (0, 1, 2, 3)
        chunk_rows = 4096 if row_local and wl.cfg.M >= 8192 else wl.cfg.M
        chunks = [(r0, min(wl.cfg.M, r0 + chunk_rows)) for r0 in range(0, wl.cfg.M, chunk_rows)]

        def step_e2e(i, capturing=False):
            k = i % wl.n_sets
            main_s = torch.cuda.current_stream()
            s_in.wait_stream(main_s)    # earlier work on the staging buffers is done (previous steps were synchronized)
            for L in order:
                L["ev_in"] = []
                for (r0, r1) in chunks:
                    with torch.cuda.stream(s_in):
                        L["x_stage"][r0:r1].copy_(L["x_host"][r0:r1], non_blocking=True)   # host -> device, pinned
                        L["ev_in"].append(s_in.record_event())
            for L in order:
                wc, ws = L["w_sets"][k]
                for ci, (r0, r1) in enumerate(chunks):
                    main_s.wait_event(L["ev_in"][ci])
                    rq.resq_linear(L["x_stage"][r0:r1], wc, ws, wl.pattern, wl.fmt, Y=L["y"][r0:r1], workspace=L["work"])
                    ev = main_s.record_event()
                    with torch.cuda.stream(s_out):
                        s_out.wait_event(ev)
                        L["y_host"][r0:r1].copy_(L["y"][r0:r1], non_blocking=True)         # device -> host
            if capturing:
                main_s.wait_stream(s_out)   # join the copy branches into the captured stream
            else:
                s_out.synchronize()
                main_s.synchronize()

        for i in range(3):
            step_e2e(i)
        run = step_e2e
        if use_graph:
            graphs = []
            wl.build_graphs(lambda k: step_e2e(k, capturing=True), into=graphs)

            def run(i):
                graphs[i % wl.n_sets].replay()       # copies in, kernels and copies out: one graph launch per step
                torch.cuda.current_stream().synchronize()
            for i in range(3):
                run(i)
        for L in wl.layers:  # the pipelined copies delivered what the device holds
            if not torch.equal(L["y_host"], L["y"].cpu()) or not torch.equal(L["x_stage"].cpu(), L["x_host"]):
                raise RuntimeError(f"end-to-end step: host copy of layer {L['spec'].name} differs from the device tensor")
        ms_e2e, _, _ = timed(run, steps)
        h2d = sum(L["x_host"].numel() * 2 for L in wl.layers)
        d2h = sum(L["y_host"].numel() * L["y_host"].element_size() for L in wl.layers)
        return {"value": world * wl.flops_step / (ms_e2e / steps * 1e-3) / 1e12, "unit": "TFLOP/s",
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / steps,
                "calls_per_layer": len(chunks), "note": "bound by the outputs crossing PCIe: d2h bytes / time = "
                f"{d2h / (ms_e2e / steps * 1e-3) / 1e9:.1f} GB/s"}

    def gemm_roofline(res, fmt_):
        """Roofline object of the dominant kernel (the GEMM) from a measure() result."""
        if "gemm_ms" not in res:
            return None
        tensor_peak, peak_src = tensor_peak_for(fmt_, res.get("clocks"))
        # the event-bracketed durations are upper bounds; the step itself bounds them from above as well
        gemm_ms = min(res["gemm_ms"] + res["reduce_ms"], res["ms_per_step"])
        bracketed = res["gemm_ms"] + res["reduce_ms"] > res["ms_per_step"]
        t = res["flops_step"] / (gemm_ms * 1e-3) / 1e12
        return {"bound": "tensor", "achieved": t, "peak": tensor_peak, "unit": "TFLOP/s", "frac": t / tensor_peak,
                "peak_source": peak_src,
                "duration": "sum of the GEMM launches of a step, CUDA events around every launch" +
                            (" (exceeded the graph-replayed step: the whole step time is used, an upper bound)" if bracketed else ""),
                "gemm_ms_per_step": gemm_ms, "launches_per_step": res["gemm_launches"],
                "avg_launch_us": gemm_ms * 1e3 / max(1, res["gemm_launches"]),
                "quantizer_avg_launch_us": res["quant_ms"] * 1e3 / max(1, res["quant_launches"]),
                "quantizer_share_of_kernel_time": res["quant_ms"] / max(1e-9, res["kernel_ms"]),
                "select_share_of_kernel_time": res["select_ms"] / max(1e-9, res["kernel_ms"]),
                "hbm_frac_of_step": res["gbs"] / world / peaks["hbm_gbs"],
                "frac_of_bf16_burst": t / (peaks["bf16_tflops"] * (4.0 if fmt_ == "mxfp4" else 1.0)),
                "frac_of_fp8_nominal": t / 4500.0, "frac_of_fp4_nominal": t / 9000.0}

    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.25)

    # ---- headline workload
    head = measure(cfg, pattern, fmt, args.steps, sampler=sampler, e2e=not args.skip_e2e and not args.group, verbose=args.verbose,
                   group=args.group)
    if args.group:
        config_desc["call"] = "one *_resq_linear_group call per step"
    config_desc["l2"] = head["l2"]
    config_desc["launch"] = "one CUDA graph replay per step" if use_graph else "eager launches"
    if args.skip_e2e or args.group:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": head["tflops"], "unit": "TFLOP/s", "ms_per_step": head["ms_per_step"],
                              "config": config_desc, "note": "profiling aid run: no e2e / roofline passes"}))
        if sampler:
            sampler.stop()
        return
    roofline = gemm_roofline(head, fmt)
    if fmt == "mxfp4":
        roofline["kernel"] = "gemm_mxfp4_native_kernel (tcgen05.mma kind::mxf4.block_scale on packed E2M1 codes; bf16 route for some layers)"
    else:
        roofline["kernel"] = "gemm_pair_kernel (tcgen05.mma cta_group::2 kind::f16 on in-kernel bf16-expanded 4-bit weights)"
    dom = max(head["per_layer"], key=lambda r: r["gemm_us"])
    tr = NCU_TRAFFIC.get((args.config, dom["layer"], pattern, fmt)) if not subset else None
    roofline["traffic"] = tr["bytes"] if tr else None
    roofline["traffic_source"] = (tr["source"] if tr else "no ncu capture of this workload's dominant launch") + \
        f"; dominant launch: {dom['layer']}, algorithmic bytes {gemm_bytes(cfg.M, dom['N'], dom['K'], pattern, fmt):.4g}"
    roofline["per_layer"] = head["per_layer"]

    extras = {}
    if rank == 0 and world == 1 and not args.headline_only and not subset:
        n_small = max(10, min(args.steps, 20))
        # ---- the other configurations with their named patterns (configs 0-3; the headline is config 4)
        per_config = []
        for ci in range(len(CONFIGS)):
            if ci == args.config:
                continue
            c = CONFIGS[ci]
            r = measure(c, c.patterns[0], "hif4", n_small, sampler=sampler)
            rf = gemm_roofline(r, "hif4")
            grouped = None
            if c.patterns[0] in (0, 1, 2) and c.M <= 1024:  # a row-local selection at decode size: also as one grouped call
                rg = measure(c, c.patterns[0], "hif4", n_small, group=True)
                grouped = {"ms_per_step": rg["ms_per_step"], "tflops": rg["tflops"], "launches_per_step": rg["launches_per_step"],
                           "frac_of_bf16_burst": rg["tflops"] / peaks["bf16_tflops"],
                           "call": "hif4_resq_linear_group over the step's layers (one quantizer launch, one GEMM launch)"}
            per_config.append({"config": ci, "name": c.name, "M": c.M, "pattern": PATTERN_NAMES[c.patterns[0]], "format": "hif4",
                               "grouped": grouped,
                               "ms_per_step": r["ms_per_step"], "tflops": r["tflops"], "gb_per_s": r["gbs"],
                               "gemm_frac_of_peak": rf["frac"], "peak_source": rf["peak_source"],
                               "quantizer_share": rf["quantizer_share_of_kernel_time"], "select_share": rf["select_share_of_kernel_time"],
                               "launches_per_step": r["launches_per_step"], "clocks": r["clocks"], "per_layer": r["per_layer"]})
        extras["per_config"] = per_config
        # ---- residual patterns and the MXFP4 twin on the headline workload
        per_pattern = []
        for name, f in (("none", "hif4"), ("dense", "hif4"), ("row50", "hif4"), ("chan50", "hif4"), ("block", "hif4"),
                        ("2:4", "mxfp4"), ("dense", "mxfp4")):
            if PATTERN_IDS[name] == pattern and f == fmt:
                continue
            r = measure(cfg, PATTERN_IDS[name], f, max(3, min(args.steps, 5)), sampler=sampler)
            rf = gemm_roofline(r, f)
            per_pattern.append({"pattern": name, "format": f, "ms_per_step": r["ms_per_step"], "tflops": r["tflops"],
                                "gemm_ms_per_step": rf["gemm_ms_per_step"], "gemm_frac_of_peak": rf["frac"],
                                "peak_source": rf["peak_source"], "quant_ms": r["quant_ms"], "select_ms": r["select_ms"]})
        extras["per_pattern"] = per_pattern
        none = next((p for p in per_pattern if p["pattern"] == "none" and p["format"] == fmt), None)
        if none:
            extras["residual_overhead_over_plain"] = {
                "whole_step": head["ms_per_step"] / none["ms_per_step"] - 1.0,
                "gemm_only": roofline["gemm_ms_per_step"] / none["gemm_ms_per_step"] - 1.0, "pattern": pattern_name}
        # ---- true decode: M = 16 ... 128 on the 3B layers, where weight streaming from HBM is the roof
        sweep = []
        c1 = CONFIGS[1]
        for M in (16, 32, 64, 128, 256):
            cM = dataclasses.replace(c1, M=M, name=f"{c1.name} M={M}")
            r = measure(cM, PATTERN_IDS["2:4"], "hif4", n_small)
            rg = measure(cM, PATTERN_IDS["2:4"], "hif4", n_small, group=True)
            sweep.append({"M": M, "us_per_step": r["ms_per_step"] * 1e3, "tflops": r["tflops"], "gb_per_s": r["gbs"],
                          "frac_of_hbm": r["gbs"] / peaks["hbm_gbs"], "launches_per_step": r["launches_per_step"],
                          "grouped_us_per_step": rg["ms_per_step"] * 1e3, "grouped_tflops": rg["tflops"],
                          "grouped_frac_of_hbm": rg["gbs"] / peaks["hbm_gbs"], "grouped_launches_per_step": rg["launches_per_step"]})
        extras["decode_sweep"] = {"workload": "config 1 layers, S_2:4, HiF4; algorithmic bytes = bf16 X + packed W + bf16 Y; "
                                              "per-layer calls, and the four layers as one grouped call",
                                  "hbm_peak_gbs": peaks["hbm_gbs"], "points": sweep}
        # ---- quantizer alone
        bpe, rows = quantizer_sweep("hif4", (256, 1024, 4096, 16384, 32768), args.verbose)
        extras["quantizer_sweep"] = {"kernel": "hif4_quantize_act", "bytes_per_element": bpe, "hbm_peak_gbs": peaks["hbm_gbs"],
                                     "best": max(rows, key=lambda r: r["GB/s"]), "worst": min(rows, key=lambda r: r["GB/s"]),
                                     "points": rows}
    if sampler:
        sampler.stop()

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        rows, tensors = oracle_sample(cfg, budget_s=20.0)
        v, cores, sample, dt = time_oracle(cfg, pattern, fmt, rows, tensors)
        cpu_baseline = {"value": v, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample,
                        "seconds": dt}

    if rank == 0:
        line = {
            "metric": METRIC, "value": head["tflops"], "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if fmt == "hif4" else "fp4 (e2m1, ue8m0 block scales) / bf16",
            "data": "synthetic", "config": config_desc,
            "gb_per_s": head["gbs"], "clocks": head["clocks"], "e2e": head["e2e"],
            "gpu_launches": int(head["launches_per_step"] * args.steps), "roofline": roofline, "cpu_baseline": cpu_baseline,
        }
        line.update(extras)
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
