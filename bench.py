#!/usr/bin/env python
"""Benchmark of the quantized UNet layer sweep (one JSON line on stdout).

A step is one pass over every quantizable layer of the SDXL-turbo-shaped 512px UNet
(794 layers) at image batch B, each layer at the widths its bit table assigns
(default: W4A8 with 10% of the layers at W8A8).  Weights are distinct per layer
(1.3 GB packed, far larger than L2); inputs are seeded and synthetic.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--batch B] [--table w4a8|a16]
  python bench.py --impl reference ...    # the CPU oracle on a bounded sample

With N > 1 (launched by torch.distributed.run) every rank runs the same sweep on its own
images: independent replicas, no data-path collective, weak scaling.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "unet_layer_sweep_throughput"
UNIT = "TOP/s"
INT8_TO_BF16_NOMINAL = 2.0  # dense int8 : bf16 tensor throughput of the part (4.5 : 2.25 POP/s)


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference", "fp16_library"],
                    help="ours: the CUDA library; reference: the CPU oracle; fp16_library: the same layers at fp16 through "
                         "torch's vendor libraries, as context for the paper's speed-up over FP16")
    ap.add_argument("--batch", type=int, default=4)
    ap.add_argument("--table", default="w4a8", choices=["w4a8", "a16"])
    ap.add_argument("--tokens", type=int, default=0,
                    help="weight-bound regime: only the linear layers of the a16 table, each on this many rows "
                         "(e.g. 16); reports the weight stream in GB/s against the HBM roofline")
    ap.add_argument("--low-bits", type=int, default=3, choices=[2, 3],
                    help="a16 table: lowest weight width; 2 gives the paper's candidate widths {2, 4, 8} at the same "
                         "3.66-bit average (the default run uses {3, 4, 8})")
    ap.add_argument("--act-asym", action="store_true",
                    help="w4a8 table: asymmetric 8-bit activations on linear layers and 3x3 convolutions (Sec. 4.1); the "
                         "default run, which the headline number is quoted on, uses symmetric ones everywhere")
    ap.add_argument("--shortcut-split", action="store_true",
                    help="w4a8 table: the resnet convolutions of the up path that read a [hidden | skip] concatenation keep "
                         "one activation scale per branch (Sec. 4.1, shortcut-splitting); not part of the default run")
    ap.add_argument("--share-qkv-quant", action="store_true",
                    help="w4a8 table: the q, k and v projections of every self-attention block share one quantization "
                         "pass of their common input (int8 codes kept, three GEMMs on them); not part of the default run")
    ap.add_argument("--fuse-projections", action="store_true",
                    help="q, k, v of every self-attention block and K, V of every cross-attention block run as one stacked "
                         "layer where the bit table gives them equal widths (same operations, fewer layers); not part of "
                         "the default run")
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the per-configuration records, the weight-bound layers and the two weight-only sweeps "
                         "that the default run appends to its line")
    return ap.parse_args()


def workload_name(args):
    if args.tokens > 0:
        return f"unet_linear_sweep_{args.table}_{args.tokens}tokens" + ("_w248" if args.low_bits == 2 else "")
    return f"unet_sweep_sdxl512_{args.table}_b{args.batch}" + ("_asym_acts" if args.act_asym else "") + \
        ("_shortcut_split" if args.shortcut_split else "") + ("_shared_qkv_quant" if args.share_qkv_quant else "") + ("_fused_projections" if args.fuse_projections else "") + \
        ("_w248" if (args.low_bits == 2 and args.table == "a16") else "")


# ----------------------------------------------------------------------------- peaks

def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows = []
        self.proc = None
        self.gpu = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.thread.join(timeout=2)
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 6:
                continue
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
            except ValueError:
                continue
            for name, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# ----------------------------------------------------------------------------- reference arm (CPU oracle)

def oracle_sample_layers(table: str, batch: int, mac_budget: float):
    """A bounded sample of the sweep for the CPU oracle: layers of distinct shapes, in census
    order, until the MAC budget is spent (at least one layer)."""
    from paper_2405_17873_b200 import synth
    layers = synth.unet_layers()
    (synth.assign_bits_w4a8 if table == "w4a8" else synth.assign_bits_weight_only)(layers)
    seen, picked, macs = set(), [], 0.0
    # cheapest distinct shapes first, so that a small budget still covers several kinds
    order = sorted(layers, key=lambda l: l.ops(batch))
    for l in order:
        key = (l.kind, l.M, l.N, l.K, l.stride, l.w_bits, l.a_bits)
        if key in seen:
            continue
        m = l.ops(batch) / 2
        if picked and macs + m > mac_budget:
            continue
        seen.add(key)
        picked.append(l)
        macs += m
    return picked


def oracle_run_layers(picked, batch: int, prepared=None):
    """One oracle pass over the sample; returns (seconds, ops, prepared inputs)."""
    from oracle import mixdq_oracle as orc
    from paper_2405_17873_b200 import synth
    if prepared is None:
        prepared = []
        for l in picked:
            X, W, b = synth.layer_inputs(l, batch, seed=5000 + l.index)
            W2 = W.reshape(l.N, -1)
            sym = l.a_bits == 8
            s, z = orc.weight_minmax_params(W2, l.w_bits, sym)
            codes = orc.quantize_weights(W2, l.w_bits, s, None if sym else z)
            extra = {}
            if l.a_bits == 8:
                if l.kind == "bos_kv":
                    extra["sx"] = orc.crossattn_act_scale(X)
                    extra["bos"] = orc.bos_row(X[0, 0], W2)
                else:
                    extra["sx"] = orc.act_scale(orc.act_absmax(X), 8)
            prepared.append((l, X, codes, s, None if sym else z, b, extra))
    t0 = time.perf_counter()
    ops = 0
    for l, X, codes, s, z, b, extra in prepared:
        if l.a_bits == 8:
            if l.kind == "conv3x3":
                orc.conv3x3_a8(X, codes.reshape(l.N, 3, 3, l.Cin), s, extra["sx"], b, l.stride)
            elif l.kind == "bos_kv":
                orc.crossattn_kv(X, codes, s, extra["sx"], extra["bos"])
            else:
                orc.linear_a8(X.reshape(-1, l.K), codes, s, extra["sx"], b)
        else:
            if l.kind == "conv3x3":
                orc.conv3x3_a16(X, codes.reshape(l.N, 3, 3, l.Cin), s, z, b, l.stride)
            else:
                orc.linear_a16(X.reshape(-1, l.K), codes, s, z, None if l.kind == "bos_kv" else b)
        ops += l.ops(batch)
    return time.perf_counter() - t0, ops, prepared


def oracle_rate_estimate(table: str) -> float:
    """MAC/s of the oracle on this host, from one small layer."""
    from oracle import mixdq_oracle as orc
    import numpy as np
    rng = np.random.default_rng(0)
    M, N, K = 128, 320, 640
    X = rng.normal(size=(M, K)).astype(np.float16)
    codes = rng.integers(0, 8, size=(N, K)).astype(np.int16)
    s = np.ones(N, np.float32)
    t0 = time.perf_counter()
    if table == "w4a8":
        orc.linear_a8(X, codes, s, np.float32(0.03), None)
    else:
        orc.linear_a16(X, codes, s, np.zeros(N, np.int32), None)
    return M * N * K / (time.perf_counter() - t0)


def cpu_baseline(table: str, batch: int, seconds: float):
    from oracle import mixdq_oracle as orc
    rate = oracle_rate_estimate(table)
    picked = oracle_sample_layers(table, batch, rate * seconds)
    dt, ops, _ = oracle_run_layers(picked, batch)
    return {"value": ops / dt / 1e12, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
            "sample": f"{len(picked)} layers of distinct shapes of the sweep ({ops / 2e9:.1f} GMAC), one pass, "
                      f"{dt:.1f} s"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import mixdq_oracle as orc
    total = args.steps + args.warmup
    rate = oracle_rate_estimate(args.table)
    per_step_s = max(0.02, min(5.0, 120.0 / max(total, 1)))
    picked = oracle_sample_layers(args.table, args.batch, rate * per_step_s)
    prepared = None
    for _ in range(args.warmup):
        _, _, prepared = oracle_run_layers(picked, args.batch, prepared)
    t, ops = 0.0, 0
    for _ in range(args.steps):
        dt, o, prepared = oracle_run_layers(picked, args.batch, prepared)
        t += dt
        ops += o
    value = ops / t / 1e12
    sample = f"{len(picked)} layers of distinct shapes per step ({ops / args.steps / 2e9:.2f} GMAC per step)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8" if args.table == "w4a8" else "f64", "data": "synthetic",
        "config": {"workload": workload_name(args), "table": args.table, "batch": args.batch},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ----------------------------------------------------------------------------- fp16 library comparator

def run_fp16_library(args):
    """Context for the paper's speed-up over FP16 (Sec. 4.3): the same 794 layers at fp16 through the vendor
    libraries (torch.nn.functional.linear / conv2d, channels-last), one step as a CUDA graph.  Not part of the
    product path and not the benchmark's arm: it prints its own line with "impl": "fp16_library"."""
    import torch
    import torch.nn.functional as F
    from paper_2405_17873_b200 import synth

    torch.cuda.set_device(0)
    B = args.batch
    layers = synth.unet_layers()
    g = torch.Generator(device="cuda").manual_seed(5)
    xs, work, ops = {}, [], 0
    for l in layers:
        if l.kind in ("conv3x3", "conv1x1"):
            k = 3 if l.kind == "conv3x3" else 1
            key = ("img", l.H, l.Cin)
            if key not in xs:
                x = torch.randn((B, l.Cin, l.H, l.H), generator=g, device="cuda", dtype=torch.float16)
                xs[key] = x.contiguous(memory_format=torch.channels_last)
            w = (torch.randn((l.N, l.Cin, k, k), generator=g, device="cuda", dtype=torch.float32) * 0.02).half()
            w = w.contiguous(memory_format=torch.channels_last)
            bias = (torch.randn((l.N,), generator=g, device="cuda") * 0.01).half()
            work.append(("conv", xs[key], w, bias, l.stride, k // 2))
        else:
            rows = B * synth.TOKENS_PER_PROMPT if l.kind == "bos_kv" else l.M * B
            key = ("rows", rows, l.K)
            if key not in xs:
                xs[key] = torch.randn((rows, l.K), generator=g, device="cuda", dtype=torch.float16)
            w = (torch.randn((l.N, l.K), generator=g, device="cuda", dtype=torch.float32) * 0.02).half()
            bias = None if l.kind == "bos_kv" else (torch.randn((l.N,), generator=g, device="cuda") * 0.01).half()
            work.append(("lin", xs[key], w, bias, 1, 0))
        ops += l.ops(B)

    def step():
        for kind, x, w, b, stride, pad in work:
            if kind == "conv":
                F.conv2d(x, w, b, stride=stride, padding=pad)
            else:
                F.linear(x, w, b)

    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream), torch.no_grad():
        for _ in range(3):
            step()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            step()
        for _ in range(max(args.warmup, 3)):
            graph.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    print(json.dumps({"impl": "fp16_library", "metric": METRIC, "value": ops / (ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                      "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
                      "dtype": "f16", "data": "synthetic",
                      "config": {"workload": f"unet_sweep_sdxl512_fp16_b{B}", "layers": len(layers), "ops_per_step": ops,
                                 "launch": "CUDA graph replay", "library": "torch " + torch.__version__ +
                                 " (cuBLAS / cuDNN), fp16 weights distinct per layer"}}))


# ----------------------------------------------------------------------------- per-configuration records

NOMINAL = {"int8_tops": 4500.0, "f16_tflops": 2250.0, "hbm_gbs": 8000.0}  # dense peaks of the part, for context


def _time_graph(torch, stream, fn, reps=10, rounds=3):
    """Average microseconds of one call of fn, from a CUDA graph of `reps` back-to-back calls replayed `rounds`
    times (events on the launching stream; one untimed replay first)."""
    with torch.cuda.stream(stream):
        fn()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for _ in range(reps):
                fn()
        g.replay()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(rounds):
            g.replay()
        t1.record()
        torch.cuda.synchronize()
    return t0.elapsed_time(t1) * 1e3 / (reps * rounds)


def _fracs(rate, measured, nominal, probe=None):
    d = {"of_measured": round(rate / measured, 4), "of_nominal": round(rate / nominal, 4)}
    if probe:
        d["of_int8_mma_probe"] = round(rate / probe, 4)
    return d


def config_records(torch, mixdq, synth, stream, peaks, probe_int8):
    """One record per stated configuration besides the layer sweep: the single W8A8 linear layer, the weight-only
    trio at 4096 and 16 tokens, the FFN pair in W4A8 / W8A8 at image batch 1 and 4, the BOS-aware K / V
    projections at prompt batch 1 and 8.  Quantization pass + GEMM per call; a graph of ten calls on one set of
    weights (warm L2) unless stated; activation scales computed at set-up."""
    dev = lambda a: torch.from_numpy(a).cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    int8_peak = peaks["bf16_tflops"] * INT8_TO_BF16_NOMINAL
    out = []

    def a8_linear(tag, X, W, b, bits):
        M, K = X.shape
        N = W.shape[0]
        Xd, Wd = dev(X), dev(W)
        s, _ = mixdq.weight_minmax_params(Wd, bits, True)
        pk = mixdq.pack_weights(Wd, bits, s)
        sx = mixdq.act_scale(Xd)
        ws = mixdq.new_workspace(mixdq.workspace_bytes(M, N, K, bits, 8))
        Y = torch.empty((M, N), dtype=torch.float16, device="cuda")
        bd = None if b is None else dev(b)
        us = _time_graph(torch, stream, lambda: mixdq.linear(Xd, pk, N, bits, s, None, 8, sx, bd, ws, status, out=Y))
        tops = 2.0 * M * N * K / us / 1e6
        rows, cols, sp = mixdq.int8_tile_plan(M, N, (K + 127) // 128, bits, with_splits=True)
        out.append({"config": tag, "M": M, "N": N, "K": K, "w_bits": bits, "a_bits": 8, "us": round(us, 2),
                    "tops": round(tops, 1), "bound": "tensor", "l2": "warm",
                    "tile": f"{rows}x{cols}" + (f", reduction over {sp} CTA pairs" if sp > 1 else ""),
                    "frac": _fracs(tops, int8_peak, NOMINAL["int8_tops"], probe_int8)})

    # 1. single linear layer, W8A8
    X, W, b = synth.single_linear(seed=0)
    a8_linear("1: single linear W8A8", X, W, b, 8)
    # 3. FFN pair (GEGLU projection, then 5120 -> 1280) with 1 % outlier channels, image batch 1 and 4
    for B in (1, 4):
        for bits in (4, 8):
            Xf = synth.ffn_input(B, seed=3000 + B)
            a8_linear(f"3: FFN-1 1280->10240 B={B}", Xf, synth.normal_f16((10240, 1280), 0.02, 3100), None, bits)
            Xg = synth.normal_f16((B * 256, 5120), 0.3, 3104)   # the size and rough range of a GEGLU output
            a8_linear(f"3: FFN-2 5120->1280 B={B}", Xg, synth.normal_f16((1280, 5120), 0.02, 3102), None, bits)
    # 4. BOS-aware K / V projections, W8A8
    for B in (1, 8):
        for N in (640, 1280):
            E = synth.text_embedding(B)
            Wk = synth.kv_weight(N, seed=4200 + N)
            Ed, Wd = dev(E), dev(Wk)
            s, _ = mixdq.weight_minmax_params(Wd, 8, True)
            pk = mixdq.pack_weights(Wd, 8, s)
            sx = mixdq.act_scale(Ed.reshape(-1, E.shape[-1]), 77)
            bos = synth.bos_projection(Ed[0, 0], Wd)
            ws = mixdq.new_workspace(mixdq.workspace_bytes(B * 76, N, 2048, 8, 8))
            Y = torch.empty((B, 77, N), dtype=torch.float16, device="cuda")
            us = _time_graph(torch, stream, lambda: mixdq.crossattn_kv(Ed, pk, N, 8, s, sx, bos, ws, status, out=Y))
            tops = 2.0 * B * 76 * N * 2048 / us / 1e6
            out.append({"config": f"4: BOS-aware K/V 2048->{N} B={B}", "M": B * 76, "N": N, "K": 2048, "w_bits": 8,
                        "a_bits": 8, "us": round(us, 2), "tops": round(tops, 1), "bound": "latency (a few tiles)",
                        "l2": "warm", "frac": _fracs(tops, int8_peak, NOMINAL["int8_tops"], probe_int8)})
    # 2. weight-only trio (W3 / W4 / W8, fp16 activations) at 4096 tokens (tensor-bound) and 16 (weight stream)
    for M in (4096, 16):
        for idx in range(3):
            X, W, b, bits = synth.weight_only_layer(idx, M)
            N, K = W.shape
            Xd, Wd = dev(X), dev(W)
            s, z = mixdq.weight_minmax_params(Wd, bits, False)
            pk = mixdq.pack_weights(Wd, bits, s, z)
            Y = torch.empty((M, N), dtype=torch.float16, device="cuda")
            bd = dev(b)
            us = _time_graph(torch, stream, lambda: mixdq.linear(Xd, pk, N, bits, s, z, 16, None, bd, None, status, out=Y))
            rec = {"config": f"2: weight-only {K}->{N} at {M} tokens", "M": M, "N": N, "K": K, "w_bits": bits,
                   "a_bits": 16, "us": round(us, 2), "l2": "warm"}
            if M >= 64:
                tf = 2.0 * M * N * K / us / 1e6
                rec.update({"tflops": round(tf, 1), "bound": "tensor",
                            "frac": _fracs(tf, peaks["bf16_tflops"], NOMINAL["f16_tflops"])})
            else:
                gbs = (pk.numel() + 8 * N + 2 * M * (K + N)) / us / 1e3
                rec.update({"gb_per_s": round(gbs, 1), "bound": "launch latency (under 0.5 MB of weights)",
                            "frac": _fracs(gbs, peaks["hbm_gbs"], NOMINAL["hbm_gbs"])})
            out.append(rec)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return out


def fused_quant_records(torch, mixdq, synth, stream):
    """The W4A8 / W8A8 linear layer as one kernel (activation quantization inside the GEMM) against quantization
    pass + GEMM, both forms forced through their explicit entry points, beside what the planner picks.  Graph of ten
    calls, warm L2.  The one-kernel form's tile width is the planner's where it selects that form, else the
    narrowest that fits one wave (256 when none does)."""
    dev = lambda a: torch.from_numpy(a).cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    out = []
    for (M, N, K) in [(4096, 640, 640), (4096, 640, 320), (1024, 640, 640), (1024, 1280, 640), (1024, 1280, 1280),
                      (16384, 320, 640), (1024, 1280, 5120)]:
        for bits in (4, 8):
            Xd = dev(synth.normal_f16((M, K), 1.0, seed=9000 + K))
            Wd = dev(synth.normal_f16((N, K), 0.02, seed=9100 + N))
            s, _ = mixdq.weight_minmax_params(Wd, bits, True)
            pk = mixdq.pack_weights(Wd, bits, s)
            sx = mixdq.act_scale(Xd)
            ws = mixdq.new_workspace(mixdq.workspace_bytes(M, N, K, bits, 8))
            Y = torch.empty((M, N), dtype=torch.float16, device="cuda")
            xq = torch.empty((M, K), dtype=torch.int8, device="cuda")
            planned = mixdq.linear_fused_quant_tile(M, N, K, bits)
            cols = planned
            if cols == 0:
                fits = [c for c in range(64, 257, 32) if -(-M // 128) * -(-N // c) <= sms]
                cols = fits[0] if fits else 256

            def two():
                mixdq.quantize_acts(Xd, sx, out=xq)
                mixdq.linear_q8(xq, pk, N, bits, s, sx, None, status, out=Y)

            t_two = _time_graph(torch, stream, two)
            t_one = _time_graph(torch, stream, lambda: mixdq.linear_a8_fused_quant(Xd, pk, N, bits, s, sx, None, cols, status, out=Y))
            t_plan = _time_graph(torch, stream, lambda: mixdq.linear(Xd, pk, N, bits, s, None, 8, sx, None, ws, status, out=Y))
            out.append({"M": M, "N": N, "K": K, "w_bits": bits, "two_kernel_us": round(t_two, 2),
                        "one_kernel_us": round(t_one, 2), "one_kernel_tile": f"128x{cols}",
                        "planned": "one kernel" if planned else "two kernels", "planned_us": round(t_plan, 2)})
    return out


def weight_bound_records(torch, mixdq, synth, stream, peaks):
    """The weight-only engine where it is bound by the weight stream: the transformer FFN layers on 16 tokens,
    with as many distinct copies of the packed weights as it takes to exceed L2 several times over, walked
    inside one graph, so that every launch streams its weights from HBM."""
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(11)
    out = []
    for (K, N, bits) in ((1280, 10240, 8), (1280, 10240, 4), (1280, 10240, 3), (5120, 1280, 4), (1280, 1280, 4)):
        W = (torch.randn((N, K), generator=g, device="cuda") * 0.02).half()
        s, z = mixdq.weight_minmax_params(W, bits, False)
        pk0 = mixdq.pack_weights(W, bits, s, z)
        copies = max(4, int(512e6 // pk0.numel()) + 1)
        pks = [pk0.clone() for _ in range(copies)]
        X = torch.randn((16, K), generator=g, device="cuda").half()
        Y = torch.empty((16, N), dtype=torch.float16, device="cuda")
        with torch.cuda.stream(stream):
            mixdq.linear(X, pks[0], N, bits, s, z, 16, None, None, None, status, out=Y)
            torch.cuda.synchronize()
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gr, stream=stream):
                for pk in pks:
                    mixdq.linear(X, pk, N, bits, s, z, 16, None, None, None, status, out=Y)
            gr.replay()
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0.record()
            gr.replay()
            gr.replay()
            t1.record()
            torch.cuda.synchronize()
        us = t0.elapsed_time(t1) * 1e3 / (2 * copies)
        alg = pk0.numel() + 8 * N + 2 * 16 * (K + N)
        gbs = alg / us / 1e3
        out.append({"layer": f"{K}->{N} at 16 tokens", "w_bits": bits, "us": round(us, 2), "gb_per_s": round(gbs, 1),
                    "algorithmic_bytes": alg, "l2": f"cold: {copies} copies of the weights walked in one graph",
                    "frac": _fracs(gbs, peaks["hbm_gbs"], NOMINAL["hbm_gbs"])})
        del pks
    return out


def sub_sweep_record(torch, UNetSweep, stream, peaks, batch, tokens, steps=10):
    """The 3.66-bit weight-only table over the whole network (tokens = 0: image batch `batch`; tokens > 0: every
    linear layer on that many rows), one step as a CUDA graph, `steps` timed replays."""
    sw = UNetSweep(batch, "a16", seed=5, tokens=tokens)
    with torch.cuda.stream(stream):
        sw.step()
        torch.cuda.synchronize()
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr, stream=stream):
            sw.step()
        for _ in range(3):
            gr.replay()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(steps):
            gr.replay()
        t1.record()
        torch.cuda.synchronize()
    ms = t0.elapsed_time(t1) / steps
    rec = {"workload": f"unet_linear_sweep_a16_{tokens}tokens" if tokens else f"unet_sweep_sdxl512_a16_b{batch}",
           "layers": len(sw.layers), "ms_per_step": round(ms, 3), "steps": steps, "device_status": int(sw.status.item()),
           "l2": "weights (distinct per layer) are larger than L2"}
    if tokens:
        alg = sum(sw.algorithmic_bytes(pl) for pl in sw.layers)
        gbs = alg / (ms * 1e-3) / 1e9
        rec.update({"bound": "hbm", "gb_per_s": round(gbs, 1), "algorithmic_bytes_per_step": alg,
                    "frac": _fracs(gbs, peaks["hbm_gbs"], NOMINAL["hbm_gbs"])})
    else:
        tf = sw.total_ops() / (ms * 1e-3) / 1e12
        rec.update({"bound": "tensor", "tflops": round(tf, 1),
                    "frac": _fracs(tf, peaks["bf16_tflops_sustained"], NOMINAL["f16_tflops"])})
    del sw
    torch.cuda.empty_cache()
    return rec


# ----------------------------------------------------------------------------- our arm

def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2405_17873_b200 import build, mixdq, replicas
    from paper_2405_17873_b200.unet_sweep import UNetSweep

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    build.build()
    mixdq.lib()  # fail here, loudly, if the CUDA library is missing

    if args.tokens > 0 and args.table != "a16":
        raise SystemExit("--tokens needs --table a16 (the weight-only engine)")
    sweep = UNetSweep(args.batch, args.table, seed=5 + rank, tokens=args.tokens, act_asym=args.act_asym, low_bits=args.low_bits,
                      shortcut_split=args.shortcut_split, share_qkv_quant=args.share_qkv_quant,
                      fuse_projections=args.fuse_projections)
    tc_layers = [pl for pl in sweep.layers if sweep.uses_tensor_int8(pl)]
    other_layers = [pl for pl in sweep.layers if not sweep.uses_tensor_int8(pl)]
    if args.table == "a16":
        tc_layers, other_layers = [], list(sweep.layers)  # all on the weight-only engine

    # warm-up outside the graphs (also sets kernel attributes), then capture one step as two graphs
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for _ in range(2):
            sweep.step()
    torch.cuda.synchronize()
    graphs, group_launches = [], []
    for group in (tc_layers, other_layers):
        if not group:
            graphs.append(None)
            group_launches.append(0)
            continue
        g = torch.cuda.CUDAGraph()
        before = mixdq.kernel_launches()
        with torch.cuda.graph(g, stream=stream):
            sweep.step(group)
        group_launches.append(mixdq.kernel_launches() - before)   # kernels recorded into the graph
        graphs.append(g)
    g_tc, g_other = graphs
    launches_per_step = sum(group_launches)

    barrier = replicas.barrier

    ev = lambda: torch.cuda.Event(enable_timing=True)

    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3)):
            if g_tc is not None:
                g_tc.replay()
            if g_other is not None:
                g_other.replay()
        torch.cuda.synchronize()

        # ---------------- timed region: inputs resident in HBM
        sampler = ClockSampler(local_rank)
        sampler.start()
        time.sleep(0.3)
        marks = []
        barrier()
        torch.cuda.synchronize()
        start, end = ev(), ev()
        start.record()
        for _ in range(args.steps):
            a, b, c = ev(), ev(), ev()
            a.record()
            if g_tc is not None:
                g_tc.replay()
            b.record()
            if g_other is not None:
                g_other.replay()
            c.record()
            marks.append((a, b, c))
        end.record()
        torch.cuda.synchronize()
        barrier()
        total_ms = start.elapsed_time(end)
        clocks = sampler.stop()
        tc_ms = sum(a.elapsed_time(b) for a, b, _ in marks) / args.steps
        other_ms = sum(b.elapsed_time(c) for _, b, c in marks) / args.steps
        status = int(sweep.status.item())

        # ---------------- end to end: host buffers in, host buffers out, every step
        x_host = {k: torch.empty_like(v, device="cpu").pin_memory().copy_(v) for k, v in sweep.x.items()}
        y_host = {k: torch.empty_like(v, device="cpu").pin_memory() for k, v in sweep.y.items()}
        h2d = sum(v.numel() * 2 for v in x_host.values())
        d2h = sum(v.numel() * 2 for v in y_host.values())

        # Three streams: the host->device copy of step i + 1 and the device->host copy of step i - 1 run
        # beside the kernels of step i.  Copies land in / leave from staging buffers; a device-to-device
        # copy at either end of the step moves them to and from the buffers the graphs are bound to.
        copy_in, copy_out = torch.cuda.Stream(), torch.cuda.Stream()
        x_stage = {k: torch.empty_like(v) for k, v in sweep.x.items()}
        y_stage = {k: torch.empty_like(v) for k, v in sweep.y.items()}
        x_staged, x_taken = torch.cuda.Event(), torch.cuda.Event()
        y_staged, y_taken = torch.cuda.Event(), torch.cuda.Event()

        def stage_inputs():           # host -> staging, on the input-copy stream
            with torch.cuda.stream(copy_in):
                copy_in.wait_event(x_taken)           # the previous contents have been consumed
                for k, v in x_host.items():
                    x_stage[k].copy_(v, non_blocking=True)
                x_staged.record(copy_in)

        def e2e_steps(n):
            x_taken.record(stream)
            y_taken.record(copy_out)
            stage_inputs()
            for i in range(n):
                stream.wait_event(x_staged)
                for k in x_stage:
                    sweep.x[k].copy_(x_stage[k], non_blocking=True)
                x_taken.record(stream)
                if i + 1 < n:
                    stage_inputs()                    # next step's inputs cross PCIe during this step's kernels
                if g_tc is not None:
                    g_tc.replay()
                if g_other is not None:
                    g_other.replay()
                stream.wait_event(y_taken)            # the previous step's outputs have left the staging buffers
                for k in y_stage:
                    y_stage[k].copy_(sweep.y[k], non_blocking=True)
                y_staged.record(stream)
                with torch.cuda.stream(copy_out):
                    copy_out.wait_event(y_staged)
                    for k, v in y_host.items():
                        v.copy_(y_stage[k], non_blocking=True)
                    y_taken.record(copy_out)
            stream.wait_event(y_taken)                # the last outputs are on the host

        e2e_steps(2)
        barrier()
        torch.cuda.synchronize()
        s2, e2 = ev(), ev()
        s2.record()
        e2e_steps(args.e2e_steps)
        e2.record()
        torch.cuda.synchronize()
        barrier()
        e2e_ms = s2.elapsed_time(e2) / args.e2e_steps

    ms_per_step = total_ms / args.steps
    ms_per_step, e2e_ms, tc_ms, other_ms = replicas.max_over_ranks([ms_per_step, e2e_ms, tc_ms, other_ms], "cuda")

    ops_step = sweep.total_ops()
    peaks = measured_peaks()
    # the largest layers one by one (the "large-M" int8 layers the 60 % tensor-roofline target is about): each as
    # a graph of ten back-to-back launches on its own weights (warm L2), against the burst peak, because such a
    # graph is over in a millisecond
    per_layer = None
    probe_int8 = None
    if args.table == "w4a8" and world == 1 and args.tokens == 0:
        # second denominator: back-to-back int8 MMAs on operands resident in shared memory, all SMs
        with torch.cuda.stream(stream):
            probe_int8 = mixdq.probe_mma_loop(1, 64)
        per_layer = []
        burst = peaks["bf16_tflops"] * INT8_TO_BF16_NOMINAL
        for name in ("up64_640#0", "res64_320_320#0", "res32_640_640#0", "up32_1280#0", "res16_1280_1280#0",
                     "res16_2560_1280#0", "ffn1_1280#0", "ffn2_1280#0", "ffn1_640#0", "attn_1280#0"):
            pl = next((q for q in sweep.layers if q.spec.name == name), None)
            if pl is None:
                continue
            reps, rounds = 10, 3
            with torch.cuda.stream(stream):
                g1 = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g1, stream=stream):
                    for _ in range(reps):
                        sweep.run_layer(pl)
                g1.replay()
                t0, t1 = ev(), ev()
                t0.record()
                for _ in range(rounds):
                    g1.replay()
                t1.record()
                torch.cuda.synchronize()
            us = t0.elapsed_time(t1) * 1e3 / (reps * rounds)
            tops = pl.spec.ops(args.batch) / us / 1e6
            kb = 9 * ((pl.spec.Cin + 127) // 128) if pl.spec.kind == "conv3x3" else (pl.spec.K + 127) // 128
            rows, cols, sp = mixdq.int8_tile_plan(pl.spec.rows(args.batch), pl.spec.N, kb, pl.spec.w_bits, with_splits=True)
            per_layer.append({"layer": name, "kind": pl.spec.kind, "M": pl.spec.rows(args.batch), "N": pl.spec.N,
                              "K": pl.spec.K, "w_bits": pl.spec.w_bits,
                              "tile": f"{rows}x{cols}" + (f", reduction over {sp} CTA pairs" if sp > 1 else ""),
                              "us": round(us, 2),
                              "tops": round(tops, 1), "frac_of_burst_peak": round(tops / burst, 3),
                              "frac_of_sustained_peak": round(tops / (peaks["bf16_tflops_sustained"] * INT8_TO_BF16_NOMINAL), 3),
                              "frac_of_int8_mma_probe": round(tops / probe_int8, 3),
                              "frac_of_nominal": round(tops / NOMINAL["int8_tops"], 3)})
    if args.table == "w4a8":
        tc_ops = sweep.total_ops(tc_layers)
        achieved = tc_ops / (tc_ms * 1e-3) / 1e12
        peak = peaks["bf16_tflops_sustained"] * INT8_TO_BF16_NOMINAL
        # (no DRAM counter figure here: the kernels have changed since the last capture of a whole step; the
        # algorithmic bytes of the step stand beside it, and per-layer captures are summarised under profiles/)
        traffic = None
        alg_bytes = sum(sweep.algorithmic_bytes(pl) for pl in tc_layers)
        roofline = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TOP/s", "frac": achieved / peak,
                    "traffic": traffic,
                    "kernel": "i8 tcgen05 kind::i8 GEMM kernels (pair_gemm_kernel on two-CTA tiles, tma_gemm_kernel, "
                              "tma_gemm_persistent_kernel) with their quant_kernel pre-pass, all tensor-core int8 layers of "
                              "the step",
                    "peak_source": f"{peaks['source']} bf16 sustained x {INT8_TO_BF16_NOMINAL:g} (nominal int8:bf16)",
                    "frac_of_nominal": achieved / NOMINAL["int8_tops"],
                    "frac_of_int8_mma_probe": (achieved / probe_int8) if probe_int8 else None,
                    "algorithmic_bytes_per_step": alg_bytes,
                    "algorithmic_gb_per_s": alg_bytes / (tc_ms * 1e-3) / 1e9,
                    "launches_per_step": group_launches[0], "layers": len(tc_layers), "ms_per_step": tc_ms}
    elif args.tokens > 0:
        # a few tokens per layer: one stream over the packed weights, bound by HBM
        alg = sum(sweep.algorithmic_bytes(pl) for pl in sweep.layers)
        achieved = alg / (other_ms * 1e-3) / 1e9
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": achieved / peaks["hbm_gbs"], "traffic": None,
                    "kernel": "wo::wo_small_kernel (packed weights streamed once, decoded in registers, mma.sync fp16), "
                              "all layers of the step",
                    "peak_source": f"{peaks['source']} copy bandwidth",
                    "launches_per_step": group_launches[1], "ms_per_step": other_ms,
                    "algorithmic_bytes_per_step": alg}
    else:
        # image batch >= 1 means hundreds of tokens per layer: the weight-only layers run on the
        # fp16 tensor cores (tcgen05 kind::f16) and are bound by that pipe, not by the weight stream
        achieved = ops_step / (other_ms * 1e-3) / 1e12
        peak = peaks["bf16_tflops_sustained"]
        alg = sum(sweep.algorithmic_bytes(pl) for pl in sweep.layers)
        roofline = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                    "traffic": None,
                    "kernel": "weight expansion to fp16 (once per layer call, into the workspace) + pair_gemm_kernel in its "
                              "tcgen05 kind::f16 mode; layers under 256 rows on wo_tc_kernel / wo_kernel; all layers of the step",
                    "peak_source": f"{peaks['source']} bf16 sustained (fp16 has the same nominal rate)",
                    "launches_per_step": group_launches[1], "ms_per_step": other_ms,
                    "algorithmic_gb_per_s": alg / (other_ms * 1e-3) / 1e9}

    if rank == 0:
        out = {
            "metric": METRIC, "value": replicas.whole_job_rate(ops_step, ms_per_step) / 1e12, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int8" if args.table == "w4a8" else "f16",
            "data": "synthetic",
            "config": {"workload": workload_name(args), "table": args.table, "batch": args.batch,
                       "layers": len(sweep.layers), "ops_per_step": ops_step,
                       "packed_weight_bytes": sweep.packed_weight_bytes(),
                       "fp16_weight_bytes": 2 * sum(pl.spec.params for pl in sweep.layers),
                       "l2": "weights (distinct per layer) are larger than L2", "launch": "CUDA graph replay"},
            "clocks": clocks,
            "e2e": {"value": replicas.whole_job_rate(ops_step, e2e_ms) / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms},
            "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline,
            "breakdown_ms": {"tensor_int8_layers": tc_ms, "other_layers": other_ms},
            "large_m_layers": per_layer,
            "device_status": status,
        }
        default_run = (world == 1 and args.table == "w4a8" and args.tokens == 0 and not args.act_asym and
                       not args.shortcut_split and not args.share_qkv_quant and not args.fuse_projections and
                       args.batch == 4 and not args.no_extras)
        if default_run:
            from paper_2405_17873_b200 import synth
            out["peaks"] = {"measured": {"hbm_gbs": peaks["hbm_gbs"], "bf16_tflops_burst": peaks["bf16_tflops"],
                                         "bf16_tflops_sustained": peaks["bf16_tflops_sustained"],
                                         "int8_mma_loop_probe_tops": round(probe_int8, 1), "source": peaks["source"]},
                            "nominal": NOMINAL}
            del sweep.workspace
            out["configs"] = config_records(torch, mixdq, synth, stream, peaks, probe_int8)
            out["fused_quantization"] = fused_quant_records(torch, mixdq, synth, stream)
            out["weight_bound_layers"] = weight_bound_records(torch, mixdq, synth, stream, peaks)
            sweep = None
            torch.cuda.empty_cache()
            out["other_sweeps"] = [sub_sweep_record(torch, UNetSweep, stream, peaks, args.batch, 0),
                                   sub_sweep_record(torch, UNetSweep, stream, peaks, args.batch, 16)]
        if world == 1 and not args.no_cpu_baseline and args.tokens == 0 and not args.act_asym and not args.shortcut_split and not args.share_qkv_quant and not args.fuse_projections and args.low_bits == 3:
            out["cpu_baseline"] = cpu_baseline(args.table, args.batch, 15.0)
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse()
    if args.impl == "reference":
        run_reference(args)
    elif args.impl == "fp16_library":
        run_fp16_library(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
