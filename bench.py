#!/usr/bin/env python
"""Benchmark of the k-means LUT linear layer (libkmq) on B200.

One "step" is one pass of the hot path over a pool of distinct weight sets:
for every bit width of the workload, `kmq_linear` is called once per pool
entry (different packed weights, codebooks, activations and outputs per call,
pool larger than L2 so no call finds its weights cached -- the protocol of the
paper's micro-benchmarks, Appendix "Benchmarking").  The calls of a step are
captured in CUDA graphs and replayed; time is taken with CUDA events on the
launching stream.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload config2]
    python bench.py --impl reference ...        # the CPU oracle on the host cores

Prints ONE JSON line (rank 0).  `value` is algorithmic bytes per second:
packed indices + codebooks + activations + outputs of every call, summed over
all ranks, divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

L2_BYTES = 126 * 1024 * 1024
FALLBACK_HBM_GBS = 6650.0

# workload -> list of (layer name, N, K, distribution, bits, M)
WORKLOADS = {
    "config2": [("square4096", 4096, 4096, "normal", b, 1) for b in (1, 2, 4)],
    "config3_m1": [(n, N, K, "student_t", 2, 1) for n, N, K in
                   (("qkv", 9216, 3072), ("o", 3072, 3072), ("gate_up", 16384, 3072), ("down", 3072, 8192))],
    "config3_m8": [(n, N, K, "student_t", 2, 8) for n, N, K in
                   (("qkv", 9216, 3072), ("o", 3072, 3072), ("gate_up", 16384, 3072), ("down", 3072, 8192))],
    "config4": [("square8192", 8192, 8192, "normal", 2, m) for m in (1, 2, 4, 8, 16, 32, 64)],
    "config5": [("down_large", 8192, 28672, "laplace", b, m) for b in (1, 4) for m in (1, 16)] +
               [("down_large", 8192, 28672, "laplace", b, 0) for b in (1, 4)],     # M = 0: kmq_dequant_to_bf16
    "tiny": [("tiny", 256, 256, "normal", b, 1) for b in (1, 2, 4)],
    # the larger batch-1 shapes of configurations 4 and 5 with random indices (no k-means fit: set-up in seconds)
    "large": [("square8192", 8192, 8192, "random", 2, 1), ("down_large", 8192, 28672, "random", 1, 1),
              ("down_large", 8192, 28672, "random", 4, 1)],
}
WORKLOAD_TEXT = {
    "config2": "single square layer N=K=4096, batch 1, b in {1,2,4}, per-row 2^b-centroid bf16 codebooks "
               "(1-D Lloyd, 20 iterations) on N(0, 0.02) weights, bf16 N(0,1) activations",
    "config3_m1": "3.9B-style decoder linear set (QKV 3072->9216, O 3072->3072, gate+up 3072->16384, "
                  "down 8192->3072), b=2, batch 1, Student-t(5) weights",
    "config3_m8": "3.9B-style decoder linear set, b=2, batch 8, Student-t(5) weights",
    "config4": "batch sweep on N=K=8192, b=2, batch in {1,2,4,8,16,32,64}",
    "config5": "large down projection N=8192 K=28672, b in {1,4}, batch in {1,16}, Laplace weights, plus the "
               "standalone kmq_dequant_to_bf16 of the full matrix (cases with M=0)",
    "tiny": "256x256 correctness layer",
    "large": "batch-1 shapes of configurations 4 and 5 (8192x8192 b=2; 8192x28672 b=1, 4) with uniformly random "
             "indices and sorted N(0, 0.02) codebooks: timing does not depend on the weight values",
}
CONFIG_ID = {"config2": 2, "config3_m1": 3, "config3_m8": 3, "config4": 4, "config5": 5, "tiny": 1, "large": 90}

# dram__bytes_read.sum + dram__bytes_write.sum per call (all launches of the call) from the ncu captures summarised
# under profiles/, keyed by (N, K, bits, M, variant); a case without an entry, or whose kernel has changed since the
# capture, reports null.
NCU_TRAFFIC_BYTES = {
    (4096, 4096, 1, 1, "tiled_select_b1"): 2146048,         # profiles/kmq_linear_tiled_4096x4096_ncu_full.md
    (4096, 4096, 2, 1, "tiled_prmt_b2"): 4251136,
    (4096, 4096, 4, 1, "tiled_pairtable_b4"): 8541184,
    (8192, 8192, 2, 1, "tiled_prmt_b2"): 16875008,          # profiles/kmq_linear_tiled_8192x8192_b2_ncu_full.md
    (8192, 28672, 1, 1, "table_lookup_b1"): 29493760 + 959488,            # main kernel + the kernel that adds the slices
    (8192, 28672, 4, 1, "split_pairtable_b4"): 117780992 + 4155392 + 486400,   # main (read + scratch written) + fix-up
}


def algorithmic_bytes(N, K, bits, M):
    if M == 0:                                   # kmq_dequant_to_bf16: packed + codebooks read, dense bf16 written
        return N * K * bits // 8 + N * (1 << bits) * 2 + 2 * N * K
    return N * K * bits // 8 + N * (1 << bits) * 2 + M * K * 2 + M * N * 2


_LAYER_CACHE = {}


def cached_layer(synth, N, K, bits, dist, config_id):
    """Weights, codebooks and indices depend on (shape, bits, distribution) only: fit them once per process."""
    key = (N, K, bits, dist, config_id)
    if key not in _LAYER_CACHE:
        _LAYER_CACHE[key] = synth.make_layer(N, K, bits, 1, dist, config_id=config_id)
    return _LAYER_CACHE[key]


def select_cases(args):
    """The cases of the workload, or the subset named by --case (e.g. "bits=1,M=1" or "layer=qkv")."""
    cases = WORKLOADS[args.workload]
    if not args.case:
        return cases
    want = dict(kv.split("=") for kv in args.case.split(","))
    keep = [c for c in cases if all(str({"layer": c[0], "N": c[1], "K": c[2], "bits": c[4], "M": c[5]}[k]) == v
                                    for k, v in want.items())]
    if not keep:
        raise SystemExit(f"--case {args.case!r} matches no case of {args.workload}")
    return keep


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# --------------------------------------------------------------------------
# clocks sampler (read-only NVML queries)
# --------------------------------------------------------------------------
class ClockSampler(threading.Thread):
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, index, period=0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons = [], set()
        self.active = False
        self.stop_flag = False
        self.max_mhz = None
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        while not self.stop_flag:
            try:
                mhz = self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)
                mask = self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
            except Exception:
                try:
                    mask = self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                except Exception:
                    mask = 0
                    mhz = None
            if self.active and mhz is not None:
                self.samples.append(mhz)
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            time.sleep(self.period)

    def summary(self):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"], "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------
# the library arm
# --------------------------------------------------------------------------
class Case:
    """One (layer, bits, M) of the workload with its pool of device buffers."""

    def __init__(self, name, N, K, dist, bits, M, config_id, torch, kmq, synth, pool_bytes, layout="auto",
                 random_weights=False):
        self.name, self.N, self.K, self.bits, self.M = name, N, K, bits, M
        self.bytes = algorithmic_bytes(N, K, bits, M)
        self.pool = max(4, -(-pool_bytes // self.bytes))
        self.dequant = M == 0
        self.random_weights = random_weights
        rng = synth.rng_for(config_id, 100 + bits * 1000 + M)
        x0 = synth.draw_activations(max(M, 1), K, synth.rng_for(config_id, synth.TENSOR_X))
        dev = torch.device("cuda")
        if random_weights:
            # timing does not depend on the weight values: uniformly random indices and sorted N(0, 0.02) codebooks,
            # drawn on the GPU, spare the minutes a k-means fit of a 235 M-weight layer takes on the host
            g = torch.Generator(device=dev).manual_seed(1000 * config_id + 10 * bits + M)
            idx = torch.randint(0, 1 << bits, (N, K), dtype=torch.uint8, device=dev, generator=g)
            cb_f = (torch.randn(N, 1 << bits, device=dev, generator=g) * 0.02).sort(dim=1).values
            codebooks = cb_f.to(torch.bfloat16).view(torch.int16).cpu().numpy().view(np.uint16)
        else:
            layer = cached_layer(synth, N, K, bits, dist, config_id)
            idx = torch.from_numpy(layer["idx"]).to(dev)
            codebooks = layer["codebooks"]
        # rows whose outputs the parity spot check recomputes with the oracle
        self.check_rows = np.unique(np.concatenate([np.arange(16), np.arange(N - 16, N),
                                                    np.random.default_rng(bits + M).choice(N, 32, replace=False)]))
        self.check_idx = idx[torch.from_numpy(self.check_rows).to(dev)].cpu().numpy()
        self.check_cb = codebooks[self.check_rows]
        # the layout in which the library is fastest for this batch (packing is the offline step)
        self.layout = {"tuned": kmq.KMQ_LAYOUT_TUNED, "table": kmq.KMQ_LAYOUT_TABLE,
                       "canonical": kmq.KMQ_LAYOUT_CANONICAL}.get(layout)
        if self.layout is None:
            self.layout = kmq.kmq_preferred_layout(N, K, bits, M) if M > 0 else kmq.KMQ_LAYOUT_TUNED
        self.layout_name = {kmq.KMQ_LAYOUT_TUNED: "tuned", kmq.KMQ_LAYOUT_TABLE: "table",
                            kmq.KMQ_LAYOUT_CANONICAL: "canonical"}[self.layout]
        words = kmq.kmq_packed_bytes(N, K, bits, self.layout) // 4
        if self.dequant:
            self.pool = max(2, -(-pool_bytes // self.bytes))
        self.packed = torch.empty((self.pool, words), dtype=torch.int32, device=dev)
        kmq.kmq_pack(idx, N, K, bits, self.packed[0], layout=self.layout)   # a1: offline packing, on the GPU
        self.packed[1:] = self.packed[0]
        del idx
        cb = torch.from_numpy(codebooks.view(np.int16)).to(dev)
        self.cb = cb.unsqueeze(0).repeat(self.pool, 1, 1).contiguous()
        Mx = max(M, 1)
        xs = np.stack([x0] + [synth.draw_activations(Mx, K, rng) for _ in range(self.pool - 1)])
        self.x_host = torch.from_numpy(xs.view(np.int16)).pin_memory()
        self.x = self.x_host.to(dev)
        if self.dequant:
            self.W = torch.zeros((self.pool, N, K), dtype=torch.int16, device=dev)
        self.y = torch.zeros((self.pool, Mx, N), dtype=torch.int16, device=dev)
        self.y_host = torch.zeros((self.pool, Mx, N), dtype=torch.int16).pin_memory()
        self.ws_bytes = 0 if self.dequant else kmq.kmq_workspace_bytes(N, K, bits, M, self.layout)
        self.ws = torch.empty(max(self.ws_bytes, 16), dtype=torch.uint8, device=dev)
        self.launches = 1 if self.dequant else kmq.kmq_linear_num_launches(N, K, bits, M, self.layout)
        self.variant = "dequant_rows" if self.dequant else kmq.kmq_linear_variant(N, K, bits, M, self.layout)
        self.kmq = kmq

    def call(self, i):
        if self.dequant:
            self.kmq.kmq_dequant_to_bf16(self.packed[i], self.cb[i], self.W[i], self.N, self.K, self.bits,
                                         layout=self.layout)
            return
        self.kmq.kmq_linear(self.packed[i], self.cb[i], self.x[i], self.y[i], self.N, self.K, self.bits, self.M,
                            self.ws, self.ws_bytes, layout=self.layout)

    def call_host(self, i):
        if self.dequant:                         # nothing to copy in or out: the weights stay on the device
            return self.call(i)
        self.kmq.kmq_linear_host(self.packed[i], self.cb[i], self.x_host[i].data_ptr(), self.y_host[i].data_ptr(),
                                 self.N, self.K, self.bits, self.M, self.x[i], self.y[i], self.ws, self.ws_bytes,
                                 layout=self.layout)


def machine_probes(torch, kmq, stream):
    """The two figures every per-call time is read against: the fixed cost of a call (a do-nothing kernel of the
    library in the same graph-replay protocol) and the read-only streaming bandwidth of a kernel of the library."""
    with torch.cuda.stream(stream):
        kmq.kmq_probe_launch()
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for _ in range(200):
                kmq.kmq_probe_launch()
        for _ in range(3):
            g.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(20):
            g.replay()
        e1.record(stream)
        stream.synchronize()
        floor_us = e0.elapsed_time(e1) * 1e3 / (20 * 200)
        nbytes = 1 << 30
        buf = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        buf.random_(0, 256)
        out = torch.empty(kmq.kmq_probe_read_out_bytes(), dtype=torch.uint8, device="cuda")
        best = float("inf")
        for _ in range(6):
            e0.record(stream)
            kmq.kmq_probe_read(buf, nbytes, out)
            e1.record(stream)
            stream.synchronize()
            best = min(best, e0.elapsed_time(e1))
        del buf
    return {"launch_floor_us": round(floor_us, 3),
            "launch_floor_how": "do-nothing kernel of the library, 200 per CUDA graph, programmatic dependent launch",
            "read_only_gbs": round(nbytes / (best * 1e-3) / 1e9, 1),
            "read_only_how": "1 GiB read once with 128-bit streaming loads, best of 6"}


# Cases timed next to the workload of --workload config2 (not part of `value`): shapes long enough for a steady-state
# HBM fraction.  (layer name, N, K, bits, M)
EXTRA_CASES = [(n, N, K, b, M) for (n, N, K, _d, b, M) in WORKLOADS["large"]]


# --------------------------------------------------------------------------
# whole decode step: every backbone linear of a Llama-style model, one CUDA graph per token
# --------------------------------------------------------------------------
# Model shapes from the paper's table of architectures (appendix "Optimization Hyperparameters": width d, layers L,
# heads, KV heads; head size 128; SwiGLU with multiplier 1.3, i.e. hidden = 1.3 * 8/3 * d rounded up to a multiple
# of 1024, which reproduces the printed parameter counts).  name -> (d, L, q heads, kv heads)
DECODE_MODELS = {"decode_4b": (3072, 24, 24, 8), "decode_12b": (4096, 48, 32, 8), "decode_31b": (6144, 60, 48, 8)}
# the paper's tokens/s at batch 1 on one L40S (864 GB/s), its own block-scaled format and Triton kernels: context only
PAPER_TOKENS_PER_S = {"decode_4b": {16: 88.8, 4.25: 190.1, 1.25: 245.6}, "decode_12b": {16: 30.0, 4.25: 79.3, 1.25: 120.0},
                      "decode_31b": {4.25: 35.4, 1.25: 60.7}}


def decode_layer_shapes(model, fused_gate_up=False):
    d, L, heads, kv = DECODE_MODELS[model]
    hidden = -(-int(1.3 * 8 * d / 3) // 1024) * 1024
    qkv = (heads + 2 * kv) * 128
    # (name, N out, K in, input: index of the call of the same layer whose output it reads, or -1 = the layer input)
    if fused_gate_up:    # the gate and up matrices stacked along N (they read the same input): one call
        return L, [("qkv", qkv, d, -1), ("o", d, d, 0), ("gate_up", 2 * hidden, d, 1), ("down", d, hidden, 2)]
    return L, [("qkv", qkv, d, -1), ("o", d, d, 0), ("gate", hidden, d, 1), ("up", hidden, d, 1), ("down", d, hidden, 2)]


def run_decode(args):
    """All backbone linears of one decoding step (batch 1) as one CUDA graph: L layers x (QKV, O, gate, up, down),
    every matrix with its own packed weights (random indices: timing does not depend on the values) and codebooks, the
    calls chained through their activations wherever the shapes of the model chain them (attention, normalisation and
    the activation function are not part of this library and are left out).  Reports tokens/s-equivalent = graph
    replays per second and the effective bandwidth over the algorithmic bytes of all calls."""
    import torch
    from paper_2602_15563_b200 import build as kb
    from paper_2602_15563_b200 import kmq, synth
    from oracle import kmq_oracle as orc
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libkmq has no CPU path")
    if int(os.environ.get("RANK", "0")) != 0:
        return
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    kb.build()
    dev = torch.device("cuda")
    peak_gbs, peak_kind = measured_peak()
    L, shapes = decode_layer_shapes(args.workload)
    d = DECODE_MODELS[args.workload][0]
    results = []
    sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")))
    sampler.start()
    stream = torch.cuda.Stream()
    for fused, bits in ((False, 1), (False, 4), (True, 1), (True, 4)):
        L, shapes = decode_layer_shapes(args.workload, fused)
        g = torch.Generator(device=dev).manual_seed(bits)
        calls, step_bytes, ws_bytes = [], 0, 16
        x0 = (torch.randn(d, device=dev, generator=g)).to(torch.bfloat16).view(torch.int16)
        for layer in range(L):
            outs = []
            for ci, (name, N, K, src) in enumerate(shapes):
                layout = kmq.kmq_preferred_layout(N, K, bits, 1)
                words = kmq.kmq_packed_bytes(N, K, bits, layout) // 4
                if layer == 0:       # packed by kmq_pack from explicit indices: these calls are checked against the oracle
                    idx = torch.randint(0, 1 << bits, (N, K), dtype=torch.uint8, device=dev, generator=g)
                    packed = torch.empty(words, dtype=torch.int32, device=dev)
                    kmq.kmq_pack(idx, N, K, bits, packed, layout=layout)
                    rows = np.unique(np.concatenate([np.arange(16), np.arange(N - 16, N)]))
                    check = (rows, idx[torch.from_numpy(rows).to(dev)].cpu().numpy())
                    del idx
                else:                # any bit pattern is a valid set of indices
                    packed = torch.randint(-2**31, 2**31 - 1, (words,), dtype=torch.int32, device=dev, generator=g)
                    check = None
                cb = (torch.randn(N, 1 << bits, device=dev, generator=g) * 0.02).sort(dim=1).values
                cb = cb.to(torch.bfloat16).view(torch.int16)
                y = torch.zeros(N, dtype=torch.int16, device=dev)
                x = (x0 if layer == 0 else calls[-1]["y"]) if src < 0 else outs[src]["y"]
                ws_bytes = max(ws_bytes, kmq.kmq_workspace_bytes(N, K, bits, 1, layout))
                c = {"name": name, "N": N, "K": K, "layout": layout, "packed": packed, "cb": cb, "x": x[:K], "y": y,
                     "check": check, "variant": kmq.kmq_linear_variant(N, K, bits, 1, layout),
                     "launches": kmq.kmq_linear_num_launches(N, K, bits, 1, layout)}
                outs.append(c)
                step_bytes += algorithmic_bytes(N, K, bits, 1)
            calls += outs
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)

        def issue():
            for c in calls:
                kmq.kmq_linear(c["packed"], c["cb"], c["x"], c["y"], c["N"], c["K"], bits, 1, ws, ws_bytes,
                               layout=c["layout"])
        with torch.cuda.stream(stream):
            issue()
            stream.synchronize()
            # parity of the first layer's calls (the chain makes every input a previous output, also checked here)
            worst = 0.0
            for c in calls[:len(shapes)]:
                rows, idx_rows = c["check"]
                ref_packed = orc.pack_canonical(idx_rows, bits)
                y_ref, s_abs = orc.linear_f64(ref_packed, c["cb"].cpu().numpy().view(np.uint16)[rows],
                                              c["x"].cpu().numpy().view(np.uint16)[None, :], c["K"], bits)
                got = c["y"].cpu().numpy().view(np.uint16)[None, rows]
                worst = max(worst, orc.check_linear(got, y_ref, s_abs))
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                issue()
            for _ in range(max(args.warmup, 3)):
                graph.replay()
            stream.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            steps = max(1, min(args.steps, 50))
            sampler.active = True
            e0.record(stream)
            for _ in range(steps):
                graph.replay()
            e1.record(stream)
            stream.synchronize()
            sampler.active = False
        ms = e0.elapsed_time(e1) / steps
        variants = sorted({f"{c['name']}:{c['variant']}" for c in calls[:len(shapes)]})
        results.append({"bits": bits, "gate_up": "one call" if fused else "two calls", "ms_per_token": round(ms, 4), "tokens_per_s_equivalent": round(1e3 / ms, 1),
                        "gbs": round(step_bytes / (ms * 1e-3) / 1e9, 1),
                        "frac_of_measured_hbm": round(step_bytes / (ms * 1e-3) / 1e9 / peak_gbs, 4),
                        "calls_per_token": len(calls), "launches_per_token": sum(c["launches"] for c in calls),
                        "bytes_per_token": step_bytes, "variants": variants, "steps": steps,
                        "parity_max_err_over_tol": round(worst, 4)})
        del calls, outs, ws, graph
        torch.cuda.empty_cache()
    sampler.stop_flag = True
    L, shapes = decode_layer_shapes(args.workload)
    best = max(results, key=lambda r: r["gbs"])
    line = {
        "metric": "kmq_linear effective HBM bandwidth (algorithmic bytes / time), batch-1 k-means LUT GEMV",
        "value": best["gbs"], "unit": "GB/s", "n_gpus": 1, "steps": best["steps"], "warmup": max(args.warmup, 3),
        "ms_per_step": best["ms_per_token"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{args.workload}: every backbone linear of one decoding step at batch 1, "
                               f"L = {L} layers x {[(n, N, K) for (n, N, K, _s) in shapes]}, one CUDA graph per token, "
                               "distinct weights per matrix (far larger than L2), random indices; timed a second time with "
                               "the gate and up matrices stacked into one call (per_bits: gate_up)",
                   "multi_gpu": "replicas only"},
        "per_bits": results,
        "roofline": {"bound": "hbm", "kernel": "all kmq_linear calls of a token", "achieved": best["gbs"],
                     "peak": peak_gbs, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                     "frac": round(best["gbs"] / peak_gbs, 4), "traffic": None},
        "gpu_launches": sum(r["launches_per_token"] * r["steps"] for r in results),
        "clocks": sampler.summary(),
        "parity": {"ok": all(r["parity_max_err_over_tol"] <= 1.0 for r in results)},
        "paper_context": {"note": "paper's tokens/s for the whole model (attention, norms and bf16 embeddings included) "
                                  "at batch 1 on one L40S (864 GB/s), by bits per weight; context only",
                          "tokens_per_s": {str(k): v for k, v in PAPER_TOKENS_PER_S[args.workload].items()}},
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------
# large batches: the fused kernel against "dequantise, then a standard bf16 GEMM"
# --------------------------------------------------------------------------
LARGE_BATCH_SHAPES = [("square8192", 8192, 8192, 2), ("gate_up", 16384, 3072, 2)]
LARGE_BATCH_M = (16, 32, 64, 96, 128, 256, 512, 1024)


def run_large_batch(args):
    """Where the fused dequantise-multiply stops paying (paper, Section 3.3: the regimes below the theoretical
    speed-up; appendix "Benchmarking": at large batch "dequantize in a separate kernel, before using a standard
    high-precision GEMM").  Per shape and batch: kmq_linear; kmq_dequant_to_bf16 followed by a bf16 GEMM of the
    vendor library (torch.matmul; a baseline leg, not a path of this library); that GEMM alone on resident bf16
    weights (the 16-bit baseline).  The measured crossover is set beside the roofline model's P_w * nu / 16."""
    import torch
    from paper_2602_15563_b200 import build as kb
    from paper_2602_15563_b200 import kmq
    from oracle import kmq_oracle as orc
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libkmq has no CPU path")
    if int(os.environ.get("RANK", "0")) != 0:
        return
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    kb.build()
    dev = torch.device("cuda")
    peak_gbs, peak_kind = measured_peak()
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            tflops = float(json.load(f)["bf16_tflops_sustained"])
        tf_kind = "measured"
    except Exception:
        tflops, tf_kind = 1400.0, "fallback"
    nu = tflops * 1e12 / (peak_gbs * 1e9)                    # the paper's nu = R_compute / R_transfer, flop per byte
    sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")))
    sampler.start()
    stream = torch.cuda.Stream()
    T = kmq.KMQ_LAYOUT_TUNED
    rows_out, launches, worst = [], 0, 0.0
    steps = max(1, min(args.steps, 20))
    for (name, N, K, bits) in LARGE_BATCH_SHAPES:
        g = torch.Generator(device=dev).manual_seed(N + K)
        pool = max(4, -(-2 * L2_BYTES // (N * K * bits // 8)))
        idx = torch.randint(0, 1 << bits, (N, K), dtype=torch.uint8, device=dev, generator=g)
        packed = torch.empty((pool, kmq.kmq_packed_bytes(N, K, bits, T) // 4), dtype=torch.int32, device=dev)
        kmq.kmq_pack(idx, N, K, bits, packed[0], layout=T)
        packed[1:] = packed[0]
        check_rows = np.unique(np.concatenate([np.arange(16), np.arange(N - 16, N)]))
        ref_packed = orc.pack_canonical(idx[torch.from_numpy(check_rows).to(dev)].cpu().numpy(), bits)
        del idx
        cb = (torch.randn(N, 1 << bits, device=dev, generator=g) * 0.02).sort(dim=1).values.to(torch.bfloat16)
        Wd = torch.empty((2, N, K), dtype=torch.bfloat16, device=dev)      # dequantised weights, two in rotation
        kmq.kmq_dequant_to_bf16(packed[0], cb, Wd[0], N, K, bits, layout=T)
        Wd[1] = Wd[0]
        p_w = bits + 16.0 * (1 << bits) / K
        for M in LARGE_BATCH_M:
            x = torch.randn(M, K, device=dev, generator=g).to(torch.bfloat16)
            y = torch.zeros(M, N, dtype=torch.bfloat16, device=dev)
            y2 = torch.zeros(M, N, dtype=torch.bfloat16, device=dev)
            ws_bytes = kmq.kmq_workspace_bytes(N, K, bits, M, T)
            ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device=dev)

            def fused(i):
                kmq.kmq_linear(packed[i % pool], cb, x, y, N, K, bits, M, ws, ws_bytes, layout=T)

            def dequant_gemm(i):
                kmq.kmq_dequant_to_bf16(packed[i % pool], cb, Wd[i % 2], N, K, bits, layout=T)
                torch.matmul(x, Wd[i % 2].t(), out=y2)

            def gemm_only(i):
                torch.matmul(x, Wd[i % 2].t(), out=y2)
            times = {}
            with torch.cuda.stream(stream):
                for leg, fn, reps in (("fused", fused, pool), ("dequant_gemm", dequant_gemm, 4), ("gemm_bf16", gemm_only, 4)):
                    fn(0)
                    stream.synchronize()
                    gr = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(gr, stream=stream):
                        for i in range(reps):
                            fn(i)
                    for _ in range(3):
                        gr.replay()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    sampler.active = True
                    e0.record(stream)
                    for _ in range(steps):
                        gr.replay()
                    e1.record(stream)
                    stream.synchronize()
                    sampler.active = False
                    times[leg] = e0.elapsed_time(e1) * 1e3 / (steps * reps)
                    if leg == "fused":
                        launches += steps * reps * kmq.kmq_linear_num_launches(N, K, bits, M, T)
                # parity of the fused result (the last call used packed[(pool - 1) % pool] = the same weights)
                y_ref, s_abs = orc.linear_f64(ref_packed, cb.view(torch.int16).cpu().numpy().view(np.uint16)[check_rows],
                                              x.view(torch.int16).cpu().numpy().view(np.uint16), K, bits)
                got = y[:, torch.from_numpy(check_rows).to(dev)].view(torch.int16).cpu().numpy().view(np.uint16)
                worst = max(worst, orc.check_linear(got, y_ref, s_abs))
            flops = 2.0 * M * N * K
            rows_out.append({"layer": name, "N": N, "K": K, "bits": bits, "M": M,
                             "variant": kmq.kmq_linear_variant(N, K, bits, M, T),
                             "fused_us": round(times["fused"], 2), "dequant_gemm_us": round(times["dequant_gemm"], 2),
                             "gemm_bf16_us": round(times["gemm_bf16"], 2),
                             "fused_tflops": round(flops / times["fused"] / 1e6, 1),
                             "fused_gbs": round(algorithmic_bytes(N, K, bits, M) / times["fused"] / 1e3, 1),
                             "fused_faster_than_dequant_gemm": bool(times["fused"] < times["dequant_gemm"]),
                             "fused_faster_than_bf16_gemm": bool(times["fused"] < times["gemm_bf16"]),
                             "model_memory_bound_up_to_m": round(p_w * nu / 16.0, 1)})
        del packed, Wd
        torch.cuda.empty_cache()
    sampler.stop_flag = True
    cross = {}
    for (name, N, K, bits) in LARGE_BATCH_SHAPES:
        ms = [r["M"] for r in rows_out if r["layer"] == name and not r["fused_faster_than_dequant_gemm"]]
        cross[name] = min(ms) if ms else None
    best = max(rows_out, key=lambda r: r["fused_tflops"])
    line = {
        "metric": "kmq_linear effective HBM bandwidth (algorithmic bytes / time), batch-1 k-means LUT GEMV",
        "value": best["fused_gbs"], "unit": "GB/s", "n_gpus": 1, "steps": steps, "warmup": 3,
        "ms_per_step": round(best["fused_us"] * 1e-3, 5), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "large_batch: fused kmq_linear against kmq_dequant_to_bf16 + bf16 GEMM and against the "
                               "bf16 GEMM alone, batches " + str(list(LARGE_BATCH_M)) + " on "
                               + str([(n, N, K, b) for (n, N, K, b) in LARGE_BATCH_SHAPES]) + ", random indices",
                   "l2": "packed weights from a pool larger than 2 x L2; dequantised weights: two buffers in rotation",
                   "multi_gpu": "replicas only"},
        "per_case": rows_out,
        "first_batch_where_dequant_plus_gemm_wins": cross,
        "roofline_model": {"nu_flop_per_byte": round(nu, 1), "tensor_tflops": tflops, "tensor_kind": f"of {tf_kind}",
                           "hbm_gbs": peak_gbs, "rule": "memory bound while m < P_w * nu / 16 (paper, theoretical model)"},
        "roofline": {"bound": "tensor", "kernel": f"kmq_linear[{best['variant']}] M={best['M']} {best['N']}x{best['K']}",
                     "achieved": best["fused_tflops"], "peak": tflops, "peak_kind": f"of {tf_kind} (sustained bf16)",
                     "unit": "TFLOP/s", "frac": round(best["fused_tflops"] / tflops, 4), "traffic": None},
        "gpu_launches": launches, "clocks": sampler.summary(),
        "parity": {"max_err_over_tol": round(worst, 4), "ok": bool(worst <= 1.0)},
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------
# the paper's own block format (shared codebook + bf16 scale per block of 64)
# --------------------------------------------------------------------------
BLOCK_CASES = [(4096, 4096, b, 1) for b in (1, 2, 4, 8)] + [(8192, 8192, b, 1) for b in (1, 2, 4)]


def block_bytes(N, K, bits, M):
    """Algorithmic bytes of one kmq_block_linear call: P_w = bits + 16/64 bits per weight (indices + scales), the
    codebook, activations in, outputs out."""
    return N * K * bits // 8 + N * (K // 64) * 2 + (1 << bits) * 2 + M * K * 2 + M * N * 2


def run_block(args):
    """kmq_block_linear (deferred scaling) at batch 1 on the paper's micro-benchmark shape (8192 x 8192) and on
    4096 x 4096, random indices and scales (timing does not depend on the values), pool of weight sets larger than
    2 x L2, one CUDA graph per case."""
    import torch
    from paper_2602_15563_b200 import build as kb
    from paper_2602_15563_b200 import kmq
    from oracle import kmq_block_oracle as blk
    from oracle import kmq_oracle as orc
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libkmq has no CPU path")
    if int(os.environ.get("RANK", "0")) != 0:
        return
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    kb.build()
    dev = torch.device("cuda")
    peak_gbs, peak_kind = measured_peak()
    sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")))
    sampler.start()
    stream = torch.cuda.Stream()
    steps = max(1, min(args.steps, 50))
    rows_out, launches, worst = [], 0, 0.0
    cases = BLOCK_CASES
    if args.case:      # e.g. "N=8192,bits=1": one case, small enough for a profiler run
        want = dict(kv.split("=") for kv in args.case.split(","))
        cases = [c for c in cases if all(str({"N": c[0], "K": c[1], "bits": c[2], "M": c[3]}[k]) == v
                                         for k, v in want.items())]
        if not cases:
            raise SystemExit(f"--case {args.case!r} matches no case of the block workload")
    for (N, K, bits, M) in cases:
        g = torch.Generator(device=dev).manual_seed(N + 7 * bits)
        nbytes = block_bytes(N, K, bits, M)
        pool = max(4, -(-2 * L2_BYTES // nbytes))
        idx = torch.randint(0, 1 << bits, (N, K), dtype=torch.uint8, device=dev, generator=g)
        wq = torch.empty((pool, N * K * bits // 8), dtype=torch.uint8, device=dev)
        kmq.kmq_block_pack(idx, N, K, bits, wq[0])
        wq[1:] = wq[0]
        rows = np.unique(np.concatenate([np.arange(16), np.arange(N - 16, N)]))
        ref_wq = blk.pack_bytes(idx[torch.from_numpy(rows).to(dev)].cpu().numpy(), bits)
        del idx
        scales = (torch.rand(N, K // 64, device=dev, generator=g) * 0.05 + 0.01).to(torch.bfloat16)
        cb = torch.linspace(-1, 1, 1 << bits, device=dev).to(torch.bfloat16)
        x = torch.randn(pool, M, K, device=dev, generator=g).to(torch.bfloat16)
        y = torch.zeros(pool, M, N, dtype=torch.bfloat16, device=dev)

        def call(i):
            kmq.kmq_block_linear(wq[i], scales, cb, x[i], y[i], N, K, bits, M, scale_order=kmq.KMQ_SCALE_DEFERRED)
        with torch.cuda.stream(stream):
            call(0)
            stream.synchronize()
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gr, stream=stream):
                for i in range(pool):
                    call(i)
            for _ in range(max(args.warmup, 3)):
                gr.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            sampler.active = True
            e0.record(stream)
            for _ in range(steps):
                gr.replay()
            e1.record(stream)
            stream.synchronize()
            sampler.active = False
        us = e0.elapsed_time(e1) * 1e3 / (steps * pool)
        launches += steps * pool
        us_table = None
        if bits != 8:
            # the same layers through the activation-table kernel, which reads its own layout (index bytes and
            # scales side by side): packed once, outside the timed region
            tab = torch.empty((pool, kmq.kmq_block_table_bytes(N, K, bits)), dtype=torch.uint8, device=dev)
            kmq.kmq_block_table_pack(wq[0], scales.view(torch.int16), N, K, bits, tab[0])
            tab[1:] = tab[0]
            wsb = kmq.kmq_block_table_workspace_bytes(N, K, bits)
            ws = torch.empty(max(wsb, 16), dtype=torch.uint8, device=dev)
            y_t = torch.zeros(pool, M, N, dtype=torch.bfloat16, device=dev)

            def call_t(i):
                kmq.kmq_block_table_linear(tab[i], cb, x[i], y_t[i], N, K, bits, M, ws, wsb)
            with torch.cuda.stream(stream):
                call_t(0)
                stream.synchronize()
                gt = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gt, stream=stream):
                    for i in range(pool):
                        call_t(i)
                for _ in range(max(args.warmup, 3)):
                    gt.replay()
                t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                sampler.active = True
                t0.record(stream)
                for _ in range(steps):
                    gt.replay()
                t1.record(stream)
                stream.synchronize()
                sampler.active = False
            us_table = t0.elapsed_time(t1) * 1e3 / (steps * pool)
            launches += steps * pool * (2 if wsb else 1)
        for i in (0, pool - 1):
            y_ref, s_abs = blk.block_linear_f64(ref_wq, scales.view(torch.int16).cpu().numpy().view(np.uint16)[rows],
                                                cb.view(torch.int16).cpu().numpy().view(np.uint16),
                                                x[i].view(torch.int16).cpu().numpy().view(np.uint16), K, bits)
            got = y[i][:, torch.from_numpy(rows).to(dev)].view(torch.int16).cpu().numpy().view(np.uint16)
            worst = max(worst, orc.check_linear(got, y_ref, s_abs))
            if us_table is not None:
                got = y_t[i][:, torch.from_numpy(rows).to(dev)].view(torch.int16).cpu().numpy().view(np.uint16)
                worst = max(worst, orc.check_linear(got, y_ref, s_abs))
        us_direct = us
        if us_table is not None:
            del tab, y_t
            us = min(us, us_table)
        gbs = nbytes / us / 1e3
        rows_out.append({"N": N, "K": K, "bits": bits, "P_w": bits + 0.25, "M": M, "pool": pool, "us_per_call": round(us, 3),
                         "us_kmq_block_linear": round(us_direct, 3),
                         "us_kmq_block_table_linear": None if us_table is None else round(us_table, 3),
                         "gbs": round(gbs, 1), "frac_of_measured_hbm": round(gbs / peak_gbs, 4), "bytes_per_call": nbytes,
                         "ideal_us_at_measured_hbm": round(nbytes / (peak_gbs * 1e3), 3)})
        del wq, x, y
        torch.cuda.empty_cache()
    sampler.stop_flag = True
    tot_b = sum(r["bytes_per_call"] * r["pool"] for r in rows_out)
    tot_us = sum(r["us_per_call"] * r["pool"] for r in rows_out)
    dom = max(rows_out, key=lambda r: r["us_per_call"] * r["pool"])
    line = {
        "metric": "kmq_linear effective HBM bandwidth (algorithmic bytes / time), batch-1 k-means LUT GEMV",
        "value": round(tot_b / tot_us / 1e3, 2), "unit": "GB/s", "n_gpus": 1, "steps": steps,
        "warmup": max(args.warmup, 3), "ms_per_step": round(tot_us * 1e-3, 5), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "block: the paper's k-means block format (shared codebook, bf16 scale per block of 64, "
                               "P_w = b + 0.25), kmq_block_linear (deferred scaling) and kmq_block_table_linear at batch 1, the "
                               "faster of the two per case, on "
                               + str([(N, K, b) for (N, K, b, _m) in cases]) + ", random indices and scales",
                   "l2": "inputs larger than L2: every call of a step uses its own weight set, pool >= 2 x 126 MB",
                   "multi_gpu": "replicas only"},
        "per_case": rows_out,
        "roofline": {"bound": "hbm", "kernel": f"block format b={dom['bits']} {dom['N']}x{dom['K']}",
                     "achieved": dom["gbs"], "peak": peak_gbs, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                     "frac": dom["frac_of_measured_hbm"], "traffic": None},
        "gpu_launches": launches, "clocks": sampler.summary(),
        "parity": {"max_err_over_tol": round(worst, 4), "ok": bool(worst <= 1.0)},
        "paper_context": PAPER_CONTEXT,
    }
    print(json.dumps(line))


# (format, N, K, bits): "rows" = a codebook per row (kmq_quantize_rows), "block" = the paper's block format
QUANTIZE_CASES = [("rows", 4096, 4096, 1), ("rows", 4096, 4096, 2), ("rows", 4096, 4096, 4), ("rows", 8192, 8192, 2),
                  ("rows", 8192, 28672, 1), ("rows", 8192, 28672, 4), ("block", 4096, 4096, 4), ("block", 8192, 8192, 1)]
QUANTIZE_SAMPLES = 32768


def run_quantize(args):
    """The quantiser side on the GPU: float32 weights -> codebooks (+ block scales) -> packed indices.  Seeded N(0,
    0.02) weights drawn on the device; every timed call reads its own copy of the weights out of a pool larger than
    L2.  The fit and the assignment are also timed on their own; sampled rows are checked against the oracle."""
    import torch
    from paper_2602_15563_b200 import build as kb
    from paper_2602_15563_b200 import kmq
    from oracle import kmq_block_oracle as blk
    from oracle import kmq_quant_oracle as qorc
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libkmq has no CPU path")
    if int(os.environ.get("RANK", "0")) != 0:
        return
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    kb.build()
    dev = torch.device("cuda")
    peak_gbs, peak_kind = measured_peak()
    sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")))
    sampler.start()
    stream = torch.cuda.Stream()
    steps = max(1, min(args.steps, 10))
    rows_out, launches, parity_ok = [], 0, True
    cpu_rows_per_s = {}

    def timed(fn, pool):
        with torch.cuda.stream(stream):
            for i in range(min(pool, max(args.warmup, 3))):
                fn(i % pool)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for it in range(steps):
                fn(it % pool)
            e1.record(stream)
            stream.synchronize()
        return e0.elapsed_time(e1) / steps

    cases = QUANTIZE_CASES
    if args.case:      # e.g. "format=rows,N=4096,bits=4": a subset small enough for a profiler run
        want = dict(kv.split("=") for kv in args.case.split(","))
        cases = [c for c in cases if all(str({"format": c[0], "N": c[1], "K": c[2], "bits": c[3]}[k]) == v
                                         for k, v in want.items())]
        if not cases:
            raise SystemExit(f"--case {args.case!r} matches no case of the quantize workload")
    for (fmt, N, K, bits) in cases:
        g = torch.Generator(device=dev).manual_seed(N + K + bits)
        pool = max(2, -(-(L2_BYTES + L2_BYTES // 2) // (N * K * 4)))
        W = torch.randn((pool, N, K), generator=g, device=dev, dtype=torch.float32) * 0.02
        Q = 1 << bits
        rows = np.unique(np.concatenate([[0, 15, 16, N - 1], np.random.default_rng(N).integers(0, N, 4)]))
        sampler.active = True
        if fmt == "rows":
            layout = kmq.kmq_preferred_layout(N, K, bits, 1)
            cb = torch.empty((N, Q), dtype=torch.int16, device=dev)
            packed = torch.empty(kmq.kmq_packed_bytes(N, K, bits, layout) // 4, dtype=torch.int32, device=dev)
            out_bytes = packed.numel() * 4 + cb.numel() * 2
            ms_all = timed(lambda i: kmq.kmq_quantize_rows(W[i], N, K, bits, 20, layout, cb, packed, stream=stream), pool)
            ms_fit = timed(lambda i: kmq.kmq_kmeans_rows(W[i], N, K, bits, 20, cb, stream=stream), pool)
            ms_assign = timed(lambda i: kmq.kmq_assign_pack(W[i], cb, N, K, bits, layout, packed, stream=stream), pool)
            launches += steps * 4
            kmq.kmq_quantize_rows(W[0], N, K, bits, 20, layout, cb, packed, stream=stream)
            idx = torch.empty((N, K), dtype=torch.uint8, device=dev)
            kmq.kmq_unpack(packed, N, K, bits, idx, layout=layout, stream=stream)
            stream.synchronize()
            sel = torch.from_numpy(rows).to(dev)
            w_rows = W[0][sel].cpu().numpy()
            t0 = time.perf_counter()
            want_cb = qorc.centroids_to_bf16(qorc.lloyd_rows(w_rows, bits))
            want_idx = qorc.nearest_centroid(w_rows, want_cb)
            cpu_rows_per_s[(N, K, bits)] = len(rows) / (time.perf_counter() - t0)
            ok = (np.array_equal(cb[sel].cpu().numpy().view(np.uint16), want_cb)
                  and np.array_equal(idx[sel].cpu().numpy(), want_idx))
            del idx, packed
        else:
            scales = torch.empty(N * K // 64, dtype=torch.int16, device=dev)
            cb = torch.empty(max(8, Q), dtype=torch.int16, device=dev)
            wq = torch.empty(kmq.kmq_block_packed_bytes(N, K, bits), dtype=torch.uint8, device=dev)
            ws = torch.empty(QUANTIZE_SAMPLES, dtype=torch.float32, device=dev)
            out_bytes = wq.numel() + scales.numel() * 2 + Q * 2
            lam = kmq.KMQ_LAMBDA_ABSMAX
            ms_all = timed(lambda i: kmq.kmq_block_quantize(W[i], N, K, bits, lam, 20, QUANTIZE_SAMPLES, scales, cb, wq,
                                                            ws, stream=stream), pool)
            ms_fit = timed(lambda i: kmq.kmq_kmeans_rows(ws, 1, QUANTIZE_SAMPLES, bits, 20, cb, stream=stream), pool)
            ms_assign = timed(lambda i: kmq.kmq_block_assign_pack(W[i], scales, cb, N, K, bits, wq, stream=stream), pool)
            launches += steps * 6
            kmq.kmq_block_quantize(W[0], N, K, bits, lam, 20, QUANTIZE_SAMPLES, scales, cb, wq, ws, stream=stream)
            stream.synchronize()
            w_rows = W[0][:256].cpu().numpy()
            s_all = scales.cpu().numpy().view(np.uint16).reshape(N, K // 64)
            cbn = cb.cpu().numpy().view(np.uint16)[:Q]
            ok = (np.array_equal(s_all[:256], qorc.block_scales(w_rows, qorc.ABSMAX))
                  and np.array_equal(wq.view(N, -1)[:256].cpu().numpy(),
                                     blk.pack_bytes(qorc.block_assign(w_rows, s_all[:256], cbn), bits)))
            del wq, scales
        sampler.active = False
        parity_ok = parity_ok and bool(ok)
        nbytes = N * K * 4 + out_bytes
        rows_out.append({"format": fmt, "N": N, "K": K, "bits": bits, "pool": pool, "ms_per_call": round(ms_all, 4),
                         "ms_fit": round(ms_fit, 4), "ms_assign_pack": round(ms_assign, 4),
                         "gbs": round(nbytes / ms_all / 1e6, 1), "frac_of_measured_hbm": round(nbytes / ms_all / 1e6 / peak_gbs, 4),
                         "assign_pack_gbs": round(nbytes / ms_assign / 1e6, 1),
                         "mweights_per_s": round(N * K / ms_all / 1e3, 1), "bytes_per_call": nbytes,
                         "ideal_ms_at_measured_hbm": round(nbytes / (peak_gbs * 1e6), 4), "parity_ok": bool(ok)})
        del W
        torch.cuda.empty_cache()
    sampler.stop_flag = True
    tot_b = sum(r["bytes_per_call"] for r in rows_out)
    tot_ms = sum(r["ms_per_call"] for r in rows_out)
    dom = max(rows_out, key=lambda r: r["ms_per_call"])
    key = (dom["N"], dom["K"], dom["bits"])
    cpu = None
    if key in cpu_rows_per_s:
        cpu = {"value": round(cpu_rows_per_s[key] * dom["K"] / 1e6, 3), "unit": "Mweights/s", "cores": _cpu_threads(),
               "kind": "oracle", "sample": f"lloyd_rows + nearest_centroid on 8 rows of the {dom['N']}x{dom['K']} b={dom['bits']} case"}
    line = {
        "metric": "quantiser throughput: float32 weights read + packed indices, codebooks and scales written, per second",
        "value": round(tot_b / tot_ms / 1e6, 2), "unit": "GB/s", "n_gpus": 1, "steps": steps,
        "warmup": max(args.warmup, 3), "ms_per_step": round(tot_ms, 4), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "quantize: per-row 1-D Lloyd fit (quantile start, 20 iterations) + nearest-centroid "
                               "assignment + packing (kmq_quantize_rows), and the block format's scales + sampled "
                               "shared-codebook fit + assignment (kmq_block_quantize, absmax, 32768 samples), on "
                               + str([(f, N, K, b) for (f, N, K, b) in cases]) + ", N(0, 0.02) float32 weights",
                   "l2": "inputs larger than L2: consecutive calls read different copies of the weights, pool >= 1.5 x 126 MB",
                   "multi_gpu": "replicas only"},
        "per_case": rows_out,
        "roofline": {"bound": "alu", "kernel": f"lloyd_rows_kernel {dom['N']}x{dom['K']} b={dom['bits']}",
                     "note": "the fit is bound by the shared-memory sorting network, not by HBM; the fraction below is "
                             "algorithmic bytes / time against the HBM peak for orientation",
                     "achieved": dom["gbs"], "peak": peak_gbs, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                     "frac": dom["frac_of_measured_hbm"], "traffic": None},
        "gpu_launches": launches, "clocks": sampler.summary(), "cpu_baseline": cpu,
        "parity": {"ok": parity_ok},
    }
    print(json.dumps(line))


def run_library(args):
    import torch
    from paper_2602_15563_b200 import build as kb
    from paper_2602_15563_b200 import kmq, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libkmq has no CPU path (use --impl reference for the oracle)")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        kb.build()
    if dist is not None:
        dist.barrier()
    kmq.lib()

    peak_gbs, peak_kind = measured_peak()
    cfg_id = CONFIG_ID[args.workload]
    pool_bytes = 2 * L2_BYTES
    cases = [Case(n, N, K, d, b, M, cfg_id, torch, kmq, synth, pool_bytes, args.layout, random_weights=(d == "random"))
             for (n, N, K, d, b, M) in select_cases(args)]
    n_main = len(cases)
    if args.workload == "config2" and not args.case and not args.no_extra:
        cases += [Case(n, N, K, "normal", b, M, 90, torch, kmq, synth, pool_bytes, args.layout, random_weights=True)
                  for (n, N, K, b, M) in EXTRA_CASES]

    stream = torch.cuda.Stream()
    graphs = []
    with torch.cuda.stream(stream):
        for c in cases:                       # warm every kernel outside capture first
            c.call(0)
        stream.synchronize()
        for c in cases:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for i in range(c.pool):
                    c.call(i)
            graphs.append(g)

    def one_step(events=None, lo=0, hi=None):
        """One pass over the cases lo .. hi-1 (default: the workload itself, without the extra cases)."""
        hi = n_main if hi is None else hi
        for j in range(lo, hi):
            if events is not None:
                events[j][0].record(stream)
            graphs[j].replay()
            if events is not None:
                events[j][1].record(stream)

    sampler = ClockSampler(local_rank)
    sampler.start()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3)):
            one_step()
        barrier()
        # ---- timed region: exactly K steps ----
        ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in cases]
              for _ in range(args.steps)]
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sampler.active = True
        t0.record(stream)
        for s in range(args.steps):
            one_step(ev[s])
        t1.record(stream)
        barrier()
        # ---- after the timed region: the extra cases, the same number of steps, their own events ----
        if len(cases) > n_main:
            for _ in range(3):
                one_step(None, n_main, len(cases))
            for s in range(args.steps):
                one_step(ev[s], n_main, len(cases))
            barrier()
        sampler.active = False
        machine = machine_probes(torch, kmq, stream) if rank == 0 and not args.quick else None
    elapsed_ms = t0.elapsed_time(t1)
    step_ms = [[ev[s][j][0].elapsed_time(ev[s][j][1]) for s in range(args.steps)] for j in range(len(cases))]
    per_case_ms = [sum(t) / args.steps for t in step_ms]
    # standard error of the mean per-call time over the K timed steps (each step = one replay of the case's graph)
    per_case_sem_ms = [(float(np.std(t, ddof=1)) / np.sqrt(len(t)) if len(t) > 1 else 0.0) for t in step_ms]

    step_bytes = sum(c.bytes * c.pool for c in cases[:n_main])
    step_calls = sum(c.pool for c in cases[:n_main])
    if dist is not None:
        t = torch.tensor([elapsed_ms], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        elapsed_ms = float(t.item())
    value = world * step_bytes * args.steps / (elapsed_ms * 1e-3) / 1e9

    # ---- end to end through the host-buffer entry point (H2D of x, D2H of y inside) ----
    e2e_steps = max(1, min(args.steps, 5))
    if args.quick:
        sampler.stop_flag = True
        if rank == 0:
            for c, ms in zip(cases, per_case_ms):
                print(f"{c.name} b={c.bits} M={c.M} [{c.variant}, {c.layout_name}]: {ms * 1e3 / c.pool:.3f} us/call, "
                      f"{c.bytes / (ms * 1e-3 / c.pool) / 1e9:.1f} GB/s")
        if dist is not None:
            dist.destroy_process_group()
        return
    with torch.cuda.stream(stream):
        for c in cases[:n_main]:
            c.call_host(0)
        barrier()
        w0 = time.perf_counter()
        for _ in range(e2e_steps):
            for c in cases[:n_main]:
                for i in range(c.pool):
                    c.call_host(i)
        torch.cuda.synchronize()
        e2e_s = time.perf_counter() - w0
    if dist is not None:
        t = torch.tensor([e2e_s], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_s = float(t.item())
    e2e_value = world * step_bytes * e2e_steps / e2e_s / 1e9
    h2d = sum(c.M * c.K * 2 * c.pool for c in cases[:n_main])
    d2h = sum(c.M * c.N * 2 * c.pool for c in cases[:n_main])

    sampler.stop_flag = True
    sampler.join(timeout=1.0)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- parity spot check of what was just timed (rank 0): sampled output rows against the oracle ----
    from oracle import kmq_oracle as orc
    worst = 0.0
    checked = 0
    for ci, c in enumerate(cases):
        rows = c.check_rows
        ref_packed = orc.pack_canonical(c.check_idx, c.bits)
        cb_rows = c.check_cb
        d_rows = torch.from_numpy(rows).cuda()
        for i in sorted({0, c.pool - 1}):
            if c.dequant:
                got = c.W[i][d_rows].cpu().numpy().view(np.uint16)
                ok = np.array_equal(got, orc.dequant_bits(ref_packed, cb_rows, c.K, c.bits))
                worst = max(worst, 0.0 if ok else float("inf"))
            else:
                x_i = c.x_host[i].numpy().view(np.uint16)
                y_ref, s = orc.linear_f64(ref_packed, cb_rows, x_i, c.K, c.bits)
                y = c.y[i][:, d_rows].cpu().numpy().view(np.uint16)
                worst = max(worst, orc.check_linear(y, y_ref, s))
                if ci < n_main:                  # the end-to-end leg ran on the workload's own cases
                    yh = c.y_host[i].numpy().view(np.uint16)[:, rows]
                    worst = max(worst, orc.check_linear(yh, y_ref, s))
            checked += 1

    # ---- per-case figures and the roofline of the dominant kernel ----
    per_case = []
    floor_us = machine["launch_floor_us"] if machine else None
    for ci, (c, ms, sem) in enumerate(zip(cases, per_case_ms, per_case_sem_ms)):
        us = ms * 1e3 / c.pool
        gbs = c.bytes / (us * 1e-6) / 1e9
        ideal_us = c.bytes / (peak_gbs * 1e9) * 1e6
        per_case.append({"layer": c.name, "N": c.N, "K": c.K, "bits": c.bits, "M": c.M, "pool": c.pool,
                         "variant": c.variant, "layout": c.layout_name, "launches_per_call": c.launches,
                         "us_per_call": round(us, 3), "us_per_call_sem": round(sem * 1e3 / c.pool, 4),
                         "gbs": round(gbs, 1), "frac_of_measured_hbm": round(gbs / peak_gbs, 4),
                         "frac_of_8tbs": round(gbs / 8000.0, 4), "bytes_per_call": c.bytes,
                         "ideal_us_at_measured_hbm": round(ideal_us, 3), "launch_floor_us": floor_us,
                         "in_value": ci < n_main,
                         "weights": "random indices, timing only" if c.random_weights else "k-means fit"})
    # the kernel with the largest share of the step: achieved = algorithmic bytes of one call / time of one call
    # (a call of two launches still moves its bytes once)
    dom = max(range(n_main), key=lambda j: per_case_ms[j])
    dc = cases[dom]
    achieved = per_case[dom]["gbs"]
    roofline = {"bound": "hbm", "kernel": f"kmq_linear[{dc.variant}] b={dc.bits} M={dc.M} {dc.N}x{dc.K}",
                "achieved": round(achieved, 1), "peak": peak_gbs, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                "frac": round(achieved / peak_gbs, 4),
                "traffic": NCU_TRAFFIC_BYTES.get((dc.N, dc.K, dc.bits, dc.M, dc.variant)),
                "algorithmic_bytes_per_launch": dc.bytes,
                "share_of_step": round(per_case_ms[dom] / sum(per_case_ms[:n_main]), 3)}
    for row, c in zip(per_case, cases):
        row["ncu_dram_bytes"] = NCU_TRAFFIC_BYTES.get((c.N, c.K, c.bits, c.M, c.variant))

    cpu = cpu_baseline(args.workload, budget_s=args.cpu_seconds)

    line = {
        "metric": "kmq_linear effective HBM bandwidth (algorithmic bytes / time), batch-1 k-means LUT GEMV",
        "value": round(value, 2), "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": round(elapsed_ms / args.steps, 5), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{args.workload}: {WORKLOAD_TEXT[args.workload]}",
                   "calls_per_step": step_calls, "bytes_per_step": step_bytes,
                   "l2": "inputs larger than L2: every call of a step uses its own weight set, pool >= 2 x 126 MB",
                   "launch": "CUDA graph per case, replayed once per step", "multi_gpu": "replicas only",
                   "packed_layout": "per case the layout kmq_preferred_layout names (see per_case), packed once by "
                                    "kmq_pack before the timed region"},
        "frac_of_measured_hbm": round(value / world / peak_gbs, 4),
        "us_per_call_mean": round(elapsed_ms * 1e3 / args.steps / step_calls, 3),
        "per_case": per_case,
        "roofline": roofline,
        "cpu_baseline": cpu,
        "e2e": {"value": round(e2e_value, 2), "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps, "api": "kmq_linear_host (x from pinned host memory, y back to host, per call)"},
        "gpu_launches": args.steps * sum(c.pool * c.launches for c in cases[:n_main]),
        "machine": machine,
        "clocks": sampler.summary(),
        "parity": {"calls_checked": checked, "max_err_over_tol": round(worst, 4), "ok": bool(worst <= 1.0)},
        "paper_context": PAPER_CONTEXT,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


# --------------------------------------------------------------------------
# the CPU oracle, timed (reported baseline and the reference arm)
# --------------------------------------------------------------------------
# The paper's own kernel timings (Appendix "Benchmarking", table of the 1 x 8192 by 8192 x 8192 product at batch 1).
# Other hardware and another format: context only, not a target and not comparable row by row.
PAPER_CONTEXT = {
    "note": "paper's numbers: one NVIDIA L40S (864 GB/s), shared 256-entry byte LUT + bf16 block scales (B = 64), "
            "Triton kernels, 8192 x 8192 at batch 1; context only",
    "bf16_16bit": {"us": 175.6, "gbs": 764, "frac_of_l40s_peak": 0.88},
    "kmeans_4p25bit": {"us": 49.5, "gbs": 721, "frac_of_l40s_peak": 0.83},
    "kmeans_1p25bit": {"us": 24.0, "gbs": 438, "frac_of_l40s_peak": 0.51},
}


def _cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return len(os.sched_getaffinity(0))


ORACLE_MAX_WEIGHTS = 1 << 24     # per oracle call: larger layers are timed on their first rows only


def _oracle_cases(workload):
    """(N_sample, K, bits, M, packed rows, codebook rows, x, bytes of the sample) per case of the workload."""
    from oracle import kmq_oracle as orc
    from paper_2602_15563_b200 import synth
    out = []
    for (name, N, K, d, b, M) in WORKLOADS[workload]:
        n = int(min(N, max(16, ORACLE_MAX_WEIGHTS // K)))
        if d == "random":
            rng = np.random.default_rng(1000 * CONFIG_ID[workload] + 10 * b + M)
            idx = rng.integers(0, 1 << b, size=(n, K), dtype=np.uint8)
            cbs = synth.f32_to_bf16_bits(np.sort(rng.standard_normal((n, 1 << b)) * 0.02, axis=1).astype(np.float32))
        else:
            layer = cached_layer(synth, N, K, b, d, CONFIG_ID[workload])
            idx, cbs = layer["idx"][:n], layer["codebooks"][:n]
        x = synth.draw_activations(max(M, 1), K, synth.rng_for(CONFIG_ID[workload], synth.TENSOR_X))
        out.append((n, K, b, M, orc.pack_canonical(idx, b), cbs, x, algorithmic_bytes(n, K, b, M)))
    return out


def _oracle_call(orc, case):
    n, K, b, M, packed, cb, x, _bytes = case
    if M == 0:
        orc.dequant_bits(packed, cb, K, b)
    else:
        orc.linear_f64(packed, cb, x, K, b)


def cpu_baseline(workload, budget_s=12.0, cases=None):
    """Time the oracle's inference part (unpack, table lookup, float64 matmul) on the host cores, on a bounded
    sample of the workload: every case once per pass, layers larger than ORACLE_MAX_WEIGHTS cut to their first rows."""
    from oracle import kmq_oracle as orc
    cases = cases or _oracle_cases(workload)
    _oracle_call(orc, cases[0])                                   # warm-up
    total_bytes, n_calls = 0, 0
    t0 = time.perf_counter()
    while True:
        for case in cases:
            _oracle_call(orc, case)
            total_bytes += case[7]
            n_calls += 1
        if time.perf_counter() - t0 >= budget_s or n_calls >= 1000:
            break
    dt = time.perf_counter() - t0
    rows = sorted({c[0] for c in cases})
    return {"value": round(total_bytes / dt / 1e9, 4), "unit": "GB/s", "cores": _cpu_threads(),
            "host_cores": len(os.sched_getaffinity(0)), "kind": "oracle",
            "sample": f"{n_calls} oracle calls ({n_calls // len(cases)} pass(es) over the {len(cases)} cases of "
                      f"{workload}, one weight set each, first {rows} rows of each layer), {dt:.1f} s",
            "us_per_call": round(dt / n_calls * 1e6, 1)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    world = int(os.environ.get("WORLD_SIZE", "1"))
    from oracle import kmq_oracle as orc
    cases = _oracle_cases(args.workload)
    step_bytes = sum(c[7] for c in cases)

    def step():
        for case in cases:
            _oracle_call(orc, case)

    steps = max(1, min(args.steps, 40))
    for _ in range(max(1, min(args.warmup, 3))):
        step()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    dt = time.perf_counter() - t0
    value = step_bytes * steps / dt / 1e9
    cores = _cpu_threads()
    sample = (f"one oracle call per case of {args.workload} per step ({len(cases)} calls, first "
              f"{sorted({c[0] for c in cases})} rows of each layer), {steps} steps")
    line = {
        "impl": "reference",
        "metric": "kmq_linear effective HBM bandwidth (algorithmic bytes / time), batch-1 k-means LUT GEMV",
        "value": round(value, 4), "unit": "GB/s", "n_gpus": world, "steps": steps, "warmup": max(1, min(args.warmup, 3)),
        "ms_per_step": round(dt / steps * 1e3, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{args.workload}: {WORKLOAD_TEXT[args.workload]}", "calls_per_step": len(cases),
                   "bytes_per_step": step_bytes},
        "cpu_baseline": {"value": round(value, 4), "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": round(value, 4), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="kmq", choices=["kmq", "reference"])
    ap.add_argument("--workload", default="config2", choices=sorted(WORKLOADS) + sorted(DECODE_MODELS) + ["large_batch", "block", "quantize"])
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--case", default="", help='subset of the workload, e.g. "bits=1,M=1" (keys: layer, N, K, bits, M)')
    ap.add_argument("--layout", default="auto", choices=["auto", "tuned", "table", "canonical"],
                    help="packed layout of the weights (auto = kmq_preferred_layout per case)")
    ap.add_argument("--no-extra", action="store_true",
                    help="config2 only: skip the three larger cases timed next to the workload (outside `value`)")
    ap.add_argument("--quick", action="store_true",
                    help="kernel timing only (no end-to-end leg, CPU baseline or parity check): for profiler runs")
    args = ap.parse_args()
    if args.impl == "reference":
        if args.workload in DECODE_MODELS or args.workload in ("large_batch", "block", "quantize"):
            raise SystemExit("the reference arm times the oracle on the layer workloads (config*, tiny, large)")
        run_reference(args)
    elif args.workload in DECODE_MODELS:
        run_decode(args)
    elif args.workload == "large_batch":
        run_large_batch(args)
    elif args.workload == "block":
        run_block(args)
    elif args.workload == "quantize":
        run_quantize(args)
    else:
        run_library(args)


if __name__ == "__main__":
    main()
