#!/usr/bin/env python
"""Benchmark of the W2A8 hot path on B200 (one process per GPU).

Workload (N = 1 and every rank of N > 1: independent replicas, no exchange):
one Llama-3-8B-shaped decoder layer -- q/o 4096x4096, k/v 4096x1024, gate/up
4096x14336, down 14336x4096 (K x N), group 64 -- run as four a8_quantize calls
and seven w2a8_gemm calls, for M = 1, 4 and 16 tokens.  One "step" is those
three passes.  Weights are packed ahead of time; successive passes rotate over
distinct resident copies of the layer so that every timed weight byte comes
from HBM, not L2.  Metric: algorithmic bytes (packed weights + scales + int8
activations + fp32 outputs of every GEMM) per second.

`python bench.py --impl reference` times the scalar CPU reference on the same
workload (a bounded sample per step) instead.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2508_06753_b200 import synth

CFG_INDEX = 1
METRIC = "W2A8 GEMM HBM GB/s at M=1-16 (Llama-3-8B decoder-layer linears, M in {1,4,16}, group 64)"
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the decode kernel on the
# 4096x14336, M=1, group-64 GEMM (ncu capture of one launch); the algorithmic bytes of that
# launch are 18,411,524.
NCU_TRAFFIC_BYTES_GATE_M1 = 18_378_752


# --------------------------------------------------------------------- accounting
def gemm_bytes(M, N, K, g):
    """Algorithmic bytes of one GEMM: packed weights + scales + int8 activations
    (+ their scales) + fp32 outputs."""
    return K * N // 4 + (K // g) * N * 4 + M * K + 4 * M + 4 * M * N


def layer_bytes(cfg, M):
    return sum(gemm_bytes(M, N, K, synth.config_group(cfg, K)) for _, K, N in cfg["shapes"])


def step_bytes(cfg):
    return sum(layer_bytes(cfg, M) for M in cfg["Ms"])


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# ------------------------------------------------------------------ distributed glue
def dist_setup(n_gpus):
    """Initialise torch.distributed when launched under torchrun; returns (rank, world)."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        if not dist.is_initialized():
            backend = os.environ.get("W2A8_BENCH_BACKEND", "nccl")
            dist.init_process_group(backend=backend)
    return rank, world


def dist_barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def aggregate(elapsed_ms: float, units: float, device=None):
    """Whole-job figures from per-rank ones: time = max over ranks, units = sum."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return elapsed_ms, units
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=device)
    u = torch.tensor([units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


# ------------------------------------------------------------------------- clocks
REASON_BITS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
               0x2: "applications_clocks_setting", 0x10: "sync_boost"}


class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons through NVML (read-only)."""

    def __init__(self, index, period_s=0.004):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples = []          # (t, sm_mhz, reasons_bitmask)
        self.max_mhz = None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def _reasons(self):
        for name in ("nvmlDeviceGetCurrentClocksEventReasons", "nvmlDeviceGetCurrentClocksThrottleReasons"):
            fn = getattr(self.nv, name, None)
            if fn is not None:
                try:
                    return int(fn(self.h))
                except Exception:
                    continue
        return 0

    def run(self):
        if not self.ok:
            return
        while not self._stop_evt.is_set():
            try:
                mhz = int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
                self.samples.append((time.perf_counter(), mhz, self._reasons()))
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()

    def summary(self, t0, t1):
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        window = "timed region"
        if len(inside) < 3:
            inside = self.samples
            window = "warm-up + timed region (timed region too short for 3 samples)"
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0,
                    "window": "unavailable"}
        bits = 0
        for s in inside:
            bits |= s[2]
        reasons = sorted(v for k, v in REASON_BITS.items() if bits & k)
        return {"sm_mhz": float(np.median([s[1] for s in inside])), "sm_max_mhz": self.max_mhz,
                "reasons": reasons, "samples": len(inside), "window": window}


# ---------------------------------------------------------------------- GPU arm
class LayerReplica:
    """R resident copies of one layer's packed weights plus the activation,
    output and workspace buffers for each M (device memory only)."""

    def __init__(self, cfg, copies, device):
        import torch
        from paper_2508_06753_b200 import binding as b
        self.torch, self.b, self.cfg = torch, b, cfg
        self.shapes = cfg["shapes"]
        self.copies = []
        for c in range(copies):
            mats = []
            for idx, (name, K, N) in enumerate(self.shapes):
                g = synth.config_group(cfg, K)
                codes, s_w = synth.make_linear(synth.shape_seed(cfg, idx) + 100 * c, K, N, g,
                                               cfg["ternary"])
                packed = b.w2_pack(torch.from_numpy(codes).to(device))
                mats.append((packed, torch.from_numpy(s_w).to(device), g))
            self.copies.append(mats)
        torch.cuda.synchronize()
        # inputs of the layer: which linear reads which activation
        self.input_of = {"q": "attn_in", "k": "attn_in", "v": "attn_in", "o": "o_in",
                         "gate": "mlp_in", "up": "mlp_in", "down": "down_in", "gemv": "attn_in"}
        self.per_m = {}
        ws_bytes = 256
        for M in cfg["Ms"]:
            bufs = {"x": {}, "a": {}, "s": {}, "y": []}
            for idx, (name, K, N) in enumerate(self.shapes):
                inp = self.input_of[name]
                if inp not in bufs["x"]:
                    bits = synth.activations_bf16(cfg["seed"] + 50 + len(bufs["x"]), M, K,
                                                  cfg["outlier_frac"])
                    bufs["x"][inp] = torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)
                    bufs["a"][inp] = torch.empty((M, K), dtype=torch.int8, device=device)
                    bufs["s"][inp] = torch.empty((M,), dtype=torch.float32, device=device)
                bufs["y"].append(torch.empty((M, N), dtype=torch.float32, device=device))
                ws_bytes = max(ws_bytes, b.w2a8_workspace_bytes(M, N, K, synth.config_group(cfg, K)))
            self.per_m[M] = bufs
        self.ws = b.new_workspace(ws_bytes, device=device)
        self.kernels_per_pass = len(self.shapes) + len(set(self.input_of[n] for n, _, _ in self.shapes))

    def run_pass(self, M, copy):
        b, bufs = self.b, self.per_m[M]
        done = set()
        for idx, (name, K, N) in enumerate(self.shapes):
            inp = self.input_of[name]
            if inp not in done:
                b.a8_quantize(bufs["x"][inp], bufs["a"][inp], bufs["s"][inp])
                done.add(inp)
            packed, s_w, g = self.copies[copy][idx]
            b.w2a8_gemm(bufs["a"][inp], bufs["s"][inp], packed, s_w, g, self.ws, bufs["y"][idx])

    def run_step(self, step_index):
        n = len(self.copies)
        for j, M in enumerate(self.cfg["Ms"]):
            self.run_pass(M, (step_index * len(self.cfg["Ms"]) + j) % n)


def build_step_graphs(rep, use_graph):
    """One CUDA graph per rotation phase (falls back to direct launches)."""
    torch = rep.torch
    n_phase = len(rep.copies)
    if not use_graph:
        return [lambda i=i: rep.run_step(i) for i in range(n_phase)], "direct"
    try:
        graphs = []
        stream = torch.cuda.Stream()
        stream.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(stream):
            for i in range(n_phase):
                rep.run_step(i)                       # warm, outside capture
            torch.cuda.synchronize()
            for i in range(n_phase):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    rep.run_step(i)
                graphs.append(g)
        torch.cuda.current_stream().wait_stream(stream)
        torch.cuda.synchronize()
        return [g.replay for g in graphs], "cuda_graph"
    except Exception as e:  # capture not possible: time direct launches instead
        sys.stderr.write(f"[bench] graph capture failed ({e}); timing direct launches\n")
        torch.cuda.synchronize()
        return [lambda i=i: rep.run_step(i) for i in range(n_phase)], "direct"


def time_steps(torch, runners, steps, warmup):
    for i in range(warmup):
        runners[i % len(runners)]()
    torch.cuda.synchronize()
    dist_barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e0.record()
    for i in range(steps):
        runners[i % len(runners)]()
    e1.record()
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    dist_barrier()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1), t0, t1


def kernel_probe(rep, M, shape_idx, reps=30):
    """Average duration of one decode-GEMM launch on its own: the same kernel and
    launch configuration the step uses, launched back to back over rotating
    weight copies (all copies of the shape together exceed 2x L2), CUDA events
    on the launching stream."""
    torch, b = rep.torch, rep.b
    name, K, N = rep.shapes[shape_idx]
    bufs = rep.per_m[M]
    inp = rep.input_of[name]
    mats = [c[shape_idx] for c in rep.copies]
    # gate and up have the same shape: use both for rotation
    twins = [i for i, (_, k2, n2) in enumerate(rep.shapes) if (k2, n2) == (K, N) and i != shape_idx]
    for t in twins:
        mats += [c[t] for c in rep.copies]
    distinct = sum(m[0].numel() * 4 + m[1].numel() * 4 for m in mats)
    b.a8_quantize(bufs["x"][inp], bufs["a"][inp], bufs["s"][inp])
    y = bufs["y"][shape_idx]

    def body():
        for packed, s_w, g in mats:
            b.w2a8_gemm(bufs["a"][inp], bufs["s"][inp], packed, s_w, g, rep.ws, y)
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(stream):
        body()
        torch.cuda.synchronize()
        try:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                body()
            run = g.replay
        except Exception:
            run = body
        for _ in range(3):
            run()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            run()
        e1.record()
        torch.cuda.synchronize()
    torch.cuda.current_stream().wait_stream(stream)
    ms = e0.elapsed_time(e1) / (reps * len(mats))
    return dict(shape=f"{K}x{N}", M=M, us_per_launch=ms * 1e3,
                bytes_per_launch=gemm_bytes(M, N, K, mats[0][2]),
                gbs=gemm_bytes(M, N, K, mats[0][2]) / (ms * 1e-3) / 1e9,
                distinct_weight_bytes=distinct, launches=reps * len(mats))


def small_shape_probe(device, peaks, l2_bytes, reps=20):
    """Extra rows (not the headline): the small square-ish matrices the paper also times (Sec. III:
    1600x1600, 2560x2560, 3840x2560, 3200x3200), where launch latency dominates.  One GEMV (M = 1,
    group 64) per launch, back to back in a CUDA graph over enough distinct weight copies to exceed
    twice the L2."""
    import torch
    from paper_2508_06753_b200 import binding as b
    rows = []
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    for K, N in ((1600, 1600), (2560, 2560), (2560, 3840), (3200, 3200)):
        g, M = 64, 1
        codes, s_w = synth.make_linear(K + N, K, N, g)
        packed = b.w2_pack(torch.from_numpy(codes).to(device))
        sw = torch.from_numpy(s_w).to(device)
        per = packed.numel() * 4 + sw.numel() * 4
        ncopy = int(np.ceil(2.2 * l2_bytes / per))
        mats = [(packed.clone(), sw.clone()) for _ in range(ncopy)]
        x = torch.from_numpy(synth.activations_bf16(K, M, K).view(np.int16)).to(device).view(torch.bfloat16)
        a, s_a = b.a8_quantize(x)
        y = torch.empty((M, N), dtype=torch.float32, device=device)
        ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g), device=device)

        def body():
            for pk, sc in mats:
                b.w2a8_gemm(a, s_a, pk, sc, g, ws, y)
        with torch.cuda.stream(stream):
            body()
            torch.cuda.synchronize()
            try:
                gr = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gr, stream=stream):
                    body()
                run = gr.replay
            except Exception:
                run = body
            for _ in range(3):
                run()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                run()
            e1.record()
            torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / (reps * ncopy)
        nbytes = gemm_bytes(M, N, K, g)
        rows.append({"shape": f"{K}x{N}", "M": M, "group": g, "us_per_launch": us, "bytes_per_launch": nbytes,
                     "gbs": nbytes / us / 1e3, "frac_of_measured_hbm": nbytes / us / 1e3 / peaks["hbm_gbs"],
                     "weight_copies": ncopy})
        del mats
    torch.cuda.current_stream().wait_stream(stream)
    return rows


def concat_probe(rep, reps=200):
    """Extra row (not the headline): the same layer with q|k|v and gate|up concatenated along N,
    i.e. 4 GEMMs + 4 a8_quantize per pass instead of 7 + 4.  Packed rows are independent, so the
    concatenated matrix is the row-wise concatenation of the packed matrices.  Reported with the
    headline's byte count so that the two are comparable."""
    torch, b, cfg = rep.torch, rep.b, rep.cfg
    names = [n for n, _, _ in rep.shapes]
    if not all(n in names for n in ("q", "k", "v", "o", "gate", "up", "down")):
        return None
    ix = {n: names.index(n) for n in names}
    fused = []
    for mats in rep.copies:
        def cat(group):
            return (torch.cat([mats[ix[n]][0] for n in group], 0).contiguous(),
                    torch.cat([mats[ix[n]][1] for n in group], 0).contiguous(), mats[ix[group[0]]][2])
        fused.append({"qkv": cat(("q", "k", "v")), "o": mats[ix["o"]], "gateup": cat(("gate", "up")),
                      "down": mats[ix["down"]]})
    out = {}
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(stream):
        for M in cfg["Ms"]:
            bufs = rep.per_m[M]
            ys = {k: torch.empty((M, v[0].shape[0]), dtype=torch.float32, device=v[0].device)
                  for k, v in fused[0].items()}
            ws = b.new_workspace(max(b.w2a8_workspace_bytes(M, v[0].shape[0], v[0].shape[1] * 16, v[2])
                                     for v in fused[0].values()), device=ys["o"].device)
            plan = (("attn_in", "qkv"), ("o_in", "o"), ("mlp_in", "gateup"), ("down_in", "down"))

            def one_pass(c):
                for inp, key in plan:
                    b.a8_quantize(bufs["x"][inp], bufs["a"][inp], bufs["s"][inp])
                    packed, s_w, g = fused[c][key]
                    b.w2a8_gemm(bufs["a"][inp], bufs["s"][inp], packed, s_w, g, ws, ys[key])
            for c in range(len(fused)):
                one_pass(c)
            torch.cuda.synchronize()
            try:
                gr = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gr, stream=stream):
                    for c in range(len(fused)):
                        one_pass(c)
                run = gr.replay
            except Exception:
                def run():
                    for c in range(len(fused)):
                        one_pass(c)
            for _ in range(3):
                run()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            n = max(reps // len(fused), 3)
            e0.record()
            for _ in range(n):
                run()
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / (n * len(fused))
            out[str(M)] = {"us_per_layer": ms * 1e3, "gbs": layer_bytes(cfg, M) / (ms * 1e-3) / 1e9}
    torch.cuda.current_stream().wait_stream(stream)
    return {"what": "q|k|v and gate|up concatenated along N: 4 GEMMs + 4 a8_quantize per layer pass; "
                    "GB/s uses the byte count of the 7-GEMM layer", "per_m": out}


def recipe16_probe(rep, peaks, group=128, reps=200):
    """Extra row (not the headline): the same layer stored the way the paper's end-to-end ternary
    section describes -- groups of 128 along K, binary16 weight scales -- with bf16 results, through
    w2a8_gemm_h16: 7 GEMMs + 4 a8_quantize per pass.  GB/s uses this recipe's own (smaller) byte
    count: 2 + 16/128 bit per weight, 2 bytes per result."""
    torch, b, cfg = rep.torch, rep.b, rep.cfg
    dev = rep.ws.device

    def bytes_of(M, N, K):
        return K * N // 4 + (K // group) * N * 2 + M * K + 4 * M + 2 * M * N

    copies = []
    for c in range(len(rep.copies)):
        mats = []
        for idx, (name, K, N) in enumerate(rep.shapes):
            if K % group:
                return None
            s_h = synth.weight_scales_h(synth.shape_seed(cfg, idx) + 100 * c, N, K // group)
            mats.append((rep.copies[c][idx][0], torch.from_numpy(s_h.view(np.int16)).to(dev).view(torch.float16)))
        copies.append(mats)
    out = {}
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(stream):
        for M in cfg["Ms"]:
            bufs = rep.per_m[M]
            ys = [torch.empty((M, N), dtype=torch.bfloat16, device=dev) for _, _, N in rep.shapes]
            ws = b.new_workspace(max(b.w2a8_workspace_bytes(M, N, K, group) for _, K, N in rep.shapes), device=dev)

            def one_pass(c):
                done = set()
                for idx, (name, K, N) in enumerate(rep.shapes):
                    inp = rep.input_of[name]
                    if inp not in done:
                        b.a8_quantize(bufs["x"][inp], bufs["a"][inp], bufs["s"][inp])
                        done.add(inp)
                    packed, s_h = copies[c][idx]
                    b.w2a8_gemm_h16(bufs["a"][inp], bufs["s"][inp], packed, s_h, group, ws, ys[idx])
            for c in range(len(copies)):
                one_pass(c)
            torch.cuda.synchronize()
            try:
                gr = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gr, stream=stream):
                    for c in range(len(copies)):
                        one_pass(c)
                run = gr.replay
            except Exception:
                def run():
                    for c in range(len(copies)):
                        one_pass(c)
            for _ in range(3):
                run()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            n = max(reps // len(copies), 3)
            e0.record()
            for _ in range(n):
                run()
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / (n * len(copies))
            nbytes = sum(bytes_of(M, N, K) for _, K, N in rep.shapes)
            out[str(M)] = {"us_per_layer": ms * 1e3, "bytes_per_layer": nbytes,
                           "gbs": nbytes / (ms * 1e-3) / 1e9,
                           "frac_of_measured_hbm": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    torch.cuda.current_stream().wait_stream(stream)
    return {"what": f"group {group}, binary16 weight scales, bf16 results (w2a8_gemm_h16): 7 GEMMs + 4 "
                    "a8_quantize per layer pass; GB/s on this recipe's own byte count", "per_m": out}


def a16_probe(rep, peaks, reps=200):
    """Extra row (not the headline): the same layer through w2a16_gemm -- bf16 activations against
    the 2-bit weights, no activation quantiser: 7 launches per pass instead of 11.  GB/s on this
    entry's own byte count (bf16 activations: 2 bytes each, no token scales)."""
    torch, b, cfg = rep.torch, rep.b, rep.cfg
    dev = rep.ws.device

    def bytes_of(M, N, K, g):
        return K * N // 4 + (K // g) * N * 4 + 2 * M * K + 4 * M * N

    out = {}
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(stream):
        for M in cfg["Ms"]:
            bufs = rep.per_m[M]

            def one_pass(c):
                for idx, (name, K, N) in enumerate(rep.shapes):
                    packed, s_w, g = rep.copies[c][idx]
                    b.w2a16_gemm(bufs["x"][rep.input_of[name]], packed, s_w, g, rep.ws, bufs["y"][idx])
            for c in range(len(rep.copies)):
                one_pass(c)
            torch.cuda.synchronize()
            try:
                gr = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gr, stream=stream):
                    for c in range(len(rep.copies)):
                        one_pass(c)
                run = gr.replay
            except Exception:
                def run():
                    for c in range(len(rep.copies)):
                        one_pass(c)
            for _ in range(3):
                run()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            n = max(reps // len(rep.copies), 3)
            e0.record()
            for _ in range(n):
                run()
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / (n * len(rep.copies))
            nbytes = sum(bytes_of(M, N, K, synth.config_group(cfg, K)) for _, K, N in rep.shapes)
            out[str(M)] = {"us_per_layer": ms * 1e3, "bytes_per_layer": nbytes, "gbs": nbytes / (ms * 1e-3) / 1e9,
                           "frac_of_measured_hbm": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    torch.cuda.current_stream().wait_stream(stream)
    return {"what": "w2a16_gemm (bf16 activations, no a8_quantize): 7 launches per layer pass; GB/s on this "
                    "entry's own byte count", "per_m": out}


def e2e_measure(rep, steps, warmup):
    """Same workload through w2a8_linear_host: pinned host activations in, host
    outputs back, copies inside the timed region."""
    torch, b, cfg = rep.torch, rep.b, rep.cfg
    dev = rep.ws.device
    host = {}
    h2d = d2h = 0
    ws_bytes = 256
    for M in cfg["Ms"]:
        xs, ys = [], []
        for idx, (name, K, N) in enumerate(rep.shapes):
            src = rep.per_m[M]["x"][rep.input_of[name]]
            xs.append(src.cpu().pin_memory())
            ys.append(torch.empty((M, N), dtype=torch.float32).pin_memory())
            h2d += M * K * 2
            d2h += M * N * 4
            ws_bytes = max(ws_bytes, b.w2a8_linear_host_workspace_bytes(M, N, K, synth.config_group(cfg, K)))
        host[M] = (xs, ys)
    ws = b.new_workspace(ws_bytes, device=dev)

    def step(i):
        n = len(rep.copies)
        for j, M in enumerate(cfg["Ms"]):
            copy = (i * len(cfg["Ms"]) + j) % n
            xs, ys = host[M]
            for idx in range(len(rep.shapes)):
                packed, s_w, g = rep.copies[copy][idx]
                b.w2a8_linear_host(xs[idx], packed, s_w, g, ys[idx], ws)

    for i in range(max(warmup, 3)):
        step(i)
    torch.cuda.synchronize()
    dist_barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        step(i)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    checksum = float(sum(float(y.sum()) for y in host[cfg["Ms"][0]][1]))
    return ms, h2d, d2h, checksum


class OracleWorkload:
    """The scalar reference on the same workload; a step may cover only the
    first n output channels of every linear (channels are independent), so a
    step can be sized to a time budget."""

    def __init__(self, cfg):
        import oracle
        oracle.build()
        self.oracle, self.cfg = oracle, cfg
        self.mats = []
        for idx, (name, K, N) in enumerate(cfg["shapes"]):
            g = synth.config_group(cfg, K)
            codes, s_w = synth.make_linear(synth.shape_seed(cfg, idx), K, N, g, cfg["ternary"])
            self.mats.append((codes, s_w, g, K, N))
        self.acts = {M: {K: synth.activations_bf16(cfg["seed"] + 50, M, K, cfg["outlier_frac"])
                         for K in sorted({m[3] for m in self.mats})} for M in cfg["Ms"]}

    def step(self, frac):
        """Returns (algorithmic bytes processed, seconds)."""
        nbytes = 0
        t0 = time.perf_counter()
        for M in self.cfg["Ms"]:
            q = {K: self.oracle.quantize(x) for K, x in self.acts[M].items()}
            for codes, s_w, g, K, N in self.mats:
                n = min(N, max(16, int(N * frac) // 16 * 16))
                a, s_a = q[K]
                self.oracle.gemm(a, s_a, codes[:n], s_w[:n], g)
                nbytes += gemm_bytes(M, n, K, g)
        return nbytes, time.perf_counter() - t0

    def frac_for(self, seconds_per_step):
        _, dt = self.step(1.0 / 64)
        _, dt = self.step(1.0 / 64)
        return float(min(1.0, max(1.0 / 896, (1.0 / 64) * seconds_per_step / max(dt, 1e-6))))


def cpu_baseline(cfg, budget_s=20.0, min_wall_s=1.5):
    """The reference as it stands on this machine's host cores, on a bounded
    sample of the benchmark workload: whole steps (restricted to a leading
    fraction of the output channels if one step alone would exceed `budget_s`),
    repeated until about `min_wall_s` seconds of wall time have been measured."""
    w = OracleWorkload(cfg)
    frac = w.frac_for(budget_s)
    tot_b, tot_s, n = 0, 0.0, 0
    while tot_s < min_wall_s and n < 64:
        nbytes, dt = w.step(frac)
        tot_b += nbytes
        tot_s += dt
        n += 1
    cores = w.oracle.num_threads()
    return dict(value=tot_b / tot_s / 1e9, unit="GB/s", cores=cores, kind="oracle",
                seconds=tot_s, cpu_core_seconds=tot_s * cores,
                sample=f"{n} step(s) (M in {cfg['Ms']}, 4 quantise + 7 GEMM calls each) restricted to "
                       f"the first {frac:.4f} of the output channels of every linear")


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = synth.CONFIGS[CFG_INDEX]
    w = OracleWorkload(cfg)
    budget = 150.0                                    # whole run, seconds
    frac = w.frac_for(budget / (args.steps + args.warmup))
    for _ in range(args.warmup):
        w.step(frac)
    tot_b, tot_s = 0, 0.0
    for _ in range(args.steps):
        nb, dt = w.step(frac)
        tot_b += nb
        tot_s += dt
    value = tot_b / tot_s / 1e9
    sample = (f"each step: M in {cfg['Ms']}, 4 quantise + 7 GEMM calls, restricted to the first "
              f"{frac:.4f} of the output channels of every linear")
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": tot_s / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int8xint2->int32, fp64 scale sum", "data": "synthetic",
        "config": {"workload": "llama3-8b decoder-layer linears (q,k,v,o,gate,up,down), group 64, "
                               "M in {1,4,16}: configuration 1", "sample": sample},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": w.oracle.num_threads(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out))


def run_ours(args):
    import torch
    rank, world = dist_setup(args.gpus)
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    from paper_2508_06753_b200 import binding as b, build
    build.build()
    b.lib()
    cfg = synth.CONFIGS[CFG_INDEX]
    peaks = load_peaks()

    l2 = torch.cuda.get_device_properties(local).L2_cache_size
    per_copy = sum(K * N // 4 + (K // synth.config_group(cfg, K)) * N * 4 for _, K, N in cfg["shapes"])
    copies = max(2, int(np.ceil(2.0 * l2 / per_copy)))
    rep = LayerReplica(cfg, copies, device)

    sampler = ClockSampler(local)
    sampler.start()
    runners, mode = build_step_graphs(rep, not args.no_graph)
    ms, t0, t1 = time_steps(torch, runners, args.steps, args.warmup)
    sampler.stop()
    clocks = sampler.summary(t0, t1)

    units = step_bytes(cfg) * args.steps
    ms_all, units_all = aggregate(ms, units, device)
    value = units_all / (ms_all * 1e-3) / 1e9

    # per-M breakdown and single-kernel probe (rank 0, after the headline timing)
    per_m = {}
    probes = []
    e2e = None
    cpu = None
    if args.only_headline:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world,
                              "steps": args.steps, "warmup": args.warmup,
                              "ms_per_step": ms_all / args.steps, "launch": mode, "clocks": clocks,
                              "gpu_launches": args.steps * len(cfg["Ms"]) * rep.kernels_per_pass}))
        return
    if rank == 0:
        for M in cfg["Ms"]:
            sub = dict(cfg, Ms=[M])
            rep_m = rep
            saved = rep.cfg
            rep.cfg = sub
            r_m, _ = build_step_graphs(rep_m, not args.no_graph)
            ms_m, _, _ = time_steps_local(torch, r_m, max(args.steps // 2, 20), 5)
            rep.cfg = saved
            per_m[str(M)] = {"us_per_layer": ms_m * 1e3, "gbs": layer_bytes(cfg, M) / (ms_m * 1e-3) / 1e9}
        big = max(range(len(cfg["shapes"])), key=lambda i: cfg["shapes"][i][1] * cfg["shapes"][i][2])
        for M in cfg["Ms"]:
            probes.append(kernel_probe(rep, M, big))
    concat = concat_probe(rep) if rank == 0 else None
    recipe16 = recipe16_probe(rep, peaks) if rank == 0 else None
    small = small_shape_probe(device, peaks, l2) if rank == 0 else None
    a16 = a16_probe(rep, peaks) if rank == 0 else None
    prefill = None
    if rank == 0 and not args.no_prefill:
        prefill = prefill_probe(device, peaks)
    e2e_ms, h2d, d2h, _ = e2e_measure(rep, max(args.steps // 10, 10), 3)
    e2e_steps = max(args.steps // 10, 10)
    e2e_ms_all, e2e_units = aggregate(e2e_ms, step_bytes(cfg) * e2e_steps, device)
    e2e = {"value": e2e_units / (e2e_ms_all * 1e-3) / 1e9, "unit": "GB/s",
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
           "api": "w2a8_linear_host, one call per linear, pinned host buffers"}
    if rank != 0:
        return
    if world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(cfg, budget_s=20.0)

    dom = probes[0]
    roofline = {"bound": "hbm", "achieved": dom["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": dom["gbs"] / peaks["hbm_gbs"], "traffic": NCU_TRAFFIC_BYTES_GATE_M1,
                "peak_source": peaks["source"],
                "kernel": "w2a8_decode_kernel<MT=1,SPP=1,TG=1,RING=4,ONE> on gate/up 4096x14336, M=1 "
                          "(largest GEMV of the layer; the M=4 and M=16 instances are in roofline_by_m)",
                "bytes_per_launch": dom["bytes_per_launch"], "us_per_launch": dom["us_per_launch"],
                "frac_of_nominal_8TBs": dom["gbs"] / NOMINAL_HBM_GBS}
    roofline_by_m = [{"M": pr["M"], "shape": pr["shape"], "achieved": pr["gbs"], "unit": "GB/s",
                      "frac": pr["gbs"] / peaks["hbm_gbs"], "us_per_launch": pr["us_per_launch"]}
                     for pr in probes]
    out = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_all / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8xint2->int32, fp32 scales",
        "data": "synthetic",
        "config": {"workload": "llama3-8b decoder-layer linears (q,k,v,o,gate,up,down), group 64, "
                               "M in {1,4,16}: configuration 1",
                   "tokens_per_step": sum(cfg["Ms"]), "parallelism": f"replicas x{world}",
                   "launch": mode, "weight_copies": copies,
                   "l2_policy": f"inputs larger than L2: {copies} resident layer copies "
                                f"({copies * per_copy / 1e6:.0f} MB) rotated, L2 = {l2 / 1e6:.0f} MB"},
        "frac_of_measured_hbm": value / world / peaks["hbm_gbs"],
        "frac_of_nominal_8TBs": value / world / NOMINAL_HBM_GBS,
        "clocks": clocks, "e2e": e2e,
        "gpu_launches": args.steps * len(cfg["Ms"]) * rep.kernels_per_pass,
        "roofline": roofline, "roofline_by_m": roofline_by_m, "cpu_baseline": cpu, "per_m": per_m,
        "kernel_probes": probes, "concatenated_qkv_gateup": concat,
        "recipe_g128_binary16_scales_bf16_out": recipe16,
        "paper_small_shapes_m1": small,
        "w2a16_no_quantiser": a16,
        "prefill": prefill,
    }
    print(json.dumps(out))


def prefill_probe(device, peaks, Ms=(512, 2048, 8192), reps=5):
    """Tensor-core path on the prefill configuration: Llama-3-8B gate/up (K=4096, N=14336)
    and down (K=14336, N=4096), group 64.  int8 TOPS = 2*M*N*K / time, GEMM alone and
    with the a8_quantize pass; CUDA events on the launching stream."""
    import torch
    from paper_2508_06753_b200 import binding as b
    cfg = synth.CONFIGS[4]
    int8_peak_burst = 2.0 * peaks["bf16_tflops"]            # nominal int8 : bf16 ratio is 2
    int8_peak_sustained = 2.0 * peaks["bf16_tflops_sustained"]
    rows = []
    for idx, (name, K, N) in enumerate(cfg["shapes"]):
        g = synth.config_group(cfg, K)
        codes, s_w = synth.make_linear(synth.shape_seed(cfg, idx), K, N, g)
        packed = b.w2_pack(torch.from_numpy(codes).to(device))
        s_w_d = torch.from_numpy(s_w).to(device)
        del codes
        for M in Ms:
            bits = synth.activations_bf16(cfg["seed"] + 7 + M, M, K)
            x = torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)
            a, s_a = b.a8_quantize(x)
            y = torch.empty((M, N), dtype=torch.float32, device=device)
            ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g), device=device)

            def gemm():
                b.w2a8_gemm(a, s_a, packed, s_w_d, g, ws, y)

            def both():
                b.a8_quantize(x, a, s_a)
                b.w2a8_gemm(a, s_a, packed, s_w_d, g, ws, y)
            out = {}
            for label, fn in (("gemm", gemm), ("quantize+gemm", both)):
                for _ in range(3):
                    fn()
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(reps):
                    fn()
                e1.record()
                torch.cuda.synchronize()
                out[label] = e0.elapsed_time(e1) / reps
            ops = 2.0 * M * N * K
            tops = ops / (out["gemm"] * 1e-3) / 1e12
            rows.append({"shape": f"{K}x{N}", "M": M, "group": g,
                         "channels_on_tensor_cores": b.w2a8_tensor_core_channels(M, N, K, g),
                         "ms_gemm": out["gemm"],
                         "ms_quantize_gemm": out["quantize+gemm"], "tops": tops,
                         "tops_with_quantize": ops / (out["quantize+gemm"] * 1e-3) / 1e12,
                         "frac_of_measured_int8_burst": tops / int8_peak_burst,
                         "frac_of_measured_int8_sustained": tops / int8_peak_sustained,
                         "frac_of_nominal_4500": tops / 4500.0,
                         "status": b.w2a8_workspace_status(ws)})
            del x, a, y, ws
        del packed
    # the same kernel with coarser scale groups on gate/up at M = 2048: the per-group drain halves
    # (group 128), quarters (256) and all but vanishes (one scale per channel)
    by_group = []
    name, K, N = cfg["shapes"][0]
    M = 2048
    bits = synth.activations_bf16(cfg["seed"] + 7 + M, M, K)
    x = torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)
    a, s_a = b.a8_quantize(x)
    y = torch.empty((M, N), dtype=torch.float32, device=device)
    for g in (64, 128, 256, K):
        codes, s_w = synth.make_linear(synth.shape_seed(cfg, 0) + g, K, N, g)
        packed = b.w2_pack(torch.from_numpy(codes).to(device))
        s_w_d = torch.from_numpy(s_w).to(device)
        del codes
        ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g), device=device)
        for _ in range(3):
            b.w2a8_gemm(a, s_a, packed, s_w_d, g, ws, y)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            b.w2a8_gemm(a, s_a, packed, s_w_d, g, ws, y)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        tops = 2.0 * M * N * K / (ms * 1e-3) / 1e12
        by_group.append({"shape": f"{K}x{N}", "M": M, "group": g, "ms_gemm": ms, "tops": tops,
                         "frac_of_measured_int8_sustained": tops / int8_peak_sustained,
                         "status": b.w2a8_workspace_status(ws)})
        del packed, s_w_d, ws
    # library int8 GEMM on the same device as a second, directly measured denominator
    lib_int8 = None
    try:
        n = 8192
        ai = torch.randint(-127, 128, (n, n), dtype=torch.int8, device=device)
        bi = torch.randint(-127, 128, (n, n), dtype=torch.int8, device=device)
        for _ in range(3):
            torch._int_mm(ai, bi)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(10):
            torch._int_mm(ai, bi)
        e1.record()
        torch.cuda.synchronize()
        lib_int8 = {"what": "torch._int_mm 8192^3 (library int8 GEMM), 10 back-to-back calls",
                    "tops": 2.0 * n ** 3 / (e0.elapsed_time(e1) / 10 * 1e-3) / 1e12}
        del ai, bi
    except Exception as exc:      # not available in this torch build: report, do not fail the bench
        lib_int8 = {"what": "torch._int_mm 8192^3", "unavailable": str(exc)[:200]}
    return {"unit": "int8 TOPS", "peak_measured_burst": int8_peak_burst,
            "peak_measured_sustained": int8_peak_sustained,
            "peak_note": "measured cuBLAS bf16 peak x 2 (nominal int8 : bf16 ratio); nominal dense int8 4500",
            "library_int8_gemm": lib_int8, "rows": rows, "by_group_m2048": by_group}


def run_kernel_profile(args):
    """Small stand-alone run of one GEMM shape for profilers: a few direct
    launches of w2a8_gemm over rotating weight copies (total > 2x L2, a few
    hundred MB), timed with CUDA events.  Prints one JSON line."""
    import torch
    from paper_2508_06753_b200 import binding as b, build
    build.build()
    K, N = (int(v) for v in args.profile_shape.split("x"))
    M, g = args.profile_m, (args.profile_group or K)
    dev = torch.device("cuda", 0)
    l2 = torch.cuda.get_device_properties(0).L2_cache_size
    per = K * N // 4 + (K // g) * N * 4
    copies = max(2, int(np.ceil(2.0 * l2 / per)))
    mats = []
    for c in range(copies):
        codes, s_w = synth.make_linear(7000 + c, K, N, g)
        mats.append((b.w2_pack(torch.from_numpy(codes).to(dev)), torch.from_numpy(s_w).to(dev)))
    x = torch.from_numpy(synth.activations_bf16(7, M, K).view(np.int16)).to(dev).view(torch.bfloat16)
    a, s_a = b.a8_quantize(x)
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g), device=dev)
    y = torch.empty((M, N), dtype=torch.float32, device=dev)
    if args.profile_entry == "a16":
        def gemm(pk, sw):
            b.w2a16_gemm(x, pk, sw, g, ws, y)
    elif args.profile_entry == "h16":
        mats = [(pk, sw.half()) for pk, sw in mats]

        def gemm(pk, sw):
            b.w2a8_gemm_h16(a, s_a, pk, sw, g, ws, y)
    else:
        def gemm(pk, sw):
            b.w2a8_gemm(a, s_a, pk, sw, g, ws, y)
    for i in range(args.profile_reps):                      # warm-up
        gemm(*mats[i % copies])
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.profile_reps):
        gemm(*mats[i % copies])
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / args.profile_reps
    print(json.dumps({"profile_shape": f"{K}x{N}", "entry": args.profile_entry, "M": M, "group": g, "copies": copies,
                      "launches": 2 * args.profile_reps, "us_per_launch_direct": us,
                      "bytes_per_launch": gemm_bytes(M, N, K, g),
                      "gbs": gemm_bytes(M, N, K, g) / us / 1e3}))


def time_steps_local(torch, runners, steps, warmup):
    for i in range(warmup):
        runners[i % len(runners)]()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        runners[i % len(runners)]()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps, None, None


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-graph", action="store_true", help="time direct launches instead of CUDA graphs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-prefill", action="store_true", help="skip the tensor-core prefill probe")
    ap.add_argument("--only-prefill", action="store_true", help="run only the prefill probe")
    ap.add_argument("--only-headline", action="store_true",
                    help="time the steps only (no per-M breakdown, kernel probe, e2e or CPU baseline); "
                         "short command for profilers")
    ap.add_argument("--profile-shape", default=None, help="KxN: run only a few launches of this GEMM")
    ap.add_argument("--profile-m", type=int, default=1)
    ap.add_argument("--profile-group", type=int, default=64)
    ap.add_argument("--profile-reps", type=int, default=10)
    ap.add_argument("--profile-entry", default="a8", choices=["a8", "h16", "a16"],
                    help="entry point the profile run launches: w2a8_gemm, w2a8_gemm_h16 or w2a16_gemm")
    args = ap.parse_args()
    if args.profile_shape:
        run_kernel_profile(args)
        return
    if args.only_prefill:
        import torch
        from paper_2508_06753_b200 import build
        build.build()
        print(json.dumps(prefill_probe(torch.device("cuda", 0), load_peaks())))
        return
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
