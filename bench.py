#!/usr/bin/env python
"""Benchmark of the W2A8 hot path on B200 (one process per GPU).

Workload (N = 1 and every rank of N > 1: independent replicas, no exchange):
one Llama-3-8B-shaped decoder layer -- q/o 4096x4096, k/v 4096x1024, gate/up
4096x14336, down 14336x4096 (K x N), group 64 -- run as four w2a8_linear_grouped
calls (q|k|v, o, gate|up, down: bf16 activations in, fp32 outputs out), for
M = 1, 4 and 16 tokens.  One "step" is those three passes; the same step as
four a8_quantize and seven w2a8_gemm calls is reported beside it.  Weights are packed ahead of time; successive passes rotate over
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
# the same for one grouped launch of the persistent kernel on gate|up, 4096x(14336+14336), M=1:
# 36,818,948 algorithmic bytes, 36,734,720 read from DRAM (the activations come from L2), 256 written
NCU_TRAFFIC_BYTES_GATEUP_M1 = 36_734_976


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
INPUT_OF = {"q": "attn_in", "k": "attn_in", "v": "attn_in", "o": "o_in", "gate": "mlp_in", "up": "mlp_in",
            "down": "down_in", "gemv": "attn_in", "gate_up": "mlp_in"}


def layer_groups(cfg):
    """The linears of a layer grouped by the activation they read, in execution order:
    [(input name, [shape indices])] -- q|k|v, o, gate|up, down for a decoder layer."""
    groups = []
    for idx, (name, K, N) in enumerate(cfg["shapes"]):
        inp = INPUT_OF[name]
        if groups and groups[-1][0] == inp:
            groups[-1][1].append(idx)
        else:
            groups.append((inp, [idx]))
    return groups


class Layer:
    """`copies` resident copies of one layer's packed weights plus the activation, output and
    workspace buffers for each M (device memory only).  Copies beyond the first are device-side
    clones: distinct addresses are what defeats L2, the values do not matter for timing."""

    def __init__(self, cfg, copies, device, Ms=None):
        import torch
        from paper_2508_06753_b200 import binding as b
        self.torch, self.b, self.cfg, self.device = torch, b, cfg, device
        self.shapes = cfg["shapes"]
        self.Ms = list(Ms if Ms is not None else cfg["Ms"])
        self.groups = layer_groups(cfg)
        first = []
        made = {}
        for idx, (name, K, N) in enumerate(self.shapes):
            g = synth.config_group(cfg, K)
            if (K, N) in made:                      # twin shape (v of k, up of gate, o of q): a clone will do
                packed, s_w = made[(K, N)]
                first.append((packed.clone(), s_w.clone(), g))
                continue
            codes, s_w = synth.make_linear(synth.shape_seed(cfg, idx), K, N, g, cfg["ternary"])
            packed = b.w2_pack(torch.from_numpy(codes).to(device))
            del codes
            made[(K, N)] = (packed, torch.from_numpy(s_w).to(device))
            first.append((packed, made[(K, N)][1], g))
        self.copies = [first] + [[(p.clone(), s.clone(), g) for p, s, g in first] for _ in range(copies - 1)]
        torch.cuda.synchronize()
        self.weight_bytes_per_copy = sum(p.numel() * 4 + s.numel() * 4 for p, s, _ in first)
        self.per_m = {}
        ws_bytes = 256
        for M in self.Ms:
            bufs = {"x": {}, "a": {}, "s": {}, "y": []}
            for idx, (name, K, N) in enumerate(self.shapes):
                inp = INPUT_OF[name]
                if inp not in bufs["x"]:
                    bits = synth.activations_bf16(cfg["seed"] + 50 + len(bufs["x"]), M, K, cfg["outlier_frac"])
                    bufs["x"][inp] = torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)
                    bufs["a"][inp] = torch.empty((M, K), dtype=torch.int8, device=device)
                    bufs["s"][inp] = torch.empty((M,), dtype=torch.float32, device=device)
                bufs["y"].append(torch.empty((M, N), dtype=torch.float32, device=device))
                ws_bytes = max(ws_bytes, b.w2a8_workspace_bytes(M, N, K, synth.config_group(cfg, K)))
            self.per_m[M] = bufs
        self.ws = b.new_workspace(ws_bytes, device=device)
        # argument blocks of the grouped entry points: one per (copy, group, M), outputs bound
        self.gargs = {}
        for c, mats in enumerate(self.copies):
            for gi, (inp, idxs) in enumerate(self.groups):
                for M in self.Ms:
                    self.gargs[(c, gi, M)] = b.Group([mats[i][0] for i in idxs], [mats[i][1] for i in idxs],
                                                     [self.per_m[M]["y"][i] for i in idxs])

    # --- the two ways to run one pass of the layer ---------------------------------------
    def pass_grouped(self, M, copy, fuse=-1):
        """One w2a8_linear_grouped call per distinct input: q|k|v, o, gate|up, down."""
        b, bufs = self.b, self.per_m[M]
        for gi, (inp, idxs) in enumerate(self.groups):
            K = self.shapes[idxs[0]][1]
            b.w2a8_linear_grouped(bufs["x"][inp], self.gargs[(copy, gi, M)], synth.config_group(self.cfg, K),
                                  self.ws, fuse=fuse, a=bufs["a"][inp], a_scale=bufs["s"][inp])

    def pass_separate(self, M, copy):
        """One a8_quantize per distinct input and one w2a8_gemm per matrix."""
        b, bufs = self.b, self.per_m[M]
        for inp, idxs in self.groups:
            b.a8_quantize(bufs["x"][inp], bufs["a"][inp], bufs["s"][inp])
            for i in idxs:
                packed, s_w, g = self.copies[copy][i]
                b.w2a8_gemm(bufs["a"][inp], bufs["s"][inp], packed, s_w, g, self.ws, bufs["y"][i])

    def launches_grouped(self, M, fuse=-1):
        """Kernel launches of pass_grouped, from what the library says it will do."""
        n = 0
        for inp, idxs in self.groups:
            K = self.shapes[idxs[0]][1]
            Ns = [self.shapes[i][2] for i in idxs]
            plan = self.b.w2a8_grouped_plan(Ns, M, K, synth.config_group(self.cfg, K), fuse)
            n += 1 if plan["fused"] else (2 if plan["one_launch"] else 1 + len(idxs))
        return n

    def launches_separate(self):
        return len(self.shapes) + len(self.groups)

    def run_step(self, step_index, mode="grouped"):
        n = len(self.copies)
        for j, M in enumerate(self.Ms):
            copy = (step_index * len(self.Ms) + j) % n
            if mode == "grouped":
                self.pass_grouped(M, copy)
            else:
                self.pass_separate(M, copy)


def copies_for(l2_bytes, bytes_per_copy, factor=2.0):
    return max(2, int(np.ceil(factor * l2_bytes / bytes_per_copy)))


def capture(torch, body, stream, use_graph=True):
    """Run `body` once on `stream` (warm), then capture it into a CUDA graph; returns the callable
    to time (the graph's replay, or `body` itself when capture is off or fails) and its kind."""
    with torch.cuda.stream(stream):
        body()
        torch.cuda.synchronize()
        if not use_graph:
            return body, "direct"
        try:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                body()
            return g.replay, "cuda_graph"
        except Exception as e:  # capture not possible: time direct launches instead
            sys.stderr.write(f"[bench] graph capture failed ({e}); timing direct launches\n")
            torch.cuda.synchronize()
            return body, "direct"


def timed_blocks(torch, run, stream, blocks=10, reps=5, warm=3):
    """CUDA-event time of `run` on `stream`: `blocks` measurements of `reps` back-to-back calls
    each, after `warm` untimed calls.  Returns milliseconds per call: mean, min and median over
    the blocks (the paper averages 10-20 iterations and reports < 3 % variation, Sec. III-A)."""
    with torch.cuda.stream(stream):
        for _ in range(warm):
            run()
        torch.cuda.synchronize()
        ts = []
        for _ in range(blocks):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                run()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) / reps)
    return {"mean": float(np.mean(ts)), "min": float(np.min(ts)), "median": float(np.median(ts)),
            "blocks": blocks, "reps_per_block": reps}


def side_stream(torch):
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    return s


def build_step_graphs(rep, use_graph, mode="grouped"):
    """One CUDA graph per rotation phase (direct launches when capture is off or fails)."""
    torch = rep.torch
    stream = side_stream(torch)
    runners, kinds = [], set()
    for i in range(len(rep.copies)):
        run, kind = capture(torch, lambda i=i: rep.run_step(i, mode), stream, use_graph)
        runners.append(run)
        kinds.add(kind)
    torch.cuda.current_stream().wait_stream(stream)
    torch.cuda.synchronize()
    return runners, ("cuda_graph" if kinds == {"cuda_graph"} else "direct"), stream


def time_steps(torch, runners, stream, steps, warmup):
    """The contract's timing: W warm-up steps, then exactly K steps between two events, bracketed
    by a barrier and a synchronize on both sides."""
    with torch.cuda.stream(stream):
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


def per_m_times(rep, mode, use_graph, blocks=10):
    """Layer pass per M on its own (graph over all weight copies), mean / min / median."""
    torch, cfg = rep.torch, rep.cfg
    stream = side_stream(torch)
    out = {}
    for M in rep.Ms:
        def body(M=M):
            for c in range(len(rep.copies)):
                if mode == "grouped":
                    rep.pass_grouped(M, c)
                else:
                    rep.pass_separate(M, c)
        run, _ = capture(torch, body, stream, use_graph)
        t = timed_blocks(torch, run, stream, blocks=blocks, reps=max(1, 40 // len(rep.copies)))
        n = len(rep.copies)
        nbytes = layer_bytes(cfg, M)
        out[str(M)] = {"us_per_layer": t["mean"] / n * 1e3, "us_min": t["min"] / n * 1e3,
                       "us_median": t["median"] / n * 1e3, "gbs": nbytes / (t["mean"] / n * 1e-3) / 1e9,
                       "bytes_per_layer": nbytes,
                       "launches_per_layer": rep.launches_grouped(M) if mode == "grouped" else rep.launches_separate()}
    torch.cuda.current_stream().wait_stream(stream)
    return out


def kernel_probe(device, peaks, l2_bytes, M, K, N, g, use_graph=True, seed=9000, count=1):
    """One GEMM launch on its own -- w2a8_gemm, or w2a8_gemm_grouped over `count` matrices of the
    same shape -- back to back in a graph over its own set of weight copies, at least twice L2 of
    distinct weight bytes, CUDA events on the launching stream."""
    import torch
    from paper_2508_06753_b200 import binding as b
    codes, s_w = synth.make_linear(seed + K + N, K, N, g)
    packed = b.w2_pack(torch.from_numpy(codes).to(device))
    sw = torch.from_numpy(s_w).to(device)
    per = (packed.numel() * 4 + sw.numel() * 4) * count
    ncopy = copies_for(l2_bytes, per, 2.2)
    mats = [[(packed.clone(), sw.clone()) for _ in range(count)] for _ in range(ncopy)]
    x = torch.from_numpy(synth.activations_bf16(seed + M, M, K).view(np.int16)).to(device).view(torch.bfloat16)
    a, s_a = b.a8_quantize(x)
    ys = [torch.empty((M, N), dtype=torch.float32, device=device) for _ in range(count)]
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g), device=device)
    groups = [b.Group([m[0] for m in grp], [m[1] for m in grp], ys) for grp in mats]

    def body():
        for grp, gargs in zip(mats, groups):
            if count == 1:
                b.w2a8_gemm(a, s_a, grp[0][0], grp[0][1], g, ws, ys[0])
            else:
                b.w2a8_gemm_grouped(a, s_a, gargs, g, ws)
    stream = side_stream(torch)
    run, kind = capture(torch, body, stream, use_graph)
    t = timed_blocks(torch, run, stream, blocks=12, reps=max(1, 48 // ncopy))
    torch.cuda.current_stream().wait_stream(stream)
    nbytes = count * gemm_bytes(M, N, K, g) - (count - 1) * (M * K + 4 * M)     # the activations are read once
    us = t["mean"] / ncopy * 1e3
    plan = b.w2a8_grouped_plan([N] * count, M, K, g, b.FUSE_OFF)
    return dict(shape=f"{K}x{N}" + (f" x{count}" if count > 1 else ""), M=M, group=g, us_per_launch=us,
                kernel="persistent" if plan["one_launch"] else "one-shot", us_min=t["min"] / ncopy * 1e3,
                us_median=t["median"] / ncopy * 1e3, bytes_per_launch=nbytes, gbs=nbytes / us / 1e3,
                frac_of_measured_hbm=nbytes / us / 1e3 / peaks["hbm_gbs"],
                distinct_weight_bytes=per * ncopy, weight_copies=ncopy, launch=kind,
                launches=t["blocks"] * t["reps_per_block"] * ncopy)


def read_ceiling_probe(device, l2_bytes):
    """Read-only ceiling measured in this job: the library's plain 128-bit load kernel over a
    buffer of four times L2, back to back."""
    import torch
    from paper_2508_06753_b200 import binding as b
    nbytes = int(4 * l2_bytes) // 4096 * 4096
    buf = torch.empty(nbytes, dtype=torch.uint8, device=device)
    buf.random_(0, 255)
    sink = torch.zeros(1, dtype=torch.int32, device=device)
    stream = side_stream(torch)
    t = timed_blocks(torch, lambda: b.w2a8_read_probe(buf, sink), stream, blocks=10, reps=5)
    torch.cuda.current_stream().wait_stream(stream)
    return {"what": "w2a8_read_probe: plain 128-bit loads of a buffer of 4 x L2, nothing else",
            "bytes": nbytes, "gbs": nbytes / (t["min"] * 1e-3) / 1e9, "gbs_mean": nbytes / (t["mean"] * 1e-3) / 1e9}


def fused_vs_separate(rep, use_graph=True):
    """The knob of Sec. II-D, measured: every w2a8_linear_grouped call of the layer with the
    quantiser inside the launch (FUSE_ON), as a launch of its own (FUSE_OFF), and as the
    library's rule picks (FUSE_AUTO); microseconds per call."""
    torch, b, cfg = rep.torch, rep.b, rep.cfg
    stream = side_stream(torch)
    rows = []
    for M in [m for m in rep.Ms if m <= 8]:
        bufs = rep.per_m[M]
        for gi, (inp, idxs) in enumerate(rep.groups):
            K = rep.shapes[idxs[0]][1]
            g = synth.config_group(cfg, K)
            Ns = [rep.shapes[i][2] for i in idxs]
            row = {"linears": "|".join(rep.shapes[i][0] for i in idxs), "M": M, "K": K, "N": Ns}
            for label, fuse in (("fused", b.FUSE_ON), ("separate", b.FUSE_OFF), ("auto", b.FUSE_AUTO)):
                def body(fuse=fuse):
                    for c in range(len(rep.copies)):
                        b.w2a8_linear_grouped(bufs["x"][inp], rep.gargs[(c, gi, M)], g, rep.ws, fuse=fuse,
                                              a=bufs["a"][inp], a_scale=bufs["s"][inp])
                run, _ = capture(torch, body, stream, use_graph)
                t = timed_blocks(torch, run, stream, blocks=6, reps=max(1, 24 // len(rep.copies)))
                row[f"us_{label}"] = t["mean"] / len(rep.copies) * 1e3
                row[f"plan_{label}"] = b.w2a8_grouped_plan(Ns, M, K, g, fuse)
            rows.append(row)
    torch.cuda.current_stream().wait_stream(stream)
    return {"what": "w2a8_linear_grouped per call: quantiser inside the persistent launch (fused), as its own "
                    "launch (separate), and the library's choice (auto)", "rows": rows}


def sweep_plan(device, peaks, l2_bytes, use_graph=True, config_index=1, Ms=(1, 4, 8, 16)):
    """What a per-shape tuner would look at (the paper picks kernel variants per shape with an
    auto-tuner, Sec. II-D): every linear group of the Llama-3-8B layer at M = 1, 4, 8, 16 through
    each way the library can run it -- one-shot kernel with one launch per matrix, persistent
    kernel with one launch per group, persistent kernel with the quantiser inside -- next to what
    the built-in rule picks.  Microseconds per group call, quantiser included."""
    import torch
    from paper_2508_06753_b200 import binding as b
    cfg = dict(synth.CONFIGS[config_index], Ms=Ms)
    per_copy = sum(K * N // 4 + (K // synth.config_group(cfg, K)) * N * 4 for _, K, N in cfg["shapes"])
    rep = Layer(cfg, copies_for(l2_bytes, per_copy), device)
    stream = side_stream(torch)
    rows = []
    saved = os.environ.get("W2A8_GEMV")
    for M in rep.Ms:
        bufs = rep.per_m[M]
        for gi, (inp, idxs) in enumerate(rep.groups):
            K = rep.shapes[idxs[0]][1]
            g = synth.config_group(cfg, K)
            Ns = [rep.shapes[i][2] for i in idxs]
            row = {"linears": "|".join(rep.shapes[i][0] for i in idxs), "M": M, "K": K, "N": Ns}
            variants = [("one_shot_per_matrix", "0", b.FUSE_OFF), ("persistent_grouped", "2", b.FUSE_OFF),
                        ("persistent_fused", "2", b.FUSE_ON), ("built_in_rule", None, b.FUSE_AUTO)]
            for label, env, fuse in variants:
                if env is None:
                    os.environ.pop("W2A8_GEMV", None)
                else:
                    os.environ["W2A8_GEMV"] = env
                if label == "persistent_fused" and not b.w2a8_grouped_plan(Ns, M, K, g, fuse)["fused"]:
                    row[label] = None
                    continue

                def body(fuse=fuse):
                    for c in range(len(rep.copies)):
                        b.w2a8_linear_grouped(bufs["x"][inp], rep.gargs[(c, gi, M)], g, rep.ws, fuse=fuse,
                                              a=bufs["a"][inp], a_scale=bufs["s"][inp])
                run, _ = capture(torch, body, stream, use_graph)
                t = timed_blocks(torch, run, stream, blocks=6, reps=max(1, 24 // len(rep.copies)))
                row[label] = round(t["mean"] / len(rep.copies) * 1e3, 3)
            best = min((v, k) for k, v in row.items() if k in ("one_shot_per_matrix", "persistent_grouped",
                                                               "persistent_fused") and v is not None)
            row["best"] = best[1]
            row["rule_vs_best"] = round(row["built_in_rule"] / best[0], 3)
            rows.append(row)
    if saved is None:
        os.environ.pop("W2A8_GEMV", None)
    else:
        os.environ["W2A8_GEMV"] = saved
    torch.cuda.current_stream().wait_stream(stream)
    return {"what": f"us per w2a8_linear_grouped call (quantiser included), configuration {config_index} "
                    f"({cfg['name']}), {len(rep.copies)} rotating weight copies", "rows": rows}


def config_row(index, device, peaks, l2_bytes, use_graph=True, cpu_budget_s=4.0):
    """One of the other benchmark configurations (0: single 2048^2 GEMV, 2: ternary layer with one
    scale per channel, 3: Llama-3-70B layer with group 128 and outliers): the layer pass per M
    through the grouped entry, GB/s on its algorithmic bytes, and the reference on the host cores."""
    import torch
    cfg = synth.CONFIGS[index]
    per_copy = sum(K * N // 4 + (K // synth.config_group(cfg, K)) * N * 4 for _, K, N in cfg["shapes"])
    rep = Layer(cfg, copies_for(l2_bytes, per_copy, 2.1), device)
    grouped = per_m_times(rep, "grouped", use_graph, blocks=8)
    for M, r in grouped.items():
        r["frac_of_measured_hbm"] = r["gbs"] / peaks["hbm_gbs"]
    row = {"config": index, "name": cfg["name"], "Ms": cfg["Ms"], "group": cfg["group"] or "K",
           "weight_copies": len(rep.copies), "distinct_weight_bytes": rep.weight_bytes_per_copy * len(rep.copies),
           "per_m": grouped}
    if index == 0:
        # launch-latency model the paper uses for its smallest shape (Sec. III-B): the time cannot
        # be below the dependent-launch latency, whatever the bandwidth
        r = grouped["1"]
        t_bw = r["bytes_per_layer"] / (peaks["hbm_gbs"] * 1e9) * 1e6
        row["latency_model"] = {"t_bandwidth_us": t_bw, "t_measured_us": r["us_per_layer"],
                                "t_launch_floor_us": r["us_per_layer"] - t_bw,
                                "model": "t = max(bytes / BW, t_launch): the measured time is the launch floor"}
    del rep
    torch.cuda.empty_cache()
    if cpu_budget_s > 0:
        row["cpu_baseline"] = cpu_baseline(cfg, budget_s=cpu_budget_s, min_wall_s=0.5, max_channels=256)
    return row


def small_shape_probe(device, peaks, l2_bytes, use_graph=True):
    """Extra rows (not the headline): the small square-ish matrices the paper also times (Sec. III:
    1600x1600, 2560x2560, 3840x2560, 3200x3200), where launch latency dominates.  One GEMV (M = 1,
    group 64) per launch."""
    rows = []
    for K, N in ((1600, 1600), (2560, 2560), (2560, 3840), (3200, 3200)):
        r = kernel_probe(device, peaks, l2_bytes, 1, K, N, 64, use_graph, seed=K)
        rows.append({k: r[k] for k in ("shape", "M", "group", "us_per_launch", "us_min", "bytes_per_launch", "gbs",
                                       "frac_of_measured_hbm", "weight_copies")})
    return rows


def recipe16_probe(rep, peaks, group=128, use_graph=True):
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
    stream = side_stream(torch)
    for M in rep.Ms:
        bufs = rep.per_m[M]
        ys = [torch.empty((M, N), dtype=torch.bfloat16, device=dev) for _, _, N in rep.shapes]
        ws = b.new_workspace(max(b.w2a8_workspace_bytes(M, N, K, group) for _, K, N in rep.shapes), device=dev)

        def body():
            for c in range(len(copies)):
                for inp, idxs in rep.groups:
                    b.a8_quantize(bufs["x"][inp], bufs["a"][inp], bufs["s"][inp])
                    for i in idxs:
                        packed, s_h = copies[c][i]
                        b.w2a8_gemm_h16(bufs["a"][inp], bufs["s"][inp], packed, s_h, group, ws, ys[i])
        run, _ = capture(torch, body, stream, use_graph)
        t = timed_blocks(torch, run, stream, blocks=6, reps=max(1, 24 // len(copies)))
        ms = t["mean"] / len(copies)
        nbytes = sum(bytes_of(M, N, K) for _, K, N in rep.shapes)
        out[str(M)] = {"us_per_layer": ms * 1e3, "bytes_per_layer": nbytes, "gbs": nbytes / (ms * 1e-3) / 1e9,
                       "frac_of_measured_hbm": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    torch.cuda.current_stream().wait_stream(stream)
    return {"what": f"group {group}, binary16 weight scales, bf16 results (w2a8_gemm_h16): 7 GEMMs + 4 "
                    "a8_quantize per layer pass; GB/s on this recipe's own byte count", "per_m": out}


def a16_probe(rep, peaks, use_graph=True):
    """Extra row (not the headline): the same layer through w2a16_gemm -- bf16 activations against
    the 2-bit weights, no activation quantiser: 7 launches per pass.  GB/s on this entry's own
    byte count (bf16 activations: 2 bytes each, no token scales)."""
    torch, b, cfg = rep.torch, rep.b, rep.cfg

    def bytes_of(M, N, K, g):
        return K * N // 4 + (K // g) * N * 4 + 2 * M * K + 4 * M * N

    out = {}
    stream = side_stream(torch)
    for M in rep.Ms:
        bufs = rep.per_m[M]

        def body():
            for c in range(len(rep.copies)):
                for idx, (name, K, N) in enumerate(rep.shapes):
                    packed, s_w, g = rep.copies[c][idx]
                    b.w2a16_gemm(bufs["x"][INPUT_OF[name]], packed, s_w, g, rep.ws, bufs["y"][idx])
        run, _ = capture(torch, body, stream, use_graph)
        t = timed_blocks(torch, run, stream, blocks=6, reps=max(1, 24 // len(rep.copies)))
        ms = t["mean"] / len(rep.copies)
        nbytes = sum(bytes_of(M, N, K, synth.config_group(cfg, K)) for _, K, N in rep.shapes)
        out[str(M)] = {"us_per_layer": ms * 1e3, "bytes_per_layer": nbytes, "gbs": nbytes / (ms * 1e-3) / 1e9,
                       "frac_of_measured_hbm": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    torch.cuda.current_stream().wait_stream(stream)
    return {"what": "w2a16_gemm (bf16 activations, no a8_quantize): 7 launches per layer pass; GB/s on this "
                    "entry's own byte count", "per_m": out}


def e2e_measure(rep, steps, warmup, use_graph=True):
    """Same workload end to end through the public API with HOST buffers: every step the bf16
    activations of that step are read from pinned host memory and the fp32 results land in pinned
    host memory (w2a8_linear_grouped_host, one call per distinct input: q|k|v, o, gate|up, down; with
    few tokens its kernels address the page-locked buffers directly, so the transfers are inside the
    kernels and inside the timed region).  Timed twice: the calls of a step captured once into a CUDA graph and replayed per step
    (what a decode loop does: fixed pinned buffers, new contents every step, one replay), and the
    same calls issued directly every step.  Returns (graph ms or None, direct ms, h2d, d2h, checksum)."""
    torch, b, cfg = rep.torch, rep.b, rep.cfg
    dev = rep.ws.device
    host = {}
    h2d = d2h = 0
    ws_bytes = 256
    for M in rep.Ms:
        xs, ys = [], []
        for gi, (inp, idxs) in enumerate(rep.groups):
            K = rep.shapes[idxs[0]][1]
            Ns = [rep.shapes[i][2] for i in idxs]
            xs.append(rep.per_m[M]["x"][inp].cpu().pin_memory())
            ys.append([torch.empty((M, n), dtype=torch.float32).pin_memory() for n in Ns])
            h2d += M * K * 2
            d2h += sum(M * n * 4 for n in Ns)
            ws_bytes = max(ws_bytes, b.w2a8_linear_grouped_host_workspace_bytes(Ns, M, K, synth.config_group(cfg, K)))
        host[M] = (xs, ys)
    ws = b.new_workspace(ws_bytes, device=dev)

    def step(i):
        n = len(rep.copies)
        for j, M in enumerate(rep.Ms):
            copy = (i * len(rep.Ms) + j) % n
            xs, ys = host[M]
            for gi, (inp, idxs) in enumerate(rep.groups):
                g = synth.config_group(cfg, rep.shapes[idxs[0]][1])
                b.w2a8_linear_grouped_host(xs[gi], rep.gargs[(copy, gi, M)], g, ys[gi], ws)

    def timed(run_step):
        for i in range(max(warmup, 3)):
            run_step(i)
        torch.cuda.synchronize()
        dist_barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            run_step(i)
            host[rep.Ms[0]][0][0][0, 0] += 0            # the host touches this step's input buffer (new contents)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    ms_direct = timed(step)
    ms_graph = None
    if use_graph:
        stream = side_stream(torch)
        replays = []
        for i in range(len(rep.copies)):
            run, kind = capture(torch, lambda i=i: step(i), stream, True)
            if kind != "cuda_graph":
                replays = None
                break
            replays.append(run)
        if replays:
            with torch.cuda.stream(stream):
                ms_graph = timed(lambda i: replays[i % len(replays)]())
        torch.cuda.current_stream().wait_stream(stream)
    checksum = float(sum(float(y.sum()) for ys in host[rep.Ms[0]][1] for y in ys))
    return ms_graph, ms_direct, h2d, d2h, checksum


class OracleWorkload:
    """The scalar reference on a benchmark configuration; a step may cover only the first n
    output channels of every linear (channels are independent), so a step can be sized to a time
    budget.  `max_channels` bounds what is generated per linear (the sample never needs more)."""

    def __init__(self, cfg, max_channels=None):
        import oracle
        oracle.build()
        self.oracle, self.cfg = oracle, cfg
        self.mats = []
        for idx, (name, K, N) in enumerate(cfg["shapes"]):
            g = synth.config_group(cfg, K)
            n_gen = N if max_channels is None else min(N, max_channels)
            codes, s_w = synth.make_linear(synth.shape_seed(cfg, idx), K, n_gen, g, cfg["ternary"])
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
                n = min(codes.shape[0], max(16, int(N * frac) // 16 * 16))
                a, s_a = q[K]
                self.oracle.gemm(a, s_a, codes[:n], s_w[:n], g)
                nbytes += gemm_bytes(M, n, K, g)
        return nbytes, time.perf_counter() - t0

    def max_frac(self):
        return min(1.0, min(m[0].shape[0] / m[4] for m in self.mats))

    def frac_for(self, seconds_per_step):
        probe = min(1.0 / 64, self.max_frac())
        _, dt = self.step(probe)
        _, dt = self.step(probe)
        return float(min(self.max_frac(), max(1.0 / 896, probe * seconds_per_step / max(dt, 1e-6))))


def cpu_baseline(cfg, budget_s=20.0, min_wall_s=1.5, max_channels=None):
    """The reference as it stands on this machine's host cores, on a bounded sample of a
    benchmark configuration: whole steps (restricted to a leading fraction of the output channels
    if one step alone would exceed `budget_s`), repeated until about `min_wall_s` seconds of wall
    time have been measured."""
    w = OracleWorkload(cfg, max_channels)
    frac = w.frac_for(budget_s)
    tot_b, tot_s, n = 0, 0.0, 0
    while tot_s < min_wall_s and n < 64:
        nbytes, dt = w.step(frac)
        tot_b += nbytes
        tot_s += dt
        n += 1
    cores = w.oracle.num_threads()
    nq, ng = len(layer_groups(cfg)), len(cfg["shapes"])
    return dict(value=tot_b / tot_s / 1e9, unit="GB/s", cores=cores, kind="oracle",
                seconds=tot_s, cpu_core_seconds=tot_s * cores,
                sample=f"{n} step(s) (M in {cfg['Ms']}, {nq} quantise + {ng} GEMM calls each) restricted to "
                       f"the first {frac:.4f} of the output channels of every linear")


WORKLOAD = ("llama3-8b decoder-layer linears (q,k,v,o,gate,up,down), group 64, M in {1,4,16}: "
            "configuration 1")


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
        "config": {"workload": WORKLOAD},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": w.oracle.num_threads(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out))


def note(msg):
    sys.stderr.write(f"[bench +{time.perf_counter() - _T0:6.1f}s] {msg}\n")
    sys.stderr.flush()


_T0 = time.perf_counter()


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
    use_graph = not args.no_graph

    l2 = torch.cuda.get_device_properties(local).L2_cache_size
    per_copy = sum(K * N // 4 + (K // synth.config_group(cfg, K)) * N * 4 for _, K, N in cfg["shapes"])
    copies = copies_for(l2, per_copy)
    rep = Layer(cfg, copies, device)
    note(f"layer resident: {copies} copies")

    # ---- headline: K steps of the layer through the grouped operator ---------------------
    sampler = ClockSampler(local)
    sampler.start()
    runners, mode, stream = build_step_graphs(rep, use_graph, "grouped")
    ms, t0, t1 = time_steps(torch, runners, stream, args.steps, args.warmup)
    sampler.stop()
    clocks = sampler.summary(t0, t1)
    units = step_bytes(cfg) * args.steps
    ms_all, units_all = aggregate(ms, units, device)
    value = units_all / (ms_all * 1e-3) / 1e9
    launches_per_step = sum(rep.launches_grouped(M) for M in rep.Ms)
    note(f"headline: {value:.1f} GB/s, {ms_all / args.steps * 1e3:.1f} us per step")

    if args.only_headline:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world,
                              "steps": args.steps, "warmup": args.warmup,
                              "ms_per_step": ms_all / args.steps, "launch": mode, "clocks": clocks,
                              "gpu_launches": args.steps * launches_per_step}))
        return

    extra = {}
    if rank == 0:
        # the same step as one a8_quantize per input and one w2a8_gemm per matrix (11 launches per pass)
        r2, _, s2 = build_step_graphs(rep, use_graph, "separate")
        ms2, _, _ = time_steps_local(torch, r2, s2, max(args.steps // 4, 20), 5)
        extra["separate_calls"] = {
            "what": "the same step as 4 a8_quantize + 7 w2a8_gemm calls per layer pass",
            "ms_per_step": ms2, "gbs": step_bytes(cfg) / (ms2 * 1e-3) / 1e9,
            "launches_per_step": rep.launches_separate() * len(rep.Ms)}
        extra["per_m"] = per_m_times(rep, "grouped", use_graph)
        extra["per_m_separate_calls"] = per_m_times(rep, "separate", use_graph, blocks=6)
        note("per-M rows done")
        name, K, N = max(cfg["shapes"], key=lambda s: s[1] * s[2])
        K, N = 4096, 14336
        # the launches with the largest share of the step: gate|up as one grouped launch (M = 1, 4),
        # gate alone (M = 16, and M = 1 for the one-shot kernel on its own), down
        probes = [kernel_probe(device, peaks, l2, 1, K, N, 64, use_graph, count=2),
                  kernel_probe(device, peaks, l2, 4, K, N, 64, use_graph, count=2),
                  kernel_probe(device, peaks, l2, 16, K, N, 64, use_graph),
                  kernel_probe(device, peaks, l2, 1, K, N, 64, use_graph),
                  kernel_probe(device, peaks, l2, 1, 14336, 4096, 64, use_graph)]
        extra["read_ceiling"] = read_ceiling_probe(device, l2)
        note("kernel probes done")
        extra["fused_vs_separate"] = fused_vs_separate(rep, use_graph)
        extra["recipe_g128_binary16_scales_bf16_out"] = recipe16_probe(rep, peaks, use_graph=use_graph)
        extra["w2a16_no_quantiser"] = a16_probe(rep, peaks, use_graph)
        extra["paper_small_shapes_m1"] = small_shape_probe(device, peaks, l2, use_graph)
        note("extra rows done")
    e2e_steps = max(args.steps // 10, 10)
    e2e_graph_ms, e2e_direct_ms, h2d, d2h, _ = e2e_measure(rep, e2e_steps, 3, use_graph)
    e2e_ms = e2e_graph_ms if e2e_graph_ms is not None else e2e_direct_ms
    e2e_ms_all, e2e_units = aggregate(e2e_ms, step_bytes(cfg) * e2e_steps, device)
    e2e = {"value": e2e_units / (e2e_ms_all * 1e-3) / 1e9, "unit": "GB/s",
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
           "ms_per_step": e2e_ms_all / e2e_steps,
           "api": "w2a8_linear_grouped_host, one call per distinct input (q|k|v, o, gate|up, down), pinned host "
                  "buffers read and written by the kernels; "
                  + ("the calls of a step captured into a CUDA graph, one replay per step"
                     if e2e_graph_ms is not None else "direct calls"),
           "direct_calls": {"value": step_bytes(cfg) * e2e_steps / (e2e_direct_ms * 1e-3) / 1e9, "unit": "GB/s",
                            "ms_per_step": e2e_direct_ms / e2e_steps}}
    if rank != 0:
        return
    del rep
    torch.cuda.empty_cache()
    cpu = None
    other = []
    if not args.no_other_configs:
        for index in (0, 2, 3):
            other.append(config_row(index, device, peaks, l2, use_graph,
                                    cpu_budget_s=0.0 if args.no_cpu_baseline or world > 1 else 4.0))
            note(f"configuration {index} done")
    prefill = None
    if not args.no_prefill:
        prefill = prefill_probe(device, peaks)
        note("prefill done")
    if world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(cfg, budget_s=20.0)
        note("cpu baseline done")

    dom = probes[0]
    ceiling = extra["read_ceiling"]["gbs"]
    roofline = {"bound": "hbm", "achieved": dom["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": dom["gbs"] / peaks["hbm_gbs"], "traffic": NCU_TRAFFIC_BYTES_GATEUP_M1,
                "peak_source": peaks["source"],
                "kernel": "w2a8_gemv_kernel<MT=1,SPP=1,ONE,BCACHE,W=8> (persistent, two 8-warp CTAs per SM) on gate|up 4096x(14336+14336) as one "
                          "grouped launch, M=1: the launch with the largest share of the step (the other large "
                          "launches, and the one-shot kernel on gate alone, are in roofline_by_m)",
                "bytes_per_launch": dom["bytes_per_launch"], "us_per_launch": dom["us_per_launch"],
                "us_min": dom["us_min"], "us_median": dom["us_median"],
                "distinct_weight_bytes": dom["distinct_weight_bytes"], "l2_bytes": l2,
                "frac_of_read_ceiling_same_job": dom["gbs"] / ceiling, "read_ceiling_gbs": ceiling,
                "frac_of_nominal_8TBs": dom["gbs"] / NOMINAL_HBM_GBS}
    roofline_by_m = [{"M": pr["M"], "shape": pr["shape"], "kernel": pr["kernel"], "achieved": pr["gbs"], "unit": "GB/s",
                      "frac": pr["gbs"] / peaks["hbm_gbs"], "frac_of_read_ceiling_same_job": pr["gbs"] / ceiling,
                      "us_per_launch": pr["us_per_launch"], "us_min": pr["us_min"], "us_median": pr["us_median"],
                      "distinct_weight_bytes": pr["distinct_weight_bytes"]} for pr in probes]
    out = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_all / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8xint2->int32, fp32 scales",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "tokens_per_step": sum(cfg["Ms"]), "parallelism": f"replicas x{world}",
                   "api": "w2a8_linear_grouped: q|k|v, o, gate|up, down -- four calls per layer pass, the seven "
                          "weight matrices where they are in memory",
                   "launch": mode, "weight_copies": copies,
                   "l2_policy": f"inputs larger than L2: {copies} resident layer copies "
                                f"({copies * per_copy / 1e6:.0f} MB) rotated, L2 = {l2 / 1e6:.0f} MB"},
        "frac_of_measured_hbm": value / world / peaks["hbm_gbs"],
        "frac_of_nominal_8TBs": value / world / NOMINAL_HBM_GBS,
        "clocks": clocks, "e2e": e2e,
        "gpu_launches": args.steps * launches_per_step,
        "roofline": roofline, "roofline_by_m": roofline_by_m, "cpu_baseline": cpu,
        "kernel_probes": probes, "other_configs": other, "prefill": prefill,
    }
    out.update(extra)
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
                         "tile_tokens": b.w2a8_tensor_core_tile_tokens(M, N, K, g),
                         "frac_of_measured_int8_sustained": tops / int8_peak_sustained,
                         "status": b.w2a8_workspace_status(ws)})
        del packed, s_w_d, ws
    # The 16-bit tensor-core kernel (tcgen05 kind::f16, the alternative kernel of Sec. II) on the
    # same gate/up problem: behind w2a16_gemm (bf16 activations as they are) and behind w2a8_gemm
    # (W2A8_TC_KIND=16: bf16 copy of the int8 activations, copy kernel included in the time)
    alt = []
    name, K, N = cfg["shapes"][0]
    g = synth.config_group(cfg, K)
    codes, s_w = synth.make_linear(synth.shape_seed(cfg, 0), K, N, g)
    packed = b.w2_pack(torch.from_numpy(codes).to(device))
    s_w_d = torch.from_numpy(s_w).to(device)
    del codes
    saved_kind = os.environ.get("W2A8_TC_KIND")
    for M in Ms:
        bits = synth.activations_bf16(cfg["seed"] + 7 + M, M, K)
        x = torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)
        a, s_a = b.a8_quantize(x)
        y = torch.empty((M, N), dtype=torch.float32, device=device)
        row = {"shape": f"{K}x{N}", "M": M, "group": g}
        for label, kind in (("w2a16_gemm", None), ("w2a8_gemm_kind16", "16")):
            if kind is None:
                os.environ.pop("W2A8_TC_KIND", None)
            else:
                os.environ["W2A8_TC_KIND"] = kind
            ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g), device=device)
            fn = (lambda: b.w2a16_gemm(x, packed, s_w_d, g, ws, y)) if kind is None else \
                 (lambda: b.w2a8_gemm(a, s_a, packed, s_w_d, g, ws, y))
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                fn()
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / reps
            row[label] = {"ms": ms, "tops": 2.0 * M * N * K / (ms * 1e-3) / 1e12, "status": b.w2a8_workspace_status(ws)}
            del ws
        alt.append(row)
    if saved_kind is None:
        os.environ.pop("W2A8_TC_KIND", None)
    else:
        os.environ["W2A8_TC_KIND"] = saved_kind
    del packed, s_w_d
    # Few output tiles (64-256 tokens on the 8B layer's matrices): the tensor-core kernel with K split
    # over the otherwise idle SMs, next to the same kernel unsplit and to the streaming kernel
    few = []
    saved = {k: os.environ.get(k) for k in ("W2A8_PREFILL", "W2A8_PF_KSPLIT")}

    def set_env(**kv):
        for k, v in kv.items():
            if v is None:
                os.environ.pop(k, None)
            else:
                os.environ[k] = v
    for (K, N) in ((4096, 4096), (14336, 4096), (4096, 14336)):
        g = 64
        codes, s_w = synth.make_linear(synth.shape_seed(cfg, 0) + K + N, K, N, g)
        packed = b.w2_pack(torch.from_numpy(codes).to(device))
        s_w_d = torch.from_numpy(s_w).to(device)
        del codes
        for M in (64, 128, 256):
            bits = synth.activations_bf16(cfg["seed"] + 11 + M, M, K)
            x = torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)
            a, s_a = b.a8_quantize(x)
            y = torch.empty((M, N), dtype=torch.float32, device=device)
            row = {"shape": f"{K}x{N}", "M": M, "group": g}
            for label, env in (("default", dict(W2A8_PREFILL=None, W2A8_PF_KSPLIT=None)),
                               ("tensor_core_unsplit", dict(W2A8_PREFILL="2", W2A8_PF_KSPLIT="1")),
                               ("streaming", dict(W2A8_PREFILL="0", W2A8_PF_KSPLIT=None))):
                set_env(**env)
                ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g), device=device)
                stream = side_stream(torch)

                def body():
                    for _ in range(4):
                        b.w2a8_gemm(a, s_a, packed, s_w_d, g, ws, y)
                run, how = capture(torch, body, stream)          # env switches are read at capture time
                t = timed_blocks(torch, run, stream, blocks=5, reps=3)
                torch.cuda.current_stream().wait_stream(stream)
                row[label] = {"us": t["mean"] / 4 * 1e3, "us_min": t["min"] / 4 * 1e3, "timing": how,
                              "kernel": b.w2a8_kernel_for(M, N, K, g),
                              "k_splits": b.w2a8_tensor_core_ksplit(M, N, K, g), "status": b.w2a8_workspace_status(ws)}
                del ws, run
            few.append(row)
        del packed, s_w_d
    set_env(**saved)
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
            "library_int8_gemm": lib_int8, "rows": rows, "by_group_m2048": by_group,
            "few_tile_k_split": few,
            "kind_f16_kernel": {"what": "16-bit tensor-core kernel (tcgen05 kind::f16, fp32 accumulators, no conversion "
                                        "in the drain): op/s counted as for the int8 kernel", "rows": alt}}


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
    elif args.profile_entry == "grouped2":
        # two matrices of the shape as one grouped launch (gate|up): pairs of neighbouring copies
        y2 = torch.empty((M, N), dtype=torch.float32, device=dev)
        pairs = {id(mats[i][0]): b.Group([mats[i][0], mats[(i + 1) % copies][0]],
                                         [mats[i][1], mats[(i + 1) % copies][1]], [y, y2]) for i in range(copies)}

        def gemm(pk, sw):
            b.w2a8_gemm_grouped(a, s_a, pairs[id(pk)], g, ws)
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


def time_steps_local(torch, runners, stream, steps, warmup):
    with torch.cuda.stream(stream):
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
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the rows of configurations 0, 2 and 3 (single GEMV, ternary layer, 70B layer)")
    ap.add_argument("--sweep-plan", action="store_true",
                    help="print the per-shape table a tuner would look at (one-shot / persistent / fused, per "
                         "linear group and M) and exit")
    ap.add_argument("--only-headline", action="store_true",
                    help="time the steps only (no per-M breakdown, kernel probe, e2e or CPU baseline); "
                         "short command for profilers")
    ap.add_argument("--sweep-config", type=int, default=1, choices=[1, 2, 3], help="configuration --sweep-plan runs")
    ap.add_argument("--sweep-ms", default="1,4,8,16", help="token counts --sweep-plan runs")
    ap.add_argument("--profile-shape", default=None, help="KxN: run only a few launches of this GEMM")
    ap.add_argument("--profile-m", type=int, default=1)
    ap.add_argument("--profile-group", type=int, default=64)
    ap.add_argument("--profile-reps", type=int, default=10)
    ap.add_argument("--profile-entry", default="a8", choices=["a8", "h16", "a16", "grouped2"],
                    help="entry point the profile run launches: w2a8_gemm, w2a8_gemm_h16 or w2a16_gemm")
    args = ap.parse_args()
    if args.profile_shape:
        run_kernel_profile(args)
        return
    if args.sweep_plan:
        import torch
        from paper_2508_06753_b200 import build
        build.build()
        dev = torch.device("cuda", 0)
        print(json.dumps(sweep_plan(dev, load_peaks(), torch.cuda.get_device_properties(0).L2_cache_size,
                                    not args.no_graph, args.sweep_config,
                                    tuple(int(m) for m in args.sweep_ms.split(",")))))
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
