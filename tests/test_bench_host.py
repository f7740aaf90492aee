"""Host-side logic of the benchmark: byte accounting, the whole-job aggregation
over ranks (two gloo ranks on CPU) and the clock-sample summary."""
import json
import os
import subprocess
import sys

import pytest

from conftest import ROOT

sys.path.insert(0, ROOT)
import bench  # noqa: E402
from paper_2508_06753_b200 import synth  # noqa: E402


def test_algorithmic_bytes_match_the_shape_table():
    # 4096x4096, group 64: 4.19 MB of packed weights + 1.05 MB of scales
    assert bench.gemm_bytes(1, 4096, 4096, 64) == 4096 * 4096 // 4 + 64 * 4096 * 4 + 4096 + 4 + 4 * 4096
    cfg = synth.CONFIGS[1]
    # one Llama-3-8B layer at M = 1: 68.4 MB
    assert abs(bench.layer_bytes(cfg, 1) / 1e6 - 68.4) < 0.1
    assert abs(bench.layer_bytes(cfg, 16) / 1e6 - 71.5) < 0.1
    assert bench.step_bytes(cfg) == sum(bench.layer_bytes(cfg, m) for m in (1, 4, 16))
    # group == K (one scale per channel): 2 bits + 32 / K bits per weight
    assert bench.gemm_bytes(1, 16, 256, 256) == 16 * 256 // 4 + 16 * 4 + 256 + 4 + 64


def test_aggregate_single_process():
    assert bench.aggregate(3.0, 10.0) == (3.0, 10.0)


_WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group(backend="gloo")
rank = dist.get_rank()
ms, units = bench.aggregate(10.0 + 5.0 * rank, 100.0 * (rank + 1))
bench.dist_barrier()
if rank == 0:
    print(json.dumps(dict(ms=ms, units=units, world=dist.get_world_size())))
dist.destroy_process_group()
"""


def test_aggregate_two_gloo_ranks(tmp_path):
    """value = units of all ranks / max time over ranks (replicas: no data-path collective)."""
    script = tmp_path / "worker.py"
    script.write_text(_WORKER.format(root=ROOT))
    port = 29500 + (os.getpid() % 2000)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    assert all(p.returncode == 0 for p in procs), [o[1][-500:] for o in outs]
    res = json.loads(outs[0][0].strip().splitlines()[-1])
    assert res == dict(ms=15.0, units=300.0, world=2)


def test_clock_summary_flags_reasons():
    s = bench.ClockSampler.__new__(bench.ClockSampler)
    s.samples = [(1.0, 1900, 0), (2.0, 1800, 0x4), (3.0, 1965, 0), (9.0, 500, 0x8)]
    s.max_mhz = 1965
    out = s.summary(0.5, 3.5)
    assert out["sm_mhz"] == 1900 and out["reasons"] == ["sw_power_cap"] and out["samples"] == 3
    out = s.summary(8.0, 10.0)          # too few samples inside: falls back to all of them
    assert "hw_slowdown" in out["reasons"] and out["samples"] == 4


def test_reference_arm_prints_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--steps", "2", "--warmup", "3"], capture_output=True, text=True, timeout=600,
                         env=dict(os.environ, OMP_NUM_THREADS="4"))
    assert out.returncode == 0, out.stderr[-1000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "GB/s" and line["steps"] == 2
    assert line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"] == {"value": line["value"], "unit": "GB/s", "h2d_bytes_per_step": 0,
                           "d2h_bytes_per_step": 0}
    assert line["metric"] == bench.METRIC
