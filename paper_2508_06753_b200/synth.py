"""Seeded synthetic inputs for the W2A8 workloads (no method arithmetic here).

The paper benchmarks on weight shapes taken from Llama-3-8B-class models with
dummy 2-bit weights (Sec. III-B, III-D); the trained checkpoints are not
needed for kernel work.  This module produces stand-ins with the same shapes
and the value distributions of the benchmark configurations: uniform 2-bit
codes (or ternary codes {1,2,3}), log-normal fp32 group scales, and bf16
N(0,1) activations with optional +-20 outliers.  It only draws random numbers
and converts formats; packing, quantising and multiplying live elsewhere.
The same host arrays feed the CPU reference and (after upload) the GPU.
"""
from __future__ import annotations

import numpy as np

# tensor ids inside one (seed) stream
_T_CODES, _T_SCALES, _T_ACT, _T_OUTLIER = 0, 1, 2, 3

# (name, K, N) of the decoder linears of one layer, in execution order.
LLAMA3_8B_LAYER = [("q", 4096, 4096), ("k", 4096, 1024), ("v", 4096, 1024), ("o", 4096, 4096),
                   ("gate", 4096, 14336), ("up", 4096, 14336), ("down", 14336, 4096)]
LLAMA3_70B_LAYER = [("q", 8192, 8192), ("k", 8192, 1024), ("v", 8192, 1024), ("o", 8192, 8192),
                    ("gate", 8192, 28672), ("up", 8192, 28672), ("down", 28672, 8192)]

# Benchmark configurations: index = position in the configuration list.
CONFIGS = {
    0: dict(name="gemv-2048", shapes=[("gemv", 2048, 2048)], Ms=[1], group=64, ternary=False,
            outlier_frac=0.0, seed=0),
    1: dict(name="llama3-8b-layer", shapes=LLAMA3_8B_LAYER, Ms=[1, 4, 16], group=64,
            ternary=False, outlier_frac=0.0, seed=1000),
    2: dict(name="llama3-8b-layer-ternary", shapes=LLAMA3_8B_LAYER, Ms=[1, 8], group=0,
            ternary=True, outlier_frac=0.0, seed=2000),  # group 0 means group = K
    3: dict(name="llama3-70b-layer", shapes=LLAMA3_70B_LAYER, Ms=[1, 8, 32], group=128,
            ternary=False, outlier_frac=0.01, seed=3000),
    4: dict(name="llama3-8b-prefill", shapes=[("gate_up", 4096, 14336), ("down", 14336, 4096)],
            Ms=[512, 2048, 8192], group=64, ternary=False, outlier_frac=0.0, seed=4000),
}


def _rng(seed: int, tensor: int) -> np.random.Generator:
    return np.random.default_rng([int(seed), int(tensor)])


def float_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_float(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def weight_codes(seed: int, N: int, K: int, ternary: bool = False) -> np.ndarray:
    """uint8 [N][K]; uniform over {0,1,2,3}, or over {1,2,3} when ternary."""
    rng = _rng(seed, _T_CODES)
    lo = 1 if ternary else 0
    return rng.integers(lo, 4, size=(N, K), dtype=np.uint8)


def weight_scales(seed: int, N: int, G: int) -> np.ndarray:
    """fp32 [N][G]; 0.02 * exp(0.5 z), z ~ N(0,1), evaluated in double."""
    z = _rng(seed, _T_SCALES).standard_normal(size=(N, G))
    return (0.02 * np.exp(0.5 * z)).astype(np.float32)


def weight_scales_h(seed: int, N: int, G: int) -> np.ndarray:
    """IEEE binary16 bit patterns uint16 [N][G]: the fp32 scales of `weight_scales` stored in 16 bits."""
    return weight_scales(seed, N, G).astype(np.float16).view(np.uint16)


def activations_bf16(seed: int, M: int, K: int, outlier_frac: float = 0.0) -> np.ndarray:
    """bf16 bit patterns uint16 [M][K]; N(0,1), optional +-20 outliers.

    With outlier_frac > 0, exactly floor(outlier_frac * K) distinct positions
    per row are overwritten with +20 or -20 (random sign).
    """
    x = _rng(seed, _T_ACT).standard_normal(size=(M, K)).astype(np.float32)
    n_out = int(np.floor(outlier_frac * K))
    if n_out > 0:
        rng = _rng(seed, _T_OUTLIER)
        for m in range(M):
            pos = rng.choice(K, size=n_out, replace=False)
            sign = rng.integers(0, 2, size=n_out) * 2 - 1
            x[m, pos] = 20.0 * sign
    return float_to_bf16_bits(x)


def make_linear(seed: int, K: int, N: int, group: int, ternary: bool = False):
    """(codes uint8 [N][K], scales fp32 [N][K/g]) for one linear layer."""
    g = K if group in (0, None) else group
    return weight_codes(seed, N, K, ternary), weight_scales(seed, N, K // g)


def config_group(cfg: dict, K: int) -> int:
    return K if cfg["group"] in (0, None) else cfg["group"]


def shape_seed(cfg: dict, shape_index: int) -> int:
    return cfg["seed"] + shape_index
