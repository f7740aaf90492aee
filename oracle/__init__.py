"""W2A8 reference ("oracle") -- test infrastructure, not the product.

Thin ctypes/numpy front end of ``w2a8_ref.c``: a plain scalar CPU statement
of the W2A8 path (pack, per-token int8 quantiser, exact int32 per-group
sums, scaled fp32 outputs).  Nothing here touches CUDA and nothing in the
CUDA package imports this module.  Only the tests, the smoke check and the
benchmark's CPU-baseline / reference legs may use it.

All arrays are C-contiguous numpy arrays; shapes use the GEMM naming
(M tokens, N output channels, K contraction, g group length).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "w2a8_ref.c")
_LIB = os.path.join(_HERE, "libw2a8_ref.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C reference into ``libw2a8_ref.so`` next to its source."""
    def stale():
        return not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale():
        import fcntl
        with open(_LIB + ".lock", "w") as lock:        # several test or bench processes may race here
            fcntl.flock(lock, fcntl.LOCK_EX)
            try:
                if force or stale():
                    tmp = _LIB + f".tmp{os.getpid()}"
                    cmd = ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared",
                           "-fPIC", "-o", tmp, _SRC, "-lm"]
                    subprocess.run(cmd, check=True)
                    os.replace(tmp, _LIB)
            finally:
                fcntl.flock(lock, fcntl.LOCK_UN)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.ref_num_threads.restype = ctypes.c_int
        _lib.ref_half_to_float.restype = ctypes.c_float
        _lib.ref_half_to_float.argtypes = [ctypes.c_uint16]
        _lib.ref_float_to_bf16.restype = ctypes.c_uint16
        _lib.ref_float_to_bf16.argtypes = [ctypes.c_float]
    return _lib


def _p(arr):
    return arr.ctypes.data_as(ctypes.c_void_p)


def num_threads() -> int:
    return int(_load().ref_num_threads())


def pack(codes: np.ndarray) -> np.ndarray:
    """codes uint8 [N][K] (0..3) -> packed uint32 [N][K/16] (W2P layout)."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    N, K = codes.shape
    assert K % 64 == 0
    out = np.empty((N, K // 16), dtype=np.uint32)
    _load().ref_pack(_p(codes), ctypes.c_int(N), ctypes.c_int(K), _p(out))
    return out


def unpack(packed: np.ndarray, K: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint32)
    N = packed.shape[0]
    assert packed.shape[1] == K // 16
    out = np.empty((N, K), dtype=np.uint8)
    _load().ref_unpack(_p(packed), ctypes.c_int(N), ctypes.c_int(K), _p(out))
    return out


def quantize(x_bf16_bits: np.ndarray):
    """bf16 bit patterns uint16 [M][K] -> (int8 [M][K], fp32 scale [M])."""
    x = np.ascontiguousarray(x_bf16_bits, dtype=np.uint16)
    M, K = x.shape
    a = np.empty((M, K), dtype=np.int8)
    s = np.empty((M,), dtype=np.float32)
    _load().ref_quantize(_p(x), ctypes.c_int(M), ctypes.c_int(K), _p(a), _p(s))
    return a, s


def partials(a: np.ndarray, codes: np.ndarray, g: int) -> np.ndarray:
    """Exact int32 per-group sums P[M][N][K/g]."""
    a = np.ascontiguousarray(a, dtype=np.int8)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    M, K = a.shape
    N = codes.shape[0]
    assert codes.shape[1] == K and K % g == 0
    P = np.empty((M, N, K // g), dtype=np.int32)
    _load().ref_partials(_p(a), _p(codes), ctypes.c_int(M), ctypes.c_int(N), ctypes.c_int(K),
                         ctypes.c_int(g), _p(P))
    return P


def gemm(a: np.ndarray, a_scale: np.ndarray, codes: np.ndarray, w_scale: np.ndarray,
         g: int) -> np.ndarray:
    """fp32 outputs y[M][N] (double accumulation, rounded once)."""
    a = np.ascontiguousarray(a, dtype=np.int8)
    a_scale = np.ascontiguousarray(a_scale, dtype=np.float32)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    w_scale = np.ascontiguousarray(w_scale, dtype=np.float32)
    M, K = a.shape
    N = codes.shape[0]
    assert codes.shape[1] == K and K % g == 0
    assert w_scale.shape == (N, K // g) and a_scale.shape == (M,)
    y = np.empty((M, N), dtype=np.float32)
    _load().ref_gemm(_p(a), _p(a_scale), _p(codes), _p(w_scale), ctypes.c_int(M),
                     ctypes.c_int(N), ctypes.c_int(K), ctypes.c_int(g), _p(y))
    return y


def half_to_float(h: int) -> float:
    """IEEE binary16 bit pattern -> value (exact)."""
    return float(_load().ref_half_to_float(int(h) & 0xFFFF))


def float_to_bf16(f: float) -> int:
    """fp32 value -> bf16 bit pattern, round to nearest even."""
    return int(_load().ref_float_to_bf16(float(np.float32(f))))


def gemm_h(a: np.ndarray, a_scale: np.ndarray, codes: np.ndarray, w_scale_h: np.ndarray, g: int):
    """16-bit recipe: w_scale_h holds binary16 bit patterns uint16 [N][K/g].

    Returns (y fp32 [M][N], the same values rounded to bf16 bit patterns uint16 [M][N]).
    """
    a = np.ascontiguousarray(a, dtype=np.int8)
    a_scale = np.ascontiguousarray(a_scale, dtype=np.float32)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    w_scale_h = np.ascontiguousarray(w_scale_h, dtype=np.uint16)
    M, K = a.shape
    N = codes.shape[0]
    assert codes.shape[1] == K and K % g == 0
    assert w_scale_h.shape == (N, K // g) and a_scale.shape == (M,)
    y32 = np.empty((M, N), dtype=np.float32)
    y16 = np.empty((M, N), dtype=np.uint16)
    _load().ref_gemm_h(_p(a), _p(a_scale), _p(codes), _p(w_scale_h), ctypes.c_int(M),
                       ctypes.c_int(N), ctypes.c_int(K), ctypes.c_int(g), _p(y32), _p(y16))
    return y32, y16


def gemm_a16(x_bf16_bits: np.ndarray, codes: np.ndarray, w_scale: np.ndarray, g: int) -> np.ndarray:
    """16-bit activations, no quantiser: fp32 y[M][N] = sum_k x[m][k] (q[n][k] - 2) s_w[n][k/g]
    (double accumulation, rounded once).  x: bf16 bit patterns uint16 [M][K]."""
    x = np.ascontiguousarray(x_bf16_bits, dtype=np.uint16)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    w_scale = np.ascontiguousarray(w_scale, dtype=np.float32)
    M, K = x.shape
    N = codes.shape[0]
    assert codes.shape[1] == K and K % g == 0 and w_scale.shape == (N, K // g)
    y = np.empty((M, N), dtype=np.float32)
    _load().ref_gemm_a16(_p(x), _p(codes), _p(w_scale), ctypes.c_int(M), ctypes.c_int(N),
                         ctypes.c_int(K), ctypes.c_int(g), _p(y))
    return y
