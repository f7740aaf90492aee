"""Pins for the oracle's 16-bit-activation product (no activation quantiser): exact rationals,
the library's float64 matrix product, integer special cases and a one-hot indexing check --
none of them reuses the oracle's code."""
from fractions import Fraction

import numpy as np
import pytest

from paper_2508_06753_b200 import synth


def _bf16_fraction(bits):
    sign = -1 if bits >> 15 else 1
    e = (bits >> 7) & 0xFF
    m = bits & 0x7F
    if e == 0:
        return sign * Fraction(m, 128) * Fraction(2) ** -126
    return sign * (1 + Fraction(m, 128)) * Fraction(2) ** (e - 127)


@pytest.mark.parametrize("g", [64, 128, 256])
def test_a16_exact_rationals_tiny(oracle, g):
    rng = np.random.default_rng(41)
    M, N, K = 2, 16, 512
    bits = synth.activations_bf16(41, M, K, 0.01)
    codes = rng.integers(0, 4, size=(N, K), dtype=np.uint8)
    s_w = synth.weight_scales(41, N, K // g)
    y = oracle.gemm_a16(bits, codes, s_w, g)
    for m in range(M):
        xs = [_bf16_fraction(int(b)) for b in bits[m]]
        for n in range(N):
            exact = sum(xs[k] * (int(codes[n, k]) - 2) * Fraction(float(s_w[n, k // g])) for k in range(K))
            scale = sum(abs(xs[k] * (int(codes[n, k]) - 2)) * Fraction(float(s_w[n, k // g])) for k in range(K))
            # one fp32 rounding of the result plus double-precision accumulation error
            assert abs(Fraction(float(y[m, n])) - exact) <= abs(exact) * Fraction(1, 2 ** 24) + scale * Fraction(1, 2 ** 44)


def test_a16_matches_library_float64_product(oracle):
    rng = np.random.default_rng(42)
    M, N, K, g = 5, 96, 1024, 128
    bits = synth.activations_bf16(42, M, K)
    codes = rng.integers(0, 4, size=(N, K), dtype=np.uint8)
    s_w = synth.weight_scales(42, N, K // g)
    y = oracle.gemm_a16(bits, codes, s_w, g)
    x = synth.bf16_bits_to_float(bits).astype(np.float64)
    w = (codes.astype(np.float64) - 2.0) * np.repeat(s_w.astype(np.float64), g, axis=1)
    ref = x @ w.T
    mag = np.abs(x) @ np.abs(w).T
    assert (np.abs(y.astype(np.float64) - ref) <= np.abs(ref) * 2.0 ** -24 + mag * 2.0 ** -44).all()


def test_a16_integer_inputs_reduce_to_integer_product(oracle):
    rng = np.random.default_rng(43)
    M, N, K, g = 3, 32, 256, 64
    xi = rng.integers(-127, 128, size=(M, K))
    bits = synth.float_to_bf16_bits(xi.astype(np.float32))          # |x| <= 127 is exact in bf16
    assert np.array_equal(synth.bf16_bits_to_float(bits), xi.astype(np.float32))
    codes = rng.integers(0, 4, size=(N, K), dtype=np.uint8)
    y = oracle.gemm_a16(bits, codes, np.ones((N, K // g), dtype=np.float32), g)
    assert np.array_equal(y.astype(np.int64), xi @ (codes.astype(np.int64) - 2).T)
    # the same integers seen as quantised activations with scale 1 give the same result bit for bit
    y8 = oracle.gemm(xi.astype(np.int8), np.ones(M, dtype=np.float32), codes,
                     np.ones((N, K // g), dtype=np.float32), g)
    assert np.array_equal(y, y8)


def test_a16_indexing_one_hot(oracle):
    M, N, K, g = 2, 32, 512, 128
    G = K // g
    rng = np.random.default_rng(44)
    codes = rng.integers(0, 4, size=(N, K), dtype=np.uint8)
    for m, k in [(0, 0), (1, 129), (0, 511)]:
        x = np.zeros((M, K), dtype=np.float32)
        x[m, k] = 3.0
        s_w = np.arange(1, N * G + 1, dtype=np.float32).reshape(N, G)
        y = oracle.gemm_a16(synth.float_to_bf16_bits(x), codes, s_w, g)
        want = np.zeros((M, N))
        want[m] = 3.0 * (codes[:, k].astype(np.float64) - 2.0) * s_w[:, k // g]
        assert np.array_equal(y.astype(np.float64), want)
    # transposed-operand trap: swapping tokens changes which row is non-zero
    assert want[0].any() and not want[1].any()
