"""Pins for the oracle's 16-bit recipe (binary16 weight scales, bf16 results).

None of these checks reuses the oracle's own code: the conversions are pinned
by exact rationals written out here, by hand-picked bit patterns and by the
library conversions of numpy / torch; the outputs by exact rational sums.
"""
from fractions import Fraction

import numpy as np
import pytest
import torch

from paper_2508_06753_b200 import synth


def _half_fraction(bits):
    """Value of a finite binary16 pattern as an exact rational."""
    sign = -1 if bits >> 15 else 1
    e = (bits >> 10) & 0x1F
    m = bits & 0x3FF
    if e == 0:
        return sign * Fraction(m, 1 << 24)
    return sign * Fraction(1024 + m, 1024) * Fraction(2) ** (e - 15)


def test_half_to_float_hand_picked(oracle):
    cases = {0x0000: 0.0, 0x3C00: 1.0, 0xC000: -2.0, 0x3555: 0.333251953125, 0x0001: 2.0 ** -24,
             0x03FF: 1023 * 2.0 ** -24, 0x0400: 2.0 ** -14, 0x7BFF: 65504.0, 0xFBFF: -65504.0,
             0x2519: 0.0199127197265625}
    for bits, value in cases.items():
        assert oracle.half_to_float(bits) == value, hex(bits)
    assert oracle.half_to_float(0x7C00) == float("inf")
    assert oracle.half_to_float(0xFC00) == float("-inf")
    assert np.isnan(oracle.half_to_float(0x7E00))
    assert np.signbit(oracle.half_to_float(0x8000))


def test_half_to_float_exhaustive(oracle):
    lib = np.arange(65536, dtype=np.uint16).view(np.float16).astype(np.float32)
    for bits in range(65536):
        got = oracle.half_to_float(bits)
        if (bits >> 10) & 0x1F == 0x1F:
            assert (np.isnan(got) and np.isnan(lib[bits])) or got == float(lib[bits])
            continue
        assert got == float(lib[bits]), hex(bits)
        if bits % 97 == 0:                       # exact rationals on a stride (the library pins all)
            assert Fraction(got) == _half_fraction(bits), hex(bits)


def _bf16_value(bits):
    sign = -1 if bits >> 15 else 1
    e = (bits >> 7) & 0xFF
    m = bits & 0x7F
    if e == 0:
        return sign * Fraction(m, 128) * Fraction(2) ** -126
    return sign * (1 + Fraction(m, 128)) * Fraction(2) ** (e - 127)


def test_float_to_bf16_hand_picked(oracle):
    f = np.float32
    assert oracle.float_to_bf16(1.0) == 0x3F80
    assert oracle.float_to_bf16(f(1) + f(2.0 ** -8)) == 0x3F80          # tie -> even (down)
    assert oracle.float_to_bf16(f(1) + f(3 * 2.0 ** -8)) == 0x3F82      # tie -> even (up)
    assert oracle.float_to_bf16(f(1) + f(2.0 ** -8) + f(2.0 ** -23)) == 0x3F81   # just above the tie
    assert oracle.float_to_bf16(f(1) + f(2.0 ** -8) - f(2.0 ** -23)) == 0x3F80   # just below the tie
    assert oracle.float_to_bf16(-0.0) == 0x8000
    assert oracle.float_to_bf16(-2.5) == 0xC020
    assert oracle.float_to_bf16(np.finfo(np.float32).max) == 0x7F80     # rounds up to infinity
    assert oracle.float_to_bf16(float("inf")) == 0x7F80
    assert oracle.float_to_bf16(np.float32(1.9921875 * 2.0 ** 127)) == 0x7F7F     # largest bf16 stays
    got = oracle.float_to_bf16(float("nan"))
    assert (got & 0x7F80) == 0x7F80 and (got & 0x7F) != 0
    assert oracle.float_to_bf16(np.float32(2.0 ** -133)) == 0x0001       # smallest bf16 subnormal
    assert oracle.float_to_bf16(np.float32(2.0 ** -134)) == 0x0000       # tie between 0 and it -> even (0)
    assert oracle.float_to_bf16(np.float32(1.5 * 2.0 ** -134)) == 0x0001


def test_float_to_bf16_is_nearest_with_ties_to_even(oracle):
    rng = np.random.default_rng(5)
    bits = rng.integers(0, 1 << 32, size=4000, dtype=np.uint64).astype(np.uint32)
    # add values sitting exactly on ties and next to them
    base = rng.integers(0x0080, 0x7F00, size=500, dtype=np.uint32) << 16
    bits = np.concatenate([bits, base | 0x8000, base | 0x8001, base | 0x7FFF, base | 0x80008000])
    vals = bits.view(np.float32)
    for u, v in zip(bits, vals):
        if not np.isfinite(v):
            continue
        got = oracle.float_to_bf16(v)
        lo = int(u) >> 16                                   # truncation: the neighbour towards zero
        hi = lo + 1                                         # next pattern away from zero
        exact = Fraction(float(v))
        d_lo = abs(exact - _bf16_value(lo))
        if (hi & 0x7F80) == 0x7F80:                         # next one is infinity: IEEE treats it as 2^128
            d_hi = abs(abs(exact) - Fraction(2) ** 128)
        else:
            d_hi = abs(exact - _bf16_value(hi))
        want = lo if d_lo < d_hi else hi if d_hi < d_lo else (lo if lo % 2 == 0 else hi)
        assert got == want, hex(int(u))


def test_float_to_bf16_matches_library_rounding(oracle):
    rng = np.random.default_rng(6)
    vals = np.concatenate([rng.standard_normal(3000).astype(np.float32) * np.float32(10.0) ** rng.integers(-30, 30, 3000),
                           np.array([0.0, -0.0, 1e-40, -1e-45, 3.3e38], dtype=np.float32)]).astype(np.float32)
    lib = torch.from_numpy(vals).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    for v, w in zip(vals, lib):
        assert oracle.float_to_bf16(v) == int(w), float(v)


def _brute_partials(a, codes, g):
    M, K = a.shape
    N = codes.shape[0]
    return np.einsum("mgk,ngk->mng", a.astype(np.int64).reshape(M, K // g, g),
                     (codes.astype(np.int64) - 2).reshape(N, K // g, g))


@pytest.mark.parametrize("g", [64, 128, 256])
def test_gemm_h_exact_rationals_tiny(oracle, g):
    rng = np.random.default_rng(31)
    M, N, K = 2, 16, 512
    a, s_a = oracle.quantize(synth.activations_bf16(31, M, K))
    codes = rng.integers(0, 4, size=(N, K), dtype=np.uint8)
    s_h = synth.weight_scales_h(31, N, K // g)
    y32, y16 = oracle.gemm_h(a, s_a, codes, s_h, g)
    P = _brute_partials(a, codes, g)
    for m in range(M):
        for n in range(N):
            exact = Fraction(float(s_a[m])) * sum(_half_fraction(int(s_h[n, gi])) * int(P[m, n, gi])
                                                  for gi in range(K // g))
            err = abs(Fraction(float(y32[m, n])) - exact)
            assert err <= abs(exact) * (Fraction(1, 2 ** 24) + Fraction(1, 10 ** 12))
            # the 16-bit result is within half a bf16 unit of the exact value (plus the fp32 rounding)
            v16 = _bf16_value(int(y16[m, n]))
            assert abs(v16 - exact) <= abs(exact) * (Fraction(1, 2 ** 8) + Fraction(1, 2 ** 23))


def test_gemm_h_bf16_is_library_rounding_of_fp32(oracle):
    rng = np.random.default_rng(32)
    M, N, K, g = 3, 48, 1024, 128
    a, s_a = oracle.quantize(synth.activations_bf16(32, M, K))
    codes = rng.integers(0, 4, size=(N, K), dtype=np.uint8)
    y32, y16 = oracle.gemm_h(a, s_a, codes, synth.weight_scales_h(32, N, K // g), g)
    lib = torch.from_numpy(y32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(y16, lib)


def test_gemm_h_scale_indexing_and_unit_scales(oracle):
    rng = np.random.default_rng(33)
    M, N, K, g = 2, 32, 512, 128
    G = K // g
    a = rng.integers(-127, 128, size=(M, K), dtype=np.int8)
    codes = rng.integers(0, 4, size=(N, K), dtype=np.uint8)
    s_a = np.ones(M, dtype=np.float32)
    P = _brute_partials(a, codes, g)
    # all scales 1.0 (0x3C00): the result is the plain integer matrix product
    y32, _ = oracle.gemm_h(a, s_a, codes, np.full((N, G), 0x3C00, dtype=np.uint16), g)
    assert np.array_equal(y32.astype(np.int64), P.sum(axis=2))
    # one non-zero scale (2.0 = 0x4000) at (n, gi): only y[:, n] is non-zero and equals 2 * P[:, n, gi]
    for n, gi in [(0, 0), (5, 3), (31, 1)]:
        s_h = np.zeros((N, G), dtype=np.uint16)
        s_h[n, gi] = 0x4000
        y32, _ = oracle.gemm_h(a, s_a, codes, s_h, g)
        want = np.zeros((M, N))
        want[:, n] = 2 * P[:, n, gi]
        assert np.array_equal(y32.astype(np.float64), want)
