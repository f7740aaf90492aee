"""Pins for the CPU reference: each check uses something other than the
reference's own code -- hand-written golden words, exact rational
arithmetic, brute force in numpy int64, closed forms and invariants."""
from fractions import Fraction

import numpy as np
import pytest

from conftest import golden_rows
from paper_2508_06753_b200 import synth


# ----------------------------------------------------------------- layout
def test_packed_bytes_closed_form(oracle):
    # 2-bit storage: K*N/4 bytes (a 256-bit load carries 128 codes, Sec. II-B)
    for N, K in [(16, 64), (32, 256), (48, 1600), (16, 448)]:
        codes = np.zeros((N, K), dtype=np.uint8)
        assert oracle.pack(codes).nbytes == K * N // 4
    assert 256 // 8 * 4 == 128


def test_golden_words(oracle):
    for row in golden_rows("w2p_words.txt"):
        codes16 = [int(v) for v in row[:16]]
        word = int(row[16], 16)
        codes = np.zeros((1, 64), dtype=np.uint8)
        codes[0, :16] = codes16
        packed = oracle.pack(codes)
        assert int(packed[0, 0]) == word, (codes16, hex(int(packed[0, 0])), hex(word))
        assert not packed[0, 1:].any()


def test_golden_word_positions(oracle):
    for K, k, idx in [(int(a), int(b), int(c)) for a, b, c in golden_rows("w2p_word_positions.txt")]:
        codes = np.zeros((2, K), dtype=np.uint8)
        codes[1, k] = 3
        packed = oracle.pack(codes)
        assert not packed[0].any()
        nz = np.flatnonzero(packed[1])
        assert nz.tolist() == [idx], (K, k, nz.tolist(), idx)


def test_shift_mask_gives_consecutive_k(oracle):
    # (word >> 2j) & 0x03030303 must be codes l = 4j..4j+3, one per byte
    rng = np.random.default_rng(7)
    codes = rng.integers(0, 4, size=(1, 64), dtype=np.uint8)
    words = oracle.pack(codes)[0]            # R = 1: natural word order
    for w in range(4):
        for j in range(4):
            lanes = (int(words[w]) >> (2 * j)) & 0x03030303
            got = [(lanes >> (8 * b)) & 0xFF for b in range(4)]
            assert got == codes[0, 16 * w + 4 * j:16 * w + 4 * j + 4].tolist()


def test_one_hot_words_all_slots(oracle):
    # 16 positions x 3 non-zero codes: the word equals code << (8*(l%4) + 2*(l//4))
    for l in range(16):
        for c in (1, 2, 3):
            codes = np.zeros((1, 64), dtype=np.uint8)
            codes[0, l] = c
            assert int(oracle.pack(codes)[0, 0]) == c << (8 * (l % 4) + 2 * (l // 4))


@pytest.mark.parametrize("N,K", [(16, 64), (16, 256), (32, 448), (16, 1600), (48, 2048)])
def test_pack_roundtrip_and_permutation(oracle, N, K):
    rng = np.random.default_rng(N * 100003 + K)
    codes = rng.integers(0, 4, size=(N, K), dtype=np.uint8)
    packed = oracle.pack(codes)
    assert packed.shape == (N, K // 16)
    assert np.array_equal(oracle.unpack(packed, K), codes)
    # every k lands in a distinct (word, slot): one-hot rows give K distinct bits
    seen = set()
    for k in range(K):
        one = np.zeros((1, K), dtype=np.uint8)
        one[0, k] = 1
        w = oracle.pack(one)[0]
        nz = np.flatnonzero(w)
        assert len(nz) == 1
        v = int(w[nz[0]])
        assert v & (v - 1) == 0
        seen.add((int(nz[0]), v))
    assert len(seen) == K


def test_unit_t_holds_quarter_t_of_each_slice(oracle):
    # In a full 256-k block the 16-byte unit t (words 4t..4t+3) holds
    # k = 64 s + 16 t + l for s = 0..3: check by labelling codes.
    K = 512
    k = np.arange(K)
    for which, fn in (("slice", lambda kk: (kk % 256) // 64), ("quarter", lambda kk: (kk % 64) // 16)):
        codes = fn(k).astype(np.uint8)[None, :]
        words = oracle.pack(codes)[0].reshape(2, 4, 4)   # [block][unit t][word in unit]
        for b in range(2):
            for t in range(4):
                for s in range(4):
                    expect = (s if which == "slice" else t) * 0x55555555
                    assert int(words[b, t, s]) == expect


def test_out_of_range_codes_are_masked(oracle):
    codes = np.full((1, 64), 0xFE, dtype=np.uint8)       # low two bits = 2
    assert (oracle.pack(codes) == 0xAAAAAAAA).all()


def test_ternary_code_map_matches_paper_encoding(oracle):
    # Fig. 3 encoding (low bit = non-zero, high bit = sign) vs value = q - 2
    for c, value, q in [(int(a), int(b), int(d)) for a, b, d in golden_rows("ternary_code_map.txt")]:
        assert q == c ^ 2
        nonzero, negative = c & 1, (c >> 1) & 1
        assert value == (0 if not nonzero else (-1 if negative else 1))
        a = np.array([[1] + [0] * 63], dtype=np.int8)
        codes = np.full((1, 64), 2, dtype=np.uint8)      # value 0 elsewhere
        codes[0, 0] = q
        assert int(oracle.partials(a, codes, 64)[0, 0, 0]) == value


# -------------------------------------------------------------- quantiser
def _rn_f32(fr):
    """Round an exact rational to the nearest fp32 (ties to even); returns a
    Fraction, or None for overflow to infinity."""
    if fr == 0:
        return Fraction(0)
    sign = -1 if fr < 0 else 1
    mag = abs(fr)
    e = mag.numerator.bit_length() - mag.denominator.bit_length()
    if Fraction(2) ** e > mag:
        e -= 1
    e = max(e, -126)
    quantum = Fraction(2) ** (e - 23)
    n = mag / quantum
    fl = n.numerator // n.denominator
    rem = n - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    out = fl * quantum
    if out >= Fraction(2) ** 128:
        return None
    return sign * out


def _round_half_even(fr):
    fl = fr.numerator // fr.denominator
    rem = fr - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    return fl


def _bf16_fraction(bits):
    sign = -1 if bits >> 15 else 1
    e = (bits >> 7) & 0xFF
    m = bits & 0x7F
    if e == 0:
        return sign * Fraction(m, 128) * Fraction(2) ** -126
    return sign * (1 + Fraction(m, 128)) * Fraction(2) ** (e - 127)


def _expected_row(bits_row):
    vals = [_bf16_fraction(int(b)) for b in bits_row]
    amax = max(abs(v) for v in vals)
    if amax == 0:
        return [0] * len(vals), Fraction(0)
    s = _rn_f32(amax / 127)
    if s == 0:
        return [0] * len(vals), Fraction(0)
    inv = _rn_f32(1 / s)
    if inv is None:
        return [0] * len(vals), Fraction(0)
    out = []
    for v in vals:
        t = _rn_f32(v * inv)
        out.append(max(-127, min(127, _round_half_even(t))))
    return out, s


def _finite_bf16_patterns():
    allb = np.arange(1 << 16, dtype=np.uint32)
    finite = ((allb >> 7) & 0xFF) != 0xFF
    return allb[finite].astype(np.uint16)


@pytest.mark.parametrize("amax_bits", [
    0x3F80,   # 1.0
    0x4040,   # 3.0
    0x4088,   # 4.25
    0x41A0,   # 20.0
    0x42FE,   # 127.0  (inverse scale exactly 1: half-way cases occur)
    0x3580,   # 2^-20
    0x5DC0,   # 3 * 2^60... large
    0x0080,   # smallest normal
])
def test_quantiser_exhaustive_against_exact_rationals(oracle, amax_bits):
    pats = _finite_bf16_patterns()
    amax = _bf16_fraction(amax_bits)
    mags = np.array([abs(_bf16_fraction(int(b))) <= amax for b in pats])
    row = np.concatenate([[np.uint16(amax_bits)], pats[mags]])
    # thin the huge set deterministically but keep every pattern near ties:
    # all patterns whose magnitude is within 2^-9 relative of amax * (j+0.5)/127
    # would be hard to single out, so simply keep all of them.
    a, s = oracle.quantize(row[None, :])
    exp_a, exp_s = _expected_row(row)
    assert Fraction(float(s[0])) == exp_s
    assert a[0].tolist() == exp_a


def test_quantiser_ties_round_to_even(oracle):
    # amax = 127 -> scale 1, inverse 1: x = k + 0.5 is a tie
    vals = np.array([127.0, 0.5, 1.5, 2.5, 3.5, -0.5, -1.5, -2.5, 126.5, -126.5, 100.5],
                    dtype=np.float32)
    a, s = oracle.quantize(synth.float_to_bf16_bits(vals)[None, :])
    assert float(s[0]) == 1.0
    assert a[0].tolist() == [127, 0, 2, 2, 4, 0, -2, -2, 126, -126, 100]


def test_quantiser_invariants(oracle):
    bits = synth.activations_bf16(11, 5, 256)
    a, s = oracle.quantize(bits)
    x = synth.bf16_bits_to_float(bits)
    # the abs-max element maps to +-127
    for m in range(5):
        j = int(np.argmax(np.abs(x[m])))
        assert abs(int(a[m, j])) == 127
        assert np.abs(a[m]).max() == 127
    # negation negates exactly
    a_neg, s_neg = oracle.quantize(bits ^ np.uint16(0x8000))
    assert np.array_equal(a_neg, -a) and np.array_equal(s_neg, s)
    # scaling by a power of two: same codes, scale scaled exactly
    x8 = synth.float_to_bf16_bits(x * 8.0)
    a8, s8 = oracle.quantize(x8)
    assert np.array_equal(a8, a) and np.array_equal(s8, s * np.float32(8.0))
    # constant rows
    c = synth.float_to_bf16_bits(np.full((1, 64), -3.25, dtype=np.float32))
    ac, sc = oracle.quantize(c)
    assert (ac == -127).all()
    assert Fraction(float(sc[0])) == _rn_f32(Fraction(13, 4) / 127)


def test_quantiser_degenerate_rows(oracle):
    zero = np.zeros((1, 64), dtype=np.uint16)
    zero[0, 3] = 0x8000                                    # -0.0
    a, s = oracle.quantize(zero)
    assert not a.any() and float(s[0]) == 0.0
    tiny = np.zeros((1, 64), dtype=np.uint16)
    tiny[0, 5] = 0x0001                                    # smallest bf16 subnormal
    a, s = oracle.quantize(tiny)                           # 1/(amax/127) overflows
    assert not a.any() and float(s[0]) == 0.0


def test_quantiser_outlier_rows(oracle):
    bits = synth.activations_bf16(5, 3, 8192, outlier_frac=0.01)
    x = synth.bf16_bits_to_float(bits)
    assert ((np.abs(x) == 20.0).sum(axis=1) == 81).all()
    a, s = oracle.quantize(bits)
    assert np.all(np.abs(a[np.abs(x) == 20.0]) == 127)
    assert np.allclose(s, 20.0 / 127.0)


# ------------------------------------------------------- integer partials
def _brute_partials(a, codes, g):
    M, K = a.shape
    N = codes.shape[0]
    v = codes.astype(np.int64) - 2
    out = np.zeros((M, N, K // g), dtype=np.int64)
    for gi in range(K // g):
        out[:, :, gi] = a[:, gi * g:(gi + 1) * g].astype(np.int64) @ v[:, gi * g:(gi + 1) * g].T
    return out


@pytest.mark.parametrize("M,N,K,g", [(1, 16, 64, 64), (2, 32, 128, 64), (3, 16, 128, 128),
                                     (3, 32, 448, 64), (2, 16, 512, 256), (1, 16, 256, 256)])
def test_partials_brute_force(oracle, M, N, K, g):
    rng = np.random.default_rng(K + N + M)
    a = rng.integers(-127, 128, size=(M, K), dtype=np.int8)
    codes = rng.integers(0, 4, size=(N, K), dtype=np.uint8)
    assert np.array_equal(oracle.partials(a, codes, g), _brute_partials(a, codes, g))


def test_partials_pure_python_triple_loop(oracle):
    rng = np.random.default_rng(3)
    M, N, K, g = 2, 16, 128, 64
    a = rng.integers(-127, 128, size=(M, K), dtype=np.int8)
    codes = rng.integers(0, 4, size=(N, K), dtype=np.uint8)
    P = oracle.partials(a, codes, g)
    for m in range(M):
        for n in range(N):
            for gi in range(K // g):
                tot = 0
                for k in range(gi * g, (gi + 1) * g):
                    tot += int(a[m, k]) * (int(codes[n, k]) - 2)
                assert int(P[m, n, gi]) == tot


def test_partials_closed_forms(oracle):
    rng = np.random.default_rng(5)
    K, g, N = 256, 64, 16
    a = rng.integers(-127, 128, size=(2, K), dtype=np.int8)
    gsum = a.astype(np.int64).reshape(2, K // g, g).sum(axis=2)
    for c in range(4):                                     # all codes equal c
        P = oracle.partials(a, np.full((N, K), c, dtype=np.uint8), g)
        assert np.array_equal(P, np.broadcast_to(((c - 2) * gsum)[:, None, :], P.shape))
    # extreme magnitudes: no overflow at the largest group in any configuration
    K = 28672
    P = oracle.partials(np.full((1, K), 127, np.int8), np.full((16, K), 3, np.uint8), K)
    assert (P == 127 * K).all()
    P = oracle.partials(np.full((1, K), -127, np.int8), np.zeros((16, K), np.uint8), K)
    assert (P == 254 * K).all() and 254 * K == 7282688


def test_partials_invariants(oracle):
    rng = np.random.default_rng(9)
    M, N, K = 3, 32, 512
    a = rng.integers(-127, 128, size=(M, K), dtype=np.int8)
    codes = rng.integers(0, 4, size=(N, K), dtype=np.uint8)
    P64 = oracle.partials(a, codes, 64)
    P128 = oracle.partials(a, codes, 128)
    PK = oracle.partials(a, codes, K)
    assert np.array_equal(P64.reshape(M, N, -1, 2).sum(axis=3), P128)      # additivity
    assert np.array_equal(P64.sum(axis=2, keepdims=True), PK)
    assert np.array_equal(oracle.partials(-a, codes, 64), -P64)            # odd in a
    perm = np.concatenate([rng.permutation(64) + 64 * i for i in range(K // 64)])
    assert np.array_equal(oracle.partials(a[:, perm], codes[:, perm], 64), P64)
    # transposed-operand trap: swapping the roles of rows must change the result shape/values
    assert not np.array_equal(P64[0, 1], P64[1, 0])


# ---------------------------------------------------------------- outputs
def test_gemm_exact_rationals_tiny(oracle):
    rng = np.random.default_rng(21)
    M, N, K, g = 2, 16, 128, 64
    bits = synth.activations_bf16(21, M, K)
    a, s_a = oracle.quantize(bits)
    codes = rng.integers(0, 4, size=(N, K), dtype=np.uint8)
    s_w = synth.weight_scales(21, N, K // g)
    y = oracle.gemm(a, s_a, codes, s_w, g)
    P = _brute_partials(a, codes, g)
    for m in range(M):
        for n in range(N):
            exact = Fraction(float(s_a[m])) * sum(Fraction(float(s_w[n, gi])) * int(P[m, n, gi])
                                                  for gi in range(K // g))
            err = abs(Fraction(float(y[m, n])) - exact)
            assert err <= abs(exact) * (Fraction(1, 2 ** 24) + Fraction(1, 10 ** 12))


def test_gemm_unit_scales_single_group_is_one_multiply(oracle):
    rng = np.random.default_rng(22)
    M, N, K = 3, 16, 256
    a, s_a = oracle.quantize(synth.activations_bf16(22, M, K))
    codes = rng.integers(0, 4, size=(N, K), dtype=np.uint8)
    y = oracle.gemm(a, s_a, codes, np.ones((N, 1), np.float32), K)
    P = _brute_partials(a, codes, K)[:, :, 0]
    expect = s_a[:, None] * P.astype(np.float32)           # exact ints < 2^24, one RN multiply
    assert np.array_equal(y, expect)


def test_gemm_reduces_to_integer_matmul(oracle):
    rng = np.random.default_rng(23)
    M, N, K, g = 2, 32, 256, 64
    a = rng.integers(-127, 128, size=(M, K), dtype=np.int8)
    codes = rng.integers(0, 4, size=(N, K), dtype=np.uint8)
    s_w = np.full((N, K // g), 0.25, np.float32)
    s_a = np.array([2.0, 0.5], np.float32)
    y = oracle.gemm(a, s_a, codes, s_w, g)
    full = a.astype(np.int64) @ (codes.astype(np.int64) - 2).T
    assert np.array_equal(y, (full * 0.25 * s_a[:, None].astype(np.float64)).astype(np.float32))


def test_gemm_scale_indexing(oracle):
    # a scale that differs for one (channel, group) must touch exactly that channel
    rng = np.random.default_rng(24)
    M, N, K, g = 1, 16, 256, 64
    a = rng.integers(1, 128, size=(M, K), dtype=np.int8)
    codes = np.full((N, K), 3, np.uint8)
    s_w = np.ones((N, K // g), np.float32)
    base = oracle.gemm(a, np.ones(M, np.float32), codes, s_w, g)
    s_w[5, 2] = 3.0
    y = oracle.gemm(a, np.ones(M, np.float32), codes, s_w, g)
    diff = (y - base)[0]
    expect = np.zeros(N, np.float32)
    expect[5] = 2.0 * a[0, 128:192].astype(np.int64).sum()
    assert np.array_equal(diff, expect)
