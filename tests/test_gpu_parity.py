"""GPU parity: the CUDA path, called through the C ABI, against the CPU
reference on the same seeded inputs.  Bit-exact for packed weights, int8
activations, activation scales and int32 per-group sums; fp32 outputs within
1e-4 * max|row| (the tolerance of the target statement)."""
import os

import numpy as np
import pytest

from conftest import Guarded
from paper_2508_06753_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 1e-4


@pytest.fixture(scope="module")
def gpu():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2508_06753_b200 import binding, build
    build.build()
    binding.lib()
    return torch, binding


def _dev(torch, arr):
    return torch.from_numpy(np.ascontiguousarray(arr)).cuda()


def _bf16_dev(torch, bits):
    return _dev(torch, bits.view(np.int16)).view(torch.bfloat16)


def _row_err_ok(y, y_ref):
    err = np.abs(y.astype(np.float64) - y_ref.astype(np.float64)).max(axis=1)
    bound = TOL * np.abs(y_ref).max(axis=1)
    return (err <= bound).all(), float((err / np.maximum(bound, 1e-30)).max())


# ------------------------------------------------------------------- pack
@pytest.mark.parametrize("N,K", [(16, 64), (16, 256), (32, 448), (48, 1600), (2048, 2048),
                                 (1024, 4096), (16, 28672), (4096, 14336)])
def test_pack_bit_exact(gpu, oracle, N, K):
    torch, b = gpu
    codes = synth.weight_codes(N + K, N, K)
    packed = b.w2_pack(_dev(torch, codes))
    torch.cuda.synchronize()
    got = packed.cpu().numpy().view(np.uint32)
    assert got.nbytes == N * K // 4 == b.w2_packed_bytes(N, K)
    assert np.array_equal(got, oracle.pack(codes))


def test_pack_masks_high_bits(gpu, oracle):
    torch, b = gpu
    rng = np.random.default_rng(1)
    codes = rng.integers(0, 256, size=(32, 512), dtype=np.uint8)
    got = b.w2_pack(_dev(torch, codes)).cpu().numpy().view(np.uint32)
    assert np.array_equal(got, oracle.pack(codes & 3))


# --------------------------------------------------------------- quantiser
@pytest.mark.parametrize("M,K,frac", [(1, 64, 0.0), (1, 2048, 0.0), (4, 4096, 0.0), (16, 14336, 0.0),
                                      (8, 8192, 0.01), (32, 28672, 0.01), (3, 1600, 0.0),
                                      (300, 4096, 0.0)])
def test_quantize_bit_exact(gpu, oracle, M, K, frac):
    torch, b = gpu
    bits = synth.activations_bf16(M * 7 + K, M, K, frac)
    a, s = b.a8_quantize(_bf16_dev(torch, bits))
    torch.cuda.synchronize()
    a_ref, s_ref = oracle.quantize(bits)
    assert np.array_equal(a.cpu().numpy(), a_ref)
    assert np.array_equal(s.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))


def test_quantize_all_bf16_patterns(gpu, oracle):
    torch, b = gpu
    allb = np.arange(1 << 16, dtype=np.uint32)
    finite = allb[((allb >> 7) & 0xFF) != 0xFF].astype(np.uint16)
    rows = []
    for amax_bits in (0x3F80, 0x4040, 0x4088, 0x41A0, 0x42FE, 0x3580, 0x5DC0, 0x0080, 0x0001, 0x7F7F):
        keep = finite[(finite & 0x7FFF) <= amax_bits]
        row = np.zeros(65536, dtype=np.uint16)
        row[:keep.size] = keep
        row[keep.size] = amax_bits
        rows.append(row)
    bits = np.stack(rows)
    a, s = b.a8_quantize(_bf16_dev(torch, bits))
    a_ref, s_ref = oracle.quantize(bits)
    assert np.array_equal(s.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(a.cpu().numpy(), a_ref)


def test_quantize_degenerate_rows(gpu, oracle):
    torch, b = gpu
    bits = synth.activations_bf16(3, 4, 256)
    bits[1, :] = 0
    bits[1, 7] = 0x8000
    bits[2, :] = 0
    bits[2, 9] = 0x0003
    a, s = b.a8_quantize(_bf16_dev(torch, bits))
    a_ref, s_ref = oracle.quantize(bits)
    assert np.array_equal(a.cpu().numpy(), a_ref)
    assert np.array_equal(s.cpu().numpy(), s_ref)
    assert not a.cpu().numpy()[1:3].any() and s_ref[1] == 0 and s_ref[2] == 0


# ------------------------------------------------------- partials / outputs
def _problem(seed, M, N, K, group, ternary=False, frac=0.0):
    g = K if group == 0 else group
    codes, s_w = synth.make_linear(seed, K, N, g, ternary)
    bits = synth.activations_bf16(seed, M, K, frac)
    return codes, s_w, bits, g


def _run_gpu(torch, b, codes, s_w, bits, g, want_partials=True):
    """The hot path through the C ABI.  Outputs, int32 sums and the workspace sit between canary
    words, checked after the calls: nothing may be written outside them."""
    M, K = bits.shape
    N = codes.shape[0]
    packed = b.w2_pack(_dev(torch, codes))
    a, s_a = b.a8_quantize(_bf16_dev(torch, bits))
    ws_bytes = (b.w2a8_workspace_bytes(M, N, K, g) + 15) // 16 * 16
    gws = Guarded(torch, (max(ws_bytes, 256),), torch.uint8)
    b.w2a8_workspace_init(gws.view)
    gy = Guarded(torch, (M, N), torch.float32, float("nan"))
    gy2 = Guarded(torch, (M, N), torch.float32, float("nan"))
    y = b.w2a8_gemm(a, s_a, packed, _dev(torch, s_w), g, gws.view, gy.view)
    y2 = b.w2a8_gemm(a, s_a, packed, _dev(torch, s_w), g, gws.view, gy2.view)
    gp = Guarded(torch, (M, N, K // g), torch.int32) if want_partials else None
    P = b.w2a8_gemm_partials(a, packed, g, gws.view, gp.view) if want_partials else None
    torch.cuda.synchronize()
    assert b.w2a8_workspace_status(gws.view) == 0
    gy.check("y"), gy2.check("y"), gws.check("workspace")
    if gp is not None:
        gp.check("partials")
    assert torch.equal(y, y2), "repeated calls must be bitwise equal"
    return (a.cpu().numpy(), s_a.cpu().numpy(), y.cpu().numpy(),
            None if P is None else P.cpu().numpy())


CASES = [
    # M, N, K, group (0 = K), ternary, outlier fraction
    (1, 2048, 2048, 64, False, 0.0),       # configuration 0 in full
    (1, 16, 64, 64, False, 0.0),           # smallest legal problem
    (2, 16, 256, 64, False, 0.0),
    (3, 48, 448, 64, False, 0.0),          # ragged K: trailing block of three slices
    (1, 1600, 1600, 64, False, 0.0),       # the paper's smallest shape (Sec. III-B)
    (5, 32, 1600, 0, True, 0.0),           # ragged K, one scale per channel
    (4, 1040, 4096, 64, False, 0.0),       # N not a multiple of anything but 16
    (8, 256, 4096, 128, False, 0.01),
    (9, 256, 2048, 128, False, 0.0),       # two token tiles, ragged
    (16, 512, 4096, 64, False, 0.0),
    (17, 128, 1024, 256, False, 0.0),
    (32, 256, 8192, 128, False, 0.01),
    (8, 128, 4096, 0, True, 0.0),          # ternary, group = K
    (1, 64, 14336, 0, True, 0.0),
    (33, 64, 512, 64, False, 0.0),         # more than one 32-token chunk
    (70, 48, 768, 128, False, 0.0),
    (1, 16, 28672, 128, False, 0.01),      # longest K of any configuration
    (1, 2560, 2560, 64, False, 0.0),       # the paper's other small shapes (Sec. III)
    (1, 3840, 2560, 64, False, 0.0),
    (4, 3200, 3200, 64, True, 0.0),
]


@pytest.mark.parametrize("M,N,K,group,ternary,frac", CASES)
def test_gemm_against_reference(gpu, oracle, M, N, K, group, ternary, frac):
    torch, b = gpu
    codes, s_w, bits, g = _problem(M * 31 + N + K, M, N, K, group, ternary, frac)
    a, s_a, y, P = _run_gpu(torch, b, codes, s_w, bits, g)
    a_ref, s_ref = oracle.quantize(bits)
    assert np.array_equal(a, a_ref) and np.array_equal(s_a.view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(P, oracle.partials(a_ref, codes, g)), "int32 per-group sums must be exact"
    ok, worst = _row_err_ok(y, oracle.gemm(a_ref, s_ref, codes, s_w, g))
    assert ok, f"worst error / bound = {worst}"


@pytest.mark.parametrize("chunks,tg", [(1, 1), (2, 2), (5, 2), (59, 1), (3, 1)])
@pytest.mark.parametrize("M,group", [(1, 64), (12, 64), (3, 128), (20, 0)])
def test_forced_chunking(gpu, oracle, chunks, tg, M, group, monkeypatch):
    """Every tile grouping and several split-K factors on a long contraction with
    a ragged last chunk and a ragged last tile group."""
    torch, b = gpu
    monkeypatch.setenv("W2A8_CHUNKS", str(chunks))
    monkeypatch.setenv("W2A8_TG", str(tg))
    N, K = 80, 14336 + 256 * 3
    codes, s_w, bits, g = _problem(99 + chunks, M, N, K, group)
    a, s_a, y, P = _run_gpu(torch, b, codes, s_w, bits, g)
    assert np.array_equal(P, oracle.partials(a, codes, g))
    ok, worst = _row_err_ok(y, oracle.gemm(a, s_a, codes, s_w, g))
    assert ok, f"worst error / bound = {worst}"


@pytest.mark.parametrize("switch", [("W2A8_CLUSTER", "0"), ("W2A8_MT", "1"), ("W2A8_MT", "3"),
                                    ("W2A8_RING", "8"), ("W2A8_MIN_WARPS", "100000")])
@pytest.mark.parametrize("M,N,K,group", [(20, 80, 14336 + 256 * 3, 64), (1, 4096, 4096, 64), (9, 1024, 4096, 128)])
def test_plan_switches(gpu, oracle, switch, M, N, K, group, monkeypatch):
    """The alternatives of the decode launch plan (split-K through the workspace instead of a
    cluster, slab widths, deeper landing slots, finer split-K) give the same exact sums."""
    torch, b = gpu
    monkeypatch.setenv(*switch)
    codes, s_w, bits, g = _problem(7 + M, M, N, K, group)
    a, s_a, y, P = _run_gpu(torch, b, codes, s_w, bits, g)
    assert np.array_equal(P, oracle.partials(a, codes, g))
    ok, worst = _row_err_ok(y, oracle.gemm(a, s_a, codes, s_w, g))
    assert ok, f"worst error / bound = {worst}"


def test_extreme_magnitudes_no_overflow(gpu, oracle):
    torch, b = gpu
    M, N, K = 2, 16, 28672
    codes = np.zeros((N, K), np.uint8)                       # value -2 everywhere
    codes[1::2] = 3                                          # value +1 on odd channels
    x = np.full((M, K), -3.0, np.float32)                    # quantises to -127
    x[1] = 3.0
    bits = synth.float_to_bf16_bits(x)
    s_w = np.ones((N, 1), np.float32)
    a, s_a, y, P = _run_gpu(torch, b, codes, s_w, bits, K)
    assert P[0, 0, 0] == 254 * K and P[1, 0, 0] == -254 * K and P[1, 1, 0] == 127 * K
    assert np.array_equal(P, oracle.partials(a, codes, K))
    ok, worst = _row_err_ok(y, oracle.gemm(a, s_a, codes, s_w, K))
    assert ok, worst
    for g in (64, 128, 256):                                 # largest sums inside one accumulator
        s_w = np.ones((N, K // g), np.float32)
        a, s_a, y, P = _run_gpu(torch, b, codes, s_w, bits, g)
        assert (P[0, 0] == 254 * g).all()
        assert np.array_equal(P, oracle.partials(a, codes, g))


def test_zero_token_row_and_zero_weights(gpu, oracle):
    torch, b = gpu
    M, N, K, g = 4, 32, 512, 64
    codes, s_w, bits, g = _problem(5, M, N, K, g)
    bits[2, :] = 0                                           # dead token
    codes[3, :] = 2                                          # channel of zeros
    a, s_a, y, P = _run_gpu(torch, b, codes, s_w, bits, g)
    assert not y[2].any() and not y[:, 3].any()
    ok, worst = _row_err_ok(y, oracle.gemm(a, s_a, codes, s_w, g))
    assert ok, worst


def test_second_device_after_first(gpu, oracle):
    """One process, two GPUs: function attributes, the SM count and the architecture check are
    kept per device, so the same shapes run on device 1 after device 0 (no peer access, no
    collectives).  Skipped where only one device is visible."""
    torch, b = gpu
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two visible devices")
    for M, N, K, g in [(1, 2048, 2048, 64), (16, 256, 4096, 64), (1, 256, 8192, 64), (256, 4096, 1024, 64)]:
        codes, s_w, bits, g = _problem(M + N, M, N, K, g)
        a_ref, s_ref = oracle.quantize(bits)
        y_ref = oracle.gemm(a_ref, s_ref, codes, s_w, g)
        for dev in (0, 1):
            with torch.cuda.device(dev):
                d = lambda x: torch.from_numpy(np.ascontiguousarray(x)).to(f"cuda:{dev}")
                packed = b.w2_pack(d(codes))
                a, s_a = b.a8_quantize(d(bits.view(np.int16)).view(torch.bfloat16))
                ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g), device=f"cuda:{dev}")
                y = b.w2a8_gemm(a, s_a, packed, d(s_w), g, ws)
                torch.cuda.synchronize()
                assert b.w2a8_workspace_status(ws) == 0
                ok, worst = _row_err_ok(y.cpu().numpy(), y_ref)
                assert ok, (dev, worst)


def test_status_word_read_back(gpu):
    """The device status word at the start of a workspace is what w2a8_workspace_status returns:
    the code a kernel leaves when one of its bounded waits gives up (-7) is written here from the
    host -- no kernel is made to time out -- and read back; a fresh workspace reads 0."""
    torch, b = gpu
    ws = b.new_workspace(4096)
    assert b.w2a8_workspace_status(ws) == 0
    ws[:4].copy_(torch.tensor([-7], dtype=torch.int32).view(torch.uint8))
    assert b.w2a8_workspace_status(ws) == -7
    assert "wait" in b.status_string(-7)
    b.w2a8_workspace_init(ws)
    assert b.w2a8_workspace_status(ws) == 0


@pytest.mark.parametrize("M,pinned", [(4, True), (4, False), (1, True), (40, True)])
def test_linear_host_end_to_end(gpu, oracle, M, pinned):
    """Host buffers in, host buffers out: page-locked buffers with few tokens are read and
    written by the kernels directly, everything else goes through staged copies."""
    torch, b = gpu
    N, K, g = 1024, 4096, 64
    codes, s_w, bits, g = _problem(77, M, N, K, g)
    packed = b.w2_pack(_dev(torch, codes))
    s_w_d = _dev(torch, s_w)
    x_host = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)
    y_host = torch.empty((M, N), dtype=torch.float32)
    if pinned:
        x_host, y_host = x_host.pin_memory(), y_host.pin_memory()
    ws = b.new_workspace(b.w2a8_linear_host_workspace_bytes(M, N, K, g))
    for _ in range(2):
        y_host.zero_()
        b.w2a8_linear_host(x_host, packed, s_w_d, g, y_host, ws)
        torch.cuda.synchronize()
        a_ref, s_ref = oracle.quantize(bits)
        ok, worst = _row_err_ok(y_host.numpy(), oracle.gemm(a_ref, s_ref, codes, s_w, g))
        assert ok, worst


@pytest.mark.parametrize("M,pinned", [(1, True), (4, True), (16, True), (4, False), (40, True)])
def test_linear_grouped_host_end_to_end(gpu, oracle, M, pinned):
    """q|k|v-like group with host buffers in and out: x crosses the bus once, every y lands in its
    host buffer; zero-copy for few tokens in page-locked buffers, staged copies otherwise."""
    torch, b = gpu
    K, Ns, g = 4096, [1024, 256, 256], 64
    mats = [synth.make_linear(300 + i, K, n, g) for i, n in enumerate(Ns)]
    bits = synth.activations_bf16(301, M, K)
    grp = b.Group([b.w2_pack(_dev(torch, c)) for c, _ in mats], [_dev(torch, s) for _, s in mats])
    x_host = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)
    ys = [torch.empty((M, n), dtype=torch.float32) for n in Ns]
    if pinned:
        x_host, ys = x_host.pin_memory(), [y.pin_memory() for y in ys]
    ws = b.new_workspace(b.w2a8_linear_grouped_host_workspace_bytes(Ns, M, K, g))
    a_ref, s_ref = oracle.quantize(bits)
    for _ in range(2):
        for y in ys:
            y.zero_()
        b.w2a8_linear_grouped_host(x_host, grp, g, ys, ws)
        torch.cuda.synchronize()
        for (codes, s_w), y in zip(mats, ys):
            ok, worst = _row_err_ok(y.numpy(), oracle.gemm(a_ref, s_ref, codes, s_w, g))
            assert ok, worst


def test_pdl_off_matches(gpu, oracle):
    # the same library with plain launches, in a child process (the switch is read once)
    import subprocess
    import sys
    code = (
        "import numpy as np, torch\n"
        "from paper_2508_06753_b200 import binding as b, synth\n"
        "import oracle\n"
        "codes, s_w = synth.make_linear(3, 2048, 256, 64)\n"
        "bits = synth.activations_bf16(3, 4, 2048)\n"
        "d = lambda x: torch.from_numpy(np.ascontiguousarray(x)).cuda()\n"
        "packed = b.w2_pack(d(codes)); a, s = b.a8_quantize(d(bits.view(np.int16)).view(torch.bfloat16))\n"
        "ws = b.new_workspace(b.w2a8_workspace_bytes(4, 256, 2048, 64))\n"
        "y = b.w2a8_gemm(a, s, packed, d(s_w), 64, ws).cpu().numpy()\n"
        "a_ref, s_ref = oracle.quantize(bits)\n"
        "ref = oracle.gemm(a_ref, s_ref, codes, s_w, 64)\n"
        "assert np.abs(y - ref).max() <= 1e-4 * np.abs(ref).max(), 'mismatch'\n"
        "print('ok')\n")
    env = dict(os.environ, W2A8_PDL="0")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, "-c", code], env=env, cwd=root, capture_output=True,
                         text=True, timeout=600)
    assert out.returncode == 0 and "ok" in out.stdout, out.stderr[-2000:]


# ---------------------------------------------- full-size shapes, sampled channels
FULL = [
    (1, "8b"), (4, "8b"), (16, "8b"), (1, "8b-ternary"), (8, "8b-ternary"), (1, "70b"), (8, "70b"), (32, "70b"),
]


@pytest.mark.parametrize("M,which", FULL)
def test_full_size_layers_sampled(gpu, oracle, M, which):
    """Every linear of a layer at full size, in the launch configuration the
    benchmark times; the reference is evaluated on 96 sampled output channels
    (channels are independent) plus the first and last 16."""
    torch, b = gpu
    cfg = {"8b": synth.CONFIGS[1], "8b-ternary": synth.CONFIGS[2], "70b": synth.CONFIGS[3]}[which]
    rng = np.random.default_rng(17)
    for idx, (name, K, N) in enumerate(cfg["shapes"]):
        if name in ("v", "up", "o"):                       # same shapes as k, gate, q
            continue
        g = synth.config_group(cfg, K)
        codes, s_w = synth.make_linear(synth.shape_seed(cfg, idx), K, N, g, cfg["ternary"])
        bits = synth.activations_bf16(synth.shape_seed(cfg, idx), M, K, cfg["outlier_frac"])
        packed = b.w2_pack(_dev(torch, codes))
        a, s_a = b.a8_quantize(_bf16_dev(torch, bits))
        ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g))
        y = b.w2a8_gemm(a, s_a, packed, _dev(torch, s_w), g, ws).cpu().numpy()
        P = b.w2a8_gemm_partials(a, packed, g, ws).cpu().numpy()
        sel = np.unique(np.concatenate([np.arange(16), np.arange(N - 16, N),
                                        rng.choice(N, size=96, replace=False)]))
        a_ref, s_ref = oracle.quantize(bits)
        assert np.array_equal(a.cpu().numpy(), a_ref)
        assert np.array_equal(P[:, sel], oracle.partials(a_ref, codes[sel], g)), name
        y_ref = oracle.gemm(a_ref, s_ref, codes[sel], s_w[sel], g)
        err = np.abs(y[:, sel].astype(np.float64) - y_ref).max(axis=1)
        assert (err <= TOL * np.abs(y_ref).max(axis=1)).all(), name
        # properties that hold for every channel: finite, and bounded by sum |s_w| * 254 g * s_a
        assert np.isfinite(y).all()
        bound = (np.abs(s_w).sum(axis=1) * 254.0 * g)[None, :] * s_ref[:, None]
        assert (np.abs(y) <= bound * (1 + 1e-5)).all()
        del packed, codes
