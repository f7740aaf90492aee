"""GPU parity of the 16-bit-activation entry (bf16 activations, no quantiser) against the CPU
reference: within 1e-4 * max|row| on random inputs, and bit-exact where every fp32 sum is exact
(integer-valued activations, unit scales)."""
import numpy as np
import pytest

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


CASES = [
    # M, N, K, group (0 = K), ternary, outlier fraction
    (1, 16, 64, 64, False, 0.0),            # smallest legal problem
    (1, 2048, 2048, 64, False, 0.0),
    (3, 48, 448, 64, False, 0.0),           # ragged K
    (1, 1600, 1600, 64, False, 0.0),
    (5, 32, 1600, 0, True, 0.0),            # one scale per channel, ragged K
    (4, 1040, 4096, 64, False, 0.01),
    (8, 256, 4096, 128, True, 0.01),
    (9, 256, 2048, 128, False, 0.0),        # two 8-token slabs
    (16, 512, 4096, 64, False, 0.0),
    (17, 128, 1024, 256, False, 0.0),
    (32, 256, 8192, 128, False, 0.01),
    (1, 256, 8192, 64, True, 0.0),          # split-K inside a cluster
    (1, 16, 28672, 128, False, 0.01),       # longest K of any configuration
    (70, 48, 768, 128, False, 0.0),         # many tokens, a shape the tensor-core kernel does not tile
    (96, 256, 1024, 64, False, 0.0),        # too few output tiles for the tensor-core kernel to pay
]


@pytest.mark.parametrize("M,N,K,group,ternary,frac", CASES)
def test_a16_against_reference(gpu, oracle, M, N, K, group, ternary, frac):
    torch, b = gpu
    g = K if group == 0 else group
    seed = M * 41 + N + K
    codes, s_w = synth.make_linear(seed, K, N, g, ternary)
    bits = synth.activations_bf16(seed, M, K, frac)
    packed = b.w2_pack(_dev(torch, codes))
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g))
    x = _bf16_dev(torch, bits)
    y = b.w2a16_gemm(x, packed, _dev(torch, s_w), g, ws)
    y2 = b.w2a16_gemm(x, packed, _dev(torch, s_w), g, ws)
    torch.cuda.synchronize()
    assert b.w2a8_workspace_status(ws) == 0
    assert torch.equal(y, y2), "repeated calls must be bitwise equal"
    ref = oracle.gemm_a16(bits, codes, s_w, g)
    err = np.abs(y.cpu().numpy().astype(np.float64) - ref.astype(np.float64)).max(axis=1)
    bound = TOL * np.abs(ref).max(axis=1)
    assert (err <= bound).all(), float((err / np.maximum(bound, 1e-30)).max())


@pytest.mark.parametrize("M,N,K,group", [(1, 64, 1024, 64), (7, 48, 1600, 64), (16, 32, 2048, 128), (12, 80, 15104, 0)])
def test_a16_exact_on_integers(gpu, M, N, K, group):
    """Integer activations |x| <= 127 and unit scales: every product and every partial sum is an
    integer below 2^24, so fp32 summation in any order is exact and the result must equal the
    integer matrix product bit for bit -- a wrong code, lane or k pairing cannot hide in a tolerance."""
    torch, b = gpu
    g = K if group == 0 else group
    rng = np.random.default_rng(M + N + K)
    xi = rng.integers(-127, 128, size=(M, K))
    codes = rng.integers(0, 4, size=(N, K), dtype=np.uint8)
    packed = b.w2_pack(_dev(torch, codes))
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g))
    x = _dev(torch, xi.astype(np.float32)).to(torch.bfloat16)
    y = b.w2a16_gemm(x, packed, torch.ones((N, K // g), dtype=torch.float32, device="cuda"), g, ws)
    torch.cuda.synchronize()
    want = xi @ (codes.astype(np.int64) - 2).T
    assert np.abs(want).max() < 2 ** 24
    assert np.array_equal(y.cpu().numpy().astype(np.int64), want)


@pytest.mark.parametrize("chunks", [2, 5, 59])
def test_a16_forced_chunking(gpu, oracle, chunks, monkeypatch):
    torch, b = gpu
    monkeypatch.setenv("W2A8_CHUNKS", str(chunks))
    M, N, K, g = 12, 80, 14336 + 256 * 3, 64
    codes, s_w = synth.make_linear(chunks, K, N, g)
    bits = synth.activations_bf16(chunks, M, K)
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g))
    y = b.w2a16_gemm(_bf16_dev(torch, bits), b.w2_pack(_dev(torch, codes)), _dev(torch, s_w), g, ws)
    torch.cuda.synchronize()
    assert b.w2a8_workspace_status(ws) == 0
    ref = oracle.gemm_a16(bits, codes, s_w, g)
    err = np.abs(y.cpu().numpy().astype(np.float64) - ref).max(axis=1)
    assert (err <= TOL * np.abs(ref).max(axis=1)).all()


@pytest.mark.parametrize("M", [1, 16])
def test_a16_full_size_gate_sampled(gpu, oracle, M):
    torch, b = gpu
    K, N, g = 4096, 14336, 64
    codes, s_w = synth.make_linear(77 + M, K, N, g)
    bits = synth.activations_bf16(77 + M, M, K, 0.01)
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g))
    y = b.w2a16_gemm(_bf16_dev(torch, bits), b.w2_pack(_dev(torch, codes)), _dev(torch, s_w), g, ws).cpu().numpy()
    rng = np.random.default_rng(29)
    sel = np.unique(np.concatenate([np.arange(16), np.arange(N - 16, N), rng.choice(N, size=96, replace=False)]))
    ref = oracle.gemm_a16(bits, codes[sel], s_w[sel], g)
    err = np.abs(y[:, sel].astype(np.float64) - ref).max(axis=1)
    assert (err <= TOL * np.abs(ref).max(axis=1)).all()
    assert np.isfinite(y).all()


TC_CASES = [
    # M, N, K, group (0 = K): shapes of the tensor-core kernel's own parity list
    (128, 128, 256, 64), (64, 128, 512, 64), (300, 256, 1024, 64), (256, 384, 2048, 128), (130, 128, 1024, 256),
    (200, 256, 1536, 512), (257, 128, 1280, 0), (640, 4096, 512, 64), (200, 19200, 256, 128),
]


@pytest.mark.parametrize("M,N,K,group", TC_CASES)
def test_a16_tensor_core_kernel(gpu, oracle, monkeypatch, M, N, K, group):
    """Many tokens: the 16-bit tensor-core kernel (tcgen05 kind::f16, bf16 operands, fp32 accumulators
    in tensor memory), forced for small shapes the dispatch rule would stream."""
    torch, b = gpu
    monkeypatch.setenv("W2A8_PREFILL", "2")
    g = K if group == 0 else group
    assert b.w2a8_kernel_for(M, N, K, g) == "tensor_core"
    codes, s_w = synth.make_linear(5 * M + N + K, K, N, g)
    bits = synth.activations_bf16(M + K, M, K, 0.01)
    packed = b.w2_pack(_dev(torch, codes))
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g))
    x = _bf16_dev(torch, bits)
    y = b.w2a16_gemm(x, packed, _dev(torch, s_w), g, ws)
    y2 = b.w2a16_gemm(x, packed, _dev(torch, s_w), g, ws)
    torch.cuda.synchronize()
    assert b.w2a8_workspace_status(ws) == 0
    assert torch.equal(y, y2)
    ref = oracle.gemm_a16(bits, codes, s_w, g)
    err = np.abs(y.cpu().numpy().astype(np.float64) - ref.astype(np.float64)).max(axis=1)
    assert (err <= TOL * np.abs(ref).max(axis=1)).all(), float((err / (TOL * np.abs(ref).max(axis=1))).max())
    # and the streaming kernel on the same problem agrees within the same tolerance
    monkeypatch.setenv("W2A8_PREFILL", "0")
    y_st = b.w2a16_gemm(x, packed, _dev(torch, s_w), g, ws)
    assert (y - y_st).abs().max() <= 2 * TOL * y.abs().max()


@pytest.mark.parametrize("M,N,K,group", [(128, 128, 1024, 64), (192, 256, 2048, 128), (96, 128, 15104 - 256 * 3 + 256, 0)])
def test_a16_tensor_core_exact_on_integers(gpu, monkeypatch, M, N, K, group):
    """Integer activations and unit scales through the tensor-core kernel: the integer matrix
    product, bit for bit."""
    torch, b = gpu
    monkeypatch.setenv("W2A8_PREFILL", "2")
    g = K if group == 0 else group
    rng = np.random.default_rng(M + N + K)
    xi = rng.integers(-127, 128, size=(M, K))
    codes = rng.integers(0, 4, size=(N, K), dtype=np.uint8)
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g))
    x = _dev(torch, xi.astype(np.float32)).to(torch.bfloat16)
    y = b.w2a16_gemm(x, b.w2_pack(_dev(torch, codes)), torch.ones((N, K // g), dtype=torch.float32, device="cuda"),
                     g, ws)
    torch.cuda.synchronize()
    assert b.w2a8_workspace_status(ws) == 0
    want = xi @ (codes.astype(np.int64) - 2).T
    assert np.abs(want).max() < 2 ** 24
    assert np.array_equal(y.cpu().numpy().astype(np.int64), want)


def test_a16_full_size_prefill_sampled_rows(gpu, oracle):
    """The prefill configuration's gate matrix at M = 2048 through w2a16_gemm as dispatched by
    default (tensor-core kernel plus the streamed last channel tile), on sampled token rows."""
    torch, b = gpu
    M, K, N, g = 2048, 4096, 14336, 64
    assert b.w2a8_kernel_for(M, N, K, g) == "tensor_core"
    codes, s_w = synth.make_linear(4100, K, N, g)
    bits = synth.activations_bf16(4101, M, K)
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g))
    y = b.w2a16_gemm(_bf16_dev(torch, bits), b.w2_pack(_dev(torch, codes)), _dev(torch, s_w), g, ws)
    torch.cuda.synchronize()
    assert b.w2a8_workspace_status(ws) == 0
    rows = sorted(set([0, 127, 1024, 1151, M - 128, M - 1] + [int(r) for r in np.random.default_rng(3).integers(0, M, 26)]))
    ref = oracle.gemm_a16(bits[rows], codes, s_w, g)
    got = y[torch.tensor(rows, device="cuda")].cpu().numpy().astype(np.float64)
    err = np.abs(got - ref).max(axis=1)
    assert (err <= TOL * np.abs(ref).max(axis=1)).all()
    assert bool(torch.isfinite(y).all())


def test_a16_argument_errors(gpu):
    torch, b = gpu
    M, N, K, g = 2, 32, 256, 64
    x = torch.zeros((M, K + 8), dtype=torch.bfloat16, device="cuda")
    packed = torch.zeros((N, K // 16), dtype=torch.int32, device="cuda")
    s_w = torch.ones((N, K // g), dtype=torch.float32, device="cuda")
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g))
    with pytest.raises(TypeError):
        b.w2a16_gemm(x[:, :K].float(), packed, s_w, g, ws)
    with pytest.raises(b.W2A8Error):                                   # activations not 16-byte aligned
        b.w2a16_gemm(x.view(-1)[1:1 + M * K].view(M, K), packed, s_w, g, ws)
    with pytest.raises(b.W2A8Error):                                   # workspace too small
        b.w2a16_gemm(x.view(-1)[:M * K].view(M, K), packed, s_w, g, ws[:8])
    torch.cuda.synchronize()
