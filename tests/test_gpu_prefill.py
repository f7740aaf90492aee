"""GPU parity of the tensor-core (tcgen05) prefill path against the CPU
reference: int32 per-group sums bit-exact, fp32 outputs within 1e-4 * max|row|."""
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


@pytest.fixture(autouse=True)
def force_tensor_core_kernel(monkeypatch):
    """Small shapes would be given to the streaming kernel by the dispatch rule; these tests are
    about the tensor-core kernel, so it is taken whenever it supports the shape."""
    monkeypatch.setenv("W2A8_PREFILL", "2")


def _dev(torch, arr):
    return torch.from_numpy(np.ascontiguousarray(arr)).cuda()


CASES = [
    # M, N, K, group (0 = K)
    (128, 128, 256, 64),        # one tile, one stage
    (64, 128, 512, 64),         # half-empty token tile
    (300, 256, 1024, 64),       # ragged token tile, several stages (ring wraps)
    (256, 384, 2048, 128),
    (130, 128, 1024, 256),
    (200, 256, 1536, 512),      # a scale group spans two stages
    (257, 128, 1280, 0),        # one scale per channel
    (512, 512, 4096, 64),       # configuration-4-like slice: K of gate/up
    (640, 4096, 512, 64),       # 160 tiles: more than one tile per persistent CTA
    (384, 6400, 768, 256),      # 150 tiles, three groups per tile (the last hand-off unit has one group)
    (200, 19200, 256, 128),     # 300 tiles of a single stage each, ragged token tiles
]


@pytest.mark.parametrize("kind", [8, 16])
@pytest.mark.parametrize("M,N,K,group", CASES)
def test_prefill_against_reference(gpu, oracle, monkeypatch, M, N, K, group, kind):
    """Both tensor-core kernels behind w2a8_gemm: the int8 one (kind::i8, int32 accumulators) and
    the 16-bit one (kind::f16 on a bf16 copy of the int8 activations, fp32 accumulators that hold the
    same integers): exact int32 group sums from either."""
    torch, b = gpu
    monkeypatch.setenv("W2A8_TC_KIND", str(kind))
    g = K if group == 0 else group
    assert b.w2a8_kernel_for(M, N, K, g) == "tensor_core"
    assert b.w2a8_tensor_core_kind(M, N, K, g) == kind
    codes, s_w = synth.make_linear(7 * M + N + K, K, N, g)
    bits = synth.activations_bf16(M + K, M, K)
    packed = b.w2_pack(_dev(torch, codes))
    a, s_a = b.a8_quantize(_dev(torch, bits.view(np.int16)).view(torch.bfloat16))
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g))
    y = b.w2a8_gemm(a, s_a, packed, _dev(torch, s_w), g, ws)
    y2 = b.w2a8_gemm(a, s_a, packed, _dev(torch, s_w), g, ws)
    P = b.w2a8_gemm_partials(a, packed, g, ws)
    torch.cuda.synchronize()
    assert b.w2a8_workspace_status(ws) == 0
    assert torch.equal(y, y2)
    a_ref, s_ref = oracle.quantize(bits)
    assert np.array_equal(a.cpu().numpy(), a_ref)
    assert np.array_equal(P.cpu().numpy(), oracle.partials(a_ref, codes, g))
    y_ref = oracle.gemm(a_ref, s_ref, codes, s_w, g)
    err = np.abs(y.cpu().numpy().astype(np.float64) - y_ref).max(axis=1)
    assert (err <= TOL * np.abs(y_ref).max(axis=1)).all(), float((err / np.abs(y_ref).max(axis=1)).max())


SPLIT_CASES = [
    # M, N, K, group, forced K splits
    (128, 256, 2048, 64, 2),
    (128, 256, 2048, 64, 4),        # two 256-k blocks per split: the smallest allowed
    (200, 128, 4096, 128, 8),       # ragged token tile
    (130, 256, 2048, 256, 4),       # a split is two groups of one block each
    (300, 384, 3072, 512, 2),       # groups of two blocks, three per split; ragged tokens
    (64, 4096, 1024, 64, 2),        # 64 work items
]


@pytest.mark.parametrize("h16", [False, True])
@pytest.mark.parametrize("M,N,K,group,split", SPLIT_CASES)
def test_k_split(gpu, oracle, monkeypatch, M, N, K, group, split, h16):
    """K split of the int8 tensor-core kernel: partial outputs per split in the workspace, added in
    split order by the second kernel.  Same result on a repeat (fixed order), within the tolerance of
    the reference, and within a few units in the last place of the unsplit kernel's result."""
    torch, b = gpu
    monkeypatch.setenv("W2A8_PF_KSPLIT", str(split))
    assert b.w2a8_kernel_for(M, N, K, group) == "tensor_core"
    assert b.w2a8_tensor_core_ksplit(M, N, K, group) == split
    codes, s_w = synth.make_linear(3 * M + N + K + split, K, N, group)
    bits = synth.activations_bf16(M + K + split, M, K)
    packed = b.w2_pack(_dev(torch, codes))
    a, s_a = b.a8_quantize(_dev(torch, bits.view(np.int16)).view(torch.bfloat16))
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, group))
    a_ref, s_ref = oracle.quantize(bits)
    if h16:
        s_h = s_w.astype(np.float16)
        run = lambda w: b.w2a8_gemm_h16(a, s_a, packed, _dev(torch, s_h), group, w)
        y_ref = oracle.gemm(a_ref, s_ref, codes, s_h.astype(np.float32), group)
    else:
        run = lambda w: b.w2a8_gemm(a, s_a, packed, _dev(torch, s_w), group, w)
        y_ref = oracle.gemm(a_ref, s_ref, codes, s_w, group)
    y = run(ws)
    y2 = run(ws)
    torch.cuda.synchronize()
    assert b.w2a8_workspace_status(ws) == 0
    assert torch.equal(y, y2)
    rowmax = np.abs(y_ref).max(axis=1)
    err = np.abs(y.cpu().numpy().astype(np.float64) - y_ref).max(axis=1)
    assert (err <= TOL * rowmax).all(), float((err / rowmax).max())
    if h16:     # bf16 result: the same fp32 sums, rounded once by the summing kernel
        y16 = b.w2a8_gemm_h16(a, s_a, packed, _dev(torch, s_h), group, ws, out_dtype=torch.bfloat16)
        assert torch.equal(y16, y.to(torch.bfloat16))
    monkeypatch.setenv("W2A8_PF_KSPLIT", "1")
    assert b.w2a8_tensor_core_ksplit(M, N, K, group) == 1
    y1 = run(b.new_workspace(b.w2a8_workspace_bytes(M, N, K, group)))
    torch.cuda.synchronize()
    diff = (y.double() - y1.double()).abs().max(dim=1).values.cpu().numpy()
    assert (diff <= 4e-6 * rowmax).all(), float((diff / rowmax).max())      # only the order of fp32 additions differs


def test_k_split_default_rule(gpu, oracle, monkeypatch):
    """Default dispatch on a few-tile shape of the benchmark layer (`down` at 128 tokens: 32 output
    tiles on 148 SMs): tensor-core kernel with K split four ways; sampled rows against the reference."""
    torch, b = gpu
    monkeypatch.delenv("W2A8_PREFILL", raising=False)
    monkeypatch.delenv("W2A8_PF_KSPLIT", raising=False)
    M, N, K, g = 128, 4096, 14336, 64
    assert b.w2a8_kernel_for(M, N, K, g) == "tensor_core"
    assert b.w2a8_tensor_core_ksplit(M, N, K, g) == 4
    assert b.w2a8_tensor_core_channels(M, N, K, g) == N
    codes, s_w = synth.make_linear(4242, K, N, g)
    bits = synth.activations_bf16(4243, M, K)
    packed = b.w2_pack(_dev(torch, codes))
    a, s_a = b.a8_quantize(_dev(torch, bits.view(np.int16)).view(torch.bfloat16))
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g))
    y = b.w2a8_gemm(a, s_a, packed, _dev(torch, s_w), g, ws).cpu().numpy()
    assert b.w2a8_workspace_status(ws) == 0
    rows = [0, 1, 63, 64, 127]
    a_ref, s_ref = oracle.quantize(bits[rows])
    assert np.array_equal(a.cpu().numpy()[rows], a_ref)
    y_ref = oracle.gemm(a_ref, s_ref, codes, s_w, g)
    err = np.abs(y[rows].astype(np.float64) - y_ref).max(axis=1)
    assert (err <= TOL * np.abs(y_ref).max(axis=1)).all()


WIDE_CASES = [
    # M, N, K: one scale per channel, 256-token tiles
    (257, 128, 1280),       # second token tile holds one token
    (130, 128, 512),        # ragged single tile, two 256-k blocks
    (512, 256, 2048),
    (1000, 384, 768),       # ragged last tile, odd number of blocks
    (300, 19200, 256),      # 300 tiles on 148 CTAs: both accumulator buffers re-used, one block per tile
]


@pytest.mark.parametrize("h16", [False, True])
@pytest.mark.parametrize("M,N,K", WIDE_CASES)
def test_wide_tiles_one_scale_per_channel(gpu, oracle, monkeypatch, M, N, K, h16):
    """The 256-token-tile kernel (group = K): against the reference, and bit for bit against the
    128-token kernel (same sums, same order of the float operations)."""
    torch, b = gpu
    g = K
    codes, s_w = synth.make_linear(5 * M + N + K, K, N, g)
    bits = synth.activations_bf16(M + 3 * K, M, K)
    packed = b.w2_pack(_dev(torch, codes))
    a, s_a = b.a8_quantize(_dev(torch, bits.view(np.int16)).view(torch.bfloat16))
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g))
    a_ref, s_ref = oracle.quantize(bits)
    if h16:
        s_h = s_w.astype(np.float16)
        run = lambda **kw: b.w2a8_gemm_h16(a, s_a, packed, _dev(torch, s_h), g, ws, **kw)
        y_ref = oracle.gemm(a_ref, s_ref, codes, s_h.astype(np.float32), g)
    else:
        run = lambda **kw: b.w2a8_gemm(a, s_a, packed, _dev(torch, s_w), g, ws)
        y_ref = oracle.gemm(a_ref, s_ref, codes, s_w, g)
    monkeypatch.setenv("W2A8_PF_WIDE", "2")
    assert b.w2a8_tensor_core_tile_tokens(M, N, K, g) == 256
    y = run()
    y2 = run()
    torch.cuda.synchronize()
    assert b.w2a8_workspace_status(ws) == 0
    assert torch.equal(y, y2)
    rowmax = np.abs(y_ref).max(axis=1)
    err = np.abs(y.cpu().numpy().astype(np.float64) - y_ref).max(axis=1)
    assert (err <= TOL * rowmax).all(), float((err / rowmax).max())
    if h16:
        y16 = run(out_dtype=torch.bfloat16)
        assert torch.equal(y16, y.to(torch.bfloat16))
    monkeypatch.setenv("W2A8_PF_WIDE", "0")
    monkeypatch.setenv("W2A8_PF_KSPLIT", "1")
    assert b.w2a8_tensor_core_tile_tokens(M, N, K, g) == 128
    y128 = run()
    torch.cuda.synchronize()
    assert torch.equal(y, y128)


def test_prefill_matches_streaming_path(gpu, monkeypatch):
    """The tensor-core path and the streaming (decode) path agree on the same problem."""
    torch, b = gpu
    M, N, K, g = 192, 256, 1024, 64
    codes, s_w = synth.make_linear(5, K, N, g)
    bits = synth.activations_bf16(5, M, K)
    packed = b.w2_pack(_dev(torch, codes))
    a, s_a = b.a8_quantize(_dev(torch, bits.view(np.int16)).view(torch.bfloat16))
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g))
    assert b.w2a8_kernel_for(M, N, K, g) == "tensor_core"
    y_tc = b.w2a8_gemm(a, s_a, packed, _dev(torch, s_w), g, ws).cpu().numpy()
    monkeypatch.setenv("W2A8_PREFILL", "0")
    assert b.w2a8_kernel_for(M, N, K, g) == "streaming"
    y_st = b.w2a8_gemm(a, s_a, packed, _dev(torch, s_w), g, ws).cpu().numpy()
    assert np.abs(y_tc - y_st).max() <= TOL * np.abs(y_st).max()


def _sample_rows(M, seed, count=128):
    """First and last row of the first, a middle and the last 128-token tile, plus seeded rows."""
    mid = (M // 128 // 2) * 128
    fixed = [0, 127, mid, mid + 127, M - 128, M - 1]
    extra = [int(r) for r in np.random.default_rng(seed).choice(M, size=count, replace=False)]
    return sorted(set(fixed + extra))


FULL_SIZE = [(M, K, N, d) for M in (512, 2048, 8192) for K, N in ((4096, 14336), (14336, 4096))
             for d in (("as_benchmarked", "tensor_core_only") if M == 2048 else ("as_benchmarked",))]


@pytest.mark.parametrize("M,K,N,dispatch", FULL_SIZE)
def test_prefill_full_size_sampled_rows(gpu, oracle, M, K, N, dispatch, monkeypatch):
    """Prefill configuration at full size (group 64) for every token count the benchmark times:
    every channel of at least 128 sampled token rows -- first and last row of the first, a middle
    and the last token tile, plus seeded ones -- against the reference, and the exact int32 sums
    of the first and the last 128-channel tile for the same rows.  "as_benchmarked" is the default
    dispatch, in which the last 128 channels of 4096x14336 are computed by the streaming kernel."""
    torch, b = gpu
    g = 64
    if dispatch == "as_benchmarked":
        monkeypatch.delenv("W2A8_PREFILL", raising=False)
        assert b.w2a8_kernel_for(M, N, K, g) == "tensor_core"
        if M <= 2048:
            assert b.w2a8_tensor_core_channels(M, N, K, g) == (111 * 128 if N == 14336 else N)
    codes, s_w = synth.make_linear(4000 + K, K, N, g)
    bits = synth.activations_bf16(4000 + N + M, M, K)
    packed = b.w2_pack(_dev(torch, codes))
    a, s_a = b.a8_quantize(_dev(torch, bits.view(np.int16)).view(torch.bfloat16))
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g))
    y = b.w2a8_gemm(a, s_a, packed, _dev(torch, s_w), g, ws)
    torch.cuda.synchronize()
    assert b.w2a8_workspace_status(ws) == 0
    rows = _sample_rows(M, K + M)
    assert len(rows) >= 128
    a_ref, s_ref = oracle.quantize(bits[rows])
    idx = torch.tensor(rows, device="cuda")
    assert np.array_equal(a[idx].cpu().numpy(), a_ref)
    y_ref = oracle.gemm(a_ref, s_ref, codes, s_w, g)
    got = y[idx].cpu().numpy().astype(np.float64)
    err = np.abs(got - y_ref).max(axis=1)
    assert (err <= TOL * np.abs(y_ref).max(axis=1)).all(), float((err / np.abs(y_ref).max(axis=1)).max())
    assert bool(torch.isfinite(y).all())
    # exact int32 sums: all tokens against the first and the last channel tile (channels are
    # independent, so their packed rows form a problem of their own), compared on the sampled rows
    monkeypatch.setenv("W2A8_PREFILL", "2")
    sel = np.concatenate([np.arange(128), np.arange(N - 128, N)])
    sub = packed[torch.from_numpy(sel).cuda()].contiguous()
    ws2 = b.new_workspace(b.w2a8_workspace_bytes(M, 256, K, g))
    assert b.w2a8_kernel_for(M, 256, K, g) == "tensor_core"
    P = b.w2a8_gemm_partials(a, sub, g, ws2)
    torch.cuda.synchronize()
    assert b.w2a8_workspace_status(ws2) == 0
    assert np.array_equal(P[idx].cpu().numpy(), oracle.partials(a_ref, codes[sel], g))


@pytest.mark.parametrize("M", [2048, 1100])
def test_wide_tiles_full_size_default_rule(gpu, oracle, monkeypatch, M):
    """One scale per channel on the gate/up shape at the default dispatch: the 256-token-tile kernel on
    the first 111 channel tiles and the streaming kernel on the last 128 channels (M = 2048), or a ragged
    token count (M = 1100); sampled token rows of every channel against the reference."""
    torch, b = gpu
    for name in ("W2A8_PREFILL", "W2A8_PF_WIDE", "W2A8_PF_KSPLIT"):
        monkeypatch.delenv(name, raising=False)
    K, N = 4096, 14336
    g = K
    assert b.w2a8_kernel_for(M, N, K, g) == "tensor_core"
    assert b.w2a8_tensor_core_tile_tokens(M, N, K, g) == 256
    if M == 2048:
        assert b.w2a8_tensor_core_channels(M, N, K, g) == 111 * 128
    codes, s_w = synth.make_linear(5100 + M, K, N, g)
    bits = synth.activations_bf16(5200 + M, M, K)
    packed = b.w2_pack(_dev(torch, codes))
    a, s_a = b.a8_quantize(_dev(torch, bits.view(np.int16)).view(torch.bfloat16))
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g))
    y = b.w2a8_gemm(a, s_a, packed, _dev(torch, s_w), g, ws)
    torch.cuda.synchronize()
    assert b.w2a8_workspace_status(ws) == 0
    assert bool(torch.isfinite(y).all())
    rows = sorted(set([0, 127, 128, 255, 256, 1023, 1024, M - 257, M - 256, M - 1] +
                      [int(r) for r in np.random.default_rng(M).choice(M, size=54, replace=False)]))
    a_ref, s_ref = oracle.quantize(bits[rows])
    idx = torch.tensor(rows, device="cuda")
    assert np.array_equal(a[idx].cpu().numpy(), a_ref)
    y_ref = oracle.gemm(a_ref, s_ref, codes, s_w, g)
    err = np.abs(y[idx].cpu().numpy().astype(np.float64) - y_ref).max(axis=1)
    assert (err <= TOL * np.abs(y_ref).max(axis=1)).all(), float((err / np.abs(y_ref).max(axis=1)).max())


def test_dispatch_rule(gpu, oracle, monkeypatch):
    """Default dispatch: few output tiles go to the streaming kernel even with many tokens; both
    choices give the reference result on a shape next to the boundary."""
    torch, b = gpu
    monkeypatch.delenv("W2A8_PREFILL", raising=False)
    assert b.w2a8_kernel_for(2048, 14336, 4096, 64) == "tensor_core"
    assert b.w2a8_kernel_for(512, 4096, 14336, 64) == "tensor_core"
    assert b.w2a8_kernel_for(128, 4096, 14336, 64) == "tensor_core"     # 32 tiles on 148 SMs: K split four ways
    assert b.w2a8_kernel_for(64, 14336, 4096, 64) == "streaming"
    assert b.w2a8_kernel_for(64, 4096, 4096, 64) == "streaming"
    assert b.w2a8_kernel_for(256, 4096, 4096, 64) == "tensor_core"
    assert b.w2a8_kernel_for(63, 14336, 4096, 64) == "streaming"        # below the token threshold
    assert b.w2a8_kernel_for(512, 1040, 4096, 64) == "streaming"        # N not a multiple of 128
    M, N, K, g = 224, 4096, 512, 64                                     # M * N just below the boundary
    assert b.w2a8_kernel_for(M, N, K, g) == "streaming"
    codes, s_w = synth.make_linear(11, K, N, g)
    bits = synth.activations_bf16(11, M, K)
    packed = b.w2_pack(_dev(torch, codes))
    a, s_a = b.a8_quantize(_dev(torch, bits.view(np.int16)).view(torch.bfloat16))
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g))
    a_ref, s_ref = oracle.quantize(bits)
    y_ref = oracle.gemm(a_ref, s_ref, codes, s_w, g)
    for mode in ("1", "2"):
        monkeypatch.setenv("W2A8_PREFILL", mode)
        y = b.w2a8_gemm(a, s_a, packed, _dev(torch, s_w), g, ws).cpu().numpy()
        assert b.w2a8_workspace_status(ws) == 0
        err = np.abs(y.astype(np.float64) - y_ref).max(axis=1)
        assert (err <= TOL * np.abs(y_ref).max(axis=1)).all(), mode


@pytest.mark.parametrize("h16", [False, True])
def test_channel_split_between_the_two_kernels(gpu, oracle, monkeypatch, h16):
    """150 channel tiles on 148 SMs: the tensor-core kernel takes 148 of them, the streaming kernel
    the last 256 channels, both writing their own columns of y."""
    torch, b = gpu
    monkeypatch.delenv("W2A8_PREFILL", raising=False)
    M, N, K, g = 128, 19200, 1024, 64
    assert b.w2a8_kernel_for(M, N, K, g) == "tensor_core"
    assert b.w2a8_tensor_core_channels(M, N, K, g) == 148 * 128
    assert b.w2a8_tensor_core_channels(2048, 14336, 4096, 64) == 111 * 128      # 1776 tiles = 12 rounds
    assert b.w2a8_tensor_core_channels(512, 14336, 4096, 64) == 111 * 128       # 444 tiles = 3 rounds
    assert b.w2a8_tensor_core_channels(512, 4096, 14336, 64) == 4096            # one round: nothing to gain
    assert b.w2a8_tensor_core_channels(16, 4096, 4096, 64) == 0
    codes = synth.weight_codes(3, N, K)
    bits = synth.activations_bf16(3, M, K)
    packed = b.w2_pack(_dev(torch, codes))
    a, s_a = b.a8_quantize(_dev(torch, bits.view(np.int16)).view(torch.bfloat16))
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g))
    a_ref, s_ref = oracle.quantize(bits)
    if h16:
        s_h = synth.weight_scales_h(3, N, K // g)
        y = b.w2a8_gemm_h16(a, s_a, packed, _dev(torch, s_h.view(np.int16)).view(torch.float16), g, ws,
                            out_dtype=torch.bfloat16)
        y_ref, _ = oracle.gemm_h(a_ref, s_ref, codes, s_h, g)
        tol = 2.0 ** -8 + TOL
        y = y.float()
    else:
        s_w = synth.weight_scales(3, N, K // g)
        y = b.w2a8_gemm(a, s_a, packed, _dev(torch, s_w), g, ws)
        y_ref = oracle.gemm(a_ref, s_ref, codes, s_w, g)
        tol = TOL
    torch.cuda.synchronize()
    assert b.w2a8_workspace_status(ws) == 0
    err = np.abs(y.cpu().numpy().astype(np.float64) - y_ref).max(axis=1)
    assert (err <= tol * np.abs(y_ref).max(axis=1)).all()
    # the same problem with the split switched off gives the same bits in the tensor-core part
    # and values within tolerance in the rest
    monkeypatch.setenv("W2A8_PF_SPLIT", "0")
    assert b.w2a8_tensor_core_channels(M, N, K, g) == N
    if not h16:
        y_all = b.w2a8_gemm(a, s_a, packed, _dev(torch, s_w), g, ws)
        torch.cuda.synchronize()
        assert torch.equal(y_all[:, :148 * 128], y[:, :148 * 128])
        assert (y_all[:, 148 * 128:] - y[:, 148 * 128:]).abs().max() <= TOL * y.abs().max()
