"""GPU parity of the persistent streaming kernel and of the grouped / fused entry points
(w2a8_gemm_grouped, w2a8_linear_grouped) against the CPU reference and against the separate
calls: outputs within 1e-4 * max|row| of the reference; a grouped launch bit-equal to one
launch per matrix through the same kernel; the fused quantiser bit-equal to a8_quantize."""
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


def _within(y, y_ref):
    err = np.abs(y.astype(np.float64) - y_ref.astype(np.float64)).max(axis=1)
    return bool((err <= TOL * np.abs(y_ref).max(axis=1)).all())


def _mats(torch, b, seed, K, Ns, g, ternary=False):
    mats = []
    for i, N in enumerate(Ns):
        codes, s_w = synth.make_linear(seed + 10 * i, K, N, g, ternary)
        mats.append((codes, s_w, b.w2_pack(_dev(torch, codes)), _dev(torch, s_w)))
    return mats


# M, K, [N...], group (0 = K)
PERSISTENT = [
    (1, 4096, [4096, 1024, 1024], 64),        # q | k | v: one block per K-lane, activations in registers
    (4, 4096, [2048, 2048], 64),
    (8, 4096, [256, 48], 128),
    (1, 2048, [2048], 64),                    # 8 blocks: two tiles side by side
    (3, 1024, [80, 16, 32, 48], 64),          # 4 blocks: four tiles side by side, ragged tile count
    (2, 768, [64], 64),                       # 3 blocks: an idle K-lane
    (5, 2560, [160], 64),                     # 10 blocks on 8 K-lanes: runs of one and two blocks
    (1, 14336, [512, 256], 64),               # 56 blocks on 16 K-lanes: runs of three and four
    (7, 14336, [128], 0),                     # one scale per channel
    (6, 8192, [1024, 1024], 128),             # two blocks per K-lane
    (1, 28672, [64], 128),
    (16, 4096, [512, 512], 64),               # two slabs of 8 tokens per tile
    (12, 14336, [64, 80], 64),
    (32, 4096, [256], 128),                   # two tiles of 16 tokens per channel tile
    (20, 2048, [96, 32], 256),
    (9, 1024, [4096], 64),                    # more tiles than one round of partial sums holds
    (1, 1024, [16 * 1500], 64),               # many rounds at one token
]


@pytest.mark.parametrize("M,K,Ns,group", PERSISTENT)
@pytest.mark.parametrize("variant", ["default", "staged", "no_bcache"])
def test_persistent_kernel_grouped(gpu, oracle, monkeypatch, M, K, Ns, group, variant):
    """Every work split of the persistent kernel, forced for all shapes: against the reference,
    and the grouped launch against one launch per matrix (bit-equal)."""
    torch, b = gpu
    monkeypatch.setenv("W2A8_GEMV", "2")
    if variant == "staged":
        monkeypatch.setenv("W2A8_GEMV_ASMEM", "1")
    elif variant == "no_bcache":
        monkeypatch.setenv("W2A8_GEMV_BCACHE", "0")
        monkeypatch.setenv("W2A8_GEMV_ASMEM", "0")
    g = K if group == 0 else group
    mats = _mats(torch, b, 31 * M + K, K, Ns, g)
    bits = synth.activations_bf16(M + K, M, K)
    a, s_a = b.a8_quantize(_bf16_dev(torch, bits))
    ws = b.new_workspace(b.w2a8_grouped_workspace_bytes(Ns, M, K, g))
    assert b.w2a8_grouped_plan(Ns, M, K, g, b.FUSE_OFF) == {"one_launch": True, "fused": False}
    grp = b.Group([m[2] for m in mats], [m[3] for m in mats])
    guards = [Guarded(torch, (M, N), torch.float32, float("nan")) for N in Ns]
    ys = b.w2a8_gemm_grouped(a, s_a, grp, g, ws, y=[gd.view for gd in guards])
    ys2 = [t.clone() for t in ys]
    b.w2a8_gemm_grouped(a, s_a, grp, g, ws, y=[gd.view for gd in guards])
    torch.cuda.synchronize()
    a_ref, s_ref = oracle.quantize(bits)
    for (codes, s_w, packed, s_w_d), y, y2, gd in zip(mats, ys, ys2, guards):
        gd.check("y")
        assert torch.equal(y, y2), "repeated calls must be bitwise equal"
        assert _within(y.cpu().numpy(), oracle.gemm(a_ref, s_ref, codes, s_w, g))
        single = b.w2a8_gemm(a, s_a, packed, s_w_d, g, ws)
        assert torch.equal(single, y), "a grouped launch must give the bits of one launch per matrix"


FUSED = [(1, 4096, [4096, 1024, 1024], 64), (1, 14336, [4096], 64), (4, 4096, [512, 512], 64),
         (8, 1024, [256], 128), (3, 2560, [160, 32], 64), (2, 28672, [64], 0), (8, 8192, [128], 64)]


@pytest.mark.parametrize("M,K,Ns,group", FUSED)
def test_fused_quantiser_matches_separate_launches(gpu, oracle, M, K, Ns, group):
    """The knob of Sec. II-D: abs-max scales inside the GEMV launch or in a launch of their own.
    Both settings give the same bits in a, a_scale and every y, and the reference's values."""
    torch, b = gpu
    g = K if group == 0 else group
    mats = _mats(torch, b, 7 * M + K, K, Ns, g)
    bits = synth.activations_bf16(3 * M + K, M, K, 0.01)
    bits[M - 1, : K // 2] = 0                       # half a row of zeros: nothing special, but cheap to have
    x = _bf16_dev(torch, bits)
    ws = b.new_workspace(b.w2a8_grouped_workspace_bytes(Ns, M, K, g))
    assert b.w2a8_grouped_plan(Ns, M, K, g, b.FUSE_ON) == {"one_launch": True, "fused": True}
    assert b.w2a8_grouped_plan(Ns, M, K, g, b.FUSE_OFF)["fused"] is False
    out = {}
    for fuse in (b.FUSE_ON, b.FUSE_OFF):
        grp = b.Group([m[2] for m in mats], [m[3] for m in mats])
        a = torch.full((M, K), 99, dtype=torch.int8, device="cuda")
        s = torch.full((M,), -1.0, dtype=torch.float32, device="cuda")
        guards = [Guarded(torch, (M, N), torch.float32, float("nan")) for N in Ns]
        for _ in range(2):
            ys = b.w2a8_linear_grouped(x, grp, g, ws, fuse=fuse, a=a, a_scale=s, y=[gd.view for gd in guards])
        torch.cuda.synchronize()
        for gd in guards:
            gd.check("y")
        out[fuse] = (a.clone(), s.clone(), [t.clone() for t in ys])
    a_ref, s_ref = oracle.quantize(bits)
    for fuse in out:
        a, s, ys = out[fuse]
        assert np.array_equal(a.cpu().numpy(), a_ref), fuse
        assert np.array_equal(s.cpu().numpy().view(np.uint32), s_ref.view(np.uint32)), fuse
        for (codes, s_w, _, _), y in zip(mats, ys):
            assert _within(y.cpu().numpy(), oracle.gemm(a_ref, s_ref, codes, s_w, g)), fuse
    if b.w2a8_grouped_plan(Ns, M, K, g, b.FUSE_OFF)["one_launch"]:
        # same kernel with and without the quantiser inside: the same bits
        for y_on, y_off in zip(out[b.FUSE_ON][2], out[b.FUSE_OFF][2]):
            assert torch.equal(y_on, y_off)


def test_fused_without_quantiser_outputs_and_dead_rows(gpu, oracle):
    torch, b = gpu
    M, K, Ns, g = 4, 4096, [256, 64], 64
    mats = _mats(torch, b, 5, K, Ns, g)
    bits = synth.activations_bf16(9, M, K)
    bits[1, :] = 0                                   # dead token
    bits[2, :] = 0
    bits[2, 5] = 0x0003                              # so small that 1 / scale overflows: dead as well
    ws = b.new_workspace(b.w2a8_grouped_workspace_bytes(Ns, M, K, g))
    grp = b.Group([m[2] for m in mats], [m[3] for m in mats])
    ys = b.w2a8_linear_grouped(_bf16_dev(torch, bits), grp, g, ws, fuse=b.FUSE_ON)      # a, a_scale: not wanted
    torch.cuda.synchronize()
    a_ref, s_ref = oracle.quantize(bits)
    for (codes, s_w, _, _), y in zip(mats, ys):
        y = y.cpu().numpy()
        assert not y[1].any() and not y[2].any()
        assert _within(y, oracle.gemm(a_ref, s_ref, codes, s_w, g))
    # without fusing, the quantiser needs its output buffers
    with pytest.raises(b.W2A8Error) as e:
        b.w2a8_linear_grouped(_bf16_dev(torch, bits), grp, g, ws, fuse=b.FUSE_OFF)
    assert e.value.status == -1


@pytest.mark.parametrize("M", [1, 4, 16])
def test_layer_groups_default_dispatch(gpu, oracle, M):
    """q|k|v and gate|up of the Llama-3-8B layer at full size, as the benchmark calls them
    (default dispatch and fuse rule), on sampled channels."""
    torch, b = gpu
    cfg = synth.CONFIGS[1]
    rng = np.random.default_rng(M)
    for names in (("q", "k", "v"), ("gate", "up")):
        shapes = [(i, s) for i, s in enumerate(cfg["shapes"]) if s[0] in names]
        K = shapes[0][1][1]
        g = synth.config_group(cfg, K)
        mats = []
        for idx, (name, _, N) in shapes:
            codes, s_w = synth.make_linear(synth.shape_seed(cfg, idx), K, N, g)
            mats.append((codes, s_w, b.w2_pack(_dev(torch, codes)), _dev(torch, s_w)))
        Ns = [m[0].shape[0] for m in mats]
        bits = synth.activations_bf16(77 + M, M, K)
        a = torch.empty((M, K), dtype=torch.int8, device="cuda")
        s = torch.empty((M,), dtype=torch.float32, device="cuda")
        ws = b.new_workspace(b.w2a8_grouped_workspace_bytes(Ns, M, K, g))
        grp = b.Group([m[2] for m in mats], [m[3] for m in mats])
        ys = b.w2a8_linear_grouped(_bf16_dev(torch, bits), grp, g, ws, a=a, a_scale=s)
        torch.cuda.synchronize()
        assert b.w2a8_workspace_status(ws) == 0
        a_ref, s_ref = oracle.quantize(bits)
        assert np.array_equal(a.cpu().numpy(), a_ref)
        for (codes, s_w, _, _), y in zip(mats, ys):
            N = codes.shape[0]
            sel = np.unique(np.concatenate([np.arange(16), np.arange(N - 16, N), rng.choice(N, 64, replace=False)]))
            assert _within(y.cpu().numpy()[:, sel], oracle.gemm(a_ref, s_ref, codes[sel], s_w[sel], g)), names
            assert bool(torch.isfinite(y).all())


def test_grouped_falls_back_to_one_launch_per_matrix(gpu, oracle, monkeypatch):
    """Shapes the persistent kernel does not take (a ragged last block; many tokens) run as
    separate launches behind the same entry points."""
    torch, b = gpu
    for M, K, Ns, g in [(3, 1600, [48, 32], 64), (96, 1024, [256, 128], 64)]:
        mats = _mats(torch, b, M, K, Ns, g)
        bits = synth.activations_bf16(M, M, K)
        assert b.w2a8_grouped_plan(Ns, M, K, g) == {"one_launch": False, "fused": False}
        a = torch.empty((M, K), dtype=torch.int8, device="cuda")
        s = torch.empty((M,), dtype=torch.float32, device="cuda")
        ws = b.new_workspace(b.w2a8_grouped_workspace_bytes(Ns, M, K, g))
        grp = b.Group([m[2] for m in mats], [m[3] for m in mats])
        ys = b.w2a8_linear_grouped(_bf16_dev(torch, bits), grp, g, ws, a=a, a_scale=s)
        torch.cuda.synchronize()
        a_ref, s_ref = oracle.quantize(bits)
        for (codes, s_w, _, _), y in zip(mats, ys):
            assert _within(y.cpu().numpy(), oracle.gemm(a_ref, s_ref, codes, s_w, g))
