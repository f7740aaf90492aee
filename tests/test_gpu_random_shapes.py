"""Seeded random shapes through the public entry points against the CPU reference: the grouped
operator (persistent kernel in both of its forms, fused and unfused quantiser, one-shot fallback)
and w2a8_gemm at prefill sizes (default dispatch and forced variants: K split, 256-token tiles,
both warp layouts).  Outputs within 1e-4 * max|row|; int8 activations bit-exact."""
import random

import numpy as np
import pytest

from paper_2508_06753_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 1e-4
SWITCHES = ("W2A8_PREFILL", "W2A8_PF_KSPLIT", "W2A8_PF_WIDE", "W2A8_PF_UNPACK_WARPS", "W2A8_GEMV", "W2A8_GEMV_WARPS",
            "W2A8_FUSE_MAX_ELEMS", "W2A8_TC_KIND")


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


def _within(y, y_ref):
    err = np.abs(y.astype(np.float64) - y_ref.astype(np.float64)).max(axis=1)
    return bool((err <= TOL * np.abs(y_ref).max(axis=1)).all())


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_grouped_operator_random_shapes(gpu, oracle, monkeypatch, seed):
    """Few tokens, K a multiple of 256, one to four matrices of ragged widths, every group size."""
    torch, b = gpu
    for name in SWITCHES:
        monkeypatch.delenv(name, raising=False)
    rng = random.Random(seed)
    plans = set()
    for _ in range(16):
        M = rng.choice([1, 1, 2, 3, 4, 5, 7, 8, 9, 12, 16, 20, 32])
        K = 256 * rng.choice([1, 2, 3, 4, 5, 8, 12, 16, 16, 16, 24, 32, 56])
        g = rng.choice([64, 64, 128, 256, K])
        if K % g:
            g = 64
        Ns = [16 * rng.choice([1, 2, 3, 5, 8, 13, 31, 64, 100]) for _ in range(rng.choice([1, 2, 3, 4]))]
        mats = [synth.make_linear(rng.randrange(1 << 20), K, N, g) for N in Ns]
        bits = synth.activations_bf16(rng.randrange(1 << 20), M, K)
        x = _dev(torch, bits.view(np.int16)).view(torch.bfloat16)
        grp = b.Group([b.w2_pack(_dev(torch, c)) for c, _ in mats], [_dev(torch, s) for _, s in mats])
        ws = b.new_workspace(max(b.w2a8_grouped_workspace_bytes(Ns, M, K, g), 256))
        a_ref, s_ref = oracle.quantize(bits)
        refs = [oracle.gemm(a_ref, s_ref, c, s_w, g) for c, s_w in mats]
        for fuse in (b.FUSE_OFF, b.FUSE_ON):
            plan = b.w2a8_grouped_plan(Ns, M, K, g, fuse)
            plans.add((plan["one_launch"], plan["fused"]))
            a = torch.empty((M, K), dtype=torch.int8, device="cuda")
            s = torch.empty(M, dtype=torch.float32, device="cuda")
            ys = b.w2a8_linear_grouped(x, grp, g, ws, fuse=fuse, a=a, a_scale=s)
            torch.cuda.synchronize()
            assert b.w2a8_workspace_status(ws) == 0
            assert np.array_equal(a.cpu().numpy(), a_ref), (M, K, Ns, g, fuse)
            assert np.array_equal(s.cpu().numpy().view(np.uint32), s_ref.view(np.uint32)), (M, K, Ns, g, fuse)
            for y, ref in zip(ys, refs):
                assert _within(y.cpu().numpy(), ref), (M, K, Ns, g, fuse)
    assert (True, False) in plans               # the draws reach the persistent kernel


@pytest.mark.parametrize("seed", [21, 22, 23])
def test_gemm_random_prefill_shapes(gpu, oracle, monkeypatch, seed):
    """64 to 1024 tokens: whatever the dispatch picks, and the tensor-core variants when forced."""
    torch, b = gpu
    rng = random.Random(seed)
    seen = set()
    for _ in range(14):
        for name in SWITCHES:
            monkeypatch.delenv(name, raising=False)
        M = rng.choice([64, 65, 100, 128, 129, 200, 256, 300, 511, 700, 1024])
        N = 128 * rng.choice([1, 2, 3, 5, 8, 32, 37, 112])
        K = 256 * rng.choice([1, 2, 3, 4, 6, 8, 16, 56])
        g = rng.choice([64, 128, 256, K, K])
        if K % g:
            g = K
        env = rng.choice([{}, {}, {"W2A8_PREFILL": "2"},
                          {"W2A8_PREFILL": "2", "W2A8_PF_KSPLIT": rng.choice(["2", "4", "8"])},
                          {"W2A8_PREFILL": "2", "W2A8_PF_WIDE": "2"},
                          {"W2A8_PREFILL": "2", "W2A8_PF_UNPACK_WARPS": rng.choice(["2", "4"])}])
        for k, v in env.items():
            monkeypatch.setenv(k, v)
        codes, s_w = synth.make_linear(rng.randrange(1 << 20), K, N, g)
        bits = synth.activations_bf16(rng.randrange(1 << 20), M, K)
        a, s_a = b.a8_quantize(_dev(torch, bits.view(np.int16)).view(torch.bfloat16))
        ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g))
        y = b.w2a8_gemm(a, s_a, b.w2_pack(_dev(torch, codes)), _dev(torch, s_w), g, ws)
        torch.cuda.synchronize()
        assert b.w2a8_workspace_status(ws) == 0, (M, N, K, g, env)
        rows = sorted(set([0, M - 1] + [rng.randrange(M) for _ in range(6)]))
        a_ref, s_ref = oracle.quantize(bits[rows])
        idx = torch.tensor(rows, device="cuda")
        assert np.array_equal(a[idx].cpu().numpy(), a_ref)
        assert _within(y[idx].cpu().numpy(), oracle.gemm(a_ref, s_ref, codes, s_w, g)), (M, N, K, g, env)
        seen.add((b.w2a8_kernel_for(M, N, K, g), b.w2a8_tensor_core_tile_tokens(M, N, K, g),
                  b.w2a8_tensor_core_ksplit(M, N, K, g) > 1))
    assert any(k == "tensor_core" for k, _, _ in seen)
