"""w2a8_gemm_static, the entry point for callers that cannot allocate or pass a
workspace (a runtime that owns all device memory, an operator slot with only
input/output pointers, a loop where allocation is forbidden): its scratch is a
fixed array inside the library.  Checked through the C ABI against w2a8_gemm,
twice in a row (the second call finds the first call's leftovers in the array).
This file is named to be collected last."""
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


@pytest.mark.parametrize("M,N,K,g", [(1, 1024, 4096, 64),      # split-K: counters and partial sums in use
                                     (4, 4096, 4096, 64),
                                     (12, 256, 14336, 128),
                                     (1, 14336, 4096, 64)])    # single chunk: no scratch traffic
def test_static_scratch_matches_workspace_entry(gpu, M, N, K, g):
    torch, b = gpu
    codes, s_w = synth.make_linear(4242 + M, K, N, g)
    packed = b.w2_pack(_dev(torch, codes))
    s_w_d = _dev(torch, s_w)
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g))
    assert b.w2a8_workspace_bytes(M, N, K, g) <= b.STATIC_SCRATCH_BYTES
    for call in range(2):
        bits = synth.activations_bf16(100 * call + M, M, K)
        a, s_a = b.a8_quantize(_dev(torch, bits.view(np.int16)).view(torch.bfloat16))
        y_ref = b.w2a8_gemm(a, s_a, packed, s_w_d, g, ws)
        y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        b.w2a8_gemm_static(a, s_a, packed, s_w_d, g, y)
        torch.cuda.synchronize()
        y, y_ref = y.cpu().numpy(), y_ref.cpu().numpy()
        err = np.abs(y.astype(np.float64) - y_ref).max(axis=1)
        assert np.isfinite(y).all()
        assert (err <= TOL * np.abs(y_ref).max(axis=1)).all(), (call, err.max())


def test_static_scratch_refuses_oversized_problems(gpu):
    torch, b = gpu
    M, N, K, g = 32, 28672, 28672, 128      # split-K partial sums alone exceed the scratch
    assert b.w2a8_workspace_bytes(M, N, K, g) > b.STATIC_SCRATCH_BYTES
    a = torch.zeros((M, K), dtype=torch.int8, device="cuda")
    s_a = torch.ones((M,), dtype=torch.float32, device="cuda")
    packed = torch.zeros((N, K // 16), dtype=torch.int32, device="cuda")
    s_w = torch.ones((N, K // g), dtype=torch.float32, device="cuda")
    with pytest.raises(b.W2A8Error) as e:
        b.w2a8_gemm_static(a, s_a, packed, s_w, g)
    assert e.value.status == -4
