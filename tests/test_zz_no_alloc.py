"""w2a8_gemm_static, the entry point for callers that cannot allocate or pass a
workspace (a runtime that owns all device memory, an operator slot with only
input/output pointers, a loop where allocation is forbidden): its scratch is a
fixed array inside the library.  Checked through the C ABI against w2a8_gemm
(same kernels, same launch configuration, so the same bits) and once against the
CPU reference, twice in a row with different activations: the second call finds
the first call's leftovers in the array.  This file is named to be collected last."""
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


# (M, N, K, group, what the scratch array is used for)
CASES = [
    (1, 256, 28672 + 128, 128, "split-K over more chunks than a cluster holds: arrival counters and partial "
                               "outputs live in the array"),
    (5, 64, 28672 + 192, 64, "the same with a ragged last chunk and several tokens"),
    (1, 1024, 4096, 64, "status word only"),
    (4, 4096, 4096, 64, "status word only"),
    (12, 256, 14336, 128, "status word only"),
    (1, 14336, 4096, 64, "status word only"),
    (512, 4096, 1024, 64, "tensor-core kernel: status word only"),
]


@pytest.mark.parametrize("M,N,K,g,why", CASES)
def test_static_scratch_matches_workspace_entry(gpu, oracle, M, N, K, g, why):
    torch, b = gpu
    codes, s_w = synth.make_linear(4242 + M, K, N, g)
    packed = b.w2_pack(_dev(torch, codes))
    s_w_d = _dev(torch, s_w)
    ws = b.new_workspace(b.w2a8_workspace_bytes(M, N, K, g))
    assert b.w2a8_workspace_bytes(M, N, K, g) <= b.STATIC_SCRATCH_BYTES
    y = torch.empty((M, N), dtype=torch.float32, device="cuda")
    for call in range(2):
        bits = synth.activations_bf16(100 * call + M, M, K)
        a, s_a = b.a8_quantize(_dev(torch, bits.view(np.int16)).view(torch.bfloat16))
        y_ref = b.w2a8_gemm(a, s_a, packed, s_w_d, g, ws)
        y.fill_(float("nan"))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        b.w2a8_gemm_static(a, s_a, packed, s_w_d, g, y)
        torch.cuda.synchronize()
        if call == 1:
            # (the first use on a device makes the CUDA runtime load the module image, which is
            # when the fixed array itself comes into being; later calls must leave memory alone)
            assert torch.cuda.mem_get_info()[0] == free_before, "the call must not allocate device memory"
        assert torch.equal(y, y_ref), (call, why)
        if call == 1:
            a_ref, s_ref = oracle.quantize(bits)
            want = oracle.gemm(a_ref, s_ref, codes, s_w, g)
            err = np.abs(y.cpu().numpy().astype(np.float64) - want).max(axis=1)
            assert (err <= TOL * np.abs(want).max(axis=1)).all(), (why, err.max())


def test_static_scratch_takes_the_split_k_workspace_path(gpu):
    """The first two cases above are only worth something if their split-K really goes through
    the scratch array: more than eight chunks cannot be summed inside a thread-block cluster."""
    torch, b = gpu
    for M, N, K, g, _ in CASES[:2]:
        assert b.w2a8_workspace_bytes(M, N, K, g) >= 256 + 9 * M * N * 4


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
