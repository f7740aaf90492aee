"""CPU-side checks of the C-ABI library: it builds, loads without a GPU, exports
every symbol the header declares, and rejects bad arguments on the host
before anything is launched."""
import ctypes
import os
import re

import pytest

from conftest import ROOT


@pytest.fixture(scope="module")
def lib():
    from paper_2508_06753_b200 import build, binding
    build.build()
    return binding.lib()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "w2a8.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    text = re.sub(r"^\s*#.*$", "", text, flags=re.M)      # preprocessor lines
    names = re.findall(r"\b([A-Za-z_][A-Za-z0-9_]*)\s*\([^;{}]*\)\s*;", text)
    return sorted(set(names))


def test_header_declares_expected_entry_points():
    names = _declared_functions()
    for must in ("w2_pack", "a8_quantize", "w2a8_gemm", "w2a8_gemm_partials", "w2a8_linear_host"):
        assert must in names


def test_library_exports_every_declared_symbol(lib):
    for name in _declared_functions():
        assert hasattr(lib, name), name


def test_binding_lists_every_declared_symbol():
    from paper_2508_06753_b200 import binding
    assert sorted(binding.EXPORTS) == _declared_functions()
    for name in binding.EXPORTS:
        assert hasattr(binding, name) or name == "w2a8_status_string"


def test_sizes_and_version(lib):
    assert lib.w2a8_version() >= 100
    assert lib.w2_packed_bytes(2048, 2048) == 2048 * 2048 // 4
    assert lib.w2_packed_bytes(16, 1600) == 16 * 1600 // 4
    assert lib.w2_packed_bytes(15, 64) == 0 and lib.w2_packed_bytes(16, 100) == 0
    assert lib.w2a8_workspace_bytes(1, 2048, 2048, 64) > 0
    assert lib.w2a8_workspace_bytes(1, 2048, 2048, 96) == 0      # group not allowed
    assert lib.w2a8_workspace_bytes(1, 2048, 2048, 192) == 0
    assert lib.w2a8_workspace_bytes(0, 2048, 2048, 64) == 0
    assert lib.w2a8_workspace_bytes(4, 4096, 14336, 14336) > 0   # group == K
    assert lib.w2a8_linear_host_workspace_bytes(4, 4096, 4096, 64) > lib.w2a8_workspace_bytes(4, 4096, 4096, 64)


def test_status_strings(lib):
    seen = set()
    for code in range(0, -8, -1):
        s = lib.w2a8_status_string(code).decode()
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 8
    assert lib.w2a8_status_string(-99).decode() == "unknown status"


def test_argument_errors_are_detected_on_the_host(lib):
    # no GPU here: every call below must return before touching the device
    buf = ctypes.create_string_buffer(1 << 16)
    base = ctypes.addressof(buf)
    p = (base + 15) // 16 * 16          # 16-byte aligned fake pointer
    NULLP, SHAPE, ALIGN, WS = -1, -2, -3, -4
    assert lib.w2_pack(None, 16, 64, p, None) == NULLP
    assert lib.w2_pack(p, 16, 65, p, None) == SHAPE
    assert lib.w2_pack(p + 4, 16, 64, p, None) == ALIGN
    assert lib.a8_quantize(None, 1, 64, p, p, None) == NULLP
    assert lib.a8_quantize(p, 0, 64, p, p, None) == SHAPE
    assert lib.a8_quantize(p, 1, 64, p + 1, p, None) == ALIGN
    assert lib.w2a8_gemm(None, p, p, p, p, 1, 16, 64, 64, p, 1 << 15, None) == NULLP
    assert lib.w2a8_gemm(p, p, p, p, p, 1, 16, 64, 32, p, 1 << 15, None) == SHAPE
    assert lib.w2a8_gemm(p, p, p, p, p, 1, 24, 64, 64, p, 1 << 15, None) == SHAPE
    assert lib.w2a8_gemm(p, p, p + 8, p, p, 1, 16, 64, 64, p, 1 << 15, None) == ALIGN
    assert lib.w2a8_gemm(p, p, p, p, p, 1, 16, 64, 64, None, 0, None) == WS
    assert lib.w2a8_gemm(p, p, p, p, p, 1, 16, 64, 64, p, 8, None) == WS
    assert lib.w2a8_gemm_partials(p, p, None, 1, 16, 64, 64, p, 1 << 15, None) == NULLP
    assert lib.w2a8_linear(None, p, p, p, p, p, 1, 16, 64, 64, p, 1 << 15, None) == NULLP
    assert lib.w2a8_linear(p, p, p, p, p, p, 1, 16, 64, 32, p, 1 << 15, None) == SHAPE
    assert lib.w2a8_linear(p, p, p, p, p, p, 1, 16, 64, 64, p, 8, None) == WS
    assert lib.w2a8_linear_host(None, 1, 64, p, p, 16, 64, p, p, 1 << 15, None) == NULLP
    assert lib.w2a8_linear_host(p, 1, 64, p, p, 16, 48, p, p, 1 << 15, None) == SHAPE
    assert lib.w2a8_linear_host(p, 1, 64, p, p, 16, 64, p, p, 16, None) == WS
    assert lib.w2a8_workspace_init(None, 16, None) == NULLP
    assert lib.w2a8_workspace_status(None, None) == NULLP


def test_grouped_entry_points_reject_bad_arguments_on_the_host(lib):
    buf = ctypes.create_string_buffer(1 << 16)
    p = (ctypes.addressof(buf) + 15) // 16 * 16
    NULLP, SHAPE, ALIGN, WS = -1, -2, -3, -4
    vp2 = (ctypes.c_void_p * 2)(p, p)
    n2 = (ctypes.c_int * 2)(16, 32)
    bad_n = (ctypes.c_int * 2)(16, 24)
    null2 = (ctypes.c_void_p * 2)(p, None)
    odd2 = (ctypes.c_void_p * 2)(p, p + 8)
    big = 1 << 15
    assert lib.w2a8_gemm_grouped(None, p, 2, vp2, vp2, vp2, n2, 1, 256, 64, p, big, None) == NULLP
    assert lib.w2a8_gemm_grouped(p, p, 2, None, vp2, vp2, n2, 1, 256, 64, p, big, None) == NULLP
    assert lib.w2a8_gemm_grouped(p, p, 2, null2, vp2, vp2, n2, 1, 256, 64, p, big, None) == NULLP
    assert lib.w2a8_gemm_grouped(p, p, 0, vp2, vp2, vp2, n2, 1, 256, 64, p, big, None) == SHAPE
    assert lib.w2a8_gemm_grouped(p, p, 5, vp2, vp2, vp2, n2, 1, 256, 64, p, big, None) == SHAPE
    assert lib.w2a8_gemm_grouped(p, p, 2, vp2, vp2, vp2, bad_n, 1, 256, 64, p, big, None) == SHAPE
    assert lib.w2a8_gemm_grouped(p, p, 2, vp2, vp2, vp2, n2, 1, 256, 96, p, big, None) == SHAPE
    assert lib.w2a8_gemm_grouped(p, p, 2, vp2, odd2, vp2, n2, 1, 256, 64, p, big, None) == ALIGN
    assert lib.w2a8_gemm_grouped(p, p, 2, vp2, vp2, vp2, n2, 1, 256, 64, None, 0, None) == WS
    assert lib.w2a8_linear_grouped(None, p, p, 2, vp2, vp2, vp2, n2, 1, 256, 64, -1, p, big, None) == NULLP
    assert lib.w2a8_linear_grouped(p, p, p, 2, vp2, vp2, vp2, n2, 1, 256, 64, 7, p, big, None) == SHAPE
    assert lib.w2a8_linear_grouped(p + 2, p, p, 2, vp2, vp2, vp2, n2, 1, 256, 64, 1, p, big, None) == ALIGN
    assert lib.w2a8_linear_grouped(p, p, p, 2, vp2, vp2, vp2, n2, 1, 256, 64, 0, p, 8, None) == WS
    assert lib.w2a8_grouped_workspace_bytes(2, n2, 1, 256, 64) >= 256
    assert lib.w2a8_grouped_workspace_bytes(2, bad_n, 1, 256, 64) == 0
    assert lib.w2a8_grouped_workspace_bytes(0, n2, 1, 256, 64) == 0
    assert lib.w2a8_grouped_plan(2, bad_n, 1, 256, 64, -1) == SHAPE
    assert lib.w2a8_linear_grouped_host(None, 1, 256, 2, vp2, vp2, n2, 64, vp2, p, big, None) == NULLP
    assert lib.w2a8_linear_grouped_host(p, 1, 256, 2, vp2, vp2, bad_n, 64, vp2, p, big, None) == SHAPE
    assert lib.w2a8_linear_grouped_host(p, 1, 256, 2, vp2, vp2, n2, 64, null2, p, 1 << 20, None) == NULLP
    assert lib.w2a8_linear_grouped_host(p, 1, 256, 2, vp2, vp2, n2, 64, vp2, p, 16, None) == WS
    assert lib.w2a8_linear_grouped_host_workspace_bytes(2, n2, 1, 256, 64) > lib.w2a8_grouped_workspace_bytes(2, n2, 1, 256, 64)
    assert lib.w2a8_read_probe(None, 1 << 20, p, None) == NULLP
    assert lib.w2a8_read_probe(p + 4, 1 << 20, p, None) == ALIGN


def test_grouped_plan_needs_no_gpu(lib, monkeypatch):
    """Which kernel a group of matrices gets and whether the quantiser goes inside is host logic:
    pinned on the linear groups of the benchmark layer (148 SMs assumed when no device is present)."""
    from paper_2508_06753_b200 import binding as b
    for name in ("W2A8_GEMV", "W2A8_FUSE_MAX_ELEMS", "W2A8_CHUNKS", "W2A8_TG", "W2A8_RING", "W2A8_MT",
                 "W2A8_CLUSTER", "W2A8_MIN_WARPS", "W2A8_RELAX"):
        monkeypatch.delenv(name, raising=False)
    qkv, gateup = [4096, 1024, 1024], [14336, 14336]
    assert b.w2a8_grouped_plan(qkv, 1, 4096, 64) == {"one_launch": True, "fused": False}       # the separate quantiser is ahead on the device
    assert b.w2a8_grouped_plan(qkv, 1, 4096, 64, b.FUSE_ON) == {"one_launch": True, "fused": True}
    monkeypatch.setenv("W2A8_FUSE_MAX_ELEMS", "8192")
    assert b.w2a8_grouped_plan(qkv, 1, 4096, 64) == {"one_launch": True, "fused": True}
    assert b.w2a8_grouped_plan(qkv, 4, 4096, 64) == {"one_launch": True, "fused": False}
    monkeypatch.delenv("W2A8_FUSE_MAX_ELEMS")
    assert b.w2a8_grouped_plan(qkv, 4, 4096, 64) == {"one_launch": True, "fused": False}
    assert b.w2a8_grouped_plan(qkv, 16, 4096, 64) == {"one_launch": True, "fused": False}
    assert b.w2a8_grouped_plan(gateup, 4, 4096, 64) == {"one_launch": True, "fused": False}
    assert b.w2a8_grouped_plan([14336], 1, 4096, 64, b.FUSE_OFF) == {"one_launch": False, "fused": False}
    assert b.w2a8_grouped_plan([4096], 1, 14336, 64) == {"one_launch": False, "fused": False}      # down
    assert b.w2a8_grouped_plan([4096], 16, 14336, 64) == {"one_launch": True, "fused": False}
    assert b.w2a8_grouped_plan([8192], 1, 28672, 128) == {"one_launch": True, "fused": False}      # 70B down
    assert b.w2a8_grouped_plan(qkv, 4, 4096, 64, b.FUSE_ON) == {"one_launch": True, "fused": True}
    assert b.w2a8_grouped_plan(qkv, 16, 4096, 64, b.FUSE_ON)["fused"] is False                     # too many tokens
    assert b.w2a8_grouped_plan([48, 32], 3, 1600, 64) == {"one_launch": False, "fused": False}     # ragged K
    assert b.w2a8_grouped_plan(qkv, 64, 4096, 64) == {"one_launch": False, "fused": False}
    monkeypatch.setenv("W2A8_GEMV", "0")
    assert b.w2a8_grouped_plan(qkv, 1, 4096, 64) == {"one_launch": False, "fused": False}
    monkeypatch.setenv("W2A8_GEMV", "2")
    assert b.w2a8_grouped_plan([14336], 1, 4096, 64, b.FUSE_OFF)["one_launch"] is True


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2508_06753_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(FileNotFoundError):
        binding.lib()


def test_dispatch_queries_need_no_gpu(lib, monkeypatch):
    """Which kernel serves a shape, and how the channels are split between the two kernels, is
    host logic: pinned here on the shapes of the benchmark configurations."""
    from paper_2508_06753_b200 import binding as b
    for name in ("W2A8_PREFILL", "W2A8_PF_SPLIT", "W2A8_PF_KSPLIT", "W2A8_TC_KIND", "W2A8_PF_WIDE"):
        monkeypatch.delenv(name, raising=False)
    # few tokens: streaming kernel
    for M in (1, 4, 16, 32, 63):
        assert b.w2a8_kernel_for(M, 14336, 4096, 64) == "streaming"
        assert b.w2a8_tensor_core_channels(M, 14336, 4096, 64) == 0
    # prefill configuration: tensor-core kernel; a ragged last round of tiles is trimmed
    assert b.w2a8_kernel_for(512, 14336, 4096, 64) == "tensor_core"
    assert b.w2a8_tensor_core_channels(512, 14336, 4096, 64) == 111 * 128       # 444 tiles = 3 x 148
    assert b.w2a8_tensor_core_channels(2048, 14336, 4096, 64) == 111 * 128      # 1776 tiles = 12 x 148
    assert b.w2a8_tensor_core_channels(8192, 14336, 4096, 64) == 14336          # the rest would cost more than a round
    assert b.w2a8_tensor_core_channels(2048, 4096, 14336, 64) == 4096
    # too few output tiles for 148 SMs: K is split so that every SM has work ...
    assert b.w2a8_kernel_for(128, 4096, 14336, 64) == "tensor_core"
    assert b.w2a8_tensor_core_ksplit(128, 4096, 14336, 64) == 4
    assert b.w2a8_tensor_core_channels(128, 4096, 14336, 64) == 4096
    assert b.w2a8_tensor_core_ksplit(256, 4096, 4096, 64) == 2
    assert b.w2a8_tensor_core_ksplit(2048, 14336, 4096, 64) == 1
    assert b.w2a8_workspace_bytes(128, 4096, 14336, 64) >= 256 + 4 * 128 * 4096 * 4
    # one scale per channel and many tokens: 256-token tiles
    assert b.w2a8_tensor_core_tile_tokens(2048, 14336, 4096, 4096) == 256
    assert b.w2a8_tensor_core_channels(2048, 14336, 4096, 4096) == 111 * 128     # 888 wide tiles = 6 x 148
    assert b.w2a8_tensor_core_tile_tokens(2048, 14336, 4096, 64) == 128
    assert b.w2a8_tensor_core_tile_tokens(4, 14336, 4096, 4096) == 0
    # ... or the streaming kernel takes it where that does not pay
    assert b.w2a8_kernel_for(64, 4096, 4096, 64) == "streaming"
    assert b.w2a8_tensor_core_ksplit(64, 4096, 4096, 64) == 0
    # shapes the tensor-core kernel does not tile
    assert b.w2a8_kernel_for(512, 1040, 4096, 64) == "streaming"
    assert b.w2a8_kernel_for(512, 4096, 4160, 64) == "streaming"
    # switches
    monkeypatch.setenv("W2A8_PREFILL", "0")
    assert b.w2a8_kernel_for(2048, 14336, 4096, 64) == "streaming"
    monkeypatch.setenv("W2A8_PREFILL", "2")
    assert b.w2a8_kernel_for(64, 128, 256, 64) == "tensor_core"
    assert b.w2a8_tensor_core_channels(512, 14336, 4096, 64) == 14336
    monkeypatch.setenv("W2A8_PREFILL", "1")
    monkeypatch.setenv("W2A8_PF_SPLIT", "0")
    assert b.w2a8_tensor_core_channels(512, 14336, 4096, 64) == 14336
    # the workspace covers the plan of the streamed remainder as well
    monkeypatch.delenv("W2A8_PF_SPLIT")
    with_split = b.w2a8_workspace_bytes(512, 14336, 4096, 64)
    monkeypatch.setenv("W2A8_PF_SPLIT", "0")
    assert with_split >= b.w2a8_workspace_bytes(512, 14336, 4096, 64) > 0
    with pytest.raises(b.W2A8Error):
        b.w2a8_kernel_for(4, 100, 4096, 64)


def test_dispatch_plan_invariants(lib, monkeypatch):
    """Host-side planning on random accepted shapes: what the report functions say is consistent
    (no device needed): channel splits are whole 128-channel tiles, K splits are whole 256-k blocks
    and whole scale groups of at least two blocks, the workspace covers the partial outputs, 256-token
    tiles only with one scale per channel."""
    import random
    from paper_2508_06753_b200 import binding as b
    for name in ("W2A8_PREFILL", "W2A8_PF_SPLIT", "W2A8_PF_KSPLIT", "W2A8_TC_KIND", "W2A8_PF_WIDE", "W2A8_GEMV"):
        monkeypatch.delenv(name, raising=False)
    rng = random.Random(5)
    seen_tc = seen_split = seen_wide = 0
    for _ in range(400):
        M = rng.choice([1, 8, 33, 64, 96, 128, 200, 256, 512, 1000, 2048, 4096])
        N = 16 * rng.choice([1, 8, 64, 256, 512, 896, 1024, 1792])
        K = 64 * rng.choice([1, 4, 8, 16, 32, 64, 128, 224])
        g = rng.choice([64, 128, 256, K])
        if K % g or (g not in (64, 128) and g % 256 and g != K):
            continue
        kernel = b.w2a8_kernel_for(M, N, K, g)
        ch, sp, tok = (b.w2a8_tensor_core_channels(M, N, K, g), b.w2a8_tensor_core_ksplit(M, N, K, g),
                       b.w2a8_tensor_core_tile_tokens(M, N, K, g))
        ws = b.w2a8_workspace_bytes(M, N, K, g)
        assert ws >= 4 and ws % 16 == 0
        if kernel == "streaming":
            assert (ch, sp, tok) == (0, 0, 0)
            continue
        seen_tc += 1
        assert M >= 64 and N % 128 == 0 and K % 256 == 0
        assert 0 < ch <= N and ch % 128 == 0 and N - ch <= 8 * 128
        assert sp in (1, 2, 4, 8) and tok in (128, 256)
        if sp > 1:
            seen_split += 1
            assert ch == N and tok == 128
            assert (K // sp) % 256 == 0 and (K // sp) % g == 0 and K // sp >= 512
            assert ws >= 256 + sp * M * N * 4
        if tok == 256:
            seen_wide += 1
            assert g == K and M >= 129 and sp == 1
    assert seen_tc > 20 and seen_split > 0 and seen_wide > 0
