"""Thin ctypes binding of the C-ABI library ``libw2a8.so`` (see include/w2a8.h).

Argument marshalling only: every step of the path runs in the CUDA kernels of
the library.  torch supplies device memory and the current stream, nothing
else.  There is no CPU fallback: if the library is missing, ``lib()`` raises.
Function names match the C entry points.
"""
from __future__ import annotations

import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libw2a8.so")

EXPORTS = [
    "w2a8_version", "w2a8_status_string", "w2_packed_bytes", "w2_pack", "a8_quantize",
    "w2a8_workspace_bytes", "w2a8_workspace_init", "w2a8_workspace_status", "w2a8_gemm", "w2a8_gemm_partials",
    "w2a8_kernel_for", "w2a8_tensor_core_channels", "w2a8_tensor_core_ksplit", "w2a8_tensor_core_tile_tokens", "w2a8_gemm_h16", "w2a16_gemm", "w2a8_linear", "w2a8_linear_host_workspace_bytes", "w2a8_linear_host", "w2a8_gemm_static",
    "w2a8_gemm_grouped", "w2a8_linear_grouped", "w2a8_grouped_workspace_bytes", "w2a8_grouped_plan",
    "w2a8_read_probe", "w2a8_tensor_core_kind",
    "w2a8_linear_grouped_host", "w2a8_linear_grouped_host_workspace_bytes",
]

_lib = None


class W2A8Error(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


def lib() -> ctypes.CDLL:
    """Load the library once; raise if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} not found: build it with `python -m paper_2508_06753_b200.build` "
                "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        L.w2a8_version.restype = i
        L.w2a8_status_string.restype = ctypes.c_char_p
        L.w2a8_status_string.argtypes = [i]
        L.w2_packed_bytes.restype = sz
        L.w2_packed_bytes.argtypes = [i, i]
        L.w2_pack.argtypes = [vp, i, i, vp, vp]
        L.a8_quantize.argtypes = [vp, i, i, vp, vp, vp]
        L.w2a8_workspace_bytes.restype = sz
        L.w2a8_workspace_bytes.argtypes = [i, i, i, i]
        L.w2a8_workspace_init.argtypes = [vp, sz, vp]
        L.w2a8_workspace_status.argtypes = [vp, vp]
        L.w2a8_gemm.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, vp, sz, vp]
        L.w2a8_gemm_h16.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, vp, sz, vp]
        L.w2a8_kernel_for.argtypes = [i, i, i, i]
        L.w2a8_tensor_core_channels.argtypes = [i, i, i, i]
        L.w2a8_tensor_core_ksplit.argtypes = [i, i, i, i]
        L.w2a8_tensor_core_tile_tokens.argtypes = [i, i, i, i]
        L.w2a16_gemm.argtypes = [vp, vp, vp, vp, i, i, i, i, vp, sz, vp]
        L.w2a8_gemm_partials.argtypes = [vp, vp, vp, i, i, i, i, vp, sz, vp]
        L.w2a8_linear.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, vp, sz, vp]
        L.w2a8_linear_host_workspace_bytes.restype = sz
        L.w2a8_linear_host_workspace_bytes.argtypes = [i, i, i, i]
        L.w2a8_linear_host.argtypes = [vp, i, i, vp, vp, i, i, vp, vp, sz, vp]
        L.w2a8_gemm_static.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, vp]
        L.w2a8_gemm_grouped.argtypes = [vp, vp, i, vp, vp, vp, vp, i, i, i, vp, sz, vp]
        L.w2a8_linear_grouped.argtypes = [vp, vp, vp, i, vp, vp, vp, vp, i, i, i, i, vp, sz, vp]
        L.w2a8_grouped_workspace_bytes.restype = sz
        L.w2a8_grouped_workspace_bytes.argtypes = [i, vp, i, i, i]
        L.w2a8_grouped_plan.argtypes = [i, vp, i, i, i, i]
        L.w2a8_linear_grouped_host_workspace_bytes.restype = sz
        L.w2a8_linear_grouped_host_workspace_bytes.argtypes = [i, vp, i, i, i]
        L.w2a8_linear_grouped_host.argtypes = [vp, i, i, i, vp, vp, vp, i, vp, vp, sz, vp]
        L.w2a8_linear_grouped_host.restype = i
        L.w2a8_tensor_core_kind.argtypes = [i, i, i, i]
        L.w2a8_tensor_core_kind.restype = i
        L.w2a8_read_probe.argtypes = [vp, sz, vp, vp]
        L.w2a8_read_probe.restype = i
        for name in ("w2_pack", "a8_quantize", "w2a8_workspace_init", "w2a8_workspace_status", "w2a8_gemm",
                     "w2a8_gemm_partials", "w2a8_linear", "w2a8_linear_host", "w2a8_gemm_static",
                     "w2a8_gemm_grouped", "w2a8_linear_grouped", "w2a8_grouped_plan"):
            getattr(L, name).restype = i
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().w2a8_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != 0:
        raise W2A8Error(status, where)


def _stream(stream=None) -> int:
    if stream is not None:
        return int(stream.cuda_stream)
    # raw handle of the current stream of the current device, without building a Stream object
    return int(torch._C._cuda_getCurrentRawStream(torch.cuda.current_device()))


def _ptr(t) -> int:
    return 0 if t is None else int(t.data_ptr())


def w2a8_version() -> int:
    return int(lib().w2a8_version())


def w2_packed_bytes(N: int, K: int) -> int:
    return int(lib().w2_packed_bytes(N, K))


def w2a8_workspace_bytes(M: int, N: int, K: int, group: int) -> int:
    return int(lib().w2a8_workspace_bytes(M, N, K, group))


def w2a8_linear_host_workspace_bytes(M: int, N: int, K: int, group: int) -> int:
    return int(lib().w2a8_linear_host_workspace_bytes(M, N, K, group))


def new_workspace(nbytes: int, device="cuda", stream=None) -> torch.Tensor:
    """Allocate and zero-fill a workspace of at least `nbytes` bytes."""
    ws = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)
    w2a8_workspace_init(ws, stream)
    return ws


def w2a8_workspace_init(workspace: torch.Tensor, stream=None):
    _check(lib().w2a8_workspace_init(_ptr(workspace), workspace.numel() * workspace.element_size(),
                                     _stream(stream)), "w2a8_workspace_init")


def w2a8_workspace_status(workspace: torch.Tensor, stream=None) -> int:
    """Device status word of a workspace (0 = ok); synchronises the stream."""
    return int(lib().w2a8_workspace_status(_ptr(workspace), _stream(stream)))


def w2_pack(codes: torch.Tensor, packed: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """codes uint8 [N][K] (device) -> packed int32 [N][K/16] (bit pattern of uint32)."""
    N, K = codes.shape
    if packed is None:
        packed = torch.empty((N, max(K // 16, 1)), dtype=torch.int32, device=codes.device)
    _check(lib().w2_pack(_ptr(codes), N, K, _ptr(packed), _stream(stream)), "w2_pack")
    return packed


def a8_quantize(x_bf16: torch.Tensor, a: torch.Tensor | None = None,
                a_scale: torch.Tensor | None = None, stream=None):
    """x bf16 [M][K] (device) -> (a int8 [M][K], a_scale fp32 [M])."""
    M, K = x_bf16.shape
    if a is None:
        a = torch.empty((M, K), dtype=torch.int8, device=x_bf16.device)
    if a_scale is None:
        a_scale = torch.empty((M,), dtype=torch.float32, device=x_bf16.device)
    _check(lib().a8_quantize(_ptr(x_bf16), M, K, _ptr(a), _ptr(a_scale), _stream(stream)),
           "a8_quantize")
    return a, a_scale


def w2a8_gemm(a: torch.Tensor, a_scale: torch.Tensor, packed: torch.Tensor, w_scale: torch.Tensor,
              group: int, workspace: torch.Tensor, y: torch.Tensor | None = None, stream=None):
    """y fp32 [M][N] = scaled W2A8 product; see w2a8_gemm in include/w2a8.h."""
    M, K = a.shape
    N = packed.shape[0]
    if y is None:
        y = torch.empty((M, N), dtype=torch.float32, device=a.device)
    _check(lib().w2a8_gemm(_ptr(a), _ptr(a_scale), _ptr(packed), _ptr(w_scale), _ptr(y), M, N, K,
                           group, _ptr(workspace), workspace.numel() * workspace.element_size(),
                           _stream(stream)), "w2a8_gemm")
    return y


def w2a8_kernel_for(M: int, N: int, K: int, group: int) -> str:
    """'streaming' or 'tensor_core': the kernel w2a8_gemm uses for this shape."""
    r = int(lib().w2a8_kernel_for(M, N, K, group))
    _check(r if r < 0 else 0, "w2a8_kernel_for")
    return "tensor_core" if r == 1 else "streaming"


def w2a8_tensor_core_kind(M: int, N: int, K: int, group: int) -> int:
    """8 (int8 kernel), 16 (16-bit kernel on a bf16 copy of the activations) or 0 (streaming)."""
    r = int(lib().w2a8_tensor_core_kind(M, N, K, group))
    _check(r if r < 0 else 0, "w2a8_tensor_core_kind")
    return r


def w2a8_tensor_core_channels(M: int, N: int, K: int, group: int) -> int:
    """Channels of the problem computed by the tensor-core kernel (0 .. N); the rest, if any, is
    computed by the streaming kernel."""
    r = int(lib().w2a8_tensor_core_channels(M, N, K, group))
    _check(r if r < 0 else 0, "w2a8_tensor_core_channels")
    return r


def w2a8_tensor_core_ksplit(M: int, N: int, K: int, group: int) -> int:
    """K splits of the tensor-core kernel for this shape (0: streaming kernel; host only)."""
    r = int(lib().w2a8_tensor_core_ksplit(M, N, K, group))
    _check(r if r < 0 else 0, "w2a8_tensor_core_ksplit")
    return r


def w2a8_tensor_core_tile_tokens(M: int, N: int, K: int, group: int) -> int:
    """Token rows per tile of the tensor-core kernel for this shape (0: streaming kernel; host only)."""
    r = int(lib().w2a8_tensor_core_tile_tokens(M, N, K, group))
    _check(r if r < 0 else 0, "w2a8_tensor_core_tile_tokens")
    return r


def w2a8_gemm_h16(a: torch.Tensor, a_scale: torch.Tensor, packed: torch.Tensor, w_scale_h: torch.Tensor,
                  group: int, workspace: torch.Tensor, y: torch.Tensor | None = None,
                  out_dtype: torch.dtype = torch.float32, stream=None):
    """w2a8_gemm with binary16 weight scales (w_scale_h: float16 [N][K/group]) and an fp32 or bf16
    result (the dtype of y, else out_dtype); see w2a8_gemm_h16 in include/w2a8.h."""
    M, K = a.shape
    N = packed.shape[0]
    if w_scale_h.dtype != torch.float16:
        raise TypeError("w_scale_h must be float16")
    if y is None:
        y = torch.empty((M, N), dtype=out_dtype, device=a.device)
    if y.dtype not in (torch.float32, torch.bfloat16):
        raise TypeError("y must be float32 or bfloat16")
    _check(lib().w2a8_gemm_h16(_ptr(a), _ptr(a_scale), _ptr(packed), _ptr(w_scale_h), _ptr(y),
                               1 if y.dtype == torch.bfloat16 else 0, M, N, K, group, _ptr(workspace),
                               workspace.numel() * workspace.element_size(), _stream(stream)),
           "w2a8_gemm_h16")
    return y


def w2a16_gemm(x: torch.Tensor, packed: torch.Tensor, w_scale: torch.Tensor, group: int,
               workspace: torch.Tensor, y: torch.Tensor | None = None, stream=None):
    """bf16 x [M][K] (device, not quantised) -> y fp32 [M][N]; see w2a16_gemm in include/w2a8.h."""
    M, K = x.shape
    N = packed.shape[0]
    if x.dtype != torch.bfloat16:
        raise TypeError("x must be bfloat16")
    if y is None:
        y = torch.empty((M, N), dtype=torch.float32, device=x.device)
    _check(lib().w2a16_gemm(_ptr(x), _ptr(packed), _ptr(w_scale), _ptr(y), M, N, K, group, _ptr(workspace),
                            workspace.numel() * workspace.element_size(), _stream(stream)), "w2a16_gemm")
    return y


def w2a8_linear(x: torch.Tensor, packed: torch.Tensor, w_scale: torch.Tensor, group: int,
                workspace: torch.Tensor, a: torch.Tensor | None = None, a_scale: torch.Tensor | None = None,
                y: torch.Tensor | None = None, stream=None):
    """bf16 x [M][K] (device) -> (y fp32 [M][N], a int8 [M][K], a_scale fp32 [M]) in one call; see
    w2a8_linear in include/w2a8.h.  a / a_scale receive what a8_quantize would write."""
    M, K = x.shape
    N = packed.shape[0]
    if a is None:
        a = torch.empty((M, K), dtype=torch.int8, device=x.device)
    if a_scale is None:
        a_scale = torch.empty((M,), dtype=torch.float32, device=x.device)
    if y is None:
        y = torch.empty((M, N), dtype=torch.float32, device=x.device)
    _check(lib().w2a8_linear(_ptr(x), _ptr(a), _ptr(a_scale), _ptr(packed), _ptr(w_scale), _ptr(y), M, N, K,
                             group, _ptr(workspace), workspace.numel() * workspace.element_size(),
                             _stream(stream)), "w2a8_linear")
    return y, a, a_scale


def w2a8_gemm_partials(a: torch.Tensor, packed: torch.Tensor, group: int, workspace: torch.Tensor,
                       partials: torch.Tensor | None = None, stream=None):
    """Exact int32 per-group sums P[M][N][K/group] (parity/debug export)."""
    M, K = a.shape
    N = packed.shape[0]
    if partials is None:
        partials = torch.empty((M, N, K // group), dtype=torch.int32, device=a.device)
    _check(lib().w2a8_gemm_partials(_ptr(a), _ptr(packed), _ptr(partials), M, N, K, group,
                                    _ptr(workspace), workspace.numel() * workspace.element_size(),
                                    _stream(stream)), "w2a8_gemm_partials")
    return partials


def w2a8_linear_host(x_host: torch.Tensor, packed: torch.Tensor, w_scale: torch.Tensor, group: int,
                     y_host: torch.Tensor, workspace: torch.Tensor, stream=None):
    """Host bf16 x [M][K] -> host fp32 y [M][N]; copies, quantiser and GEMM enqueued on the stream."""
    M, K = x_host.shape
    N = packed.shape[0]
    _check(lib().w2a8_linear_host(_ptr(x_host), M, K, _ptr(packed), _ptr(w_scale), N, group,
                                  _ptr(y_host), _ptr(workspace),
                                  workspace.numel() * workspace.element_size(), _stream(stream)),
           "w2a8_linear_host")
    return y_host


FUSE_AUTO, FUSE_OFF, FUSE_ON = -1, 0, 1


class Group:
    """Host-side argument block of the grouped entry points: the arrays of device pointers and of
    N, built once for a set of weight matrices (and, optionally, outputs) and reused every call."""

    def __init__(self, packed, w_scale, y=None):
        self.packed, self.w_scale = list(packed), list(w_scale)
        self.count = len(self.packed)
        self.N = [int(p.shape[0]) for p in self.packed]
        self.K = int(self.packed[0].shape[1]) * 16
        self._pk = (ctypes.c_void_p * self.count)(*[_ptr(p) for p in self.packed])
        self._sc = (ctypes.c_void_p * self.count)(*[_ptr(s) for s in self.w_scale])
        self._n = (ctypes.c_int * self.count)(*self.N)
        self.y = None
        self._y = None
        if y is not None:
            self.bind_outputs(y)

    def bind_outputs(self, y):
        self.y = list(y)
        self._y = (ctypes.c_void_p * self.count)(*[_ptr(t) for t in self.y])


def w2a8_grouped_workspace_bytes(N, M: int, K: int, group: int) -> int:
    arr = (ctypes.c_int * len(N))(*[int(n) for n in N])
    return int(lib().w2a8_grouped_workspace_bytes(len(N), arr, M, K, group))


def w2a8_grouped_plan(N, M: int, K: int, group: int, fuse: int = FUSE_AUTO) -> dict:
    """What a grouped call will do: {'one_launch': bool, 'fused': bool}."""
    arr = (ctypes.c_int * len(N))(*[int(n) for n in N])
    r = int(lib().w2a8_grouped_plan(len(N), arr, M, K, group, fuse))
    _check(r if r < 0 else 0, "w2a8_grouped_plan")
    return {"one_launch": bool(r & 1), "fused": bool(r & 2)}


def w2a8_gemm_grouped(a: torch.Tensor, a_scale: torch.Tensor, grp: Group, group: int,
                      workspace: torch.Tensor, y=None, stream=None):
    """y[i] = W2A8(a; matrix i) for the matrices of `grp`; see w2a8_gemm_grouped in include/w2a8.h."""
    M, K = a.shape
    if y is not None:
        grp.bind_outputs(y)
    elif grp.y is None or grp.y[0].shape[0] != M:
        grp.bind_outputs([torch.empty((M, n), dtype=torch.float32, device=a.device) for n in grp.N])
    _check(lib().w2a8_gemm_grouped(_ptr(a), _ptr(a_scale), grp.count, grp._pk, grp._sc, grp._y, grp._n, M, K,
                                   group, _ptr(workspace), workspace.numel() * workspace.element_size(),
                                   _stream(stream)), "w2a8_gemm_grouped")
    return grp.y


def w2a8_linear_grouped(x: torch.Tensor, grp: Group, group: int, workspace: torch.Tensor, fuse: int = FUSE_AUTO,
                        a: torch.Tensor | None = None, a_scale: torch.Tensor | None = None, y=None, stream=None):
    """bf16 x [M][K] (device) -> y[i] fp32 [M][N_i] for the matrices of `grp`; a / a_scale (optional when the
    call fuses) receive what a8_quantize would write.  See w2a8_linear_grouped in include/w2a8.h."""
    M, K = x.shape
    if y is not None:
        grp.bind_outputs(y)
    elif grp.y is None or grp.y[0].shape[0] != M:
        grp.bind_outputs([torch.empty((M, n), dtype=torch.float32, device=x.device) for n in grp.N])
    _check(lib().w2a8_linear_grouped(_ptr(x), _ptr(a), _ptr(a_scale), grp.count, grp._pk, grp._sc, grp._y,
                                     grp._n, M, K, group, fuse, _ptr(workspace),
                                     workspace.numel() * workspace.element_size(), _stream(stream)),
           "w2a8_linear_grouped")
    return grp.y


def w2a8_linear_grouped_host_workspace_bytes(N, M: int, K: int, group: int) -> int:
    arr = (ctypes.c_int * len(N))(*[int(n) for n in N])
    return int(lib().w2a8_linear_grouped_host_workspace_bytes(len(N), arr, M, K, group))


def w2a8_linear_grouped_host(x_host: torch.Tensor, grp: Group, group: int, y_host, workspace: torch.Tensor,
                             stream=None):
    """Host bf16 x [M][K] -> host fp32 y_host[i] [M][N_i] for the matrices of `grp` (device); x is
    brought over and quantised once.  See w2a8_linear_grouped_host in include/w2a8.h."""
    M, K = x_host.shape
    ys = (ctypes.c_void_p * grp.count)(*[_ptr(t) for t in y_host])
    _check(lib().w2a8_linear_grouped_host(_ptr(x_host), M, K, grp.count, grp._pk, grp._sc, grp._n, group, ys,
                                          _ptr(workspace), workspace.numel() * workspace.element_size(),
                                          _stream(stream)), "w2a8_linear_grouped_host")
    return y_host


def w2a8_read_probe(buffer: torch.Tensor, sink: torch.Tensor, stream=None):
    """Enqueue one read-only pass over `buffer` (see w2a8_read_probe in include/w2a8.h)."""
    _check(lib().w2a8_read_probe(_ptr(buffer), buffer.numel() * buffer.element_size(), _ptr(sink),
                                 _stream(stream)), "w2a8_read_probe")


STATIC_SCRATCH_BYTES = 8 << 20


def w2a8_gemm_static(a: torch.Tensor, a_scale: torch.Tensor, packed: torch.Tensor,
                     w_scale: torch.Tensor, group: int, y: torch.Tensor | None = None, stream=None):
    """w2a8_gemm for callers with no workspace to give: the kernel's scratch is a fixed
    array inside the library (at most STATIC_SCRATCH_BYTES; larger problems raise), so
    nothing is allocated on the library side.  Calls share that array: keep them on one
    stream.  See w2a8_gemm_static in include/w2a8.h."""
    M, K = a.shape
    N = packed.shape[0]
    if y is None:
        y = torch.empty((M, N), dtype=torch.float32, device=a.device)
    _check(lib().w2a8_gemm_static(_ptr(a), _ptr(a_scale), _ptr(packed), _ptr(w_scale), _ptr(y), M, N, K,
                                  group, _stream(stream)), "w2a8_gemm_static")
    return y
