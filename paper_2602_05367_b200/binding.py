"""ctypes binding of the C ABI in include/rabit.h.  Marshalling only: every step of the layer
runs inside the CUDA library."""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# RABIT_LIBRARY selects another build of the same library (e.g. librabit_trace.so, built with --trace)
_LIB_PATH = os.environ.get("RABIT_LIBRARY") or os.path.join(_HERE, "librabit.so")

_c_void_p = ctypes.c_void_p
_c_int = ctypes.c_int
_c_size_t = ctypes.c_size_t


class RabitError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"rabit error {code}: {message}")
        self.code = code


def _load() -> ctypes.CDLL:
    if not os.path.exists(_LIB_PATH):
        raise ImportError(
            f"{_LIB_PATH} is missing: build it with `python paper_2602_05367_b200/build.py` "
            "(there is no CPU fallback)")
    lib = ctypes.CDLL(_LIB_PATH)
    lib.rabit_layout_version.restype = _c_int
    lib.rabit_packed_bytes.restype = _c_size_t
    lib.rabit_packed_bytes.argtypes = [_c_int, _c_int, _c_int]
    lib.rabit_pack_host.restype = _c_int
    lib.rabit_pack_host.argtypes = [_c_void_p, _c_void_p, _c_void_p, _c_int, _c_int, _c_int, _c_void_p, _c_size_t]
    lib.rabit_unpack_host.restype = _c_int
    lib.rabit_unpack_host.argtypes = [_c_void_p, _c_size_t, _c_void_p, _c_void_p, _c_void_p]
    lib.rabit_pack.restype = _c_int
    lib.rabit_pack.argtypes = [_c_void_p, _c_void_p, _c_void_p, _c_int, _c_int, _c_int, _c_void_p, _c_size_t,
                               _c_void_p, ctypes.POINTER(_c_void_p)]
    lib.rabit_derive_pack.restype = _c_int
    lib.rabit_derive_pack.argtypes = [_c_void_p, _c_void_p, _c_void_p, _c_int, _c_int, _c_int, _c_void_p, _c_size_t,
                                      _c_void_p, ctypes.POINTER(_c_void_p)]
    lib.rabit_linear.restype = _c_int
    lib.rabit_linear.argtypes = [_c_void_p, _c_void_p, _c_void_p, _c_int, _c_void_p]
    lib.rabit_stage_bytes.restype = _c_size_t
    lib.rabit_stage_bytes.argtypes = [_c_void_p, _c_int]
    lib.rabit_linear_host.restype = _c_int
    lib.rabit_linear_host.argtypes = [_c_void_p, _c_void_p, _c_void_p, _c_int, _c_void_p, _c_size_t, _c_void_p]
    lib.rabit_linear_group.restype = _c_int
    lib.rabit_linear_group.argtypes = [_c_void_p, _c_void_p, _c_void_p, _c_int, _c_int, _c_void_p]
    lib.rabit_linear_static_scratch.restype = _c_int
    lib.rabit_linear_static_scratch.argtypes = [_c_void_p, _c_void_p, _c_void_p, _c_int, _c_void_p]
    lib.rabit_group_stage_bytes.restype = _c_size_t
    lib.rabit_group_stage_bytes.argtypes = [_c_void_p, _c_int, _c_int]
    lib.rabit_linear_group_host.restype = _c_int
    lib.rabit_linear_group_host.argtypes = [_c_void_p, _c_void_p, _c_void_p, _c_int, _c_int, _c_void_p, _c_size_t, _c_void_p]
    lib.rabit_layer_status.restype = _c_int
    lib.rabit_layer_status.argtypes = [_c_void_p, _c_int, _c_void_p]
    lib.rabit_selftest_bounded_wait.restype = _c_int
    lib.rabit_selftest_bounded_wait.argtypes = [_c_void_p, _c_int, _c_void_p]
    lib.rabit_selftest_f16_plan.restype = _c_int
    lib.rabit_selftest_f16_plan.argtypes = [_c_int, _c_int, _c_int, _c_int, _c_int, _c_void_p, _c_int]
    lib.rabit_selftest_stream_read.restype = _c_int
    lib.rabit_selftest_stream_read.argtypes = [_c_void_p, _c_size_t, _c_void_p, _c_void_p]
    lib.rabit_unpack.restype = _c_int
    lib.rabit_unpack.argtypes = [_c_void_p, _c_void_p, _c_void_p, _c_void_p, _c_void_p]
    for name in ("rabit_layer_K", "rabit_layer_M", "rabit_layer_N"):
        getattr(lib, name).restype = _c_int
        getattr(lib, name).argtypes = [_c_void_p]
    lib.rabit_set_variant.restype = _c_int
    lib.rabit_set_variant.argtypes = [_c_void_p, _c_int]
    lib.rabit_free.restype = _c_int
    lib.rabit_free.argtypes = [_c_void_p]
    lib.rabit_trace_begin.restype = _c_int
    lib.rabit_trace_begin.argtypes = [_c_void_p, _c_size_t]
    lib.rabit_trace_launches.restype = _c_int
    lib.rabit_trace_launches.argtypes = [_c_void_p, _c_int]
    lib.rabit_last_error.restype = ctypes.c_char_p
    return lib


_lib = _load()


def lib_path() -> str:
    return _LIB_PATH


def raw_lib() -> ctypes.CDLL:
    """The loaded CDLL, for tests that exercise the ABI with raw pointers."""
    return _lib


def last_error() -> str:
    return _lib.rabit_last_error().decode()


def _check(rc: int) -> None:
    if rc != 0:
        raise RabitError(rc, last_error())


def layout_version() -> int:
    return int(_lib.rabit_layout_version())


def packed_bytes(K: int, M: int, N: int) -> int:
    return int(_lib.rabit_packed_bytes(K, M, N))


def _host_arrays(planes, g, h) -> Tuple[np.ndarray, np.ndarray, np.ndarray, int, int, int]:
    planes = np.ascontiguousarray(planes, dtype=np.uint32)
    g16 = np.ascontiguousarray(g, dtype=np.float16).view(np.uint16)
    h16 = np.ascontiguousarray(h, dtype=np.float16).view(np.uint16)
    if planes.ndim != 3 or g16.ndim != 2 or h16.ndim != 2:
        raise ValueError("planes must be [K][M][N/32], g [K][M], h [K][N]")
    K, M, W = planes.shape
    N = h16.shape[1]
    if g16.shape != (K, M) or h16.shape[0] != K or W * 32 != N:
        raise ValueError("inconsistent shapes between planes, g and h")
    return planes, g16, h16, K, M, N


def pack_host(planes, g, h) -> np.ndarray:
    """Packed image as a uint8 array (no GPU needed)."""
    planes, g16, h16, K, M, N = _host_arrays(planes, g, h)
    nbytes = packed_bytes(K, M, N)
    if nbytes == 0:
        raise RabitError(-2, f"unsupported shape K={K} M={M} N={N}")
    out = np.empty(nbytes, dtype=np.uint8)
    _check(_lib.rabit_pack_host(planes.ctypes.data, g16.ctypes.data, h16.ctypes.data, K, M, N,
                                out.ctypes.data, out.nbytes))
    return out


def unpack_host(image: np.ndarray, K: int, M: int, N: int):
    image = np.ascontiguousarray(image, dtype=np.uint8)
    planes = np.empty((K, M, N // 32), dtype=np.uint32)
    g = np.empty((K, M), dtype=np.uint16)
    h = np.empty((K, N), dtype=np.uint16)
    _check(_lib.rabit_unpack_host(image.ctypes.data, image.nbytes, planes.ctypes.data, g.ctypes.data, h.ctypes.data))
    return planes, g.view(np.float16), h.view(np.float16)


class RabitLayer:
    """Owns one descriptor and the torch buffer that holds its packed image."""

    def __init__(self, handle: int, dev_buf, K: int, M: int, N: int):
        self._handle = _c_void_p(handle)
        self.dev_buf = dev_buf          # keeps the device memory alive
        self.K, self.M, self.N = K, M, N
        self._stage = None              # device staging buffer of rabit_linear_host

    @property
    def handle(self) -> ctypes.c_void_p:
        if self._handle is None:
            raise RabitError(-1, "layer already freed")
        return self._handle

    def set_variant(self, variant: int) -> None:
        """Kernel family for later rabit_linear calls of this layer: 0 automatic, 1 plain, 2 integer tensor-core GEMV,
        3 tcgen05 GEMM (exact expansion), 4 tcgen05 GEMM on dequantised fp16 weight tiles (never chosen automatically),
        5 table-driven GEMV."""
        _check(_lib.rabit_set_variant(self.handle, variant))

    def status(self, clear: bool = False, stream: int = 0) -> int:
        """0 if every kernel of this layer completed its waits, RABIT_DEVICE_FAULT (-5) otherwise; synchronises."""
        return int(_lib.rabit_layer_status(self.handle, 1 if clear else 0, _c_void_p(stream)))

    def unpack(self, stream: int = 0):
        planes = np.empty((self.K, self.M, self.N // 32), dtype=np.uint32)
        g = np.empty((self.K, self.M), dtype=np.uint16)
        h = np.empty((self.K, self.N), dtype=np.uint16)
        _check(_lib.rabit_unpack(self.handle, planes.ctypes.data, g.ctypes.data, h.ctypes.data, _c_void_p(stream)))
        return planes, g.view(np.float16), h.view(np.float16)

    def free(self) -> None:
        if self._handle is not None:
            _lib.rabit_free(self._handle)
            self._handle = None
            self.dev_buf = None
            self._stage = None

    def __del__(self):  # pragma: no cover
        try:
            self.free()
        except Exception:
            pass


def rabit_pack(planes, g, h, device="cuda:0", stream: Optional[int] = None) -> RabitLayer:
    """Pack on the host, upload into a torch-allocated device buffer, return the layer."""
    import torch

    planes, g16, h16, K, M, N = _host_arrays(planes, g, h)
    nbytes = packed_bytes(K, M, N)
    if nbytes == 0:
        raise RabitError(-2, f"unsupported shape K={K} M={M} N={N}")
    dev = torch.device(device)
    buf = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    st = torch.cuda.current_stream(dev).cuda_stream if stream is None else stream
    out = _c_void_p()
    with torch.cuda.device(dev):
        _check(_lib.rabit_pack(planes.ctypes.data, g16.ctypes.data, h16.ctypes.data, K, M, N,
                               _c_void_p(buf.data_ptr()), nbytes, _c_void_p(st), ctypes.byref(out)))
    return RabitLayer(out.value, buf, K, M, N)


def rabit_derive_pack(W, g, h, stream: Optional[int] = None) -> RabitLayer:
    """Derive the sign planes of every path from the CUDA float32 weight W [M][N] and the fp16 scales
    g [K][M], h [K][N] (host arrays) on the device, packed in place; returns the layer."""
    import torch

    if W.dtype != torch.float32 or not W.is_cuda or not W.is_contiguous() or W.dim() != 2:
        raise ValueError("W must be a contiguous CUDA float32 matrix")
    g16 = np.ascontiguousarray(g, dtype=np.float16).view(np.uint16)
    h16 = np.ascontiguousarray(h, dtype=np.float16).view(np.uint16)
    K, M = g16.shape
    N = h16.shape[1]
    if tuple(W.shape) != (M, N) or h16.shape[0] != K:
        raise ValueError("inconsistent shapes between W, g and h")
    nbytes = packed_bytes(K, M, N)
    if nbytes == 0:
        raise RabitError(-2, f"unsupported shape K={K} M={M} N={N}")
    buf = torch.empty(nbytes, dtype=torch.uint8, device=W.device)
    st = torch.cuda.current_stream(W.device).cuda_stream if stream is None else stream
    out = _c_void_p()
    with torch.cuda.device(W.device):
        _check(_lib.rabit_derive_pack(_c_void_p(W.data_ptr()), g16.ctypes.data, h16.ctypes.data, K, M, N,
                                      _c_void_p(buf.data_ptr()), nbytes, _c_void_p(st), ctypes.byref(out)))
    return RabitLayer(out.value, buf, K, M, N)


def rabit_linear(layer: RabitLayer, x, y=None, stream: Optional[int] = None):
    """y[b] = layer(x[b]); x is a CUDA fp16 tensor [batch][N] (or [N]); returns y [batch][M]."""
    import torch

    if x.dtype != torch.float16 or not x.is_cuda or not x.is_contiguous():
        raise ValueError("x must be a contiguous CUDA float16 tensor")
    xb = x if x.dim() == 2 else x.view(1, -1)
    if xb.shape[1] != layer.N:
        raise ValueError(f"x has {xb.shape[1]} columns, layer expects {layer.N}")
    batch = xb.shape[0]
    if y is None:
        y = torch.empty((batch, layer.M), dtype=torch.float16, device=x.device)
    elif y.dtype != torch.float16 or not y.is_cuda or not y.is_contiguous() or y.numel() != batch * layer.M:
        raise ValueError("y must be a contiguous CUDA float16 tensor of batch*M elements")
    st = torch.cuda.current_stream(x.device).cuda_stream if stream is None else stream
    _check(_lib.rabit_linear(layer.handle, _c_void_p(xb.data_ptr()), _c_void_p(y.data_ptr()), batch, _c_void_p(st)))
    return y if x.dim() == 2 else y.view(-1)


def rabit_linear_group(layers, xs, ys, stream: Optional[int] = None):
    """Independent layers in one launch: ys[l] = layers[l](xs[l]).  xs may repeat one tensor (projections
    that share their input).  All tensors are contiguous CUDA float16, [batch][N_l] and [batch][M_l]."""
    import torch

    n = len(layers)
    if n < 1 or len(xs) != n or len(ys) != n:
        raise ValueError("layers, xs and ys must have the same, non-zero length")
    batch = 1 if xs[0].dim() == 1 else xs[0].shape[0]
    for L, x, y in zip(layers, xs, ys):
        if x.dtype != torch.float16 or not x.is_cuda or not x.is_contiguous() or x.numel() != batch * L.N:
            raise ValueError("every x must be a contiguous CUDA float16 tensor of batch*N elements")
        if y.dtype != torch.float16 or not y.is_cuda or not y.is_contiguous() or y.numel() != batch * L.M:
            raise ValueError("every y must be a contiguous CUDA float16 tensor of batch*M elements")
    st = torch.cuda.current_stream(xs[0].device).cuda_stream if stream is None else stream
    h = (_c_void_p * n)(*[L.handle for L in layers])
    xp = (_c_void_p * n)(*[x.data_ptr() for x in xs])
    yp = (_c_void_p * n)(*[y.data_ptr() for y in ys])
    _check(_lib.rabit_linear_group(h, xp, yp, n, batch, _c_void_p(st)))
    return ys


def rabit_linear_group_host(layers, xs_host, ys_host, stream: Optional[int] = None):
    """Host-buffer form of rabit_linear_group: CPU float16 tensors in and out (pinned for asynchronous copies);
    an input tensor that occurs several times is copied once.  Returns without synchronising."""
    import torch

    n = len(layers)
    if n < 1 or len(xs_host) != n or len(ys_host) != n:
        raise ValueError("layers, xs_host and ys_host must have the same, non-zero length")
    batch = 1 if xs_host[0].dim() == 1 else xs_host[0].shape[0]
    for L, x, y in zip(layers, xs_host, ys_host):
        if x.dtype != torch.float16 or x.is_cuda or not x.is_contiguous() or x.numel() != batch * L.N:
            raise ValueError("every x must be a contiguous CPU float16 tensor of batch*N elements")
        if y.dtype != torch.float16 or y.is_cuda or not y.is_contiguous() or y.numel() != batch * L.M:
            raise ValueError("every y must be a contiguous CPU float16 tensor of batch*M elements")
    h = (_c_void_p * n)(*[L.handle for L in layers])
    need = int(_lib.rabit_group_stage_bytes(h, n, batch))
    first = layers[0]
    if first._stage is None or first._stage.numel() < need:
        first._stage = torch.empty(need, dtype=torch.uint8, device=first.dev_buf.device)
    st = torch.cuda.current_stream(first.dev_buf.device).cuda_stream if stream is None else stream
    xp = (_c_void_p * n)(*[x.data_ptr() for x in xs_host])
    yp = (_c_void_p * n)(*[y.data_ptr() for y in ys_host])
    _check(_lib.rabit_linear_group_host(h, xp, yp, n, batch, _c_void_p(first._stage.data_ptr()), need, _c_void_p(st)))
    return ys_host


class PreparedGroupHost:
    """A rabit_linear_group_host call with its arguments checked and marshalled once: calling the object enqueues
    the same copies and launch again on the given stream (the tensors are kept alive and read / written in place),
    without the per-call checks of rabit_linear_group_host.  Returns without synchronising."""

    def __init__(self, layers, xs_host, ys_host):
        import torch

        n = len(layers)
        if n < 1 or len(xs_host) != n or len(ys_host) != n:
            raise ValueError("layers, xs_host and ys_host must have the same, non-zero length")
        batch = 1 if xs_host[0].dim() == 1 else xs_host[0].shape[0]
        for L, x, y in zip(layers, xs_host, ys_host):
            if x.dtype != torch.float16 or x.is_cuda or not x.is_contiguous() or x.numel() != batch * L.N:
                raise ValueError("every x must be a contiguous CPU float16 tensor of batch*N elements")
            if y.dtype != torch.float16 or y.is_cuda or not y.is_contiguous() or y.numel() != batch * L.M:
                raise ValueError("every y must be a contiguous CPU float16 tensor of batch*M elements")
        self._keep = (list(layers), list(xs_host), list(ys_host))
        self._device = layers[0].dev_buf.device
        self._h = (_c_void_p * n)(*[L.handle for L in layers])
        self._xp = (_c_void_p * n)(*[x.data_ptr() for x in xs_host])
        self._yp = (_c_void_p * n)(*[y.data_ptr() for y in ys_host])
        self._n, self._batch = n, batch
        self._need = int(_lib.rabit_group_stage_bytes(self._h, n, batch))
        self._stage = torch.empty(self._need, dtype=torch.uint8, device=self._device)
        self._stage_ptr = _c_void_p(self._stage.data_ptr())
        self.ys_host = ys_host

    def __call__(self, stream: Optional[int] = None):
        if stream is None:
            import torch
            stream = torch.cuda.current_stream(self._device).cuda_stream
        rc = _lib.rabit_linear_group_host(self._h, self._xp, self._yp, self._n, self._batch, self._stage_ptr, self._need, _c_void_p(stream))
        if rc != 0:
            _check(rc)
        return self.ys_host


def rabit_linear_host(layer: RabitLayer, x_host, y_host, stream: Optional[int] = None):
    """Host-buffer form: x_host / y_host are CPU float16 tensors (pinned for asynchronous copies)
    of shape [batch][N] (or [N]) and [batch][M]; the copies and the kernel are enqueued on the
    stream and the call returns without synchronising."""
    import torch

    if x_host.dtype != torch.float16 or x_host.is_cuda or not x_host.is_contiguous():
        raise ValueError("x_host must be a contiguous CPU float16 tensor")
    if y_host.dtype != torch.float16 or y_host.is_cuda or not y_host.is_contiguous():
        raise ValueError("y_host must be a contiguous CPU float16 tensor")
    batch = 1 if x_host.dim() == 1 else x_host.shape[0]
    if x_host.numel() != batch * layer.N or y_host.numel() != batch * layer.M:
        raise ValueError("x_host / y_host sizes do not match the layer")
    need = int(_lib.rabit_stage_bytes(layer.handle, batch))
    if layer._stage is None or layer._stage.numel() < need:
        layer._stage = torch.empty(need, dtype=torch.uint8, device=layer.dev_buf.device)
    st = torch.cuda.current_stream(layer.dev_buf.device).cuda_stream if stream is None else stream
    _check(_lib.rabit_linear_host(layer.handle, _c_void_p(x_host.data_ptr()), _c_void_p(y_host.data_ptr()), batch,
                                  _c_void_p(layer._stage.data_ptr()), need, _c_void_p(st)))
    return y_host


def rabit_linear_static_scratch(layer: RabitLayer, x, y, stream: Optional[int] = None):
    """rabit_linear for batch 1..16 that keeps its reduction scratch in the library's own fixed
    4 MiB device array, so nothing is allocated for the call (the caller passes x and y).  All
    calls share that array: keep them on one stream."""
    import torch

    if x.dtype != torch.float16 or not x.is_cuda or not x.is_contiguous():
        raise ValueError("x must be a contiguous CUDA float16 tensor")
    if y.dtype != torch.float16 or not y.is_cuda or not y.is_contiguous():
        raise ValueError("y must be a contiguous CUDA float16 tensor")
    batch = 1 if x.dim() == 1 else x.shape[0]
    if x.numel() != batch * layer.N or y.numel() != batch * layer.M:
        raise ValueError("x / y sizes do not match the layer")
    st = torch.cuda.current_stream(x.device).cuda_stream if stream is None else stream
    with torch.cuda.device(x.device):
        _check(_lib.rabit_linear_static_scratch(layer.handle, _c_void_p(x.data_ptr()), _c_void_p(y.data_ptr()), batch, _c_void_p(st)))
    return y


def rabit_free(layer: RabitLayer) -> None:
    layer.free()
