"""ctypes binding of the C-ABI library (``include/nm.h``): same names, argument marshalling only.

Every function takes torch CUDA tensors (used purely as device memory) and passes their
``data_ptr()`` plus ``torch.cuda.current_stream().cuda_stream`` to the library.  No step of the
method runs in Python or in torch: if ``libnm_b200.so`` is missing the import fails loudly, and
there is no CPU path.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# NM_LIBRARY selects another build of the same library (e.g. the self-checking libnm_b200_debug.so that
# `python -m paper_2507_17301_b200.build -DNM_DEBUG_BOUNDS` makes)
LIB_PATH = os.environ.get("NM_LIBRARY") or os.path.join(_HERE, "libnm_b200.so")

NM_OK = 0
NM_ERR_INVALID_ARG = -1
NM_ERR_UNSUPPORTED = -2
NM_ERR_CUDA = -3
NM_ERR_ALLOC = -4
NM_ERR_TIMEOUT = -5
NM_ERR_INTERNAL = -6


class NmError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__(f"{_status_string(status)}: {text}")
        self.status = status


class nm_plan_t(ctypes.Structure):
    _fields_ = [("variant", ctypes.c_int), ("bn", ctypes.c_int), ("stages", ctypes.c_int),
                ("split", ctypes.c_int), ("kblk", ctypes.c_int), ("loads", ctypes.c_int),
                ("issuers", ctypes.c_int), ("ksplit", ctypes.c_int), ("reserved", ctypes.c_int * 8)]

    def as_dict(self):
        return {"variant": self.variant, "bn": self.bn, "stages": self.stages, "split": self.split,
                "kblk": self.kblk, "loads": self.loads, "issuers": self.issuers, "ksplit": self.ksplit}


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is not built; run `python -m paper_2507_17301_b200.build` "
            "(there is no fallback path without the CUDA library)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i, fp = ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(ctypes.c_float)
    ip = ctypes.POINTER(ctypes.c_int)
    pp = ctypes.POINTER(nm_plan_t)
    lib.nm_prune.argtypes = [vp, i, i, i, i, i, i, i, vp, ctypes.POINTER(vp)]
    lib.nm_prune_noalloc.argtypes = [vp, i, i, i, i, i, i, i, vp, vp, vp]
    lib.nm_weights_dims.argtypes = [vp, ip, ip, ip, ip, ip]
    lib.nm_weights_export.argtypes = [vp, vp, vp, vp]
    lib.nm_weights_import.argtypes = [vp, vp, i, i, i, i, i, i, i, vp, ctypes.POINTER(vp)]
    lib.nm_weights_check.argtypes = [vp, vp]
    lib.nm_selftest_wait_expiry.argtypes = [vp, vp]
    lib.nm_selftest_wait_expiry.restype = ctypes.c_int
    lib.nm_maxpool2d.argtypes = [vp] + [i] * 10 + [vp, vp]
    lib.nm_maxpool2d.restype = ctypes.c_int
    lib.nm_weights_retained_l1.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
    lib.nm_weights_retained_l1.restype = ctypes.c_int
    lib.nm_plan_scratch_bytes.argtypes = [vp] + [i] * 9 + [pp, ctypes.POINTER(ctypes.c_size_t)]
    lib.nm_weights_reserve.argtypes = [vp, ctypes.c_size_t]
    lib.nm_weights_free.argtypes = [vp]
    conv_geom = [i] * 9
    lib.nm_conv2d.argtypes = [vp, vp] + conv_geom + [vp, i, vp, pp, vp]
    lib.nm_conv2d_res.argtypes = [vp, vp] + conv_geom + [vp, vp, i, vp, pp, vp]
    lib.nm_conv2d_res.restype = ctypes.c_int
    lib.nm_conv2d_host.argtypes = [vp, vp, vp] + conv_geom + [vp, vp, i, vp, vp, pp, vp]
    lib.nm_autotune.argtypes = [vp, vp] + conv_geom + [vp, i, vp, vp, pp, fp]
    lib.nm_autotune_tile.argtypes = [vp, i, i, i, i, i, i, ip, i, vp] + conv_geom + [vp, i, vp, vp, ip, pp, fp]
    for name in ("nm_plan_scratch_bytes", "nm_weights_reserve"):
        getattr(lib, name).restype = ctypes.c_int
    for name in ("nm_prune", "nm_prune_noalloc", "nm_weights_dims", "nm_weights_export", "nm_weights_import", "nm_weights_check",
                 "nm_weights_free", "nm_conv2d", "nm_conv2d_host", "nm_autotune", "nm_autotune_tile"):
        getattr(lib, name).restype = ctypes.c_int
    lib.nm_plan_key.argtypes = [i] * 18 + [ctypes.c_char_p, ctypes.c_size_t]
    lib.nm_plan_key.restype = ctypes.c_int
    lib.nm_plan_cache_store.argtypes = [ctypes.c_char_p, ctypes.c_char_p, pp]
    lib.nm_plan_cache_store.restype = ctypes.c_int
    lib.nm_plan_cache_lookup.argtypes = [ctypes.c_char_p, ctypes.c_char_p, pp]
    lib.nm_plan_cache_lookup.restype = ctypes.c_int
    lib.nm_status_string.argtypes = [ctypes.c_int]
    lib.nm_status_string.restype = ctypes.c_char_p
    lib.nm_last_error.argtypes = []
    lib.nm_last_error.restype = ctypes.c_char_p
    lib.nm_launch_count.argtypes = []
    lib.nm_launch_count.restype = ctypes.c_uint64
    return lib


_lib = _load()

EXPORTS = ("nm_plan_key", "nm_plan_cache_store", "nm_plan_cache_lookup", "nm_selftest_wait_expiry", "nm_maxpool2d", "nm_weights_retained_l1", "nm_conv2d_res", "nm_plan_scratch_bytes", "nm_weights_reserve", "nm_prune", "nm_prune_noalloc", "nm_weights_dims", "nm_weights_export", "nm_weights_import", "nm_weights_check",
           "nm_weights_free", "nm_conv2d", "nm_conv2d_host", "nm_autotune", "nm_autotune_tile",
           "nm_status_string", "nm_last_error", "nm_launch_count")


def _status_string(s: int) -> str:
    return _lib.nm_status_string(s).decode()


def nm_last_error() -> str:
    return _lib.nm_last_error().decode()


def nm_launch_count() -> int:
    return int(_lib.nm_launch_count())


def _check(status: int):
    if status != NM_OK:
        raise NmError(status, nm_last_error())


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dev_f32(t: torch.Tensor, what: str) -> int:
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
        raise TypeError(f"{what} must be a contiguous float32 CUDA tensor")
    return t.data_ptr()


def _pair(v):
    return (v, v) if isinstance(v, int) else (int(v[0]), int(v[1]))


class Weights:
    """Owner of one ``nm_weights_t*`` handle (freed with the object)."""

    def __init__(self, handle: int):
        self._h = ctypes.c_void_p(handle)
        dims = [ctypes.c_int() for _ in range(5)]
        _check(_lib.nm_weights_dims(self._h, *[ctypes.byref(d) for d in dims]))
        self.c_out, self.k, self.kk, self.n_tiles, self.tile_t = (d.value for d in dims)

    @property
    def handle(self):
        return self._h

    def free(self):
        if self._h is not None and self._h.value:
            _lib.nm_weights_free(self._h)
        self._h = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def nm_prune(w_dense: torch.Tensor, n_keep: int, m_group: int, tile_t: int) -> Weights:
    """``w_dense``: CUDA fp32 OHWI ``[c_out, kh, kw, c_in]``.  Returns the compressed-weight handle."""
    ptr = _dev_f32(w_dense, "w_dense")
    if w_dense.dim() != 4:
        raise TypeError("w_dense must be [c_out, kh, kw, c_in]")
    c_out, kh, kw, c_in = w_dense.shape
    out = ctypes.c_void_p()
    _check(_lib.nm_prune(ptr, c_out, kh, kw, c_in, n_keep, m_group, tile_t, _stream(), ctypes.byref(out)))
    return Weights(out.value)


NM_NOALLOC_MAX_CELLS = 1 << 19


def nm_prune_noalloc(w_dense: torch.Tensor, n_keep: int, m_group: int, tile_t: int, values: torch.Tensor,
                     indices: torch.Tensor) -> None:
    """Pruning for callers that must not allocate on the device (a plug-in inside a server that owns
    all GPU memory, a loop that cannot afford cudaMalloc's synchronisation): the caller passes the
    output tensors ``values [c_out, kk]`` fp32 and ``indices [n_tiles, kk]`` uint16, the library uses
    its built-in scratch array and allocates nothing.  Problems with more than
    ``NM_NOALLOC_MAX_CELLS`` (tile, column) cells are refused; calls must not overlap on the GPU."""
    ptr = _dev_f32(w_dense, "w_dense")
    if w_dense.dim() != 4:
        raise TypeError("w_dense must be [c_out, kh, kw, c_in]")
    c_out, kh, kw, c_in = w_dense.shape
    vptr = _dev_f32(values, "values")
    if not (indices.is_cuda and indices.dtype == torch.uint16 and indices.is_contiguous()):
        raise TypeError("indices must be a contiguous uint16 CUDA tensor")
    if n_keep >= 1 and m_group >= n_keep and tile_t >= 1:   # otherwise the library reports the bad argument
        k = kh * kw * c_in
        kk = (k // m_group) * n_keep + min(k % m_group, n_keep)
        n_tiles = -(-c_out // tile_t)
        if values.numel() < c_out * kk or indices.numel() < n_tiles * kk:
            raise TypeError(f"values needs {c_out * kk} elements and indices {n_tiles * kk} "
                            f"(got {values.numel()} and {indices.numel()})")
    _check(_lib.nm_prune_noalloc(ptr, c_out, kh, kw, c_in, n_keep, m_group, tile_t, vptr, indices.data_ptr(),
                                 _stream()))


def nm_weights_export(w: Weights):
    """Returns ``(values [c_out, kk] fp32, indices [n_tiles, kk] uint16)`` as CUDA tensors."""
    values = torch.empty((w.c_out, w.kk), dtype=torch.float32, device="cuda")
    indices = torch.empty((w.n_tiles, w.kk), dtype=torch.uint16, device="cuda")
    _check(_lib.nm_weights_export(w.handle, values.data_ptr(), indices.data_ptr(), _stream()))
    return values, indices


def nm_weights_import(values: torch.Tensor, indices: torch.Tensor, kh: int, kw: int, c_in: int, n_keep: int,
                      m_group: int, tile_t: int) -> Weights:
    vptr = _dev_f32(values, "values")
    if not (indices.is_cuda and indices.dtype == torch.uint16 and indices.is_contiguous()):
        raise TypeError("indices must be a contiguous uint16 CUDA tensor")
    out = ctypes.c_void_p()
    _check(_lib.nm_weights_import(vptr, indices.data_ptr(), values.shape[0], kh, kw, c_in, n_keep, m_group, tile_t,
                                  _stream(), ctypes.byref(out)))
    return Weights(out.value)


def nm_plan_scratch_bytes(w: Weights, x_shape, stride, pad, dil, plan: nm_plan_t) -> int:
    """Scratch bytes `plan` needs on this layer (0 for most plans)."""
    stride, pad, dil = _pair(stride), _pair(pad), _pair(dil)
    b, h, wd, _ = x_shape
    out = ctypes.c_size_t()
    _check(_lib.nm_plan_scratch_bytes(w.handle, b, h, wd, stride[0], stride[1], pad[0], pad[1], dil[0], dil[1],
                                      ctypes.byref(plan), ctypes.byref(out)))
    return int(out.value)


def nm_weights_reserve(w: Weights, nbytes: int):
    """Reserves handle-owned scratch memory (allocates; call outside the timed / captured region)."""
    _check(_lib.nm_weights_reserve(w.handle, nbytes))


def nm_maxpool2d(x: torch.Tensor, kernel=3, stride=2, pad=1, y: torch.Tensor | None = None) -> torch.Tensor:
    """Max pooling of CUDA fp32 NHWC activations; allocates ``y`` unless given."""
    kernel, stride, pad = _pair(kernel), _pair(stride), _pair(pad)
    b, h, wd, c = x.shape
    if y is None:
        ho = (h + 2 * pad[0] - kernel[0]) // stride[0] + 1
        wo = (wd + 2 * pad[1] - kernel[1]) // stride[1] + 1
        y = torch.empty((b, max(ho, 1), max(wo, 1), c), dtype=torch.float32, device=x.device)
    _check(_lib.nm_maxpool2d(_dev_f32(x, "x"), b, h, wd, c, kernel[0], kernel[1], stride[0], stride[1], pad[0], pad[1],
                             _dev_f32(y, "y"), _stream()))
    return y


def nm_weights_retained_l1(w: Weights):
    """Returns ``(kept, total)``: L1 mass of the retained weights and of all weights of the layer."""
    kept, total = ctypes.c_double(), ctypes.c_double()
    _check(_lib.nm_weights_retained_l1(w.handle, ctypes.byref(kept), ctypes.byref(total)))
    return float(kept.value), float(total.value)


def nm_plan_key(c_out, kh, kw, c_in, n_keep, m_group, tile_t, x_shape, stride=1, pad=0, dil=1, has_bias=True,
                relu=False) -> str:
    """Key of a layer in the plan cache file (geometry, pattern, tile width, batch and image size, bias / ReLU)."""
    stride, pad, dil = _pair(stride), _pair(pad), _pair(dil)
    b, h, wd, _ = x_shape
    buf = ctypes.create_string_buffer(384)
    _check(_lib.nm_plan_key(c_out, kh, kw, c_in, n_keep, m_group, tile_t, b, h, wd, stride[0], stride[1], pad[0], pad[1],
                            dil[0], dil[1], int(bool(has_bias)), int(bool(relu)), buf, len(buf)))
    return buf.value.decode()


def nm_plan_cache_store(path: str, key: str, plan: nm_plan_t) -> None:
    _check(_lib.nm_plan_cache_store(path.encode(), key.encode(), ctypes.byref(plan)))


def nm_plan_cache_lookup(path: str, key: str):
    """The cached plan of `key`, or None when the file or the key is missing."""
    plan = nm_plan_t()
    status = _lib.nm_plan_cache_lookup(path.encode(), key.encode(), ctypes.byref(plan))
    if status == NM_ERR_UNSUPPORTED:
        return None
    _check(status)
    return plan


def nm_selftest_wait_expiry(w: Weights):
    """Makes a bounded device-side wait run out on purpose; the next ``nm_weights_check`` raises NM_ERR_TIMEOUT."""
    _check(_lib.nm_selftest_wait_expiry(w.handle, _stream()))


def nm_weights_check(w: Weights):
    _check(_lib.nm_weights_check(w.handle, _stream()))


def out_shape(x_shape, kh, kw, c_out, stride, pad, dil):
    b, h, wd, _ = x_shape
    ho = (h + 2 * pad[0] - dil[0] * (kh - 1) - 1) // stride[0] + 1
    wo = (wd + 2 * pad[1] - dil[1] * (kw - 1) - 1) // stride[1] + 1
    return (b, ho, wo, c_out)


def nm_conv2d(w: Weights, x: torch.Tensor, kh: int, kw: int, stride=1, pad=0, dil=1, bias=None, relu=False,
              y: torch.Tensor | None = None, plan: nm_plan_t | None = None,
              residual: torch.Tensor | None = None) -> torch.Tensor:
    """``x``: CUDA fp32 NHWC.  Allocates ``y`` (NHWC) unless given.  Asynchronous on the current stream.
    With ``residual`` (NHWC, the output's shape) it calls ``nm_conv2d_res``: act(conv + bias + residual)."""
    stride, pad, dil = _pair(stride), _pair(pad), _pair(dil)
    xp = _dev_f32(x, "x")
    b, h, wd, _ = x.shape
    if y is None:
        if min(stride) < 1 or min(dil) < 1:  # let the library report it
            y = torch.empty(4, dtype=torch.float32, device=x.device)
        else:
            shape = out_shape(x.shape, kh, kw, w.c_out, stride, pad, dil)
            y = torch.empty([max(d, 1) for d in shape], dtype=torch.float32, device=x.device)
    yp = _dev_f32(y, "y")
    bp = _dev_f32(bias, "bias") if bias is not None else None
    pl = ctypes.byref(plan) if plan is not None else None
    if residual is None:
        _check(_lib.nm_conv2d(w.handle, xp, b, h, wd, stride[0], stride[1], pad[0], pad[1], dil[0], dil[1], bp,
                              int(bool(relu)), yp, pl, _stream()))
    else:
        if tuple(residual.shape) != tuple(y.shape):
            raise TypeError("residual must have the output's shape")
        _check(_lib.nm_conv2d_res(w.handle, xp, b, h, wd, stride[0], stride[1], pad[0], pad[1], dil[0], dil[1], bp,
                                  _dev_f32(residual, "residual"), int(bool(relu)), yp, pl, _stream()))
    return y


def nm_conv2d_host(w: Weights, x_host: torch.Tensor, x_dev: torch.Tensor, stride, pad, dil, bias_host, bias_dev,
                   relu, y_host: torch.Tensor, y_dev: torch.Tensor, plan: nm_plan_t | None = None):
    """Host-buffer form: H2D(x, bias) -> conv -> D2H(y) on the current stream (no synchronisation)."""
    stride, pad, dil = _pair(stride), _pair(pad), _pair(dil)
    b, h, wd, _ = x_host.shape
    for t, what in ((x_host, "x_host"), (y_host, "y_host")):
        if t.is_cuda or t.dtype != torch.float32 or not t.is_contiguous():
            raise TypeError(f"{what} must be a contiguous float32 host tensor")
    _check(_lib.nm_conv2d_host(
        w.handle, x_host.data_ptr(), _dev_f32(x_dev, "x_dev"), b, h, wd, stride[0], stride[1], pad[0], pad[1],
        dil[0], dil[1], bias_host.data_ptr() if bias_host is not None else None,
        _dev_f32(bias_dev, "bias_dev") if bias_dev is not None else None, int(bool(relu)), y_host.data_ptr(),
        _dev_f32(y_dev, "y_dev"), ctypes.byref(plan) if plan is not None else None, _stream()))


def nm_autotune(w: Weights, x: torch.Tensor, stride=1, pad=0, dil=1, bias=None, relu=False,
                y_scratch: torch.Tensor | None = None, kh: int = 1, kw: int = 1):
    """Returns ``(plan, milliseconds)`` of the fastest candidate for this layer."""
    stride, pad, dil = _pair(stride), _pair(pad), _pair(dil)
    b, h, wd, _ = x.shape
    if y_scratch is None:
        y_scratch = torch.empty(out_shape(x.shape, kh, kw, w.c_out, stride, pad, dil), dtype=torch.float32,
                                device=x.device)
    plan = nm_plan_t()
    ms = ctypes.c_float()
    _check(_lib.nm_autotune(w.handle, _dev_f32(x, "x"), b, h, wd, stride[0], stride[1], pad[0], pad[1], dil[0],
                            dil[1], _dev_f32(bias, "bias") if bias is not None else None, int(bool(relu)),
                            _dev_f32(y_scratch, "y_scratch"), _stream(), ctypes.byref(plan), ctypes.byref(ms)))
    return plan, float(ms.value)


def nm_autotune_tile(w_dense: torch.Tensor, n_keep: int, m_group: int, tile_candidates, x: torch.Tensor, stride=1,
                     pad=0, dil=1, bias=None, relu=False, y_scratch: torch.Tensor | None = None):
    """Returns ``(tile_t, plan, milliseconds)``: the fastest pruning tile width and its plan."""
    stride, pad, dil = _pair(stride), _pair(pad), _pair(dil)
    c_out, kh, kw, c_in = w_dense.shape
    b, h, wd, _ = x.shape
    if y_scratch is None:
        y_scratch = torch.empty(out_shape(x.shape, kh, kw, c_out, stride, pad, dil), dtype=torch.float32,
                                device=x.device)
    cands = (ctypes.c_int * len(tile_candidates))(*tile_candidates)
    plan, ms, tile = nm_plan_t(), ctypes.c_float(), ctypes.c_int()
    _check(_lib.nm_autotune_tile(_dev_f32(w_dense, "w_dense"), c_out, kh, kw, c_in, n_keep, m_group, cands,
                                 len(tile_candidates), _dev_f32(x, "x"), b, h, wd, stride[0], stride[1], pad[0],
                                 pad[1], dil[0], dil[1], _dev_f32(bias, "bias") if bias is not None else None,
                                 int(bool(relu)), _dev_f32(y_scratch, "y_scratch"), _stream(), ctypes.byref(tile),
                                 ctypes.byref(plan), ctypes.byref(ms)))
    return int(tile.value), plan, float(ms.value)
