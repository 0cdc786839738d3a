"""CPU oracle (test infrastructure only) for column-wise N:M pruning + sparse conv.

Thin ctypes loader around ``nm_oracle.c``.  It compiles the C file with gcc on first
use and exposes numpy-in / numpy-out wrappers.  Nothing here is used by, imported
from, or shared with the CUDA library: tests, the smoke check and the CPU-baseline
leg of the benchmark are the only callers.

Each wrapper names the passage of the paper its C function follows; the C file's
header lists the readings taken where the paper is silent and the pins that hold
the oracle to something other than itself.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "nm_oracle.c")
_LIB_PATH = os.path.join(_HERE, "libnm_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile ``nm_oracle.c`` into ``libnm_oracle.so`` beside it (gcc, -O2, OpenMP)."""
    stale = (not os.path.exists(_LIB_PATH)) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB_PATH + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-Wall", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        fp = ctypes.POINTER(ctypes.c_float)
        up = ctypes.POINTER(ctypes.c_uint16)
        i = ctypes.c_int
        lib.nm_oracle_kept_count.argtypes = [i, i, i]
        lib.nm_oracle_kept_count.restype = i
        lib.nm_oracle_threads.argtypes = []
        lib.nm_oracle_threads.restype = i
        lib.nm_oracle_prune.argtypes = [fp, i, i, i, i, i, fp, up]
        lib.nm_oracle_prune.restype = i
        lib.nm_oracle_expand.argtypes = [fp, up, i, i, i, i, fp]
        lib.nm_oracle_expand.restype = i
        lib.nm_oracle_conv2d.argtypes = [fp, up] + [i] * 6 + [fp] + [i] * 9 + [fp, i, fp]
        lib.nm_oracle_conv2d.restype = i
        lib.nm_oracle_conv2d_res.argtypes = [fp, up] + [i] * 6 + [fp] + [i] * 9 + [fp, fp, i, fp]
        lib.nm_oracle_conv2d_res.restype = i
        lib.nm_oracle_maxpool2d.argtypes = [fp] + [i] * 10 + [fp]
        lib.nm_oracle_maxpool2d.restype = i
        _lib = lib
    return _lib


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))


def _u16(a):
    a = np.ascontiguousarray(a, dtype=np.uint16)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16))


def threads() -> int:
    """Threads the conv oracle's outer loop runs on (OpenMP default)."""
    return int(_load().nm_oracle_threads())


def kept_count(k: int, n_keep: int, m_group: int) -> int:
    """Columns retained out of ``k``: N per full group of M (Sec. 2.1, Sec. 3.1)."""
    return int(_load().nm_oracle_kept_count(k, n_keep, m_group))


def prune(w: np.ndarray, n_keep: int, m_group: int, tile_t: int):
    """Column-wise N:M pruning at tile level (Sec. 3.1; compressed form of Sec. 2.1).

    ``w``: dense fp32 weights ``[c_out, kh, kw, c_in]`` (OHWI) or already flat ``[c_out, k]``.
    Returns ``(values [c_out, kk] fp32, indices [n_tiles, kk] uint16)``.
    """
    w = np.asarray(w, dtype=np.float32)
    c_out = w.shape[0]
    w2, wp = _f32(w.reshape(c_out, -1))
    k = w2.shape[1]
    if n_keep < 1 or m_group < n_keep or tile_t < 1:
        raise ValueError("need 1 <= n_keep <= m_group and tile_t >= 1")
    kk = kept_count(k, n_keep, m_group)
    n_tiles = -(-c_out // tile_t)
    values = np.zeros((c_out, kk), dtype=np.float32)
    indices = np.zeros((n_tiles, kk), dtype=np.uint16)
    rc = _load().nm_oracle_prune(
        wp, c_out, k, n_keep, m_group, tile_t,
        values.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
        indices.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16)),
    )
    if rc != kk:
        raise ValueError(f"nm_oracle_prune rejected its arguments (rc={rc})")
    return values, indices


def expand(values: np.ndarray, indices: np.ndarray, k: int, tile_t: int) -> np.ndarray:
    """Zero-expand the compressed form back to dense ``[c_out, k]`` (Fig. 1 reversed)."""
    values, vp = _f32(values)
    indices, ip = _u16(indices)
    c_out, kk = values.shape
    out = np.empty((c_out, k), dtype=np.float32)
    rc = _load().nm_oracle_expand(vp, ip, c_out, k, kk, tile_t,
                                  out.ctypes.data_as(ctypes.POINTER(ctypes.c_float)))
    if rc != 0:
        raise ValueError("nm_oracle_expand rejected its arguments")
    return out


def conv2d_res(values, indices, kh, kw, c_in, tile_t, x, stride=(1, 1), pad=(0, 0), dil=(1, 1),
               bias=None, residual=None, relu=False) -> np.ndarray:
    """``conv2d`` followed by the shortcut addition of a residual block before the activation
    (the block structure of the ResNets measured in Sec. 4.5): ``act(conv + bias + residual)``,
    the addition in fp64 before the single rounding.  ``residual``: NHWC fp32 of the output's shape."""
    values, vp = _f32(values)
    indices, ip = _u16(indices)
    x, xp = _f32(x)
    c_out, kk = values.shape
    b, h, w, ci = x.shape
    if ci != c_in:
        raise ValueError("x channel count does not match c_in")
    ho = (h + 2 * pad[0] - dil[0] * (kh - 1) - 1) // stride[0] + 1
    wo = (w + 2 * pad[1] - dil[1] * (kw - 1) - 1) // stride[1] + 1
    y = np.empty((b, ho, wo, c_out), dtype=np.float32)
    null = ctypes.POINTER(ctypes.c_float)()
    bp = null
    if bias is not None:
        bias, bp = _f32(bias)
    rp = null
    if residual is not None:
        residual, rp = _f32(residual)
        if residual.shape != y.shape:
            raise ValueError("residual must have the output's shape")
    rc = _load().nm_oracle_conv2d_res(
        vp, ip, c_out, kh, kw, c_in, kk, tile_t, xp, b, h, w,
        stride[0], stride[1], pad[0], pad[1], dil[0], dil[1], bp, rp, int(bool(relu)),
        y.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
    )
    if rc != 0:
        raise ValueError("nm_oracle_conv2d_res rejected its arguments")
    return y


def conv2d(values, indices, kh, kw, c_in, tile_t, x, stride=(1, 1), pad=(0, 0), dil=(1, 1),
           bias=None, relu=False) -> np.ndarray:
    """Sparse conv on the retained columns (Algorithm 1 over the patch matrix of Sec. 2.2).

    ``x``: NHWC fp32 ``[batch, h, w, c_in]``.  Returns NHWC fp32 ``[batch, ho, wo, c_out]``;
    fp64 products and sum in ascending retained-column order, one rounding at the end.
    """
    values, vp = _f32(values)
    indices, ip = _u16(indices)
    x, xp = _f32(x)
    c_out, kk = values.shape
    b, h, w, ci = x.shape
    if ci != c_in:
        raise ValueError("x channel count does not match c_in")
    ho = (h + 2 * pad[0] - dil[0] * (kh - 1) - 1) // stride[0] + 1
    wo = (w + 2 * pad[1] - dil[1] * (kw - 1) - 1) // stride[1] + 1
    y = np.empty((b, ho, wo, c_out), dtype=np.float32)
    if bias is not None:
        bias, bp = _f32(bias)
    else:
        bp = ctypes.POINTER(ctypes.c_float)()
    rc = _load().nm_oracle_conv2d(
        vp, ip, c_out, kh, kw, c_in, kk, tile_t, xp, b, h, w,
        stride[0], stride[1], pad[0], pad[1], dil[0], dil[1], bp, int(bool(relu)),
        y.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
    )
    if rc != 0:
        raise ValueError("nm_oracle_conv2d rejected its arguments")
    return y


def maxpool2d(x, kernel=(3, 3), stride=(2, 2), pad=(1, 1)) -> np.ndarray:
    """Max pooling over NHWC fp32 (between the stem and the first block of the ResNets of Sec. 4.5);
    window positions outside the image do not take part."""
    x, xp = _f32(x)
    b, h, w, c = x.shape
    ho = (h + 2 * pad[0] - kernel[0]) // stride[0] + 1
    wo = (w + 2 * pad[1] - kernel[1]) // stride[1] + 1
    if ho < 1 or wo < 1:
        raise ValueError("the window does not fit the padded image")
    y = np.empty((b, ho, wo, c), dtype=np.float32)
    rc = _load().nm_oracle_maxpool2d(xp, b, h, w, c, kernel[0], kernel[1], stride[0], stride[1], pad[0], pad[1],
                                     y.ctypes.data_as(ctypes.POINTER(ctypes.c_float)))
    if rc != 0:
        raise ValueError("nm_oracle_maxpool2d rejected its arguments")
    return y
