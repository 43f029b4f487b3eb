"""ctypes front end of the CPU oracle (``f8ref.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library never imports this module and
this module never imports the CUDA binding; the only thing both sides share is
the seeded input generator (layer descriptions and integer tensors).

``build()`` compiles ``f8ref.c`` with gcc into ``libf8ref.so`` next to it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "f8ref.c")
_LIB = os.path.join(_HERE, "libf8ref.so")
_lib = None

# dtype / layer-kind codes of the layer descriptions: defined once, by the input generator
from paper_2202_05239_b200.synth import U8, S8, S32, CONV, DWCONV, MAXPOOL, GAP, LINEAR, SIBLING  # noqa: E402


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-Wall", "-Wextra",
                               "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.f8ref_shift_round_clip.restype = ctypes.c_int64
        _lib.f8ref_shift_round_clip.argtypes = [ctypes.c_int64, ctypes.c_int, ctypes.c_int64, ctypes.c_int64]
    return _lib


def threads() -> int:
    """Threads the OpenMP loops will use (the affinity mask unless OMP_NUM_THREADS says otherwise)."""
    env = os.environ.get("OMP_NUM_THREADS")
    return int(env) if env else len(os.sched_getaffinity(0))


def _ptr(a: Optional[np.ndarray]):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.c_void_p)


_NP = {U8: np.uint8, S8: np.int8, S32: np.int32}


def _dtype_code(a: np.ndarray) -> int:
    return {np.dtype(np.uint8): U8, np.dtype(np.int8): S8}[a.dtype]


def _check(status: int, what: str):
    if status != 0:
        raise RuntimeError(f"oracle {what} failed with status {status}"
                           + (" (accumulator outside int32)" if status == 2 else ""))


def shift_round_clip(acc: int, s: int, lo: int, hi: int) -> int:
    return int(lib().f8ref_shift_round_clip(acc, s, lo, hi))


def conv2d(x, w, bias, *, stride, pad, fl_x, fl_w, fl_y, y_dtype, residual=None, fl_r=0):
    n, h, wd, ci = x.shape
    co, kh, kw, ci2 = w.shape
    assert ci2 == ci and w.dtype == np.int8
    ho, wo = (h + 2 * pad - kh) // stride + 1, (wd + 2 * pad - kw) // stride + 1
    y = np.empty((n, ho, wo, co), dtype=_NP[y_dtype])
    if residual is not None:
        assert residual.shape == y.shape
    st = lib().f8ref_conv2d(n, h, wd, ci, co, kh, kw, stride, pad, _dtype_code(x), fl_x, fl_w, fl_y, y_dtype,
                            _ptr(x), _ptr(w), _ptr(bias), _ptr(residual),
                            _dtype_code(residual) if residual is not None else 0, fl_r, _ptr(y))
    _check(st, "conv2d")
    return y


S32_RELU = 3      # output kind of conv2d_siblings only: the 32-bit value behind a ReLU, max(v, 0), unrounded
_NP_OUT = {U8: np.uint8, S8: np.int8, S32: np.int32, S32_RELU: np.int32}


def conv2d_siblings(x, w, bias, *, stride, pad, fl_x, fl_w, y1_kind, fl_y1, y2_kind=None, fl_y2=0, residual=None, fl_r=0):
    """One accumulator, one output per child layer, each with its private fractional length (Sec. 4.3); the shortcut
    may be an 8-bit tensor or an int32 tensor in format fl_r.  Returns (y1, y2) with y2 None when not asked for."""
    n, h, wd, ci = x.shape
    co, kh, kw, ci2 = w.shape
    assert ci2 == ci and w.dtype == np.int8
    ho, wo = (h + 2 * pad - kh) // stride + 1, (wd + 2 * pad - kw) // stride + 1
    y1 = np.empty((n, ho, wo, co), dtype=_NP_OUT[y1_kind])
    y2 = np.empty((n, ho, wo, co), dtype=_NP_OUT[y2_kind]) if y2_kind is not None else None
    res_kind = 0
    if residual is not None:
        assert residual.shape == y1.shape and residual.flags["C_CONTIGUOUS"]
        res_kind = 2 if residual.dtype == np.int32 else _dtype_code(residual)
    st = lib().f8ref_conv2d_siblings(n, h, wd, ci, co, kh, kw, stride, pad, _dtype_code(x), fl_x, fl_w,
                                     _ptr(x), _ptr(w), _ptr(bias), _ptr(residual), res_kind, fl_r,
                                     _ptr(y1), y1_kind, fl_y1, _ptr(y2), y2_kind if y2_kind is not None else 0, fl_y2)
    _check(st, "conv2d_siblings")
    return y1, y2


def dwconv(x, w, bias, *, stride, pad, fl_x, fl_w, fl_y, y_dtype, residual=None, fl_r=0):
    n, h, wd, c = x.shape
    c2, kh, kw = w.shape
    assert c2 == c and w.dtype == np.int8
    ho, wo = (h + 2 * pad - kh) // stride + 1, (wd + 2 * pad - kw) // stride + 1
    y = np.empty((n, ho, wo, c), dtype=_NP[y_dtype])
    st = lib().f8ref_dwconv(n, h, wd, c, kh, kw, stride, pad, _dtype_code(x), fl_x, fl_w, fl_y, y_dtype,
                            _ptr(x), _ptr(w), _ptr(bias), _ptr(residual),
                            _dtype_code(residual) if residual is not None else 0, fl_r, _ptr(y))
    _check(st, "dwconv")
    return y


def linear(x, w, bias, *, fl_x, fl_w, fl_y, y_dtype):
    n, k = x.shape
    out, k2 = w.shape
    assert k2 == k and w.dtype == np.int8
    y = np.empty((n, out), dtype=_NP[y_dtype])
    st = lib().f8ref_linear(n, k, out, _dtype_code(x), fl_x, fl_w, fl_y, y_dtype, _ptr(x), _ptr(w), _ptr(bias),
                            _ptr(y))
    _check(st, "linear")
    return y


def maxpool(x, *, k, stride, pad):
    n, h, wd, c = x.shape
    ho, wo = (h + 2 * pad - k) // stride + 1, (wd + 2 * pad - k) // stride + 1
    y = np.empty((n, ho, wo, c), dtype=x.dtype)
    _check(lib().f8ref_maxpool(n, h, wd, c, k, stride, pad, _dtype_code(x), _ptr(x), _ptr(y)), "maxpool")
    return y


def gap(x, *, fl_x, fl_y):
    n, h, wd, c = x.shape
    y = np.empty((n, c), dtype=x.dtype)
    _check(lib().f8ref_gap(n, h, wd, c, _dtype_code(x), fl_x, fl_y, _ptr(x), _ptr(y)), "gap")
    return y


def run_layer(layer, x: np.ndarray, residual: Optional[np.ndarray] = None) -> np.ndarray:
    """Evaluate one generated layer description on host tensors."""
    x = np.ascontiguousarray(x)
    if layer.kind == CONV:
        return conv2d(x, layer.weight, layer.bias, stride=layer.stride, pad=layer.pad, fl_x=layer.fl_x,
                      fl_w=layer.fl_w, fl_y=layer.fl_y, y_dtype=layer.y_dtype, residual=residual, fl_r=layer.fl_r)
    if layer.kind == DWCONV:
        return dwconv(x, layer.weight, layer.bias, stride=layer.stride, pad=layer.pad, fl_x=layer.fl_x,
                      fl_w=layer.fl_w, fl_y=layer.fl_y, y_dtype=layer.y_dtype, residual=residual, fl_r=layer.fl_r)
    if layer.kind == MAXPOOL:
        return maxpool(x, k=layer.kh, stride=layer.stride, pad=layer.pad)
    if layer.kind == GAP:
        return gap(x, fl_x=layer.fl_x, fl_y=layer.fl_y)
    if layer.kind == LINEAR:
        return linear(x.reshape(x.shape[0], -1), layer.weight, layer.bias, fl_x=layer.fl_x, fl_w=layer.fl_w,
                      fl_y=layer.fl_y, y_dtype=layer.y_dtype)
    raise ValueError(f"unknown layer kind {layer.kind}")


def run_layer_with_sibling(layer, sibling, x: np.ndarray, residual: Optional[np.ndarray] = None):
    """A dense convolution whose 32-bit sum has a second consumer (`sibling`: a SIBLING layer description, or None),
    or whose shortcut / output stays in 32 bits (Sec. 4.3): returns (output, sibling output or None)."""
    assert layer.kind == CONV
    return conv2d_siblings(np.ascontiguousarray(x), layer.weight, layer.bias, stride=layer.stride, pad=layer.pad,
                           fl_x=layer.fl_x, fl_w=layer.fl_w, y1_kind=layer.y_dtype, fl_y1=layer.fl_y,
                           y2_kind=sibling.y_dtype if sibling is not None else None,
                           fl_y2=sibling.fl_y if sibling is not None else 0, residual=residual, fl_r=layer.fl_r)


def _needs_sibling_form(layer, nxt) -> bool:
    return layer.kind == CONV and ((nxt is not None and nxt.kind == SIBLING) or layer.y_dtype == S32_RELU or
                                   (layer.res >= 0 and layer.r_dtype == S32))


def net_forward(layers: Sequence, image: np.ndarray, keep_all: bool = True) -> List[np.ndarray]:
    """Run a layer list; returns every tensor (tensor 0 = image, layer i -> tensor i+1).

    With ``keep_all=False`` tensors are dropped once no later layer reads them
    (entries become ``None``), which bounds host memory for large batches.
    """
    last_use = {}
    for i, l in enumerate(layers):
        last_use[l.src] = i
        if l.res >= 0:
            last_use[l.res] = i
    tensors: List[Optional[np.ndarray]] = [np.ascontiguousarray(image)]
    pending = None            # the output of a sibling layer, computed together with its parent
    for i, l in enumerate(layers):
        r = tensors[l.res] if l.res >= 0 else None
        nxt = layers[i + 1] if i + 1 < len(layers) else None
        if l.kind == SIBLING:
            tensors.append(pending)
            pending = None
        elif _needs_sibling_form(l, nxt):
            y, pending = run_layer_with_sibling(l, nxt if nxt is not None and nxt.kind == SIBLING else None, tensors[l.src], r)
            tensors.append(y)
        else:
            tensors.append(run_layer(l, tensors[l.src], r))
        if not keep_all:
            for t in {l.src, l.res}:
                if t >= 0 and last_use.get(t, -1) <= i:
                    tensors[t] = None
    return tensors
