"""Thin Python binding over the C-ABI CUDA library (``libf8net.so``).

Only argument marshalling happens here: every function forwards device pointers
of torch tensors (torch supplies memory and streams) to the entry point of the
same name in ``include/f8net.h``.  There is no CPU fallback: importing this
module fails if the library has not been built.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np
import torch

from . import synth

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libf8net.so")

if not os.path.exists(_LIB_PATH):
    raise ImportError(
        f"{_LIB_PATH} is missing: build the CUDA library first "
        "(python -m paper_2202_05239_b200.build, or __graft_entry__.build())")

_lib = ctypes.CDLL(_LIB_PATH)

F8_OK = 0
F8_U8, F8_S8, F8_S32, F8_S32_RELU = 0, 1, 2, 3
STATUS_NAMES = ["F8_OK", "F8_ERR_NULL", "F8_ERR_SHAPE", "F8_ERR_DTYPE", "F8_ERR_FL_RANGE", "F8_ERR_SHIFT_RANGE",
                "F8_ERR_ALIGN", "F8_ERR_ACC_BOUND", "F8_ERR_WORKSPACE", "F8_ERR_UNSUPPORTED", "F8_ERR_CUDA",
                "F8_ERR_TIMEOUT"]


class ConvDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("n", "h", "w", "c", "c_out", "kh", "kw", "stride", "pad", "x_dtype", "y_dtype", "r_dtype",
                 "fl_x", "fl_w", "fl_y", "fl_r")]


class LayerDesc(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int), ("src", ctypes.c_int), ("res", ctypes.c_int), ("conv", ConvDesc)]


class F8Error(RuntimeError):
    def __init__(self, status: int, message: str):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{name}: {message}")


_vp, _ci, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
_lib.f8_conv2d_fixed.argtypes = [ctypes.POINTER(ConvDesc), _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.f8_dwconv_fixed.argtypes = _lib.f8_conv2d_fixed.argtypes
_lib.f8_linear_fixed.argtypes = [_ci] * 8 + [_vp, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.f8_maxpool_fixed.argtypes = [_ci] * 8 + [_vp, _vp, _vp]
_lib.f8_global_avgpool_fixed.argtypes = [_ci] * 7 + [_vp, _vp, _vp]
_lib.f8_conv_workspace_bytes.argtypes = [ctypes.POINTER(ConvDesc)]
_lib.f8_conv_workspace_bytes.restype = _sz
_lib.f8_net_create.argtypes = [ctypes.POINTER(LayerDesc), _ci, ctypes.POINTER(_vp), ctypes.POINTER(_vp), _ci,
                               ctypes.POINTER(_vp)]
_lib.f8_net_workspace_bytes.argtypes = [_vp, _ci]
_lib.f8_net_workspace_bytes.restype = _sz
_lib.f8_net_forward.argtypes = [_vp, _ci, _vp, _vp, _vp, _sz, ctypes.POINTER(_vp), _vp]
_lib.f8_net_last_launch_count.argtypes = [_vp]
_lib.f8_net_set_profiling.argtypes = [_vp, _ci]
_lib.f8_net_get_layer_ms.argtypes = [_vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int)]
_lib.f8_net_destroy.argtypes = [_vp]
_lib.f8_net_destroy.restype = None
_lib.f8_status_str.argtypes = [_ci]
_lib.f8_status_str.restype = ctypes.c_char_p
_lib.f8_last_error.restype = ctypes.c_char_p
_lib.f8_mma_i8_probe.argtypes = [_ci, ctypes.POINTER(ctypes.c_double), _vp]
_lib.f8_debug_force_direct.argtypes = [_ci]
_lib.f8_debug_force_direct.restype = None


def _check(status: int):
    if status != F8_OK:
        raise F8Error(status, _lib.f8_last_error().decode())


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("tensors must be contiguous CUDA tensors")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def conv_desc(layer: "synth.Layer", n: int) -> ConvDesc:
    return ConvDesc(n, layer.h, layer.w, layer.c, layer.c_out, layer.kh, layer.kw, layer.stride, layer.pad,
                    layer.x_dtype, layer.y_dtype, layer.r_dtype, layer.fl_x, layer.fl_w, layer.fl_y, layer.fl_r)


_TORCH_DTYPE = {F8_U8: torch.uint8, F8_S8: torch.int8, F8_S32: torch.int32, F8_S32_RELU: torch.int32}


def torch_dtype(code: int) -> torch.dtype:
    return _TORCH_DTYPE[code]


def to_device(a: Optional[np.ndarray], device="cuda") -> Optional[torch.Tensor]:
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(device)


# ------------------------------------------------------------------ entry points (same names as the C ABI)

def f8_conv2d_fixed(desc: ConvDesc, x, w, bias, residual, y, workspace=None, stream=None):
    _check(_lib.f8_conv2d_fixed(ctypes.byref(desc), _ptr(x), _ptr(w), _ptr(bias), _ptr(residual), _ptr(y),
                                _ptr(workspace), workspace.numel() if workspace is not None else 0, _stream(stream)))


_lib.f8_conv2d_siblings_fixed.argtypes = [ctypes.POINTER(ConvDesc), _ci, _ci, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]


def f8_conv2d_siblings_fixed(desc: ConvDesc, y2_dtype, fl_y2, x, w, bias, residual, y, y2, workspace=None, stream=None):
    """One 32-bit sum, one output per consumer with its private fractional length; 32-bit shortcuts allowed (Sec. 4.3)."""
    _check(_lib.f8_conv2d_siblings_fixed(ctypes.byref(desc), y2_dtype, fl_y2, _ptr(x), _ptr(w), _ptr(bias), _ptr(residual),
                                         _ptr(y), _ptr(y2), _ptr(workspace),
                                         workspace.numel() if workspace is not None else 0, _stream(stream)))


_lib.f8_conv_pointwise_fixed.argtypes = [ctypes.POINTER(ConvDesc), ctypes.POINTER(ConvDesc)] + [_vp] * 9


def f8_conv_pointwise_fixed(conv: ConvDesc, pw: ConvDesc, x, w_conv, bias_conv, w_pw, bias_pw, residual, y_mid, y, stream=None):
    """A 64 -> 64 convolution and the 64 -> 256 pointwise layer behind it in one launch (y_mid: optional copy of the first output)."""
    _check(_lib.f8_conv_pointwise_fixed(ctypes.byref(conv), ctypes.byref(pw), _ptr(x), _ptr(w_conv), _ptr(bias_conv), _ptr(w_pw),
                                        _ptr(bias_pw), _ptr(residual), _ptr(y_mid), _ptr(y), _stream(stream)))


def f8_dwconv_fixed(desc: ConvDesc, x, w, bias, residual, y, workspace=None, stream=None):
    _check(_lib.f8_dwconv_fixed(ctypes.byref(desc), _ptr(x), _ptr(w), _ptr(bias), _ptr(residual), _ptr(y),
                                _ptr(workspace), workspace.numel() if workspace is not None else 0, _stream(stream)))


def f8_linear_fixed(n, k, out, x_dtype, y_dtype, fl_x, fl_w, fl_y, x, w, bias, y, workspace=None, stream=None):
    _check(_lib.f8_linear_fixed(n, k, out, x_dtype, y_dtype, fl_x, fl_w, fl_y, _ptr(x), _ptr(w), _ptr(bias), _ptr(y),
                                _ptr(workspace), workspace.numel() if workspace is not None else 0, _stream(stream)))


def f8_maxpool_fixed(n, h, w, c, k, stride, pad, x_dtype, x, y, stream=None):
    _check(_lib.f8_maxpool_fixed(n, h, w, c, k, stride, pad, x_dtype, _ptr(x), _ptr(y), _stream(stream)))


def f8_global_avgpool_fixed(n, h, w, c, x_dtype, fl_x, fl_y, x, y, stream=None):
    _check(_lib.f8_global_avgpool_fixed(n, h, w, c, x_dtype, fl_x, fl_y, _ptr(x), _ptr(y), _stream(stream)))


_lib.f8_stem_conv2d_fixed_static.argtypes = [ctypes.POINTER(ConvDesc), _vp, _vp, _vp, _vp, _ci, _vp]
F8_STATIC_STEM_MAX_BYTES = 16 * 1024 * 1024


def f8_stem_conv2d_fixed_static(desc: ConvDesc, x, w, bias, y, check_previous: bool = False, stream=None):
    """First-layer convolution whose scratch memory is a fixed array inside the library: nothing is allocated.

    For callers that cannot obtain device memory when they need the result (the device is owned by another
    allocator, or allocation is forbidden on their path).  Same result as ``f8_conv2d_fixed``; calls share the
    array, so do not let two of them overlap on the GPU.
    """
    _check(_lib.f8_stem_conv2d_fixed_static(ctypes.byref(desc), _ptr(x), _ptr(w), _ptr(bias), _ptr(y),
                                            1 if check_previous else 0, _stream(stream)))


class FoldDesc(ctypes.Structure):
    _fields_ = [("c_out", ctypes.c_int), ("k", ctypes.c_int), ("fl_x", ctypes.c_int), ("fl_w_min", ctypes.c_int),
                ("fl_w_max", ctypes.c_int), ("eta_in", ctypes.c_double), ("eta_out", ctypes.c_double)]


_lib.f8_fold_workspace_bytes.argtypes = [ctypes.POINTER(FoldDesc)]
_lib.f8_fold_workspace_bytes.restype = _sz
_lib.f8_fold_quantize_fixed.argtypes = [ctypes.POINTER(FoldDesc)] + [_vp] * 9 + [_sz, _vp]


def f8_fold_workspace_bytes(desc: FoldDesc) -> int:
    return int(_lib.f8_fold_workspace_bytes(ctypes.byref(desc)))


def f8_fold_quantize_fixed(desc: FoldDesc, w, gamma, sigma, beta, mu, w_q, bias_q, fl_w, workspace, stream=None):
    """Eq. 6 + Eq. 1 + signed quantiser for one Conv-BN block; every tensor on the device, fl_w a 1-element int32."""
    _check(_lib.f8_fold_quantize_fixed(ctypes.byref(desc), _ptr(w), _ptr(gamma), _ptr(sigma), _ptr(beta), _ptr(mu),
                                       _ptr(w_q), _ptr(bias_q), _ptr(fl_w), _ptr(workspace),
                                       workspace.numel() * workspace.element_size(), _stream(stream)))


_lib.f8_format_study_workspace_bytes.restype = _sz
_lib.f8_format_study_fixed.argtypes = [_vp, ctypes.c_longlong, _ci, _vp, _vp, _vp, _sz, _vp]


def f8_format_study_workspace_bytes() -> int:
    return int(_lib.f8_format_study_workspace_bytes())


def f8_format_study_fixed(x, unsigned: bool, err, best_fl, workspace, stream=None):
    """Sec. 3.3's experiment on the device sample x (fp32): err (9 float64) and best_fl (1 int32) are device tensors."""
    _check(_lib.f8_format_study_fixed(_ptr(x), x.numel(), 1 if unsigned else 0, _ptr(err), _ptr(best_fl), _ptr(workspace),
                                      workspace.numel() * workspace.element_size(), _stream(stream)))


_lib.f8_requantize_dual_fixed.argtypes = [ctypes.c_longlong, _vp, _ci, _vp, _ci, _ci, _vp, _ci, _ci, _vp]


def f8_requantize_dual_fixed(acc, fa, y1, y1_dtype, fl_y1, y2=None, y2_dtype=F8_U8, fl_y2=0, stream=None):
    """int32 tensor in format fa -> one or two 8-bit tensors, each with its own fractional length (Sec. 4.3)."""
    _check(_lib.f8_requantize_dual_fixed(acc.numel(), _ptr(acc), fa, _ptr(y1), y1_dtype, fl_y1, _ptr(y2), y2_dtype, fl_y2,
                                         _stream(stream)))


def f8_conv_workspace_bytes(desc: ConvDesc) -> int:
    return int(_lib.f8_conv_workspace_bytes(ctypes.byref(desc)))


def f8_device_status():
    _check(_lib.f8_device_status())


def f8_mma_i8_probe(iters: int, stream=None) -> float:
    ops = ctypes.c_double(0.0)
    _check(_lib.f8_mma_i8_probe(iters, ctypes.byref(ops), _stream(stream)))
    return ops.value


_lib.f8_tc_launch_count.restype = ctypes.c_longlong


def f8_tc_launch_count() -> int:
    return int(_lib.f8_tc_launch_count())


def f8_debug_force_direct(on: bool):
    _lib.f8_debug_force_direct(1 if on else 0)


_lib.f8_debug_plan_options.argtypes = [ctypes.c_uint]
_lib.f8_debug_plan_options.restype = None
_lib.f8_debug_last_plan.argtypes = [ctypes.POINTER(ctypes.c_int), _ci]
_lib.f8_debug_set_wait_limit_ms.argtypes = [ctypes.c_double]
_lib.f8_debug_set_wait_limit_ms.restype = None
_lib.f8_debug_wait_timeout_probe.argtypes = [ctypes.c_double, _vp]

# f8_debug_plan_options bits (planning choices switched off) and f8_debug_last_plan flags
PLAN_OFF_RESIDENT_WEIGHTS, PLAN_OFF_WINDOWED, PLAN_OFF_DUAL_ISSUE, PLAN_OFF_ALT_PRODUCERS = 1, 2, 4, 8
PLAN_OFF_PAIRS, PLAN_OFF_DW_WALK, PLAN_OFF_STEM_KERNEL, PLAN_OFF_STEM_POOL_FUSION = 16, 32, 64, 128
PLAN_OFF_LAYER_OVERLAP, PLAN_OFF_LANES, PLAN_SYNC_LAYERS, PLAN_OFF_DW_DP4A = 256, 512, 1024, 2048
PLAN_OFF_TILE_GROUPS = 4096
PLAN_OFF_LAYER_FUSION = 8192
PLAN_RESIDENT_WEIGHTS, PLAN_WINDOWED, PLAN_DUAL_ISSUE, PLAN_ALT_PRODUCERS = 1, 2, 4, 8
PLAN_PLAIN_MATRIX, PLAN_STAGED_EPILOGUE, PLAN_PAIRS, PLAN_ROW_TILES = 16, 32, 64, 128
PLAN_TILE_GROUPS = 256


def f8_debug_plan_options(off_mask: int):
    _lib.f8_debug_plan_options(off_mask)


_lib.f8_debug_set_micro_batch.argtypes = [_ci]
_lib.f8_debug_set_micro_batch.restype = None
_lib.f8_net_micro_batching.argtypes = [_vp, ctypes.POINTER(_ci)]


def f8_debug_set_micro_batch(images: int):
    """Micro-batch of f8_net_forward's depth-first runs: 0 off (default), -1 the L2-size rule, > 0 that many images."""
    _lib.f8_debug_set_micro_batch(images)


_lib.f8_debug_set_lanes.argtypes = [_ci]
_lib.f8_debug_set_lanes.restype = None
_lib.f8_net_lanes.argtypes = [_vp]
_lib.f8_net_fused_pairs.argtypes = [_vp]


def f8_debug_set_lanes(lanes: int):
    """Concurrent lanes of f8_net_forward: 0 the library's rule, 1 or 2 that many."""
    _lib.f8_debug_set_lanes(lanes)


def f8_debug_last_plan() -> dict:
    """What the most recent tensor-core plan decided (which code path a layer takes, how many tiles per CTA)."""
    v = (ctypes.c_int * 10)()
    _lib.f8_debug_last_plan(v, 10)
    keys = ("flags", "epilogue", "bn", "kb", "stages", "group", "m_tiles", "n_tiles", "ctas", "out_bufs")
    return dict(zip(keys, [int(x) for x in v]))


def f8_debug_set_wait_limit_ms(ms: float):
    _lib.f8_debug_set_wait_limit_ms(ms)


def f8_debug_wait_timeout_probe(limit_ms: float, stream=None):
    _check(_lib.f8_debug_wait_timeout_probe(limit_ms, _stream(stream)))


def layer_output_shape(layer: "synth.Layer", n: int):
    if layer.kind in (synth.CONV, synth.DWCONV):
        return (n, layer.ho, layer.wo, layer.c_out)
    if layer.kind == synth.MAXPOOL:
        return (n, layer.ho, layer.wo, layer.c)
    if layer.kind == synth.GAP:
        return (n, layer.c)
    return (n, layer.c_out)


def run_layer(layer: "synth.Layer", x: torch.Tensor, residual: Optional[torch.Tensor] = None, params=None,
              stream=None, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """One generated layer through the single-layer entry points; returns the output tensor (`out` if given)."""
    n = x.shape[0]
    w, b = params if params is not None else (to_device(layer.weight), to_device(layer.bias))
    if out is not None:
        y = out
        if layer.kind in (synth.CONV, synth.DWCONV):
            fn = f8_conv2d_fixed if layer.kind == synth.CONV else f8_dwconv_fixed
            fn(conv_desc(layer, n), x, w, b, residual, y, stream=stream)
        elif layer.kind == synth.LINEAR:
            f8_linear_fixed(n, layer.c, layer.c_out, layer.x_dtype, layer.y_dtype, layer.fl_x, layer.fl_w, layer.fl_y,
                            x, w, b, y, stream=stream)
        elif layer.kind == synth.MAXPOOL:
            f8_maxpool_fixed(n, layer.h, layer.w, layer.c, layer.kh, layer.stride, layer.pad, layer.x_dtype, x, y,
                             stream=stream)
        elif layer.kind == synth.GAP:
            f8_global_avgpool_fixed(n, layer.h, layer.w, layer.c, layer.x_dtype, layer.fl_x, layer.fl_y, x, y,
                                    stream=stream)
        else:
            raise ValueError(layer.kind)
        return y
    if layer.kind in (synth.CONV, synth.DWCONV):
        y = torch.empty((n, layer.ho, layer.wo, layer.c_out), dtype=torch_dtype(layer.y_dtype), device=x.device)
        fn = f8_conv2d_fixed if layer.kind == synth.CONV else f8_dwconv_fixed
        fn(conv_desc(layer, n), x, w, b, residual, y, stream=stream)
    elif layer.kind == synth.LINEAR:
        y = torch.empty((n, layer.c_out), dtype=torch_dtype(layer.y_dtype), device=x.device)
        f8_linear_fixed(n, layer.c, layer.c_out, layer.x_dtype, layer.y_dtype, layer.fl_x, layer.fl_w, layer.fl_y,
                        x, w, b, y, stream=stream)
    elif layer.kind == synth.MAXPOOL:
        y = torch.empty((n, layer.ho, layer.wo, layer.c), dtype=x.dtype, device=x.device)
        f8_maxpool_fixed(n, layer.h, layer.w, layer.c, layer.kh, layer.stride, layer.pad, layer.x_dtype, x, y,
                         stream=stream)
    elif layer.kind == synth.GAP:
        y = torch.empty((n, layer.c), dtype=x.dtype, device=x.device)
        f8_global_avgpool_fixed(n, layer.h, layer.w, layer.c, layer.x_dtype, layer.fl_x, layer.fl_y, x, y,
                                stream=stream)
    else:
        raise ValueError(layer.kind)
    return y


class Net:
    """Owner of an ``f8_net`` object built from generated layer descriptions."""

    def __init__(self, layers: Sequence["synth.Layer"], max_batch: int):
        self.layers = list(layers)
        self.max_batch = max_batch
        n = len(self.layers)
        descs, wptrs, bptrs, self._keep = _layer_tables(self.layers)
        handle = _vp()
        _check(_lib.f8_net_create(descs, n, wptrs, bptrs, max_batch, ctypes.byref(handle)))
        self._h = handle
        self._ws = None
        last = self.layers[-1]
        self.out_shape = (last.c_out,) if last.kind in (synth.LINEAR, synth.GAP) else (last.ho, last.wo, last.c_out)
        self.out_dtype = torch_dtype(last.y_dtype)

    def workspace_bytes(self, batch: int) -> int:
        return int(_lib.f8_net_workspace_bytes(self._h, batch))

    def layer_output(self, i: int, batch: int, device="cuda") -> torch.Tensor:
        l = self.layers[i]
        shape = (batch, l.c_out) if l.kind in (synth.LINEAR, synth.GAP) else (batch, l.ho, l.wo, l.c_out)
        return torch.empty(shape, dtype=torch_dtype(l.y_dtype), device=device)

    def forward(self, x: torch.Tensor, out: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                dump: Optional[Sequence[Optional[torch.Tensor]]] = None, stream=None) -> torch.Tensor:
        """f8_net_forward: ``x`` [batch,h,w,c] device tensor -> ``out`` (allocated if not given)."""
        batch = x.shape[0]
        if out is None:
            out = torch.empty((batch,) + self.out_shape, dtype=self.out_dtype, device=x.device)
        need = self.workspace_bytes(batch)
        if workspace is None:
            if self._ws is None or self._ws.numel() < need or self._ws.device != x.device:
                self._ws = torch.empty(need, dtype=torch.uint8, device=x.device)
            workspace = self._ws
        dptr = None
        if dump is not None:
            dptr = (_vp * len(self.layers))()
            for i, t in enumerate(dump):
                if t is not None:
                    dptr[i] = t.data_ptr()
        _check(_lib.f8_net_forward(self._h, batch, _ptr(x), _ptr(out), _ptr(workspace), workspace.numel(), dptr,
                                   _stream(stream)))
        return out

    def set_profiling(self, on: bool):
        _check(_lib.f8_net_set_profiling(self._h, 1 if on else 0))

    def layer_ms(self):
        """(ms per layer, ran-on-tensor-cores flag per layer) of the last profiled forward pass."""
        n = len(self.layers)
        ms = (ctypes.c_float * n)()
        tc = (ctypes.c_int * n)()
        _check(_lib.f8_net_get_layer_ms(self._h, ms, tc))
        return list(ms), [bool(v) for v in tc]

    @property
    def last_launch_count(self) -> int:
        return int(_lib.f8_net_last_launch_count(self._h))

    @property
    def lanes(self) -> int:
        return int(_lib.f8_net_lanes(self._h))

    @property
    def fused_pairs(self) -> int:
        """Launches of the last forward pass that ran two layers at once."""
        return int(_lib.f8_net_fused_pairs(self._h))

    def micro_batching(self):
        """(number of runs of layers the last forward pass executed depth-first over micro-batches, smallest micro-batch)."""
        images = _ci(0)
        runs = int(_lib.f8_net_micro_batching(self._h, ctypes.byref(images)))
        return runs, int(images.value)

    def close(self):
        if self._h:
            _lib.f8_net_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def _layer_tables(layers):
    """ctypes tables f8_net_create / f8_net_host_create take: descriptors, host weight and bias pointers (+ the arrays
    that must stay alive while the call runs)."""
    n = len(layers)
    descs = (LayerDesc * n)()
    wptrs = (_vp * n)()
    bptrs = (_vp * n)()
    keep = []
    for i, l in enumerate(layers):
        descs[i] = LayerDesc(l.kind, l.src, l.res, conv_desc(l, 1))
        if l.weight is not None:
            w = np.ascontiguousarray(l.weight, dtype=np.int8)
            keep.append(w)
            wptrs[i] = w.ctypes.data
        if l.bias is not None:
            b = np.ascontiguousarray(l.bias, dtype=np.int32)
            keep.append(b)
            bptrs[i] = b.ctypes.data
    return descs, wptrs, bptrs, keep


_lib.f8_net_host_create.argtypes = [ctypes.POINTER(LayerDesc), _ci, ctypes.POINTER(_vp), ctypes.POINTER(_vp), _ci, _ci,
                                    ctypes.POINTER(_vp)]
_lib.f8_net_forward_host.argtypes = [_vp, _vp, _vp]
_lib.f8_net_host_wait.argtypes = [_vp]
_lib.f8_net_host_streams.argtypes = [_vp, ctypes.POINTER(_vp), ctypes.POINTER(_vp), ctypes.POINTER(_vp)]
_lib.f8_net_host_launches_per_pass.argtypes = [_vp]
_lib.f8_net_host_destroy.argtypes = [_vp]
_lib.f8_net_host_destroy.restype = None


class HostPipeline:
    """Forward passes from (pinned) host buffers through ``f8_net_forward_host``: while the GPU runs batch i, the copy
    engines upload batch i+1 and download the logits of batch i-1.  Slots, device buffers, streams and events all
    belong to the library object; this class only passes host pointers.  submit() returns at once; result `i` is in
    its host buffer after wait()."""

    def __init__(self, layers: Sequence["synth.Layer"], batch: int, depth: int = 2, device="cuda"):
        self.batch = batch
        self.depth = depth
        dev = torch.device(device)
        with torch.cuda.device(dev if dev.index is not None else torch.cuda.current_device()):
            descs, wptrs, bptrs, keep = _layer_tables(list(layers))
            handle = _vp()
            _check(_lib.f8_net_host_create(descs, len(layers), wptrs, bptrs, batch, depth, ctypes.byref(handle)))
            self._h = handle
            up, comp, down = _vp(), _vp(), _vp()
            _check(_lib.f8_net_host_streams(self._h, ctypes.byref(up), ctypes.byref(comp), ctypes.byref(down)))
            self.up_stream = torch.cuda.ExternalStream(up.value)
            self.compute_stream = torch.cuda.ExternalStream(comp.value)
            self.down_stream = torch.cuda.ExternalStream(down.value)
        del keep

    def submit(self, x_host: torch.Tensor, y_host: torch.Tensor):
        if x_host.is_cuda or y_host.is_cuda or not x_host.is_contiguous() or not y_host.is_contiguous():
            raise ValueError("submit() takes contiguous host tensors")
        _check(_lib.f8_net_forward_host(self._h, ctypes.c_void_p(x_host.data_ptr()), ctypes.c_void_p(y_host.data_ptr())))

    def wait(self):
        _check(_lib.f8_net_host_wait(self._h))

    @property
    def launches_per_step(self) -> int:
        return int(_lib.f8_net_host_launches_per_pass(self._h))

    def close(self):
        if self._h:
            _lib.f8_net_host_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
