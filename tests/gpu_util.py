"""Helpers shared by the GPU parity tests (not collected by pytest)."""
import numpy as np
import torch

from paper_2202_05239_b200 import synth


def api():
    from paper_2202_05239_b200 import api as _api
    return _api


def random_conv_layer(rng, *, h, w, c, c_out, k, stride, pad, x_signed, y_dtype, with_res, kind=synth.CONV,
                      fl_x=None, fl_w=None, fl_y=None, fl_r=None, wide=False):
    """A layer with uniformly random codes (all byte values occur, including -128 and 255)."""
    depthwise = kind == synth.DWCONV
    fan_in = k * k * (1 if depthwise else c)
    wshape = (c, k, k) if depthwise else (c_out, k, k, c)
    if wide:
        wgt = rng.integers(-128, 128, size=wshape).astype(np.int8)
    else:   # keep accumulators in a range where the output is not always clipped
        wgt = np.clip(np.round(rng.normal(0, 12, size=wshape)), -128, 127).astype(np.int8)
    fl_x = int(rng.integers(0, 8)) if fl_x is None else fl_x
    fl_w = int(rng.integers(3, 11)) if fl_w is None else fl_w
    x_dtype = synth.S8 if x_signed else synth.U8
    # choose fl_y so that typical accumulators land inside the 8-bit range
    typical = 12.0 * 80.0 * np.sqrt(fan_in)
    s = max(0, int(np.ceil(np.log2(typical / 64.0))))
    if fl_y is None:
        fl_y = int(np.clip(fl_x + fl_w - s, 0, 7))
    r_dtype = synth.S8 if rng.integers(0, 2) else synth.U8
    fl_r = int(rng.integers(0, 8)) if fl_r is None else fl_r
    bias = rng.integers(-(1 << 14), 1 << 14, size=c_out).astype(np.int32)
    layer = synth.Layer(kind, "rand", 0, 1 if with_res else -1, h, w, c, c_out, k, k, stride, pad, x_dtype, y_dtype,
                        r_dtype, fl_x, fl_w, fl_y, fl_r, wgt, bias)
    return layer


def random_input(rng, n, layer):
    if layer.x_dtype == synth.S8:
        return rng.integers(-128, 128, size=(n, layer.h, layer.w, layer.c)).astype(np.int8)
    return rng.integers(0, 256, size=(n, layer.h, layer.w, layer.c)).astype(np.uint8)


def random_residual(rng, n, layer):
    shape = (n, layer.ho, layer.wo, layer.c_out)
    if layer.r_dtype == synth.S8:
        return rng.integers(-128, 128, size=shape).astype(np.int8)
    return rng.integers(0, 256, size=shape).astype(np.uint8)


def check_layer(ref, layer, x, res=None, force_direct=False, expect_tc=None):
    """Runs one layer on the GPU through the C ABI and on the oracle; asserts bit-exact equality."""
    a = api()
    want = ref.run_layer(layer, x, res)
    a.f8_debug_force_direct(force_direct)
    before = a.f8_tc_launch_count()
    try:
        got = a.run_layer(layer, a.to_device(x), a.to_device(res) if res is not None else None)
        torch.cuda.synchronize()
        a.f8_device_status()
    finally:
        a.f8_debug_force_direct(False)
    if expect_tc is not None:
        assert (a.f8_tc_launch_count() - before == 1) == expect_tc, "layer did not take the expected path"
    got = got.cpu().numpy().reshape(want.shape)
    bad = np.argwhere(got != want)
    assert bad.shape[0] == 0, f"{bad.shape[0]} of {want.size} elements differ; first at {bad[0]}: got {got[tuple(bad[0])]} want {want[tuple(bad[0])]}"
