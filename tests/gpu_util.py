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


GUARD = 4096          # bytes of poison on either side of every output buffer
POISON = 0xA5


class Guarded:
    """An output tensor inside a poison-filled allocation: `t` is the tensor the kernel writes, `intact()` says whether
    the bands in front of and behind it still hold the poison (a stand-in for a memory checker: an out-of-bounds
    store next to an output shows up here).  The tensor itself starts out poisoned too, so an element a kernel
    forgot to write is very unlikely to compare equal."""

    def __init__(self, shape, dtype, device="cuda"):
        self.nbytes = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        pad = (-self.nbytes) % 256
        self.raw = torch.full((GUARD + self.nbytes + pad + GUARD,), POISON, dtype=torch.uint8, device=device)
        self.t = self.raw[GUARD:GUARD + self.nbytes].view(dtype).view(shape)

    def intact(self) -> bool:
        head, tail = self.raw[:GUARD], self.raw[GUARD + self.nbytes:]
        return bool((head == POISON).all().item()) and bool((tail == POISON).all().item())


def assert_equal_arrays(got, want, what=""):
    bad = np.argwhere(got != want)
    assert bad.shape[0] == 0, (f"{what}{bad.shape[0]} of {want.size} elements differ; first at {bad[0]}: "
                               f"got {got[tuple(bad[0])]} want {want[tuple(bad[0])]}")


def check_layer(ref, layer, x, res=None, force_direct=False, expect_tc=None, plan_off=0, expect_flags=0,
                forbid_flags=0, min_tiles_per_cta=0):
    """Runs one layer on the GPU through the C ABI and on the oracle; asserts bit-exact equality and that nothing
    next to the output buffer was touched.  plan_off switches planning choices off (the alternative code paths);
    expect_flags / forbid_flags / min_tiles_per_cta assert what the tensor-core plan decided."""
    a = api()
    want = ref.run_layer(layer, x, res)
    a.f8_debug_force_direct(force_direct)
    a.f8_debug_plan_options(plan_off)
    before = a.f8_tc_launch_count()
    out = Guarded(a.layer_output_shape(layer, x.shape[0]), a.torch_dtype(layer.y_dtype))
    try:
        got = a.run_layer(layer, a.to_device(x), a.to_device(res) if res is not None else None, out=out.t)
        torch.cuda.synchronize()
        a.f8_device_status()
    finally:
        a.f8_debug_force_direct(False)
        a.f8_debug_plan_options(0)
    if expect_tc is not None:
        assert (a.f8_tc_launch_count() - before == 1) == expect_tc, "layer did not take the expected path"
    if expect_flags or forbid_flags or min_tiles_per_cta:
        plan = a.f8_debug_last_plan()
        assert plan["flags"] & expect_flags == expect_flags, f"plan {plan} lacks flags {expect_flags}"
        assert plan["flags"] & forbid_flags == 0, f"plan {plan} has one of the flags {forbid_flags}"
        tiles = plan["m_tiles"] * plan["n_tiles"]
        assert tiles >= min_tiles_per_cta * plan["ctas"], f"plan {plan}: fewer than {min_tiles_per_cta} tiles per CTA"
    assert out.intact(), "the kernel wrote outside its output buffer"
    assert_equal_arrays(got.cpu().numpy().reshape(want.shape), want)
