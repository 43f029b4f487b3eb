"""GPU parity (bit-exact, tolerance 0) of the CUDA-core kernels against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2202_05239_b200 import synth
from gpu_util import api, check_layer, random_conv_layer, random_input, random_residual

pytestmark = pytest.mark.gpu


def test_single_conv_case_config(ref):
    layer, x = synth.single_conv_case(0)
    check_layer(ref, layer, x, force_direct=True)
    check_layer(ref, layer, x)


@pytest.mark.parametrize("case", range(12))
def test_direct_conv_random_shapes(ref, case):
    rng = np.random.default_rng(100 + case)
    k = [1, 3, 3, 5, 7, 1, 3, 2, 3, 1, 3, 4][case]
    stride = [1, 1, 2, 1, 2, 2, 1, 2, 3, 1, 2, 1][case]
    pad = [0, 1, 1, 2, 3, 0, 0, 1, 1, 0, 1, 2][case]
    c = [3, 16, 5, 8, 3, 24, 32, 7, 12, 64, 20, 4][case]
    c_out = [8, 16, 7, 24, 64, 144, 10, 1, 33, 1000, 16, 6][case]
    h, w = 9 + case, 7 + 2 * case
    layer = random_conv_layer(rng, h=h, w=w, c=c, c_out=c_out, k=k, stride=stride, pad=pad, x_signed=bool(case % 2),
                              y_dtype=[synth.U8, synth.S8, synth.S32][case % 3], with_res=case % 4 == 1)
    x = random_input(rng, 3, layer)
    res = random_residual(rng, 3, layer) if layer.res >= 0 else None
    check_layer(ref, layer, x, res, force_direct=True)


@pytest.mark.parametrize("case", range(8))
def test_depthwise(ref, case):
    rng = np.random.default_rng(200 + case)
    c = [32, 96, 144, 5, 16, 384, 24, 960][case]
    stride = 1 + case % 2
    h = [56, 28, 14, 9, 112, 14, 33, 7][case]
    layer = random_conv_layer(rng, h=h, w=h + case % 3, c=c, c_out=c, k=3, stride=stride, pad=1,
                              x_signed=case in (3, 6), y_dtype=synth.S8 if case in (2, 5) else synth.U8,
                              with_res=case in (1, 3), kind=synth.DWCONV, fl_w=6)
    x = random_input(rng, 2, layer)
    res = random_residual(rng, 2, layer) if layer.res >= 0 else None
    check_layer(ref, layer, x, res)


@pytest.mark.parametrize("c,h,w,n,stride,x_signed,y_dtype", [
    (32, 112, 112, 3, 1, False, synth.U8), (512, 14, 14, 5, 1, False, synth.U8), (1024, 7, 7, 4, 1, True, synth.S8),
    (8, 5, 1, 2, 1, False, synth.U8), (4, 1, 9, 3, 1, True, synth.U8), (96, 37, 23, 2, 1, False, synth.S8),
    (64, 112, 112, 2, 2, False, synth.U8), (256, 28, 28, 3, 2, True, synth.U8), (512, 14, 14, 4, 2, False, synth.S8),
    (16, 7, 5, 2, 2, False, synth.U8), (12, 1, 2, 3, 2, True, synth.U8), (48, 33, 18, 2, 2, False, synth.U8)])
def test_depthwise_packed_dot_products(ref, c, h, w, n, stride, x_signed, y_dtype):
    """The dp4a depthwise kernels with every byte value on both sides (-128 weights against 255 / -128 activations),
    widths of one and two, odd sizes, single rows."""
    rng = np.random.default_rng(c * 1000 + h)
    layer = random_conv_layer(rng, h=h, w=w, c=c, c_out=c, k=3, stride=stride, pad=1, x_signed=x_signed, y_dtype=y_dtype,
                              with_res=False, kind=synth.DWCONV, fl_w=4, wide=True)
    check_layer(ref, layer, random_input(rng, n, layer))
    # the older kernels behind the planning switch give the same bits
    from paper_2202_05239_b200 import api as a
    if c <= 96:
        check_layer(ref, layer, random_input(rng, n, layer), plan_off=a.PLAN_OFF_DW_DP4A)


@pytest.mark.parametrize("c,signed,h,k,stride,pad", [(64, False, 112, 3, 2, 1), (16, True, 9, 3, 2, 1), (20, False, 11, 2, 2, 0),
                                                      (7, True, 10, 3, 1, 1), (128, False, 7, 3, 2, 1)])
def test_maxpool(ref, c, signed, h, k, stride, pad):
    rng = np.random.default_rng(c)
    dt = synth.S8 if signed else synth.U8
    layer = synth.Layer(synth.MAXPOOL, "pool", 0, -1, h, h + 1, c, c, k, k, stride, pad, dt, dt, synth.U8, 5, 0, 5, 0)
    x = random_input(rng, 2, layer)
    if signed:
        x[0, :4, :4, :] = rng.integers(-128, -90, size=x[0, :4, :4, :].shape)    # all-negative windows
    check_layer(ref, layer, x)


@pytest.mark.parametrize("c,signed,h,w,fl_x,fl_y", [(2048, False, 7, 7, 5, 6), (1280, False, 7, 7, 6, 7), (24, True, 5, 3, 4, 4),
                                                     (512, False, 1, 1, 5, 5), (100, True, 8, 8, 7, 2),
                                                     # 257 positions: the largest sum the 16-bit lanes of the packed kernel hold;
                                                     # 258: one more (the byte-wise kernel); 6 channels: not a multiple of four
                                                     (8, False, 257, 1, 4, 4), (8, True, 257, 1, 4, 4), (8, False, 129, 2, 4, 4),
                                                     (6, True, 4, 4, 5, 5)])
def test_global_average_pool(ref, c, signed, h, w, fl_x, fl_y):
    rng = np.random.default_rng(c + h)
    dt = synth.S8 if signed else synth.U8
    layer = synth.Layer(synth.GAP, "gap", 0, -1, h, w, c, c, 1, 1, 1, 0, dt, dt, synth.U8, fl_x, 0, fl_y, 0)
    x = random_input(rng, 5, layer)
    x[0, :, :, 0] = -128 if signed else 255          # a channel of extreme values: the largest / smallest possible sum
    x[1, :, :, 1] = 127 if signed else 0
    check_layer(ref, layer, x)


@pytest.mark.parametrize("n,k,out,y_dtype", [(4, 512, 1000, synth.S32), (1, 2048, 1000, synth.S32), (3, 33, 10, synth.S8),
                                             (2, 1280, 1000, synth.U8)])
def test_linear(ref, n, k, out, y_dtype):
    rng = np.random.default_rng(n * k)
    wgt = np.clip(np.round(rng.normal(0, 20, size=(out, k))), -128, 127).astype(np.int8)
    bias = rng.integers(-5000, 5000, size=out).astype(np.int32)
    layer = synth.Layer(synth.LINEAR, "fc", 0, -1, 1, 1, k, out, 1, 1, 1, 0, synth.U8, y_dtype, synth.U8, 6, 9, 3, 0, wgt, bias)
    x = rng.integers(0, 256, size=(n, k)).astype(np.uint8)
    check_layer(ref, layer, x, force_direct=True)


def test_requant_corner_shifts(ref):
    """Negative shifts (left shift then clip), shift 0, large shifts, and both residual alignment directions."""
    rng = np.random.default_rng(7)
    for fl_x, fl_w, fl_y, fl_r, y_dtype in [(0, 0, 7, 7, synth.S8), (0, -2, 6, 0, synth.U8), (7, 18, 0, 3, synth.U8),
                                            (4, 4, 8, 8, synth.U8), (3, 3, 6, 2, synth.S8), (8, 10, 8, 0, synth.U8)]:
        layer = random_conv_layer(rng, h=6, w=6, c=8, c_out=8, k=1, stride=1, pad=0, x_signed=False, y_dtype=y_dtype,
                                  with_res=True, fl_x=fl_x, fl_w=fl_w, fl_y=fl_y, fl_r=fl_r, wide=True)
        layer.r_dtype = synth.U8 if fl_r == 8 else layer.r_dtype
        if fl_w + fl_x > 20:
            layer.bias = rng.integers(-(1 << 29), 1 << 29, size=8).astype(np.int32)
        x = random_input(rng, 1, layer)
        check_layer(ref, layer, x, random_residual(rng, 1, layer), force_direct=True)


def test_empty_batch_is_accepted():
    a = api()
    layer, x = synth.single_conv_case(0)
    y = a.run_layer(layer, a.to_device(x[:0]))
    assert y.shape[0] == 0
