"""GPU parity (bit-exact) of the paper's sibling handling (Sec. 4.3 "Clipping-Level Sharing and Private Fractional
Length", Fig. 4): one 32-bit sum quantised once per consumer with that consumer's private fractional length, and
shortcuts that stay in 32 bits -- as a single layer call (f8_conv2d_siblings_fixed) and inside a network
(F8_LAYER_SIBLING layers, int32 residual tensors), against the oracle."""
import numpy as np
import pytest
import torch

from paper_2202_05239_b200 import synth
from gpu_util import api, Guarded, assert_equal_arrays, random_conv_layer, random_input
from test_gpu_c_nets import _compare_net

pytestmark = pytest.mark.gpu

U8, S8, S32, S32R = synth.U8, synth.S8, synth.S32, synth.S32_RELU

# (h, w, c, c_out, k, stride, n, x_signed, y1_kind, y2_kind, residual kind or None, on tensor cores)
CASES = [
    (28, 28, 128, 128, 1, 1, 4, False, U8, S8, None, True),      # two 8-bit children, no shortcut
    (28, 28, 128, 256, 1, 1, 4, False, U8, S32R, U8, True),      # 8-bit shortcut in; 8-bit child + 32-bit shortcut out
    (28, 28, 64, 64, 3, 1, 6, False, U8, S32R, S32, True),       # 32-bit shortcut in and out (identity block)
    (56, 56, 64, 128, 1, 2, 3, False, S32, None, None, True),    # down-sampling convolution handing on its raw sum
    (28, 28, 128, 128, 3, 1, 3, True, S8, U8, S32, True),        # signed input, 32-bit shortcut, signed + unsigned children
    (56, 56, 64, 64, 3, 1, 32, False, U8, U8, S32, True),        # many tiles per CTA (784 tiles)
    (14, 14, 24, 40, 3, 1, 2, False, U8, S8, S32, False),        # channel counts off the 16-byte rule: CUDA-core kernel
    (9, 9, 16, 16, 3, 2, 1, True, S32R, S32, S8, False),         # small tensor: CUDA-core kernel, both outputs 32-bit
    (12, 12, 32, 24, 1, 1, 40, False, U8, S32, U8, True),        # c_out = 24 on the tensor cores: ragged stores of both outputs
]


@pytest.mark.parametrize("case", range(len(CASES)))
def test_sibling_outputs_and_32_bit_shortcuts(ref, case):
    a = api()
    h, w, c, c_out, k, stride, n, xs, k1, k2, rk, on_tc = CASES[case]
    rng = np.random.default_rng(4000 + case)
    layer = random_conv_layer(rng, h=h, w=w, c=c, c_out=c_out, k=k, stride=stride, pad=k // 2, x_signed=xs, y_dtype=U8,
                              with_res=False)
    x = random_input(rng, n, layer)
    fa = layer.fl_x + layer.fl_w
    res, fl_r = None, 0
    if rk == S32:
        fl_r = int(rng.integers(max(0, fa - 4), fa + 5))
        res = rng.integers(-(1 << 16), 1 << 16, size=(n, layer.ho, layer.wo, c_out)).astype(np.int32)
    elif rk is not None:
        fl_r = int(rng.integers(0, 8))
        res = (rng.integers(-128, 128, size=(n, layer.ho, layer.wo, c_out)).astype(np.int8) if rk == S8
               else rng.integers(0, 256, size=(n, layer.ho, layer.wo, c_out)).astype(np.uint8))
    f = max(fa, fl_r) if res is not None else fa
    fl1 = int(np.clip(f - 9 + rng.integers(0, 3), 0, 7))
    fl2 = int(np.clip(fl1 + rng.integers(-2, 3), 0, 7))
    want1, want2 = ref.conv2d_siblings(x, layer.weight, layer.bias, stride=stride, pad=k // 2, fl_x=layer.fl_x,
                                       fl_w=layer.fl_w, y1_kind=k1, fl_y1=fl1, y2_kind=k2, fl_y2=fl2, residual=res, fl_r=fl_r)
    desc = a.conv_desc(layer, n)
    desc.y_dtype, desc.fl_y = k1, fl1
    if res is not None:
        desc.r_dtype, desc.fl_r = rk, fl_r
    shape = (n, layer.ho, layer.wo, c_out)
    y1 = Guarded(shape, a.torch_dtype(k1))
    y2 = Guarded(shape, a.torch_dtype(k2)) if k2 is not None else None
    before = a.f8_tc_launch_count()
    a.f8_conv2d_siblings_fixed(desc, k2 if k2 is not None else 0, fl2, a.to_device(x), a.to_device(layer.weight),
                               a.to_device(layer.bias), a.to_device(res) if res is not None else None, y1.t,
                               y2.t if y2 is not None else None)
    torch.cuda.synchronize()
    a.f8_device_status()
    assert (a.f8_tc_launch_count() - before == 1) == on_tc
    assert y1.intact() and (y2 is None or y2.intact())
    assert_equal_arrays(y1.t.cpu().numpy(), want1, "first output: ")
    if y2 is not None:
        assert_equal_arrays(y2.t.cpu().numpy(), want2, "second output: ")
    # an 8-bit child is exactly what the single-output entry point gives for that format
    if k1 in (U8, S8) and rk != S32:
        single = torch.empty(shape, dtype=a.torch_dtype(k1), device="cuda")
        a.f8_conv2d_fixed(desc, a.to_device(x), a.to_device(layer.weight), a.to_device(layer.bias),
                          a.to_device(res) if res is not None else None, single)
        torch.cuda.synchronize()
        assert torch.equal(single, y1.t)


def test_sibling_validation():
    a = api()
    rng = np.random.default_rng(1)
    layer = random_conv_layer(rng, h=8, w=8, c=16, c_out=16, k=1, stride=1, pad=0, x_signed=False, y_dtype=U8, with_res=False)
    desc = a.conv_desc(layer, 1)
    x = torch.zeros((1, 8, 8, 16), dtype=torch.uint8, device="cuda")
    w, b = a.to_device(layer.weight), a.to_device(layer.bias)
    y = torch.empty((1, 8, 8, 16), dtype=torch.uint8, device="cuda")
    y2 = torch.empty((1, 8, 8, 16), dtype=torch.uint8, device="cuda")
    with pytest.raises(a.F8Error) as e:
        a.f8_conv2d_siblings_fixed(desc, 7, 3, x, w, b, None, y, y2)       # unknown dtype of the second output
    assert e.value.status == 3
    with pytest.raises(a.F8Error) as e:
        a.f8_conv2d_siblings_fixed(desc, U8, 9, x, w, b, None, y, y2)      # fractional length outside the 8-bit range
    assert e.value.status == 4
    desc.r_dtype, desc.fl_r = S32, 40
    r = torch.zeros((1, 8, 8, 16), dtype=torch.int32, device="cuda")
    with pytest.raises(a.F8Error) as e:
        a.f8_conv2d_siblings_fixed(desc, U8, 3, x, w, b, r, y, y2)         # format of the 32-bit shortcut out of range
    assert e.value.status == 4
    desc.r_dtype, desc.fl_r = S32, 4
    with pytest.raises(a.F8Error) as e:
        a.f8_conv2d_fixed(desc, x, w, b, r, y)                             # the plain entry point takes 8-bit shortcuts only
    assert e.value.status == 3


@pytest.mark.parametrize("batch,image,direct", [(3, 224, False), (64, 224, False), (2, 64, True), (1, 224, False)])
def test_resnet18_with_sibling_layers_every_layer(ref, batch, image, direct):
    """The ResNet-18-shaped network with the paper's sibling handling: every tensor, 8-bit and 32-bit, bit-exact."""
    _compare_net(ref, "resnet18_siblings", batch, image, force_direct=direct)


def test_the_two_readings_of_a_shortcut_differ_by_one_code_where_they_first_differ(ref):
    """One 8-bit tensor per activation (shortcut re-read in 8 bits) against the paper's reading (shortcut kept in 32
    bits): same weights, both on the GPU.  Up to the first block that adds a 32-bit shortcut the two networks are
    identical; that block's output differs by one code at most, because the 8-bit shortcut was rounded once more
    (elements whose 8-bit shortcut saturated are excluded: the 32-bit value is not clipped)."""
    a = api()
    batch, image = 4, 224
    x = synth.draw_image(batch, 1, image, image)
    outs = {}
    for name in ("resnet18", "resnet18_siblings"):
        layers = synth.make_net(name, 0, image=image)
        net = a.Net(layers, batch)
        dump = [net.layer_output(i, batch) for i in range(len(layers))]
        net.forward(a.to_device(x), dump=dump)
        torch.cuda.synchronize()
        a.f8_device_status()
        outs[name] = {l.name: d.cpu().numpy().astype(np.int64) for l, d in zip(layers, dump)}
        net.close()
    one, two = outs["resnet18"], outs["resnet18_siblings"]
    for name in ("stem", "pool", "s0b0.conv1", "s0b0.conv2", "s0b1.conv1"):
        assert np.array_equal(one[name], two[name]), name
    first = "s0b1.conv2"          # adds the output of s0b0.conv2: 8 bits in one reading, 32 bits in the other
    unsaturated = one["s0b0.conv2"] < 255
    diff = np.abs(one[first] - two[first])
    assert diff[unsaturated].max() <= 1
    assert (diff > 0).any()        # the extra rounding is visible
