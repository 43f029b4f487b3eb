"""GPU parity (bit-exact) of the first-layer kernel: stride-2 convolution over an image with at most four channels,
read by the tensor cores as overlapping windows of packed row pairs, alone and fused with the 3x3 / 2 max pool."""
import numpy as np
import pytest
import torch

from paper_2202_05239_b200 import synth
from gpu_util import api

pytestmark = pytest.mark.gpu

# (h, w, c, c_out, k, pad, batch, y_dtype, with_pool)
STEM_CASES = [
    (224, 224, 3, 64, 7, 3, 2, synth.U8, True),     # the ResNet stem
    (70, 66, 3, 32, 7, 3, 5, synth.U8, True),       # odd output height (35): the last pooled row has two input rows
    (61, 45, 3, 48, 3, 1, 7, synth.U8, True),       # 3x3 stem, three 16-channel chunks per pixel, odd sizes
    (96, 96, 1, 16, 5, 2, 3, synth.S8, True),       # one channel, 5x5, signed output (signed max)
    (130, 250, 4, 64, 7, 3, 2, synth.U8, False),    # four channels, 125 outputs per row
    (64, 64, 3, 128, 7, 3, 9, synth.U8, True),      # 128 output channels; bands cross image boundaries
    (40, 40, 2, 256, 3, 1, 4, synth.S8, False),     # 256 output channels: both accumulators fill tensor memory
    (256, 256, 3, 32, 3, 1, 3, synth.U8, False),    # 128 outputs per row (a full MMA tile), MobileNet-style stem
]


def _stem_net(rng, h, w, c, c_out, k, pad, y_dtype, with_pool):
    wgt = np.clip(np.round(rng.normal(0, 20, size=(c_out, k, k, c))), -128, 127).astype(np.int8)
    wgt[0, 0, 0, 0], wgt[-1, -1, -1, -1] = -128, 127
    bias = rng.integers(-(1 << 12), 1 << 12, size=c_out).astype(np.int32)
    fl_x, fl_w = 6, 7
    s = int(np.ceil(np.log2(20.0 * 60.0 * np.sqrt(k * k * c) / 48.0)))
    conv = synth.Layer(synth.CONV, "stem", 0, -1, h, w, c, c_out, k, k, 2, pad, synth.S8, y_dtype, synth.U8,
                       fl_x, fl_w, fl_x + fl_w - s, 0, wgt, bias)
    layers = [conv]
    if with_pool:
        layers.append(synth.Layer(synth.MAXPOOL, "pool", 1, -1, conv.ho, conv.wo, c_out, c_out, 3, 3, 2, 1, y_dtype, y_dtype,
                                  synth.U8, conv.fl_y, 0, conv.fl_y, 0))
    return layers


@pytest.mark.parametrize("case", range(len(STEM_CASES)))
def test_stem_kernel(ref, case):
    h, w, c, c_out, k, pad, batch, y_dtype, with_pool = STEM_CASES[case]
    rng = np.random.default_rng(900 + case)
    layers = _stem_net(rng, h, w, c, c_out, k, pad, y_dtype, with_pool)
    x = rng.integers(-128, 128, size=(batch, h, w, c)).astype(np.int8)
    want = ref.net_forward(layers, x)
    a = api()
    net = a.Net(layers, batch)
    xd = a.to_device(x)
    # every layer's output asked for: the convolution runs alone, the pool in its own kernel
    before = a.f8_tc_launch_count()
    dump = [net.layer_output(i, batch) for i in range(len(layers))]
    out = net.forward(xd, dump=dump)
    torch.cuda.synchronize()
    a.f8_device_status()
    assert a.f8_tc_launch_count() - before == 1, "the first layer did not run on the tensor cores"
    assert net.last_launch_count == len(layers)
    for i in range(len(layers)):
        got = dump[i].cpu().numpy().reshape(want[i + 1].shape)
        assert int((got != want[i + 1]).sum()) == 0, f"layer {i} differs"
    assert np.array_equal(out.cpu().numpy().reshape(want[-1].shape), want[-1])
    # only the final output asked for: one kernel computes convolution and pool
    out.zero_()
    out = net.forward(xd, out=out)
    torch.cuda.synchronize()
    a.f8_device_status()
    assert net.last_launch_count == 1
    got = out.cpu().numpy().reshape(want[-1].shape)
    bad = np.argwhere(got != want[-1])
    assert bad.shape[0] == 0, f"{bad.shape[0]} of {got.size} differ, first at {bad[0]}"
    if with_pool:
        # the pooled output asked for as a dump as well (still fused)
        d2 = [None, net.layer_output(1, batch)]
        net.forward(xd, dump=d2)
        torch.cuda.synchronize()
        assert net.last_launch_count == 1
        assert np.array_equal(d2[1].cpu().numpy().reshape(want[2].shape), want[2])
    net.close()


def test_stem_pool_fusion_needs_a_single_consumer(ref):
    """A second reader of the convolution's output (here a residual-free 1x1 layer) keeps the layers apart."""
    rng = np.random.default_rng(77)
    layers = _stem_net(rng, 64, 64, 3, 32, 7, 3, synth.U8, True)
    conv = layers[0]
    w2 = np.clip(np.round(rng.normal(0, 20, size=(16, 1, 1, 32))), -128, 127).astype(np.int8)
    b2 = rng.integers(-100, 100, size=16).astype(np.int32)
    layers.append(synth.Layer(synth.CONV, "side", 1, -1, conv.ho, conv.wo, 32, 16, 1, 1, 1, 0, synth.U8, synth.U8, synth.U8,
                              conv.fl_y, 6, conv.fl_y, 0, w2, b2))
    x = rng.integers(-128, 128, size=(6, 64, 64, 3)).astype(np.int8)
    want = ref.net_forward(layers, x)
    a = api()
    net = a.Net(layers, 6)
    out = net.forward(a.to_device(x))
    torch.cuda.synchronize()
    a.f8_device_status()
    assert net.last_launch_count == 3
    assert np.array_equal(out.cpu().numpy().reshape(want[-1].shape), want[-1])
    net.close()
