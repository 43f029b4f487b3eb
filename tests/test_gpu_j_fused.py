"""GPU parity (bit-exact) of the two-layer kernel: a 64 -> 64 convolution and the 64 -> 256 pointwise layer behind it in one
launch (f8_conv_pointwise_fixed), against the oracle's two single-layer calls; and of networks whose bottleneck tails
f8_net_forward runs that way."""
import numpy as np
import pytest
import torch

from paper_2202_05239_b200 import synth
from gpu_util import Guarded, api, assert_equal_arrays, random_conv_layer, random_input, random_residual

pytestmark = pytest.mark.gpu

# (h, w, k, stride, pad, n, x_signed, y_dtype of the second layer, shortcut, copy of the first output)
FUSED_CASES = [
    (56, 56, 3, 1, 1, 4, False, synth.U8, True, True),       # 98 tiles: one per CTA
    (56, 56, 3, 1, 1, 32, False, synth.U8, True, False),     # 784 tiles: five or six per CTA, every ring wraps
    (30, 30, 3, 1, 1, 9, False, synth.S8, False, True),      # ragged last tile, signed output, no shortcut
    (28, 28, 1, 1, 0, 12, True, synth.U8, True, True),       # a single tap per tile, signed input
    (31, 31, 3, 2, 0, 10, True, synth.S8, True, False),      # stride 2 without padding
    (20, 20, 4, 1, 1, 12, False, synth.U8, False, True),     # sixteen taps: more taps than stages (two rounds per tile)
    (56, 56, 3, 1, 1, 64, False, synth.U8, True, True),      # 1568 tiles: ten or eleven per CTA
    (56, 56, 3, 1, 1, 256, False, synth.U8, True, False),    # the bench shape: 6272 tiles, tensors beyond the L2 cache
]


def _pair(rng, h, w, k, stride, pad, xs, y_dtype, with_res):
    first = random_conv_layer(rng, h=h, w=w, c=64, c_out=64, k=k, stride=stride, pad=pad, x_signed=xs, y_dtype=synth.U8,
                              with_res=False)
    second = random_conv_layer(rng, h=first.ho, w=first.wo, c=64, c_out=256, k=1, stride=1, pad=0, x_signed=False,
                               y_dtype=y_dtype, with_res=with_res, fl_x=first.fl_y)
    return first, second


@pytest.mark.parametrize("case", range(len(FUSED_CASES)))
def test_conv_pointwise_fused(ref, case):
    a = api()
    h, w, k, stride, pad, n, xs, y_dtype, with_res, dump = FUSED_CASES[case]
    rng = np.random.default_rng(1500 + case)
    first, second = _pair(rng, h, w, k, stride, pad, xs, y_dtype, with_res)
    x = random_input(rng, n, first)
    assert x.size >= 128 * 1024
    res = random_residual(rng, n, second) if with_res else None
    want_mid = ref.run_layer(first, x, None)
    want = ref.run_layer(second, want_mid, res)
    # the cases must exercise the clip as well as the interior of the 8-bit range
    assert 0.02 < np.mean(want_mid == 0) < 0.98
    y_mid = Guarded((n, first.ho, first.wo, 64), torch.uint8) if dump else None
    y = Guarded((n, first.ho, first.wo, 256), a.torch_dtype(y_dtype))
    before = a.f8_tc_launch_count()
    a.f8_conv_pointwise_fixed(a.conv_desc(first, n), a.conv_desc(second, n), a.to_device(x), a.to_device(first.weight),
                              a.to_device(first.bias), a.to_device(second.weight), a.to_device(second.bias),
                              a.to_device(res) if with_res else None, y_mid.t if dump else None, y.t)
    torch.cuda.synchronize()
    a.f8_device_status()
    assert a.f8_tc_launch_count() - before == 1
    assert y.intact(), "the kernel wrote outside its output buffer"
    if dump:
        assert y_mid.intact(), "the kernel wrote outside the copy of the first layer's output"
        assert_equal_arrays(y_mid.t.cpu().numpy(), want_mid, "first layer: ")
    assert_equal_arrays(y.t.cpu().numpy(), want, "second layer: ")


def test_conv_pointwise_fused_rejects_what_it_cannot_run():
    a = api()
    rng = np.random.default_rng(1600)
    first, second = _pair(rng, 56, 56, 3, 1, 1, False, synth.U8, False)
    n = 2
    x = a.to_device(random_input(rng, n, first))
    w1, b1, w2, b2 = (a.to_device(t) for t in (first.weight, first.bias, second.weight, second.bias))
    y = torch.empty((n, 56, 56, 256), dtype=torch.uint8, device="cuda")
    d1, d2 = a.conv_desc(first, n), a.conv_desc(second, n)
    d2.fl_x = (d2.fl_x + 1) % 8           # the second layer no longer continues the first
    with pytest.raises(a.F8Error) as e:
        a.f8_conv_pointwise_fixed(d1, d2, x, w1, b1, w2, b2, None, None, y)
    assert a.STATUS_NAMES[e.value.status] == "F8_ERR_DTYPE"
    d2 = a.conv_desc(second, n)
    d2.c_out = 128                         # a width the kernel does not take
    with pytest.raises(a.F8Error) as e:
        a.f8_conv_pointwise_fixed(d1, d2, x, w1, b1, w2, b2, None, None, y)
    assert a.STATUS_NAMES[e.value.status] == "F8_ERR_UNSUPPORTED"
    d1 = a.conv_desc(first, 0)
    d2 = a.conv_desc(second, 0)
    a.f8_conv_pointwise_fixed(d1, d2, x, w1, b1, w2, b2, None, None, y)      # an empty batch is not an error


def test_conv_pointwise_fused_many_launches(ref):
    """Forty launches back to back (no synchronisation in between) over rotating buffers, every output compared with the
    oracle's: the two producer warps, the issuer and the epilogue run at whatever skew the memory system gives them."""
    a = api()
    rng = np.random.default_rng(1700)
    first, second = _pair(rng, 56, 56, 3, 1, 1, False, synth.U8, True)
    n, sets = 48, 4
    w1, b1, w2, b2 = (a.to_device(t) for t in (first.weight, first.bias, second.weight, second.bias))
    xs, rs, wants, ys = [], [], [], []
    for _ in range(sets):
        x = random_input(rng, n, first)
        res = random_residual(rng, n, second)
        wants.append(ref.run_layer(second, ref.run_layer(first, x, None), res))
        xs.append(a.to_device(x))
        rs.append(a.to_device(res))
    d1, d2 = a.conv_desc(first, n), a.conv_desc(second, n)
    for rep in range(10):
        ys = [Guarded((n, 56, 56, 256), torch.uint8) for _ in range(sets)]
        for i in range(sets):
            a.f8_conv_pointwise_fixed(d1, d2, xs[i], w1, b1, w2, b2, rs[i], None, ys[i].t)
        torch.cuda.synchronize()
        a.f8_device_status()
        for i in range(sets):
            assert ys[i].intact()
            assert_equal_arrays(ys[i].t.cpu().numpy(), wants[i], f"round {rep}, set {i}: ")
