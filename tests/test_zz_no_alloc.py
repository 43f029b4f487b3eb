"""The entry point that allocates nothing (``f8_stem_conv2d_fixed_static``).

Some users of this library cannot call cudaMalloc when they need a result: the device may be fully reserved
by another memory pool, or allocation may be forbidden on their code path.  For them the first-layer
convolution exists in a form whose scratch memory is a fixed array inside the library.  This test calls it
through the C ABI twice in a row (the second call with a smaller batch and other data, so anything the first
call left in the shared array would show) and compares each result, bit for bit, with ``f8_conv2d_fixed``.
It lives in a file that pytest collects last so that a failure here cannot hide the other tests.
"""
import numpy as np
import pytest
import torch

from paper_2202_05239_b200 import synth

pytestmark = pytest.mark.gpu


def _stem_layer(seed):
    layers = synth.make_net("resnet50", seed)
    return layers[0]            # 7x7 / 2, 3 -> 64 channels, signed input, ReLU output


def _run_both(api, layer, x_host):
    n = x_host.shape[0]
    x = api.to_device(x_host)
    w, b = api.to_device(layer.weight), api.to_device(layer.bias)
    desc = api.conv_desc(layer, n)
    want = torch.empty((n, layer.ho, layer.wo, layer.c_out), dtype=torch.uint8, device="cuda")
    api.f8_conv2d_fixed(desc, x, w, b, None, want)
    got = torch.full_like(want, 0xAB)
    api.f8_stem_conv2d_fixed_static(desc, x, w, b, got, check_previous=True)
    torch.cuda.synchronize()
    return got, want


def test_static_stem_matches_existing_entry_point_twice_in_a_row():
    from paper_2202_05239_b200 import api
    layer = _stem_layer(0)
    before = torch.cuda.memory_allocated()
    got1, want1 = _run_both(api, layer, synth.draw_image(6, 11))
    assert torch.equal(got1, want1)
    # second call: fewer images, different data, different weights; the shared array still holds call one
    layer2 = _stem_layer(5)
    got2, want2 = _run_both(api, layer2, synth.draw_image(3, 12))
    assert torch.equal(got2, want2)
    del got1, want1, got2, want2
    assert torch.cuda.memory_allocated() <= before      # nothing of torch's is retained by the calls


def test_static_stem_rejects_what_it_cannot_hold():
    from paper_2202_05239_b200 import api
    layer = _stem_layer(0)
    w, b = api.to_device(layer.weight), api.to_device(layer.bias)
    x = torch.zeros((1, 224, 224, 3), dtype=torch.int8, device="cuda")
    y = torch.empty((1, 112, 112, 64), dtype=torch.uint8, device="cuda")
    with pytest.raises(api.F8Error) as e:        # 64 images need more than the 16 MiB array: split the batch
        api.f8_stem_conv2d_fixed_static(api.conv_desc(layer, 64), x, w, b, y)
    assert e.value.status == 8 and "split the batch" in str(e.value)
    small = synth.Layer(synth.CONV, "tiny", 0, -1, 16, 16, 3, 64, 7, 7, 2, 3, synth.S8, synth.U8, synth.U8, 6, 9, 6, 0,
                        layer.weight, layer.bias)
    with pytest.raises(api.F8Error) as e:        # below 128 KiB the ordinary entry point is the one to use
        api.f8_stem_conv2d_fixed_static(api.conv_desc(small, 1), x, w, b, y)
    assert e.value.status == 9
