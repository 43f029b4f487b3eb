"""The entry point that allocates nothing (``f8_stem_conv2d_fixed_static``).

Some users of this library cannot call cudaMalloc when they need a result: the device may be fully reserved
by another memory pool, or allocation may be forbidden on their code path.  For them the first-layer
convolution exists in a form whose scratch memory is a fixed array inside the library.  This test calls it
through the C ABI twice in a row (the second call with a smaller batch and other data, so anything the first
call left in the shared array would show) and compares each result, bit for bit, with ``f8_conv2d_fixed`` and
with the CPU oracle.  It lives in a file that pytest collects last so that a failure here cannot hide the
other tests.
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


def test_static_stem_matches_existing_entry_point_twice_in_a_row(ref):
    from paper_2202_05239_b200 import api
    layer = _stem_layer(0)
    before = torch.cuda.memory_allocated()
    x1 = synth.draw_image(6, 11)
    got1, want1 = _run_both(api, layer, x1)
    assert torch.equal(got1, want1)
    assert np.array_equal(got1.cpu().numpy(), ref.run_layer(layer, x1))
    # second call: fewer images, different data, different weights; the shared array still holds call one
    layer2 = _stem_layer(5)
    x2 = synth.draw_image(3, 12)
    got2, want2 = _run_both(api, layer2, x2)
    assert torch.equal(got2, want2)
    assert np.array_equal(got2.cpu().numpy(), ref.run_layer(layer2, x2))
    del got1, want1, got2, want2
    assert torch.cuda.memory_allocated() <= before      # nothing of torch's is retained by the calls


def test_static_stem_leaves_device_memory_alone_and_covers_its_branches(ref):
    """After a warm-up call (the first call on a device looks the array's address up), further calls must leave the
    amount of free device memory exactly as it was: torch's own counter would not see a cudaMalloc inside the
    library, the driver's does.  The shapes cover the other branches of the entry point: more than four channels,
    signed output, a filter row of more than eight taps, a caller's stream without the status check."""
    from paper_2202_05239_b200 import api
    rng = np.random.default_rng(77)
    side = torch.cuda.Stream()
    cases = [   # (h, w, c, c_out, k, stride, pad, n, x_signed, y_dtype)
        (96, 96, 8, 32, 3, 2, 1, 4, True, synth.S8),
        (160, 160, 3, 48, 11, 4, 5, 3, False, synth.U8),
        (128, 128, 5, 64, 5, 2, 2, 2, True, synth.U8),
    ]
    layer0 = _stem_layer(0)
    _run_both(api, layer0, synth.draw_image(2, 1))          # warm-up: address look-up, torch's pools
    torch.cuda.synchronize()
    for h, w, c, c_out, k, stride, pad, n, xs, y_dtype in cases:
        wgt = np.clip(np.round(rng.normal(0, 20, size=(c_out, k, k, c))), -128, 127).astype(np.int8)
        bias = rng.integers(-4000, 4000, size=c_out).astype(np.int32)
        layer = synth.Layer(synth.CONV, "stem", 0, -1, h, w, c, c_out, k, k, stride, pad, synth.S8 if xs else synth.U8,
                            y_dtype, synth.U8, 6, 8, 3, 0, wgt, bias)
        x_host = (rng.integers(-128, 128, size=(n, h, w, c)).astype(np.int8) if xs
                  else rng.integers(0, 256, size=(n, h, w, c)).astype(np.uint8))
        x, wd, bd = api.to_device(x_host), api.to_device(wgt), api.to_device(bias)
        y = torch.full((n, layer.ho, layer.wo, c_out), 0x5A, dtype=api.torch_dtype(y_dtype), device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        try:
            with torch.cuda.stream(side):
                api.f8_stem_conv2d_fixed_static(api.conv_desc(layer, n), x, wd, bd, y, check_previous=False, stream=side)
        except api.F8Error as e:
            assert e.status == 9, str(e)        # a shape it does not take must say so, not compute something else
            continue
        side.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the amount of free device memory"
        assert np.array_equal(y.cpu().numpy(), ref.run_layer(layer, x_host)), f"case {(h, w, c, c_out, k, stride)}"


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
