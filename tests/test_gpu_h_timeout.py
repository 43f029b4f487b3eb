"""Failure detection on the device, exercised without harming the GPU: every barrier wait inside the kernels is
bounded, and a wait that runs out records itself in the device status word and lets its kernel return.  Here a
one-thread kernel waits (about a millisecond) on a barrier nothing ever arrives at; the library must report the
time-out with the site of the wait, the context must stay usable, and an ordinary layer must still be bit-exact."""
import numpy as np
import pytest
import torch

from paper_2202_05239_b200 import synth
from gpu_util import api, check_layer, random_conv_layer, random_input

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_the_device_stays_usable(ref):
    a = api()
    a.f8_device_status()                                  # clean to begin with
    a.f8_debug_wait_timeout_probe(1.0)
    torch.cuda.synchronize()                              # the kernel returned by itself
    rng = np.random.default_rng(1)
    layer = random_conv_layer(rng, h=28, w=28, c=128, c_out=128, k=1, stride=1, pad=0, x_signed=False, y_dtype=synth.U8,
                              with_res=False)
    # while the record is pending, a call that would enqueue work reports it instead (no synchronisation involved)
    x = a.to_device(random_input(rng, 2, layer))
    y = torch.empty((2, layer.ho, layer.wo, layer.c_out), dtype=torch.uint8, device="cuda")
    with pytest.raises(a.F8Error) as e:
        a.f8_conv2d_fixed(a.conv_desc(layer, 2), x, a.to_device(layer.weight), a.to_device(layer.bias), None, y)
    assert e.value.status == 11
    with pytest.raises(a.F8Error) as e:
        a.f8_device_status()
    assert e.value.status == 11                           # F8_ERR_TIMEOUT
    assert "site 199" in str(e.value)
    a.f8_device_status()                                  # reading the word cleared it
    check_layer(ref, layer, random_input(rng, 2, layer), expect_tc=True)


def test_net_forward_reports_a_time_out_left_by_an_earlier_pass(ref):
    """A kernel that gives up a wait also stores its code to a word in host memory, which f8_net_forward looks at on
    entry: the time-out is reported by the next pass without anybody calling f8_device_status (and without a
    synchronisation inside the library)."""
    a = api()
    a.f8_device_status()
    layers = synth.make_net("resnet18", 0, image=64)
    net = a.Net(layers, 2)
    x = a.to_device(synth.draw_image(2, 1, 64, 64))
    net.forward(x)
    torch.cuda.synchronize()
    net.forward(x)                                         # nothing to report
    a.f8_debug_wait_timeout_probe(0.5)                     # a time-out between two passes
    net.forward(x)                                         # this pass ends with the word already set
    torch.cuda.synchronize()
    with pytest.raises(a.F8Error) as e:
        net.forward(x)
    assert e.value.status == 11
    with pytest.raises(a.F8Error):
        a.f8_device_status()                               # details and reset
    a.f8_device_status()
    want = ref.net_forward(layers, synth.draw_image(2, 1, 64, 64), keep_all=False)[-1]
    assert np.array_equal(net.forward(x).cpu().numpy(), want)
    net.close()
