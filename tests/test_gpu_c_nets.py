"""Whole-network parity through f8_net_forward: every layer's output equals the oracle's, bit for bit."""
import numpy as np
import pytest
import torch

from paper_2202_05239_b200 import synth
from gpu_util import api, Guarded, assert_equal_arrays

pytestmark = pytest.mark.gpu


def _layer_shape(l, batch):
    return (batch, l.c_out) if l.kind in (synth.LINEAR, synth.GAP) else (batch, l.ho, l.wo, l.c_out)


def _compare_net(ref, name, batch, image, force_direct=False, seed=0, plan_off=0, micro_batch=0, lanes=0):
    """Every layer's output against the oracle.  The dump buffers, the network output and the workspace sit between
    poisoned guard bands that must come back untouched."""
    a = api()
    layers = synth.make_net(name, seed, image=image)
    x = synth.draw_image(batch, seed + 1, image, image)
    want = ref.net_forward(layers, x)
    a.f8_debug_force_direct(force_direct)
    a.f8_debug_plan_options(plan_off)
    a.f8_debug_set_micro_batch(micro_batch)
    a.f8_debug_set_lanes(lanes)
    before = a.f8_tc_launch_count()
    try:
        net = a.Net(layers, batch)
        guards = [Guarded(_layer_shape(l, batch), a.torch_dtype(l.y_dtype)) for l in layers]
        dump = [g.t for g in guards]
        out = Guarded((batch,) + net.out_shape, net.out_dtype)
        ws = Guarded((net.workspace_bytes(batch),), torch.uint8)
        net.forward(a.to_device(x), out=out.t, workspace=ws.t, dump=dump)
        torch.cuda.synchronize()
        a.f8_device_status()
    finally:
        a.f8_debug_force_direct(False)
        a.f8_debug_plan_options(0)
        a.f8_debug_set_micro_batch(0)
        a.f8_debug_set_lanes(0)
    if lanes:
        assert net.lanes == lanes
    if micro_batch:
        runs, images = net.micro_batching()
        assert runs >= 1 and images == micro_batch, "the forward pass was not micro-batched"
    for i, l in enumerate(layers):
        got = dump[i].cpu().numpy().reshape(want[i + 1].shape)
        assert_equal_arrays(got, want[i + 1], f"{name} layer {i} ({l.name}): ")
        assert guards[i].intact(), f"{name} layer {i} ({l.name}): bytes next to the dump buffer were overwritten"
    assert np.array_equal(out.t.cpu().numpy(), want[-1])
    assert out.intact() and ws.intact(), "bytes next to the output or the workspace were overwritten"
    # one launch per layer, except that a sibling layer is written by its parent's launch and a first layer may take
    # the pooling layer behind it along
    # ... and a 64 -> 64 convolution runs in one launch with the 64 -> 256 pointwise layer behind it
    fused = net.fused_pairs
    if plan_off & a.PLAN_OFF_LAYER_FUSION or force_direct:
        assert fused == 0
    elif name == "resnet50" and image == 224 and not micro_batch:
        assert fused == 3 * (2 if lanes == 2 else 1), "the three bottleneck tails of the first stage should each be one launch"
    assert net.last_launch_count >= sum(1 for l in layers if l.kind != synth.SIBLING) - 1 - fused
    tc = a.f8_tc_launch_count() - before
    if force_direct:
        assert tc == 0
    elif image == 224 and not micro_batch and lanes != 2:
        # every dense layer whose input is at least 128 KiB and has c % 16 == 0 (or is a packed stem)
        assert tc >= sum(1 for l in layers if l.kind == synth.CONV and l.c % 16 == 0 and batch * l.h * l.w * l.c >= 131072) - fused
    net.close()


@pytest.mark.parametrize("name", ["resnet18", "resnet50", "mobilenetv2", "mobilenetv1"])
def test_net_parity_cuda_core_path(ref, name):
    _compare_net(ref, name, 2, 64, force_direct=True)


@pytest.mark.parametrize("name,batch,image", [("resnet18", 3, 224), ("resnet50", 2, 224), ("mobilenetv2", 3, 224),
                                              ("resnet50", 1, 224), ("resnet18", 5, 96), ("mobilenetv1", 3, 224),
                                              ("mobilenetv2", 1, 224), ("resnet18", 1, 224), ("mobilenetv1", 1, 224)])
def test_net_parity(ref, name, batch, image):
    _compare_net(ref, name, batch, image)


@pytest.mark.parametrize("name", ["resnet50", "resnet18", "mobilenetv2", "mobilenetv1"])
def test_net_parity_batch_64_every_layer(ref, name):
    """Throughput batches: at 64 images every CTA of the tensor-core kernel walks many tiles in the early stages."""
    _compare_net(ref, name, 64, 224)


def _off_masks():
    from paper_2202_05239_b200 import api as a
    return [a.PLAN_OFF_STEM_KERNEL, a.PLAN_OFF_STEM_POOL_FUSION, a.PLAN_OFF_LAYER_OVERLAP, a.PLAN_OFF_LANES,
            a.PLAN_OFF_DUAL_ISSUE | a.PLAN_OFF_ALT_PRODUCERS, a.PLAN_OFF_RESIDENT_WEIGHTS, a.PLAN_OFF_PAIRS,
            a.PLAN_SYNC_LAYERS, a.PLAN_OFF_LAYER_FUSION]


@pytest.mark.parametrize("case", range(9))
def test_net_parity_with_planning_choices_switched_off(ref, case):
    """The alternative code paths behind f8_debug_plan_options give the same bits."""
    _compare_net(ref, "resnet50", 4, 224, plan_off=_off_masks()[case])


@pytest.mark.parametrize("name,batch,micro,direct", [("resnet50", 8, 3, False), ("resnet18", 7, 2, False), ("mobilenetv2", 5, 2, False),
                                                     ("mobilenetv1", 6, 4, False), ("resnet18_siblings", 5, 2, False),
                                                     ("resnet50", 3, 1, True), ("resnet50", 64, 16, False)])
def test_net_parity_micro_batched(ref, name, batch, micro, direct):
    """Depth-first execution of runs of layers over micro-batches (tensors inside a run hold one micro-batch and are
    reused; the last micro-batch may be ragged): every layer's output is unchanged."""
    _compare_net(ref, name, batch, 224 if not direct else 64, force_direct=direct, micro_batch=micro)


@pytest.mark.parametrize("name,batch,micro", [("resnet50", 5, 0), ("resnet18", 2, 0), ("mobilenetv2", 7, 0), ("mobilenetv1", 4, 0),
                                              ("resnet18_siblings", 3, 0), ("resnet50", 9, 2)])
def test_net_parity_two_lanes(ref, name, batch, micro):
    """The batch cut into two halves (the first one larger when the batch is odd) that run as two passes on two
    streams, launched alternately -- optionally with micro-batched runs inside each lane: every layer unchanged."""
    _compare_net(ref, name, batch, 224, lanes=2, micro_batch=micro)


@pytest.mark.parametrize("which", ["walk", "strip"])
def test_mobilenet_parity_with_the_older_depthwise_kernels(ref, which):
    """Stride-1 depthwise layers default to the packed-dot-product kernel; the row-walking kernel and the strip kernel
    behind it stay selectable and must give the same bits."""
    a = api()
    off = a.PLAN_OFF_DW_DP4A | (a.PLAN_OFF_DW_WALK if which == "strip" else 0)
    _compare_net(ref, "mobilenetv1", 3, 224, plan_off=off)


def _sampled_full_batch(ref, name, batch, samples):
    """The timed configuration: one full-batch launch with every layer dumped; images are independent, so the oracle
    checks a sample of them one by one, every layer."""
    a = api()
    layers = synth.make_net(name, 0)
    x = synth.draw_image(batch, 1)
    net = a.Net(layers, batch)
    dump = [net.layer_output(i, batch) for i in range(len(layers))]
    out = net.forward(a.to_device(x), dump=dump)
    torch.cuda.synchronize()
    a.f8_device_status()
    for i in samples:
        want = ref.net_forward(layers, x[i:i + 1])
        for li, l in enumerate(layers):
            got = dump[li][i:i + 1].cpu().numpy().reshape(want[li + 1].shape)
            assert_equal_arrays(got, want[li + 1], f"{name} image {i} layer {li} ({l.name}): ")
        assert np.array_equal(out[i:i + 1].cpu().numpy(), want[-1])
    del dump
    net.close()


@pytest.mark.parametrize("name,batch", [("resnet18", 256), ("resnet50", 256), ("mobilenetv1", 256)])
def test_full_batch_sampled_images_every_layer(ref, name, batch):
    _sampled_full_batch(ref, name, batch, (0, 101, 255))


def test_resnet50_full_batch_sampled_images(ref):
    """The benchmark configuration (batch 256): images are independent, so the oracle checks a sample of
    them one by one against the logits of the full-batch launch."""
    a = api()
    batch = 256
    layers = synth.make_net("resnet50", 0)
    x = synth.draw_image(batch, 1)
    net = a.Net(layers, batch)
    out = net.forward(a.to_device(x))
    torch.cuda.synchronize()
    a.f8_device_status()
    got = out.cpu().numpy()
    for i in (0, 77, 128, 255):
        want = ref.net_forward(layers, x[i:i + 1], keep_all=False)[-1]
        assert np.array_equal(got[i:i + 1], want), f"image {i}"
    # a second pass over the same buffers gives the same bits (no state leaks between calls)
    out2 = net.forward(a.to_device(x))
    torch.cuda.synchronize()
    assert torch.equal(out, out2)
    net.close()


def test_resnet50_many_back_to_back_passes():
    """Long runs: several hundred forward passes queued without synchronising (each layer's prologue overlaps the tail of
    the one before, across passes too), then the pipelined host-to-host path.  Barrier-protocol mistakes that a single
    pass never meets show up here as a device fault, a timed-out wait or different bits."""
    a = api()
    batch = 256
    layers = synth.make_net("resnet50", 0)
    x_host = torch.from_numpy(synth.draw_image(batch, 3)).pin_memory()
    x = x_host.cuda()
    net = a.Net(layers, batch)
    out = torch.empty((batch, 1000), dtype=torch.int32, device="cuda")
    ws = torch.empty(net.workspace_bytes(batch), dtype=torch.uint8, device="cuda")
    net.forward(x, out=out, workspace=ws)
    torch.cuda.synchronize()
    first = out.clone()
    for _ in range(500):
        net.forward(x, out=out, workspace=ws)
    torch.cuda.synchronize()
    a.f8_device_status()
    assert torch.equal(out, first)
    pipe = a.HostPipeline(layers, batch, depth=2)
    ys = [torch.empty((batch, 1000), dtype=torch.int32).pin_memory() for _ in range(2)]
    for i in range(300):
        pipe.submit(x_host, ys[i & 1])
    pipe.wait()
    a.f8_device_status()
    assert torch.equal(ys[0], first.cpu()) and torch.equal(ys[1], first.cpu())
    pipe.close()
    net.close()


def test_workspace_too_small_is_rejected():
    a = api()
    layers = synth.make_net("resnet18", 0, image=64)
    net = a.Net(layers, 2)
    x = a.to_device(synth.draw_image(2, 0, 64, 64))
    ws = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(a.F8Error) as e:
        net.forward(x, workspace=ws)
    assert e.value.status == 8
    net.close()


def test_host_pipeline_matches_oracle(ref):
    """Pipelined host-to-host forward passes (copies overlapped with compute, two slots): five different batches in
    flight one after the other, every result equal to the oracle's logits."""
    a = api()
    batch, image = 3, 96
    layers = synth.make_net("resnet18", 0, image=image)
    pipe = a.HostPipeline(layers, batch, depth=2)
    xs = [torch.from_numpy(synth.draw_image(batch, 10 + i, image, image)).pin_memory() for i in range(5)]
    ys = [torch.empty((batch, 1000), dtype=torch.int32).pin_memory() for _ in range(5)]
    for x, y in zip(xs, ys):
        pipe.submit(x, y)
    pipe.wait()
    a.f8_device_status()
    for i, (x, y) in enumerate(zip(xs, ys)):
        want = ref.net_forward(layers, x.numpy(), keep_all=False)[-1]
        assert np.array_equal(y.numpy(), want), f"batch {i}"
    pipe.close()
