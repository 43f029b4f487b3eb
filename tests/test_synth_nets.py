"""The synthetic networks: shapes are consistent and, run through the oracle, activations stay alive."""
import numpy as np
import pytest

from paper_2202_05239_b200 import synth


@pytest.mark.parametrize("name,n_layers,gmac", [("resnet18", 23, 1.814), ("resnet50", 56, 4.089), ("mobilenetv2", 54, 0.3008), ("mobilenetv1", 29, 0.5688)])
def test_shapes_and_macs(name, n_layers, gmac):
    layers = synth.make_net(name, 0)
    assert len(layers) == n_layers
    assert abs(synth.net_macs_per_image(layers) / 1e9 - gmac) < 2e-3
    shapes = [(224, 224, 3)]
    for l in layers:
        assert shapes[l.src] == (l.h, l.w, l.c)
        if l.res >= 0:
            assert shapes[l.res] == (l.ho, l.wo, l.c_out)
        assert 0 <= l.fl_x <= 8 and 0 <= l.fl_y <= 16
        shapes.append((l.ho, l.wo, l.c_out))
    assert shapes[-1] == (1, 1, 1000)


def test_generators_are_seeded():
    a = synth.make_net("resnet18", 3)
    b = synth.make_net("resnet18", 3)
    c = synth.make_net("resnet18", 4)
    assert all(np.array_equal(x.weight, y.weight) for x, y in zip(a, b) if x.weight is not None)
    assert not np.array_equal(a[0].weight, c[0].weight)
    assert np.array_equal(synth.draw_image(2, 5), synth.draw_image(2, 5))


@pytest.mark.parametrize("name", ["resnet18", "resnet50", "mobilenetv2", "mobilenetv1"])
def test_activations_are_not_degenerate(ref, name):
    """The analytic FL choice keeps every layer's codes spread out (neither all zero nor all clipped)."""
    layers = synth.make_net(name, 0, image=96)
    t = ref.net_forward(layers, synth.draw_image(1, 0, 96, 96))
    for l, y in zip(layers, t[1:]):
        if l.y_dtype == synth.S32:
            continue
        v = y.astype(np.int64)
        hi = 255 if l.y_dtype == synth.U8 else 127
        assert (np.abs(v) == hi).mean() < 0.05, l.name
        assert (v == 0).mean() < 0.8, l.name
        assert v.std() > 8, l.name
