"""Host-only checks of the C-ABI library: it loads, exports every declared symbol, and rejects bad
arguments before touching the device (so these run without a GPU)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2202_05239_b200 import build
    return ctypes.CDLL(build.build())


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "f8net.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(f8_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_entry_points():
    names = _declared_symbols()
    for required in ("f8_conv2d_fixed", "f8_dwconv_fixed", "f8_linear_fixed", "f8_net_forward"):
        assert required in names


@pytest.mark.parametrize("name", _declared_symbols())
def test_symbol_is_exported(lib, name):
    assert hasattr(lib, name)


def _desc(**kw):
    from paper_2202_05239_b200.api import ConvDesc
    base = dict(n=1, h=8, w=8, c=16, c_out=16, kh=3, kw=3, stride=1, pad=1, x_dtype=0, y_dtype=0, r_dtype=0,
                fl_x=4, fl_w=7, fl_y=4, fl_r=0)
    base.update(kw)
    return ConvDesc(**base)


@pytest.mark.parametrize("kw,status", [
    (dict(h=0), 2), (dict(kh=20), 2), (dict(x_dtype=2), 3), (dict(y_dtype=7), 3), (dict(fl_x=9), 4),
    (dict(x_dtype=1, fl_x=8), 4), (dict(fl_w=40), 4), (dict(fl_y=9), 4), (dict(fl_x=8, fl_w=24, fl_y=0), 5),
    (dict(c=40000, kh=3, kw=3, h=3, w=3), 7),
])
def test_validation_rejects_without_launching(lib, kw, status):
    from paper_2202_05239_b200 import api
    d = _desc(**kw)
    fake = ctypes.c_void_p(0x1000)       # never dereferenced: validation fails first
    st = api._lib.f8_conv2d_fixed(ctypes.byref(d), fake, fake, None, None, fake, None, 0, None)
    assert st == status, api._lib.f8_last_error()
    assert api._lib.f8_status_str(st).decode() == api.STATUS_NAMES[status]


def test_null_and_alignment_are_reported(lib):
    from paper_2202_05239_b200 import api
    d = _desc()
    assert api._lib.f8_conv2d_fixed(ctypes.byref(d), None, None, None, None, None, None, 0, None) == 1
    a, bad = ctypes.c_void_p(0x1000), ctypes.c_void_p(0x1004)
    assert api._lib.f8_conv2d_fixed(ctypes.byref(d), bad, a, None, None, a, None, 0, None) == 6
    assert api._lib.f8_conv2d_fixed(None, a, a, None, None, a, None, 0, None) == 1
    # residual alignment shift out of range: fl_x + fl_w = 31 vs fl_r = 0
    d = _desc(fl_x=7, fl_w=24, fl_r=0, y_dtype=2, c=1, kh=1, kw=1, pad=0)
    assert api._lib.f8_conv2d_fixed(ctypes.byref(d), a, a, None, a, a, None, 0, None) == 5


def test_depthwise_needs_equal_channels_and_empty_batch_is_a_noop(lib):
    from paper_2202_05239_b200 import api
    a = ctypes.c_void_p(0x1000)
    d = _desc(c_out=32)
    assert api._lib.f8_dwconv_fixed(ctypes.byref(d), a, a, None, None, a, None, 0, None) == 2
    d = _desc(n=0)
    assert api._lib.f8_conv2d_fixed(ctypes.byref(d), None, None, None, None, None, None, 0, None) == 0
    assert api._lib.f8_maxpool_fixed(0, 8, 8, 16, 3, 2, 1, 0, None, None, None) == 0
    assert api._lib.f8_maxpool_fixed(1, 8, 8, 16, 3, 2, 3, 0, a, a, None) == 2
    assert api._lib.f8_global_avgpool_fixed(1, 7, 7, 16, 0, 9, 4, a, a, None) == 4


def test_net_create_validates_graph_and_accumulator_bound(lib):
    import numpy as np
    from paper_2202_05239_b200 import api, synth
    layers = synth.make_net("resnet18", 0, image=32)
    # break the chain: a layer whose input format disagrees with its producer
    layers[3].fl_x += 1
    with pytest.raises(api.F8Error) as e:
        api.Net(layers, 1)
    assert e.value.status == 3
    # an int32 bias that makes the accumulator bound fail
    layers = synth.make_net("resnet18", 0, image=32)
    layers[0].bias = np.full_like(layers[0].bias, 2 ** 31 - 1)
    with pytest.raises(api.F8Error) as e:
        api.Net(layers, 1)
    assert e.value.status == 7


@pytest.mark.parametrize("kw,status", [
    (dict(c_out=0), 2), (dict(k=-3), 2), (dict(fl_x=9), 4), (dict(fl_w_min=5, fl_w_max=4), 4), (dict(fl_w_max=30), 4),
    (dict(eta_out=0.0), 2), (dict(eta_in=float("nan")), 2),
])
def test_fold_validation_rejects_without_launching(lib, kw, status):
    from paper_2202_05239_b200 import api
    base = dict(c_out=8, k=16, fl_x=4, fl_w_min=0, fl_w_max=7, eta_in=0.5, eta_out=0.25)
    base.update(kw)
    d = api.FoldDesc(**base)
    fake = ctypes.c_void_p(0x1000)       # never dereferenced: validation fails first
    st = api._lib.f8_fold_quantize_fixed(ctypes.byref(d), *([fake] * 9), 1 << 20, None)
    assert st == status, api._lib.f8_last_error()


def test_fold_workspace_and_null_are_reported(lib):
    from paper_2202_05239_b200 import api
    d = api.FoldDesc(8, 16, 4, 0, 7, 0.5, 0.25)
    fake = ctypes.c_void_p(0x1000)
    assert api._lib.f8_fold_quantize_fixed(ctypes.byref(d), *([fake] * 8), None, 0, None) == 8
    assert api._lib.f8_fold_quantize_fixed(ctypes.byref(d), *([fake] * 9), 16, None) == 8
    assert api._lib.f8_fold_quantize_fixed(ctypes.byref(d), None, *([fake] * 8), 1 << 20, None) == 1
    assert api._lib.f8_fold_workspace_bytes(ctypes.byref(d)) >= 16384
