"""Pins for the CPU oracle: everything here runs without a GPU.

The oracle is checked against things it did not produce: hand-worked values
(tests/golden), the real-valued definition of Eq. 2 / Eq. 6 evaluated exactly
with Python fractions, torch float64 library routines on the integer tensors,
algebraic identities, and the paper's own identities (Eq. 4, the private-FL
identity of the appendix, the error claim behind Eq. 1).
"""
import json
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from paper_2202_05239_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
U8, S8, S32 = synth.U8, synth.S8, synth.S32


# ---------------------------------------------------------------- P1: hand-worked scalars

def _scalar_cases():
    out = []
    with open(os.path.join(GOLDEN, "shift_round_clip.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                out.append(tuple(int(t) for t in line.split()))
    return out


@pytest.mark.parametrize("acc,s,lo,hi,expected", _scalar_cases())
def test_shift_round_clip_golden(ref, acc, s, lo, hi, expected):
    assert ref.shift_round_clip(acc, s, lo, hi) == expected


def _layer_cases():
    out = {}
    with open(os.path.join(GOLDEN, "conv_handworked.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                d = json.loads(line)
                out[d["name"]] = d
    return out


@pytest.mark.parametrize("name", ["sobel_3x3_s1_p1", "sobel_3x3_s2_p1"])
def test_conv_handworked(ref, name):
    d = _layer_cases()[name]
    x = np.array(d["x"], dtype=np.uint8)[None, :, :, None]
    w = np.array(d["w"], dtype=np.int8)[None, :, :, None]
    y = ref.conv2d(x, w, None, stride=d["stride"], pad=d["pad"], fl_x=0, fl_w=0, fl_y=0, y_dtype=S32)
    assert y[0, :, :, 0].tolist() == d["raw"]


def test_dot_and_residual_handworked(ref):
    cases = _layer_cases()
    d = cases["dot3_bias"]
    x = np.array(d["x"], dtype=np.uint8)[None, :]
    w = np.array(d["w"], dtype=np.int8)[None, :]
    b = np.array([d["bias"]], dtype=np.int32)
    kw = dict(fl_x=d["fl_x"], fl_w=d["fl_w"], fl_y=d["fl_y"])
    assert ref.linear(x, w, b, y_dtype=S32, **kw)[0, 0] == d["raw"]
    assert ref.linear(x, w, b, y_dtype=U8, **kw)[0, 0] == d["u8"]
    # the same dot product as a 1x1 conv whose bias brings the accumulator to 15400, plus a residual
    r = cases["residual_align"]
    bias = np.array([r["acc"] - 13989], dtype=np.int32)
    res = np.array([[[[r["r"]]]]], dtype=np.uint8)
    y = ref.conv2d(x.reshape(1, 1, 1, 3), w.reshape(1, 1, 1, 3), bias, stride=1, pad=0, fl_x=4, fl_w=7,
                   fl_y=r["fl_y"], y_dtype=U8, residual=res, fl_r=r["fl_r"])
    assert y.item() == r["u8"]
    y32 = ref.conv2d(x.reshape(1, 1, 1, 3), w.reshape(1, 1, 1, 3), bias, stride=1, pad=0, fl_x=4, fl_w=7,
                     fl_y=0, y_dtype=S32, residual=res, fl_r=r["fl_r"])
    assert y32.item() == r["aligned_sum"]


def test_gap_handworked(ref):
    d = _layer_cases()["gap_7x7"]
    x = np.array([(37 * i) % 256 for i in range(49)], dtype=np.uint8).reshape(1, 7, 7, 1)
    assert int(x.sum()) == d["sum"]
    assert ref.gap(x, fl_x=d["fl_x"], fl_y=d["fl_y"]).item() == d["u8"]


# ---------------------------------------------------------------- P2/P5: the real-valued definition, exactly

def _quant_real(v: Fraction, fl: int, lo: int, hi: int) -> int:
    """Eq. 2 / signed fix_quant as written: clip(v 2^FL) then round (half up); returns the code."""
    t = v * Fraction(2) ** fl
    t = min(max(t, Fraction(lo)), Fraction(hi))
    return math.floor(t + Fraction(1, 2))


def _brute_conv(x, w, b, res, stride, pad, fl_x, fl_w, fl_y, fl_r, lo, hi):
    n, h, wd, ci = x.shape
    co, kh, kw, _ = w.shape
    ho, wo = (h + 2 * pad - kh) // stride + 1, (wd + 2 * pad - kw) // stride + 1
    y = np.zeros((n, ho, wo, co), dtype=np.int64)
    for i in range(n):
        for oh in range(ho):
            for ow in range(wo):
                for oc in range(co):
                    v = Fraction(int(b[oc]), 2 ** (fl_x + fl_w))
                    for r in range(kh):
                        for s in range(kw):
                            ih, iw = oh * stride + r - pad, ow * stride + s - pad
                            if 0 <= ih < h and 0 <= iw < wd:
                                for c in range(ci):
                                    v += Fraction(int(w[oc, r, s, c]), 2 ** fl_w) * Fraction(int(x[i, ih, iw, c]), 2 ** fl_x)
                    if res is not None:
                        v += Fraction(int(res[i, oh, ow, oc]), 2 ** fl_r)
                    y[i, oh, ow, oc] = _quant_real(v, fl_y, lo, hi)
    return y


@pytest.mark.parametrize("seed", range(6))
def test_conv_equals_real_valued_definition(ref, seed):
    rng = np.random.default_rng(seed)
    signed_x = bool(seed % 2)
    relu = seed % 3 != 0
    stride = 1 + seed % 2
    k = [1, 3, 3, 5, 3, 1][seed]
    pad = k // 2 if seed != 3 else 1
    n, h, wd, ci, co = 2, 5 + seed % 3, 6, 3 + seed, 4
    x = rng.integers(-128 if signed_x else 0, 128 if signed_x else 256, size=(n, h, wd, ci)).astype(
        np.int8 if signed_x else np.uint8)
    w = rng.integers(-128, 128, size=(co, k, k, ci)).astype(np.int8)
    fl_x, fl_w = int(rng.integers(0, 8)), int(rng.integers(0, 10))
    b = rng.integers(-3000, 3000, size=co).astype(np.int32)
    ho, wo = (h + 2 * pad - k) // stride + 1, (wd + 2 * pad - k) // stride + 1
    use_res = seed % 2 == 0
    res = rng.integers(0, 256, size=(n, ho, wo, co)).astype(np.uint8) if use_res else None
    fl_r = int(rng.integers(0, 9))
    for fl_y in (0, 3, 7, min(8, fl_x + fl_w + 2)):
        lo, hi = (0, 255) if relu else (-127, 127)
        got = ref.conv2d(x, w, b, stride=stride, pad=pad, fl_x=fl_x, fl_w=fl_w, fl_y=fl_y,
                         y_dtype=U8 if relu else S8, residual=res, fl_r=fl_r)
        want = _brute_conv(x, w, b, res, stride, pad, fl_x, fl_w, fl_y, fl_r, lo, hi)
        assert np.array_equal(got.astype(np.int64), want)


def test_double_precision_invariant(ref):
    """code == clip(floor(acc 2^(FLy-FA) + 0.5)) evaluated in double (exact for |acc| < 2^31)."""
    rng = np.random.default_rng(1)
    acc = np.concatenate([rng.integers(-2 ** 31, 2 ** 31, size=4000), rng.integers(-70000, 70000, size=4000),
                          np.arange(-1100, 1100)])
    for s in (-8, -3, 0, 1, 2, 7, 12, 20, 31):
        for lo, hi in ((0, 255), (-127, 127)):
            want = np.clip(np.floor(acc.astype(np.float64) * 2.0 ** (-s) + 0.5), lo, hi).astype(np.int64)
            got = np.array([ref.shift_round_clip(int(a), s, lo, hi) for a in acc])
            assert np.array_equal(got, want)


def test_round_then_clip_equals_clip_then_round(ref):
    for acc in range(-40000, 40000, 37):
        for s in (1, 4, 7):
            for lo, hi in ((0, 255), (-127, 127)):
                v = Fraction(acc, 2 ** s)
                clip_then_round = math.floor(min(max(v, lo), hi) + Fraction(1, 2))
                assert ref.shift_round_clip(acc, s, lo, hi) == clip_then_round


# ---------------------------------------------------------------- P3: library routines on float64 copies

@pytest.mark.parametrize("k,stride,pad,signed", [(3, 1, 1, False), (3, 2, 1, True), (1, 1, 0, False), (1, 2, 0, True),
                                                 (7, 2, 3, True), (5, 1, 0, False), (3, 2, 0, False)])
def test_conv_accumulator_vs_torch(ref, k, stride, pad, signed):
    rng = np.random.default_rng(k * 10 + stride)
    n, h, wd, ci, co = 2, 13, 11, 5, 7
    x = rng.integers(-128 if signed else 0, 128 if signed else 256, size=(n, h, wd, ci)).astype(
        np.int8 if signed else np.uint8)
    w = rng.integers(-128, 128, size=(co, k, k, ci)).astype(np.int8)
    b = rng.integers(-10 ** 5, 10 ** 5, size=co).astype(np.int32)
    got = ref.conv2d(x, w, b, stride=stride, pad=pad, fl_x=3, fl_w=4, fl_y=0, y_dtype=S32)
    xt = torch.from_numpy(x.astype(np.float64)).permute(0, 3, 1, 2)
    wt = torch.from_numpy(w.astype(np.float64)).permute(0, 3, 1, 2)
    want = F.conv2d(xt, wt, torch.from_numpy(b.astype(np.float64)), stride=stride, padding=pad)
    assert np.array_equal(got.astype(np.float64), want.permute(0, 2, 3, 1).numpy())


def test_dwconv_accumulator_vs_torch(ref):
    rng = np.random.default_rng(5)
    n, h, wd, c = 2, 9, 10, 6
    x = rng.integers(0, 256, size=(n, h, wd, c)).astype(np.uint8)
    w = rng.integers(-128, 128, size=(c, 3, 3)).astype(np.int8)
    for stride in (1, 2):
        got = ref.dwconv(x, w, None, stride=stride, pad=1, fl_x=0, fl_w=0, fl_y=0, y_dtype=S32)
        xt = torch.from_numpy(x.astype(np.float64)).permute(0, 3, 1, 2)
        wt = torch.from_numpy(w.astype(np.float64))[:, None]
        want = F.conv2d(xt, wt, None, stride=stride, padding=1, groups=c)
        assert np.array_equal(got.astype(np.float64), want.permute(0, 2, 3, 1).numpy())


def test_maxpool_and_linear_vs_torch(ref):
    rng = np.random.default_rng(6)
    x = rng.integers(0, 256, size=(2, 11, 12, 5)).astype(np.uint8)
    got = ref.maxpool(x, k=3, stride=2, pad=1)
    want = F.max_pool2d(torch.from_numpy(x.astype(np.float64)).permute(0, 3, 1, 2), 3, 2, 1).permute(0, 2, 3, 1)
    assert np.array_equal(got.astype(np.float64), want.numpy())
    xs = rng.integers(-128, 128, size=(2, 7, 9, 3)).astype(np.int8)      # all-negative windows must stay negative
    xs[0, :3, :3, 0] = -100
    got = ref.maxpool(xs, k=3, stride=2, pad=1)
    want = F.max_pool2d(torch.from_numpy(xs.astype(np.float64)).permute(0, 3, 1, 2), 3, 2, 1).permute(0, 2, 3, 1)
    assert np.array_equal(got.astype(np.float64), want.numpy())
    a = rng.integers(0, 256, size=(4, 33)).astype(np.uint8)
    w = rng.integers(-128, 128, size=(10, 33)).astype(np.int8)
    b = rng.integers(-1000, 1000, size=10).astype(np.int32)
    got = ref.linear(a, w, b, fl_x=5, fl_w=7, fl_y=0, y_dtype=S32)
    want = F.linear(torch.from_numpy(a.astype(np.float64)), torch.from_numpy(w.astype(np.float64)),
                    torch.from_numpy(b.astype(np.float64)))
    assert np.array_equal(got.astype(np.float64), want.numpy())


# ---------------------------------------------------------------- P4: algebra

def test_identity_kernel_returns_input(ref):
    rng = np.random.default_rng(7)
    x = rng.integers(0, 256, size=(1, 6, 5, 4)).astype(np.uint8)
    w = np.zeros((4, 3, 3, 4), dtype=np.int8)
    for c in range(4):
        w[c, 1, 1, c] = 64                      # 1.0 in format FL_w = 6
    y = ref.conv2d(x, w, None, stride=1, pad=1, fl_x=5, fl_w=6, fl_y=5, y_dtype=U8)
    assert np.array_equal(y, x)


def test_zero_weights_pass_residual_through(ref):
    rng = np.random.default_rng(8)
    x = rng.integers(0, 256, size=(1, 4, 4, 8)).astype(np.uint8)
    r = rng.integers(-127, 128, size=(1, 4, 4, 3)).astype(np.int8)
    w = np.zeros((3, 1, 1, 8), dtype=np.int8)
    y = ref.conv2d(x, w, None, stride=1, pad=0, fl_x=4, fl_w=7, fl_y=3, y_dtype=S8, residual=r, fl_r=3)
    assert np.array_equal(y, r)
    # a coarser output format halves (rounding half up), a finer one doubles and saturates
    y = ref.conv2d(x, w, None, stride=1, pad=0, fl_x=4, fl_w=7, fl_y=2, y_dtype=S8, residual=r, fl_r=3)
    assert np.array_equal(y, np.floor(r.astype(np.float64) / 2 + 0.5).astype(np.int8))
    y = ref.conv2d(x, w, None, stride=1, pad=0, fl_x=4, fl_w=7, fl_y=4, y_dtype=S8, residual=r, fl_r=3)
    assert np.array_equal(y, np.clip(r.astype(np.int64) * 2, -127, 127).astype(np.int8))


def test_depthwise_is_block_diagonal_dense(ref):
    rng = np.random.default_rng(9)
    c = 5
    x = rng.integers(0, 256, size=(2, 7, 8, c)).astype(np.uint8)
    wd = rng.integers(-128, 128, size=(c, 3, 3)).astype(np.int8)
    b = rng.integers(-500, 500, size=c).astype(np.int32)
    dense = np.zeros((c, 3, 3, c), dtype=np.int8)
    for ch in range(c):
        dense[ch, :, :, ch] = wd[ch]
    for stride in (1, 2):
        kw = dict(stride=stride, pad=1, fl_x=4, fl_w=6, fl_y=3, y_dtype=U8)
        assert np.array_equal(ref.dwconv(x, wd, b, **kw), ref.conv2d(x, dense, b, **kw))


def test_linear_is_1x1_conv_and_gap_is_unit_depthwise(ref):
    rng = np.random.default_rng(10)
    a = rng.integers(0, 256, size=(3, 20)).astype(np.uint8)
    w = rng.integers(-128, 128, size=(6, 20)).astype(np.int8)
    b = rng.integers(-500, 500, size=6).astype(np.int32)
    kw = dict(fl_x=6, fl_w=7, fl_y=4, y_dtype=S8)
    y1 = ref.linear(a, w, b, **kw)
    y2 = ref.conv2d(a.reshape(3, 1, 1, 20), w.reshape(6, 1, 1, 20), b, stride=1, pad=0, **kw)
    assert np.array_equal(y1, y2.reshape(3, 6))
    x = rng.integers(0, 256, size=(2, 7, 7, 4)).astype(np.uint8)
    g = ref.gap(x, fl_x=5, fl_y=6)
    ones = np.ones((4, 7, 7), dtype=np.int8)
    # unit weights with FL_w = 6 = ceil(log2 49): the accumulator has format FL_x + 6
    d = ref.dwconv(x, ones, None, stride=1, pad=0, fl_x=5, fl_w=6, fl_y=6, y_dtype=U8)
    assert np.array_equal(g, d.reshape(2, 4))


def test_scaling_identities_and_saturation(ref):
    rng = np.random.default_rng(11)
    x = rng.integers(0, 100, size=(1, 5, 5, 6)).astype(np.uint8)
    w = rng.integers(-128, 128, size=(4, 3, 3, 6)).astype(np.int8)
    y1 = ref.conv2d(x, w, None, stride=1, pad=1, fl_x=4, fl_w=7, fl_y=4, y_dtype=S8)
    # the codes 2x in format FL_x + 1 stand for the same real numbers
    y2 = ref.conv2d((2 * x).astype(np.uint8), w, None, stride=1, pad=1, fl_x=5, fl_w=7, fl_y=4, y_dtype=S8)
    assert np.array_equal(y1, y2)
    # linearity of the accumulator in the weights
    w2 = rng.integers(-60, 60, size=w.shape).astype(np.int8)
    w1 = rng.integers(-60, 60, size=w.shape).astype(np.int8)
    kw = dict(stride=1, pad=1, fl_x=0, fl_w=0, fl_y=0, y_dtype=S32)
    assert np.array_equal(ref.conv2d(x, w1, None, **kw) + ref.conv2d(x, w2, None, **kw),
                          ref.conv2d(x, (w1 + w2).astype(np.int8), None, **kw))
    ones = np.full((1, 3, 3, 8), 255, dtype=np.uint8)
    hi = np.full((2, 3, 3, 8), 127, dtype=np.int8)
    lo = np.full((2, 3, 3, 8), -128, dtype=np.int8)
    assert (ref.conv2d(ones, hi, None, stride=1, pad=1, fl_x=4, fl_w=7, fl_y=4, y_dtype=U8) == 255).all()
    assert (ref.conv2d(ones, lo, None, stride=1, pad=1, fl_x=4, fl_w=7, fl_y=4, y_dtype=U8) == 0).all()
    assert (ref.conv2d(ones, lo, None, stride=1, pad=1, fl_x=4, fl_w=7, fl_y=4, y_dtype=S8) == -127).all()


def test_maxpool_commutes_with_requantisation(ref):
    """max is monotone, so pooling before or after a (monotone) format change gives the same codes."""
    rng = np.random.default_rng(12)
    x = rng.integers(0, 256, size=(1, 9, 9, 4)).astype(np.uint8)
    ident = np.zeros((4, 1, 1, 4), dtype=np.int8)
    for c in range(4):
        ident[c, 0, 0, c] = 1
    requant = lambda t: ref.conv2d(t, ident, None, stride=1, pad=0, fl_x=6, fl_w=0, fl_y=4, y_dtype=U8)
    assert np.array_equal(ref.maxpool(requant(x), k=3, stride=2, pad=1), requant(ref.maxpool(x, k=3, stride=2, pad=1)))


def test_accumulator_range_is_reported(ref):
    x = np.full((1, 1, 1, 4), 255, dtype=np.uint8)
    w = np.full((1, 1, 1, 4), 127, dtype=np.int8)
    b = np.array([2 ** 31 - 1000], dtype=np.int32)
    with pytest.raises(RuntimeError):
        ref.conv2d(x, w, b, stride=1, pad=0, fl_x=0, fl_w=0, fl_y=0, y_dtype=U8)


# ---------------------------------------------------------------- P6: the paper's identities

def _fix_quant_real(ref, xs, fl, signed):
    """Real-valued fix_quant of Eq. 2 / its signed form through the oracle's integer quantizer.

    Inputs are put on a 2^-24 grid first so that the numerator is an exact integer."""
    lo, hi = (-127, 127) if signed else (0, 255)
    num = np.floor(xs * 2.0 ** 24 + 0.5).astype(np.int64)
    return np.array([ref.shift_round_clip(int(a), 24 - fl, lo, hi) for a in num]) * 2.0 ** (-fl)


def test_pact_equals_scaled_fix_quant(ref):
    """Eq. 4: PACT(x) = eta fix_quant(x / eta), eta = 2^FL alpha / (2^WL - 1), with M = 2^WL - 1."""
    rng = np.random.default_rng(13)
    m = 255.0
    for fl in (0, 3, 5, 8):
        alpha = m / 2.0 ** fl * 2.0 ** int(rng.integers(-2, 3))    # eta a power of two keeps x/eta on the grid
        eta = 2.0 ** fl * alpha / m
        x = np.floor(rng.normal(0, alpha / 2, size=2000) * 2.0 ** 12 + 0.5) / 2.0 ** 12
        pact = alpha / m * np.floor(m / alpha * np.clip(x, 0, alpha) + 0.5)
        assert np.allclose(pact, eta * _fix_quant_real(ref, x / eta, fl, False), rtol=0, atol=1e-12)


def test_private_fractional_length_is_a_shift(ref):
    """Appendix on private FLs: at a shared clipping level, quantising with FL instead of the master's
    FL^m is fix_quant with the clipping level scaled by 2^(FL^m - FL); in codes, the sibling with the
    coarser format equals the rounded right shift of the finer one wherever neither clips."""
    rng = np.random.default_rng(14)
    acc = rng.integers(-2 ** 14, 2 ** 14, size=3000)
    for fl_m, fl in ((6, 5), (6, 4), (5, 3)):
        fine = np.array([ref.shift_round_clip(int(a), 12 - fl_m, -10 ** 9, 10 ** 9) for a in acc])
        coarse = np.array([ref.shift_round_clip(int(a), 12 - fl, -10 ** 9, 10 ** 9) for a in acc])
        # both stand for the same real number to within half a step of the coarser format
        assert np.all(np.abs(fine * 2.0 ** -fl_m - coarse * 2.0 ** -fl) <= 2.0 ** -(fl + 1) + 2.0 ** -(fl_m + 1))
        # and the ranges differ exactly by the power of two
        assert 255 * 2.0 ** -fl == 2.0 ** (fl_m - fl) * 255 * 2.0 ** -fl_m


@pytest.mark.parametrize("signed", [True, False])
def test_eq1_format_keeps_relative_error_below_one_percent(ref, signed):
    """Sec. 3.3: with the FL of Eq. 1 the relative (squared) quantisation error of 10 000 Gaussian
    samples stays below 1 % for sigma in [0.1, 40] (signed) / [0.1, 100] (unsigned, rectified)."""
    rng = np.random.default_rng(15)
    sigmas = [0.1, 0.3, 1.0, 3.0, 10.0, 30.0, 40.0] if signed else [0.1, 0.5, 2.0, 8.0, 30.0, 100.0]
    for sigma in sigmas:
        x = rng.normal(0.0, sigma, size=10000)
        if not signed:
            x = np.maximum(x, 0.0)
        fl = synth.fl_signed(sigma) if signed else synth.fl_unsigned(sigma)
        q = _fix_quant_real(ref, x, fl, signed)
        rel = float(((q - x) ** 2).sum() / (x ** 2).sum())
        assert rel < 0.01, (sigma, fl, rel)
        # and no other format is dramatically better: Eq. 1 picks (nearly) the best candidate
        best = min(float(((_fix_quant_real(ref, x, f, signed) - x) ** 2).sum() / (x ** 2).sum())
                   for f in range(0, 8 if signed else 9))
        assert rel <= 4.0 * best + 1e-6, (sigma, fl, rel, best)
