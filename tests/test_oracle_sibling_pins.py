"""Pins of the oracle's sibling handling (``conv2d_siblings``): one 32-bit sum quantised once per child layer with
the child's private fractional length, and a shortcut that may stay in 32 bits (Sec. 4.3 "Clipping-Level Sharing and
Private Fractional Length", Fig. 4, appendix on private fractional lengths).  None of these checks calls the function
under test to produce its own expectation: they use hand-worked numbers, exact rational arithmetic, and the
single-output oracle functions that are pinned elsewhere."""
from fractions import Fraction

import numpy as np
import pytest

from paper_2202_05239_b200.synth import U8, S8, S32


def _round_half_up(fr: Fraction) -> int:
    return (fr + Fraction(1, 2)).__floor__()


def _pixel(ref, x, w, bias, r, fl_r, kinds, fls, fl_x=4, fl_w=7):
    """A 1x1 convolution on one pixel: returns the outputs for the given child kinds."""
    xa = np.array(x, dtype=np.uint8).reshape(1, 1, 1, -1)
    wa = np.array(w, dtype=np.int8).reshape(1, 1, 1, -1)
    ba = np.array([bias], dtype=np.int32)
    ra = None if r is None else np.array([r], dtype=np.int32 if abs(r) > 255 or isinstance(r, np.int32) else np.uint8).reshape(1, 1, 1, 1)
    out = []
    for kind, fl in zip(kinds, fls):
        y1, _ = ref.conv2d_siblings(xa, wa, ba, stride=1, pad=0, fl_x=fl_x, fl_w=fl_w, y1_kind=kind, fl_y1=fl,
                                    residual=ra, fl_r=fl_r)
        out.append(int(y1.reshape(-1)[0]))
    return out


def test_hand_worked_sum_with_a_32_bit_shortcut(ref):
    # 200*77 - 17*128 + 255*3 = 13989; bias 1411 -> acc = 15400 in format 11 (real 7.51953125)
    x, w, bias = [200, 17, 255], [77, -128, 3], 1411
    assert 200 * 77 - 17 * 128 + 255 * 3 + bias == 15400
    # shortcut 597 in format 9 (real 1.166015625): F = 11, v = 15400 + 597 * 4 = 17788 (real 8.685546875)
    r32 = np.int32(597)
    got = _pixel(ref, x, w, bias, r32, 9, [U8, S8, S32, ref.S32_RELU], [4, 3, 0, 0])
    # FL 4: (17788 + 64) >> 7 = 139 (real * 16 = 138.97);  FL 3: (17788 + 128) >> 8 = 69 (real * 8 = 69.48)
    assert got == [139, 69, 17788, 17788]
    # shortcut finer than the accumulator: 9551 in format 13 -> F = 13, v = 15400 * 4 + 9551 = 71151
    r32 = np.int32(9551)
    got = _pixel(ref, x, w, bias, r32, 13, [U8, S32], [4, 0])
    assert got == [(71151 + 256) >> 9, 71151] and got[0] == 139
    # a negative sum: shortcut -80000 in format 13 -> v = 61600 - 80000 = -18400 (real -2.24609375)
    r32 = np.int32(-80000)
    got = _pixel(ref, x, w, bias, r32, 13, [U8, S8, S32, ref.S32_RELU], [4, 4, 0, 0])
    # signed FL 4: real * 16 = -35.94 -> -36; unsigned clips to 0; the ReLU'd 32-bit value is 0
    assert got == [0, -36, -18400, 0]


def test_the_8_bit_shortcut_case_of_the_single_output_oracle_is_reproduced(ref):
    """acc 15400 (format 11) + 8-bit shortcut 37 in format 5 -> 17768 -> FL 4: 139 (worked for the single-output
    function); the sibling function must agree and its 32-bit child must be the aligned sum itself."""
    got = _pixel(ref, [200, 17, 255], [77, -128, 3], 1411, 37, 5, [U8, S32], [4, 0])
    assert got == [139, 15400 + (37 << 6)]


@pytest.mark.parametrize("seed", range(6))
def test_two_children_equal_two_single_output_calls(ref, seed):
    rng = np.random.default_rng(seed)
    n, h, w, ci, co, k = 2, 7, 6, 5, 9, 3
    stride, pad = (1, 1) if seed % 2 == 0 else (2, 0)
    x = rng.integers(0, 256, size=(n, h, w, ci)).astype(np.uint8) if seed % 3 else rng.integers(-128, 128, size=(n, h, w, ci)).astype(np.int8)
    wgt = rng.integers(-128, 128, size=(co, k, k, ci)).astype(np.int8)
    bias = rng.integers(-3000, 3000, size=co).astype(np.int32)
    fl_x, fl_w = int(rng.integers(0, 8)), int(rng.integers(2, 10))
    ho, wo = (h + 2 * pad - k) // stride + 1, (w + 2 * pad - k) // stride + 1
    res = rng.integers(0, 256, size=(n, ho, wo, co)).astype(np.uint8) if seed % 2 else None
    fl_r = int(rng.integers(0, 9))
    fl1, fl2 = int(rng.integers(0, 9)), int(rng.integers(0, 8))
    y1, y2 = ref.conv2d_siblings(x, wgt, bias, stride=stride, pad=pad, fl_x=fl_x, fl_w=fl_w, y1_kind=U8, fl_y1=fl1,
                                 y2_kind=S8, fl_y2=fl2, residual=res, fl_r=fl_r)
    kw = dict(stride=stride, pad=pad, fl_x=fl_x, fl_w=fl_w, residual=res, fl_r=fl_r)
    assert np.array_equal(y1, ref.conv2d(x, wgt, bias, fl_y=fl1, y_dtype=U8, **kw))
    assert np.array_equal(y2, ref.conv2d(x, wgt, bias, fl_y=fl2, y_dtype=S8, **kw))
    # the 32-bit child is the raw accumulator of the single-output function
    y32, y32r = ref.conv2d_siblings(x, wgt, bias, stride=stride, pad=pad, fl_x=fl_x, fl_w=fl_w, y1_kind=S32, fl_y1=0,
                                    y2_kind=ref.S32_RELU, fl_y2=0, residual=res, fl_r=fl_r)
    assert np.array_equal(y32, ref.conv2d(x, wgt, bias, fl_y=0, y_dtype=S32, **kw))
    assert np.array_equal(y32r, np.maximum(y32, 0))
    # every 8-bit child is the rounding shift + clip of that 32-bit value (scalar function, pinned by the golden table)
    f = max(fl_x + fl_w, fl_r) if res is not None else fl_x + fl_w
    flat32 = y32.reshape(-1)
    for i in rng.integers(0, flat32.size, size=200):
        assert ref.shift_round_clip(int(flat32[i]), f - fl1, 0, 255) == int(y1.reshape(-1)[i])
        assert ref.shift_round_clip(int(flat32[i]), f - fl2, -127, 127) == int(y2.reshape(-1)[i])


@pytest.mark.parametrize("seed", range(4))
def test_32_bit_shortcut_against_exact_rational_arithmetic(ref, seed):
    """Brute force on a tiny layer: the real-valued definition in Fractions, shortcut given as a 32-bit value."""
    rng = np.random.default_rng(100 + seed)
    n, h, w, ci, co, k, stride, pad = 1, 4, 5, 3, 4, 3, 1, 1
    x = rng.integers(-128, 128, size=(n, h, w, ci)).astype(np.int8)
    wgt = rng.integers(-128, 128, size=(co, k, k, ci)).astype(np.int8)
    bias = rng.integers(-2000, 2000, size=co).astype(np.int32)
    fl_x, fl_w, fl_r = int(rng.integers(0, 8)), int(rng.integers(2, 9)), int(rng.integers(4, 16))
    res = rng.integers(-(1 << 17), 1 << 17, size=(n, h, w, co)).astype(np.int32)
    fl1, fl2 = int(rng.integers(0, 9)), int(rng.integers(0, 8))
    y1, y2 = ref.conv2d_siblings(x, wgt, bias, stride=stride, pad=pad, fl_x=fl_x, fl_w=fl_w, y1_kind=U8, fl_y1=fl1,
                                 y2_kind=S8, fl_y2=fl2, residual=res, fl_r=fl_r)
    y3, _ = ref.conv2d_siblings(x, wgt, bias, stride=stride, pad=pad, fl_x=fl_x, fl_w=fl_w, y1_kind=ref.S32_RELU, fl_y1=0,
                                residual=res, fl_r=fl_r)
    f = max(fl_x + fl_w, fl_r)
    for oh in range(h):
        for ow in range(w):
            for oc in range(co):
                v = Fraction(int(bias[oc]), 1 << (fl_x + fl_w)) + Fraction(int(res[0, oh, ow, oc]), 1 << fl_r)
                for r in range(k):
                    for s in range(k):
                        ih, iw = oh + r - pad, ow + s - pad
                        if 0 <= ih < h and 0 <= iw < w:
                            for c in range(ci):
                                v += Fraction(int(x[0, ih, iw, c]), 1 << fl_x) * Fraction(int(wgt[oc, r, s, c]), 1 << fl_w)
                assert int(y1[0, oh, ow, oc]) == min(255, max(0, _round_half_up(v * (1 << fl1))))
                assert int(y2[0, oh, ow, oc]) == min(127, max(-127, _round_half_up(v * (1 << fl2))))
                assert int(y3[0, oh, ow, oc]) == max(0, int(v * (1 << f)))       # exact integer in format F


def test_a_sum_outside_int32_is_reported(ref):
    x = np.full((1, 1, 1, 1), 255, dtype=np.uint8)
    wgt = np.full((1, 1, 1, 1), 127, dtype=np.int8)
    res = np.full((1, 1, 1, 1), (1 << 30), dtype=np.int32)
    with pytest.raises(RuntimeError):      # shortcut in format 0 against an accumulator in format 4: 2^30 * 16 overflows
        ref.conv2d_siblings(x, wgt, None, stride=1, pad=0, fl_x=2, fl_w=2, y1_kind=U8, fl_y1=0, residual=res, fl_r=0)


def test_private_formats_only_rescale(ref):
    """Appendix on private fractional lengths: two children that share the clipping level but use formats d bits apart
    read the same real value, the coarser one within half of its own step (plus the finer one's rounding)."""
    rng = np.random.default_rng(9)
    x = rng.integers(0, 256, size=(1, 6, 6, 8)).astype(np.uint8)
    wgt = rng.integers(-20, 20, size=(8, 1, 1, 8)).astype(np.int8)
    y_f, y_c = ref.conv2d_siblings(x, wgt, None, stride=1, pad=0, fl_x=5, fl_w=6, y1_kind=U8, fl_y1=5, y2_kind=U8, fl_y2=3)
    unclipped = (y_f < 255) & (y_c < 255)
    real_f, real_c = y_f.astype(np.float64) / 32.0, y_c.astype(np.float64) / 8.0
    assert np.max(np.abs(real_f - real_c)[unclipped]) <= 1 / 16.0 + 1 / 64.0 + 1e-12
