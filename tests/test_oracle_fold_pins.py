"""Pins of the weight-compile oracle (oracle/f8fold.py) against what the paper and the mathematics fix: printed
values of Eq. 1, the derivation behind Eq. 6 evaluated in floating point with a real BatchNorm, hand-worked codes of
the signed quantiser, Eq. 4, and the paper's claim about the error at the optimal fractional length."""
import math

import numpy as np
import pytest

from oracle import f8fold


def test_eq1_printed_thresholds():
    # Eq. 1: FL* = floor(log2(40 / sigma)) signed, floor(log2(70 / sigma)) unsigned.
    # Sec. 3.3 states the usable range: signed sigma from 0.1 up to about 40, unsigned up to about 100 --
    # i.e. FL* runs from 8 (sigma 0.1: log2 400 = 8.64) down to 0 (sigma 40: log2 1 = 0).
    assert f8fold.optimal_fl_signed(0.1) == 8
    assert f8fold.optimal_fl_signed(40.0) == 0
    assert f8fold.optimal_fl_signed(1.0) == 5          # log2 40 = 5.32
    assert f8fold.optimal_fl_signed(0.3) == 7          # log2 133.3 = 7.06
    assert f8fold.optimal_fl_signed(0.32) == 6         # log2 125 = 6.97
    assert f8fold.optimal_fl_unsigned(0.1) == 9        # log2 700 = 9.45
    assert f8fold.optimal_fl_unsigned(70.0) == 0
    assert f8fold.optimal_fl_unsigned(1.0) == 6        # log2 70 = 6.13
    # thresholds are equidistant on the log scale (Sec. 3.3): halving sigma adds one bit
    for s in (0.07, 0.5, 3.0, 19.0):
        assert f8fold.optimal_fl_signed(s / 2) == f8fold.optimal_fl_signed(s) + 1


def test_signed_quantiser_hand_values():
    # appendix "Double Side Quantization": clip(x * 2^FL, -127, 127) then round; WL = 8
    q = f8fold.fix_quant_signed_codes
    assert q(np.array([0.5]), 7)[0] == 64
    assert q(np.array([1.0]), 7)[0] == 127                # 128 clips to 127
    assert q(np.array([-1.004]), 7)[0] == -127            # -128.5 clips to -127
    assert q(np.array([0.37]), 5)[0] == 12                # 11.84 -> 12
    assert q(np.array([0.390625]), 5)[0] == 13            # 12.5: tie rounds up
    assert q(np.array([-0.390625]), 5)[0] == -12          # -12.5: tie rounds up (towards +inf)
    assert q(np.array([-0.40]), 5)[0] == -13              # -12.8 -> -13
    assert q(np.array([3.0]), 0)[0] == 3


def test_eq6_is_the_folded_conv_bn_pact_chain():
    """The argument of fix_quant in Eq. 6 equals (1 / eta_out) * BN(conv(W, eta_in * q)) computed the long way."""
    rng = np.random.default_rng(3)
    c_out, k = 7, 45
    w = rng.normal(0, 0.2, (c_out, k))
    gamma, beta = rng.normal(1, 0.3, c_out), rng.normal(0, 0.5, c_out)
    mu, sigma = rng.normal(0, 1, c_out), rng.uniform(0.3, 2.0, c_out)
    eta_in, eta_out = f8fold.eta_fix(5, 6.1), f8fold.eta_fix(4, 11.7)
    q = rng.integers(0, 256, k) / 2.0 ** 5                 # fixed-point input activations of the block
    y = w @ (eta_in * q)                                   # convolution on the de-quantised input
    x = gamma / sigma * (y - mu) + beta                    # BatchNorm with running statistics
    long_way = x / eta_out
    short = f8fold.effective_weight(w, gamma, sigma, eta_in, eta_out) @ q + f8fold.effective_bias(gamma, sigma, beta, mu, eta_out)
    assert np.allclose(short, long_way, rtol=1e-12, atol=1e-12)
    # a dropped mean, a wrong sign or eta ratio upside down would show
    wrong = f8fold.effective_weight(w, gamma, sigma, eta_out, eta_in) @ q + f8fold.effective_bias(gamma, sigma, beta, mu, eta_out)
    assert not np.allclose(wrong, long_way, rtol=1e-3)


def test_eq4_pact_as_fix_quant():
    """Eq. 4 with M = 2^WL - 1: PACT(x) = eta * fix_quant(x / eta), unsigned 8-bit."""
    rng = np.random.default_rng(4)
    for fl in (2, 4, 7):
        alpha = float(rng.uniform(0.5, 9.0))
        x = rng.uniform(-1.0, 1.5 * alpha, 2000)
        m = 255.0
        pact = alpha / m * np.floor(m / alpha * np.clip(x, 0, alpha) + 0.5)
        eta = f8fold.eta_fix(fl, alpha)
        fixq = np.floor(np.clip(x / eta * 2.0 ** fl, 0, 255) + 0.5) / 2.0 ** fl
        assert np.allclose(pact, eta * fixq, rtol=0, atol=1e-12)


def test_fold_quantize_special_cases():
    rng = np.random.default_rng(5)
    w = rng.normal(0, 0.05, (16, 27))
    one, zero = np.ones(16), np.zeros(16)
    # identity BatchNorm and equal scaling factors: plain quantisation of W with FL from Eq. 1
    wq, bq, fl, std = f8fold.fold_quantize(w, one, one, zero, zero, 0.3, 0.3, fl_x=6, fl_max=24)
    assert fl == math.floor(math.log2(40 / np.std(w)))
    assert np.array_equal(wq, np.clip(np.floor(w * 2.0 ** fl + 0.5), -127, 127).astype(np.int8))
    assert not bq.any()
    # the bias is expressed in the accumulator format FL_x + FL_w: beta = 0.75, eta_out = 0.5 -> 1.5 * 2^(6 + fl)
    wq2, bq2, fl2, _ = f8fold.fold_quantize(w, one, one, zero + 0.75, zero, 0.3, 0.5, fl_x=6, fl_max=24)
    assert fl2 == math.floor(math.log2(40 / (np.std(w) * 0.6)))
    assert np.all(bq2 == int(1.5 * 2 ** (6 + fl2)))
    # doubling gamma halves nothing but the format: one bit less, same codes (up to the clip)
    wq3, _, fl3, _ = f8fold.fold_quantize(w, 2 * one, one, zero, zero, 0.3, 0.3, fl_x=6, fl_max=24)
    assert fl3 == fl - 1
    assert np.array_equal(wq3, wq)
    # clamp of the fractional length
    assert f8fold.fold_quantize(w, one, one, zero, zero, 0.3, 0.3, fl_x=6, fl_max=7)[2] == 7


def test_error_at_the_optimal_fractional_length_is_small():
    """Sec. 3.3: with the format of Eq. 1, zero-mean Gaussian values are quantised with a relative error below 1 % for
    standard deviations from 0.1 to about 40 (signed).  Relative error = ||q - x||^2 / ||x||^2."""
    rng = np.random.default_rng(6)
    for sigma in (0.1, 0.35, 1.0, 4.0, 17.0, 39.0):
        x = rng.normal(0, sigma, 10000)
        fl = f8fold.optimal_fl_signed(float(np.std(x)))
        q = f8fold.fix_quant_signed_codes(x, fl) / 2.0 ** fl
        assert np.sum((q - x) ** 2) / np.sum(x ** 2) < 0.01, sigma
