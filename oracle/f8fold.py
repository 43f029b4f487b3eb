"""CPU oracle of the weight "compile" step: BatchNorm folding, scaling-factor absorption and fixed-point
quantisation of the effective weight and bias of one Conv-BN block (Eq. 6, Eq. 1, signed form of Eq. 2).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``.  The CUDA library never imports this module and this module never
imports the CUDA binding.  Everything is float64 (the paper does not fix a precision), written term by term in the
order of the equations, with numpy as the only library.

For output channel i and input index j of block l (Sec. 4.3 and the appendix "Derivation of Effective Weight"):

    W_eff[i, j] = (gamma_i / sigma_i) * (eta_in / eta_out) * W[i, j]                 effective weight, Eq. 6
    b_eff[i]    = (beta_i - (gamma_i / sigma_i) * mu_i) / eta_out                     effective bias, Eq. 6
    FL_w        = floor(log2(40 / std(W_eff)))  clamped to [fl_min, fl_max]           Eq. 1, signed branch
    w_q[i, j]   = round(clip(W_eff[i, j] * 2^FL_w, -127, 127))                        signed fix_quant (appendix), WL = 8
    b_q[i]      = round(b_eff[i] * 2^(FL_x + FL_w))                                    int32, accumulator format

eta_in = eta_fix of this block's input quantiser, eta_out = eta_fix of the next block's (Eq. 5:
eta_fix = 2^FL * alpha / (2^WL - 1)); the caller evaluates Eq. 5 and passes the two numbers.  `round` is round half
up, floor(v + 1/2), as everywhere in this repository; std is the population standard deviation over the whole tensor.
"""
from __future__ import annotations

import math

import numpy as np


def eta_fix(fl: int, alpha: float, wl: int = 8) -> float:
    """Eq. 5: the scaling factor left over when PACT with clipping level alpha is written as fix_quant (Eq. 4)."""
    return (2.0 ** fl) * alpha / (2.0 ** wl - 1.0)


def optimal_fl_signed(std: float) -> int:
    """Eq. 1, signed branch, as printed."""
    return int(math.floor(math.log2(40.0 / std)))


def optimal_fl_unsigned(std: float) -> int:
    """Eq. 1, unsigned branch, as printed."""
    return int(math.floor(math.log2(70.0 / std)))


def effective_weight(w, gamma, sigma, eta_in: float, eta_out: float) -> np.ndarray:
    """Effective weight of Eq. 6; w is [c_out, k], gamma / sigma are [c_out]."""
    w = np.asarray(w, dtype=np.float64)
    scale = (np.asarray(gamma, np.float64) / np.asarray(sigma, np.float64)) * (np.float64(eta_in) / np.float64(eta_out))
    return scale[:, None] * w


def effective_bias(gamma, sigma, beta, mu, eta_out: float) -> np.ndarray:
    """Effective bias of Eq. 6."""
    g, s = np.asarray(gamma, np.float64), np.asarray(sigma, np.float64)
    return (np.asarray(beta, np.float64) - (g / s) * np.asarray(mu, np.float64)) / np.float64(eta_out)


def fix_quant_signed_codes(v: np.ndarray, fl: int, wl: int = 8) -> np.ndarray:
    """Integer codes of the signed quantiser (appendix "Double Side Quantization"): clip to +-(2^(WL-1) - 1), round."""
    lim = 2.0 ** (wl - 1) - 1.0
    return np.floor(np.clip(np.asarray(v, np.float64) * (2.0 ** fl), -lim, lim) + 0.5)


def fold_quantize(w, gamma, sigma, beta, mu, eta_in: float, eta_out: float, fl_x: int, fl_min: int = 0, fl_max: int = 7):
    """Returns (w_q int8 [c_out, k], b_q int32 [c_out], FL_w, std of the effective weight)."""
    w_eff = effective_weight(w, gamma, sigma, eta_in, eta_out)
    b_eff = effective_bias(gamma, sigma, beta, mu, eta_out)
    std = float(np.std(w_eff))
    fl_w = min(fl_max, max(fl_min, optimal_fl_signed(std)))
    w_q = fix_quant_signed_codes(w_eff, fl_w).astype(np.int8)
    b = np.floor(b_eff * (2.0 ** (fl_x + fl_w)) + 0.5)
    b_q = np.clip(b, -(2.0 ** 31), 2.0 ** 31 - 1).astype(np.int32)
    return w_q, b_q, fl_w, std
