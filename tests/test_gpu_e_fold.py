"""GPU parity of the weight compile step (f8_fold_quantize_fixed: Eq. 6 effective weight / bias, Eq. 1 format, signed
quantiser) against the float64 oracle: integer codes and bias bit for bit, the chosen fractional length equal."""
import math

import numpy as np
import pytest
import torch

from oracle import f8fold
from gpu_util import api

pytestmark = pytest.mark.gpu

# (c_out, k, weight sigma, fl_x, fl_max)
FOLD_CASES = [
    (64, 147, 0.12, 6, 24),        # a 7x7x3 stem
    (256, 576, 0.06, 5, 24),       # 3x3x64
    (2048, 512, 0.03, 4, 24),      # 1x1, a million weights: several chunks per block, all blocks busy
    (1000, 2048, 0.02, 3, 24),     # fully connected
    (17, 5, 0.5, 0, 24),           # tiny and ragged
    (96, 4608, 0.8, 8, 7),         # rows longer than a chunk; paper's FL range 0..7
    (32, 27, 30.0, 2, 7),          # large weights: FL clamps at 0 and codes saturate
]


def _run(w, gamma, sigma, beta, mu, eta_in, eta_out, fl_x, fl_min, fl_max):
    a = api()
    c_out, k = w.shape
    d = a.FoldDesc(c_out, k, fl_x, fl_min, fl_max, eta_in, eta_out)
    dev = [a.to_device(t.astype(np.float32)) for t in (w, gamma, sigma, beta, mu)]
    w_q = torch.empty((c_out, k), dtype=torch.int8, device="cuda")
    b_q = torch.empty(c_out, dtype=torch.int32, device="cuda")
    fl = torch.full((1,), -99, dtype=torch.int32, device="cuda")
    ws = torch.empty(a.f8_fold_workspace_bytes(d), dtype=torch.uint8, device="cuda")
    a.f8_fold_quantize_fixed(d, *dev, w_q, b_q, fl, ws)
    torch.cuda.synchronize()
    return w_q.cpu().numpy(), b_q.cpu().numpy(), int(fl.item())


@pytest.mark.parametrize("case", range(len(FOLD_CASES)))
def test_fold_quantize(case):
    c_out, k, wsig, fl_x, fl_max = FOLD_CASES[case]
    rng = np.random.default_rng(1200 + case)
    # fp32 inputs (what a trained model holds); the oracle reads the same fp32 values as float64
    w = rng.normal(0, wsig, (c_out, k)).astype(np.float32)
    gamma = rng.normal(1.0, 0.3, c_out).astype(np.float32)
    sigma = rng.uniform(0.2, 3.0, c_out).astype(np.float32)
    beta = rng.normal(0, 0.4, c_out).astype(np.float32)
    mu = rng.normal(0, 1.0, c_out).astype(np.float32)
    eta_in = f8fold.eta_fix(fl_x, float(rng.uniform(2.0, 8.0)))
    eta_out = f8fold.eta_fix(int(rng.integers(2, 7)), float(rng.uniform(2.0, 8.0)))
    want_w, want_b, want_fl, std = f8fold.fold_quantize(w, gamma, sigma, beta, mu, eta_in, eta_out, fl_x, 0, fl_max)
    got_w, got_b, got_fl = _run(w, gamma, sigma, beta, mu, eta_in, eta_out, fl_x, 0, fl_max)
    # the one place where the summation order can show: 40 / std within rounding of a power of two
    frac = math.log2(40.0 / std) % 1.0
    assert min(frac, 1.0 - frac) > 1e-9, "case sits on a format boundary: pick another seed"
    assert got_fl == want_fl
    assert int((got_w != want_w).sum()) == 0
    assert int((got_b != want_b).sum()) == 0


def test_fold_constant_and_identity_cases():
    # identity BatchNorm, equal scaling factors: the plain signed quantiser with the format of Eq. 1
    rng = np.random.default_rng(99)
    w = rng.normal(0, 0.07, (48, 144)).astype(np.float32)
    one, zero = np.ones(48, np.float32), np.zeros(48, np.float32)
    got_w, got_b, got_fl = _run(w, one, one, zero, zero, 0.25, 0.25, 5, 0, 24)
    fl = math.floor(math.log2(40.0 / float(np.std(w.astype(np.float64)))))
    assert got_fl == fl
    assert np.array_equal(got_w, np.clip(np.floor(w.astype(np.float64) * 2.0 ** fl + 0.5), -127, 127).astype(np.int8))
    assert not got_b.any()
    # all weights equal: zero standard deviation, the finest allowed format is taken and nothing divides by zero
    c = np.full((8, 16), 0.25, np.float32)
    got_w, _, got_fl = _run(c, np.ones(8, np.float32), np.ones(8, np.float32), np.zeros(8, np.float32),
                            np.zeros(8, np.float32), 1.0, 1.0, 4, 0, 7)
    assert got_fl == 7 and np.all(got_w == 32)


def test_compiled_block_runs_through_the_fixed_point_conv(ref):
    """Float Conv-BN-ReLU with PACT input / output quantisation against the compiled fixed-point layer: the 8-bit
    outputs agree with the float chain within one code almost everywhere (weights are quantised, activations are not
    re-rounded: the chain is Eq. 6 evaluated with W_eff in place of its 8-bit codes)."""
    from paper_2202_05239_b200 import synth
    a = api()
    rng = np.random.default_rng(7)
    n, h, c, c_out, kk = 2, 20, 32, 48, 3
    fl_x, alpha_x, fl_y, alpha_y = 5, 6.0, 4, 12.0
    eta_in, eta_out = f8fold.eta_fix(fl_x, alpha_x), f8fold.eta_fix(fl_y, alpha_y)
    w = rng.normal(0, math.sqrt(2.0 / (kk * kk * c)), (c_out, kk, kk, c)).astype(np.float32)
    gamma = rng.uniform(0.6, 1.4, c_out).astype(np.float32)
    sigma = rng.uniform(0.8, 1.6, c_out).astype(np.float32)
    beta = rng.normal(0, 0.3, c_out).astype(np.float32)
    mu = rng.normal(0, 0.3, c_out).astype(np.float32)
    got_w, got_b, got_fl = _run(w.reshape(c_out, -1), gamma, sigma, beta, mu, eta_in, eta_out, fl_x, 0, 24)
    x = rng.integers(0, 256, (n, h, h, c)).astype(np.uint8)
    layer = synth.Layer(synth.CONV, "compiled", 0, -1, h, h, c, c_out, kk, kk, 1, 1, synth.U8, synth.U8, synth.U8,
                        fl_x, got_fl, fl_y, 0, got_w.reshape(c_out, kk, kk, c), got_b)
    y = a.run_layer(layer, a.to_device(x)).cpu().numpy().astype(np.float64)
    assert np.array_equal(y, ref.run_layer(layer, x).astype(np.float64))
    # the float chain: de-quantised input -> conv -> BatchNorm -> PACT(alpha_y) expressed in output codes (Eq. 4)
    xt = torch.from_numpy(x.astype(np.float64) / 2.0 ** fl_x * eta_in).permute(0, 3, 1, 2)

    def chain(weights, gam, sig, bet, mean):
        wt = torch.from_numpy(weights).permute(0, 3, 1, 2)
        conv = torch.nn.functional.conv2d(xt, wt, padding=1).permute(0, 2, 3, 1).numpy()
        bn = gam / sig * (conv - mean) + bet
        return np.floor(np.clip(bn / eta_out * 2.0 ** fl_y, 0, 255) + 0.5)

    # with the compiled parameters put back into float form (W = eta_out / eta_in * w_q 2^-FL_w, identity BatchNorm,
    # beta = eta_out * b_q 2^-(FL_x + FL_w)) the float chain IS the fixed-point layer: every code agrees, except
    # where float rounding of the scaled sum meets an exact tie of the quantiser
    w_back = got_w.reshape(c_out, kk, kk, c).astype(np.float64) / 2.0 ** got_fl * (eta_out / eta_in)
    b_back = got_b.astype(np.float64) / 2.0 ** (fl_x + got_fl) * eta_out
    same = chain(w_back, 1.0, 1.0, b_back, 0.0)
    assert np.mean(same == y) > 0.999 and np.max(np.abs(same - y)) <= 1
    # with the original float parameters the difference is the weights' quantisation error only
    codes = chain(w.astype(np.float64), gamma.astype(np.float64), sigma.astype(np.float64), beta.astype(np.float64),
                  mu.astype(np.float64))
    err = np.linalg.norm(codes - y) / np.linalg.norm(codes)
    assert err < 0.05, err
    assert np.mean(np.abs(codes - y) <= 2) > 0.9
