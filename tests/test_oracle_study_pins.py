"""Pins of the statistical-study oracle (oracle/f8study.py) against the paper: Sec. 3.3's error claim, the
almost-linear relation between log sigma and the best format that Eq. 1 summarises, and closed-form cases."""
import math

import numpy as np

from oracle import f8study


def _sample(sigma, seed, n=10000):          # the paper's experiment: 10 000 zero-mean Gaussian values per sigma
    return np.random.default_rng(seed).normal(0.0, sigma, n)


def test_error_at_best_format_below_one_percent():
    # Sec. 3.3: < 1 % for sigma from 0.1 to about 40 (signed) and 0.1 to 100 (unsigned, after ReLU)
    for i, sigma in enumerate((0.1, 0.3, 1.0, 3.0, 10.0, 30.0, 39.0)):
        assert f8study.best_format(_sample(sigma, i), False)[1].min() < 0.01
    for i, sigma in enumerate((0.1, 0.5, 2.0, 9.0, 40.0, 99.0)):
        assert f8study.best_format(_sample(sigma, 50 + i), True)[1].min() < 0.01
    # far outside the range no format is good
    assert f8study.best_format(_sample(400.0, 7), False)[1].min() > 0.01
    assert f8study.best_format(_sample(0.002, 8), False)[1].min() > 0.01


def test_best_format_follows_eq1():
    """Eq. 1 is a fit to the jumping points of the best format: away from those points the experiment and the
    formula agree, and near them they differ by at most one."""
    agree = total = 0
    for i, lg in enumerate(np.linspace(math.log2(0.35), math.log2(38.0), 40)):
        sigma = 2.0 ** lg
        x = _sample(sigma, 100 + i)
        best, _ = f8study.best_format(x, False)
        want = min(7, max(0, math.floor(math.log2(40.0 / float(np.std(x))))))
        assert abs(best - want) <= 1, (sigma, best, want)
        agree += best == want
        total += 1
    assert agree >= 0.7 * total
    agree = total = 0
    for i, lg in enumerate(np.linspace(math.log2(0.3), math.log2(60.0), 40)):
        sigma = 2.0 ** lg
        x = _sample(sigma, 200 + i)
        best, _ = f8study.best_format(x, True)
        want = min(8, max(0, math.floor(math.log2(70.0 / sigma))))
        assert abs(best - want) <= 1, (sigma, best, want)
        agree += best == want
        total += 1
    assert agree >= 0.7 * total


def test_halving_sigma_shifts_the_whole_curve_by_one_format():
    # q_FL(x / 2) = q_{FL-1}(x) / 2 exactly: the error curves of Fig. 2 are translates of each other on the log axis
    x = _sample(3.0, 9)
    e1 = f8study.relative_errors(x, False)
    e2 = f8study.relative_errors(x / 2.0, False)
    assert np.allclose(e2[1:], e1[:-1], rtol=1e-12)
    u1 = f8study.relative_errors(x, True)
    u2 = f8study.relative_errors(x / 2.0, True)
    assert np.allclose(u2[1:], u1[:-1], rtol=1e-12)


def test_closed_form_cases():
    # values on the grid of a format are exact in that format and in every finer one that does not clip
    x = np.array([0.5, -1.25, 3.0, -0.75, 2.25])
    err = f8study.relative_errors(x, False)
    assert err[2] == 0.0 and err[3] == 0.0 and err[5] == 0.0
    assert err[7] > 0.0                                   # 3.0 * 128 clips at 127
    # one value, by hand: x = 0.3, FL = 2 -> round(1.2) / 4 = 0.25, error (0.05 / 0.3)^2
    assert math.isclose(f8study.relative_errors(np.array([0.3]), False)[2], (0.05 / 0.3) ** 2, rel_tol=1e-12)
    # unsigned study: negative samples are rectified first and then contribute nothing
    eu = f8study.relative_errors(np.array([-5.0, 0.3]), True)
    assert math.isclose(eu[2], (0.05 / 0.3) ** 2, rel_tol=1e-12)
    # a tie at 0.5 rounds up: x = 0.125, FL = 2 -> 0.5 -> 1 -> 0.25
    assert math.isclose(f8study.relative_errors(np.array([0.125]), True)[2], 1.0, rel_tol=1e-12)
