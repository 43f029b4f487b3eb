"""CPU oracle of the statistical study behind the format rule (Sec. 3.3, Fig. 2 / Fig. 3, appendix "More Details for
Statistical Analysis"): relative quantisation error of a sample under every 8-bit fixed-point format, and the format
with the smallest error.

TEST INFRASTRUCTURE ONLY: imported by ``tests/``.  float64 numpy, term by term.

    unsigned (after ReLU):  q_FL(x) = round(clip(max(x, 0) * 2^FL, 0, 255)) / 2^FL          FL = 0 .. 8      (Eq. 2)
    signed:                 q_FL(x) = round(clip(x * 2^FL, -127, 127)) / 2^FL               FL = 0 .. 7      (appendix)
    err[FL] = sum (q_FL(x) - x')^2 / sum x'^2            x' = x, or max(x, 0) for the unsigned study
    FL*     = argmin_FL err[FL]      (smallest FL on a tie)

The paper does not define its "relative error"; the squared-norm ratio is the reading under which its statement
"below 1 % from sigma = 0.1 to about 40 (signed) / 100 (unsigned)" holds.  round = floor(v + 1/2).
"""
from __future__ import annotations

import numpy as np


def relative_errors(x, unsigned: bool) -> np.ndarray:
    x = np.asarray(x, dtype=np.float64)
    ref = np.maximum(x, 0.0) if unsigned else x
    lo, hi, n_fl = (0.0, 255.0, 9) if unsigned else (-127.0, 127.0, 8)
    den = np.sum(ref * ref)
    err = np.empty(n_fl)
    for fl in range(n_fl):
        q = np.floor(np.clip(ref * 2.0 ** fl, lo, hi) + 0.5) / 2.0 ** fl
        err[fl] = np.sum((q - ref) ** 2) / den
    return err


def best_format(x, unsigned: bool):
    err = relative_errors(x, unsigned)
    return int(np.argmin(err)), err
