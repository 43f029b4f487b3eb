"""GPU parity of the statistical-study kernel (f8_format_study_fixed) against the float64 oracle: the per-format
relative errors agree to summation-order rounding (1e-11 relative) and the best format is the same."""
import numpy as np
import pytest
import torch

from oracle import f8study
from gpu_util import api

pytestmark = pytest.mark.gpu

RTOL = 1e-11      # both sides sum float64 terms that are equal bit for bit; only the order of the additions differs


def _run(x, unsigned):
    a = api()
    xd = a.to_device(x)
    err = torch.full((9,), -7.0, dtype=torch.float64, device="cuda")
    best = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    ws = torch.empty(a.f8_format_study_workspace_bytes(), dtype=torch.uint8, device="cuda")
    a.f8_format_study_fixed(xd, unsigned, err, best, ws)
    torch.cuda.synchronize()
    return err.cpu().numpy(), int(best.item())


@pytest.mark.parametrize("unsigned", [False, True])
@pytest.mark.parametrize("sigma,n", [(0.1, 10000), (1.0, 10000), (7.0, 10000), (38.0, 10000), (0.02, 1), (3.0, 257),
                                     (0.6, 3_000_001)])
def test_study_matches_oracle(sigma, n, unsigned):
    rng = np.random.default_rng(int(sigma * 1000) + n + (1 if unsigned else 0))
    x = rng.normal(0.0, sigma, n).astype(np.float32)
    if n == 1:
        x[0] = abs(x[0]) + 0.01          # the unsigned study needs one positive value
    want_best, want = f8study.best_format(x, unsigned)
    got, got_best = _run(x, unsigned)
    n_fl = 9 if unsigned else 8
    assert np.allclose(got[:n_fl], want, rtol=RTOL, atol=0.0)
    if not unsigned:
        assert got[8] == -1.0
    # the best format is unique unless two errors are within rounding of each other
    order = np.sort(want)
    if order[1] - order[0] > 1e-9 * order[0]:
        assert got_best == want_best
