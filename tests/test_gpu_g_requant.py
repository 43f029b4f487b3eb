"""GPU parity (bit-exact) of f8_requantize_dual_fixed: one int32 tensor quantised for two consumers with private
fractional lengths (Sec. 4.3), against the oracle's rounding shift + clip."""
import numpy as np
import pytest
import torch

from paper_2202_05239_b200 import synth
from gpu_util import api

pytestmark = pytest.mark.gpu


def _want(ref, acc, fa, fl, dtype):
    """Every element through the oracle's own quantiser: a fully connected layer with a zero input and zero weights
    hands each int32 value, as the bias in accumulator format fa, to the oracle's rounding shift + clip."""
    n = acc.size
    y = ref.linear(np.zeros((1, 1), dtype=np.uint8), np.zeros((n, 1), dtype=np.int8), np.ascontiguousarray(acc),
                   fl_x=0, fl_w=fa, fl_y=fl, y_dtype=dtype)
    return y.reshape(n).astype(np.int64)


@pytest.mark.parametrize("n,fa,fl1,d1,fl2,d2", [
    (1 << 20, 12, 4, synth.U8, 5, synth.S8),      # two consumers: unsigned FL 4, signed FL 5
    (1000003, 11, 7, synth.S8, 0, synth.U8),       # ragged length; shifts 4 and 11
    (4099, 3, 8, synth.U8, 7, synth.S8),           # negative shifts: left shift then clip
    (17, 20, 3, synth.U8, None, None),             # one consumer only
    (1 << 22, 14, 6, synth.U8, 4, synth.U8),       # siblings sharing the clipping level, formats two bits apart
])
def test_requantize_dual(ref, n, fa, fl1, d1, fl2, d2):
    a = api()
    rng = np.random.default_rng(n % 1000 + fa)
    acc = rng.integers(-(1 << (fa + 5)), 1 << (fa + 5), size=n).astype(np.int32)
    acc[:8] = [0, 1 << (fa - 1 if fa > 0 else 0), -(1 << 30), (1 << 31) - 1, -(1 << 31), 3, -3, 255 << max(fa - 4, 0)]
    accd = a.to_device(acc)
    y1 = torch.empty(n, dtype=a.torch_dtype(d1), device="cuda")
    y2 = torch.empty(n, dtype=a.torch_dtype(d2), device="cuda") if d2 is not None else None
    a.f8_requantize_dual_fixed(accd, fa, y1, d1, fl1, y2, d2 if d2 is not None else 0, fl2 if fl2 is not None else 0)
    torch.cuda.synchronize()
    assert np.array_equal(y1.cpu().numpy().astype(np.int64), _want(ref, acc, fa, fl1, d1))
    if y2 is not None:
        assert np.array_equal(y2.cpu().numpy().astype(np.int64), _want(ref, acc, fa, fl2, d2))


def test_private_formats_versus_realigning_one_tensor(ref):
    """Quantising the 32-bit value for each consumer (the paper) against storing one 8-bit tensor and re-aligning it at
    the coarser consumer (the single-tensor reading the network executor uses): the latter rounds twice, so the two may
    differ, but by one code at most."""
    a = api()
    rng = np.random.default_rng(5)
    fa, fine, coarse = 13, 6, 4
    acc = rng.integers(0, 255 << (fa - coarse), size=1 << 16).astype(np.int32)
    y_f = torch.empty(acc.size, dtype=torch.uint8, device="cuda")
    y_c = torch.empty(acc.size, dtype=torch.uint8, device="cuda")
    a.f8_requantize_dual_fixed(a.to_device(acc), fa, y_f, synth.U8, fine, y_c, synth.U8, coarse)
    torch.cuda.synchronize()
    direct = y_c.cpu().numpy().astype(np.int64)
    twice = np.clip((y_f.cpu().numpy().astype(np.int64) + 2) >> 2, 0, 255)      # fine tensor re-aligned by fine - coarse = 2 bits
    unclipped = y_f.cpu().numpy() < 255
    assert np.max(np.abs(direct - twice)[unclipped]) <= 1
    assert np.any(direct != twice)          # the double rounding is visible: the readings are not identical
