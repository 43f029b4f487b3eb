"""GPU parity (bit-exact) of the tensor-core implicit-GEMM path (tcgen05.mma kind::i8 + TMA im2col)."""
import numpy as np
import pytest
import torch

from paper_2202_05239_b200 import synth
from gpu_util import api, check_layer, random_conv_layer, random_input, random_residual

pytestmark = pytest.mark.gpu


def test_tensor_core_probe_runs():
    a = api()
    ops = a.f8_mma_i8_probe(64)
    torch.cuda.synchronize()
    a.f8_device_status()
    assert ops == 2.0 * 128 * 256 * 32 * 64 * torch.cuda.get_device_properties(0).multi_processor_count


# (h, w, c, c_out, k, stride, pad, n, x_signed, y_dtype, res)
TC_CASES = [
    (56, 56, 64, 64, 1, 1, 0, 1, False, synth.U8, False),      # plain GEMM, one K chunk (64-byte swizzle)
    (28, 28, 128, 128, 1, 1, 0, 2, False, synth.U8, True),     # 128-byte swizzle + residual
    (28, 28, 256, 64, 1, 1, 0, 1, True, synth.S8, False),      # two K chunks, signed in / out
    (14, 14, 1024, 256, 1, 1, 0, 3, False, synth.U8, False),   # 8 K chunks, ragged M (588 pixels)
    (56, 56, 64, 64, 3, 1, 1, 1, False, synth.U8, False),      # 3x3 halo through im2col
    (28, 28, 128, 128, 3, 2, 1, 2, False, synth.U8, True),     # 3x3 stride 2
    (56, 56, 256, 512, 1, 2, 0, 1, False, synth.S8, False),    # 1x1 stride 2 (downsample), two N tiles
    (15, 17, 32, 48, 3, 1, 1, 17, True, synth.U8, False),       # odd sizes, 32-byte swizzle, N tile 48
    (9, 9, 144, 24, 1, 1, 0, 13, False, synth.S8, True),       # c = 144 (ragged K chunk), c_out = 24
    (12, 12, 96, 576, 1, 1, 0, 10, True, synth.U8, False),     # three N tiles with a ragged last one
    (7, 7, 512, 512, 3, 1, 1, 6, False, synth.U8, False),      # 36 K iterations, tiles span several images
    (8, 8, 2048, 1000, 1, 1, 0, 2, False, synth.S32, False),   # int32 output, ragged N
    (33, 20, 16, 96, 1, 1, 0, 13, True, synth.U8, False),      # c = 16: half-empty 32-byte K chunk
    (20, 20, 64, 32, 5, 1, 2, 6, False, synth.U8, False),      # 5x5
    (31, 31, 64, 64, 3, 2, 0, 3, False, synth.U8, False),      # stride 2 without padding
    (28, 28, 128, 128, 3, 1, 1, 2, False, synth.U8, False),    # windowed 3x3: four whole rows per tile
    (28, 28, 128, 128, 3, 1, 1, 3, True, synth.S8, True),      # windowed 3x3 with residual, signed in / out
    (30, 22, 128, 64, 3, 1, 1, 5, False, synth.U8, False),     # windowed 3x3: five rows of 24 positions, six bands
    (14, 14, 128, 128, 3, 1, 1, 9, False, synth.U8, True),     # windowed 3x3: second band of an image is partial
    (12, 40, 256, 32, 3, 1, 1, 3, True, synth.U8, False),      # windowed 3x3 with two channel chunks
]


@pytest.mark.parametrize("case", range(len(TC_CASES)))
def test_tensor_core_conv(ref, case):
    h, w, c, c_out, k, stride, pad, n, xs, y_dtype, with_res = TC_CASES[case]
    rng = np.random.default_rng(300 + case)
    layer = random_conv_layer(rng, h=h, w=w, c=c, c_out=c_out, k=k, stride=stride, pad=pad, x_signed=xs, y_dtype=y_dtype,
                              with_res=with_res)
    x = random_input(rng, n, layer)
    assert x.size >= 128 * 1024, "case must be large enough for the tensor-core path"
    res = random_residual(rng, n, layer) if with_res else None
    check_layer(ref, layer, x, res, expect_tc=True)


# pointwise layers on tensors below 128 KiB: activations are read as a plain matrix (no im2col map)
# (h, w, c, c_out, n, x_signed, y_dtype, res)
SMALL_POINTWISE = [
    (1, 1, 1280, 1000, 64, False, synth.S32, False),    # a fully connected layer at batch 64 (80 KB)
    (7, 7, 160, 960, 1, True, synth.U8, False),          # batch-1 inference: 7.8 KB, one ragged M tile
    (7, 7, 960, 160, 2, False, synth.S8, True),          # 94 KB, residual, eight K chunks
    (3, 5, 320, 48, 9, False, synth.U8, False),          # 135 pixels: two M tiles, the second nearly empty
]


@pytest.mark.parametrize("case", range(len(SMALL_POINTWISE)))
def test_small_pointwise_on_tensor_cores(ref, case):
    h, w, c, c_out, n, xs, y_dtype, with_res = SMALL_POINTWISE[case]
    rng = np.random.default_rng(700 + case)
    layer = random_conv_layer(rng, h=h, w=w, c=c, c_out=c_out, k=1, stride=1, pad=0, x_signed=xs, y_dtype=y_dtype,
                              with_res=with_res)
    x = random_input(rng, n, layer)
    assert 4096 <= x.size < 128 * 1024
    res = random_residual(rng, n, layer) if with_res else None
    check_layer(ref, layer, x, res, expect_tc=True)


# layers that are not pointwise on tensors below 128 KiB (single-image inference): whole output rows per tile, one tiled
# load per filter tap (no im2col map)
# (h, w, c, c_out, k, stride, pad, n, x_signed, y_dtype, res)
SMALL_ROW_TILED = [
    (28, 28, 128, 128, 3, 1, 1, 1, False, synth.U8, False),     # 98 KB: four rows per tile, seven bands
    (14, 14, 256, 256, 3, 1, 1, 1, False, synth.U8, True),      # nine rows per tile, second band partial; residual
    (7, 7, 512, 512, 3, 1, 1, 2, True, synth.S8, False),        # 49 of 128 tile rows used; two N tiles, streamed weights
    (14, 14, 512, 512, 3, 2, 1, 1, False, synth.U8, False),     # stride 2: boxes traversed with the convolution stride
    (28, 28, 96, 48, 1, 2, 0, 1, True, synth.U8, False),        # 1x1 stride 2 (a down-sampling shortcut), ragged K chunk
    (15, 17, 32, 40, 3, 1, 1, 3, False, synth.S32, False),      # int32 output through the generic epilogue, odd sizes
    (20, 20, 64, 32, 5, 1, 2, 2, False, synth.U8, True),        # 5x5
    (9, 31, 16, 24, 3, 2, 0, 5, True, synth.S8, False),         # no padding, stride 2, c_out = 24
    (6, 100, 128, 64, 3, 1, 1, 1, False, synth.U8, False),      # one row of 100 positions per tile
    (6, 100, 64, 64, 3, 1, 1, 2, False, synth.U8, False),       # the same with 64-byte rows: row tiles
]


@pytest.mark.parametrize("case", range(len(SMALL_ROW_TILED)))
def test_small_layers_row_tiled_on_tensor_cores(ref, case):
    from paper_2202_05239_b200 import api as a
    h, w, c, c_out, k, stride, pad, n, xs, y_dtype, with_res = SMALL_ROW_TILED[case]
    rng = np.random.default_rng(800 + case)
    layer = random_conv_layer(rng, h=h, w=w, c=c, c_out=c_out, k=k, stride=stride, pad=pad, x_signed=xs, y_dtype=y_dtype,
                              with_res=with_res)
    x = random_input(rng, n, layer)
    assert 4096 <= x.size < 128 * 1024
    res = random_residual(rng, n, layer) if with_res else None
    # the first and the last case are also eligible for the windowed mode (which reads through a tiled map as well)
    check_layer(ref, layer, x, res, expect_tc=True, expect_flags=a.PLAN_WINDOWED if case in (0, 8) else a.PLAN_ROW_TILES)


def test_extreme_operands_on_tensor_cores(ref):
    """-128 weights against 255 / -128 activations: the signedness selection of the MMA must be right."""
    rng = np.random.default_rng(5)
    for xs in (False, True):
        layer = random_conv_layer(rng, h=32, w=32, c=128, c_out=64, k=1, stride=1, pad=0, x_signed=xs, y_dtype=synth.S32,
                                  with_res=False, wide=True)
        layer.weight[:] = -128
        layer.weight[1::2] = 127
        x = random_input(rng, 1, layer)
        x[:] = -128 if xs else 255
        check_layer(ref, layer, x, expect_tc=True)


@pytest.mark.parametrize("index", range(6))
def test_layer_sweep_shapes(ref, index):
    """The CNN layer-shape sweep at its stated batch of 32 (the oracle needs a fraction of a second per layer)."""
    layer, x = synth.sweep_case(index, batch=32, seed=0)
    check_layer(ref, layer, x, expect_tc=True)


# Cases in which every CTA walks several tiles: the accumulator double buffer, the stage ring, the output ring and the
# second issuer's tile alternation all wrap around.  One case per plan mode and epilogue variant; the mode is asserted.
#   (h, w, c, c_out, k, stride, n, x_signed, y_dtype, res, plan_off, expect, forbid)
def _modes():
    from paper_2202_05239_b200 import api as a
    RW, WIN, DUAL, ALT, STAGED = (a.PLAN_RESIDENT_WEIGHTS, a.PLAN_WINDOWED, a.PLAN_DUAL_ISSUE, a.PLAN_ALT_PRODUCERS,
                                  a.PLAN_STAGED_EPILOGUE)
    return [
        # resident weights, two issuers, u8
        (56, 56, 64, 64, 1, 1, 32, False, synth.U8, False, 0, RW | DUAL | STAGED, WIN),
        # resident weights, 256-wide tile, residual, u8 and s8 outputs
        (56, 56, 64, 256, 1, 1, 32, False, synth.U8, True, 0, RW | STAGED, 0),
        (56, 56, 64, 256, 1, 1, 32, True, synth.S8, True, 0, RW | STAGED, 0),
        # signed output without residual, resident weights, 3x3 through im2col, two issuers
        (56, 56, 64, 64, 3, 1, 32, False, synth.S8, False, 0, RW | DUAL | STAGED, WIN),
        # streamed weights, two N tiles, second producer pair
        (28, 28, 512, 512, 1, 1, 50, False, synth.U8, False, 0, ALT | STAGED, RW),
        # the same without the second producer pair
        (28, 28, 512, 512, 1, 1, 50, False, synth.U8, False, a.PLAN_OFF_ALT_PRODUCERS, STAGED, RW | ALT),
        # K-heavy 3x3 through im2col, streamed weights
        (14, 14, 256, 256, 3, 1, 400, False, synth.U8, False, 0, STAGED, RW),
        # windowed 3x3 with residual
        (28, 28, 128, 128, 3, 1, 100, False, synth.U8, True, 0, WIN | RW | STAGED, 0),
        # the same layer through im2col (windowed mode off), then with streamed weights as well
        (28, 28, 128, 128, 3, 1, 100, False, synth.U8, True, a.PLAN_OFF_WINDOWED, STAGED, WIN),
        (28, 28, 128, 128, 3, 1, 100, False, synth.U8, True, a.PLAN_OFF_RESIDENT_WEIGHTS, STAGED, WIN | RW),
        # one issuer where two are the default
        (56, 56, 64, 64, 1, 1, 32, False, synth.U8, False, a.PLAN_OFF_DUAL_ISSUE, RW | STAGED, DUAL),
        # int32 output: generic epilogue with direct stores, many tiles
        (56, 56, 256, 64, 1, 1, 32, False, synth.S32, False, 0, 0, STAGED),
        # stride 2 with residual and streamed weights
        (56, 56, 128, 128, 3, 2, 100, False, synth.U8, True, 0, STAGED, 0),
    ]


# CTA pairs (tcgen05 cta_group::2): K-heavy layers with 256-wide tiles; 256-row tiles shared by two CTAs
# (h, w, c, c_out, k, stride, n, x_signed, y_dtype, res)
PAIR_CASES = [
    (14, 14, 1024, 256, 1, 1, 64, False, synth.U8, False),      # eight K chunks, 98 M tiles: 49 pair tiles
    (14, 14, 512, 256, 3, 1, 33, True, synth.U8, False),        # 3x3 through im2col, signed input; 51 M tiles: the last pair is half empty
    (7, 7, 512, 512, 3, 1, 64, True, synth.S8, False),          # two N tiles, 36 K iterations, signed
    (14, 14, 1024, 2048, 1, 2, 40, False, synth.S8, False),     # stride-2 shortcut convolution, eight N tiles
    (7, 7, 2048, 512, 1, 1, 256, False, synth.U8, False),       # 98 M tiles x 2 N tiles on 74 pairs: several tiles per pair
    (9, 9, 1024, 256, 1, 1, 3, False, synth.U8, False),         # 243 pixels: one pair, second CTA nearly empty
    (14, 14, 256, 256, 3, 1, 96, False, synth.U8, True),        # K-heavy layer with a shortcut (basic residual block): 74 pair tiles
    (7, 7, 512, 512, 3, 1, 64, False, synth.S8, True),          # the same with two N tiles and a signed output
    (13, 13, 256, 256, 3, 1, 5, True, synth.U8, True),          # ragged: 845 pixels, the last pair tile half empty, signed input
]


@pytest.mark.parametrize("case", range(len(PAIR_CASES)))
def test_cta_pairs(ref, case):
    from paper_2202_05239_b200 import api as a
    h, w, c, c_out, k, stride, n, xs, y_dtype, with_res = PAIR_CASES[case]
    rng = np.random.default_rng(1200 + case)
    layer = random_conv_layer(rng, h=h, w=w, c=c, c_out=c_out, k=k, stride=stride, pad=k // 2, x_signed=xs, y_dtype=y_dtype,
                              with_res=with_res)
    x = random_input(rng, n, layer)
    res = random_residual(rng, n, layer) if with_res else None
    check_layer(ref, layer, x, res, expect_tc=True, expect_flags=a.PLAN_PAIRS)
    if case in (0, 2):      # the same layer on single CTAs
        check_layer(ref, layer, x, res, expect_tc=True, plan_off=a.PLAN_OFF_PAIRS, forbid_flags=a.PLAN_PAIRS)


# Pointwise layers with a single K chunk and narrow tiles: several M tiles share one stage use and one accumulator hand-over
# (h, w, c, c_out, n, x_signed, y_dtype)
GROUP_CASES = [
    (56, 56, 64, 64, 100, False, synth.U8),       # groups of four 64-wide tiles; 2450 M tiles
    (56, 56, 64, 64, 97, True, synth.S8),         # 2377 M tiles: the last group holds one tile, and that one is ragged
    (112, 112, 32, 64, 25, False, synth.U8),      # 32-byte K chunk
    (56, 56, 64, 128, 50, False, synth.U8),       # groups of two 128-wide tiles
    (56, 56, 128, 96, 50, True, synth.U8),        # 96 of 128 columns exist: the last two chunks of every tile are skipped
    (56, 56, 16, 32, 100, False, synth.S8),       # 16 channels in a 32-byte chunk, 32-wide tiles: half of the accumulator unused
]


@pytest.mark.parametrize("case", range(len(GROUP_CASES)))
def test_groups_of_m_tiles(ref, case):
    from paper_2202_05239_b200 import api as a
    h, w, c, c_out, n, xs, y_dtype = GROUP_CASES[case]
    rng = np.random.default_rng(1500 + case)
    layer = random_conv_layer(rng, h=h, w=w, c=c, c_out=c_out, k=1, stride=1, pad=0, x_signed=xs, y_dtype=y_dtype, with_res=False)
    x = random_input(rng, n, layer)
    check_layer(ref, layer, x, None, expect_tc=True, expect_flags=a.PLAN_TILE_GROUPS | a.PLAN_RESIDENT_WEIGHTS)
    if case in (1, 4):      # the same layer with one tile per hand-over
        check_layer(ref, layer, x, None, expect_tc=True, plan_off=a.PLAN_OFF_TILE_GROUPS, forbid_flags=a.PLAN_TILE_GROUPS)


@pytest.mark.parametrize("case", range(13))
def test_many_tiles_per_cta_in_every_plan_mode(ref, case):
    h, w, c, c_out, k, stride, n, xs, y_dtype, with_res, off, expect, forbid = _modes()[case]
    rng = np.random.default_rng(900 + case)
    layer = random_conv_layer(rng, h=h, w=w, c=c, c_out=c_out, k=k, stride=stride, pad=k // 2, x_signed=xs,
                              y_dtype=y_dtype, with_res=with_res)
    x = random_input(rng, n, layer)
    res = random_residual(rng, n, layer) if with_res else None
    check_layer(ref, layer, x, res, expect_tc=True, plan_off=off, expect_flags=expect, forbid_flags=forbid,
                min_tiles_per_cta=4)


def test_linear_on_tensor_cores(ref):
    rng = np.random.default_rng(11)
    n, k, out = 256, 2048, 1000
    wgt = np.clip(np.round(rng.normal(0, 20, size=(out, k))), -128, 127).astype(np.int8)
    bias = rng.integers(-5000, 5000, size=out).astype(np.int32)
    layer = synth.Layer(synth.LINEAR, "fc", 0, -1, 1, 1, k, out, 1, 1, 1, 0, synth.U8, synth.S32, synth.U8, 6, 9, 3, 0, wgt, bias)
    x = rng.integers(0, 256, size=(n, k)).astype(np.uint8)
    check_layer(ref, layer, x, expect_tc=True)
