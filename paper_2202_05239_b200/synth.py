"""Seeded synthetic inputs: layer descriptions, integer tensors and FL tables.

This module only *draws* things: 8-bit tensors, int8 weights, int32 biases and
the per-layer fractional lengths (FL) that go with them.  It performs none of
the fixed-point layer arithmetic (no convolution, no rounding shift, no clip
of an accumulator); both the CUDA library and the CPU oracle consume what it
returns, so neither depends on the other.

Recipe (synthetic stand-ins for the trained ImageNet networks of the paper's
Sec. 5, which need data and weights that are not available):

* weights of a layer with fan-in ``n`` are real Gaussians ``N(0, sigma)`` with
  the He value ``sigma = sqrt(2/n)``; "BN folded" is modelled the way a freshly
  initialised BatchNorm behaves: the folded scale (gamma / running std in
  Eq. 6) is ``1/std`` of the layer's own pre-activation, so every conv output
  has unit variance before the activation.  The pre-activation std is tracked
  analytically through the net (Gaussian moment propagation), never measured
  by running a layer;
* the weight format follows "3 sigma fits the 8-bit range":
  ``FL_w = floor(log2(127 / (3 std(W))))`` on the drawn real tensor, and the
  integer code is ``clip(floor(W 2^FL_w + 1/2), -128, 127)``;
* activation formats follow the paper's Eq. 1 on the modelled pre-activation
  std: unsigned ``floor(log2(70/sigma))`` in [0, 8] after ReLU, signed
  ``floor(log2(40/sigma))`` in [0, 7] otherwise;
* biases are ``floor(N(0, 0.1) 2^(FL_x+FL_w) + 1/2)`` (accumulator format);
* images are ``clip(floor(N(0,1) 64 + 1/2), -127, 127)`` int8 with FL 6.

Tensor numbering inside a net: tensor 0 is the image, layer ``i`` writes
tensor ``i + 1``; ``src`` / ``res`` are tensor numbers (``res = -1``: none).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np

U8, S8, S32 = 0, 1, 2
S32_RELU = 3      # output kind of sibling handling only: the 32-bit sum behind a ReLU (stored like S32)
CONV, DWCONV, MAXPOOL, GAP, LINEAR = 0, 1, 2, 3, 4
SIBLING = 5       # a second consumer's view of the previous layer's 32-bit sum, with its private format (Sec. 4.3)
KIND_NAMES = {CONV: "conv", DWCONV: "dwconv", MAXPOOL: "maxpool", GAP: "gap", LINEAR: "linear", SIBLING: "sibling"}


@dataclass
class Layer:
    kind: int
    name: str
    src: int                      # input tensor number
    res: int                      # residual tensor number or -1
    h: int                        # input height / width / channels (per image)
    w: int
    c: int
    c_out: int
    kh: int = 1
    kw: int = 1
    stride: int = 1
    pad: int = 0
    x_dtype: int = U8
    y_dtype: int = U8             # U8: clip [0,255] (ReLU); S8: clip [-127,127]; S32: raw accumulator
    r_dtype: int = U8
    fl_x: int = 0
    fl_w: int = 0
    fl_y: int = 0
    fl_r: int = 0
    weight: Optional[np.ndarray] = None   # conv: [c_out,kh,kw,c]; dwconv: [c,kh,kw]; linear: [out,k]
    bias: Optional[np.ndarray] = None     # [c_out] int32, accumulator format
    ho: int = field(init=False, default=0)
    wo: int = field(init=False, default=0)

    def __post_init__(self):
        if self.kind in (CONV, DWCONV, MAXPOOL, SIBLING):
            self.ho = (self.h + 2 * self.pad - self.kh) // self.stride + 1
            self.wo = (self.w + 2 * self.pad - self.kw) // self.stride + 1
        else:
            self.ho, self.wo = 1, 1

    @property
    def macs_per_image(self) -> int:
        if self.kind == CONV:
            return self.ho * self.wo * self.c_out * self.kh * self.kw * self.c
        if self.kind == DWCONV:
            return self.ho * self.wo * self.c * self.kh * self.kw
        if self.kind == LINEAR:
            return self.c * self.c_out
        return 0

    def bytes_per_image(self) -> int:
        """Algorithmic activation bytes per image: input + output (+ residual)."""
        ysz = 4 if self.y_dtype in (S32, S32_RELU) else 1
        out = self.ho * self.wo * self.c_out * ysz
        if self.kind == SIBLING:
            return out                      # a second output of the parent's launch: written, nothing read
        rsz = 4 if self.r_dtype == S32 else 1
        return self.h * self.w * self.c + out + (self.ho * self.wo * self.c_out * rsz if self.res >= 0 else 0)

    def param_bytes(self) -> int:
        b = 0
        if self.weight is not None:
            b += self.weight.size
        if self.bias is not None:
            b += 4 * self.bias.size
        return b


# --------------------------------------------------------------------------
# small helpers (random draws and format choices only)
# --------------------------------------------------------------------------

def _rng(seed: int, *stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, *stream])))


def round_half_up(v: np.ndarray) -> np.ndarray:
    return np.floor(v + 0.5)


def fl_weight(std: float) -> int:
    """Largest FL such that three standard deviations still fit in [-127, 127]."""
    return int(math.floor(math.log2(127.0 / (3.0 * std))))


def fl_unsigned(std: float) -> int:
    """Eq. 1, unsigned branch, clamped to the unsigned 8-bit range of Eq. 2."""
    return int(min(8, max(0, math.floor(math.log2(70.0 / std)))))


def fl_signed(std: float) -> int:
    """Eq. 1, signed branch, clamped to the signed 8-bit range."""
    return int(min(7, max(0, math.floor(math.log2(40.0 / std)))))


def draw_weight(rng: np.random.Generator, shape: Tuple[int, ...], sigma: float) -> Tuple[np.ndarray, int]:
    real = rng.normal(0.0, sigma, size=shape)
    flw = fl_weight(float(real.std()))
    code = np.clip(round_half_up(real * 2.0 ** flw), -128, 127).astype(np.int8)
    return code, flw


def draw_bias(rng: np.random.Generator, n: int, fa: int, sigma: float = 0.1) -> np.ndarray:
    return round_half_up(rng.normal(0.0, sigma, size=n) * 2.0 ** fa).astype(np.int32)


def draw_image(batch: int, seed: int, h: int = 224, w: int = 224, c: int = 3) -> np.ndarray:
    """int8 NHWC images, FL 6 (a normalised, signed network input)."""
    rng = _rng(seed, 7001)
    return np.clip(round_half_up(rng.normal(0.0, 1.0, size=(batch, h, w, c)) * 64.0), -127, 127).astype(np.int8)


def draw_unsigned_activation(rng: np.random.Generator, shape, fl: int) -> np.ndarray:
    return np.clip(round_half_up(np.abs(rng.normal(0.0, 1.0, size=shape)) * 2.0 ** fl), 0, 255).astype(np.uint8)


# --------------------------------------------------------------------------
# single-layer cases
# --------------------------------------------------------------------------

def single_conv_case(seed: int = 0):
    """One 3x3 conv on a 1x16x16x16 uint8 image, all tensors uniform.

    x U[0,255] FL 4; w U[-128,127] FL 7; bias U[-2^12, 2^12] in format 11;
    output FL 4, ReLU + clip [0,255].
    """
    rng = _rng(seed, 1)
    x = rng.integers(0, 256, size=(1, 16, 16, 16), dtype=np.int64).astype(np.uint8)
    wgt = rng.integers(-128, 128, size=(16, 3, 3, 16), dtype=np.int64).astype(np.int8)
    bias = rng.integers(-(1 << 12), (1 << 12) + 1, size=16, dtype=np.int64).astype(np.int32)
    layer = Layer(CONV, "conv3x3_16", 0, -1, 16, 16, 16, 16, 3, 3, 1, 1, U8, U8, U8, 4, 7, 4, 0, wgt, bias)
    return layer, x


SWEEP_SHAPES = [
    # name,            h,  c_in, c_out, k
    ("c3x3_56_64", 56, 64, 64, 3),
    ("c3x3_28_128", 28, 128, 128, 3),
    ("c3x3_14_256", 14, 256, 256, 3),
    ("c3x3_7_512", 7, 512, 512, 3),
    ("c1x1_56_256_64", 56, 256, 64, 1),
    ("c1x1_14_1024_256", 14, 1024, 256, 1),
]


def sweep_case(index: int, batch: int = 32, seed: int = 0):
    """One layer of the CNN layer-shape sweep: He weights, |N(0,1)| activations FL 5, output FL 5."""
    name, h, ci, co, k = SWEEP_SHAPES[index]
    rng = _rng(seed, 2, index)
    fan_in = k * k * ci
    wgt, flw = draw_weight(rng, (co, k, k, ci), math.sqrt(2.0 / fan_in))
    bias = draw_bias(rng, co, 5 + flw)
    x = draw_unsigned_activation(rng, (batch, h, h, ci), 5)
    layer = Layer(CONV, name, 0, -1, h, h, ci, co, k, k, 1, k // 2, U8, U8, U8, 5, flw, 5, 0, wgt, bias)
    return layer, x


# --------------------------------------------------------------------------
# moment model used to pick activation FLs without running any layer
# --------------------------------------------------------------------------

@dataclass
class _Stat:
    """Mean / variance of the *real* values a tensor stands for (Gaussian model)."""
    mean: float
    var: float
    dtype: int
    fl: int
    h: int
    w: int
    c: int

    @property
    def m2(self) -> float:
        return self.mean * self.mean + self.var


def _phi(z: float) -> float:
    return math.exp(-0.5 * z * z) / math.sqrt(2.0 * math.pi)


def _Phi(z: float) -> float:
    return 0.5 * (1.0 + math.erf(z / math.sqrt(2.0)))


def _relu_moments(mu: float, var: float) -> Tuple[float, float]:
    """Mean and variance of max(0, z), z ~ N(mu, var)."""
    sd = math.sqrt(var)
    a = mu / sd
    m1 = mu * _Phi(a) + sd * _phi(a)
    m2 = (mu * mu + var) * _Phi(a) + mu * sd * _phi(a)
    return m1, max(m2 - m1 * m1, 1e-12)


class _NetBuilder:
    def __init__(self, seed: int, stream: int, h: int, w: int, c: int):
        self.seed, self.stream = seed, stream
        self.layers: List[Layer] = []
        self.drawn = 0            # layers that drew random numbers so far (sibling layers draw none)
        # image: N(0,1) real values in s8 FL 6
        self.stats: List[_Stat] = [_Stat(0.0, 1.0, S8, 6, h, w, c)]

    def _rng(self) -> np.random.Generator:
        # one stream per layer, numbered without the sibling layers: a net with sibling layers draws the same
        # weights as the same net without them
        return _rng(self.seed, self.stream, len(self.layers) - sum(1 for l in self.layers if l.kind == SIBLING))

    def _finish(self, layer: Layer, pre_mean: float, pre_var: float, relu: bool, keep32: bool = False) -> int:
        sd = math.sqrt(pre_var)
        if relu:
            layer.y_dtype, layer.fl_y = U8, fl_unsigned(sd)
            m1, v = _relu_moments(pre_mean, pre_var)
        else:
            layer.y_dtype, layer.fl_y = S8, fl_signed(sd)
            m1, v = pre_mean, pre_var
        fl_out = layer.fl_y
        if keep32:      # the sum itself, in the format of the aligned sum
            layer.y_dtype = S32_RELU if relu else S32
            fl_out = max(layer.fl_x + layer.fl_w, layer.fl_r) if layer.res >= 0 else layer.fl_x + layer.fl_w
        self.layers.append(layer)
        self.stats.append(_Stat(m1, v, S32 if keep32 else layer.y_dtype, fl_out, layer.ho, layer.wo, layer.c_out))
        return len(self.stats) - 1

    def sibling(self, name: str, parent: int, y_dtype: int, fl_y: int = 0) -> int:
        """Second consumer of the sum that produced tensor `parent` (which must be the newest tensor)."""
        assert parent == len(self.stats) - 1 and self.layers[-1].kind == CONV
        p, ps = self.layers[-1], self.stats[parent]
        layer = Layer(SIBLING, name, parent, -1, ps.h, ps.w, ps.c, ps.c, 1, 1, 1, 0, p.x_dtype, y_dtype, U8,
                      p.fl_x, p.fl_w, fl_y, 0)
        self.layers.append(layer)
        wide = y_dtype in (S32, S32_RELU)
        fl_sum = max(p.fl_x + p.fl_w, p.fl_r) if p.res >= 0 else p.fl_x + p.fl_w
        self.stats.append(_Stat(ps.mean, ps.var, S32 if wide else y_dtype, fl_sum if wide else fl_y, ps.h, ps.w, ps.c))
        return len(self.stats) - 1

    def conv(self, name: str, src: int, c_out: int, k: int, stride: int, relu: bool, res: int = -1,
             depthwise: bool = False, keep32: bool = False) -> int:
        s = self.stats[src]
        rng = self._rng()
        fan_in = k * k * (1 if depthwise else s.c)
        # He draw, then the folded BatchNorm scale 1/std(pre-activation): net sigma below
        sigma = math.sqrt(2.0 / fan_in) / math.sqrt(2.0 * s.m2)
        shape = (s.c, k, k) if depthwise else (c_out, k, k, s.c)
        wgt, flw = draw_weight(rng, shape, sigma)
        fa = s.fl + flw
        bias = draw_bias(rng, c_out, fa)
        layer = Layer(DWCONV if depthwise else CONV, name, src, res, s.h, s.w, s.c, c_out, k, k, stride, k // 2,
                      s.dtype, U8, U8, s.fl, flw, 0, 0, wgt, bias)
        pre_mean, pre_var = 0.0, fan_in * sigma * sigma * s.m2 + 0.01
        if res >= 0:
            r = self.stats[res]
            layer.r_dtype, layer.fl_r = r.dtype, r.fl
            pre_mean += r.mean
            pre_var += r.var
        return self._finish(layer, pre_mean, pre_var, relu, keep32)

    def maxpool(self, name: str, src: int, k: int = 3, stride: int = 2, pad: int = 1) -> int:
        s = self.stats[src]
        layer = Layer(MAXPOOL, name, src, -1, s.h, s.w, s.c, s.c, k, k, stride, pad, s.dtype, s.dtype, U8,
                      s.fl, 0, s.fl, 0)
        self.layers.append(layer)
        # max of k*k neighbouring rectified unit Gaussians (rough: mean 1.35 sd, variance 0.45 var)
        sd = math.sqrt(s.var / 0.34) if s.dtype == U8 else math.sqrt(s.var)
        self.stats.append(_Stat(1.35 * sd, 0.45 * sd * sd, s.dtype, s.fl, layer.ho, layer.wo, s.c))
        return len(self.stats) - 1

    def gap(self, name: str, src: int) -> int:
        s = self.stats[src]
        hw = s.h * s.w
        d = max(0, math.ceil(math.log2(hw)))
        scale = hw / float(1 << d)
        mean, var = s.mean * scale, s.var * hw / float(1 << d) ** 2
        size = math.sqrt(mean * mean + var)
        fl = fl_unsigned(size) if s.dtype == U8 else fl_signed(size)
        layer = Layer(GAP, name, src, -1, s.h, s.w, s.c, s.c, 1, 1, 1, 0, s.dtype, s.dtype, U8, s.fl, 0, fl, 0)
        self.layers.append(layer)
        self.stats.append(_Stat(mean, var, s.dtype, fl, 1, 1, s.c))
        return len(self.stats) - 1

    def linear(self, name: str, src: int, out: int) -> int:
        s = self.stats[src]
        rng = self._rng()
        k = s.c
        sigma = 1.0 / math.sqrt(k * s.m2)
        wgt, flw = draw_weight(rng, (out, k), sigma)
        bias = draw_bias(rng, out, s.fl + flw)
        layer = Layer(LINEAR, name, src, -1, 1, 1, k, out, 1, 1, 1, 0, s.dtype, S32, U8, s.fl, flw, s.fl + flw, 0,
                      wgt, bias)
        self.layers.append(layer)
        self.stats.append(_Stat(0.0, 1.0, S32, s.fl + flw, 1, 1, out))
        return len(self.stats) - 1


# --------------------------------------------------------------------------
# network shapes (widths and block counts as in the public architecture papers;
# the paper under study names the networks but does not list their layers)
# --------------------------------------------------------------------------

def resnet18(seed: int = 0, image: int = 224, siblings: bool = False) -> List[Layer]:
    """siblings=False: every activation is one 8-bit tensor that all of its consumers read (re-aligned by shifts
    where their formats differ).  siblings=True: the handling the paper describes for layers with two children
    (Sec. 4.3, Fig. 4) -- the sum of a block's last layer stays in 32 bits and is quantised once per child: the next
    block's first convolution reads the master format, its down-sampling convolution (where there is one) a private
    format one bit finer (a synthetic stand-in: trained formats are not available), and an identity shortcut takes
    the 32-bit value itself (behind the ReLU, unrounded); a down-sampling convolution also hands its sum on in 32 bits.
    Weights are the same in both variants."""
    b = _NetBuilder(seed, 18, image, image, 3)
    t = b.conv("stem", 0, 64, 7, 2, True)
    t = b.maxpool("pool", t)
    t_private, t_wide = None, None          # the newest block output in a private 8-bit format / in 32 bits
    widths = [64, 128, 256, 512]
    for si, width in enumerate(widths):
        for bi in range(2):
            stride = 2 if (bi == 0 and si > 0) else 1
            short = t_wide if t_wide is not None else t
            if stride != 1 or b.stats[t].c != width:
                short = b.conv(f"s{si}b{bi}.down", t_private if t_private is not None else t, width, 1, stride, False,
                               keep32=siblings)
            u = b.conv(f"s{si}b{bi}.conv1", t, width, 3, stride, True)
            t = b.conv(f"s{si}b{bi}.conv2", u, width, 3, 1, True, res=short)
            t_private, t_wide = None, None
            last = si == len(widths) - 1 and bi == 1
            if siblings and not last:
                if bi == 1:      # the next block starts a stage: its down-sampling convolution is the second child
                    t_private = b.sibling(f"s{si}b{bi}.conv2.private", t, U8, min(8, b.stats[t].fl + 1))
                else:            # the next block adds this block's output back in: kept in 32 bits
                    t_wide = b.sibling(f"s{si}b{bi}.conv2.wide", t, S32_RELU)
    t = b.gap("gap", t)
    b.linear("fc", t, 1000)
    return b.layers


def resnet50(seed: int = 0, image: int = 224) -> List[Layer]:
    b = _NetBuilder(seed, 50, image, image, 3)
    t = b.conv("stem", 0, 64, 7, 2, True)
    t = b.maxpool("pool", t)
    for si, (width, blocks) in enumerate(zip([64, 128, 256, 512], [3, 4, 6, 3])):
        for bi in range(blocks):
            stride = 2 if (bi == 0 and si > 0) else 1     # stride on the 3x3 of the bottleneck
            short = t
            if bi == 0:
                short = b.conv(f"s{si}b{bi}.down", t, 4 * width, 1, stride, False)
            u = b.conv(f"s{si}b{bi}.conv1", t, width, 1, 1, True)
            u = b.conv(f"s{si}b{bi}.conv2", u, width, 3, stride, True)
            t = b.conv(f"s{si}b{bi}.conv3", u, 4 * width, 1, 1, True, res=short)
    t = b.gap("gap", t)
    b.linear("fc", t, 1000)
    return b.layers


def mobilenetv2(seed: int = 0, image: int = 224) -> List[Layer]:
    b = _NetBuilder(seed, 2, image, image, 3)
    t = b.conv("stem", 0, 32, 3, 2, True)
    cfg = [(1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2), (6, 96, 3, 1), (6, 160, 3, 2), (6, 320, 1, 1)]
    bi = 0
    for expand, c_out, repeats, first_stride in cfg:
        for r in range(repeats):
            stride = first_stride if r == 0 else 1
            c_in = b.stats[t].c
            u = t
            if expand != 1:
                u = b.conv(f"b{bi}.expand", u, c_in * expand, 1, 1, True)
            u = b.conv(f"b{bi}.dw", u, b.stats[u].c, 3, stride, True, depthwise=True)
            use_res = stride == 1 and c_in == c_out
            t = b.conv(f"b{bi}.project", u, c_out, 1, 1, False, res=t if use_res else -1)
            bi += 1
    t = b.conv("head", t, 1280, 1, 1, True)
    t = b.gap("gap", t)
    b.linear("fc", t, 1000)
    return b.layers


def mobilenetv1(seed: int = 0, image: int = 224) -> List[Layer]:
    """13 depthwise-separable blocks (3x3 depthwise + 1x1 pointwise, ReLU after both, no shortcuts), widths and strides of the
    public MobileNet architecture at width multiplier 1."""
    b = _NetBuilder(seed, 1, image, image, 3)
    t = b.conv("stem", 0, 32, 3, 2, True)
    cfg = [(64, 1), (128, 2), (128, 1), (256, 2), (256, 1), (512, 2), (512, 1), (512, 1), (512, 1), (512, 1), (512, 1),
           (1024, 2), (1024, 1)]
    for bi, (c_out, stride) in enumerate(cfg):
        t = b.conv(f"b{bi}.dw", t, b.stats[t].c, 3, stride, True, depthwise=True)
        t = b.conv(f"b{bi}.pw", t, c_out, 1, 1, True)
    t = b.gap("gap", t)
    b.linear("fc", t, 1000)
    return b.layers


NETS = {"resnet18": resnet18, "resnet50": resnet50, "mobilenetv2": mobilenetv2, "mobilenetv1": mobilenetv1}


def resnet18_siblings(seed: int = 0, image: int = 224) -> List[Layer]:
    return resnet18(seed, image, siblings=True)


NETS["resnet18_siblings"] = resnet18_siblings


def make_net(name: str, seed: int = 0, image: int = 224) -> List[Layer]:
    return NETS[name](seed, image)


def net_macs_per_image(layers: List[Layer]) -> int:
    return sum(l.macs_per_image for l in layers)


def net_bytes(layers: List[Layer], batch: int) -> int:
    """Layer-wise algorithmic bytes for one forward pass of ``batch`` images."""
    return sum(batch * l.bytes_per_image() + l.param_bytes() for l in layers)
