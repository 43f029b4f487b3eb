/*
 * f8ref.c -- CPU oracle for F8Net's fixed-point 8-bit inference arithmetic.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is checked against.  Nothing in the product path includes,
 * links or calls it, and it shares no code, header, table or helper with the
 * CUDA sources.
 *
 * What it computes (paper: Eq. 2 = unsigned fix_quant, the signed fix_quant of
 * the appendix "Double Side Quantization", Eq. 6 = fix_quant of effective
 * weight x fixed-point activation + effective bias, Sec. 4.3 / Fig. 4 = the
 * residual siblings that differ only by bit shifts):
 *
 *   every tensor element is an 8-bit integer code q with a per-tensor
 *   fractional length FL, standing for the real number q * 2^-FL.
 *   A layer evaluates, for each output element,
 *
 *       v  = sum_taps (w 2^-FLw)(x 2^-FLx) + b 2^-(FLx+FLw) [+ r 2^-FLr]
 *       y  = clip(round(v * 2^FLy), lo, hi)                (the integer code)
 *
 *   with [lo,hi] = [0,255] for the unsigned quantizer (Eq. 2, used after
 *   ReLU / PACT) and [-127,127] for the signed one.  All terms are dyadic
 *   rationals, so v * 2^F is an exact integer for F = max(FLx+FLw, FLr); the
 *   function below forms that integer in int64 and applies the quantizer as
 *   one rounding shift.
 *
 * Readings where the paper is silent (each is restated where it is used):
 *   - round() is round-half-up, floor(v + 1/2);
 *   - rounding then clipping (equal to the paper's clip-then-round because the
 *     clip bounds are integers and the rounding is monotone);
 *   - a negative shift is an exact left shift followed by the clip;
 *   - the shortcut operand of a residual add is an 8-bit tensor, added to the
 *     accumulator before the single rounding;
 *   - max pooling ignores padded taps; global average pooling is a sum
 *     followed by a rounding shift by ceil(log2(H*W)) + FLx - FLy.
 *
 * Pins: tests/test_oracle_*.py check these functions against hand-worked
 * values (tests/golden/), exact evaluation of the real-valued definition in
 * double / Python integers, torch float64 conv2d / max_pool2d / linear on the
 * integer tensors, and algebraic identities.  The network-level choices
 * (topology, pooling, calibration of FLs) have no counterpart in the paper:
 * for those, parity is pinned only by the stated reading.
 *
 * Loop nests are direct (n, oh, ow, co, kh, kw, ci); the only concession to
 * run time is an OpenMP pragma over (n, oh).  No blocking, no intrinsics.
 */
#include <stdint.h>
#include <stddef.h>

#define F8REF_OK            0
#define F8REF_ERR_ARG       1
#define F8REF_ERR_ACC_RANGE 2   /* an accumulator left the int32 range */

/* Eq. 2 / signed fix_quant on an exact integer numerator.
 * acc stands for the real value acc * 2^-FA; the result is the integer code of
 * fix_quant with fractional length FLy, s = FA - FLy:
 *     round(acc * 2^-s) with ties toward +infinity, then clip to [lo, hi]. */
int64_t f8ref_shift_round_clip(int64_t acc, int s, int64_t lo, int64_t hi)
{
    int64_t t;
    if (s > 0) {
        /* floor((acc + 2^(s-1)) / 2^s): >> on a negative int64 is an arithmetic
         * shift with gcc, i.e. floor division by a power of two. */
        t = (acc + ((int64_t)1 << (s - 1))) >> s;
    } else {
        t = acc * ((int64_t)1 << (-s));
    }
    if (t < lo) t = lo;
    if (t > hi) t = hi;
    return t;
}

static int64_t load8(const void *p, size_t i, int is_signed)
{
    return is_signed ? (int64_t)((const int8_t *)p)[i] : (int64_t)((const uint8_t *)p)[i];
}

/* Common tail of every layer (Eq. 6 argument -> Eq. 2): bias is already inside
 * acc.  Aligns the optional residual code r (format FLr) with the accumulator
 * (format FA) on the finer of the two formats -- a pure shift, Sec. 4.3 and the
 * appendix on private fractional lengths -- adds, and quantizes once. */
static int finish(int64_t acc, int fa, int has_res, int64_t r, int fl_r, int fl_y,
                  int y_kind /*0 u8, 1 s8, 2 s32 raw*/, void *y, size_t yi)
{
    if (acc > INT32_MAX || acc < INT32_MIN) return F8REF_ERR_ACC_RANGE;
    if (has_res) {
        int f = fa > fl_r ? fa : fl_r;
        acc = acc * ((int64_t)1 << (f - fa)) + r * ((int64_t)1 << (f - fl_r));
        fa = f;
        if (acc > INT32_MAX || acc < INT32_MIN) return F8REF_ERR_ACC_RANGE;
    }
    if (y_kind == 2) {               /* raw accumulator, format FA, no quantizer */
        ((int32_t *)y)[yi] = (int32_t)acc;
    } else if (y_kind == 0) {        /* Eq. 2: unsigned, [0, 2^8 - 1] */
        ((uint8_t *)y)[yi] = (uint8_t)f8ref_shift_round_clip(acc, fa - fl_y, 0, 255);
    } else {                         /* signed fix_quant: [-2^7 + 1, 2^7 - 1] */
        ((int8_t *)y)[yi] = (int8_t)f8ref_shift_round_clip(acc, fa - fl_y, -127, 127);
    }
    return F8REF_OK;
}

/*
 * Dense convolution layer (Eq. 6 with the sum running over a kh x kw x ci
 * window; cross-correlation, zero outside the image).
 *   x   : [n, h, w, ci]   u8 (x_signed = 0) or s8 (x_signed = 1), format fl_x
 *   wgt : [co, kh, kw, ci] s8, format fl_w
 *   bias: [co] int32 in the accumulator format fl_x + fl_w, may be NULL (= 0)
 *   res : NULL or [n, ho, wo, co] 8-bit (r_signed), format fl_r
 *   y   : [n, ho, wo, co]; y_kind 0 = u8 clip [0,255], 1 = s8 clip [-127,127],
 *         2 = int32 raw accumulator (fl_y ignored)
 */
int f8ref_conv2d(int n, int h, int w, int ci, int co, int kh, int kw, int stride, int pad,
                 int x_signed, int fl_x, int fl_w, int fl_y, int y_kind,
                 const void *x, const int8_t *wgt, const int32_t *bias,
                 const void *res, int r_signed, int fl_r, void *y)
{
    if (n < 0 || h <= 0 || w <= 0 || ci <= 0 || co <= 0 || kh <= 0 || kw <= 0 || stride <= 0 || pad < 0)
        return F8REF_ERR_ARG;
    const int ho = (h + 2 * pad - kh) / stride + 1;
    const int wo = (w + 2 * pad - kw) / stride + 1;
    if (ho <= 0 || wo <= 0) return F8REF_ERR_ARG;
    int status = F8REF_OK;
#pragma omp parallel for collapse(2) schedule(static)
    for (int in = 0; in < n; ++in)
        for (int oh = 0; oh < ho; ++oh)
            for (int ow = 0; ow < wo; ++ow)
                for (int oc = 0; oc < co; ++oc) {
                    int64_t acc = 0;
                    for (int r = 0; r < kh; ++r)
                        for (int s = 0; s < kw; ++s) {
                            const int ih = oh * stride + r - pad;
                            const int iw = ow * stride + s - pad;
                            if (ih < 0 || ih >= h || iw < 0 || iw >= w) continue;
                            for (int c = 0; c < ci; ++c) {
                                const size_t xi = (((size_t)in * h + ih) * w + iw) * ci + c;
                                const size_t wi = (((size_t)oc * kh + r) * kw + s) * ci + c;
                                acc += load8(x, xi, x_signed) * (int64_t)wgt[wi];
                            }
                        }
                    if (bias) acc += bias[oc];
                    const size_t yi = (((size_t)in * ho + oh) * wo + ow) * co + oc;
                    const int64_t rv = res ? load8(res, yi, r_signed) : 0;
                    const int st = finish(acc, fl_x + fl_w, res != NULL, rv, fl_r, fl_y, y_kind, y, yi);
                    if (st != F8REF_OK) {
#pragma omp atomic write
                        status = st;
                    }
                }
    return status;
}

/*
 * Sibling consumers of one 32-bit value (Sec. 4.3 "Clipping-Level Sharing and Private Fractional Length", Fig. 4;
 * appendix "Private Fractional Lengths Enabling Different Clipping-Levels").  The paper keeps the sum of a layer
 * in 32 bits and quantizes it once per child layer with that child's own fractional length; a shortcut stays in
 * 32 bits until it is added.  For one output element:
 *
 *     acc  = sum_taps x*w + bias                              format FA = FLx + FLw
 *     F    = max(FA, FLr)          v = acc * 2^(F-FA) + r * 2^(F-FLr)        (r: 8-bit code or 32-bit value)
 *     child k (k = 1, 2):  kind 0: clip(round(v * 2^(FLk - F)), 0, 255)      Eq. 2
 *                          kind 1: clip(round(v * 2^(FLk - F)), -127, 127)   signed form
 *                          kind 2: v itself, int32 in format F
 *                          kind 3: max(v, 0), int32 in format F  (the value behind a ReLU, still unrounded:
 *                                  reading -- the paper says such values "are stored in 32-bit" and only
 *                                  "quantized into 8-bit for multiplication"; it does not spell the clip out)
 * Same loop nest as f8ref_conv2d; res_kind 0 u8, 1 s8, 2 int32; y2 may be NULL.
 */
static int finish_child(int64_t v, int f, int kind, int fl, void *y, size_t yi)
{
    if (kind == 2) ((int32_t *)y)[yi] = (int32_t)v;
    else if (kind == 3) ((int32_t *)y)[yi] = (int32_t)(v > 0 ? v : 0);
    else if (kind == 0) ((uint8_t *)y)[yi] = (uint8_t)f8ref_shift_round_clip(v, f - fl, 0, 255);
    else if (kind == 1) ((int8_t *)y)[yi] = (int8_t)f8ref_shift_round_clip(v, f - fl, -127, 127);
    else return F8REF_ERR_ARG;
    return F8REF_OK;
}

int f8ref_conv2d_siblings(int n, int h, int w, int ci, int co, int kh, int kw, int stride, int pad,
                          int x_signed, int fl_x, int fl_w,
                          const void *x, const int8_t *wgt, const int32_t *bias,
                          const void *res, int res_kind, int fl_r,
                          void *y1, int y1_kind, int fl_y1, void *y2, int y2_kind, int fl_y2)
{
    if (n < 0 || h <= 0 || w <= 0 || ci <= 0 || co <= 0 || kh <= 0 || kw <= 0 || stride <= 0 || pad < 0)
        return F8REF_ERR_ARG;
    if (!y1 || (res && (res_kind < 0 || res_kind > 2))) return F8REF_ERR_ARG;
    const int ho = (h + 2 * pad - kh) / stride + 1;
    const int wo = (w + 2 * pad - kw) / stride + 1;
    if (ho <= 0 || wo <= 0) return F8REF_ERR_ARG;
    int status = F8REF_OK;
#pragma omp parallel for collapse(2) schedule(static)
    for (int in = 0; in < n; ++in)
        for (int oh = 0; oh < ho; ++oh)
            for (int ow = 0; ow < wo; ++ow)
                for (int oc = 0; oc < co; ++oc) {
                    int64_t acc = 0;
                    for (int r = 0; r < kh; ++r)
                        for (int s = 0; s < kw; ++s) {
                            const int ih = oh * stride + r - pad;
                            const int iw = ow * stride + s - pad;
                            if (ih < 0 || ih >= h || iw < 0 || iw >= w) continue;
                            for (int c = 0; c < ci; ++c) {
                                const size_t xi = (((size_t)in * h + ih) * w + iw) * ci + c;
                                const size_t wi = (((size_t)oc * kh + r) * kw + s) * ci + c;
                                acc += load8(x, xi, x_signed) * (int64_t)wgt[wi];
                            }
                        }
                    if (bias) acc += bias[oc];
                    const size_t yi = (((size_t)in * ho + oh) * wo + ow) * co + oc;
                    int st = F8REF_OK;
                    int f = fl_x + fl_w;
                    int64_t v = acc;
                    if (acc > INT32_MAX || acc < INT32_MIN) st = F8REF_ERR_ACC_RANGE;
                    if (res) {
                        const int64_t rv = res_kind == 2 ? (int64_t)((const int32_t *)res)[yi] : load8(res, yi, res_kind == 1);
                        f = f > fl_r ? f : fl_r;
                        v = acc * ((int64_t)1 << (f - (fl_x + fl_w))) + rv * ((int64_t)1 << (f - fl_r));
                        if (v > INT32_MAX || v < INT32_MIN) st = F8REF_ERR_ACC_RANGE;
                    }
                    if (st == F8REF_OK) st = finish_child(v, f, y1_kind, fl_y1, y1, yi);
                    if (st == F8REF_OK && y2) st = finish_child(v, f, y2_kind, fl_y2, y2, yi);
                    if (st != F8REF_OK) {
#pragma omp atomic write
                        status = st;
                    }
                }
    return status;
}

/*
 * Depthwise convolution layer: one kh x kw filter per channel (MobileNet's
 * depthwise layers).  wgt : [c, kh, kw] s8.  Everything else as f8ref_conv2d.
 */
int f8ref_dwconv(int n, int h, int w, int c, int kh, int kw, int stride, int pad,
                 int x_signed, int fl_x, int fl_w, int fl_y, int y_kind,
                 const void *x, const int8_t *wgt, const int32_t *bias,
                 const void *res, int r_signed, int fl_r, void *y)
{
    if (n < 0 || h <= 0 || w <= 0 || c <= 0 || kh <= 0 || kw <= 0 || stride <= 0 || pad < 0)
        return F8REF_ERR_ARG;
    const int ho = (h + 2 * pad - kh) / stride + 1;
    const int wo = (w + 2 * pad - kw) / stride + 1;
    if (ho <= 0 || wo <= 0) return F8REF_ERR_ARG;
    int status = F8REF_OK;
#pragma omp parallel for collapse(2) schedule(static)
    for (int in = 0; in < n; ++in)
        for (int oh = 0; oh < ho; ++oh)
            for (int ow = 0; ow < wo; ++ow)
                for (int ch = 0; ch < c; ++ch) {
                    int64_t acc = 0;
                    for (int r = 0; r < kh; ++r)
                        for (int s = 0; s < kw; ++s) {
                            const int ih = oh * stride + r - pad;
                            const int iw = ow * stride + s - pad;
                            if (ih < 0 || ih >= h || iw < 0 || iw >= w) continue;
                            const size_t xi = (((size_t)in * h + ih) * w + iw) * c + ch;
                            const size_t wi = ((size_t)ch * kh + r) * kw + s;
                            acc += load8(x, xi, x_signed) * (int64_t)wgt[wi];
                        }
                    if (bias) acc += bias[ch];
                    const size_t yi = (((size_t)in * ho + oh) * wo + ow) * c + ch;
                    const int64_t rv = res ? load8(res, yi, r_signed) : 0;
                    const int st = finish(acc, fl_x + fl_w, res != NULL, rv, fl_r, fl_y, y_kind, y, yi);
                    if (st != F8REF_OK) {
#pragma omp atomic write
                        status = st;
                    }
                }
    return status;
}

/*
 * Fully connected layer: Eq. 6 with the sum over k inputs.
 *   x : [n, k] 8-bit, wgt : [out, k] s8, bias : [out] int32 (format fl_x+fl_w),
 *   y : [n, out]; y_kind as above (2 = int32 logits in format fl_x + fl_w).
 */
int f8ref_linear(int n, int k, int out, int x_signed, int fl_x, int fl_w, int fl_y, int y_kind,
                 const void *x, const int8_t *wgt, const int32_t *bias, void *y)
{
    if (n < 0 || k <= 0 || out <= 0) return F8REF_ERR_ARG;
    int status = F8REF_OK;
#pragma omp parallel for schedule(static)
    for (int in = 0; in < n; ++in)
        for (int o = 0; o < out; ++o) {
            int64_t acc = 0;
            for (int j = 0; j < k; ++j)
                acc += load8(x, (size_t)in * k + j, x_signed) * (int64_t)wgt[(size_t)o * k + j];
            if (bias) acc += bias[o];
            const int st = finish(acc, fl_x + fl_w, 0, 0, 0, fl_y, y_kind, y, (size_t)in * out + o);
            if (st != F8REF_OK) {
#pragma omp atomic write
                status = st;
            }
        }
    return status;
}

/*
 * Max pooling (not in the paper; reading: integer max over the taps that fall
 * inside the image, format unchanged).  x, y : 8-bit NHWC of the same
 * signedness.
 */
int f8ref_maxpool(int n, int h, int w, int c, int k, int stride, int pad, int x_signed,
                  const void *x, void *y)
{
    if (n < 0 || h <= 0 || w <= 0 || c <= 0 || k <= 0 || stride <= 0 || pad < 0 || pad >= k)
        return F8REF_ERR_ARG;
    const int ho = (h + 2 * pad - k) / stride + 1;
    const int wo = (w + 2 * pad - k) / stride + 1;
    if (ho <= 0 || wo <= 0) return F8REF_ERR_ARG;
#pragma omp parallel for collapse(2) schedule(static)
    for (int in = 0; in < n; ++in)
        for (int oh = 0; oh < ho; ++oh)
            for (int ow = 0; ow < wo; ++ow)
                for (int ch = 0; ch < c; ++ch) {
                    int64_t m = INT64_MIN;
                    for (int r = 0; r < k; ++r)
                        for (int s = 0; s < k; ++s) {
                            const int ih = oh * stride + r - pad;
                            const int iw = ow * stride + s - pad;
                            if (ih < 0 || ih >= h || iw < 0 || iw >= w) continue;
                            const int64_t v = load8(x, (((size_t)in * h + ih) * w + iw) * c + ch, x_signed);
                            if (v > m) m = v;
                        }
                    const size_t yi = (((size_t)in * ho + oh) * wo + ow) * c + ch;
                    if (x_signed) ((int8_t *)y)[yi] = (int8_t)m;
                    else          ((uint8_t *)y)[yi] = (uint8_t)m;
                }
    return F8REF_OK;
}

/*
 * Global average pooling (not in the paper; reading: the division by H*W is
 * replaced by the next power of two 2^d, d = ceil(log2(H*W)), so the layer is
 * a sum followed by the fixed-point quantizer with shift d + fl_x - fl_y; the
 * constant H*W / 2^d belongs to the following layer's effective weight, the
 * way Eq. 6 absorbs scale ratios).
 *   x : [n, h, w, c] 8-bit, y : [n, c] 8-bit of the same signedness.
 */
int f8ref_gap(int n, int h, int w, int c, int x_signed, int fl_x, int fl_y,
              const void *x, void *y)
{
    if (n < 0 || h <= 0 || w <= 0 || c <= 0) return F8REF_ERR_ARG;
    int d = 0;
    while (((int64_t)1 << d) < (int64_t)h * w) ++d;
#pragma omp parallel for schedule(static)
    for (int in = 0; in < n; ++in)
        for (int ch = 0; ch < c; ++ch) {
            int64_t sum = 0;
            for (int ih = 0; ih < h; ++ih)
                for (int iw = 0; iw < w; ++iw)
                    sum += load8(x, (((size_t)in * h + ih) * w + iw) * c + ch, x_signed);
            const size_t yi = (size_t)in * c + ch;
            if (x_signed) ((int8_t *)y)[yi] = (int8_t)f8ref_shift_round_clip(sum, d + fl_x - fl_y, -127, 127);
            else          ((uint8_t *)y)[yi] = (uint8_t)f8ref_shift_round_clip(sum, d + fl_x - fl_y, 0, 255);
        }
    return F8REF_OK;
}
