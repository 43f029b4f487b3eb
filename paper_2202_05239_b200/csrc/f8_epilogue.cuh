// Device-side tail of every layer: residual alignment, rounding shift, clip (Eq. 2 / signed form, Eq. 6).
#pragma once

#include "f8_internal.h"

// Round-half-up arithmetic right shift without forming v + 2^(s-1) (which could overflow):
// floor((v + 2^(s-1)) / 2^s) = (v >> s) + bit (s-1) of v, for 1 <= s <= 31.
__device__ __forceinline__ int f8_rshift_round(int v, int s) {
    return (v >> s) + ((v >> (s - 1)) & 1);
}

// One consumer's view of the aligned 32-bit sum v: the quantizer of Eq. 2 / its signed form with this consumer's
// shift, or the 32-bit value itself (kind F8_S32), or that value behind a ReLU (F8_S32_RELU).
__device__ __forceinline__ int f8_quantize_child(int v, int y_kind, int s, int lo, int hi) {
    if (y_kind == F8_S32) return v;
    if (y_kind == F8_S32_RELU) return max(v, 0);
    int t;
    if (s > 0) {
        t = f8_rshift_round(v, s);
    } else {
        // left shift by at most 8; clamping first keeps the product inside int32 and
        // cannot change the clipped result because |lo|, |hi| <= 255 < 256
        t = min(max(v, -256), 256) << (-s);
    }
    return min(max(t, lo), hi);
}

// acc already holds sum + bias.  r is the residual operand (ignored unless q.has_res): the accumulator and the
// shortcut are brought to the finer of their two formats by shifts and added (Sec. 4.3).
__device__ __forceinline__ int f8_align_add(int acc, int r, const F8Requant &q) {
    return q.has_res ? (acc << q.sh_acc) + (r << q.sh_res) : acc;
}

__device__ __forceinline__ int f8_requant(int acc, int r, const F8Requant &q) {
    return f8_quantize_child(f8_align_add(acc, r, q), q.y_kind, q.s, q.lo, q.hi);
}

__device__ __forceinline__ int f8_load8(const void *p, size_t i, int is_signed) {
    return is_signed ? (int)((const int8_t *)p)[i] : (int)((const uint8_t *)p)[i];
}

// Extract byte j (0..3) of a packed word as a signed / unsigned code.
__device__ __forceinline__ int f8_byte(uint32_t word, int j, int is_signed) {
    const uint32_t b = (word >> (8 * j)) & 0xffu;
    return is_signed ? (int)(int8_t)b : (int)b;
}

__device__ __forceinline__ uint32_t f8_pack4(int a, int b, int c, int d) {
    return (uint32_t)(a & 0xff) | ((uint32_t)(b & 0xff) << 8) | ((uint32_t)(c & 0xff) << 16) |
           ((uint32_t)(d & 0xff) << 24);
}
