// CUDA-core kernels: generic direct convolution (any shape), depthwise convolution, pooling and the
// stem packing pre-pass.  Depthwise and pooling layers are not dense contractions: they are bound by
// HBM traffic, so these kernels are organised around wide, coalesced NHWC accesses.
#include "f8_epilogue.cuh"

namespace {

// Programmatic dependent launch (see the tensor-core kernel): every kernel here first waits for the grids
// before it -- all of its inputs may come from them -- and then lets the grid after it start its prologue.
__device__ __forceinline__ void grid_dependency_sync() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

template <typename... KArgs, typename... Args>
cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, int block, bool overlap_previous, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3((unsigned)block);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap_previous ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}


__device__ __forceinline__ int dp4a_us(uint32_t a, uint32_t b, int c) {   // u8 x s8
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ int dp4a_ss(uint32_t a, uint32_t b, int c) {   // s8 x s8
    int d;
    asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

__device__ __forceinline__ void store_out(void *y, size_t i, int v, int y_kind) {
    if (y_kind == F8_S32 || y_kind == F8_S32_RELU) ((int32_t *)y)[i] = v;
    else ((uint8_t *)y)[i] = (uint8_t)(v & 0xff);
}

// ---------------------------------------------------------------------------------------
// Generic direct convolution: one thread per output element, channel fastest so that a warp
// shares its input window.  Used for shapes the tensor-core path does not take.
// ---------------------------------------------------------------------------------------
template <bool VEC4>
__global__ void __launch_bounds__(256) conv_direct_kernel(F8ConvGeom g, F8Requant q, const uint8_t *__restrict__ x,
                                                          const int8_t *__restrict__ w,
                                                          const int32_t *__restrict__ bias,
                                                          const void *__restrict__ res, void *__restrict__ y,
                                                          F8Sibling sib) {
    grid_dependency_sync();
    const size_t total = (size_t)g.n * g.ho * g.wo * g.c_out;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (size_t)gridDim.x * blockDim.x) {
        const int co = (int)(idx % g.c_out);
        size_t pix = idx / g.c_out;
        const int ow = (int)(pix % g.wo);
        pix /= g.wo;
        const int oh = (int)(pix % g.ho);
        const int in = (int)(pix / g.ho);
        int acc = bias ? bias[co] : 0;
        for (int r = 0; r < g.kh; ++r) {
            const int ih = oh * g.stride_h + r - g.pad_h;
            if (ih < 0 || ih >= g.h) continue;
            for (int s = 0; s < g.kw; ++s) {
                const int iw = ow * g.stride_w + s - g.pad_w;
                if (iw < 0 || iw >= g.w) continue;
                const uint8_t *xp = x + (((size_t)in * g.h + ih) * g.w + iw) * g.c;
                const int8_t *wp = w + (((size_t)co * g.kh + r) * g.kw + s) * g.c;
                if (VEC4) {
                    const uint32_t *x4 = (const uint32_t *)xp;
                    const uint32_t *w4 = (const uint32_t *)wp;
                    const int nc = g.c >> 2;
                    if (g.x_signed) {
                        for (int c = 0; c < nc; ++c) acc = dp4a_ss(x4[c], w4[c], acc);
                    } else {
                        for (int c = 0; c < nc; ++c) acc = dp4a_us(x4[c], w4[c], acc);
                    }
                } else {
                    for (int c = 0; c < g.c; ++c) {
                        const int xv = g.x_signed ? (int)(int8_t)xp[c] : (int)xp[c];
                        acc += xv * (int)wp[c];
                    }
                }
            }
        }
        const int rv = q.has_res ? (q.r_s32 ? ((const int32_t *)res)[idx] : f8_load8(res, idx, q.r_signed)) : 0;
        // one 32-bit sum, one quantisation per consumer (Sec. 4.3)
        const int v = f8_align_add(acc, rv, q);
        store_out(y, idx, f8_quantize_child(v, q.y_kind, q.s, q.lo, q.hi), q.y_kind);
        if (sib.y2) store_out(sib.y2, idx, f8_quantize_child(v, sib.y_kind, sib.s, sib.lo, sib.hi), sib.y_kind);
    }
}

// ---------------------------------------------------------------------------------------
// Depthwise kh x kw convolution.  One thread owns 4 consecutive channels of one output pixel:
// every tap is one 32-bit load that a warp coalesces into a 128-byte row segment.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) dwconv_vec4_kernel(F8ConvGeom g, F8Requant q, const uint8_t *__restrict__ x,
                                                          const int8_t *__restrict__ w,
                                                          const int32_t *__restrict__ bias,
                                                          const void *__restrict__ res, void *__restrict__ y) {
    grid_dependency_sync();
    const int c4 = g.c >> 2;
    const size_t total = (size_t)g.n * g.ho * g.wo * c4;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (size_t)gridDim.x * blockDim.x) {
        const int cg = (int)(idx % c4);
        size_t pix = idx / c4;
        const int ow = (int)(pix % g.wo);
        pix /= g.wo;
        const int oh = (int)(pix % g.ho);
        const int in = (int)(pix / g.ho);
        const int c0 = cg * 4;
        int acc[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[j] = bias ? bias[c0 + j] : 0;
        const int taps = g.kh * g.kw;
        for (int r = 0; r < g.kh; ++r) {
            const int ih = oh * g.stride_h + r - g.pad_h;
            if (ih < 0 || ih >= g.h) continue;
            for (int s = 0; s < g.kw; ++s) {
                const int iw = ow * g.stride_w + s - g.pad_w;
                if (iw < 0 || iw >= g.w) continue;
                const uint32_t xw = *(const uint32_t *)(x + (((size_t)in * g.h + ih) * g.w + iw) * g.c + c0);
                const int t = r * g.kw + s;
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    acc[j] += f8_byte(xw, j, g.x_signed) * (int)w[(size_t)(c0 + j) * taps + t];
            }
        }
        const size_t o = (((size_t)in * g.ho + oh) * g.wo + ow) * g.c + c0;
        uint32_t rw = 0;
        if (q.has_res) rw = *(const uint32_t *)((const uint8_t *)res + o);
        int out[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) out[j] = f8_requant(acc[j], f8_byte(rw, j, q.r_signed), q);
        if (q.y_kind == F8_S32) {
            *(int4 *)((int32_t *)y + o) = make_int4(out[0], out[1], out[2], out[3]);
        } else {
            *(uint32_t *)((uint8_t *)y + o) = f8_pack4(out[0], out[1], out[2], out[3]);
        }
    }
}

// ---------------------------------------------------------------------------------------
// Depthwise 3x3, pad 1, stride S (1 or 2): the layers of MobileNet.  One thread owns 4 consecutive
// channels and a strip of TW output pixels along W.  The nine filter taps of its channels stay in
// registers and every input word (4 channels of one pixel) is loaded and unpacked once per filter row
// and reused by all outputs of the strip that touch it, so the kernel does about one load and four
// unpacks per eight multiply-accumulates instead of one load per multiply-accumulate.  Consecutive
// threads take consecutive channel groups: loads and stores coalesce over the channel dimension.
// Depthwise is not a contraction over channels, so this stays on the CUDA cores (IMAD); it is bound
// by instruction issue, not by HBM.
// ---------------------------------------------------------------------------------------
// Byte j of a word as a sign-extended int with one PRMT: selector nibble j picks the byte, nibble 8|j
// replicates its sign bit (the intrinsic __byte_perm ignores that bit, hence the inline PTX).
__device__ __forceinline__ int prmt_s8(uint32_t word, int j) {
    int r;
    const uint32_t sel = (uint32_t)(j | ((8 | j) << 4) | ((8 | j) << 8) | ((8 | j) << 12));
    asm("prmt.b32 %0, %1, 0, %2;" : "=r"(r) : "r"(word), "r"(sel));
    return r;
}

// FAST: 8-bit output with shift 1..24 -> rounding constant folded into the bias, plain shift, saturating pack.
template <int S, int TW, bool XS, bool FAST>
__global__ void __launch_bounds__(128) dwconv3x3_strip_kernel(F8ConvGeom g, F8Requant q, const uint8_t *__restrict__ x,
                                                              const int8_t *__restrict__ w,
                                                              const int32_t *__restrict__ bias,
                                                              const void *__restrict__ res, void *__restrict__ y,
                                                              int strips, int total) {
    grid_dependency_sync();
    constexpr int SPAN = (TW - 1) * S + 3;          // input pixels a strip touches along W
    const int c4 = g.c >> 2;
    // all index arithmetic in 32 bits (the launcher checks that every offset fits)
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        const int cg = idx % c4;
        int t = idx / c4;
        const int strip = t % strips;
        t /= strips;
        const int oh = t % g.ho;
        const int in = t / g.ho;
        const int c0 = cg * 4;
        const int ow0 = strip * TW;
        int wt[9][4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int k = 0; k < 9; ++k) wt[k][j] = (int)w[(c0 + j) * 9 + k];
        int acc[TW][4];
        int4 b = bias ? *(const int4 *)(bias + c0) : make_int4(0, 0, 0, 0);
        if (FAST) {
            const int rnd = 1 << (q.s - 1);
            b.x = (b.x << q.sh_acc) + rnd; b.y = (b.y << q.sh_acc) + rnd;
            b.z = (b.z << q.sh_acc) + rnd; b.w = (b.w << q.sh_acc) + rnd;
        }
#pragma unroll
        for (int o = 0; o < TW; ++o) { acc[o][0] = 0; acc[o][1] = 0; acc[o][2] = 0; acc[o][3] = 0; }
        const int iw0 = ow0 * S - 1;
#pragma unroll
        for (int r = 0; r < 3; ++r) {
            const int ih = oh * S + r - 1;
            if (ih < 0 || ih >= g.h) continue;
            const uint8_t *row = x + (size_t)((in * g.h + ih) * g.w) * g.c + c0;
            uint32_t words[SPAN];
#pragma unroll
            for (int xx = 0; xx < SPAN; ++xx) {
                const int iw = iw0 + xx;
                words[xx] = (iw >= 0 && iw < g.w) ? __ldg((const uint32_t *)(row + iw * g.c)) : 0u;
            }
#pragma unroll
            for (int xx = 0; xx < SPAN; ++xx) {
                int v[4];
#pragma unroll
                for (int j = 0; j < 4; ++j)   // byte j as an int: one PRMT (selector 8|j replicates the sign bit)
                    v[j] = XS ? prmt_s8(words[xx], j) : (int)__byte_perm(words[xx], 0, 0x4440 | j);
#pragma unroll
                for (int s = 0; s < 3; ++s) {
                    // input column xx feeds output o through tap s when xx = o * S + s
                    if ((xx - s) >= 0 && (xx - s) % S == 0 && (xx - s) / S < TW) {
                        const int o = (xx - s) / S;
#pragma unroll
                        for (int j = 0; j < 4; ++j) acc[o][j] += v[j] * wt[r * 3 + s][j];
                    }
                }
            }
        }
        const int out_row = ((in * g.ho + oh) * g.wo) * g.c + c0;
        const int bb[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int o = 0; o < TW; ++o) {
            const int ow = ow0 + o;
            if (ow >= g.wo) break;
            const int off = out_row + ow * g.c;
            uint32_t rw = 0;
            if (q.has_res) rw = *(const uint32_t *)((const uint8_t *)res + off);
            if (FAST) {
                int tv[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    int v = (acc[o][j] << q.sh_acc) + bb[j];
                    if (q.has_res) v += f8_byte(rw, j, q.r_signed) << q.sh_res;
                    v >>= q.s;
                    tv[j] = q.y_kind == F8_S8 ? max(v, -127) : v;
                }
                uint32_t hi2, word;
                if (q.y_kind == F8_S8) {
                    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, 0;" : "=r"(hi2) : "r"(tv[3]), "r"(tv[2]));
                    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(word) : "r"(tv[1]), "r"(tv[0]), "r"(hi2));
                } else {
                    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, 0;" : "=r"(hi2) : "r"(tv[3]), "r"(tv[2]));
                    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(word) : "r"(tv[1]), "r"(tv[0]), "r"(hi2));
                }
                *(uint32_t *)((uint8_t *)y + off) = word;
            } else {
                int out[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) out[j] = f8_requant(acc[o][j] + bb[j], f8_byte(rw, j, q.r_signed), q);
                if (q.y_kind == F8_S32) *(int4 *)((int32_t *)y + off) = make_int4(out[0], out[1], out[2], out[3]);
                else *(uint32_t *)((uint8_t *)y + off) = f8_pack4(out[0], out[1], out[2], out[3]);
            }
        }
    }
}

// ---------------------------------------------------------------------------------------
// Depthwise 3x3, pad 1, stride 1, walking down the image.  One thread owns 4 consecutive channels, a strip of 2 (or 4)
// output columns and a band of output rows.  It keeps the accumulators of the three output rows that are open (an input row
// feeds the output rows above, at and below it), so every input word is loaded and unpacked ONCE and the filter taps
// are loaded once per band: about 15 instructions per output instead of the 36 of the strip kernel, whose threads
// re-read and re-unpack every input row three times and re-load the taps for every output row.
// ---------------------------------------------------------------------------------------

template <bool XS, int DW_WALK_SPAN>
__device__ __forceinline__ void dw_walk_unpack(const uint32_t (&words)[DW_WALK_SPAN], int (&v)[DW_WALK_SPAN][4]) {
#pragma unroll
    for (int xx = 0; xx < DW_WALK_SPAN; ++xx)
#pragma unroll
        for (int j = 0; j < 4; ++j) v[xx][j] = XS ? prmt_s8(words[xx], j) : (int)__byte_perm(words[xx], 0, 0x4440 | j);
}

// input row `ih` (already unpacked) into the three open output rows: slot (K + 1 - r) mod 3 holds output row ih + 1 - r
template <int K, int DW_WALK_COLS>
__device__ __forceinline__ void dw_walk_accumulate(const int (&v)[DW_WALK_COLS + 2][4], const int (&wt)[9][4],
                                                   int (&acc)[3][DW_WALK_COLS][4]) {
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        constexpr int dummy = 0;
        (void)dummy;
        const int slot = (K + 1 - r + 3) % 3;
#pragma unroll
        for (int o = 0; o < DW_WALK_COLS; ++o)
#pragma unroll
            for (int sx = 0; sx < 3; ++sx)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    // the top tap row opens output row ih + 1: its first product starts the sum
                    if (r == 0 && sx == 0) acc[slot][o][j] = v[o][j] * wt[0][j];
                    else acc[slot][o][j] += v[o + sx][j] * wt[r * 3 + sx][j];
                }
    }
}

// DW_WALK_COLS output columns per thread (4: fewest instructions; 2: half the registers, more warps per SM)
template <bool XS, bool SIGNED_OUT, int DW_WALK_COLS>
__global__ void __launch_bounds__(128) dwconv3x3_walk_kernel(F8ConvGeom g, F8Requant q, const uint8_t *__restrict__ x,
                                                             const int8_t *__restrict__ w,
                                                             const int32_t *__restrict__ bias, uint8_t *__restrict__ y,
                                                             int strips, int bands, int band_rows, int total) {
    grid_dependency_sync();
    constexpr int DW_WALK_SPAN = DW_WALK_COLS + 2;
    const int c4 = g.c >> 2;
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        const int cg = idx % c4;
        int t = idx / c4;
        const int strip = t % strips;
        t /= strips;
        const int band = t % bands;
        const int in = t / bands;
        const int c0 = cg * 4;
        const int ow0 = strip * DW_WALK_COLS;
        const int oh0 = band * band_rows, oh1 = min(g.ho, oh0 + band_rows);
        int wt[9][4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int k = 0; k < 9; ++k) wt[k][j] = (int)w[(c0 + j) * 9 + k];
        int4 b = bias ? *(const int4 *)(bias + c0) : make_int4(0, 0, 0, 0);
        const int rnd = 1 << (q.s - 1);
        const int bb[4] = {b.x + rnd, b.y + rnd, b.z + rnd, b.w + rnd};
        int acc[3][DW_WALK_COLS][4];
#pragma unroll
        for (int a = 0; a < 3; ++a)
#pragma unroll
            for (int o = 0; o < DW_WALK_COLS; ++o)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[a][o][j] = 0;
        // column offsets (bytes) of the six input columns; columns outside the image read as zero
        const int iw0 = ow0 - 1;
        bool col_ok[DW_WALK_SPAN];
#pragma unroll
        for (int xx = 0; xx < DW_WALK_SPAN; ++xx) col_ok[xx] = iw0 + xx >= 0 && iw0 + xx < g.w;
        const int row_stride = g.w * g.c;
        const uint8_t *img = x + (size_t)in * g.h * row_stride + c0 + iw0 * g.c;

        auto load_row = [&](int ih, uint32_t (&words)[DW_WALK_SPAN]) {
            const bool row_ok = ih >= 0 && ih < g.h;
            const uint8_t *rp = img + (size_t)ih * row_stride;
#pragma unroll
            for (int xx = 0; xx < DW_WALK_SPAN; ++xx)
                words[xx] = (row_ok && col_ok[xx]) ? __ldg((const uint32_t *)(rp + xx * g.c)) : 0u;
        };
        // output row `oh` is complete: shift, clip, pack, store (its slot is re-opened by the next top-tap products)
        auto emit = [&](int oh, int (&a)[DW_WALK_COLS][4]) {
            if (oh >= oh0 && oh < oh1) {
                uint8_t *out = y + ((size_t)(in * g.ho + oh) * g.wo + ow0) * g.c + c0;
#pragma unroll
                for (int o = 0; o < DW_WALK_COLS; ++o) {
                    if (ow0 + o < g.wo) {
                        int tv[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const int vv = (a[o][j] + bb[j]) >> q.s;
                            tv[j] = SIGNED_OUT ? max(vv, -127) : vv;
                        }
                        uint32_t hi2, word;
                        if (SIGNED_OUT) {
                            asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, 0;" : "=r"(hi2) : "r"(tv[3]), "r"(tv[2]));
                            asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(word) : "r"(tv[1]), "r"(tv[0]), "r"(hi2));
                        } else {
                            asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, 0;" : "=r"(hi2) : "r"(tv[3]), "r"(tv[2]));
                            asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(word) : "r"(tv[1]), "r"(tv[0]), "r"(hi2));
                        }
                        *(uint32_t *)(out + o * g.c) = word;
                    }
                }
            }
        };

        // input rows oh0 - 1 .. oh1, three per trip so that the slots are compile-time; the next row's words are
        // requested before the current row is used
        uint32_t cur[DW_WALK_SPAN], nxt[DW_WALK_SPAN];
        int ih = oh0 - 1;
        load_row(ih, cur);
        while (ih <= oh1) {
            int v[DW_WALK_SPAN][4];
            // K = 0: input row ih feeds slots 1 (row ih + 1), 0 (row ih), 2 (row ih - 1, now complete)
            load_row(ih + 1, nxt);
            dw_walk_unpack<XS, DW_WALK_SPAN>(cur, v);
            dw_walk_accumulate<0, DW_WALK_COLS>(v, wt, acc);
            emit(ih - 1, acc[2]);
            if (++ih > oh1) break;
            // K = 1: slots 2 (row ih + 1), 1 (row ih), 0 (row ih - 1)
            load_row(ih + 1, cur);
            dw_walk_unpack<XS, DW_WALK_SPAN>(nxt, v);
            dw_walk_accumulate<1, DW_WALK_COLS>(v, wt, acc);
            emit(ih - 1, acc[0]);
            if (++ih > oh1) break;
            // K = 2: slots 0 (row ih + 1), 2 (row ih), 1 (row ih - 1)
            load_row(ih + 1, nxt);
            dw_walk_unpack<XS, DW_WALK_SPAN>(cur, v);
            dw_walk_accumulate<2, DW_WALK_COLS>(v, wt, acc);
            emit(ih - 1, acc[1]);
            if (++ih > oh1) break;
#pragma unroll
            for (int xx = 0; xx < DW_WALK_SPAN; ++xx) cur[xx] = nxt[xx];
        }
    }
}

// ---------------------------------------------------------------------------------------
// Depthwise 3x3, pad 1, stride 1 with packed dot products.  Same walk as above (a thread owns 4 consecutive channels
// and 2 output columns and walks down a band of rows with the three open output rows in registers), but the
// multiply-accumulates run as dp4a: the four words of an input row that a thread needs (columns ow0 - 1 .. ow0 + 2,
// four channels each) are transposed in registers into one word per channel holding that channel's four columns
// (8 PRMT), and a filter row of a channel is kept as one packed word [w0 w1 w2 0], applied to that word for the left
// output column and to the word shifted down by one column for the right one, so that one dp4a does the three products of
// a filter row.  Per input row and thread: 4 copies, 8 permutes, 4 shifts and 24 dp4a for 72 multiply-accumulates, against
// 72 multiply-adds and 16 unpacks before.
// ---------------------------------------------------------------------------------------
template <bool XS>
__device__ __forceinline__ int dw_dot4(uint32_t x, uint32_t w, int acc) {
    return XS ? dp4a_ss(x, w, acc) : dp4a_us(x, w, acc);
}

// input row (transposed: t[j] = the four columns of channel j) into the three open output rows; slot (K + 1 - r) mod 3
// holds output row ih + 1 - r.  The top filter row opens an output row: its product starts the sum.
template <int K, bool XS>
__device__ __forceinline__ void dw_dp4a_accumulate(const uint32_t (&t)[4], const uint32_t (&wa)[3][4], const int (&open)[4],
                                                   int (&acc)[3][2][4]) {
    // the right output column reads columns 1..3: the same packed filter row against the word shifted down by one column
    uint32_t tr[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) tr[j] = t[j] >> 8;
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        const int slot = (K + 1 - r + 3) % 3;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            // open[j] = bias + rounding constant: the value an output row's sum starts from
            acc[slot][0][j] = dw_dot4<XS>(t[j], wa[r][j], r == 0 ? open[j] : acc[slot][0][j]);
            acc[slot][1][j] = dw_dot4<XS>(tr[j], wa[r][j], r == 0 ? open[j] : acc[slot][1][j]);
        }
    }
}

// Input rows reach the thread through a private ring in shared memory filled by asynchronous copies issued DW_AHEAD rows
// ahead (no registers are tied up by loads in flight, so every thread keeps 4 * DW_AHEAD words on their way: with
// loads into registers, one row ahead, the kernel was bound by memory latency at a quarter of the HBM bandwidth).
constexpr int DW_AHEAD = 8;

__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

// four saturated bytes (channels 0..3 of one output pixel) from four sums that still carry the rounding constant
template <bool SIGNED_OUT>
__device__ __forceinline__ uint32_t dw_pack4(const int (&a)[4], int s) {
    int tv[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int vv = a[j] >> s;
        tv[j] = SIGNED_OUT ? max(vv, -127) : vv;
    }
    uint32_t hi2, word;
    if (SIGNED_OUT) {
        asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, 0;" : "=r"(hi2) : "r"(tv[3]), "r"(tv[2]));
        asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(word) : "r"(tv[1]), "r"(tv[0]), "r"(hi2));
    } else {
        asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, 0;" : "=r"(hi2) : "r"(tv[3]), "r"(tv[2]));
        asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(word) : "r"(tv[1]), "r"(tv[0]), "r"(hi2));
    }
    return word;
}

// Addresses are 32-bit offsets that advance by a row per step (tensors on this path are below 2 GiB): with the offsets
// recomputed from the row index for every copy and every store, address arithmetic was more than a third of the
// instructions of a kernel that is bound by instruction issue.
template <bool XS, bool SIGNED_OUT>
__global__ void __launch_bounds__(128) dwconv3x3_dp4a_kernel(F8ConvGeom g, F8Requant q, const uint8_t *__restrict__ x,
                                                             const int8_t *__restrict__ w,
                                                             const int32_t *__restrict__ bias, uint8_t *__restrict__ y,
                                                             int strips, int bands, int band_rows, int total) {
    grid_dependency_sync();
    __shared__ uint32_t ring[DW_AHEAD][4][128];          // [row slot][column][thread]: a thread only touches its own words
    constexpr uint32_t SLOT_BYTES = 4 * 128 * 4, RING_BYTES = DW_AHEAD * SLOT_BYTES;
    const uint32_t ring_base = (uint32_t)__cvta_generic_to_shared(&ring[0][0][threadIdx.x]);
    const int c4 = g.c >> 2;
    const uint32_t row_stride = (uint32_t)(g.w * g.c), out_stride = (uint32_t)(g.wo * g.c);
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        const int cg = idx % c4;
        int tt = idx / c4;
        const int strip = tt % strips;
        tt /= strips;
        const int band = tt % bands;
        const int in = tt / bands;
        const int c0 = cg * 4;
        const int ow0 = strip * 2;
        const int oh0 = band * band_rows, oh1 = min(g.ho, oh0 + band_rows);
        // filter rows as packed words: bytes (w0, w1, w2, 0)
        uint32_t wa[3][4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int r = 0; r < 3; ++r) {
                const uint32_t b0 = (uint8_t)w[(c0 + j) * 9 + 3 * r], b1 = (uint8_t)w[(c0 + j) * 9 + 3 * r + 1],
                               b2 = (uint8_t)w[(c0 + j) * 9 + 3 * r + 2];
                wa[r][j] = b0 | (b1 << 8) | (b2 << 16);
            }
        int4 b = bias ? *(const int4 *)(bias + c0) : make_int4(0, 0, 0, 0);
        const int rnd = 1 << (q.s - 1);
        const int bb[4] = {b.x + rnd, b.y + rnd, b.z + rnd, b.w + rnd};
        int acc[3][2][4];
#pragma unroll
        for (int a = 0; a < 3; ++a)
#pragma unroll
            for (int o = 0; o < 2; ++o)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[a][o][j] = bb[j];
        const int iw0 = ow0 - 1;
        uint32_t col_off[4];                // byte offset of the column inside a row (0 for columns outside the image)
        int col_bytes[4];                   // 4, or 0 for a column outside the image (the copy then writes zeros)
#pragma unroll
        for (int xx = 0; xx < 4; ++xx) {
            const bool ok = (unsigned)(iw0 + xx) < (unsigned)g.w;
            col_off[xx] = ok ? (uint32_t)(iw0 + xx) * (uint32_t)g.c : 0u;
            col_bytes[xx] = ok ? 4 : 0;
        }
        const uint32_t img_off = (uint32_t)in * (uint32_t)g.h * row_stride + (uint32_t)c0;
        const bool right_ok = ow0 + 1 < g.wo;

        // input rows oh0 - 1 .. oh1 are requested in order, DW_AHEAD rows ahead of their use (rows outside the image and
        // requests past the band are zero fills that keep the group count regular)
        int req_ih = oh0 - 1;
        uint32_t req_off = img_off + (uint32_t)req_ih * row_stride;       // (wraps for row -1: used only for rows inside)
        uint32_t req_slot = 0;                                            // byte offset of the ring slot
        auto request_next = [&]() {
            const bool row_ok = (unsigned)req_ih < (unsigned)g.h && req_ih <= oh1;
            const uint32_t off = row_ok ? req_off : img_off;
#pragma unroll
            for (int xx = 0; xx < 4; ++xx) {
                const int bytes = row_ok ? col_bytes[xx] : 0;
                asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(ring_base + req_slot + (uint32_t)xx * 512u),
                             "l"(x + (off + col_off[xx])), "r"(bytes)
                             : "memory");
            }
            cp_async_commit();
            ++req_ih;
            req_off += row_stride;
            req_slot = (req_slot + SLOT_BYTES) & (RING_BYTES - 1);
        };
        // the four words of the oldest requested row, transposed: words of four channels per column -> words of four
        // columns per channel
        uint32_t take_slot = 0;
        auto take_row = [&](uint32_t (&t)[4]) {
            cp_async_wait<DW_AHEAD - 1>();
            uint32_t cw[4];
#pragma unroll
            for (int xx = 0; xx < 4; ++xx) cw[xx] = lds32(ring_base + take_slot + (uint32_t)xx * 512u);
            take_slot = (take_slot + SLOT_BYTES) & (RING_BYTES - 1);
            const uint32_t lo01 = __byte_perm(cw[0], cw[1], 0x5140), hi01 = __byte_perm(cw[0], cw[1], 0x7362);
            const uint32_t lo23 = __byte_perm(cw[2], cw[3], 0x5140), hi23 = __byte_perm(cw[2], cw[3], 0x7362);
            t[0] = __byte_perm(lo01, lo23, 0x5410);
            t[1] = __byte_perm(lo01, lo23, 0x7632);
            t[2] = __byte_perm(hi01, hi23, 0x5410);
            t[3] = __byte_perm(hi01, hi23, 0x7632);
        };
        // output rows leave in order, starting two rows above the band (those two belong to the band above)
        int emit_left = -2;                                               // rows until the first one of this band
        uint32_t out_off = ((uint32_t)(in * g.ho + oh0) * (uint32_t)g.wo + (uint32_t)ow0) * (uint32_t)g.c + (uint32_t)c0;
        auto emit = [&](int (&a)[2][4]) {
            if (emit_left >= 0) {
                *(uint32_t *)(y + out_off) = dw_pack4<SIGNED_OUT>(a[0], q.s);
                if (right_ok) *(uint32_t *)(y + out_off + (uint32_t)g.c) = dw_pack4<SIGNED_OUT>(a[1], q.s);
                out_off += out_stride;
            }
            ++emit_left;
        };

        static_assert((RING_BYTES & (RING_BYTES - 1)) == 0, "ring size must be a power of two");
#pragma unroll
        for (int d = 0; d < DW_AHEAD; ++d) request_next();
        int ih = oh0 - 1;
        uint32_t t[4];
        // three rows per trip so that the accumulator slots are compile-time; output row ih - 1 closes with input row ih
        while (ih <= oh1) {
            take_row(t);
            request_next();
            dw_dp4a_accumulate<0, XS>(t, wa, bb, acc);
            emit(acc[2]);
            if (++ih > oh1) break;
            take_row(t);
            request_next();
            dw_dp4a_accumulate<1, XS>(t, wa, bb, acc);
            emit(acc[0]);
            if (++ih > oh1) break;
            take_row(t);
            request_next();
            dw_dp4a_accumulate<2, XS>(t, wa, bb, acc);
            emit(acc[1]);
            ++ih;
        }
        cp_async_wait<0>();          // nothing of this item is in flight when the ring is reused for the next one
    }
}

// The same for stride 2.  A thread owns 4 channels and 2 output columns, i.e. the five input columns 2 ow0 - 1 .. 2 ow0 + 3:
// columns 0..2 feed the left output, columns 2..4 the right one, so a filter row is one packed word (w0 w1 w2 0) for both
// and the transposition yields two words per channel (12 PRMT).  Output row oh takes input rows 2 oh - 1, 2 oh and 2 oh + 1;
// an odd input row closes one output row and opens the next, so a single set of accumulators walks down the band.
template <bool XS, bool SIGNED_OUT>
__global__ void __launch_bounds__(128) dwconv3x3s2_dp4a_kernel(F8ConvGeom g, F8Requant q, const uint8_t *__restrict__ x,
                                                               const int8_t *__restrict__ w,
                                                               const int32_t *__restrict__ bias, uint8_t *__restrict__ y,
                                                               int strips, int bands, int band_rows, int total) {
    grid_dependency_sync();
    __shared__ uint32_t ring[DW_AHEAD][5][128];
    constexpr uint32_t SLOT_BYTES = 5 * 128 * 4;
    const uint32_t ring_base = (uint32_t)__cvta_generic_to_shared(&ring[0][0][threadIdx.x]);
    const int c4 = g.c >> 2;
    const uint32_t row_stride = (uint32_t)(g.w * g.c), out_stride = (uint32_t)(g.wo * g.c);
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        const int cg = idx % c4;
        int tt = idx / c4;
        const int strip = tt % strips;
        tt /= strips;
        const int band = tt % bands;
        const int in = tt / bands;
        const int c0 = cg * 4;
        const int ow0 = strip * 2;
        const int oh0 = band * band_rows, oh1 = min(g.ho, oh0 + band_rows);
        uint32_t wr[3][4];                  // filter row r of channel j: bytes (w0, w1, w2, 0)
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int r = 0; r < 3; ++r) {
                const uint32_t b0 = (uint8_t)w[(c0 + j) * 9 + 3 * r], b1 = (uint8_t)w[(c0 + j) * 9 + 3 * r + 1],
                               b2 = (uint8_t)w[(c0 + j) * 9 + 3 * r + 2];
                wr[r][j] = b0 | (b1 << 8) | (b2 << 16);
            }
        int4 b = bias ? *(const int4 *)(bias + c0) : make_int4(0, 0, 0, 0);
        const int rnd = 1 << (q.s - 1);
        const int bb[4] = {b.x + rnd, b.y + rnd, b.z + rnd, b.w + rnd};
        const int iw0 = 2 * ow0 - 1;
        uint32_t col_off[5];
        int col_bytes[5];
#pragma unroll
        for (int xx = 0; xx < 5; ++xx) {
            const bool ok = (unsigned)(iw0 + xx) < (unsigned)g.w;
            col_off[xx] = ok ? (uint32_t)(iw0 + xx) * (uint32_t)g.c : 0u;
            col_bytes[xx] = ok ? 4 : 0;
        }
        const uint32_t img_off = (uint32_t)in * (uint32_t)g.h * row_stride + (uint32_t)c0;
        const int last_row = 2 * (oh1 - 1) + 1;            // last input row of the band
        const bool right_ok = ow0 + 1 < g.wo;

        // input rows 2 oh0 - 1 .. last_row, requested in order DW_AHEAD rows ahead of their use (32-bit offsets that advance
        // by a row per request; rows outside the image or past the band are zero fills)
        int req_ih = 2 * oh0 - 1;
        uint32_t req_off = img_off + (uint32_t)req_ih * row_stride;
        int req_slot = 0;
        auto request_next = [&]() {
            const bool row_ok = (unsigned)req_ih < (unsigned)g.h && req_ih <= last_row;
            const uint32_t off = row_ok ? req_off : img_off;
            const uint32_t dst = ring_base + (uint32_t)req_slot * SLOT_BYTES;
#pragma unroll
            for (int xx = 0; xx < 5; ++xx) {
                const int bytes = row_ok ? col_bytes[xx] : 0;
                asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst + (uint32_t)xx * 512u),
                             "l"(x + (off + col_off[xx])), "r"(bytes)
                             : "memory");
            }
            cp_async_commit();
            ++req_ih;
            req_off += row_stride;
            req_slot = (req_slot + 1) & (DW_AHEAD - 1);
        };
        // ta[j]: columns 0..3 of channel j (the left output reads bytes 0..2); tb[j]: columns 2, 3, 4 (the right output)
        int take_slot = 0;
        auto take_row = [&](uint32_t (&ta)[4], uint32_t (&tb)[4]) {
            cp_async_wait<DW_AHEAD - 1>();
            const uint32_t src = ring_base + (uint32_t)take_slot * SLOT_BYTES;
            take_slot = (take_slot + 1) & (DW_AHEAD - 1);
            uint32_t cw[5];
#pragma unroll
            for (int xx = 0; xx < 5; ++xx) cw[xx] = lds32(src + (uint32_t)xx * 512u);
            const uint32_t lo01 = __byte_perm(cw[0], cw[1], 0x5140), hi01 = __byte_perm(cw[0], cw[1], 0x7362);
            const uint32_t lo23 = __byte_perm(cw[2], cw[3], 0x5140), hi23 = __byte_perm(cw[2], cw[3], 0x7362);
            ta[0] = __byte_perm(lo01, lo23, 0x5410);
            ta[1] = __byte_perm(lo01, lo23, 0x7632);
            ta[2] = __byte_perm(hi01, hi23, 0x5410);
            ta[3] = __byte_perm(hi01, hi23, 0x7632);
            tb[0] = __byte_perm(lo23, cw[4], 0x4410);
            tb[1] = __byte_perm(lo23, cw[4], 0x5532);
            tb[2] = __byte_perm(hi23, cw[4], 0x6610);
            tb[3] = __byte_perm(hi23, cw[4], 0x7732);
        };
        uint32_t out_off = ((uint32_t)(in * g.ho + oh0) * (uint32_t)g.wo + (uint32_t)ow0) * (uint32_t)g.c + (uint32_t)c0;
        auto emit = [&](const int (&a)[2][4]) {
            *(uint32_t *)(y + out_off) = dw_pack4<SIGNED_OUT>(a[0], q.s);
            if (right_ok) *(uint32_t *)(y + out_off + (uint32_t)g.c) = dw_pack4<SIGNED_OUT>(a[1], q.s);
            out_off += out_stride;
        };

#pragma unroll
        for (int d = 0; d < DW_AHEAD; ++d) request_next();
        int acc[2][4];
        uint32_t ta[4], tb[4];
        // the row above the band opens the first output row
        take_row(ta, tb);
        request_next();
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            acc[0][j] = dw_dot4<XS>(ta[j], wr[0][j], bb[j]);
            acc[1][j] = dw_dot4<XS>(tb[j], wr[0][j], bb[j]);
        }
        for (int oh = oh0; oh < oh1; ++oh) {
            take_row(ta, tb);                               // the middle filter row
            request_next();
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                acc[0][j] = dw_dot4<XS>(ta[j], wr[1][j], acc[0][j]);
                acc[1][j] = dw_dot4<XS>(tb[j], wr[1][j], acc[1][j]);
            }
            take_row(ta, tb);                               // the bottom filter row of this output row, the top one of the next
            request_next();
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                acc[0][j] = dw_dot4<XS>(ta[j], wr[2][j], acc[0][j]);
                acc[1][j] = dw_dot4<XS>(tb[j], wr[2][j], acc[1][j]);
            }
            emit(acc);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                acc[0][j] = dw_dot4<XS>(ta[j], wr[0][j], bb[j]);
                acc[1][j] = dw_dot4<XS>(tb[j], wr[0][j], bb[j]);
            }
        }
        cp_async_wait<0>();
    }
}

__global__ void __launch_bounds__(256) dwconv_scalar_kernel(F8ConvGeom g, F8Requant q, const uint8_t *__restrict__ x,
                                                            const int8_t *__restrict__ w,
                                                            const int32_t *__restrict__ bias,
                                                            const void *__restrict__ res, void *__restrict__ y) {
    grid_dependency_sync();
    const size_t total = (size_t)g.n * g.ho * g.wo * g.c;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (size_t)gridDim.x * blockDim.x) {
        const int ch = (int)(idx % g.c);
        size_t pix = idx / g.c;
        const int ow = (int)(pix % g.wo);
        pix /= g.wo;
        const int oh = (int)(pix % g.ho);
        const int in = (int)(pix / g.ho);
        int acc = bias ? bias[ch] : 0;
        for (int r = 0; r < g.kh; ++r) {
            const int ih = oh * g.stride_h + r - g.pad_h;
            if (ih < 0 || ih >= g.h) continue;
            for (int s = 0; s < g.kw; ++s) {
                const int iw = ow * g.stride_w + s - g.pad_w;
                if (iw < 0 || iw >= g.w) continue;
                acc += f8_load8(x, (((size_t)in * g.h + ih) * g.w + iw) * g.c + ch, g.x_signed) *
                       (int)w[((size_t)ch * g.kh + r) * g.kw + s];
            }
        }
        const int rv = q.has_res ? f8_load8(res, idx, q.r_signed) : 0;
        store_out(y, idx, f8_requant(acc, rv, q), q.y_kind);
    }
}

// ---------------------------------------------------------------------------------------
// Max pooling: one thread per (output pixel, VEC channels); taps outside the image are skipped.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t max4(uint32_t a, uint32_t b, int is_signed) {
    return is_signed ? __vmaxs4(a, b) : __vmaxu4(a, b);
}

template <int WORDS>   // WORDS 32-bit words (4 channels each) per thread: 4 -> 16-byte accesses
__global__ void __launch_bounds__(256) maxpool_kernel(int n, int h, int w, int c, int ho, int wo, int k, int stride,
                                                      int pad, int x_signed, const uint8_t *__restrict__ x,
                                                      uint8_t *__restrict__ y) {
    grid_dependency_sync();
    const int cg = c / (4 * WORDS);
    const size_t total = (size_t)n * ho * wo * cg;
    const uint32_t identity = x_signed ? 0x80808080u : 0u;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (size_t)gridDim.x * blockDim.x) {
        const int g = (int)(idx % cg);
        size_t pix = idx / cg;
        const int ow = (int)(pix % wo);
        pix /= wo;
        const int oh = (int)(pix % ho);
        const int in = (int)(pix / ho);
        uint32_t m[WORDS];
#pragma unroll
        for (int j = 0; j < WORDS; ++j) m[j] = identity;
        for (int r = 0; r < k; ++r) {
            const int ih = oh * stride + r - pad;
            if (ih < 0 || ih >= h) continue;
            for (int s = 0; s < k; ++s) {
                const int iw = ow * stride + s - pad;
                if (iw < 0 || iw >= w) continue;
                const uint32_t *p = (const uint32_t *)(x + (((size_t)in * h + ih) * w + iw) * c) + g * WORDS;
                if (WORDS == 4) {
                    const uint4 v = *(const uint4 *)p;
                    m[0] = max4(m[0], v.x, x_signed);
                    m[1 % WORDS] = max4(m[1 % WORDS], v.y, x_signed);
                    m[2 % WORDS] = max4(m[2 % WORDS], v.z, x_signed);
                    m[3 % WORDS] = max4(m[3 % WORDS], v.w, x_signed);
                } else {
#pragma unroll
                    for (int j = 0; j < WORDS; ++j) m[j] = max4(m[j], p[j], x_signed);
                }
            }
        }
        uint32_t *o = (uint32_t *)(y + (((size_t)in * ho + oh) * wo + ow) * c) + g * WORDS;
        if (WORDS == 4) *(uint4 *)o = make_uint4(m[0], m[1 % WORDS], m[2 % WORDS], m[3 % WORDS]);
        else {
#pragma unroll
            for (int j = 0; j < WORDS; ++j) o[j] = m[j];
        }
    }
}

// 3x3 / stride 2 / pad 1 max-pool, c % 16 == 0: a thread owns 16 channels of a block of 2 x 4 outputs.  It walks the
// five input rows of the block once; per row it loads the nine columns once, takes the horizontal maxima of the four
// windows and folds them into the one or two output rows the input row belongs to (5.6 loads per output instead
// of 9).  Out-of-range taps contribute the identity of max (padding never wins).
template <bool SIGNED>
__global__ void __launch_bounds__(128) maxpool3x3s2_kernel(int n, int h, int w, int c, int ho, int wo,
                                                           const uint8_t *__restrict__ x, uint8_t *__restrict__ y) {
    grid_dependency_sync();
    constexpr int TH = 2, TW = 4;
    const int cg = c / 16;
    const int wb = (wo + TW - 1) / TW, hb = (ho + TH - 1) / TH;
    const size_t total = (size_t)n * hb * wb * cg;
    const uint32_t ident = SIGNED ? 0x80808080u : 0u;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (size_t)gridDim.x * blockDim.x) {
        const int g = (int)(idx % cg);
        size_t t = idx / cg;
        const int bw = (int)(t % wb);
        t /= wb;
        const int bh = (int)(t % hb);
        const int img = (int)(t / hb);
        const int oh0 = bh * TH, ow0 = bw * TW;
        uint4 acc[TH][TW];
#pragma unroll
        for (int a = 0; a < TH; ++a)
#pragma unroll
            for (int b = 0; b < TW; ++b) acc[a][b] = make_uint4(ident, ident, ident, ident);
#pragma unroll
        for (int r = 0; r < 2 * TH + 1; ++r) {
            const int ih = 2 * oh0 - 1 + r;
            if (ih < 0 || ih >= h) continue;
            const uint8_t *row = x + (((size_t)img * h + ih) * w) * c + g * 16;
            uint4 v[2 * TW + 1];
#pragma unroll
            for (int j = 0; j < 2 * TW + 1; ++j) {
                const int iw = 2 * ow0 - 1 + j;
                v[j] = (iw >= 0 && iw < w) ? *(const uint4 *)(row + (size_t)iw * c) : make_uint4(ident, ident, ident, ident);
            }
#pragma unroll
            for (int b = 0; b < TW; ++b) {
                uint4 m;
                if (SIGNED) {
                    m.x = __vmaxs4(__vmaxs4(v[2 * b].x, v[2 * b + 1].x), v[2 * b + 2].x);
                    m.y = __vmaxs4(__vmaxs4(v[2 * b].y, v[2 * b + 1].y), v[2 * b + 2].y);
                    m.z = __vmaxs4(__vmaxs4(v[2 * b].z, v[2 * b + 1].z), v[2 * b + 2].z);
                    m.w = __vmaxs4(__vmaxs4(v[2 * b].w, v[2 * b + 1].w), v[2 * b + 2].w);
                } else {
                    m.x = __vmaxu4(__vmaxu4(v[2 * b].x, v[2 * b + 1].x), v[2 * b + 2].x);
                    m.y = __vmaxu4(__vmaxu4(v[2 * b].y, v[2 * b + 1].y), v[2 * b + 2].y);
                    m.z = __vmaxu4(__vmaxu4(v[2 * b].z, v[2 * b + 1].z), v[2 * b + 2].z);
                    m.w = __vmaxu4(__vmaxu4(v[2 * b].w, v[2 * b + 1].w), v[2 * b + 2].w);
                }
                // input row r of the block feeds output row a when r is one of 2a, 2a+1, 2a+2
#pragma unroll
                for (int a = 0; a < TH; ++a)
                    if (r >= 2 * a && r <= 2 * a + 2) {
                        acc[a][b].x = SIGNED ? __vmaxs4(acc[a][b].x, m.x) : __vmaxu4(acc[a][b].x, m.x);
                        acc[a][b].y = SIGNED ? __vmaxs4(acc[a][b].y, m.y) : __vmaxu4(acc[a][b].y, m.y);
                        acc[a][b].z = SIGNED ? __vmaxs4(acc[a][b].z, m.z) : __vmaxu4(acc[a][b].z, m.z);
                        acc[a][b].w = SIGNED ? __vmaxs4(acc[a][b].w, m.w) : __vmaxu4(acc[a][b].w, m.w);
                    }
            }
        }
#pragma unroll
        for (int a = 0; a < TH; ++a)
#pragma unroll
            for (int b = 0; b < TW; ++b)
                if (oh0 + a < ho && ow0 + b < wo)
                    *(uint4 *)(y + ((((size_t)img * ho + oh0 + a) * wo + ow0 + b) * c) + g * 16) = acc[a][b];
    }
}

__global__ void __launch_bounds__(256) maxpool_scalar_kernel(int n, int h, int w, int c, int ho, int wo, int k,
                                                             int stride, int pad, int x_signed,
                                                             const uint8_t *__restrict__ x, uint8_t *__restrict__ y) {
    grid_dependency_sync();
    const size_t total = (size_t)n * ho * wo * c;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (size_t)gridDim.x * blockDim.x) {
        const int ch = (int)(idx % c);
        size_t pix = idx / c;
        const int ow = (int)(pix % wo);
        pix /= wo;
        const int oh = (int)(pix % ho);
        const int in = (int)(pix / ho);
        int m = -1000;
        for (int r = 0; r < k; ++r) {
            const int ih = oh * stride + r - pad;
            if (ih < 0 || ih >= h) continue;
            for (int s = 0; s < k; ++s) {
                const int iw = ow * stride + s - pad;
                if (iw < 0 || iw >= w) continue;
                m = max(m, f8_load8(x, (((size_t)in * h + ih) * w + iw) * c + ch, x_signed));
            }
        }
        y[idx] = (uint8_t)(m & 0xff);
    }
}

// ---------------------------------------------------------------------------------------
// Global average pooling: sum over h*w, rounding shift, clip.  A block handles one image and a
// slab of channels; threads run over channels so that every row read is coalesced.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) gap_kernel(int hw, int c, int x_signed, int s, const uint8_t *__restrict__ x,
                                                  uint8_t *__restrict__ y) {
    grid_dependency_sync();
    const int in = blockIdx.y;
    const int ch = blockIdx.x * blockDim.x + threadIdx.x;
    if (ch >= c) return;
    const uint8_t *p = x + (size_t)in * hw * c + ch;
    int sum = 0;
    for (int i = 0; i < hw; ++i) {
        const uint8_t b = p[(size_t)i * c];
        sum += x_signed ? (int)(int8_t)b : (int)b;
    }
    F8Requant q;
    q.sh_acc = q.sh_res = 0;
    q.s = s;
    q.lo = x_signed ? -127 : 0;
    q.hi = x_signed ? 127 : 255;
    q.y_kind = x_signed ? F8_S8 : F8_U8;
    q.has_res = 0;
    q.r_signed = 0;
    y[(size_t)in * c + ch] = (uint8_t)(f8_requant(sum, 0, q) & 0xff);
}

// The same with four channels per thread: 4-byte loads, and the four sums kept in two registers of two 16-bit lanes each
// (channels 0 / 2 and 1 / 3), which cannot overflow while hw * 255 < 65536.  Signed inputs are made unsigned by flipping
// the top bit of every byte (x + 128); the 128 * hw this adds to every sum is taken off at the end.
__global__ void __launch_bounds__(256) gap4_kernel(int hw, int c, int x_signed, int s, const uint8_t *__restrict__ x,
                                                   uint8_t *__restrict__ y) {
    grid_dependency_sync();
    const int in = blockIdx.y;
    const int c4 = blockIdx.x * blockDim.x + threadIdx.x;
    const int stride = c >> 2;
    if (c4 >= stride) return;
    const uint32_t *p = (const uint32_t *)(x + (size_t)in * hw * c) + c4;
    const uint32_t flip = x_signed ? 0x80808080u : 0u;
    uint32_t even = 0, odd = 0;
#pragma unroll 7
    for (int i = 0; i < hw; ++i) {
        const uint32_t w = __ldg(p + (size_t)i * stride) ^ flip;
        even += w & 0x00ff00ffu;
        odd += (w >> 8) & 0x00ff00ffu;
    }
    const int off = x_signed ? 128 * hw : 0;
    const int sum[4] = {(int)(even & 0xffffu) - off, (int)(odd & 0xffffu) - off, (int)(even >> 16) - off, (int)(odd >> 16) - off};
    F8Requant q;
    q.sh_acc = q.sh_res = 0;
    q.s = s;
    q.lo = x_signed ? -127 : 0;
    q.hi = x_signed ? 127 : 255;
    q.y_kind = x_signed ? F8_S8 : F8_U8;
    q.has_res = 0;
    q.r_signed = 0;
    uint32_t word = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) word |= (uint32_t)(f8_requant(sum[j], 0, q) & 0xff) << (8 * j);
    *(uint32_t *)(y + (size_t)in * c + 4 * c4) = word;
}

// ---------------------------------------------------------------------------------------
// Stem packing: [n,h,w,c<=8] -> [n,h,wp,8], pixel iw lands at column iw + left; all other bytes 0.
// One thread writes one 8-byte output pixel.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) pack_stem_kernel(int n, int h, int w, int c, int wp, int left,
                                                        const uint8_t *__restrict__ x, uint2 *__restrict__ y) {
    grid_dependency_sync();
    const size_t total = (size_t)n * h * wp;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (size_t)gridDim.x * blockDim.x) {
        const int col = (int)(idx % wp);
        const size_t row = idx / wp;           // n*h + ih
        const int iw = col - left;
        uint32_t lo = 0, hi = 0;
        if (iw >= 0 && iw < w) {
            const uint8_t *p = x + (row * w + iw) * c;
            for (int j = 0; j < c; ++j) {
                const uint32_t b = p[j];
                if (j < 4) lo |= b << (8 * j);
                else hi |= b << (8 * (j - 4));
            }
        }
        y[idx] = make_uint2(lo, hi);
    }
}

// ---------------------------------------------------------------------------------------
// Row-pair stem packing: [n,h,w,c] -> [n,hp,wp] cells of 2*CPAD bytes (CPAD = 4 for c <= 4, else 8); the cell
// at column iw + left of pair p holds pixel iw of image row 2p (first CPAD bytes) and of row 2p+1 (last CPAD
// bytes), channels first, zero filled.  One thread per cell.
// ---------------------------------------------------------------------------------------
template <int CPAD>
__global__ void __launch_bounds__(256) pack_stem_pairs_kernel(int n, int h, int w, int c, int hp, int wp, int left,
                                                              const uint8_t *__restrict__ x, uint32_t *__restrict__ y) {
    grid_dependency_sync();
    constexpr int WORDS = CPAD / 4;            // 32-bit words per pixel
    const size_t total = (size_t)n * hp * wp;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (size_t)gridDim.x * blockDim.x) {
        const int col = (int)(idx % wp);
        const size_t np = idx / wp;            // n*hp + pair
        const int pair = (int)(np % hp);
        const size_t img = np / hp;
        const int iw = col - left;
        uint32_t word[2 * WORDS];
#pragma unroll
        for (int i = 0; i < 2 * WORDS; ++i) word[i] = 0;
        if (iw >= 0 && iw < w) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int ih = 2 * pair + e;
                if (ih < h) {
                    const uint8_t *px = x + ((img * h + ih) * w + iw) * c;
#pragma unroll
                    for (int j = 0; j < CPAD; ++j)
                        if (j < c) word[WORDS * e + (j >> 2)] |= (uint32_t)px[j] << (8 * (j & 3));
                }
            }
        }
        if (WORDS == 1) ((uint2 *)y)[idx] = make_uint2(word[0], word[1]);
        else ((uint4 *)y)[idx] = make_uint4(word[0], word[1], word[2 * WORDS - 2], word[2 * WORDS - 1]);
    }
}

inline int grid_for(size_t total, int block) {
    size_t blocks = (total + block - 1) / block;
    const size_t cap = 148 * 16;   // a few waves of a grid-stride loop on 148 SMs
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

}   // namespace

cudaError_t f8_launch_conv_direct(const F8ConvGeom &g, const F8Requant &q, const void *x, const int8_t *w,
                                  const int32_t *bias, const void *res, void *y, cudaStream_t st, bool overlap_previous,
                                  const F8Sibling *sib) {
    const size_t total = (size_t)g.n * g.ho * g.wo * g.c_out;
    if (total == 0) return cudaSuccess;
    const bool vec = (g.c % 4 == 0) && (((uintptr_t)x | (uintptr_t)w) % 4 == 0);
    const F8Sibling sb = sib ? *sib : F8Sibling();
    if (vec)
        launch_k(conv_direct_kernel<true>, grid_for(total, 256), 256, overlap_previous, st, g, q, (const uint8_t *)x, w, bias, res, y, sb);
    else
        launch_k(conv_direct_kernel<false>, grid_for(total, 256), 256, overlap_previous, st, g, q, (const uint8_t *)x, w, bias, res, y, sb);
    return cudaGetLastError();
}

cudaError_t f8_launch_dwconv(const F8ConvGeom &g, const F8Requant &q, const void *x, const int8_t *w,
                             const int32_t *bias, const void *res, void *y, cudaStream_t st, bool overlap_previous) {
    const size_t total = (size_t)g.n * g.ho * g.wo * g.c;
    if (total == 0) return cudaSuccess;
    const bool strip_ok = g.c % 4 == 0 && g.kh == 3 && g.kw == 3 && g.pad_h == 1 && g.pad_w == 1 &&
                          g.stride_h == g.stride_w && (g.stride_h == 1 || g.stride_h == 2) &&
                          (((uintptr_t)x | (uintptr_t)y | (uintptr_t)res | (uintptr_t)bias) & 15) == 0 &&
                          (size_t)g.n * g.h * g.w * g.c < (1u << 31) && total * (q.y_kind == F8_S32 ? 4 : 1) < (1u << 31);
    const bool walk_ok = strip_ok && g.stride_h == 1 && !q.has_res && q.y_kind != F8_S32 && q.s >= 1 && q.s <= 24 &&
                         q.sh_acc == 0 && !(f8_plan_options_off() & F8_PLAN_OFF_DW_WALK);
    const bool dp4a_ok = strip_ok && !q.has_res && (q.y_kind == F8_U8 || q.y_kind == F8_S8) && q.s >= 1 &&
                         q.s <= 24 && q.sh_acc == 0 && !(f8_plan_options_off() & F8_PLAN_OFF_DW_DP4A);
    if (dp4a_ok && g.stride_h == 2) {
        const int strips = (g.wo + 1) / 2;
        int band_rows = g.ho;
        while (band_rows > 4 && (long long)g.n * ((g.ho + band_rows - 1) / band_rows) * strips * (g.c / 4) < 148 * 128 * 8)
            band_rows = (band_rows + 1) / 2;
        const int bands = (g.ho + band_rows - 1) / band_rows;
        const int threads = g.n * bands * strips * (g.c / 4);
        const int grid = grid_for((size_t)threads, 128);
        const uint8_t *xp = (const uint8_t *)x;
#define F8_DW_DP4A2(XS_, SO_) \
    launch_k(dwconv3x3s2_dp4a_kernel<XS_, SO_>, grid, 128, overlap_previous, st, g, q, xp, w, bias, (uint8_t *)y, strips, bands, band_rows, threads)
        const bool so = q.y_kind == F8_S8;
        if (g.x_signed) { if (so) F8_DW_DP4A2(true, true); else F8_DW_DP4A2(true, false); }
        else { if (so) F8_DW_DP4A2(false, true); else F8_DW_DP4A2(false, false); }
#undef F8_DW_DP4A2
    } else if (dp4a_ok) {
        const int strips = (g.wo + 1) / 2;
        int band_rows = g.ho;
        while (band_rows > 8 && (long long)g.n * ((g.ho + band_rows - 1) / band_rows) * strips * (g.c / 4) < 148 * 128 * 8)
            band_rows = (band_rows + 1) / 2;
        const int bands = (g.ho + band_rows - 1) / band_rows;
        const int threads = g.n * bands * strips * (g.c / 4);
        const int grid = grid_for((size_t)threads, 128);
        const uint8_t *xp = (const uint8_t *)x;
#define F8_DW_DP4A(XS_, SO_) \
    launch_k(dwconv3x3_dp4a_kernel<XS_, SO_>, grid, 128, overlap_previous, st, g, q, xp, w, bias, (uint8_t *)y, strips, bands, band_rows, threads)
        const bool so = q.y_kind == F8_S8;
        if (g.x_signed) { if (so) F8_DW_DP4A(true, true); else F8_DW_DP4A(true, false); }
        else { if (so) F8_DW_DP4A(false, true); else F8_DW_DP4A(false, false); }
#undef F8_DW_DP4A
    } else if (walk_ok) {
        // two columns per thread measured slightly ahead of four (96 against 128 registers: 20 against 16 warps per SM)
        const int wcols = 2;
        const int strips = (g.wo + wcols - 1) / wcols;
        // bands of output rows: long enough to amortise the two extra input rows and the tap loads, short enough to
        // give every SM several blocks
        int band_rows = g.ho;
        while (band_rows > 8 && (long long)g.n * ((g.ho + band_rows - 1) / band_rows) * strips * (g.c / 4) < 148 * 128 * 8)
            band_rows = (band_rows + 1) / 2;
        const int bands = (g.ho + band_rows - 1) / band_rows;
        const int threads = g.n * bands * strips * (g.c / 4);
        const int grid = grid_for((size_t)threads, 128);
        const uint8_t *xp = (const uint8_t *)x;
#define F8_DW_WALK(XS_, SO_, C_) \
    launch_k(dwconv3x3_walk_kernel<XS_, SO_, C_>, grid, 128, overlap_previous, st, g, q, xp, w, bias, (uint8_t *)y, strips, bands, band_rows, threads)
        const bool so = q.y_kind == F8_S8;
        if (wcols == 2) {
            if (g.x_signed) { if (so) F8_DW_WALK(true, true, 2); else F8_DW_WALK(true, false, 2); }
            else { if (so) F8_DW_WALK(false, true, 2); else F8_DW_WALK(false, false, 2); }
        } else {
            if (g.x_signed) { if (so) F8_DW_WALK(true, true, 4); else F8_DW_WALK(true, false, 4); }
            else { if (so) F8_DW_WALK(false, true, 4); else F8_DW_WALK(false, false, 4); }
        }
#undef F8_DW_WALK
    } else if (strip_ok) {
        const int tw = g.stride_h == 1 ? 8 : 4;
        const int strips = (g.wo + tw - 1) / tw;
        const int threads = g.n * g.ho * strips * (g.c / 4);
        const int grid = grid_for((size_t)threads, 128);
        const uint8_t *xp = (const uint8_t *)x;
        const bool fast = q.y_kind != F8_S32 && q.s >= 1 && q.s <= 24;
#define F8_DW_LAUNCH(S_, TW_, XS_, FAST_) \
    launch_k(dwconv3x3_strip_kernel<S_, TW_, XS_, FAST_>, grid, 128, overlap_previous, st, g, q, xp, w, bias, res, y, strips, threads)
        if (g.stride_h == 1) {
            if (g.x_signed) { if (fast) F8_DW_LAUNCH(1, 8, true, true); else F8_DW_LAUNCH(1, 8, true, false); }
            else { if (fast) F8_DW_LAUNCH(1, 8, false, true); else F8_DW_LAUNCH(1, 8, false, false); }
        } else {
            if (g.x_signed) { if (fast) F8_DW_LAUNCH(2, 4, true, true); else F8_DW_LAUNCH(2, 4, true, false); }
            else { if (fast) F8_DW_LAUNCH(2, 4, false, true); else F8_DW_LAUNCH(2, 4, false, false); }
        }
#undef F8_DW_LAUNCH
    } else if (g.c % 4 == 0)
        launch_k(dwconv_vec4_kernel, grid_for(total / 4, 256), 256, overlap_previous, st, g, q, (const uint8_t *)x, w, bias, res, y);
    else
        launch_k(dwconv_scalar_kernel, grid_for(total, 256), 256, overlap_previous, st, g, q, (const uint8_t *)x, w, bias, res, y);
    return cudaGetLastError();
}

cudaError_t f8_launch_maxpool(int n, int h, int w, int c, int k, int stride, int pad, int x_signed, const void *x,
                              void *y, cudaStream_t st, bool overlap_previous) {
    const int ho = (h + 2 * pad - k) / stride + 1, wo = (w + 2 * pad - k) / stride + 1;
    const size_t total = (size_t)n * ho * wo * c;
    if (total == 0) return cudaSuccess;
    const size_t blocks8 = (size_t)n * ((ho + 1) / 2) * ((wo + 3) / 4) * (c / 16);
    if (c % 16 == 0 && k == 3 && stride == 2 && pad == 1 && ((uintptr_t)x | (uintptr_t)y) % 16 == 0) {
        if (x_signed)
            launch_k(maxpool3x3s2_kernel<true>, grid_for(blocks8, 128), 128, overlap_previous, st, n, h, w, c, ho, wo, (const uint8_t *)x, (uint8_t *)y);
        else
            launch_k(maxpool3x3s2_kernel<false>, grid_for(blocks8, 128), 128, overlap_previous, st, n, h, w, c, ho, wo, (const uint8_t *)x, (uint8_t *)y);
    } else if (c % 16 == 0)
        launch_k(maxpool_kernel<4>, grid_for(total / 16, 256), 256, overlap_previous, st, n, h, w, c, ho, wo, k, stride, pad, x_signed,
                                                                     (const uint8_t *)x, (uint8_t *)y);
    else if (c % 4 == 0)
        launch_k(maxpool_kernel<1>, grid_for(total / 4, 256), 256, overlap_previous, st, n, h, w, c, ho, wo, k, stride, pad, x_signed,
                                                                    (const uint8_t *)x, (uint8_t *)y);
    else
        launch_k(maxpool_scalar_kernel, grid_for(total, 256), 256, overlap_previous, st, n, h, w, c, ho, wo, k, stride, pad, x_signed,
                                                                    (const uint8_t *)x, (uint8_t *)y);
    return cudaGetLastError();
}

cudaError_t f8_launch_gap(int n, int h, int w, int c, int x_signed, int s, const void *x, void *y, cudaStream_t st,
                          bool overlap_previous) {
    if (n == 0) return cudaSuccess;
    if (c % 4 == 0 && (long long)h * w * 255 < 65536 && (((uintptr_t)x | (uintptr_t)y) & 3) == 0) {
        dim3 grid4((c / 4 + 255) / 256, n);
        launch_k(gap4_kernel, grid4, 256, overlap_previous, st, h * w, c, x_signed, s, (const uint8_t *)x, (uint8_t *)y);
        return cudaGetLastError();
    }
    dim3 grid((c + 255) / 256, n);
    launch_k(gap_kernel, grid, 256, overlap_previous, st, h * w, c, x_signed, s, (const uint8_t *)x, (uint8_t *)y);
    return cudaGetLastError();
}

cudaError_t f8_launch_pack_stem(int n, int h, int w, int c, int wp, int left, const void *x, void *y,
                                cudaStream_t st, bool overlap_previous) {
    const size_t total = (size_t)n * h * wp;
    if (total == 0) return cudaSuccess;
    launch_k(pack_stem_kernel, grid_for(total, 256), 256, overlap_previous, st, n, h, w, c, wp, left, (const uint8_t *)x, (uint2 *)y);
    return cudaGetLastError();
}

cudaError_t f8_launch_pack_stem_pairs(int n, int h, int w, int c, int cpad, int hp, int wp, int left, const void *x,
                                      void *y, cudaStream_t st, bool overlap_previous) {
    const size_t total = (size_t)n * hp * wp;
    if (total == 0) return cudaSuccess;
    if (cpad == 4)
        launch_k(pack_stem_pairs_kernel<4>, grid_for(total, 256), 256, overlap_previous, st, n, h, w, c, hp, wp, left, (const uint8_t *)x, (uint32_t *)y);
    else
        launch_k(pack_stem_pairs_kernel<8>, grid_for(total, 256), 256, overlap_previous, st, n, h, w, c, hp, wp, left, (const uint8_t *)x, (uint32_t *)y);
    return cudaGetLastError();
}
