// First layer of an image network on the tensor cores: a kh x kw convolution with stride 2 over an image with at
// most four channels (a2 - a4 fused: bias, rounding shift, clip), optionally followed in the same kernel by the
// 3x3 / stride 2 / pad 1 max pool that ResNet-style networks put behind it.
//
// The layer is a GEMM with a tiny K (7 x 7 x 3 = 147) and a huge M, and its input rows overlap heavily, so it is
// organised around the image rather than around an im2col gather:
//   * A CTA walks down a band of output rows.  For every PAIR of image rows it builds, in shared memory, a line of
//     8-byte cells: cell `col` holds pixel col - pad of both rows (4 bytes each, zero filled).  The kw-tap window
//     of output column ox over that row pair is then the 8 * kw bytes that start at cell 2 * ox, i.e. at byte
//     16 * ox: windows of neighbouring outputs overlap and are 16 bytes apart.
//   * That is exactly a K-major operand without swizzle whose 8 x 16-byte core matrices are 128 contiguous bytes
//     (row pitch 16 bytes), with 16 bytes between core matrices along K and 128 bytes between 8-row groups: the
//     tensor core reads the overlapping windows straight from the line, nothing is expanded.  One output row
//     (up to 128 pixels = the M of one tcgen05.mma) takes `kh2` row pairs x (window bytes / 32) instructions.
//   * The weights ([K / 16][c_out][16] bytes, the same core-matrix form) stay in shared memory.
//   * Two accumulators in tensor memory: the MMAs of row oy + 1 run while eight warps requantise row oy into a
//     ring of three finished rows, from which either the row itself or, every second row, one pooled row is
//     written to global memory with 16-byte accesses.
// The CTA is synchronised with two block barriers per row and one mbarrier wait (bounded) for the accumulator;
// several CTAs share an SM and fill each other's gaps.
#include <algorithm>
#include <stdio.h>
#include <stdlib.h>

#include "f8_epilogue.cuh"
#include "f8_tc_ptx.cuh"

namespace {

constexpr int STEM_EPI_WARPS = 8;
constexpr int STEM_THREADS = 32 * (STEM_EPI_WARPS + 1);     // warp 8 issues the MMAs
constexpr int STEM_PAIR_SLOTS = 8;                           // ring of packed row pairs (a window needs <= 7, plus one)
constexpr int STEM_SLOT_BYTES = 2176;                        // 128 windows 16 bytes apart, 64 bytes long, rounded up
constexpr int STEM_MAX_CELLS = 264;                          // cells a slot can hold (2112 bytes)

struct StemParams {
    int n, h, w, c;            // image, c <= 4
    int ho, wo, c_out;         // convolution output, wo <= 128
    int kh2;                   // row pairs one window covers
    int top;                   // the first pair of output row oy is oy - top
    int left;                  // zero cells in front of a line (the left padding)
    int hp;                    // row pairs per image
    int slices;                // 32-byte K slices per row pair
    int ncell;                 // cells of a line that can reach a valid output
    int pool;                  // 1: write the 3x3 / 2 / pad 1 max pool of the layer's output instead of the output
    int po, pwo;               // pooled height / width
    int rows_per_img;          // po or ho: output rows this launch writes per image
    int acc_cols;              // TMEM columns of one accumulator
    int cpr;                   // 16-byte chunks per output pixel (c_out / 16)
    int swz_shift, swz_mask;   // chunk swizzle of the finished-row ring: chunk ^ ((px >> shift) & mask)
    uint32_t idesc;
    uint32_t a_desc_hi, b_desc_hi;   // upper descriptor words (byte offsets between core matrices)
    uint32_t a_desc_lbo_sbo, b_desc_lbo_sbo;   // bits 16.. of the lower word (leading byte offset)
    int s;                     // rounding shift, 1..24
    int signed_out;
    int x_signed;
    const uint8_t *x;
    const int8_t *wk;          // [K / 16][c_out][16]
    const int32_t *bias;
    uint8_t *y;
    int *status;
    int tag;
    unsigned long long wait_limit;   // bound of the accumulator wait in SM cycles (0: the default)
};

__device__ __forceinline__ uint32_t ldg32(const uint8_t *p) { return __ldg((const uint32_t *)p); }

// The (up to four) channel bytes of the pixel that starts `off` bytes into the image tensor, zero extended to 32 bits.
// FAST: the tensor is 4-byte aligned and a multiple of 4 bytes long, so aligned words may be read up to its last one.
template <bool FAST>
__device__ __forceinline__ uint32_t load_pixel(const uint8_t *x, uint32_t off, uint32_t last_word, int c) {
    if (FAST) {
        if (c == 4) return ldg32(x + off);
        const uint32_t a = off & ~3u;
        const uint32_t w0 = ldg32(x + a), w1 = ldg32(x + min(a + 4u, last_word));
        return __funnelshift_r(w0, w1, (off & 3u) * 8u) & (0xffffffffu >> (32 - 8 * c));
    }
    uint32_t word = 0;
#pragma unroll
    for (int ch = 0; ch < 4; ++ch)
        if (ch < c) word |= (uint32_t)__ldg(x + off + ch) << (8 * ch);
    return word;
}

// CPR: 16-byte chunks per output pixel when known at compile time (0: read it from the parameters).
template <int CPR, bool POOL, bool SIGNED, bool FAST>
__global__ void __launch_bounds__(STEM_THREADS, 3) f8_stem_tc_kernel(const StemParams p, const int grid_units_total) {
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ __align__(8) uint64_t acc_bar[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cpr = CPR ? CPR : p.cpr;
    const uint32_t c_out = (uint32_t)cpr * 16u;
    const int k_bytes = p.kh2 * p.slices * 32;
    const uint32_t w_bytes = (uint32_t)k_bytes * c_out;
    const uint32_t row_bytes = 128u * c_out;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t pair_base = smem_base + w_bytes;
    const uint32_t rows_base = pair_base + STEM_PAIR_SLOTS * STEM_SLOT_BYTES;     // two finished / running-maximum rows
    const uint32_t bias_base = rows_base + 2 * row_bytes;
    uint8_t *const pair_ptr = smem + w_bytes;

    // ---- prologue (reads only parameters that no earlier work in the stream writes)
    {
        uint4 *z = (uint4 *)pair_ptr;     // cells past the image are never written again: they stay zero
        for (int i = threadIdx.x; i < STEM_PAIR_SLOTS * STEM_SLOT_BYTES / 16; i += STEM_THREADS) z[i] = make_uint4(0, 0, 0, 0);
        const uint4 *wg = (const uint4 *)p.wk;
        uint4 *ws = (uint4 *)smem;
        for (int i = threadIdx.x; i < (int)(w_bytes / 16); i += STEM_THREADS) ws[i] = __ldg(wg + i);
        int *bs = (int *)(smem + (bias_base - smem_base));
        const int rnd = 1 << (p.s - 1);
        for (int i = threadIdx.x; i < (int)c_out; i += STEM_THREADS) bs[i] = (p.bias ? __ldg(p.bias + i) : 0) + rnd;
    }
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&acc_bar[0]), 1);
        mbar_init(smem_u32(&acc_bar[1]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == STEM_EPI_WARPS) tmem_alloc(smem_u32(&tmem_base_slot), (uint32_t)(2 * p.acc_cols));
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // weights: generic writes, read by the tensor core
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    grid_launch_dependents();
    grid_dependency_wait();        // the image / the output buffer may belong to earlier work in the stream

    volatile int *abortp = &abort_flag;
    const WaitCtx wc = make_wait_ctx(&abort_flag, p.status, p.wait_limit);
    const int tagbits = p.tag << 8;
    const long long total = grid_units_total;
    const int u_begin = (int)(total * blockIdx.x / gridDim.x), u_end = (int)(total * (blockIdx.x + 1) / gridDim.x);
    const uint32_t rsel[4] = {0, 0, 0, 0};
    int k = 0;                       // rows issued so far by this CTA: accumulator k & 1, barrier parity (k >> 1) & 1

    // ---- per-thread constants
    // packing: this thread owns cell `col` (and col + STEM_THREADS) of every line
    const uint32_t img_row_bytes = (uint32_t)p.w * p.c;
    uint32_t cell_off[2];            // byte offset of the cell's pixel inside an image row
    bool cell_on[2], cell_px[2];     // the cell exists / holds a pixel (else zero padding)
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int col = threadIdx.x + i * STEM_THREADS, iw = col - p.left;
        cell_on[i] = col < p.ncell;
        cell_px[i] = cell_on[i] && iw >= 0 && iw < p.w;
        cell_off[i] = cell_px[i] ? (uint32_t)iw * p.c : 0u;
    }
    const uint32_t last_word = (uint32_t)p.n * p.h * img_row_bytes - 4u;
    // epilogue: this thread owns output pixel px and the 16-byte chunks [ch0, ch1) of it
    const int quarter = warp & 3, half = (warp >> 2) & 1;
    const int px = quarter * 32 + lane;
    const int ch_per = (cpr + 1) >> 1;
    const int ch0 = half * ch_per, ch1 = min(cpr, ch0 + ch_per);
    const uint32_t swz = ((uint32_t)px >> p.swz_shift) & (uint32_t)p.swz_mask;
    const uint32_t px_off = (uint32_t)px * c_out;

    auto load_cells = [&](int img, int pr, uint2 (&cell)[2]) {
        const uint32_t r0 = ((uint32_t)img * p.h + 2u * pr) * img_row_bytes;
        const bool second = 2 * pr + 1 < p.h;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            cell[i] = make_uint2(0u, 0u);
            if (cell_px[i]) {
                cell[i].x = load_pixel<FAST>(p.x, r0 + cell_off[i], last_word, p.c);
                if (second) cell[i].y = load_pixel<FAST>(p.x, r0 + img_row_bytes + cell_off[i], last_word, p.c);
            }
        }
    };
    auto store_cells = [&](int pr, const uint2 (&cell)[2]) {
        uint2 *line = (uint2 *)(pair_ptr + (pr & (STEM_PAIR_SLOTS - 1)) * STEM_SLOT_BYTES);
#pragma unroll
        for (int i = 0; i < 2; ++i)
            if (cell_on[i]) line[threadIdx.x + i * STEM_THREADS] = cell[i];
    };
    // issue the MMAs of output row oy into accumulator kk & 1 (one thread).  A lone thread pays for every instruction
    // it executes, so the descriptors are assembled from 32-bit words inside one asm block per row pair.
    const uint32_t a_lo0 = p.a_desc_lbo_sbo | ((pair_base & 0x3ffffu) >> 4), b_lo0 = p.b_desc_lbo_sbo | ((smem_base & 0x3ffffu) >> 4);
    const uint32_t b_slice = 2u * c_out;                 // 16-byte units between the K slices of the weights
    auto issue_row = [&](int oy, int kk) {
        const uint32_t d_tmem = tmem_base + (uint32_t)((kk & 1) * p.acc_cols);
        uint32_t accumulate = 0;
        uint32_t b_lo = b_lo0;
        for (int j = 0; j < p.kh2; ++j, b_lo += b_slice * p.slices) {
            const int pr = oy - p.top + j;
            if (pr < 0 || pr >= p.hp) continue;          // rows above / below the image contribute nothing
            const uint32_t a_lo = a_lo0 + (uint32_t)(pr & (STEM_PAIR_SLOTS - 1)) * (STEM_SLOT_BYTES / 16);
            if (p.slices == 2)
                asm volatile("{\n\t.reg .pred p, t;\n\t.reg .b64 a, b;\n\t.reg .b32 x, y;\n\tsetp.ne.b32 p, %7, 0;\n\t"
                             "setp.eq.b32 t, 0, 0;\n\tmov.b64 a, {%1, %3};\n\tmov.b64 b, {%2, %4};\n\t"
                             "tcgen05.mma.cta_group::1.kind::i8 [%0], a, b, %6, p;\n\t"
                             "add.u32 x, %1, 2;\n\tadd.u32 y, %2, %5;\n\tmov.b64 a, {x, %3};\n\tmov.b64 b, {y, %4};\n\t"
                             "tcgen05.mma.cta_group::1.kind::i8 [%0], a, b, %6, t;\n\t}" ::"r"(d_tmem),
                             "r"(a_lo), "r"(b_lo), "r"(p.a_desc_hi), "r"(p.b_desc_hi), "r"(b_slice), "r"(p.idesc), "r"(accumulate)
                             : "memory");
            else
                asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 a, b;\n\tsetp.ne.b32 p, %6, 0;\n\t"
                             "mov.b64 a, {%1, %3};\n\tmov.b64 b, {%2, %4};\n\t"
                             "tcgen05.mma.cta_group::1.kind::i8 [%0], a, b, %5, p;\n\t}" ::"r"(d_tmem),
                             "r"(a_lo), "r"(b_lo), "r"(p.a_desc_hi), "r"(p.b_desc_hi), "r"(p.idesc), "r"(accumulate)
                             : "memory");
            accumulate = 1;
        }
        mma_commit(smem_u32(&acc_bar[kk & 1]));
    };

    for (int u = u_begin; u < u_end;) {
        const int img = u / p.rows_per_img, r0 = u - img * p.rows_per_img;
        const int r1 = min(p.rows_per_img, r0 + (u_end - u));            // rows [r0, r1) of this image are ours
        u += r1 - r0;
        const int oy_first = POOL ? max(0, 2 * r0 - 1) : r0;
        const int oy_last = POOL ? min(p.ho - 1, 2 * (r1 - 1) + 1) : r1 - 1;

        // ---- lines of the first row's window; the line the second row adds stays in registers for now
        uint2 cell[2];
        for (int j = 0; j < p.kh2; ++j) {
            const int pr = oy_first - p.top + j;
            if (pr < 0 || pr >= p.hp) continue;
            load_cells(img, pr, cell);
            store_cells(pr, cell);
        }
        {
            const int pn = oy_first + 1 - p.top + p.kh2 - 1;
            if (oy_first + 1 <= oy_last && pn >= 0 && pn < p.hp) load_cells(img, pn, cell);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncthreads();
        if (warp == STEM_EPI_WARPS) {
            if (lane == 0) {
                tc_fence_after();
                issue_row(oy_first, k);
            }
            __syncwarp();
        }

        for (int oy = oy_first; oy <= oy_last; ++oy, ++k) {
            // ---- the line that row oy + 1 adds to the window
            if (oy + 1 <= oy_last) {
                const int pn = oy + 1 - p.top + p.kh2 - 1;
                if (pn >= 0 && pn < p.hp) store_cells(pn, cell);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncthreads();
            {
                // cells for the row after next: in flight while this row is converted
                const int pn2 = oy + 2 - p.top + p.kh2 - 1;
                if (oy + 2 <= oy_last && pn2 >= 0 && pn2 < p.hp) load_cells(img, pn2, cell);
            }
            // pooling: row oy closes the pooled row oy >> 1 when it is odd (or the last row) and opens the next one
            const bool closes = (oy & 1) || oy == p.ho - 1;
            // row 0 has no row above it: it starts the running maximum of pooled row 0 instead of joining one
            const bool opens = oy == 0;
            const int py = oy >> 1;
            if (warp == STEM_EPI_WARPS) {
                if (lane == 0 && oy + 1 <= oy_last) {
                    tc_fence_after();
                    issue_row(oy + 1, k + 1);
                }
                __syncwarp();
            } else {
                // ---- epilogue of row oy: thread = output pixel, 16 channels per accumulator load
                // the accumulator is usually a few hundred cycles away: sleep on the barrier (the hardware wakes the
                // thread when the phase completes or after the hinted time) before falling back to the bounded poll
                bool got = false;
#pragma unroll 1
                for (int t = 0; t < 4 && !got; ++t) got = mbar_try_wait_hint(smem_u32(&acc_bar[k & 1]), (uint32_t)(k >> 1) & 1u, 4000u);
                if (!got) got = mbar_wait(smem_u32(&acc_bar[k & 1]), (uint32_t)(k >> 1) & 1u, wc, tagbits | 120);
                if (__all_sync(0xffffffffu, got)) {
                    tc_fence_after();
                    const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)((k & 1) * p.acc_cols);
                    // POOL: buffer py & 1 holds the running maximum of the pooled row that is open
                    const uint32_t cur = rows_base + (POOL ? (uint32_t)(py & 1) * row_bytes : 0u) + px_off;
                    const uint32_t nxt = rows_base + (uint32_t)((py + 1) & 1) * row_bytes + px_off;
#pragma unroll
                    for (int ci = 0; ci < (CPR ? (CPR + 1) / 2 : 8); ++ci) {
                        const int ch = ch0 + ci;
                        if (ch >= ch1) break;
                        int v[16];
                        tmem_ld16(t_addr + ch * 16, v);
                        tmem_ld_wait();
                        const uint4 o = epilogue_fast16<false, SIGNED>(v, bias_base + 64 * ch, make_uint4(0, 0, 0, 0), 1, 0, rsel, p.s);
                        const uint32_t co = ((uint32_t)ch ^ swz) << 4;
                        if (!POOL) {
                            sts128(cur + co, o);
                        } else {
                            uint4 m = o;
                            if (!opens) {
                                const uint4 t = lds128(cur + co);
                                m.x = SIGNED ? __vmaxs4(t.x, o.x) : __vmaxu4(t.x, o.x);
                                m.y = SIGNED ? __vmaxs4(t.y, o.y) : __vmaxu4(t.y, o.y);
                                m.z = SIGNED ? __vmaxs4(t.z, o.z) : __vmaxu4(t.z, o.z);
                                m.w = SIGNED ? __vmaxs4(t.w, o.w) : __vmaxu4(t.w, o.w);
                            }
                            sts128(cur + co, m);
                            if (oy & 1) sts128(nxt + co, o);      // an odd row is also the top row of the next pooled row
                        }
                    }
                    tc_fence_before();
                }
            }
            __syncthreads();
            if (*abortp) break;

            // ---- write: the finished row, or the pooled row it closes (maximum over three neighbouring columns)
            if (!POOL) {
                uint8_t *dst = p.y + ((size_t)img * p.ho + oy) * (size_t)p.wo * c_out;
                for (int it = threadIdx.x; it < p.wo * cpr; it += STEM_THREADS) {
                    const int x0 = it / cpr, ch = it - x0 * cpr;
                    const uint32_t sw = ((uint32_t)x0 >> p.swz_shift) & (uint32_t)p.swz_mask;
                    *(uint4 *)(dst + (size_t)it * 16) = lds128(rows_base + (uint32_t)x0 * c_out + (((uint32_t)ch ^ sw) << 4));
                }
            } else if (closes && py >= r0 && py < r1) {
                const uint32_t src = rows_base + (uint32_t)(py & 1) * row_bytes;
                uint8_t *dst = p.y + ((size_t)img * p.po + py) * (size_t)p.pwo * c_out;
                for (int it = threadIdx.x; it < p.pwo * cpr; it += STEM_THREADS) {
                    const int ppx = it / cpr, ch = it - ppx * cpr;
                    const int cx = 2 * ppx;
                    const uint32_t sw1 = ((uint32_t)cx >> p.swz_shift) & (uint32_t)p.swz_mask;
                    uint4 m = lds128(src + (uint32_t)cx * c_out + (((uint32_t)ch ^ sw1) << 4));
                    if (cx > 0) {
                        const uint32_t sw0 = ((uint32_t)(cx - 1) >> p.swz_shift) & (uint32_t)p.swz_mask;
                        const uint4 t = lds128(src + (uint32_t)(cx - 1) * c_out + (((uint32_t)ch ^ sw0) << 4));
                        m.x = SIGNED ? __vmaxs4(t.x, m.x) : __vmaxu4(t.x, m.x);
                        m.y = SIGNED ? __vmaxs4(t.y, m.y) : __vmaxu4(t.y, m.y);
                        m.z = SIGNED ? __vmaxs4(t.z, m.z) : __vmaxu4(t.z, m.z);
                        m.w = SIGNED ? __vmaxs4(t.w, m.w) : __vmaxu4(t.w, m.w);
                    }
                    if (cx + 1 < p.wo) {
                        const uint32_t sw2 = ((uint32_t)(cx + 1) >> p.swz_shift) & (uint32_t)p.swz_mask;
                        const uint4 t = lds128(src + (uint32_t)(cx + 1) * c_out + (((uint32_t)ch ^ sw2) << 4));
                        m.x = SIGNED ? __vmaxs4(t.x, m.x) : __vmaxu4(t.x, m.x);
                        m.y = SIGNED ? __vmaxs4(t.y, m.y) : __vmaxu4(t.y, m.y);
                        m.z = SIGNED ? __vmaxs4(t.z, m.z) : __vmaxu4(t.z, m.z);
                        m.w = SIGNED ? __vmaxs4(t.w, m.w) : __vmaxu4(t.w, m.w);
                    }
                    *(uint4 *)(dst + (size_t)it * 16) = m;
                }
            }
        }
        if (*abortp) break;
        __syncthreads();      // the buffers are reused by the next band: everybody is done reading
    }
    if (*abortp && threadIdx.x == 0) {
        // aborting: give the MMAs already issued time to finish before tensor memory is released
        const unsigned long long t0 = clock64();
        while (!mbar_try_wait(smem_u32(&acc_bar[k & 1]), (uint32_t)(k >> 1) & 1u) &&
               (unsigned long long)(clock64() - t0) < DRAIN_LIMIT_CYCLES) {
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == STEM_EPI_WARPS) {
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)(2 * p.acc_cols));
    }
}

}   // namespace

static size_t stem_smem_bytes(int kh2, int slices, int c_out) {
    return (size_t)kh2 * slices * 32 * c_out + STEM_PAIR_SLOTS * STEM_SLOT_BYTES + 2 * 128 * (size_t)c_out + 4 * (size_t)c_out;
}

bool f8_stem_tc_supported(const F8ConvGeom &g, const F8Requant &q, int kh2, int slices) {
    if (g.c > 4 || g.stride_h != 2 || g.stride_w != 2) return false;
    if (g.wo > 128 || g.wo < 1 || g.c_out % 16 != 0 || g.c_out > 256) return false;
    if (q.has_res || (q.y_kind != F8_U8 && q.y_kind != F8_S8) || q.s < 1 || q.s > 24) return false;
    if (kh2 < 1 || kh2 >= STEM_PAIR_SLOTS || slices < 1 || slices > 2) return false;       // windows of at most 64 bytes
    if (2 * (g.wo - 1) + slices * 4 > STEM_MAX_CELLS) return false;
    if ((size_t)g.n * g.h * g.w * g.c >= 0x7fffffffull || (size_t)g.n * std::max(g.ho, 1) >= 0x7fffffffull) return false;
    return stem_smem_bytes(kh2, slices, g.c_out) <= 200 * 1024;
}

namespace {
typedef void (*StemKernel)(const StemParams, const int);
template <int CPR, bool POOL, bool SIGNED>
StemKernel pick_fast(bool fast) {
    return fast ? f8_stem_tc_kernel<CPR, POOL, SIGNED, true> : f8_stem_tc_kernel<CPR, POOL, SIGNED, false>;
}
template <int CPR>
StemKernel pick_kernel(bool pool, bool sgn, bool fast) {
    if (pool) return sgn ? pick_fast<CPR, true, true>(fast) : pick_fast<CPR, true, false>(fast);
    return sgn ? pick_fast<CPR, false, true>(fast) : pick_fast<CPR, false, false>(fast);
}
}   // namespace

cudaError_t f8_launch_stem_tc(const F8ConvGeom &g, const F8Requant &q, int kh2, int top, int left, int slices, int pool,
                              const void *x, const int8_t *w_core, const int32_t *bias, void *y, int *status_word, int tag,
                              cudaStream_t st, bool overlap_previous) {
    if (g.n == 0) return cudaSuccess;
    StemParams p = {};
    p.n = g.n; p.h = g.h; p.w = g.w; p.c = g.c;
    p.ho = g.ho; p.wo = g.wo; p.c_out = g.c_out;
    p.kh2 = kh2; p.top = top; p.left = left; p.hp = (g.h + 1) / 2; p.slices = slices;
    p.ncell = std::min(STEM_MAX_CELLS, 2 * (g.wo - 1) + slices * 4);
    p.pool = pool;
    p.po = (g.ho - 1) / 2 + 1;
    p.pwo = (g.wo - 1) / 2 + 1;
    p.rows_per_img = pool ? p.po : g.ho;
    p.acc_cols = 32;
    while (p.acc_cols < g.c_out) p.acc_cols *= 2;
    p.cpr = g.c_out / 16;
    const bool pow2 = (p.cpr & (p.cpr - 1)) == 0;
    p.swz_shift = p.cpr == 4 ? 1 : (p.cpr == 2 ? 2 : 0);
    p.swz_mask = (pow2 && p.cpr > 1) ? std::min(p.cpr, 8) - 1 : 0;
    p.idesc = (2u << 4) | ((g.x_signed ? 1u : 0u) << 7) | (1u << 10) | ((uint32_t)(g.c_out >> 3) << 17) | ((128u >> 4) << 24);
    // K-major operands without swizzle: core matrices of 8 rows x 16 bytes are 128 contiguous bytes; the leading
    // byte offset is the distance between core matrices along K, the stride byte offset the one between 8-row groups.
    // A (overlapping windows): 16 bytes along K, 128 bytes along M.  B ([K/16][c_out][16]): c_out * 16 along K, 128 along N.
    const uint32_t a_lbo = 16, a_sbo = 128, b_lbo = (uint32_t)g.c_out * 16, b_sbo = 128;
    p.a_desc_lbo_sbo = (a_lbo >> 4) << 16;
    p.b_desc_lbo_sbo = (b_lbo >> 4) << 16;
    p.a_desc_hi = (a_sbo >> 4) | (1u << 14);     // stride byte offset at bit 32, descriptor version 1 at bit 46, no swizzle
    p.b_desc_hi = (b_sbo >> 4) | (1u << 14);
    p.s = q.s;
    p.signed_out = q.y_kind == F8_S8 ? 1 : 0;
    p.x_signed = g.x_signed;
    p.x = (const uint8_t *)x; p.wk = w_core; p.bias = bias; p.y = (uint8_t *)y; p.status = status_word; p.tag = tag;
    p.wait_limit = f8_wait_limit_cycles();

    const bool fast = ((uintptr_t)x & 3) == 0 && ((size_t)g.n * g.h * g.w * g.c) % 4 == 0;
    const bool sgn = p.signed_out != 0;
    StemKernel kernel = p.cpr == 4 ? pick_kernel<4>(pool != 0, sgn, fast)
                        : (p.cpr == 2 ? pick_kernel<2>(pool != 0, sgn, fast) : pick_kernel<0>(pool != 0, sgn, fast));
    const size_t smem = stem_smem_bytes(kh2, slices, g.c_out);
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(200 * 1024));
    // several CTAs are meant to share an SM: ask for the largest shared-memory carve-out (the default preference
    // sizes it for a single CTA of this kernel)
    if (e == cudaSuccess) e = cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 148, occ = 1;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    // CTAs that fit an SM, from the kernel's own resource use (the runtime's occupancy query answers 1 for this
    // kernel whatever the carve-out): registers, shared memory, threads, and two accumulators each in tensor memory
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, kernel) == cudaSuccess && fa.numRegs > 0) {
        const int regs_per_cta = ((fa.numRegs + 7) / 8 * 8) * STEM_THREADS;
        const int by_regs = 65536 / regs_per_cta;
        const int by_smem = (int)((227 * 1024) / (smem + fa.sharedSizeBytes + 1024));
        const int by_threads = 2048 / STEM_THREADS;
        occ = std::min(std::min(by_regs, by_smem), by_threads);
    }
    occ = std::min(occ, 512 / (2 * p.acc_cols));
    occ = std::max(1, std::min(occ, 4));
    const long long units = (long long)g.n * p.rows_per_img;
    // bands of at least four output rows (each band recomputes one row above it when pooling)
    long long grid = std::min<long long>((long long)sms * occ, std::max<long long>(1, units / 4));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(STEM_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap_previous ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, p, (int)units);
}
