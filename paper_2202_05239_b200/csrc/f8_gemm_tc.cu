// Dense convolution / pointwise / fully connected layers as an implicit GEMM on the Blackwell tensor
// cores:  D[M = output pixels, N = output channels] = A[M, K = taps x channels] * B[N, K]^T.
//
//   * A tiles (128 output pixels x KB channels of one filter tap) are gathered straight from the NHWC
//     activation tensor by TMA in im2col mode (zero fill outside the image and past the last pixel);
//     B tiles (BN output channels x KB) come from the OHWI weight tensor by tiled TMA.  Both land in
//     shared memory in the swizzled K-major layout tcgen05.mma reads.
//   * One thread issues tcgen05.mma.kind::i8 (u8|s8 x s8 -> s32); the 128 x BN int32 accumulator lives
//     in tensor memory, double buffered so the epilogue of tile i overlaps the main loop of tile i+1.
//   * Sixteen epilogue warps read the accumulator with tcgen05.ld (one output pixel per thread, 16
//     consecutive channels per load), add the bias, align and add the residual, apply the rounding
//     shift and clip (Eq. 2 / signed form applied to Eq. 6).  The 8-bit result goes to a swizzled staging
//     tile in shared memory; a mover thread stores finished tiles with one TMA instruction per 128-byte
//     column slab and a fetcher thread brings in the residual tiles the same way, two tiles ahead.  All
//     hand-offs are mbarriers, nobody waits at a block-wide barrier, and global memory only sees
//     full-line accesses.  Shapes that do not fit this scheme (int32 output, c_out not a multiple of
//     16) use direct stores.
//   * Persistent CTAs (one per SM) walk the tile list; tiles that share an A tile are adjacent so that
//     the activation tensor is read from HBM once and from L2 afterwards.
//
// Every mbarrier wait is bounded: when a wait does not complete the kernel raises a shared abort flag,
// writes the device status word, drains what it started and returns; it never spins forever or traps.
#include <cuda.h>
#include <cudaTypedefs.h>

#include <stdlib.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>

#include "f8_epilogue.cuh"
#include "f8_tc_ptx.cuh"

namespace {

constexpr int TILE_M = 128;
constexpr int NUM_EPI_WARPS = 16;          // four warps per TMEM lane quarter, each takes a quarter of the columns
// The TMA serves the loads of one thread strictly one after the other, and one load occupies it for
// several hundred cycles whatever the box size, so a single issuing thread caps a CTA at roughly ten
// bytes per clock.  Loads issued by different threads (lanes of one warp included) overlap: every
// (stage, sub-chunk) pair therefore has its own lane.  Issuing a TMA instruction also holds the issuing
// warp for a few hundred cycles, so activations and weights are requested by two different warps.
constexpr int A_PROD_WARP = 0;             // requests activation tiles
constexpr int MMA_WARP = 1;
constexpr int MOVER_WARP = 2;              // one thread stores finished output tiles
constexpr int FETCH_WARP = 3;              // one thread fetches residual tiles
constexpr int FIRST_EPI_WARP = 4;          // warps 4..19; warp & 3 is the TMEM lane quarter
constexpr int B_PROD_WARP = FIRST_EPI_WARP + NUM_EPI_WARPS;   // requests weight tiles
// Issuing a tcgen05.mma costs its thread 70-100 cycles, more than the tensor pipe needs for a tile of up to
// 128 columns; a second issuer (alternate tiles, the other accumulator) keeps the pipe fed for such layers.
constexpr int MMA2_WARP = B_PROD_WARP + 1;
// A producer warp spends roughly a thousand cycles per stage use (wait for the stage, announce, issue, loop), and with
// streamed weights the few stages that fit make the ring latency bound: a second pair of producer warps takes every
// other stage use.
constexpr int A2_PROD_WARP = MMA2_WARP + 1;
constexpr int B2_PROD_WARP = MMA2_WARP + 2;
constexpr int NUM_THREADS = 32 * (B2_PROD_WARP + 1);
constexpr int MAX_STAGES = 16;
constexpr int MAX_OUT_BUFS = 4;             // ring of staged output tiles; with a residual, the residual tile lands in the
                                            // buffer first and the epilogue converts it in place
constexpr int TMEM_COLS = 512;
// Shared memory budget of stages, staging and resident weights: the 227 KiB a block may have, minus the control block
// in front of them and up to 1023 bytes of alignment slack (the kernel has no static shared memory).
constexpr size_t SMEM_LIMIT = 225 * 1024;
constexpr uint32_t CONTROL_BYTES = 1024;

struct TcControl {
    uint64_t bars[2 * MAX_STAGES + 5];        // full[], empty[], tfull[2], tempty[2], bres
    uint64_t epi_bars[3 * MAX_OUT_BUFS];      // out_full[], out_free[], res_full[]
    uint32_t tmem_base_slot;
    int abort_flag;
};
static_assert(sizeof(TcControl) <= CONTROL_BYTES, "control block does not fit its slot");

// Division by a run-time constant without a divide instruction (a 32-bit divide costs a lone thread well over a
// hundred cycles): q = (n * mul) >> shift is exact for 0 <= n < 2^31 with mul = floor(2^shift / d) + 1,
// shift = 31 + ceil(log2 d).
struct FastDiv {
    uint32_t mul, shift;
};
__device__ __forceinline__ int fast_div(int n, FastDiv d) { return (int)(((uint64_t)(uint32_t)n * d.mul) >> d.shift); }

struct TcParams {
    int M;                    // total output pixels
    int ho, wo;
    int c_out;
    int kh, kw;
    int stride_h, stride_w, pad_h, pad_w;
    int c_chunks;             // K chunks per tap
    int kb;                   // bytes (= int8 elements) of K per stage: 32, 64 or 128
    int bn;                   // N tile, multiple of 16, <= 256
    int m_tiles, n_tiles;
    FastDiv div_n_tiles, div_wo, div_ho;
    int stages;
    int group;                // k-iterations per stage (1..8)
    int uses;                 // stage uses per tile: ceil(k_iters / group)
    int dual_issue;           // 1: two MMA-issuing threads (needs stages >= 2 * uses)
    int a_plain;              // 1: pointwise layer on a small tensor: activations read as a plain [M, C] matrix (tiled map)
    int pair;                 // 1: CTA pairs (the PAIR instantiation): 256-row tiles, half of a weight tile per CTA
    int pair_tiles;           // 256-row tiles x N tiles
    int alt;                  // 1: two pairs of producer warps, pair h takes the stage uses of parity h (streamed weights,
                              // one MMA issuer: fills may then complete out of order, the consumer is in order)
    int sup;                  // 0, or the number of M tiles (2..4) that share one stage use and one accumulator hand-over: layers
                              // with a single k-iteration and narrow tiles, where the per-tile hand-overs between the roles cost
                              // more than the tile's work.  M tile j of such a group takes columns j * bn of the accumulator and
                              // column slab j of the staged output
    int sup_tiles;            // groups of `sup` M tiles
    int epi_groups;           // 1, 2 or 4: the tile's columns are split over this many groups of four epilogue warps (one warp per
                              // tensor-memory lane quarter); the warps of the other groups stay out of the tile loop
    uint32_t sub_bytes;       // A + B bytes of one k-iteration (each rounded to 1024)
    uint32_t stage_bytes;     // group * sub_bytes
    uint32_t a_bytes;         // bytes of the A part (rounded to 1024)
    uint32_t tx_a, tx_b;      // bytes the A / B load of a k-iteration delivers
    uint32_t tx_sub;          // bytes a k-iteration adds to its stage's full barrier
    int b_res;                // 1: the whole weight tensor stays in shared memory for the life of the CTA
    uint32_t b_bytes;         // bytes of one B tile (rounded to 1024)
    uint32_t bres_off;        // resident weights: tile (n_t, k-iteration) at bres_off + (n_t * k_iters + k) * b_bytes
    uint32_t idesc;           // tcgen05 instruction descriptor
    uint64_t desc_hi;         // constant upper part of the shared-memory matrix descriptors
    const int32_t *bias;
    const uint8_t *res;
    uint8_t *y;
    int vec_bytes;            // widest aligned store the output rows allow: 16, 8, 4 or 1
    int epi;                  // EPI_* epilogue variant
    // staged epilogue: the output tile (and the residual tile) pass through shared memory in column
    // slabs of slab_w bytes per row, written / read by TMA with the matching swizzle (few, large TMA
    // operations: the TMA serves roughly one operation per hundred cycles whatever its size)
    int slab_w;               // 16, 32, 64 or 128 bytes
    int slab_chunks;          // slab_w / 16
    int n_slabs;              // bn / slab_w
    uint32_t swz_mask;        // 7, 3, 1 or 0: address bits 7.. XORed into the 16-byte chunk index
    uint32_t out_bytes;       // TILE_M * bn
    int out_bufs;             // staged output tiles in the ring (2..MAX_OUT_BUFS)
    uint32_t out_off, bias_off;   // byte offsets behind the stages: two output tiles, two residual
                                           // tiles, int32 bias' of all padded columns
    uint32_t ktab_off;        // table of k-iteration coordinates (8 bytes each)
    F8Requant q;
    F8Sibling sib;            // second consumer of the same sums (generic epilogue only)
    int vec_bytes2;           // widest aligned store of the second output's rows
    int mul_acc, mul_res;     // 2^q.sh_acc, 2^q.sh_res (kept opaque to the compiler, see the epilogue)
    int *status;
    // Windowed 3x3 (stride 1, pad 1, resident weights).  A tile is win_r whole output rows of one image; its M index runs
    // over the rows of the zero-padded image (win_wp = W + 2 positions per row, the last two of each row are discarded).
    // The padded input rows win_r + 2 rows tall are loaded ONCE per channel chunk as they lie in memory; the window of
    // filter tap (r, s) is then the same shared-memory tile read from (r * win_wp + s) pixel rows further down, so the
    // activations cross the L2 -> SM path once instead of nine times.
    int win;
    // Row-tiled geometry (rows = 1): a tile is win_r whole output rows of one image (win_wp positions per row, win_bands
    // tiles per image), stored / fetched with 4-D tensor maps.  The windowed mode uses it with win_wp = W + 2; small
    // tensors (for which no im2col map is made) use it with win_wp = W_out and one tiled load per filter tap, whose box
    // starts at the tap's offset and whose out-of-image elements are zero filled (rowt = 1).
    int rows, rowt;
    int win_r, win_wp, win_bands;
    FastDiv div_bands;
    uint32_t tx_win;          // bytes of one window load
    uint32_t tx_res;          // bytes of one residual tile load
    int tag;                  // caller's label of this launch (layer index + 1), reported with a timed-out wait
    unsigned long long wait_limit;   // bound of every mbarrier wait in SM cycles (0: the default, about two seconds)
};

// ----------------------------------------------------------------------------- epilogue helpers

// Writes 16 consecutive channels of one output row for one consumer of the aligned sums v[].
__device__ __forceinline__ void store_chunk(uint8_t *ybase, int y_kind, int s, int lo, int hi, const int (&v)[16], size_t o,
                                            int nvalid, int c_out, int vec_bytes) {
    int t[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) t[j] = f8_quantize_child(v[j], y_kind, s, lo, hi);
    if (y_kind == F8_S32 || y_kind == F8_S32_RELU) {
        int32_t *y32 = (int32_t *)ybase + o;
        if (nvalid == 16 && (c_out & 3) == 0) {
#pragma unroll
            for (int j = 0; j < 4; ++j) *(int4 *)(y32 + 4 * j) = make_int4(t[4 * j], t[4 * j + 1], t[4 * j + 2], t[4 * j + 3]);
        } else {
            for (int j = 0; j < nvalid; ++j) y32[j] = t[j];
        }
        return;
    }
    uint32_t ow[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) ow[j] = f8_pack4(t[4 * j], t[4 * j + 1], t[4 * j + 2], t[4 * j + 3]);
    uint8_t *yo = ybase + o;
    if (nvalid == 16 && vec_bytes == 16) {
        *(uint4 *)yo = make_uint4(ow[0], ow[1], ow[2], ow[3]);
    } else if (vec_bytes >= 8 && (nvalid & 7) == 0) {
        for (int j = 0; j < nvalid / 8; ++j) *(uint2 *)(yo + 8 * j) = make_uint2(ow[2 * j], ow[2 * j + 1]);
    } else if (vec_bytes >= 4 && (nvalid & 3) == 0) {
        for (int j = 0; j < nvalid / 4; ++j) *(uint32_t *)(yo + 4 * j) = ow[j];
    } else {
        for (int j = 0; j < nvalid; ++j) yo[j] = (uint8_t)(ow[j >> 2] >> (8 * (j & 3)));
    }
}

// Generic epilogue with direct stores: any output kind, any channel count, an 8-bit or 32-bit shortcut, and
// optionally a second consumer of the same sums with its private fractional length (Sec. 4.3).
__device__ __forceinline__ void epilogue_chunk(const TcParams &p, const int (&acc)[16], size_t row, int co0,
                                               bool row_valid) {
    // how many of the 16 channels exist
    const int nvalid = min(16, p.c_out - co0);
    int v[16];
    const size_t o = row * (size_t)p.c_out + co0;
    int r[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) r[j] = 0;
    if (p.q.has_res && row_valid) {
        if (p.q.r_s32) {
            const int32_t *r32 = (const int32_t *)p.res + o;
            if (nvalid == 16 && (p.c_out & 3) == 0) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int4 t = *(const int4 *)(r32 + 4 * j);
                    r[4 * j] = t.x; r[4 * j + 1] = t.y; r[4 * j + 2] = t.z; r[4 * j + 3] = t.w;
                }
            } else {
                for (int j = 0; j < nvalid; ++j) r[j] = r32[j];
            }
        } else {
            uint32_t rw[4] = {0u, 0u, 0u, 0u};
            if ((p.c_out & 15) == 0 && nvalid == 16) {      // 8-bit rows of c_out bytes: 16-byte aligned chunks
                const uint4 t = *(const uint4 *)(p.res + o);
                rw[0] = t.x; rw[1] = t.y; rw[2] = t.z; rw[3] = t.w;
            } else {
                for (int j = 0; j < nvalid; ++j) rw[j >> 2] |= (uint32_t)p.res[o + j] << (8 * (j & 3));
            }
#pragma unroll
            for (int j = 0; j < 16; ++j) r[j] = f8_byte(rw[j >> 2], j & 3, p.q.r_signed);
        }
    }
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const int b = (j < nvalid && p.bias) ? __ldg(p.bias + co0 + j) : 0;
        v[j] = f8_align_add(acc[j] + b, r[j], p.q);
    }
    if (!row_valid) return;
    store_chunk(p.y, p.q.y_kind, p.q.s, p.q.lo, p.q.hi, v, o, nvalid, p.c_out, p.vec_bytes);
    if (p.sib.y2) store_chunk((uint8_t *)p.sib.y2, p.sib.y_kind, p.sib.s, p.sib.lo, p.sib.hi, v, o, nvalid, p.c_out, p.vec_bytes2);
}

// ----------------------------------------------------------------------------- the kernel

enum { EPI_GENERIC = 0, EPI_U8 = 1, EPI_U8_RES = 2, EPI_S8 = 3, EPI_S8_RES = 4 };

// MODE 0: one 128-row tile per hand-over.  MODE 2: groups of M tiles (TcParams::sup).  MODE 1 (PAIR below):
// PAIR: two CTAs of a cluster share 256-row tiles (tcgen05 cta_group::2): each loads its own 128 rows of activations and
// half of the weight tile, so a weight byte crosses the L2 -> SM path once per 256 rows; the even CTA issues the MMAs.
template <int EPI, int MODE>
__global__ void __launch_bounds__(NUM_THREADS, 1)
f8_conv_gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                       const __grid_constant__ CUtensorMap map_y, const __grid_constant__ CUtensorMap map_r,
                       const TcParams p) {
    constexpr bool PAIR = MODE == 1;                                // CTA pairs
    constexpr bool SUP = MODE == 2;                                 // groups of M tiles per hand-over (TcParams::sup)
    constexpr bool STAGED = EPI != EPI_GENERIC;                     // output (and residual) through shared memory + TMA
    constexpr bool RES = EPI == EPI_U8_RES || EPI == EPI_S8_RES;
    constexpr bool SGN = EPI == EPI_S8 || EPI == EPI_S8_RES;

    extern __shared__ uint8_t smem_raw[];
    // stage buffers need 1024-byte alignment for the 128-byte swizzle
    uint8_t *smem_aligned = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    // Barriers, the tensor-memory address and the abort flag live in the first KiB of the aligned buffer: the same
    // place in every instantiation of this kernel (the kernel has no static shared memory of its own, so the
    // compiler lays nothing out).  Everything else follows behind it.
    TcControl &ctl = *(TcControl *)smem_aligned;
    uint8_t *smem = smem_aligned + CONTROL_BYTES;
    uint64_t *const bars = ctl.bars;
    uint64_t *const epi_bars = ctl.epi_bars;         // out_full[], out_free[], res_full[]
    uint32_t &tmem_base_slot = ctl.tmem_base_slot;
    int &abort_flag = ctl.abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    // persistent workers: CTAs, or CTA pairs (rank 0 = the even CTA, which owns the stage barriers and issues the MMAs)
    const uint32_t cta_rank = PAIR ? cluster_cta_rank() : 0u;
    const int worker = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int n_workers = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    const uint32_t full_bar = smem_u32(&bars[0]);
    const uint32_t empty_bar = smem_u32(&bars[MAX_STAGES]);
    const uint32_t tfull_bar = smem_u32(&bars[2 * MAX_STAGES]);
    const uint32_t tempty_bar = smem_u32(&bars[2 * MAX_STAGES + 2]);
    const uint32_t bres_bar = smem_u32(&bars[2 * MAX_STAGES + 4]);   // resident weights have landed
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t out_full = smem_u32(&epi_bars[0]), out_free = smem_u32(&epi_bars[MAX_OUT_BUFS]);
    const uint32_t res_full = smem_u32(&epi_bars[2 * MAX_OUT_BUFS]);

    if (threadIdx.x == 32) {
        // the first copy through a tensor map otherwise pays for fetching the map itself, at the head of every layer
        prefetch_tensormap(&map_a);
        prefetch_tensormap(&map_b);
        if (STAGED) prefetch_tensormap(&map_y);
        if (RES) prefetch_tensormap(&map_r);
    }
    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(full_bar + 8 * s, p.win ? 1 : 2);   // per use: one arrival (with its byte count) per producer warp
            mbar_init(empty_bar + 8 * s, 1);
        }
        mbar_init(bres_bar, 1);
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull_bar + 8 * a, 1);
            mbar_init(tempty_bar + 8 * a, (PAIR ? 8 : 4) * p.epi_groups);     // the active epilogue warps (of both CTAs)
        }
        for (int a = 0; a < MAX_OUT_BUFS; ++a) {
            mbar_init(out_full + 8 * a, 4 * p.epi_groups);   // every active epilogue warp has written its part of the tile
            mbar_init(out_free + 8 * a, 1);               // the store has finished reading the tile
            mbar_init(res_full + 8 * a, 1);               // the residual tile has landed in the buffer (transaction count)
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    {
        // coordinates of every k-iteration (filter tap and channel chunk), once per CTA
        uint2 *ktab = (uint2 *)(smem + p.ktab_off);
        for (int i = threadIdx.x; i < p.kh * p.kw * p.c_chunks; i += NUM_THREADS) {
            const int tap = i / p.c_chunks, cc = i - tap * p.c_chunks;
            const int r = tap / p.kw, sx = tap - r * p.kw;
            ktab[i] = make_uint2((uint32_t)(cc * p.kb), ((uint32_t)tap << 16) | ((uint32_t)r << 8) | (uint32_t)sx);
        }
    }
    if (warp == MMA_WARP) {
        if (PAIR) tmem_alloc_pair(smem_u32(&tmem_base_slot), TMEM_COLS);
        else tmem_alloc(smem_u32(&tmem_base_slot), TMEM_COLS);
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();      // the partner's barriers exist before anything is sent to them
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    // the next grid in the stream may be scheduled from here on: its CTAs take over an SM when this grid's
    // CTA there has exited, and run their prologue while the rest of this grid finishes
    grid_launch_dependents();

    // per worker: 128-row tiles, 256-row tiles of a pair, or groups of p.sup M tiles
    const int total_tiles = PAIR ? p.pair_tiles : (SUP ? p.sup_tiles : p.m_tiles * p.n_tiles);
    const int k_iters = p.kh * p.kw * p.c_chunks;
    const WaitCtx wc = make_wait_ctx(&abort_flag, p.status, p.wait_limit);
    const int tagbits = p.tag << 8;     // status word of a timed-out wait: tag << 8 | site

    if (warp == A_PROD_WARP || warp == B_PROD_WARP || ((warp == A2_PROD_WARP || warp == B2_PROD_WARP) && p.alt)) {
        // ------------------------------------------------------------------ TMA producer warps
        // A stage holds `group` consecutive k-iterations of one tile (fewer at the tile's end).  Each producer
        // warp makes one pass per stage use: it waits for the stage, then lane (st*group + j) & 31 issues the
        // load of sub-chunk j with the coordinates of its k-iteration from a table built at kernel start.
        // There is no per-k-iteration loop (a single warp spends a few hundred cycles of loop overhead per
        // iteration, which used to bound layers with many short k-iterations), and consecutive loads sit in
        // different per-thread TMA queues, so they overlap.
        const uint2 *ktab = (const uint2 *)(smem + p.ktab_off);
        const int opnd = (warp == A_PROD_WARP || warp == A2_PROD_WARP) ? 0 : 1;
        const int half = (warp == A2_PROD_WARP || warp == B2_PROD_WARP) ? 1 : 0;      // which uses this warp takes (p.alt)
        int use_idx = 0;
        if (opnd == 1 && p.b_res) {
            // Resident weights: when all B tiles fit beside the pipeline, they are loaded once and every tile
            // of this CTA reuses them; the stages then carry activations only (the weight re-reads are what
            // saturates the L2 -> SM path of layers with few output channels).
            const int n_loads = p.n_tiles * k_iters;
            if (lane == 0) mbar_expect_tx(bres_bar, (uint32_t)n_loads * p.tx_b);
            __syncwarp();
            for (int i = lane; i < n_loads; i += 32) {
                const int n_t = i / k_iters, k = i - n_t * k_iters;
                const uint2 e = ktab[k];
                tma_load_3d(smem_base + p.bres_off + (uint32_t)i * p.b_bytes, &map_b, bres_bar, (int)e.x, (int)(e.y >> 16),
                            n_t * p.bn);
            }
        }
        {
        // With resident weights the weight warp has nothing left to request: it takes the odd sub-chunks of
        // the activation loads off the activation warp (issuing a TMA instruction holds a warp for a few
        // hundred cycles per participating lane, which otherwise bounds layers with short tiles).
        const bool a_helper = opnd == 1 && p.b_res;
        const int j_mask = p.b_res ? 1 : 0, j_want = a_helper ? 1 : 0;     // which sub-chunks this warp requests
        if (opnd == 0 || a_helper) grid_dependency_wait();      // activations come from the previous grid; weights do not
        int stage = 0;
        uint32_t phase = 0;
        bool have_last = false;
        int last_stage = 0;
        uint32_t last_phase = 0;            // stage / phase of this lane's most recent load (for the drain on abort)
        bool ok = true;
        if (p.win) {
            // one load per (tile, channel chunk): the padded rows of the band, requested by the lane that owns the stage
            for (int tile = worker; ok && opnd == 0 && tile < total_tiles; tile += n_workers) {
                const int m_t = fast_div(tile, p.div_n_tiles);
                const int img = fast_div(m_t, p.div_bands);
                const int y0 = (m_t - img * p.win_bands) * p.win_r;
                for (int cc = 0; cc < p.c_chunks; ++cc) {
                    if (!__all_sync(0xffffffffu, mbar_wait(empty_bar + 8 * stage, phase ^ 1, wc, tagbits | 101))) {
                        ok = false;
                        break;
                    }
                    if (lane == (stage & 31)) {
                        const uint32_t fb = full_bar + 8 * stage;
                        mbar_expect_tx(fb, p.tx_win);
                        tma_load_4d(smem_base + stage * p.stage_bytes, &map_a, fb, cc * p.kb, -1, y0 - 1, img);
                        have_last = true;
                        last_stage = stage;
                        last_phase = phase;
                    }
                    if (++stage == p.stages) { stage = 0; phase ^= 1; }
                }
            }
        } else if (SUP) {
            // one stage use per group of M tiles: sub-chunk j is the activation tile of M tile first + j (a single k-iteration
            // per tile; the weights are resident, so the two producer warps share the sub-chunks as usual)
            for (int tile = worker; ok && tile < total_tiles; tile += n_workers) {
                if (!__all_sync(0xffffffffu, mbar_wait(empty_bar + 8 * stage, phase ^ 1, wc, tagbits | 101))) {
                    ok = false;
                    break;
                }
                const int first_m = tile * p.sup;
                const int subs = min(p.sup, p.m_tiles - first_m);
                const uint32_t fb = full_bar + 8 * stage;
                if (lane == 0) {
                    const uint32_t bytes = (uint32_t)(opnd == 0 ? (subs + 1) >> 1 : subs >> 1) * p.tx_a;
                    if (bytes) mbar_expect_tx(fb, bytes);
                    else mbar_arrive(fb);
                }
                __syncwarp();
                const int j = (lane - stage * p.sup) & 31;
                if (j < subs && (j & 1) == opnd) {
                    const int m0 = (first_m + j) * TILE_M;
                    const uint32_t dst = smem_base + stage * p.stage_bytes + j * p.a_bytes;
                    if (p.a_plain) {
                        tma_load_2d(dst, &map_a, fb, 0, m0);
                    } else {
                        const int t1 = fast_div(m0, p.div_wo);
                        const int ow = m0 - t1 * p.wo;
                        const int img = fast_div(t1, p.div_ho);
                        const int oh = t1 - img * p.ho;
                        tma_load_im2col(dst, &map_a, fb, 0, ow * p.stride_w - p.pad_w, oh * p.stride_h - p.pad_h, img, 0, 0);
                    }
                    have_last = true;
                    last_stage = stage;
                    last_phase = phase;
                }
                if (++stage == p.stages) { stage = 0; phase ^= 1; }
            }
        } else if (p.rowt)
        // small tensors: the same pipeline, but a tile is win_r whole output rows of one image and every filter tap is a
        // tiled load whose box starts at the tap's offset (out-of-image elements are zero filled)
        for (int tile = worker; ok && tile < total_tiles; tile += n_workers) {
            const int m_q = fast_div(tile, p.div_n_tiles), n_t = tile - m_q * p.n_tiles;
            const int m_t = PAIR ? 2 * m_q + (int)cta_rank : m_q;
            const int m0 = m_t * TILE_M;
            // output rows y0 .. y0 + win_r - 1; tap (r, s) starts at input (s - pad, y0 * stride + r - pad)
            const int img = fast_div(m_t, p.div_bands);
            const int base_w = -p.pad_w;
            const int base_h = (m_t - img * p.win_bands) * p.win_r * p.stride_h - p.pad_h;
            const int n_base = n_t * p.bn;
            for (int kc = 0; kc < k_iters; kc += p.group, ++use_idx) {
                if (p.alt && (use_idx & 1) != half) {
                    // the other pair's use.  This warp waits only for the stages of its own uses, and the single,
                    // in-order MMA issuer cannot pass one of those without it: it never falls a barrier phase behind.
                    if (++stage == p.stages) { stage = 0; phase ^= 1; }
                    continue;
                }
                if (!__all_sync(0xffffffffu, mbar_wait(empty_bar + 8 * stage, phase ^ 1, wc, tagbits | 101))) {
                    ok = false;
                    break;
                }
                const int subs = min(p.group, k_iters - kc);
                const uint32_t fb = full_bar + 8 * stage;
                // Two arrivals per stage use, one from each producer warp, and each announces the bytes of its own loads
                // BEFORE it issues them: the barrier's byte count never runs ahead of what has been announced, and both
                // warps are needed for every use, so neither can fall a barrier phase behind the pipeline (a parity wait
                // cannot tell a phase from the one two later).  A helper without a load in this use just arrives.
                if (lane == 0) {
                    uint32_t bytes;
                    if (opnd == 0) bytes = (uint32_t)(p.b_res ? (subs + 1) >> 1 : subs) * p.tx_a;
                    else bytes = p.b_res ? (uint32_t)(subs >> 1) * p.tx_a : (uint32_t)subs * p.tx_b;
                    if (bytes) mbar_expect_tx(fb, bytes);
                    else mbar_arrive(fb);
                }
                __syncwarp();
                const int j = (lane - stage * p.group) & 31;
                if (j < subs && (j & j_mask) == j_want) {
                    const uint2 e = ktab[kc + j];       // x: first channel of the chunk, y: tap << 16 | r << 8 | s
                    const uint32_t dst = smem_base + stage * p.stage_bytes + j * p.sub_bytes;
                    if (opnd == 0 || a_helper)
                        tma_load_4d(dst, &map_a, fb, (int)e.x, base_w + (int)(e.y & 0xff), base_h + (int)((e.y >> 8) & 0xff), img);
                    else
                        tma_load_3d(dst + p.a_bytes, &map_b, fb, (int)e.x, (int)(e.y >> 16), n_base);
                    have_last = true;
                    last_stage = stage;
                    last_phase = phase;
                }
                if (++stage == p.stages) { stage = 0; phase ^= 1; }
            }
        }
        else
        for (int tile = worker; ok && tile < total_tiles; tile += n_workers) {
            const int m_q = fast_div(tile, p.div_n_tiles), n_t = tile - m_q * p.n_tiles;
            const int m_t = PAIR ? 2 * m_q + (int)cta_rank : m_q;
            const int m0 = m_t * TILE_M;
            const int t1 = fast_div(m0, p.div_wo);
            const int ow = m0 - t1 * p.wo;
            const int img = fast_div(t1, p.div_ho);
            const int oh = t1 - img * p.ho;
            const int base_w = ow * p.stride_w - p.pad_w;
            const int base_h = oh * p.stride_h - p.pad_h;
            const int n_base = n_t * p.bn;
            for (int kc = 0; kc < k_iters; kc += p.group, ++use_idx) {
                if (p.alt && (use_idx & 1) != half) {
                    // the other pair's use.  This warp waits only for the stages of its own uses, and the single,
                    // in-order MMA issuer cannot pass one of those without it: it never falls a barrier phase behind.
                    if (++stage == p.stages) { stage = 0; phase ^= 1; }
                    continue;
                }
                if (!__all_sync(0xffffffffu, mbar_wait(empty_bar + 8 * stage, phase ^ 1, wc, tagbits | 101))) {
                    ok = false;
                    break;
                }
                const int subs = min(p.group, k_iters - kc);
                const uint32_t fb = full_bar + 8 * stage;
                // Two arrivals per stage use, one from each producer warp, and each announces the bytes of its own loads
                // BEFORE it issues them: the barrier's byte count never runs ahead of what has been announced, and both
                // warps are needed for every use, so neither can fall a barrier phase behind the pipeline (a parity wait
                // cannot tell a phase from the one two later).  A helper without a load in this use just arrives.
                // (A pair has one barrier per stage, in its even CTA: the even CTA's warps announce the bytes of both CTAs,
                // the odd CTA's loads complete there without an arrival of their own.)
                if (lane == 0 && (!PAIR || cta_rank == 0)) {
                    uint32_t bytes;
                    if (opnd == 0) bytes = (uint32_t)(p.b_res ? (subs + 1) >> 1 : subs) * p.tx_a;
                    else bytes = p.b_res ? (uint32_t)(subs >> 1) * p.tx_a : (uint32_t)subs * p.tx_b;
                    if (PAIR) bytes *= 2;
                    if (bytes) mbar_expect_tx(fb, bytes);
                    else mbar_arrive(fb);
                }
                __syncwarp();
                const int j = (lane - stage * p.group) & 31;
                if (j < subs && (j & j_mask) == j_want) {
                    const uint2 e = ktab[kc + j];       // x: first channel of the chunk, y: tap << 16 | r << 8 | s
                    const uint32_t dst = smem_base + stage * p.stage_bytes + j * p.sub_bytes;
                    if (PAIR) {
                        // this CTA's 128 rows of activations, its half of the weight tile; completion on the even CTA's barrier
                        if (opnd == 0 && p.a_plain)
                            tma_load_2d_pair(dst, &map_a, fb, (int)e.x, m0);
                        else if (opnd == 0)
                            tma_load_im2col_pair(dst, &map_a, fb, (int)e.x, base_w, base_h, img, (uint16_t)(e.y & 0xff),
                                                 (uint16_t)((e.y >> 8) & 0xff));
                        else
                            tma_load_3d_pair(dst + p.a_bytes, &map_b, fb, (int)e.x, (int)(e.y >> 16),
                                             n_base + (int)cta_rank * (p.bn >> 1));
                    } else if ((opnd == 0 || a_helper) && p.a_plain)
                        tma_load_2d(dst, &map_a, fb, (int)e.x, m0);
                    else if (opnd == 0 || a_helper)
                        tma_load_im2col(dst, &map_a, fb, (int)e.x, base_w, base_h, img, (uint16_t)(e.y & 0xff),
                                        (uint16_t)((e.y >> 8) & 0xff));
                    else
                        tma_load_3d(dst + p.a_bytes, &map_b, fb, (int)e.x, (int)(e.y >> 16), n_base);
                    have_last = true;
                    last_stage = stage;
                    last_phase = phase;
                }
                if (++stage == p.stages) { stage = 0; phase ^= 1; }
            }
        }
        if (!ok && have_last) {
            // Drain: loads of one thread are served in order, so waiting (bounded) for the most recent one
            // covers everything this lane has in flight before the CTA's shared memory goes away.
            const unsigned long long t0 = clock64();
            while (!mbar_try_wait(full_bar + 8 * last_stage, last_phase) &&
                   (unsigned long long)(clock64() - t0) < DRAIN_LIMIT_CYCLES) {
            }
        }
        // the resident weights must have landed before this CTA's shared memory may go away (they have, unless
        // the kernel is aborting: the MMA issuers wait for them before their first instruction)
        if (a_helper) mbar_wait(bres_bar, 0, wc, tagbits | 110);
        }
    } else if (warp == MMA_WARP || warp == MMA2_WARP) {
        // ------------------------------------------------------------------ MMA issuers
        // With two issuers, issuer q takes the CTA's tiles with (local & 1) == q, i.e. accumulator q, and steps
        // over the stage uses of the other issuer's tiles.  A parity wait can only tell a phase from its
        // neighbour, so an issuer must never wait on a stage whose previous use has not been filled yet: the
        // plan enables the second issuer only when stages >= 2 * uses per tile, which guarantees that (the
        // previous use of the stage then belongs to a tile this issuer, or the other one before it, is done with).
        const int q_issuer = warp == MMA_WARP ? 0 : 1;
        if (PAIR && cta_rank != 0) {
            // The odd CTA of a pair issues nothing; the commits of the even CTA's issuer arrive on its barriers too.  Before
            // the CTA may go, the arrivals that free its last stage uses must have landed (see below).
            if (lane == 0 && q_issuer == 0) {
                int local = 0;
                for (int tile = worker; tile < total_tiles; tile += n_workers) ++local;
                const int total_uses = local * p.uses;
                for (int g = max(0, total_uses - p.stages); g < total_uses; ++g)
                    mbar_wait(empty_bar + 8 * (g % p.stages), (uint32_t)(g / p.stages) & 1u, wc, tagbits | 113);
            }
        } else if (lane == 0 && (q_issuer == 0 || p.dual_issue)) {
            int stage = 0;
            uint32_t phase = 0;
            int local = 0;
            bool ok = true;
            bool committed_any = false;
            int last_acc = 0;
            uint32_t last_acc_phase = 0;
            // descriptor words: the low one holds the start address (16-byte units, 14 bits) and LBO
            const uint32_t desc_lo0 = (uint32_t)p.desc_hi | ((smem_base & 0x3ffffu) >> 4);
            const uint32_t desc_hi32 = (uint32_t)(p.desc_hi >> 32);
            uint32_t stage_lo = desc_lo0;
            const uint32_t stage16 = p.stage_bytes >> 4, sub16 = p.sub_bytes >> 4, a16 = p.a_bytes >> 4;
            const uint32_t b16 = p.b_bytes >> 4, bres_lo = desc_lo0 + (p.bres_off >> 4);
            const uint32_t b_step = p.b_res ? b16 : sub16;
            if (p.b_res && !mbar_wait(bres_bar, 0, wc, tagbits | 111)) ok = false;
            const int mmas = p.kb >> 5;      // 1, 2 or 4 instructions per stage
            for (int tile = worker; ok && tile < total_tiles; tile += n_workers, ++local) {
                const int acc = local & 1;
                if (p.dual_issue && acc != q_issuer) {
                    // the other issuer's tile: step over its stage uses
                    stage += p.uses;
                    while (stage >= p.stages) { stage -= p.stages; phase ^= 1; }
                    stage_lo = desc_lo0 + (uint32_t)stage * stage16;
                    continue;
                }
                const uint32_t acc_phase = (local >> 1) & 1;
                if (!mbar_wait(tempty_bar + 8 * acc, acc_phase ^ 1, wc, tagbits | 102)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * 256;   // two 256-column accumulators
                uint32_t b_tile_lo = 0;
                if (p.b_res) {
                    const int n_t = tile - fast_div(tile, p.div_n_tiles) * p.n_tiles;
                    b_tile_lo = bres_lo + (uint32_t)(n_t * k_iters) * b16;
                }
                if (SUP) {
                    // one stage use: the activation tiles of up to p.sup M tiles, each accumulated (a single k-iteration) into
                    // its own column range of this accumulator
                    if (!mbar_wait(full_bar + 8 * stage, phase, wc, tagbits | 103)) { ok = false; break; }
                    tc_fence_after();
                    const int subs = min(p.sup, p.m_tiles - tile * p.sup);
                    uint32_t a_lo = stage_lo;
                    for (int j = 0; j < subs; ++j, a_lo += a16) {
                        const uint32_t d_sub = d_tmem + (uint32_t)(j * p.bn);
                        if (mmas == 4) mma_i8_sub<4>(d_sub, a_lo, b_tile_lo, desc_hi32, p.idesc, 0u);
                        else if (mmas == 2) mma_i8_sub<2>(d_sub, a_lo, b_tile_lo, desc_hi32, p.idesc, 0u);
                        else mma_i8_sub<1>(d_sub, a_lo, b_tile_lo, desc_hi32, p.idesc, 0u);
                    }
                    mma_commit(empty_bar + 8 * stage);
                    stage_lo += stage16;
                    if (++stage == p.stages) { stage = 0; phase ^= 1; stage_lo = desc_lo0; }
                } else if (p.win) {
                    // one stage use per channel chunk; the nine taps read the same tile at shifted row offsets
                    const uint32_t kb16 = (uint32_t)p.kb >> 4;
                    for (int cc = 0; cc < p.c_chunks; ++cc) {
                        if (!mbar_wait(full_bar + 8 * stage, phase, wc, tagbits | 103)) { ok = false; break; }
                        tc_fence_after();
                        uint32_t first = cc != 0 ? 1u : 0u;
                        uint32_t b_lo = b_tile_lo + (uint32_t)cc * b16;
                        for (int r = 0; r < 3; ++r) {
                            uint32_t a_lo = stage_lo + (uint32_t)(r * p.win_wp) * kb16;
                            for (int sx = 0; sx < 3; ++sx) {
                                if (mmas == 4) mma_i8_sub<4>(d_tmem, a_lo, b_lo, desc_hi32, p.idesc, first);
                                else if (mmas == 2) mma_i8_sub<2>(d_tmem, a_lo, b_lo, desc_hi32, p.idesc, first);
                                else mma_i8_sub<1>(d_tmem, a_lo, b_lo, desc_hi32, p.idesc, first);
                                first = 1u;
                                a_lo += kb16;
                                b_lo += (uint32_t)p.c_chunks * b16;
                            }
                        }
                        mma_commit(empty_bar + 8 * stage);
                        stage_lo += stage16;
                        if (++stage == p.stages) { stage = 0; phase ^= 1; stage_lo = desc_lo0; }
                    }
                } else
                for (int kc = 0; kc < k_iters; kc += p.group) {
                    if (!mbar_wait(full_bar + 8 * stage, phase, wc, tagbits | 103)) { ok = false; break; }
                    tc_fence_after();
                    const int subs = min(p.group, k_iters - kc);
                    const uint32_t first = kc != 0 ? 1u : 0u;      // the tile's first MMA overwrites the accumulator
                    const uint32_t b_lo = p.b_res ? b_tile_lo + (uint32_t)kc * b16 : stage_lo + a16;
                    if (PAIR) {
                        // 256-row instructions over both CTAs' tiles (128-byte K chunks only); the commit frees the stage in both
                        uint32_t a_lo = stage_lo, bb_lo = b_lo;
                        for (int j = 0; j < subs; ++j, a_lo += sub16, bb_lo += b_step)
                            mma_i8_sub_pair4(d_tmem, a_lo, bb_lo, desc_hi32, p.idesc, j == 0 ? first : 1u);
                        mma_commit_pair(empty_bar + 8 * stage);
                    } else {
                    if (mmas == 4) mma_i8_stage<4>(d_tmem, stage_lo, b_lo, sub16, b_step, desc_hi32, p.idesc, subs, first);
                    else if (mmas == 2) mma_i8_stage<2>(d_tmem, stage_lo, b_lo, sub16, b_step, desc_hi32, p.idesc, subs, first);
                    else mma_i8_stage<1>(d_tmem, stage_lo, b_lo, sub16, b_step, desc_hi32, p.idesc, subs, first);
                    mma_commit(empty_bar + 8 * stage);    // frees the stage when these MMAs have read it
                    }
                    stage_lo += stage16;
                    if (++stage == p.stages) { stage = 0; phase ^= 1; stage_lo = desc_lo0; }
                }
                if (!ok) break;
                if (PAIR) mma_commit_pair(tfull_bar + 8 * acc);      // both CTAs' halves of the accumulator are complete
                else mma_commit(tfull_bar + 8 * acc);          // accumulator complete
                committed_any = true;
                last_acc = acc;
                last_acc_phase = acc_phase;
            }
            if (ok && local > 0) {
                // The commits that free the last stage uses arrive on barriers nobody waits for any more (the producers
                // are done).  Such an arrival must not land after this CTA has gone: the next kernel's CTA takes over
                // the SM at once and keeps its own barriers at the same shared-memory addresses.  So every issuer waits
                // for the last arrival on each stage that came from one of its own tiles.
                const int uses_tile = p.win ? p.c_chunks : p.uses;      // (p.sup: one use per group of M tiles, p.uses == 1)
                const int total_uses = local * uses_tile;
                for (int g = max(0, total_uses - p.stages); g < total_uses; ++g) {
                    const int t_of_g = g / uses_tile;
                    if (p.dual_issue && (t_of_g & 1) != q_issuer) continue;
                    mbar_wait(empty_bar + 8 * (g % p.stages), (uint32_t)(g / p.stages) & 1u, wc, tagbits | 112);
                }
            }
            if (!ok && committed_any) {
                // let the tensor pipe finish what was issued before TMEM is released
                const unsigned long long t0 = clock64();
                while (!mbar_try_wait(tfull_bar + 8 * last_acc, last_acc_phase) &&
                       (unsigned long long)(clock64() - t0) < DRAIN_LIMIT_CYCLES) {
                }
            }
        }
    } else if (warp == MOVER_WARP) {
        // ------------------------------------------------------------------ output mover
        if (STAGED && lane == 0) {
            grid_dependency_wait();     // the output may overwrite a tensor the previous grid still reads
            // stores: a tile leaves from its buffer of the ring once all epilogue warps have written it
            int b = 0;
            uint32_t bphase = 0;
            for (int tile = worker; tile < total_tiles; tile += n_workers) {
                const int m_q = fast_div(tile, p.div_n_tiles), n_t = tile - m_q * p.n_tiles;
            const int m_t = PAIR ? 2 * m_q + (int)cta_rank : m_q;
                if (!mbar_wait(out_full + 8 * b, bphase, wc, tagbits | 108)) break;
                const uint32_t src = smem_base + p.out_off + b * p.out_bytes;
                if (SUP) {
                    // column slab sl of the staged tile is M tile tile * sup + sl
                    const int subs = min(p.sup, p.m_tiles - tile * p.sup);
                    for (int sl = 0; sl < subs; ++sl)
                        tma_store_2d(&map_y, src + sl * (TILE_M * p.slab_w), 0, (tile * p.sup + sl) * TILE_M);
                } else if (p.rows) {
                    const int img = fast_div(m_t, p.div_bands);
                    const int y0 = (m_t - img * p.win_bands) * p.win_r;
                    // positions W and W + 1 of every row and rows below the image are clipped by the hardware
                    for (int sl = 0; sl < p.n_slabs; ++sl)
                        if (n_t * p.bn + sl * p.slab_w < p.c_out)
                            tma_store_4d(&map_y, src + sl * (TILE_M * p.slab_w), n_t * p.bn + sl * p.slab_w, 0, y0, img);
                } else
                for (int sl = 0; sl < p.n_slabs; ++sl)
                    if (n_t * p.bn + sl * p.slab_w < p.c_out)
                        tma_store_2d(&map_y, src + sl * (TILE_M * p.slab_w), n_t * p.bn + sl * p.slab_w, m_t * TILE_M);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                // the buffer is free again as soon as the store has read it (the next tiles use the others)
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                mbar_arrive(out_free + 8 * b);
                if (++b == p.out_bufs) { b = 0; bphase ^= 1; }
            }
            asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        }
    } else if (warp == FETCH_WARP) {
        // ------------------------------------------------------------------ residual fetcher
        if (RES && lane == 0) {
            grid_dependency_wait();
            // residual tiles go straight into the output ring (the epilogue converts them in place): a buffer is
            // loaded as soon as the store of the tile that used it before has read it, up to out_bufs - 1 tiles ahead
            int local = 0;
            int rb = 0;
            uint32_t rphase = 0;
            bool ok = true;
            for (int tile = worker; tile < total_tiles; tile += n_workers, ++local) {
                const int m_q = fast_div(tile, p.div_n_tiles), n_t = tile - m_q * p.n_tiles;
            const int m_t = PAIR ? 2 * m_q + (int)cta_rank : m_q;
                if (!mbar_wait(out_free + 8 * rb, rphase ^ 1, wc, tagbits | 106)) { ok = false; break; }
                const uint32_t fb = res_full + 8 * rb;
                mbar_expect_tx(fb, p.tx_res);
                if (p.rows) {
                    const int img = fast_div(m_t, p.div_bands);
                    const int y0 = (m_t - img * p.win_bands) * p.win_r;
                    for (int sl = 0; sl < p.n_slabs; ++sl)
                        tma_load_4d(smem_base + p.out_off + rb * p.out_bytes + sl * (TILE_M * p.slab_w), &map_r, fb,
                                    n_t * p.bn + sl * p.slab_w, 0, y0, img);
                } else
                for (int sl = 0; sl < p.n_slabs; ++sl)
                    tma_load_2d(smem_base + p.out_off + rb * p.out_bytes + sl * (TILE_M * p.slab_w), &map_r, fb,
                                n_t * p.bn + sl * p.slab_w, m_t * TILE_M);
                if (++rb == p.out_bufs) { rb = 0; rphase ^= 1; }
            }
            if (!ok && local > 0) {
                // aborting: give the loads that are still in flight time to land (walk back over the ring)
                for (int i = 0; i < p.out_bufs && local - 1 - i >= 0; ++i) {
                    const int l = local - 1 - i;
                    const unsigned long long t0 = clock64();
                    while (!mbar_try_wait(res_full + 8 * (l % p.out_bufs), (uint32_t)(l / p.out_bufs) & 1u) &&
                           (unsigned long long)(clock64() - t0) < DRAIN_LIMIT_CYCLES) {
                    }
                }
            }
        }
    } else if (warp >= FIRST_EPI_WARP && warp < FIRST_EPI_WARP + NUM_EPI_WARPS) {
        // ------------------------------------------------------------------ epilogue warps
        const int quarter = warp & 3;               // TMEM lanes 32*quarter .. +31 belong to this warp
        const int ew = warp - FIRST_EPI_WARP;
        const int group = ew >> 2;                  // which quarter of the tile's columns this warp converts
        const int chunks = (SUP ? p.sup * p.bn : p.bn) / 16;
        const int per_group = (chunks + p.epi_groups - 1) / p.epi_groups;     // <= 4 chunks of 16 columns per warp
        const int ch_begin = min(group * per_group, chunks);
        const int nch = min(ch_begin + per_group, chunks) - ch_begin;
        const int mul_acc = p.mul_acc, mul_res = p.mul_res;     // 2^sh_acc, 2^sh_res
        int local = 0;
        int ob = 0;                 // buffer of the output ring for the current tile and the parity of its use
        uint32_t ophase = 0;
        bool ok = true;
        if (STAGED) {
            {
                // bias' = (bias << sh_acc) + 2^(s-1) for every (padded) output column, once per CTA.  Only these warps
                // read the table, so they build it -- behind a barrier of their own -- while the producers and the MMA
                // issuers are already at work: the prologue of a CTA starts when the previous layer's CTA has left the SM,
                // and a round trip to global memory there would be paid by every layer.
                int *bias_all = (int *)(smem + p.bias_off);
                const int rnd = 1 << (p.q.s - 1);
                for (int i = (int)threadIdx.x - FIRST_EPI_WARP * 32; i < p.n_tiles * p.bn; i += NUM_EPI_WARPS * 32)
                    bias_all[i] = ((i < p.c_out && p.bias) ? (__ldg(p.bias + i) << p.q.sh_acc) : 0) + rnd;
                asm volatile("bar.sync 1, %0;" ::"n"(NUM_EPI_WARPS * 32) : "memory");
            }
            const int tile_row = quarter * 32 + lane;
            const int sup_sub = SUP ? (ch_begin * 16) / p.bn : 0, sup_col0 = ch_begin * 16 - sup_sub * p.bn;
            // Narrow tiles are converted by fewer warps: the MMA-issuing threads share their scheduler partitions with the
            // epilogue warps, and every warp that is ready to issue slows them down.
            const int my_tiles_end = group < p.epi_groups ? total_tiles : 0;
            // PRMT selectors that turn byte k of a residual word into an int (zero- or sign-extended)
            uint32_t rsel[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) rsel[k] = p.q.r_signed ? (0x8880u | (0x1111u * k)) : (0x4440u | k);
            // where this thread's 16-byte chunks live inside a staged tile (same for every tile)
            uint32_t so[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int ch = ch_begin + i;
                uint32_t off = (uint32_t)tile_row * p.slab_w + (ch % p.slab_chunks) * 16;
                off ^= ((off >> 7) & p.swz_mask) << 4;
                so[i] = (uint32_t)(ch / p.slab_chunks) * (TILE_M * p.slab_w) + off;
            }
            for (int tile = worker; tile < my_tiles_end; tile += n_workers, ++local) {
                const int acc = local & 1;                   // accumulator, output buffer and residual buffer in use
                const uint32_t acc_phase = (local >> 1) & 1;
                const int n_t = tile - fast_div(tile, p.div_n_tiles) * p.n_tiles;
                int c_first = n_t * p.bn + ch_begin * 16;
                int my_nch = min(nch, max(0, (p.c_out - c_first) / 16));      // chunks that exist in c_out
                if (SUP) {
                    // this warp's chunks lie in M tile sup_sub of the group (a chunk range never straddles two of them)
                    c_first = sup_col0;
                    my_nch = sup_sub < min(p.sup, p.m_tiles - tile * p.sup) ? min(nch, max(0, (p.c_out - c_first) / 16)) : 0;
                }
                const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * 256 + ch_begin * 16;
                // The buffer first (it holds the residual tile, which implies that its previous store has left, or it is
                // free): that wait is over long before the accumulator is complete, so it costs the chain accumulator ->
                // epilogue -> accumulator nothing.
                bool got;
                if (RES) got = mbar_wait(res_full + 8 * ob, ophase, wc, tagbits | 107);
                else got = mbar_wait(out_free + 8 * ob, ophase ^ 1, wc, tagbits | 109);
                got = mbar_wait(tfull_bar + 8 * acc, acc_phase, wc, tagbits | 104) && got;
                if (!__all_sync(0xffffffffu, got)) { ok = false; break; }
                tc_fence_after();
                const uint32_t out_buf = smem_base + p.out_off + ob * p.out_bytes;
                const uint32_t res_buf = out_buf;       // in place: a thread reads and then overwrites its own 16 bytes
                const uint32_t bias_s = smem_base + p.bias_off + 4 * c_first;
                // The accumulator goes back to the MMA issuer as soon as this warp's last load from it has completed -- before
                // the last chunk is converted and written.
                auto release_acc = [&]() {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        if (PAIR && cta_rank != 0) mbar_arrive_cluster(tempty_bar + 8 * acc, 0);     // the issuer's barrier
                        else mbar_arrive(tempty_bar + 8 * acc);
                    }
                };
                int va[16], vb[16];
                if (my_nch > 0) tmem_ld16(t_addr, va);
                else release_acc();
#pragma unroll
                for (int i = 0; i < 4; i += 2) {
                    if (i < my_nch) {
                        uint4 rw = make_uint4(0, 0, 0, 0);
                        if (RES) rw = lds128(res_buf + so[i]);
                        tmem_ld_wait();
                        if (i + 1 < my_nch) tmem_ld16(t_addr + (i + 1) * 16, vb);
                        else release_acc();
                        sts128(out_buf + so[i], epilogue_fast16<RES, SGN>(va, bias_s + 64 * (i), rw, mul_acc, mul_res, rsel, p.q.s));
                    }
                    if (i + 1 < my_nch) {
                        uint4 rw = make_uint4(0, 0, 0, 0);
                        if (RES) rw = lds128(res_buf + so[i + 1]);
                        tmem_ld_wait();
                        if (i + 2 < my_nch) tmem_ld16(t_addr + (i + 2) * 16, va);
                        else release_acc();
                        sts128(out_buf + so[i + 1], epilogue_fast16<RES, SGN>(vb, bias_s + 64 * (i + 1), rw, mul_acc, mul_res, rsel, p.q.s));
                    }
                }
                // the output part is written: make the writes visible to the TMA and tell the mover (and, through it, the
                // fetcher)
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(out_full + 8 * ob);
                if (++ob == p.out_bufs) { ob = 0; ophase ^= 1; }
            }
        } else {
            grid_dependency_wait();     // direct stores (and residual reads) from these warps
            const int tile_row = quarter * 32 + lane;   // this thread's row of the tile
            for (int tile = worker; ok && tile < total_tiles; tile += n_workers, ++local) {
                const int acc = local & 1;
                const uint32_t acc_phase = (local >> 1) & 1;
                const int m_q = fast_div(tile, p.div_n_tiles), n_t = tile - m_q * p.n_tiles;
            const int m_t = PAIR ? 2 * m_q + (int)cta_rank : m_q;
                const int n0 = n_t * p.bn;
                size_t row = (size_t)m_t * TILE_M + tile_row;
                bool row_valid = row < (size_t)p.M;
                if (p.rows) {
                    // row-tiled geometry: tile row -> (row of the band, position in the row) -> output pixel
                    const int img = fast_div(m_t, p.div_bands);
                    const int y0 = (m_t - img * p.win_bands) * p.win_r;
                    const int ry = tile_row / p.win_wp, rx = tile_row - ry * p.win_wp;
                    row_valid = ry < p.win_r && y0 + ry < p.ho && rx < p.wo;
                    row = ((size_t)img * p.ho + (size_t)(y0 + ry)) * p.wo + rx;
                }
                const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * 256 + ch_begin * 16;
                if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar + 8 * acc, acc_phase, wc, tagbits | 104))) { ok = false; break; }
                tc_fence_after();
                for (int i = 0; i < nch; ++i) {
                    const int co0 = n0 + (ch_begin + i) * 16;
                    if (co0 >= p.c_out) break;                   // uniform across the warp
                    int v[16];
                    tmem_ld16(t_addr + i * 16, v);
                    tmem_ld_wait();
                    epilogue_chunk(p, v, row, co0, row_valid);
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(tempty_bar + 8 * acc);
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    // a pair leaves together: the issuer's instructions read the partner's shared memory and tensor memory, and arrivals
    // go to the partner's barriers
    if (PAIR) cluster_sync_all();
    if (warp == MMA_WARP) {
        tc_fence_after();
        if (PAIR) tmem_dealloc_pair(tmem_base, TMEM_COLS);
        else tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ----------------------------------------------------------------------------- MMA-only probe

__global__ void __launch_bounds__(NUM_THREADS, 1) f8_mma_probe_kernel(int iters, int *status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // 128 x 128 A and 256 x 128 B int8 tiles; the values do not matter for a rate measurement
    for (int i = threadIdx.x; i < (128 + 256) * 128 / 4; i += blockDim.x) ((uint32_t *)smem)[i] = 0x01010101u * (i & 3);
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == MMA_WARP) tmem_alloc(smem_u32(&tmem_base_slot), TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    if (warp == MMA_WARP && lane == 0) {
        const uint32_t a_addr = smem_u32(smem), b_addr = a_addr + 128 * 128;
        const uint64_t hi = smem_desc_hi(128);
        const uint64_t a_desc = hi | (uint64_t)((a_addr & 0x3ffffu) >> 4);
        const uint64_t b_desc = hi | (uint64_t)((b_addr & 0x3ffffu) >> 4);
        // u8 x s8 -> s32, M 128, N 256
        const uint32_t idesc = (2u << 4) | (0u << 7) | (1u << 10) | ((256u >> 3) << 17) | ((128u >> 4) << 24);
        for (int i = 0; i < iters; ++i)
            mma_i8(tmem_base + (i & 1) * 256, a_desc + 2 * (i & 3), b_desc + 2 * (i & 3), idesc, i > 1 ? 1u : 0u);
        mma_commit(smem_u32(&bar));
        mbar_wait(smem_u32(&bar), 0, make_wait_ctx(&abort_flag, status, 0), 105);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == MMA_WARP) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ----------------------------------------------------------------------------- time-out probe

// The time-out path of the bounded waits, exercised without harming anything: a barrier with one expected arrival that
// nobody makes.  The wait gives up after `limit_cycles`, records itself in the status word and the kernel returns.
__global__ void __launch_bounds__(32, 1) f8_wait_probe_kernel(unsigned long long limit_cycles, int *status) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_wait(smem_u32(&bar), 0, make_wait_ctx(&abort_flag, status, limit_cycles), 199);
    }
}

// ----------------------------------------------------------------------------- host side

PFN_cuTensorMapEncodeTiled_v12000 g_encode_tiled = nullptr;
PFN_cuTensorMapEncodeIm2col_v12000 g_encode_im2col = nullptr;

bool load_driver_entry_points() {
    if (g_encode_tiled && g_encode_im2col) return true;
    void *f = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &qr) != cudaSuccess || !f ||
        qr != cudaDriverEntryPointSuccess)
        return false;
    g_encode_tiled = (PFN_cuTensorMapEncodeTiled_v12000)f;
    f = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &f, cudaEnableDefault, &qr) != cudaSuccess || !f ||
        qr != cudaDriverEntryPointSuccess)
        return false;
    g_encode_im2col = (PFN_cuTensorMapEncodeIm2col_v12000)f;
    return true;
}

FastDiv make_fast_div(int d) {
    uint32_t l = 0;
    while ((1u << l) < (uint32_t)d) ++l;
    FastDiv f;
    f.shift = 31 + l;
    f.mul = (uint32_t)(((uint64_t)1 << f.shift) / (uint32_t)d + 1);
    return f;
}

int choose_kb(int c) { return c >= 96 ? 128 : (c >= 48 ? 64 : 32); }

int choose_bn(int c_out) {
    if (c_out >= 256) return 256;
    return (c_out + 15) / 16 * 16;
}

// N tile of the staged epilogue: a power of two up to 128, or 256 (two 128-byte slabs) when no residual
// buffers are needed; the TMA store clips columns beyond c_out.
int choose_bn_staged(int c_out, bool has_res, int kb) {
    // with a residual the four staging tiles of a 256-wide tile leave room for the pipeline only when
    // the K chunks are 64 bytes or less
    if (c_out > 128 && (!has_res || kb <= 64)) return 256;
    int bn = 16;
    while (bn < c_out && bn < 128) bn *= 2;
    return bn;
}

CUtensorMapSwizzle swizzle_for(int kb) {
    return kb == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : (kb == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
}

}   // namespace

struct F8TcPlan {
    CUtensorMap map_a;
    CUtensorMap map_b;
    CUtensorMap map_y;
    CUtensorMap map_r;
    TcParams p;
    int grid;
    size_t smem;
};

size_t f8_tc_plan_size() { return sizeof(F8TcPlan); }
void f8_tc_plan_set_tag(F8TcPlan *plan, int tag) { plan->p.tag = tag; }

// Whole output rows fit a tile and the boxes of a tap stay inside the limits of a tiled tensor map.
bool f8_tc_rowtile_ok(const F8ConvGeom &g) {
    if (g.wo > TILE_M || g.pad_h_end >= 0) return false;
    const int r = std::min(TILE_M / g.wo, g.ho);
    return g.wo * g.stride_w <= 256 && r * g.stride_h <= 256 && g.stride_w <= 8 && g.stride_h <= 8;
}

bool f8_tc_supported(const F8ConvGeom &g, size_t x_bytes) {
    if (g.c % 16 != 0) return false;                 // TMA strides are multiples of 16 bytes
    // im2col tensor maps of tensors below 128 KiB are avoided.  A pointwise layer (1x1, stride 1, no padding) needs no
    // im2col: its activations are a plain [pixels, channels] matrix read through a tiled map, whatever their size;
    // other layers on small tensors take whole output rows per tile and one tiled load per filter tap; what fits
    // neither goes to the CUDA-core kernel.
    const bool pointwise = g.kh == 1 && g.kw == 1 && g.stride_h == 1 && g.stride_w == 1 && g.pad_h == 0 && g.pad_w == 0;
    if (x_bytes < 4096) return false;
    if (x_bytes < 128 * 1024 && !pointwise && !f8_tc_rowtile_ok(g)) return false;
    if (g.kh > 255 || g.kw > 255) return false;
    if ((long long)g.n * g.ho * g.wo > 0x7fffff00ll) return false;
    return true;
}

cudaError_t f8_tc_plan_init(F8TcPlan *plan, const F8ConvGeom &g, const F8Requant &q, const F8TcTensorView &xv,
                            const int8_t *w, const int32_t *bias, const void *res, void *y, int *status_word,
                            const char **why, const F8Sibling *sib) {
    *why = "";
    if (!load_driver_entry_points()) {
        *why = "cuTensorMapEncode entry points not available";
        return cudaErrorNotSupported;
    }
    memset(plan, 0, sizeof(*plan));
    TcParams &p = plan->p;
    p.epi_groups = 4;
    p.M = g.n * g.ho * g.wo;
    p.ho = g.ho;
    p.wo = g.wo;
    p.c_out = g.c_out;
    p.kh = g.kh;
    p.kw = g.kw;
    p.stride_h = g.stride_h;
    p.stride_w = g.stride_w;
    p.pad_h = g.pad_h;
    p.pad_w = g.pad_w;
    p.kb = choose_kb(g.c);
    // residual layers are bound by the epilogue, not by the main loop: prefer 64-byte K chunks so that a
    // 256-wide tile (half the tiles, half the A re-reads) still leaves room for the pipeline stages
    // (not the K-heavy ones -- a 3x3 layer with a shortcut, as in basic residual blocks: those keep 128-byte chunks and
    // 256-wide tiles, which makes them CTA pairs; the three 32-KiB buffers of the output ring leave three 32-KiB stages)
    const bool k_heavy_res = q.has_res && g.c % 128 == 0 && g.c_out % 256 == 0 && g.kh * g.kw * (g.c / 128) >= 8;
    if (q.has_res && g.c_out > 128 && p.kb == 128 && g.c <= 256 && !k_heavy_res) p.kb = 64;
    p.c_chunks = (g.c + p.kb - 1) / p.kb;
    p.epi = EPI_GENERIC;
    const bool has_sib = sib && sib->y2;
    if ((q.y_kind == F8_U8 || q.y_kind == F8_S8) && q.s >= 1 && q.s <= 24 && g.c_out % 16 == 0 && !has_sib && !q.r_s32)
        p.epi = q.y_kind == F8_U8 ? (q.has_res ? EPI_U8_RES : EPI_U8) : (q.has_res ? EPI_S8_RES : EPI_S8);
    const bool staged = p.epi != EPI_GENERIC;
    p.bn = staged ? (k_heavy_res ? 256 : choose_bn_staged(g.c_out, q.has_res != 0, p.kb)) : choose_bn(g.c_out);
    p.m_tiles = (p.M + TILE_M - 1) / TILE_M;
    if (!staged) {
        // few output pixels (a fully connected layer): narrower N tiles until every SM has one, the weights are
        // what has to be streamed and each CTA then streams its own slice of them
        int sm_count = 148, dev0 = 0;
        cudaGetDevice(&dev0);
        cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev0);
        while (p.bn > 32 && p.bn % 32 == 0 && (long long)p.m_tiles * ((g.c_out + p.bn - 1) / p.bn) < sm_count) p.bn /= 2;
    }
    p.n_tiles = (g.c_out + p.bn - 1) / p.bn;
    p.div_n_tiles = make_fast_div(p.n_tiles);
    p.div_wo = make_fast_div(g.wo);
    p.div_ho = make_fast_div(g.ho);
    p.a_bytes = (uint32_t)(TILE_M * p.kb + 1023) / 1024 * 1024;
    // CTA pairs for the K-heavy layers with 256-wide tiles, whose main loop is bound by the bytes a CTA has to pull
    // through the L2 -> SM path per tensor-core cycle (48 KiB per 128-byte K chunk alone, 32 KiB in a pair: the weight
    // tile is split between the two CTAs)
    {
        const unsigned off0 = f8_plan_options_off();
        const size_t xb = (size_t)xv.dim_c * xv.dim_w * xv.dim_h * xv.dim_n;
        p.pair = (staged && p.kb == 128 && g.c % 128 == 0 && p.bn == 256 && g.c_out % 256 == 0 &&
                  g.kh * g.kw * ((g.c + p.kb - 1) / p.kb) >= 8 && xb >= 128 * 1024 && p.m_tiles >= 2 && !(off0 & F8_PLAN_OFF_PAIRS)) ? 1 : 0;
    }
    const int bn_load = p.pair ? p.bn / 2 : p.bn;        // rows of a weight tile one CTA loads
    const uint32_t b_bytes = (uint32_t)(bn_load * p.kb + 1023) / 1024 * 1024;
    p.b_bytes = b_bytes;
    p.sub_bytes = p.a_bytes + b_bytes;
    p.tx_a = (uint32_t)(TILE_M * p.kb);
    p.tx_b = (uint32_t)(bn_load * p.kb);
    p.pair_tiles = ((p.m_tiles + 1) / 2) * p.n_tiles;
    size_t staging = 0;
    if (staged) {
        p.slab_w = p.bn < 128 ? p.bn : 128;
        p.slab_chunks = p.slab_w / 16;
        p.n_slabs = p.bn / p.slab_w;
        p.swz_mask = p.slab_w == 128 ? 7u : (p.slab_w == 64 ? 3u : (p.slab_w == 32 ? 1u : 0u));
        p.out_bytes = (uint32_t)(TILE_M * p.bn + 1023) / 1024 * 1024;
        const size_t bias_bytes = ((size_t)p.n_tiles * p.bn * 4 + 1023) / 1024 * 1024;
        // Output ring.  Without a residual two buffers overlap the epilogue of a tile with the store of the one
        // before.  With a residual a buffer goes through load -> convert in place -> store, and a residual tile takes
        // about as long to arrive from HBM as a tile takes to compute: three buffers (four when they are small).
        p.out_bufs = !q.has_res ? 2 : (p.out_bytes <= 16 * 1024 ? 4 : 3);
        // 64-wide tiles: eight epilogue warps (two chunks each) instead of sixteen -- measured, 3x3 64 -> 64 at 56 x 56 61 -> 57 us
        // (one warp per quarter: the same); 128-wide tiles show no difference and keep all sixteen
        p.epi_groups = p.bn <= 64 ? 2 : 4;
        // Groups of M tiles (see TcParams::sup): pointwise layers with one k-iteration, one N tile of at most 128 columns and
        // no residual; enough tiles that every CTA still gets several groups
        p.sup = 0;
        {
            const bool one_k = g.kh == 1 && g.kw == 1 && g.c <= p.kb;
            const int gsz = p.bn <= 64 ? 4 : 2;
            if (one_k && !q.has_res && p.bn <= 128 && g.c_out <= p.bn && g.c_out % 16 == 0 && !p.pair && g.stride_h == 1 &&
                g.stride_w == 1 && g.pad_h == 0 && g.pad_w == 0 && p.m_tiles >= 148 * 4 * gsz &&
                !(f8_plan_options_off() & (F8_PLAN_OFF_TILE_GROUPS | F8_PLAN_OFF_RESIDENT_WEIGHTS))) {
                p.sup = gsz;
                p.sup_tiles = (p.m_tiles + gsz - 1) / gsz;
                p.slab_w = p.bn;
                p.slab_chunks = p.slab_w / 16;
                p.n_slabs = gsz;
                p.swz_mask = p.slab_w == 128 ? 7u : (p.slab_w == 64 ? 3u : (p.slab_w == 32 ? 1u : 0u));
                p.out_bytes = (uint32_t)(TILE_M * p.bn * gsz + 1023) / 1024 * 1024;
                p.out_bufs = 2;
                p.epi_groups = 4;
            }
        }
        staging = (size_t)p.out_bytes * p.out_bufs + bias_bytes;
    }
    const size_t ktab_bytes = ((size_t)g.kh * g.kw * p.c_chunks * 8 + 1023) / 1024 * 1024;
    if (ktab_bytes > 16 * 1024 || g.kh * g.kw > 0xffff) {
        *why = "too many k-iterations for the coordinate table";
        return cudaErrorInvalidValue;
    }
    staging += ktab_bytes;
    // k-iterations per stage: every stage use costs the MMA thread a wait, a fence and a commit (a few hundred
    // cycles of a lone thread, as much as several MMAs), so K chunks are grouped -- as long as two stages and one
    // lane per load remain; measured, fewer and larger stage uses beat a deeper ring of small ones
    const int k_iters = g.kh * g.kw * p.c_chunks;
    size_t avail = SMEM_LIMIT - 1024 - staging;
    // resident weights: one N tile, and room left for at least four activation tiles in flight (with only two, a
    // 3x3 layer of 128 channels waits on every im2col load: measured 62 us against 48 us with streamed weights)
    const size_t b_all = (size_t)p.n_tiles * k_iters * b_bytes;
    const unsigned off = f8_plan_options_off();
    p.b_res = (!p.pair && p.n_tiles == 1 && b_all + 4 * (size_t)p.a_bytes <= avail && b_all + 32 * 1024 <= avail &&
               !(off & F8_PLAN_OFF_RESIDENT_WEIGHTS)) ? 1 : 0;
    if (p.b_res) {
        avail -= b_all;
        p.sub_bytes = p.a_bytes;
    }
    if (p.sup && !p.b_res) {
        *why = "tile groups need resident weights";
        return cudaErrorInvalidValue;
    }
    p.tx_sub = p.tx_a + (p.b_res ? 0u : p.tx_b);
    p.tx_res = p.out_bytes;
    // Windowed mode for 3x3 / stride 1 / pad 1 layers whose weights can stay resident: whole padded rows are loaded once
    // per tile and every filter tap reads them at a shifted row offset.  Worth it when whole rows fill most of a tile
    // and the im2col loads are what bounds the layer: measured, 128-channel layers gain 1.8x (the resident weights
    // leave room for two im2col stages only); 64-channel layers gain nothing (62 against 64 us: their tiles are bound
    // by the MMA-issuing threads, which need about 150 cycles per N = 64 instruction while the epilogue warps of their
    // scheduler partition are busy -- an MMA-only loop issues one every 52 cycles -- and whole-row tiles are 12.5 % more
    // tiles).
    p.win = 0;
    if (staged && !p.pair && p.kb == 128 && g.kh == 3 && g.kw == 3 && g.stride_h == 1 && g.stride_w == 1 && g.pad_h == 1 && g.pad_w == 1 &&
        g.pad_h_end < 0 && p.n_tiles == 1 && g.w + 2 <= TILE_M && g.w == g.wo && g.h == g.ho && g.c % p.kb == 0 &&
        !(off & (F8_PLAN_OFF_WINDOWED | F8_PLAN_OFF_RESIDENT_WEIGHTS))) {
        const int wp = g.w + 2;
        const int r = std::min(TILE_M / wp, g.ho);
        const int bands = (g.ho + r - 1) / r;
        const double fill = (double)g.ho * g.wo / ((double)bands * TILE_M);
        const uint32_t box_bytes = (uint32_t)p.kb * wp * (r + 2);
        const uint32_t win_stage = (box_bytes + 1023) / 1024 * 1024;
        const size_t bias_bytes = ((size_t)p.n_tiles * p.bn * 4 + 1023) / 1024 * 1024;
        int ob = p.out_bufs;
        // at least two window stages beside the weights; give up output buffers before giving up the mode
        while (ob > 1 && b_all + 2 * (size_t)win_stage + (size_t)p.out_bytes * ob + bias_bytes + ktab_bytes + 1024 > SMEM_LIMIT) --ob;
        const bool fits = b_all + 2 * (size_t)win_stage + (size_t)p.out_bytes * ob + bias_bytes + ktab_bytes + 1024 <= SMEM_LIMIT;
        if (fill >= 0.7 && fits) {
            p.win = 1;
            p.win_r = r;
            p.win_wp = wp;
            p.win_bands = bands;
            p.div_bands = make_fast_div(bands);
            p.tx_win = box_bytes;
            p.tx_res = (uint32_t)p.bn * wp * r;
            p.out_bufs = ob;
            staging = (size_t)p.out_bytes * ob + bias_bytes + ktab_bytes;
            p.b_res = 1;
            p.m_tiles = g.n * bands;
            p.sub_bytes = win_stage;
        }
    }
    p.rows = p.win;
    p.rowt = 0;
    // Small tensors: no im2col map is made for tensors below 128 KiB.  Pointwise layers read them as a plain matrix; other
    // layers take whole output rows per tile and fetch every filter tap with an ordinary tiled load.
    const bool dense_x = xv.stride_w == xv.dim_c && xv.stride_h == xv.dim_c * xv.dim_w && xv.stride_n == xv.dim_c * xv.dim_w * xv.dim_h;
    const bool pointwise = g.kh == 1 && g.kw == 1 && g.stride_h == 1 && g.stride_w == 1 && g.pad_h == 0 && g.pad_w == 0;
    const bool small_x = xv.dim_c * xv.dim_w * xv.dim_h * xv.dim_n < 128 * 1024;
    if (small_x && !pointwise && !p.win) {
        if (!dense_x || !f8_tc_rowtile_ok(g)) {
            *why = "small tensor whose rows do not fit a tile";
            return cudaErrorInvalidValue;
        }
        const int r = std::min(TILE_M / g.wo, g.ho);
        p.rows = p.rowt = 1;
        p.win_r = r;
        p.win_wp = g.wo;
        p.win_bands = (g.ho + r - 1) / r;
        p.div_bands = make_fast_div(p.win_bands);
        p.m_tiles = g.n * p.win_bands;
        p.tx_a = (uint32_t)p.kb * g.wo * r;            // bytes one tap's box delivers (zero fill included)
        p.tx_sub = p.tx_a + (p.b_res ? 0u : p.tx_b);
        p.tx_res = (uint32_t)p.bn * g.wo * r;
    }
    if (p.win) {
        p.group = 1;
        p.stage_bytes = p.sub_bytes;
        int stages = (int)((SMEM_LIMIT - 1024 - staging - b_all) / p.stage_bytes);
        if (stages > MAX_STAGES) stages = MAX_STAGES;
        p.stages = stages;
        p.uses = p.c_chunks;
    } else {
    const int uses = (k_iters + 7) / 8;                  // at most eight k-iterations per stage, evenly split
    int group = (k_iters + uses - 1) / uses;
    while (group > 1 && avail / ((size_t)group * p.sub_bytes) < 2) --group;
    group = (k_iters + (k_iters + group - 1) / group - 1) / ((k_iters + group - 1) / group);   // same uses, evenly split
    if (p.pair) group = 1;      // 32-KiB stage uses, as many stages in flight as fit
    if (p.sup) group = p.sup;   // a stage use holds the activation tiles of a group of M tiles (sub_bytes == a_bytes)
    p.group = group;
    p.stage_bytes = (uint32_t)group * p.sub_bytes;
    int stages = (int)(avail / p.stage_bytes);
    if (stages > 32 / group) stages = 32 / group;     // one lane per (stage, sub-chunk)
    if (stages > MAX_STAGES) stages = MAX_STAGES;
    if (stages < 2) {
        *why = "stage does not fit";
        return cudaErrorInvalidValue;
    }
    p.stages = stages;
    p.uses = p.sup ? 1 : (k_iters + group - 1) / group;
    }
    const int stages = p.stages;
    p.dual_issue = (p.bn <= 128 && stages >= 2 * p.uses && !p.sup && !(off & F8_PLAN_OFF_DUAL_ISSUE)) ? 1 : 0;
    p.alt = (!p.b_res && !p.dual_issue && !p.win && p.stages >= 2 && !(off & F8_PLAN_OFF_ALT_PRODUCERS)) ? 1 : 0;
    p.out_off = (uint32_t)(p.stages * p.stage_bytes);
    p.bias_off = p.out_off + (uint32_t)p.out_bufs * p.out_bytes;
    p.ktab_off = (uint32_t)(p.stages * p.stage_bytes + staging - ktab_bytes);
    p.bres_off = (uint32_t)(p.stages * p.stage_bytes + staging);
    // instruction descriptor: D = s32 (2 at bit 4), A format at bit 7 (0 = u8, 1 = s8), B = s8 at bit 10,
    // both operands K-major, N/8 at bit 17, M/16 at bit 24
    p.idesc = (2u << 4) | ((g.x_signed ? 1u : 0u) << 7) | (1u << 10) | ((uint32_t)(p.bn >> 3) << 17) |
              ((uint32_t)((p.pair ? 2 * TILE_M : TILE_M) >> 4) << 24);
    p.desc_hi = smem_desc_hi(p.kb);
    p.bias = bias;
    p.res = (const uint8_t *)res;
    p.y = (uint8_t *)y;
    p.q = q;
    p.mul_acc = 1 << q.sh_acc;
    p.mul_res = 1 << q.sh_res;
    p.status = status_word;
    const int ysz = (q.y_kind == F8_S32 || q.y_kind == F8_S32_RELU) ? 4 : 1;
    const size_t row_bytes = (size_t)g.c_out * ysz;
    p.vec_bytes = (row_bytes % 16 == 0) ? 16 : (row_bytes % 8 == 0 ? 8 : (row_bytes % 4 == 0 ? 4 : 1));
    if (has_sib) p.sib = *sib;
    {
        const size_t rb2 = (size_t)g.c_out * ((p.sib.y_kind == F8_S32 || p.sib.y_kind == F8_S32_RELU) ? 4 : 1);
        p.vec_bytes2 = (rb2 % 16 == 0) ? 16 : (rb2 % 8 == 0 ? 8 : (rb2 % 4 == 0 ? 4 : 1));
    }

    p.a_plain = (g.kh == 1 && g.kw == 1 && g.stride_h == 1 && g.stride_w == 1 && g.pad_h == 0 && g.pad_w == 0 && dense_x &&
                 xv.dim_c * xv.dim_w * xv.dim_h * xv.dim_n < 128 * 1024) ? 1 : 0;
    if (p.a_plain) {
        // A: [M, C] bytes, box = 128 pixels x kb channels; rows past the last pixel are zero filled
        cuuint64_t dims[2] = {xv.dim_c, (cuuint64_t)p.M};
        cuuint64_t strides[1] = {xv.dim_c};
        cuuint32_t box[2] = {(cuuint32_t)p.kb, (cuuint32_t)TILE_M};
        cuuint32_t estr[2] = {1, 1};
        CUresult r = g_encode_tiled(&plan->map_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(xv.base), dims, strides,
                                    box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(p.kb),
                                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) {
            *why = "cuTensorMapEncodeTiled rejected the activation matrix";
            return cudaErrorInvalidValue;
        }
    } else if (p.rowt) {
        // A: plain tiles of win_r output rows: one box per filter tap, traversed with the convolution stride (a box of
        // n * stride elements delivers n of them), out-of-image elements zero filled
        cuuint64_t dims[4] = {xv.dim_c, xv.dim_w, xv.dim_h, xv.dim_n};
        cuuint64_t strides[3] = {xv.stride_w, xv.stride_h, xv.stride_n};
        cuuint32_t box[4] = {(cuuint32_t)p.kb, (cuuint32_t)(g.wo * g.stride_w), (cuuint32_t)(p.win_r * g.stride_h), 1};
        cuuint32_t estr[4] = {1, (cuuint32_t)g.stride_w, (cuuint32_t)g.stride_h, 1};
        CUresult r = g_encode_tiled(&plan->map_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(xv.base), dims, strides,
                                    box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(p.kb),
                                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) {
            *why = "cuTensorMapEncodeTiled rejected the activation tensor";
            return cudaErrorInvalidValue;
        }
    } else if (p.win) {
        // A: the same tensor as plain tiles of win_r + 2 padded rows (coordinates -1 are zero filled)
        cuuint64_t dims[4] = {xv.dim_c, xv.dim_w, xv.dim_h, xv.dim_n};
        cuuint64_t strides[3] = {xv.stride_w, xv.stride_h, xv.stride_n};
        cuuint32_t box[4] = {(cuuint32_t)p.kb, (cuuint32_t)p.win_wp, (cuuint32_t)(p.win_r + 2), 1};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        CUresult r = g_encode_tiled(&plan->map_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(xv.base), dims, strides,
                                    box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(p.kb),
                                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) {
            *why = "cuTensorMapEncodeTiled rejected the activation tensor";
            return cudaErrorInvalidValue;
        }
    } else
    // A: activation tensor (C, W, H, N) in im2col mode.  Corners follow the usual forward-convolution
    // rule: lower = -pad, upper = pad - (k - 1); the traversal stride is the convolution stride.
    {
        cuuint64_t dims[4] = {xv.dim_c, xv.dim_w, xv.dim_h, xv.dim_n};
        cuuint64_t strides[3] = {xv.stride_w, xv.stride_h, xv.stride_n};
        int lower[2] = {-g.pad_w, -g.pad_h};
        int upper[2] = {g.pad_w - (g.kw - 1), (g.pad_h_end >= 0 ? g.pad_h_end : g.pad_h) - (g.kh - 1)};
        cuuint32_t estr[4] = {1, (cuuint32_t)g.stride_w, (cuuint32_t)g.stride_h, 1};
        CUresult r = g_encode_im2col(&plan->map_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(xv.base), dims,
                                     strides, lower, upper, (cuuint32_t)p.kb, (cuuint32_t)TILE_M, estr,
                                     CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(p.kb), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) {
            *why = "cuTensorMapEncodeIm2col rejected the activation tensor";
            return cudaErrorInvalidValue;
        }
    }
    // B: weights (C, taps, C_out), box (kb, 1, bn)
    {
        cuuint64_t dims[3] = {(cuuint64_t)g.c, (cuuint64_t)(g.kh * g.kw), (cuuint64_t)g.c_out};
        cuuint64_t strides[2] = {(cuuint64_t)g.c, (cuuint64_t)g.c * g.kh * g.kw};
        cuuint32_t box[3] = {(cuuint32_t)p.kb, 1, (cuuint32_t)bn_load};
        cuuint32_t estr[3] = {1, 1, 1};
        CUresult r = g_encode_tiled(&plan->map_b, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<int8_t *>(w), dims,
                                    strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(p.kb),
                                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) {
            *why = "cuTensorMapEncodeTiled rejected the weight tensor";
            return cudaErrorInvalidValue;
        }
    }
    // output / residual [M, c_out] bytes, one box = one column slab of a tile
    plan->map_y = plan->map_b;
    plan->map_r = plan->map_b;
    if (staged && p.rows) {
        // output / residual as (C_out, W, H, N); one box = one column slab of win_r rows of W + 2 positions
        cuuint64_t dims[4] = {(cuuint64_t)g.c_out, (cuuint64_t)g.wo, (cuuint64_t)g.ho, (cuuint64_t)g.n};
        cuuint64_t strides[3] = {(cuuint64_t)g.c_out, (cuuint64_t)g.c_out * g.wo, (cuuint64_t)g.c_out * g.wo * g.ho};
        cuuint32_t box[4] = {(cuuint32_t)p.slab_w, (cuuint32_t)p.win_wp, (cuuint32_t)p.win_r, 1};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        const CUtensorMapSwizzle sw = p.slab_w == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                      : (p.slab_w == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                         : (p.slab_w == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE));
        CUresult r = g_encode_tiled(&plan->map_y, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, y, dims, strides, box, estr,
                                    CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r == CUDA_SUCCESS && q.has_res)
            r = g_encode_tiled(&plan->map_r, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(res), dims, strides, box,
                               estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) {
            *why = "cuTensorMapEncodeTiled rejected the output tensor";
            return cudaErrorInvalidValue;
        }
    } else if (staged) {
        cuuint64_t dims[2] = {(cuuint64_t)g.c_out, (cuuint64_t)p.M};
        cuuint64_t strides[1] = {(cuuint64_t)g.c_out};
        cuuint32_t box[2] = {(cuuint32_t)p.slab_w, (cuuint32_t)TILE_M};
        cuuint32_t estr[2] = {1, 1};
        const CUtensorMapSwizzle sw = p.slab_w == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                      : (p.slab_w == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                         : (p.slab_w == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE));
        CUresult r = g_encode_tiled(&plan->map_y, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, y, dims, strides, box, estr,
                                    CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r == CUDA_SUCCESS && q.has_res)
            r = g_encode_tiled(&plan->map_r, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(res), dims, strides, box,
                               estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) {
            *why = "cuTensorMapEncodeTiled rejected the output tensor";
            return cudaErrorInvalidValue;
        }
    }
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int total_tiles = p.sup ? p.sup_tiles : p.m_tiles * p.n_tiles;
    plan->grid = total_tiles < sms ? total_tiles : sms;
    if (p.pair) plan->grid = 2 * std::min(p.pair_tiles, sms / 2);        // clusters of two; trimmed to what fits at launch
    // at least half of an SM's shared memory so that two CTAs (each owning all of TMEM) never share an SM
    plan->smem = (size_t)p.stages * p.stage_bytes + staging + (p.b_res ? b_all : 0) + 1024 + CONTROL_BYTES;
    if (plan->smem < 120 * 1024) plan->smem = 120 * 1024;
    p.wait_limit = f8_wait_limit_cycles();
    // what the plan decided, for tests that must know which code path a case exercises
    {
        int *info = f8_last_plan_info();
        info[0] = (p.b_res ? F8_PLAN_RESIDENT_WEIGHTS : 0) | (p.win ? F8_PLAN_WINDOWED : 0) | (p.dual_issue ? F8_PLAN_DUAL_ISSUE : 0) |
                  (p.alt ? F8_PLAN_ALT_PRODUCERS : 0) | (p.a_plain ? F8_PLAN_PLAIN_MATRIX : 0) | (staged ? F8_PLAN_STAGED_EPILOGUE : 0) | (p.rowt ? F8_PLAN_ROW_TILES : 0) |
                  (p.pair ? F8_PLAN_PAIRS : 0) | (p.sup ? F8_PLAN_TILE_GROUPS : 0);
        info[1] = p.epi; info[2] = p.bn; info[3] = p.kb; info[4] = p.stages; info[5] = p.group;
        info[6] = p.m_tiles; info[7] = p.n_tiles; info[8] = plan->grid; info[9] = staged ? p.out_bufs : 0;
    }
    // the opt-in to large dynamic shared memory is a per-device attribute of each kernel
    static bool attr_set[64] = {false};
    if (dev < 0 || dev >= 64) {
        *why = "device index out of range";
        return cudaErrorInvalidDevice;
    }
    if (!attr_set[dev]) {
        const int bytes = (int)(SMEM_LIMIT + CONTROL_BYTES);
        cudaError_t e = cudaFuncSetAttribute(f8_conv_gemm_tc_kernel<EPI_GENERIC, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(f8_conv_gemm_tc_kernel<EPI_U8, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(f8_conv_gemm_tc_kernel<EPI_U8_RES, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(f8_conv_gemm_tc_kernel<EPI_S8, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(f8_conv_gemm_tc_kernel<EPI_S8_RES, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(f8_conv_gemm_tc_kernel<EPI_U8, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(f8_conv_gemm_tc_kernel<EPI_U8_RES, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(f8_conv_gemm_tc_kernel<EPI_S8, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(f8_conv_gemm_tc_kernel<EPI_S8_RES, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(f8_conv_gemm_tc_kernel<EPI_U8, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(f8_conv_gemm_tc_kernel<EPI_S8, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e != cudaSuccess) {
            *why = "cudaFuncSetAttribute(MaxDynamicSharedMemorySize) failed";
            return e;
        }
        attr_set[dev] = true;
    }
    return cudaSuccess;
}

namespace {
template <int EPI, int MODE>
cudaError_t launch_variant(const F8TcPlan *plan, bool overlap_previous, cudaStream_t st) {
    constexpr bool PAIR = MODE == 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)plan->grid);
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = plan->smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n = 0;
    if (PAIR) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = 2;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    if (overlap_previous) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    if (PAIR) {
        // persistent pairs: no more clusters than the device can hold at once
        int clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&clusters, f8_conv_gemm_tc_kernel<EPI, MODE>, &cfg) == cudaSuccess && clusters > 0 &&
            2 * clusters < plan->grid)
            cfg.gridDim = dim3((unsigned)(2 * clusters));
        else
            (void)cudaGetLastError();
    }
    return cudaLaunchKernelEx(&cfg, f8_conv_gemm_tc_kernel<EPI, MODE>, plan->map_a, plan->map_b, plan->map_y, plan->map_r, plan->p);
}
}   // namespace

cudaError_t f8_tc_launch(const F8TcPlan *plan, bool overlap_previous, cudaStream_t st) {
    if (plan->p.M == 0) return cudaSuccess;
    if (plan->p.pair) {
        switch (plan->p.epi) {
            case EPI_U8: return launch_variant<EPI_U8, 1>(plan, overlap_previous, st);
            case EPI_U8_RES: return launch_variant<EPI_U8_RES, 1>(plan, overlap_previous, st);
            case EPI_S8: return launch_variant<EPI_S8, 1>(plan, overlap_previous, st);
            case EPI_S8_RES: return launch_variant<EPI_S8_RES, 1>(plan, overlap_previous, st);
            default: return cudaErrorInvalidValue;
        }
    }
    if (plan->p.sup) {
        switch (plan->p.epi) {
            case EPI_U8: return launch_variant<EPI_U8, 2>(plan, overlap_previous, st);
            case EPI_S8: return launch_variant<EPI_S8, 2>(plan, overlap_previous, st);
            default: return cudaErrorInvalidValue;
        }
    }
    switch (plan->p.epi) {
        case EPI_U8: return launch_variant<EPI_U8, 0>(plan, overlap_previous, st);
        case EPI_U8_RES: return launch_variant<EPI_U8_RES, 0>(plan, overlap_previous, st);
        case EPI_S8: return launch_variant<EPI_S8, 0>(plan, overlap_previous, st);
        case EPI_S8_RES: return launch_variant<EPI_S8_RES, 0>(plan, overlap_previous, st);
        default: return launch_variant<EPI_GENERIC, 0>(plan, overlap_previous, st);
    }
}

cudaError_t f8_tc_wait_probe(unsigned long long limit_cycles, int *status_word, cudaStream_t st) {
    // never the unbounded default: a probe waits a hundred milliseconds at most
    if (limit_cycles == 0 || limit_cycles > 250000000ull) limit_cycles = 250000000ull;
    f8_wait_probe_kernel<<<1, 32, 0, st>>>(limit_cycles, status_word);
    return cudaGetLastError();
}

cudaError_t f8_tc_probe(int iters, double *ops, int *status_word, cudaStream_t st) {
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const size_t smem = 120 * 1024;
    cudaError_t e = cudaFuncSetAttribute(f8_mma_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    f8_mma_probe_kernel<<<sms, NUM_THREADS, smem, st>>>(iters, status_word);
    *ops = 2.0 * 128 * 256 * 32 * (double)iters * sms;
    return cudaGetLastError();
}
