// Two layers in one kernel: a dense convolution with 64 input and 64 output channels followed by the pointwise
// (1x1) convolution that expands its output to 256 channels, with or without a shortcut -- the tail of a ResNet
// bottleneck block at its widest resolution.  Eq. 6 is applied per layer, so running two layers in one launch
// changes no result: the first layer's 8-bit output tile (128 pixels x 64 channels, quantised by Eq. 2) is written
// to shared memory in the swizzled K-major layout tcgen05.mma reads and is the A operand of the second GEMM at
// once; it never travels to global memory (unless the caller asks for a copy).
//
//   producers (2 warps)   one im2col TMA load per filter tap and tile, every tap in its own lane and stage
//   MMA issuer (1 thread) GEMM 1: taps x (128 x 64 x 64) into one of two 64-column accumulators;
//                         GEMM 2 of the previous tile: 128 x 256 x 64 from the staged tile into a 256-column one
//   16 epilogue warps     tile l: accumulator 1 -> bias, rounding shift, clip -> staged tile;
//                         tile l - 1: accumulator 2 -> bias, shortcut, rounding shift, clip -> output ring
//   mover / fetcher       TMA stores of finished output tiles, TMA loads of shortcut tiles into the ring
//
// Both weight tensors stay in shared memory for the life of the CTA.  Every wait is bounded (see f8_tc_ptx.cuh).
#include <cuda.h>
#include <cudaTypedefs.h>

#include <string.h>

#include <algorithm>

#include "f8_internal.h"
#include "f8_tc_ptx.cuh"

namespace {

constexpr int FT_TILE_M = 128;
constexpr int FT_C = 64;                  // channels of the first layer's input and output
constexpr int FT_N2 = 256;                // output channels of the pointwise layer
constexpr int FT_MAX_STAGES = 16;
constexpr int FT_MAX_OUT_BUFS = 4;
constexpr int FT_EPI_WARPS = 16;
constexpr int FT_A_WARP = 0, FT_MMA_WARP = 1, FT_MOVER_WARP = 2, FT_FETCH_WARP = 3, FT_FIRST_EPI = 4;
constexpr int FT_A2_WARP = FT_FIRST_EPI + FT_EPI_WARPS;
constexpr int FT_MMA2_WARP = FT_A2_WARP + 2;        // (the warp in between would share the first issuer's scheduler)
constexpr int FT_THREADS = 32 * (FT_MMA2_WARP + 1);
constexpr uint32_t FT_A_BYTES = FT_TILE_M * FT_C;          // one tap of a tile
constexpr uint32_t FT_W1_BYTES = FT_C * FT_C;              // one tap of the first layer's weights
constexpr uint32_t FT_W2_BYTES = FT_N2 * FT_C;
constexpr uint32_t FT_T_BYTES = FT_TILE_M * FT_C;          // the staged 8-bit tile between the layers
constexpr uint32_t FT_OUT_BYTES = FT_TILE_M * FT_N2;
constexpr uint32_t FT_CONTROL_BYTES = 1024;
constexpr size_t FT_SMEM_LIMIT = 225 * 1024;
constexpr int FT_TMEM_COLS = 512;
constexpr int FT_ACC2_COL = 256;

// Stage and accumulator barriers sit where the single-layer kernel keeps its own, the rest behind them.
struct FtControl {
    uint64_t full[FT_MAX_STAGES], empty[FT_MAX_STAGES];
    uint64_t tfull1[2], tempty1[2], wres;
    uint64_t out_full[FT_MAX_OUT_BUFS], out_free[FT_MAX_OUT_BUFS], res_full[FT_MAX_OUT_BUFS];
    uint64_t tmid_full, tmid_free, tfull2, tempty2;
    uint32_t tmem_base_slot;
    int abort_flag;
};
static_assert(sizeof(FtControl) <= FT_CONTROL_BYTES, "control block does not fit its slot");

struct FtDiv {
    uint32_t mul, shift;
};
__device__ __forceinline__ int ft_div(int n, FtDiv d) { return (int)(((uint64_t)(uint32_t)n * d.mul) >> d.shift); }

struct FtParams {
    int M;                      // output pixels
    int ho, wo;
    int kh, kw, stride, pad;
    int taps;                   // kh * kw <= 16
    int m_tiles;
    FtDiv div_wo, div_ho;
    int stages, out_bufs;
    int group, groups;          // taps per stage, stages uses per tile
    uint32_t w1_off, w2_off, t_off, out_off, bias_off;      // byte offsets behind the control block
    uint32_t idesc1, idesc2;
    uint64_t desc_hi;
    const int32_t *bias1, *bias2;
    int s1;                     // rounding shift of the first layer (1..24); its output is unsigned 8-bit
    int mul1;                   // 1 (opaque to the compiler, as the factors of the second layer are)
    int sh_acc2, s2, mul_acc2, mul_res2, r_signed;
    uint8_t *y_mid;             // optional copy of the first layer's output (NULL: none)
    int *status;
    int tag;
    unsigned long long wait_limit;
};

// ----------------------------------------------------------------------------- the kernel

template <bool RES, bool SGN>
__global__ void __launch_bounds__(FT_THREADS, 1)
f8_conv_pw_fused_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w1,
                           const __grid_constant__ CUtensorMap map_w2, const __grid_constant__ CUtensorMap map_y,
                           const __grid_constant__ CUtensorMap map_r, const FtParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem_aligned = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    FtControl &ctl = *(FtControl *)smem_aligned;
    uint8_t *smem = smem_aligned + FT_CONTROL_BYTES;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int worker = (int)blockIdx.x, n_workers = (int)gridDim.x;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t full_bar = smem_u32(&ctl.full[0]), empty_bar = smem_u32(&ctl.empty[0]);
    const uint32_t tfull1 = smem_u32(&ctl.tfull1[0]), tempty1 = smem_u32(&ctl.tempty1[0]);
    const uint32_t wres_bar = smem_u32(&ctl.wres);
    const uint32_t out_full = smem_u32(&ctl.out_full[0]), out_free = smem_u32(&ctl.out_free[0]);
    const uint32_t res_full = smem_u32(&ctl.res_full[0]);
    const uint32_t tmid_full = smem_u32(&ctl.tmid_full), tmid_free = smem_u32(&ctl.tmid_free);
    const uint32_t tfull2 = smem_u32(&ctl.tfull2), tempty2 = smem_u32(&ctl.tempty2);

    if (threadIdx.x == 32) {
        prefetch_tensormap(&map_a);
        prefetch_tensormap(&map_w1);
        prefetch_tensormap(&map_w2);
        prefetch_tensormap(&map_y);
        if (RES) prefetch_tensormap(&map_r);
    }
    if (threadIdx.x == 0) {
        ctl.abort_flag = 0;
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(full_bar + 8 * s, p.group);  // every lane that requests a tap of the group announces its bytes
            mbar_init(empty_bar + 8 * s, 1);       // commit of the MMAs that read the stage
        }
        mbar_init(wres_bar, 1);
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull1 + 8 * a, 1);
            mbar_init(tempty1 + 8 * a, FT_EPI_WARPS);
        }
        mbar_init(tmid_full, FT_EPI_WARPS);        // every epilogue warp has written its part of the staged tile
        mbar_init(tmid_free, 1);                   // GEMM 2 has read the staged tile
        mbar_init(tfull2, 1);
        mbar_init(tempty2, FT_EPI_WARPS);
        for (int b = 0; b < FT_MAX_OUT_BUFS; ++b) {
            mbar_init(out_full + 8 * b, FT_EPI_WARPS);
            mbar_init(out_free + 8 * b, 1);
            mbar_init(res_full + 8 * b, 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == FT_MMA_WARP) tmem_alloc(smem_u32(&ctl.tmem_base_slot), FT_TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl.tmem_base_slot;
    grid_launch_dependents();

    const int n_local = worker < p.m_tiles ? (p.m_tiles - worker + n_workers - 1) / n_workers : 0;
    const WaitCtx wc = make_wait_ctx(&ctl.abort_flag, p.status, p.wait_limit);
    const int tagbits = p.tag << 8;

    if (warp == FT_A_WARP || warp == FT_A2_WARP) {
        // ------------------------------------------------------------------ TMA producers
        // A stage holds a group of G consecutive taps of one tile (one barrier pair per group: every wait, fence and commit
        // costs the lone MMA-issuing thread a few hundred cycles, as much as several MMAs).  Group k of local tile l is
        // use u = l * groups + k of the ring: stage u mod S, use u div S.  Warp h requests the uses of parity h, every
        // tap in a lane of its own (loads issued by different threads overlap).  S is even, so a stage is always
        // refilled by the same warp: the wait for its previous refill comes earlier in that warp's program order, and
        // a parity wait (which can only tell a phase from its neighbour) cannot take an older release for the last one.
        const int half = warp == FT_A2_WARP ? 1 : 0;
        if (half == 1) {
            // the weights of both layers, once per CTA: nothing the previous grid writes
            const int n_loads = p.taps + 1;
            if (lane == 0) mbar_expect_tx(wres_bar, (uint32_t)p.taps * FT_W1_BYTES + FT_W2_BYTES);
            __syncwarp();
            if (lane < p.taps) tma_load_3d(smem_base + p.w1_off + (uint32_t)lane * FT_W1_BYTES, &map_w1, wres_bar, 0, lane, 0);
            else if (lane == n_loads - 1) tma_load_3d(smem_base + p.w2_off, &map_w2, wres_bar, 0, 0, 0);
        }
        grid_dependency_wait();
        const int G = p.group, NG = p.groups, S = p.stages, per_round = S >> 1;
        const int gi = lane / G, ti = lane - gi * G;       // this lane's group among the warp's groups of a tile, tap in the group
        bool ok = true, have_last = false;
        int last_slot = 0;
        uint32_t last_par = 0;
        for (int l = 0; l < n_local; ++l) {
            const int m0 = (worker + l * n_workers) * FT_TILE_M;
            const int t1 = ft_div(m0, p.div_wo);
            const int ow = m0 - t1 * p.wo;
            const int img = ft_div(t1, p.div_ho);
            const int oh = t1 - img * p.ho;
            const int u0 = l * NG;
            const int k0 = (half - u0) & 1;                          // this warp's first group of the tile
            const int n_mine = k0 < NG ? (NG - k0 + 1) >> 1 : 0;     // groups k0, k0 + 2, ...
            const int k = k0 + 2 * gi, u = u0 + k, tap = k * G + ti;
            const int slot = u % S, use = u / S;
            const int r = tap / p.kw, sx = tap - r * p.kw;
            // at most S / 2 of the warp's groups at a time: they lie in different stages, and a stage a later round needs
            // is freed by loads that were requested in an earlier one
            for (int r0 = 0; ok && r0 < n_mine; r0 += per_round) {
                const bool act = gi < n_mine && gi >= r0 && gi < r0 + per_round;
                bool got = true;
                if (act) got = mbar_wait(empty_bar + 8 * slot, (uint32_t)(use & 1) ^ 1u, wc, tagbits | 201);
                if (!__all_sync(0xffffffffu, got)) { ok = false; break; }
                if (act) {
                    const uint32_t fb = full_bar + 8 * slot;
                    if (tap < p.taps) {
                        mbar_expect_tx(fb, FT_A_BYTES);
                        tma_load_im2col(smem_base + (uint32_t)(slot * G + ti) * FT_A_BYTES, &map_a, fb, 0, ow * p.stride - p.pad,
                                        oh * p.stride - p.pad, img, (uint16_t)sx, (uint16_t)r);
                        have_last = true;
                        last_slot = slot;
                        last_par = (uint32_t)(use & 1);
                    } else {
                        mbar_arrive(fb);        // a tap the last group does not have
                    }
                }
            }
            if (!ok) break;
        }
        if (!ok && have_last) {
            const unsigned long long t0 = clock64();
            while (!mbar_try_wait(full_bar + 8 * last_slot, last_par) && (unsigned long long)(clock64() - t0) < DRAIN_LIMIT_CYCLES) {
            }
        }
        // the weights must have landed before this CTA's shared memory may go away
        if (half == 1 && lane == 0) mbar_wait(wres_bar, 0, wc, tagbits | 210);
    } else if (warp == FT_MMA_WARP) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0 && n_local > 0) {
            const uint32_t desc_lo0 = (uint32_t)p.desc_hi | ((smem_base & 0x3ffffu) >> 4);
            const uint32_t desc_hi32 = (uint32_t)(p.desc_hi >> 32);
            const uint32_t w1_lo = desc_lo0 + (p.w1_off >> 4);
            bool ok = mbar_wait(wres_bar, 0, wc, tagbits | 211);
            bool committed_any = false;
            int last_acc = 0;
            uint32_t last_acc_phase = 0;
            int slot = 0, use = 0;
            const int G = p.group, NG = p.groups;
            for (int l = 0; ok && l < n_local; ++l) {
                const int acc = l & 1;
                if (!mbar_wait(tempty1 + 8 * acc, (uint32_t)((l >> 1) & 1) ^ 1u, wc, tagbits | 202)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)acc * FT_C;
                int tap = 0;
                for (int k = 0; k < NG; ++k) {
                    if (!mbar_wait(full_bar + 8 * slot, (uint32_t)(use & 1), wc, tagbits | 203)) { ok = false; break; }
                    tc_fence_after();
                    uint32_t a_lo = desc_lo0 + (uint32_t)(slot * G) * (FT_A_BYTES >> 4);
                    for (int t = 0; t < G && tap < p.taps; ++t, ++tap, a_lo += FT_A_BYTES >> 4)
                        mma_i8_sub<2>(d_tmem, a_lo, w1_lo + (uint32_t)tap * (FT_W1_BYTES >> 4), desc_hi32, p.idesc1, tap != 0 ? 1u : 0u);
                    mma_commit(empty_bar + 8 * slot);
                    if (++slot == p.stages) { slot = 0; ++use; }
                }
                if (!ok) break;
                mma_commit(tfull1 + 8 * acc);
                committed_any = true;
                last_acc = acc;
                last_acc_phase = (uint32_t)((l >> 1) & 1);
            }
            if (ok) {
                // the releases of the last stage uses, which nobody else waits for, must land before the CTA goes
                const int total = n_local * NG;
                for (int g = max(0, total - p.stages); g < total; ++g)
                    mbar_wait(empty_bar + 8 * (g % p.stages), (uint32_t)(g / p.stages) & 1u, wc, tagbits | 212);
            } else if (committed_any) {
                // let the tensor pipe finish what was issued before tensor memory is released
                const unsigned long long t0 = clock64();
                while (!mbar_try_wait(tfull1 + 8 * last_acc, last_acc_phase) && (unsigned long long)(clock64() - t0) < DRAIN_LIMIT_CYCLES) {
                }
            }
        }
    } else if (warp == FT_MMA2_WARP) {
        // ------------------------------------------------------------------ second issuer: the pointwise GEMM
        // GEMM 2 of local tile i: the staged tile times the pointwise weights, as soon as the first layer's epilogue has
        // written the tile and the second layer's epilogue has read the previous result out of the accumulator.  A thread
        // of its own, so that these waits do not sit between the first issuer's instructions.
        if (lane == 0 && n_local > 0) {
            const uint32_t desc_lo0 = (uint32_t)p.desc_hi | ((smem_base & 0x3ffffu) >> 4);
            const uint32_t desc_hi32 = (uint32_t)(p.desc_hi >> 32);
            const uint32_t w2_lo = desc_lo0 + (p.w2_off >> 4), t_lo = desc_lo0 + (p.t_off >> 4);
            bool ok = mbar_wait(wres_bar, 0, wc, tagbits | 214);
            int i = 0;
            for (; ok && i < n_local; ++i) {
                if (!mbar_wait(tmid_full, (uint32_t)(i & 1), wc, tagbits | 205)) { ok = false; break; }
                if (!mbar_wait(tempty2, (uint32_t)(i & 1) ^ 1u, wc, tagbits | 206)) { ok = false; break; }
                tc_fence_after();
                mma_i8_sub<2>(tmem_base + FT_ACC2_COL, t_lo, w2_lo, desc_hi32, p.idesc2, 0u);
                mma_commit(tmid_free);
                mma_commit(tfull2);
            }
            // the last release of the staged tile has no other waiter
            if (ok) mbar_wait(tmid_free, (uint32_t)((n_local - 1) & 1), wc, tagbits | 213);
        }
    } else if (warp == FT_MOVER_WARP) {
        // ------------------------------------------------------------------ output mover
        if (lane == 0) {
            grid_dependency_wait();
            int b = 0;
            uint32_t bphase = 0;
            for (int l = 0; l < n_local; ++l) {
                const int m0 = (worker + l * n_workers) * FT_TILE_M;
                if (!mbar_wait(out_full + 8 * b, bphase, wc, tagbits | 208)) break;
                const uint32_t src = smem_base + p.out_off + (uint32_t)b * FT_OUT_BYTES;
                tma_store_2d(&map_y, src, 0, m0);
                tma_store_2d(&map_y, src + FT_TILE_M * 128, 128, m0);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                mbar_arrive(out_free + 8 * b);
                if (++b == p.out_bufs) { b = 0; bphase ^= 1; }
            }
            asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        }
    } else if (warp == FT_FETCH_WARP) {
        // ------------------------------------------------------------------ shortcut fetcher
        if (RES && lane == 0) {
            grid_dependency_wait();
            int rb = 0, l = 0;
            uint32_t rphase = 0;
            bool ok = true;
            for (; l < n_local; ++l) {
                const int m0 = (worker + l * n_workers) * FT_TILE_M;
                if (!mbar_wait(out_free + 8 * rb, rphase ^ 1u, wc, tagbits | 207)) { ok = false; break; }
                const uint32_t fb = res_full + 8 * rb;
                const uint32_t dst = smem_base + p.out_off + (uint32_t)rb * FT_OUT_BYTES;
                mbar_expect_tx(fb, FT_OUT_BYTES);
                tma_load_2d(dst, &map_r, fb, 0, m0);
                tma_load_2d(dst + FT_TILE_M * 128, &map_r, fb, 128, m0);
                if (++rb == p.out_bufs) { rb = 0; rphase ^= 1; }
            }
            if (!ok) {
                for (int i = 0; i < p.out_bufs && l - 1 - i >= 0; ++i) {
                    const int k = l - 1 - i;
                    const unsigned long long t0 = clock64();
                    while (!mbar_try_wait(res_full + 8 * (k % p.out_bufs), (uint32_t)(k / p.out_bufs) & 1u) &&
                           (unsigned long long)(clock64() - t0) < DRAIN_LIMIT_CYCLES) {
                    }
                }
            }
        }
    }
    else if (warp >= FT_FIRST_EPI && warp < FT_FIRST_EPI + FT_EPI_WARPS) {
        // ------------------------------------------------------------------ epilogue warps
        const int quarter = warp & 3;                       // TMEM lanes 32 * quarter .. + 31
        const int g = (warp - FT_FIRST_EPI) >> 2;           // chunk of accumulator 1, column quarter of accumulator 2
        {
            // bias' = (bias << sh_acc) + 2^(s - 1) of both layers, once per CTA, behind a barrier of these warps only
            int *bias_all = (int *)(smem + p.bias_off);
            for (int i = (int)threadIdx.x - FT_FIRST_EPI * 32; i < FT_C + FT_N2; i += FT_EPI_WARPS * 32) {
                if (i < FT_C) bias_all[i] = (p.bias1 ? __ldg(p.bias1 + i) : 0) + (1 << (p.s1 - 1));
                else bias_all[i] = ((p.bias2 ? __ldg(p.bias2 + i - FT_C) : 0) << p.sh_acc2) + (1 << (p.s2 - 1));
            }
            asm volatile("bar.sync 1, %0;" ::"n"(FT_EPI_WARPS * 32) : "memory");
        }
        if (p.y_mid) grid_dependency_wait();     // direct stores of the first layer's output
        const int row = quarter * 32 + lane;
        uint32_t rsel[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) rsel[k] = p.r_signed ? (0x8880u | (0x1111u * k)) : (0x4440u | k);
        // this thread's 16 bytes of the staged tile (64-byte rows, 64-byte swizzle)
        uint32_t so1 = (uint32_t)row * FT_C + (uint32_t)g * 16;
        so1 ^= ((so1 >> 7) & 3u) << 4;
        // and its four 16-byte chunks of an output tile (two slabs of 128-byte rows, 128-byte swizzle)
        uint32_t so2[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t off = (uint32_t)row * 128 + (uint32_t)((g & 1) * 4 + i) * 16;
            off ^= ((off >> 7) & 7u) << 4;
            so2[i] = (uint32_t)(g >> 1) * (FT_TILE_M * 128) + off;
        }
        const uint32_t bias1_s = smem_base + p.bias_off + 64 * g;
        const uint32_t bias2_s = smem_base + p.bias_off + 4 * FT_C + 256 * g;
        const uint32_t t_buf = smem_base + p.t_off;
        const int mul_acc2 = p.mul_acc2, mul_res2 = p.mul_res2, mul1 = p.mul1;
        int ob = 0;
        uint32_t ophase = 0;
        // second layer's epilogue of local tile i
        auto epi2 = [&](int i) -> bool {
            bool got;
            if (RES) got = mbar_wait(res_full + 8 * ob, ophase, wc, tagbits | 221);
            else got = mbar_wait(out_free + 8 * ob, ophase ^ 1u, wc, tagbits | 222);
            got = mbar_wait(tfull2, (uint32_t)(i & 1), wc, tagbits | 223) && got;
            if (!__all_sync(0xffffffffu, got)) return false;
            tc_fence_after();
            const uint32_t out_buf = smem_base + p.out_off + (uint32_t)ob * FT_OUT_BYTES;
            const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + FT_ACC2_COL + g * 64;
            auto release_acc = [&]() {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(tempty2);
            };
            int va[16], vb[16];
            tmem_ld16(t_addr, va);
#pragma unroll
            for (int c = 0; c < 4; c += 2) {
                {
                    uint4 rw = make_uint4(0, 0, 0, 0);
                    if (RES) rw = lds128(out_buf + so2[c]);
                    tmem_ld_wait();
                    tmem_ld16(t_addr + (c + 1) * 16, vb);
                    sts128(out_buf + so2[c], epilogue_fast16<RES, SGN>(va, bias2_s + 64 * c, rw, mul_acc2, mul_res2, rsel, p.s2));
                }
                {
                    uint4 rw = make_uint4(0, 0, 0, 0);
                    if (RES) rw = lds128(out_buf + so2[c + 1]);
                    tmem_ld_wait();
                    if (c + 2 < 4) tmem_ld16(t_addr + (c + 2) * 16, va);
                    else release_acc();
                    sts128(out_buf + so2[c + 1], epilogue_fast16<RES, SGN>(vb, bias2_s + 64 * (c + 1), rw, mul_acc2, mul_res2, rsel, p.s2));
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(out_full + 8 * ob);
            if (++ob == p.out_bufs) { ob = 0; ophase ^= 1; }
            return true;
        };
        bool ok = true;
        for (int l = 0; ok && l < n_local; ++l) {
            // first layer's epilogue of local tile l: accumulator 1 -> the staged tile
            const int acc = l & 1;
            if (!__all_sync(0xffffffffu, mbar_wait(tfull1 + 8 * acc, (uint32_t)((l >> 1) & 1), wc, tagbits | 224))) { ok = false; break; }
            tc_fence_after();
            int v[16];
            tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)acc * FT_C + g * 16, v);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty1 + 8 * acc);
            const uint4 o = epilogue_fast16<false, false>(v, bias1_s, make_uint4(0, 0, 0, 0), mul1, 0, rsel, p.s1);
            // the staged tile is free once GEMM 2 of the previous tile has read it
            if (!__all_sync(0xffffffffu, mbar_wait(tmid_free, (uint32_t)(l & 1) ^ 1u, wc, tagbits | 225))) { ok = false; break; }
            sts128(t_buf + so1, o);
            if (p.y_mid) {
                const size_t m = (size_t)(worker + l * n_workers) * FT_TILE_M + row;
                if (m < (size_t)p.M) *(uint4 *)(p.y_mid + m * FT_C + g * 16) = o;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(tmid_full);
            if (l >= 1) ok = epi2(l - 1);
        }
        if (ok && n_local > 0) epi2(n_local - 1);
    }

    if (*(volatile int *)&ctl.abort_flag) {
        // A wait gave up: the roles have left their loops with copies and tensor-core work possibly still on their way to
        // this CTA's shared memory, barriers and tensor memory.  Give them time to land before the CTA goes (the
        // failure is already on record; this only keeps it from turning into a fault).
        const unsigned long long t0 = clock64();
        while ((unsigned long long)(clock64() - t0) < 400000ull) {
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == FT_MMA_WARP) {
        tc_fence_after();
        tmem_dealloc(tmem_base, FT_TMEM_COLS);
    }
}

// ----------------------------------------------------------------------------- host side

PFN_cuTensorMapEncodeTiled_v12000 ft_encode_tiled = nullptr;
PFN_cuTensorMapEncodeIm2col_v12000 ft_encode_im2col = nullptr;

bool ft_load_driver_entry_points() {
    if (ft_encode_tiled && ft_encode_im2col) return true;
    void *f = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &qr) != cudaSuccess || !f ||
        qr != cudaDriverEntryPointSuccess)
        return false;
    ft_encode_tiled = (PFN_cuTensorMapEncodeTiled_v12000)f;
    f = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &f, cudaEnableDefault, &qr) != cudaSuccess || !f ||
        qr != cudaDriverEntryPointSuccess)
        return false;
    ft_encode_im2col = (PFN_cuTensorMapEncodeIm2col_v12000)f;
    return true;
}

FtDiv ft_make_div(int d) {
    uint32_t l = 0;
    while ((1u << l) < (uint32_t)d) ++l;
    FtDiv f;
    f.shift = 31 + l;
    f.mul = (uint32_t)(((uint64_t)1 << f.shift) / (uint32_t)d + 1);
    return f;
}

}   // namespace

struct F8FusedPlan {
    CUtensorMap map_a, map_w1, map_w2, map_y, map_r;
    FtParams p;
    int grid;
    size_t smem;
    int res, sgn;
};

size_t f8_fused_plan_size() { return sizeof(F8FusedPlan); }
void f8_fused_plan_set_tag(F8FusedPlan *plan, int tag) { plan->p.tag = tag; }

bool f8_fused_supported(const F8ConvGeom &g1, const F8Requant &q1, int c_out2, const F8Requant &q2) {
    if (g1.c != FT_C || g1.c_out != FT_C || c_out2 != FT_N2) return false;
    if (g1.kh * g1.kw > 16 || g1.kh > 255 || g1.kw > 255 || g1.stride_h != g1.stride_w || g1.pad_h != g1.pad_w || g1.pad_h_end >= 0) return false;
    if ((size_t)g1.n * g1.h * g1.w * g1.c < 128 * 1024) return false;        // no im2col map for small tensors
    if ((long long)g1.n * g1.ho * g1.wo > 0x7fffff00ll) return false;
    // the first layer feeds the second as unsigned 8-bit codes (ReLU + clip of Eq. 2), without a shortcut of its own
    if (q1.y_kind != F8_U8 || q1.has_res || q1.s < 1 || q1.s > 24) return false;
    if ((q2.y_kind != F8_U8 && q2.y_kind != F8_S8) || q2.r_s32 || q2.s < 1 || q2.s > 24) return false;
    return true;
}

cudaError_t f8_fused_plan_init(F8FusedPlan *plan, const F8ConvGeom &g1, const F8Requant &q1, const F8Requant &q2, const void *x,
                               const int8_t *w1, const int32_t *bias1, const int8_t *w2, const int32_t *bias2, const void *res,
                               void *y_mid, void *y, int *status_word, const char **why) {
    *why = "";
    if (!ft_load_driver_entry_points()) {
        *why = "cuTensorMapEncode entry points not available";
        return cudaErrorNotSupported;
    }
    if (!f8_fused_supported(g1, q1, FT_N2, q2) || (q2.has_res != 0) != (res != nullptr)) {
        *why = "shape outside the fused kernel's range";
        return cudaErrorInvalidValue;
    }
    memset(plan, 0, sizeof(*plan));
    FtParams &p = plan->p;
    p.M = g1.n * g1.ho * g1.wo;
    p.ho = g1.ho;
    p.wo = g1.wo;
    p.kh = g1.kh;
    p.kw = g1.kw;
    p.stride = g1.stride_h;
    p.pad = g1.pad_h;
    p.taps = g1.kh * g1.kw;
    p.m_tiles = (p.M + FT_TILE_M - 1) / FT_TILE_M;
    p.div_wo = ft_make_div(g1.wo);
    p.div_ho = ft_make_div(g1.ho);
    // shared memory: stages | first layer's weights | pointwise weights | staged tile | output ring | bias tables.
    // With a shortcut a buffer of the ring goes through load -> convert in place -> store: three of them.
    // Two buffers in the output ring (with a shortcut a buffer goes through load -> convert in place -> store; a third
    // buffer measured no faster than two, and costs four stages).
    p.out_bufs = 2;
    p.group = p.taps >= 3 ? 3 : p.taps;
    p.groups = (p.taps + p.group - 1) / p.group;
    const size_t stage_bytes = (size_t)p.group * FT_A_BYTES;
    const size_t fixed = (size_t)p.taps * FT_W1_BYTES + FT_W2_BYTES + FT_T_BYTES + (size_t)p.out_bufs * FT_OUT_BYTES + 2048;
    int stages = (int)((FT_SMEM_LIMIT - fixed) / stage_bytes);
    if (stages > FT_MAX_STAGES) stages = FT_MAX_STAGES;
    stages &= ~1;           // even: a stage is always refilled by the same producer warp
    if (stages < 2) {
        *why = "stages do not fit";
        return cudaErrorInvalidValue;
    }
    p.stages = stages;
    p.w1_off = (uint32_t)(stages * stage_bytes);
    p.w2_off = p.w1_off + (uint32_t)p.taps * FT_W1_BYTES;
    p.t_off = p.w2_off + FT_W2_BYTES;
    p.out_off = p.t_off + FT_T_BYTES;
    p.bias_off = p.out_off + (uint32_t)p.out_bufs * FT_OUT_BYTES;
    plan->smem = (size_t)p.bias_off + 2048 + FT_CONTROL_BYTES + 1024;
    // instruction descriptors: D = s32, A format (0 = u8, 1 = s8), B = s8, both K-major, N / 8, M / 16
    p.idesc1 = (2u << 4) | ((g1.x_signed ? 1u : 0u) << 7) | (1u << 10) | ((uint32_t)(FT_C >> 3) << 17) | ((uint32_t)(FT_TILE_M >> 4) << 24);
    p.idesc2 = (2u << 4) | (0u << 7) | (1u << 10) | ((uint32_t)(FT_N2 >> 3) << 17) | ((uint32_t)(FT_TILE_M >> 4) << 24);
    p.desc_hi = smem_desc_hi(FT_C);
    p.bias1 = bias1;
    p.bias2 = bias2;
    p.s1 = q1.s;
    p.mul1 = 1;
    p.sh_acc2 = q2.sh_acc;
    p.s2 = q2.s;
    p.mul_acc2 = 1 << q2.sh_acc;
    p.mul_res2 = 1 << q2.sh_res;
    p.r_signed = q2.r_signed;
    p.y_mid = (uint8_t *)y_mid;
    p.status = status_word;
    p.wait_limit = f8_wait_limit_cycles();
    plan->res = q2.has_res ? 1 : 0;
    plan->sgn = q2.y_kind == F8_S8 ? 1 : 0;
    {
        // A: the activation tensor (C, W, H, N) in im2col mode: lower corner -pad, upper corner pad - (k - 1)
        cuuint64_t dims[4] = {(cuuint64_t)g1.c, (cuuint64_t)g1.w, (cuuint64_t)g1.h, (cuuint64_t)g1.n};
        cuuint64_t strides[3] = {(cuuint64_t)g1.c, (cuuint64_t)g1.c * g1.w, (cuuint64_t)g1.c * g1.w * g1.h};
        int lower[2] = {-g1.pad_w, -g1.pad_h};
        int upper[2] = {g1.pad_w - (g1.kw - 1), g1.pad_h - (g1.kh - 1)};
        cuuint32_t estr[4] = {1, (cuuint32_t)g1.stride_w, (cuuint32_t)g1.stride_h, 1};
        CUresult r = ft_encode_im2col(&plan->map_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(x), dims, strides, lower, upper,
                                      (cuuint32_t)FT_C, (cuuint32_t)FT_TILE_M, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                      CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) {
            *why = "cuTensorMapEncodeIm2col rejected the activation tensor";
            return cudaErrorInvalidValue;
        }
    }
    {
        // weights (C, taps, C_out): one box per tap of the first layer, one box for the whole pointwise layer
        cuuint64_t dims1[3] = {(cuuint64_t)FT_C, (cuuint64_t)p.taps, (cuuint64_t)FT_C};
        cuuint64_t str1[2] = {(cuuint64_t)FT_C, (cuuint64_t)FT_C * p.taps};
        cuuint32_t box1[3] = {(cuuint32_t)FT_C, 1, (cuuint32_t)FT_C};
        cuuint64_t dims2[3] = {(cuuint64_t)FT_C, 1, (cuuint64_t)FT_N2};
        cuuint64_t str2[2] = {(cuuint64_t)FT_C, (cuuint64_t)FT_C};
        cuuint32_t box2[3] = {(cuuint32_t)FT_C, 1, (cuuint32_t)FT_N2};
        cuuint32_t estr[3] = {1, 1, 1};
        CUresult r = ft_encode_tiled(&plan->map_w1, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<int8_t *>(w1), dims1, str1, box1, estr,
                                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r == CUDA_SUCCESS)
            r = ft_encode_tiled(&plan->map_w2, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<int8_t *>(w2), dims2, str2, box2, estr,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) {
            *why = "cuTensorMapEncodeTiled rejected a weight tensor";
            return cudaErrorInvalidValue;
        }
    }
    {
        // output / shortcut [M, 256] bytes, one box = a 128-byte column slab of a tile
        cuuint64_t dims[2] = {(cuuint64_t)FT_N2, (cuuint64_t)p.M};
        cuuint64_t strides[1] = {(cuuint64_t)FT_N2};
        cuuint32_t box[2] = {128, (cuuint32_t)FT_TILE_M};
        cuuint32_t estr[2] = {1, 1};
        CUresult r = ft_encode_tiled(&plan->map_y, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, y, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        plan->map_r = plan->map_y;
        if (r == CUDA_SUCCESS && res)
            r = ft_encode_tiled(&plan->map_r, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(res), dims, strides, box, estr,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) {
            *why = "cuTensorMapEncodeTiled rejected the output tensor";
            return cudaErrorInvalidValue;
        }
    }
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    plan->grid = std::min(p.m_tiles, sms);
    static bool attr_set[64] = {false};
    if (dev < 0 || dev >= 64) {
        *why = "device index out of range";
        return cudaErrorInvalidDevice;
    }
    if (!attr_set[dev]) {
        const int bytes = (int)(FT_SMEM_LIMIT + FT_CONTROL_BYTES + 1024);
        cudaError_t e = cudaFuncSetAttribute(f8_conv_pw_fused_tc_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(f8_conv_pw_fused_tc_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(f8_conv_pw_fused_tc_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(f8_conv_pw_fused_tc_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e != cudaSuccess) {
            *why = "cudaFuncSetAttribute(MaxDynamicSharedMemorySize) failed";
            return e;
        }
        attr_set[dev] = true;
    }
    return cudaSuccess;
}

namespace {
template <bool RES, bool SGN>
cudaError_t ft_launch_variant(const F8FusedPlan *plan, bool overlap_previous, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)plan->grid);
    cfg.blockDim = dim3(FT_THREADS);
    cfg.dynamicSmemBytes = plan->smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    int n = 0;
    if (overlap_previous) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, f8_conv_pw_fused_tc_kernel<RES, SGN>, plan->map_a, plan->map_w1, plan->map_w2, plan->map_y, plan->map_r,
                              plan->p);
}
}   // namespace

cudaError_t f8_fused_launch(const F8FusedPlan *plan, bool overlap_previous, cudaStream_t st) {
    if (plan->p.M == 0) return cudaSuccess;
    if (plan->res) return plan->sgn ? ft_launch_variant<true, true>(plan, overlap_previous, st) : ft_launch_variant<true, false>(plan, overlap_previous, st);
    return plan->sgn ? ft_launch_variant<false, true>(plan, overlap_previous, st) : ft_launch_variant<false, false>(plan, overlap_previous, st);
}
