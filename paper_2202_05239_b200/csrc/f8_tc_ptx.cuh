// PTX wrappers and the branch-free requantising epilogue shared by the tensor-core kernels (mbarriers with bounded
// waits, TMA loads / stores, tcgen05 allocation, MMA issue, accumulator loads, shared-memory matrix descriptors).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

constexpr unsigned long long WAIT_LIMIT_CYCLES = 4000000000ull;   // default bound of a wait: ~2 s at 2 GHz
constexpr unsigned MIN_POLLS_BEFORE_TIMEOUT = 1u << 16;             // failed polls a wait needs before it may give up
constexpr unsigned long long DRAIN_LIMIT_CYCLES = 200000000ull;

// What a bounded wait needs besides the barrier: where to raise the CTA's abort flag, where to record the wait
// that gave up, and how long to try.  limit_cycles is a launch parameter (0 = the default above).
struct WaitCtx {
    volatile int *abort_flag;
    int *status;
    unsigned long long limit_cycles;
    unsigned min_polls;
};
__device__ __forceinline__ WaitCtx make_wait_ctx(volatile int *abort_flag, int *status, unsigned long long limit_cycles) {
    WaitCtx c;
    c.abort_flag = abort_flag;
    c.status = status;
    c.limit_cycles = limit_cycles ? limit_cycles : WAIT_LIMIT_CYCLES;
    // a short limit is a test of the time-out path itself: it must not wait for the poll count of a real run
    c.min_polls = limit_cycles && limit_cycles < (1ull << 28) ? 256u : MIN_POLLS_BEFORE_TIMEOUT;
    return c;
}

// ----------------------------------------------------------------------------- PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Programmatic dependent launch.  A grid launched with the programmatic-serialization attribute may start
// while its predecessor in the stream is still running; grid_dependency_wait() returns once every
// predecessor has completed and its writes are visible (at once for an ordinary launch).  Everything that
// reads activations or writes the output sits behind it; the prologue and the weight loads do not.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// One attempt that may suspend the thread for up to about `ns` nanoseconds while the phase is incomplete.
__device__ __forceinline__ bool mbar_try_wait_hint(uint32_t bar, uint32_t parity, uint32_t ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(ns)
        : "memory");
    return ok != 0;
}

// Bounded wait.  Returns false when the kernel is aborting (this wait or another one ran out).
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, const WaitCtx &wc, int code) {
    volatile int *abort_flag = wc.abort_flag;
    int *status = wc.status;
    const unsigned long long t0 = clock64();
    unsigned long long g0 = 0;
    unsigned spins = 0;
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 63u) == 0) {
            // wall clock of a wait that is already long (reading it costs the warp a microsecond or so)
            if (spins == 4096u || (spins == 64u && wc.min_polls < 4096u)) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g0));
            if (*abort_flag) return false;
            // both conditions: the cycle counter keeps running while the context is switched out (a profiler
            // replaying the kernel does that for seconds), the poll count does not
            if (spins >= wc.min_polls && (unsigned long long)(clock64() - t0) > wc.limit_cycles) {
                *abort_flag = 1;
                if (atomicCAS(status, 0, code) == 0) {
                    // the first wait to give up leaves a description: CTA, thread, barrier address, parity
                    status[1] = (int)blockIdx.x;
                    status[2] = (int)threadIdx.x;
                    status[3] = (int)bar;
                    status[4] = (int)parity;
                    unsigned long long g1;
                    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g1));
                    const unsigned long long dc = clock64() - t0, dg = g1 - g0;
                    status[5] = (int)spins;
                    status[6] = (int)(dc >> 20);       // SM cycles / 2^20
                    status[7] = (int)(dg >> 10);       // wall-clock microseconds (ns / 1024) since the 4096th poll (the 64th under a short test limit)
                    // words 32 / 33 of the status buffer may hold the address of a word in host memory that the library
                    // reads without synchronising (0: none): the code goes there as well
                    int *host_copy = *(int *volatile *)(status + 32);
                    if (host_copy) {
                        *(volatile int *)host_copy = code;
                        __threadfence_system();
                    }
                }
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const WaitCtx &wc, int code) {
    if (mbar_try_wait(bar, parity)) return true;
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, wc, code);
}

__device__ __forceinline__ void tma_load_im2col(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c, int w,
                                                int h, int n, uint16_t off_w, uint16_t off_h) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};" ::"r"(dst),
        "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1,
                                            int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(dst),
        "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
        "l"(map), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2,
                                            int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(dst),
        "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
__device__ __forceinline__ void tma_store_4d(const CUtensorMap *map, uint32_t src, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];" ::"l"(map), "r"(src),
                 "r"(c0), "r"(c1), "r"(c2), "r"(c3)
                 : "memory");
}
// shared -> global tile store; rows / columns outside the tensor are clipped by the hardware
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, uint32_t src, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(map), "r"(src),
                 "r"(c0), "r"(c1)
                 : "memory");
}

// Brings a tensor map (a kernel parameter) into the descriptor cache ahead of its first use by a bulk tensor copy.
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]^T, int8 operands, int32 accumulate.
__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// The K = 32 slices of one sub-chunk (kb / 32 of them), issued from one asm block.  A lone thread pays a few
// cycles for every instruction it executes, and the tensor pipe is only kept busy when an MMA costs the
// issuing thread no more than a handful of them: the shared-memory descriptors of the slices differ only
// in their low words (start address, 16-byte units), so those are advanced with 32-bit adds inside the
// block and the constant high word (SBO, version, swizzle mode) is attached by a register-pair move.
#define F8_MMA_I8 "tcgen05.mma.cta_group::1.kind::i8 [%0], a, b, %4, "
#define F8_MMA_NEXT(off) \
    "add.u32 x, %1, " #off ";\n\tadd.u32 y, %2, " #off ";\n\tmov.b64 a, {x, %3};\n\tmov.b64 b, {y, %3};\n\t" F8_MMA_I8 "t;\n\t"
template <int MMAS>
__device__ __forceinline__ void mma_i8_sub(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi,
                                           uint32_t idesc, uint32_t accumulate) {
    if (MMAS == 1)
        asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 a, b;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                     "mov.b64 a, {%1, %3};\n\tmov.b64 b, {%2, %3};\n\t" F8_MMA_I8 "p;\n\t}" ::"r"(d_tmem),
                     "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate)
                     : "memory");
    else if (MMAS == 2)
        asm volatile("{\n\t.reg .pred p, t;\n\t.reg .b64 a, b;\n\t.reg .b32 x, y;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                     "setp.eq.b32 t, 0, 0;\n\tmov.b64 a, {%1, %3};\n\tmov.b64 b, {%2, %3};\n\t" F8_MMA_I8 "p;\n\t"
                     F8_MMA_NEXT(2) "}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate)
                     : "memory");
    else
        asm volatile("{\n\t.reg .pred p, t;\n\t.reg .b64 a, b;\n\t.reg .b32 x, y;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                     "setp.eq.b32 t, 0, 0;\n\tmov.b64 a, {%1, %3};\n\tmov.b64 b, {%2, %3};\n\t" F8_MMA_I8 "p;\n\t"
                     F8_MMA_NEXT(2) F8_MMA_NEXT(4) F8_MMA_NEXT(6) "}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi),
                     "r"(idesc), "r"(accumulate)
                     : "memory");
}

// All sub-chunks of one stage use; `a_lo` / `b_lo` are the low descriptor words of its first A / B tile.
template <int MMAS>
__device__ __forceinline__ void mma_i8_stage(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t a_step,
                                             uint32_t b_step, uint32_t desc_hi, uint32_t idesc, int subs,
                                             uint32_t accumulate_first) {
    mma_i8_sub<MMAS>(d_tmem, a_lo, b_lo, desc_hi, idesc, accumulate_first);
    for (int j = 1; j < subs; ++j) {
        a_lo += a_step;
        b_lo += b_step;
        mma_i8_sub<MMAS>(d_tmem, a_lo, b_lo, desc_hi, idesc, 1u);
    }
}
// mbarrier arrives once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                 : "memory");
}

// ----------------------------------------------------------------------------- CTA pairs (tcgen05 cta_group::2)
// Two CTAs of a cluster work on one 256-row tile: each holds its own 128 rows of A and half of the B tile in its shared
// memory (same offsets in both), the even CTA issues the instructions, each tensor core accumulates its 128 rows in its own
// tensor memory.  Loads of the odd CTA complete on the even CTA's barrier; commits arrive on the barriers of both.

__device__ __forceinline__ uint32_t cluster_cta_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.aligned;" ::: "memory");
}
// arrive on the barrier at the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar, uint32_t rank) {
    asm volatile(
        "{\n\t.reg .b32 remote;\n\t"
        "mapa.shared::cluster.u32 remote, %0, %1;\n\t"
        "mbarrier.arrive.shared::cluster.b64 _, [remote];\n\t}" ::"r"(bar), "r"(rank)
        : "memory");
}
// the barrier at the same offset in the even CTA of the pair (the CTA rank is bit 24 of a shared-window address)
__device__ __forceinline__ uint32_t pair_leader_bar(uint32_t bar) { return bar & 0xFEFFFFFFu; }

__device__ __forceinline__ void tma_load_im2col_pair(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c, int w, int h,
                                                     int n, uint16_t off_w, uint16_t off_h) {
    asm volatile(
        "cp.async.bulk.tensor.4d.im2col.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};" ::"r"(dst),
        "l"(map), "r"(pair_leader_bar(bar)), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(dst),
        "l"(map), "r"(pair_leader_bar(bar)), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
        "l"(map), "r"(pair_leader_bar(bar)), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// arrives on the barrier at this offset in both CTAs of the pair once every MMA issued so far by this thread has completed
__device__ __forceinline__ void mma_commit_pair(uint32_t bar) {
    const uint16_t both = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
                 "h"(both)
                 : "memory");
}
// The K = 32 slices of one 128-byte sub-chunk (four of them) as 256-row instructions of the pair, from one asm block.
#define F8_MMA_I8_PAIR "tcgen05.mma.cta_group::2.kind::i8 [%0], a, b, %4, {%6, %6, %6, %6, %6, %6, %6, %6}, "
#define F8_MMA_NEXT_PAIR(off) \
    "add.u32 x, %1, " #off ";\n\tadd.u32 y, %2, " #off ";\n\tmov.b64 a, {x, %3};\n\tmov.b64 b, {y, %3};\n\t" F8_MMA_I8_PAIR "t;\n\t"
__device__ __forceinline__ void mma_i8_sub_pair4(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc,
                                                 uint32_t accumulate) {
    const uint32_t zero = 0;      // no output lane is disabled
    asm volatile("{\n\t.reg .pred p, t;\n\t.reg .b64 a, b;\n\t.reg .b32 x, y;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                 "setp.eq.b32 t, 0, 0;\n\tmov.b64 a, {%1, %3};\n\tmov.b64 b, {%2, %3};\n\t" F8_MMA_I8_PAIR "p;\n\t"
                 F8_MMA_NEXT_PAIR(2) F8_MMA_NEXT_PAIR(4) F8_MMA_NEXT_PAIR(6) "}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi),
                 "r"(idesc), "r"(accumulate), "r"(zero)
                 : "memory");
}

// 16 consecutive accumulator columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, int (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, "
        "%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile whose rows are `kb` bytes long and swizzled with
// the matching TMA mode: 8-row groups are 8*kb bytes apart (stride byte offset), the leading offset
// is unused (1), descriptor version 1, layout code 2 / 4 / 6 for 128 / 64 / 32-byte swizzle.
__host__ __device__ inline uint64_t smem_desc_hi(int kb) {
    const uint64_t layout = kb == 128 ? 2 : (kb == 64 ? 4 : 6);
    const uint64_t sbo = (uint64_t)(8 * kb) >> 4;
    return ((uint64_t)1 << 16) | (sbo << 32) | ((uint64_t)1 << 46) | (layout << 61);
}

// Branch-free epilogue for the common case (8-bit output, 1 <= s <= 24, c_out % 16 == 0).
//   v = acc * 2^sh_acc + bias'          bias' = (bias << sh_acc) + 2^(s-1), staged in shared memory
//   v += r << sh_res                    (RES only)
//   t = v >> s                          = floor((acc' + 2^(s-1)) / 2^s), round half up (the same floor taken as the high
//                                       word of v * 2^(32-s), to move it to the multiplier pipe, measured 2 % slower)
//   y = clamp(t, lo, hi)                saturating pack; the signed quantizer additionally excludes -128
// cvt.pack.sat packs two saturated values into the low half of d and moves the low half of c above
// them: d = (c << 16) | (sat(a) << 8) | sat(b).
// The integer ALU pipe (shifts, byte permutes, 3-input adds, packs) issues a warp instruction every other
// cycle and is what bounds this code, so work is kept off it: the two scalings are multiply-adds whose
// power-of-two factors arrive as opaque kernel parameters (the FMA pipe; a visible 1 << n would be turned
// into shifts), a residual byte costs one PRMT whose selector (zero- or sign-extending) sits in a register,
// and bias / residual / output go through explicit shared-space accesses.
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint4 v) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

template <bool RES, bool SIGNED_OUT>
__device__ __forceinline__ uint4 epilogue_fast16(const int (&acc)[16], uint32_t bias_addr, uint4 rw, int mul_acc,
                                                 int mul_res, const uint32_t (&rsel)[4], int s) {
    int t[16];
    const uint32_t rwords[4] = {rw.x, rw.y, rw.z, rw.w};
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        const uint4 b = lds128(bias_addr + 16 * g);
        const int bb[4] = {(int)b.x, (int)b.y, (int)b.z, (int)b.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int j = 4 * g + k;
#ifdef F8_EPILOGUE_SHIFTS_ONLY
            // the letter of the method: alignment by shift instructions (the factors are powers of two)
            int v = (acc[j] << (31 - __clz(mul_acc))) + bb[k];
            if (RES) {
                int r;
                asm("prmt.b32 %0, %1, 0, %2;" : "=r"(r) : "r"(rwords[g]), "r"(rsel[k]));
                v += r << (31 - __clz(mul_res));
            }
#else
            int v = acc[j] * mul_acc + bb[k];
            if (RES) {
                int r;
                asm("prmt.b32 %0, %1, 0, %2;" : "=r"(r) : "r"(rwords[g]), "r"(rsel[k]));
                v += r * mul_res;
            }
#endif
            v >>= s;
            t[j] = SIGNED_OUT ? max(v, -127) : v;
        }
    }
    uint32_t o[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        uint32_t hi2;
        if (SIGNED_OUT) {
            asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, 0;" : "=r"(hi2) : "r"(t[4 * g + 3]), "r"(t[4 * g + 2]));
            asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(o[g]) : "r"(t[4 * g + 1]), "r"(t[4 * g]), "r"(hi2));
        } else {
            asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, 0;" : "=r"(hi2) : "r"(t[4 * g + 3]), "r"(t[4 * g + 2]));
            asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(o[g]) : "r"(t[4 * g + 1]), "r"(t[4 * g]), "r"(hi2));
        }
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

}   // namespace
