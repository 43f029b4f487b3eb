// Internal declarations shared by the CUDA sources of the library (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/f8net.h"

// How an int32 accumulator becomes an output element: bias has already been added.
//   v = has_res ? (acc << sh_acc) + (r << sh_res) : acc
//   y_kind 2: store v as int32
//   else    : t = s > 0 ? rounding right shift of v by s : v << -s ; y = clamp(t, lo, hi)
struct F8Requant {
    int sh_acc;     // F - (fl_x + fl_w), F = max(fl_x + fl_w, fl_r)   (0 without residual)
    int sh_res;     // F - fl_r
    int s;          // F - fl_y   in [-8, 31]
    int lo, hi;     // clip bounds of the output quantizer
    int y_kind;     // F8_U8 / F8_S8 / F8_S32 / F8_S32_RELU
    int has_res;
    int r_signed;
    int r_s32 = 0;  // the residual operand is an int32 tensor (a shortcut kept in 32 bits, Sec. 4.3)
};

// A second consumer of the same 32-bit sum, quantised with its private fractional length (Sec. 4.3).
struct F8Sibling {
    void *y2 = nullptr;     // nullptr: none
    int y_kind = 0;         // F8_U8 / F8_S8 / F8_S32 / F8_S32_RELU
    int s = 0;              // F - fl_y2
    int lo = 0, hi = 0;
};

// Geometry of one convolution-shaped launch (dense or depthwise).
struct F8ConvGeom {
    int n, h, w, c;         // input
    int ho, wo, c_out;      // output
    int kh, kw;
    int stride_h, stride_w;
    int pad_h, pad_w;
    int x_signed;
    int pad_h_end = -1;     // padding below the last row when it differs from pad_h (-1: symmetric)
};

// ---- CUDA-core kernels (f8_direct.cu) -------------------------------------------------
// overlap_previous: launch with programmatic stream serialization (the kernel itself waits for the grids
// before it prior to touching memory, so this is always safe; it lets launch latency overlap their tail).
cudaError_t f8_launch_conv_direct(const F8ConvGeom &g, const F8Requant &q, const void *x, const int8_t *w,
                                  const int32_t *bias, const void *res, void *y, cudaStream_t st,
                                  bool overlap_previous = false, const F8Sibling *sib = nullptr);
cudaError_t f8_launch_dwconv(const F8ConvGeom &g, const F8Requant &q, const void *x, const int8_t *w,
                             const int32_t *bias, const void *res, void *y, cudaStream_t st,
                             bool overlap_previous = false);
cudaError_t f8_launch_maxpool(int n, int h, int w, int c, int k, int stride, int pad, int x_signed,
                              const void *x, void *y, cudaStream_t st, bool overlap_previous = false);
cudaError_t f8_launch_gap(int n, int h, int w, int c, int x_signed, int s, const void *x, void *y,
                          cudaStream_t st, bool overlap_previous = false);
// channel-padding pre-pass for 3-channel stems: [n,h,w,c] -> [n,h,wp,8] with `left` zero pixels in front
cudaError_t f8_launch_pack_stem(int n, int h, int w, int c, int wp, int left, const void *x, void *y,
                                cudaStream_t st, bool overlap_previous = false);

// row-pair packing for stride-2 stems: [n,h,w,c<=8] -> [n,hp,wp] cells of 2*cpad bytes (cpad 4 or 8 >= c); the cell
// at column iw + left of row pair p holds pixel iw of image rows 2p and 2p+1 (cpad bytes each, zero filled)
cudaError_t f8_launch_pack_stem_pairs(int n, int h, int w, int c, int cpad, int hp, int wp, int left, const void *x,
                                      void *y, cudaStream_t st, bool overlap_previous = false);

// ---- tensor-core implicit GEMM (f8_gemm_tc.cu) ----------------------------------------
struct F8TcPlan;   // opaque: tensor maps + launch parameters of one conv launch

// Activation tensor as the TMA sees it: extents and byte strides of (C, W, H, N).
struct F8TcTensorView {
    const void *base;
    uint64_t dim_c, dim_w, dim_h, dim_n;
    uint64_t stride_w, stride_h, stride_n;   // bytes (stride of C is 1)
};

// True when this geometry can run on the tensor-core path.
bool f8_tc_supported(const F8ConvGeom &g, size_t x_bytes);
bool f8_tc_rowtile_ok(const F8ConvGeom &g);
size_t f8_tc_plan_size();
// Encodes tensor maps and tile schedule; returns cudaSuccess or an error (no launch).
cudaError_t f8_tc_plan_init(F8TcPlan *plan, const F8ConvGeom &g, const F8Requant &q, const F8TcTensorView &xv,
                            const int8_t *w /* [c_out][kh][kw][g.c] */, const int32_t *bias, const void *res,
                            void *y, int *status_word, const char **why, const F8Sibling *sib = nullptr);
// Label reported (with the wait's site) when a bounded wait of this launch gives up; 0 = none.
void f8_tc_plan_set_tag(F8TcPlan *plan, int tag);
// overlap_previous: the grid may start before the preceding work of the stream has finished; only its weight
// and bias reads then run early, so it is for callers whose weights no earlier work in the stream writes.
cudaError_t f8_tc_launch(const F8TcPlan *plan, bool overlap_previous, cudaStream_t st);
cudaError_t f8_tc_probe(int iters, double *ops, int *status_word, cudaStream_t st);
// One thread waits `limit_cycles` on a barrier nothing arrives at, records the time-out (site 199) and returns.
cudaError_t f8_tc_wait_probe(unsigned long long limit_cycles, int *status_word, cudaStream_t st);

// ---- two layers in one launch (f8_fused_tc.cu): a dense convolution 64 -> 64 channels (unsigned 8-bit output, no shortcut)
// followed by the pointwise convolution 64 -> 256 behind it (8-bit output, optional 8-bit shortcut).  The first layer's
// output stays in shared memory; y_mid (may be NULL) receives a copy of it.
struct F8FusedPlan;
bool f8_fused_supported(const F8ConvGeom &g1, const F8Requant &q1, int c_out2, const F8Requant &q2);
size_t f8_fused_plan_size();
cudaError_t f8_fused_plan_init(F8FusedPlan *plan, const F8ConvGeom &g1, const F8Requant &q1, const F8Requant &q2, const void *x,
                               const int8_t *w1, const int32_t *bias1, const int8_t *w2, const int32_t *bias2, const void *res,
                               void *y_mid, void *y, int *status_word, const char **why);
void f8_fused_plan_set_tag(F8FusedPlan *plan, int tag);
cudaError_t f8_fused_launch(const F8FusedPlan *plan, bool overlap_previous, cudaStream_t st);

// ---- first-layer kernel (f8_stem_tc.cu): stride-2 convolution over an image with <= 4 channels, optionally fused
// with the 3x3 / 2 / pad 1 max pool behind it.  kh2 row pairs per window starting `top` pairs above the output row,
// `left` zero cells in front of a row, `slices` 32-byte K slices per row pair; w_core is [K / 16][c_out][16].
bool f8_stem_tc_supported(const F8ConvGeom &g, const F8Requant &q, int kh2, int slices);
cudaError_t f8_launch_stem_tc(const F8ConvGeom &g, const F8Requant &q, int kh2, int top, int left, int slices, int pool,
                              const void *x, const int8_t *w_core, const int32_t *bias, void *y, int *status_word, int tag,
                              cudaStream_t st, bool overlap_previous);

// Device status word (0 = fine); allocated once per device on first use, together with a host-visible copy of its
// first word that kernels write through (f8_status_host_code reads it without synchronising).
int *f8_status_word();
int f8_status_host_code();

// Planning choices switched off by f8_debug_plan_options (F8_PLAN_OFF_* bits), the bound of in-kernel waits in SM
// cycles (0 = default) and the record of the last tensor-core plan (10 ints, see f8_debug_last_plan).
unsigned f8_plan_options_off();
unsigned long long f8_wait_limit_cycles();
int *f8_last_plan_info();

// Records a message for f8_last_error() and returns `s` (for entry points defined outside f8_api.cu).
f8_status f8_set_error(f8_status s, const char *message);
