// C ABI: argument validation, dispatch to the kernels, and the whole-network executor.
#include <cuda_runtime.h>

#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <memory>
#include <new>
#include <vector>

#include "f8_internal.h"

namespace {

thread_local char g_err[512] = "";
bool g_force_direct = false;
long long g_tc_launches = 0;
unsigned g_plan_off = 0;                      // F8_PLAN_OFF_* bits (test hook)
unsigned long long g_wait_limit_cycles = 0;   // 0: the kernels' default
int g_last_plan[10] = {0};
int g_micro_batch = 0;                        // 0: no micro-batching; > 0: this micro-batch in every eligible run; -1: the L2 rule
int g_lanes = 0;                              // 0: automatic; 1 / 2: that many concurrent lanes in f8_net_forward

f8_status fail(f8_status s, const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return s;
}

f8_status cuda_fail(cudaError_t e, const char *what) {
    return fail(F8_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

bool aligned16(const void *p) { return ((uintptr_t)p & 15) == 0; }

int ceil_log2(long long v) {
    int d = 0;
    while ((1ll << d) < v) ++d;
    return d;
}

// Validates one conv-shaped descriptor and derives geometry + requantisation parameters.
f8_status check_conv(const f8_conv_desc *d, bool depthwise, bool has_res, F8ConvGeom *g, F8Requant *q,
                     bool siblings = false /* accept a 32-bit shortcut and the F8_S32_RELU output */) {
    if (!d) return fail(F8_ERR_NULL, "descriptor is NULL");
    if (d->n < 0 || d->h <= 0 || d->w <= 0 || d->c <= 0 || d->c_out <= 0 || d->kh <= 0 || d->kw <= 0 ||
        d->stride <= 0 || d->pad < 0)
        return fail(F8_ERR_SHAPE, "non-positive extent in descriptor");
    if (depthwise && d->c_out != d->c) return fail(F8_ERR_SHAPE, "depthwise layers need c_out == c");
    const int ho = (d->h + 2 * d->pad - d->kh) / d->stride + 1;
    const int wo = (d->w + 2 * d->pad - d->kw) / d->stride + 1;
    if (d->h + 2 * d->pad < d->kh || d->w + 2 * d->pad < d->kw || ho <= 0 || wo <= 0)
        return fail(F8_ERR_SHAPE, "filter larger than the padded image");
    if ((long long)d->n * ho * wo * d->c_out >= (1ll << 40) || (long long)d->n * d->h * d->w * d->c >= (1ll << 40))
        return fail(F8_ERR_SHAPE, "tensor too large");
    if (d->x_dtype != F8_U8 && d->x_dtype != F8_S8) return fail(F8_ERR_DTYPE, "x_dtype must be F8_U8 or F8_S8");
    if (d->y_dtype != F8_U8 && d->y_dtype != F8_S8 && d->y_dtype != F8_S32 && !(siblings && d->y_dtype == F8_S32_RELU))
        return fail(F8_ERR_DTYPE, "y_dtype must be F8_U8, F8_S8 or F8_S32");
    if (d->fl_x < 0 || d->fl_x > (d->x_dtype == F8_U8 ? 8 : 7))
        return fail(F8_ERR_FL_RANGE, "fl_x = %d outside the 8-bit format range", d->fl_x);
    if (d->fl_w < -8 || d->fl_w > 24) return fail(F8_ERR_FL_RANGE, "fl_w = %d outside [-8, 24]", d->fl_w);
    int fa = d->fl_x + d->fl_w;
    q->sh_acc = q->sh_res = 0;
    q->has_res = has_res ? 1 : 0;
    q->r_signed = 0;
    q->r_s32 = 0;
    if (has_res) {
        const bool r32 = siblings && d->r_dtype == F8_S32;
        if (d->r_dtype != F8_U8 && d->r_dtype != F8_S8 && !r32) return fail(F8_ERR_DTYPE, "r_dtype must be F8_U8 or F8_S8");
        if (d->fl_r < 0 || d->fl_r > (r32 ? 31 : (d->r_dtype == F8_U8 ? 8 : 7)))
            return fail(F8_ERR_FL_RANGE, "fl_r = %d outside the accepted range", d->fl_r);
        q->r_s32 = r32 ? 1 : 0;
        const int f = std::max(fa, d->fl_r);
        q->sh_acc = f - fa;
        q->sh_res = f - d->fl_r;
        q->r_signed = d->r_dtype == F8_S8;
        if (q->sh_acc > 22 || q->sh_res > 22)
            return fail(F8_ERR_SHIFT_RANGE, "residual alignment shift %d / %d exceeds 22", q->sh_acc, q->sh_res);
        fa = f;
    }
    q->y_kind = d->y_dtype;
    if (d->y_dtype == F8_S32 || d->y_dtype == F8_S32_RELU) {
        q->s = 0;
        q->lo = q->hi = 0;
    } else {
        if (d->fl_y < 0 || d->fl_y > (d->y_dtype == F8_U8 ? 8 : 7))
            return fail(F8_ERR_FL_RANGE, "fl_y = %d outside the 8-bit format range", d->fl_y);
        q->s = fa - d->fl_y;
        if (q->s < -8 || q->s > 31) return fail(F8_ERR_SHIFT_RANGE, "requantisation shift %d outside [-8, 31]", q->s);
        q->lo = d->y_dtype == F8_U8 ? 0 : -127;
        q->hi = d->y_dtype == F8_U8 ? 255 : 127;
    }
    // shape-level accumulator bound: |sum| <= K * 255 * 128 (or 128 * 128) must leave room for bias / residual
    const long long k = (long long)d->kh * d->kw * (depthwise ? 1 : d->c);
    const long long worst = k * (d->x_dtype == F8_U8 ? 255ll : 128ll) * 128ll;
    if ((worst << q->sh_acc) >= (1ll << 30))
        return fail(F8_ERR_ACC_BOUND, "K = %lld taps cannot be guaranteed to fit the int32 accumulator", k);
    g->n = d->n; g->h = d->h; g->w = d->w; g->c = d->c;
    g->ho = ho; g->wo = wo; g->c_out = d->c_out;
    g->kh = d->kh; g->kw = d->kw;
    g->stride_h = g->stride_w = d->stride;
    g->pad_h = g->pad_w = d->pad;
    g->x_signed = d->x_dtype == F8_S8;
    return F8_OK;
}

F8TcTensorView dense_view(const void *x, const F8ConvGeom &g) {
    F8TcTensorView v;
    v.base = x;
    v.dim_c = g.c; v.dim_w = g.w; v.dim_h = g.h; v.dim_n = g.n;
    v.stride_w = (uint64_t)g.c;
    v.stride_h = (uint64_t)g.c * g.w;
    v.stride_n = (uint64_t)g.c * g.w * g.h;
    return v;
}

struct PlanDeleter { void operator()(F8TcPlan *p) const { free(p); } };
using PlanPtr = std::unique_ptr<F8TcPlan, PlanDeleter>;

// tensor maps inside the plan are 64-byte aligned objects
PlanPtr alloc_plan() {
    const size_t size = (f8_tc_plan_size() + 63) / 64 * 64;
    void *p = aligned_alloc(64, size);
    if (p) memset(p, 0, size);
    return PlanPtr((F8TcPlan *)p);
}

struct FusedPlanDeleter { void operator()(F8FusedPlan *p) const { free(p); } };
using FusedPlanPtr = std::unique_ptr<F8FusedPlan, FusedPlanDeleter>;

FusedPlanPtr alloc_fused_plan() {
    const size_t size = (f8_fused_plan_size() + 63) / 64 * 64;
    void *p = aligned_alloc(64, size);
    if (p) memset(p, 0, size);
    return FusedPlanPtr((F8FusedPlan *)p);
}

// The second consumer of a layer's sum: its quantizer relative to the format F of the aligned sum.
f8_status make_sibling(const f8_conv_desc *d, const F8Requant &q, int y2_dtype, int fl_y2, void *y2, F8Sibling *sib) {
    if (y2_dtype != F8_U8 && y2_dtype != F8_S8 && y2_dtype != F8_S32 && y2_dtype != F8_S32_RELU)
        return fail(F8_ERR_DTYPE, "y2_dtype must be F8_U8, F8_S8, F8_S32 or F8_S32_RELU");
    sib->y2 = y2;
    sib->y_kind = y2_dtype;
    sib->s = 0;
    sib->lo = sib->hi = 0;
    if (y2_dtype == F8_U8 || y2_dtype == F8_S8) {
        if (fl_y2 < 0 || fl_y2 > (y2_dtype == F8_U8 ? 8 : 7))
            return fail(F8_ERR_FL_RANGE, "fl_y2 = %d outside the 8-bit format range", fl_y2);
        const int f = d->fl_x + d->fl_w + q.sh_acc;        // format of the aligned sum
        sib->s = f - fl_y2;
        if (sib->s < -8 || sib->s > 31) return fail(F8_ERR_SHIFT_RANGE, "requantisation shift %d of the second output outside [-8, 31]", sib->s);
        sib->lo = y2_dtype == F8_U8 ? 0 : -127;
        sib->hi = y2_dtype == F8_U8 ? 255 : 127;
    }
    return F8_OK;
}

f8_status run_dense(const F8ConvGeom &g, const F8Requant &q, const void *x, const int8_t *w, const int32_t *bias,
                    const void *res, void *y, cudaStream_t st, const F8Sibling *sib = nullptr) {
    if (g.n == 0) return F8_OK;
    const size_t x_bytes = (size_t)g.n * g.h * g.w * g.c;
    if (!g_force_direct && f8_tc_supported(g, x_bytes)) {
        PlanPtr plan = alloc_plan();
        if (!plan) return fail(F8_ERR_CUDA, "out of host memory");
        const char *why = "";
        cudaError_t e = f8_tc_plan_init(plan.get(), g, q, dense_view(x, g), w, bias, res, y, f8_status_word(), &why, sib);
        if (e == cudaSuccess) {
            e = f8_tc_launch(plan.get(), false, st);   // the caller's weights may come from earlier work in the stream
            if (e != cudaSuccess) return cuda_fail(e, "tensor-core conv launch");
            ++g_tc_launches;
            return F8_OK;
        }
        if (e != cudaErrorInvalidValue && e != cudaErrorNotSupported) return cuda_fail(e, why);
        // the tensor map could not be encoded for this shape: take the CUDA-core kernel
        (void)cudaGetLastError();
    }
    cudaError_t e = f8_launch_conv_direct(g, q, x, w, bias, res, y, st, false, sib);
    if (e != cudaSuccess) return cuda_fail(e, "direct conv launch");
    return F8_OK;
}

}   // namespace

f8_status f8_set_error(f8_status s, const char *message) { return fail(s, "%s", message); }

unsigned f8_plan_options_off() { return g_plan_off; }
unsigned long long f8_wait_limit_cycles() { return g_wait_limit_cycles; }
int *f8_last_plan_info() { return g_last_plan; }

namespace {
int *g_status_words[64] = {nullptr};
volatile int *g_status_host[64] = {nullptr};     // page-locked host word a kernel that gives up a wait writes its code to
}   // namespace

int *f8_status_word() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!g_status_words[dev]) {
        int *p = nullptr;
        if (cudaMalloc(&p, 256) != cudaSuccess) return nullptr;
        cudaMemset(p, 0, 256);
        // a host-visible copy of the first word: kernels store to it through its device address (words 32 / 33 of the
        // buffer), the host reads it directly -- f8_net_forward can then report a time-out without touching a stream
        int *h = nullptr, *h_dev = nullptr;
        if (cudaHostAlloc((void **)&h, 64, cudaHostAllocMapped) == cudaSuccess && cudaHostGetDevicePointer((void **)&h_dev, h, 0) == cudaSuccess) {
            memset(h, 0, 64);
            cudaMemcpy(p + 32, &h_dev, sizeof(h_dev), cudaMemcpyHostToDevice);
            g_status_host[dev] = h;
        } else {
            (void)cudaGetLastError();
        }
        g_status_words[dev] = p;
    }
    return g_status_words[dev];
}

// 0, or the code of a wait some kernel on the current device has given up since the last f8_device_status().
int f8_status_host_code() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64 || !g_status_host[dev]) return 0;
    return *g_status_host[dev];
}

// A kernel that gives up a bounded wait also stores its code to a host-visible word.  Every entry point that enqueues work
// looks at it first (a plain host load, no synchronisation), so an incomplete earlier result is reported by the next call.
static f8_status pending_timeout() {
    if (const int v = f8_status_host_code())
        return fail(F8_ERR_TIMEOUT, "a kernel abandoned a bounded wait (site %d, layer %d): the output of that launch is incomplete; "
                    "f8_device_status() gives the details and clears the record", v & 0xff, (v >> 8) - 1);
    return F8_OK;
}

extern "C" {

const char *f8_status_str(f8_status s) {
    switch (s) {
        case F8_OK: return "F8_OK";
        case F8_ERR_NULL: return "F8_ERR_NULL";
        case F8_ERR_SHAPE: return "F8_ERR_SHAPE";
        case F8_ERR_DTYPE: return "F8_ERR_DTYPE";
        case F8_ERR_FL_RANGE: return "F8_ERR_FL_RANGE";
        case F8_ERR_SHIFT_RANGE: return "F8_ERR_SHIFT_RANGE";
        case F8_ERR_ALIGN: return "F8_ERR_ALIGN";
        case F8_ERR_ACC_BOUND: return "F8_ERR_ACC_BOUND";
        case F8_ERR_WORKSPACE: return "F8_ERR_WORKSPACE";
        case F8_ERR_UNSUPPORTED: return "F8_ERR_UNSUPPORTED";
        case F8_ERR_CUDA: return "F8_ERR_CUDA";
        case F8_ERR_TIMEOUT: return "F8_ERR_TIMEOUT";
    }
    return "F8_ERR_?";
}

const char *f8_last_error(void) { return g_err; }

long long f8_tc_launch_count(void) { return g_tc_launches; }

// Test hook: non-zero routes every dense layer to the CUDA-core kernel.
void f8_debug_force_direct(int on) { g_force_direct = on != 0; }

void f8_debug_plan_options(unsigned off_mask) { g_plan_off = off_mask; }

void f8_debug_set_micro_batch(int images) { g_micro_batch = images > 0 ? images : (images < 0 ? -1 : 0); }

void f8_debug_set_lanes(int lanes) { g_lanes = lanes == 1 || lanes == 2 ? lanes : 0; }

int f8_debug_last_plan(int *info, int n) {
    if (!info || n <= 0) return 0;
    const int m = n < 10 ? n : 10;
    for (int i = 0; i < m; ++i) info[i] = g_last_plan[i];
    return m;
}

void f8_debug_set_wait_limit_ms(double ms) {
    int dev = 0, khz = 1965000;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev);
    g_wait_limit_cycles = ms > 0 ? (unsigned long long)(ms * (double)khz) : 0ull;
    if (ms > 0 && g_wait_limit_cycles == 0) g_wait_limit_cycles = 1;
}

f8_status f8_debug_wait_timeout_probe(double limit_ms, void *cuda_stream) {
    if (!(limit_ms > 0) || limit_ms > 100.0) return fail(F8_ERR_SHAPE, "limit_ms must be in (0, 100]");
    int *w = f8_status_word();
    if (!w) return fail(F8_ERR_CUDA, "no status word");
    int dev = 0, khz = 1965000;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev);
    unsigned long long cycles = (unsigned long long)(limit_ms * (double)khz);
    if (cycles == 0) cycles = 1;
    cudaError_t e = f8_tc_wait_probe(cycles, w, (cudaStream_t)cuda_stream);
    if (e != cudaSuccess) return cuda_fail(e, "wait probe launch");
    return F8_OK;
}

f8_status f8_device_status(void) {
    int *w = f8_status_word();
    if (!w) return fail(F8_ERR_CUDA, "no status word");
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceSynchronize");
    int v[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    e = cudaMemcpy(v, w, sizeof(v), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e, "status read");
    {
        int dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64 && g_status_host[dev]) *g_status_host[dev] = 0;
    }
    if (v[0] != 0) {
        cudaMemset(w, 0, sizeof(v));
        return fail(F8_ERR_TIMEOUT, "a kernel abandoned a bounded wait (site %d, layer %d, block %d, thread %d, barrier 0x%x, parity %d; "
                    "%d polls, %.0f Mcycles, %.3f ms)",
                    v[0] & 0xff, (v[0] >> 8) - 1, v[1], v[2], (unsigned)v[3], v[4], v[5], v[6] * 1.048576, v[7] * 1.024e-3);
    }
    return F8_OK;
}

size_t f8_conv_workspace_bytes(const f8_conv_desc *) { return 0; }

f8_status f8_conv2d_fixed(const f8_conv_desc *desc, const void *x, const int8_t *w, const int32_t *bias,
                          const void *residual, void *y, void *, size_t, void *cuda_stream) {
    F8ConvGeom g;
    F8Requant q;
    f8_status s = check_conv(desc, false, residual != nullptr, &g, &q);
    if (s != F8_OK) return s;
    if (g.n == 0) return F8_OK;
    if (!x || !w || !y) return fail(F8_ERR_NULL, "x, w and y must not be NULL");
    if (!aligned16(x) || !aligned16(w) || !aligned16(y) || !aligned16(residual) || !aligned16(bias))
        return fail(F8_ERR_ALIGN, "device pointers must be 16-byte aligned");
    if (pending_timeout() != F8_OK) return F8_ERR_TIMEOUT;
    return run_dense(g, q, x, w, bias, residual, y, (cudaStream_t)cuda_stream);
}

f8_status f8_conv2d_siblings_fixed(const f8_conv_desc *desc, int y2_dtype, int fl_y2, const void *x, const int8_t *w,
                                   const int32_t *bias, const void *residual, void *y, void *y2, void *, size_t,
                                   void *cuda_stream) {
    F8ConvGeom g;
    F8Requant q;
    f8_status s = check_conv(desc, false, residual != nullptr, &g, &q, true);
    if (s != F8_OK) return s;
    F8Sibling sib;
    if (y2) {
        s = make_sibling(desc, q, y2_dtype, fl_y2, y2, &sib);
        if (s != F8_OK) return s;
    }
    if (g.n == 0) return F8_OK;
    if (!x || !w || !y) return fail(F8_ERR_NULL, "x, w and y must not be NULL");
    if (!aligned16(x) || !aligned16(w) || !aligned16(y) || !aligned16(y2) || !aligned16(residual) || !aligned16(bias))
        return fail(F8_ERR_ALIGN, "device pointers must be 16-byte aligned");
    if (pending_timeout() != F8_OK) return F8_ERR_TIMEOUT;
    return run_dense(g, q, x, w, bias, residual, y, (cudaStream_t)cuda_stream, y2 ? &sib : nullptr);
}

f8_status f8_conv_pointwise_fixed(const f8_conv_desc *conv, const f8_conv_desc *pw, const void *x, const int8_t *w_conv,
                                  const int32_t *bias_conv, const int8_t *w_pw, const int32_t *bias_pw, const void *residual,
                                  void *y_mid, void *y, void *cuda_stream) {
    F8ConvGeom g1, g2;
    F8Requant q1, q2;
    f8_status s = check_conv(conv, false, false, &g1, &q1);
    if (s != F8_OK) return s;
    s = check_conv(pw, false, residual != nullptr, &g2, &q2);
    if (s != F8_OK) return s;
    if (pw->n != conv->n || pw->h != g1.ho || pw->w != g1.wo || pw->c != conv->c_out || pw->kh != 1 || pw->kw != 1 || pw->stride != 1 ||
        pw->pad != 0)
        return fail(F8_ERR_SHAPE, "the second layer must be a 1x1 convolution over the first layer's output");
    if (pw->x_dtype != conv->y_dtype || pw->fl_x != conv->fl_y)
        return fail(F8_ERR_DTYPE, "the second layer's input format must be the first layer's output format");
    if (g1.n == 0) return F8_OK;
    if (!x || !w_conv || !w_pw || !y) return fail(F8_ERR_NULL, "x, both weight tensors and y must not be NULL");
    if (!aligned16(x) || !aligned16(w_conv) || !aligned16(w_pw) || !aligned16(y) || !aligned16(y_mid) || !aligned16(residual) ||
        !aligned16(bias_conv) || !aligned16(bias_pw))
        return fail(F8_ERR_ALIGN, "device pointers must be 16-byte aligned");
    if (!f8_fused_supported(g1, q1, g2.c_out, q2))
        return fail(F8_ERR_UNSUPPORTED, "the two-layer kernel takes 64 -> 64 -> 256 channels, an unsigned 8-bit tensor between the layers, "
                                        "shifts in 1..24 and an input of at least 128 KiB");
    if (pending_timeout() != F8_OK) return F8_ERR_TIMEOUT;
    const size_t size = (f8_fused_plan_size() + 63) / 64 * 64;
    F8FusedPlan *plan = (F8FusedPlan *)aligned_alloc(64, size);
    if (!plan) return fail(F8_ERR_CUDA, "out of host memory");
    const char *why = "";
    cudaError_t e = f8_fused_plan_init(plan, g1, q1, q2, x, w_conv, bias_conv, w_pw, bias_pw, residual, y_mid, y, f8_status_word(), &why);
    if (e == cudaSuccess) e = f8_fused_launch(plan, false, (cudaStream_t)cuda_stream);
    free(plan);
    if (e != cudaSuccess) return cuda_fail(e, *why ? why : "two-layer kernel launch");
    ++g_tc_launches;
    return F8_OK;
}

f8_status f8_dwconv_fixed(const f8_conv_desc *desc, const void *x, const int8_t *w, const int32_t *bias,
                          const void *residual, void *y, void *, size_t, void *cuda_stream) {
    F8ConvGeom g;
    F8Requant q;
    f8_status s = check_conv(desc, true, residual != nullptr, &g, &q);
    if (s != F8_OK) return s;
    if (g.n == 0) return F8_OK;
    if (!x || !w || !y) return fail(F8_ERR_NULL, "x, w and y must not be NULL");
    if (!aligned16(x) || !aligned16(w) || !aligned16(y) || !aligned16(residual) || !aligned16(bias))
        return fail(F8_ERR_ALIGN, "device pointers must be 16-byte aligned");
    if (pending_timeout() != F8_OK) return F8_ERR_TIMEOUT;
    cudaError_t e = f8_launch_dwconv(g, q, x, w, bias, residual, y, (cudaStream_t)cuda_stream);
    if (e != cudaSuccess) return cuda_fail(e, "depthwise launch");
    return F8_OK;
}

f8_status f8_linear_fixed(int n, int k, int out, int x_dtype, int y_dtype, int fl_x, int fl_w, int fl_y, const void *x,
                          const int8_t *w, const int32_t *bias, void *y, void *, size_t, void *cuda_stream) {
    f8_conv_desc d;
    memset(&d, 0, sizeof(d));
    d.n = n; d.h = 1; d.w = 1; d.c = k; d.c_out = out; d.kh = d.kw = 1; d.stride = 1; d.pad = 0;
    d.x_dtype = x_dtype; d.y_dtype = y_dtype; d.fl_x = fl_x; d.fl_w = fl_w; d.fl_y = fl_y;
    return f8_conv2d_fixed(&d, x, w, bias, nullptr, y, nullptr, 0, cuda_stream);
}

f8_status f8_maxpool_fixed(int n, int h, int w, int c, int k, int stride, int pad, int x_dtype, const void *x, void *y,
                           void *cuda_stream) {
    if (n < 0 || h <= 0 || w <= 0 || c <= 0 || k <= 0 || stride <= 0 || pad < 0 || pad >= k || h + 2 * pad < k ||
        w + 2 * pad < k)
        return fail(F8_ERR_SHAPE, "bad pooling geometry");
    if (x_dtype != F8_U8 && x_dtype != F8_S8) return fail(F8_ERR_DTYPE, "x_dtype must be F8_U8 or F8_S8");
    if (n == 0) return F8_OK;
    if (!x || !y) return fail(F8_ERR_NULL, "x and y must not be NULL");
    if (!aligned16(x) || !aligned16(y)) return fail(F8_ERR_ALIGN, "device pointers must be 16-byte aligned");
    if (pending_timeout() != F8_OK) return F8_ERR_TIMEOUT;
    cudaError_t e = f8_launch_maxpool(n, h, w, c, k, stride, pad, x_dtype == F8_S8, x, y, (cudaStream_t)cuda_stream);
    if (e != cudaSuccess) return cuda_fail(e, "max-pool launch");
    return F8_OK;
}

f8_status f8_global_avgpool_fixed(int n, int h, int w, int c, int x_dtype, int fl_x, int fl_y, const void *x, void *y,
                                  void *cuda_stream) {
    if (n < 0 || h <= 0 || w <= 0 || c <= 0 || (long long)h * w > (1 << 22)) return fail(F8_ERR_SHAPE, "bad pooling geometry");
    if (x_dtype != F8_U8 && x_dtype != F8_S8) return fail(F8_ERR_DTYPE, "x_dtype must be F8_U8 or F8_S8");
    const int fmax = x_dtype == F8_U8 ? 8 : 7;
    if (fl_x < 0 || fl_x > fmax || fl_y < 0 || fl_y > fmax) return fail(F8_ERR_FL_RANGE, "fl outside the 8-bit format range");
    const int s = ceil_log2((long long)h * w) + fl_x - fl_y;
    if (s < -8 || s > 31) return fail(F8_ERR_SHIFT_RANGE, "shift %d outside [-8, 31]", s);
    if (n == 0) return F8_OK;
    if (!x || !y) return fail(F8_ERR_NULL, "x and y must not be NULL");
    if (!aligned16(x) || !aligned16(y)) return fail(F8_ERR_ALIGN, "device pointers must be 16-byte aligned");
    if (pending_timeout() != F8_OK) return F8_ERR_TIMEOUT;
    cudaError_t e = f8_launch_gap(n, h, w, c, x_dtype == F8_S8, s, x, y, (cudaStream_t)cuda_stream);
    if (e != cudaSuccess) return cuda_fail(e, "global-average-pool launch");
    return F8_OK;
}

f8_status f8_mma_i8_probe(int iters, double *ops, void *cuda_stream) {
    if (!ops) return fail(F8_ERR_NULL, "ops is NULL");
    if (iters <= 0 || iters > (1 << 24)) return fail(F8_ERR_SHAPE, "iters out of range");
    cudaError_t e = f8_tc_probe(iters, ops, f8_status_word(), (cudaStream_t)cuda_stream);
    if (e != cudaSuccess) return cuda_fail(e, "probe launch");
    return F8_OK;
}

}   // extern "C"

// ===========================================================================================
// Whole-network executor
// ===========================================================================================

namespace {

struct NetLayer {
    f8_layer_desc d;
    F8ConvGeom g;            // per-image geometry (n filled per call)
    F8Requant q;
    int8_t *w = nullptr;     // device parameters (owned)
    int32_t *b = nullptr;
    // stem packing (3-channel inputs on the tensor-core path)
    bool packed = false;
    int pack_wp = 0, pack_left = 0, pack_kw8 = 0;   // pack_kw8: bytes of one window row (kw cells of 16 bytes, padded)
    int pack_cpad = 8;     // bytes per pixel inside a cell (4 when c <= 4); a cell is two rows = 2 * pack_cpad bytes
    int pack_hp = 0, pack_kh = 0, pack_top = 0, pack_bottom = 0;   // row pairs: count, taps, padding above / below
    int8_t *w_packed = nullptr;
    int8_t *w_core = nullptr;   // the same window weights as [K / 16][c_out][16] (core-matrix order) for the stem kernel
    size_t out_bytes_per_image = 0;
    F8Sibling sib;              // F8_LAYER_SIBLING: this layer's quantizer of its parent's sum (y2 filled per plan)
    bool has_sibling = false;   // the next layer is an F8_LAYER_SIBLING of this one
};

struct Step {
    int kind = 0;             // layer kind, or -1 for the stem packing pre-pass
    int layer = -1;
    const void *x = nullptr;
    const void *res = nullptr;
    void *y = nullptr;
    bool use_tc = false;
    bool fused_pool = false;  // kind -2: the stem kernel also computes the max pool that follows (layer + 1)
    bool has_sib = false;     // the launch also writes the output of the sibling layer behind it (layer + 1)
    F8Sibling sib;
    int img0 = 0;             // first image of the batch this step works on (lanes, micro-batched runs)
    int lane = 0;             // 0: the caller's stream; 1: the network's second stream
    PlanPtr plan;
    // kind -3: this layer and the pointwise layer behind it (layer + 1) in one launch; y is that layer's output,
    // y_mid NULL or where a copy of this layer's own output goes
    FusedPlanPtr fplan;
    void *y_mid = nullptr;
    F8ConvGeom g;
};

}   // namespace

struct f8_net {
    std::vector<NetLayer> layers;
    std::vector<int> t_h, t_w, t_c, t_elem;     // per tensor: per-image shape and element size
    bool overlap_layers = true;                  // programmatic dependent launch between layers
    bool sync_layers = false;                    // synchronize after every launch (fault attribution)
    unsigned plan_options = 0;                   // F8_PLAN_OFF_* mask the cached plan was made under
    int plan_micro = 0, plan_lanes = 0;          // micro-batch / lane settings the cached plan was made under
    bool plan_profiling = false;
    int last_lanes = 1;
    // second lane: its own stream, joined to the caller's stream by events
    cudaStream_t lane_stream = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    int last_regions = 0, last_micro = 0;        // micro-batched runs of the cached plan and the smallest micro-batch
    std::vector<int> t_cp;                       // per tensor: channels as stored (intermediate 8-bit tensors are padded
                                                 // to a multiple of 16 so that every dense layer can use the TMA path)
    int max_batch = 0;
    // cached execution plan
    int plan_batch = -1;
    const void *plan_x = nullptr;
    void *plan_y = nullptr, *plan_ws = nullptr;
    bool plan_force_direct = false;
    bool plan_dump_first = false;                // the cached plan keeps the output of a fusable first layer
    bool plan_dumping = false;                   // the cached plan was made for a pass that copies layer outputs
    std::vector<Step> steps;
    std::vector<size_t> t_off;                   // workspace offset per tensor
    size_t pack_off = 0;
    int last_launches = 0;
    // optional per-layer timing
    bool profiling = false;
    std::vector<cudaEvent_t> events;             // steps + 1 events of the last profiled forward
    std::vector<int> event_layer;                // layer each step belongs to
};

namespace {

size_t round256(size_t v) { return (v + 255) / 256 * 256; }

size_t tensor_bytes(const f8_net *net, int t, int batch) {
    return (size_t)batch * net->t_h[t] * net->t_w[t] * net->t_cp[t] * net->t_elem[t];
}

// A run of consecutive layers executed depth-first over micro-batches: layers first..last run on images
// [0, mb), then on [mb, 2 mb), ...  Tensors that live entirely inside the run are allocated for mb images only and are
// reused by every micro-batch, so a producer's output is still in the L2 cache when its consumer reads it (and is
// overwritten there before it is ever written back); tensors that enter or leave the run keep their full size.
struct Region { int first, last, mb; };

size_t tensor_image_bytes(const f8_net *net, int t) {
    return (size_t)net->t_h[t] * net->t_w[t] * net->t_cp[t] * net->t_elem[t];
}

// Bytes one image moves through layer i when every tensor comes from / goes to memory.
size_t layer_image_bytes(const f8_net *net, int i) {
    const NetLayer &L = net->layers[i];
    if (L.d.kind == F8_LAYER_SIBLING) return tensor_image_bytes(net, i + 1);
    size_t b = tensor_image_bytes(net, L.d.src) + tensor_image_bytes(net, i + 1);
    if (L.q.has_res && L.d.res >= 0) b += tensor_image_bytes(net, L.d.res);
    return b;
}

std::vector<Region> plan_regions(const f8_net *net, int batch) {
    std::vector<Region> out;
    if (g_micro_batch == 0) return out;
    const int nl = (int)net->layers.size();
    int dev = 0, l2 = 64 << 20, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) {
        cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    }
    int i = 0;
    while (i < nl) {
        // a run of layers whose outputs have the same spatial size (one stage of a network)
        const int oh = net->t_h[i + 1], ow = net->t_w[i + 1];
        int j = i;
        while (j + 1 < nl && net->t_h[j + 2] == oh && net->t_w[j + 2] == ow) ++j;
        int first = i;
        // a pooling layer that opens the run brings the convolution in front of it along (the two may be one kernel)
        if (first > 0 && net->layers[first].d.kind == F8_LAYER_MAXPOOL && net->layers[first].d.src == first &&
            net->layers[first - 1].d.kind == F8_LAYER_CONV && (out.empty() || out.back().last < first - 1))
            --first;
        if ((long long)oh * ow > 1 && j - first + 1 >= 3 && j < nl - 1) {
            size_t worst = 0;
            bool beyond_l2 = false;
            for (int l = first; l <= j; ++l) {
                const size_t b = layer_image_bytes(net, l);
                worst = std::max(worst, b);
                if (b * (size_t)batch > (size_t)l2) beyond_l2 = true;
            }
            int mb = 0;
            if (g_micro_batch > 0) {
                mb = g_micro_batch;
            } else if (beyond_l2 && worst > 0) {
                // the largest power of two whose heaviest layer moves at most half of the cache
                mb = 1;
                while ((size_t)(2 * mb) * worst <= (size_t)l2 / 2) mb *= 2;
                // every dense layer must still fill the machine a few times over, or the tail of each launch costs
                // more than the memory traffic saved
                for (int l = first; l <= j && mb > 0; ++l) {
                    const NetLayer &L = net->layers[l];
                    if (L.d.kind != F8_LAYER_CONV) continue;
                    const long long tiles = (((long long)mb * L.g.ho * L.g.wo + 127) / 128) * ((L.g.c_out + 255) / 256);
                    if (tiles < 2ll * sms) mb = 0;
                }
            }
            if (mb > 0 && mb < batch) out.push_back({first, j, mb});
        }
        i = j + 1;
    }
    return out;
}

// Lanes: the batch is cut into two halves that run as two independent forward passes on two streams, launched
// alternately layer by layer.  Every launch starts and ends with a few microseconds in which most SMs idle (the
// last tiles of a layer drain, the first tiles of the next one wait for memory); the idea is that with a second,
// independent launch queue the SMs one lane leaves idle take blocks of the other lane.  Images are independent, so
// no result changes.
int lanes_for(const f8_net *net, int batch) {
    if (g_plan_off & F8_PLAN_OFF_LANES) return 1;
    if (g_lanes == 1 || batch < 2 || net->profiling) return 1;
    // measured slower than one lane on every configuration tried (the waiting blocks of a lane's next launch hold the
    // SMs its sibling could use): two lanes only on request
    return g_lanes == 2 ? 2 : 1;
}
int lane_images(int batch, int lanes, int lane) {
    const int first = (batch + lanes - 1) / lanes;
    return lane == 0 ? first : batch - first;
}

// Which run a layer belongs to (-1: none), and which tensors live entirely inside one run.
void classify_tensors(const f8_net *net, const std::vector<Region> &regions, std::vector<int> *layer_region,
                      std::vector<int> *tensor_region /* run a tensor is internal to, or -1 */) {
    const int nl = (int)net->layers.size();
    layer_region->assign(nl, -1);
    for (int r = 0; r < (int)regions.size(); ++r)
        for (int l = regions[r].first; l <= regions[r].last; ++l) (*layer_region)[l] = r;
    tensor_region->assign(nl + 1, -1);
    for (int t = 1; t < nl; ++t) {
        const int producer = net->layers[t - 1].d.kind == F8_LAYER_SIBLING ? t - 2 : t - 1;
        const int r = (*layer_region)[producer];
        if (r < 0 || (*layer_region)[t - 1] != r) continue;
        bool inside = true;
        for (int l = 0; l < nl && inside; ++l) {
            const NetLayer &L = net->layers[l];
            const bool reads = L.d.src == t || (L.q.has_res && L.d.res == t && L.d.kind != F8_LAYER_SIBLING);
            if (reads && (*layer_region)[l] != r) inside = false;
        }
        if (inside) (*tensor_region)[t] = r;
    }
}

// Assigns workspace offsets: tensors whose lifetimes do not overlap may share memory (first fit).
// Layer i and the pointwise layer behind it may run as one launch (the two-layer kernel): layer i + 1 is a 1x1 convolution
// that alone reads layer i's output, and the channel counts are the kernel's.  (Whether they do is decided per plan: the
// batch must make the input large enough, and both layers must lie in the same run of the schedule.)
bool pair_candidate(const f8_net *net, int i) {
    const int nl = (int)net->layers.size();
    if (i + 1 >= nl) return false;
    const NetLayer &L = net->layers[i], &P = net->layers[i + 1];
    if (L.d.kind != F8_LAYER_CONV || L.packed || L.has_sibling || L.q.has_res) return false;
    if (P.d.kind != F8_LAYER_CONV || P.has_sibling || P.packed || P.d.src != i + 1 || P.g.kh != 1 || P.g.kw != 1 || P.g.stride_h != 1 ||
        P.g.stride_w != 1 || P.g.pad_h != 0 || P.g.pad_w != 0)
        return false;
    if (P.q.has_res && P.d.res == i + 1) return false;
    if (net->t_cp[i + 1] != L.g.c_out) return false;
    for (int l2 = i + 2; l2 < nl; ++l2)
        if (net->layers[l2].d.src == i + 1 || (net->layers[l2].q.has_res && net->layers[l2].d.res == i + 1)) return false;
    F8ConvGeom g = L.g;
    g.n = net->max_batch;   // the size rule is checked again with the real batch when a plan is made
    return f8_fused_supported(g, L.q, P.g.c_out, P.q);
}

size_t assign_offsets(const f8_net *net, int batch, std::vector<size_t> *off, size_t *pack_off,
                      const std::vector<Region> &regions) {
    const int nl = (int)net->layers.size();
    const int nt = nl + 1;
    std::vector<int> layer_region, tensor_region;
    classify_tensors(net, regions, &layer_region, &tensor_region);
    std::vector<int> last(nt, -1), born(nt, 0);
    for (int i = 0; i < nl; ++i) {
        last[net->layers[i].d.src] = i;
        if (net->layers[i].d.res >= 0) last[net->layers[i].d.res] = i;
    }
    for (int t = 1; t < nt; ++t) {
        // written by layer t-1; a sibling's tensor is written by the launch of the layer before it
        born[t] = net->layers[t - 1].d.kind == F8_LAYER_SIBLING ? t - 2 : t - 1;
        last[t] = std::max(last[t], born[t]);
    }
    // the two-layer kernel writes the second layer's output while it still reads the first layer's input: that output is
    // born with the first layer's launch, so that it shares memory with nothing the launch reads
    for (int i = 0; i + 1 < nl; ++i)
        if (pair_candidate(net, i)) born[i + 2] = std::min(born[i + 2], i);
    // A full-size tensor that a micro-batched run writes is filled slice by slice over the whole run, and one that the
    // run reads is read again by every micro-batch: both are live from the run's first layer to its last.
    for (int t = 1; t < nt; ++t) {
        if (tensor_region[t] >= 0) continue;
        const int rp = layer_region[born[t]];
        if (rp >= 0) { born[t] = std::min(born[t], regions[rp].first); last[t] = std::max(last[t], regions[rp].last); }
        for (int l = 0; l < nl; ++l) {
            const NetLayer &L = net->layers[l];
            const bool reads = L.d.src == t || (L.d.res == t && L.d.res >= 0);
            if (reads && layer_region[l] >= 0) last[t] = std::max(last[t], regions[layer_region[l]].last);
        }
    }
    struct Live { size_t off, size; int until; };
    std::vector<Live> live;
    off->assign(nt, 0);
    size_t top = 0;
    // in order of birth (a tensor a run writes in full may be born before tensors with smaller numbers)
    std::vector<int> order;
    for (int t = 1; t < nt - 1; ++t) order.push_back(t);      // tensor 0 = caller's x, tensor nt-1 = caller's y
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return born[a] < born[b]; });
    for (int t : order) {
        const int images = tensor_region[t] >= 0 ? std::min(batch, regions[tensor_region[t]].mb) : batch;
        const size_t size = round256((size_t)images * tensor_image_bytes(net, t));
        live.erase(std::remove_if(live.begin(), live.end(), [&](const Live &l) { return l.until < born[t]; }), live.end());
        std::sort(live.begin(), live.end(), [](const Live &a, const Live &b) { return a.off < b.off; });
        size_t pos = 0;
        for (const Live &l : live) {
            if (pos + size <= l.off) break;
            pos = std::max(pos, l.off + l.size);
        }
        (*off)[t] = pos;
        live.push_back({pos, size, last[t]});
        top = std::max(top, pos + size);
    }
    *pack_off = top;
    size_t pack = 0;
    for (const NetLayer &l : net->layers)
        if (l.packed) pack = std::max(pack, round256((size_t)batch * l.pack_hp * l.pack_wp * 2 * l.pack_cpad));
    return top + pack;
}

void free_layers(f8_net *net) {
    for (NetLayer &l : net->layers) {
        if (l.w) cudaFree(l.w);
        if (l.b) cudaFree(l.b);
        if (l.w_packed) cudaFree(l.w_packed);
        if (l.w_core) cudaFree(l.w_core);
    }
}

}   // namespace

extern "C" {

f8_status f8_net_create(const f8_layer_desc *layers, int n_layers, const int8_t *const *host_weights,
                        const int32_t *const *host_bias, int max_batch, f8_net **out) {
    if (!layers || !out) return fail(F8_ERR_NULL, "layers / out is NULL");
    if (n_layers <= 0 || max_batch <= 0) return fail(F8_ERR_SHAPE, "n_layers and max_batch must be positive");
    std::unique_ptr<f8_net> net(new (std::nothrow) f8_net);
    if (!net) return fail(F8_ERR_CUDA, "out of host memory");
    net->max_batch = max_batch;
    net->layers.resize(n_layers);
    // tensor 0 shape comes from the first layer that reads it
    net->t_h.assign(n_layers + 1, 0);
    net->t_w.assign(n_layers + 1, 0);
    net->t_c.assign(n_layers + 1, 0);
    net->t_elem.assign(n_layers + 1, 1);
    std::vector<int> t_dtype(n_layers + 1, -1), t_fl(n_layers + 1, 0);
    std::vector<long long> t_bound(n_layers + 1, 0);       // largest magnitude an element of a 32-bit tensor can take
    auto cleanup = [&](f8_status s) { free_layers(net.get()); return s; };
    for (int i = 0; i < n_layers; ++i) {
        NetLayer &L = net->layers[i];
        L.d = layers[i];
        f8_conv_desc &d = L.d.conv;
        d.n = 1;
        if (L.d.kind == F8_LAYER_SIBLING) {
            // a second consumer of the 32-bit sum of the layer right before it, with its private format (Sec. 4.3)
            if (i == 0 || L.d.src != i || net->layers[i - 1].d.kind != F8_LAYER_CONV)
                return cleanup(fail(F8_ERR_SHAPE, "layer %d: a sibling layer must directly follow the dense convolution whose output tensor it names", i));
            NetLayer &P = net->layers[i - 1];
            const int yd = d.y_dtype, fy = d.fl_y;
            const f8_status s = make_sibling(&P.d.conv, P.q, yd, fy, nullptr, &L.sib);
            if (s != F8_OK) {
                char msg[400];
                snprintf(msg, sizeof(msg), "layer %d: %.300s", i, g_err);
                return cleanup(fail(s, "%s", msg));
            }
            d = P.d.conv;
            d.y_dtype = yd;
            d.fl_y = fy;
            L.d.res = -1;
            L.g = P.g;
            L.q = P.q;
            P.has_sibling = true;
            const bool wide = yd == F8_S32 || yd == F8_S32_RELU;
            net->t_h[i + 1] = net->t_h[i]; net->t_w[i + 1] = net->t_w[i]; net->t_c[i + 1] = net->t_c[i];
            net->t_elem[i + 1] = wide ? 4 : 1;
            t_dtype[i + 1] = wide ? F8_S32 : yd;
            t_fl[i + 1] = wide ? P.d.conv.fl_x + P.d.conv.fl_w + P.q.sh_acc : fy;
            t_bound[i + 1] = t_bound[i];       // the same sum as the parent's output
            continue;
        }
        if (L.d.src < 0 || L.d.src > i) return cleanup(fail(F8_ERR_SHAPE, "layer %d: src %d is not an earlier tensor", i, L.d.src));
        if (L.d.res > i) return cleanup(fail(F8_ERR_SHAPE, "layer %d: res %d is not an earlier tensor", i, L.d.res));
        const int kind = L.d.kind;
        if (kind == F8_LAYER_LINEAR) { d.h = d.w = 1; d.kh = d.kw = 1; d.stride = 1; d.pad = 0; }
        if (kind == F8_LAYER_GAP) { d.kh = d.kw = 1; d.stride = 1; d.pad = 0; d.c_out = d.c; d.y_dtype = d.x_dtype; d.fl_w = 0; }
        if (kind == F8_LAYER_MAXPOOL) { d.c_out = d.c; d.y_dtype = d.x_dtype; d.fl_w = 0; d.fl_y = d.fl_x; }
        const bool has_res = L.d.res >= 0 && (kind == F8_LAYER_CONV || kind == F8_LAYER_DWCONV);
        f8_status s;
        switch (kind) {
            case F8_LAYER_CONV:
                s = check_conv(&d, false, has_res, &L.g, &L.q, true);
                break;
            case F8_LAYER_LINEAR:
                s = check_conv(&d, false, has_res, &L.g, &L.q);
                break;
            case F8_LAYER_DWCONV:
                s = check_conv(&d, true, has_res, &L.g, &L.q);
                break;
            case F8_LAYER_MAXPOOL:
                if (d.kh != d.kw || d.pad >= d.kh) return cleanup(fail(F8_ERR_SHAPE, "layer %d: bad pooling window", i));
                s = check_conv(&d, true, false, &L.g, &L.q);
                break;
            case F8_LAYER_GAP: {
                f8_conv_desc t = d;
                t.kh = t.h; t.kw = t.w;
                t.fl_w = ceil_log2((long long)d.h * d.w);    // the power-of-two "average" enters as a format shift
                s = check_conv(&t, true, false, &L.g, &L.q);
                L.g.kh = L.g.kw = 1;
                break;
            }
            default:
                return cleanup(fail(F8_ERR_UNSUPPORTED, "layer %d: unknown kind %d", i, kind));
        }
        if (s != F8_OK) {
            char msg[400];
            snprintf(msg, sizeof(msg), "layer %d: %s", i, g_err);
            return cleanup(fail(s, "%s", msg));
        }
        // shapes / dtypes must chain
        const int src = L.d.src;
        if (src == 0 && net->t_h[0] == 0) {
            net->t_h[0] = d.h; net->t_w[0] = d.w; net->t_c[0] = d.c;
            t_dtype[0] = d.x_dtype; t_fl[0] = d.fl_x;
        }
        if (net->t_h[src] != d.h || net->t_w[src] != d.w || net->t_c[src] != d.c)
            return cleanup(fail(F8_ERR_SHAPE, "layer %d: input shape does not match tensor %d", i, src));
        if (t_dtype[src] != d.x_dtype || t_fl[src] != d.fl_x)
            return cleanup(fail(F8_ERR_DTYPE, "layer %d: x_dtype / fl_x do not match the producer of tensor %d", i, src));
        const int ho = kind == F8_LAYER_GAP ? 1 : L.g.ho, wo = kind == F8_LAYER_GAP ? 1 : L.g.wo;
        if (has_res) {
            const int r = L.d.res;
            if (net->t_h[r] != ho || net->t_w[r] != wo || net->t_c[r] != d.c_out)
                return cleanup(fail(F8_ERR_SHAPE, "layer %d: residual tensor %d has the wrong shape", i, r));
            if (t_dtype[r] != d.r_dtype || t_fl[r] != d.fl_r)
                return cleanup(fail(F8_ERR_DTYPE, "layer %d: r_dtype / fl_r do not match the producer of tensor %d", i, r));
        }
        net->t_h[i + 1] = ho; net->t_w[i + 1] = wo; net->t_c[i + 1] = d.c_out;
        const bool wide_out = d.y_dtype == F8_S32 || d.y_dtype == F8_S32_RELU;
        net->t_elem[i + 1] = wide_out ? 4 : 1;
        t_dtype[i + 1] = wide_out ? F8_S32 : d.y_dtype;
        t_fl[i + 1] = wide_out ? d.fl_x + d.fl_w + L.q.sh_acc : d.fl_y;
        if (has_res && L.q.r_s32 && d.c_out % 16 != 0)
            return cleanup(fail(F8_ERR_UNSUPPORTED, "layer %d: a 32-bit shortcut needs c_out to be a multiple of 16", i));
        L.out_bytes_per_image = (size_t)ho * wo * d.c_out * net->t_elem[i + 1];

        // parameters
        const bool has_params = kind == F8_LAYER_CONV || kind == F8_LAYER_DWCONV || kind == F8_LAYER_LINEAR;
        if (!has_params) continue;
        const int8_t *hw = host_weights ? host_weights[i] : nullptr;
        const int32_t *hb = host_bias ? host_bias[i] : nullptr;
        if (!hw) return cleanup(fail(F8_ERR_NULL, "layer %d: weights missing", i));
        const size_t per_out = (size_t)d.kh * d.kw * (kind == F8_LAYER_DWCONV ? 1 : d.c);
        // exact accumulator bound per output channel from the actual parameters
        const long long xmax = d.x_dtype == F8_U8 ? 255 : 128;
        const long long rmax = has_res ? (L.q.r_s32 ? t_bound[L.d.res] : (d.r_dtype == F8_U8 ? 255 : 128)) : 0;
        long long layer_bound = 0;
        for (int co = 0; co < d.c_out; ++co) {
            long long sum = 0;
            for (size_t j = 0; j < per_out; ++j) sum += llabs((long long)hw[co * per_out + j]);
            long long bound = sum * xmax + (hb ? llabs((long long)hb[co]) : 0);
            bound = (bound << L.q.sh_acc) + (rmax << L.q.sh_res);
            layer_bound = std::max(layer_bound, bound);
            if (L.q.y_kind != F8_S32 && L.q.y_kind != F8_S32_RELU && L.q.s >= 1) bound += 1ll << (L.q.s - 1);      // room for the rounding constant
            if (bound >= (1ll << 31) - 1)
                return cleanup(fail(F8_ERR_ACC_BOUND, "layer %d channel %d: accumulator bound %lld exceeds int32", i, co, bound));
        }
        t_bound[i + 1] = layer_bound;       // what a 32-bit output of this layer (its own or a sibling's) can reach
    }
    // Stored channel counts: intermediate 8-bit tensors whose channel count is not a multiple of 16 (24 in
    // MobileNetV2) are padded with channels that are identically zero -- zero weights and bias produce them,
    // zero weights consume them -- so the arithmetic of the real channels is untouched.
    net->t_cp = net->t_c;
    for (int t = 1; t < n_layers; ++t)
        if (net->t_elem[t] == 1 && net->t_c[t] % 16 != 0) net->t_cp[t] = (net->t_c[t] + 15) / 16 * 16;
    // both outputs of a launch have the same number of stored channels
    for (int i = 1; i < n_layers; ++i)
        if (net->layers[i].d.kind == F8_LAYER_SIBLING) {
            if (i + 1 == n_layers && net->t_cp[i] != net->t_c[i])
                return cleanup(fail(F8_ERR_UNSUPPORTED, "layer %d: the network output cannot be the sibling of a layer with padded channels", i));
            net->t_cp[i + 1] = net->t_cp[i];
        }
    // second pass (everything validated): upload the parameters
    for (int i = 0; i < n_layers; ++i) {
        NetLayer &L = net->layers[i];
        const f8_conv_desc &d = L.d.conv;
        const int kind = L.d.kind;
        const int cp_in = net->t_cp[L.d.src], cp_out = net->t_cp[i + 1];
        L.g.c = cp_in;
        L.g.c_out = cp_out;
        L.out_bytes_per_image = (size_t)net->t_h[i + 1] * net->t_w[i + 1] * cp_out * net->t_elem[i + 1];
        if (kind != F8_LAYER_CONV && kind != F8_LAYER_DWCONV && kind != F8_LAYER_LINEAR) continue;
        const int8_t *hw = host_weights[i];
        const int32_t *hb = host_bias ? host_bias[i] : nullptr;
        std::vector<int8_t> w_padded;
        std::vector<int32_t> b_padded;
        const int taps = d.kh * d.kw;
        if (cp_in != d.c || cp_out != d.c_out) {
            if (kind == F8_LAYER_DWCONV) {
                w_padded.assign((size_t)cp_out * taps, 0);
                memcpy(w_padded.data(), hw, (size_t)d.c * taps);
            } else {
                w_padded.assign((size_t)cp_out * taps * cp_in, 0);
                for (int co = 0; co < d.c_out; ++co)
                    for (int t = 0; t < taps; ++t)
                        memcpy(&w_padded[((size_t)co * taps + t) * cp_in], &hw[((size_t)co * taps + t) * d.c], (size_t)d.c);
            }
            hw = w_padded.data();
            if (hb) {
                b_padded.assign((size_t)cp_out, 0);
                memcpy(b_padded.data(), hb, 4 * (size_t)d.c_out);
                hb = b_padded.data();
            }
        }
        const size_t wn = (size_t)taps * (kind == F8_LAYER_DWCONV ? 1 : cp_in) * cp_out;
        cudaError_t e = cudaMalloc(&L.w, round256(wn));
        if (e == cudaSuccess) e = cudaMemcpy(L.w, hw, wn, cudaMemcpyHostToDevice);
        if (e == cudaSuccess && hb) {
            e = cudaMalloc(&L.b, round256(4 * (size_t)cp_out));
            if (e == cudaSuccess) e = cudaMemcpy(L.b, hb, 4 * (size_t)cp_out, cudaMemcpyHostToDevice);
        }
        if (e != cudaSuccess) return cleanup(cuda_fail(e, "parameter upload"));
        hw = host_weights[i];     // the stem packing below reads the caller's layout

        // 3-channel (<= 8) stems with stride 2.  The image is re-packed into cells of 16 bytes that hold one
        // pixel of two consecutive rows (8 bytes each), so that the kw-tap window of an output column over a
        // row PAIR is one contiguous, 16-byte aligned run of kw16 bytes.  The layer then is a kh' x 1
        // convolution with stride 1 over kw16 "channels" of an overlapping strided view (kh' row pairs cover
        // the kh rows; taps that fall outside the filter get zero weights), which the tensor-core path takes
        // with few, long TMA rows.  Kernel row r sits in pair j, half e with r = 2j + e + pad - 2*top.
        if (kind == F8_LAYER_CONV && cp_in == d.c && cp_out == d.c_out && d.c <= 8 && d.stride == 2 &&
            d.kw * 16 <= 256 && !L.has_sibling && !L.q.r_s32 && d.y_dtype != F8_S32_RELU) {
            L.packed = true;
            L.pack_left = d.pad;
            L.pack_cpad = d.c <= 4 ? 4 : 8;
            const int cb = 2 * L.pack_cpad;                       // bytes per cell
            L.pack_kw8 = (d.kw * cb + 31) / 32 * 32;
            L.pack_wp = std::max(d.w + d.pad, (L.g.wo - 1) * d.stride + L.pack_kw8 / cb);
            L.pack_wp = (L.pack_wp + 1) / 2 * 2;                  // rows of cells stay 16-byte multiples
            L.pack_hp = (d.h + 1) / 2;
            L.pack_top = (d.pad + 1) / 2;
            L.pack_kh = (d.kh - 1 - d.pad >= 0 ? (d.kh - 1 - d.pad) / 2 : -((d.pad - d.kh + 2) / 2)) + L.pack_top + 1;
            L.pack_bottom = L.g.ho - L.pack_hp - L.pack_top + L.pack_kh - 1;
            std::vector<int8_t> wp((size_t)d.c_out * L.pack_kh * L.pack_kw8, 0);
            for (int co = 0; co < d.c_out; ++co)
                for (int j = 0; j < L.pack_kh; ++j)
                    for (int e2 = 0; e2 < 2; ++e2) {
                        const int r = 2 * j + e2 + d.pad - 2 * L.pack_top;
                        if (r < 0 || r >= d.kh) continue;
                        for (int s2 = 0; s2 < d.kw; ++s2)
                            for (int ch = 0; ch < d.c; ++ch)
                                wp[((size_t)co * L.pack_kh + j) * L.pack_kw8 + s2 * cb + e2 * L.pack_cpad + ch] =
                                    hw[(((size_t)co * d.kh + r) * d.kw + s2) * d.c + ch];
                    }
            if (L.pack_kh < 1 || L.pack_bottom < 0) L.packed = false;      // degenerate geometry: CUDA-core kernel
            if (!L.packed) continue;
            e = cudaMalloc(&L.w_packed, round256(wp.size()));
            if (e == cudaSuccess) e = cudaMemcpy(L.w_packed, wp.data(), wp.size(), cudaMemcpyHostToDevice);
            if (e != cudaSuccess) return cleanup(cuda_fail(e, "packed stem weights upload"));
            if (L.pack_cpad == 4) {
                // core-matrix order for the stem kernel: 16 consecutive K bytes of one output channel are contiguous,
                // then the output channels, then the K chunks
                const size_t kb = (size_t)L.pack_kh * L.pack_kw8;
                std::vector<int8_t> wc(kb * d.c_out, 0);
                for (int co = 0; co < d.c_out; ++co)
                    for (size_t k = 0; k < kb; ++k) wc[((k / 16) * d.c_out + co) * 16 + k % 16] = wp[(size_t)co * kb + k];
                e = cudaMalloc(&L.w_core, round256(wc.size()));
                if (e == cudaSuccess) e = cudaMemcpy(L.w_core, wc.data(), wc.size(), cudaMemcpyHostToDevice);
                if (e != cudaSuccess) return cleanup(cuda_fail(e, "stem weights upload"));
            }
        }
    }
    (void)f8_status_word();         // creates the device status word and its host-visible copy
    if (cudaStreamCreateWithFlags(&net->lane_stream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&net->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&net->ev_join, cudaEventDisableTiming) != cudaSuccess) {
        (void)cudaGetLastError();
        f8_net *raw = net.release();
        f8_net_destroy(raw);
        return fail(F8_ERR_CUDA, "could not create the second lane's stream");
    }
    *out = net.release();
    return F8_OK;
}

size_t f8_net_workspace_bytes(const f8_net *net, int batch) {
    if (!net || batch <= 0) return 0;
    std::vector<size_t> off;
    size_t pack_off;
    // enough for one lane and for two (a profiled pass runs as one lane whatever the rule says)
    size_t most = 0;
    for (int lanes = 1; lanes <= (batch >= 2 ? 2 : 1); ++lanes) {
        size_t total = 256;
        for (int lane = 0; lane < lanes; ++lane) {
            const int n = lane_images(batch, lanes, lane);
            total += round256(assign_offsets(net, n, &off, &pack_off, plan_regions(net, n)));
        }
        most = std::max(most, total);
    }
    return most;
}

int f8_net_last_launch_count(const f8_net *net) { return net ? net->last_launches : 0; }

int f8_net_lanes(const f8_net *net) { return net ? net->last_lanes : 0; }

int f8_net_fused_pairs(const f8_net *net) {
    int n = 0;
    if (net)
        for (const Step &stp : net->steps) n += stp.kind == -3 ? 1 : 0;
    return n;
}

int f8_net_micro_batching(const f8_net *net, int *images) {
    if (images) *images = net ? net->last_micro : 0;
    return net ? net->last_regions : 0;
}

f8_status f8_net_set_profiling(f8_net *net, int on) {
    if (!net) return fail(F8_ERR_NULL, "net is NULL");
    net->profiling = on != 0;
    net->event_layer.clear();
    return F8_OK;
}

f8_status f8_net_get_layer_ms(f8_net *net, float *ms, int *on_tensor_cores) {
    if (!net || !ms) return fail(F8_ERR_NULL, "net / ms is NULL");
    const int nl = (int)net->layers.size();
    for (int i = 0; i < nl; ++i) ms[i] = 0.f;
    if (on_tensor_cores) for (int i = 0; i < nl; ++i) on_tensor_cores[i] = 0;
    if (net->event_layer.empty()) return fail(F8_ERR_UNSUPPORTED, "no profiled forward pass recorded");
    cudaError_t e = cudaEventSynchronize(net->events[net->event_layer.size()]);
    if (e != cudaSuccess) return cuda_fail(e, "cudaEventSynchronize");
    for (size_t k = 0; k < net->event_layer.size(); ++k) {
        float t = 0.f;
        e = cudaEventElapsedTime(&t, net->events[k], net->events[k + 1]);
        if (e != cudaSuccess) return cuda_fail(e, "cudaEventElapsedTime");
        ms[net->event_layer[k]] += t;
    }
    if (on_tensor_cores)
        for (const Step &stp : net->steps)
            if (stp.kind >= 0 && stp.use_tc) on_tensor_cores[stp.layer] = 1;
            else if (stp.kind == -3) on_tensor_cores[stp.layer] = on_tensor_cores[stp.layer + 1] = 1;
    return F8_OK;
}

void f8_net_destroy(f8_net *net) {
    if (!net) return;
    for (cudaEvent_t ev : net->events) cudaEventDestroy(ev);
    if (net->ev_fork) cudaEventDestroy(net->ev_fork);
    if (net->ev_join) cudaEventDestroy(net->ev_join);
    if (net->lane_stream) cudaStreamDestroy(net->lane_stream);
    free_layers(net);
    delete net;
}

f8_status f8_net_forward(f8_net *net, int batch, const void *x, void *y, void *workspace, size_t workspace_bytes,
                         void *const *layer_dump, void *cuda_stream) {
    if (!net) return fail(F8_ERR_NULL, "net is NULL");
    if (batch < 0 || batch > net->max_batch) return fail(F8_ERR_SHAPE, "batch %d outside [0, %d]", batch, net->max_batch);
    if (batch == 0) { net->last_launches = 0; return F8_OK; }
    if (!x || !y) return fail(F8_ERR_NULL, "x and y must not be NULL");
    if (!aligned16(x) || !aligned16(y) || !aligned16(workspace)) return fail(F8_ERR_ALIGN, "device pointers must be 16-byte aligned");
    const size_t need = f8_net_workspace_bytes(net, batch);
    if (need > 256 && (!workspace || workspace_bytes < need))
        return fail(F8_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", need, workspace_bytes);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int nl = (int)net->layers.size();
    // A kernel that gives up a bounded wait also stores its code to a host-visible word: an earlier pass (or anything
    // else on this device) that left its output incomplete is reported here, without a synchronisation.
    if (pending_timeout() != F8_OK) return F8_ERR_TIMEOUT;

    // a first layer whose output is asked for cannot be fused with the pooling layer behind it
    bool dump_fusable = false;
    if (layer_dump)
        for (int i = 0; i < nl; ++i)
            if (net->layers[i].w_core && layer_dump[i]) dump_fusable = true;
    const bool replan = net->plan_batch != batch || net->plan_x != x || net->plan_y != y || net->plan_ws != workspace ||
                        net->plan_force_direct != g_force_direct || net->plan_dump_first != dump_fusable ||
                        net->plan_dumping != (layer_dump != nullptr) ||
                        net->plan_options != g_plan_off || net->plan_micro != g_micro_batch || net->plan_lanes != g_lanes ||
                        net->plan_profiling != net->profiling;
    net->overlap_layers = !(g_plan_off & F8_PLAN_OFF_LAYER_OVERLAP);
    net->sync_layers = (g_plan_off & F8_PLAN_SYNC_LAYERS) != 0;
    if (replan) {
        net->steps.clear();
        net->plan_batch = -1;
        const int lanes = lanes_for(net, batch);
        net->last_lanes = lanes;
        net->last_regions = 0;
        net->last_micro = 0;
        // every lane is a forward pass of its own over its share of the images, with its own part of the workspace
        struct Lane {
            int img0 = 0, n = 0;
            uint8_t *ws = nullptr;
            std::vector<size_t> t_off;
            size_t pack_off = 0;
            std::vector<Region> regions;
            std::vector<int> layer_region, tensor_region;
            std::vector<Step> steps;
            int skip_layer = -1;      // a pooling layer the stem kernel has taken over
        };
        std::vector<Lane> lane_list(lanes);
        {
            uint8_t *base = (uint8_t *)workspace;
            int img = 0;
            for (int k = 0; k < lanes; ++k) {
                Lane &ln = lane_list[k];
                ln.img0 = img;
                ln.n = lane_images(batch, lanes, k);
                img += ln.n;
                ln.regions = plan_regions(net, ln.n);
                ln.ws = base;
                base += round256(assign_offsets(net, ln.n, &ln.t_off, &ln.pack_off, ln.regions));
                classify_tensors(net, ln.regions, &ln.layer_region, &ln.tensor_region);
                net->last_regions = std::max(net->last_regions, (int)ln.regions.size());
                for (const Region &r : ln.regions) net->last_micro = net->last_micro ? std::min(net->last_micro, r.mb) : r.mb;
            }
        }
        const size_t x_image_bytes = (size_t)net->t_h[0] * net->t_w[0] * net->t_c[0];
        const size_t y_image_bytes = (size_t)net->t_h[nl] * net->t_w[nl] * net->t_c[nl] * net->t_elem[nl];

        // Plans layer i for images [img0, img0 + n) of the batch.  Inside a micro-batched run (in_run) tensors that live
        // entirely in the run hold one micro-batch and always start at their base address; all other tensors are
        // addressed at the slice of these images.
        // img0: first image relative to the lane's share
        auto plan_layer = [&](Lane &ln, int lane_index, int i, int n, int img0, bool in_run) {
            NetLayer &L = net->layers[i];
            int &skip_layer = ln.skip_layer;
            const std::vector<int> &layer_region = ln.layer_region, &tensor_region = ln.tensor_region;
            if (i == skip_layer || L.d.kind == F8_LAYER_SIBLING) return;      // a sibling is written by its parent's launch
            auto tensor_ptr = [&](int t) -> void * {
                // the caller's tensors are addressed by the image's place in the whole batch
                if (t == 0) return (uint8_t *)const_cast<void *>(x) + (size_t)(ln.img0 + img0) * x_image_bytes;
                if (t == nl) return (uint8_t *)y + (size_t)(ln.img0 + img0) * y_image_bytes;
                uint8_t *base = ln.ws + ln.t_off[t];
                if (in_run && tensor_region[t] < 0) base += (size_t)img0 * tensor_image_bytes(net, t);
                return base;
            };
            Step stp;
            stp.kind = L.d.kind;
            stp.layer = i;
            stp.lane = lane_index;
            stp.img0 = ln.img0 + img0;
            stp.x = tensor_ptr(L.d.src);
            stp.res = (L.q.has_res) ? tensor_ptr(L.d.res) : nullptr;
            stp.y = tensor_ptr(i + 1);
            stp.g = L.g;
            stp.g.n = n;
            if (L.has_sibling) {
                stp.has_sib = true;
                stp.sib = net->layers[i + 1].sib;
                stp.sib.y2 = tensor_ptr(i + 2);
            }
            if ((L.d.kind == F8_LAYER_CONV || L.d.kind == F8_LAYER_LINEAR) && !g_force_direct) {
                const char *why = "";
                if (L.packed && L.w_core && !(g_plan_off & F8_PLAN_OFF_STEM_KERNEL) &&
                    f8_stem_tc_supported(stp.g, L.q, L.pack_kh, L.pack_kw8 / 32)) {
                    // the stem kernel; it also takes the 3x3 / 2 / pad 1 max pool behind the layer when nothing else
                    // reads the layer's output
                    bool fuse = !dump_fusable && i + 1 < nl && !(g_plan_off & F8_PLAN_OFF_STEM_POOL_FUSION) &&
                                layer_region[i] == layer_region[i + 1];
                    if (fuse) {
                        const NetLayer &P = net->layers[i + 1];
                        fuse = P.d.kind == F8_LAYER_MAXPOOL && P.d.src == i + 1 && P.d.conv.kh == 3 && P.d.conv.kw == 3 &&
                               P.d.conv.stride == 2 && P.d.conv.pad == 1;
                        for (int l = i + 2; fuse && l < nl; ++l)
                            if (net->layers[l].d.src == i + 1 || (net->layers[l].q.has_res && net->layers[l].d.res == i + 1)) fuse = false;
                    }
                    stp.kind = -2;
                    stp.fused_pool = fuse;
                    if (fuse) {
                        stp.y = tensor_ptr(i + 2);
                        skip_layer = i + 1;
                    }
                } else if (L.packed) {
                    F8ConvGeom pg = stp.g;
                    pg.c = L.pack_kw8; pg.kw = 1; pg.stride_w = 1; pg.pad_w = 0;
                    pg.kh = L.pack_kh; pg.stride_h = 1; pg.pad_h = L.pack_top; pg.pad_h_end = L.pack_bottom;
                    pg.h = L.pack_hp;
                    void *pbuf = ln.ws + ln.pack_off;
                    const uint64_t cb = 2 * (uint64_t)L.pack_cpad;
                    const size_t pbytes = (size_t)n * L.pack_hp * L.pack_wp * cb;
                    if (f8_tc_supported(pg, pbytes)) {
                        F8TcTensorView v;
                        v.base = pbuf;
                        v.dim_c = L.pack_kw8; v.dim_w = L.g.wo; v.dim_h = L.pack_hp; v.dim_n = n;
                        v.stride_w = (uint64_t)L.g.stride_w * cb;
                        v.stride_h = (uint64_t)L.pack_wp * cb;
                        v.stride_n = (uint64_t)L.pack_wp * cb * L.pack_hp;
                        PlanPtr plan = alloc_plan();
                        if (plan && f8_tc_plan_init(plan.get(), pg, L.q, v, L.w_packed, L.b, stp.res, stp.y,
                                                    f8_status_word(), &why) == cudaSuccess) {
                            Step pre;
                            pre.kind = -1;
                            pre.layer = i;
                            pre.img0 = ln.img0 + img0;
                            pre.lane = lane_index;
                            pre.x = stp.x;
                            pre.y = pbuf;
                            pre.g = stp.g;
                            ln.steps.push_back(std::move(pre));
                            stp.use_tc = true;
                            f8_tc_plan_set_tag(plan.get(), i + 1);
                            stp.plan = std::move(plan);
                        }
                    }
                } else if ([&]() -> bool {
                               // This layer and the pointwise layer behind it in one launch (the tail of a bottleneck block):
                               // the next layer is a 1x1 convolution that alone reads this layer's output, both lie in the
                               // same run of the schedule, and the shapes are the two-layer kernel's.
                               if (g_plan_off & F8_PLAN_OFF_LAYER_FUSION) return false;
                               if (!pair_candidate(net, i) || layer_region[i] != layer_region[i + 1]) return false;
                               const NetLayer &P = net->layers[i + 1];
                               if (!f8_fused_supported(stp.g, L.q, P.g.c_out, P.q)) return false;
                               FusedPlanPtr fp = alloc_fused_plan();
                               if (!fp) return false;
                               const void *res2 = P.q.has_res ? tensor_ptr(P.d.res) : nullptr;
                               void *mid = layer_dump ? tensor_ptr(i + 1) : nullptr;      // only a pass that copies outputs keeps it
                               if (f8_fused_plan_init(fp.get(), stp.g, L.q, P.q, stp.x, L.w, L.b, P.w, P.b, res2, mid, tensor_ptr(i + 2),
                                                      f8_status_word(), &why) != cudaSuccess) {
                                   (void)cudaGetLastError();
                                   return false;
                               }
                               f8_fused_plan_set_tag(fp.get(), i + 2);
                               stp.kind = -3;
                               stp.use_tc = true;
                               stp.y = tensor_ptr(i + 2);
                               stp.y_mid = mid;
                               stp.fplan = std::move(fp);
                               skip_layer = i + 1;
                               return true;
                           }()) {
                    // planned above
                } else if (f8_tc_supported(stp.g, (size_t)n * L.g.h * L.g.w * L.g.c)) {
                    PlanPtr plan = alloc_plan();
                    if (plan && f8_tc_plan_init(plan.get(), stp.g, L.q, dense_view(stp.x, stp.g), L.w, L.b, stp.res,
                                                stp.y, f8_status_word(), &why, stp.has_sib ? &stp.sib : nullptr) == cudaSuccess) {
                        stp.use_tc = true;
                        f8_tc_plan_set_tag(plan.get(), i + 1);
                        stp.plan = std::move(plan);
                    }
                }
            }
            ln.steps.push_back(std::move(stp));
        };
        for (int k = 0; k < lanes; ++k) {
            Lane &ln = lane_list[k];
            for (int i = 0; i < nl;) {
                const int r = ln.layer_region[i];
                if (r < 0) {
                    plan_layer(ln, k, i, ln.n, 0, false);
                    ++i;
                    continue;
                }
                // depth first: the whole run on one micro-batch, then on the next
                for (int img0 = 0; img0 < ln.n; img0 += ln.regions[r].mb) {
                    ln.skip_layer = -1;
                    for (int l = ln.regions[r].first; l <= ln.regions[r].last; ++l)
                        plan_layer(ln, k, l, std::min(ln.regions[r].mb, ln.n - img0), img0, true);
                }
                i = ln.regions[r].last + 1;
                ln.skip_layer = -1;
            }
        }
        // launch order: the lanes take turns, one launch each
        {
            size_t longest = 0;
            for (const Lane &ln : lane_list) longest = std::max(longest, ln.steps.size());
            for (size_t j = 0; j < longest; ++j)
                for (Lane &ln : lane_list)
                    if (j < ln.steps.size()) net->steps.push_back(std::move(ln.steps[j]));
        }
        net->plan_batch = batch;
        net->plan_x = x;
        net->plan_y = y;
        net->plan_ws = workspace;
        net->plan_force_direct = g_force_direct;
        net->plan_dump_first = dump_fusable;
        net->plan_dumping = layer_dump != nullptr;
        net->plan_options = g_plan_off;
        net->plan_micro = g_micro_batch;
        net->plan_lanes = g_lanes;
        net->plan_profiling = net->profiling;
    }

    int launches = 0;
    const bool prof = net->profiling;
    if (prof) {
        while (net->events.size() < net->steps.size() + 1) {
            cudaEvent_t ev;
            if (cudaEventCreate(&ev) != cudaSuccess) return fail(F8_ERR_CUDA, "cudaEventCreate failed");
            net->events.push_back(ev);
        }
        net->event_layer.clear();
        cudaEventRecord(net->events[0], st);
    }
    const cudaStream_t caller_stream = st;
    const bool two_lanes = net->last_lanes == 2;
    if (two_lanes) {
        // the second lane starts when the caller's stream has reached this point ...
        cudaError_t e = cudaEventRecord(net->ev_fork, caller_stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(net->lane_stream, net->ev_fork, 0);
        if (e != cudaSuccess) return cuda_fail(e, "second lane fork");
    }
    for (Step &stp : net->steps) {
        NetLayer &L = net->layers[stp.layer];
        cudaError_t e = cudaSuccess;
        st = stp.lane == 1 ? net->lane_stream : caller_stream;
        switch (stp.kind) {
            case -2:
                e = f8_launch_stem_tc(stp.g, L.q, L.pack_kh, L.pack_top, L.pack_left, L.pack_kw8 / 32, stp.fused_pool ? 1 : 0, stp.x,
                                      L.w_core, L.b, stp.y, f8_status_word(), stp.layer + 1, st, net->overlap_layers);
                ++g_tc_launches;
                break;
            case -3:
                e = f8_fused_launch(stp.fplan.get(), net->overlap_layers, st);
                ++g_tc_launches;
                break;
            case -1:
                e = f8_launch_pack_stem_pairs(stp.g.n, L.g.h, L.g.w, L.g.c, L.pack_cpad, L.pack_hp, L.pack_wp, L.pack_left, stp.x, stp.y, st,
                                              net->overlap_layers);
                break;
            case F8_LAYER_CONV:
            case F8_LAYER_LINEAR:
                // the net owns its weights (uploaded at creation), so a layer's prologue and weight loads may
                // overlap the tail of the previous layer
                if (stp.use_tc) { e = f8_tc_launch(stp.plan.get(), net->overlap_layers, st); ++g_tc_launches; }
                else e = f8_launch_conv_direct(stp.g, L.q, stp.x, L.w, L.b, stp.res, stp.y, st, net->overlap_layers,
                                               stp.has_sib ? &stp.sib : nullptr);
                break;
            case F8_LAYER_DWCONV:
                e = f8_launch_dwconv(stp.g, L.q, stp.x, L.w, L.b, stp.res, stp.y, st, net->overlap_layers);
                break;
            case F8_LAYER_MAXPOOL:
                e = f8_launch_maxpool(stp.g.n, L.g.h, L.g.w, L.g.c, L.d.conv.kh, L.d.conv.stride, L.d.conv.pad, L.g.x_signed,
                                      stp.x, stp.y, st, net->overlap_layers);
                break;
            case F8_LAYER_GAP:
                e = f8_launch_gap(stp.g.n, L.g.h, L.g.w, L.g.c, L.g.x_signed, L.q.s, stp.x, stp.y, st, net->overlap_layers);
                break;
        }
        if (e != cudaSuccess) return fail(F8_ERR_CUDA, "launch of layer %d: %s", stp.layer, cudaGetErrorString(e));
        if (net->sync_layers) {     // debugging aid: a device-side fault is then reported with the layer that raised it
            e = cudaStreamSynchronize(st);
            if (e != cudaSuccess) return fail(F8_ERR_CUDA, "layer %d failed on the device: %s", stp.layer, cudaGetErrorString(e));
        }
        ++launches;
        if (prof) {
            cudaEventRecord(net->events[launches], st);
            net->event_layer.push_back(stp.fused_pool || stp.kind == -3 ? stp.layer + 1 : stp.layer);
        }
        // copies of the outputs this step wrote: its layer's (the pooling layer's when fused), and a sibling's
        auto dump_layer = [&](int out_layer, const void *src) -> cudaError_t {
            if (!layer_dump || !layer_dump[out_layer]) return cudaSuccess;
            const int c_true = net->t_c[out_layer + 1], c_stored = net->t_cp[out_layer + 1];
            const size_t elem = (size_t)net->t_elem[out_layer + 1];
            const size_t pixels_per_image = (size_t)net->t_h[out_layer + 1] * net->t_w[out_layer + 1];
            const size_t pixels = (size_t)stp.g.n * pixels_per_image;
            uint8_t *dst = (uint8_t *)layer_dump[out_layer] + (size_t)stp.img0 * pixels_per_image * c_true * elem;
            if (c_true == c_stored)
                return cudaMemcpyAsync(dst, src, pixels * c_true * elem, cudaMemcpyDeviceToDevice, st);
            // drop the zero padding channels: one row per pixel
            return cudaMemcpy2DAsync(dst, c_true * elem, src, c_stored * elem, c_true * elem, pixels,
                                     cudaMemcpyDeviceToDevice, st);
        };
        if (stp.kind != -1) {
            e = dump_layer(stp.fused_pool || stp.kind == -3 ? stp.layer + 1 : stp.layer, stp.y);
            if (e == cudaSuccess && stp.kind == -3 && stp.y_mid) e = dump_layer(stp.layer, stp.y_mid);
            if (e == cudaSuccess && stp.has_sib) e = dump_layer(stp.layer + 1, stp.sib.y2);
            if (e != cudaSuccess) return cuda_fail(e, "layer dump copy");
        }
    }
    st = caller_stream;
    if (two_lanes) {
        // ... and the caller's stream continues when the second lane has finished
        cudaError_t e = cudaEventRecord(net->ev_join, net->lane_stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(caller_stream, net->ev_join, 0);
        if (e != cudaSuccess) return cuda_fail(e, "second lane join");
    }
    net->last_launches = launches;
    return F8_OK;
}

}   // extern "C"

// ===========================================================================================
// Forward passes from host buffers: copies of neighbouring passes overlap the compute
// ===========================================================================================

struct f8_net_host {
    int depth = 0, batch = 0;
    size_t x_bytes = 0, y_bytes = 0, ws_bytes = 0;
    std::vector<f8_net *> nets;                  // one per slot: execution plans are cached per set of buffer addresses
    std::vector<void *> x_dev, y_dev, ws;
    cudaStream_t up = nullptr, compute = nullptr, down = nullptr;
    std::vector<cudaEvent_t> ev_in, ev_done, ev_out;
    long long count = 0;
};

extern "C" {

void f8_net_host_destroy(f8_net_host *p) {
    if (!p) return;
    if (p->up) cudaStreamSynchronize(p->up);
    if (p->compute) cudaStreamSynchronize(p->compute);
    if (p->down) cudaStreamSynchronize(p->down);
    for (f8_net *n : p->nets) f8_net_destroy(n);
    for (void *b : p->x_dev) cudaFree(b);
    for (void *b : p->y_dev) cudaFree(b);
    for (void *b : p->ws) cudaFree(b);
    for (cudaEvent_t e : p->ev_in) cudaEventDestroy(e);
    for (cudaEvent_t e : p->ev_done) cudaEventDestroy(e);
    for (cudaEvent_t e : p->ev_out) cudaEventDestroy(e);
    if (p->up) cudaStreamDestroy(p->up);
    if (p->compute) cudaStreamDestroy(p->compute);
    if (p->down) cudaStreamDestroy(p->down);
    delete p;
}

f8_status f8_net_host_create(const f8_layer_desc *layers, int n_layers, const int8_t *const *host_weights,
                             const int32_t *const *host_bias, int batch, int depth, f8_net_host **out) {
    if (!out) return fail(F8_ERR_NULL, "out is NULL");
    if (batch <= 0 || depth < 1 || depth > 8) return fail(F8_ERR_SHAPE, "batch must be positive and depth in 1..8");
    std::unique_ptr<f8_net_host, void (*)(f8_net_host *)> p(new (std::nothrow) f8_net_host, f8_net_host_destroy);
    if (!p) return fail(F8_ERR_CUDA, "out of host memory");
    p->depth = depth;
    p->batch = batch;
    for (int i = 0; i < depth; ++i) {
        f8_net *n = nullptr;
        const f8_status s = f8_net_create(layers, n_layers, host_weights, host_bias, batch, &n);
        if (s != F8_OK) return s;
        p->nets.push_back(n);
    }
    const f8_net *n0 = p->nets[0];
    const int nl = (int)n0->layers.size();
    p->x_bytes = (size_t)batch * n0->t_h[0] * n0->t_w[0] * n0->t_c[0];
    p->y_bytes = (size_t)batch * n0->t_h[nl] * n0->t_w[nl] * n0->t_c[nl] * n0->t_elem[nl];
    p->ws_bytes = f8_net_workspace_bytes(n0, batch);
    cudaError_t e = cudaStreamCreateWithFlags(&p->up, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p->compute, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p->down, cudaStreamNonBlocking);
    for (int i = 0; i < depth && e == cudaSuccess; ++i) {
        void *b = nullptr;
        e = cudaMalloc(&b, round256(p->x_bytes));
        if (e == cudaSuccess) { p->x_dev.push_back(b); e = cudaMalloc(&b, round256(p->y_bytes)); }
        if (e == cudaSuccess) { p->y_dev.push_back(b); e = cudaMalloc(&b, round256(p->ws_bytes)); }
        if (e == cudaSuccess) p->ws.push_back(b);
        cudaEvent_t ev[3] = {nullptr, nullptr, nullptr};
        for (int k = 0; k < 3 && e == cudaSuccess; ++k) e = cudaEventCreateWithFlags(&ev[k], cudaEventDisableTiming);
        if (ev[0]) p->ev_in.push_back(ev[0]);
        if (ev[1]) p->ev_done.push_back(ev[1]);
        if (ev[2]) p->ev_out.push_back(ev[2]);
    }
    if (e != cudaSuccess) return cuda_fail(e, "host pipeline set-up");
    *out = p.release();
    return F8_OK;
}

f8_status f8_net_forward_host(f8_net_host *p, const void *host_x, void *host_y) {
    if (!p) return fail(F8_ERR_NULL, "pipeline is NULL");
    if (!host_x || !host_y) return fail(F8_ERR_NULL, "host_x and host_y must not be NULL");
    const int b = (int)(p->count % p->depth);
    // upload: once the slot's previous forward pass has read its input
    cudaError_t e = cudaStreamWaitEvent(p->up, p->ev_done[b], 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(p->x_dev[b], host_x, p->x_bytes, cudaMemcpyHostToDevice, p->up);
    if (e == cudaSuccess) e = cudaEventRecord(p->ev_in[b], p->up);
    // forward pass: once the input is there and the slot's previous result has left its output buffer
    if (e == cudaSuccess) e = cudaStreamWaitEvent(p->compute, p->ev_in[b], 0);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(p->compute, p->ev_out[b], 0);
    if (e != cudaSuccess) return cuda_fail(e, "host pipeline upload");
    const f8_status s = f8_net_forward(p->nets[b], p->batch, p->x_dev[b], p->y_dev[b], p->ws[b], round256(p->ws_bytes), nullptr,
                                       p->compute);
    if (s != F8_OK) return s;
    e = cudaEventRecord(p->ev_done[b], p->compute);
    // download
    if (e == cudaSuccess) e = cudaStreamWaitEvent(p->down, p->ev_done[b], 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(host_y, p->y_dev[b], p->y_bytes, cudaMemcpyDeviceToHost, p->down);
    if (e == cudaSuccess) e = cudaEventRecord(p->ev_out[b], p->down);
    if (e != cudaSuccess) return cuda_fail(e, "host pipeline download");
    ++p->count;
    return F8_OK;
}

f8_status f8_net_host_wait(f8_net_host *p) {
    if (!p) return fail(F8_ERR_NULL, "pipeline is NULL");
    cudaError_t e = cudaStreamSynchronize(p->up);
    if (e == cudaSuccess) e = cudaStreamSynchronize(p->compute);
    if (e == cudaSuccess) e = cudaStreamSynchronize(p->down);
    if (e != cudaSuccess) return cuda_fail(e, "host pipeline wait");
    return F8_OK;
}

f8_status f8_net_host_streams(f8_net_host *p, void **upload, void **compute, void **download) {
    if (!p) return fail(F8_ERR_NULL, "pipeline is NULL");
    if (upload) *upload = p->up;
    if (compute) *compute = p->compute;
    if (download) *download = p->down;
    return F8_OK;
}

int f8_net_host_launches_per_pass(const f8_net_host *p) { return p && !p->nets.empty() ? p->nets[0]->last_launches : 0; }

}   // extern "C"

