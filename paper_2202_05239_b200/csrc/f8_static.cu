// f8_stem_conv2d_fixed_static: the packed-stem convolution with all of its scratch memory in a
// file-scope device array, for callers that cannot allocate (see include/f8net.h).
#include <cuda_runtime.h>

#include <stdio.h>
#include <string.h>

#include "f8_internal.h"

namespace {

constexpr size_t STATUS_BYTES = 256;                 // [0, 256): status word of the kernels launched here
constexpr size_t WEIGHT_BYTES = 64 * 1024;           // [256, 256 + 64 KiB): weights re-packed to 8 bytes per tap
constexpr size_t INPUT_OFFSET = STATUS_BYTES + WEIGHT_BYTES;
constexpr size_t SCRATCH_BYTES = INPUT_OFFSET + F8_STATIC_STEM_MAX_BYTES;

// Part of the library image: every GPU that loads the library holds these bytes until the process exits.
// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[SCRATCH_BYTES];

// [c_out][kh][kw][c] -> [c_out][kh][kw8], tap s of the filter row at bytes 8*s .. 8*s + c - 1, zeros elsewhere.
// Writes every byte of the packed tensor, so nothing of an earlier call survives.
__global__ void __launch_bounds__(256) pack_stem_weights_kernel(const int8_t *__restrict__ w, int8_t *__restrict__ wp,
                                                                int c_out, int kh, int kw, int c, int kw8) {
    const int total = c_out * kh * kw8;
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        const int in_row = idx % kw8;
        const int row = idx / kw8;                   // co * kh + r
        const int s = in_row >> 3, ch = in_row & 7;
        wp[idx] = (s < kw && ch < c) ? w[((size_t)row * kw + s) * c + ch] : (int8_t)0;
    }
}

unsigned char *g_scratch_addr[64] = {nullptr};       // device address of the array, per device

// plan storage: tensor maps are 64-byte aligned objects; no heap allocation on this path
alignas(64) unsigned char g_plan_storage[4096];

}   // namespace

extern "C" f8_status f8_stem_conv2d_fixed_static(const f8_conv_desc *d, const void *x, const int8_t *w,
                                                 const int32_t *bias, void *y, int check_previous, void *cuda_stream) {
    if (!d) return f8_set_error(F8_ERR_NULL, "descriptor is NULL");
    if (d->n < 0 || d->h <= 0 || d->w <= 0 || d->c <= 0 || d->c_out <= 0 || d->kh <= 0 || d->kw <= 0 || d->stride <= 0 ||
        d->pad < 0 || d->h + 2 * d->pad < d->kh || d->w + 2 * d->pad < d->kw)
        return f8_set_error(F8_ERR_SHAPE, "non-positive or inconsistent extent in descriptor");
    if (d->c > 8 || d->stride % 2 != 0 || d->kw > 32 || d->kh > 255)
        return f8_set_error(F8_ERR_UNSUPPORTED, "f8_stem_conv2d_fixed_static takes c <= 8, an even stride and kw <= 32");
    if (d->x_dtype != F8_U8 && d->x_dtype != F8_S8) return f8_set_error(F8_ERR_DTYPE, "x_dtype must be F8_U8 or F8_S8");
    if (d->y_dtype != F8_U8 && d->y_dtype != F8_S8) return f8_set_error(F8_ERR_DTYPE, "y_dtype must be F8_U8 or F8_S8");
    if (d->fl_x < 0 || d->fl_x > (d->x_dtype == F8_U8 ? 8 : 7) || d->fl_y < 0 || d->fl_y > (d->y_dtype == F8_U8 ? 8 : 7) ||
        d->fl_w < -8 || d->fl_w > 24)
        return f8_set_error(F8_ERR_FL_RANGE, "fractional length outside the accepted range");
    const int s = d->fl_x + d->fl_w - d->fl_y;
    if (s < -8 || s > 31) return f8_set_error(F8_ERR_SHIFT_RANGE, "requantisation shift outside [-8, 31]");
    if ((long long)d->kh * d->kw * d->c * 255 * 128 >= (1ll << 30))
        return f8_set_error(F8_ERR_ACC_BOUND, "filter too large for the int32 accumulator");
    if (d->n == 0) return F8_OK;
    if (!x || !w || !y) return f8_set_error(F8_ERR_NULL, "x, w and y must not be NULL");
    if ((((uintptr_t)x | (uintptr_t)w | (uintptr_t)y | (uintptr_t)bias) & 15) != 0)
        return f8_set_error(F8_ERR_ALIGN, "device pointers must be 16-byte aligned");

    const int ho = (d->h + 2 * d->pad - d->kh) / d->stride + 1;
    const int wo = (d->w + 2 * d->pad - d->kw) / d->stride + 1;
    const int kw8 = (d->kw * 8 + 31) / 32 * 32;
    int wp = d->w + d->pad;
    if (wp < (wo - 1) * d->stride + kw8 / 8) wp = (wo - 1) * d->stride + kw8 / 8;
    wp = (wp + 1) / 2 * 2;                            // rows stay multiples of 16 bytes
    const size_t packed_bytes = (size_t)d->n * d->h * wp * 8;
    const size_t weight_bytes = (size_t)d->c_out * d->kh * kw8;
    if (packed_bytes > F8_STATIC_STEM_MAX_BYTES) {
        char msg[200];
        snprintf(msg, sizeof(msg), "padded input copy needs %zu bytes, the static array holds %zu: split the batch",
                 packed_bytes, (size_t)F8_STATIC_STEM_MAX_BYTES);
        return f8_set_error(F8_ERR_WORKSPACE, msg);
    }
    if (weight_bytes > WEIGHT_BYTES) return f8_set_error(F8_ERR_WORKSPACE, "re-packed weights exceed 64 KiB");

    F8ConvGeom g;
    g.n = d->n; g.h = d->h; g.w = d->w; g.c = kw8;     // the layer as the tensor cores see it: kh x 1 over kw8 channels
    g.ho = ho; g.wo = wo; g.c_out = d->c_out;
    g.kh = d->kh; g.kw = 1;
    g.stride_h = d->stride; g.stride_w = 1;
    g.pad_h = d->pad; g.pad_w = 0;
    g.x_signed = d->x_dtype == F8_S8;
    if (!f8_tc_supported(g, packed_bytes))
        return f8_set_error(F8_ERR_UNSUPPORTED, "input too small for this entry point (padded copy below 128 KiB): use f8_conv2d_fixed");
    if (f8_tc_plan_size() > sizeof(g_plan_storage)) return f8_set_error(F8_ERR_UNSUPPORTED, "plan storage too small");

    // once per device, with that device current: the device address behind the array's name
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= 64) return f8_set_error(F8_ERR_CUDA, "cudaGetDevice failed");
    if (!g_scratch_addr[dev]) {
        unsigned char *ptr = nullptr;
        e = cudaGetSymbolAddress((void **)&ptr, g_static_scratch);
        if (e != cudaSuccess || !ptr) {
            char msg[200];
            snprintf(msg, sizeof(msg), "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
            return f8_set_error(F8_ERR_CUDA, msg);
        }
        g_scratch_addr[dev] = ptr;
    }
    unsigned char *scratch = g_scratch_addr[dev];
    int *status_word = (int *)scratch;
    int8_t *w_packed = (int8_t *)(scratch + STATUS_BYTES);
    unsigned char *x_packed = scratch + INPUT_OFFSET;
    cudaStream_t st = (cudaStream_t)cuda_stream;

    if (check_previous) {
        e = cudaStreamSynchronize(st);
        int v = 0;
        if (e == cudaSuccess) e = cudaMemcpy(&v, status_word, sizeof(int), cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) return f8_set_error(F8_ERR_CUDA, cudaGetErrorString(e));
        if (v != 0) {
            cudaMemsetAsync(status_word, 0, sizeof(int), st);
            return f8_set_error(F8_ERR_TIMEOUT, "a kernel of an earlier call abandoned a bounded wait");
        }
    }

    F8Requant q;
    q.sh_acc = q.sh_res = 0;
    q.s = s;
    q.lo = d->y_dtype == F8_U8 ? 0 : -127;
    q.hi = d->y_dtype == F8_U8 ? 255 : 127;
    q.y_kind = d->y_dtype;
    q.has_res = 0;
    q.r_signed = 0;

    F8TcTensorView v;                                  // overlapping strided view of the padded copy
    v.base = x_packed;
    v.dim_c = (uint64_t)kw8; v.dim_w = (uint64_t)wo; v.dim_h = (uint64_t)d->h; v.dim_n = (uint64_t)d->n;
    v.stride_w = (uint64_t)d->stride * 8;
    v.stride_h = (uint64_t)wp * 8;
    v.stride_n = (uint64_t)wp * 8 * d->h;
    F8TcPlan *plan = (F8TcPlan *)g_plan_storage;
    const char *why = "";
    e = f8_tc_plan_init(plan, g, q, v, w_packed, bias, nullptr, y, status_word, &why);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        char msg[300];
        snprintf(msg, sizeof(msg), "%s: %s", why, cudaGetErrorString(e));
        return f8_set_error(e == cudaErrorInvalidValue || e == cudaErrorNotSupported ? F8_ERR_UNSUPPORTED : F8_ERR_CUDA, msg);
    }
    const int total_w = (int)weight_bytes;
    pack_stem_weights_kernel<<<(total_w + 255) / 256, 256, 0, st>>>(w, w_packed, d->c_out, d->kh, d->kw, d->c, kw8);
    e = cudaGetLastError();
    if (e == cudaSuccess) e = f8_launch_pack_stem(d->n, d->h, d->w, d->c, wp, d->pad, x, x_packed, st);
    if (e == cudaSuccess) e = f8_tc_launch(plan, false, st);
    if (e != cudaSuccess) return f8_set_error(F8_ERR_CUDA, cudaGetErrorString(e));
    return F8_OK;
}
