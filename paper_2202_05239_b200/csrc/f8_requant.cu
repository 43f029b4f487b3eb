// Sibling layers with private fractional lengths (Sec. 4.3 "Clipping-Level Sharing", appendix "Private Fractional
// Lengths"): a value that feeds several layers is kept in 32 bits and quantised once per consumer, each with its own
// format; the formats differ by powers of two, so each consumer's view costs a shift.  This kernel takes the int32 tensor a layer produced (format fa,
// e.g. the F8_S32 output of a convolution) and emits one or two 8-bit tensors:
//
//     y_k = clip(rshift_round(acc, fa - fl_k), lo_k, hi_k)        k = 1, 2;   rshift_round = round half up
//
// Purely bound by memory traffic (4 bytes read, 1 or 2 written per element): 16-byte loads, 4-byte stores per output.
#include "f8_epilogue.cuh"

namespace {

__device__ __forceinline__ uint32_t requant4(const int4 a, const F8Requant &q) {
    return f8_pack4(f8_requant(a.x, 0, q), f8_requant(a.y, 0, q), f8_requant(a.z, 0, q), f8_requant(a.w, 0, q));
}

__global__ void __launch_bounds__(256) requant_dual_kernel(const int32_t *__restrict__ acc, long long n, F8Requant q1, F8Requant q2,
                                                            uint8_t *__restrict__ y1, uint8_t *__restrict__ y2, int vec) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (vec) {
        const long long n4 = n >> 2;
        long long i = i0;
        // four independent 16-byte loads in flight per thread
        for (; i + 3 * stride < n4; i += 4 * stride) {
            int4 a[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) a[u] = __ldg((const int4 *)acc + i + u * stride);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                ((uint32_t *)y1)[i + u * stride] = requant4(a[u], q1);
                if (y2) ((uint32_t *)y2)[i + u * stride] = requant4(a[u], q2);
            }
        }
        for (; i < n4; i += stride) {
            const int4 a = __ldg((const int4 *)acc + i);
            ((uint32_t *)y1)[i] = requant4(a, q1);
            if (y2) ((uint32_t *)y2)[i] = requant4(a, q2);
        }
        for (long long i = (n4 << 2) + i0; i < n; i += stride) {       // ragged tail
            const int a = __ldg(acc + i);
            y1[i] = (uint8_t)(f8_requant(a, 0, q1) & 0xff);
            if (y2) y2[i] = (uint8_t)(f8_requant(a, 0, q2) & 0xff);
        }
    } else {
        for (long long i = i0; i < n; i += stride) {
            const int a = __ldg(acc + i);
            y1[i] = (uint8_t)(f8_requant(a, 0, q1) & 0xff);
            if (y2) y2[i] = (uint8_t)(f8_requant(a, 0, q2) & 0xff);
        }
    }
}

bool make_q(int fa, int fl_y, int y_dtype, F8Requant *q) {
    if (y_dtype != F8_U8 && y_dtype != F8_S8) return false;
    if (fl_y < 0 || fl_y > (y_dtype == F8_U8 ? 8 : 7)) return false;
    q->sh_acc = 0; q->sh_res = 0; q->has_res = 0; q->r_signed = 0;
    q->s = fa - fl_y;
    q->y_kind = y_dtype;
    q->lo = y_dtype == F8_U8 ? 0 : -127;
    q->hi = y_dtype == F8_U8 ? 255 : 127;
    return true;
}

}   // namespace

extern "C" f8_status f8_requantize_dual_fixed(long long n, const int32_t *acc, int fa, void *y1, int y1_dtype, int fl_y1, void *y2,
                                              int y2_dtype, int fl_y2, void *cuda_stream) {
    if (!acc || !y1) return f8_set_error(F8_ERR_NULL, "acc and y1 must not be NULL");
    if (n < 0) return f8_set_error(F8_ERR_SHAPE, "n must not be negative");
    if (fa < -8 || fa > 32) return f8_set_error(F8_ERR_FL_RANGE, "accumulator format outside [-8, 32]");
    F8Requant q1, q2;
    if (!make_q(fa, fl_y1, y1_dtype, &q1)) return f8_set_error(y1_dtype == F8_U8 || y1_dtype == F8_S8 ? F8_ERR_FL_RANGE : F8_ERR_DTYPE, "y1: 8-bit dtype with fl in its range");
    q2 = q1;
    if (y2 && !make_q(fa, fl_y2, y2_dtype, &q2)) return f8_set_error(y2_dtype == F8_U8 || y2_dtype == F8_S8 ? F8_ERR_FL_RANGE : F8_ERR_DTYPE, "y2: 8-bit dtype with fl in its range");
    if (q1.s < -8 || q1.s > 31 || (y2 && (q2.s < -8 || q2.s > 31))) return f8_set_error(F8_ERR_SHIFT_RANGE, "shift fa - fl_y outside [-8, 31]");
    if (((uintptr_t)acc & 3)) return f8_set_error(F8_ERR_ALIGN, "acc must be 4-byte aligned");
    if (n == 0) return F8_OK;
    const int vec = (((uintptr_t)acc & 15) == 0 && ((uintptr_t)y1 & 3) == 0 && (!y2 || ((uintptr_t)y2 & 3) == 0)) ? 1 : 0;
    long long blocks = (n / 4 + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (blocks < 1) blocks = 1;
    requant_dual_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)cuda_stream>>>(acc, n, q1, q2, (uint8_t *)y1, (uint8_t *)y2, vec);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return f8_set_error(F8_ERR_CUDA, cudaGetErrorString(e));
    return F8_OK;
}
