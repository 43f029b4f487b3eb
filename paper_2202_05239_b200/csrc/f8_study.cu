// Statistical study behind the format rule (Sec. 3.3, Fig. 2 / Fig. 3): for a sample of real values, the relative
// quantisation error under every 8-bit fixed-point format and the format with the smallest error.
//
//     unsigned (after ReLU):  q_FL(x) = floor(clip(max(x, 0) * 2^FL, 0, 255) + 1/2) / 2^FL      FL = 0 .. 8   (Eq. 2)
//     signed:                 q_FL(x) = floor(clip(x * 2^FL, -127, 127) + 1/2) / 2^FL           FL = 0 .. 7   (appendix)
//     err[FL] = sum (q_FL(x) - x')^2 / sum x'^2,   x' = x or max(x, 0);   FL* = first FL with the smallest err
//
// float64 throughout; scaling by powers of two is exact, so a sample's quantised value is exact and only the two
// sums are rounded.  Their order is fixed (per-thread strided partial sums, block tree, blocks in index order), so
// the result is reproducible; it differs from another summation order by rounding only.
// One pass over the sample: every thread carries the nine numerators and the denominator.
#include <math.h>

#include "f8_internal.h"

namespace {

constexpr int STUDY_THREADS = 256;
constexpr int STUDY_MAX_BLOCKS = 1024;
constexpr int STUDY_SLOTS = 10;          // nine numerators and the denominator

__global__ void __launch_bounds__(STUDY_THREADS) study_partial_kernel(const float *__restrict__ x, long long n, int is_unsigned,
                                                                      double *__restrict__ partial) {
    const int n_fl = is_unsigned ? 9 : 8;
    const double lo = is_unsigned ? 0.0 : -127.0, hi = is_unsigned ? 255.0 : 127.0;
    double acc[STUDY_SLOTS];
#pragma unroll
    for (int i = 0; i < STUDY_SLOTS; ++i) acc[i] = 0.0;
    for (long long i = (long long)blockIdx.x * STUDY_THREADS + threadIdx.x; i < n; i += (long long)gridDim.x * STUDY_THREADS) {
        double v = (double)__ldg(x + i);
        if (is_unsigned) v = fmax(v, 0.0);
        acc[9] += v * v;
        double up = 1.0, down = 1.0;
#pragma unroll
        for (int fl = 0; fl < 9; ++fl) {
            if (fl < n_fl) {
                const double q = __dmul_rn(floor(__dadd_rn(fmin(fmax(__dmul_rn(v, up), lo), hi), 0.5)), down);
                const double d = __dsub_rn(q, v);
                acc[fl] += d * d;
            }
            up *= 2.0;
            down *= 0.5;
        }
    }
    __shared__ double red[STUDY_THREADS];
    for (int slot = 0; slot < STUDY_SLOTS; ++slot) {
        red[threadIdx.x] = acc[slot];
        __syncthreads();
        for (int step = STUDY_THREADS / 2; step > 0; step >>= 1) {
            if ((int)threadIdx.x < step) red[threadIdx.x] += red[threadIdx.x + step];
            __syncthreads();
        }
        if (threadIdx.x == 0) partial[(size_t)blockIdx.x * STUDY_SLOTS + slot] = red[0];
        __syncthreads();
    }
}

__global__ void __launch_bounds__(32) study_final_kernel(const double *__restrict__ partial, int blocks, int is_unsigned,
                                                         double *__restrict__ err, int *__restrict__ best_fl) {
    __shared__ double tot[STUDY_SLOTS];
    if (threadIdx.x < STUDY_SLOTS) {
        double s = 0.0;
        for (int b = 0; b < blocks; ++b) s += partial[(size_t)b * STUDY_SLOTS + threadIdx.x];
        tot[threadIdx.x] = s;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const int n_fl = is_unsigned ? 9 : 8;
        int best = 0;
        double best_err = 0.0;
        for (int fl = 0; fl < 9; ++fl) {
            const double e = fl < n_fl ? tot[fl] / tot[9] : -1.0;      // a format that does not exist: -1
            err[fl] = e;
            if (fl < n_fl && (fl == 0 || e < best_err)) { best = fl; best_err = e; }
        }
        *best_fl = best;
    }
}

}   // namespace

extern "C" {

size_t f8_format_study_workspace_bytes(void) { return (size_t)STUDY_MAX_BLOCKS * STUDY_SLOTS * sizeof(double); }

f8_status f8_format_study_fixed(const float *x, long long n, int is_unsigned, double *err, int *best_fl, void *workspace,
                                size_t workspace_bytes, void *cuda_stream) {
    if (!x || !err || !best_fl) return f8_set_error(F8_ERR_NULL, "a required pointer is NULL");
    if (n <= 0) return f8_set_error(F8_ERR_SHAPE, "the sample must not be empty");
    if (!workspace || workspace_bytes < f8_format_study_workspace_bytes()) return f8_set_error(F8_ERR_WORKSPACE, "workspace smaller than f8_format_study_workspace_bytes()");
    if (((uintptr_t)workspace & 7) || ((uintptr_t)err & 7) || ((uintptr_t)x & 3) || ((uintptr_t)best_fl & 3))
        return f8_set_error(F8_ERR_ALIGN, "workspace and err must be 8-byte aligned, x and best_fl 4-byte aligned");
    cudaStream_t st = (cudaStream_t)cuda_stream;
    long long want = (n + STUDY_THREADS * 8 - 1) / (STUDY_THREADS * 8);
    const int blocks = (int)(want < 1 ? 1 : (want > STUDY_MAX_BLOCKS ? STUDY_MAX_BLOCKS : want));
    study_partial_kernel<<<blocks, STUDY_THREADS, 0, st>>>(x, n, is_unsigned ? 1 : 0, (double *)workspace);
    study_final_kernel<<<1, 32, 0, st>>>((const double *)workspace, blocks, is_unsigned ? 1 : 0, err, best_fl);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return f8_set_error(F8_ERR_CUDA, cudaGetErrorString(e));
    return F8_OK;
}

}   // extern "C"
