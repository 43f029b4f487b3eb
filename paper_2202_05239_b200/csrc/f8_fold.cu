// Weight "compile" step of one Conv-BN block, on the device: BatchNorm folding and scaling-factor absorption into the
// effective weight and bias (Eq. 6), choice of the weight format from the standard deviation (Eq. 1, signed branch),
// and the signed 8-bit quantiser (appendix "Double Side Quantization").
//
//     scale_i   = (gamma_i / sigma_i) * (eta_in / eta_out)
//     W_eff     = scale_i * W[i, j]                       b_eff = (beta_i - (gamma_i / sigma_i) * mu_i) / eta_out
//     FL_w      = floor(log2(40 / std(W_eff)))  clamped   std = population standard deviation of the whole tensor
//     w_q       = floor(clip(W_eff * 2^FL_w, -127, 127) + 1/2)
//     b_q       = floor(b_eff * 2^(FL_x + FL_w) + 1/2)    saturated to int32
//
// Floating point decides integer codes here, so the arithmetic is fixed: float64, one correctly rounded IEEE operation
// per step in the order written above (explicit _rn intrinsics: no contraction into fused multiply-adds), scaling by
// powers of two is exact, and floor(log2(r)) is taken from the exponent of r.  Only the summation order of the
// variance is free; it is fixed too (per-block partial sums reduced in index order), so results are reproducible.
//
// The work is four small launches: row scales -> partial sums -> format and bias -> quantised weights.  It is bound by memory
// traffic: the fp32 weights are read twice and one byte per weight is written.
#include <math.h>

#include "f8_internal.h"

namespace {

constexpr int FOLD_THREADS = 256;
constexpr int FOLD_CHUNK = 4096;         // weights of one row handled by one block iteration
constexpr int FOLD_MAX_BLOCKS = 1024;

struct FoldParams {
    int c_out, k;
    int chunks_per_row;
    long long items;                      // c_out * chunks_per_row
    double ratio;                         // eta_in / eta_out
    double eta_out;
    int fl_x, fl_min, fl_max;
    int vec4;                             // k % 4 == 0 and w 16-byte, w_q 4-byte aligned: four weights per thread and access
    const float *w, *gamma, *sigma, *beta, *mu;
    int8_t *w_q;
    int32_t *b_q;
    int *fl_w;
    double *partial;                      // [blocks][2], then [2]: mean, std
    double *scale;                        // [c_out]: (gamma / sigma) * ratio, written by the first launch
};

__global__ void __launch_bounds__(FOLD_THREADS) fold_scale_kernel(const FoldParams p) {
    const int i = blockIdx.x * FOLD_THREADS + threadIdx.x;
    if (i < p.c_out) p.scale[i] = __dmul_rn(__ddiv_rn((double)__ldg(p.gamma + i), (double)__ldg(p.sigma + i)), p.ratio);
}

__device__ __forceinline__ double row_scale(const FoldParams &p, int row) { return p.scale[row]; }

__global__ void __launch_bounds__(FOLD_THREADS) fold_stats_kernel(const FoldParams p) {
    double s1 = 0.0, s2 = 0.0;
    for (long long item = blockIdx.x; item < p.items; item += gridDim.x) {
        const int row = (int)(item / p.chunks_per_row), chunk = (int)(item - (long long)row * p.chunks_per_row);
        const double sc = row_scale(p, row);
        const float *wr = p.w + (size_t)row * p.k;
        const int j1 = min(p.k, (chunk + 1) * FOLD_CHUNK);
        if (p.vec4) {       // rows are multiples of four weights and 16-byte aligned: one 16-byte load per thread
            for (int j = chunk * FOLD_CHUNK + 4 * threadIdx.x; j < j1; j += 4 * FOLD_THREADS) {
                const float4 f = __ldg((const float4 *)(wr + j));
                const double v0 = __dmul_rn(sc, (double)f.x), v1 = __dmul_rn(sc, (double)f.y);
                const double v2 = __dmul_rn(sc, (double)f.z), v3 = __dmul_rn(sc, (double)f.w);
                s1 += (v0 + v1) + (v2 + v3);
                s2 += (v0 * v0 + v1 * v1) + (v2 * v2 + v3 * v3);
            }
        } else
        for (int j = chunk * FOLD_CHUNK + threadIdx.x; j < j1; j += FOLD_THREADS) {
            const double v = __dmul_rn(sc, (double)__ldg(wr + j));
            s1 += v;
            s2 += v * v;
        }
    }
    // block reduction in a fixed order
    __shared__ double r1[FOLD_THREADS], r2[FOLD_THREADS];
    r1[threadIdx.x] = s1;
    r2[threadIdx.x] = s2;
    __syncthreads();
    for (int step = FOLD_THREADS / 2; step > 0; step >>= 1) {
        if ((int)threadIdx.x < step) {
            r1[threadIdx.x] += r1[threadIdx.x + step];
            r2[threadIdx.x] += r2[threadIdx.x + step];
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        p.partial[2 * blockIdx.x] = r1[0];
        p.partial[2 * blockIdx.x + 1] = r2[0];
    }
}

__global__ void __launch_bounds__(FOLD_THREADS) fold_format_kernel(const FoldParams p, const int blocks) {
    __shared__ double r1[FOLD_THREADS], r2[FOLD_THREADS];
    __shared__ int fl_s;
    double s1 = 0.0, s2 = 0.0;
    for (int b = threadIdx.x; b < blocks; b += FOLD_THREADS) {
        s1 += p.partial[2 * b];
        s2 += p.partial[2 * b + 1];
    }
    r1[threadIdx.x] = s1;
    r2[threadIdx.x] = s2;
    __syncthreads();
    for (int step = FOLD_THREADS / 2; step > 0; step >>= 1) {
        if ((int)threadIdx.x < step) {
            r1[threadIdx.x] += r1[threadIdx.x + step];
            r2[threadIdx.x] += r2[threadIdx.x + step];
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const double n = (double)p.c_out * (double)p.k;
        const double mean = r1[0] / n;
        double var = r2[0] / n - mean * mean;
        if (!(var > 0.0)) var = 0.0;
        const double sd = sqrt(var);
        int fl = p.fl_max;                                   // a constant tensor: the finest format allowed
        if (sd > 0.0) {
            const double r = __ddiv_rn(40.0, sd);            // Eq. 1, signed: floor(log2(40 / sigma)) = exponent of r
            fl = isfinite(r) ? ilogb(r) : p.fl_max;
        }
        fl = max(p.fl_min, min(p.fl_max, fl));
        fl_s = fl;
        *p.fl_w = fl;
        p.partial[2 * blocks] = mean;
        p.partial[2 * blocks + 1] = sd;
    }
    __syncthreads();
    const int fa = p.fl_x + fl_s;
    for (int i = threadIdx.x; i < p.c_out; i += FOLD_THREADS) {
        const double gs = __ddiv_rn((double)__ldg(p.gamma + i), (double)__ldg(p.sigma + i));
        const double be = __ddiv_rn(__dsub_rn((double)__ldg(p.beta + i), __dmul_rn(gs, (double)__ldg(p.mu + i))), p.eta_out);
        double t = floor(__dadd_rn(scalbn(be, fa), 0.5));
        t = fmin(fmax(t, -2147483648.0), 2147483647.0);
        p.b_q[i] = (int32_t)t;
    }
}

__global__ void __launch_bounds__(FOLD_THREADS) fold_quant_kernel(const FoldParams p) {
    const int fl = *p.fl_w;
    const double pow2 = scalbn(1.0, fl);          // multiplying by a power of two is exact
    for (long long item = blockIdx.x; item < p.items; item += gridDim.x) {
        const int row = (int)(item / p.chunks_per_row), chunk = (int)(item - (long long)row * p.chunks_per_row);
        const double sc = row_scale(p, row);
        const float *wr = p.w + (size_t)row * p.k;
        int8_t *qr = p.w_q + (size_t)row * p.k;
        const int j1 = min(p.k, (chunk + 1) * FOLD_CHUNK);
        if (p.vec4) {
            for (int j = chunk * FOLD_CHUNK + 4 * threadIdx.x; j < j1; j += 4 * FOLD_THREADS) {
                const float4 f = __ldg((const float4 *)(wr + j));
                const float in[4] = {f.x, f.y, f.z, f.w};
                uint32_t packed = 0;
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const double v = __dmul_rn(__dmul_rn(sc, (double)in[t]), pow2);
                    const int q = (int)floor(__dadd_rn(fmin(fmax(v, -127.0), 127.0), 0.5));
                    packed |= (uint32_t)(q & 0xff) << (8 * t);
                }
                *(uint32_t *)(qr + j) = packed;
            }
        } else
        for (int j = chunk * FOLD_CHUNK + threadIdx.x; j < j1; j += FOLD_THREADS) {
            const double v = __dmul_rn(__dmul_rn(sc, (double)__ldg(wr + j)), pow2);
            qr[j] = (int8_t)(int)floor(__dadd_rn(fmin(fmax(v, -127.0), 127.0), 0.5));
        }
    }
}

int fold_blocks(long long items) { return (int)std::min<long long>(items, FOLD_MAX_BLOCKS); }

}   // namespace

extern "C" {

size_t f8_fold_workspace_bytes(const f8_fold_desc *d) {
    return (size_t)(2 * FOLD_MAX_BLOCKS + 2 + (d && d->c_out > 0 ? d->c_out : 0)) * sizeof(double);
}

f8_status f8_fold_quantize_fixed(const f8_fold_desc *d, const float *w, const float *gamma, const float *sigma,
                                 const float *beta, const float *mu, int8_t *w_q, int32_t *bias_q, int *fl_w,
                                 void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!d || !w || !gamma || !sigma || !beta || !mu || !w_q || !bias_q || !fl_w) return f8_set_error(F8_ERR_NULL, "a required pointer is NULL");
    if (d->c_out <= 0 || d->k <= 0 || (long long)d->c_out * d->k >= (1ll << 31)) return f8_set_error(F8_ERR_SHAPE, "c_out and k must be positive and c_out * k below 2^31");
    if (d->fl_x < 0 || d->fl_x > 8 || d->fl_w_min < -8 || d->fl_w_max > 24 || d->fl_w_min > d->fl_w_max)
        return f8_set_error(F8_ERR_FL_RANGE, "fl_x must lie in [0, 8] and [fl_w_min, fl_w_max] inside [-8, 24]");
    if (!(d->eta_in > 0.0) || !(d->eta_out > 0.0) || !isfinite(d->eta_in) || !isfinite(d->eta_out))
        return f8_set_error(F8_ERR_SHAPE, "eta_in and eta_out must be positive and finite");
    if (!workspace || workspace_bytes < f8_fold_workspace_bytes(d)) return f8_set_error(F8_ERR_WORKSPACE, "workspace smaller than f8_fold_workspace_bytes()");
    if (((uintptr_t)workspace & 7) || ((uintptr_t)w & 3) || ((uintptr_t)bias_q & 3) || ((uintptr_t)fl_w & 3))
        return f8_set_error(F8_ERR_ALIGN, "workspace must be 8-byte aligned, w / bias_q / fl_w 4-byte aligned");
    FoldParams p;
    p.c_out = d->c_out; p.k = d->k;
    p.chunks_per_row = (d->k + FOLD_CHUNK - 1) / FOLD_CHUNK;
    p.items = (long long)d->c_out * p.chunks_per_row;
    p.ratio = d->eta_in / d->eta_out;
    p.eta_out = d->eta_out;
    p.fl_x = d->fl_x; p.fl_min = d->fl_w_min; p.fl_max = d->fl_w_max;
    p.vec4 = (d->k % 4 == 0 && ((uintptr_t)w & 15) == 0 && ((uintptr_t)w_q & 3) == 0) ? 1 : 0;
    p.w = w; p.gamma = gamma; p.sigma = sigma; p.beta = beta; p.mu = mu;
    p.w_q = w_q; p.b_q = bias_q; p.fl_w = fl_w; p.partial = (double *)workspace;
    p.scale = p.partial + 2 * FOLD_MAX_BLOCKS + 2;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int blocks = fold_blocks(p.items);
    fold_scale_kernel<<<(d->c_out + FOLD_THREADS - 1) / FOLD_THREADS, FOLD_THREADS, 0, st>>>(p);
    fold_stats_kernel<<<blocks, FOLD_THREADS, 0, st>>>(p);
    fold_format_kernel<<<1, FOLD_THREADS, 0, st>>>(p, blocks);
    fold_quant_kernel<<<blocks, FOLD_THREADS, 0, st>>>(p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return f8_set_error(F8_ERR_CUDA, cudaGetErrorString(e));
    return F8_OK;
}

}   // extern "C"
