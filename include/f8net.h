/*
 * f8net.h -- C ABI of the fixed-point 8-bit inference library for NVIDIA B200 (sm_100a).
 *
 * The library evaluates the inference arithmetic of F8Net ("Fixed-Point 8-bit Only
 * Multiplication for Network Quantization"): every tensor element is an 8-bit
 * integer code q with a per-tensor fractional length FL and stands for q * 2^-FL
 * (word length 8 everywhere, Sec. 4.3).  A layer multiplies 8-bit activations by
 * 8-bit effective weights, accumulates in int32, adds the effective bias (Eq. 6),
 * optionally adds a shortcut tensor after aligning its format by a bit shift
 * (Sec. 4.3 "Clipping-Level Sharing", Fig. 4), and applies the fixed-point
 * quantizer of the consumer, Eq. 2 (unsigned, clip [0, 255]; this is also the
 * ReLU / PACT clip, Eq. 4) or its signed form from the appendix (clip
 * [-127, 127]).  Because all formats are powers of two, the quantizer is a
 * rounding arithmetic shift by  s = FL_x + FL_w - FL_y  followed by the clip;
 * no int32 or floating-point multiplication by a learned scale is needed for
 * rescaling.  (Where an accumulator or a shortcut has to be moved to a finer
 * format, the tensor-core epilogue does that left shift as a multiply-add with
 * the power of two 2^shift, which this GPU executes on a less loaded pipe; the
 * result is the shift's, bit for bit.  Building with -DF8_EPILOGUE_SHIFTS_ONLY
 * uses shift instructions instead.)
 *
 * For one output element, with FA = FL_x + FL_w:
 *
 *     acc = sum_taps x * w + bias                         exact, int32
 *     if residual:  F = max(FA, FL_r)
 *                   acc = (acc << (F - FA)) + (r << (F - FL_r)),  FA = F
 *     s   = FA - FL_y
 *     t   = s > 0 ? floor((acc + 2^(s-1)) / 2^s) : acc * 2^(-s)    (round half up)
 *     y   = min(hi, max(lo, t))
 *
 * Conventions for every entry point
 *   - Pointers named x, w, bias, residual, y, workspace are DEVICE pointers unless
 *     the name starts with host_.  Tensors are dense, NHWC (channel fastest),
 *     16-byte aligned.  The caller owns every buffer; the library allocates no
 *     output and keeps no pointer after the call returns (f8_net objects own a
 *     device copy of their parameters, see f8_net_create).
 *   - cuda_stream is a cudaStream_t passed as void* (NULL = default stream).
 *     Calls validate their arguments on the host, enqueue work on the stream and
 *     return without synchronising.
 *   - Errors are reported by the return code; nothing is launched when validation
 *     fails.  f8_last_error() gives a message for the calling thread's last
 *     failure.  Kernels never trap: a wait that does not complete within its
 *     bound makes the kernel return early (its output is then incomplete) and
 *     records itself in a device status word and in a host-visible copy of it.
 *     Every entry point that enqueues work looks at that copy first (a host
 *     load, no synchronisation) and returns F8_ERR_TIMEOUT without enqueuing
 *     anything while a record is pending; f8_device_status() synchronises,
 *     reports the details and clears it.
 *   - Preconditions the library cannot check on device data: every accumulator
 *     (including the aligned residual sum) fits in int32.  f8_net_create checks
 *     this bound from the host copies of the parameters.  The single-layer entry
 *     points only see the shapes: they reject layers whose worst case
 *     K * 255 * 128 * 2^sh_acc reaches 2^30 and otherwise rely on the caller for
 *         |sum + bias| * 2^sh_acc + 255 * 2^sh_res + 2^(s-1) < 2^31
 *     (sh_acc / sh_res: the alignment shifts of accumulator and residual, s the
 *     requantisation shift): the fast epilogue adds the rounding constant 2^(s-1)
 *     to the bias once per layer and forms this sum in int32; a bias beyond that
 *     bound wraps silently.
 */
#ifndef F8NET_H
#define F8NET_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    F8_OK = 0,
    F8_ERR_NULL = 1,          /* a required pointer is NULL */
    F8_ERR_SHAPE = 2,         /* non-positive or inconsistent extents */
    F8_ERR_DTYPE = 3,         /* dtype code not valid in this position */
    F8_ERR_FL_RANGE = 4,      /* fractional length outside the accepted range */
    F8_ERR_SHIFT_RANGE = 5,   /* a shift amount outside [-8, 31] (requantisation) or [0, 22] (alignment) */
    F8_ERR_ALIGN = 6,         /* a pointer is not 16-byte aligned */
    F8_ERR_ACC_BOUND = 7,     /* the int32 accumulator bound cannot be guaranteed */
    F8_ERR_WORKSPACE = 8,     /* workspace missing or too small */
    F8_ERR_UNSUPPORTED = 9,   /* valid request the library does not implement */
    F8_ERR_CUDA = 10,         /* a CUDA runtime / driver call failed */
    F8_ERR_TIMEOUT = 11       /* a kernel gave up on a bounded wait (see f8_device_status) */
} f8_status;

typedef enum { F8_U8 = 0, F8_S8 = 1, F8_S32 = 2,
               F8_S32_RELU = 3      /* output of the sibling entry points only: int32, max(value, 0) */
} f8_dtype;

/*
 * One convolution-shaped layer (Eq. 6).  Input x is [n, h, w, c]; the output is
 * [n, ho, wo, c_out] with ho = (h + 2 pad - kh) / stride + 1 (same for wo);
 * dilation 1; cross-correlation; taps outside the image contribute 0.
 *   x_dtype  F8_U8 or F8_S8, format fl_x (0..8 unsigned, 0..7 signed; Eq. 2 and its signed form)
 *   weights  int8 in [-128, 127], format fl_w (-8..24: the arithmetic only sees the shift)
 *   y_dtype  F8_U8: quantizer of Eq. 2, clip [0, 255] (this is ReLU + PACT clip);
 *            F8_S8: signed quantizer, clip [-127, 127];
 *            F8_S32: raw accumulator in format fl_x + fl_w (fl_y ignored)
 *   r_dtype / fl_r describe the residual tensor and are read only when the
 *            residual pointer of the call is not NULL.
 */
typedef struct {
    int n, h, w, c;
    int c_out, kh, kw, stride, pad;
    int x_dtype, y_dtype, r_dtype;
    int fl_x, fl_w, fl_y, fl_r;
} f8_conv_desc;

/* Dense convolution (Eq. 6; residual add of Sec. 4.3; quantizer Eq. 2 / signed form).
 *   w_ohwi [c_out, kh, kw, c] int8; bias [c_out] int32 in format fl_x + fl_w or NULL (zero);
 *   residual NULL or [n, ho, wo, c_out] 8-bit (r_dtype, fl_r); y [n, ho, wo, c_out].
 * Layers with c % 16 == 0 whose input is at least 128 KiB run on the tensor cores
 * (tcgen05.mma kind::i8); every other shape takes a CUDA-core kernel with the same
 * result.  workspace: f8_conv_workspace_bytes(desc) bytes (may be 0 -> NULL allowed). */
f8_status f8_conv2d_fixed(const f8_conv_desc *desc, const void *x, const int8_t *w_ohwi, const int32_t *bias,
                          const void *residual, void *y, void *workspace, size_t workspace_bytes,
                          void *cuda_stream);

/* One 32-bit sum, several consumers (Sec. 4.3 "Clipping-Level Sharing and Private Fractional Length", Fig. 4;
 * appendix "Private Fractional Lengths Enabling Different Clipping-Levels").  The paper keeps a layer's sum in
 * 32 bits and quantizes it once per child layer with that child's own fractional length, and keeps a shortcut in
 * 32 bits until it is added.  This call is f8_conv2d_fixed with
 *   - a second output y2 (NULL: none) of dtype y2_dtype with its private fl_y2, produced from the same sum;
 *   - desc->r_dtype == F8_S32 allowed: the residual is an int32 tensor in format fl_r (0..31);
 *   - F8_S32_RELU allowed for y_dtype / y2_dtype: the sum behind a ReLU, max(v, 0), unrounded, int32 in the format
 *     F = max(fl_x + fl_w, fl_r) of the aligned sum (F8_S32: the sum itself).
 * Both 8-bit outputs equal what two f8_conv2d_fixed calls with fl_y and fl_y2 would give.  Precondition as for every
 * layer: the aligned sum fits int32.  Runs with direct stores (not the staged TMA epilogue); same validation errors. */
f8_status f8_conv2d_siblings_fixed(const f8_conv_desc *desc, int y2_dtype, int fl_y2, const void *x,
                                   const int8_t *w_ohwi, const int32_t *bias, const void *residual, void *y, void *y2,
                                   void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Two consecutive layers in one launch: a dense convolution `conv` (Eq. 6, quantizer of Eq. 2) and the pointwise (1x1,
 * stride 1, no padding) convolution `pw` that reads its output, with the optional shortcut add of Sec. 4.3 behind the
 * second layer -- the last two layers of a ResNet bottleneck block (Sec. 5 workloads).  Eq. 6 holds per layer, so both
 * outputs are exactly what f8_conv2d_fixed(conv) followed by f8_conv2d_fixed(pw) give; the difference is that the
 * first layer's output tile goes from the epilogue straight into the second GEMM through shared memory and is not
 * written to device memory unless y_mid is given.
 *   conv  c = 64, c_out = 64, any kh * kw <= 16, stride, pad; y_dtype F8_U8; input at least 128 KiB; no shortcut
 *   pw    n / h / w / c = conv's output, c_out = 256, x_dtype / fl_x = conv's y_dtype / fl_y, y_dtype F8_U8 or F8_S8;
 *         r_dtype / fl_r describe `residual` ([n, ho, wo, 256] 8-bit, NULL: none)
 *   both requantisation shifts must lie in 1..24
 *   w_conv [64, kh, kw, 64], w_pw [256, 64] int8; bias_conv [64], bias_pw [256] int32 or NULL; all pointers DEVICE,
 *   16-byte aligned; y_mid NULL or [n, ho, wo, 64] (receives the first layer's output); y [n, ho, wo, 256].
 * Errors: as f8_conv2d_fixed for each descriptor; F8_ERR_SHAPE / F8_ERR_DTYPE when pw does not continue conv;
 * F8_ERR_UNSUPPORTED for shapes outside the list above (call the two layers separately). */
f8_status f8_conv_pointwise_fixed(const f8_conv_desc *conv, const f8_conv_desc *pw, const void *x, const int8_t *w_conv,
                                  const int32_t *bias_conv, const int8_t *w_pw, const int32_t *bias_pw, const void *residual,
                                  void *y_mid, void *y, void *cuda_stream);

/* Depthwise convolution (one kh x kw filter per channel; MobileNet layers of Sec. 5),
 * c_out must equal c.  w_chw [c, kh, kw] int8.  Everything else as f8_conv2d_fixed. */
f8_status f8_dwconv_fixed(const f8_conv_desc *desc, const void *x, const int8_t *w_chw, const int32_t *bias,
                          const void *residual, void *y, void *workspace, size_t workspace_bytes,
                          void *cuda_stream);

/* Fully connected layer: Eq. 6 with the sum over k inputs.  x [n, k] 8-bit, w_out_k [out, k] int8,
 * bias [out] int32 (format fl_x + fl_w) or NULL, y [n, out] of y_dtype (F8_S32 = logits in
 * format fl_x + fl_w, the values "stored in 32-bit" of Sec. 4.3). */
f8_status f8_linear_fixed(int n, int k, int out, int x_dtype, int y_dtype, int fl_x, int fl_w, int fl_y,
                          const void *x, const int8_t *w_out_k, const int32_t *bias, void *y,
                          void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Max pooling k x k / stride with padding (not in the paper: integer max over the taps inside
 * the image; codes and format unchanged).  x, y 8-bit NHWC of dtype x_dtype. */
f8_status f8_maxpool_fixed(int n, int h, int w, int c, int k, int stride, int pad, int x_dtype,
                           const void *x, void *y, void *cuda_stream);

/* Global average pooling (not in the paper): sum over h*w followed by the quantizer of Eq. 2
 * (or its signed form) with shift ceil(log2(h*w)) + fl_x - fl_y; y [n, c] of dtype x_dtype. */
f8_status f8_global_avgpool_fixed(int n, int h, int w, int c, int x_dtype, int fl_x, int fl_y,
                                  const void *x, void *y, void *cuda_stream);

size_t f8_conv_workspace_bytes(const f8_conv_desc *desc);

/* ---------------------------------------------------------------- whole networks */

typedef enum { F8_LAYER_CONV = 0, F8_LAYER_DWCONV = 1, F8_LAYER_MAXPOOL = 2, F8_LAYER_GAP = 3,
               F8_LAYER_LINEAR = 4,
               F8_LAYER_SIBLING = 5     /* a second consumer's view of the previous layer's 32-bit sum */
} f8_layer_kind;

/* Tensor 0 is the network input; layer i writes tensor i + 1.  src / res name tensors
 * (res = -1: no residual).  conv.n is ignored (the batch is given per call); for
 * F8_LAYER_LINEAR conv.c = inputs and conv.c_out = outputs; for pooling layers only the
 * geometry, x_dtype and fl_x / fl_y are read.
 *
 * Sibling consumers (Sec. 4.3, Fig. 4): an F8_LAYER_SIBLING layer i must directly follow a dense convolution
 * (layer i - 1) and name that layer's output tensor as src (src = i).  Its tensor i + 1 is the SAME 32-bit sum
 * quantised with this layer's own conv.y_dtype / conv.fl_y (F8_U8, F8_S8, or F8_S32 / F8_S32_RELU to keep it in
 * 32 bits, e.g. as the shortcut of the next block); the other fields are ignored.  Both tensors are written by
 * one launch.  Dense convolutions inside a network may name an int32 tensor as their residual (r_dtype F8_S32,
 * fl_r = the format that tensor was produced in: fl_x + fl_w of its producer, or max(fl_x + fl_w, fl_r) if the
 * producer had a residual itself). */
typedef struct {
    int kind;
    int src;
    int res;
    f8_conv_desc conv;
} f8_layer_desc;

typedef struct f8_net f8_net;

/* Builds a network object from HOST copies of the parameters (host_weights[i] / host_bias[i]
 * may be NULL for layers without parameters).  Validates every layer, checks the int32
 * accumulator bound of each output channel from the actual weights (F8_ERR_ACC_BOUND),
 * copies (and where needed re-packs) the parameters to the current device.  The last
 * layer's output is the network output.  Must be called with the target device current. */
f8_status f8_net_create(const f8_layer_desc *layers, int n_layers, const int8_t *const *host_weights,
                        const int32_t *const *host_bias, int max_batch, f8_net **out);

/* Bytes of device workspace f8_net_forward needs for this batch (all intermediate tensors). */
size_t f8_net_workspace_bytes(const f8_net *net, int batch);

/* One forward pass (the fixed-point inference path end to end).  x: [batch, h, w, c] network
 * input; y: the last layer's output ([batch, out] int32 logits for a net ending in a linear
 * layer).  layer_dump: NULL, or an array of n_layers device pointers; a non-NULL entry i
 * receives a copy of layer i's output (for parity checks).
 * Schedule: layers run one after the other over the whole batch on cuda_stream.  Two alternatives exist, both off
 * by default because they measured slower on this GPU (every extra launch costs about 5 us of drained SMs):
 * f8_debug_set_lanes(2) cuts the batch into two halves that run as two independent passes, one on cuda_stream and
 * one on a stream the network owns, launched alternately (the call returns with cuda_stream waiting for both);
 * f8_debug_set_micro_batch executes a run of layers with equal output size depth-first over micro-batches so that
 * the tensors inside the run stay in the L2 cache.  Images are independent, so neither changes a result.  Status: if a kernel of an earlier pass on this object gave up a bounded
 * wait, the call returns F8_ERR_TIMEOUT before enqueuing anything (see f8_device_status). */
f8_status f8_net_forward(f8_net *net, int batch, const void *x, void *y, void *workspace,
                         size_t workspace_bytes, void *const *layer_dump, void *cuda_stream);

/* Number of kernels the last f8_net_forward on this object enqueued. */
int f8_net_last_launch_count(const f8_net *net);

/* Number of those kernels that ran two layers at once (a 64 -> 64 convolution and the 64 -> 256 pointwise layer that
 * alone reads its output: see f8_conv_pointwise_fixed).  f8_net_forward does that wherever the shapes allow; the
 * first layer's output then exists in device memory only in a pass that asks for layer dumps. */
int f8_net_fused_pairs(const f8_net *net);

/* Per-layer timing.  With profiling on, f8_net_forward records a CUDA event after every kernel it
 * enqueues; f8_net_get_layer_ms waits for the last profiled pass and writes the device time of
 * each layer (ms[n_layers]; a stem's packing pre-pass is added to its layer) and, if
 * on_tensor_cores is not NULL, 1 for layers that ran on the tcgen05 path. */
f8_status f8_net_set_profiling(f8_net *net, int on);
f8_status f8_net_get_layer_ms(f8_net *net, float *ms, int *on_tensor_cores);

void f8_net_destroy(f8_net *net);

/* ---------------------------------------------------------------- forward passes from host buffers */

/* The same forward pass for callers whose images and results live in HOST memory (the end-to-end path).  The
 * object owns `depth` slots, each with its own network object, device input / output buffers and workspace
 * (allocated here, on the current device), and three streams: while the GPU computes pass i, the copy engines
 * upload the input of pass i + 1 and download the result of pass i - 1.  Every step of the arithmetic still runs
 * in f8_net_forward.
 *   f8_net_forward_host   host_x: [batch, h, w, c] network input, host_y: the last layer's output, both in HOST
 *                         memory (page-locked memory is needed for the copies to overlap; pageable memory works but
 *                         serialises them).  One cudaMemcpyAsync each way per call.  Returns at once; host_x may be
 *                         reused and host_y read after f8_net_host_wait (or after `depth` further calls).
 *   f8_net_host_wait      blocks until everything submitted so far has finished.
 *   f8_net_host_streams   the three streams (cudaStream_t as void*), so that a caller can record its own events
 *                         around a run of calls.
 * Errors as f8_net_create / f8_net_forward; F8_ERR_SHAPE for depth outside 1..8. */
typedef struct f8_net_host f8_net_host;
f8_status f8_net_host_create(const f8_layer_desc *layers, int n_layers, const int8_t *const *host_weights,
                             const int32_t *const *host_bias, int batch, int depth, f8_net_host **out);
f8_status f8_net_forward_host(f8_net_host *pipe, const void *host_x, void *host_y);
f8_status f8_net_host_wait(f8_net_host *pipe);
f8_status f8_net_host_streams(f8_net_host *pipe, void **upload, void **compute, void **download);
int f8_net_host_launches_per_pass(const f8_net_host *pipe);
void f8_net_host_destroy(f8_net_host *pipe);

/* ---------------------------------------------------------------- one 32-bit value, several consumers */

/* A value with several consumers is "stored in 32-bit" and quantised once per consumer with that consumer's own
 * fractional length (Sec. 4.3, "Clipping-Level Sharing and Private Fractional Length"; appendix "Private Fractional
 * Lengths Enabling Different Clipping-Levels": the cost is only some bit shifting).  acc [n] int32 in format fa
 * (for instance the F8_S32 output of f8_conv2d_fixed, fa = fl_x + fl_w) ->
 *     y1[i] = clip(rshift_round(acc[i], fa - fl_y1))    and, when y2 != NULL,    y2[i] = clip(rshift_round(acc[i], fa - fl_y2))
 * with the unsigned clip [0, 255] (Eq. 2; also the ReLU) for F8_U8 and [-127, 127] (appendix) for F8_S8; a negative
 * shift multiplies.  All pointers DEVICE; y1 / y2 [n] bytes.  Errors: F8_ERR_NULL, F8_ERR_SHAPE (n < 0),
 * F8_ERR_DTYPE, F8_ERR_FL_RANGE, F8_ERR_SHIFT_RANGE (fa - fl outside [-8, 31]), F8_ERR_ALIGN (acc not 4-byte aligned). */
f8_status f8_requantize_dual_fixed(long long n, const int32_t *acc, int fa, void *y1, int y1_dtype, int fl_y1,
                                   void *y2, int y2_dtype, int fl_y2, void *cuda_stream);

/* ---------------------------------------------------------------- weight compile step */

/* One Conv-BN block's parameters turned into what the layer entry points above consume (Sec. 4.2 - 4.3):
 *
 *     W_eff[i, j] = (gamma_i / sigma_i) * (eta_in / eta_out) * W[i, j]         effective weight, Eq. 6
 *     b_eff[i]    = (beta_i - (gamma_i / sigma_i) * mu_i) / eta_out             effective bias, Eq. 6
 *     FL_w        = floor(log2(40 / std(W_eff))), clamped to [fl_w_min, fl_w_max]   Eq. 1, signed branch
 *     w_q         = round(clip(W_eff * 2^FL_w, -127, 127))                      signed fix_quant (appendix), WL = 8
 *     bias_q      = round(b_eff * 2^(fl_x + FL_w)), saturated to int32          accumulator format
 *
 * gamma, beta: BatchNorm weight and bias; sigma, mu: its running standard deviation and mean (sigma is the
 * standard deviation itself, already including any epsilon); eta_in / eta_out: the fix scaling factors of Eq. 5,
 * eta_fix = 2^FL * alpha / 255, of this block's input quantiser and of the next block's.  std is the population
 * standard deviation over the whole tensor; round is round half up.  All arithmetic is float64 with one IEEE
 * operation per step in the order written, so the integer codes are reproducible.
 *
 * w [c_out, k] fp32 (k = kh * kw * c_in in the layout the convolution will use, e.g. OHWI), gamma / sigma /
 * beta / mu [c_out] fp32, w_q [c_out, k] int8, bias_q [c_out] int32, fl_w one int -- all DEVICE pointers; the
 * chosen fractional length is written to *fl_w on the device (read it back after the stream has finished).
 * workspace: at least f8_fold_workspace_bytes() bytes of device memory, 8-byte aligned; its contents need not be
 * initialised and are overwritten.  Four kernels are enqueued on the stream; nothing is synchronised.
 * Errors: F8_ERR_NULL, F8_ERR_SHAPE (extents, non-positive eta), F8_ERR_FL_RANGE, F8_ERR_WORKSPACE,
 * F8_ERR_ALIGN; nothing is launched when validation fails. */
typedef struct {
    int c_out, k;
    int fl_x;                   /* fractional length of the block's input activations, 0..8 */
    int fl_w_min, fl_w_max;     /* accepted range of the weight format, inside [-8, 24] (the paper: 0..7) */
    double eta_in, eta_out;
} f8_fold_desc;

size_t f8_fold_workspace_bytes(const f8_fold_desc *desc);
f8_status f8_fold_quantize_fixed(const f8_fold_desc *desc, const float *w, const float *gamma, const float *sigma,
                                 const float *beta, const float *mu, int8_t *w_q, int32_t *bias_q, int *fl_w,
                                 void *workspace, size_t workspace_bytes, void *cuda_stream);

/* ---------------------------------------------------------------- statistical study of the formats */

/* The experiment of Sec. 3.3 (Fig. 2, Fig. 3; appendix "More Details for Statistical Analysis") on a caller-given
 * sample x [n] fp32 (DEVICE): relative quantisation error  err[FL] = sum (q_FL(x') - x')^2 / sum x'^2  for every
 * 8-bit format -- unsigned, Eq. 2, FL = 0..8, with x' = max(x, 0) (the sample "processed by ReLU"), or signed
 * (appendix), FL = 0..7, x' = x -- and the format with the smallest error (the smaller FL on a tie), which Eq. 1
 * approximates from the standard deviation.  err: 9 doubles on the DEVICE (err[8] = -1 for the signed study),
 * best_fl: one int on the DEVICE.  float64 arithmetic, fixed summation order.  workspace: at least
 * f8_format_study_workspace_bytes() bytes of device memory, 8-byte aligned, contents irrelevant.  Two kernels are
 * enqueued; nothing is synchronised.  Errors: F8_ERR_NULL, F8_ERR_SHAPE (n <= 0), F8_ERR_WORKSPACE, F8_ERR_ALIGN. */
size_t f8_format_study_workspace_bytes(void);
f8_status f8_format_study_fixed(const float *x, long long n, int is_unsigned, double *err, int *best_fl,
                                void *workspace, size_t workspace_bytes, void *cuda_stream);

/* ---------------------------------------------------------------- diagnostics */

const char *f8_status_str(f8_status s);
const char *f8_last_error(void);

/* Synchronises the device and returns F8_ERR_TIMEOUT if any kernel since the last call
 * abandoned a bounded wait (the word is cleared), F8_ERR_CUDA on a CUDA error, else F8_OK. */
f8_status f8_device_status(void);

/* Number of tensor-core (tcgen05) convolution kernels this process has launched so far; lets a
 * caller confirm which path a layer took. */
long long f8_tc_launch_count(void);

/* Test hook: non-zero routes every dense layer to the CUDA-core kernel (same results). */
void f8_debug_force_direct(int on);

/* Test hook: switches planning choices off so that the alternative code paths can be checked against
 * the oracle (results never change; the default, 0, is the fastest plan).  Process-wide; takes effect for
 * plans made after the call (f8_net objects plan again when the mask has changed).
 *   F8_PLAN_OFF_RESIDENT_WEIGHTS  weights are streamed through the pipeline even where they would fit in shared memory
 *   F8_PLAN_OFF_WINDOWED          3x3 stride-1 layers gather their taps by im2col instead of reading whole padded rows
 *   F8_PLAN_OFF_DUAL_ISSUE        one MMA-issuing thread per CTA
 *   F8_PLAN_OFF_ALT_PRODUCERS     one pair of TMA producer warps
 *   F8_PLAN_OFF_PAIRS             no two-CTA tiles (tcgen05 cta_group::2)
 *   F8_PLAN_OFF_DW_DP4A           depthwise 3x3 layers do not use the packed-dot-product kernels
 *   F8_PLAN_OFF_TILE_GROUPS       pointwise layers with a single K chunk do not hand several M tiles over at once
 *   F8_PLAN_OFF_DW_WALK           depthwise 3x3 stride-1 layers do not use the row-walking kernel (with both off: the strip kernel)
 *   F8_PLAN_OFF_STEM_KERNEL       first layers take the packed-row-pair GEMM instead of the first-layer kernel
 *   F8_PLAN_OFF_STEM_POOL_FUSION  the max pool behind a first layer runs as its own kernel
 *   F8_PLAN_OFF_LAYER_OVERLAP     f8_net_forward launches without programmatic dependent launch
 *   F8_PLAN_OFF_LAYER_FUSION      f8_net_forward runs a 64 -> 64 convolution and the 64 -> 256 pointwise layer behind it as two launches
 *   F8_PLAN_OFF_LANES             f8_net_forward runs the whole batch as one sequence of launches on the caller's stream
 *   F8_PLAN_SYNC_LAYERS           f8_net_forward synchronises after every launch, so that a device fault is
 *                                 reported with the layer that raised it */
enum {
    F8_PLAN_OFF_RESIDENT_WEIGHTS = 1, F8_PLAN_OFF_WINDOWED = 2, F8_PLAN_OFF_DUAL_ISSUE = 4, F8_PLAN_OFF_ALT_PRODUCERS = 8,
    F8_PLAN_OFF_PAIRS = 16, F8_PLAN_OFF_DW_WALK = 32, F8_PLAN_OFF_STEM_KERNEL = 64, F8_PLAN_OFF_STEM_POOL_FUSION = 128,
    F8_PLAN_OFF_LAYER_OVERLAP = 256, F8_PLAN_OFF_LANES = 512, F8_PLAN_SYNC_LAYERS = 1024, F8_PLAN_OFF_DW_DP4A = 2048,
    F8_PLAN_OFF_TILE_GROUPS = 4096, F8_PLAN_OFF_LAYER_FUSION = 8192
};
void f8_debug_plan_options(unsigned off_mask);

/* The micro-batch schedule of f8_net_forward (off by default: on this GPU the extra launches cost more than the
 * memory traffic they save).  images = -1: a run of layers whose tensors exceed the L2 cache at the full batch is
 * executed depth-first over micro-batches sized to half the cache, provided every dense layer of the run still has
 * two tiles per SM; images > 0 forces that micro-batch for every run of three or more layers with equal output
 * size; 0 switches it off.  f8_net_micro_batching reports what the last forward pass of a network did: the number
 * of micro-batched runs (return value) and the smallest micro-batch (*images). */
void f8_debug_set_micro_batch(int images);
int f8_net_micro_batching(const f8_net *net, int *images);

/* Lanes of f8_net_forward: 0 = the library's rule (one lane: two measured slower on this GPU), 1 / 2 = that many.
 * f8_net_lanes reports what the last forward pass used. */
void f8_debug_set_lanes(int lanes);
int f8_net_lanes(const f8_net *net);

/* What the most recent tensor-core plan of this process decided (n <= 10 ints are written, the count is returned):
 * [0] flags below, [1] epilogue variant (0 generic, 1 u8, 2 u8 + residual, 3 s8, 4 s8 + residual), [2] N tile,
 * [3] K bytes per chunk, [4] pipeline stages, [5] K chunks per stage, [6] M tiles, [7] N tiles, [8] CTAs launched,
 * [9] staged output buffers.  Lets a test assert which path a case took and how many tiles each CTA walked. */
enum {
    F8_PLAN_RESIDENT_WEIGHTS = 1, F8_PLAN_WINDOWED = 2, F8_PLAN_DUAL_ISSUE = 4, F8_PLAN_ALT_PRODUCERS = 8,
    F8_PLAN_PLAIN_MATRIX = 16, F8_PLAN_STAGED_EPILOGUE = 32, F8_PLAN_PAIRS = 64, F8_PLAN_ROW_TILES = 128,
    F8_PLAN_TILE_GROUPS = 256
};
int f8_debug_last_plan(int *info, int n);

/* Bound of every in-kernel barrier wait, in milliseconds at the maximum SM clock (0 restores the default of
 * about two seconds).  Process-wide; for kernels launched after the call. */
void f8_debug_set_wait_limit_ms(double ms);

/* Failure-detection check that harms nothing: one thread of a one-block kernel waits, with the given bound, on a
 * barrier that nothing will ever arrive at.  The wait runs out, the kernel records it in the device status word
 * (site 199) and returns normally; the next f8_device_status() reports F8_ERR_TIMEOUT. */
f8_status f8_debug_wait_timeout_probe(double limit_ms, void *cuda_stream);

/* Tensor-core probe: every SM issues `iters` back-to-back tcgen05.mma kind::i8
 * 128 x 256 x 32 instructions on resident shared-memory tiles (no global traffic).
 * Returns the number of int8 operations (2 per multiply-accumulate) issued in *ops so that
 * the caller can time the launch and obtain the attainable INT8 rate of the device. */
f8_status f8_mma_i8_probe(int iters, double *ops, void *cuda_stream);

/* ---------------------------------------------------------------- a call that allocates nothing */

/* Largest input, in bytes of its 8-bytes-per-pixel padded copy (n * h * wp * 8, wp about w + pad), that
 * f8_stem_conv2d_fixed_static accepts: 40 images of 224 x 224 at once. */
#define F8_STATIC_STEM_MAX_BYTES ((size_t)16 * 1024 * 1024)

/* The paper has no counterpart to this entry point; it exists for callers that may not allocate
 * device memory at the moment they need a result: code running under a framework that has reserved
 * the whole device for its own pool, a real-time loop that must not take the allocator's lock, or a
 * host that hands this library a fixed memory budget.  Every other entry point either takes a caller
 * workspace or (f8_net_create, the first use of the status word) calls cudaMalloc.
 *
 * It computes the same thing as f8_conv2d_fixed for a few-channel first layer ("stem": c <= 8, even
 * stride, kw <= 32, no residual, 8-bit output), on the tensor cores: the image is widened to 8 bytes
 * per pixel, the weights are re-packed to match, and the convolution runs over that copy.  The copy,
 * the packed weights and the kernel's status word live in one array that is part of the library image
 * (about 16 MiB of device memory on every GPU that loads the library, until the process exits).  The
 * call makes no cudaMalloc / cudaFree and calls no allocating routine; x, w_ohwi, bias and y are the
 * caller's device buffers as in f8_conv2d_fixed.
 *
 *   - Inputs whose padded copy exceeds F8_STATIC_STEM_MAX_BYTES are rejected with F8_ERR_WORKSPACE;
 *     inputs whose padded copy is below 128 KiB, or shapes outside the list above, with
 *     F8_ERR_UNSUPPORTED (use f8_conv2d_fixed for those).
 *   - The first call on a device looks up the array's device address (once per device, with that
 *     device current).  Make that first call outside any stream capture.
 *   - All calls share the array and it keeps what the previous call left there.  Each call rewrites
 *     every byte it later reads, so earlier contents never leak into a result, but two calls whose
 *     GPU work overlaps (different streams, different host threads) race on it: serialise them.
 *   - check_previous != 0 first synchronises the stream and returns F8_ERR_TIMEOUT if a kernel of an
 *     earlier call on this device gave up on a bounded wait (f8_device_status does not see this
 *     entry point's status word); with 0 the call never synchronises. */
f8_status f8_stem_conv2d_fixed_static(const f8_conv_desc *desc, const void *x, const int8_t *w_ohwi,
                                      const int32_t *bias, void *y, int check_previous, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* F8NET_H */
