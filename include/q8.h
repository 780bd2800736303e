/*
 * q8 -- 8-bit quantized CNN inference primitives for NVIDIA B200 (sm_100a).
 *
 * C ABI of the library.  Every entry point returns a q8_status.  No exception
 * crosses this boundary, nothing aborts, no kernel traps.
 *
 * Conventions
 *  - "device pointer" = memory reachable from the current CUDA device; the
 *    caller owns every buffer, the library allocates no device memory.
 *  - `stream` is a cudaStream_t passed as void* (NULL = default stream).  All
 *    device work is enqueued on it asynchronously; only q8_read_status blocks.
 *  - Activations are NHWC, weights are KRSC (Cout, R, S, Cin), both contiguous
 *    in the channel dimension.  Quantized payloads are u8, s8 or s32; the
 *    quantization factor q of a tensor is one host-side fp32 number.
 *  - Rounding is round-half-to-even everywhere; every fp32 step is a single
 *    IEEE operation (no fused multiply-add), so results are reproducible bit
 *    for bit.
 */
#ifndef Q8_H_
#define Q8_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum q8_status {
  Q8_OK = 0,
  Q8_ERR_INVALID_ARG = 1, /* null pointer, non-positive extent, unknown enum */
  Q8_ERR_UNSUPPORTED = 2, /* legal request that no kernel here can run */
  Q8_ERR_ALIGNMENT = 3,   /* pointer or stride not aligned as documented */
  Q8_ERR_WORKSPACE = 4,   /* workspace missing or too small */
  Q8_ERR_CUDA = 5,        /* CUDA runtime/driver error; text in q8_last_error() */
  Q8_ERR_TIMEOUT = 6,     /* a bounded device-side wait gave up (status word set) */
  Q8_ERR_NONFINITE = 7    /* NaN/Inf where a finite value is required */
} q8_status;

typedef enum q8_dtype { Q8_U8 = 0, Q8_S8 = 1, Q8_S32 = 2, Q8_F32 = 3 } q8_dtype;

/* Which convolution kernel to use. */
typedef enum q8_conv_algo {
  Q8_ALGO_AUTO = 0,   /* tensor-core kernel when the shape allows it, else direct */
  Q8_ALGO_UMMA = 1,   /* tcgen05 implicit GEMM; Q8_ERR_UNSUPPORTED if not eligible */
  Q8_ALGO_DIRECT = 2  /* CUDA-core direct convolution, any shape */
} q8_conv_algo;

/* ------------------------------------------------------------------------
 * Library info and errors (host only).
 * ---------------------------------------------------------------------- */
const char* q8_version(void);
/* Text of the last error raised on the calling thread ("" if none). */
const char* q8_last_error(void);
/* Blocks until `stream` is idle, then reads and clears the device status word.
 * Returns Q8_ERR_TIMEOUT if a kernel gave up on a bounded wait since the last
 * call (its outputs are then undefined), Q8_OK otherwise. */
int q8_read_status(void* stream);

/* ------------------------------------------------------------------------
 * Calibration (Sec. "8-bit Low Precision Inference", calibration paragraph:
 * each tensor's factor is max|r| / (2^p - 1)).
 * ---------------------------------------------------------------------- */

/* *d_running_max = max(*d_running_max, max_i |x[i]|).
 * x: device, n fp32 values (n may be 0).  d_running_max: device, one fp32 the
 * caller sets to 0 before the first batch.  A NaN/Inf in x makes the result
 * NaN/Inf (largest bit pattern wins); q8_factor then reports it. */
int q8_calibrate_maxabs(const float* x, size_t n, float* d_running_max, void* stream);

/* The same for every row of a row-major [rows][cols] matrix: d_running_max[r] = max(d_running_max[r],
 * max_c |x[r][c]|).  For one factor per output channel of a weight tensor [K][R*S*C] (the paper takes one
 * factor per tensor; per-channel factors are an extension the convolution supports through scale_count = K).
 * x: device.  d_running_max: device, rows fp32 values the caller zeroes first. */
int q8_calibrate_maxabs_rows(const float* x, size_t rows, size_t cols, float* d_running_max, void* stream);

/* Host helper: *q = maxabs / (2^p - 1) as one fp32 division; *q = 1 when
 * maxabs == 0.  p in [1,31].  Q8_ERR_NONFINITE if maxabs is NaN/Inf/negative. */
int q8_factor(float maxabs, int p, float* q);

/* Host helper: *s = fp32(q_x * q_w / q_y) formed in fp64 -- the single
 * requantisation multiplier of Eq. (int8_affine) (accumulator factor q_W q_x by
 * the product rule of Eq. (arithmetics), re-expressed at q_y). */
int q8_requant_scale(float q_x, float q_w, float q_y, float* s);

/* Host helper: *q_b = q_x * q_w (one fp32 multiply), the factor at which the
 * int32 bias is quantized so that it can be added to the accumulator. */
int q8_bias_factor(float q_x, float q_w, float* q_b);

/* ------------------------------------------------------------------------
 * Eq. (Q): z = clamp(Round(x / q)), and Eq. (D): r = q * z.
 * ---------------------------------------------------------------------- */

/* z[i] = clamp(Round(x[i] / q), lo, hi) with (lo,hi) = (0,255) for Q8_U8,
 * (-128,127) for Q8_S8, (-2^31, 2^31-1) for Q8_S32.  fp32 IEEE division.  NaN
 * maps to 0.  x, z: device, n elements, same layout.  q must be finite, > 0. */
int q8_quantize(const float* x, size_t n, float q, int out_type, void* z, void* stream);

/* Eq. (Q) with one factor per row of a row-major [rows][cols] matrix: z[r][c] = clamp(Round(x[r][c] / q[r])).
 * d_q: DEVICE array of rows factors, each finite and > 0 (not checked: a bad factor yields saturated or
 * zero codes for its row).  out_type: Q8_U8, Q8_S8 or Q8_S32.  x, z: device, same layout. */
int q8_quantize_rows(const float* x, size_t rows, size_t cols, const float* d_q, int out_type, void* z,
                     void* stream);

/* As q8_quantize for an NHWC tensor of `pixels` x C values, but the output has
 * C_pad >= C channels per pixel and channels C..C_pad-1 are written as 0 (the
 * exact code of 0.0 under a symmetric quantizer).  Lets a 3-channel image feed
 * kernels that need 16-byte aligned pixels.  out_type: Q8_U8 or Q8_S8. */
int q8_quantize_pad_channels(const float* x, size_t pixels, int C, int C_pad, float q, int out_type,
                             void* z, void* stream);

/* The same for an image batch x[N][H][W][C] written into z[N][H][W_pad][C_pad] (W_pad >= W, C_pad >= C): pixels
 * beyond W and channels beyond C are zero.  A stride-2 first layer reads its input as pixel pairs, which needs
 * an even row length; a zero column on the right is never read or acts as the zero padding it replaces, as long
 * as it does not add an output column (the caller checks that).  Errors as q8_quantize_pad_channels. */
int q8_quantize_pad_image(const float* x, int N, int H, int W, int C, int W_pad, int C_pad, float q, int out_type,
                          void* z, void* stream);

/* r[i] = q * float(z[i]).  in_type: Q8_U8, Q8_S8 or Q8_S32. */
int q8_dequantize(const void* z, int in_type, size_t n, float q, float* r, void* stream);

/* ------------------------------------------------------------------------
 * Batch-norm folding (Sec. "Model Optimization"):
 *   a = gamma / sqrt(var + eps);  w' = a w;  b' = a (b - mean) + beta,
 * evaluated in fp64 and rounded once to fp32.
 * w, w_out: device [K][elems_per_k] (may alias).  b: device [K] or NULL (= 0).
 * gamma, beta, mean, var, b_out: device [K].
 * ---------------------------------------------------------------------- */
int q8_fold_bn(const float* w, const float* b, const float* gamma, const float* beta, const float* mean,
               const float* var, double eps, int K, size_t elems_per_k, float* w_out, float* b_out,
               void* stream);

/* ------------------------------------------------------------------------
 * Quantized convolution with fused epilogue (Eq. int8_affine,
 * Eq. int8_affine_fused; "+" and "x" of Eq. arithmetics; conv+ReLU and
 * conv+eltwise-sum fusion of Sec. "Model Optimization"):
 *
 *   acc[n,p,q,k] = sum_{r,s,c} x[n, p*stride_h - pad_h + r*dil_h,
 *                                   q*stride_w - pad_w + s*dil_w, c] * w[k,r,s,c]
 *                  + bias[k]                          (int32, zero padding)
 *   v = float(acc) * scale[k or 0]                    (one fp32 multiply)
 *   v = v + float(residual[n,p,q,k]) * residual_scale (product, then sum)
 *   v = max(v, 0)                                     (if relu)
 *   y = clamp(Round(v)) as u8 [0,255] or s8 [-128,127]; or v (Q8_F32); or
 *       acc (Q8_S32, raw accumulator, scale/residual/relu ignored)
 * with P = (H + 2 pad_h - dil_h (R-1) - 1) / stride_h + 1 (floor), same for Q.
 *
 * y is written at y[((n*P + p)*Q + q) * y_ldc + y_c_offset + k]: with
 * y_ldc > K the layer writes a channel slice of a wider tensor (concatenation
 * in place).  y_ldc = 0 means K.
 * ---------------------------------------------------------------------- */
typedef struct q8_conv_desc {
  int32_t N, H, W, C;       /* input  NHWC */
  int32_t K, R, S;          /* filter KRSC (C shared) */
  int32_t stride_h, stride_w;
  int32_t pad_h, pad_w;
  int32_t dil_h, dil_w;
  int32_t x_type;           /* Q8_U8 or Q8_S8 */
  int32_t res_type;         /* Q8_U8 or Q8_S8 (ignored without residual) */
  int32_t y_type;           /* Q8_U8, Q8_S8, Q8_F32 or Q8_S32 */
  int32_t relu;             /* 0/1 */
  int32_t scale_count;      /* 1 (per tensor) or K (per output channel) */
  int32_t y_ldc;            /* channels per output pixel in memory, 0 = K */
  int32_t y_c_offset;       /* first channel written */
  int32_t algo;             /* q8_conv_algo */
} q8_conv_desc;

/* Bytes of device scratch with which q8_conv2d runs `d` fastest: 0 for most shapes.  Layers whose
 * output has too few 128-row tiles to occupy the GPU (small images with long reductions, fully
 * connected layers) split the reduction R*S*C into parts; every part writes raw int32 partial sums
 * to the workspace (splits * N*P*Q * K * 4 bytes) and a second kernel adds them up, adds the bias and
 * applies the epilogue.  Integer addition is exact, so the result does not depend on the split.
 * Host only. */
int q8_conv2d_workspace_bytes(const q8_conv_desc* d, size_t* bytes);

/* Which kernel q8_conv2d would pick for `d`: writes Q8_ALGO_UMMA or
 * Q8_ALGO_DIRECT.  Host only. */
int q8_conv2d_query_algo(const q8_conv_desc* d, int* algo);

/* x: device NHWC (x_type).  w: device KRSC s8.  bias: device s32[K] or NULL.
 * scale: device fp32[scale_count].  residual: device [N,P,Q,K] dense (res_type)
 * or NULL.  y: device, see above.  workspace: device, 16-byte aligned, workspace_bytes long, or NULL.
 * It is optional: with less than q8_conv2d_workspace_bytes() the layer runs unsplit (same result,
 * slower for the shapes that would split).  Contents undefined afterwards.
 * Alignment: the tensor-core kernel needs x, w, y, residual 16-byte aligned, C
 * a multiple of 16, and for u8/s8 output y_ldc and y_c_offset multiples of 16;
 * Q8_ALGO_AUTO falls back to the direct kernel otherwise.
 * Errors: Q8_ERR_INVALID_ARG (null/extent/enum, R*S*C > 65793 which could
 * overflow int32), Q8_ERR_UNSUPPORTED (Q8_ALGO_UMMA on an ineligible shape),
 * Q8_ERR_WORKSPACE, Q8_ERR_CUDA.  Nothing is launched on error. */
int q8_conv2d(const q8_conv_desc* d, const void* x, const int8_t* w, const int32_t* bias,
              const float* scale, const void* residual, float residual_scale, void* y,
              void* workspace, size_t workspace_bytes, void* stream);

/* Two convolutions in one launch: layer 1 (descriptor d1: any filter with stride 1 that the tensor-core kernel
 * tiles with halo patches, 32, 64 or 128 output channels, 8-bit output, no residual) followed by layer 2 (d2: 1x1,
 * stride 1, no padding, reading exactly layer 1's output tensor, 8-bit output, optional fused residual sum).
 * Each layer computes what q8_conv2d computes for its descriptor (Eq. int8_affine / int8_affine_fused, bias,
 * requantization, ReLU, residual rule of Eq. arithmetics); the 8-bit tensor between them stays in shared memory
 * and is never written (the paper's "Model Optimization" section fuses the element-wise operations into the
 * convolution before them; this keeps the tensor between two convolutions on chip as well).  The result in y
 * equals q8_conv2d(d2, q8_conv2d(d1, x, ...), ...) bit for bit.
 * x: device, d1's input.  w1/bias1/scale1 and w2/bias2/scale2: device, as for q8_conv2d (bias nullable,
 * scale_count 1 or K entries).  residual: device [N][P][Q][d2->K] of d2->res_type or NULL.  y: device, d2's
 * output (y_ldc / y_c_offset of d2 honoured; d1's are ignored).  All pointers 16-byte aligned.
 * Ordering contract: weights, biases and multipliers are read BEFORE the kernel orders itself behind the
 * previous kernel of the stream, so they must not be produced by the library call enqueued immediately
 * before on the same stream (activations and the residual may be).
 * q8_conv2d_then_1x1_supported sets *supported to 1 if the pair can run this way (host only, no launch).
 * Errors: Q8_ERR_INVALID_ARG, Q8_ERR_UNSUPPORTED (pair not eligible: the message names the reason; run the two
 * layers with q8_conv2d instead), Q8_ERR_CUDA.  Nothing is launched on error. */
int q8_conv2d_then_1x1_supported(const q8_conv_desc* d1, const q8_conv_desc* d2, int* supported);
int q8_conv2d_then_1x1(const q8_conv_desc* d1, const q8_conv_desc* d2, const void* x, const int8_t* w1,
                       const int32_t* bias1, const float* scale1, const int8_t* w2, const int32_t* bias2,
                       const float* scale2, const void* residual, float residual_scale, void* y, void* stream);

/* Measurement aid (the paper has no counterpart): issue rate of the int8 tensor-core instruction behind Eq.
 * int8_affine's contraction, used as the measured "int8 tensor peak" of the convolution roofline.  Launches `ctas`
 * CTAs (one per SM is the intended use); each issues `instructions` tcgen05.mma.kind::i8 of shape 128 x bn x 32 back
 * to back on zeroed shared-memory operands, cycling over `chains` TMEM accumulators (1: each instruction depends on
 * its predecessor), and writes the SM cycles from first issue to last completion to cycles_dev[cta] (device, `ctas`
 * entries, caller-owned).  Asynchronous on `stream`; a bounded wait that runs out shows in q8_read_status.
 * MACs per CTA = instructions * 128 * bn * 32.  bn: multiple of 16 in [16,256]; chains * max(bn,32) <= 512.
 * Errors: Q8_ERR_INVALID_ARG, Q8_ERR_CUDA. */
int q8_int8_mma_rate(int bn, int chains, int instructions, int ctas, unsigned long long* cycles_dev, void* stream);

/* Test aid (the paper has no counterpart): every wait inside the tensor-core kernels is bounded; when one runs
 * out, the kernel sets a bit of the device status word, all roles of the CTA drain and the kernel returns, and the
 * next q8_read_status reports Q8_ERR_TIMEOUT and clears the word.  This call makes that happen without any fault:
 * it launches one small CTA whose first warp waits `limit_us` microseconds (1 .. 1 000 000) on a barrier nothing
 * signals, and whose second warp waits with the library's normal limit (2 s) and must leave early because the first
 * gave up.  Asynchronous on `stream`; afterwards q8_read_status(stream) returns Q8_ERR_TIMEOUT (site mask 0x5)
 * once, then Q8_OK.  Errors: Q8_ERR_INVALID_ARG, Q8_ERR_CUDA. */
int q8_selftest_bounded_wait(unsigned int limit_us, void* stream);

/* q8_conv2d for callers that cannot allocate device memory (the paper has no counterpart; this is a
 * property of the library, not of the method).  Meant for hosts where every byte of device memory was
 * handed out before this library is called, or where cudaMalloc is off limits because it stalls the
 * device: the scratch of the split reduction (see q8_conv2d_workspace_bytes) is a fixed array of
 * q8_static_workspace_bytes() = 16 MiB inside the library image instead of a caller buffer.
 *  - Every GPU on which the library is used holds that array until the process exits.  Under CUDA's default
 *    lazy module loading the device sets the 16 MiB (and the library's kernel images) aside at the first call
 *    into the library on that device, not when the process starts: a host that hands out all remaining device
 *    memory must make that first call before it does so, or the call fails with Q8_ERR_CUDA (out of memory).
 *    q8_static_workspace_bytes() is such a first call: besides returning the size it looks the array up on
 *    the current device (and returns the size alone where there is no usable device).
 *  - A layer that would need more scratch is refused with Q8_ERR_WORKSPACE (nothing is launched);
 *    q8_conv2d with workspace = NULL still runs it, unsplit.  Layers that need none just run.
 *  - The first call on each device (of q8_static_workspace_bytes or q8_conv2d_static_workspace) looks up
 *    the array's device address (cudaGetSymbolAddress, with that device current).  Make that first call
 *    outside any stream capture.  Later calls leave the amount of free device memory unchanged.
 *  - All calls share the one array and it keeps the previous call's contents.  Nothing needs clearing
 *    (each call writes every partial sum before reading it), but two calls whose kernels overlap on the
 *    GPU (different streams, or threads) race on it: serialise them.
 *  - No cudaMalloc, cudaFree or other allocating call is made.
 * Arguments, result and errors otherwise as q8_conv2d. */
size_t q8_static_workspace_bytes(void);
int q8_conv2d_static_workspace(const q8_conv_desc* d, const void* x, const int8_t* w, const int32_t* bias,
                               const float* scale, const void* residual, float residual_scale, void* y,
                               void* stream);

/* ------------------------------------------------------------------------
 * Channel concatenation of quantized branches under one factor (the paper
 * gives no rule; the caller passes the shared factor, normally the largest
 * branch factor as in the "+" rule of Eq. arithmetics).  Branch i is written
 * as clamp(Round(float(z) * fp32(q_i / q_out))) (ratio formed in fp64), or
 * copied unchanged when that ratio is exactly 1.
 * xs: host array of n_in device pointers, branch i is [pixels][channels[i]].
 * channels, in_factors: host arrays.  y: device [pixels][sum channels].
 * t: Q8_U8 or Q8_S8.  n_in <= 8.
 * ---------------------------------------------------------------------- */
int q8_concat(int n_in, const void* const* xs, const int* channels, const float* in_factors,
              float out_factor, int t, size_t pixels, void* y, void* stream);

/* One branch of such a concatenation, written into a channel slice of a wider tensor: for branches that
 * cannot be produced in place (a pooled tensor whose factor differs from the shared one) while the
 * convolution branches write their slices themselves (q8_conv_desc y_ldc / y_c_offset).
 * x: device [pixels][channels].  y: device [pixels][y_ldc]; channels y_c_offset .. y_c_offset+channels-1
 * are written, the rest of y is untouched.  Same arithmetic as q8_concat.
 * Errors: Q8_ERR_INVALID_ARG (null pointer, channels <= 0, slice outside y_ldc, type not U8/S8),
 * Q8_ERR_NONFINITE (factor not finite positive). */
int q8_concat_branch(const void* x, int channels, float in_factor, float out_factor, int t, size_t pixels,
                     void* y, int y_ldc, int y_c_offset, void* stream);

/* ------------------------------------------------------------------------
 * Pooling between quantized layers (not described in the paper; needed to
 * run whole networks in int8).  The factor is unchanged.
 * max: maximum over the in-image cells of the window.
 * avg: clamp(Round(float(sum of in-image cells) * fp32(1/(kh*kw)))) -- full
 *      window divisor, padding counts as zero.
 * ceil_mode: output extent rounds up (last window may hang over the edge).
 * x: device NHWC, y: device [N,P,Q,C]; t: Q8_U8 or Q8_S8.
 * ---------------------------------------------------------------------- */
int q8_pool_out_extent(int H, int k, int stride, int pad, int ceil_mode, int* out);
int q8_maxpool2d(const void* x, int t, int N, int H, int W, int C, int kh, int kw, int stride_h,
                 int stride_w, int pad_h, int pad_w, int ceil_mode, void* y, void* stream);
int q8_avgpool2d(const void* x, int t, int N, int H, int W, int C, int kh, int kw, int stride_h,
                 int stride_w, int pad_h, int pad_w, int ceil_mode, void* y, void* stream);

/* ------------------------------------------------------------------------
 * The SSD tail and the FP32 route for signed sums.  The paper runs SSD with a detection-output layer
 * (artifact appendix) and sends potentially negative activations through FP32 (Sec. "8-bit Low Precision
 * Inference", calibration paragraph) but prints no arithmetic for them; these calls follow the detector's
 * published definition with every floating-point step one IEEE fp32 operation in a fixed order.
 * ---------------------------------------------------------------------- */

/* L2 normalisation across the channels of each pixel, on unsigned 8-bit codes:
 *   S = sum_c z_c^2 (integer),  r = 1 / sqrt(float(S) * (qx * qx) + eps)   (one IEEE division per pixel),
 *   y_c = clamp(Round((float(z_c) * mult[c]) * r), 0, 255),   mult[c] = gamma_c qx / qy (formed by the caller).
 * x, y: device [pixels][C] u8 (may not overlap); d_mult: device [C] fp32.  The fast path needs C % 4 == 0,
 * x and y 4-byte aligned and d_mult 16-byte aligned; anything else takes a scalar kernel.  An all-zero pixel
 * with eps == 0 gives code 0.  Asynchronous on `stream`.
 * Errors: Q8_ERR_INVALID_ARG (null pointer, C outside 1..65536), Q8_ERR_NONFINITE (qx not finite positive, eps
 * negative or not finite), Q8_ERR_CUDA. */
int q8_l2norm(const void* x, size_t pixels, int C, float qx, float eps, const float* d_mult, void* y, void* stream);

/* The FP32 route of a residual sum whose summands may be negative: a and b are dequantized (fp32) convolution
 * outputs, y = clamp(Round(max(a + b, 0) / q), 0, 255) as u8 (one fp32 add, one IEEE division, Round half to even).
 * a, b: device fp32 [n]; y: device u8 [n].  Vector path when a, b are 16-byte and y 4-byte aligned.
 * Errors: Q8_ERR_INVALID_ARG, Q8_ERR_NONFINITE (q not finite positive), Q8_ERR_CUDA. */
int q8_add_relu_quantize(const float* a, const float* b, size_t n, float q, void* y, void* stream);

/* Detection output for a batch of N images.
 * Inputs: n_sources (<= 8) head tensors.  Source i has cells[i] cells per image and boxes_per_cell[i] boxes per
 * cell; its localisation values for image n, cell k, box b are the four floats at
 * loc[i] + (n * cells[i] + k) * loc_stride[i] + 4 b, its class logits the `classes` floats at
 * conf[i] + (n * cells[i] + k) * conf_stride[i] + classes * b (strides in floats; device pointers in HOST arrays;
 * a merged head passes the same base twice with an offset).  Boxes are numbered source by source, cell by cell, box
 * by box: P = sum cells * boxes_per_cell in all.  d_priors: device [P][4] fp32 (centre x, centre y, width, height),
 * 16-byte aligned.  variances: HOST [4].
 * Steps: corners = decode(loc, prior, variances) (centre-size code, exp by a fixed fp32 recipe, no clipping);
 * probabilities = softmax(logits); per image and class other than `background` (-1: none): boxes with probability
 * > conf_thresh, best nms_top_k by probability (ties: lower box index), greedy suppression of boxes whose overlap
 * (intersection over union) with a kept box exceeds nms_thresh; per image the best keep_top_k of all kept (ties:
 * lower class, lower box index).
 * Outputs: d_out device [N][keep_top_k][6] fp32 rows (class, probability, xmin, ymin, xmax, ymax), best first, rows
 * beyond the count zero; d_counts device [N] int32.
 * workspace: device, 256-byte aligned, q8_detection_output_workspace_bytes(...) bytes, caller-owned; three kernels
 * are enqueued on `stream`, nothing is allocated.
 * Limits: P <= 16384, nms_top_k <= 512, (foreground classes) * nms_top_k <= 16384, N <= 65535.
 * Errors: Q8_ERR_INVALID_ARG, Q8_ERR_UNSUPPORTED (a limit), Q8_ERR_NONFINITE (thresholds), Q8_ERR_ALIGNMENT,
 * Q8_ERR_WORKSPACE, Q8_ERR_CUDA.  Nothing is launched on error. */
int q8_detection_output_workspace_bytes(int N, int P, int classes, int background, int nms_top_k, int keep_top_k,
                                        size_t* bytes);
int q8_detection_output(int n_sources, const float* const* loc, const int* loc_stride, const float* const* conf,
                        const int* conf_stride, const int* cells, const int* boxes_per_cell, const float* d_priors,
                        const float* variances, int N, int classes, int background, float conf_thresh,
                        float nms_thresh, int nms_top_k, int keep_top_k, void* workspace, size_t workspace_bytes,
                        float* d_out, int* d_counts, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* Q8_H_ */
