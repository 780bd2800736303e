// q8 oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
//
// A plain, slow, single-threaded-per-image CPU statement of what the 8-bit
// quantized convolution path computes, written from the paper's equations.
// Only tests, the smoke check and the benchmark's CPU-baseline leg may call
// it; the CUDA library never does, and the two share no code.
//
// Every function names the passage of the paper it follows.  Where the paper
// is silent or inconsistent the reading taken is stated next to the code.
//
// Parity status: every function below is pinned by CPU tests against closed
// forms, hand-computed cases, invariants or an independent formulation
// (see tests/test_oracle_pins.py).  Nothing here is "parity unpinned" except
// the whole-network accuracy of the paper's Table 3, which needs datasets
// and trained weights that are not available.
//
// Build: g++ -O2 -ffp-contract=off -fno-fast-math -shared -fPIC (see build.py).

#include <cmath>
#include <cstddef>
#include <cstdint>
#include <thread>
#include <vector>

extern "C" {

// ---------------------------------------------------------------------------
// Calibration: the factor of a tensor is max|r| / (2^p - 1)  (Sec. "8-bit Low
// Precision Inference", calibration paragraph).
// ---------------------------------------------------------------------------

// Sequential max of absolute values.  `init` is the running maximum carried
// over from earlier calibration batches (0 for the first one).
float q8o_maxabs(const float* r, size_t n, float init) {
  float m = init;
  for (size_t i = 0; i < n; ++i) {
    float a = std::fabs(r[i]);
    if (a > m) m = a;
  }
  return m;
}

// factor = max / (2^p - 1), one fp32 division.  Reading: an all-zero tensor
// (max == 0) gets factor 1 so that Q stays defined.
float q8o_factor(float maxabs, int p) {
  if (maxabs == 0.0f) return 1.0f;
  float denom = (float)((1ll << p) - 1);
  return maxabs / denom;
}

// ---------------------------------------------------------------------------
// Eq. (Q): z = max(min(Round(r / q), hi), lo), Round = half-to-even.
// The literal bounds are lo = -2^p, hi = 2^p - 1; storage types narrow them
// (u8: [0,255], s8: [-128,127], s32: [-2^31, 2^31-1]) and the caller passes
// the pair it wants.  The quotient is one fp32 IEEE division.  NaN maps to 0.
// ---------------------------------------------------------------------------
void q8o_quantize(const float* r, size_t n, float q, double lo, double hi, int32_t* z) {
  for (size_t i = 0; i < n; ++i) {
    float t = r[i] / q;
    float rounded = std::nearbyintf(t);  // default rounding mode: nearest-even
    double d = (double)rounded;
    int32_t v;
    if (rounded != rounded) v = 0;
    else if (d < lo) v = (int32_t)lo;
    else if (d > hi) v = (int32_t)hi;
    else v = (int32_t)d;
    z[i] = v;
  }
}

// Eq. (D): r' = q * z, one fp32 multiply of q with float(z).
void q8o_dequantize(const int32_t* z, size_t n, float q, float* r) {
  for (size_t i = 0; i < n; ++i) r[i] = q * (float)z[i];
}

// ---------------------------------------------------------------------------
// Eq. (arithmetics), first line:  z1_q1 + z2_q2 = Q_p(D(z1_q1) + D(z2_q2), max(q1,q2)).
// Returns the factor of the sum.
// ---------------------------------------------------------------------------
float q8o_eltwise_add(const int32_t* z1, float q1, const int32_t* z2, float q2, size_t n,
                      double lo, double hi, int32_t* z) {
  float qo = q1 > q2 ? q1 : q2;
  std::vector<float> sum(n);
  for (size_t i = 0; i < n; ++i) {
    float a = q1 * (float)z1[i];
    float b = q2 * (float)z2[i];
    sum[i] = a + b;
  }
  q8o_quantize(sum.data(), n, qo, lo, hi, z);
  return qo;
}

// ---------------------------------------------------------------------------
// Batch-norm folding (Sec. "Model Optimization"):
//   a = gamma / sqrt(var + eps),  w' = a * w,  b' = a * (b - mean) + beta,
// evaluated in fp64 and rounded once to fp32.  Weights are [K][elems_per_k].
// ---------------------------------------------------------------------------
void q8o_fold_bn_f64(const float* w, const float* b, const float* gamma, const float* beta,
                     const float* mean, const float* var, double eps, int K, size_t elems_per_k,
                     double* w_out, double* b_out) {
  for (int k = 0; k < K; ++k) {
    double a = (double)gamma[k] / std::sqrt((double)var[k] + eps);
    for (size_t e = 0; e < elems_per_k; ++e)
      w_out[(size_t)k * elems_per_k + e] = a * (double)w[(size_t)k * elems_per_k + e];
    double b0 = b ? (double)b[k] : 0.0;
    b_out[k] = a * (b0 - (double)mean[k]) + (double)beta[k];
  }
}

// The fp32 model parameters: the fp64 values above rounded once to fp32.
void q8o_fold_bn(const float* w, const float* b, const float* gamma, const float* beta,
                 const float* mean, const float* var, double eps, int K, size_t elems_per_k,
                 float* w_out, float* b_out) {
  std::vector<double> wd((size_t)K * elems_per_k), bd(K);
  q8o_fold_bn_f64(w, b, gamma, beta, mean, var, eps, K, elems_per_k, wd.data(), bd.data());
  for (size_t i = 0; i < wd.size(); ++i) w_out[i] = (float)wd[i];
  for (int k = 0; k < K; ++k) b_out[k] = (float)bd[k];
}

// Combined requantisation scale s = q_x * q_w / q_y, formed in fp64 and rounded
// once to fp32 (reading of Eq. int8_affine: the accumulator carries factor
// q_W * q_x by the product rule, and Q_{8,q_y} divides by q_y).
float q8o_requant_scale(float qx, float qw, float qy) {
  return (float)((double)qx * (double)qw / (double)qy);
}

// Factor of the int32 bias: the product q_x * q_w as one fp32 multiply (reading
// of the subscript printed as a sum in Eq. int8_affine).
float q8o_bias_factor(float qx, float qw) { return qx * qw; }

// ---------------------------------------------------------------------------
// Integer convolution accumulator (Eq. arithmetics second line, Eq. int8_affine):
//   acc[n,p,q,k] = sum_{r,s,c} x[n, p*st_h - pad_h + r*dil_h, q*st_w - pad_w + s*dil_w, c]
//                              * w[k,r,s,c]  (+ bias[k]),
// zero outside the image, int32 accumulation.  x is NHWC (u8 or s8 bytes),
// w is KRSC s8, acc is [N,P,Q,K].  Images are independent; `threads` > 1 only
// hands whole images to std::threads, the loop nest per image is unchanged.
// ---------------------------------------------------------------------------
static void conv_acc_image(const uint8_t* x, int x_signed, const int8_t* w, const int32_t* bias,
                           int H, int W, int C, int K, int R, int S, int st_h, int st_w,
                           int pad_h, int pad_w, int dil_h, int dil_w, int P, int Q,
                           int32_t* acc) {
  for (int p = 0; p < P; ++p)
    for (int q = 0; q < Q; ++q)
      for (int k = 0; k < K; ++k) {
        int32_t a = 0;
        for (int r = 0; r < R; ++r) {
          int h = p * st_h - pad_h + r * dil_h;
          if (h < 0 || h >= H) continue;
          for (int s = 0; s < S; ++s) {
            int ww = q * st_w - pad_w + s * dil_w;
            if (ww < 0 || ww >= W) continue;
            const uint8_t* xp = x + ((size_t)h * W + ww) * C;
            const int8_t* wp = w + (((size_t)k * R + r) * S + s) * C;
            for (int c = 0; c < C; ++c) {
              int32_t xv = x_signed ? (int32_t)(int8_t)xp[c] : (int32_t)xp[c];
              a += xv * (int32_t)wp[c];
            }
          }
        }
        if (bias) a = (int32_t)((uint32_t)a + (uint32_t)bias[k]);
        acc[((size_t)p * Q + q) * K + k] = a;
      }
}

void q8o_conv_acc(const uint8_t* x, int x_signed, const int8_t* w, const int32_t* bias,
                  int N, int H, int W, int C, int K, int R, int S, int st_h, int st_w,
                  int pad_h, int pad_w, int dil_h, int dil_w, int32_t* acc, int threads) {
  int P = (H + 2 * pad_h - dil_h * (R - 1) - 1) / st_h + 1;
  int Q = (W + 2 * pad_w - dil_w * (S - 1) - 1) / st_w + 1;
  size_t x_img = (size_t)H * W * C, a_img = (size_t)P * Q * K;
  auto run = [&](int n0, int n1) {
    for (int n = n0; n < n1; ++n)
      conv_acc_image(x + n * x_img, x_signed, w, bias, H, W, C, K, R, S, st_h, st_w, pad_h, pad_w,
                     dil_h, dil_w, P, Q, acc + n * a_img);
  };
  if (threads <= 1 || N == 1) {
    run(0, N);
  } else {
    if (threads > N) threads = N;
    std::vector<std::thread> pool;
    for (int t = 0; t < threads; ++t) {
      int n0 = (int)((long long)N * t / threads), n1 = (int)((long long)N * (t + 1) / threads);
      pool.emplace_back(run, n0, n1);
    }
    for (auto& th : pool) th.join();
  }
}

// ---------------------------------------------------------------------------
// Epilogue of the quantized affine layer (Eq. int8_affine / int8_affine_fused,
// the "+" rule for the fused residual, ReLU fusion of Sec. "Model Optimization"):
//   v = float(acc) * s[k]                 one fp32 multiply
//   v = v + float(res) * s_res            product rounded, then sum rounded
//   v = max(v, 0)                         if relu
//   y = clamp(Round(v), lo, hi)           y_type 0: u8 [0,255], 1: s8 [-128,127]
//   y = v                                 y_type 3: fp32 (dequantized output)
//   y = acc                               y_type 2: raw int32
// acc is [M][K]; y is written at y[m * ldc + c_off + k] so that a layer can
// write into a slice of a wider (concatenated) tensor.
// ---------------------------------------------------------------------------
void q8o_epilogue(const int32_t* acc, size_t M, int K, const float* scale, int scale_count,
                  const uint8_t* res, int res_signed, float res_scale, int relu, int y_type,
                  void* y, size_t ldc, size_t c_off) {
  for (size_t m = 0; m < M; ++m)
    for (int k = 0; k < K; ++k) {
      int32_t a = acc[m * K + k];
      size_t o = m * ldc + c_off + k;
      if (y_type == 2) { ((int32_t*)y)[o] = a; continue; }
      float v = (float)a;
      v = v * scale[scale_count == 1 ? 0 : k];
      if (res) {
        uint8_t rb = res[m * K + k];
        float rv = res_signed ? (float)(int8_t)rb : (float)rb;
        float t = rv * res_scale;
        v = v + t;
      }
      if (relu) v = v > 0.0f ? v : 0.0f;
      if (y_type == 3) { ((float*)y)[o] = v; continue; }
      float rounded = std::nearbyintf(v);
      if (y_type == 0) {
        ((uint8_t*)y)[o] = (uint8_t)(rounded < 0.0f ? 0.0f : rounded > 255.0f ? 255.0f : rounded);
      } else {
        ((int8_t*)y)[o] = (int8_t)(rounded < -128.0f ? -128.0f : rounded > 127.0f ? 127.0f : rounded);
      }
    }
}

// ---------------------------------------------------------------------------
// Channel concatenation of quantized branches under one output factor
// (reading: the shared factor is chosen by the caller, normally the max of the
// branch factors as in the "+" rule).  Each branch is re-expressed as
//   z' = clamp(Round(float(z) * s_i)),  s_i = fp32(q_i / q_out) formed in fp64,
// and copied unchanged when s_i == 1.
// ---------------------------------------------------------------------------
void q8o_concat(int n_in, const uint8_t* const* xs, const int* channels, const float* in_factors,
                float out_factor, int is_signed, size_t pixels, uint8_t* y) {
  size_t ctot = 0;
  for (int i = 0; i < n_in; ++i) ctot += channels[i];
  size_t off = 0;
  for (int i = 0; i < n_in; ++i) {
    float s = (float)((double)in_factors[i] / (double)out_factor);
    for (size_t px = 0; px < pixels; ++px)
      for (int c = 0; c < channels[i]; ++c) {
        uint8_t b = xs[i][px * channels[i] + c];
        uint8_t o;
        if (s == 1.0f) {
          o = b;
        } else {
          float v = (is_signed ? (float)(int8_t)b : (float)b) * s;
          float rounded = std::nearbyintf(v);
          if (is_signed) o = (uint8_t)(int8_t)(rounded < -128.0f ? -128.0f : rounded > 127.0f ? 127.0f : rounded);
          else o = (uint8_t)(rounded < 0.0f ? 0.0f : rounded > 255.0f ? 255.0f : rounded);
        }
        y[px * ctot + off + c] = o;
      }
    off += channels[i];
  }
}

// ---------------------------------------------------------------------------
// Pooling glue between quantized layers (the paper is silent; readings):
// max-pool takes the maximum of the in-image window cells, factor unchanged;
// avg-pool is Round(float(sum of in-image cells) * fp32(1 / (kh*kw))) with the
// full-window divisor (padding counts as zero), factor unchanged.
// `ceil_mode` rounds the output extent up and drops windows that start past
// the padded image.
// ---------------------------------------------------------------------------
static int pool_out(int H, int k, int st, int pad, int ceil_mode) {
  int num = H + 2 * pad - k;
  int o = (ceil_mode ? (num + st - 1) / st : num / st) + 1;
  if (ceil_mode && (o - 1) * st >= H + pad) --o;
  return o;
}

int q8o_pool_out(int H, int k, int st, int pad, int ceil_mode) { return pool_out(H, k, st, pad, ceil_mode); }

void q8o_pool(const uint8_t* x, int is_signed, int is_avg, int N, int H, int W, int C, int kh, int kw,
              int st_h, int st_w, int pad_h, int pad_w, int ceil_mode, uint8_t* y) {
  int P = pool_out(H, kh, st_h, pad_h, ceil_mode), Q = pool_out(W, kw, st_w, pad_w, ceil_mode);
  float inv = 1.0f / (float)(kh * kw);
  for (int n = 0; n < N; ++n)
    for (int p = 0; p < P; ++p)
      for (int q = 0; q < Q; ++q)
        for (int c = 0; c < C; ++c) {
          int32_t sum = 0, mx = is_signed ? -128 : 0;
          bool any = false;
          for (int r = 0; r < kh; ++r) {
            int h = p * st_h - pad_h + r;
            if (h < 0 || h >= H) continue;
            for (int s = 0; s < kw; ++s) {
              int w = q * st_w - pad_w + s;
              if (w < 0 || w >= W) continue;
              uint8_t b = x[(((size_t)n * H + h) * W + w) * C + c];
              int32_t v = is_signed ? (int32_t)(int8_t)b : (int32_t)b;
              sum += v;
              if (!any || v > mx) mx = v;
              any = true;
            }
          }
          int32_t o;
          if (is_avg) {
            float v = (float)sum * inv;
            float rounded = std::nearbyintf(v);
            float lo = is_signed ? -128.0f : 0.0f, hi = is_signed ? 127.0f : 255.0f;
            o = (int32_t)(rounded < lo ? lo : rounded > hi ? hi : rounded);
          } else {
            o = mx;
          }
          y[(((size_t)n * P + p) * Q + q) * C + c] = (uint8_t)o;
        }
}

int q8o_hw_threads() { return (int)std::thread::hardware_concurrency(); }

}  // extern "C"
