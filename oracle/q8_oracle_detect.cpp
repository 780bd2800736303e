// q8 oracle, SSD tail -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
//
// The paper runs SSD "with a DetectOutput layer added to calculate the mAP" (artifact appendix) and sends
// potentially negative activations through FP32 (Sec. "8-bit Low Precision Inference", calibration paragraph),
// but prints no arithmetic for either.  What follows is the published SSD definition (L2 normalisation of
// conv4_3 with a learned per-channel scale; box decoding from centre-size priors with variances; softmax
// confidences; per-class greedy non-maximum suppression; a per-image limit on kept detections) written out
// step by step, with every floating-point step one IEEE fp32 operation in a stated order, so that the CUDA
// library can be compared bit by bit.  Readings taken where the definition leaves a choice are stated at the
// function they concern.  Pins: tests/test_oracle_detect.py.
//
// Build: part of libq8_oracle.so (see build.py), -O2 -ffp-contract=off -fno-fast-math.

#include <algorithm>
#include <cmath>
#include <cstddef>
#include <cstdint>
#include <cstring>
#include <vector>

extern "C" {

// ---------------------------------------------------------------------------
// L2 normalisation across the channels of one pixel, on 8-bit codes:
//   x_c = q_x z_c,  v_c = gamma_c x_c / sqrt(sum_c x_c^2 + eps),  y_c = Q_8(v_c, q_y)
// evaluated as
//   S = sum_c z_c^2 (integer, exact),  r = 1 / sqrt(float(S) * (q_x * q_x) + eps),
//   y_c = clamp(Round((float(z_c) * m_c) * r), 0, 255)   with  m_c = gamma_c q_x / q_y  (q8o_l2norm_mult),
// five fp32 operations per pixel (one division) and two multiplies per value.  Reading: the definition divides by
// the norm; one reciprocal per pixel and a multiply per value is the same quantity to within an fp32 rounding and
// costs a tenth of a division per value.  Input codes are unsigned (the layer follows a ReLU).
// ---------------------------------------------------------------------------
float q8o_l2norm_mult(float gamma, float qx, float qy) {
  return (float)((double)gamma * (double)qx / (double)qy);  // formed in fp64, rounded once
}

void q8o_l2norm(const uint8_t* x, size_t pixels, int C, float qx, float eps, const float* mult, uint8_t* y) {
  const float qx2 = qx * qx;
  for (size_t p = 0; p < pixels; ++p) {
    const uint8_t* xp = x + p * (size_t)C;
    int64_t S = 0;
    for (int c = 0; c < C; ++c) S += (int64_t)xp[c] * xp[c];
    const float fS = (float)S;
    const float t = fS * qx2;
    const float d = std::sqrt(t + eps);
    const float rd = 1.0f / d;
    for (int c = 0; c < C; ++c) {
      const float num = (float)xp[c] * mult[c];
      const float r = std::nearbyintf(num * rd);  // 0 * inf (an all-zero pixel with eps = 0) gives NaN, which maps to 0
      y[p * (size_t)C + c] = (uint8_t)(!(r > 0.0f) ? 0.0f : (r > 255.0f ? 255.0f : r));
    }
  }
}

// ---------------------------------------------------------------------------
// exp(x) in fp32 by a fixed recipe (the library's and the C library's exponentials differ in their last bit,
// and a confidence decides which boxes survive): x is clamped to [-87, 88]; k = Round(x * log2(e));
// r = x - k ln2 in two fused steps (Cody-Waite split of ln2); exp(r) by the degree-7 Taylor polynomial in
// Horner form with fused multiply-adds (|r| <= 0.35: truncation below 6e-9); the result is p * 2^k, exact.
// Accurate to about 2 units in the last place (pinned against the C library in the tests).
// ---------------------------------------------------------------------------
float q8o_exp(float x) {
  x = x < -87.0f ? -87.0f : (x > 88.0f ? 88.0f : x);
  const float k = std::nearbyintf(x * 1.44269504088896341f);
  float r = std::fmaf(-k, 0.693145751953125f, x);          // ln2, high part (exact product for |k| < 2^11)
  r = std::fmaf(-k, 1.42860682030941723e-6f, r);           // ln2, low part
  float p = 1.0f / 5040.0f;
  p = std::fmaf(p, r, 1.0f / 720.0f);
  p = std::fmaf(p, r, 1.0f / 120.0f);
  p = std::fmaf(p, r, 1.0f / 24.0f);
  p = std::fmaf(p, r, 1.0f / 6.0f);
  p = std::fmaf(p, r, 0.5f);
  p = std::fmaf(p, r, 1.0f);
  p = std::fmaf(p, r, 1.0f);
  const int32_t bits = ((int32_t)k + 127) << 23;            // 2^k, k in [-126, 127]
  float scale;
  std::memcpy(&scale, &bits, 4);
  return p * scale;
}

// Softmax over the classes of one box: e_c = exp(x_c - max_c x), p_c = e_c / sum_c e_c, the sum taken in class
// order, each step one fp32 operation.
void q8o_softmax(const float* conf, size_t boxes, int classes, float* prob) {
  for (size_t b = 0; b < boxes; ++b) {
    const float* x = conf + b * (size_t)classes;
    float m = x[0];
    for (int c = 1; c < classes; ++c) m = x[c] > m ? x[c] : m;
    float sum = 0.0f;
    for (int c = 0; c < classes; ++c) {
      const float e = q8o_exp(x[c] - m);
      prob[b * (size_t)classes + c] = e;
      sum = sum + e;
    }
    for (int c = 0; c < classes; ++c) prob[b * (size_t)classes + c] = prob[b * (size_t)classes + c] / sum;
  }
}

// ---------------------------------------------------------------------------
// Box decoding (centre-size code, variances applied to the regression output):
//   cx = (v0 * l0) * pw + pcx,  cy = (v1 * l1) * ph + pcy,  w = exp(v2 * l2) * pw,  h = exp(v3 * l3) * ph,
//   box = (cx - w/2, cy - h/2, cx + w/2, cy + h/2)      (halves as one multiply by 0.5; no clipping).
// priors: [P][4] as (pcx, pcy, pw, ph); loc: [N][P][4]; boxes: [N][P][4] as (xmin, ymin, xmax, ymax).
// ---------------------------------------------------------------------------
void q8o_decode_boxes(const float* loc, const float* priors, const float* var, int N, int P, float* boxes) {
  for (int n = 0; n < N; ++n)
    for (int p = 0; p < P; ++p) {
      const float* l = loc + ((size_t)n * P + p) * 4;
      const float* pr = priors + (size_t)p * 4;
      const float cx = (var[0] * l[0]) * pr[2] + pr[0];
      const float cy = (var[1] * l[1]) * pr[3] + pr[1];
      const float w = q8o_exp(var[2] * l[2]) * pr[2];
      const float h = q8o_exp(var[3] * l[3]) * pr[3];
      const float hw = w * 0.5f, hh = h * 0.5f;
      float* b = boxes + ((size_t)n * P + p) * 4;
      b[0] = cx - hw; b[1] = cy - hh; b[2] = cx + hw; b[3] = cy + hh;
    }
}

// Jaccard overlap of two corner boxes: intersection over union, 0 when they do not intersect.
float q8o_iou(const float* a, const float* b) {
  const float ix0 = a[0] > b[0] ? a[0] : b[0], iy0 = a[1] > b[1] ? a[1] : b[1];
  const float ix1 = a[2] < b[2] ? a[2] : b[2], iy1 = a[3] < b[3] ? a[3] : b[3];
  const float iw = ix1 - ix0, ih = iy1 - iy0;
  if (!(iw > 0.0f) || !(ih > 0.0f)) return 0.0f;
  const float inter = iw * ih;
  const float area_a = (a[2] - a[0]) * (a[3] - a[1]), area_b = (b[2] - b[0]) * (b[3] - b[1]);
  return inter / ((area_a + area_b) - inter);
}

// ---------------------------------------------------------------------------
// Detection output for a batch.  Per image and per class other than `background`:
//   1. candidates: boxes whose class probability exceeds conf_thresh, ordered by probability, highest first
//      (equal probabilities: lower box index first), cut to the first nms_top_k;
//   2. greedy suppression in that order: a candidate is kept unless its overlap with an already kept box of the
//      same class exceeds nms_thresh.
// Per image, all kept (class, box) pairs are ordered by probability, highest first (ties: lower class, then lower
// box index) and cut to keep_top_k.  Row i of the image's output: (class, probability, xmin, ymin, xmax, ymax);
// counts[n] rows are valid.  out: [N][keep_top_k][6], rows beyond the count are zero.
// Reading: the output order is the selection order (the definition's own order, by class, is a permutation of it).
// ---------------------------------------------------------------------------
void q8o_detection_output(const float* loc, const float* conf, const float* priors, const float* var, int N, int P,
                          int classes, int background, float conf_thresh, float nms_thresh, int nms_top_k,
                          int keep_top_k, float* out, int32_t* counts) {
  std::vector<float> boxes((size_t)N * P * 4), prob((size_t)N * P * classes);
  q8o_decode_boxes(loc, priors, var, N, P, boxes.data());
  q8o_softmax(conf, (size_t)N * P, classes, prob.data());
  struct Det { float score; int cls; int box; };
  for (int n = 0; n < N; ++n) {
    std::vector<Det> kept_all;
    const float* bx = boxes.data() + (size_t)n * P * 4;
    for (int c = 0; c < classes; ++c) {
      if (c == background) continue;
      std::vector<Det> cand;
      for (int p = 0; p < P; ++p) {
        const float s = prob[((size_t)n * P + p) * classes + c];
        if (s > conf_thresh) cand.push_back({s, c, p});
      }
      std::sort(cand.begin(), cand.end(), [](const Det& a, const Det& b) { return a.score != b.score ? a.score > b.score : a.box < b.box; });
      if ((int)cand.size() > nms_top_k) cand.resize(nms_top_k);
      std::vector<Det> kept;
      for (const Det& d : cand) {
        bool keep = true;
        for (const Det& k : kept)
          if (q8o_iou(bx + (size_t)d.box * 4, bx + (size_t)k.box * 4) > nms_thresh) { keep = false; break; }
        if (keep) kept.push_back(d);
      }
      kept_all.insert(kept_all.end(), kept.begin(), kept.end());
    }
    std::sort(kept_all.begin(), kept_all.end(), [](const Det& a, const Det& b) {
      if (a.score != b.score) return a.score > b.score;
      if (a.cls != b.cls) return a.cls < b.cls;
      return a.box < b.box;
    });
    if ((int)kept_all.size() > keep_top_k) kept_all.resize(keep_top_k);
    counts[n] = (int32_t)kept_all.size();
    float* o = out + (size_t)n * keep_top_k * 6;
    std::memset(o, 0, sizeof(float) * (size_t)keep_top_k * 6);
    for (size_t i = 0; i < kept_all.size(); ++i) {
      const Det& d = kept_all[i];
      o[i * 6] = (float)d.cls; o[i * 6 + 1] = d.score;
      for (int j = 0; j < 4; ++j) o[i * 6 + 2 + j] = bx[(size_t)d.box * 4 + j];
    }
  }
}

// ---------------------------------------------------------------------------
// The FP32 route the paper takes for potentially negative activations, for a residual block whose shortcut is a
// convolution without ReLU: both summands arrive as FP32 (dequantized convolution outputs), the sum and the ReLU
// are FP32, and the result is quantized for the next 8-bit convolution:
//   y = Q_8(max(a + b, 0), q_y)      (one fp32 add, one fp32 division, Round half to even, clamp to [0, 255]).
// ---------------------------------------------------------------------------
void q8o_add_relu_quantize(const float* a, const float* b, size_t n, float qy, uint8_t* y) {
  for (size_t i = 0; i < n; ++i) {
    float v = a[i] + b[i];
    v = v > 0.0f ? v : 0.0f;
    const float r = std::nearbyintf(v / qy);
    y[i] = (uint8_t)(r > 255.0f ? 255.0f : r);
  }
}

}  // extern "C"
