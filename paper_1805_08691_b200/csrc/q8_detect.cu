// The SSD tail of the 8-bit path and the FP32 route for signed residual sums.
//
// The paper runs SSD with a detection-output layer (artifact appendix) and sends potentially negative activations
// through FP32 (Sec. "8-bit Low Precision Inference", calibration paragraph) without printing arithmetic for either;
// the kernels below follow the detector's published definition, every floating-point step one IEEE fp32 operation
// in a fixed order (the library is built without contraction; fused steps are written as fused):
//   * L2 normalisation across channels on 8-bit codes (one warp per pixel, integer sum of squares by dp4a);
//   * Q_8(max(a + b, 0), q): the FP32 sum, ReLU and re-quantization of two dequantized convolution outputs;
//   * detection output: box decoding and softmax (one thread per box), per (image, class) candidate selection by a
//     bitonic sort in shared memory and greedy suppression over a bit matrix of overlaps, per-image selection of
//     the best detections.
#include <atomic>
#include <cfloat>
#include <cmath>

#include "q8_internal.h"

namespace q8 {
namespace {

// ------------------------------------------------------------------------------------------ L2 normalisation
//   S = sum_c z_c^2,  r = 1 / sqrt(float(S) * (q_x * q_x) + eps),  y_c = clamp(Round((float(z_c) * m_c) * r), 0, 255)
__device__ __forceinline__ unsigned int l2_word(unsigned int w, const float4 m, float r) {
  // byte -> float without a conversion instruction: 0x4B0000bb is 2^23 + b exactly
  const float f0 = __fsub_rn(__uint_as_float(__byte_perm(w, 0x4B000000u, 0x7540u)), 8388608.0f);
  const float f1 = __fsub_rn(__uint_as_float(__byte_perm(w, 0x4B000000u, 0x7541u)), 8388608.0f);
  const float f2 = __fsub_rn(__uint_as_float(__byte_perm(w, 0x4B000000u, 0x7542u)), 8388608.0f);
  const float f3 = __fsub_rn(__uint_as_float(__byte_perm(w, 0x4B000000u, 0x7543u)), 8388608.0f);
  const float v0 = __fmul_rn(__fmul_rn(f0, m.x), r), v1 = __fmul_rn(__fmul_rn(f1, m.y), r);
  const float v2 = __fmul_rn(__fmul_rn(f2, m.z), r), v3 = __fmul_rn(__fmul_rn(f3, m.w), r);
  unsigned int b0, b1, b2, b3;
  asm("cvt.rni.sat.u8.f32 %0, %1;" : "=r"(b0) : "f"(v0));
  asm("cvt.rni.sat.u8.f32 %0, %1;" : "=r"(b1) : "f"(v1));
  asm("cvt.rni.sat.u8.f32 %0, %1;" : "=r"(b2) : "f"(v2));
  asm("cvt.rni.sat.u8.f32 %0, %1;" : "=r"(b3) : "f"(v3));
  return __byte_perm(__byte_perm(b0, b1, 0x0040u), __byte_perm(b2, b3, 0x0040u), 0x5410u);
}

__device__ __forceinline__ float l2_recip(unsigned int s, float qx2, float eps) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  return __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(__fmul_rn((float)s, qx2), eps)));
}

// A warp takes two pixels per step (all loads of both are issued before the first sum is reduced), C a multiple of
// 4 and rows 4-byte aligned: a lane takes words lane, lane + 32, ... of each pixel, kept in registers (kL2Words
// words per lane: up to 512 channels; wider rows take the kernel below).
constexpr int kL2Words = 4;
__global__ void __launch_bounds__(256) l2norm_kernel(const unsigned int* __restrict__ x, size_t pixels, int cw, float qx2,
                                                     float eps, const float4* __restrict__ mult, unsigned int* __restrict__ y) {
  const int lane = threadIdx.x & 31;
  const size_t warp = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = ((size_t)gridDim.x * blockDim.x) >> 5;
  float4 m[kL2Words];
#pragma unroll
  for (int j = 0; j < kL2Words; ++j) m[j] = lane + 32 * j < cw ? __ldg(mult + lane + 32 * j) : make_float4(0.f, 0.f, 0.f, 0.f);
  for (size_t p = 2 * warp; p < pixels; p += 2 * nwarps) {
    const bool two = p + 1 < pixels;
    const unsigned int* row0 = x + p * (size_t)cw;
    const unsigned int* row1 = row0 + (two ? cw : 0);
    unsigned int w0[kL2Words], w1[kL2Words];
#pragma unroll
    for (int j = 0; j < kL2Words; ++j) {
      const int i = lane + 32 * j;
      w0[j] = i < cw ? __ldcs(row0 + i) : 0u;
      w1[j] = i < cw ? __ldcs(row1 + i) : 0u;
    }
    unsigned int s0 = 0, s1 = 0;  // at most 2048 channels of 255^2: far below 2^32
#pragma unroll
    for (int j = 0; j < kL2Words; ++j) { s0 = __dp4a(w0[j], w0[j], s0); s1 = __dp4a(w1[j], w1[j], s1); }
    const float r0 = l2_recip(s0, qx2, eps), r1 = l2_recip(s1, qx2, eps);
    unsigned int* out0 = y + p * (size_t)cw;
#pragma unroll
    for (int j = 0; j < kL2Words; ++j) {
      const int i = lane + 32 * j;
      if (i < cw) {
        __stcs(out0 + i, l2_word(w0[j], m[j], r0));
        if (two) __stcs(out0 + cw + i, l2_word(w1[j], m[j], r1));
      }
    }
  }
}

// Rows wider than the registers of the kernel above hold (C % 4 == 0): one warp per pixel, the row is read twice.
__global__ void __launch_bounds__(256) l2norm_wide_kernel(const unsigned int* __restrict__ x, size_t pixels, int cw, float qx2,
                                                          float eps, const float4* __restrict__ mult, unsigned int* __restrict__ y) {
  const int lane = threadIdx.x & 31;
  const size_t warp = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = ((size_t)gridDim.x * blockDim.x) >> 5;
  for (size_t p = warp; p < pixels; p += nwarps) {
    const unsigned int* row = x + p * (size_t)cw;
    unsigned int s = 0;  // at most 65536 channels of 255^2: below 2^32
    for (int i = lane; i < cw; i += 32) {
      const unsigned int v = __ldg(row + i);
      s = __dp4a(v, v, s);
    }
    const float r = l2_recip(s, qx2, eps);
    unsigned int* out = y + p * (size_t)cw;
    for (int i = lane; i < cw; i += 32) out[i] = l2_word(__ldg(row + i), __ldg(mult + i), r);
  }
}

// any C: one thread per pixel
__global__ void __launch_bounds__(256) l2norm_scalar_kernel(const unsigned char* __restrict__ x, size_t pixels, int C, float qx2,
                                                            float eps, const float* __restrict__ mult, unsigned char* __restrict__ y) {
  const size_t n = (size_t)gridDim.x * blockDim.x;
  for (size_t p = (size_t)blockIdx.x * blockDim.x + threadIdx.x; p < pixels; p += n) {
    const unsigned char* row = x + p * (size_t)C;
    unsigned long long s = 0;
    for (int c = 0; c < C; ++c) s += (unsigned int)row[c] * (unsigned int)row[c];
    const float r = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(__fmul_rn((float)s, qx2), eps)));
    for (int c = 0; c < C; ++c) {
      unsigned int b;
      asm("cvt.rni.sat.u8.f32 %0, %1;" : "=r"(b) : "f"(__fmul_rn(__fmul_rn((float)row[c], mult[c]), r)));
      y[p * (size_t)C + c] = (unsigned char)b;
    }
  }
}

// ------------------------------------------------------------------------------------------ FP32 route of a sum
// y = clamp(Round(max(a + b, 0) / q), 0, 255): 32 bytes of fp32 in, 4 bytes out per thread and step.
__device__ __forceinline__ unsigned int arq1(float a, float b, float q) {
  unsigned int r;
  asm("cvt.rni.sat.u8.f32 %0, %1;" : "=r"(r) : "f"(__fdiv_rn(fmaxf(__fadd_rn(a, b), 0.0f), q)));
  return r;
}
__global__ void __launch_bounds__(512) add_relu_quantize_kernel(const float4* __restrict__ a, const float4* __restrict__ b, size_t n4,
                                                                float q, unsigned int* __restrict__ y) {
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  for (; i + nthreads < n4; i += 2 * nthreads) {
    const float4 a0 = __ldcs(a + i), b0 = __ldcs(b + i), a1 = __ldcs(a + i + nthreads), b1 = __ldcs(b + i + nthreads);
    y[i] = arq1(a0.x, b0.x, q) | (arq1(a0.y, b0.y, q) << 8) | (arq1(a0.z, b0.z, q) << 16) | (arq1(a0.w, b0.w, q) << 24);
    y[i + nthreads] = arq1(a1.x, b1.x, q) | (arq1(a1.y, b1.y, q) << 8) | (arq1(a1.z, b1.z, q) << 16) | (arq1(a1.w, b1.w, q) << 24);
  }
  for (; i < n4; i += nthreads) {
    const float4 a0 = __ldcs(a + i), b0 = __ldcs(b + i);
    y[i] = arq1(a0.x, b0.x, q) | (arq1(a0.y, b0.y, q) << 8) | (arq1(a0.z, b0.z, q) << 16) | (arq1(a0.w, b0.w, q) << 24);
  }
}
__global__ void __launch_bounds__(256) add_relu_quantize_tail_kernel(const float* __restrict__ a, const float* __restrict__ b,
                                                                     size_t first, size_t n, float q, unsigned char* __restrict__ y) {
  const size_t i = first + (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) y[i] = (unsigned char)arq1(a[i], b[i], q);
}

// ------------------------------------------------------------------------------------------ detection output
// exp(x) by a fixed recipe, so that a confidence has the same bits wherever it is computed: clamp to [-87, 88],
// k = Round(x log2 e), r = x - k ln2 in two fused steps, degree-7 Taylor polynomial by fused Horner steps, times 2^k.
__device__ __forceinline__ float exp_fixed(float x) {
  x = x < -87.0f ? -87.0f : (x > 88.0f ? 88.0f : x);
  const float k = rintf(__fmul_rn(x, 1.44269504088896341f));
  float r = __fmaf_rn(-k, 0.693145751953125f, x);
  r = __fmaf_rn(-k, 1.42860682030941723e-6f, r);
  float p = 1.0f / 5040.0f;
  p = __fmaf_rn(p, r, 1.0f / 720.0f);
  p = __fmaf_rn(p, r, 1.0f / 120.0f);
  p = __fmaf_rn(p, r, 1.0f / 24.0f);
  p = __fmaf_rn(p, r, 1.0f / 6.0f);
  p = __fmaf_rn(p, r, 0.5f);
  p = __fmaf_rn(p, r, 1.0f);
  p = __fmaf_rn(p, r, 1.0f);
  return __fmul_rn(p, __int_as_float(((int)k + 127) << 23));
}

constexpr int kMaxSources = 8;
constexpr int kRegClasses = 24;   // class counts up to this keep a box's logits in registers
struct DetSources {
  const float* loc[kMaxSources];
  const float* conf[kMaxSources];
  int loc_stride[kMaxSources], conf_stride[kMaxSources];  // floats between consecutive cells
  int cells[kMaxSources], boxes[kMaxSources];              // cells per image, boxes per cell
  int first[kMaxSources + 1];                              // first prior of each source
  int n;
};

// One thread per (image, prior): decoded corner box and the softmax of its class logits.
//   cx = (v0 l0) pw + pcx, cy = (v1 l1) ph + pcy, w = exp(v2 l2) pw, h = exp(v3 l3) ph, corners = centre -+ half
//   e_c = exp(x_c - max x), p_c = e_c / sum_c e_c (sum in class order)
// boxes: [N][P] float4; prob: [N][classes][P] (class-major, for the per-class pass).
__global__ void __launch_bounds__(256) decode_softmax_kernel(const __grid_constant__ DetSources src, const float4* __restrict__ priors,
                                                             float v0, float v1, float v2, float v3, int N, int P, int classes,
                                                             float4* __restrict__ boxes, float* __restrict__ prob) {
  const size_t total = (size_t)N * P;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int n = (int)(i / P), p = (int)(i - (size_t)n * P);
    int s = 0;
#pragma unroll
    for (int j = 1; j < kMaxSources; ++j)
      if (j < src.n && p >= src.first[j]) s = j;
    const int local = p - src.first[s];
    const int cell = local / src.boxes[s], b = local - cell * src.boxes[s];
    const size_t pix = (size_t)n * src.cells[s] + cell;
    const float* l = src.loc[s] + pix * src.loc_stride[s] + b * 4;
    const float* x = src.conf[s] + pix * src.conf_stride[s] + (size_t)b * classes;
    const float4 pr = __ldg(priors + p);
    const float cx = __fadd_rn(__fmul_rn(__fmul_rn(v0, l[0]), pr.z), pr.x);
    const float cy = __fadd_rn(__fmul_rn(__fmul_rn(v1, l[1]), pr.w), pr.y);
    const float w = __fmul_rn(exp_fixed(__fmul_rn(v2, l[2])), pr.z);
    const float h = __fmul_rn(exp_fixed(__fmul_rn(v3, l[3])), pr.w);
    const float hw = __fmul_rn(w, 0.5f), hh = __fmul_rn(h, 0.5f);
    boxes[i] = make_float4(__fsub_rn(cx, hw), __fsub_rn(cy, hh), __fadd_rn(cx, hw), __fadd_rn(cy, hh));
    float* pr_out = prob + (size_t)n * classes * P + p;
    if (classes <= kRegClasses) {
      // the logits and then the exponentials stay in registers: one exponential per class instead of two
      float e[kRegClasses];
#pragma unroll
      for (int c = 0; c < kRegClasses; ++c) e[c] = c < classes ? x[c] : -FLT_MAX;
      float m = e[0];
#pragma unroll
      for (int c = 1; c < kRegClasses; ++c) m = (c < classes && e[c] > m) ? e[c] : m;
      float sum = 0.0f;
#pragma unroll
      for (int c = 0; c < kRegClasses; ++c)
        if (c < classes) {
          e[c] = exp_fixed(__fsub_rn(e[c], m));
          sum = __fadd_rn(sum, e[c]);
        }
#pragma unroll
      for (int c = 0; c < kRegClasses; ++c)
        if (c < classes) pr_out[(size_t)c * P] = __fdiv_rn(e[c], sum);
    } else {
      float m = x[0];
      for (int c = 1; c < classes; ++c) m = x[c] > m ? x[c] : m;
      float sum = 0.0f;
      for (int c = 0; c < classes; ++c) sum = __fadd_rn(sum, exp_fixed(__fsub_rn(x[c], m)));
      for (int c = 0; c < classes; ++c) pr_out[(size_t)c * P] = __fdiv_rn(exp_fixed(__fsub_rn(x[c], m)), sum);
    }
  }
}

// Ascending bitonic sort of n (a power of two) 64-bit keys in shared memory by the whole block.
__device__ void bitonic_sort(unsigned long long* keys, int n) {
  for (int k = 2; k <= n; k <<= 1)
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const int ixj = i ^ j;
        if (ixj > i) {
          const unsigned long long a = keys[i], b = keys[ixj];
          if ((a > b) == ((i & k) == 0)) { keys[i] = b; keys[ixj] = a; }
        }
      }
      __syncthreads();
    }
}

// Overlap of two corner boxes (intersection over union; 0 when they do not intersect).
__device__ __forceinline__ float iou(const float4 a, const float4 b) {
  const float ix0 = a.x > b.x ? a.x : b.x, iy0 = a.y > b.y ? a.y : b.y;
  const float ix1 = a.z < b.z ? a.z : b.z, iy1 = a.w < b.w ? a.w : b.w;
  const float iw = __fsub_rn(ix1, ix0), ih = __fsub_rn(iy1, iy0);
  if (!(iw > 0.0f) || !(ih > 0.0f)) return 0.0f;
  const float inter = __fmul_rn(iw, ih);
  const float area_a = __fmul_rn(__fsub_rn(a.z, a.x), __fsub_rn(a.w, a.y)), area_b = __fmul_rn(__fsub_rn(b.z, b.x), __fsub_rn(b.w, b.y));
  return __fdiv_rn(inter, __fsub_rn(__fadd_rn(area_a, area_b), inter));
}

constexpr int kNmsThreads = 512;     // per (image, class) block
constexpr int kTopThreads = 1024;    // per image block
constexpr int kMaxTopK = 512;        // candidates that enter the suppression of one class
constexpr int kMaxSort = 16384;      // boxes per image; keys the per-image block sorts in shared memory
constexpr int kSelBits = 11;         // key bits per histogram pass of the pre-selection
constexpr int kSelBins = 1 << kSelBits;
constexpr int kSelCap = 2048;        // keys handed to the per-class sort

// Warp 0 only: the first bin at which the running sum of hist reaches `need` (need <= the total), and the sum of
// the bins before it.
__device__ int select_bin(const int* hist, int need, int* below) {
  const int lane = threadIdx.x & 31;
  constexpr int kPer = kSelBins / 32;
  int local = 0;
  for (int j = 0; j < kPer; ++j) local += hist[lane * kPer + j];
  int incl = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  const unsigned int reached = __ballot_sync(0xffffffffu, incl >= need);
  const int src = reached ? __ffs(reached) - 1 : 31;
  int bin = 0, bel = 0;
  if (lane == src) {
    int cum = incl - local, j = 0;
    for (; j < kPer - 1; ++j) {
      const int h = hist[lane * kPer + j];
      if (cum + h >= need) break;
      cum += h;
    }
    bin = lane * kPer + j;
    bel = cum;
  }
  *below = __shfl_sync(0xffffffffu, bel, src);
  return __shfl_sync(0xffffffffu, bin, src);
}

__device__ __forceinline__ unsigned long long nms_key(float s, int p) {
  return ((unsigned long long)(~__float_as_uint(s)) << 32) | (unsigned int)p;
}

// One block per (image, class other than background).  Keys order candidates (probability > conf_thresh) by
// probability, highest first, then by box index: (~bits of the positive probability) << 32 | box; they are unique.
// Only the best top_k can matter.  The probabilities of the class (P floats, L2 resident) are read once per pass: the
// first pass counts the candidates and fills a histogram of the leading kSelBits key bits; up to kSelCap candidates
// are simply collected, more are narrowed by a radix selection (per pass: the bin in which the running count
// reaches top_k; keys below it are in, keys in it go to the next pass over the next bits) until the keys at or below
// the chosen prefix number at most kSelCap; with unique keys that ends at the latest when all 64 bits are fixed.
// The collected keys are sorted (bitonic, shared memory), the best top_k and their boxes copied out, their overlaps
// written as a bit matrix (over the sort area) and one warp walks the candidates in order.
__global__ void __launch_bounds__(kNmsThreads) nms_class_kernel(const float4* __restrict__ boxes, const float* __restrict__ prob, int P,
                                                                int classes, int background, float conf_thresh, float nms_thresh,
                                                                int top_k, unsigned int work_bytes,
                                                                unsigned long long* __restrict__ kept_keys,
                                                                int* __restrict__ kept_count) {
  // work_bytes: room for kSelCap keys and for top_k rows of the overlap matrix, whichever is larger
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned long long* work = reinterpret_cast<unsigned long long*>(smem_raw);
  unsigned long long* top = reinterpret_cast<unsigned long long*>(smem_raw + work_bytes);
  float4* tbox = reinterpret_cast<float4*>(top + kMaxTopK);
  int* hist = reinterpret_cast<int*>(tbox + kMaxTopK);
  unsigned int* mask = reinterpret_cast<unsigned int*>(smem_raw);
  __shared__ int cnt, sel_bin, sel_below, sel_in_bin, sel_cnt;
  const int n = blockIdx.y;
  int c = blockIdx.x;
  if (background >= 0 && c >= background) ++c;  // blockIdx.x runs over the foreground classes
  if (threadIdx.x == 0) { cnt = 0; sel_cnt = 0; }
  for (int i = threadIdx.x; i < kSelBins; i += blockDim.x) hist[i] = 0;
  __syncthreads();
  const float* sc = prob + ((size_t)n * classes + c) * P;
  for (int p0 = threadIdx.x; p0 < P; p0 += 4 * blockDim.x) {
    float s[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) s[u] = p0 + u * blockDim.x < P ? sc[p0 + u * blockDim.x] : -1.0f;
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (s[u] > conf_thresh) {
        atomicAdd(&cnt, 1);
        atomicAdd(&hist[nms_key(s[u], 0) >> (64 - kSelBits)], 1);
      }
  }
  __syncthreads();
  int m = cnt;
  int shift = 64;                    // keys with (key >> shift) <= limit are collected; 64: all candidates
  unsigned long long limit = 0;
  if (m > kSelCap) {                 // (the whole block takes this branch or none of it does)
    int need = top_k, accepted = 0;  // accepted: keys below the prefix chosen so far
    int width = kSelBits;            // bits of the digit the histogram holds
    shift = 64 - kSelBits;
    for (;;) {
      if (threadIdx.x < 32) {
        int below;
        const int b = select_bin(hist, need, &below);
        if (threadIdx.x == 0) { sel_bin = b; sel_below = below; sel_in_bin = hist[b]; }
      }
      __syncthreads();
      limit = (limit << width) | (unsigned int)sel_bin;
      accepted += sel_below;
      need -= sel_below;
      m = accepted + sel_in_bin;
      if (m <= kSelCap || shift == 0) break;
      const int ns = shift >= kSelBits ? shift - kSelBits : 0;
      width = shift - ns;
      const unsigned int dmask = (1u << width) - 1u;
      for (int i = threadIdx.x; i < kSelBins; i += blockDim.x) hist[i] = 0;
      __syncthreads();
      for (int p = threadIdx.x; p < P; p += blockDim.x) {
        const float s = sc[p];
        if (s > conf_thresh) {
          const unsigned long long key = nms_key(s, p);
          if ((key >> shift) == limit) atomicAdd(&hist[(unsigned int)(key >> ns) & dmask], 1);
        }
      }
      __syncthreads();
      shift = ns;
    }
  }
  for (int p = threadIdx.x; p < P; p += blockDim.x) {
    const float s = sc[p];
    if (s > conf_thresh) {
      const unsigned long long key = nms_key(s, p);
      if (shift == 64 || (key >> shift) <= limit) work[atomicAdd(&sel_cnt, 1)] = key;
    }
  }
  int size = 1;
  while (size < m) size <<= 1;
  __syncthreads();
  for (int i = m + threadIdx.x; i < size; i += blockDim.x) work[i] = ~0ull;
  __syncthreads();
  bitonic_sort(work, size);
  const int k = m < top_k ? m : top_k;
  const float4* bx = boxes + (size_t)n * P;
  for (int i = threadIdx.x; i < k; i += blockDim.x) {
    top[i] = work[i];
    tbox[i] = bx[(unsigned int)work[i]];
  }
  __syncthreads();
  const int W = (k + 31) >> 5;
  for (int item = threadIdx.x; item < k * W; item += blockDim.x) {
    const int i = item / W, w = item - i * W;
    unsigned int bits = 0;
    const float4 bi = tbox[i];
    for (int b = 0; b < 32; ++b) {
      const int j = w * 32 + b;
      if (j > i && j < k && iou(tbox[j], bi) > nms_thresh) bits |= 1u << b;
    }
    mask[item] = bits;
  }
  __syncthreads();
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    unsigned int removed = 0;  // lane l holds word l of the removed set (W <= 16)
    int nk = 0;
    unsigned long long* out = kept_keys + ((size_t)n * classes + c) * top_k;
    for (int i = 0; i < k; ++i) {
      const unsigned int word = __shfl_sync(0xffffffffu, removed, i >> 5);
      if (!((word >> (i & 31)) & 1u)) {
        if (lane < W) removed |= mask[i * W + lane];
        if (lane == 0) out[nk] = top[i];
        ++nk;
      }
    }
    if (lane == 0) kept_count[n * classes + c] = nk;
  }
}

// One block per image: the kept detections of all classes ordered by probability (ties: class, then box), the first
// keep_top_k written as rows (class, probability, xmin, ymin, xmax, ymax); unused rows are zero.
__global__ void __launch_bounds__(kTopThreads) keep_top_kernel(const float4* __restrict__ boxes, const unsigned long long* __restrict__ kept_keys,
                                                               const int* __restrict__ kept_count, int P, int classes, int background,
                                                               int top_k, int keep_top_k, float* __restrict__ out,
                                                               int* __restrict__ counts) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(smem_raw);
  const int n = blockIdx.x;
  int m = 0;  // every thread walks the class counts itself: no shared counter, no barrier per class
  for (int c = 0; c < classes; ++c) {
    if (c == background) continue;
    const int kc = kept_count[n * classes + c];
    const unsigned long long* kk = kept_keys + ((size_t)n * classes + c) * top_k;
    for (int i = threadIdx.x; i < kc; i += blockDim.x) {
      const unsigned long long key = kk[i];
      keys[m + i] = (key & 0xffffffff00000000ull) | ((unsigned long long)c << 16) | (key & 0xffffull);
    }
    m += kc;
  }
  int size = 1;
  while (size < m) size <<= 1;
  for (int i = m + threadIdx.x; i < size; i += blockDim.x) keys[i] = ~0ull;
  __syncthreads();
  bitonic_sort(keys, size);
  const int k = m < keep_top_k ? m : keep_top_k;
  float* o = out + (size_t)n * keep_top_k * 6;
  for (int i = threadIdx.x; i < keep_top_k; i += blockDim.x) {
    float row[6] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (i < k) {
      const unsigned long long key = keys[i];
      const float4 b = boxes[(size_t)n * P + (unsigned int)(key & 0xffffull)];
      row[0] = (float)(unsigned int)((key >> 16) & 0xffffull);
      row[1] = __uint_as_float(~(unsigned int)(key >> 32));
      row[2] = b.x; row[3] = b.y; row[4] = b.z; row[5] = b.w;
    }
#pragma unroll
    for (int j = 0; j < 6; ++j) o[i * 6 + j] = row[j];
  }
  if (threadIdx.x == 0) counts[n] = k;
}

size_t align256(size_t v) { return (v + 255) / 256 * 256; }
struct DetLayout { size_t boxes, prob, keys, counts, total; };
DetLayout det_layout(int N, int P, int classes, int top_k) {
  DetLayout L;
  L.boxes = 0;
  L.prob = align256((size_t)N * P * 16);
  L.keys = L.prob + align256((size_t)N * classes * P * 4);
  L.counts = L.keys + align256((size_t)N * classes * top_k * 8);
  L.total = L.counts + align256((size_t)N * classes * 4);
  return L;
}

}  // namespace
}  // namespace q8

using namespace q8;

extern "C" {

int q8_l2norm(const void* x, size_t pixels, int C, float qx, float eps, const float* d_mult, void* y, void* stream) {
  clear_error();
  if ((!x || !y || !d_mult) && pixels) return fail(Q8_ERR_INVALID_ARG, "q8_l2norm: null pointer");
  if (C <= 0 || C > 65536) return fail(Q8_ERR_INVALID_ARG, "q8_l2norm: need 0 < C <= 65536");
  if (!(qx > 0.f) || std::isinf(qx) || !(eps >= 0.f) || std::isinf(eps)) return fail(Q8_ERR_NONFINITE, "q8_l2norm: factor must be finite positive, eps finite and >= 0");
  if (pixels == 0) return Q8_OK;
  volatile float qx2 = qx * qx;  // one fp32 multiply
  cudaStream_t s = as_stream(stream);
  const bool vec = C % 4 == 0 && (reinterpret_cast<uintptr_t>(x) & 3u) == 0 && (reinterpret_cast<uintptr_t>(y) & 3u) == 0 && aligned16(d_mult);
  if (vec) {
    const size_t cap = (size_t)sm_count() * 8;
    if (C / 4 <= 32 * kL2Words) {
      const size_t blocks = (pixels + 15) / 16;  // eight warps of two pixels per block and step
      l2norm_kernel<<<(unsigned)(blocks < cap ? blocks : cap), 256, 0, s>>>(static_cast<const unsigned int*>(x), pixels, C / 4, qx2, eps,
                                                                              reinterpret_cast<const float4*>(d_mult), static_cast<unsigned int*>(y));
      return check_launch("l2norm_kernel");
    }
    const size_t blocks = (pixels + 7) / 8;
    l2norm_wide_kernel<<<(unsigned)(blocks < cap ? blocks : cap), 256, 0, s>>>(static_cast<const unsigned int*>(x), pixels, C / 4, qx2, eps,
                                                                                 reinterpret_cast<const float4*>(d_mult), static_cast<unsigned int*>(y));
    return check_launch("l2norm_wide_kernel");
  }
  const size_t blocks = (pixels + 255) / 256, cap = (size_t)sm_count() * 8;
  l2norm_scalar_kernel<<<(unsigned)(blocks < cap ? blocks : cap), 256, 0, s>>>(static_cast<const unsigned char*>(x), pixels, C, qx2, eps, d_mult,
                                                                                 static_cast<unsigned char*>(y));
  return check_launch("l2norm_scalar_kernel");
}

int q8_add_relu_quantize(const float* a, const float* b, size_t n, float q, void* y, void* stream) {
  clear_error();
  if ((!a || !b || !y) && n) return fail(Q8_ERR_INVALID_ARG, "q8_add_relu_quantize: null pointer");
  if (!(q > 0.f) || std::isinf(q)) return fail(Q8_ERR_NONFINITE, "q8_add_relu_quantize: factor must be finite and positive");
  if (n == 0) return Q8_OK;
  cudaStream_t s = as_stream(stream);
  size_t done = 0;
  if (aligned16(a) && aligned16(b) && (reinterpret_cast<uintptr_t>(y) & 3u) == 0 && n >= 4) {
    const size_t n4 = n / 4, blocks = (n4 + 511) / 512, cap = (size_t)sm_count() * 4;
    add_relu_quantize_kernel<<<(unsigned)(blocks < cap ? blocks : cap), 512, 0, s>>>(reinterpret_cast<const float4*>(a), reinterpret_cast<const float4*>(b),
                                                                                        n4, q, static_cast<unsigned int*>(y));
    done = n4 * 4;
  }
  if (done < n) {
    const size_t rest = n - done;
    if (rest > 0x7fffffffu * 256ull) return fail(Q8_ERR_UNSUPPORTED, "q8_add_relu_quantize: unaligned tensors above 2^39 elements");
    add_relu_quantize_tail_kernel<<<(unsigned)((rest + 255) / 256), 256, 0, s>>>(a, b, done, n, q, static_cast<unsigned char*>(y));
  }
  return check_launch("add_relu_quantize_kernel");
}

static int det_check(int N, int P, int classes, int background, int nms_top_k, int keep_top_k) {
  if (N <= 0 || P <= 0 || classes <= 0 || nms_top_k <= 0 || keep_top_k <= 0 || background < -1 || background >= classes)
    return fail(Q8_ERR_INVALID_ARG, "q8_detection_output: bad extent or class index");
  const int fg = classes - (background >= 0 ? 1 : 0);
  if (fg <= 0) return fail(Q8_ERR_INVALID_ARG, "q8_detection_output: no foreground class");
  if (P > kMaxSort || nms_top_k > kMaxTopK || classes > 65535 || (long long)fg * nms_top_k > kMaxSort || N > 65535)
    return fail(Q8_ERR_UNSUPPORTED, "q8_detection_output: limits are %d boxes per image, nms_top_k <= %d, (classes - 1) * nms_top_k <= %d, N <= 65535",
                kMaxSort, kMaxTopK, kMaxSort);
  return Q8_OK;
}

int q8_detection_output_workspace_bytes(int N, int P, int classes, int background, int nms_top_k, int keep_top_k, size_t* bytes) {
  clear_error();
  if (!bytes) return fail(Q8_ERR_INVALID_ARG, "q8_detection_output_workspace_bytes: null pointer");
  const int rc = det_check(N, P, classes, background, nms_top_k, keep_top_k);
  if (rc != Q8_OK) return rc;
  *bytes = det_layout(N, P, classes, nms_top_k).total;
  return Q8_OK;
}

int q8_detection_output(int n_sources, const float* const* loc, const int* loc_stride, const float* const* conf,
                        const int* conf_stride, const int* cells, const int* boxes_per_cell, const float* d_priors,
                        const float* variances, int N, int classes, int background, float conf_thresh, float nms_thresh,
                        int nms_top_k, int keep_top_k, void* workspace, size_t workspace_bytes, float* d_out, int* d_counts,
                        void* stream) {
  clear_error();
  if (n_sources <= 0 || n_sources > kMaxSources || !loc || !loc_stride || !conf || !conf_stride || !cells || !boxes_per_cell ||
      !d_priors || !variances || !d_out || !d_counts)
    return fail(Q8_ERR_INVALID_ARG, "q8_detection_output: null pointer or more than %d sources", kMaxSources);
  if (classes <= 0) return fail(Q8_ERR_INVALID_ARG, "q8_detection_output: classes must be positive");
  DetSources src{};
  src.n = n_sources;
  long long P = 0;
  for (int i = 0; i < n_sources; ++i) {
    if (!loc[i] || !conf[i] || cells[i] <= 0 || boxes_per_cell[i] <= 0 || loc_stride[i] < boxes_per_cell[i] * 4 ||
        (long long)conf_stride[i] < (long long)boxes_per_cell[i] * classes)
      return fail(Q8_ERR_INVALID_ARG, "q8_detection_output: source %d: null pointer, empty, or a cell stride below its values", i);
    src.loc[i] = loc[i]; src.conf[i] = conf[i];
    src.loc_stride[i] = loc_stride[i]; src.conf_stride[i] = conf_stride[i];
    src.cells[i] = cells[i]; src.boxes[i] = boxes_per_cell[i];
    src.first[i] = (int)P;
    P += (long long)cells[i] * boxes_per_cell[i];
    if (P > kMaxSort) return fail(Q8_ERR_UNSUPPORTED, "q8_detection_output: more than %d boxes per image", kMaxSort);
  }
  src.first[n_sources] = (int)P;
  const int rc = det_check(N, (int)P, classes, background, nms_top_k, keep_top_k);
  if (rc != Q8_OK) return rc;
  if (!std::isfinite(conf_thresh) || !std::isfinite(nms_thresh) || conf_thresh < 0.f)
    return fail(Q8_ERR_NONFINITE, "q8_detection_output: thresholds must be finite, the confidence threshold not negative");
  if (!aligned16(d_priors)) return fail(Q8_ERR_ALIGNMENT, "q8_detection_output: priors not 16-byte aligned");
  const DetLayout L = det_layout(N, (int)P, classes, nms_top_k);
  if (!workspace || workspace_bytes < L.total || (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return fail(Q8_ERR_WORKSPACE, "q8_detection_output: workspace of %zu bytes, 256-byte aligned, needed", L.total);
  cudaStream_t s = as_stream(stream);
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  float4* boxes = reinterpret_cast<float4*>(ws + L.boxes);
  float* prob = reinterpret_cast<float*>(ws + L.prob);
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(ws + L.keys);
  int* kcount = reinterpret_cast<int*>(ws + L.counts);
  {
    const size_t total = (size_t)N * P, blocks = (total + 255) / 256, cap = (size_t)sm_count() * 8;
    decode_softmax_kernel<<<(unsigned)(blocks < cap ? blocks : cap), 256, 0, s>>>(src, reinterpret_cast<const float4*>(d_priors), variances[0],
                                                                                    variances[1], variances[2], variances[3], N, (int)P,
                                                                                    classes, boxes, prob);
    const int rc2 = check_launch("decode_softmax_kernel");
    if (rc2 != Q8_OK) return rc2;
  }
  const int fg = classes - (background >= 0 ? 1 : 0);
  {
    const unsigned int W = (unsigned)(nms_top_k + 31) / 32;
    unsigned int work_bytes = (unsigned)kSelCap * 8u;
    if (work_bytes < (unsigned)nms_top_k * W * 4u) work_bytes = (unsigned)nms_top_k * W * 4u;
    work_bytes = (work_bytes + 15u) & ~15u;
    const size_t smem = (size_t)work_bytes + (size_t)kMaxTopK * (8 + 16) + (size_t)kSelBins * 4;
    const int dev = current_device();
    static std::atomic<size_t> configured[kMaxDevices];
    if (dev < 0 || configured[dev].load() < smem) {
      const int rc2 = check_cuda(cudaFuncSetAttribute(nms_class_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem), "cudaFuncSetAttribute(nms_class_kernel)");
      if (rc2 != Q8_OK) return rc2;
      if (dev >= 0) configured[dev].store(smem);
    }
    nms_class_kernel<<<dim3((unsigned)fg, (unsigned)N), kNmsThreads, smem, s>>>(boxes, prob, (int)P, classes, background, conf_thresh, nms_thresh,
                                                                               nms_top_k, work_bytes, keys, kcount);
    const int rc2 = check_launch("nms_class_kernel");
    if (rc2 != Q8_OK) return rc2;
  }
  {
    int cap = 1;
    while (cap < fg * nms_top_k) cap <<= 1;
    const size_t smem = (size_t)cap * 8;
    const int dev = current_device();
    static std::atomic<size_t> configured[kMaxDevices];
    if (dev < 0 || configured[dev].load() < smem) {
      const int rc2 = check_cuda(cudaFuncSetAttribute(keep_top_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem), "cudaFuncSetAttribute(keep_top_kernel)");
      if (rc2 != Q8_OK) return rc2;
      if (dev >= 0) configured[dev].store(smem);
    }
    keep_top_kernel<<<(unsigned)N, kTopThreads, smem, s>>>(boxes, keys, kcount, (int)P, classes, background, nms_top_k, keep_top_k, d_out, d_counts);
  }
  return check_launch("keep_top_kernel");
}

}  // extern "C"
