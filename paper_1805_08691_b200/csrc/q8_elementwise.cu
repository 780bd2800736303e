// Bandwidth-bound kernels around the quantized convolution: max-abs calibration,
// quantize (Eq. Q), dequantize (Eq. D), BN folding, concat, pooling.
//
// All of them stream their operands once with 16-byte accesses; grids are sized
// as a multiple of the SM count so every SM keeps several loads in flight.
#include <cmath>

#include "q8_internal.h"

namespace q8 {
namespace {

constexpr int kThreads = 512;

int grid_for(size_t work_items, int per_block, int blocks_per_sm) {
  size_t need = (work_items + per_block - 1) / per_block;
  size_t cap = (size_t)sm_count() * blocks_per_sm;
  if (need < 1) need = 1;
  return (int)(need < cap ? need : cap);
}

// ---------------------------------------------------------------------------------------------
// max |x|: bits of a non-negative float order like unsigned integers, and NaN/Inf patterns sit
// above every finite value, so an unsigned atomicMax both reduces and propagates non-finite input.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned int abs_bits(float v) { return __float_as_uint(v) & 0x7fffffffu; }

__global__ void __launch_bounds__(kThreads) maxabs_kernel(const float* __restrict__ x, size_t n,
                                                          unsigned int* __restrict__ running) {
  unsigned int m = 0;
  // head: scalar until 16-byte aligned
  size_t head = ((16 - (reinterpret_cast<uintptr_t>(x) & 15u)) & 15u) / 4;
  if (head > n) head = n;
  const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  if (tid < head) m = abs_bits(x[tid]);
  const float4* x4 = reinterpret_cast<const float4*>(x + head);
  const size_t n4 = (n - head) / 4;
  size_t i = tid;
  // four independent 16-byte loads in flight per thread
  for (; i + 3 * nthreads < n4; i += 4 * nthreads) {
    float4 a = __ldcs(x4 + i), b = __ldcs(x4 + i + nthreads), c = __ldcs(x4 + i + 2 * nthreads),
           d = __ldcs(x4 + i + 3 * nthreads);
    m = max(m, max(max(abs_bits(a.x), abs_bits(a.y)), max(abs_bits(a.z), abs_bits(a.w))));
    m = max(m, max(max(abs_bits(b.x), abs_bits(b.y)), max(abs_bits(b.z), abs_bits(b.w))));
    m = max(m, max(max(abs_bits(c.x), abs_bits(c.y)), max(abs_bits(c.z), abs_bits(c.w))));
    m = max(m, max(max(abs_bits(d.x), abs_bits(d.y)), max(abs_bits(d.z), abs_bits(d.w))));
  }
  for (; i < n4; i += nthreads) {
    float4 a = __ldcs(x4 + i);
    m = max(m, max(max(abs_bits(a.x), abs_bits(a.y)), max(abs_bits(a.z), abs_bits(a.w))));
  }
  const size_t tail0 = head + n4 * 4;
  if (tail0 + tid < n) m = max(m, abs_bits(x[tail0 + tid]));

#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
  __shared__ unsigned int warp_max[kThreads / 32];
  if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x < 32) {
    m = threadIdx.x < kThreads / 32 ? warp_max[threadIdx.x] : 0u;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (threadIdx.x == 0 && m != 0) atomicMax(running, m);
  }
}

// ---------------------------------------------------------------------------------------------
// Eq. (Q).  One fp32 IEEE division, round-to-nearest-even conversion (saturating, NaN -> 0), clamp.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ int quant1(float v, float q, int lo, int hi) {
  int z = __float2int_rn(__fdiv_rn(v, q));
  return min(max(z, lo), hi);
}

__device__ __forceinline__ unsigned int pack4(int a, int b, int c, int d) {
  return (unsigned int)(a & 0xff) | ((unsigned int)(b & 0xff) << 8) | ((unsigned int)(c & 0xff) << 16) |
         ((unsigned int)(d & 0xff) << 24);
}

// One float4 in, four bytes out per thread and step: a warp reads 512 contiguous bytes and writes 128.
// Four independent steps are in flight per thread.  n4 = number of float4.  Requires x 16-byte and z
// 4-byte aligned.
__global__ void __launch_bounds__(kThreads) quantize8_vec_kernel(const float4* __restrict__ x, size_t n4,
                                                                 float q, int lo, int hi,
                                                                 unsigned int* __restrict__ z) {
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  for (; i + 3 * nthreads < n4; i += 4 * nthreads) {
    const float4 a = __ldcs(x + i), b = __ldcs(x + i + nthreads), c = __ldcs(x + i + 2 * nthreads), d = __ldcs(x + i + 3 * nthreads);
    __stcs(z + i, pack4(quant1(a.x, q, lo, hi), quant1(a.y, q, lo, hi), quant1(a.z, q, lo, hi), quant1(a.w, q, lo, hi)));
    __stcs(z + i + nthreads, pack4(quant1(b.x, q, lo, hi), quant1(b.y, q, lo, hi), quant1(b.z, q, lo, hi), quant1(b.w, q, lo, hi)));
    __stcs(z + i + 2 * nthreads, pack4(quant1(c.x, q, lo, hi), quant1(c.y, q, lo, hi), quant1(c.z, q, lo, hi), quant1(c.w, q, lo, hi)));
    __stcs(z + i + 3 * nthreads, pack4(quant1(d.x, q, lo, hi), quant1(d.y, q, lo, hi), quant1(d.z, q, lo, hi), quant1(d.w, q, lo, hi)));
  }
  for (; i < n4; i += nthreads) {
    const float4 a = __ldcs(x + i);
    __stcs(z + i, pack4(quant1(a.x, q, lo, hi), quant1(a.y, q, lo, hi), quant1(a.z, q, lo, hi), quant1(a.w, q, lo, hi)));
  }
}

template <typename OutT>
__global__ void __launch_bounds__(kThreads) quantize_scalar_kernel(const float* __restrict__ x, size_t begin,
                                                                   size_t n, float q, int lo, int hi,
                                                                   OutT* __restrict__ z) {
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  for (size_t i = begin + (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += nthreads)
    z[i] = (OutT)quant1(x[i], q, lo, hi);
}

__global__ void __launch_bounds__(kThreads) quantize32_vec_kernel(const float4* __restrict__ x, size_t n4, float q,
                                                                  int4* __restrict__ z) {
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += nthreads) {
    float4 a = __ldcs(x + i);
    int4 o;
    o.x = __float2int_rn(__fdiv_rn(a.x, q));
    o.y = __float2int_rn(__fdiv_rn(a.y, q));
    o.z = __float2int_rn(__fdiv_rn(a.z, q));
    o.w = __float2int_rn(__fdiv_rn(a.w, q));
    __stcs(z + i, o);
  }
}

// One factor per row: a block walks rows (grid stride), its threads the columns.
__global__ void __launch_bounds__(256) maxabs_rows_kernel(const float* __restrict__ x, size_t rows, size_t cols,
                                                          unsigned int* __restrict__ running) {
  __shared__ unsigned int warp_max[8];
  for (size_t r = blockIdx.x; r < rows; r += gridDim.x) {
    const float* row = x + r * cols;
    unsigned int m = 0;
    for (size_t c = threadIdx.x; c < cols; c += blockDim.x) m = max(m, abs_bits(row[c]));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
#pragma unroll
      for (int w = 1; w < 8; ++w) m = max(m, warp_max[w]);
      atomicMax(running + r, m);
    }
    __syncthreads();
  }
}

template <typename OutT>
__global__ void __launch_bounds__(256) quantize_rows_kernel(const float* __restrict__ x, size_t rows, size_t cols,
                                                            const float* __restrict__ q, int lo, int hi,
                                                            OutT* __restrict__ z) {
  for (size_t r = blockIdx.x; r < rows; r += gridDim.x) {
    const float qr = q[r];
    const float* row = x + r * cols;
    OutT* out = z + r * cols;
    for (size_t c = threadIdx.x; c < cols; c += blockDim.x) out[c] = (OutT)quant1(row[c], qr, lo, hi);
  }
}

// NHWC pixels with C real channels -> C_pad channels, zeros appended.  One thread per pixel group.
template <typename OutT>
__global__ void __launch_bounds__(kThreads) quantize_pad_kernel(const float* __restrict__ x, size_t pixels, int C,
                                                                int C_pad, float q, int lo, int hi,
                                                                OutT* __restrict__ z) {
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  const size_t total = pixels * (size_t)C_pad;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += nthreads) {
    size_t px = i / C_pad;
    int c = (int)(i - px * C_pad);
    z[i] = c < C ? (OutT)quant1(x[px * C + c], q, lo, hi) : (OutT)0;
  }
}

// The same with one 16-byte store per thread: thread = (pixel, group of 16 output channels).  A warp reads
// 32 consecutive pixels (contiguous floats when C <= 16) and writes 512 contiguous bytes.
__global__ void __launch_bounds__(kThreads) quantize_pad16_kernel(const float* __restrict__ x, size_t pixels, int C,
                                                                  int groups, float q, int lo, int hi,
                                                                  uint4* __restrict__ z) {
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  const size_t total = pixels * (size_t)groups;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += nthreads) {
    const size_t px = i / groups;
    const int c0 = (int)(i - px * groups) * 16;
    const float* src = x + px * C + c0;
    int v[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = (c0 + j < C) ? quant1(__ldcs(src + j), q, lo, hi) : 0;
    z[i] = make_uint4(pack4(v[0], v[1], v[2], v[3]), pack4(v[4], v[5], v[6], v[7]), pack4(v[8], v[9], v[10], v[11]),
                      pack4(v[12], v[13], v[14], v[15]));
  }
}

// Image batch with padded rows and channels: thread = (output pixel, group of 16 output channels).
__global__ void __launch_bounds__(kThreads) quantize_pad_image_kernel(const float* __restrict__ x, size_t rows, int W, int C,
                                                                      int W_pad, int groups, float q, int lo, int hi,
                                                                      uint4* __restrict__ z) {
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  const size_t per_row = (size_t)W_pad * groups;
  const size_t total = rows * per_row;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += nthreads) {
    const size_t row = i / per_row;
    const unsigned int rem = (unsigned int)(i - row * per_row);
    const int w = (int)(rem / (unsigned)groups), c0 = (int)(rem % (unsigned)groups) * 16;
    int v[16];
    const float* src = x + (row * W + w) * C + c0;
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = (w < W && c0 + j < C) ? quant1(__ldcs(src + j), q, lo, hi) : 0;
    z[i] = make_uint4(pack4(v[0], v[1], v[2], v[3]), pack4(v[4], v[5], v[6], v[7]), pack4(v[8], v[9], v[10], v[11]),
                      pack4(v[12], v[13], v[14], v[15]));
  }
}

// Images: 3 channels -> 16, rows of W pixels padded to W_pad output pixels.  A warp takes 128 output pixels of one
// row: their 384 floats travel to shared memory as asynchronous copies (16 bytes each where the chunk starts on a
// 16-byte boundary, else 4), the copies of the warp's next chunk are in flight while every lane quantizes four pixels
// of the present one (three conflict-free shared-memory reads each), and the warp writes 512 contiguous bytes per
// store.  (One thread per pixel reads 12-byte and writes 16-byte pieces 48 / 64 bytes apart: a third / a quarter
// of every sector per instruction, measured 61 % of the copy bandwidth; without the second buffer the loads and
// the arithmetic of a warp alternate, 66 %.)
constexpr int kPadThreads = 256;

__device__ __forceinline__ void cp_async4(float* dst, const float* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((unsigned)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async16(float* dst, const float* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((unsigned)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}

__global__ void __launch_bounds__(kPadThreads, 8) quantize_pad3_rows_kernel(const float* __restrict__ x, size_t rows, size_t W,
                                                                            size_t W_pad, float q, int lo, int hi,
                                                                            uint4* __restrict__ z) {
  __shared__ __align__(16) float stage[2][kPadThreads / 32][384];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const size_t chunks_per_row = (W_pad + 127) / 128, chunks = rows * chunks_per_row;
  const size_t nwarps = (size_t)gridDim.x * (kPadThreads / 32);
  auto fetch = [&](size_t ch, int buf) {
    if (ch < chunks) {
      const size_t r = ch / chunks_per_row, w0 = (ch - r * chunks_per_row) * 128;
      const size_t in_px = w0 < W ? (W - w0 < 128 ? W - w0 : 128) : 0;      // real pixels of this chunk
      const float* src = x + (r * W + w0) * 3;
      float* st = stage[buf][warp];
      if (in_px == 128 && (reinterpret_cast<uintptr_t>(src) & 15) == 0) {
#pragma unroll
        for (int k = 0; k < 3; ++k) cp_async16(st + (k * 32 + lane) * 4, src + (k * 32 + lane) * 4);
      } else {
        const int nf = (int)in_px * 3;
#pragma unroll
        for (int k = 0; k < 12; ++k) {
          const int f = k * 32 + lane;
          if (f < nf) cp_async4(st + f, src + f);
        }
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  size_t ch = (size_t)blockIdx.x * (kPadThreads / 32) + warp;
  int buf = 0;
  fetch(ch, 0);
  for (; ch < chunks; ch += nwarps, buf ^= 1) {
    fetch(ch + nwarps, buf ^ 1);
    asm volatile("cp.async.wait_group 1;" ::: "memory");
    __syncwarp();
    const size_t r = ch / chunks_per_row, w0 = (ch - r * chunks_per_row) * 128;
    const size_t in_px = w0 < W ? (W - w0 < 128 ? W - w0 : 128) : 0;
    const size_t out_px = W_pad - w0 < 128 ? W_pad - w0 : 128;
    const float* st = stage[buf][warp];
    uint4* out = z + r * W_pad + w0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int px = k * 32 + lane;
      if ((size_t)px < out_px) {
        unsigned int w = 0u;
        if ((size_t)px < in_px) w = pack4(quant1(st[3 * px], q, lo, hi), quant1(st[3 * px + 1], q, lo, hi), quant1(st[3 * px + 2], q, lo, hi), 0);
        __stcs(out + px, make_uint4(w, 0u, 0u, 0u));
      }
    }
    __syncwarp();
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// ---------------------------------------------------------------------------------------------
// Eq. (D): r = q * float(z), one fp32 multiply.
// ---------------------------------------------------------------------------------------------
template <bool kSigned>
__device__ __forceinline__ float4 deq4(unsigned int w, float q) {
  float4 r;
  if (kSigned) {
    r.x = __fmul_rn(q, (float)(int)(signed char)(w & 0xff));
    r.y = __fmul_rn(q, (float)(int)(signed char)((w >> 8) & 0xff));
    r.z = __fmul_rn(q, (float)(int)(signed char)((w >> 16) & 0xff));
    r.w = __fmul_rn(q, (float)(int)(signed char)(w >> 24));
  } else {
    r.x = __fmul_rn(q, (float)(w & 0xff));
    r.y = __fmul_rn(q, (float)((w >> 8) & 0xff));
    r.z = __fmul_rn(q, (float)((w >> 16) & 0xff));
    r.w = __fmul_rn(q, (float)(w >> 24));
  }
  return r;
}

// Four bytes in, one float4 out per thread and step (a warp reads 128 contiguous bytes and writes 512),
// four independent steps in flight.  n4 = number of 4-byte groups.
template <bool kSigned>
__global__ void __launch_bounds__(kThreads) dequantize8_vec_kernel(const unsigned int* __restrict__ z, size_t n4, float q,
                                                                   float4* __restrict__ r) {
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  for (; i + 3 * nthreads < n4; i += 4 * nthreads) {
    const unsigned int a = __ldcs(z + i), b = __ldcs(z + i + nthreads), c = __ldcs(z + i + 2 * nthreads), d = __ldcs(z + i + 3 * nthreads);
    __stcs(r + i, deq4<kSigned>(a, q));
    __stcs(r + i + nthreads, deq4<kSigned>(b, q));
    __stcs(r + i + 2 * nthreads, deq4<kSigned>(c, q));
    __stcs(r + i + 3 * nthreads, deq4<kSigned>(d, q));
  }
  for (; i < n4; i += nthreads) __stcs(r + i, deq4<kSigned>(__ldcs(z + i), q));
}

template <typename InT>
__global__ void __launch_bounds__(kThreads) dequantize_scalar_kernel(const InT* __restrict__ z, size_t begin,
                                                                     size_t n, float q, float* __restrict__ r) {
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  for (size_t i = begin + (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += nthreads)
    r[i] = __fmul_rn(q, (float)z[i]);
}

// ---------------------------------------------------------------------------------------------
// BN folding in fp64, rounded once to fp32.  grid = (chunks, K).
// ---------------------------------------------------------------------------------------------
__global__ void fold_bn_kernel(const float* __restrict__ w, const float* __restrict__ b,
                               const float* __restrict__ gamma, const float* __restrict__ beta,
                               const float* __restrict__ mean, const float* __restrict__ var, double eps,
                               size_t elems_per_k, float* __restrict__ w_out, float* __restrict__ b_out) {
  const int k = blockIdx.y;
  const double a = __ddiv_rn((double)gamma[k], __dsqrt_rn(__dadd_rn((double)var[k], eps)));
  const size_t base = (size_t)k * elems_per_k;
  for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < elems_per_k; e += (size_t)gridDim.x * blockDim.x)
    w_out[base + e] = (float)__dmul_rn(a, (double)w[base + e]);
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    double b0 = b ? (double)b[k] : 0.0;
    b_out[k] = (float)__dadd_rn(__dmul_rn(a, __dsub_rn(b0, (double)mean[k])), (double)beta[k]);
  }
}

// ---------------------------------------------------------------------------------------------
// Concat: one launch per branch; re-expresses the branch at the shared factor.
// ---------------------------------------------------------------------------------------------
template <bool kSigned>
__device__ __forceinline__ int requant_byte(unsigned int b, float s) {
  float v = kSigned ? (float)(int)(signed char)b : (float)b;
  int z = __float2int_rn(__fmul_rn(v, s));
  return kSigned ? min(max(z, -128), 127) : min(max(z, 0), 255);
}

template <bool kSigned>
__device__ __forceinline__ unsigned int requant_word(unsigned int w, float s) {
  return pack4(requant_byte<kSigned>(w & 0xff, s), requant_byte<kSigned>((w >> 8) & 0xff, s),
               requant_byte<kSigned>((w >> 16) & 0xff, s), requant_byte<kSigned>(w >> 24, s));
}

// Packed fp32 pairs: two independent IEEE operations (round to nearest even) per instruction.
__device__ __forceinline__ unsigned long long pack_f2(float a, float b) {
  unsigned long long d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(a), "f"(b));
  return d;
}
__device__ __forceinline__ void unpack_f2(unsigned long long d, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(d));
}
__device__ __forceinline__ unsigned long long fmul2(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ unsigned long long fsub2(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// The same re-expression for multipliers in (0, 1] (the shared factor is the largest branch factor, so this is the
// case in practice): |z * s| <= |z| needs no clamp, the byte becomes a float exactly through the 2^23 trick (signed
// bytes biased by 128), one fp32 multiply, and round-half-even by adding 1.5 * 2^23, whose low mantissa byte is the
// result in two's complement.  Less than half the instructions of the general form, which bounds this kernel.
template <bool kSigned>
__device__ __forceinline__ unsigned int requant_word_small(unsigned int w, float s) {
  const unsigned int u = kSigned ? (w ^ 0x80808080u) : w;
  const float off = kSigned ? 8388736.0f : 8388608.0f;
  const unsigned long long off2 = pack_f2(off, off), s2 = pack_f2(s, s);
  float v0, v1, v2, v3;
  unpack_f2(fmul2(fsub2(pack_f2(__uint_as_float(__byte_perm(u, 0x4B000000u, 0x7540u)),
                                __uint_as_float(__byte_perm(u, 0x4B000000u, 0x7541u))), off2), s2), v0, v1);
  unpack_f2(fmul2(fsub2(pack_f2(__uint_as_float(__byte_perm(u, 0x4B000000u, 0x7542u)),
                                __uint_as_float(__byte_perm(u, 0x4B000000u, 0x7543u))), off2), s2), v2, v3);
  const unsigned int z0 = __float_as_uint(__fadd_rn(v0, 12582912.0f)), z1 = __float_as_uint(__fadd_rn(v1, 12582912.0f));
  const unsigned int z2 = __float_as_uint(__fadd_rn(v2, 12582912.0f)), z3 = __float_as_uint(__fadd_rn(v3, 12582912.0f));
  return __byte_perm(__byte_perm(z0, z1, 0x0040u), __byte_perm(z2, z3, 0x0040u), 0x5410u);
}

// vec path: channels, c_total and c_off multiples of 16, pointers 16-byte aligned.
// One thread moves 16-byte groups i0, i0 + nthreads, ... of a branch; two loads are issued before the first of
// them is used, with all 2048 threads of an SM resident (a loop whose body branches on the kind of multiplier kept one load in flight per thread and ran at
// 0.67 of the copy bandwidth).  kMode 0: general multiplier, 1: copy, 2: multiplier in (0, 1).
template <bool kSigned, int kMode>
__device__ __forceinline__ uint4 concat_word(uint4 v, float s) {
  if (kMode == 2) {
    v.x = requant_word_small<kSigned>(v.x, s);
    v.y = requant_word_small<kSigned>(v.y, s);
    v.z = requant_word_small<kSigned>(v.z, s);
    v.w = requant_word_small<kSigned>(v.w, s);
  } else if (kMode == 0) {
    v.x = requant_word<kSigned>(v.x, s);
    v.y = requant_word<kSigned>(v.y, s);
    v.z = requant_word<kSigned>(v.z, s);
    v.w = requant_word<kSigned>(v.w, s);
  }
  return v;
}

template <bool kSigned, int kMode>
__device__ __forceinline__ void concat_span(const uint4* __restrict__ x, size_t total, int cvec, int ctot_vec,
                                            int coff_vec, float s, size_t i, size_t nthreads, uint4* __restrict__ y) {
  // (pixel, 16-byte group) of this thread's element, advanced by additions: one division per thread
  size_t px = i / cvec;
  int c = (int)(i - px * cvec);
  const size_t dpx = nthreads / cvec;
  const int dc = (int)(nthreads - dpx * cvec);
  constexpr int kBatch = 2;
  for (; i + (kBatch - 1) * nthreads < total; i += kBatch * nthreads) {
    uint4 v[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) v[u] = __ldcs(x + i + u * nthreads);
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      y[px * ctot_vec + coff_vec + c] = concat_word<kSigned, kMode>(v[u], s);
      px += dpx;
      c += dc;
      if (c >= cvec) { c -= cvec; ++px; }
    }
  }
  for (; i < total; i += nthreads) {
    y[px * ctot_vec + coff_vec + c] = concat_word<kSigned, kMode>(__ldcs(x + i), s);
    px += dpx;
    c += dc;
    if (c >= cvec) { c -= cvec; ++px; }
  }
}

template <bool kSigned>
__device__ __forceinline__ void concat_span_mode(int mode, const uint4* __restrict__ x, size_t total, int cvec,
                                                 int ctot_vec, int coff_vec, float s, size_t i, size_t nthreads,
                                                 uint4* __restrict__ y) {
  if (mode == 1) concat_span<kSigned, 1>(x, total, cvec, ctot_vec, coff_vec, s, i, nthreads, y);
  else if (mode == 2) concat_span<kSigned, 2>(x, total, cvec, ctot_vec, coff_vec, s, i, nthreads, y);
  else concat_span<kSigned, 0>(x, total, cvec, ctot_vec, coff_vec, s, i, nthreads, y);
}

template <bool kSigned>
__global__ void __launch_bounds__(kThreads, 4) concat_vec_kernel(const uint4* __restrict__ x, size_t pixels, int cvec,
                                                              int ctot_vec, int coff_vec, float s, int copy_only,
                                                              uint4* __restrict__ y) {
  concat_span_mode<kSigned>(copy_only, x, pixels * (size_t)cvec, cvec, ctot_vec, coff_vec, s,
                            (size_t)blockIdx.x * blockDim.x + threadIdx.x, (size_t)gridDim.x * blockDim.x, y);
}

// All branches in one launch: a block belongs to one branch (its range of block indices is proportional to the
// branch's bytes) and moves that branch with the blocks of its range.
struct ConcatBranch {
  const uint4* x;
  int cvec, coff_vec;
  float s;
  int mode;            // 0: general multiplier, 1: copy, 2: multiplier in (0, 1)
  unsigned int block0; // first block of this branch
};
struct ConcatBranches {
  ConcatBranch b[8];
  int n;
  unsigned int blocks;  // all branches
};

template <bool kSigned>
__global__ void __launch_bounds__(kThreads, 4) concat_multi_kernel(const __grid_constant__ ConcatBranches br, size_t pixels,
                                                                int ctot_vec, uint4* __restrict__ y) {
  int k = 0;
#pragma unroll
  for (int j = 1; j < 8; ++j)
    if (j < br.n && blockIdx.x >= br.b[j].block0) k = j;
  const ConcatBranch& me = br.b[k];
  const unsigned int nblocks = (k + 1 < br.n ? br.b[k + 1].block0 : br.blocks) - me.block0;
  concat_span_mode<kSigned>(me.mode, me.x, pixels * (size_t)me.cvec, me.cvec, ctot_vec, me.coff_vec, me.s,
                            (size_t)(blockIdx.x - me.block0) * blockDim.x + threadIdx.x,
                            (size_t)nblocks * blockDim.x, y);
}

template <bool kSigned>
__global__ void __launch_bounds__(kThreads) concat_scalar_kernel(const unsigned char* __restrict__ x, size_t pixels,
                                                                 int ch, int ctot, int coff, float s, int copy_only,
                                                                 unsigned char* __restrict__ y) {
  const size_t total = pixels * (size_t)ch;
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += nthreads) {
    size_t px = i / ch;
    int c = (int)(i - px * ch);
    unsigned int b = x[i];
    y[px * ctot + coff + c] = copy_only == 1 ? (unsigned char)b : (unsigned char)requant_byte<kSigned>(b, s);
  }
}

// ---------------------------------------------------------------------------------------------
// Pooling: one thread per output pixel and group of 4 channels (C % 4 == 0) or single channel.
// ---------------------------------------------------------------------------------------------
template <bool kSigned, bool kAvg, int kVec>
__global__ void __launch_bounds__(256) pool_kernel(const unsigned char* __restrict__ x, int N, int H, int W, int C,
                                                   int kh, int kw, int st_h, int st_w, int pad_h, int pad_w, int P,
                                                   int Q, float inv, unsigned char* __restrict__ y) {
  const int cg = C / kVec;
  const size_t total = (size_t)N * P * Q * cg;
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += nthreads) {
    int c = (int)(i % cg) * kVec;
    size_t t = i / cg;
    int q = (int)(t % Q);
    t /= Q;
    int p = (int)(t % P);
    int n = (int)(t / P);
    int acc[kVec];
#pragma unroll
    for (int j = 0; j < kVec; ++j) acc[j] = kAvg ? 0 : (kSigned ? -128 : 0);
    for (int r = 0; r < kh; ++r) {
      int h = p * st_h - pad_h + r;
      if (h < 0 || h >= H) continue;
      for (int s = 0; s < kw; ++s) {
        int w = q * st_w - pad_w + s;
        if (w < 0 || w >= W) continue;
        const unsigned char* px = x + (((size_t)n * H + h) * W + w) * C + c;
        unsigned int word;
        if (kVec == 4) word = *reinterpret_cast<const unsigned int*>(px);
        else word = *px;
#pragma unroll
        for (int j = 0; j < kVec; ++j) {
          unsigned int b = (word >> (8 * j)) & 0xff;
          int v = kSigned ? (int)(signed char)b : (int)b;
          acc[j] = kAvg ? acc[j] + v : max(acc[j], v);
        }
      }
    }
    unsigned char* out = y + (((size_t)n * P + p) * Q + q) * C + c;
    int o[kVec];
#pragma unroll
    for (int j = 0; j < kVec; ++j) {
      if (kAvg) {
        int z = __float2int_rn(__fmul_rn((float)acc[j], inv));
        o[j] = kSigned ? min(max(z, -128), 127) : min(max(z, 0), 255);
      } else {
        o[j] = acc[j];
      }
    }
    if (kVec == 4) *reinterpret_cast<unsigned int*>(out) = pack4(o[0], o[1], o[2], o[3]);
    else *out = (unsigned char)o[0];
  }
}

// Max pooling with 16 channels per thread: 16-byte loads and stores, byte-wise SIMD maximum (exact).
template <bool kSigned>
__global__ void __launch_bounds__(256) maxpool16_kernel(const uint4* __restrict__ x, int N, int H, int W, int cg, int kh,
                                                        int kw, int st_h, int st_w, int pad_h, int pad_w, int P, int Q,
                                                        uint4* __restrict__ y) {
  const size_t total = (size_t)N * P * Q * cg;
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += nthreads) {
    const int c = (int)(i % cg);
    size_t t = i / cg;
    const int q = (int)(t % Q);
    t /= Q;
    const int p = (int)(t % P);
    const int n = (int)(t / P);
    const unsigned int init = kSigned ? 0x80808080u : 0u;
    uint4 m = make_uint4(init, init, init, init);
    for (int r = 0; r < kh; ++r) {
      const int h = p * st_h - pad_h + r;
      if (h < 0 || h >= H) continue;
      for (int s = 0; s < kw; ++s) {
        const int w = q * st_w - pad_w + s;
        if (w < 0 || w >= W) continue;
        const uint4 v = __ldg(x + (((size_t)n * H + h) * W + w) * cg + c);
        if (kSigned) { m.x = __vmaxs4(m.x, v.x); m.y = __vmaxs4(m.y, v.y); m.z = __vmaxs4(m.z, v.z); m.w = __vmaxs4(m.w, v.w); }
        else { m.x = __vmaxu4(m.x, v.x); m.y = __vmaxu4(m.y, v.y); m.z = __vmaxu4(m.z, v.z); m.w = __vmaxu4(m.w, v.w); }
      }
    }
    y[i] = m;
  }
}

// Average pooling with 16 channels per thread.  Bytes are summed as pairs of 16-bit lanes (window of at most
// 256 cells: 256 * 255 < 2^16); signed bytes are biased by +128 first and the bias of the cells that were
// inside the image is taken off the sum.  Then float(sum) * fp32(1/(kh kw)), round half even, clamp.
template <bool kSigned>
__global__ void __launch_bounds__(256) avgpool16_kernel(const uint4* __restrict__ x, int N, int H, int W, int cg, int kh,
                                                        int kw, int st_h, int st_w, int pad_h, int pad_w, int P, int Q,
                                                        float inv, uint4* __restrict__ y) {
  const size_t total = (size_t)N * P * Q * cg;
  const size_t nthreads = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += nthreads) {
    const int c = (int)(i % cg);
    size_t t = i / cg;
    const int q = (int)(t % Q);
    t /= Q;
    const int p = (int)(t % P);
    const int n = (int)(t / P);
    unsigned int even[4] = {0, 0, 0, 0}, odd[4] = {0, 0, 0, 0};  // bytes 0,2 and bytes 1,3 of each word
    int cells = 0;
    for (int r = 0; r < kh; ++r) {
      const int h = p * st_h - pad_h + r;
      if (h < 0 || h >= H) continue;
      for (int s = 0; s < kw; ++s) {
        const int w = q * st_w - pad_w + s;
        if (w < 0 || w >= W) continue;
        uint4 v = __ldg(x + (((size_t)n * H + h) * W + w) * cg + c);
        if (kSigned) { v.x ^= 0x80808080u; v.y ^= 0x80808080u; v.z ^= 0x80808080u; v.w ^= 0x80808080u; }
        const unsigned int word[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          even[j] += word[j] & 0x00ff00ffu;
          odd[j] += (word[j] >> 8) & 0x00ff00ffu;
        }
        ++cells;
      }
    }
    const int bias = kSigned ? 128 * cells : 0;
    unsigned int out[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int sum[4] = {(int)(even[j] & 0xffffu) - bias, (int)(odd[j] & 0xffffu) - bias, (int)(even[j] >> 16) - bias,
                          (int)(odd[j] >> 16) - bias};
      int o[4];
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int z = __float2int_rn(__fmul_rn((float)sum[b], inv));
        o[b] = kSigned ? min(max(z, -128), 127) : min(max(z, 0), 255);
      }
      out[j] = pack4(o[0], o[1], o[2], o[3]);
    }
    y[i] = make_uint4(out[0], out[1], out[2], out[3]);
  }
}

// 3x3 and 2x2 windows, 16 channels per thread, 32-bit index arithmetic: the window is unrolled so that all of
// its (predicated) 16-byte loads are in flight together; cells outside the image do not take part.
template <bool kSigned, bool kAvg, int KH, int KW>
__global__ void __launch_bounds__(256) pool16_window_kernel(const uint4* __restrict__ x, int H, int W, int cg, int st_h,
                                                            int st_w, int pad_h, int pad_w, int P, int Q, float inv,
                                                            unsigned int total, uint4* __restrict__ y) {
  // Average: the result is a function of the window sum alone, so each block tabulates it once, with the
  // defining arithmetic clamp(Round(float(sum) * inv)); entry j is the code for sum j - kOff.  The kernel is
  // bound by integer instructions, and the table replaces seven of them per element by one shared-memory load.
  constexpr int kOff = kSigned ? 128 * KH * KW : 0;
  constexpr int kEntries = 255 * KH * KW + 1;
  __shared__ unsigned char table[kAvg ? kEntries : 1];
  if (kAvg) {
    for (int j = threadIdx.x; j < kEntries; j += blockDim.x) {
      const int z = __float2int_rn(__fmul_rn((float)(j - kOff), inv));
      table[j] = (unsigned char)(kSigned ? min(max(z, -128), 127) : min(max(z, 0), 255));
    }
    __syncthreads();
  }
  const unsigned int nthreads = gridDim.x * blockDim.x;
  for (unsigned int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += nthreads) {
    const unsigned int c = i % (unsigned)cg;
    unsigned int t = i / (unsigned)cg;
    const int q = (int)(t % (unsigned)Q);
    t /= (unsigned)Q;
    const int p = (int)(t % (unsigned)P);
    const unsigned int n = t / (unsigned)P;
    const int h0 = p * st_h - pad_h, w0 = q * st_w - pad_w;
    const uint4* img = x + (size_t)n * H * W * cg + c;
    uint4 v[KH * KW];
    bool ok[KH * KW];
#pragma unroll
    for (int r = 0; r < KH; ++r)
#pragma unroll
      for (int s = 0; s < KW; ++s) {
        const int h = h0 + r, w = w0 + s;
        ok[r * KW + s] = h >= 0 && h < H && w >= 0 && w < W;
        v[r * KW + s] = ok[r * KW + s] ? __ldg(img + ((size_t)h * W + w) * cg) : make_uint4(0u, 0u, 0u, 0u);
      }
    if (!kAvg) {
      const unsigned int init = kSigned ? 0x80808080u : 0u;
      uint4 m = make_uint4(init, init, init, init);
#pragma unroll
      for (int k = 0; k < KH * KW; ++k) {
        if (!ok[k]) continue;
        if (kSigned) { m.x = __vmaxs4(m.x, v[k].x); m.y = __vmaxs4(m.y, v[k].y); m.z = __vmaxs4(m.z, v[k].z); m.w = __vmaxs4(m.w, v[k].w); }
        else { m.x = __vmaxu4(m.x, v[k].x); m.y = __vmaxu4(m.y, v[k].y); m.z = __vmaxu4(m.z, v[k].z); m.w = __vmaxu4(m.w, v[k].w); }
      }
      y[i] = m;
    } else {
      unsigned int even[4] = {0, 0, 0, 0}, odd[4] = {0, 0, 0, 0};
      int cells = 0;
#pragma unroll
      for (int k = 0; k < KH * KW; ++k) {
        if (!ok[k]) continue;
        const unsigned int flip = kSigned ? 0x80808080u : 0u;
        const unsigned int word[4] = {v[k].x ^ flip, v[k].y ^ flip, v[k].z ^ flip, v[k].w ^ flip};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          even[j] += word[j] & 0x00ff00ffu;
          odd[j] += __byte_perm(word[j], 0u, 0x4341u);  // bytes 1 and 3 as 16-bit lanes
        }
        ++cells;
      }
      // table index = lane sum - 128 * cells + kOff (signed input was biased by 128 per cell)
      const unsigned int adj = kSigned ? (unsigned int)(128 * (KH * KW - cells)) * 0x00010001u : 0u;
      unsigned int out[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const unsigned int e = even[j] + adj, o = odd[j] + adj;
        out[j] = (unsigned int)table[e & 0xffffu] | ((unsigned int)table[o & 0xffffu] << 8) |
                 ((unsigned int)table[e >> 16] << 16) | ((unsigned int)table[o >> 16] << 24);
      }
      y[i] = make_uint4(out[0], out[1], out[2], out[3]);
    }
  }
}

template <bool kSigned, bool kAvg, int KH, int KW>
void launch_pool16_window(const void* x, int N, int H, int W, int cg, int st_h, int st_w, int pad_h, int pad_w, int P, int Q,
                          float inv, void* y, cudaStream_t s) {
  const unsigned int total = (unsigned int)((size_t)N * P * Q * cg);
  pool16_window_kernel<kSigned, kAvg, KH, KW><<<grid_for(total, 256, 8), 256, 0, s>>>(
      static_cast<const uint4*>(x), H, W, cg, st_h, st_w, pad_h, pad_w, P, Q, inv, total, static_cast<uint4*>(y));
}

// 3x3 windows with stride 1 or 2, 16 channels per thread, as vertical strips: a thread owns one output column and
// kRows consecutive output rows and slides down the image, reducing each input row of its three columns once
// (three 16-byte loads) and keeping the last rows' partial results in registers.  The one-thread-per-output form
// above issues nine loads per output (measured 29 % of the copy bandwidth for stride 1, 50 % for stride 2); here an
// output costs two (stride 1, two columns per thread) or six (stride 2) loads.
// Average: bytes are summed as 16-bit lanes (signed input biased by +128 per in-image cell); the rounding of
// clamp(Round(float(sum) * fp32(1/9))) is taken by one fused multiply-add per value (see pool_combine3; a
// full-window divisor keeps the result inside the 8-bit range, so the clamp never acts).
// Maximum: the same 16-bit lanes (signed input made unsigned by flipping the sign bits), reduced with the native
// two-lane maximum of two or three operands; the byte-wise SIMD maximum is emulated by about ten instructions per
// word (measured: 415 warp instructions per 512 output bytes, ALU pipe 72 % busy, 0.56 of the copy bandwidth).
struct PoolRow {
  unsigned int a[4], b[4];  // a = lanes of bytes 0,2; b = lanes of bytes 1,3 (sums, or maxima of sign-flipped bytes)
  int cells;                // average, signed input: in-image cells that went into the sums
};

__device__ __forceinline__ unsigned int max_u16x2(unsigned int a, unsigned int b) {
  unsigned int d;
  asm("max.u16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}

template <bool kSigned, bool kAvg>
__device__ __forceinline__ PoolRow pool_row3(const uint4* __restrict__ img, int h, int H, int W, int cg, int w0) {
  PoolRow r;
#pragma unroll
  for (int j = 0; j < 4; ++j) { r.a[j] = 0u; r.b[j] = 0u; }
  r.cells = 0;
  if (h < 0 || h >= H) return r;
  const uint4* row = img + (size_t)h * W * cg;
  const unsigned int flip = kSigned ? 0x80808080u : 0u;
  uint4 v[3];
  bool ok[3];
#pragma unroll
  for (int s = 0; s < 3; ++s) {
    ok[s] = w0 + s >= 0 && w0 + s < W;
    v[s] = ok[s] ? __ldg(row + (size_t)(w0 + s) * cg) : make_uint4(flip, flip, flip, flip);
  }
  unsigned int e[3][4], o[3][4];
#pragma unroll
  for (int s = 0; s < 3; ++s) {
    const unsigned int word[4] = {v[s].x, v[s].y, v[s].z, v[s].w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const unsigned int wj = word[j] ^ flip;  // outside the image: 0, the identity of both reductions
      e[s][j] = wj & 0x00ff00ffu;
      o[s][j] = __byte_perm(wj, 0u, 0x4341u);  // bytes 1 and 3 as 16-bit lanes
    }
    if (ok[s]) ++r.cells;
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    if (kAvg) { r.a[j] = e[0][j] + e[1][j] + e[2][j]; r.b[j] = o[0][j] + o[1][j] + o[2][j]; }
    else { r.a[j] = __vimax3_u16x2(e[0][j], e[1][j], e[2][j]); r.b[j] = __vimax3_u16x2(o[0][j], o[1][j], o[2][j]); }
  }
  return r;
}

template <bool kSigned, bool kAvg>
__device__ __forceinline__ uint4 pool_combine3(const PoolRow& r0, const PoolRow& r1, const PoolRow& r2) {
  unsigned int out[4];
  if (!kAvg) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const unsigned int e = __vimax3_u16x2(r0.a[j], r1.a[j], r2.a[j]);
      const unsigned int o = __vimax3_u16x2(r0.b[j], r1.b[j], r2.b[j]);
      out[j] = __byte_perm(e, o, 0x6240u) ^ (kSigned ? 0x80808080u : 0u);
    }
  } else {
    // One fused multiply-add per value.  bits(0x4B10LLLL) is the float 9 * 2^20 + n exactly (n = the lane, for signed
    // input raised to sum + 128 * 9 first); times fp32(1/9) that is 2^20 + n/9 + d with 0 < d < 0.01, and adding the
    // integer 1.5 * 2^23 - 2^20 (- 128 for signed input) rounds once, half to even at unit spacing, leaving
    // Round(n/9) in the low mantissa bits.  n/9 lies at least 1/18 from a tie, so d changes nothing, and neither does
    // the rounding of the definition's own fp32 product: the same integer as clamp(Round(float(sum) * fp32(1/9)))
    // for every possible window sum (checked exhaustively on the host in the tests).
    const unsigned int adj = kSigned ? (unsigned int)(128 * (9 - (r0.cells + r1.cells + r2.cells))) * 0x00010001u : 0u;
    const float c = kSigned ? (12582912.0f - 1048576.0f - 128.0f) : (12582912.0f - 1048576.0f);
    constexpr float kInv9 = 1.0f / 9.0f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const unsigned int e = r0.a[j] + r1.a[j] + r2.a[j] + adj, o = r0.b[j] + r1.b[j] + r2.b[j] + adj;
      const unsigned int z0 = __float_as_uint(__fmaf_rn(__uint_as_float(__byte_perm(e, 0x4B100000u, 0x7610u)), kInv9, c));
      const unsigned int z1 = __float_as_uint(__fmaf_rn(__uint_as_float(__byte_perm(o, 0x4B100000u, 0x7610u)), kInv9, c));
      const unsigned int z2 = __float_as_uint(__fmaf_rn(__uint_as_float(__byte_perm(e, 0x4B100000u, 0x7632u)), kInv9, c));
      const unsigned int z3 = __float_as_uint(__fmaf_rn(__uint_as_float(__byte_perm(o, 0x4B100000u, 0x7632u)), kInv9, c));
      out[j] = __byte_perm(__byte_perm(z0, z1, 0x0040u), __byte_perm(z2, z3, 0x0040u), 0x5410u);
    }
  }
  return make_uint4(out[0], out[1], out[2], out[3]);
}

// Lanes of one input pixel; outside the image: zero, the identity of both reductions.
template <bool kSigned, bool kAvg>
__device__ __forceinline__ PoolRow pool_pixel(const uint4* __restrict__ row, int w, int W, int cg, bool row_ok) {
  PoolRow r;
  const unsigned int flip = kSigned ? 0x80808080u : 0u;
  const bool ok = row_ok && w >= 0 && w < W;
  const uint4 v = ok ? __ldg(row + (size_t)w * cg) : make_uint4(flip, flip, flip, flip);
  const unsigned int word[4] = {v.x, v.y, v.z, v.w};
  r.cells = ok ? 1 : 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const unsigned int wj = word[j] ^ flip;
    r.a[j] = wj & 0x00ff00ffu;
    r.b[j] = __byte_perm(wj, 0u, 0x4341u);
  }
  return r;
}

template <bool kSigned, bool kAvg>
__device__ __forceinline__ PoolRow pool_join(const PoolRow& x, const PoolRow& y) {
  PoolRow r;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    if (!kAvg) { r.a[j] = max_u16x2(x.a[j], y.a[j]); r.b[j] = max_u16x2(x.b[j], y.b[j]); }
    else { r.a[j] = x.a[j] + y.a[j]; r.b[j] = x.b[j] + y.b[j]; }
  }
  r.cells = x.cells + y.cells;
  return r;
}

// Stride 1: a thread owns TWO adjacent output columns and kRows output rows: four loads per input row serve two
// outputs (the two middle pixels are reduced once for both).
template <bool kSigned, bool kAvg, int kRows>
__global__ void __launch_bounds__(256) pool3_strip2_kernel(const uint4* __restrict__ x, int H, int W, int cg, int pad_h,
                                                           int pad_w, int P, int Q, int strips, float inv, unsigned int total,
                                                           uint4* __restrict__ y) {
  const int Q2 = (Q + 1) >> 1;
  const unsigned int nthreads = gridDim.x * blockDim.x;
  for (unsigned int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += nthreads) {
    const unsigned int c = i % (unsigned)cg;
    unsigned int t = i / (unsigned)cg;
    const int q = (int)(t % (unsigned)Q2) * 2;
    t /= (unsigned)Q2;
    const int strip = (int)(t % (unsigned)strips);
    const unsigned int n = t / (unsigned)strips;
    const int p0 = strip * kRows, p1 = min(P, p0 + kRows);
    const int w0 = q - pad_w;
    const bool two = q + 1 < Q;
    const uint4* img = x + (size_t)n * H * W * cg + c;
    uint4* out = y + ((size_t)n * P * Q + (size_t)p0 * Q + q) * cg + c;
    PoolRow ra[3], rb[3];  // the last three input rows, reduced over the columns of output q and of output q + 1
    auto load_row = [&](int h, PoolRow& oa, PoolRow& ob) {
      const bool row_ok = h >= 0 && h < H;
      const uint4* row = img + (size_t)(row_ok ? h : 0) * W * cg;
      const PoolRow x0 = pool_pixel<kSigned, kAvg>(row, w0, W, cg, row_ok);
      const PoolRow x1 = pool_pixel<kSigned, kAvg>(row, w0 + 1, W, cg, row_ok);
      const PoolRow x2 = pool_pixel<kSigned, kAvg>(row, w0 + 2, W, cg, row_ok);
      const PoolRow x3 = pool_pixel<kSigned, kAvg>(row, w0 + 3, W, cg, row_ok && two);
      const PoolRow mid = pool_join<kSigned, kAvg>(x1, x2);
      oa = pool_join<kSigned, kAvg>(x0, mid);
      ob = pool_join<kSigned, kAvg>(mid, x3);
    };
    int h = p0 - pad_h;
    load_row(h, ra[0], rb[0]);
    load_row(h + 1, ra[1], rb[1]);
#pragma unroll 1
    for (int p = p0; p < p1; ++p, ++h, out += (size_t)Q * cg) {
      load_row(h + 2, ra[2], rb[2]);
      out[0] = pool_combine3<kSigned, kAvg>(ra[0], ra[1], ra[2]);
      if (two) out[cg] = pool_combine3<kSigned, kAvg>(rb[0], rb[1], rb[2]);
      ra[0] = ra[1]; ra[1] = ra[2];
      rb[0] = rb[1]; rb[1] = rb[2];
    }
  }
}

template <bool kSigned, bool kAvg, int kStride, int kRows>
__global__ void __launch_bounds__(256) pool3_strip_kernel(const uint4* __restrict__ x, int H, int W, int cg, int pad_h,
                                                          int pad_w, int P, int Q, int strips, float inv, unsigned int total,
                                                          uint4* __restrict__ y) {
  const unsigned int nthreads = gridDim.x * blockDim.x;
  for (unsigned int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += nthreads) {
    const unsigned int c = i % (unsigned)cg;
    unsigned int t = i / (unsigned)cg;
    const int q = (int)(t % (unsigned)Q);
    t /= (unsigned)Q;
    const int strip = (int)(t % (unsigned)strips);
    const unsigned int n = t / (unsigned)strips;
    const int p0 = strip * kRows, p1 = min(P, p0 + kRows);
    const int w0 = q * kStride - pad_w;
    const uint4* img = x + (size_t)n * H * W * cg + c;
    uint4* out = y + ((size_t)n * P * Q + (size_t)p0 * Q + q) * cg + c;
    int h = p0 * kStride - pad_h;
    PoolRow r0 = pool_row3<kSigned, kAvg>(img, h, H, W, cg, w0);
    PoolRow r1 = pool_row3<kSigned, kAvg>(img, h + 1, H, W, cg, w0);
    for (int p = p0; p < p1; ++p, h += kStride, out += (size_t)Q * cg) {
      const PoolRow r2 = pool_row3<kSigned, kAvg>(img, h + 2, H, W, cg, w0);
      *out = pool_combine3<kSigned, kAvg>(r0, r1, r2);
      if (kStride == 1) {
        r0 = r1;
        r1 = r2;
      } else {
        r0 = r2;
        if (p + 1 < p1) r1 = pool_row3<kSigned, kAvg>(img, h + 3, H, W, cg, w0);
      }
    }
  }
}

template <bool kSigned, bool kAvg, int kStride>
void launch_pool3_strip(const void* x, int N, int H, int W, int cg, int pad_h, int pad_w, int P, int Q, float inv, void* y,
                        cudaStream_t s) {
  // One strip per thread and a block per 256 strips: with a grid capped at the resident blocks, a tensor of 1.3
  // times that many strips ran two rounds with the second a third full.  Four output rows per strip: two and eight
  // were both measured slower for stride 2 (0.585 and 0.58 against 0.64 of the copy bandwidth).
  constexpr int kRows = 4;
  const int strips = (P + kRows - 1) / kRows;
  if (kStride == 1) {
    const unsigned int total = (unsigned int)((size_t)N * strips * ((Q + 1) / 2) * cg);
    pool3_strip2_kernel<kSigned, kAvg, kRows><<<(total + 255u) / 256u, 256, 0, s>>>(
        static_cast<const uint4*>(x), H, W, cg, pad_h, pad_w, P, Q, strips, inv, total, static_cast<uint4*>(y));
    return;
  }
  const unsigned int total = (unsigned int)((size_t)N * strips * Q * cg);
  pool3_strip_kernel<kSigned, kAvg, kStride, kRows><<<(total + 255u) / 256u, 256, 0, s>>>(
      static_cast<const uint4*>(x), H, W, cg, pad_h, pad_w, P, Q, strips, inv, total, static_cast<uint4*>(y));
}

// Global average pooling (the window is the whole image, one output pixel): a block takes one image and 64
// channels; thread (g, c) sums every 16th pixel of channel word c, the 16 partial sums meet in shared memory.
template <bool kSigned>
__global__ void __launch_bounds__(256) global_avgpool_kernel(const unsigned int* __restrict__ x, int pixels, int cw,
                                                             float inv, unsigned int* __restrict__ y) {
  __shared__ int part[16][16][4];
  const int c = threadIdx.x & 15, g = threadIdx.x >> 4;
  const int word = blockIdx.x * 16 + c;          // 32-bit word (4 channels) of a pixel
  const int n = blockIdx.y;
  int sum[4] = {0, 0, 0, 0};
  if (word < cw) {
    const unsigned int* img = x + (size_t)n * pixels * cw + word;
    for (int p = g; p < pixels; p += 16) {
      const unsigned int w = __ldg(img + (size_t)p * cw);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const unsigned int b = (w >> (8 * j)) & 0xffu;
        sum[j] += kSigned ? (int)(signed char)b : (int)b;
      }
    }
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) part[g][c][j] = sum[j];
  __syncthreads();
  if (g == 0 && word < cw) {
    int o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int t = 0;
#pragma unroll
      for (int k = 0; k < 16; ++k) t += part[k][c][j];
      const int z = __float2int_rn(__fmul_rn((float)t, inv));
      o[j] = kSigned ? min(max(z, -128), 127) : min(max(z, 0), 255);
    }
    y[(size_t)n * cw + word] = pack4(o[0], o[1], o[2], o[3]);
  }
}

int pool_extent(int H, int k, int st, int pad, int ceil_mode) {
  int num = H + 2 * pad - k;
  int o = (ceil_mode ? (num + st - 1) / st : num / st) + 1;
  if (ceil_mode && (o - 1) * st >= H + pad) --o;
  return o;
}

template <bool kAvg>
int launch_pool(const void* x, int t, int N, int H, int W, int C, int kh, int kw, int st_h, int st_w, int pad_h,
                int pad_w, int ceil_mode, void* y, void* stream) {
  clear_error();
  if (!x || !y) return fail(Q8_ERR_INVALID_ARG, "pool: null pointer");
  if (t != Q8_U8 && t != Q8_S8) return fail(Q8_ERR_INVALID_ARG, "pool: type must be Q8_U8 or Q8_S8");
  if (N <= 0 || H <= 0 || W <= 0 || C <= 0 || kh <= 0 || kw <= 0 || st_h <= 0 || st_w <= 0 || pad_h < 0 || pad_w < 0 ||
      pad_h >= kh || pad_w >= kw)
    return fail(Q8_ERR_INVALID_ARG, "pool: bad extents");
  int P = pool_extent(H, kh, st_h, pad_h, ceil_mode), Q = pool_extent(W, kw, st_w, pad_w, ceil_mode);
  if (P <= 0 || Q <= 0) return fail(Q8_ERR_INVALID_ARG, "pool: empty output");
  float inv = 1.0f / (float)(kh * kw);
  cudaStream_t s = as_stream(stream);
  if (kAvg && P == 1 && Q == 1 && kh == H && kw == W && pad_h == 0 && pad_w == 0 && C % 4 == 0 && N <= 65535 &&
      (reinterpret_cast<uintptr_t>(x) & 3u) == 0 && (reinterpret_cast<uintptr_t>(y) & 3u) == 0) {
    const int cw = C / 4;
    const dim3 grid((unsigned)((cw + 15) / 16), (unsigned)N);
    if (t == Q8_S8) global_avgpool_kernel<true><<<grid, 256, 0, s>>>(static_cast<const unsigned int*>(x), H * W, cw, inv, static_cast<unsigned int*>(y));
    else global_avgpool_kernel<false><<<grid, 256, 0, s>>>(static_cast<const unsigned int*>(x), H * W, cw, inv, static_cast<unsigned int*>(y));
    return check_launch("global_avgpool_kernel");
  }
  if (C % 16 == 0 && aligned16(x) && aligned16(y) && kh == kw && (kh == 3 || kh == 2) &&
      (size_t)N * P * Q * (C / 16) < (1ull << 31) && (size_t)N * H * W * (C / 16) < (1ull << 31)) {
    const int cg = C / 16;
    // strips of four output rows once that still gives every SM a few warps
    if (kh == 3 && st_h == st_w && (st_h == 1 || st_h == 2) && (size_t)N * ((P + 3) / 4) * Q * cg >= (size_t)sm_count() * 256) {
      if (st_h == 1) {
        if (t == Q8_S8) launch_pool3_strip<true, kAvg, 1>(x, N, H, W, cg, pad_h, pad_w, P, Q, inv, y, s);
        else launch_pool3_strip<false, kAvg, 1>(x, N, H, W, cg, pad_h, pad_w, P, Q, inv, y, s);
      } else {
        if (t == Q8_S8) launch_pool3_strip<true, kAvg, 2>(x, N, H, W, cg, pad_h, pad_w, P, Q, inv, y, s);
        else launch_pool3_strip<false, kAvg, 2>(x, N, H, W, cg, pad_h, pad_w, P, Q, inv, y, s);
      }
      return check_launch("pool3_strip_kernel");
    }
    if (kh == 3) {
      if (t == Q8_S8) launch_pool16_window<true, kAvg, 3, 3>(x, N, H, W, cg, st_h, st_w, pad_h, pad_w, P, Q, inv, y, s);
      else launch_pool16_window<false, kAvg, 3, 3>(x, N, H, W, cg, st_h, st_w, pad_h, pad_w, P, Q, inv, y, s);
    } else {
      if (t == Q8_S8) launch_pool16_window<true, kAvg, 2, 2>(x, N, H, W, cg, st_h, st_w, pad_h, pad_w, P, Q, inv, y, s);
      else launch_pool16_window<false, kAvg, 2, 2>(x, N, H, W, cg, st_h, st_w, pad_h, pad_w, P, Q, inv, y, s);
    }
    return check_launch("pool16_window_kernel");
  }
  if (!kAvg && C % 16 == 0 && aligned16(x) && aligned16(y)) {
    const int cg = C / 16;
    const int grid16 = grid_for((size_t)N * P * Q * cg, 256, 8);
    if (t == Q8_S8) maxpool16_kernel<true><<<grid16, 256, 0, s>>>(static_cast<const uint4*>(x), N, H, W, cg, kh, kw, st_h, st_w, pad_h, pad_w, P, Q, static_cast<uint4*>(y));
    else maxpool16_kernel<false><<<grid16, 256, 0, s>>>(static_cast<const uint4*>(x), N, H, W, cg, kh, kw, st_h, st_w, pad_h, pad_w, P, Q, static_cast<uint4*>(y));
    return check_launch("maxpool16_kernel");
  }
  if (kAvg && C % 16 == 0 && kh * kw <= 256 && aligned16(x) && aligned16(y)) {
    const int cg = C / 16;
    const int grid16 = grid_for((size_t)N * P * Q * cg, 256, 8);
    if (t == Q8_S8) avgpool16_kernel<true><<<grid16, 256, 0, s>>>(static_cast<const uint4*>(x), N, H, W, cg, kh, kw, st_h, st_w, pad_h, pad_w, P, Q, inv, static_cast<uint4*>(y));
    else avgpool16_kernel<false><<<grid16, 256, 0, s>>>(static_cast<const uint4*>(x), N, H, W, cg, kh, kw, st_h, st_w, pad_h, pad_w, P, Q, inv, static_cast<uint4*>(y));
    return check_launch("avgpool16_kernel");
  }
  bool vec = (C % 4 == 0) && ((reinterpret_cast<uintptr_t>(x) & 3u) == 0) && ((reinterpret_cast<uintptr_t>(y) & 3u) == 0);
  size_t total = (size_t)N * P * Q * (vec ? C / 4 : C);
  int grid = grid_for(total, 256, 8);
  const unsigned char* xp = static_cast<const unsigned char*>(x);
  unsigned char* yp = static_cast<unsigned char*>(y);
#define Q8_POOL(SG, V) pool_kernel<SG, kAvg, V><<<grid, 256, 0, s>>>(xp, N, H, W, C, kh, kw, st_h, st_w, pad_h, pad_w, P, Q, inv, yp)
  if (t == Q8_S8) { if (vec) Q8_POOL(true, 4); else Q8_POOL(true, 1); }
  else { if (vec) Q8_POOL(false, 4); else Q8_POOL(false, 1); }
#undef Q8_POOL
  return check_launch("pool_kernel");
}

}  // namespace
}  // namespace q8

using namespace q8;

extern "C" {

int q8_calibrate_maxabs(const float* x, size_t n, float* d_running_max, void* stream) {
  clear_error();
  if (!d_running_max || (!x && n)) return fail(Q8_ERR_INVALID_ARG, "q8_calibrate_maxabs: null pointer");
  if (reinterpret_cast<uintptr_t>(x) & 3u) return fail(Q8_ERR_ALIGNMENT, "q8_calibrate_maxabs: x not 4-byte aligned");
  if (n == 0) return Q8_OK;
  int grid = grid_for((n + 3) / 4, kThreads * 4, 4);
  maxabs_kernel<<<grid, kThreads, 0, as_stream(stream)>>>(x, n, reinterpret_cast<unsigned int*>(d_running_max));
  return check_launch("maxabs_kernel");
}

int q8_calibrate_maxabs_rows(const float* x, size_t rows, size_t cols, float* d_running_max, void* stream) {
  clear_error();
  if (!d_running_max || (!x && rows && cols)) return fail(Q8_ERR_INVALID_ARG, "q8_calibrate_maxabs_rows: null pointer");
  if (reinterpret_cast<uintptr_t>(x) & 3u) return fail(Q8_ERR_ALIGNMENT, "q8_calibrate_maxabs_rows: x not 4-byte aligned");
  if (rows == 0 || cols == 0) return Q8_OK;
  const int grid = (int)(rows < (size_t)sm_count() * 8 ? rows : (size_t)sm_count() * 8);
  maxabs_rows_kernel<<<grid, 256, 0, as_stream(stream)>>>(x, rows, cols, reinterpret_cast<unsigned int*>(d_running_max));
  return check_launch("maxabs_rows_kernel");
}

int q8_quantize_rows(const float* x, size_t rows, size_t cols, const float* d_q, int out_type, void* z, void* stream) {
  clear_error();
  if ((!x || !z || !d_q) && rows && cols) return fail(Q8_ERR_INVALID_ARG, "q8_quantize_rows: null pointer");
  if (out_type != Q8_U8 && out_type != Q8_S8 && out_type != Q8_S32) return fail(Q8_ERR_INVALID_ARG, "q8_quantize_rows: bad out_type");
  if (rows == 0 || cols == 0) return Q8_OK;
  const int grid = (int)(rows < (size_t)sm_count() * 8 ? rows : (size_t)sm_count() * 8);
  cudaStream_t s = as_stream(stream);
  if (out_type == Q8_U8) quantize_rows_kernel<unsigned char><<<grid, 256, 0, s>>>(x, rows, cols, d_q, 0, 255, static_cast<unsigned char*>(z));
  else if (out_type == Q8_S8) quantize_rows_kernel<signed char><<<grid, 256, 0, s>>>(x, rows, cols, d_q, -128, 127, static_cast<signed char*>(z));
  else quantize_rows_kernel<int><<<grid, 256, 0, s>>>(x, rows, cols, d_q, INT32_MIN, INT32_MAX, static_cast<int*>(z));
  return check_launch("quantize_rows_kernel");
}

int q8_factor(float maxabs, int p, float* q) {
  clear_error();
  if (!q || p < 1 || p > 31) return fail(Q8_ERR_INVALID_ARG, "q8_factor: bad argument");
  if (!(maxabs >= 0.0f) || std::isinf(maxabs)) return fail(Q8_ERR_NONFINITE, "q8_factor: max-abs is not a finite non-negative number");
  if (maxabs == 0.0f) { *q = 1.0f; return Q8_OK; }
  volatile float denom = (float)((1ll << p) - 1);
  volatile float r = maxabs / denom;
  *q = r;
  return Q8_OK;
}

int q8_requant_scale(float q_x, float q_w, float q_y, float* s) {
  clear_error();
  if (!s) return fail(Q8_ERR_INVALID_ARG, "q8_requant_scale: null pointer");
  if (!(q_x > 0.f) || !(q_w > 0.f) || !(q_y > 0.f) || std::isinf(q_x) || std::isinf(q_w) || std::isinf(q_y))
    return fail(Q8_ERR_NONFINITE, "q8_requant_scale: factors must be finite and positive");
  volatile double prod = (double)q_x * (double)q_w;
  volatile double quo = prod / (double)q_y;
  *s = (float)quo;
  return Q8_OK;
}

int q8_bias_factor(float q_x, float q_w, float* q_b) {
  clear_error();
  if (!q_b) return fail(Q8_ERR_INVALID_ARG, "q8_bias_factor: null pointer");
  volatile float r = q_x * q_w;
  *q_b = r;
  return Q8_OK;
}

int q8_quantize(const float* x, size_t n, float q, int out_type, void* z, void* stream) {
  clear_error();
  if ((!x || !z) && n) return fail(Q8_ERR_INVALID_ARG, "q8_quantize: null pointer");
  if (!(q > 0.f) || std::isinf(q)) return fail(Q8_ERR_NONFINITE, "q8_quantize: factor must be finite and positive");
  if (out_type != Q8_U8 && out_type != Q8_S8 && out_type != Q8_S32) return fail(Q8_ERR_INVALID_ARG, "q8_quantize: bad out_type");
  if (n == 0) return Q8_OK;
  cudaStream_t s = as_stream(stream);
  if (out_type == Q8_S32) {
    if (aligned16(x) && aligned16(z)) {
      size_t n4 = n / 4;
      if (n4) quantize32_vec_kernel<<<grid_for(n4, kThreads, 8), kThreads, 0, s>>>(reinterpret_cast<const float4*>(x), n4, q, static_cast<int4*>(z));
      if (n4 * 4 < n) quantize_scalar_kernel<int><<<1, kThreads, 0, s>>>(x, n4 * 4, n, q, INT32_MIN, INT32_MAX, static_cast<int*>(z));
    } else {
      quantize_scalar_kernel<int><<<grid_for(n, kThreads, 8), kThreads, 0, s>>>(x, 0, n, q, INT32_MIN, INT32_MAX, static_cast<int*>(z));
    }
    return check_launch("quantize32");
  }
  const int lo = out_type == Q8_U8 ? 0 : -128, hi = out_type == Q8_U8 ? 255 : 127;
  if (aligned16(x) && aligned16(z)) {
    size_t n4 = n / 4;
    if (n4) quantize8_vec_kernel<<<grid_for(n4, kThreads * 4, 4), kThreads, 0, s>>>(reinterpret_cast<const float4*>(x), n4, q, lo, hi, static_cast<unsigned int*>(z));
    if (n4 * 4 < n) quantize_scalar_kernel<unsigned char><<<1, kThreads, 0, s>>>(x, n4 * 4, n, q, lo, hi, static_cast<unsigned char*>(z));
  } else {
    quantize_scalar_kernel<unsigned char><<<grid_for(n, kThreads, 8), kThreads, 0, s>>>(x, 0, n, q, lo, hi, static_cast<unsigned char*>(z));
  }
  return check_launch("quantize8");
}

int q8_quantize_pad_channels(const float* x, size_t pixels, int C, int C_pad, float q, int out_type, void* z, void* stream) {
  clear_error();
  if ((!x || !z) && pixels) return fail(Q8_ERR_INVALID_ARG, "q8_quantize_pad_channels: null pointer");
  if (C <= 0 || C_pad < C) return fail(Q8_ERR_INVALID_ARG, "q8_quantize_pad_channels: need 0 < C <= C_pad");
  if (!(q > 0.f) || std::isinf(q)) return fail(Q8_ERR_NONFINITE, "q8_quantize_pad_channels: factor must be finite and positive");
  if (out_type != Q8_U8 && out_type != Q8_S8) return fail(Q8_ERR_INVALID_ARG, "q8_quantize_pad_channels: bad out_type");
  if (pixels == 0) return Q8_OK;
  const int lo = out_type == Q8_U8 ? 0 : -128, hi = out_type == Q8_U8 ? 255 : 127;
  if (C == 3 && C_pad == 16 && aligned16(z)) {
    quantize_pad3_rows_kernel<<<grid_for((pixels + 127) / 128, kPadThreads / 32, 8), kPadThreads, 0, as_stream(stream)>>>(
        x, 1, pixels, pixels, q, lo, hi, static_cast<uint4*>(z));
    return check_launch("quantize_pad3_rows_kernel");
  }
  if (C_pad % 16 == 0 && aligned16(z)) {
    const int groups = C_pad / 16;
    quantize_pad16_kernel<<<grid_for(pixels * groups, kThreads, 8), kThreads, 0, as_stream(stream)>>>(
        x, pixels, C, groups, q, lo, hi, static_cast<uint4*>(z));
    return check_launch("quantize_pad16_kernel");
  }
  quantize_pad_kernel<unsigned char><<<grid_for(pixels * C_pad, kThreads, 8), kThreads, 0, as_stream(stream)>>>(
      x, pixels, C, C_pad, q, lo, hi, static_cast<unsigned char*>(z));
  return check_launch("quantize_pad_kernel");
}

int q8_quantize_pad_image(const float* x, int N, int H, int W, int C, int W_pad, int C_pad, float q, int out_type, void* z,
                          void* stream) {
  clear_error();
  if (N < 0 || H < 0 || W < 0 || C <= 0 || W_pad < W || C_pad < C || C_pad % 16)
    return fail(Q8_ERR_INVALID_ARG, "q8_quantize_pad_image: need W_pad >= W, C_pad >= C > 0, C_pad a multiple of 16");
  if (W_pad == W) return q8_quantize_pad_channels(x, (size_t)N * H * W, C, C_pad, q, out_type, z, stream);
  const size_t rows = (size_t)N * H;
  if ((!x || !z) && rows && W) return fail(Q8_ERR_INVALID_ARG, "q8_quantize_pad_image: null pointer");
  if (!(q > 0.f) || std::isinf(q)) return fail(Q8_ERR_NONFINITE, "q8_quantize_pad_image: factor must be finite and positive");
  if (out_type != Q8_U8 && out_type != Q8_S8) return fail(Q8_ERR_INVALID_ARG, "q8_quantize_pad_image: bad out_type");
  if (!aligned16(z)) return fail(Q8_ERR_ALIGNMENT, "q8_quantize_pad_image: z not 16-byte aligned");
  if (rows == 0 || W_pad == 0) return Q8_OK;
  const int lo = out_type == Q8_U8 ? 0 : -128, hi = out_type == Q8_U8 ? 255 : 127;
  const int groups = C_pad / 16;
  if (C == 3 && C_pad == 16) {
    const size_t chunks = rows * (((size_t)W_pad + 127) / 128);
    quantize_pad3_rows_kernel<<<grid_for(chunks, kPadThreads / 32, 8), kPadThreads, 0, as_stream(stream)>>>(
        x, rows, (size_t)W, (size_t)W_pad, q, lo, hi, static_cast<uint4*>(z));
    return check_launch("quantize_pad3_rows_kernel");
  }
  quantize_pad_image_kernel<<<grid_for(rows * W_pad * groups, kThreads, 8), kThreads, 0, as_stream(stream)>>>(
      x, rows, W, C, W_pad, groups, q, lo, hi, static_cast<uint4*>(z));
  return check_launch("quantize_pad_image_kernel");
}

int q8_dequantize(const void* z, int in_type, size_t n, float q, float* r, void* stream) {
  clear_error();
  if ((!z || !r) && n) return fail(Q8_ERR_INVALID_ARG, "q8_dequantize: null pointer");
  if (in_type != Q8_U8 && in_type != Q8_S8 && in_type != Q8_S32) return fail(Q8_ERR_INVALID_ARG, "q8_dequantize: bad in_type");
  if (!std::isfinite(q)) return fail(Q8_ERR_NONFINITE, "q8_dequantize: factor must be finite");
  if (n == 0) return Q8_OK;
  cudaStream_t s = as_stream(stream);
  if (in_type == Q8_S32) {
    dequantize_scalar_kernel<int><<<grid_for(n, kThreads, 8), kThreads, 0, s>>>(static_cast<const int*>(z), 0, n, q, r);
    return check_launch("dequantize32");
  }
  size_t done = 0;
  if (aligned16(z) && aligned16(r)) {
    size_t n4 = n / 4;
    if (n4) {
      int grid = grid_for(n4, kThreads * 4, 4);
      if (in_type == Q8_S8) dequantize8_vec_kernel<true><<<grid, kThreads, 0, s>>>(static_cast<const unsigned int*>(z), n4, q, reinterpret_cast<float4*>(r));
      else dequantize8_vec_kernel<false><<<grid, kThreads, 0, s>>>(static_cast<const unsigned int*>(z), n4, q, reinterpret_cast<float4*>(r));
    }
    done = n4 * 4;
  }
  if (done < n) {
    int grid = grid_for(n - done, kThreads, 8);
    if (in_type == Q8_S8) dequantize_scalar_kernel<signed char><<<grid, kThreads, 0, s>>>(static_cast<const signed char*>(z), done, n, q, r);
    else dequantize_scalar_kernel<unsigned char><<<grid, kThreads, 0, s>>>(static_cast<const unsigned char*>(z), done, n, q, r);
  }
  return check_launch("dequantize8");
}

int q8_fold_bn(const float* w, const float* b, const float* gamma, const float* beta, const float* mean,
               const float* var, double eps, int K, size_t elems_per_k, float* w_out, float* b_out, void* stream) {
  clear_error();
  if (!w || !gamma || !beta || !mean || !var || !w_out || !b_out) return fail(Q8_ERR_INVALID_ARG, "q8_fold_bn: null pointer");
  if (K <= 0 || K > 65535 || elems_per_k == 0) return fail(Q8_ERR_INVALID_ARG, "q8_fold_bn: need 0 < K <= 65535 and elems_per_k > 0");
  if (!(eps >= 0.0)) return fail(Q8_ERR_INVALID_ARG, "q8_fold_bn: eps must be >= 0");
  int chunks = (int)((elems_per_k + 255) / 256);
  if (chunks > 64) chunks = 64;
  fold_bn_kernel<<<dim3(chunks, K), 256, 0, as_stream(stream)>>>(w, b, gamma, beta, mean, var, eps, elems_per_k, w_out, b_out);
  return check_launch("fold_bn_kernel");
}

int q8_concat_branch(const void* x, int channels, float in_factor, float out_factor, int t, size_t pixels, void* y,
                     int y_ldc, int y_c_offset, void* stream) {
  clear_error();
  if (!x || !y || channels <= 0 || y_c_offset < 0 || (long long)y_c_offset + channels > (long long)y_ldc)
    return fail(Q8_ERR_INVALID_ARG, "q8_concat_branch: bad argument");
  if (t != Q8_U8 && t != Q8_S8) return fail(Q8_ERR_INVALID_ARG, "q8_concat_branch: type must be Q8_U8 or Q8_S8");
  if (!(out_factor > 0.f) || std::isinf(out_factor) || !(in_factor > 0.f) || std::isinf(in_factor))
    return fail(Q8_ERR_NONFINITE, "q8_concat_branch: factors must be finite and positive");
  if (pixels == 0) return Q8_OK;
  cudaStream_t s = as_stream(stream);
  volatile double ratio = (double)in_factor / (double)out_factor;
  float sc = (float)ratio;
  int copy_only = sc == 1.0f ? 1 : ((sc > 0.0f && sc < 1.0f) ? 2 : 0);  // 2: the clamp-free form (vector kernel)
  const int ch = channels, ctot = y_ldc, off = y_c_offset;
  bool vec = (ch % 16 == 0) && (ctot % 16 == 0) && (off % 16 == 0) && aligned16(x) && aligned16(y);
  if (vec) {
    int grid = grid_for(pixels * (ch / 16), kThreads, 4);
    if (t == Q8_S8) concat_vec_kernel<true><<<grid, kThreads, 0, s>>>(static_cast<const uint4*>(x), pixels, ch / 16, ctot / 16, off / 16, sc, copy_only, static_cast<uint4*>(y));
    else concat_vec_kernel<false><<<grid, kThreads, 0, s>>>(static_cast<const uint4*>(x), pixels, ch / 16, ctot / 16, off / 16, sc, copy_only, static_cast<uint4*>(y));
  } else {
    int grid = grid_for(pixels * ch, kThreads, 8);
    if (t == Q8_S8) concat_scalar_kernel<true><<<grid, kThreads, 0, s>>>(static_cast<const unsigned char*>(x), pixels, ch, ctot, off, sc, copy_only, static_cast<unsigned char*>(y));
    else concat_scalar_kernel<false><<<grid, kThreads, 0, s>>>(static_cast<const unsigned char*>(x), pixels, ch, ctot, off, sc, copy_only, static_cast<unsigned char*>(y));
  }
  return check_launch("concat_kernel");
}

int q8_concat(int n_in, const void* const* xs, const int* channels, const float* in_factors, float out_factor,
              int t, size_t pixels, void* y, void* stream) {
  clear_error();
  if (n_in <= 0 || n_in > 8 || !xs || !channels || !in_factors || !y) return fail(Q8_ERR_INVALID_ARG, "q8_concat: bad argument");
  if (t != Q8_U8 && t != Q8_S8) return fail(Q8_ERR_INVALID_ARG, "q8_concat: type must be Q8_U8 or Q8_S8");
  if (!(out_factor > 0.f) || std::isinf(out_factor)) return fail(Q8_ERR_NONFINITE, "q8_concat: out_factor must be finite and positive");
  long long ctot = 0;
  for (int i = 0; i < n_in; ++i) {
    if (!xs[i] || channels[i] <= 0) return fail(Q8_ERR_INVALID_ARG, "q8_concat: branch %d null or empty", i);
    if (!(in_factors[i] > 0.f) || std::isinf(in_factors[i])) return fail(Q8_ERR_NONFINITE, "q8_concat: factor %d not finite positive", i);
    ctot += channels[i];
  }
  if (ctot > 0x7fffffffLL) return fail(Q8_ERR_INVALID_ARG, "q8_concat: too many channels");
  if (pixels == 0) return Q8_OK;
  // one launch for all branches when every branch takes the 16-byte path
  bool vec = n_in > 1 && ctot % 16 == 0 && aligned16(y);
  for (int i = 0; i < n_in && vec; ++i) vec = channels[i] % 16 == 0 && aligned16(xs[i]);
  if (vec) {
    ConcatBranches br{};
    br.n = n_in;
    size_t items = pixels * (size_t)(ctot / 16);
    const unsigned int grid = (unsigned int)grid_for(items, kThreads, 4);
    unsigned int next = 0;
    int coff = 0;
    for (int i = 0; i < n_in; ++i) {
      volatile double ratio = (double)in_factors[i] / (double)out_factor;
      float sc = (float)ratio;
      br.b[i].x = static_cast<const uint4*>(xs[i]);
      br.b[i].cvec = channels[i] / 16;
      br.b[i].coff_vec = coff / 16;
      br.b[i].s = sc;
      br.b[i].mode = sc == 1.0f ? 1 : ((sc > 0.0f && sc < 1.0f) ? 2 : 0);
      br.b[i].block0 = next;
      unsigned long long share = ((unsigned long long)grid * (unsigned long long)channels[i] + ctot - 1) / ctot;
      next += (unsigned int)(share < 1 ? 1 : share);
      coff += channels[i];
    }
    br.blocks = next;
    cudaStream_t s = as_stream(stream);
    if (t == Q8_S8) concat_multi_kernel<true><<<next, kThreads, 0, s>>>(br, pixels, (int)(ctot / 16), static_cast<uint4*>(y));
    else concat_multi_kernel<false><<<next, kThreads, 0, s>>>(br, pixels, (int)(ctot / 16), static_cast<uint4*>(y));
    return check_launch("concat_multi_kernel");
  }
  int off = 0;
  for (int i = 0; i < n_in; ++i) {
    int rc = q8_concat_branch(xs[i], channels[i], in_factors[i], out_factor, t, pixels, y, (int)ctot, off, stream);
    if (rc != Q8_OK) return rc;
    off += channels[i];
  }
  return Q8_OK;
}

int q8_pool_out_extent(int H, int k, int stride, int pad, int ceil_mode, int* out) {
  clear_error();
  if (!out || H <= 0 || k <= 0 || stride <= 0 || pad < 0) return fail(Q8_ERR_INVALID_ARG, "q8_pool_out_extent: bad argument");
  *out = pool_extent(H, k, stride, pad, ceil_mode);
  return Q8_OK;
}

int q8_maxpool2d(const void* x, int t, int N, int H, int W, int C, int kh, int kw, int stride_h, int stride_w,
                 int pad_h, int pad_w, int ceil_mode, void* y, void* stream) {
  return launch_pool<false>(x, t, N, H, W, C, kh, kw, stride_h, stride_w, pad_h, pad_w, ceil_mode, y, stream);
}

int q8_avgpool2d(const void* x, int t, int N, int H, int W, int C, int kh, int kw, int stride_h, int stride_w,
                 int pad_h, int pad_w, int ceil_mode, void* y, void* stream) {
  return launch_pool<true>(x, t, N, H, W, C, kh, kw, stride_h, stride_w, pad_h, pad_w, ceil_mode, y, stream);
}

}  // extern "C"
