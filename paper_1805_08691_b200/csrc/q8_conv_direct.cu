// Direct quantized convolution on CUDA cores: any shape, any alignment.
//
// Used for shapes the tensor-core kernel does not take (channel counts that are not a multiple
// of 16, unaligned pointers, very small inputs).  One thread per output element; consecutive
// threads take consecutive output channels of one pixel, so the activation reads are warp
// broadcasts and the stores are contiguous.
#include "q8_epilogue.cuh"
#include "q8_internal.h"

namespace q8 {
namespace {

struct DirectParams {
  int N, H, W, C, K, R, S, st_h, st_w, pad_h, pad_w, dil_h, dil_w, P, Q;
  int x_signed, res_signed, y_type, relu, scale_count, ldc, c_off;
  long long total;  // N*P*Q*K
  const unsigned char* x;
  const signed char* w;
  const int* bias;
  const float* scale;
  const unsigned char* res;
  float res_scale;
  void* y;
};

__global__ void __launch_bounds__(256) conv_direct_kernel(const DirectParams p) {
  const long long nthreads = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < p.total; i += nthreads) {
    const int k = (int)(i % p.K);
    const long long m = i / p.K;
    const int q = (int)(m % p.Q);
    const long long t = m / p.Q;
    const int pp = (int)(t % p.P);
    const int n = (int)(t / p.P);
    int acc = 0;
    for (int r = 0; r < p.R; ++r) {
      const int h = pp * p.st_h - p.pad_h + r * p.dil_h;
      if (h < 0 || h >= p.H) continue;
      for (int s = 0; s < p.S; ++s) {
        const int ww = q * p.st_w - p.pad_w + s * p.dil_w;
        if (ww < 0 || ww >= p.W) continue;
        const unsigned char* xp = p.x + (((size_t)n * p.H + h) * p.W + ww) * p.C;
        const signed char* wp = p.w + (((size_t)k * p.R + r) * p.S + s) * p.C;
        if (p.x_signed) {
          for (int c = 0; c < p.C; ++c) acc += (int)(signed char)xp[c] * (int)wp[c];
        } else {
          for (int c = 0; c < p.C; ++c) acc += (int)xp[c] * (int)wp[c];
        }
      }
    }
    if (p.bias) acc += p.bias[k];
    const size_t o = (size_t)m * p.ldc + p.c_off + k;
    if (p.y_type == Q8_S32) {
      static_cast<int*>(p.y)[o] = acc;
      continue;
    }
    int res = 0;
    if (p.res) {
      unsigned char rb = p.res[(size_t)m * p.K + k];
      res = p.res_signed ? (int)(signed char)rb : (int)rb;
    }
    const float v = requant_value(acc, p.scale[p.scale_count == 1 ? 0 : k], p.res != nullptr, res, p.res_scale, p.relu != 0);
    if (p.y_type == Q8_F32) static_cast<float*>(p.y)[o] = v;
    else if (p.y_type == Q8_U8) static_cast<unsigned char*>(p.y)[o] = (unsigned char)round_clamp_u8(v);
    else static_cast<signed char*>(p.y)[o] = (signed char)round_clamp_s8(v);
  }
}

}  // namespace

int launch_conv_direct(const ConvArgs& a) {
  DirectParams p;
  const q8_conv_desc& d = a.d;
  p.N = d.N; p.H = d.H; p.W = d.W; p.C = d.C; p.K = d.K; p.R = d.R; p.S = d.S;
  p.st_h = d.stride_h; p.st_w = d.stride_w; p.pad_h = d.pad_h; p.pad_w = d.pad_w; p.dil_h = d.dil_h; p.dil_w = d.dil_w;
  p.P = a.P; p.Q = a.Q;
  p.x_signed = d.x_type == Q8_S8; p.res_signed = d.res_type == Q8_S8; p.y_type = d.y_type; p.relu = d.relu;
  p.scale_count = d.scale_count; p.ldc = a.ldc; p.c_off = a.c_off;
  p.total = a.M * d.K;
  p.x = static_cast<const unsigned char*>(a.x); p.w = reinterpret_cast<const signed char*>(a.w);
  p.bias = a.bias; p.scale = a.scale; p.res = static_cast<const unsigned char*>(a.residual);
  p.res_scale = a.residual_scale; p.y = a.y;
  long long blocks = (p.total + 255) / 256;
  if (blocks > 148ll * 64) blocks = 148ll * 64;
  conv_direct_kernel<<<(int)blocks, 256, 0, a.stream>>>(p);
  return check_launch("conv_direct_kernel");
}

}  // namespace q8
