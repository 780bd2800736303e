// Second pass of a split-K convolution: sums the int32 partial accumulators the tensor-core kernel wrote
// into the workspace ([split][M][K], exact integer addition), adds the bias and applies the same epilogue
// as the fused path: requantise, + residual, ReLU, round, clamp, store (u8 / s8 / fp32), optionally into a
// channel slice of a wider tensor.
#include "q8_epilogue.cuh"
#include "q8_internal.h"

namespace q8 {
namespace {

struct ReduceParams {
  const int* ws;
  long long split_stride;  // M * K
  int splits;
  long long M;
  int K;
  const int* bias;
  const float* scale;
  int scale_count;
  const unsigned char* res;
  int res_signed;
  float res_scale;
  void* y;
  int y_type, ldc, c_off, relu;
};

// One thread per four consecutive channels of one pixel (K % 4 == 0): 16-byte loads of the partial sums.
template <int kVec>
__global__ void __launch_bounds__(256) splitk_reduce_kernel(const ReduceParams p) {
  const int kg = p.K / kVec;
  const long long total = p.M * kg;
  const long long nthreads = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += nthreads) {
    const long long m = i / kg;
    const int k0 = (int)(i - m * kg) * kVec;
    int acc[kVec];
#pragma unroll
    for (int j = 0; j < kVec; ++j) acc[j] = p.bias ? p.bias[k0 + j] : 0;
    const int* src = p.ws + m * p.K + k0;
    for (int sp = 0; sp < p.splits; ++sp, src += p.split_stride) {
      if (kVec == 4) {
        const int4 v = *reinterpret_cast<const int4*>(src);
        acc[0] += v.x; acc[1] += v.y; acc[2] += v.z; acc[3] += v.w;
      } else {
        acc[0] += src[0];
      }
    }
    const size_t o = (size_t)m * p.ldc + p.c_off + k0;
#pragma unroll
    for (int j = 0; j < kVec; ++j) {
      int r = 0;
      if (p.res) {
        const unsigned char rb = p.res[(size_t)m * p.K + k0 + j];
        r = p.res_signed ? (int)(signed char)rb : (int)rb;
      }
      const float v = requant_value(acc[j], p.scale[p.scale_count == 1 ? 0 : k0 + j], p.res != nullptr, r, p.res_scale, p.relu != 0);
      if (p.y_type == Q8_F32) static_cast<float*>(p.y)[o + j] = v;
      else if (p.y_type == Q8_U8) static_cast<unsigned char*>(p.y)[o + j] = (unsigned char)round_clamp_u8(v);
      else static_cast<signed char*>(p.y)[o + j] = (signed char)round_clamp_s8(v);
    }
  }
}

}  // namespace

int launch_splitk_reduce(const ConvArgs& a, int splits) {
  ReduceParams p;
  p.ws = static_cast<const int*>(a.workspace);
  p.split_stride = a.M * a.d.K;
  p.splits = splits;
  p.M = a.M;
  p.K = a.d.K;
  p.bias = a.bias;
  p.scale = a.scale;
  p.scale_count = a.d.scale_count;
  p.res = static_cast<const unsigned char*>(a.residual);
  p.res_signed = a.d.res_type == Q8_S8;
  p.res_scale = a.residual_scale;
  p.y = a.y;
  p.y_type = a.d.y_type;
  p.ldc = a.ldc;
  p.c_off = a.c_off;
  p.relu = a.d.relu;
  const bool vec = a.d.K % 4 == 0;
  const long long items = a.M * (vec ? a.d.K / 4 : a.d.K);
  long long blocks = (items + 255) / 256;
  if (blocks > 148ll * 8) blocks = 148ll * 8;
  if (vec) splitk_reduce_kernel<4><<<(int)blocks, 256, 0, a.stream>>>(p);
  else splitk_reduce_kernel<1><<<(int)blocks, 256, 0, a.stream>>>(p);
  return check_launch("splitk_reduce_kernel");
}

}  // namespace q8
