// Requantisation epilogue shared by the convolution kernels (device side).
//
//   v = float(acc) * s;  v += float(res) * s_res;  v = max(v,0);  y = clamp(Round(v))
//
// Each step is one IEEE fp32 operation (explicit _rn intrinsics, never contracted into an FMA),
// the int->float conversion and the final rounding are round-to-nearest-even.
#pragma once
#include <cstdint>

namespace q8 {

__device__ __forceinline__ float requant_value(int acc, float s, bool has_res, int res, float s_res, bool relu) {
  float v = __fmul_rn(__int2float_rn(acc), s);
  if (has_res) v = __fadd_rn(v, __fmul_rn(__int2float_rn(res), s_res));
  if (relu) v = v > 0.0f ? v : 0.0f;
  return v;
}

__device__ __forceinline__ int round_clamp_u8(float v) { return min(max(__float2int_rn(v), 0), 255); }
__device__ __forceinline__ int round_clamp_s8(float v) { return min(max(__float2int_rn(v), -128), 127); }

}  // namespace q8
