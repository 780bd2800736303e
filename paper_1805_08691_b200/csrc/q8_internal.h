// Internal declarations shared by the translation units of libq8 (host side).
#pragma once

#include <cuda_runtime.h>

#include <cstdarg>
#include <cstddef>
#include <cstdint>

#include "q8.h"

namespace q8 {

// Records the message returned by q8_last_error() on this thread and returns `code`.
int fail(int code, const char* fmt, ...);
void clear_error();

// Returns Q8_OK or records the CUDA error text and returns Q8_ERR_CUDA.
int check_cuda(cudaError_t e, const char* what);
int check_launch(const char* kernel);

// Device status word (bit mask of timeout sites), zero when healthy.
unsigned int* status_word_device_ptr();

// Host-side caches are kept per device (function attributes, the SM count and symbol addresses belong to a
// device, and one process may drive several from several threads).
constexpr int kMaxDevices = 64;
// Index of the current device, or -1 if it cannot be read or is not below kMaxDevices (callers then skip their cache).
int current_device();
// Multiprocessor count of the current device (148 if it cannot be read).
int sm_count();

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline int conv_out_extent(int H, int pad, int dil, int R, int stride) {
  return (H + 2 * pad - dil * (R - 1) - 1) / stride + 1;
}

struct ConvArgs {
  q8_conv_desc d;
  int P, Q;
  long long M;  // N*P*Q
  const void* x;
  const int8_t* w;
  const int32_t* bias;
  const float* scale;
  const void* residual;
  float residual_scale;
  void* y;
  int ldc, c_off;
  void* workspace;
  size_t workspace_bytes;
  cudaStream_t stream;
};

// Eligibility of the tensor-core kernel for a descriptor (pointer alignment checked at launch).
bool umma_shape_eligible(const q8_conv_desc& d, const char** why);
int launch_conv_umma(const ConvArgs& a);
// Number of split-K parts the tensor-core kernel uses for this layer when it is given a workspace of
// splits * M * K int32 (1: none).  Host only.
int umma_plan_splits(const q8_conv_desc& d, int P, int Q, long long M);
// Sums the split-K partial accumulators in a.workspace, adds the bias and applies the epilogue of `a`.
int launch_splitk_reduce(const ConvArgs& a, int splits);
int launch_conv_direct(const ConvArgs& a);
// A stride-1 convolution followed by a 1x1 convolution over its output, in one launch (q8_conv_fused.cu).
// Descriptors validated by the caller; `why` names the first reason a pair cannot run fused.
bool fused_pair_eligible(const q8_conv_desc& d1, const q8_conv_desc& d2, const char** why);
int launch_conv_fused(const q8_conv_desc& d1, const q8_conv_desc& d2, const void* x, const int8_t* w1, const int32_t* bias1,
                      const float* scale1, const int8_t* w2, const int32_t* bias2, const float* scale2, const void* residual,
                      float residual_scale, void* y, cudaStream_t stream);

}  // namespace q8
