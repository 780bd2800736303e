// Host entry points of libq8 that are not tied to one kernel file: errors, status word,
// descriptor validation and dispatch of q8_conv2d.
#include <atomic>
#include <cstdio>
#include <cstring>

#include "q8_internal.h"

namespace q8 {

namespace {
thread_local char g_last_error[512] = "";
__device__ unsigned int g_status_word = 0;
}  // namespace

int fail(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_last_error, sizeof(g_last_error), fmt, ap);
  va_end(ap);
  return code;
}

void clear_error() { g_last_error[0] = '\0'; }

int check_cuda(cudaError_t e, const char* what) {
  if (e == cudaSuccess) return Q8_OK;
  return fail(Q8_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

int check_launch(const char* kernel) { return check_cuda(cudaGetLastError(), kernel); }

int current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
  return dev;
}

int sm_count() {
  static std::atomic<int> cached[kMaxDevices];  // zero-initialised; racing threads store the same value
  const int dev = current_device();
  int n = dev >= 0 ? cached[dev].load(std::memory_order_relaxed) : 0;
  if (n == 0) {
    int cur = 0;
    if (cudaGetDevice(&cur) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, cur) != cudaSuccess || n <= 0) n = 148;
    if (dev >= 0) cached[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}

unsigned int* status_word_device_ptr() {
  // One lookup per device; the symbol address is a device address obtained from the runtime.
  static thread_local int cached_dev = -1;
  static thread_local unsigned int* cached_ptr = nullptr;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
  if (dev != cached_dev) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_status_word) != cudaSuccess) return nullptr;
    cached_ptr = static_cast<unsigned int*>(p);
    cached_dev = dev;
  }
  return cached_ptr;
}

namespace {

int validate_desc(const q8_conv_desc* d, int* P, int* Q) {
  if (!d) return fail(Q8_ERR_INVALID_ARG, "conv: null descriptor");
  if (d->N <= 0 || d->H <= 0 || d->W <= 0 || d->C <= 0 || d->K <= 0 || d->R <= 0 || d->S <= 0)
    return fail(Q8_ERR_INVALID_ARG, "conv: extents must be positive");
  if (d->stride_h <= 0 || d->stride_w <= 0 || d->dil_h <= 0 || d->dil_w <= 0 || d->pad_h < 0 || d->pad_w < 0)
    return fail(Q8_ERR_INVALID_ARG, "conv: stride/dilation must be positive, padding non-negative");
  if (d->x_type != Q8_U8 && d->x_type != Q8_S8) return fail(Q8_ERR_INVALID_ARG, "conv: x_type must be Q8_U8 or Q8_S8");
  if (d->y_type < Q8_U8 || d->y_type > Q8_F32) return fail(Q8_ERR_INVALID_ARG, "conv: bad y_type");
  if (d->res_type != Q8_U8 && d->res_type != Q8_S8) return fail(Q8_ERR_INVALID_ARG, "conv: res_type must be Q8_U8 or Q8_S8");
  if (d->scale_count != 1 && d->scale_count != d->K) return fail(Q8_ERR_INVALID_ARG, "conv: scale_count must be 1 or K");
  if (d->algo < Q8_ALGO_AUTO || d->algo > Q8_ALGO_DIRECT) return fail(Q8_ERR_INVALID_ARG, "conv: bad algo");
  // |x| <= 255, |w| <= 128: R*S*C terms stay inside int32 up to floor(2^31 / (255*128))
  if ((long long)d->R * d->S * d->C > 65793) return fail(Q8_ERR_INVALID_ARG, "conv: R*S*C > 65793 could overflow the int32 accumulator");
  int p = conv_out_extent(d->H, d->pad_h, d->dil_h, d->R, d->stride_h);
  int q = conv_out_extent(d->W, d->pad_w, d->dil_w, d->S, d->stride_w);
  if (p <= 0 || q <= 0) return fail(Q8_ERR_INVALID_ARG, "conv: empty output");
  if ((long long)d->N * p * q > 0x7fffffffll - 256) return fail(Q8_ERR_INVALID_ARG, "conv: N*P*Q too large");
  int ldc = d->y_ldc == 0 ? d->K : d->y_ldc;
  if (d->y_c_offset < 0 || ldc < d->y_c_offset + d->K) return fail(Q8_ERR_INVALID_ARG, "conv: y_ldc < y_c_offset + K");
  *P = p;
  *Q = q;
  return Q8_OK;
}

}  // namespace
}  // namespace q8

using namespace q8;

extern "C" {

const char* q8_version(void) { return "q8 0.1 (sm_100a)"; }

const char* q8_last_error(void) { return g_last_error; }

int q8_read_status(void* stream) {
  clear_error();
  int rc = check_cuda(cudaStreamSynchronize(as_stream(stream)), "q8_read_status: synchronize");
  if (rc != Q8_OK) return rc;
  unsigned int* dptr = status_word_device_ptr();
  if (!dptr) return fail(Q8_ERR_CUDA, "q8_read_status: no status word on this device");
  unsigned int host = 0;
  rc = check_cuda(cudaMemcpy(&host, dptr, sizeof(host), cudaMemcpyDeviceToHost), "q8_read_status: read");
  if (rc != Q8_OK) return rc;
  if (host != 0) {
    unsigned int zero = 0;
    cudaMemcpy(dptr, &zero, sizeof(zero), cudaMemcpyHostToDevice);
    return fail(Q8_ERR_TIMEOUT, "a kernel gave up on a bounded wait (site mask 0x%x)", host);
  }
  return Q8_OK;
}

int q8_conv2d_workspace_bytes(const q8_conv_desc* d, size_t* bytes) {
  clear_error();
  int P, Q;
  int rc = validate_desc(d, &P, &Q);
  if (rc != Q8_OK) return rc;
  if (!bytes) return fail(Q8_ERR_INVALID_ARG, "q8_conv2d_workspace_bytes: null pointer");
  *bytes = 0;
  if (d->algo != Q8_ALGO_DIRECT && d->y_type != Q8_S32) {
    const long long M = (long long)d->N * P * Q;
    const int splits = umma_plan_splits(*d, P, Q, M);
    if (splits > 1) *bytes = (size_t)splits * (size_t)M * (size_t)d->K * sizeof(int32_t);
  }
  return Q8_OK;
}

int q8_conv2d_query_algo(const q8_conv_desc* d, int* algo) {
  clear_error();
  int P, Q;
  int rc = validate_desc(d, &P, &Q);
  if (rc != Q8_OK) return rc;
  if (!algo) return fail(Q8_ERR_INVALID_ARG, "q8_conv2d_query_algo: null pointer");
  const char* why = nullptr;
  if (d->algo == Q8_ALGO_DIRECT) *algo = Q8_ALGO_DIRECT;
  else *algo = umma_shape_eligible(*d, &why) ? Q8_ALGO_UMMA : Q8_ALGO_DIRECT;
  return Q8_OK;
}

int q8_conv2d(const q8_conv_desc* d, const void* x, const int8_t* w, const int32_t* bias, const float* scale,
              const void* residual, float residual_scale, void* y, void* workspace, size_t workspace_bytes,
              void* stream) {
  clear_error();
  ConvArgs a;
  int rc = validate_desc(d, &a.P, &a.Q);
  if (rc != Q8_OK) return rc;
  if (!x || !w || !y) return fail(Q8_ERR_INVALID_ARG, "q8_conv2d: null x, w or y");
  if (!scale && d->y_type != Q8_S32) return fail(Q8_ERR_INVALID_ARG, "q8_conv2d: null scale");
  a.d = *d;
  a.M = (long long)d->N * a.P * a.Q;
  a.x = x; a.w = w; a.bias = bias; a.scale = scale;
  a.residual = d->y_type == Q8_S32 ? nullptr : residual;
  a.residual_scale = residual_scale;
  a.y = y;
  a.ldc = d->y_ldc == 0 ? d->K : d->y_ldc;
  a.c_off = d->y_c_offset;
  a.workspace = workspace; a.workspace_bytes = workspace_bytes;
  a.stream = as_stream(stream);

  if (d->algo == Q8_ALGO_DIRECT) return launch_conv_direct(a);
  const char* why = "";
  bool ok = umma_shape_eligible(*d, &why);
  if (ok) {
    const bool out8 = d->y_type == Q8_U8 || d->y_type == Q8_S8;
    if (!aligned16(x) || !aligned16(w)) { ok = false; why = "x or w not 16-byte aligned"; }
    else if (out8 && (!aligned16(y) || a.ldc % 16 || a.c_off % 16)) { ok = false; why = "8-bit output needs y, y_ldc, y_c_offset aligned to 16"; }
    else if (a.residual && !aligned16(a.residual)) { ok = false; why = "residual not 16-byte aligned"; }
  }
  if (!ok) {
    if (d->algo == Q8_ALGO_UMMA) return fail(Q8_ERR_UNSUPPORTED, "q8_conv2d: tensor-core kernel not eligible: %s", why);
    return launch_conv_direct(a);
  }
  return launch_conv_umma(a);
}

int q8_conv2d_then_1x1_supported(const q8_conv_desc* d1, const q8_conv_desc* d2, int* supported) {
  clear_error();
  int P, Q;
  int rc = validate_desc(d1, &P, &Q);
  if (rc != Q8_OK) return rc;
  rc = validate_desc(d2, &P, &Q);
  if (rc != Q8_OK) return rc;
  if (!supported) return fail(Q8_ERR_INVALID_ARG, "q8_conv2d_then_1x1_supported: null pointer");
  const char* why = "";
  *supported = (d1->algo != Q8_ALGO_DIRECT && d2->algo != Q8_ALGO_DIRECT && fused_pair_eligible(*d1, *d2, &why)) ? 1 : 0;
  return Q8_OK;
}

int q8_conv2d_then_1x1(const q8_conv_desc* d1, const q8_conv_desc* d2, const void* x, const int8_t* w1, const int32_t* bias1,
                       const float* scale1, const int8_t* w2, const int32_t* bias2, const float* scale2,
                       const void* residual, float residual_scale, void* y, void* stream) {
  clear_error();
  int P, Q;
  int rc = validate_desc(d1, &P, &Q);
  if (rc != Q8_OK) return rc;
  rc = validate_desc(d2, &P, &Q);
  if (rc != Q8_OK) return rc;
  if (!x || !w1 || !w2 || !y || !scale1 || !scale2) return fail(Q8_ERR_INVALID_ARG, "q8_conv2d_then_1x1: null x, w1, w2, y, scale1 or scale2");
  if (!aligned16(x) || !aligned16(w1) || !aligned16(w2) || !aligned16(y))
    return fail(Q8_ERR_UNSUPPORTED, "q8_conv2d_then_1x1: x, w1, w2 and y must be 16-byte aligned");
  return launch_conv_fused(*d1, *d2, x, w1, bias1, scale1, w2, bias2, scale2, residual, residual_scale, y, as_stream(stream));
}

}  // extern "C"
