// q8_conv2d_static_workspace: the split-K convolution for callers that may not allocate device memory.
//
// Some hosts of this library cannot hand q8_conv2d a workspace: a plug-in inside an inference server
// whose device memory was budgeted and handed out before the plug-in was loaded, a real-time loop in
// which cudaMalloc is forbidden because it synchronises the whole device, code that runs while another
// component owns the allocator.  For them the partial sums of the split reduction live in a fixed array
// that is part of the library image.  The price: every GPU that loads the library carries the array until
// the process exits, the size is capped, and all calls share it.
#include <atomic>

#include "q8_internal.h"

namespace q8 {
namespace {

constexpr size_t kStaticWorkspaceBytes = 16u << 20;  // 16 MiB, see q8_static_workspace_bytes()

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress, never an
// address a kernel may be given.
static __device__ __align__(256) unsigned char g_static_workspace[kStaticWorkspaceBytes];

// Device address of the array on each device, looked up once per device with that device current.  Two threads
// that make the first call on a device at the same time both look the address up and store the same value.
std::atomic<void*> g_static_workspace_ptr[kMaxDevices];

int static_workspace(void** ptr) {
  int dev = 0;
  int rc = check_cuda(cudaGetDevice(&dev), "q8_conv2d_static_workspace: cudaGetDevice");
  if (rc != Q8_OK) return rc;
  if (dev < 0 || dev >= kMaxDevices) return fail(Q8_ERR_UNSUPPORTED, "q8_conv2d_static_workspace: device index %d not supported", dev);
  void* p = g_static_workspace_ptr[dev].load(std::memory_order_acquire);
  if (!p) {
    // With lazy module loading (the CUDA default) this lookup is also the moment the device sets the 16 MiB
    // aside, together with the library's kernel images.
    rc = check_cuda(cudaGetSymbolAddress((void**)&p, g_static_workspace), "q8_conv2d_static_workspace: cudaGetSymbolAddress");
    if (rc != Q8_OK) return rc;
    g_static_workspace_ptr[dev].store(p, std::memory_order_release);
  }
  *ptr = p;
  return Q8_OK;
}

}  // namespace
}  // namespace q8

using namespace q8;

extern "C" {

size_t q8_static_workspace_bytes(void) {
  // Also the set-up call: looks the array up on the current device, so that a host can pay for it (and have the
  // device set the memory aside) at a moment of its choosing.  Without a usable device only the size is returned.
  void* ws = nullptr;
  if (static_workspace(&ws) != Q8_OK) clear_error();
  return kStaticWorkspaceBytes;
}

int q8_conv2d_static_workspace(const q8_conv_desc* d, const void* x, const int8_t* w, const int32_t* bias,
                               const float* scale, const void* residual, float residual_scale, void* y,
                               void* stream) {
  size_t need = 0;
  int rc = q8_conv2d_workspace_bytes(d, &need);  // validates the descriptor
  if (rc != Q8_OK) return rc;
  if (need > kStaticWorkspaceBytes)
    return fail(Q8_ERR_WORKSPACE,
                "q8_conv2d_static_workspace: this layer's split reduction needs %zu bytes of scratch, the built-in "
                "workspace holds %zu; use q8_conv2d with a caller-provided workspace (or none)",
                need, kStaticWorkspaceBytes);
  void* ws = nullptr;
  rc = static_workspace(&ws);
  if (rc != Q8_OK) return rc;
  // Nothing in the array has to be cleared between calls: every partial sum of a layer is written by
  // the first kernel before the second one reads it.
  return q8_conv2d(d, x, w, bias, scale, residual, residual_scale, y, ws, need, stream);
}

}  // extern "C"
