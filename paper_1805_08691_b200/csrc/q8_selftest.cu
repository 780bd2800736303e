// Self-test of the bounded-wait machinery the tensor-core kernels rely on: a wait that nothing will ever satisfy
// must run out, set the device status word and let the other roles of the CTA drain, instead of hanging the GPU.
// The kernel below waits on mbarriers that are initialised and never signalled: warp 0 with the caller's (short)
// limit, warp 1 with the library's normal limit, which it must leave early through the CTA's abort flag.
#include "q8_umma_common.cuh"

namespace q8 {
namespace {

__global__ void __launch_bounds__(64, 1) bounded_wait_kernel(unsigned long long limit_ns, unsigned int* status) {
  __shared__ __align__(8) unsigned long long never[2];
  __shared__ int abort_flag;
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&never[0]), 1);
    mbar_init(smem_u32(&never[1]), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  volatile int* abortp = &abort_flag;
  if (warp == 0) {
    // phase 0 of a fresh barrier never completes: no thread arrives
    const bool ok = mbar_wait_slow(smem_u32(&never[0]), 0u, abortp, limit_ns);
    if (!ok && lane == 0) {
      abort_flag = 1;
      atomicOr(status, kTimeoutProducer);
    }
  } else {
    const bool ok = mbar_wait(smem_u32(&never[1]), 0u, abortp);  // leaves when warp 0 has given up
    if (!ok && lane == 0) atomicOr(status, kTimeoutEpilogue);
  }
}

}  // namespace
}  // namespace q8

using namespace q8;

extern "C" int q8_selftest_bounded_wait(unsigned int limit_us, void* stream) {
  clear_error();
  if (limit_us < 1 || limit_us > 1000000u) return fail(Q8_ERR_INVALID_ARG, "q8_selftest_bounded_wait: limit must be 1 us .. 1 s");
  unsigned int* status = status_word_device_ptr();
  if (!status) return fail(Q8_ERR_CUDA, "q8_selftest_bounded_wait: status word not available");
  bounded_wait_kernel<<<1, 64, 0, as_stream(stream)>>>((unsigned long long)limit_us * 1000ull, status);
  return check_launch("bounded_wait_kernel");
}
