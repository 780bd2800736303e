// Issue-rate probe of the int8 tensor-core instruction the convolution kernels are built on
// (tcgen05.mma.cta_group::1.kind::i8, 128 x bn x 32 per instruction, operands in shared memory, int32
// accumulators in TMEM).  It is the measured stand-in for the "int8 tensor peak" in the roofline of the
// quantized convolution: one CTA per SM issues `instructions` MMAs back to back from one lane, cycling over
// `chains` accumulators (1 = every instruction depends on the one before it through its accumulator), and
// reports the SM cycles from the first issue to the completion of the last.
#include "q8_umma_common.cuh"

namespace q8 {
namespace {

__global__ void __launch_bounds__(128, 1) mma_rate_kernel(int bn, int chains, int instructions, unsigned long long* cycles,
                                                          unsigned int* status) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long done_bar;
  __shared__ uint32_t tmem_holder;
  __shared__ int abort_flag;
  const uint32_t raw_base = smem_u32(smem_raw);
  const uint32_t base = (raw_base + 1023u) & ~1023u;
  unsigned char* const base_ptr = smem_raw + (base - raw_base);
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  // operands: A = 128 rows x 128 bytes, B = bn rows x 128 bytes (K-major, 128-byte swizzle); all zero
  const int bytes = (kBM + bn) * 128;
  for (int i = threadIdx.x * 16; i < bytes; i += blockDim.x * 16) *reinterpret_cast<uint4*>(base_ptr + i) = make_uint4(0u, 0u, 0u, 0u);
  fence_proxy_async_smem();
  if (warp == 0) {
    if (lane == 0) { mbar_init(smem_u32(&done_bar), 1); abort_flag = 0; }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncwarp();
    tmem_alloc(smem_u32(&tmem_holder), 512u);
    tmem_relinquish();
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_base = tmem_holder;
  if (warp == 0) {
    const uint64_t hi = ((uint64_t)((unsigned)((8 * 128) >> 4) | (1u << 14) | (2u << 29)) << 32) | (1ull << 16);
    const uint64_t a_d = hi | ((base >> 4) & 0x3fffu), b_d = hi | (((base + kBM * 128) >> 4) & 0x3fffu);
    const uint32_t idesc = (2u << 4) | (1u << 10) | ((unsigned)(bn >> 3) << 17) | ((unsigned)(kBM >> 4) << 24);
    const uint32_t stride = bn < 32 ? 32u : (uint32_t)bn;
    const long long t0 = clock64();
    if (lane == 0) {
      int chain = 0;
      for (int i = 0; i < instructions; ++i) {
        const uint32_t k = (uint32_t)(i & 3) * 2u;
        umma_i8(tmem_base + (uint32_t)chain * stride, a_d + k, b_d + k, idesc, i >= chains ? 1u : 0u);
        if (++chain == chains) chain = 0;
      }
      umma_commit(smem_u32(&done_bar));
    }
    __syncwarp();
    const bool ok = mbar_wait(smem_u32(&done_bar), 0u, &abort_flag);
    const long long t1 = clock64();
    if (lane == 0) {
      cycles[blockIdx.x] = (unsigned long long)(t1 - t0);
      if (!ok) atomicOr(status, kTimeoutMma);
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 0) {
    tcgen05_fence_after();
    tmem_dealloc(tmem_base, 512u);
  }
}

}  // namespace
}  // namespace q8

using namespace q8;

extern "C" int q8_int8_mma_rate(int bn, int chains, int instructions, int ctas, unsigned long long* cycles_dev, void* stream) {
  clear_error();
  if (bn < 16 || bn > 256 || bn % 16) return fail(Q8_ERR_INVALID_ARG, "q8_int8_mma_rate: bn must be a multiple of 16 in [16, 256]");
  if (chains < 1 || chains * (bn < 32 ? 32 : bn) > 512) return fail(Q8_ERR_INVALID_ARG, "q8_int8_mma_rate: chains * bn must fit 512 TMEM columns");
  if (instructions < 1 || instructions > (1 << 24) || ctas < 1 || ctas > 65535) return fail(Q8_ERR_INVALID_ARG, "q8_int8_mma_rate: bad instruction or CTA count");
  if (!cycles_dev) return fail(Q8_ERR_INVALID_ARG, "q8_int8_mma_rate: null result buffer");
  unsigned int* status = status_word_device_ptr();
  if (!status) return fail(Q8_ERR_CUDA, "q8_int8_mma_rate: status word not available");
  const size_t dyn = 1024 + (size_t)(kBM + bn) * 128;
  static std::atomic<bool> configured[kMaxDevices];
  const int dev = current_device();
  if (dev < 0 || !configured[dev].load(std::memory_order_acquire)) {
    int rc = check_cuda(cudaFuncSetAttribute(mma_rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 1024 + (kBM + 256) * 128),
                        "q8_int8_mma_rate: set shared memory size");
    if (rc != Q8_OK) return rc;
    if (dev >= 0) configured[dev].store(true, std::memory_order_release);
  }
  mma_rate_kernel<<<ctas, 128, dyn, as_stream(stream)>>>(bn, chains, instructions, cycles_dev, status);
  return check_launch("mma_rate_kernel");
}
