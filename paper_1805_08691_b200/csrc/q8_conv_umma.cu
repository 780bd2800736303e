// Quantized convolution as an implicit GEMM on the 5th-generation tensor cores (sm_100a).
//
//   D[M = N*P*Q pixels, Cout] (int32, in TMEM) = A[M, R*S*C] (u8/s8) x B[Cout, R*S*C]^T (s8)
//
// One CTA computes one 128 x BN output tile:
//   warp 0   : TMA producer.  A tiles come from the NHWC activation tensor through an im2col
//              tensor map (one filter tap (r,s) and one channel block per load; padding is the
//              map's zero fill, which is the exact code of 0.0 under a symmetric quantizer), or
//              through a plain 2-D tiled map for 1x1 / stride 1 / no padding.  B tiles come from
//              the KRSC weights through a 3-D tiled map.  Both land in the K-major swizzled
//              layout tcgen05.mma reads.
//   warp 1   : allocates TMEM, one lane issues tcgen05.mma.kind::i8 (128 x BN x 32 per instruction),
//              tcgen05.commit releases smem stages and finally publishes the accumulator.
//   warps 2-5: epilogue.  tcgen05.ld (one accumulator row per thread), + bias, requantise,
//              + residual, ReLU, round, clamp, 16-byte stores.
// Stages are handed over with mbarriers; every wait is bounded in wall-clock time and on expiry
// sets a bit in the library's status word instead of hanging.
#include <cuda.h>

#include <initializer_list>

#include "q8_epilogue.cuh"
#include "q8_internal.h"

namespace q8 {
namespace {

constexpr int kBM = 128;
constexpr int kUmmaThreads = 192;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s per wait

enum StatusBits : unsigned int {
  kTimeoutProducer = 1u,
  kTimeoutMma = 2u,
  kTimeoutEpilogue = 4u,
};

struct UmmaParams {
  int M, K;                  // GEMM rows (pixels) and Cout
  int PQ, Q;                 // pixels per image, output width
  int stride_h, stride_w, pad_h, pad_w, dil_h, dil_w;
  int S;                     // filter width
  int c_blocks;              // ceil(C / BK)
  int k_iters;               // R * S * c_blocks
  int stages;                // smem stages in use (<= template maximum)
  int a_im2col;              // 1: im2col tensor map, 0: 2-D tiled [M][C]
  unsigned int idesc;        // tcgen05 instruction descriptor
  const int* bias;
  const float* scale;
  int scale_count;
  const unsigned char* res;
  int res_signed, res_vec;
  float res_scale;
  void* y;
  int y_type, y_vec, ldc, c_off, relu;
  unsigned int* status;
};

// ------------------------------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// Waits for the phase with the given parity.  Gives up after kWaitLimitNs or when another role of
// this CTA has already given up; the caller then records the site and leaves its loop.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_timer_ns();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 0xffu) == 0) {
      if (*abort_flag) return false;
      if (global_timer_ns() - t0 > kWaitLimitNs) return false;
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}

// im2col load of a 4-D (C, W, H, N) tensor: `pixelsPerColumn` output pixels starting at base pixel
// (w, h, n), filter-tap offsets (off_w, off_h) added to every pixel, `channelsPerPixel` channels from c.
__device__ __forceinline__ void tma_load_im2col_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c, int w,
                                                   int h, int n, unsigned short off_w, unsigned short off_h) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h)
      : "memory");
}

__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t holder_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(holder_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}

// D[tmem] (+)= A[smem desc] * B[smem desc]^T, 8-bit integer inputs, int32 accumulate.
__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// The mbarrier gets one arrival once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 lanes x 16 consecutive 32-bit columns: thread i of the warp receives row (lane base + i).
__device__ __forceinline__ void tmem_ld_16(uint32_t taddr, int (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major operand tile whose rows are BK bytes (= one swizzle
// span): 8-row groups are 8*BK bytes apart (stride byte offset), the leading byte offset is unused
// for swizzled K-major tiles and set to 1, descriptor version 1, swizzle mode from BK.
template <int BK>
__device__ __forceinline__ uint64_t make_kmajor_desc(uint32_t smem_addr) {
  constexpr uint64_t layout = BK == 128 ? 2 : (BK == 64 ? 4 : 6);
  return (uint64_t)((smem_addr >> 4) & 0x3fffu) | (1ull << 16) | ((uint64_t)((8 * BK) >> 4) << 32) | (1ull << 46) |
         (layout << 61);
}

__device__ __forceinline__ unsigned int pack4(int a, int b, int c, int d) {
  return (unsigned int)(a & 0xff) | ((unsigned int)(b & 0xff) << 8) | ((unsigned int)(c & 0xff) << 16) |
         ((unsigned int)(d & 0xff) << 24);
}

__host__ __device__ constexpr int tmem_cols_for(int bn) { return bn <= 32 ? 32 : (bn <= 64 ? 64 : (bn <= 128 ? 128 : 256)); }

// ------------------------------------------------------------------------------------------ kernel
template <int BN, int BK, int MAX_STAGES>
__global__ void __launch_bounds__(kUmmaThreads) conv_umma_kernel(const __grid_constant__ CUtensorMap tmA,
                                                                 const __grid_constant__ CUtensorMap tmB,
                                                                 const UmmaParams p) {
  constexpr uint32_t A_BYTES = kBM * BK, B_BYTES = BN * BK, STAGE_BYTES = A_BYTES + B_BYTES;
  constexpr uint32_t TMEM_COLS = tmem_cols_for(BN);
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long full_bar[MAX_STAGES];
  __shared__ __align__(8) unsigned long long empty_bar[MAX_STAGES];
  __shared__ __align__(8) unsigned long long accum_bar;
  __shared__ uint32_t tmem_holder;
  __shared__ int abort_flag;
  __shared__ float s_scale[BN];
  __shared__ int s_bias[BN];

  const uint32_t tiles = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * kBM;
  const int n0 = blockIdx.y * BN;
  const int stages = p.stages;

  if (threadIdx.x == 0) {
    prefetch_tensormap(&tmA);
    prefetch_tensormap(&tmB);
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    mbar_init(smem_u32(&accum_bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_holder), TMEM_COLS);
    tmem_relinquish();
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_base = tmem_holder;
  volatile int* abortp = &abort_flag;

  if (threadIdx.x == 0) {
    // ------------------------------------------------------------------ TMA producer
    int w0 = 0, h0 = 0, img = 0;
    if (p.a_im2col) {
      img = m0 / p.PQ;
      const int rem = m0 - img * p.PQ;
      const int p0 = rem / p.Q, q0 = rem - p0 * p.Q;
      h0 = p0 * p.stride_h - p.pad_h;
      w0 = q0 * p.stride_w - p.pad_w;
    }
    int stage = 0;
    uint32_t phase = 0;
    int r = 0, s = 0, cb = 0;
    for (int it = 0; it < p.k_iters; ++it) {
      if (!mbar_wait(smem_u32(&empty_bar[stage]), phase ^ 1u, abortp)) {
        abort_flag = 1;
        atomicOr(p.status, kTimeoutProducer);
        break;
      }
      const uint32_t bar = smem_u32(&full_bar[stage]);
      const uint32_t a_dst = tiles + stage * STAGE_BYTES, b_dst = a_dst + A_BYTES;
      mbar_arrive_expect_tx(bar, STAGE_BYTES);
      if (p.a_im2col)
        tma_load_im2col_4d(a_dst, &tmA, bar, cb * BK, w0, h0, img, (unsigned short)(s * p.dil_w), (unsigned short)(r * p.dil_h));
      else
        tma_load_2d(a_dst, &tmA, bar, cb * BK, m0);
      tma_load_3d(b_dst, &tmB, bar, cb * BK, r * p.S + s, n0);
      if (++cb == p.c_blocks) { cb = 0; if (++s == p.S) { s = 0; ++r; } }
      if (++stage == stages) { stage = 0; phase ^= 1u; }
    }
  } else if (threadIdx.x == 32) {
    // ------------------------------------------------------------------ MMA issuer
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int it = 0; it < p.k_iters; ++it) {
      if (!mbar_wait(smem_u32(&full_bar[stage]), phase, abortp)) {
        abort_flag = 1;
        atomicOr(p.status, kTimeoutMma);
        ok = false;
        break;
      }
      tcgen05_fence_after();
      const uint32_t a_src = tiles + stage * STAGE_BYTES, b_src = a_src + A_BYTES;
      const uint64_t a_desc = make_kmajor_desc<BK>(a_src), b_desc = make_kmajor_desc<BK>(b_src);
#pragma unroll
      for (int k = 0; k < BK / 32; ++k)  // 32 bytes of K per instruction: +2 in 16-byte address units
        umma_i8(tmem_base, a_desc + 2 * k, b_desc + 2 * k, p.idesc, (it > 0 || k > 0) ? 1u : 0u);
      umma_commit(smem_u32(&empty_bar[stage]));
      if (++stage == stages) { stage = 0; phase ^= 1u; }
    }
    if (ok) umma_commit(smem_u32(&accum_bar));
  } else if (warp >= 2) {
    // ------------------------------------------------------------------ epilogue
    const int et = threadIdx.x - 64;
    for (int j = et; j < BN; j += 128) {
      const int n = n0 + j;
      s_bias[j] = (p.bias && n < p.K) ? p.bias[n] : 0;
      s_scale[j] = p.scale ? (p.scale_count == 1 ? p.scale[0] : (n < p.K ? p.scale[n] : 0.f)) : 0.f;
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");
    bool ok = mbar_wait(smem_u32(&accum_bar), 0, abortp);
    if (!ok && lane == 0) {
      abort_flag = 1;
      atomicOr(p.status, kTimeoutEpilogue);
    }
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      tcgen05_fence_after();
      const int quad = warp & 3;
      const int row = quad * 32 + lane;
      const long long m = (long long)m0 + row;
      const bool row_ok = m < p.M;
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16);
      const bool has_res = p.res != nullptr;
#pragma unroll 1
      for (int ch = 0; ch < BN / 16; ++ch) {
        int acc[16];
        __syncwarp();
        tmem_ld_16(taddr + ch * 16, acc);
        tmem_ld_wait();
        const int nb = n0 + ch * 16;
        if (!row_ok || nb >= p.K) continue;
        const int valid = min(16, p.K - nb);
#pragma unroll
        for (int j = 0; j < 16; ++j) acc[j] += s_bias[ch * 16 + j];
        const size_t o = (size_t)m * p.ldc + p.c_off + nb;
        if (p.y_type == Q8_S32) {
          int* yp = static_cast<int*>(p.y) + o;
          if (p.y_vec && valid == 16) {
#pragma unroll
            for (int j = 0; j < 4; ++j) reinterpret_cast<int4*>(yp)[j] = make_int4(acc[4 * j], acc[4 * j + 1], acc[4 * j + 2], acc[4 * j + 3]);
          } else {
            for (int j = 0; j < valid; ++j) yp[j] = acc[j];
          }
          continue;
        }
        int res[16];
        if (has_res) {
          const unsigned char* rp = p.res + (size_t)m * p.K + nb;
          if (p.res_vec && valid == 16) {
            const uint4 rv = *reinterpret_cast<const uint4*>(rp);
            const unsigned int w[4] = {rv.x, rv.y, rv.z, rv.w};
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const unsigned int b = (w[j >> 2] >> (8 * (j & 3))) & 0xffu;
              res[j] = p.res_signed ? (int)(signed char)b : (int)b;
            }
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const unsigned int b = j < valid ? rp[j] : 0u;
              res[j] = p.res_signed ? (int)(signed char)b : (int)b;
            }
          }
        }
        float v[16];
#pragma unroll
        for (int j = 0; j < 16; ++j)
          v[j] = requant_value(acc[j], s_scale[ch * 16 + j], has_res, has_res ? res[j] : 0, p.res_scale, p.relu != 0);
        if (p.y_type == Q8_F32) {
          float* yp = static_cast<float*>(p.y) + o;
          if (p.y_vec && valid == 16) {
#pragma unroll
            for (int j = 0; j < 4; ++j) reinterpret_cast<float4*>(yp)[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
          } else {
            for (int j = 0; j < valid; ++j) yp[j] = v[j];
          }
        } else {
          int z[16];
          if (p.y_type == Q8_U8) {
#pragma unroll
            for (int j = 0; j < 16; ++j) z[j] = round_clamp_u8(v[j]);
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) z[j] = round_clamp_s8(v[j]);
          }
          unsigned char* yp = static_cast<unsigned char*>(p.y) + o;
          if (valid == 16) {
            *reinterpret_cast<uint4*>(yp) = make_uint4(pack4(z[0], z[1], z[2], z[3]), pack4(z[4], z[5], z[6], z[7]),
                                                      pack4(z[8], z[9], z[10], z[11]), pack4(z[12], z[13], z[14], z[15]));
          } else {
            for (int j = 0; j < valid; ++j) yp[j] = (unsigned char)z[j];
          }
        }
      }
    }
  }

  tcgen05_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tcgen05_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ------------------------------------------------------------------------------------------ host
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
typedef CUresult (*EncodeIm2colFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const int*, const int*, cuuint32_t, cuuint32_t, const cuuint32_t*,
                                   CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);

struct DriverFns {
  EncodeTiledFn tiled = nullptr;
  EncodeIm2colFn im2col = nullptr;
  bool tried = false;
};

DriverFns& driver_fns() {
  static DriverFns f;
  if (!f.tried) {
    f.tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess && qr == cudaDriverEntryPointSuccess)
      f.tiled = reinterpret_cast<EncodeTiledFn>(p);
    p = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &p, cudaEnableDefault, &qr) == cudaSuccess && qr == cudaDriverEntryPointSuccess)
      f.im2col = reinterpret_cast<EncodeIm2colFn>(p);
  }
  return f;
}

int pick_bk(int C) {
  int best = 32, best_pad = ((C + 31) / 32) * 32;
  for (int bk : {64, 128}) {
    int padded = ((C + bk - 1) / bk) * bk;
    if (padded <= best_pad) { best = bk; best_pad = padded; }
  }
  return best;
}

int pick_bn(int K) {
  if (K <= 16) return 16;
  if (K <= 32) return 32;
  if (K <= 64) return 64;
  if (K <= 128) return 128;
  // wider tiles re-read A less often; take 256 unless it pads Cout by more than 128 would
  int pad128 = ((K + 127) / 128) * 128, pad256 = ((K + 255) / 256) * 256;
  return pad256 <= pad128 ? 256 : 128;
}

constexpr int max_stages_for(int bn, int bk) {
  int stage = (kBM + bn) * bk;
  int n = (stage > 33 * 1024 ? 196 * 1024 : 98 * 1024) / stage;
  return n < 2 ? 2 : (n > 8 ? 8 : n);
}

CUtensorMapSwizzle swizzle_for(int bk) {
  return bk == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : (bk == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
}

template <int BN, int BK>
int launch_tile(const CUtensorMap& tmA, const CUtensorMap& tmB, UmmaParams& p, cudaStream_t stream) {
  constexpr int MAXS = max_stages_for(BN, BK);
  constexpr int STAGE_BYTES = (kBM + BN) * BK;
  auto kernel = conv_umma_kernel<BN, BK, MAXS>;
  p.stages = p.k_iters < MAXS ? p.k_iters : MAXS;
  size_t dyn = (size_t)p.stages * STAGE_BYTES + 1024;  // + slack for the 1024-byte round-up
  // TMEM holds 512 columns per SM: keep (resident CTAs) x (columns per CTA) within it by making
  // each CTA large enough in shared memory that no more than 512/cols of them fit on an SM.
  const int max_ctas = 512 / tmem_cols_for(BN);
  const size_t min_dyn = (size_t)233472 / (max_ctas + 1) + 1;
  if (dyn < min_dyn) dyn = min_dyn;
  static bool configured = false;  // per instantiation
  if (!configured) {
    size_t cap = (size_t)MAXS * STAGE_BYTES + 1024;
    if (cap < min_dyn) cap = min_dyn;
    int rc = check_cuda(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cap),
                        "conv_umma: set shared memory size");
    if (rc != Q8_OK) return rc;
    configured = true;
  }
  dim3 grid((unsigned)((p.M + kBM - 1) / kBM), (unsigned)((p.K + BN - 1) / BN));
  kernel<<<grid, kUmmaThreads, dyn, stream>>>(tmA, tmB, p);
  return check_launch("conv_umma_kernel");
}

template <int BN>
int launch_bk(int bk, const CUtensorMap& tmA, const CUtensorMap& tmB, UmmaParams& p, cudaStream_t stream) {
  switch (bk) {
    case 128: return launch_tile<BN, 128>(tmA, tmB, p, stream);
    case 64: return launch_tile<BN, 64>(tmA, tmB, p, stream);
    default: return launch_tile<BN, 32>(tmA, tmB, p, stream);
  }
}

}  // namespace

bool umma_shape_eligible(const q8_conv_desc& d, const char** why) {
  const char* dummy;
  if (!why) why = &dummy;
  if (d.C % 16) { *why = "C is not a multiple of 16"; return false; }
  const bool plain = d.R == 1 && d.S == 1 && d.stride_h == 1 && d.stride_w == 1 && d.pad_h == 0 && d.pad_w == 0;
  if (!plain) {
    // im2col tensor maps: corners are 8-bit signed, tap offsets 8-bit unsigned, strides at most 8
    const int up_w = d.pad_w - (d.S - 1) * d.dil_w, up_h = d.pad_h - (d.R - 1) * d.dil_h;
    if (d.pad_w > 128 || d.pad_h > 128 || up_w < -128 || up_h < -128 || up_w > 127 || up_h > 127) { *why = "padding/dilation outside the im2col corner range"; return false; }
    if ((d.S - 1) * d.dil_w > 255 || (d.R - 1) * d.dil_h > 255) { *why = "filter extent outside the im2col offset range"; return false; }
    if (d.stride_h > 8 || d.stride_w > 8) { *why = "stride > 8"; return false; }
    if ((long long)d.N * d.H * d.W * d.C < 131072) { *why = "activation tensor smaller than 128 KiB"; return false; }
  }
  return true;
}

int launch_conv_umma(const ConvArgs& a) {
  const q8_conv_desc& d = a.d;
  DriverFns& fn = driver_fns();
  if (!fn.tiled || !fn.im2col) return fail(Q8_ERR_CUDA, "conv_umma: cuTensorMapEncode* entry points not available");
  unsigned int* status = status_word_device_ptr();
  if (!status) return fail(Q8_ERR_CUDA, "conv_umma: status word not available");

  const int BK = pick_bk(d.C), BN = pick_bn(d.K);
  const bool plain = d.R == 1 && d.S == 1 && d.stride_h == 1 && d.stride_w == 1 && d.pad_h == 0 && d.pad_w == 0;
  const CUtensorMapSwizzle swz = swizzle_for(BK);

  CUtensorMap tmA, tmB;
  CUresult cr;
  if (plain) {
    cuuint64_t dims[2] = {(cuuint64_t)d.C, (cuuint64_t)a.M};
    cuuint64_t strides[1] = {(cuuint64_t)d.C};
    cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)kBM};
    cuuint32_t estr[2] = {1, 1};
    cr = fn.tiled(&tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(a.x), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else {
    cuuint64_t dims[4] = {(cuuint64_t)d.C, (cuuint64_t)d.W, (cuuint64_t)d.H, (cuuint64_t)d.N};
    cuuint64_t strides[3] = {(cuuint64_t)d.C, (cuuint64_t)d.W * d.C, (cuuint64_t)d.H * d.W * d.C};
    int lower[2] = {-d.pad_w, -d.pad_h};
    int upper[2] = {d.pad_w - (d.S - 1) * d.dil_w, d.pad_h - (d.R - 1) * d.dil_h};
    cuuint32_t estr[4] = {1, (cuuint32_t)d.stride_w, (cuuint32_t)d.stride_h, 1};
    cr = fn.im2col(&tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(a.x), dims, strides, lower, upper,
                   (cuuint32_t)BK, (cuuint32_t)kBM, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  if (cr != CUDA_SUCCESS) return fail(Q8_ERR_CUDA, "conv_umma: activation tensor map rejected (CUresult %d)", (int)cr);
  {
    cuuint64_t dims[3] = {(cuuint64_t)d.C, (cuuint64_t)d.R * d.S, (cuuint64_t)d.K};
    cuuint64_t strides[2] = {(cuuint64_t)d.C, (cuuint64_t)d.R * d.S * d.C};
    cuuint32_t box[3] = {(cuuint32_t)BK, 1, (cuuint32_t)BN};
    cuuint32_t estr[3] = {1, 1, 1};
    cr = fn.tiled(&tmB, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<int8_t*>(a.w), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  if (cr != CUDA_SUCCESS) return fail(Q8_ERR_CUDA, "conv_umma: weight tensor map rejected (CUresult %d)", (int)cr);

  UmmaParams p;
  p.M = (int)a.M; p.K = d.K; p.PQ = a.P * a.Q; p.Q = a.Q;
  p.stride_h = d.stride_h; p.stride_w = d.stride_w; p.pad_h = d.pad_h; p.pad_w = d.pad_w; p.dil_h = d.dil_h; p.dil_w = d.dil_w;
  p.S = d.S;
  p.c_blocks = (d.C + BK - 1) / BK;
  p.k_iters = d.R * d.S * p.c_blocks;
  p.stages = 0;
  p.a_im2col = plain ? 0 : 1;
  // instruction descriptor: D = s32 (2 << 4); A format at bit 7 (0 = u8, 1 = s8); B = s8 at bit 10;
  // both operands K-major; N/8 at bit 17; M/16 at bit 24.
  p.idesc = (2u << 4) | ((d.x_type == Q8_S8 ? 1u : 0u) << 7) | (1u << 10) | ((unsigned)(BN >> 3) << 17) | ((unsigned)(kBM >> 4) << 24);
  p.bias = a.bias; p.scale = a.scale; p.scale_count = d.scale_count;
  p.res = static_cast<const unsigned char*>(a.residual);
  p.res_signed = d.res_type == Q8_S8;
  p.res_vec = a.residual && d.K % 16 == 0 && aligned16(a.residual);
  p.res_scale = a.residual_scale;
  p.y = a.y; p.y_type = d.y_type; p.ldc = a.ldc; p.c_off = a.c_off; p.relu = d.relu;
  p.y_vec = (d.y_type == Q8_F32 || d.y_type == Q8_S32) ? (aligned16(a.y) && a.ldc % 4 == 0 && a.c_off % 4 == 0) : 1;
  p.status = status;

  switch (BN) {
    case 16: return launch_bk<16>(BK, tmA, tmB, p, a.stream);
    case 32: return launch_bk<32>(BK, tmA, tmB, p, a.stream);
    case 64: return launch_bk<64>(BK, tmA, tmB, p, a.stream);
    case 128: return launch_bk<128>(BK, tmA, tmB, p, a.stream);
    default: return launch_bk<256>(BK, tmA, tmB, p, a.stream);
  }
}

}  // namespace q8
