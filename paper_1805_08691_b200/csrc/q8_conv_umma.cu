// Quantized convolution as an implicit GEMM on the 5th-generation tensor cores (sm_100a).
//
//   D[M = N*P*Q pixels, Cout] (int32, in TMEM) = A[M, R*S*C] (u8/s8) x B[Cout, R*S*C]^T (s8)
//
// Persistent kernel: one CTA per SM walks over 128 x BN output tiles.
//   warp 0    : TMA producer.  A tiles come from the NHWC activation tensor through an im2col tensor
//               map (one filter tap (r,s) and one channel block per load; padding is the map's zero
//               fill, the exact code of 0.0 under a symmetric quantizer) or, for 1x1 / stride 1 / no
//               padding, through a 2-D tiled map.  B tiles come from the KRSC weights through a 3-D
//               tiled map.  Both land in the K-major swizzled layout tcgen05.mma reads.  The residual
//               tile of the fused eltwise sum is fetched by TMA as well, ahead of its epilogue.
//   warp 1    : allocates TMEM (two accumulator buffers), one lane issues tcgen05.mma.kind::i8
//               (128 x BN x 32 per instruction); tcgen05.commit releases smem stages and publishes
//               each finished accumulator.
//   warps 2-9 : epilogue.  tcgen05.ld (one accumulator row per thread), + bias, requantise,
//               + residual, ReLU, round, clamp, into a swizzled smem tile that one thread hands to a
//               TMA store.  The epilogue of tile i overlaps the loads and MMAs of tile i+1.
// Every mbarrier wait is bounded in wall-clock time; on expiry a bit of the library's status word
// is set and all roles drain instead of hanging.
#include <cuda.h>

#include <cstring>
#include <initializer_list>

#include "q8_epilogue.cuh"
#include "q8_internal.h"

namespace q8 {
namespace {

constexpr int kBM = 128;
constexpr int kEpiWarps = 8;
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kUmmaThreads = 64 + kEpiThreads;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s per wait
constexpr int kSmemLimit = 232448;                           // 227 KiB opt-in maximum per CTA
constexpr int kStaticSmemReserve = 4096;                     // barriers, bias/scale staging

enum StatusBits : unsigned int {
  kTimeoutProducer = 1u,
  kTimeoutMma = 2u,
  kTimeoutEpilogue = 4u,
};

enum ResMode : int { kResNone = 0, kResTma = 1, kResGlobal = 2 };

struct UmmaParams {
  int M, K;                  // GEMM rows (pixels) and Cout
  int PQ, Q;                 // pixels per image, output width
  int stride_h, stride_w, pad_h, pad_w, dil_h, dil_w;
  int S;                     // filter width
  int c_blocks;              // ceil(C / BK)
  int k_iters;               // R * S * c_blocks
  int stages;                // smem stages in use (<= template maximum)
  int m_tiles, n_tiles;
  int a_im2col;              // 1: im2col tensor map, 0: 2-D tiled [M][C]
  unsigned int idesc;        // tcgen05 instruction descriptor
  const int* bias;
  const float* scale;
  int scale_count;
  const unsigned char* res;
  int res_mode, res_signed;
  float res_scale;
  void* y;
  int y_type, y_vec, y_tma, ldc, c_off, relu;
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

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
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

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

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

__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory"); }

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

// TMEM columns for two accumulator buffers of BN columns (power of two, at least 32).
__host__ __device__ constexpr int tmem_cols_for(int bn) { return bn <= 16 ? 32 : (bn <= 32 ? 64 : (bn <= 64 ? 128 : (bn <= 128 ? 256 : 512))); }
// 8-bit output / residual tiles are kept in smem as panels of at most one 128-byte swizzle span;
// panel_mask is the XOR mask the TMA swizzle applies to 16-byte chunk indices.
__host__ __device__ constexpr int panel_bytes_for(int bn) { return bn < 128 ? bn : 128; }
__host__ __device__ constexpr int panel_mask_for(int pw) { return pw == 128 ? 7 : (pw == 64 ? 3 : (pw == 32 ? 1 : 0)); }

// ------------------------------------------------------------------------------------------ kernel
template <int BN, int BK, int MAX_STAGES>
__global__ void __launch_bounds__(kUmmaThreads, 1) conv_umma_kernel(const __grid_constant__ CUtensorMap tmA,
                                                                    const __grid_constant__ CUtensorMap tmB,
                                                                    const __grid_constant__ CUtensorMap tmRes,
                                                                    const __grid_constant__ CUtensorMap tmY,
                                                                    const UmmaParams p) {
  constexpr uint32_t A_BYTES = kBM * BK, B_BYTES = BN * BK, STAGE_BYTES = A_BYTES + B_BYTES;
  constexpr uint32_t TMEM_COLS = tmem_cols_for(BN);
  constexpr int PW = panel_bytes_for(BN), PANELS = BN / PW, PMASK = panel_mask_for(PW);
  constexpr uint32_t TILE8_BYTES = kBM * BN;  // one 8-bit output / residual tile
  constexpr int NCHUNK = BN / 16;

  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long full_bar[MAX_STAGES];
  __shared__ __align__(8) unsigned long long empty_bar[MAX_STAGES];
  __shared__ __align__(8) unsigned long long acc_full[2], acc_empty[2], res_full[2], res_empty[2];
  __shared__ uint32_t tmem_holder;
  __shared__ int abort_flag;
  __shared__ int epi_ok;
  __shared__ float s_scale[BN];
  __shared__ int s_bias[BN];

  // dynamic smem: [stages][A|B], then two 8-bit output staging tiles, then two residual tiles
  const uint32_t raw_base = smem_u32(smem_raw);
  const uint32_t tiles_base = (raw_base + 1023u) & ~1023u;
  const int stages = p.stages;
  const uint32_t out_base = (tiles_base + (uint32_t)stages * STAGE_BYTES + 1023u) & ~1023u;
  const uint32_t res_base = out_base + (p.y_tma ? 2u * TILE8_BYTES : 0u);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_tiles = p.m_tiles * p.n_tiles;

  if (threadIdx.x == 0) {
    prefetch_tensormap(&tmA);
    prefetch_tensormap(&tmB);
    if (p.res_mode == kResTma) prefetch_tensormap(&tmRes);
    if (p.y_tma) prefetch_tensormap(&tmY);
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&acc_full[i]), 1);
      mbar_init(smem_u32(&acc_empty[i]), 1);
      mbar_init(smem_u32(&res_full[i]), 1);
      mbar_init(smem_u32(&res_empty[i]), 1);
    }
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
    int stage = 0;
    uint32_t phase = 0;
    int lt = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++lt) {
      const int m0 = (tile / p.n_tiles) * kBM, n0 = (tile % p.n_tiles) * BN;
      if (p.res_mode == kResTma) {
        const int rb = lt & 1;
        if (!mbar_wait(smem_u32(&res_empty[rb]), ((uint32_t)(lt >> 1) & 1u) ^ 1u, abortp)) { ok = false; break; }
        const uint32_t bar = smem_u32(&res_full[rb]);
        mbar_arrive_expect_tx(bar, TILE8_BYTES);
#pragma unroll
        for (int pn = 0; pn < PANELS; ++pn)
          tma_load_2d(res_base + rb * TILE8_BYTES + pn * (kBM * PW), &tmRes, bar, n0 + pn * PW, m0);
      }
      int w0 = 0, h0 = 0, img = 0;
      if (p.a_im2col) {
        img = m0 / p.PQ;
        const int rem = m0 - img * p.PQ;
        const int p0 = rem / p.Q, q0 = rem - p0 * p.Q;
        h0 = p0 * p.stride_h - p.pad_h;
        w0 = q0 * p.stride_w - p.pad_w;
      }
      int r = 0, s = 0, cb = 0;
      for (int it = 0; it < p.k_iters; ++it) {
        if (!mbar_wait(smem_u32(&empty_bar[stage]), phase ^ 1u, abortp)) { ok = false; break; }
        const uint32_t bar = smem_u32(&full_bar[stage]);
        const uint32_t a_dst = tiles_base + stage * STAGE_BYTES, b_dst = a_dst + A_BYTES;
        mbar_arrive_expect_tx(bar, STAGE_BYTES);
        if (p.a_im2col)
          tma_load_im2col_4d(a_dst, &tmA, bar, cb * BK, w0, h0, img, (unsigned short)(s * p.dil_w), (unsigned short)(r * p.dil_h));
        else
          tma_load_2d(a_dst, &tmA, bar, cb * BK, m0);
        tma_load_3d(b_dst, &tmB, bar, cb * BK, r * p.S + s, n0);
        if (++cb == p.c_blocks) { cb = 0; if (++s == p.S) { s = 0; ++r; } }
        if (++stage == stages) { stage = 0; phase ^= 1u; }
      }
    }
    if (!ok) {
      abort_flag = 1;
      atomicOr(p.status, kTimeoutProducer);
    }
  } else if (threadIdx.x == 32) {
    // ------------------------------------------------------------------ MMA issuer
    int stage = 0;
    uint32_t phase = 0;
    int lt = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++lt) {
      const int ab = lt & 1;
      if (!mbar_wait(smem_u32(&acc_empty[ab]), ((uint32_t)(lt >> 1) & 1u) ^ 1u, abortp)) { ok = false; break; }
      tcgen05_fence_after();
      const uint32_t d_tmem = tmem_base + (uint32_t)(ab * BN);
      for (int it = 0; it < p.k_iters; ++it) {
        if (!mbar_wait(smem_u32(&full_bar[stage]), phase, abortp)) { ok = false; break; }
        tcgen05_fence_after();
        const uint32_t a_src = tiles_base + stage * STAGE_BYTES, b_src = a_src + A_BYTES;
        const uint64_t a_desc = make_kmajor_desc<BK>(a_src), b_desc = make_kmajor_desc<BK>(b_src);
#pragma unroll
        for (int k = 0; k < BK / 32; ++k)  // 32 bytes of K per instruction: +2 in 16-byte address units
          umma_i8(d_tmem, a_desc + 2 * k, b_desc + 2 * k, p.idesc, (it > 0 || k > 0) ? 1u : 0u);
        umma_commit(smem_u32(&empty_bar[stage]));
        if (++stage == stages) { stage = 0; phase ^= 1u; }
      }
      if (ok) umma_commit(smem_u32(&acc_full[ab]));
    }
    if (!ok) {
      abort_flag = 1;
      atomicOr(p.status, kTimeoutMma);
    }
  } else if (warp >= 2) {
    // ------------------------------------------------------------------ epilogue (8 warps)
    const int et = threadIdx.x - 64;
    const int quad = warp & 3;         // TMEM lane quadrant this warp may read
    const int half = (warp - 2) >> 2;  // which interleaved half of the 16-column chunks
    const int row = quad * 32 + lane;
    const bool leader = et == 0;
    const bool out8 = p.y_type == Q8_U8 || p.y_type == Q8_S8;
    unsigned char* const smem_tiles = smem_raw + (tiles_base - raw_base);  // generic pointer to tiles_base
    int lt = 0;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++lt) {
      const int m0 = (tile / p.n_tiles) * kBM, n0 = (tile % p.n_tiles) * BN;
      const int ab = lt & 1;
      const uint32_t par = (uint32_t)(lt >> 1) & 1u;
      if (leader) {
        bool ok = mbar_wait(smem_u32(&acc_full[ab]), par, abortp);
        if (ok && p.res_mode == kResTma) ok = mbar_wait(smem_u32(&res_full[ab]), par, abortp);
        if (!ok) {
          abort_flag = 1;
          atomicOr(p.status, kTimeoutEpilogue);
        }
        if (p.y_tma) bulk_wait_read<1>();  // the store that last used this staging tile has read it
        epi_ok = ok ? 1 : 0;
      }
      for (int j = et; j < BN; j += kEpiThreads) {
        const int n = n0 + j;
        s_bias[j] = (p.bias && n < p.K) ? p.bias[n] : 0;
        s_scale[j] = p.scale ? (p.scale_count == 1 ? p.scale[0] : (n < p.K ? p.scale[n] : 0.f)) : 0.f;
      }
      epi_bar_sync();
      if (!epi_ok) break;
      tcgen05_fence_after();

      const long long m = (long long)m0 + row;
      const bool row_ok = m < p.M;
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(ab * BN);
      unsigned char* const stage_out = smem_tiles + (out_base - tiles_base) + ab * TILE8_BYTES;
      const unsigned char* const stage_res = smem_tiles + (res_base - tiles_base) + ab * TILE8_BYTES;
      const bool has_res = p.res_mode != kResNone;
#pragma unroll 1
      for (int ch = half; ch < NCHUNK; ch += 2) {
        int acc[16];
        __syncwarp();
        tmem_ld_16(taddr + ch * 16, acc);
        tmem_ld_wait();
        const int nb = n0 + ch * 16;
        // 16-byte chunk (row, ch) of an 8-bit tile: panel, byte offset inside it, swizzled
        const int pn = (ch * 16) / PW;
        uint32_t off = (uint32_t)row * PW + (uint32_t)((ch * 16) % PW);
        off ^= ((off >> 7) & PMASK) << 4;
        off += pn * (kBM * PW);
#pragma unroll
        for (int j = 0; j < 16; ++j) acc[j] += s_bias[ch * 16 + j];

        if (p.y_type == Q8_S32) {
          if (row_ok && nb < p.K) {
            const int valid = min(16, p.K - nb);
            int* yp = static_cast<int*>(p.y) + (size_t)m * p.ldc + p.c_off + nb;
            if (p.y_vec && valid == 16) {
#pragma unroll
              for (int j = 0; j < 4; ++j) reinterpret_cast<int4*>(yp)[j] = make_int4(acc[4 * j], acc[4 * j + 1], acc[4 * j + 2], acc[4 * j + 3]);
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j)
                if (j < valid) yp[j] = acc[j];
            }
          }
          continue;
        }
        unsigned int rw[4] = {0u, 0u, 0u, 0u};
        if (p.res_mode == kResTma) {
          const uint4 rv = *reinterpret_cast<const uint4*>(stage_res + off);
          rw[0] = rv.x; rw[1] = rv.y; rw[2] = rv.z; rw[3] = rv.w;
        } else if (p.res_mode == kResGlobal) {
          if (row_ok && nb < p.K) {
            const int valid = min(16, p.K - nb);
            const unsigned char* rp = p.res + (size_t)m * p.K + nb;
#pragma unroll
            for (int j = 0; j < 16; ++j)
              if (j < valid) rw[j >> 2] |= (unsigned int)rp[j] << (8 * (j & 3));
          }
        }
        float v[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const unsigned int b = (rw[j >> 2] >> (8 * (j & 3))) & 0xffu;
          const int rz = p.res_signed ? (int)(signed char)b : (int)b;
          v[j] = requant_value(acc[j], s_scale[ch * 16 + j], has_res, rz, p.res_scale, p.relu != 0);
        }
        if (p.y_type == Q8_F32) {
          if (row_ok && nb < p.K) {
            const int valid = min(16, p.K - nb);
            float* yp = static_cast<float*>(p.y) + (size_t)m * p.ldc + p.c_off + nb;
            if (p.y_vec && valid == 16) {
#pragma unroll
              for (int j = 0; j < 4; ++j) reinterpret_cast<float4*>(yp)[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j)
                if (j < valid) yp[j] = v[j];
            }
          }
          continue;
        }
        int z[16];
        if (p.y_type == Q8_U8) {
#pragma unroll
          for (int j = 0; j < 16; ++j) z[j] = round_clamp_u8(v[j]);
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) z[j] = round_clamp_s8(v[j]);
        }
        *reinterpret_cast<uint4*>(stage_out + off) =
            make_uint4(pack4(z[0], z[1], z[2], z[3]), pack4(z[4], z[5], z[6], z[7]), pack4(z[8], z[9], z[10], z[11]),
                       pack4(z[12], z[13], z[14], z[15]));
      }
      // after this barrier every TMEM read, residual read and staging write of the tile is done
      tcgen05_fence_before();
      if (out8) fence_proxy_async_smem();
      epi_bar_sync();
      if (leader) {
        mbar_arrive(smem_u32(&acc_empty[ab]));
        if (p.res_mode == kResTma) mbar_arrive(smem_u32(&res_empty[ab]));
        if (p.y_tma) {
#pragma unroll
          for (int pn = 0; pn < PANELS; ++pn)
            tma_store_2d(&tmY, out_base + ab * TILE8_BYTES + pn * (kBM * PW), p.c_off + n0 + pn * PW, m0);
          bulk_commit();
        }
      }
    }
    if (leader && p.y_tma) bulk_wait_all();
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

int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    if (n <= 0) n = 148;
  }
  return n;
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
  int n = 200 * 1024 / ((kBM + bn) * bk);
  return n < 2 ? 2 : (n > 12 ? 12 : n);
}

// Dynamic shared memory besides the A/B stages: alignment slack and the epilogue tiles.
int fixed_smem_bytes(int bn, bool y_tma, bool res_tma) {
  return 2048 + (y_tma ? 2 * kBM * bn : 0) + (res_tma ? 2 * kBM * bn : 0);
}

int stages_that_fit(int bn, int bk, bool y_tma, bool res_tma) {
  return (kSmemLimit - kStaticSmemReserve - fixed_smem_bytes(bn, y_tma, res_tma)) / ((kBM + bn) * bk);
}

CUtensorMapSwizzle swizzle_for_bytes(int row_bytes) {
  return row_bytes >= 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                          : (row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                             : (row_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE));
}

template <int BN, int BK>
int launch_tile(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmRes, const CUtensorMap& tmY,
                UmmaParams& p, cudaStream_t stream) {
  constexpr int MAXS = max_stages_for(BN, BK);
  constexpr int STAGE_BYTES = (kBM + BN) * BK;
  auto kernel = conv_umma_kernel<BN, BK, MAXS>;
  int stages = stages_that_fit(BN, BK, p.y_tma != 0, p.res_mode == kResTma);
  if (stages > MAXS) stages = MAXS;
  if (stages < 2) return fail(Q8_ERR_UNSUPPORTED, "conv_umma: tile does not fit in shared memory");
  p.stages = stages;
  // at least 120 KiB so that one CTA owns an SM and with it the whole TMEM
  size_t dyn = (size_t)fixed_smem_bytes(BN, p.y_tma != 0, p.res_mode == kResTma) + (size_t)stages * STAGE_BYTES;
  if (dyn < 120 * 1024) dyn = 120 * 1024;
  static bool configured = false;  // per instantiation
  if (!configured) {
    int rc = check_cuda(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit - kStaticSmemReserve),
                        "conv_umma: set shared memory size");
    if (rc != Q8_OK) return rc;
    configured = true;
  }
  p.m_tiles = (p.M + kBM - 1) / kBM;
  p.n_tiles = (p.K + BN - 1) / BN;
  const long long tiles = (long long)p.m_tiles * p.n_tiles;
  const int grid = (int)(tiles < sm_count() ? tiles : sm_count());
  kernel<<<grid, kUmmaThreads, dyn, stream>>>(tmA, tmB, tmRes, tmY, p);
  return check_launch("conv_umma_kernel");
}

template <int BN>
int launch_bk(int bk, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmRes, const CUtensorMap& tmY,
              UmmaParams& p, cudaStream_t stream) {
  switch (bk) {
    case 128: return launch_tile<BN, 128>(tmA, tmB, tmRes, tmY, p, stream);
    case 64: return launch_tile<BN, 64>(tmA, tmB, tmRes, tmY, p, stream);
    default: return launch_tile<BN, 32>(tmA, tmB, tmRes, tmY, p, stream);
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

  const bool plain = d.R == 1 && d.S == 1 && d.stride_h == 1 && d.stride_w == 1 && d.pad_h == 0 && d.pad_w == 0;
  const bool out8 = d.y_type == Q8_U8 || d.y_type == Q8_S8;
  int res_mode = kResNone;
  if (a.residual) res_mode = (d.K % 16 == 0 && aligned16(a.residual)) ? kResTma : kResGlobal;
  const int BK = pick_bk(d.C);
  int BN = pick_bn(d.K);
  // the widest tile leaves too little room for A/B stages next to its epilogue tiles: narrow it
  if (BN == 256 && stages_that_fit(BN, BK, out8, res_mode == kResTma) < 3) BN = 128;
  const CUtensorMapSwizzle swz = swizzle_for_bytes(BK);
  const int PW = panel_bytes_for(BN);

  CUtensorMap tmA, tmB, tmRes, tmY;
  memset(&tmRes, 0, sizeof(tmRes));
  memset(&tmY, 0, sizeof(tmY));
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

  if (res_mode == kResTma) {
    cuuint64_t dims[2] = {(cuuint64_t)d.K, (cuuint64_t)a.M};
    cuuint64_t strides[1] = {(cuuint64_t)d.K};
    cuuint32_t box[2] = {(cuuint32_t)PW, (cuuint32_t)kBM};
    cuuint32_t estr[2] = {1, 1};
    cr = fn.tiled(&tmRes, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(a.residual), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for_bytes(PW), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return fail(Q8_ERR_CUDA, "conv_umma: residual tensor map rejected (CUresult %d)", (int)cr);
  }
  if (out8) {
    // the map ends at the last channel this layer owns, so the store clips ragged Cout tiles and
    // never touches a neighbouring slice of a concatenated tensor
    cuuint64_t dims[2] = {(cuuint64_t)(a.c_off + d.K), (cuuint64_t)a.M};
    cuuint64_t strides[1] = {(cuuint64_t)a.ldc};
    cuuint32_t box[2] = {(cuuint32_t)PW, (cuuint32_t)kBM};
    cuuint32_t estr[2] = {1, 1};
    cr = fn.tiled(&tmY, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, a.y, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  swizzle_for_bytes(PW), CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return fail(Q8_ERR_CUDA, "conv_umma: output tensor map rejected (CUresult %d)", (int)cr);
  }

  UmmaParams p;
  p.M = (int)a.M; p.K = d.K; p.PQ = a.P * a.Q; p.Q = a.Q;
  p.stride_h = d.stride_h; p.stride_w = d.stride_w; p.pad_h = d.pad_h; p.pad_w = d.pad_w; p.dil_h = d.dil_h; p.dil_w = d.dil_w;
  p.S = d.S;
  p.c_blocks = (d.C + BK - 1) / BK;
  p.k_iters = d.R * d.S * p.c_blocks;
  p.stages = 0; p.m_tiles = 0; p.n_tiles = 0;
  p.a_im2col = plain ? 0 : 1;
  // instruction descriptor: D = s32 (2 << 4); A format at bit 7 (0 = u8, 1 = s8); B = s8 at bit 10;
  // both operands K-major; N/8 at bit 17; M/16 at bit 24.
  p.idesc = (2u << 4) | ((d.x_type == Q8_S8 ? 1u : 0u) << 7) | (1u << 10) | ((unsigned)(BN >> 3) << 17) | ((unsigned)(kBM >> 4) << 24);
  p.bias = a.bias; p.scale = a.scale; p.scale_count = d.scale_count;
  p.res = static_cast<const unsigned char*>(a.residual);
  p.res_mode = res_mode;
  p.res_signed = d.res_type == Q8_S8;
  p.res_scale = a.residual_scale;
  p.y = a.y; p.y_type = d.y_type; p.ldc = a.ldc; p.c_off = a.c_off; p.relu = d.relu;
  p.y_tma = out8 ? 1 : 0;
  p.y_vec = out8 ? 1 : (aligned16(a.y) && a.ldc % 4 == 0 && a.c_off % 4 == 0);
  p.status = status;

  switch (BN) {
    case 16: return launch_bk<16>(BK, tmA, tmB, tmRes, tmY, p, a.stream);
    case 32: return launch_bk<32>(BK, tmA, tmB, tmRes, tmY, p, a.stream);
    case 64: return launch_bk<64>(BK, tmA, tmB, tmRes, tmY, p, a.stream);
    case 128: return launch_bk<128>(BK, tmA, tmB, tmRes, tmY, p, a.stream);
    default: return launch_bk<256>(BK, tmA, tmB, tmRes, tmY, p, a.stream);
  }
}

}  // namespace q8
