// Device and host helpers shared by the tensor-core convolution kernels (q8_conv_umma.cu, q8_conv_fused.cu):
// launch constants, the kernel parameter block, the tile walker, single-instruction PTX wrappers (mbarrier, TMA,
// tcgen05), the requantizing epilogue of one accumulator row, and the host-side planning helpers (driver entry
// points for tensor maps, halo tiling, channel-block and tile-width choice).  Everything here has internal linkage.
#pragma once
#include <cuda.h>

#include <atomic>
#include <cstdlib>
#include <cstring>
#include <initializer_list>

#include "q8_internal.h"

namespace q8 {
namespace {

constexpr int kBM = 128;
constexpr int kCtrlWarps = 6;            // producer, MMA 0, buffers/residual, store, MMA 1, spare
constexpr int kCtrlThreads = kCtrlWarps * 32;
constexpr int kMmaWarps = 3;             // at most this many MMA-issuing lanes; tile lt belongs to lane lt % mma_lanes
constexpr int kGroupThreads = 128;      // one epilogue group
constexpr int kMaxStages = 8;           // A stages
constexpr int kMaxBStages = 8;          // weight ring
constexpr int kMaxAcc = 4;
constexpr int kMaxSlots = 8;            // 8-bit tile buffers over all groups
constexpr int kMaxTaps = 64;            // halo mode keeps a descriptor offset per tap in shared memory
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s per wait
constexpr int kSmemLimit = 232448;                           // 227 KiB opt-in maximum per CTA
constexpr int kStaticSmemReserve = 2048;                     // barriers, tap table and flags

enum StatusBits : unsigned int {
  kTimeoutProducer = 1u,
  kTimeoutMma = 2u,
  kTimeoutEpilogue = 4u,
  kTimeoutResidual = 8u,
  kTimeoutStore = 16u,
};

enum ResMode : int { kResNone = 0, kResTma = 1, kResGlobal = 2 };
enum AMode : int { kAPlain = 0, kAIm2col = 1, kAHalo = 2 };
enum BMode : int { kBStage = 0, kBResident = 1, kBRing = 2 };

// Division by a launch-time constant without the ~35-instruction software divide, which costs a
// lone control lane some 200 cycles: q = (umulhi(x, m) + x) >> l for 0 <= x < 2^31 (Granlund-Montgomery).
struct FastDiv {
  unsigned int m, l;
  int d;
#ifdef __CUDACC__
  __device__ __forceinline__ int div(int x) const { return (int)((__umulhi((unsigned int)x, m) + (unsigned int)x) >> l); }
#endif
};

struct UmmaParams {
  int M, K;                  // GEMM rows (pixels) and Cout
  int P, Q, PQ;              // output height, width, pixels per image
  int stride_h, stride_w, pad_h, pad_w, dil_h, dil_w;
  int R, S, taps;            // filter height, width, R * S
  int C_pad, c_blocks;       // channels rounded up to whole K blocks, number of K blocks
  int bn, bk, ksteps;        // tile width (multiple of 16), K bytes per block (32/64/128), bk / 32
  int a_mode, b_mode;
  int k_iters, kb;           // plain/im2col: taps * c_blocks (tap, block) iterations, kb of them per A stage
  int tw, th, twb, hb;       // halo: tile and patch extents in pixels (pixel pairs along W when halo_sw == 2)
  int halo_sw, halo_e, c_true;  // halo: stride along W (1 or 2), parity of pad_w, channels per input pixel
  unsigned int tap_shift16[kMaxTaps];  // halo: descriptor start offset of every tap, in 16-byte units
  int p_tiles, q_tiles;      // halo: tiles per image column / row
  int stages, b_stages;      // A stages, weight-ring stages
  int nacc, acc_stride, tmem_cols;  // TMEM accumulators, columns between them, allocation (power of two)
  int nbuf;                  // 8-bit tile buffers per epilogue group (0: none)
  int m_tiles, n_tiles;
  FastDiv fd_ntiles, fd_perimg, fd_qtiles, fd_pq, fd_q;  // n_tiles, p_tiles*q_tiles, q_tiles, P*Q, Q
  int splits, kps;           // split-K: work item = (tile, split), each split runs kps of the k_iters iterations
  FastDiv fd_splits, fd_cblocks, fd_s;  // splits, c_blocks, S
  long long split_stride;    // elements between the partial results of two splits in the workspace
  unsigned int idesc;        // tcgen05 instruction descriptor
  unsigned int desc_hi;      // high word of the shared-memory matrix descriptors
  unsigned int a_sub_bytes;  // plain/im2col: one 128 x bk block; halo: bytes of one patch load
  unsigned int b_tile_bytes; // bn * bk
  unsigned int b_sub_bytes;  // b_tile_bytes rounded up to 1 KiB (placement inside a stage); ring: one ring stage
  int cta2;                  // 1: CTA pairs (clusters of two) issue tcgen05.mma.cta_group::2 over two m tiles that
                             // share the n tile; each CTA holds its own A patch and half of the weight tile rows
  int m_tiles_real;          // cta2: number of real m tiles (m_tiles counts pairs)
  int fast_taps;             // halo: tap count of a filter whose issue loop is unrolled (3x3, 5x5, 7 x 4 pairs), else 0
  unsigned int row16, col16; // halo: descriptor shift, in 16-byte units, of one filter row / one filter column
  int mma_lanes;             // 3 with four accumulators (narrow tiles are bound by the issue rate of a lone lane), else 2
  int epi_split;             // 1: every epilogue group takes a share of the columns of every tile (short launches)
  int b_T, b_chunks;         // weight ring: filter taps per ring stage (one TMA operation), stages per channel block
  unsigned int a_stage_bytes;
  unsigned int tile8_bytes;
  unsigned int res_tx_bytes; // bytes one residual tile load delivers
  unsigned int off_a, off_bring, off_bufs, off_chan;  // from the 1 KiB aligned base; resident weights at 0
  int pw_shift, pmask, panels;  // 8-bit tiles live in smem as panels of 2^pw_shift bytes per row
  int k_pad;                 // n_tiles * bn channels of bias/scale staged in smem
  const int* bias;
  const float* scale;
  int scale_count;
  const unsigned char* res;
  int res_mode, res_signed;
  float res_scale;
  void* y;
  int y_type, y_vec, out8, ldc, c_off, relu;
  unsigned int* status;
};

// Walks the tiles of one role: tile = first, first + step, ...; tile -> (m tile, n tile) with the
// n tiles of one m tile adjacent (they share the A operand through L2), and for halo tiles
// m tile -> (image, tile row, tile column).  Only additions after init().
template <bool kPair>
struct TileIterT {
  int tile, step;    // work item index (tile * splits + split) and its stride
  int sp, d_sp;      // split-K part of the work item
  int mt, nt;        // m tile, n tile
  int img, pt, qt;   // halo: image, tile row, tile column
  int d_mt, d_nt, d_img, d_pt, d_qt;
  int rank;          // cta2: this CTA's rank in its pair; work items are pairs of m tiles (2 * pair + rank)
  bool valid;        // cta2: the m tile exists (the last pair of an odd count has a phantom second tile)

  // cta2: plain re-decoding, a handful of multiply-shift divisions per tile of several thousand cycles
  __device__ __forceinline__ void decode_pair(const UmmaParams& p) {
    const int mp = p.fd_ntiles.div(tile);
    nt = tile - mp * p.n_tiles;
    mt = 2 * mp + rank;
    valid = mt < p.m_tiles_real;
    const int per_img = p.p_tiles * p.q_tiles;
    img = p.fd_perimg.div(mt);
    const int r = mt - img * per_img;
    pt = p.fd_qtiles.div(r);
    qt = r - pt * p.q_tiles;
  }

  __device__ __forceinline__ void init(const UmmaParams& p, int first, int step_, int rank_ = 0) {
    tile = first; step = step_;
    rank = rank_; valid = true;
    if constexpr (kPair) { sp = d_sp = 0; decode_pair(p); return; }
    int t0 = first, dt = step_;  // output tile and its stride
    sp = d_sp = 0;
    if (p.splits > 1) {
      t0 = p.fd_splits.div(first); sp = first - t0 * p.splits;
      dt = p.fd_splits.div(step_); d_sp = step_ - dt * p.splits;
    }
    mt = p.fd_ntiles.div(t0); nt = t0 - mt * p.n_tiles;
    d_mt = p.fd_ntiles.div(dt); d_nt = dt - d_mt * p.n_tiles;
    img = pt = qt = d_img = d_pt = d_qt = 0;
    if (p.a_mode == kAHalo) {
      const int per_img = p.p_tiles * p.q_tiles;
      img = p.fd_perimg.div(mt);
      int r = mt - img * per_img;
      pt = p.fd_qtiles.div(r); qt = r - pt * p.q_tiles;
      d_img = p.fd_perimg.div(d_mt);
      r = d_mt - d_img * per_img;
      d_pt = p.fd_qtiles.div(r); d_qt = r - d_pt * p.q_tiles;
    }
  }
  __device__ __forceinline__ void next(const UmmaParams& p) {
    tile += step;
    if constexpr (kPair) { decode_pair(p); return; }
    int carry = 0;
    sp += d_sp;
    if (sp >= p.splits) { sp -= p.splits; carry = 1; }
    nt += d_nt + carry; carry = 0;
    if (nt >= p.n_tiles) { nt -= p.n_tiles; carry = 1; }
    mt += d_mt + carry;
    if (p.a_mode == kAHalo) {
      qt += d_qt + carry; carry = 0;
      if (qt >= p.q_tiles) { qt -= p.q_tiles; carry = 1; }
      pt += d_pt + carry; carry = 0;
      if (pt >= p.p_tiles) { pt -= p.p_tiles; carry = 1; }
      img += d_img + carry;
    }
  }
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

// Waits are warp collective: every role runs as a whole converged warp (its loop counters, addresses and
// descriptors then are warp-uniform values, which the instructions that take uniform operands, tcgen05.mma and
// the TMA copies, need: computed by a single diverged lane they cost a dozen extra moves per instruction),
// all 32 lanes poll, and the votes make the outcome uniform by construction.
// Slow path of a wait, out of line to keep the role loops small.  Gives up after about
// kWaitLimitNs or when another role of this CTA has already given up; the caller then records the
// site and leaves its loop.  The wall clock is only read once the wait has lasted a while.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                            unsigned long long limit_ns = kWaitLimitNs) {
  unsigned long long t0 = 0;
  uint32_t spins = 0;
  for (;;) {
    if (__all_sync(0xffffffffu, mbar_try_wait(bar, parity) ? 1 : 0)) return true;
    if ((++spins & 0x3ffu) == 0) {
      int give_up = *abort_flag;
      const unsigned long long now = global_timer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) give_up = 1;
      if (__any_sync(0xffffffffu, give_up)) return false;
    }
  }
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (__all_sync(0xffffffffu, mbar_try_wait(bar, parity) ? 1 : 0)) return true;
  return mbar_wait_slow(bar, parity, abort_flag);
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

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}

__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
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

// ---- CTA pairs (cta_group::2).  The leader (even rank) issues the MMAs; operands sit at the same shared-memory
// offsets in both CTAs; loads of either CTA signal the leader's barrier; commits arrive in both CTAs.
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, uint32_t leader_bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(leader_bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* map, uint32_t leader_bar, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(leader_bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t holder_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(holder_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void umma_i8_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrives on the barrier at this offset in both CTAs of the pair once the MMAs issued so far have completed
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((unsigned short)3)
               : "memory");
}

// D[tmem] (+)= A[smem desc] * B[smem desc]^T, 8-bit integer inputs, int32 accumulate.  The issuing
// lane retires about one instruction every six cycles, so the issue path is kept to the bare
// instruction: descriptors live in 64-bit registers and the always-accumulate form has a constant
// predicate.
__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_i8_acc(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.eq.u32 p, 0, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc)
      : "memory");
}

// kSteps instructions over one K block of kSteps * 32 bytes: +2 in 16-byte address units per step.
template <int kSteps>
__device__ __forceinline__ void umma_i8_block(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate_first) {
  umma_i8(d_tmem, a_desc, b_desc, idesc, accumulate_first);
#pragma unroll
  for (int k = 1; k < kSteps; ++k) umma_i8_acc(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc);
}

// All taps of an R x S filter (kTrans: tap order (s, r) of the pixel-pair view, else (r, s)) on one channel block
// against resident weight tiles, fully unrolled: the descriptor shift of tap (r, s) is r * row16 + s * col16.
template <int kR, int kS, bool kTrans, int kSteps>
__device__ __forceinline__ void issue_taps(uint32_t d_tmem, uint64_t a_d, uint32_t row16, uint32_t col16, uint64_t bres,
                                           uint32_t btile16, uint32_t idesc, uint32_t accumulate_first) {
  uint32_t coff[kS];
#pragma unroll
  for (int t = 0; t < kS; ++t) coff[t] = (uint32_t)t * col16;
  uint64_t rowb = a_d;  // descriptor of filter row r, advanced by additions
#pragma unroll
  for (int r = 0; r < kR; ++r) {
#pragma unroll
    for (int t = 0; t < kS; ++t) {
      const int tap = kTrans ? t * kR + r : r * kS + t;  // position of the tap's weight tile
      umma_i8_block<kSteps>(d_tmem, rowb + coff[t], bres + (uint32_t)tap * btile16, idesc,
                            (r == 0 && t == 0) ? accumulate_first : 1u);
    }
    rowb += row16;
  }
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
// Waits for this thread's TMEM loads.  The registers are named as operands so that no use of them
// can be scheduled ahead of the wait.
__device__ __forceinline__ void tmem_ld_wait(int (&v)[16]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]), "+r"(v[8]),
                 "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15])
               :
               : "memory");
}

// {lo byte, next byte} = {sat(b), sat(a)}, upper half = low half of c.
__device__ __forceinline__ unsigned int pack_sat_u8(int a, int b, unsigned int c) {
  unsigned int d;
  asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ unsigned int pack_sat_s8(int a, int b, unsigned int c) {
  unsigned int d;
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
// bytes (z0, z1, z2, z3), z0 lowest, each saturated to the 8-bit range
template <bool kSigned>
__device__ __forceinline__ unsigned int pack4_sat(int z0, int z1, int z2, int z3) {
  return kSigned ? pack_sat_s8(z1, z0, pack_sat_s8(z3, z2, 0u)) : pack_sat_u8(z1, z0, pack_sat_u8(z3, z2, 0u));
}

// Packed fp32 arithmetic: two independent IEEE operations (round to nearest even, no contraction) in one
// instruction slot.  The epilogue of a layer with a short reduction is bound by instruction issue.
__device__ __forceinline__ unsigned long long pack_f2(float a, float b) {
  unsigned long long d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(a), "f"(b));
  return d;
}
__device__ __forceinline__ void unpack_f2(unsigned long long d, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(d));
}
__device__ __forceinline__ unsigned long long fmul2(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ unsigned long long fsub2(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// ------------------------------------------------------------------------------------------ epilogue
struct EpiTile {
  const int* s_bias;       // smem, k_pad entries
  const float* s_scale;    // smem, k_pad entries
  unsigned char* buf;      // this tile's 8-bit buffer (residual in, output out) or nullptr
  long long m;             // output pixel (row of the [M][Cout] result) of this thread
  long long y_off;         // element offset of this work item's output (split-K partial results), else 0
  int srow;                // row of this thread's pixel inside the 8-bit tile buffer
  uint32_t row_base, swz;  // byte offset of that row inside a panel, and the row's swizzle term (set by epi_row_setup)
  int n0;                  // first channel of the tile
  bool row_ok;             // the pixel exists (inside the image and below M)
  bool smem_ok;            // this accumulator row maps to a pixel of the tile (always, except halo tiles)
};

// Position of a thread's row in the swizzled 8-bit tile buffers: constant for the thread's lifetime.  A panel is
// 128 rows of 2^pw_shift bytes; the 16-byte chunk index of a row is XORed with address bits 7.. (the swizzle the
// TMA and the tensor core use), which for rows of one swizzle span depend on the row alone.
__device__ __forceinline__ void epi_row_setup(const UmmaParams& p, EpiTile& t) {
  t.row_base = (uint32_t)t.srow << p.pw_shift;
  t.swz = ((t.row_base >> 7) & (uint32_t)p.pmask) << 4;
}

// One 16-column chunk of one accumulator row.  kOut: Q8_U8, Q8_S8, Q8_S32 or Q8_F32.  kRes: kResNone, kResTma
// (a residual from the tile buffer if p.res_mode says so, else none: decided at run time) or kResGlobal.  Fewer
// distinct kernels matter more than one uniform branch per chunk: a launch of another kernel function than
// the one before it starts with cold instruction caches, which costs a layer of a network 2 to 6 us, so the
// layers with and without a residual sum share their kernels.  (One straight-line arm per case, chosen per
// chunk or per row, made the register allocator spill.)
//   v = float(acc + bias) * s;  v += float(res) * s_res;  v = max(v, 0);  y = clamp(Round(v))
// Each step is one IEEE fp32 operation (the library is built without FMA contraction).
template <int kOut, int kRes>
__device__ __forceinline__ void epilogue_chunk(const UmmaParams& p, const EpiTile& t, int ch, const int (&raw)[16]) {
  const int c16 = ch * 16;
  const int nb = t.n0 + c16;
  int acc[16];
  {
    const int4* bp = reinterpret_cast<const int4*>(t.s_bias + nb);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int4 b = bp[j];
      acc[4 * j] = raw[4 * j] + b.x; acc[4 * j + 1] = raw[4 * j + 1] + b.y;
      acc[4 * j + 2] = raw[4 * j + 2] + b.z; acc[4 * j + 3] = raw[4 * j + 3] + b.w;
    }
  }
  if (kOut == Q8_S32) {
    if (t.row_ok && nb < p.K) {
      const int valid = min(16, p.K - nb);
      int* yp = static_cast<int*>(p.y) + t.y_off + (size_t)t.m * p.ldc + p.c_off + nb;
      if (p.y_vec && valid == 16) {
#pragma unroll
        for (int j = 0; j < 4; ++j) reinterpret_cast<int4*>(yp)[j] = make_int4(acc[4 * j], acc[4 * j + 1], acc[4 * j + 2], acc[4 * j + 3]);
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (j < valid) yp[j] = acc[j];
      }
    }
    return;
  }
  // position of this thread's 16 bytes inside the swizzled 8-bit tile buffer
  uint32_t off = 0;
  if (kOut == Q8_U8 || kOut == Q8_S8 || (kRes == kResTma && p.res_mode == kResTma)) {
    const int pn = c16 >> p.pw_shift;
    off = t.row_base + (((uint32_t)(c16 & ((1 << p.pw_shift) - 1))) ^ t.swz) + (uint32_t)pn * ((uint32_t)kBM << p.pw_shift);
  }
  unsigned long long v2[8];  // v[2i], v[2i + 1]
  float v[16];
  {
    const float4* sp = reinterpret_cast<const float4*>(t.s_scale + nb);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float4 s = sp[j];
      v2[2 * j] = fmul2(pack_f2(__int2float_rn(acc[4 * j]), __int2float_rn(acc[4 * j + 1])), pack_f2(s.x, s.y));
      v2[2 * j + 1] = fmul2(pack_f2(__int2float_rn(acc[4 * j + 2]), __int2float_rn(acc[4 * j + 3])), pack_f2(s.z, s.w));
    }
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) unpack_f2(v2[j], v[2 * j], v[2 * j + 1]);
  unsigned int rw[4] = {0u, 0u, 0u, 0u};
  if (kRes == kResTma && (kOut == Q8_U8 || kOut == Q8_S8)) {
    // the tile buffer always exists for 8-bit outputs: its bytes are read ahead of the (uniform) branch on
    // whether they are a residual, so that the load is in flight with those of bias and scale
    const uint4 rv = *reinterpret_cast<const uint4*>(t.buf + off);
    rw[0] = rv.x; rw[1] = rv.y; rw[2] = rv.z; rw[3] = rv.w;
  }
  if (kRes == kResGlobal || (kRes == kResTma && p.res_mode != kResNone)) {
    if (kRes == kResTma) {
      if (kOut != Q8_U8 && kOut != Q8_S8) {
        const uint4 rv = *reinterpret_cast<const uint4*>(t.buf + off);
        rw[0] = rv.x; rw[1] = rv.y; rw[2] = rv.z; rw[3] = rv.w;
      }
    } else if (t.row_ok && nb < p.K) {
      const int valid = min(16, p.K - nb);
      const unsigned char* rp = p.res + (size_t)t.m * p.K + nb;
#pragma unroll
      for (int j = 0; j < 16; ++j)
        if (j < valid) rw[j >> 2] |= (unsigned int)rp[j] << (8 * (j & 3));
    }
    // byte b -> float without a conversion instruction: 0x4B0000bb is 2^23 + b exactly; a signed
    // byte is first biased by 128
    const unsigned int sign_mask = p.res_signed ? 0x80808080u : 0u;
    const float magic = p.res_signed ? 8388736.0f : 8388608.0f;
    const unsigned long long magic2 = pack_f2(magic, magic), rs2 = pack_f2(p.res_scale, p.res_scale);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const unsigned int w = rw[j >> 1] ^ sign_mask;
      const float r0 = __uint_as_float(__byte_perm(w, 0x4B000000u, 0x7540u | (unsigned)((2 * j) & 3)));
      const float r1 = __uint_as_float(__byte_perm(w, 0x4B000000u, 0x7540u | (unsigned)((2 * j + 1) & 3)));
      // the sum stays scalar: the assembler contracts a packed multiply followed by a packed add into one
      // fused operation (one rounding instead of two), which would break the two-rounding definition
      float t0, t1;
      unpack_f2(fmul2(fsub2(pack_f2(r0, r1), magic2), rs2), t0, t1);
      v[2 * j] = __fadd_rn(v[2 * j], t0);
      v[2 * j + 1] = __fadd_rn(v[2 * j + 1], t1);
    }
  }
  if (kOut == Q8_F32) {
    if (p.relu) {
#pragma unroll
      for (int j = 0; j < 16; ++j) v[j] = fmaxf(v[j], 0.0f);
    }
    if (t.row_ok && nb < p.K) {
      const int valid = min(16, p.K - nb);
      float* yp = static_cast<float*>(p.y) + (size_t)t.m * p.ldc + p.c_off + nb;
      if (p.y_vec && valid == 16) {
#pragma unroll
        for (int j = 0; j < 4; ++j) reinterpret_cast<float4*>(yp)[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (j < valid) yp[j] = v[j];
      }
    }
    return;
  }
  // 8-bit output: the saturating pack clamps to [0,255] (which also is the ReLU) or [-128,127]
  if (kOut == Q8_S8 && p.relu) {
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = fmaxf(v[j], 0.0f);
  }
  int z[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) z[j] = __float2int_rn(v[j]);
  uint4 o;
  o.x = pack4_sat<kOut == Q8_S8>(z[0], z[1], z[2], z[3]);
  o.y = pack4_sat<kOut == Q8_S8>(z[4], z[5], z[6], z[7]);
  o.z = pack4_sat<kOut == Q8_S8>(z[8], z[9], z[10], z[11]);
  o.w = pack4_sat<kOut == Q8_S8>(z[12], z[13], z[14], z[15]);
  if (t.smem_ok) *reinterpret_cast<uint4*>(t.buf + off) = o;
}

// All chunks of one accumulator row, TMEM loads one chunk ahead of the arithmetic.  The accumulator
// is released (acc_empty) as soon as its last chunk is in registers.
template <int kOut, int kRes, bool kPair>
__device__ __forceinline__ void epilogue_row(const UmmaParams& p, const EpiTile& t, uint32_t taddr, uint32_t acc_empty_bar,
                                             int lane, const int ch0, const int nchunk) {
  // chunks ch0 .. nchunk-1 of 16 columns each
  int ra[16], rb[16];
  if (ch0 >= nchunk) {  // no columns for this warp in this tile: it still hands the accumulator back
    tcgen05_fence_before();
    __syncwarp();
    if (lane == 0) { if constexpr (kPair) mbar_arrive_cluster(acc_empty_bar); else mbar_arrive(acc_empty_bar); }
    return;
  }
  tmem_ld_16(taddr + ch0 * 16, ra);
#pragma unroll 1
  for (int ch = ch0; ch < nchunk; ch += 2) {
    tmem_ld_wait(ra);
    const bool more1 = ch + 1 < nchunk;
    if (more1) tmem_ld_16(taddr + (ch + 1) * 16, rb);
    else {
      // every accumulator value of this warp is in registers: hand the TMEM buffer back
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) { if constexpr (kPair) mbar_arrive_cluster(acc_empty_bar); else mbar_arrive(acc_empty_bar); }
    }
    epilogue_chunk<kOut, kRes>(p, t, ch, ra);
    if (more1) {
      tmem_ld_wait(rb);
      const bool more2 = ch + 2 < nchunk;
      if (more2) tmem_ld_16(taddr + (ch + 2) * 16, ra);
      else {
        tcgen05_fence_before();
        __syncwarp();
        if (lane == 0) { if constexpr (kPair) mbar_arrive_cluster(acc_empty_bar); else mbar_arrive(acc_empty_bar); }
      }
      epilogue_chunk<kOut, kRes>(p, t, ch + 1, rb);
    }
  }
}

// ------------------------------------------------------------------------------------------ MMA role
struct MmaRoleArgs {
  uint32_t base, tmem_base;
  uint32_t a_full, a_empty, b_full, b_empty, acc_full, acc_empty, bres_full, turn;
  const uint32_t* tap_shift16;
  int first_tile, tile_step, total_tiles;  // this CTA's work items: first_tile, first_tile + tile_step, ... below total_tiles
  volatile int* abortp;
};

// The single MMA-issuing lane.  kSteps (K block bytes / 32) is a compile-time constant so that the
// instructions of one K block are straight-line code.  Returns false if a wait gave up.
template <int kSteps>
__device__ __forceinline__ bool mma_role(const UmmaParams& p, const MmaRoleArgs& r, const int who) {
  // This lane's tiles are lt = who, who + kMmaWarps, ... of the CTA's sequence; the stage, weight-ring
  // and accumulator positions of a tile follow from lt alone.  A parity wait is only meaningful for
  // the use of a barrier that is in flight, so a lane starts the stage waits of tile lt only after
  // the lane of tile lt - 1 has passed all of its own (the turn barriers); the per-tile bookkeeping
  // and the accumulator wait run ahead of that.
  TileIterT<false> ti;
  const int L = p.mma_lanes;
  const bool lane0 = (threadIdx.x & 31u) == 0;  // the whole warp walks the schedule, this lane issues
  ti.init(p, r.first_tile + who * r.tile_step, L * r.tile_step);
  const uint32_t nstages = (uint32_t)p.stages, nbst = (uint32_t)p.b_stages;
  // descriptors: high word constant; low word = start address >> 4 (shared memory ends below 256 KiB,
  // the 14-bit field never wraps) plus the leading-byte-offset field (bits 16-29), unused for swizzled
  // K-major tiles and set to 1
  const uint64_t hi = ((uint64_t)p.desc_hi << 32) | (1ull << 16);
  const uint64_t a_d0 = hi | (((r.base + p.off_a) >> 4) & 0x3fffu), bring_d0 = hi | (((r.base + p.off_bring) >> 4) & 0x3fffu);
  const uint64_t bres_d0 = hi | ((r.base >> 4) & 0x3fffu);
  const uint32_t stage16 = p.a_stage_bytes >> 4, asub16 = p.a_sub_bytes >> 4, bsub16 = p.b_sub_bytes >> 4, btile16 = p.b_tile_bytes >> 4;
  const uint32_t idesc = p.idesc;
  const int taps = p.taps, c_blocks = p.c_blocks, k_iters = p.kps, kb = p.kb;  // k iterations of one work item
  const bool halo = p.a_mode == kAHalo, ring = p.b_mode == kBRing, b_in_stage = p.b_mode == kBStage;
  // ring positions of tile lt = who, and how far the other lanes' tiles move them between two of ours
  const uint32_t spt = halo ? (uint32_t)c_blocks : (uint32_t)((k_iters + kb - 1) / kb);  // A stages per tile
  const int bT = p.b_T;
  const uint32_t bpt = (uint32_t)(p.b_chunks * c_blocks);                                 // ring stages per tile
  const uint32_t skip_a = (uint32_t)(L - 1) * spt, skip_b = (uint32_t)(L - 1) * bpt;
  uint32_t stage = ((uint32_t)who * spt) % nstages, phase = (((uint32_t)who * spt) / nstages) & 1u;
  uint32_t bs = 0, bphase = 0;
  if (ring) { bs = ((uint32_t)who * bpt) % nbst; bphase = (((uint32_t)who * bpt) / nbst) & 1u; }
  uint64_t a_d = a_d0 + stage * stage16;
  uint64_t bring_d = bring_d0 + bs * bsub16;
  const uint32_t nacc = (uint32_t)p.nacc;
  uint32_t ab = (uint32_t)who % nacc, acc_par = 1u ^ (((uint32_t)who / nacc) & 1u);  // accumulator and the parity of its empty barrier
  uint32_t my_k = 0;  // number of tiles this lane has issued
  const uint32_t turn_next = r.turn + (uint32_t)((who + 1) % L) * 8u;  // the next lane's turn barrier
  const uint32_t turn_mine = r.turn + (uint32_t)who * 8u;
  if (p.b_mode == kBResident && !mbar_wait(r.bres_full, 0u, r.abortp)) return false;
  const int fast_taps = halo ? p.fast_taps : 0;  // 9: 3x3, 25: 5x5, 28: 7x7 as pixel pairs, else 0
  uint32_t shift9[9];
#pragma unroll
  for (int t = 0; t < 9; ++t) shift9[t] = fast_taps == 9 ? r.tap_shift16[t] : 0u;
  for (; ti.tile < r.total_tiles; ti.next(p)) {
    if (!mbar_wait(r.acc_empty + ab * 8u, acc_par, r.abortp)) return false;
    // turn[w] counts the tiles the other lane has finished waiting for: tile number k of lane 0 needs
    // k of them, tile number k of lane 1 needs k + 1
    if (who == 0) { if (my_k > 0 && !mbar_wait(turn_mine, (my_k - 1) & 1u, r.abortp)) return false; }
    else if (!mbar_wait(turn_mine, my_k & 1u, r.abortp)) return false;
    tcgen05_fence_after();
    const uint32_t d_tmem = r.tmem_base + ab * (uint32_t)p.acc_stride;
    uint32_t accum = 0;
    // resident weights: tile (nt, cb, tap) sits at ((nt * c_blocks + cb) * taps + tap) * b_tile_bytes
    const uint64_t bres_nt = bres_d0 + (uint32_t)(ti.nt * c_blocks * taps) * btile16;
    if (halo) {
      uint64_t bres = bres_nt;  // (cb, tap) is exactly the order of the loops below
      for (int cb = 0; cb < c_blocks; ++cb) {
        if (!mbar_wait(r.a_full + stage * 8u, phase, r.abortp)) return false;
        const bool last_cb = cb == c_blocks - 1;
        if (last_cb && !ring && lane0) mbar_arrive(turn_next);  // this tile's last wait is behind us
        tcgen05_fence_after();
        if (ring && bT == 1) {
          // (kept apart from the multi-tap loop below: every extra instruction of this lone lane costs ~6 cycles)
          for (int tap = 0; tap < taps; ++tap) {
            if (!mbar_wait(r.b_full + bs * 8u, bphase, r.abortp)) return false;
            tcgen05_fence_after();
            if (lane0) {
              if (last_cb && tap == taps - 1) mbar_arrive(turn_next);
              umma_i8_block<kSteps>(d_tmem, a_d + r.tap_shift16[tap], bring_d, idesc, accum);
              umma_commit(r.b_empty + bs * 8u);
            }
            accum = 1;
            bring_d += bsub16;
            if (++bs == nbst) { bs = 0; bphase ^= 1u; bring_d = bring_d0; }
          }
        } else if (ring && fast_taps == 9 && bT == 3) {
          // 3x3 in ring stages of one filter row each: straight-line issue with the shifts in registers
#pragma unroll
          for (int row = 0; row < 3; ++row) {
            if (!mbar_wait(r.b_full + bs * 8u, bphase, r.abortp)) return false;
            tcgen05_fence_after();
            if (lane0) {
              if (last_cb && row == 2) mbar_arrive(turn_next);
#pragma unroll
              for (int t = 0; t < 3; ++t)
                umma_i8_block<kSteps>(d_tmem, a_d + shift9[3 * row + t], bring_d + (uint32_t)t * btile16, idesc, (row == 0 && t == 0) ? accum : 1u);
              umma_commit(r.b_empty + bs * 8u);
            }
            accum = 1;
            bring_d += bsub16;
            if (++bs == nbst) { bs = 0; bphase ^= 1u; bring_d = bring_d0; }
          }
        } else if (ring) {
          for (int tap0 = 0; tap0 < taps; tap0 += bT) {
            if (!mbar_wait(r.b_full + bs * 8u, bphase, r.abortp)) return false;
            tcgen05_fence_after();
            const int nt = min(bT, taps - tap0);
            if (lane0) {
              if (last_cb && tap0 + bT >= taps) mbar_arrive(turn_next);
              uint64_t bd = bring_d;
              for (int t = 0; t < nt; ++t, bd += btile16) {
                umma_i8_block<kSteps>(d_tmem, a_d + r.tap_shift16[tap0 + t], bd, idesc, accum);
                accum = 1;
              }
              umma_commit(r.b_empty + bs * 8u);
            }
            accum = 1;
            bring_d += bsub16;
            if (++bs == nbst) { bs = 0; bphase ^= 1u; bring_d = bring_d0; }
          }
        } else if (fast_taps == 9) {
          // common filters: tap shifts in registers, straight-line issue (this lane pays ~6 cycles per
          // instruction, more per branch, and a shared-memory load per tap otherwise)
          // 3x3: the nine shifts live in registers (measured faster than forming them by additions)
          if (lane0) {
#pragma unroll
            for (int tap = 0; tap < 9; ++tap)
              umma_i8_block<kSteps>(d_tmem, a_d + shift9[tap], bres + (uint32_t)tap * btile16, idesc, tap == 0 ? accum : 1u);
          }
          accum = 1;
          bres += 9u * btile16;
        } else if (fast_taps == 25) {
          if (lane0) issue_taps<5, 5, false, kSteps>(d_tmem, a_d, p.row16, p.col16, bres, btile16, idesc, accum);
          accum = 1;
          bres += 25u * btile16;
        } else if (fast_taps == 28) {
          if (lane0) issue_taps<7, 4, true, kSteps>(d_tmem, a_d, p.row16, p.col16, bres, btile16, idesc, accum);
          accum = 1;
          bres += 28u * btile16;
        } else {
          if (lane0) {
            uint64_t bt = bres;
#pragma unroll 3
            for (int tap = 0; tap < taps; ++tap) {
              umma_i8_block<kSteps>(d_tmem, a_d + r.tap_shift16[tap], bt, idesc, accum);
              accum = 1;
              bt += btile16;
            }
          }
          accum = 1;
          bres += (uint32_t)taps * btile16;
        }
        if (lane0) umma_commit(r.a_empty + stage * 8u);
        a_d += stage16;
        if (++stage == nstages) { stage = 0; phase ^= 1u; a_d = a_d0; }
      }
    } else {
      uint64_t bres_tap = bres_nt, bres = bres_nt;  // iterations run over taps with the channel blocks innermost
      int cb = 0;
      if (p.splits > 1) {
        const int it0 = ti.sp * k_iters, tap0 = p.fd_cblocks.div(it0);
        cb = it0 - tap0 * c_blocks;
        bres_tap += (uint32_t)tap0 * btile16;
        bres = bres_tap + (uint32_t)(cb * taps) * btile16;
      }
      const uint32_t b_off16 = (uint32_t)kb * asub16;
      for (int it = 0; it < k_iters;) {
        const int nsub = min(kb, k_iters - it);
        if (!mbar_wait(r.a_full + stage * 8u, phase, r.abortp)) return false;
        if (it + nsub >= k_iters && lane0) mbar_arrive(turn_next);  // this tile's last wait is behind us
        tcgen05_fence_after();
        uint64_t sa = a_d, sb = a_d + b_off16;
        for (int j = 0; j < nsub; ++j) {
          if (lane0) umma_i8_block<kSteps>(d_tmem, sa, b_in_stage ? sb : bres, idesc, accum);
          accum = 1;
          sa += asub16;
          sb += bsub16;
          bres += (uint32_t)taps * btile16;
          if (++cb == c_blocks) { cb = 0; bres_tap += btile16; bres = bres_tap; }
        }
        if (lane0) umma_commit(r.a_empty + stage * 8u);
        it += nsub;
        a_d += stage16;
        if (++stage == nstages) { stage = 0; phase ^= 1u; a_d = a_d0; }
      }
    }
    ++my_k;
    if (lane0) umma_commit(r.acc_full + ab * 8u);
    ab += (uint32_t)L;
    while (ab >= nacc) { ab -= nacc; acc_par ^= 1u; }
    // step over the stages and ring tiles of the other lanes' tiles
    stage += skip_a;
    while (stage >= nstages) { stage -= nstages; phase ^= 1u; }
    a_d = a_d0 + stage * stage16;
    if (ring) {
      bs += skip_b;
      while (bs >= nbst) { bs -= nbst; bphase ^= 1u; }
      bring_d = bring_d0 + bs * bsub16;
    }
  }
  return true;
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
};

// Looked up once per process; the function-local static is initialised by exactly one thread, and the others
// wait for it (C++11), so no caller can see half-filled pointers.
const DriverFns& driver_fns() {
  static const DriverFns f = [] {
    DriverFns r;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess && qr == cudaDriverEntryPointSuccess)
      r.tiled = reinterpret_cast<EncodeTiledFn>(p);
    p = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &p, cudaEnableDefault, &qr) == cudaSuccess && qr == cudaDriverEntryPointSuccess)
      r.im2col = reinterpret_cast<EncodeIm2colFn>(p);
    return r;
  }();
  return f;
}


int pick_bk(int C) {
  // A pipeline iteration costs one TMA operation per operand (several hundred cycles whatever its size), so the
  // widest channel block that C reaches wins even when it pads C: out-of-range channels are zero filled by TMA
  // and cost tensor-core time only, which a short reduction has to spare.
  return C <= 32 ? 32 : (C <= 64 ? 64 : 128);
}

// Tile width: the multiple of 16 (power-of-two panels keep the 8-bit tile layout simple) that pads
// Cout least; short reductions are bandwidth bound and take narrower tiles, which leaves room for
// four TMEM accumulators and more tile buffers.
int pick_bn(int K, int kgemm) {
  const int cap = kgemm <= 640 ? 128 : 256;
  const double k_steps = (kgemm + 31) / 32, k_iters = (kgemm + 127) / 128;
  int best = 16;
  double best_cost = -1.0;
  for (int w = 16; w <= cap; w += 16) {
    const int n_tiles = (K + w - 1) / w;
    // cycles per 128-row block of the output: every tile of columns runs the whole reduction again (one
    // 128 x w x 32 MMA takes max(59, 0.53 w) cycles, a pipeline iteration about 550), the epilogue pays for
    // every padded column
    const double mma = k_steps * (0.53 * w > 59.0 ? 0.53 * w : 59.0), feed = k_iters * 550.0;
    const double cost = n_tiles * ((mma > feed ? mma : feed) + 200.0) + (double)n_tiles * w * 8.0;
    if (best_cost < 0 || cost <= best_cost) { best = w; best_cost = cost; }
  }
  return best;
}

CUtensorMapSwizzle swizzle_for_bytes(int row_bytes) {
  return row_bytes >= 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                          : (row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                             : (row_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE));
}

unsigned int round_up(unsigned int v, unsigned int a) { return (v + a - 1) / a * a; }

FastDiv make_fastdiv(int d) {
  FastDiv f;
  f.d = d < 1 ? 1 : d;
  unsigned int l = 0;
  while ((1ull << l) < (unsigned long long)f.d) ++l;
  f.l = l;
  f.m = (unsigned int)(((1ull << 32) * ((1ull << l) - (unsigned long long)f.d)) / (unsigned long long)f.d + 1ull);
  return f;
}

// Developer knobs for sweeps of tile shapes and pipeline depths.  They exist only in builds made with
// -DQ8_TUNE_KNOBS (the library proper never reads the environment) and are honoured only when Q8_TUNE is set.
// Every knob is confined to the range [lo, hi] that the plan supports at that point (the default always lies
// inside it); a value outside the range, or not a number, is ignored, so a typo cannot produce a launch whose
// shared-memory or TMEM plan does not hold.
//   Q8_PDL 0/1 dependent launch, Q8_HALO 0/1 halo tiles, Q8_BN tile width (multiple of 16), Q8_LANES 2/3 MMA warps,
//   Q8_SPLIT 0/1 column-split epilogue (only where the plan allows it), Q8_G 2/4 epilogue groups, Q8_BRES 0 weights
//   not resident, Q8_CTA2 0 no CTA pairs, Q8_CTA2SPLIT, Q8_CTA2MIN pair-mode thresholds, Q8_BT taps per weight-ring
//   stage, Q8_KB channel blocks per A stage, Q8_NBUF tile buffers per group, Q8_BSTAGES / Q8_STAGES ring depths (at
//   most what fits), Q8_GRID number of CTAs (at most the default).
int tune_env(const char* name, int dflt, int lo, int hi) {
#ifdef Q8_TUNE_KNOBS
  static const bool enabled = getenv("Q8_TUNE") != nullptr;
  if (!enabled) return dflt;
  const char* v = getenv(name);
  if (!v || !*v) return dflt;
  char* end = nullptr;
  const long x = strtol(v, &end, 10);
  if (end == v || *end != '\0' || x < lo || x > hi) return dflt;
  return (int)x;
#else
  (void)name; (void)lo; (void)hi;
  return dflt;
#endif
}

// Halo tiling of a stride-1 filter: TH x TW output pixels per tile, (TH + ext_h) x (TW + ext_w)
// input pixels per patch, TH * (TW + ext_w) <= 128 accumulator rows.  Picks the extents that waste
// the fewest accumulator rows, preferring less halo among near-equals.
struct HaloTile {
  int tw, th, twb, hb;
  double eff;  // useful output pixels per computed accumulator row
  int sw;      // stride along W: 1, or 2 = the input is read as pixel pairs [N, H, W/2, 2C]
  int s_eff;   // filter taps along W in that view
  int pad_w_eff, e;  // left padding in that view; parity of pad_w
};

// Stride 2 along W needs no data movement: with W even, NHWC memory is also a tensor of pixel pairs with 2C
// channels, and output column q reads pairs q + t' - pad', t' = 0 .. S'-1, i.e. a stride-1 filter of
// S' = ceil((S + e) / 2) taps (e = pad_w & 1).  Stride along H is served by tiles of one output row.
bool choose_halo_tile(const q8_conv_desc& d, int P, int Q, HaloTile* out) {
  const int sw = d.stride_w;
  if (sw != 1 && sw != 2) return false;
  int s_eff = d.S, pad_eff = d.pad_w, e = 0, dil_w = d.dil_w;
  if (sw == 2) {
    if (d.W % 2 || d.dil_w != 1 || (d.C != 16 && d.C != 32 && d.C != 64)) return false;
    e = d.pad_w & 1;
    s_eff = (d.S + e + 1) / 2;
    pad_eff = (d.pad_w + e) / 2;
    dil_w = 1;
    // this view keeps the weights resident in shared memory
    const int BN = pick_bn(d.K, d.R * d.S * d.C);
    if ((long long)((d.K + BN - 1) / BN) * BN * d.R * s_eff * 2 * d.C > 80 * 1024) return false;
  }
  const int taps = d.R * s_eff;
  if (taps < 2 || taps > kMaxTaps) return false;
  const int ext_w = (s_eff - 1) * dil_w, ext_h = (d.R - 1) * d.dil_h;
  HaloTile best = {0, 0, 0, 0, 0.0, sw, s_eff, pad_eff, e};
  double best_score = 0.0;
  for (int tw = 1; tw <= Q && tw + ext_w <= kBM; ++tw) {
    const int twb = tw + ext_w;
    int th = d.stride_h == 1 ? kBM / twb : 1;
    if (th > P) th = P;
    if (th < 1) continue;
    const int hb = (th - 1) * d.stride_h + ext_h + 1;
    if (hb > 256 || twb > 256) continue;
    const long long tiles = (long long)((Q + tw - 1) / tw) * ((P + th - 1) / th);
    const double eff = (double)P * Q / ((double)tiles * kBM);
    const double halo = (double)hb * twb / ((double)th * tw);
    const double score = eff / (1.0 + 0.04 * halo);
    if (score > best_score) { best_score = score; best.tw = tw; best.th = th; best.twb = twb; best.hb = hb; best.eff = eff; }
  }
  // Tiny images waste accumulator rows (a 7x7 image fills 49 of 128 rows).  Where the im2col path is
  // open it is the better choice for them (it can split the reduction); tensors below its size limit
  // still take halo tiles rather than leave the tensor cores.
  const bool im2col_closed = (long long)d.N * d.H * d.W * d.C < 131072;
  if (!im2col_closed && best.eff < 0.5) return false;
  if (best.tw == 0) return false;
  *out = best;
  return true;
}

}  // namespace
}  // namespace q8
