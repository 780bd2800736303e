// Quantized convolution as an implicit GEMM on the 5th-generation tensor cores (sm_100a).
//
//   D[M = N*P*Q pixels, Cout] (int32, in TMEM) = A[M, R*S*C] (u8/s8) x B[Cout, R*S*C]^T (s8)
//
// Persistent kernel: one CTA per SM walks over output tiles of 128 accumulator rows x BN channels.
// A lone control warp executes roughly one instruction every 6-10 cycles and every TMA operation
// occupies the SM's copy engine for at least ~370 cycles whatever its size, so the pipeline moves
// few, large pieces:
//
//   A operand, three sources
//     plain  : 1x1 / stride 1 / no padding.  The activation tensor is the [M][C] matrix itself; a
//              stage holds several consecutive 128 x BK channel blocks (2-D tiled loads).
//     halo   : stride 1 filters.  A tile is TH x TW output pixels of one image.  One 4-D tiled load
//              brings the (TH + halo) x (TW + halo) input patch of a channel block, zero filled
//              outside the image (the exact code of 0.0 under a symmetric quantizer).  Every filter
//              tap (r, s) is then the same patch read from a start address shifted by
//              (r*dil_h * patch width + s*dil_w) pixels: accumulator row i = pp * patch width + qq
//              is output pixel (pp, qq); rows with qq >= TW are computed and dropped.  Each input
//              byte crosses the L2 port about 1.5 times instead of R*S times.
//     im2col : everything else (strided, tiny images): one im2col-mode load per tap and channel
//              block, several of them per stage.
//   B operand (KRSC weights), three sources
//     resident : the whole layer's weights sit in shared memory for the CTA's lifetime;
//     ring     : (halo) BN x BK tiles per tap and channel block through their own ring, several taps per
//                stage (one TMA operation) for tiles up to 128 columns;
//     stage    : (plain, im2col) one BN x BK tile next to each A block of a stage.
//
// Roles (one lane each unless noted):
//   warp 0     : TMA producer of A patches / blocks and of B tiles;
//   warps 1, 4 : tcgen05.mma.kind::i8 issue (128 x BN x 32 per instruction, int32 accumulators in a
//                ring of up to four TMEM buffers), alternate tiles each, so that the per-tile
//                bookkeeping of one lane overlaps the issue of the other; tcgen05.commit releases
//                stages and publishes accumulators.  Warp 1 also owns the TMEM allocation;
//   warp 2     : hands 8-bit tile buffers to the epilogue groups, filled by TMA with the residual
//                tile of the fused eltwise sum when there is one;
//   warp 3     : sends finished 8-bit tiles to global memory with TMA stores, recycles the buffers;
//   warps 6..  : G epilogue groups of four warps; group g owns every G-th tile of the CTA, or, in launches
//                with at most two tiles per CTA, a share of the columns of every tile.  A thread
//                owns one accumulator row: tcgen05.ld, + bias, requantise, + residual, ReLU, round,
//                clamp; the 16 bytes go back into the buffer the residual came from (same swizzled
//                position), which then is the source of the TMA store.
// The kernel is launched with programmatic stream serialization: its set-up overlaps the tail of the kernel
// before it, and every global access comes after griddepcontrol.wait.
// All hand-offs are mbarriers, there is no block-wide barrier after the prologue.  Every wait is
// bounded in wall-clock time; on expiry a bit of the library's status word is set and all roles drain
// instead of hanging.
#include <cuda.h>

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

// Slow path of a wait, out of line to keep the role loops small.  Gives up after about
// kWaitLimitNs or when another role of this CTA has already given up; the caller then records the
// site and leaves its loop.  The wall clock is only read once the wait has lasted a while.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  unsigned long long t0 = 0;
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 0x3ffu) == 0) {
      if (*abort_flag) return false;
      const unsigned long long now = global_timer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitLimitNs) return false;
    }
  }
  return true;
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
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
  int n0;                  // first channel of the tile
  bool row_ok;             // the pixel exists (inside the image and below M)
  bool smem_ok;            // this accumulator row maps to a pixel of the tile (always, except halo tiles)
};

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
    off = ((uint32_t)t.srow << p.pw_shift) + (uint32_t)(c16 & ((1 << p.pw_shift) - 1));
    off ^= ((off >> 7) & (uint32_t)p.pmask) << 4;
    off += (uint32_t)pn * ((uint32_t)kBM << p.pw_shift);
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
  int total_tiles;
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
  ti.init(p, blockIdx.x + who * (int)gridDim.x, L * (int)gridDim.x);
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
        if (last_cb && !ring) mbar_arrive(turn_next);  // this tile's last wait is behind us
        tcgen05_fence_after();
        if (ring && bT == 1) {
          // (kept apart from the multi-tap loop below: every extra instruction of this lone lane costs ~6 cycles)
          for (int tap = 0; tap < taps; ++tap) {
            if (!mbar_wait(r.b_full + bs * 8u, bphase, r.abortp)) return false;
            if (last_cb && tap == taps - 1) mbar_arrive(turn_next);
            tcgen05_fence_after();
            umma_i8_block<kSteps>(d_tmem, a_d + r.tap_shift16[tap], bring_d, idesc, accum);
            accum = 1;
            umma_commit(r.b_empty + bs * 8u);
            bring_d += bsub16;
            if (++bs == nbst) { bs = 0; bphase ^= 1u; bring_d = bring_d0; }
          }
        } else if (ring && fast_taps == 9 && bT == 3) {
          // 3x3 in ring stages of one filter row each: straight-line issue with the shifts in registers
#pragma unroll
          for (int row = 0; row < 3; ++row) {
            if (!mbar_wait(r.b_full + bs * 8u, bphase, r.abortp)) return false;
            if (last_cb && row == 2) mbar_arrive(turn_next);
            tcgen05_fence_after();
#pragma unroll
            for (int t = 0; t < 3; ++t)
              umma_i8_block<kSteps>(d_tmem, a_d + shift9[3 * row + t], bring_d + (uint32_t)t * btile16, idesc, (row == 0 && t == 0) ? accum : 1u);
            accum = 1;
            umma_commit(r.b_empty + bs * 8u);
            bring_d += bsub16;
            if (++bs == nbst) { bs = 0; bphase ^= 1u; bring_d = bring_d0; }
          }
        } else if (ring) {
          for (int tap0 = 0; tap0 < taps; tap0 += bT) {
            if (!mbar_wait(r.b_full + bs * 8u, bphase, r.abortp)) return false;
            if (last_cb && tap0 + bT >= taps) mbar_arrive(turn_next);
            tcgen05_fence_after();
            const int nt = min(bT, taps - tap0);
            uint64_t bd = bring_d;
            for (int t = 0; t < nt; ++t, bd += btile16) {
              umma_i8_block<kSteps>(d_tmem, a_d + r.tap_shift16[tap0 + t], bd, idesc, accum);
              accum = 1;
            }
            umma_commit(r.b_empty + bs * 8u);
            bring_d += bsub16;
            if (++bs == nbst) { bs = 0; bphase ^= 1u; bring_d = bring_d0; }
          }
        } else if (fast_taps == 9) {
          // common filters: tap shifts in registers, straight-line issue (this lane pays ~6 cycles per
          // instruction, more per branch, and a shared-memory load per tap otherwise)
          // 3x3: the nine shifts live in registers (measured faster than forming them by additions)
#pragma unroll
          for (int tap = 0; tap < 9; ++tap)
            umma_i8_block<kSteps>(d_tmem, a_d + shift9[tap], bres + (uint32_t)tap * btile16, idesc, tap == 0 ? accum : 1u);
          accum = 1;
          bres += 9u * btile16;
        } else if (fast_taps == 25) {
          issue_taps<5, 5, false, kSteps>(d_tmem, a_d, p.row16, p.col16, bres, btile16, idesc, accum);
          accum = 1;
          bres += 25u * btile16;
        } else if (fast_taps == 28) {
          issue_taps<7, 4, true, kSteps>(d_tmem, a_d, p.row16, p.col16, bres, btile16, idesc, accum);
          accum = 1;
          bres += 28u * btile16;
        } else {
#pragma unroll 3
          for (int tap = 0; tap < taps; ++tap) {
            umma_i8_block<kSteps>(d_tmem, a_d + r.tap_shift16[tap], bres, idesc, accum);
            accum = 1;
            bres += btile16;
          }
        }
        umma_commit(r.a_empty + stage * 8u);
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
        if (it + nsub >= k_iters) mbar_arrive(turn_next);  // this tile's last wait is behind us
        tcgen05_fence_after();
        uint64_t sa = a_d, sb = a_d + b_off16;
        for (int j = 0; j < nsub; ++j) {
          umma_i8_block<kSteps>(d_tmem, sa, b_in_stage ? sb : bres, idesc, accum);
          accum = 1;
          sa += asub16;
          sb += bsub16;
          bres += (uint32_t)taps * btile16;
          if (++cb == c_blocks) { cb = 0; bres_tap += btile16; bres = bres_tap; }
        }
        umma_commit(r.a_empty + stage * 8u);
        it += nsub;
        a_d += stage16;
        if (++stage == nstages) { stage = 0; phase ^= 1u; a_d = a_d0; }
      }
    }
    ++my_k;
    umma_commit(r.acc_full + ab * 8u);
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

// The MMA lanes of the leader CTA of a pair (halo tiles, weight ring): the same schedule as mma_role, with
// tcgen05.mma.cta_group::2 over both CTAs' tiles and commits that arrive in both CTAs.
template <int kSteps>
__device__ __forceinline__ bool mma_role_pair(const UmmaParams& p, const MmaRoleArgs& r, const int who, const int vblock,
                                              const int vgrid) {
  TileIterT<true> ti;
  const int L = p.mma_lanes;
  ti.init(p, vblock + who * vgrid, L * vgrid, 0);
  const uint32_t nstages = (uint32_t)p.stages, nbst = (uint32_t)p.b_stages;
  const uint64_t hi = ((uint64_t)p.desc_hi << 32) | (1ull << 16);
  const uint64_t a_d0 = hi | (((r.base + p.off_a) >> 4) & 0x3fffu), bring_d0 = hi | (((r.base + p.off_bring) >> 4) & 0x3fffu);
  const uint32_t stage16 = p.a_stage_bytes >> 4, bsub16 = p.b_sub_bytes >> 4, btile16 = p.b_tile_bytes >> 4;
  const uint32_t idesc = p.idesc;
  const int taps = p.taps, c_blocks = p.c_blocks, bT = p.b_T;
  const uint32_t spt = (uint32_t)c_blocks, bpt = (uint32_t)(p.b_chunks * c_blocks);
  const uint32_t skip_a = (uint32_t)(L - 1) * spt, skip_b = (uint32_t)(L - 1) * bpt;
  uint32_t stage = ((uint32_t)who * spt) % nstages, phase = (((uint32_t)who * spt) / nstages) & 1u;
  uint32_t bs = ((uint32_t)who * bpt) % nbst, bphase = (((uint32_t)who * bpt) / nbst) & 1u;
  uint64_t a_d = a_d0 + stage * stage16, bring_d = bring_d0 + bs * bsub16;
  const uint32_t nacc = (uint32_t)p.nacc;
  uint32_t ab = (uint32_t)who % nacc, acc_par = 1u ^ (((uint32_t)who / nacc) & 1u);
  uint32_t my_k = 0;
  const uint32_t turn_next = r.turn + (uint32_t)((who + 1) % L) * 8u;
  const uint32_t turn_mine = r.turn + (uint32_t)who * 8u;
  const bool fast9 = p.fast_taps == 9 && bT == 3;
  uint32_t shift9[9];
#pragma unroll
  for (int t = 0; t < 9; ++t) shift9[t] = fast9 ? r.tap_shift16[t] : 0u;
  for (; ti.tile < r.total_tiles; ti.next(p)) {
    if (!mbar_wait(r.acc_empty + ab * 8u, acc_par, r.abortp)) return false;
    if (who == 0) { if (my_k > 0 && !mbar_wait(turn_mine, (my_k - 1) & 1u, r.abortp)) return false; }
    else if (!mbar_wait(turn_mine, my_k & 1u, r.abortp)) return false;
    tcgen05_fence_after();
    const uint32_t d_tmem = r.tmem_base + ab * (uint32_t)p.acc_stride;
    uint32_t accum = 0;
    for (int cb = 0; cb < c_blocks; ++cb) {
      if (!mbar_wait(r.a_full + stage * 8u, phase, r.abortp)) return false;
      const bool last_cb = cb == c_blocks - 1;
      tcgen05_fence_after();
      if (fast9) {
        // 3x3 in ring stages of one filter row each: straight-line issue with the shifts in registers
#pragma unroll
        for (int row = 0; row < 3; ++row) {
          if (!mbar_wait(r.b_full + bs * 8u, bphase, r.abortp)) return false;
          if (last_cb && row == 2) mbar_arrive(turn_next);
          tcgen05_fence_after();
#pragma unroll
          for (int t = 0; t < 3; ++t) {
            const uint64_t ad = a_d + shift9[3 * row + t], bd = bring_d + (uint32_t)t * btile16;
            umma_i8_pair(d_tmem, ad, bd, idesc, (row == 0 && t == 0) ? accum : 1u);
#pragma unroll
            for (int k = 1; k < kSteps; ++k) umma_i8_pair(d_tmem, ad + 2 * k, bd + 2 * k, idesc, 1u);
          }
          accum = 1;
          umma_commit_pair(r.b_empty + bs * 8u);
          bring_d += bsub16;
          if (++bs == nbst) { bs = 0; bphase ^= 1u; bring_d = bring_d0; }
        }
      }
      for (int tap0 = 0; !fast9 && tap0 < taps; tap0 += bT) {
        if (!mbar_wait(r.b_full + bs * 8u, bphase, r.abortp)) return false;
        if (last_cb && tap0 + bT >= taps) mbar_arrive(turn_next);
        tcgen05_fence_after();
        const int nt = min(bT, taps - tap0);
        uint64_t bd = bring_d;
        for (int t = 0; t < nt; ++t, bd += btile16) {
          const uint64_t ad = a_d + r.tap_shift16[tap0 + t];
          umma_i8_pair(d_tmem, ad, bd, idesc, accum);
#pragma unroll
          for (int k = 1; k < kSteps; ++k) umma_i8_pair(d_tmem, ad + 2 * k, bd + 2 * k, idesc, 1u);
          accum = 1;
        }
        umma_commit_pair(r.b_empty + bs * 8u);
        bring_d += bsub16;
        if (++bs == nbst) { bs = 0; bphase ^= 1u; bring_d = bring_d0; }
      }
      umma_commit_pair(r.a_empty + stage * 8u);
      a_d += stage16;
      if (++stage == nstages) { stage = 0; phase ^= 1u; a_d = a_d0; }
    }
    ++my_k;
    umma_commit_pair(r.acc_full + ab * 8u);
    ab += (uint32_t)L;
    while (ab >= nacc) { ab -= nacc; acc_par ^= 1u; }
    stage += skip_a;
    while (stage >= nstages) { stage -= nstages; phase ^= 1u; }
    a_d = a_d0 + stage * stage16;
    bs += skip_b;
    while (bs >= nbst) { bs -= nbst; bphase ^= 1u; }
    bring_d = bring_d0 + bs * bsub16;
  }
  return true;
}

// ------------------------------------------------------------------------------------------ kernel
// G epilogue groups; one instantiation per output type and residual source keeps a single epilogue
// body in each kernel (several of them in one kernel made the register allocator spill).
// kCta2: the CTA-pair variant (its cta_group::2 instructions make the kernel launchable as clusters of two only).
template <int G, int kOut, int kRes, bool kCta2>
__global__ void __launch_bounds__(kCtrlThreads + G * kGroupThreads, 1)
    conv_umma_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                     const __grid_constant__ CUtensorMap tmRes, const __grid_constant__ CUtensorMap tmY,
                     const __grid_constant__ UmmaParams p) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long a_full[kMaxStages], a_empty[kMaxStages];
  __shared__ __align__(8) unsigned long long b_full[kMaxBStages], b_empty[kMaxBStages];
  __shared__ __align__(8) unsigned long long acc_full[kMaxAcc], acc_empty[kMaxAcc];
  __shared__ __align__(8) unsigned long long buf_full[kMaxSlots], buf_empty[kMaxSlots];
  __shared__ __align__(8) unsigned long long store_ready[kMaxSlots];  // per buffer: a buffer is recycled by the store
                                                                        // lane between two uses, so no phase can be skipped
  __shared__ __align__(8) unsigned long long bres_full;
  __shared__ __align__(8) unsigned long long mma_turn[kMmaWarps];
  __shared__ uint32_t tap_shift16[kMaxTaps];  // halo: descriptor start offset of a tap, in 16-byte units
  __shared__ uint32_t tmem_holder;
  __shared__ int abort_flag;

  // dynamic smem: [resident weights] [A stages] [weight ring] [G*nbuf 8-bit tile buffers] [bias, scale]
  const uint32_t raw_base = smem_u32(smem_raw);
  const uint32_t base = (raw_base + 1023u) & ~1023u;
  unsigned char* const base_ptr = smem_raw + (base - raw_base);
  int* const s_bias = reinterpret_cast<int*>(base_ptr + p.off_chan);
  float* const s_scale = reinterpret_cast<float*>(base_ptr + p.off_chan) + p.k_pad;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // CTA pairs: both CTAs walk the same sequence of work items (pairs of m tiles); rank 1 takes the second tile
  int cta_rank = 0;
  if constexpr (kCta2) cta_rank = (int)cluster_ctarank();
  const int vblock = kCta2 ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int vgrid = kCta2 ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  const int total_tiles = p.m_tiles * p.n_tiles * p.splits;  // work items
  const int slots = p.epi_split ? p.nbuf : G * p.nbuf;  // split mode: nbuf counts the buffers of the CTA

  // Programmatic dependent launch: the next kernel of the stream may be scheduled onto SMs as they fall idle
  // (it waits below, like this one, before it touches global memory), and this kernel's own set-up (barriers,
  // TMEM allocation, descriptor prefetch) runs while the previous kernel drains.  Both are no-ops for a
  // launch without the attribute.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // Prologue.  Each control lane initialises the barriers it owns.  Warp 0 only signals the
  // start-up barrier (bar.arrive) and goes straight to its loads, so that the first bytes are on
  // their way while the others allocate TMEM and fetch bias and scale; everybody else waits on it.
  const int nthreads = kCtrlThreads + G * kGroupThreads;
  if (warp == 0) {
    // one barrier per lane: a lone lane would spend ~50 cycles on each
    if (lane < p.stages) { mbar_init(smem_u32(&a_full[lane]), 1); mbar_init(smem_u32(&a_empty[lane]), 1); }
    else if (lane >= 8 && lane - 8 < p.b_stages) { mbar_init(smem_u32(&b_full[lane - 8]), 1); mbar_init(smem_u32(&b_empty[lane - 8]), 1); }
    else if (lane == 16) { mbar_init(smem_u32(&bres_full), 1); abort_flag = 0; }
    else if (lane == 17) prefetch_tensormap(&tmA);
    else if (lane == 18) prefetch_tensormap(&tmB);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncwarp();
    asm volatile("griddepcontrol.wait;" ::: "memory");  // everything the previous kernel wrote is visible from here
    if constexpr (kCta2) cluster_sync_all();  // the peer's barriers exist before anything signals them
    asm volatile("bar.arrive 1, %0;" ::"r"(nthreads) : "memory");
  } else {
    if (warp == 1) {
      // one arrival per epilogue warp that reads the accumulator: a group's four, or all of them in split mode
      if (lane < p.nacc) { mbar_init(smem_u32(&acc_full[lane]), 1); mbar_init(smem_u32(&acc_empty[lane]), (p.epi_split ? 4 * G : 4) * (kCta2 ? 2 : 1)); }
      else if (lane >= 8 && lane - 8 < kMmaWarps) mbar_init(smem_u32(&mma_turn[lane - 8]), 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    } else if (warp == 2) {
      if (lane < slots) { mbar_init(smem_u32(&buf_full[lane]), 1); mbar_init(smem_u32(&buf_empty[lane]), 1); }
      else if (lane == 16 && p.res_mode == kResTma) prefetch_tensormap(&tmRes);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    } else if (warp == 3) {
      if (lane < slots) mbar_init(smem_u32(&store_ready[lane]), p.epi_split ? G * kGroupThreads : kGroupThreads);
      else if (lane == 16 && p.out8) prefetch_tensormap(&tmY);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
      __syncwarp();
      if constexpr (kCta2) {
        tmem_alloc_pair(smem_u32(&tmem_holder), (uint32_t)p.tmem_cols);
        tmem_relinquish_pair();
      } else {
        tmem_alloc(smem_u32(&tmem_holder), (uint32_t)p.tmem_cols);
        tmem_relinquish();
      }
    }
    if (p.a_mode == kAHalo && threadIdx.x >= 32 && threadIdx.x - 32 < p.taps) tap_shift16[threadIdx.x - 32] = p.tap_shift16[threadIdx.x - 32];
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // bias and scale of every channel, once per CTA (zero beyond Cout; one scale replicated if per tensor)
    for (int i = threadIdx.x - 32; i < p.k_pad; i += nthreads - 32) {
      s_bias[i] = (p.bias && i < p.K) ? p.bias[i] : 0;
      s_scale[i] = p.scale ? (p.scale_count == 1 ? p.scale[0] : (i < p.K ? p.scale[i] : 0.f)) : 0.f;
    }
    tcgen05_fence_before();
    if constexpr (kCta2) {
      __syncwarp();
      cluster_sync_all();
    }
    asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory");
    tcgen05_fence_after();
  }
  const uint32_t tmem_base = warp == 0 ? 0u : tmem_holder;  // warp 0 never touches TMEM
  volatile int* abortp = &abort_flag;

  if (threadIdx.x == 0) {
    // ------------------------------------------------------------------ A / B producer
    TileIterT<kCta2> ti;
    ti.init(p, vblock, vgrid, cta_rank);
    const uint32_t nstages = (uint32_t)p.stages, nbst = (uint32_t)p.b_stages;
    const uint32_t afull0 = smem_u32(&a_full[0]), aempty0 = smem_u32(&a_empty[0]);
    const uint32_t bfull0 = smem_u32(&b_full[0]), bempty0 = smem_u32(&b_empty[0]);
    const uint32_t a0 = base + p.off_a, bring0 = base + p.off_bring;
    uint32_t stage = 0, phase = 0, a_dst = a0;
    uint32_t bs = 0, bphase = 0, b_dst = bring0;
    bool ok = true;
    if (p.b_mode == kBResident) {
      // every weight tile of the layer, once: one load per (n tile, channel block) brings all taps,
      // laid out [tap][bn rows][bk bytes], i.e. one K-major operand tile per tap
      const uint32_t bar = smem_u32(&bres_full);
      uint32_t dst = base;
      mbar_arrive_expect_tx(bar, (uint32_t)(p.n_tiles * p.c_blocks * p.taps) * p.b_tile_bytes);
      if (p.a_mode == kAHalo && p.halo_sw == 2) {
        // pixel-pair taps: tap t' of a filter row covers s = 2t' - e and 2t' - e + 1, whose weights are 2C
        // contiguous bytes of the (s, c) axis; a start left of s = 0 is zero filled.  One load per t' brings
        // all R filter rows: tile order (t', r).
        for (int nt = 0; nt < p.n_tiles; ++nt)
          for (int t = 0; t < p.S; ++t, dst += (uint32_t)p.R * p.b_tile_bytes) tma_load_3d(dst, &tmB, bar, (2 * t - p.halo_e) * p.c_true, nt * p.bn, 0);
      } else {
        for (int nt = 0; nt < p.n_tiles; ++nt)
          for (int c = 0; c < p.C_pad; c += p.bk, dst += (uint32_t)p.taps * p.b_tile_bytes) tma_load_3d(dst, &tmB, bar, c, nt * p.bn, 0);
      }
    }
    if (p.a_mode == kAHalo) {
      const uint32_t b_tx = (uint32_t)p.b_T * p.b_tile_bytes;
      for (; ti.tile < total_tiles && ok; ti.next(p)) {
        const int n0 = ti.nt * p.bn + (kCta2 ? cta_rank * (p.bn >> 1) : 0);
        const int q0 = ti.qt * p.tw - p.pad_w, p0 = ti.pt * p.th * p.stride_h - p.pad_h;
        for (int c = 0; c < p.C_pad && ok; c += p.bk) {
          if (!mbar_wait(aempty0 + stage * 8u, phase ^ 1u, abortp)) { ok = false; break; }
          const uint32_t bar = afull0 + stage * 8u;
          if constexpr (kCta2) {
            // the leader's barrier counts the bytes of both CTAs' patches
            if (cta_rank == 0) mbar_arrive_expect_tx(bar, 2u * p.a_sub_bytes);
            tma_load_4d_pair(a_dst, &tmA, map_to_cta(bar, 0), c, q0, p0, ti.img);
          } else {
            mbar_arrive_expect_tx(bar, p.a_sub_bytes);
            tma_load_4d(a_dst, &tmA, bar, c, q0, p0, ti.img);
          }
          a_dst += p.a_stage_bytes;
          if (++stage == nstages) { stage = 0; phase ^= 1u; a_dst = a0; }
          if (p.b_mode == kBRing) {
            // one operation brings the weight tiles of b_T taps (a box that runs past the last tap is zero filled
            // and still counts in full): the copy engine spends ~600 cycles per operation whatever its size
            for (int tap = 0; tap < p.taps; tap += p.b_T) {
              if (!mbar_wait(bempty0 + bs * 8u, bphase ^ 1u, abortp)) { ok = false; break; }
              const uint32_t bbar = bfull0 + bs * 8u;
              if constexpr (kCta2) {
                if (cta_rank == 0) mbar_arrive_expect_tx(bbar, 2u * b_tx);
                tma_load_3d_pair(b_dst, &tmB, map_to_cta(bbar, 0), c, n0, tap);
              } else {
                mbar_arrive_expect_tx(bbar, b_tx);
                tma_load_3d(b_dst, &tmB, bbar, c, n0, tap);
              }
              b_dst += p.b_sub_bytes;
              if (++bs == nbst) { bs = 0; bphase ^= 1u; b_dst = bring0; }
            }
          }
        }
      }
    } else {
      const uint32_t sub_tx = p.a_sub_bytes + (p.b_mode == kBStage ? p.b_tile_bytes : 0u);
      const uint32_t b_in_stage = (uint32_t)p.kb * p.a_sub_bytes;
      for (; ti.tile < total_tiles && ok; ti.next(p)) {
        const int m0 = ti.mt * kBM, n0 = ti.nt * p.bn;
        int w0 = 0, h0 = 0, img = 0;
        if (p.a_mode == kAIm2col) {
          img = p.fd_pq.div(m0);
          const int rem = m0 - img * p.PQ;
          const int pr = p.fd_q.div(rem), qc = rem - pr * p.Q;
          h0 = pr * p.stride_h - p.pad_h;
          w0 = qc * p.stride_w - p.pad_w;
        }
        int c = 0, tap = 0, s = 0, off_w = 0, off_h = 0;
        if (p.splits > 1) {  // this split starts at iteration sp * kps = (tap, channel block)
          const int it0 = ti.sp * p.kps;
          tap = p.fd_cblocks.div(it0);
          c = (it0 - tap * p.c_blocks) * p.bk;
          const int r0 = p.fd_s.div(tap);
          s = tap - r0 * p.S;
          off_w = s * p.dil_w; off_h = r0 * p.dil_h;
        }
        for (int it = 0; it < p.kps;) {
          const int nsub = min(p.kb, p.kps - it);
          if (!mbar_wait(aempty0 + stage * 8u, phase ^ 1u, abortp)) { ok = false; break; }
          const uint32_t bar = afull0 + stage * 8u;
          mbar_arrive_expect_tx(bar, (uint32_t)nsub * sub_tx);
          uint32_t dst = a_dst, bdst = a_dst + b_in_stage;
          for (int j = 0; j < nsub; ++j) {
            if (p.a_mode == kAIm2col) tma_load_im2col_4d(dst, &tmA, bar, c, w0, h0, img, (unsigned short)off_w, (unsigned short)off_h);
            else tma_load_2d(dst, &tmA, bar, c, m0);
            if (p.b_mode == kBStage) tma_load_3d(bdst, &tmB, bar, c, tap, n0);
            dst += p.a_sub_bytes;
            bdst += p.b_sub_bytes;
            c += p.bk;
            if (c >= p.C_pad) {  // next tap
              c = 0; ++tap; ++s; off_w += p.dil_w;
              if (s == p.S) { s = 0; off_w = 0; off_h += p.dil_h; }
            }
          }
          it += nsub;
          a_dst += p.a_stage_bytes;
          if (++stage == nstages) { stage = 0; phase ^= 1u; a_dst = a0; }
        }
      }
    }
    if (!ok) {
      abort_flag = 1;
      atomicOr(p.status, kTimeoutProducer);
    }
  } else if (threadIdx.x == 32 || threadIdx.x == 128 || (threadIdx.x == 160 && p.mma_lanes == 3)) {
    // ------------------------------------------------------------------ MMA issuers (lane 0 of warps 1, 4 and 5)
    const int who = threadIdx.x == 32 ? 0 : (threadIdx.x == 128 ? 1 : 2);
    MmaRoleArgs ra;
    ra.base = base; ra.tmem_base = tmem_base; ra.total_tiles = total_tiles; ra.abortp = abortp;
    ra.a_full = smem_u32(&a_full[0]); ra.a_empty = smem_u32(&a_empty[0]);
    ra.b_full = smem_u32(&b_full[0]); ra.b_empty = smem_u32(&b_empty[0]);
    ra.acc_full = smem_u32(&acc_full[0]); ra.acc_empty = smem_u32(&acc_empty[0]);
    ra.bres_full = smem_u32(&bres_full); ra.tap_shift16 = tap_shift16; ra.turn = smem_u32(&mma_turn[0]);
    bool ok = true;
    if constexpr (kCta2) {
      if (cta_rank == 0) ok = p.ksteps == 4 ? mma_role_pair<4>(p, ra, who, vblock, vgrid) : mma_role_pair<2>(p, ra, who, vblock, vgrid);
    } else {
      if (p.ksteps == 4) ok = mma_role<4>(p, ra, who);
      else if (p.ksteps == 2) ok = mma_role<2>(p, ra, who);
      else ok = mma_role<1>(p, ra, who);
    }
    if (!ok) {
      abort_flag = 1;
      atomicOr(p.status, kTimeoutMma);
    }
  } else if (threadIdx.x == 64) {
    // ------------------------------------------------------------------ tile-buffer / residual producer
    if (p.nbuf > 0) {
      TileIterT<kCta2> ti;
      ti.init(p, vblock, vgrid, cta_rank);
      const uint32_t bfull0 = smem_u32(&buf_full[0]), bempty0 = smem_u32(&buf_empty[0]);
      const uint32_t nslots = (uint32_t)slots;
      uint32_t slot = 0, par = 1;  // slots are used round robin over all groups: tile lt -> slot lt % (G*nbuf)
      bool ok = true;
      const int pw = 1 << p.pw_shift;
      const uint32_t panel_bytes = (uint32_t)kBM << p.pw_shift;
      for (; ti.tile < total_tiles; ti.next(p)) {
        if (!mbar_wait(bempty0 + slot * 8u, par, abortp)) { ok = false; break; }
        const uint32_t bar = bfull0 + slot * 8u;
        if (p.res_mode == kResTma && ti.valid) {
          uint32_t dst = base + p.off_bufs + slot * p.tile8_bytes;
          mbar_arrive_expect_tx(bar, p.res_tx_bytes);
          if (p.a_mode == kAHalo) {
            for (int pn = 0, c = ti.nt * p.bn; pn < p.panels; ++pn, c += pw, dst += panel_bytes) tma_load_4d(dst, &tmRes, bar, c, ti.qt * p.tw, ti.pt * p.th, ti.img);
          } else {
            for (int pn = 0, c = ti.nt * p.bn; pn < p.panels; ++pn, c += pw, dst += panel_bytes) tma_load_2d(dst, &tmRes, bar, c, ti.mt * kBM);
          }
        } else {
          mbar_arrive(bar);
        }
        if (++slot == nslots) { slot = 0; par ^= 1u; }
      }
      if (!ok) {
        abort_flag = 1;
        atomicOr(p.status, kTimeoutResidual);
      }
    }
  } else if (threadIdx.x == 96) {
    // ------------------------------------------------------------------ output store / buffer recycler
    if (p.nbuf > 0) {
      TileIterT<kCta2> ti;
      ti.init(p, vblock, vgrid, cta_rank);
      const uint32_t bempty0 = smem_u32(&buf_empty[0]), ready0 = smem_u32(&store_ready[0]);
      const uint32_t nslots = (uint32_t)slots;
      uint32_t slot = 0, spar = 0;  // tile lt uses buffer lt % (G*nbuf); its use number (lt / (G*nbuf)) gives the parity
      int prev_slot = -1;
      bool ok = true;
      const int pw = 1 << p.pw_shift;
      const uint32_t panel_bytes = (uint32_t)kBM << p.pw_shift;
      for (; ti.tile < total_tiles; ti.next(p)) {
        if (!mbar_wait(ready0 + slot * 8u, spar, abortp)) { ok = false; break; }
        if (p.out8) {
          uint32_t src = base + p.off_bufs + slot * p.tile8_bytes;
          if (!ti.valid) {
            // second tile of the last pair of an odd count: nothing to store
          } else if (p.a_mode == kAHalo) {
            for (int pn = 0, c = p.c_off + ti.nt * p.bn; pn < p.panels; ++pn, c += pw, src += panel_bytes) tma_store_4d(&tmY, src, c, ti.qt * p.tw, ti.pt * p.th, ti.img);
          } else {
            for (int pn = 0, c = p.c_off + ti.nt * p.bn; pn < p.panels; ++pn, c += pw, src += panel_bytes) tma_store_2d(&tmY, src, c, ti.mt * kBM);
          }
          bulk_commit();
          // the store before this one has read its buffer: hand that buffer back
          bulk_wait_read<1>();
          if (prev_slot >= 0) mbar_arrive(bempty0 + (uint32_t)prev_slot * 8u);
          prev_slot = (int)slot;
        } else {
          mbar_arrive(bempty0 + slot * 8u);
        }
        if (++slot == nslots) { slot = 0; spar ^= 1u; }
      }
      if (p.out8) {
        bulk_wait_read<0>();  // the CTA's shared memory must outlive the reads of its last stores
        if (prev_slot >= 0) mbar_arrive(bempty0 + (uint32_t)prev_slot * 8u);
      }
      if (!ok) {
        abort_flag = 1;
        atomicOr(p.status, kTimeoutStore);
      }
    }
  } else if (warp >= kCtrlWarps) {
    // ------------------------------------------------------------------ epilogue groups
    const int g = (warp - kCtrlWarps) >> 2;
    const int quad = warp & 3;  // TMEM lane quadrant this warp may read
    const int row = quad * 32 + lane;  // accumulator row of this thread
    EpiTile t;
    t.s_bias = s_bias;
    t.s_scale = s_scale;
    // halo tiles: accumulator row -> pixel (pp, qq) of the patch grid; rows right of the tile are dropped
    int pp = 0, qq = 0;
    t.srow = row;
    t.smem_ok = true;
    if (p.a_mode == kAHalo) {
      pp = row / p.twb;  // once per thread
      qq = row - pp * p.twb;
      t.smem_ok = pp < p.th && qq < p.tw;
      t.srow = t.smem_ok ? pp * p.tw + qq : 0;
    }
    // this group's tiles are lt = g, g + G, ... of the CTA's sequence; ring positions advance by additions
    // pair mode: the accumulators of both CTAs are handed back on the leader's barriers
    const uint32_t accf0 = smem_u32(&acc_full[0]);
    uint32_t acce0 = smem_u32(&acc_empty[0]);
    if constexpr (kCta2) acce0 = map_to_cta(acce0, 0);
    const uint32_t bfull0 = smem_u32(&buf_full[0]), ready0 = smem_u32(&store_ready[0]);
    const uint32_t nslots = (uint32_t)slots, nacc = (uint32_t)p.nacc;
    // split mode: every group works on every tile and takes the chunks [ch0, ch1) of its columns, so that a
    // launch with one or two tiles per CTA does not leave three of four groups idle
    const bool split = p.epi_split != 0;
    const int tile_step = split ? 1 : G;
    const int nchunk_all = p.bn >> 4;
    const int ch0 = split ? (g * nchunk_all) / G : 0, ch1 = split ? ((g + 1) * nchunk_all) / G : nchunk_all;
    uint32_t ab = split ? 0u : (uint32_t)g % nacc, acc_par = split ? 0u : ((uint32_t)g / nacc) & 1u;
    uint32_t slot = split ? 0u : (uint32_t)g, slot_par = 0;
    TileIterT<kCta2> ti;
    ti.init(p, vblock + (split ? 0 : g) * vgrid, tile_step * vgrid, cta_rank);
    for (; ti.tile < total_tiles; ti.next(p)) {
      bool ok = mbar_wait(accf0 + ab * 8u, acc_par, abortp);
      if (p.nbuf > 0 && ok) ok = mbar_wait(bfull0 + slot * 8u, slot_par, abortp);
      ok = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
      if (!ok) {
        if (lane == 0) {
          abort_flag = 1;
          atomicOr(p.status, kTimeoutEpilogue);
        }
        break;
      }
      tcgen05_fence_after();
      t.n0 = ti.nt * p.bn;
      t.y_off = (long long)ti.sp * p.split_stride;
      if (p.a_mode == kAHalo) {
        const int pr = ti.pt * p.th + pp, qc = ti.qt * p.tw + qq;
        t.row_ok = t.smem_ok && pr < p.P && qc < p.Q && ti.valid;
        t.m = ((long long)ti.img * p.P + pr) * p.Q + qc;
      } else {
        t.m = (long long)ti.mt * kBM + row;
        t.row_ok = t.m < p.M;
      }
      t.buf = p.nbuf > 0 ? base_ptr + p.off_bufs + (size_t)slot * p.tile8_bytes : nullptr;
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + ab * (uint32_t)p.acc_stride;
      epilogue_row<kOut, kRes, kCta2>(p, t, taddr, acce0 + ab * 8u, lane, ch0, ch1);
      if (p.nbuf > 0) {
        // this thread's reads and writes of the buffer are done; the store thread takes over
        if (p.out8) fence_proxy_async_smem();
        mbar_arrive(ready0 + slot * 8u);
      }
      ab += (uint32_t)tile_step;
      while (ab >= nacc) { ab -= nacc; acc_par ^= 1u; }
      slot += (uint32_t)tile_step;
      if (slot >= nslots) { slot -= nslots; slot_par ^= 1u; }
    }
  }

  tcgen05_fence_before();
  __syncthreads();
  if constexpr (kCta2) cluster_sync_all();  // the peer may still read this CTA's weight halves and signal its barriers until here
  if (warp == 1) {
    __syncwarp();
    tcgen05_fence_after();
    if constexpr (kCta2) tmem_dealloc_pair(tmem_base, (uint32_t)p.tmem_cols);
    else tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
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

// Developer knobs for sweeps of tile shapes and pipeline depths: honoured only when Q8_TUNE is set in the
// environment (looked up once per process), so that a normal launch never reads the environment.
int tune_env(const char* name, int dflt) {
  static const bool enabled = getenv("Q8_TUNE") != nullptr;
  if (!enabled) return dflt;
  const char* v = getenv(name);
  return v && *v ? atoi(v) : dflt;
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

template <int G, int kOut, int kRes, bool kCta2>
int launch_variant(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmRes, const CUtensorMap& tmY,
                   const UmmaParams& p, size_t dyn, int grid, cudaStream_t stream) {
  auto kernel = conv_umma_kernel<G, kOut, kRes, kCta2>;
  static bool configured = false;  // per instantiation
  if (!configured) {
    int rc = check_cuda(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit - kStaticSmemReserve),
                        "conv_umma: set shared memory size");
    if (rc != Q8_OK) return rc;
    configured = true;
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3((unsigned)(kCtrlThreads + G * kGroupThreads));
  cfg.dynamicSmemBytes = dyn;
  cfg.stream = stream;
  // let this kernel's set-up overlap the tail of the kernel before it in the stream
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = tune_env("Q8_PDL", 1) ? 1 : 0;
  if (p.cta2) {  // CTA pairs: clusters of two, beside the dependent launch
    const int pdl = (int)cfg.numAttrs;
    attr[pdl].id = cudaLaunchAttributeClusterDimension;
    attr[pdl].val.clusterDim.x = 2;
    attr[pdl].val.clusterDim.y = 1;
    attr[pdl].val.clusterDim.z = 1;
    cfg.numAttrs = pdl + 1;
  }
  const cudaError_t le = cudaLaunchKernelEx(&cfg, kernel, tmA, tmB, tmRes, tmY, p);
  if (le != cudaSuccess) {
    cudaGetLastError();
    return fail(Q8_ERR_CUDA, "conv_umma: launch failed (%s; grid %d, block %d, shared memory %zu, cluster %d)", cudaGetErrorString(le),
                grid, kCtrlThreads + G * kGroupThreads, dyn, p.cta2 ? 2 : 1);
  }
  return check_launch("conv_umma_kernel");
}

template <int G>
int launch_groups(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmRes, const CUtensorMap& tmY,
                  const UmmaParams& p, size_t dyn, int grid, cudaStream_t stream) {
#define Q8_LAUNCH(OUT, RES) return launch_variant<G, OUT, RES, false>(tmA, tmB, tmRes, tmY, p, dyn, grid, stream)
  // kResTma stands for "a residual through the tile buffers, or none"
  const bool global_res = p.res_mode == kResGlobal;
  if (p.y_type == Q8_U8) {
    if (global_res) Q8_LAUNCH(Q8_U8, kResGlobal);
    Q8_LAUNCH(Q8_U8, kResTma);
  }
  if (p.y_type == Q8_S8) {
    if (global_res) Q8_LAUNCH(Q8_S8, kResGlobal);
    Q8_LAUNCH(Q8_S8, kResTma);
  }
  if (p.y_type == Q8_F32) {
    if (global_res) Q8_LAUNCH(Q8_F32, kResGlobal);
    Q8_LAUNCH(Q8_F32, kResTma);
  }
  Q8_LAUNCH(Q8_S32, kResTma);
#undef Q8_LAUNCH
}

bool is_plain(const q8_conv_desc& d) {
  return d.R == 1 && d.S == 1 && d.stride_h == 1 && d.stride_w == 1 && d.pad_h == 0 && d.pad_w == 0;
}

}  // namespace

bool umma_shape_eligible(const q8_conv_desc& d, const char** why) {
  const char* dummy;
  if (!why) why = &dummy;
  if (d.C % 16) { *why = "C is not a multiple of 16"; return false; }
  if (d.K > 4096) { *why = "more than 4096 output channels"; return false; }
  if (is_plain(d)) return true;
  HaloTile ht;
  const int P = conv_out_extent(d.H, d.pad_h, d.dil_h, d.R, d.stride_h), Q = conv_out_extent(d.W, d.pad_w, d.dil_w, d.S, d.stride_w);
  if (choose_halo_tile(d, P, Q, &ht)) return true;
  // im2col tensor maps: corners are 8-bit signed, tap offsets 8-bit unsigned, strides at most 8
  const int up_w = d.pad_w - (d.S - 1) * d.dil_w, up_h = d.pad_h - (d.R - 1) * d.dil_h;
  if (d.pad_w > 128 || d.pad_h > 128 || up_w < -128 || up_h < -128 || up_w > 127 || up_h > 127) { *why = "padding/dilation outside the im2col corner range"; return false; }
  if ((d.S - 1) * d.dil_w > 255 || (d.R - 1) * d.dil_h > 255) { *why = "filter extent outside the im2col offset range"; return false; }
  if (d.stride_h > 8 || d.stride_w > 8) { *why = "stride > 8"; return false; }
  if ((long long)d.N * d.H * d.W * d.C < 131072) { *why = "activation tensor smaller than 128 KiB"; return false; }
  return true;
}

// Split-K plan: layers whose output tiles cannot occupy a quarter of the SMs split the reduction over
// (tap, channel block) iterations into `splits` equal parts; every part writes raw int32 partial sums
// (integer addition is associative, so the result stays bit exact).  Only the plain and im2col operand
// paths split.  Returns 1 when the layer runs unsplit.
int umma_plan_splits(const q8_conv_desc& d, int P, int Q, long long M) {
  if (!umma_shape_eligible(d, nullptr)) return 1;
  HaloTile ht;
  if (!is_plain(d) && choose_halo_tile(d, P, Q, &ht)) return 1;
  const int BK = pick_bk(d.C), BN = pick_bn(d.K, d.R * d.S * d.C);
  const long long tiles = ((M + kBM - 1) / kBM) * ((d.K + BN - 1) / BN);
  const int k_iters = d.R * d.S * ((d.C + BK - 1) / BK);
  const int sms = sm_count();
  // a split costs a second (small) kernel and the partial-sum traffic: it pays once most SMs would idle
  if (tiles * 4 > sms) return 1;
  int best = 1;
  for (int sp = 2; sp <= 16 && tiles * sp <= sms; ++sp)
    if (k_iters % sp == 0 && k_iters / sp >= 4) best = sp;
  return best;
}

namespace {
constexpr int kPlanNoFit = -1000;  // internal: this tile shape needs more shared memory than an SM has
int launch_conv_umma_plan(const ConvArgs& a, int splits, int bk_cap, bool allow_halo);

// Tries tile shapes from the preferred one down: halo patches of dilated filters on wide channel blocks can
// exceed shared memory, narrower channel blocks shrink them; im2col loads need the least.
int launch_conv_umma_impl(const ConvArgs& a, int splits) {
  static const struct { int bk_cap; bool halo; } kTries[] = {{128, true}, {64, true}, {32, true}, {128, false}, {64, false}};
  for (const auto& t : kTries) {
    const int rc = launch_conv_umma_plan(a, splits, t.bk_cap, t.halo);
    if (rc != kPlanNoFit) return rc;
  }
  return fail(Q8_ERR_UNSUPPORTED, "conv_umma: no tile shape of this layer fits in shared memory");
}
}  // namespace

int launch_conv_umma(const ConvArgs& a) {
  const q8_conv_desc& d = a.d;
  const int splits = umma_plan_splits(d, a.P, a.Q, a.M);
  const size_t need = splits > 1 ? (size_t)splits * (size_t)a.M * d.K * sizeof(int) : 0;
  if (splits > 1 && d.y_type != Q8_S32 && a.workspace && a.workspace_bytes >= need && aligned16(a.workspace)) {
    // pass 1: raw partial accumulators of every split into the workspace; pass 2: sum, bias, epilogue
    ConvArgs part = a;
    part.d.y_type = Q8_S32;
    part.d.relu = 0;
    part.y = a.workspace;
    part.ldc = d.K;
    part.c_off = 0;
    part.bias = nullptr;
    part.residual = nullptr;
    int rc = launch_conv_umma_impl(part, splits);
    if (rc != Q8_OK) return rc;
    return launch_splitk_reduce(a, splits);
  }
  return launch_conv_umma_impl(a, 1);
}

namespace {
int launch_conv_umma_plan(const ConvArgs& a, int splits, int bk_cap, bool allow_halo) {
  const q8_conv_desc& d = a.d;
  DriverFns& fn = driver_fns();
  if (!fn.tiled || !fn.im2col) return fail(Q8_ERR_CUDA, "conv_umma: cuTensorMapEncode* entry points not available");
  unsigned int* status = status_word_device_ptr();
  if (!status) return fail(Q8_ERR_CUDA, "conv_umma: status word not available");

  const bool out8 = d.y_type == Q8_U8 || d.y_type == Q8_S8;
  int res_mode = kResNone;
  if (a.residual) res_mode = (d.K % 16 == 0 && aligned16(a.residual)) ? kResTma : kResGlobal;
  UmmaParams p;
  memset(&p, 0, sizeof(p));
  HaloTile ht = {0, 0, 0, 0, 0.0, 1, d.S, d.pad_w, 0};
  p.a_mode = is_plain(d) ? kAPlain : ((allow_halo && tune_env("Q8_HALO", 1) && choose_halo_tile(d, a.P, a.Q, &ht)) ? kAHalo : kAIm2col);
  const bool paired = p.a_mode == kAHalo && ht.sw == 2;  // input read as pixel pairs with 2C channels
  const int c_eff = paired ? 2 * d.C : d.C;
  const int BK = pick_bk(c_eff) < bk_cap ? pick_bk(c_eff) : bk_cap;
  const int BN = tune_env("Q8_BN", pick_bn(d.K, d.R * d.S * d.C));
  const CUtensorMapSwizzle swz = swizzle_for_bytes(BK);
  p.bn = BN; p.bk = BK; p.ksteps = BK / 32;
  p.P = a.P; p.Q = a.Q; p.PQ = a.P * a.Q; p.M = (int)a.M; p.K = d.K;
  p.stride_h = d.stride_h; p.stride_w = d.stride_w; p.pad_h = d.pad_h; p.pad_w = d.pad_w; p.dil_h = d.dil_h; p.dil_w = d.dil_w;
  p.R = d.R; p.S = d.S; p.taps = d.R * d.S;
  p.halo_sw = 1; p.halo_e = 0; p.c_true = d.C;
  if (p.a_mode == kAHalo) {
    p.S = ht.s_eff; p.taps = d.R * ht.s_eff; p.pad_w = ht.pad_w_eff;
    p.halo_sw = ht.sw; p.halo_e = ht.e;
    const int dil_w = paired ? 1 : d.dil_w;
    p.row16 = (unsigned)(d.dil_h * ht.twb) * (unsigned)(BK >> 4);
    p.col16 = (unsigned)dil_w * (unsigned)(BK >> 4);
    p.fast_taps = (!paired && d.R == 3 && ht.s_eff == 3) ? 9 : ((!paired && d.R == 5 && ht.s_eff == 5) ? 25 : ((paired && d.R == 7 && ht.s_eff == 4) ? 28 : 0));
    for (int r = 0; r < d.R; ++r)
      for (int t = 0; t < ht.s_eff; ++t) {
        // tap order = order of the weight tiles in shared memory: (r, s) normally, (t', r) for pixel pairs
        const int tap = paired ? t * d.R + r : r * ht.s_eff + t;
        p.tap_shift16[tap] = (unsigned)((r * d.dil_h * ht.twb + t * dil_w) * BK) >> 4;
      }
  }
  p.c_blocks = (c_eff + BK - 1) / BK;
  p.C_pad = p.c_blocks * BK;
  p.k_iters = p.taps * p.c_blocks;
  p.splits = splits;
  p.kps = p.k_iters / splits;  // the plan only splits evenly
  p.fd_splits = make_fastdiv(splits);
  p.fd_cblocks = make_fastdiv(p.c_blocks);
  p.fd_s = make_fastdiv(d.S);
  p.split_stride = (long long)a.M * a.ldc;
  // 8-bit tile buffers: panels as wide as the largest power of two dividing BN, at most one swizzle span
  int pw = BN & -BN;
  if (pw > 128) pw = 128;
  p.pw_shift = 0;
  while ((1 << p.pw_shift) < pw) ++p.pw_shift;
  p.pmask = pw == 128 ? 7 : (pw == 64 ? 3 : (pw == 32 ? 1 : 0));
  p.panels = BN / pw;
  p.n_tiles = (d.K + BN - 1) / BN;
  p.k_pad = p.n_tiles * BN;
  if (p.a_mode == kAHalo) {
    p.tw = ht.tw; p.th = ht.th; p.twb = ht.twb; p.hb = ht.hb;
    p.q_tiles = (a.Q + ht.tw - 1) / ht.tw;
    p.p_tiles = (a.P + ht.th - 1) / ht.th;
    p.m_tiles = d.N * p.p_tiles * p.q_tiles;
  } else {
    p.m_tiles = (int)((a.M + kBM - 1) / kBM);
  }
  p.fd_ntiles = make_fastdiv(p.n_tiles);
  p.fd_perimg = make_fastdiv(p.a_mode == kAHalo ? p.p_tiles * p.q_tiles : 1);
  p.fd_qtiles = make_fastdiv(p.a_mode == kAHalo ? p.q_tiles : 1);
  p.fd_pq = make_fastdiv(p.PQ);
  p.fd_q = make_fastdiv(p.Q);
  p.tile8_bytes = (unsigned)(kBM * BN);  // a multiple of 2 KiB
  p.acc_stride = 32;
  while (p.acc_stride < BN) p.acc_stride *= 2;
  p.nacc = 512 / p.acc_stride < kMaxAcc ? 512 / p.acc_stride : kMaxAcc;
  p.tmem_cols = p.nacc * p.acc_stride;  // a power of two in [32, 512]
  // With two accumulators a third lane could wait on an accumulator barrier two phases ahead (the release it waits
  // for may belong to a tile that another lane has not issued yet); with four, the tile that last used the
  // accumulator was issued before this lane's previous tile.
  p.mma_lanes = tune_env("Q8_LANES", p.nacc >= 4 ? 3 : 2);
  if (p.mma_lanes > 2 && p.nacc < 4) p.mma_lanes = 2;
  p.b_tile_bytes = (unsigned)(BN * BK);
  p.b_sub_bytes = round_up(p.b_tile_bytes, 1024u);

  // ---- shared memory plan: [resident weights] [A stages] [weight ring] [8-bit tile buffers] [bias, scale]
  const bool use_bufs = out8 || res_mode == kResTma;
  // Launches with at most two work items per CTA cannot keep several groups busy on different tiles: there all
  // four groups share every tile, each taking a quarter of its columns (any tile width, both accumulators).
  {
    const long long items = (long long)p.m_tiles * p.n_tiles * splits;
    const long long ctas = items < sm_count() ? items : sm_count();
    p.epi_split = tune_env("Q8_SPLIT", ((items + ctas - 1) / ctas <= 2 && BN >= 64 && d.y_type != Q8_S32) ? 1 : 0);
  }
  int G = tune_env("Q8_G", (BN > 128 && !p.epi_split) ? 2 : 4);
  if (G > p.nacc && !p.epi_split) G = 2;  // a group may run at most one accumulator phase ahead of the MMA warp
  const unsigned chan_bytes = round_up((unsigned)p.k_pad * 8u, 1024u);
  const unsigned budget = (unsigned)(kSmemLimit - kStaticSmemReserve) - 1024u /* alignment slack */ - chan_bytes;
  // Weights stay resident when the whole layer's B operand is small: no per-tile weight traffic at all.
  // A tile of bn*bk bytes keeps every tap tile aligned to the swizzle pattern.
  const unsigned b_all = (unsigned)(p.n_tiles * p.c_blocks * p.taps) * p.b_tile_bytes;
  const bool resident = tune_env("Q8_BRES", (b_all <= 80u * 1024u && p.taps <= 256 && p.b_tile_bytes % (8u * BK) == 0) ? 1 : 0) != 0;
  p.b_mode = resident ? kBResident : (p.a_mode == kAHalo ? kBRing : kBStage);
  const unsigned bres_bytes = resident ? round_up(b_all, 1024u) : 0u;
  // CTA pairs for the large layers with 256-wide tiles and streamed weights.  There the shared-memory port is
  // the limit: every 128 x 256 x 128 block reads 48 KB of operands while TMA writes 32 KB of weights.  With
  // tcgen05.mma.cta_group::2 two CTAs work on two m tiles of the same n tile, each holds half of the weight
  // rows, and both the operand reads and the weight writes per SM drop by a third and a half.
  p.cta2 = 0;
  p.m_tiles_real = p.m_tiles;
  {
    // Worth it once every SM pair has two work items (28x28 3x3 128->128, batch 64: 16.0 -> 15.0 us).  Shorter
    // launches gain a microsecond alone but lose inside a network whose branches run on several streams
    // (clusters need two free SMs of one pair at the same time), so they stay single CTAs.  Tile widths whose
    // halves keep whole 16-row groups.  Layers with resident weights stay single CTAs: they are bound by the
    // issue rate of the MMA lanes, which a third lane cures better (300x300 64->64: 167 us with two lanes, 154 us
    // as pairs, 135 us with three lanes).
    const long long pair_items = (long long)((p.m_tiles + 1) / 2) * p.n_tiles;
    const bool can = p.a_mode == kAHalo && !paired && p.b_mode == kBRing && BN >= 96 && BN % 32 == 0 && out8 &&
                     res_mode != kResGlobal && splits == 1 && (BK == 128 || BK == 64) &&
                     (!p.epi_split || tune_env("Q8_CTA2SPLIT", 0)) &&
                     pair_items >= tune_env("Q8_CTA2MIN", 2 * (sm_count() / 2));
    if (can && tune_env("Q8_CTA2", 1)) {
      p.cta2 = 1;
      p.m_tiles = (p.m_tiles + 1) / 2;              // work items are pairs of m tiles
      {
        const long long items = (long long)p.m_tiles * p.n_tiles, clusters = sm_count() / 2;
        const long long per = (items + (items < clusters ? items : clusters) - 1) / (items < clusters ? items : clusters);
        p.epi_split = tune_env("Q8_SPLIT", per <= 2 ? 1 : 0);
        G = tune_env("Q8_G", (BN > 128 && !p.epi_split) ? 2 : 4);
        if (G > p.nacc && !p.epi_split) G = 2;
      }
      p.b_tile_bytes = (unsigned)((BN / 2) * BK);   // this CTA's half of the weight rows
      p.b_sub_bytes = round_up(p.b_tile_bytes, 1024u);
    }
  }
  p.b_T = 1;
  p.b_chunks = p.taps;
  unsigned min_pipe;
  if (p.a_mode == kAHalo) {
    // the taps read up to (ext_h * twb + ext_w) pixels beyond accumulator row 127
    const unsigned reach = (unsigned)(kBM + (d.R - 1) * d.dil_h * ht.twb + (ht.s_eff - 1) * (paired ? 1 : d.dil_w)) * BK;
    p.a_sub_bytes = (unsigned)(BK * ht.twb * ht.hb);
    p.a_stage_bytes = round_up(reach > p.a_sub_bytes ? reach : p.a_sub_bytes, 1024u);
    p.kb = 1;
    // (measured: a gain with four accumulators, i.e. tiles up to 128 columns; a loss with two)
    if (p.b_mode == kBRing && p.b_tile_bytes % (8u * BK) == 0 && (p.nacc >= 4 || p.cta2)) {
      // Weight ring stages of several filter taps, one TMA operation each (the copy engine spends ~600 cycles
      // per operation whatever its size): as many taps as fit in about 48 KiB while two such stages fit beside
      // two activation stages and one tile buffer per epilogue group, spread evenly over a channel block.
      const unsigned fixed = bres_bytes + (use_bufs ? (unsigned)(p.epi_split ? 2 : G) * p.tile8_bytes : 0u) + 2u * p.a_stage_bytes;
      const unsigned avail = budget > fixed ? budget - fixed : 0u;
      int T = (int)(48u * 1024u / p.b_tile_bytes);
      if (T > (int)(avail / (2u * p.b_tile_bytes))) T = (int)(avail / (2u * p.b_tile_bytes));
      T = tune_env("Q8_BT", T);
      if (T > p.taps) T = p.taps;
      if (T < 1) T = 1;
      p.b_chunks = (p.taps + T - 1) / T;
      p.b_T = (p.taps + p.b_chunks - 1) / p.b_chunks;
      p.b_chunks = (p.taps + p.b_T - 1) / p.b_T;
      p.b_sub_bytes = round_up((unsigned)p.b_T * p.b_tile_bytes, 1024u);
    }
    min_pipe = 2u * p.a_stage_bytes + (p.b_mode == kBRing ? (p.b_T > 1 ? 2u : 3u) * p.b_sub_bytes : 0u);
  } else {
    p.a_sub_bytes = (unsigned)(kBM * BK);
    const unsigned unit = p.a_sub_bytes + (p.b_mode == kBStage ? p.b_sub_bytes : 0u);
    int kb = (int)(40u * 1024u / unit);
    if (kb < 1) kb = 1;
    if (kb > p.kps) kb = p.kps;
    p.kb = tune_env("Q8_KB", kb);
    p.a_stage_bytes = (unsigned)p.kb * unit;
    min_pipe = 2u * p.a_stage_bytes;
  }
  p.nbuf = 0;
  if (use_bufs) {
    // two buffers per group when that still leaves a comfortable pipeline
    p.nbuf = (budget >= bres_bytes + 2u * G * p.tile8_bytes + 2u * min_pipe && 2 * G <= kMaxSlots) ? 2 : 1;
    p.nbuf = tune_env("Q8_NBUF", p.nbuf);
    if (p.epi_split) p.nbuf = 2;  // one buffer per tile in flight; a CTA has at most two tiles
  }
  const unsigned buf_bytes = (unsigned)(p.epi_split ? p.nbuf : G * p.nbuf) * p.tile8_bytes;
  if (budget < bres_bytes + buf_bytes + min_pipe) return kPlanNoFit;
  unsigned rest = budget - bres_bytes - buf_bytes;
  p.b_stages = 0;
  if (p.b_mode == kBRing) {
    int bst = (int)((rest - 2u * p.a_stage_bytes) / p.b_sub_bytes);
    if (bst > kMaxBStages) bst = kMaxBStages;
    p.b_stages = tune_env("Q8_BSTAGES", bst);
    rest -= (unsigned)p.b_stages * p.b_sub_bytes;
  }
  int stages = (int)(rest / p.a_stage_bytes);
  if (stages > kMaxStages) stages = kMaxStages;
  p.stages = tune_env("Q8_STAGES", stages);
  p.off_a = bres_bytes;
  p.off_bring = p.off_a + (unsigned)p.stages * p.a_stage_bytes;
  p.off_bufs = p.off_bring + (unsigned)p.b_stages * p.b_sub_bytes;
  p.off_chan = p.off_bufs + buf_bytes;
  size_t dyn = 1024u + p.off_chan + chan_bytes;
  if (dyn > (size_t)(kSmemLimit - kStaticSmemReserve)) return kPlanNoFit;
  // at least 120 KiB so that one CTA owns an SM and with it the whole TMEM
  if (dyn < 120 * 1024) dyn = 120 * 1024;

  // ---- tensor maps
  CUtensorMap tmA, tmB, tmRes, tmY;
  memset(&tmRes, 0, sizeof(tmRes));
  memset(&tmY, 0, sizeof(tmY));
  CUresult cr;
  const cuuint32_t ones[4] = {1, 1, 1, 1};
  if (p.a_mode == kAPlain) {
    cuuint64_t dims[2] = {(cuuint64_t)d.C, (cuuint64_t)a.M};
    cuuint64_t strides[1] = {(cuuint64_t)d.C};
    cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)kBM};
    cr = fn.tiled(&tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(a.x), dims, strides, box, ones,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else {
    cuuint64_t dims[4] = {(cuuint64_t)d.C, (cuuint64_t)d.W, (cuuint64_t)d.H, (cuuint64_t)d.N};
    cuuint64_t strides[3] = {(cuuint64_t)d.C, (cuuint64_t)d.W * d.C, (cuuint64_t)d.H * d.W * d.C};
    if (p.a_mode == kAHalo) {
      if (paired) { dims[0] = (cuuint64_t)c_eff; dims[1] = (cuuint64_t)(d.W / 2); strides[0] = (cuuint64_t)c_eff; }
      cuuint32_t box[4] = {(cuuint32_t)BK, (cuuint32_t)ht.twb, (cuuint32_t)ht.hb, 1};
      cr = fn.tiled(&tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(a.x), dims, strides, box, ones,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    } else {
      int lower[2] = {-d.pad_w, -d.pad_h};
      int upper[2] = {d.pad_w - (d.S - 1) * d.dil_w, d.pad_h - (d.R - 1) * d.dil_h};
      cuuint32_t estr[4] = {1, (cuuint32_t)d.stride_w, (cuuint32_t)d.stride_h, 1};
      cr = fn.im2col(&tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(a.x), dims, strides, lower, upper,
                     (cuuint32_t)BK, (cuuint32_t)kBM, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
  }
  if (cr != CUDA_SUCCESS) return fail(Q8_ERR_CUDA, "conv_umma: activation tensor map rejected (CUresult %d)", (int)cr);
  if (resident && paired) {
    // (S*C, K, R) view of the KRSC weights: a box of 2C bytes along the (s, c) axis is one pixel-pair tap
    cuuint64_t dims[3] = {(cuuint64_t)d.S * d.C, (cuuint64_t)d.K, (cuuint64_t)d.R};
    cuuint64_t strides[2] = {(cuuint64_t)d.R * d.S * d.C, (cuuint64_t)d.S * d.C};
    cuuint32_t box[3] = {(cuuint32_t)BK, (cuuint32_t)BN, (cuuint32_t)d.R};
    cr = fn.tiled(&tmB, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<int8_t*>(a.w), dims, strides, box, ones,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else if (resident) {
    // (C, K, taps) view of the KRSC weights: one box brings bn rows of every tap
    cuuint64_t dims[3] = {(cuuint64_t)d.C, (cuuint64_t)d.K, (cuuint64_t)p.taps};
    cuuint64_t strides[2] = {(cuuint64_t)p.taps * d.C, (cuuint64_t)d.C};
    cuuint32_t box[3] = {(cuuint32_t)BK, (cuuint32_t)BN, (cuuint32_t)p.taps};
    cr = fn.tiled(&tmB, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<int8_t*>(a.w), dims, strides, box, ones,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else if (p.b_mode == kBRing) {
    // (C, K, taps) view: one box brings bn rows of b_T consecutive taps, one K-major tile per tap
    cuuint64_t dims[3] = {(cuuint64_t)d.C, (cuuint64_t)d.K, (cuuint64_t)p.taps};
    cuuint64_t strides[2] = {(cuuint64_t)p.taps * d.C, (cuuint64_t)d.C};
    cuuint32_t box[3] = {(cuuint32_t)BK, (cuuint32_t)(p.cta2 ? BN / 2 : BN), (cuuint32_t)p.b_T};
    cr = fn.tiled(&tmB, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<int8_t*>(a.w), dims, strides, box, ones,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else {
    cuuint64_t dims[3] = {(cuuint64_t)d.C, (cuuint64_t)p.taps, (cuuint64_t)d.K};
    cuuint64_t strides[2] = {(cuuint64_t)d.C, (cuuint64_t)p.taps * d.C};
    cuuint32_t box[3] = {(cuuint32_t)BK, 1, (cuuint32_t)BN};
    cr = fn.tiled(&tmB, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<int8_t*>(a.w), dims, strides, box, ones,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  if (cr != CUDA_SUCCESS) return fail(Q8_ERR_CUDA, "conv_umma: weight tensor map rejected (CUresult %d)", (int)cr);

  // Residual and output tiles: [M][channels] matrices, or for halo tiles (channels, Q, P, N) tensors whose
  // TH x TW box lands as TH*TW dense rows.  The output map ends at the last channel this layer owns,
  // so the store clips ragged Cout tiles and never touches a neighbouring slice of a concatenated tensor.
  auto encode_rows = [&](CUtensorMap* tm, void* ptr, int channels, int ld, CUtensorMapL2promotion promo) -> CUresult {
    if (p.a_mode == kAHalo) {
      cuuint64_t dims[4] = {(cuuint64_t)channels, (cuuint64_t)a.Q, (cuuint64_t)a.P, (cuuint64_t)d.N};
      cuuint64_t strides[3] = {(cuuint64_t)ld, (cuuint64_t)a.Q * ld, (cuuint64_t)a.P * a.Q * ld};
      cuuint32_t box[4] = {(cuuint32_t)pw, (cuuint32_t)ht.tw, (cuuint32_t)ht.th, 1};
      return fn.tiled(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, ptr, dims, strides, box, ones, CU_TENSOR_MAP_INTERLEAVE_NONE,
                      swizzle_for_bytes(pw), promo, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    cuuint64_t dims[2] = {(cuuint64_t)channels, (cuuint64_t)a.M};
    cuuint64_t strides[1] = {(cuuint64_t)ld};
    cuuint32_t box[2] = {(cuuint32_t)pw, (cuuint32_t)kBM};
    return fn.tiled(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, ptr, dims, strides, box, ones, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    swizzle_for_bytes(pw), promo, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  };
  if (res_mode == kResTma) {
    cr = encode_rows(&tmRes, const_cast<void*>(a.residual), d.K, d.K, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
    if (cr != CUDA_SUCCESS) return fail(Q8_ERR_CUDA, "conv_umma: residual tensor map rejected (CUresult %d)", (int)cr);
  }
  if (out8) {
    cr = encode_rows(&tmY, a.y, a.c_off + d.K, a.ldc, CU_TENSOR_MAP_L2_PROMOTION_NONE);
    if (cr != CUDA_SUCCESS) return fail(Q8_ERR_CUDA, "conv_umma: output tensor map rejected (CUresult %d)", (int)cr);
  }
  p.res_tx_bytes = (unsigned)BN * (p.a_mode == kAHalo ? (unsigned)(ht.tw * ht.th) : (unsigned)kBM);

  // instruction descriptor: D = s32 (2 << 4); A format at bit 7 (0 = u8, 1 = s8); B = s8 at bit 10;
  // both operands K-major; N/8 at bit 17; M/16 at bit 24.
  p.idesc = (2u << 4) | ((d.x_type == Q8_S8 ? 1u : 0u) << 7) | (1u << 10) | ((unsigned)(BN >> 3) << 17) |
            ((unsigned)((p.cta2 ? 2 * kBM : kBM) >> 4) << 24);
  // shared-memory matrix descriptor of a K-major operand tile whose rows are BK bytes (= one swizzle
  // span): 8-row groups are 8*BK bytes apart (stride byte offset, bits 32-45), the leading byte offset
  // (bits 16-29) is unused for swizzled K-major tiles and set to 1, descriptor version 1 (bit 46),
  // swizzle mode from BK (bits 61-63).  Only the high word is kept here; the low word is
  // (start address >> 4) | (1 << 16).
  {
    const unsigned layout = BK == 128 ? 2u : (BK == 64 ? 4u : 6u);
    p.desc_hi = (unsigned)((8 * BK) >> 4) | (1u << 14) | (layout << 29);
  }
  p.bias = a.bias; p.scale = a.scale; p.scale_count = d.scale_count;
  p.res = static_cast<const unsigned char*>(a.residual);
  p.res_mode = res_mode;
  p.res_signed = d.res_type == Q8_S8;
  p.res_scale = a.residual_scale;
  p.y = a.y; p.y_type = d.y_type; p.ldc = a.ldc; p.c_off = a.c_off; p.relu = d.relu;
  p.out8 = out8 ? 1 : 0;
  p.y_vec = out8 ? 1 : (aligned16(a.y) && a.ldc % 4 == 0 && a.c_off % 4 == 0);
  p.status = status;

  const long long tiles = (long long)p.m_tiles * p.n_tiles * splits;  // work items
  int grid = (int)(tiles < sm_count() ? tiles : sm_count());
  grid = tune_env("Q8_GRID", grid);
  if (p.cta2) {  // one cluster of two CTAs per work item in flight
    const long long pairs = sm_count() / 2;
    grid = 2 * (int)(tiles < pairs ? tiles : pairs);
  }
  if (p.cta2) {
    // planned only for 8-bit outputs, residual by TMA or none.  These are the large 3x3 layers, which seldom
    // take a residual: their kernels keep that choice at compile time.
#define Q8_PAIR(GG)                                                                                                      \
  do {                                                                                                                   \
    if (d.y_type == Q8_U8) {                                                                                             \
      if (res_mode == kResTma) return launch_variant<GG, Q8_U8, kResTma, true>(tmA, tmB, tmRes, tmY, p, dyn, grid, a.stream); \
      return launch_variant<GG, Q8_U8, kResNone, true>(tmA, tmB, tmRes, tmY, p, dyn, grid, a.stream);                    \
    }                                                                                                                    \
    if (res_mode == kResTma) return launch_variant<GG, Q8_S8, kResTma, true>(tmA, tmB, tmRes, tmY, p, dyn, grid, a.stream); \
    return launch_variant<GG, Q8_S8, kResNone, true>(tmA, tmB, tmRes, tmY, p, dyn, grid, a.stream);                      \
  } while (0)
    if (G == 2) Q8_PAIR(2);
    Q8_PAIR(4);
#undef Q8_PAIR
  }
  if (G == 2) return launch_groups<2>(tmA, tmB, tmRes, tmY, p, dyn, grid, a.stream);
  return launch_groups<4>(tmA, tmB, tmRes, tmY, p, dyn, grid, a.stream);
}
}  // namespace

}  // namespace q8
