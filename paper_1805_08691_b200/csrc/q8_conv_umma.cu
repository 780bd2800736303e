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
#include "q8_umma_common.cuh"

namespace q8 {
namespace {

// The MMA lanes of the leader CTA of a pair (halo tiles, weight ring): the same schedule as mma_role, with
// tcgen05.mma.cta_group::2 over both CTAs' tiles and commits that arrive in both CTAs.
template <int kSteps>
__device__ __forceinline__ bool mma_role_pair(const UmmaParams& p, const MmaRoleArgs& r, const int who, const int vblock,
                                              const int vgrid) {
  TileIterT<true> ti;
  const int L = p.mma_lanes;
  const bool lane0 = (threadIdx.x & 31u) == 0;
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
          tcgen05_fence_after();
          if (lane0) {
            if (last_cb && row == 2) mbar_arrive(turn_next);
#pragma unroll
            for (int t = 0; t < 3; ++t) {
              const uint64_t ad = a_d + shift9[3 * row + t], bd = bring_d + (uint32_t)t * btile16;
              umma_i8_pair(d_tmem, ad, bd, idesc, (row == 0 && t == 0) ? accum : 1u);
#pragma unroll
              for (int k = 1; k < kSteps; ++k) umma_i8_pair(d_tmem, ad + 2 * k, bd + 2 * k, idesc, 1u);
            }
            umma_commit_pair(r.b_empty + bs * 8u);
          }
          accum = 1;
          bring_d += bsub16;
          if (++bs == nbst) { bs = 0; bphase ^= 1u; bring_d = bring_d0; }
        }
      }
      for (int tap0 = 0; !fast9 && tap0 < taps; tap0 += bT) {
        if (!mbar_wait(r.b_full + bs * 8u, bphase, r.abortp)) return false;
        tcgen05_fence_after();
        const int nt = min(bT, taps - tap0);
        if (lane0) {
          if (last_cb && tap0 + bT >= taps) mbar_arrive(turn_next);
          uint64_t bd = bring_d;
          for (int t = 0; t < nt; ++t, bd += btile16) {
            const uint64_t ad = a_d + r.tap_shift16[tap0 + t];
            umma_i8_pair(d_tmem, ad, bd, idesc, accum);
#pragma unroll
            for (int k = 1; k < kSteps; ++k) umma_i8_pair(d_tmem, ad + 2 * k, bd + 2 * k, idesc, 1u);
            accum = 1;
          }
          umma_commit_pair(r.b_empty + bs * 8u);
        }
        accum = 1;
        bring_d += bsub16;
        if (++bs == nbst) { bs = 0; bphase ^= 1u; bring_d = bring_d0; }
      }
      if (lane0) umma_commit_pair(r.a_empty + stage * 8u);
      a_d += stage16;
      if (++stage == nstages) { stage = 0; phase ^= 1u; a_d = a_d0; }
    }
    ++my_k;
    if (lane0) umma_commit_pair(r.acc_full + ab * 8u);
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
  // the warp index through a broadcast, so that the compiler treats it, and the role it selects, as warp uniform
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  const bool lane0 = lane == 0;
  // CTA pairs: both CTAs walk the same sequence of work items (pairs of m tiles); rank 1 takes the second tile
  int cta_rank = 0;
  if constexpr (kCta2) cta_rank = __shfl_sync(0xffffffffu, (int)cluster_ctarank(), 0);
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
  // start-up barriers (bar.arrive) and goes straight to its loads, so that the first bytes are on
  // their way while the others allocate TMEM.  Single CTAs keep the epilogue warps off the critical path: the
  // control warps meet on barrier 1 among themselves and start; the epilogue warps first touch every line of the
  // kernel parameters (the control warps' first reads of them would otherwise miss the constant cache one after
  // the other), fetch bias and scale, and join on barrier 3, which the control warps only signal.
  const int nthreads = kCtrlThreads + G * kGroupThreads;
  if (!kCta2 && warp >= kCtrlWarps) {
    const unsigned int* words = reinterpret_cast<const unsigned int*>(&p);
    unsigned int touched = 0;
    for (int i = ((int)threadIdx.x - kCtrlThreads) * 16; i < (int)(sizeof(UmmaParams) / 4); i += G * kGroupThreads * 16) touched ^= words[i];
    asm volatile("" ::"r"(touched));
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (int i = (int)threadIdx.x - kCtrlThreads; i < p.k_pad; i += G * kGroupThreads) {
      s_bias[i] = (p.bias && i < p.K) ? p.bias[i] : 0;
      s_scale[i] = p.scale ? (p.scale_count == 1 ? p.scale[0] : (i < p.K ? p.scale[i] : 0.f)) : 0.f;
    }
    asm volatile("bar.sync 3, %0;" ::"r"(nthreads) : "memory");
    tcgen05_fence_after();
  } else if (warp == 0) {
    // one barrier per lane: a lone lane would spend ~50 cycles on each
    if (lane < p.stages) { mbar_init(smem_u32(&a_full[lane]), 1); mbar_init(smem_u32(&a_empty[lane]), 1); }
    else if (lane >= 8 && lane - 8 < p.b_stages) { mbar_init(smem_u32(&b_full[lane - 8]), 1); mbar_init(smem_u32(&b_empty[lane - 8]), 1); }
    else if (lane == 16) { mbar_init(smem_u32(&bres_full), 1); abort_flag = 0; }
    else if (lane == 17) prefetch_tensormap(&tmA);
    else if (lane == 18) prefetch_tensormap(&tmB);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncwarp();
    asm volatile("griddepcontrol.wait;" ::: "memory");  // everything the previous kernel wrote is visible from here
    if constexpr (kCta2) {
      cluster_sync_all();  // the peer's barriers exist before anything signals them
      asm volatile("bar.arrive 1, %0;" ::"r"(nthreads) : "memory");
    } else {
      asm volatile("bar.arrive 1, %0;" ::"r"(kCtrlThreads) : "memory");
      asm volatile("bar.arrive 3, %0;" ::"r"(nthreads) : "memory");
    }
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
    if constexpr (kCta2) {
      // bias and scale of every channel, once per CTA (zero beyond Cout; one scale replicated if per tensor)
      for (int i = threadIdx.x - 32; i < p.k_pad; i += nthreads - 32) {
        s_bias[i] = (p.bias && i < p.K) ? p.bias[i] : 0;
        s_scale[i] = p.scale ? (p.scale_count == 1 ? p.scale[0] : (i < p.K ? p.scale[i] : 0.f)) : 0.f;
      }
      tcgen05_fence_before();
      __syncwarp();
      cluster_sync_all();
      asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory");
    } else {
      tcgen05_fence_before();
      asm volatile("bar.arrive 3, %0;" ::"r"(nthreads) : "memory");      // the epilogue warps wait for this set-up
      asm volatile("bar.sync 1, %0;" ::"r"(kCtrlThreads) : "memory");    // the control warps only for each other
    }
    tcgen05_fence_after();
  }
  const uint32_t tmem_base = warp == 0 ? 0u : tmem_holder;  // warp 0 never touches TMEM
  volatile int* abortp = &abort_flag;

  if (warp == 0) {
    // ------------------------------------------------------------------ A / B producer (whole warp; lane 0 issues)
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
      if (!lane0) {
        // only lane 0 issues
      } else if (p.a_mode == kAHalo && p.halo_sw == 2) {
        mbar_arrive_expect_tx(bar, (uint32_t)(p.n_tiles * p.c_blocks * p.taps) * p.b_tile_bytes);
        // pixel-pair taps: tap t' of a filter row covers s = 2t' - e and 2t' - e + 1, whose weights are 2C
        // contiguous bytes of the (s, c) axis; a start left of s = 0 is zero filled.  One load per t' brings
        // all R filter rows: tile order (t', r).
        for (int nt = 0; nt < p.n_tiles; ++nt)
          for (int t = 0; t < p.S; ++t, dst += (uint32_t)p.R * p.b_tile_bytes) tma_load_3d(dst, &tmB, bar, (2 * t - p.halo_e) * p.c_true, nt * p.bn, 0);
      } else {
        mbar_arrive_expect_tx(bar, (uint32_t)(p.n_tiles * p.c_blocks * p.taps) * p.b_tile_bytes);
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
          if (!lane0) {
          } else if constexpr (kCta2) {
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
              if (!lane0) {
              } else if constexpr (kCta2) {
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
          if (lane0) mbar_arrive_expect_tx(bar, (uint32_t)nsub * sub_tx);
          uint32_t dst = a_dst, bdst = a_dst + b_in_stage;
          for (int j = 0; j < nsub; ++j) {
            if (!lane0) {
            } else if (p.a_mode == kAIm2col) tma_load_im2col_4d(dst, &tmA, bar, c, w0, h0, img, (unsigned short)off_w, (unsigned short)off_h);
            else tma_load_2d(dst, &tmA, bar, c, m0);
            if (lane0 && p.b_mode == kBStage) tma_load_3d(bdst, &tmB, bar, c, tap, n0);
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
    if (!ok && lane0) {
      abort_flag = 1;
      atomicOr(p.status, kTimeoutProducer);
    }
  } else if (warp == 1 || warp == 4 || (warp == 5 && p.mma_lanes == 3)) {
    // ------------------------------------------------------------------ MMA issuers (warps 1, 4 and 5; lane 0 issues)
    const int who = warp == 1 ? 0 : warp - 3;
    MmaRoleArgs ra;
    ra.base = base; ra.tmem_base = tmem_base; ra.total_tiles = total_tiles; ra.abortp = abortp;
    ra.first_tile = (int)blockIdx.x; ra.tile_step = (int)gridDim.x;
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
    if (!ok && lane0) {
      abort_flag = 1;
      atomicOr(p.status, kTimeoutMma);
    }
  } else if (warp == 2) {
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
        if (!lane0) {
        } else if (p.res_mode == kResTma && ti.valid) {
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
      if (!ok && lane0) {
        abort_flag = 1;
        atomicOr(p.status, kTimeoutResidual);
      }
    }
  } else if (warp == 3) {
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
        if (!lane0) {
        } else if (p.out8) {
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
      if (p.out8 && lane0) {
        bulk_wait_read<0>();  // the CTA's shared memory must outlive the reads of its last stores
        if (prev_slot >= 0) mbar_arrive(bempty0 + (uint32_t)prev_slot * 8u);
      }
      if (!ok && lane0) {
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
    epi_row_setup(p, t);
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
template <int G, int kOut, int kRes, bool kCta2>
int launch_variant(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmRes, const CUtensorMap& tmY,
                   const UmmaParams& p, size_t dyn, int grid, cudaStream_t stream) {
  auto kernel = conv_umma_kernel<G, kOut, kRes, kCta2>;
  static std::atomic<bool> configured[kMaxDevices];  // per instantiation and device (the attribute is per device)
  const int dev = current_device();
  if (dev < 0 || !configured[dev].load(std::memory_order_acquire)) {
    int rc = check_cuda(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit - kStaticSmemReserve),
                        "conv_umma: set shared memory size");
    if (rc != Q8_OK) return rc;
    // every tensor-core kernel of the library asks for the largest shared-memory carve-out, so that consecutive
    // launches of different kernels or shapes never make the SMs switch their L1 / shared-memory split
    rc = check_cuda(cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared),
                    "conv_umma: set shared memory carve-out");
    if (rc != Q8_OK) return rc;
    if (dev >= 0) configured[dev].store(true, std::memory_order_release);
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
  cfg.numAttrs = tune_env("Q8_PDL", 1, 0, 1) ? 1 : 0;
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
  const DriverFns& fn = driver_fns();
  if (!fn.tiled || !fn.im2col) return fail(Q8_ERR_CUDA, "conv_umma: cuTensorMapEncode* entry points not available");
  unsigned int* status = status_word_device_ptr();
  if (!status) return fail(Q8_ERR_CUDA, "conv_umma: status word not available");

  const bool out8 = d.y_type == Q8_U8 || d.y_type == Q8_S8;
  int res_mode = kResNone;
  if (a.residual) res_mode = (d.K % 16 == 0 && aligned16(a.residual)) ? kResTma : kResGlobal;
  UmmaParams p;
  memset(&p, 0, sizeof(p));
  HaloTile ht = {0, 0, 0, 0, 0.0, 1, d.S, d.pad_w, 0};
  p.a_mode = is_plain(d) ? kAPlain : ((allow_halo && tune_env("Q8_HALO", 1, 0, 1) && choose_halo_tile(d, a.P, a.Q, &ht)) ? kAHalo : kAIm2col);
  const bool paired = p.a_mode == kAHalo && ht.sw == 2;  // input read as pixel pairs with 2C channels
  const int c_eff = paired ? 2 * d.C : d.C;
  const int BK = pick_bk(c_eff) < bk_cap ? pick_bk(c_eff) : bk_cap;
  int BN = pick_bn(d.K, d.R * d.S * d.C);
  {
    // Few output tiles (small images with many channels): 128-wide tiles run the tensor pipe at the same rate
    // per column as 256-wide ones, and twice as many CTAs get work.
    const long long m_tiles = p.a_mode == kAHalo ? (long long)d.N * ((a.P + ht.th - 1) / ht.th) * ((a.Q + ht.tw - 1) / ht.tw)
                                                 : (a.M + kBM - 1) / kBM;
    if (splits == 1 && BN == 256 && d.K % 256 == 0 && m_tiles * (d.K / 256) * 2 <= sm_count()) BN = 128;
  }
  {
    const int want = tune_env("Q8_BN", BN, 16, 256);
    if (want % 16 == 0) BN = want;
  }
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
  p.mma_lanes = tune_env("Q8_LANES", p.nacc >= 4 ? 3 : 2, 2, 3);
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
    const int may = (BN >= 64 && d.y_type != Q8_S32) ? 1 : 0;
    p.epi_split = tune_env("Q8_SPLIT", ((items + ctas - 1) / ctas <= 2 && may) ? 1 : 0, 0, may);
  }
  int G = tune_env("Q8_G", (BN > 128 && !p.epi_split) ? 2 : 4, 2, 4);
  if (G == 3) G = 4;
  if (G > p.nacc && !p.epi_split) G = 2;  // a group may run at most one accumulator phase ahead of the MMA warp
  const unsigned chan_bytes = round_up((unsigned)p.k_pad * 8u, 1024u);
  const unsigned budget = (unsigned)(kSmemLimit - kStaticSmemReserve) - 1024u /* alignment slack */ - chan_bytes;
  // Weights stay resident when the whole layer's B operand is small: no per-tile weight traffic at all.
  // A tile of bn*bk bytes keeps every tap tile aligned to the swizzle pattern.
  const unsigned b_all = (unsigned)(p.n_tiles * p.c_blocks * p.taps) * p.b_tile_bytes;
  const int can_reside = (b_all <= 80u * 1024u && p.taps <= 256 && p.b_tile_bytes % (8u * BK) == 0) ? 1 : 0;
  const bool resident = tune_env("Q8_BRES", can_reside, 0, can_reside) != 0;
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
                     (!p.epi_split || tune_env("Q8_CTA2SPLIT", 0, 0, 1)) &&
                     pair_items >= tune_env("Q8_CTA2MIN", 2 * (sm_count() / 2), 1, 1 << 30);
    if (can && tune_env("Q8_CTA2", 1, 0, 1)) {
      p.cta2 = 1;
      p.m_tiles = (p.m_tiles + 1) / 2;              // work items are pairs of m tiles
      {
        const long long items = (long long)p.m_tiles * p.n_tiles, clusters = sm_count() / 2;
        const long long per = (items + (items < clusters ? items : clusters) - 1) / (items < clusters ? items : clusters);
        p.epi_split = tune_env("Q8_SPLIT", per <= 2 ? 1 : 0, 0, 1);
        G = tune_env("Q8_G", (BN > 128 && !p.epi_split) ? 2 : 4, 2, 4);
        if (G == 3) G = 4;
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
      T = tune_env("Q8_BT", T, 1, T > 1 ? T : 1);
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
    p.kb = tune_env("Q8_KB", kb, 1, kb);
    p.a_stage_bytes = (unsigned)p.kb * unit;
    min_pipe = 2u * p.a_stage_bytes;
  }
  p.nbuf = 0;
  if (use_bufs) {
    // two buffers per group when that still leaves a comfortable pipeline
    p.nbuf = (budget >= bres_bytes + 2u * G * p.tile8_bytes + 2u * min_pipe && 2 * G <= kMaxSlots) ? 2 : 1;
    p.nbuf = tune_env("Q8_NBUF", p.nbuf, 1, p.nbuf);
    if (p.epi_split) p.nbuf = 2;  // one buffer per tile in flight; a CTA has at most two tiles
  }
  const unsigned buf_bytes = (unsigned)(p.epi_split ? p.nbuf : G * p.nbuf) * p.tile8_bytes;
  if (budget < bres_bytes + buf_bytes + min_pipe) return kPlanNoFit;
  unsigned rest = budget - bres_bytes - buf_bytes;
  p.b_stages = 0;
  if (p.b_mode == kBRing) {
    int bst = (int)((rest - 2u * p.a_stage_bytes) / p.b_sub_bytes);
    if (bst > kMaxBStages) bst = kMaxBStages;
    p.b_stages = tune_env("Q8_BSTAGES", bst, 2, bst > 2 ? bst : 2);
    rest -= (unsigned)p.b_stages * p.b_sub_bytes;
  }
  int stages = (int)(rest / p.a_stage_bytes);
  if (stages > kMaxStages) stages = kMaxStages;
  p.stages = tune_env("Q8_STAGES", stages, 2, stages > 2 ? stages : 2);
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
  grid = tune_env("Q8_GRID", grid, 1, grid);
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
