// Two quantized convolutions in one launch: a stride-1 filter (layer 1, e.g. the 3x3 of a residual bottleneck)
// followed by a 1x1 convolution over its output (layer 2, e.g. the expanding 1x1 with the fused residual sum).
// The 8-bit output tile of layer 1 never leaves the SM: the epilogue writes it to shared memory in the K-major
// swizzled layout a tcgen05 A operand has, and layer 2 multiplies it with weights resident in shared memory.
// (Sec. "Model Optimization" of the paper fuses the element-wise ops into the convolution before them; this goes
// one step further and also keeps the tensor between two convolutions on chip.)
//
//   layer 1:  D1[128 rows of one halo tile, Cout1]   = patch (TMA, shifted descriptors per tap) x W1^T
//             E1: + bias1, * scale1, ReLU, round, clamp -> T[slot] (u8/s8, [128][Cout1], swizzled)
//   layer 2:  D2[128, 128-column chunk j of Cout2]   = T[slot] x W2[chunk j]^T          for every chunk j
//             E2: + bias2, * scale2, + residual * s_res, ReLU, round, clamp -> tile buffer -> TMA store
//
// Warps (whole warps walk the schedules, lane 0 issues):
//   0      TMA producer of layer 1 (input patches, weight ring), and of all resident weights before the kernel
//          orders itself behind its predecessor in the stream;
//   1      MMA issue of layer 1 (owns the TMEM allocation);
//   2      MMA issue of layer 2;
//   3      tile buffers of layer 2: residual tiles in (TMA), finished output tiles out (TMA store);
//   4-7    E1, one group of four warps;
//   8-19   E2, three groups of four warps; group g owns accumulator g of layer 2 and every third chunk.
// TMEM (512 columns): three layer-2 accumulators of 128 columns, the rest holds one to two layer-1 accumulators.
// Every hand-off is an mbarrier with a bounded wait (status word + drain on expiry), as in q8_conv_umma.cu.
#include "q8_umma_common.cuh"

namespace q8 {
namespace {

constexpr int kFCtrlWarps = 4;
constexpr int kFE2Groups = 3;
constexpr int kFThreads = (kFCtrlWarps + 4 + 4 * kFE2Groups) * 32;  // 640
constexpr int kFAcc2Cols = 128;                                      // columns of one layer-2 accumulator
constexpr int kFMaxTb = 4;                                           // slots of the intermediate tile ring
constexpr int kFMaxSlots = 6;                                        // layer-2 tile buffers

struct FusedParams {
  UmmaParams l1;  // layer 1: halo tiles, one tile of columns (bn = Cout1), one MMA warp; its 8-bit tile fields
                  // (pw_shift, pmask) describe the intermediate tile T
  UmmaParams l2;  // layer 2: bn = chunk width, n_tiles = chunks, bk = ksteps * 32 = Cout1; 8-bit tile fields
                  // describe the output tile buffers; y / ldc / c_off / residual as in the single-layer kernel
  int ntb;                       // slots of the T ring
  unsigned int off_w2, off_tb;   // resident W2 tiles, T ring (from the 1 KiB aligned base)
  unsigned int tb_bytes;         // 128 * Cout1
  unsigned int off_chan2;        // bias2 / scale2 staging
  int nslots;                    // layer-2 tile buffers (3 or 6)
  int acc1_col;                  // first TMEM column of the layer-1 accumulators
};

// One (m tile, chunk) item of layer 2 in this CTA's sequence, with the tile's image coordinates.
struct ItemIter {
  TileIterT<false> ti;
  int j, left;
  __device__ __forceinline__ void init(const UmmaParams& l1, int t0, int j0, int count) {
    ti.init(l1, t0, 1);
    j = j0;
    left = count;
  }
  __device__ __forceinline__ bool done() const { return left <= 0; }
  __device__ __forceinline__ void next(const UmmaParams& l1, int chunks) {
    --left;
    if (++j == chunks) { j = 0; ti.next(l1); }
  }
};

template <int kOut1, int kOut2>
__global__ void __launch_bounds__(kFThreads, 1)
    conv_fused_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB1,
                      const __grid_constant__ CUtensorMap tmB2, const __grid_constant__ CUtensorMap tmRes,
                      const __grid_constant__ CUtensorMap tmY, const __grid_constant__ FusedParams p) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long a_full[kMaxStages], a_empty[kMaxStages];
  __shared__ __align__(8) unsigned long long b_full[kMaxBStages], b_empty[kMaxBStages];
  __shared__ __align__(8) unsigned long long acc1_full[2], acc1_empty[2];
  __shared__ __align__(8) unsigned long long acc2_full[kFE2Groups], acc2_empty[kFE2Groups];
  __shared__ __align__(8) unsigned long long tb_full[kFMaxTb], tb_empty[kFMaxTb];
  __shared__ __align__(8) unsigned long long buf_full[kFMaxSlots], store_ready[kFMaxSlots];
  __shared__ __align__(8) unsigned long long w1_full, w2_full, mma_turn;
  __shared__ uint32_t tap_shift16[kMaxTaps];
  __shared__ uint32_t tmem_holder;
  __shared__ int abort_flag;

  // dynamic smem: [W1 resident] [W2 resident] [A stages] [W1 ring] [T ring] [layer-2 tile buffers] [bias1, scale1] [bias2, scale2]
  const uint32_t raw_base = smem_u32(smem_raw);
  const uint32_t base = (raw_base + 1023u) & ~1023u;
  unsigned char* const base_ptr = smem_raw + (base - raw_base);
  int* const s_bias1 = reinterpret_cast<int*>(base_ptr + p.l1.off_chan);
  float* const s_scale1 = reinterpret_cast<float*>(base_ptr + p.l1.off_chan) + p.l1.k_pad;
  int* const s_bias2 = reinterpret_cast<int*>(base_ptr + p.off_chan2);
  float* const s_scale2 = reinterpret_cast<float*>(base_ptr + p.off_chan2) + p.l2.k_pad;
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  const bool lane0 = lane == 0;
  // Work split.  The unit is one item = (m tile, chunk of layer-2 output channels); items are numbered tile by tile
  // and every CTA takes a contiguous range of them, so that the CTAs' loads differ by at most one item (whole tiles
  // per CTA would leave most SMs idle for up to a tile's time at the end).  A CTA whose range starts or ends inside a
  // tile computes layer 1 of that tile as well: the tensor pipe has time to spare, the epilogue of layer 2 has not.
  const int chunks = p.l2.n_tiles;
  int t0, j0, j1, my_items, my_tiles;
  {
    const int total = p.l1.m_tiles * chunks, per = total / (int)gridDim.x, rem = total - per * (int)gridDim.x;
    const int c = (int)blockIdx.x;
    my_items = per + (c < rem ? 1 : 0);
    const int begin = c * per + (c < rem ? c : rem), last = begin + my_items - 1;
    t0 = begin / chunks;
    j0 = begin - t0 * chunks;
    const int t1 = last / chunks;
    j1 = last - t1 * chunks + 1;
    my_tiles = my_items > 0 ? t1 - t0 + 1 : 0;
  }

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // Prologue.  Weights, biases and multipliers are constants of the layer pair: they are fetched BEFORE the kernel
  // orders itself behind the previous kernel of the stream (griddepcontrol.wait), so that under a programmatic
  // dependent launch they arrive while that kernel drains.  Only activations (input patches, residual tiles)
  // wait for it.  The control warps meet on barrier 1 among themselves and start; the epilogue warps touch every line
  // of the kernel parameters (warming the constant cache for the control warps), stage bias and multipliers, and
  // join on barrier 3, which the control warps only signal.
  if (warp >= kFCtrlWarps) {
    const unsigned int* words = reinterpret_cast<const unsigned int*>(&p);
    unsigned int touched = 0;
    const int et = (int)threadIdx.x - kFCtrlWarps * 32, en = kFThreads - kFCtrlWarps * 32;
    for (int i = et * 16; i < (int)(sizeof(FusedParams) / 4); i += en * 16) touched ^= words[i];
    asm volatile("" ::"r"(touched));
    // bias and multiplier of every channel of both layers (zero beyond Cout; one multiplier replicated if per tensor)
    for (int i = et; i < p.l1.k_pad; i += en) {
      s_bias1[i] = (p.l1.bias && i < p.l1.K) ? p.l1.bias[i] : 0;
      s_scale1[i] = p.l1.scale_count == 1 ? p.l1.scale[0] : (i < p.l1.K ? p.l1.scale[i] : 0.f);
    }
    for (int i = et; i < p.l2.k_pad; i += en) {
      s_bias2[i] = (p.l2.bias && i < p.l2.K) ? p.l2.bias[i] : 0;
      s_scale2[i] = p.l2.scale_count == 1 ? p.l2.scale[0] : (i < p.l2.K ? p.l2.scale[i] : 0.f);
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("bar.sync 3, %0;" ::"r"(kFThreads) : "memory");
    tcgen05_fence_after();
  } else if (warp == 0) {
    if (lane < p.l1.stages) { mbar_init(smem_u32(&a_full[lane]), 1); mbar_init(smem_u32(&a_empty[lane]), 1); }
    else if (lane >= 8 && lane - 8 < p.l1.b_stages) { mbar_init(smem_u32(&b_full[lane - 8]), 1); mbar_init(smem_u32(&b_empty[lane - 8]), 1); }
    else if (lane == 16) { mbar_init(smem_u32(&w1_full), 1); mbar_init(smem_u32(&w2_full), 1); abort_flag = 0; }
    else if (lane == 17) prefetch_tensormap(&tmA);
    else if (lane == 18) prefetch_tensormap(&tmB1);
    else if (lane == 19) prefetch_tensormap(&tmB2);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncwarp();
    if (lane0) {
      // layer-2 weights: one K-major tile of bn2 x Cout1 bytes per chunk
      const uint32_t bar2 = smem_u32(&w2_full);
      mbar_arrive_expect_tx(bar2, (uint32_t)chunks * p.l2.b_tile_bytes);
      uint32_t dst = base + p.off_w2;
      for (int j = 0; j < chunks; ++j, dst += p.l2.b_tile_bytes) tma_load_2d(dst, &tmB2, bar2, 0, j * p.l2.bn);
      if (p.l1.b_mode == kBResident) {
        // layer-1 weights, [tap][bn1 rows][bk bytes] per channel block
        const uint32_t bar1 = smem_u32(&w1_full);
        mbar_arrive_expect_tx(bar1, (uint32_t)(p.l1.c_blocks * p.l1.taps) * p.l1.b_tile_bytes);
        uint32_t d1 = base;
        for (int c = 0; c < p.l1.C_pad; c += p.l1.bk, d1 += (uint32_t)p.l1.taps * p.l1.b_tile_bytes) tma_load_3d(d1, &tmB1, bar1, c, 0, 0);
      }
    }
    __syncwarp();
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("bar.arrive 1, %0;" ::"r"(kFCtrlWarps * 32) : "memory");
    asm volatile("bar.arrive 3, %0;" ::"r"(kFThreads) : "memory");
  } else {
    if (warp == 1) {
      if (lane < p.l1.nacc) { mbar_init(smem_u32(&acc1_full[lane]), 1); mbar_init(smem_u32(&acc1_empty[lane]), 4); }
      else if (lane == 8) mbar_init(smem_u32(&mma_turn), 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      __syncwarp();
      tmem_alloc(smem_u32(&tmem_holder), 512u);
      tmem_relinquish();
    } else if (warp == 2) {
      if (lane < kFE2Groups) { mbar_init(smem_u32(&acc2_full[lane]), 1); mbar_init(smem_u32(&acc2_empty[lane]), 4); }
      else if (lane >= 8 && lane - 8 < p.ntb) { mbar_init(smem_u32(&tb_full[lane - 8]), kGroupThreads); mbar_init(smem_u32(&tb_empty[lane - 8]), 1); }
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    } else if (warp == 3) {
      if (lane < p.nslots) { mbar_init(smem_u32(&buf_full[lane]), 1); mbar_init(smem_u32(&store_ready[lane]), kGroupThreads); }
      else if (lane == 16 && p.l2.res_mode == kResTma) prefetch_tensormap(&tmRes);
      else if (lane == 17) prefetch_tensormap(&tmY);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x >= 32 && (int)threadIdx.x - 32 < p.l1.taps) tap_shift16[threadIdx.x - 32] = p.l1.tap_shift16[threadIdx.x - 32];
    asm volatile("griddepcontrol.wait;" ::: "memory");
    tcgen05_fence_before();
    asm volatile("bar.arrive 3, %0;" ::"r"(kFThreads) : "memory");
    asm volatile("bar.sync 1, %0;" ::"r"(kFCtrlWarps * 32) : "memory");
    tcgen05_fence_after();
  }
  const uint32_t tmem_base = warp == 0 ? 0u : tmem_holder;
  volatile int* abortp = &abort_flag;

  if (warp == 0) {
    // ------------------------------------------------------------------ layer-1 producer: patches and the weight ring
    TileIterT<false> ti;
    ti.init(p.l1, t0, 1);
    const UmmaParams& q = p.l1;
    const uint32_t nstages = (uint32_t)q.stages, nbst = (uint32_t)q.b_stages;
    const uint32_t afull0 = smem_u32(&a_full[0]), aempty0 = smem_u32(&a_empty[0]);
    const uint32_t bfull0 = smem_u32(&b_full[0]), bempty0 = smem_u32(&b_empty[0]);
    const uint32_t a0 = base + q.off_a, bring0 = base + q.off_bring;
    uint32_t stage = 0, phase = 0, a_dst = a0;
    uint32_t bs = 0, bphase = 0, b_dst = bring0;
    const uint32_t b_tx = (uint32_t)q.b_T * q.b_tile_bytes;
    bool ok = true;
    for (int k = 0; k < my_tiles && ok; ++k, ti.next(q)) {
      const int q0 = ti.qt * q.tw - q.pad_w, p0 = ti.pt * q.th - q.pad_h;
      for (int c = 0; c < q.C_pad && ok; c += q.bk) {
        if (!mbar_wait(aempty0 + stage * 8u, phase ^ 1u, abortp)) { ok = false; break; }
        if (lane0) {
          const uint32_t bar = afull0 + stage * 8u;
          mbar_arrive_expect_tx(bar, q.a_sub_bytes);
          tma_load_4d(a_dst, &tmA, bar, c, q0, p0, ti.img);
        }
        a_dst += q.a_stage_bytes;
        if (++stage == nstages) { stage = 0; phase ^= 1u; a_dst = a0; }
        if (q.b_mode == kBRing) {
          for (int tap = 0; tap < q.taps; tap += q.b_T) {
            if (!mbar_wait(bempty0 + bs * 8u, bphase ^ 1u, abortp)) { ok = false; break; }
            if (lane0) {
              const uint32_t bbar = bfull0 + bs * 8u;
              mbar_arrive_expect_tx(bbar, b_tx);
              tma_load_3d(b_dst, &tmB1, bbar, c, 0, tap);
            }
            b_dst += q.b_sub_bytes;
            if (++bs == nbst) { bs = 0; bphase ^= 1u; b_dst = bring0; }
          }
        }
      }
    }
    if (!ok && lane0) { abort_flag = 1; atomicOr(p.l1.status, kTimeoutProducer); }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ layer-1 MMA issue
    MmaRoleArgs ra;
    ra.base = base; ra.tmem_base = tmem_base + (uint32_t)p.acc1_col; ra.total_tiles = t0 + my_tiles; ra.abortp = abortp;
    ra.first_tile = t0; ra.tile_step = 1;
    ra.a_full = smem_u32(&a_full[0]); ra.a_empty = smem_u32(&a_empty[0]);
    ra.b_full = smem_u32(&b_full[0]); ra.b_empty = smem_u32(&b_empty[0]);
    ra.acc_full = smem_u32(&acc1_full[0]); ra.acc_empty = smem_u32(&acc1_empty[0]);
    ra.bres_full = smem_u32(&w1_full); ra.tap_shift16 = tap_shift16; ra.turn = smem_u32(&mma_turn);
    bool ok;
    if (p.l1.ksteps == 4) ok = mma_role<4>(p.l1, ra, 0);
    else if (p.l1.ksteps == 2) ok = mma_role<2>(p.l1, ra, 0);
    else ok = mma_role<1>(p.l1, ra, 0);
    if (!ok && lane0) { abort_flag = 1; atomicOr(p.l1.status, kTimeoutMma); }
  } else if (warp == 2) {
    // ------------------------------------------------------------------ layer-2 MMA issue: T[slot] x W2[chunk]^T
    const UmmaParams& q = p.l2;
    const uint64_t hi = ((uint64_t)q.desc_hi << 32) | (1ull << 16);
    const uint64_t t_d0 = hi | (((base + p.off_tb) >> 4) & 0x3fffu), w_d0 = hi | (((base + p.off_w2) >> 4) & 0x3fffu);
    const uint32_t tb16 = p.tb_bytes >> 4, wt16 = q.b_tile_bytes >> 4;
    const uint32_t tbf0 = smem_u32(&tb_full[0]), tbe0 = smem_u32(&tb_empty[0]);
    const uint32_t a2f0 = smem_u32(&acc2_full[0]), a2e0 = smem_u32(&acc2_empty[0]);
    const uint32_t ntb = (uint32_t)p.ntb;
    uint32_t slot = 0, tpar = 0, g = 0, gpar = 1;  // T slot and its parity; accumulator (= group) and the parity of its empty barrier
    bool ok = mbar_wait(smem_u32(&w2_full), 0u, abortp);
    for (int k = 0; k < my_tiles && ok; ++k) {
      if (!mbar_wait(tbf0 + slot * 8u, tpar, abortp)) { ok = false; break; }
      const uint64_t t_d = t_d0 + slot * tb16;
      const int jb = k == 0 ? j0 : 0, je = k == my_tiles - 1 ? j1 : chunks;  // this CTA's chunks of the tile
      uint64_t w_d = w_d0 + (uint32_t)jb * wt16;
      for (int j = jb; j < je; ++j, w_d += wt16) {
        if (!mbar_wait(a2e0 + g * 8u, gpar, abortp)) { ok = false; break; }
        tcgen05_fence_after();
        if (lane0) {
          const uint32_t d_tmem = tmem_base + g * (uint32_t)kFAcc2Cols;
          if (q.ksteps == 4) umma_i8_block<4>(d_tmem, t_d, w_d, q.idesc, 0u);
          else if (q.ksteps == 2) umma_i8_block<2>(d_tmem, t_d, w_d, q.idesc, 0u);
          else umma_i8_block<1>(d_tmem, t_d, w_d, q.idesc, 0u);
          umma_commit(a2f0 + g * 8u);
        }
        if (++g == (uint32_t)kFE2Groups) { g = 0; gpar ^= 1u; }
      }
      if (lane0) umma_commit(tbe0 + slot * 8u);  // T[slot] may be overwritten once these MMAs have read it
      if (++slot == ntb) { slot = 0; tpar ^= 1u; }
    }
    if (!ok && lane0) { abort_flag = 1; atomicOr(p.l1.status, kTimeoutMma); }
  } else if (warp == 3) {
    // ------------------------------------------------------------------ layer-2 tile buffers: residual in, output out
    // Item i of the CTA's sequence uses buffer i % nslots.  A buffer goes: residual tile arrives (buf_full) -> an E2
    // group turns it into the output tile (store_ready) -> TMA store -> once the store has read it, the residual
    // of item i + nslots is loaded into it.
    const UmmaParams& q = p.l2;
    const uint32_t bfull0 = smem_u32(&buf_full[0]), ready0 = smem_u32(&store_ready[0]);
    const uint32_t nslots = (uint32_t)p.nslots;
    const int pw = 1 << q.pw_shift;
    const uint32_t panel_bytes = (uint32_t)kBM << q.pw_shift;
    const UmmaParams& h = p.l1;  // tile geometry
    auto load_residual = [&](const ItemIter& it, uint32_t s) {
      const uint32_t bar = bfull0 + s * 8u;
      if (q.res_mode == kResTma) {
        uint32_t dst = base + q.off_bufs + s * q.tile8_bytes;
        mbar_arrive_expect_tx(bar, q.res_tx_bytes);
        for (int pn = 0, c = it.j * q.bn; pn < q.panels; ++pn, c += pw, dst += panel_bytes)
          tma_load_4d(dst, &tmRes, bar, c, it.ti.qt * h.tw, it.ti.pt * h.th, it.ti.img);
      } else {
        mbar_arrive(bar);
      }
    };
    ItemIter ld, st;
    ld.init(h, t0, j0, my_items);
    st.init(h, t0, j0, my_items);
    if (lane0)
      for (uint32_t s = 0; s < nslots && !ld.done(); ++s, ld.next(h, chunks)) load_residual(ld, s);
    else
      for (uint32_t s = 0; s < nslots && !ld.done(); ++s) ld.next(h, chunks);
    uint32_t slot = 0, spar = 0;
    int prev_slot = -1;
    bool ok = true;
    for (; !st.done(); st.next(h, chunks)) {
      if (!mbar_wait(ready0 + slot * 8u, spar, abortp)) { ok = false; break; }
      if (lane0) {
        uint32_t src = base + q.off_bufs + slot * q.tile8_bytes;
        for (int pn = 0, c = q.c_off + st.j * q.bn; pn < q.panels; ++pn, c += pw, src += panel_bytes)
          tma_store_4d(&tmY, src, c, st.ti.qt * h.tw, st.ti.pt * h.th, st.ti.img);
        bulk_commit();
        bulk_wait_read<1>();  // the store before this one has read its buffer: that buffer takes the next residual
        if (prev_slot >= 0 && !ld.done()) load_residual(ld, (uint32_t)prev_slot);
      }
      if (prev_slot >= 0 && !ld.done()) ld.next(h, chunks);
      prev_slot = (int)slot;
      if (++slot == nslots) { slot = 0; spar ^= 1u; }
    }
    if (lane0) bulk_wait_read<0>();  // the CTA's shared memory must outlive the reads of its last stores
    if (!ok && lane0) { abort_flag = 1; atomicOr(p.l1.status, kTimeoutStore); }
  } else if (warp < kFCtrlWarps + 4) {
    // ------------------------------------------------------------------ E1: layer-1 accumulator -> T[slot]
    const UmmaParams& q = p.l1;
    const int quad = warp & 3, row = quad * 32 + lane;
    EpiTile t;
    t.s_bias = s_bias1;
    t.s_scale = s_scale1;
    const int pp = row / q.twb, qq = row - pp * q.twb;  // accumulator row -> pixel of the patch grid
    t.smem_ok = pp < q.th && qq < q.tw;
    t.srow = t.smem_ok ? pp * q.tw + qq : 0;
    epi_row_setup(q, t);
    t.n0 = 0; t.y_off = 0; t.m = 0; t.row_ok = false;
    const uint32_t accf0 = smem_u32(&acc1_full[0]), acce0 = smem_u32(&acc1_empty[0]);
    const uint32_t tbf0 = smem_u32(&tb_full[0]), tbe0 = smem_u32(&tb_empty[0]);
    const uint32_t nacc = (uint32_t)q.nacc, ntb = (uint32_t)p.ntb;
    uint32_t ab = 0, apar = 0, slot = 0, tpar = 1;
    const int nchunk = q.bn >> 4;
    for (int k = 0; k < my_tiles; ++k) {
      bool ok = mbar_wait(accf0 + ab * 8u, apar, abortp);
      if (ok) ok = mbar_wait(tbe0 + slot * 8u, tpar, abortp);
      if (!ok) {
        if (lane0) { abort_flag = 1; atomicOr(q.status, kTimeoutEpilogue); }
        break;
      }
      tcgen05_fence_after();
      t.buf = base_ptr + p.off_tb + (size_t)slot * p.tb_bytes;
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)p.acc1_col + ab * (uint32_t)q.acc_stride;
      epilogue_row<kOut1, kResTma, false>(q, t, taddr, acce0 + ab * 8u, lane, 0, nchunk);
      fence_proxy_async_smem();  // the tile is read by the tensor core (async proxy)
      mbar_arrive(tbf0 + slot * 8u);
      if (++ab == nacc) { ab = 0; apar ^= 1u; }
      if (++slot == ntb) { slot = 0; tpar ^= 1u; }
    }
  } else {
    // ------------------------------------------------------------------ E2 groups: layer-2 accumulator g -> tile buffer
    const UmmaParams& q = p.l2;
    const int g = (warp - kFCtrlWarps - 4) >> 2;
    const int quad = warp & 3, row = quad * 32 + lane;
    EpiTile t;
    t.s_bias = s_bias2;
    t.s_scale = s_scale2;
    t.srow = row;                               // T rows are the tile's pixels in dense order
    t.smem_ok = row < p.l1.th * p.l1.tw;
    epi_row_setup(q, t);
    t.y_off = 0; t.m = 0; t.row_ok = false;
    const uint32_t accf = smem_u32(&acc2_full[g]), acce = smem_u32(&acc2_empty[g]);
    const uint32_t bfull0 = smem_u32(&buf_full[0]), ready0 = smem_u32(&store_ready[0]);
    const uint32_t nslots = (uint32_t)p.nslots;
    const int items = my_items;
    uint32_t apar = 0, slot = (uint32_t)g % nslots, spar = ((uint32_t)g / nslots) & 1u;
    int j = (j0 + g) % chunks;
    const int nchunk = q.bn >> 4;
    const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)g * (uint32_t)kFAcc2Cols;
    for (int i = g; i < items; i += kFE2Groups) {
      bool ok = mbar_wait(accf, apar, abortp);
      if (ok) ok = mbar_wait(bfull0 + slot * 8u, spar, abortp);
      if (!ok) {
        if (lane0) { abort_flag = 1; atomicOr(p.l1.status, kTimeoutEpilogue); }
        break;
      }
      tcgen05_fence_after();
      t.n0 = j * q.bn;
      t.buf = base_ptr + q.off_bufs + (size_t)slot * q.tile8_bytes;
      epilogue_row<kOut2, kResTma, false>(q, t, taddr, acce, lane, 0, nchunk);
      fence_proxy_async_smem();
      mbar_arrive(ready0 + slot * 8u);
      apar ^= 1u;
      slot += (uint32_t)kFE2Groups;
      while (slot >= nslots) { slot -= nslots; spar ^= 1u; }
      j += kFE2Groups;
      while (j >= chunks) j -= chunks;
    }
  }

  tcgen05_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tcgen05_fence_after();
    tmem_dealloc(tmem_base, 512u);
  }
}

template <int kOut1, int kOut2>
int launch_fused_variant(const CUtensorMap& tmA, const CUtensorMap& tmB1, const CUtensorMap& tmB2, const CUtensorMap& tmRes,
                         const CUtensorMap& tmY, const FusedParams& p, size_t dyn, int grid, cudaStream_t stream) {
  auto kernel = conv_fused_kernel<kOut1, kOut2>;
  static std::atomic<bool> configured[kMaxDevices];
  const int dev = current_device();
  if (dev < 0 || !configured[dev].load(std::memory_order_acquire)) {
    int rc = check_cuda(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit - kStaticSmemReserve),
                        "conv_fused: set shared memory size");
    if (rc != Q8_OK) return rc;
    rc = check_cuda(cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared),
                    "conv_fused: set shared memory carve-out");
    if (rc != Q8_OK) return rc;
    if (dev >= 0) configured[dev].store(true, std::memory_order_release);
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3((unsigned)kFThreads);
  cfg.dynamicSmemBytes = dyn;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t le = cudaLaunchKernelEx(&cfg, kernel, tmA, tmB1, tmB2, tmRes, tmY, p);
  if (le != cudaSuccess) {
    cudaGetLastError();
    return fail(Q8_ERR_CUDA, "conv_fused: launch failed (%s; grid %d, shared memory %zu)", cudaGetErrorString(le), grid, dyn);
  }
  return check_launch("conv_fused_kernel");
}

// The plan of a layer pair, or the reason it cannot run fused.
struct FusedPlan {
  FusedParams p;
  HaloTile ht;
  int BK1, P, Q;
  size_t dyn;
};

bool plan_fused(const q8_conv_desc& d1, const q8_conv_desc& d2, FusedPlan* out, const char** why) {
  const char* dummy;
  if (!why) why = &dummy;
  const int P = conv_out_extent(d1.H, d1.pad_h, d1.dil_h, d1.R, d1.stride_h), Q = conv_out_extent(d1.W, d1.pad_w, d1.dil_w, d1.S, d1.stride_w);
  if (P <= 0 || Q <= 0) { *why = "empty output"; return false; }
  if (d1.C % 16) { *why = "C of the first layer is not a multiple of 16"; return false; }
  if (d1.stride_h != 1 || d1.stride_w != 1) { *why = "first layer must have stride 1"; return false; }
  if (d1.K != 32 && d1.K != 64 && d1.K != 128) { *why = "first layer must have 32, 64 or 128 output channels"; return false; }
  if (d1.y_type != Q8_U8 && d1.y_type != Q8_S8) { *why = "the tensor between the layers must be 8-bit"; return false; }
  if (d2.R != 1 || d2.S != 1 || d2.stride_h != 1 || d2.stride_w != 1 || d2.pad_h || d2.pad_w) { *why = "second layer must be 1x1, stride 1, no padding"; return false; }
  if (d2.N != d1.N || d2.H != P || d2.W != Q || d2.C != d1.K || d2.x_type != d1.y_type) { *why = "second layer does not read the first layer's output"; return false; }
  if (d2.y_type != Q8_U8 && d2.y_type != Q8_S8) { *why = "second layer must have an 8-bit output"; return false; }
  if (d2.K % 16 || d2.K > 4096) { *why = "Cout of the second layer must be a multiple of 16, at most 4096"; return false; }
  const int ldc = d2.y_ldc == 0 ? d2.K : d2.y_ldc;
  if (ldc % 16 || d2.y_c_offset % 16) { *why = "y_ldc and y_c_offset must be multiples of 16"; return false; }
  HaloTile ht;
  if (d1.R * d1.S < 2 || !choose_halo_tile(d1, P, Q, &ht) || ht.sw != 1) { *why = "first layer has no halo tiling"; return false; }
  if (ht.eff < 0.5) { *why = "images too small for halo tiles"; return false; }

  FusedPlan pl;
  memset(&pl, 0, sizeof(pl));
  pl.ht = ht; pl.P = P; pl.Q = Q;
  UmmaParams& a = pl.p.l1;
  UmmaParams& b = pl.p.l2;
  // ---- layer 1: as the single-layer kernel plans a halo layer, with one tile of Cout1 columns
  const int BK1 = pick_bk(d1.C), BN1 = d1.K;
  pl.BK1 = BK1;
  a.bn = BN1; a.bk = BK1; a.ksteps = BK1 / 32;
  a.P = P; a.Q = Q; a.PQ = P * Q; a.M = d1.N * P * Q; a.K = d1.K;
  a.stride_h = 1; a.stride_w = 1; a.pad_h = d1.pad_h; a.pad_w = d1.pad_w; a.dil_h = d1.dil_h; a.dil_w = d1.dil_w;
  a.R = d1.R; a.S = d1.S; a.taps = d1.R * d1.S;
  a.halo_sw = 1; a.halo_e = 0; a.c_true = d1.C;
  a.a_mode = kAHalo;
  a.row16 = (unsigned)(d1.dil_h * ht.twb) * (unsigned)(BK1 >> 4);
  a.col16 = (unsigned)d1.dil_w * (unsigned)(BK1 >> 4);
  a.fast_taps = (d1.R == 3 && d1.S == 3) ? 9 : ((d1.R == 5 && d1.S == 5) ? 25 : 0);
  for (int r = 0; r < d1.R; ++r)
    for (int t = 0; t < d1.S; ++t) a.tap_shift16[r * d1.S + t] = (unsigned)((r * d1.dil_h * ht.twb + t * d1.dil_w) * BK1) >> 4;
  a.c_blocks = (d1.C + BK1 - 1) / BK1;
  a.C_pad = a.c_blocks * BK1;
  a.k_iters = a.taps * a.c_blocks; a.splits = 1; a.kps = a.k_iters; a.kb = 1;
  a.fd_splits = make_fastdiv(1); a.fd_cblocks = make_fastdiv(a.c_blocks); a.fd_s = make_fastdiv(d1.S);
  a.pw_shift = 0;
  while ((1 << a.pw_shift) < BN1) ++a.pw_shift;                     // T rows are Cout1 bytes: one panel
  a.pmask = BN1 == 128 ? 7 : (BN1 == 64 ? 3 : 1);
  a.panels = 1;
  a.n_tiles = 1; a.k_pad = BN1;
  a.tw = ht.tw; a.th = ht.th; a.twb = ht.twb; a.hb = ht.hb;
  a.q_tiles = (Q + ht.tw - 1) / ht.tw; a.p_tiles = (P + ht.th - 1) / ht.th;
  a.m_tiles = d1.N * a.p_tiles * a.q_tiles; a.m_tiles_real = a.m_tiles;
  a.fd_ntiles = make_fastdiv(1); a.fd_perimg = make_fastdiv(a.p_tiles * a.q_tiles); a.fd_qtiles = make_fastdiv(a.q_tiles);
  a.fd_pq = make_fastdiv(a.PQ); a.fd_q = make_fastdiv(Q);
  a.tile8_bytes = (unsigned)(kBM * BN1);
  a.acc_stride = BN1 < 32 ? 32 : BN1;
  a.nacc = (512 - kFE2Groups * kFAcc2Cols) / a.acc_stride;
  if (a.nacc > 2) a.nacc = 2;
  a.tmem_cols = 512;
  a.mma_lanes = 1;
  a.b_tile_bytes = (unsigned)(BN1 * BK1);
  a.b_sub_bytes = round_up(a.b_tile_bytes, 1024u);
  a.res_mode = kResNone; a.relu = d1.relu; a.out8 = 1; a.y_type = d1.y_type; a.y_vec = 1;
  a.scale_count = d1.scale_count;
  // ---- layer 2: chunks of up to 128 output channels over the K = Cout1 bytes of a T row
  const int BN2 = d2.K >= kFAcc2Cols ? kFAcc2Cols : d2.K;
  b.bn = BN2; b.bk = d1.K; b.ksteps = d1.K / 32;
  b.K = d2.K; b.M = a.M; b.P = P; b.Q = Q; b.PQ = P * Q;
  b.n_tiles = (d2.K + BN2 - 1) / BN2;
  b.k_pad = b.n_tiles * BN2;
  int pw = BN2 & -BN2;
  if (pw > 128) pw = 128;
  while ((1 << b.pw_shift) < pw) ++b.pw_shift;
  b.pmask = pw == 128 ? 7 : (pw == 64 ? 3 : (pw == 32 ? 1 : 0));
  b.panels = BN2 / pw;
  b.tile8_bytes = (unsigned)(kBM * BN2);
  b.b_tile_bytes = (unsigned)(BN2 * d1.K);
  b.res_tx_bytes = (unsigned)BN2 * (unsigned)(ht.tw * ht.th);
  b.relu = d2.relu; b.out8 = 1; b.y_type = d2.y_type; b.y_vec = 1;
  b.scale_count = d2.scale_count;
  b.ldc = ldc; b.c_off = d2.y_c_offset;
  b.res_signed = d2.res_type == Q8_S8;
  // ---- shared memory
  const unsigned chan1 = round_up((unsigned)a.k_pad * 8u, 256u), chan2 = round_up((unsigned)b.k_pad * 8u, 256u);
  const unsigned budget = (unsigned)(kSmemLimit - kStaticSmemReserve) - 1024u - chan1 - chan2;
  const unsigned w1_all = (unsigned)(a.c_blocks * a.taps) * a.b_tile_bytes;
  const unsigned w2_all = (unsigned)b.n_tiles * b.b_tile_bytes;
  if (w2_all > 64u * 1024u) { *why = "second layer's weights exceed 64 KiB"; return false; }
  const unsigned reach = (unsigned)(kBM + (d1.R - 1) * d1.dil_h * ht.twb + (d1.S - 1) * d1.dil_w) * BK1;
  a.a_sub_bytes = (unsigned)(BK1 * ht.twb * ht.hb);
  a.a_stage_bytes = round_up(reach > a.a_sub_bytes ? reach : a.a_sub_bytes, 1024u);
  pl.p.tb_bytes = (unsigned)(kBM * BN1);
  const unsigned w2_bytes = round_up(w2_all, 1024u);
  // weights of layer 1 resident when that leaves room for two patch stages, two T slots and three tile buffers
  const bool resident = w1_all <= 80u * 1024u && a.b_tile_bytes % (8u * BK1) == 0 &&
                        budget >= round_up(w1_all, 1024u) + w2_bytes + 2u * a.a_stage_bytes + 2u * pl.p.tb_bytes + 3u * b.tile8_bytes;
  a.b_mode = resident ? kBResident : kBRing;
  const unsigned w1_bytes = resident ? round_up(w1_all, 1024u) : 0u;
  a.b_T = 1; a.b_chunks = a.taps;
  unsigned ring_min = 0;
  if (!resident) {
    if (a.b_tile_bytes % (8u * BK1)) { *why = "weight tiles of the first layer do not keep the swizzle alignment"; return false; }
    // ring stages of several taps (one TMA operation each), two of them
    const unsigned fixed = w2_bytes + 2u * a.a_stage_bytes + 1u * pl.p.tb_bytes + 3u * b.tile8_bytes;
    const unsigned avail = budget > fixed ? budget - fixed : 0u;
    int T = (int)(48u * 1024u / a.b_tile_bytes);
    if (T > (int)(avail / (2u * a.b_tile_bytes))) T = (int)(avail / (2u * a.b_tile_bytes));
    if (T > a.taps) T = a.taps;
    if (T < 1) { *why = "no room for the first layer's weight ring"; return false; }
    a.b_chunks = (a.taps + T - 1) / T;
    a.b_T = (a.taps + a.b_chunks - 1) / a.b_chunks;
    a.b_chunks = (a.taps + a.b_T - 1) / a.b_T;
    a.b_sub_bytes = round_up((unsigned)a.b_T * a.b_tile_bytes, 1024u);
    ring_min = 2u * a.b_sub_bytes;
  }
  const unsigned need_min = w1_bytes + w2_bytes + 2u * a.a_stage_bytes + ring_min + 1u * pl.p.tb_bytes + 3u * b.tile8_bytes;
  if (budget < need_min) { *why = "the layer pair does not fit in shared memory"; return false; }
  unsigned rest = budget - need_min;
  pl.p.ntb = 1;
  pl.p.nslots = 3;
  if (rest >= pl.p.tb_bytes) { pl.p.ntb = 2; rest -= pl.p.tb_bytes; }
  if (rest >= 3u * b.tile8_bytes + a.a_stage_bytes) { pl.p.nslots = 6; rest -= 3u * b.tile8_bytes; }
  a.b_stages = 0;
  if (!resident) {
    a.b_stages = 2;
    while (a.b_stages < 4 && rest >= a.b_sub_bytes + a.a_stage_bytes) { ++a.b_stages; rest -= a.b_sub_bytes; }
  }
  a.stages = 2 + (int)(rest / a.a_stage_bytes);
  if (a.stages > kMaxStages) a.stages = kMaxStages;
  pl.p.off_w2 = w1_bytes;
  a.off_a = w1_bytes + w2_bytes;
  a.off_bring = a.off_a + (unsigned)a.stages * a.a_stage_bytes;
  pl.p.off_tb = a.off_bring + (unsigned)a.b_stages * a.b_sub_bytes;
  b.off_bufs = pl.p.off_tb + (unsigned)pl.p.ntb * pl.p.tb_bytes;
  a.off_chan = b.off_bufs + (unsigned)pl.p.nslots * b.tile8_bytes;
  pl.p.off_chan2 = a.off_chan + chan1;
  pl.dyn = 1024u + pl.p.off_chan2 + chan2;
  if (pl.dyn > (size_t)(kSmemLimit - kStaticSmemReserve)) { *why = "the layer pair does not fit in shared memory"; return false; }
  pl.p.acc1_col = kFE2Groups * kFAcc2Cols;
  // ---- instruction and matrix descriptors (see q8_conv_umma.cu)
  a.idesc = (2u << 4) | ((d1.x_type == Q8_S8 ? 1u : 0u) << 7) | (1u << 10) | ((unsigned)(BN1 >> 3) << 17) | ((unsigned)(kBM >> 4) << 24);
  b.idesc = (2u << 4) | ((d1.y_type == Q8_S8 ? 1u : 0u) << 7) | (1u << 10) | ((unsigned)(BN2 >> 3) << 17) | ((unsigned)(kBM >> 4) << 24);
  {
    const unsigned layout = BK1 == 128 ? 2u : (BK1 == 64 ? 4u : 6u);
    a.desc_hi = (unsigned)((8 * BK1) >> 4) | (1u << 14) | (layout << 29);
    const int BK2 = d1.K;
    const unsigned layout2 = BK2 == 128 ? 2u : (BK2 == 64 ? 4u : 6u);
    b.desc_hi = (unsigned)((8 * BK2) >> 4) | (1u << 14) | (layout2 << 29);
  }
  if (out) *out = pl;
  return true;
}

}  // namespace

bool fused_pair_eligible(const q8_conv_desc& d1, const q8_conv_desc& d2, const char** why) {
  return plan_fused(d1, d2, nullptr, why);
}

int launch_conv_fused(const q8_conv_desc& d1, const q8_conv_desc& d2, const void* x, const int8_t* w1, const int32_t* bias1,
                      const float* scale1, const int8_t* w2, const int32_t* bias2, const float* scale2, const void* residual,
                      float residual_scale, void* y, cudaStream_t stream) {
  const DriverFns& fn = driver_fns();
  if (!fn.tiled) return fail(Q8_ERR_CUDA, "conv_fused: cuTensorMapEncodeTiled entry point not available");
  unsigned int* status = status_word_device_ptr();
  if (!status) return fail(Q8_ERR_CUDA, "conv_fused: status word not available");
  FusedPlan pl;
  const char* why = "";
  if (!plan_fused(d1, d2, &pl, &why)) return fail(Q8_ERR_UNSUPPORTED, "q8_conv2d_then_1x1: %s", why);
  if (residual && !aligned16(residual)) return fail(Q8_ERR_UNSUPPORTED, "q8_conv2d_then_1x1: residual not 16-byte aligned");
  FusedParams& p = pl.p;
  const HaloTile& ht = pl.ht;
  const int BK1 = pl.BK1, P = pl.P, Q = pl.Q;
  p.l1.bias = bias1; p.l1.scale = scale1; p.l1.status = status;
  p.l2.bias = bias2; p.l2.scale = scale2; p.l2.status = status;
  p.l2.res = static_cast<const unsigned char*>(residual);
  p.l2.res_mode = residual ? kResTma : kResNone;
  p.l2.res_scale = residual_scale;
  p.l2.y = y;

  CUtensorMap tmA, tmB1, tmB2, tmRes, tmY;
  memset(&tmRes, 0, sizeof(tmRes));
  const cuuint32_t ones[4] = {1, 1, 1, 1};
  CUresult cr;
  {
    cuuint64_t dims[4] = {(cuuint64_t)d1.C, (cuuint64_t)d1.W, (cuuint64_t)d1.H, (cuuint64_t)d1.N};
    cuuint64_t strides[3] = {(cuuint64_t)d1.C, (cuuint64_t)d1.W * d1.C, (cuuint64_t)d1.H * d1.W * d1.C};
    cuuint32_t box[4] = {(cuuint32_t)BK1, (cuuint32_t)ht.twb, (cuuint32_t)ht.hb, 1};
    cr = fn.tiled(&tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(x), dims, strides, box, ones,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for_bytes(BK1), CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return fail(Q8_ERR_CUDA, "conv_fused: activation tensor map rejected (CUresult %d)", (int)cr);
  }
  {
    // (C, K, taps) view of the KRSC weights: a box brings Cout1 rows of all taps (resident) or of b_T taps (ring)
    cuuint64_t dims[3] = {(cuuint64_t)d1.C, (cuuint64_t)d1.K, (cuuint64_t)p.l1.taps};
    cuuint64_t strides[2] = {(cuuint64_t)p.l1.taps * d1.C, (cuuint64_t)d1.C};
    cuuint32_t box[3] = {(cuuint32_t)BK1, (cuuint32_t)d1.K, (cuuint32_t)(p.l1.b_mode == kBResident ? p.l1.taps : p.l1.b_T)};
    cr = fn.tiled(&tmB1, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<int8_t*>(w1), dims, strides, box, ones,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for_bytes(BK1), CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return fail(Q8_ERR_CUDA, "conv_fused: first weight tensor map rejected (CUresult %d)", (int)cr);
  }
  {
    // W2 is a [Cout2][Cout1] matrix: one box per chunk of output channels
    cuuint64_t dims[2] = {(cuuint64_t)d1.K, (cuuint64_t)d2.K};
    cuuint64_t strides[1] = {(cuuint64_t)d1.K};
    cuuint32_t box[2] = {(cuuint32_t)d1.K, (cuuint32_t)p.l2.bn};
    cr = fn.tiled(&tmB2, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(w2), dims, strides, box, ones,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for_bytes(d1.K), CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return fail(Q8_ERR_CUDA, "conv_fused: second weight tensor map rejected (CUresult %d)", (int)cr);
  }
  const int pw = 1 << p.l2.pw_shift;
  auto encode_rows = [&](CUtensorMap* tm, void* ptr, int channels, int ld, CUtensorMapL2promotion promo) -> CUresult {
    cuuint64_t dims[4] = {(cuuint64_t)channels, (cuuint64_t)Q, (cuuint64_t)P, (cuuint64_t)d1.N};
    cuuint64_t strides[3] = {(cuuint64_t)ld, (cuuint64_t)Q * ld, (cuuint64_t)P * Q * ld};
    cuuint32_t box[4] = {(cuuint32_t)pw, (cuuint32_t)ht.tw, (cuuint32_t)ht.th, 1};
    return fn.tiled(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, ptr, dims, strides, box, ones, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    swizzle_for_bytes(pw), promo, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  };
  if (residual) {
    cr = encode_rows(&tmRes, const_cast<void*>(residual), d2.K, d2.K, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
    if (cr != CUDA_SUCCESS) return fail(Q8_ERR_CUDA, "conv_fused: residual tensor map rejected (CUresult %d)", (int)cr);
  }
  cr = encode_rows(&tmY, y, p.l2.c_off + d2.K, p.l2.ldc, CU_TENSOR_MAP_L2_PROMOTION_NONE);
  if (cr != CUDA_SUCCESS) return fail(Q8_ERR_CUDA, "conv_fused: output tensor map rejected (CUresult %d)", (int)cr);

  const long long items = (long long)p.l1.m_tiles * p.l2.n_tiles;
  const int grid = (int)(items < sm_count() ? items : sm_count());
  if (d1.y_type == Q8_U8) {
    if (d2.y_type == Q8_U8) return launch_fused_variant<Q8_U8, Q8_U8>(tmA, tmB1, tmB2, tmRes, tmY, p, pl.dyn, grid, stream);
    return launch_fused_variant<Q8_U8, Q8_S8>(tmA, tmB1, tmB2, tmRes, tmY, p, pl.dyn, grid, stream);
  }
  if (d2.y_type == Q8_U8) return launch_fused_variant<Q8_S8, Q8_U8>(tmA, tmB1, tmB2, tmRes, tmY, p, pl.dyn, grid, stream);
  return launch_fused_variant<Q8_S8, Q8_S8>(tmA, tmB1, tmB2, tmRes, tmY, p, pl.dyn, grid, stream);
}

}  // namespace q8
