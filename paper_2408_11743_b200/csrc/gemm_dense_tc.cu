// Dense W4A16 layer for sm_100a, batch sizes from 17 rows: tcgen05 tensor cores with the WEIGHTS as the A operand in
// tensor memory, 128 batch rows per accumulator tile; larger batches are slabs of 128 rows inside one launch.
//
// The warp-level MMA (mma.sync) of the small-batch kernel runs at about a tenth of the tcgen05 rate on
// this architecture and is out of steam above batch 16.  Here the product is computed transposed, as the
// paper does for its sparse kernel (Section 4: C = (B^T A^T)^T): per 256-column tile of W and 128-row
// k-block
//     D_t[128 channels x MPAD batch rows] += W_t^T[128 x 128] . A^T[128 x MPAD],   t = 0, 1
// with UMMA shape M = 128 (output channels on the TMEM lanes), N = MPAD (batch), K = 16.
//
// One CTA per SM, 512 threads:
//   warps 0..7    dequantisers: thread = one output channel of the tile.  It reads its 128 codes of the
//                 k-block (four 16-byte shared loads), converts them to fp16 (q - 8) with the
//                 exponent-bias trick (Section 3.4 "Dequantization and Tensor Cores"), multiplies by the
//                 group scale (Section 3.4 "Groups and Instruction Ordering": applied in the main loop)
//                 and writes the 128 values into its TMEM lane with tcgen05.st (64 columns, two k per
//                 column).  Two or three A-operand slots let conversion of k-block i+1 overlap the MMAs of i.
//                 At the end of a column segment the same warps read the accumulators back (tcgen05.ld),
//                 run the fix-up and store C.
//   warps 8, 9    producers: per k-block one 16 KB bulk copy of packed weights (evict-first), the row of
//                 group scales, and one TMA tensor tile per 64-wide half of the activations (128-byte
//                 swizzle = the canonical K-major UMMA layout, rows >= M zero-filled), into a ring of stages.
//   warps 10..13  MMA issuers.  Issuing one tcgen05.mma occupies its thread for about 75 cycles, more than a
//                 128 x 64 x 16 product takes to execute, so four warps issue: up to batch 64 per tile t and half
//                 h of the k-block (each half into an accumulator of its own), at batch 128 per tile and half of
//                 the batch rows (N = 64).  One
//                 tcgen05.commit per stage and warp signals that the A slot and the stage are free.  Warp 10
//                 owns the TMEM allocation.
//   warps 14, 15  idle (they complete the last warpgroup for setmaxnreg).
//
// Partition: every column tile is cut into S k-ranges, one per CTA, where that keeps most SMs busy (one
// epilogue per CTA, all CTAs alike); else even stripes over all units.  Fix-up of a shared tile: above 32
// rows and when the S CTAs of every tile fit on the device as one wave of thread-block clusters, every CTA
// fetches its share of the batch rows from the partial tiles in the other CTAs' shared memory (fixed order
// of the sum); otherwise every contributor adds its partial tile into an fp32 tile
// in the workspace with L2 reductions and the last arriver stores C.  Bounded waits and programmatic
// dependent launch are those of the small-batch kernel (gemm_dense.cu).
#include <stdlib.h>

#include "device_utils.cuh"
#include "marlin_internal.cuh"
#include "tc_utils.cuh"

namespace marlin_b200 {
namespace {


// ---------------------------------------------------------------------------------------------
// geometry
// ---------------------------------------------------------------------------------------------
constexpr int kTcThreads = 512;
constexpr int kDequantWarps = 8;
constexpr int kDequantThreads = kDequantWarps * 32;
constexpr int kTcProducerWarps = 2;  // warps 8, 9
constexpr int kMmaWarp = 10;         // first of the MMA-issuing warps (it also owns the TMEM allocation)
constexpr int kTcMaxStages = 8;
constexpr int kTileN = 256;          // columns of W per CTA tile: two UMMA tiles of 128 channels
constexpr int kTmemCols = 512;
constexpr int kAuxRegs = 40;         // registers per thread of the copy and MMA warps
constexpr int kDequantRegs = 216;    // 512 threads start with 128 each: 2 x 128 x (128 - 40) / 256 = 88 more

// SP: the 2:4 variant (Section 4).  A stage then holds the 64 kept codes per column of the k-block (8 KB) and the
// metadata words of the 256 tensor-memory lanes (4 KB); an A-operand slot holds 32 columns of kept values and 4
// columns of metadata per 128-channel tile.
// FMT: 0 = dense 4-bit codes, 1 = the 2:4 variant, 2 = dense 8-bit codes (W = (q - 128) * s: a stage holds 128 bytes per
// column, [8 vectors][256 columns][16 bytes], the conversion places a byte under the exponent 0x64 with one byte
// permute per pair of weights and subtracts 1152; everything after the conversion is the 4-bit path).
constexpr int kFmtDense4 = 0, kFmtSparse4 = 1, kFmtDense8 = 2;
template <int MPAD, int FMT>
struct TcGeometry {
  static constexpr bool SP = FMT == kFmtSparse4;
  static constexpr bool W8 = FMT == kFmtDense8;
  static constexpr int A_HALF_BYTES = MPAD * 128;
  static constexpr int A_BYTES = 2 * A_HALF_BYTES;
  static constexpr int W_BYTES = SP ? 2 * kChunkBytes : (W8 ? 8 * kChunkBytes : 4 * kChunkBytes);
  static constexpr int META_BYTES = SP ? kChunkBytes : 0;
  static constexpr int STAGE_BYTES = A_BYTES + W_BYTES + META_BYTES;
  static constexpr int SC_ROW_BYTES = kTileN * 2;                   // one row of the tile's group scales
  static constexpr int SC_ZP_OFF = 4 * SC_ROW_BYTES;                // the zero points of those groups, if the layer has any
  static constexpr int SC_BYTES = 8 * SC_ROW_BYTES;                 // scales of one stage: up to four rows (groups of 32), then zero points
  static constexpr int FIXED_BYTES = 1024 + kTcMaxStages * SC_BYTES; // barriers + scale ring
  static constexpr int ALIGN_SLACK = 1024;
  static constexpr int STAGES =
      (kSmemBudget - FIXED_BYTES - ALIGN_SLACK) / STAGE_BYTES > kTcMaxStages
          ? kTcMaxStages
          : (kSmemBudget - FIXED_BYTES - ALIGN_SLACK) / STAGE_BYTES;
  static constexpr int SMEM_BYTES = FIXED_BYTES + ALIGN_SLACK + STAGES * STAGE_BYTES;
  // Issuing one tcgen05.mma occupies its thread for about 75 cycles, more than a 128 x 64 x 16 product takes
  // to execute, and a commit or a wait costs the thread as much again while the pipe drains.  So four warps
  // issue, two per 128-channel tile.  Up to batch 64 they split the k-block, each half into an accumulator of
  // its own (the epilogue adds the two).  At batch 128 there is no room for four full accumulators: the two
  // warps of a tile split the batch instead, 64 rows each (N = 64), which are the two halves of the tile's one
  // 128-column accumulator.
  static constexpr int MMA_WARPS = 4;
  static constexpr int KH = MPAD <= 64 ? 2 : 1;            // k-halves with accumulators of their own
  static constexpr int NH = MPAD <= 64 ? 1 : 2;            // halves of the batch per tile
  static constexpr int MMA_N = MPAD / NH;                  // N of one MMA
  static constexpr int D_COLS = 2 * KH * MPAD;             // accumulator of (tile t, half h) at column (t * KH + h) * MPAD
  // then as many A-operand slots as fit in the 512 columns: 2 tiles x 64 columns each; 2:4: 2 tiles x 32 columns of
  // kept values, then 2 tiles x 4 columns of metadata (even column numbers: the instruction names a pair of
  // metadata columns and which of the two)
  static constexpr int TILE_A_COLS = SP ? 32 : 64;
  static constexpr int SLOT_COLS = SP ? 72 : 128;
  static constexpr int A_SLOTS = (kTmemCols - D_COLS) / SLOT_COLS > 4 ? 4 : (kTmemCols - D_COLS) / SLOT_COLS;
  static constexpr int A_COL0 = kTmemCols - A_SLOTS * SLOT_COLS;
  static_assert(A_COL0 % 2 == 0 && SLOT_COLS % 2 == 0, "metadata columns must start on an even column");
  static_assert(A_SLOTS >= 2 && A_COL0 >= D_COLS, "tensor memory");
  static_assert(STAGE_BYTES % 1024 == 0, "swizzled tiles need 1024-byte alignment");
};

// ---------------------------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------------------------
// GR: the layer has group scales (multiplied into the weights in the loop); otherwise one scale per column,
// applied to the accumulators in the epilogue.
template <int MPAD, bool GR, int FMT>
__global__ void __launch_bounds__(kTcThreads, 1)
gemm_dense_tc_kernel(const GemmParams p, const __grid_constant__ CUtensorMap tmap_a) {
  using G = TcGeometry<MPAD, FMT>;
  constexpr bool SP = G::SP;
  constexpr bool W8 = G::W8;
  constexpr int NSTAGES = G::STAGES;
  constexpr int NSLOTS = G::A_SLOTS;
  constexpr int NM = G::MMA_WARPS;
  constexpr int KH = G::KH;
  extern __shared__ __align__(128) uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem);          // [8]  weights and scales of a stage have landed
  uint64_t* xfull = reinterpret_cast<uint64_t*>(smem + 256);   // [8]  activation tile of a stage has landed
  uint64_t* empty = reinterpret_cast<uint64_t*>(smem + 64);    // [8]  the codes of a stage are in registers
  uint64_t* afull = reinterpret_cast<uint64_t*>(smem + 128);   // [4]  A-operand slot written
  uint64_t* mdone = reinterpret_cast<uint64_t*>(smem + 160);   // [8]  the MMAs of a stage have completed
  uint64_t* dfull = reinterpret_cast<uint64_t*>(smem + 224);   //      accumulators of a segment complete
  uint64_t* dempty = reinterpret_cast<uint64_t*>(smem + 232);  //      accumulators read out
  uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(smem + 240);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + 244);
  volatile int* last_flag = reinterpret_cast<volatile int*>(smem + 248);
  uint8_t* sc_ring = smem + 1024;  // [stage][256] fp16 scales, copied with the stage
  uint8_t* stage0 = smem + G::FIXED_BYTES;

  // the warp index, broadcast from lane 0 so that the compiler knows it is the same in all lanes (every role branch
  // and loop bound below depends on it: otherwise each warp-wide instruction gets a divergence check)
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
  const int lane = threadIdx.x & 31;
  const uint32_t worker = blockIdx.x;
  const uint32_t U = p.units, P = p.workers, KB = p.kb;
  // split > 0: one k-range of one column tile per CTA (the last range of a tile ends where the next tile begins)
  // whole: the stripes are cut at tile boundaries (many more tiles than workers: nothing is shared, no fix-up)
  const uint32_t u0 = p.split   ? split_begin32(worker, KB, p.split)
                      : p.whole ? stripe_begin32(worker, (uint32_t)p.ncols, P) * KB
                                : stripe_begin32(worker, U, P);
  const uint32_t u1 = p.split   ? split_begin32(worker + 1, KB, p.split)
                      : p.whole ? stripe_begin32(worker + 1, (uint32_t)p.ncols, P) * KB
                                : stripe_begin32(worker + 1, U, P);

  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGES; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&xfull[s], 1);
      mbar_init(&empty[s], kDequantWarps);
      mbar_init(&mdone[s], NM);
    }
    for (int a = 0; a < NSLOTS; ++a) mbar_init(&afull[a], kDequantWarps);
    mbar_init(dfull, NM);
    mbar_init(dempty, kDequantWarps);
    *abort_flag = 0;
    *last_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp) {
    tmem_alloc(tmem_base_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_base_slot;

  if (warp >= kDequantWarps) {
    setmaxnreg_dec<kAuxRegs>();
    if (warp < kDequantWarps + kTcProducerWarps) {
      // ------------------------------- producers --------------------------------------------
      const int pw = warp - kDequantWarps;
      if (lane == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_a) : "memory");
      // one slab: every weight byte is read once; several slabs read the layer once each, from the L2 after the first
      // (normal priority: marked to stay, the weights of the layers before would crowd the L2)
      const uint64_t pol_w = p.slabs > 1 ? policy_evict_normal() : policy_evict_first();
      const uint64_t pol_a = policy_evict_last();
      // weights and activations complete barriers of their own: the converting warps need only the former, and
      // on the first pass over the ring those arrive before the dependency wait
      // groups of 128 rows and more: one scale row per k-block; groups of 64 or 32 rows: two or four, which the
      // packed layout keeps together per (k-block, column tile)
      const uint32_t sc_copy = (uint32_t)p.sub_groups * G::SC_ROW_BYTES;
      const bool zp = p.zq != nullptr;  // zero points: rows of the same shape and order as the scales, copied beside them
      const uint32_t tx_bytes = G::W_BYTES + G::META_BYTES + (p.grouped ? sc_copy : 0) + (zp ? sc_copy : 0);
      auto scale_off = [&](uint32_t col, uint32_t kb) -> size_t {
        if (p.sub_groups > 1) return ((size_t)kb * (p.N / kTileN) + col) * sc_copy;
        const uint32_t gi = p.group_shift >= 0 ? (kb >> p.group_shift) : (kb / (uint32_t)p.kb_per_group);
        return ((size_t)gi * p.N + (size_t)col * kTileN) * 2;
      };
      auto scale_src = [&](uint32_t col, uint32_t kb) -> const uint8_t* { return p.sq + scale_off(col, kb); };
      // weights of (kb, col): the four chunks of a 256-column tile are adjacent, k-blocks follow one another
      auto weight_src = [&](uint32_t col, uint32_t kb) -> const uint8_t* {
        return p.wq + ((size_t)col * KB + kb) * (size_t)G::W_BYTES;
      };
      // 2:4: the metadata records follow the same order in a buffer of their own
      auto meta_src = [&](uint32_t col, uint32_t kb) -> const uint8_t* {
        return p.meta + ((size_t)col * KB + kb) * (size_t)G::META_BYTES;
      };
      // first pass over the ring: weights before the dependency wait, activations after it
      uint32_t u = u0 + pw;
      int s = pw;
#ifdef MARLIN_TEST_HOOKS
      const bool withhold = worker == 0 && pw == 1 && p.status[7] == kTestWithholdMagic;  // stage 1 belongs to producer 1
#else
      constexpr bool withhold = false;
#endif
      if (lane == 0) {
        for (; u < u1 && s < NSTAGES; u += kTcProducerWarps, s += kTcProducerWarps) {
          const uint32_t vcol = u / KB, kb = u - vcol * KB;
          const uint32_t col = vcol / p.slabs;
          if (withhold && s == 1) continue;
          mbar_expect_tx(&full[s], tx_bytes);
          bulk_g2s(stage0 + (size_t)s * G::STAGE_BYTES + G::A_BYTES, weight_src(col, kb), G::W_BYTES, &full[s], pol_w);
          if constexpr (SP)
            bulk_g2s(stage0 + (size_t)s * G::STAGE_BYTES + G::A_BYTES + G::W_BYTES, meta_src(col, kb), G::META_BYTES,
                     &full[s], pol_w);
          if (p.grouped) bulk_g2s(sc_ring + (size_t)s * G::SC_BYTES, scale_src(col, kb), sc_copy, &full[s], pol_w);
          if (zp) bulk_g2s(sc_ring + (size_t)s * G::SC_BYTES + G::SC_ZP_OFF, p.zq + scale_off(col, kb), sc_copy, &full[s], pol_w);
        }
      }
      __syncwarp();
      pdl_wait_prior_grids();
      u = u0 + pw;
      s = pw;
      for (; u < u1 && s < NSTAGES; u += kTcProducerWarps, s += kTcProducerWarps) {
        const uint32_t vcol = u / KB, kb = u - vcol * KB;
        const uint32_t slab = vcol % p.slabs;
        if (lane == 0) mbar_expect_tx(&xfull[s], G::A_BYTES);
        __syncwarp();
        if (lane < 2)
          tma_load_2d(stage0 + (size_t)s * G::STAGE_BYTES + lane * G::A_HALF_BYTES, &tmap_a,
                      (int)(kb * kTileK + lane * 64), (int)(slab * MPAD), &xfull[s], pol_a);
      }
      uint32_t ph = 1;
      s -= NSTAGES;
      for (; u < u1; u += kTcProducerWarps) {
        const uint32_t vcol = u / KB, kb = u - vcol * KB;
        const uint32_t col = vcol / p.slabs, slab = vcol - col * p.slabs;
        // the stage is free when its codes are in registers and the MMAs that read its activations are done
        mbar_wait<200>(&empty[s], ph ^ 1u, abort_flag, p.status);
        mbar_wait<200>(&mdone[s], ph ^ 1u, abort_flag, p.status);
        uint8_t* st = stage0 + (size_t)s * G::STAGE_BYTES;
        if (lane == 0) {
          mbar_expect_tx(&full[s], tx_bytes);
          bulk_g2s(st + G::A_BYTES, weight_src(col, kb), G::W_BYTES, &full[s], pol_w);
          if constexpr (SP) bulk_g2s(st + G::A_BYTES + G::W_BYTES, meta_src(col, kb), G::META_BYTES, &full[s], pol_w);
          if (p.grouped) bulk_g2s(sc_ring + (size_t)s * G::SC_BYTES, scale_src(col, kb), sc_copy, &full[s], pol_w);
          if (zp) bulk_g2s(sc_ring + (size_t)s * G::SC_BYTES + G::SC_ZP_OFF, p.zq + scale_off(col, kb), sc_copy, &full[s], pol_w);
          mbar_expect_tx(&xfull[s], G::A_BYTES);
        }
        __syncwarp();
        if (lane < 2)
          tma_load_2d(st + lane * G::A_HALF_BYTES, &tmap_a, (int)(kb * kTileK + lane * 64), (int)(slab * MPAD), &xfull[s],
                      pol_a);
        s += kTcProducerWarps;
        if (s >= NSTAGES) { s -= NSTAGES; ph ^= 1u; }
      }
      if (*abort_flag) {
        for (int x = 0; x < 1000; ++x) __nanosleep(1000);
      }
    } else if (warp >= kMmaWarp && warp < kMmaWarp + NM) {
      // ------------------------------- MMA issuers --------------------------------------------
      constexpr uint32_t idesc = instr_desc_f16(128, G::MMA_N);
      constexpr int KS = 8 / KH;           // K = 16 steps per warp and stage
      const int mw = warp - kMmaWarp;
      const int t = mw & 1;                // 128-channel tile
      const int h = KH == 2 ? mw >> 1 : 0;        // half of the k-block
      const int nh = G::NH == 2 ? mw >> 1 : 0;    // half of the batch rows
      const uint32_t d_tmem = tmem_base + (uint32_t)((t * KH + h) * MPAD + nh * G::MMA_N);
      // rows 64 nh .. of the activation tile: eight 1024-byte groups of eight rows further on
      const uint32_t b_rows_off = (uint32_t)(nh * G::MMA_N * 128);
      uint32_t it = 0;   // stage counter of this CTA
      uint32_t seg = 0;  // segment counter
      uint32_t u = u0;
      while (u < u1) {
        const uint32_t kb0 = u % KB;
        const uint32_t len = min(KB - kb0, u1 - u);
        // the accumulators are overwritten by the first MMA of the segment: the previous one must be read out
        mbar_wait(dempty, (seg & 1u) ^ 1u, abort_flag, p.status);
        for (uint32_t x = 0; x < len; ++x, ++it) {
          const int s = (int)(it % NSTAGES);
          const int slot = (int)(it % NSLOTS);
          mbar_wait(&xfull[s], (it / NSTAGES) & 1u, abort_flag, p.status);
          mbar_wait(&afull[slot], (it / NSLOTS) & 1u, abort_flag, p.status);
          tc_fence_after_sync();
          if (lane == 0) {
            // descriptor of the first K = 16 step of the stage; the others differ in the address field only
            const uint64_t desc0 = smem_desc_k_sw128(smem_u32(stage0 + (size_t)s * G::STAGE_BYTES) + b_rows_off);
            const uint32_t slot_col = tmem_base + (uint32_t)(G::A_COL0 + slot * G::SLOT_COLS);
            const uint32_t a_tmem = slot_col + (uint32_t)(t * G::TILE_A_COLS);
            if constexpr (!SP) {
#pragma unroll
              for (int k2 = 0; k2 < KS; ++k2) {
                const int ks = h * KS + k2;
                const uint64_t bdesc = desc0 + (uint64_t)(((ks >> 2) * G::A_HALF_BYTES + (ks & 3) * 32) >> 4);
                tc_mma_ts(d_tmem, a_tmem + ks * 8, bdesc, idesc, (x == 0 && k2 == 0) ? 0u : 1u);
              }
            } else {
              // 2:4 (Section 4): one instruction takes 32 rows of k (16 kept values per channel = 8 columns of
              // the slot) and the metadata column of that step; four steps per k-block
              const uint32_t e_tmem = slot_col + (uint32_t)(2 * G::TILE_A_COLS + t * 4);
#pragma unroll
              for (int k2 = 0; k2 < KS / 2; ++k2) {
                const int i = h * (KS / 2) + k2;
                const uint64_t bdesc = desc0 + (uint64_t)(((i >> 1) * G::A_HALF_BYTES + (i & 1) * 64) >> 4);
                tc_mma_sp_ts(d_tmem, a_tmem + i * 8, bdesc, e_tmem + (uint32_t)(i & ~1), idesc | kIdescSparse | (uint32_t)(i & 1),
                             (x == 0 && k2 == 0) ? 0u : 1u);
              }
            }
            // one arrival when these MMAs are done: the A slot may be rewritten, the activation tile refilled
            tc_commit(&mdone[s]);
            if (x + 1 == len) tc_commit(dfull);
          }
          __syncwarp();
        }
        u += len;
        ++seg;
      }
    }
    if (p.cluster) {
      // every thread of every CTA of the cluster takes part in the two barriers of the epilogue
      cluster_sync_all();
      cluster_sync_all();
    }
    // ---- the TMEM owner waits for everybody who touches tensor memory, then frees it ----
    if (warp == kMmaWarp) {
      named_bar_sync(2, kDequantThreads + 32);
      tc_fence_after_sync();
      tmem_dealloc(tmem_base, kTmemCols);
    }
    return;
  }

  // --------------------------------- dequantisers / epilogue ----------------------------------
  setmaxnreg_inc<kDequantRegs>();
  const int tile = warp >> 2;                 // which 128 channels of the 256-column tile
  const uint32_t lane_win = (uint32_t)(warp & 3) * 32u;  // this warp's TMEM lanes
  const int n256 = tile * 128 + (int)lane_win + lane;    // column of the thread inside the CTA tile
  const int q = n256 >> 6, n64 = n256 & 63;
  const int j = n64 >> 4, b = (n64 >> 3) & 1, g = n64 & 7;
  const uint32_t vec_off = (uint32_t)q * kChunkBytes + (uint32_t)(((2 * j + b) * 32 + 4 * g) * 16);
  const int spos = q * 64 + 8 * g + 2 * j + b;  // position of this column's scale inside the tile's 256 scales
  const int ctid = threadIdx.x;
  const uint32_t tmem_lane = tmem_base + (lane_win << 16);

  uint32_t it = 0, seg = 0;
  uint32_t u = u0;
  bool waited_for_prior_grid = false;
  while (u < u1) {
    // virtual column tile = (column tile of W, slab of MPAD batch rows): batches above 128 rows replicate the
    // layer in the unit numbering (Section 3.4, last paragraph), slab after slab of one column tile
    const uint32_t vcol = u / KB;
    const uint32_t col = vcol / p.slabs, slab = vcol - col * p.slabs;
    const int m_lim = p.M - (int)slab * MPAD;   // rows of this slab that exist
    const uint32_t kb0 = u % KB;
    const uint32_t len = min(KB - kb0, u1 - u);
    const uint16_t* sptr = reinterpret_cast<const uint16_t*>(p.sq) + (size_t)col * kTileN + spos;

    uint32_t sv4[4] = {0, 0, 0, 0};  // {scale, scale} of this thread's column for the four 32-row quarters of the k-block
    // the subtrahends of the conversion per quarter: {1024 + z, 1024 + z} and {-(64 + z), -(64 + z)}, z = 8 without zero points
    uint32_t zlo4[4] = {0x64086408u, 0x64086408u, 0x64086408u, 0x64086408u};
    uint32_t zhi4[4] = {0xd480d480u, 0xd480d480u, 0xd480d480u, 0xd480d480u};
    const bool zp = p.zq != nullptr;
    float sc_col = 1.f;  // the column's single scale
    if constexpr (!GR) sc_col = __half2float(__ushort_as_half(__ldg(sptr)));
    for (uint32_t x = 0; x < len; ++x, ++it) {
      const int s = (int)(it % NSTAGES);
      const int slot = (int)(it % NSLOTS);
      mbar_wait(&full[s], (it / NSTAGES) & 1u, abort_flag, p.status);
      if constexpr (GR) {
        // the scale row of the k-block came with the stage (a global read here would be a cold DRAM access)
        const uint32_t sbase = smem_u32(sc_ring) + (uint32_t)s * G::SC_BYTES + (uint32_t)spos * 2;
#pragma unroll
        for (int qd = 0; qd < 4; ++qd) {
          // quarter qd lies in scale row qd * sub_groups / 4 of the stage (row 0 for groups of 128 rows and more)
          const uint32_t sv = lds16(sbase + (uint32_t)((qd * p.sub_groups) >> 2) * G::SC_ROW_BYTES);
          sv4[qd] = sv | (sv << 16);
        }
        if (zp) {
#pragma unroll
          for (int qd = 0; qd < 4; ++qd) {
            const uint32_t zv = lds16(sbase + G::SC_ZP_OFF + (uint32_t)((qd * p.sub_groups) >> 2) * G::SC_ROW_BYTES);
            const uint32_t z2 = zv | (zv << 16);
            zlo4[qd] = hadd2_u32(z2, 0x64006400u);   // 1024 + z
            zhi4[qd] = hsub2_u32(0xd400d400u, z2);   // -64 - z
          }
        }
      }
      const uint32_t wbase = smem_u32(stage0) + (uint32_t)s * G::STAGE_BYTES + G::A_BYTES + ((SP || W8) ? (uint32_t)n256 * 16u : vec_off);
      uint4 v[W8 ? 8 : 4];
      if constexpr (W8) {
#pragma unroll
        for (int c = 0; c < 8; ++c) v[c] = lds128(wbase + c * 256 * 16);  // codes of rows 16c .. 16c + 15 of this column
      } else if constexpr (!SP) {
#pragma unroll
        for (int c = 0; c < 4; ++c) v[c] = lds128(wbase + (uint32_t)(((c + (g >> 1)) & 3) * 16));  // rows 16c.. sit in slot (c + g/2) % 4
      } else {
        v[0] = lds128(wbase);                        // kept values 0..31 of this column
        v[1] = lds128(wbase + 256 * 16);             // kept values 32..63
        v[2] = lds128(wbase + (uint32_t)G::W_BYTES); // the four metadata words of this tensor-memory lane
      }

      if (it >= (uint32_t)NSLOTS) {
        // the slot was last read by the MMAs of stage it - NSLOTS
        const uint32_t jt = it - NSLOTS;
        mbar_wait(&mdone[jt % NSTAGES], (jt / NSTAGES) & 1u, abort_flag, p.status);
      }
      tc_fence_after_sync();
      const uint32_t slot_col = tmem_lane + (uint32_t)(G::A_COL0 + slot * G::SLOT_COLS);
      if constexpr (W8) {
        const uint32_t a_col = slot_col + (uint32_t)(tile * 64);
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          uint32_t r[32];
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const uint4 vv = v[4 * hh + c];
            const uint32_t w4[4] = {vv.x, vv.y, vv.z, vv.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              // bytes (b0, b1) and (b2, b3) of the word under the exponent of 1024: 1024 + b, minus 1152 = b - 128
              const uint32_t lo = hsub2_u32(__byte_perm(w4[e], 0x64646464u, 0x4140), 0x64806480u);
              const uint32_t hi = hsub2_u32(__byte_perm(w4[e], 0x64646464u, 0x4342), 0x64806480u);
              // rows 64hh + 16c ..: quarter 2hh + c / 2 of the k-block
              r[8 * c + 2 * e] = GR ? hmul2_u32(lo, sv4[2 * hh + (c >> 1)]) : lo;
              r[8 * c + 2 * e + 1] = GR ? hmul2_u32(hi, sv4[2 * hh + (c >> 1)]) : hi;
            }
          }
          tc_st_x32(a_col + (uint32_t)(32 * hh), r);  // column = row / 2
        }
      } else if constexpr (!SP) {
        const uint32_t a_col = slot_col + (uint32_t)(tile * 64);
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          // 64 rows of k = 32 columns of the slot, written with one store
          uint32_t r[32];
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const uint32_t w0 = hh == 0 ? v[c].x : v[c].z, w1 = hh == 0 ? v[c].y : v[c].w;
            uint32_t lo[4], hi[4];
            dequant8_zp(w0, lo, zlo4[2 * hh + (c >> 1)], zhi4[2 * hh + (c >> 1)]);  // rows 64hh + 16c + 0..7
            dequant8_zp(w1, hi, zlo4[2 * hh + (c >> 1)], zhi4[2 * hh + (c >> 1)]);  // rows 64hh + 16c + 8..15
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              // rows 64hh + 16c ..: quarter 2hh + c / 2 of the k-block
              r[8 * c + e] = GR ? hmul2_u32(lo[e], sv4[2 * hh + (c >> 1)]) : lo[e];
              r[8 * c + 4 + e] = GR ? hmul2_u32(hi[e], sv4[2 * hh + (c >> 1)]) : hi[e];
            }
          }
          tc_st_x32(a_col + (uint32_t)(32 * hh), r);  // column = row / 2
        }
      } else {
        // 64 kept values = 32 columns: column G holds the two kept values of the k-block's group G of four rows
        uint32_t r[32];
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          const uint32_t w[4] = {v[c].x, v[c].y, v[c].z, v[c].w};
#pragma unroll
          for (int wi = 0; wi < 4; ++wi) {
            uint32_t a[4];
            dequant8(w[wi], a);
#pragma unroll
            // kept pair 16c + 4wi + e = group of four original rows: quarter 2c + wi / 2 of the k-block
            for (int e = 0; e < 4; ++e) r[16 * c + 4 * wi + e] = GR ? hmul2_u32(a[e], sv4[2 * c + (wi >> 1)]) : a[e];
          }
        }
        tc_st_x32(slot_col + (uint32_t)(tile * 32), r);
        const uint32_t mw[4] = {v[2].x, v[2].y, v[2].z, v[2].w};
        tc_st_x4(slot_col + (uint32_t)(64 + tile * 4), mw);
      }
      // The codes have been converted, so the shared loads that fetched them have certainly delivered: only now is
      // the weight part of the stage released.  (An arrival issued right behind the loads can be performed before a
      // multi-wavefront shared load has read its data: with a weight ring refilled without waiting for the MMAs, a
      // refill that followed at once overwrote codes still being read.)
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[s]);
      tc_wait_st();
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&afull[slot]);
    }

    // ---- segment end: read the accumulators, fix-up across CTAs, store C ----
    mbar_wait(dfull, seg & 1u, abort_flag, p.status);
    tc_fence_after_sync();
    ++seg;
    if (!waited_for_prior_grid) {
      // first write to C or the workspace: the previous kernel of the stream must be done with them
      pdl_wait_prior_grids();
      waited_for_prior_grid = true;
    }
    const int first_w = p.split ? (int)(vcol * p.split) : (int)stripe_owner32(vcol * KB, U, P);
    const int last_w = p.split ? (int)(vcol * p.split + p.split - 1) : (int)stripe_owner32((vcol + 1) * KB - 1, U, P);
    const bool shared_tile = !p.whole && last_w > first_w;
    if (p.cluster) {
      // The CTAs of this column tile form a thread-block cluster and finish side by side, so the partial
      // tiles never leave the SMs.  Every CTA puts its partial tile into its own stage ring (free by now), a
      // cluster barrier publishes them, and every CTA fetches, for its share of the batch rows (blocks of four
      // rows are dealt out to the ranks), the S partials from the shared memory of the CTAs that hold them,
      // adds them in rank order and stores that part of C.  Fixed order of the fp32 sum, no atomics, no
      // workspace.  Distributed shared memory is slow here (20-30 GB/s per SM, loads and stores alike, and worse
      // with many requests in flight), so this epilogue still costs microseconds at 128 rows; pushing the tiles
      // with remote stores, with asynchronous remote stores, or exchanging them through the L2 under the same
      // barriers were all slower.
      constexpr int R4 = MPAD / 4;              // blocks of four batch rows
      const int S = (int)p.split;
      const int r = (int)cluster_ctarank();
      // (the partial tile goes into this CTA's OWN ring, which is quiet once its accumulators are complete: no
      // barrier is needed before it; the others read it only after the barrier below)
      const uint32_t mine_s = smem_u32(stage0); // [block of four rows][256 columns] float4
#pragma unroll 1
      for (int cc = 0; cc < MPAD / 32; ++cc) {
        float part[32];
        tc_ld_x32(tmem_lane + (uint32_t)(tile * KH * MPAD + cc * 32), part);
        if constexpr (KH == 2) {
          float part2[32];
          tc_ld_x32(tmem_lane + (uint32_t)((tile * KH + 1) * MPAD + cc * 32), part2);
          tc_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) part[e] += part2[e];
        } else {
          tc_wait_ld();
        }
        if constexpr (!GR) {
#pragma unroll
          for (int e = 0; e < 32; ++e) part[e] *= sc_col;
        }
#pragma unroll
        for (int m4 = 0; m4 < 8; ++m4)
          *reinterpret_cast<float4*>(stage0 + (size_t)((cc * 8 + m4) * kTileN + n256) * 16) =
              make_float4(part[4 * m4], part[4 * m4 + 1], part[4 * m4 + 2], part[4 * m4 + 3]);
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(dempty);
      cluster_sync_all();                       // every CTA's partial tile is in its shared memory
      const int b0 = r * R4 / S, b1 = (r + 1) * R4 / S;
      // the sums go through a row-major fp16 tile behind the partial tile, so that C is written with 16-byte
      // stores along its rows
      uint16_t* out = reinterpret_cast<uint16_t*>(stage0 + (size_t)R4 * kTileN * 16);
      for (int blk = b0; blk < b1; ++blk) {
        const int li = blk - b0;
        const uint32_t at = mine_s + (uint32_t)((blk * kTileN + n256) * 16);
        float4 sum = ld_cluster_f32x4(at, 0u);
        for (int src = 1; src < S; ++src) {
          const float4 v = ld_cluster_f32x4(at, (uint32_t)src);
          sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
        }
        out[(4 * li + 0) * kTileN + n256] = __half_as_ushort(__float2half_rn(sum.x));
        out[(4 * li + 1) * kTileN + n256] = __half_as_ushort(__float2half_rn(sum.y));
        out[(4 * li + 2) * kTileN + n256] = __half_as_ushort(__float2half_rn(sum.z));
        out[(4 * li + 3) * kTileN + n256] = __half_as_ushort(__float2half_rn(sum.w));
      }
      named_bar_sync(1, kDequantThreads);
      {
        const int rows_here = 4 * (b1 - b0);
        if (!p.swiglu) {
          for (int vec = ctid; vec < rows_here * (kTileN / 8); vec += kDequantThreads) {
            const int row = vec / (kTileN / 8), c16 = vec % (kTileN / 8);
            const int m = 4 * b0 + row;
            if (m < m_lim)
              *reinterpret_cast<uint4*>(p.C + ((size_t)slab * MPAD + m) * p.N + (size_t)col * kTileN + c16 * 8) =
                  *reinterpret_cast<const uint4*>(out + row * kTileN + c16 * 8);
          }
        } else {
          // fused activation: every block of 16 columns is eight gate channels and the same eight up channels
          const int ldc = p.N / 2;
          for (int vec = ctid; vec < rows_here * (kTileN / 16); vec += kDequantThreads) {
            const int row = vec / (kTileN / 16), c2 = vec % (kTileN / 16);
            const int m = 4 * b0 + row;
            if (m < m_lim)
              *reinterpret_cast<uint4*>(p.C + ((size_t)slab * MPAD + m) * ldc + (size_t)col * (kTileN / 2) + c2 * 8) =
                  swiglu8(*reinterpret_cast<const uint4*>(out + row * kTileN + (2 * c2) * 8),
                          *reinterpret_cast<const uint4*>(out + row * kTileN + (2 * c2 + 1) * 8));
          }
        }
      }
      cluster_sync_all();                       // nobody reads this CTA's shared memory any more
      u += len;
      continue;
    }
    // The column tile may be shared by several CTAs.  With up to 128 rows a partial tile is large and
    // a small layer splits every column many ways, so the sum is left to the L2: every contributor
    // adds its partial into the tile's fp32 accumulation buffer with fire-and-forget reductions
    // (float4 index = (m / 4) * 256 + column: coalesced over columns), the last arriver reads the
    // total, clears the buffer for the next call and stores C.  (The order of these fp32 additions
    // is not fixed, so the last bits of a shared tile can differ from run to run.)
    // One accumulation tile and one counter per virtual column tile; where there are more of those than workers,
    // per tile that can be shared, numbered by the first worker on it (at most one tile runs over the end of a
    // worker's stripe).
    const uint32_t fix = (uint32_t)p.ncols <= P ? vcol : (uint32_t)first_w;
    float4* mine = reinterpret_cast<float4*>(p.tc_tiles + (size_t)fix * (kTileN * MPAD)) + n256;
    uint16_t* cptr = p.C + (size_t)slab * MPAD * p.N + (size_t)col * kTileN + n256;
    // Row m of this thread's column goes to C.  With the fused activation the thread of a gate channel (columns
    // 0..7 of a block of 16) fetches the up channel's value from the lane eight further on and stores
    // silu(gate) * up into a C of half the width; every lane of the warp takes part in the exchange.
    const int ldc = p.N / 2;
    uint16_t* hptr = p.C + (size_t)slab * MPAD * ldc + (size_t)col * (kTileN / 2) + (n256 >> 4) * 8 + (n256 & 7);
    auto put_plain = [&](int m, float v) {
      if (m < m_lim) cptr[(size_t)m * p.N] = __half_as_ushort(__float2half_rn(v));
    };
    auto put_act = [&](int m, float v) {
      const uint32_t h = __half_as_ushort(__float2half_rn(v));
      const uint32_t other = __shfl_xor_sync(0xffffffffu, h, 8);
      if ((lane & 8) == 0 && m < m_lim) hptr[(size_t)m * ldc] = (uint16_t)(swiglu2(h, other) & 0xffffu);
    };
    if (p.swiglu && !shared_tile) {
      // fused activation on a tile of its own: 32 batch rows at a time (the exchange between lanes and the
      // activation need registers of their own)
#pragma unroll 1
      for (int cc = 0; cc < MPAD / 32; ++cc) {
        float part[32];
        tc_ld_x32(tmem_lane + (uint32_t)(tile * KH * MPAD + cc * 32), part);
        if constexpr (KH == 2) {
          float part2[32];
          tc_ld_x32(tmem_lane + (uint32_t)((tile * KH + 1) * MPAD + cc * 32), part2);
          tc_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) part[e] += part2[e];
        } else {
          tc_wait_ld();
        }
#pragma unroll
        for (int e = 0; e < 32; ++e) put_act(cc * 32 + e, GR ? part[e] : part[e] * sc_col);
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(dempty);
      u += len;
      continue;
    }
    // All accumulators of this thread's channel out of tensor memory first: the MMAs of the next segment may then
    // start while the partial tile goes to the L2 or C is stored.
    float acc[MPAD];
#pragma unroll
    for (int cc = 0; cc < MPAD / 32; ++cc) {
      tc_ld_x32(tmem_lane + (uint32_t)(tile * KH * MPAD + cc * 32), reinterpret_cast<float(&)[32]>(acc[32 * cc]));
      if constexpr (KH == 2) {
        float part2[32];
        tc_ld_x32(tmem_lane + (uint32_t)((tile * KH + 1) * MPAD + cc * 32), part2);
        tc_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) acc[32 * cc + e] += part2[e];
      }
    }
    tc_wait_ld();
    tc_fence_before_sync();
    __syncwarp();
    if (lane == 0) mbar_arrive(dempty);
    if constexpr (!GR) {
#pragma unroll
      for (int e = 0; e < MPAD; ++e) acc[e] *= sc_col;
    }
    if (shared_tile) {
#pragma unroll
      for (int m4 = 0; m4 < MPAD / 4; ++m4)
        red_add_f32x4(mine + m4 * kTileN, acc[4 * m4], acc[4 * m4 + 1], acc[4 * m4 + 2], acc[4 * m4 + 3]);
    } else {
#pragma unroll
      for (int m = 0; m < MPAD; ++m) put_plain(m, acc[m]);
    }

    if (shared_tile) {
      named_bar_sync(1, kDequantThreads);
      if (ctid == 0) {
        const int old = atom_add_acq_rel_gpu(&p.counters[fix], 1);
        const int is_last = (old == last_w - first_w) ? 1 : 0;
        if (is_last) p.counters[fix] = 0;
        *last_flag = is_last;
      }
      named_bar_sync(1, kDequantThreads);
      if (*last_flag != 0) {
        if (!p.swiglu) {
          // all loads of the total in flight at once: this CTA is alone on the critical path of the tile
          float4 t4[MPAD / 4];
#pragma unroll
          for (int m4 = 0; m4 < MPAD / 4; ++m4) t4[m4] = ld_cg_f4(mine + m4 * kTileN);
#pragma unroll
          for (int m4 = 0; m4 < MPAD / 4; ++m4) mine[m4 * kTileN] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
          for (int m4 = 0; m4 < MPAD / 4; ++m4) {
            const int m = 4 * m4;
            put_plain(m, t4[m4].x);
            put_plain(m + 1, t4[m4].y);
            put_plain(m + 2, t4[m4].z);
            put_plain(m + 3, t4[m4].w);
          }
        } else {
          // fused activation: 32 batch rows at a time
#pragma unroll 1
          for (int c8 = 0; c8 < MPAD / 32; ++c8) {
            float4 t4[8];
#pragma unroll
            for (int m4 = 0; m4 < 8; ++m4) t4[m4] = ld_cg_f4(mine + (c8 * 8 + m4) * kTileN);
#pragma unroll
            for (int m4 = 0; m4 < 8; ++m4) mine[(c8 * 8 + m4) * kTileN] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int m4 = 0; m4 < 8; ++m4) {
              const int m = 4 * (c8 * 8 + m4);
              put_act(m, t4[m4].x);
              put_act(m + 1, t4[m4].y);
              put_act(m + 2, t4[m4].z);
              put_act(m + 3, t4[m4].w);
            }
          }
        }
      }
      named_bar_sync(1, kDequantThreads);  // last_flag may be rewritten by the next segment
    }
    u += len;
  }
  // everybody is done with tensor memory
  tc_fence_before_sync();
  named_bar_sync(2, kDequantThreads + 32);
}

template <int MPAD, bool GR, int FMT>
cudaError_t launch_tc(const GemmParams& p, int workers, cudaStream_t stream) {
  using G = TcGeometry<MPAD, FMT>;
  auto kernel = gemm_dense_tc_kernel<MPAD, GR, FMT>;
  static bool attr_set[64] = {};
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, G::SMEM_BYTES);
    if (err != cudaSuccess) return err;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  alignas(64) CUtensorMap tmap;
  if (!make_a_tensor_map(&tmap, p.A, p.M, p.K, MPAD)) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(workers);
  cfg.blockDim = dim3(kTcThreads);
  cfg.dynamicSmemBytes = G::SMEM_BYTES;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  GemmParams q = p;
  q.cluster = 0;
  if (p.cluster) {
    // the S CTAs of a column tile as one thread-block cluster, if this device can co-schedule such a cluster
    // (all of them at once: a GPC holds only so many clusters of a size, and a second wave would cost far
    // more than the reduction through the L2 that is the alternative)
    static int max_clusters[64][9] = {};  // per device and cluster size: clusters resident at once (0 unknown, -1 none)
    const int S = (int)p.split;
    int nmax = (dev >= 0 && dev < 64) ? max_clusters[dev][S] : 0;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)S;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    if (nmax == 0) {
      cfg.numAttrs = 2;
      int n = 0;
      nmax = (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) == cudaSuccess && n > 0) ? n : -1;
      (void)cudaGetLastError();
      if (dev >= 0 && dev < 64) max_clusters[dev][S] = nmax;
    }
    const int ok = (nmax > 0 && (long long)nmax * S >= workers) ? 1 : -1;  // all clusters of THIS grid at once
    cfg.numAttrs = ok > 0 ? 2 : 1;
    q.cluster = ok > 0 ? 1u : 0u;
  }
  return cudaLaunchKernelEx(&cfg, kernel, q, tmap);
}

}  // namespace


bool tc_path_supported(int m_slab, int K, int N) {
  return m_slab >= 1 && N % kTileN == 0 && K % kTileK == 0;
}

int tc_max_rows(int K, int N, int sm_count) {
  // the device's 32-bit stripe arithmetic: slabs * tiles * k-blocks * workers stays below 2^31
  const long long per_slab = (long long)(N / kTileN) * (K / kTileK) * (sm_count < kMaxWorkers ? sm_count : kMaxWorkers);
  long long slabs = ((1ll << 31) - 1) / per_slab;
  if (slabs < 1) slabs = 1;
  if (slabs > (1 << 16)) slabs = 1 << 16;
  return (int)slabs * kTcMaxSlabM;
}

size_t tc_fixup_tiles(int M, int N, int workers) {
  // accumulation tiles of the fix-up: one per column tile up to 128 rows; above, one per (column tile, slab) or, if
  // those outnumber the workers, one per worker
  if (M <= kTcMaxSlabM) return (size_t)(N / kTileN);
  const long long vcols = (long long)(N / kTileN) * ((M + kTcMaxSlabM - 1) / kTcMaxSlabM);
  return (size_t)(vcols < workers ? vcols : workers);
}

int tc_mpad(int m_slab) { return m_slab <= 32 ? 32 : (m_slab <= 64 ? 64 : 128); }

cudaError_t launch_gemm_dense_tc(GemmParams p, int sm_count, bool sparse24, cudaStream_t stream, bool w8) {
  // stripe plan for 256-column tiles
  // above 128 rows the layer is replicated in the unit numbering, once per slab of 128 rows (Section 3.4, last
  // paragraph): one launch, its stripes running over (column tile, slab, k-block)
  p.slabs = (uint32_t)((p.M + kTcMaxSlabM - 1) / kTcMaxSlabM);
  p.ncols = (p.N / kTileN) * (int)p.slabs;
  const long long units = (long long)p.ncols * (p.K / kTileK);
  long long workers = sm_count < kMaxWorkers ? sm_count : kMaxWorkers;
  if (workers > units) workers = units;
  p.units = (uint32_t)units;
  // With up to 128 rows the epilogue of a segment (accumulators out of tensor memory, L2 reductions, arrival
  // count) takes microseconds during which the CTA converts nothing, and under even stripes most CTAs run it
  // twice.  So each tile is cut into S k-ranges instead, one per CTA (one epilogue per CTA, all CTAs alike),
  // wherever that leaves few SMs idle, or where what the idle SMs would have taken costs less than the second
  // epilogues of even stripes (about ten k-blocks of a CTA's time, six up to 32 rows: layers of 8-16 column tiles up
  // to K of about 16 K; measured on B200 over 25 shapes at 64 and 128 rows, e.g. 8192 x 2048 at 128 rows: 14.7 us with eight
  // k-ranges on 64 SMs against 20.0 us with even stripes on 148).
  p.split = 0;
  {
    long long S = workers / p.ncols;
    if (S > (long long)p.kb) S = p.kb;
    if (S > 8) S = 8;  // the CTAs of a tile form a thread-block cluster: at most the portable size
    // at least four k-blocks per CTA (2048 x 4096 at 64 rows: 7.4 us with four k-ranges, 8.9 with eight); two up
    // to 32 rows, where the epilogue is light (the same layer at 32 rows: 6.2 us with eight k-ranges, 6.5 with four)
    const long long min_kb = p.M <= 32 ? 2 : 4;
    if (S > (long long)p.kb / min_kb) S = p.kb / min_kb;
    const char* e = getenv("MARLIN_B200_TC_SPLIT");  // tuning knob: 0 forces even stripes
    bool chosen = false;
    // Above 64 rows the partial tiles are large.  Clusters of eight all fit on the device only for up to eight
    // column tiles; beyond that eight k-ranges per tile go through the L2, which costs about 5 us more than the
    // exchange inside clusters: shorter layers take four or six longer k-ranges instead (measured at 128 rows:
    // 4096 x 4096 13.3 us with four against 15.7 with eight; 8192 x 4096 17.5 with six, 18.8 with eight, 19.0 with
    // four; 14336 x 4096 23.3 with six, 23.8 with eight; 28672 x 4096 33.8 with eight, 37.1 with six).
    if (S == 8 && p.M > 64 && p.ncols > 8 && p.kb <= 120 && 4 * p.ncols * 100 >= workers * 40) {
      S = p.kb <= 56 ? 4 : 6;
      chosen = true;
    } else if (S == 8 && p.M > 32 && p.ncols > 8 && p.kb <= 32 && 4 * p.ncols * 100 >= workers * 40) {
      // 33-64 rows: the same on the shortest layers (2:4, 4096 x 4096 at 64 rows: 7.6 us with four k-ranges in
      // clusters, 8.9 with eight through the L2; the dense layer runs 10.1 and 10.0)
      S = 4;
      chosen = true;
    }
    if (e && atoi(e) >= 2 && atoi(e) <= 8 && atoi(e) <= workers / p.ncols) {  // tuning knob: 2..8 k-ranges per tile
      S = atoi(e);
      chosen = true;
    }
    // k-blocks per CTA that the idle SMs of the split cost, against even stripes on all of them
    // (up to 32 rows the second epilogue is cheaper: six k-blocks; 14336 x 2048 at 32 rows: 11.6 us even, 12.7 split)
    const bool idle_is_cheap = S >= 2 && (double)p.kb * (1.0 / (double)S - (double)p.ncols / (double)workers) <
                                             (p.M <= 32 ? 6.0 : 10.0);
    if (S >= 2 && (S * p.ncols * 100 >= workers * 85 || chosen || idle_is_cheap) && !(e && atoi(e) == 0)) {
      p.split = (uint32_t)S;
      workers = S * p.ncols;
    }
  }
  {
    const char* e = getenv("MARLIN_B200_TC_CLUSTER");  // tuning knob: 0 = reduce through the L2 instead
    // from 33 rows up: below that the partial tiles are small and the L2 path is as fast
    p.cluster = (p.split >= 2 && p.M > 32 && !(e && atoi(e) == 0)) ? 1u : 0u;
  }
  // Many more (column tile, slab) pairs than workers: stripes cut at tile boundaries leave little imbalance and need
  // no fix-up at all.
  p.whole = 0;
  if (p.split == 0 && p.ncols >= workers) {
    const long long per = (p.ncols + workers - 1) / workers;
    if (per * workers * 100 <= (long long)p.ncols * 106) p.whole = 1;
  }
  p.workers = (uint32_t)workers;
  const int mpad = tc_mpad(p.M < kTcMaxSlabM ? p.M : kTcMaxSlabM);
  if (w8) {
    if (p.grouped) {
      if (mpad == 32) return launch_tc<32, true, kFmtDense8>(p, (int)workers, stream);
      if (mpad == 64) return launch_tc<64, true, kFmtDense8>(p, (int)workers, stream);
      return launch_tc<128, true, kFmtDense8>(p, (int)workers, stream);
    }
    if (mpad == 32) return launch_tc<32, false, kFmtDense8>(p, (int)workers, stream);
    if (mpad == 64) return launch_tc<64, false, kFmtDense8>(p, (int)workers, stream);
    return launch_tc<128, false, kFmtDense8>(p, (int)workers, stream);
  }
  if (sparse24) {
    if (p.grouped) {
      if (mpad == 32) return launch_tc<32, true, true>(p, (int)workers, stream);
      if (mpad == 64) return launch_tc<64, true, true>(p, (int)workers, stream);
      return launch_tc<128, true, true>(p, (int)workers, stream);
    }
    if (mpad == 32) return launch_tc<32, false, true>(p, (int)workers, stream);
    if (mpad == 64) return launch_tc<64, false, true>(p, (int)workers, stream);
    return launch_tc<128, false, true>(p, (int)workers, stream);
  }
  if (p.grouped) {
    if (mpad == 32) return launch_tc<32, true, false>(p, (int)workers, stream);
    if (mpad == 64) return launch_tc<64, true, false>(p, (int)workers, stream);
    return launch_tc<128, true, false>(p, (int)workers, stream);
  }
  if (mpad == 32) return launch_tc<32, false, false>(p, (int)workers, stream);
  if (mpad == 64) return launch_tc<64, false, false>(p, (int)workers, stream);
  return launch_tc<128, false, false>(p, (int)workers, stream);
}

}  // namespace marlin_b200
