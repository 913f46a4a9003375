// Dense W4A16 layer for sm_100a, batch sizes 1..64 per launch, 128-column tiles: tcgen05 tensor cores with the
// WEIGHTS as the A operand in tensor memory and the group scales applied to the fp32 accumulators ("deferred"
// scaling).  It serves the layers whose N is a multiple of 128 but not of 256 at batch sizes above 16 (which the
// 256-column tcgen05 kernel cannot take and the warp-level kernel would need several launches for); on the
// shapes those two kernels serve it is the slower one (measured), because its per-k-block chain conversion ->
// tensor-memory store -> MMA -> accumulator read-back is latency-bound with the operand slots and accumulators
// that fit in the 512 columns of tensor memory.
//
// The product is computed transposed, as the paper does for its sparse kernel (Section 4: C = (B^T A^T)^T):
// per 128-column tile of W and 128-row k-block
//     D[128 channels x MPAD batch rows] = W_t^T[128 x 128] . A^T[128 x MPAD]        (eight UMMAs of K = 16)
// into an accumulator of its own in tensor memory, which a drain warp reads back, multiplies by the k-block's
// group scale s[g, n] (one scalar per thread: thread = output channel) and adds to fp32 registers.  So the
// weights go through the tensor core unscaled, as small integers (Section 3.4 "Groups and Instruction
// Ordering" multiplies them in fp16 in the loop: four more ALU instructions per eight weights and one more
// rounding).  Up to 32 rows the codes even keep the offset of the exponent trick (1024 + q, 64 + q: five ALU
// instructions per eight weights instead of nine, Section 3.4 "Dequantization and Tensor Cores") and the drain
// takes corr[m] = sum_k a[m][k] * (1032 or 72) off every accumulator; the MMA warps compute corr with the
// warp-level MMA from the activation tile.
//
// One CTA per SM, warp-specialised, 768 threads:
//   warps 0..3    drain / epilogue.  Warp q owns TMEM lanes 32q..32q+31 = 32 output channels.  64 accumulator
//                 columns (4, 2 or 1 k-blocks) at a time: wait for the MMAs' commits, tcgen05.ld, release the
//                 accumulators and stages, out[m] += s * (acc[m] - corr[m]).  At the end of a column segment:
//                 fix-up across the CTAs that share the tile, fp32 -> fp16, store C.  The scales come straight
//                 from global memory, fetched sixteen k-blocks ahead.
//   warps 4..15   three dequantiser sets of four warps; set j converts the k-blocks it = j, j + 3, ... of the
//                 CTA, so the sets are in different phases of their work.  Thread = one output channel: four
//                 16-byte shared loads give its 128 codes of the k-block, two tcgen05.st put the 128 fp16 values
//                 into one of the A-operand slots.
//   warps 16, 17  producers: per k-block one 8 KB bulk copy of packed weights (L2 evict-first) and one TMA
//                 tensor tile of the activations (3-D box: both 64-wide halves, 128-byte swizzle = the
//                 canonical K-major UMMA layout; rows >= M zero-filled), into a ring of stages.  The weights
//                 of the first pass over the ring are requested before the programmatic dependency wait
//                 (Section 3.4 "Memory Load Pipelining", across the kernel boundary).
//   warps 18..23  MMA issuers, k-blocks round-robin (issuing a tcgen05.mma occupies its thread for longer
//                 than a small-N product takes to execute); one tcgen05.commit per k-block tells the drain
//                 that the accumulator is complete and the dequantisers that the A slot is free; the drain's
//                 release tells the producers that the stage is free.  Warp 18 owns the TMEM allocation.
//
// Partition (Section 3.4 "Striped Partitioning"): the (128-column tile, k-block) units are numbered tile by
// tile and cut into `workers` even stripes (floor/ceil balanced), so every SM streams the same number of
// bytes.  Fix-up of a tile shared by several CTAs: every contributor writes its fp32 partial tile to a slot of
// the workspace and bumps the tile's arrival counter (acq_rel); whoever arrives last adds all partials in
// worker order (the same order whoever is last: results are reproducible bit for bit) and stores C.  Nobody
// spins on another CTA.  Every mbarrier wait is bounded (device_utils.cuh).
#include <stdlib.h>

#include "device_utils.cuh"
#include "marlin_internal.cuh"
#include "tc_utils.cuh"

namespace marlin_b200 {
namespace {

// ---------------------------------------------------------------------------------------------
// geometry
// ---------------------------------------------------------------------------------------------
constexpr int kTdTileN = 128;           // columns of W per CTA tile = TMEM lanes = M of the UMMA
constexpr int kTdSets = 3;              // dequantiser sets
constexpr int kTdDrainWarps = 4;
constexpr int kTdDequantWarp0 = kTdDrainWarps;
constexpr int kTdProducerWarp0 = kTdDequantWarp0 + 4 * kTdSets;   // 16
constexpr int kTdProducers = 2;
constexpr int kTdMmaWarp0 = kTdProducerWarp0 + kTdProducers;      // 18
constexpr int kTdMmaWarps = 6;
constexpr int kTdThreads = (kTdMmaWarp0 + kTdMmaWarps) * 32;      // 768
constexpr int kTdDrainThreads = kTdDrainWarps * 32;
constexpr int kTdMaxStages = 32;
constexpr int kTdTmemCols = 512;
constexpr int kTdAuxRegs = 40;          // producers and MMA issuers
// Register re-allocation (setmaxnreg) moves registers inside the pool the CTA was launched with: 768 threads
// x 80 registers.  What the warpgroups hold afterwards must not exceed that pool, or the increase never returns.
constexpr int kTdLaunchRegs = 80;       // 65536 / 768, rounded down to a multiple of 8: what ptxas gives the kernel
constexpr int kTdDequantRegs = 88;
constexpr int kTdDrainRegs = 136;
static_assert(12 * 32 * kTdDequantRegs + 4 * 32 * kTdDrainRegs + 8 * 32 * kTdAuxRegs <= kTdThreads * kTdLaunchRegs,
              "setmaxnreg budget exceeds the registers the CTA is launched with");

template <int MPAD>
struct TdGeometry {
  static constexpr int A_HALF_BYTES = MPAD * 128;               // MPAD rows x 64 fp16
  static constexpr int A_BYTES = 2 * A_HALF_BYTES;
  static constexpr int W_BYTES = 2 * kChunkBytes;               // 128 columns x 128 rows of codes
  static constexpr int STAGE_BYTES = A_BYTES + W_BYTES;         // multiple of 1024
  // Up to 32 rows the codes are converted without the subtraction of the bias trick (1024 + q, 64 + q) and the
  // drain takes sum_k a[m][k] * (1032 or 72) off each accumulator; the MMA warps compute that correction.
  static constexpr bool BIASED = MPAD <= 32;
  static constexpr int CORR_RING = 32;                          // k-blocks whose corrections are kept
  static constexpr int CORR_BYTES = BIASED ? CORR_RING * MPAD * 4 : 0;
  // barriers and flags (2048), sixteen rows of parked scales (4096), corrections
  static constexpr int BAR_BYTES = 2048 + 16 * kTdTileN * 2 + CORR_BYTES;
  static constexpr int ALIGN_SLACK = 1024;
  static constexpr int STAGES_FIT = (kSmemBudget - ALIGN_SLACK - BAR_BYTES) / STAGE_BYTES;
  static constexpr int STAGES = STAGES_FIT > kTdMaxStages ? kTdMaxStages : STAGES_FIT;
  static constexpr int FIXED_BYTES = BAR_BYTES;
  static constexpr int SMEM_BYTES = FIXED_BYTES + ALIGN_SLACK + STAGES * STAGE_BYTES;
  // tensor memory: four A-operand slots of 64 columns (128 rows of k, two per column) in the upper half,
  // accumulators of MPAD columns from column 0
  static constexpr int SLOTS = MPAD == 16 ? 5 : 4;
  static constexpr int A_COL0 = kTdTmemCols - SLOTS * 64;
  static constexpr int SETS = A_COL0 / MPAD > 12 ? 12 : A_COL0 / MPAD;
  // A waiter must see a barrier's phase before the barrier completes the phase after next.  The chains
  // producer -> dequantiser -> MMA -> drain -> producer keep every waiter within one ring pass of the event it
  // waits for as long as the slots and accumulators in flight fit inside the ring.
  static_assert(SLOTS + SETS <= STAGES, "ring too short for the operand slots and accumulators in flight");
  static_assert(STAGES >= kTdProducers && STAGES >= kTdSets && STAGES >= kTdMmaWarps, "ring too short");
  static_assert(SMEM_BYTES <= kSmemBudget, "shared memory");
  static_assert(STAGE_BYTES % 1024 == 0, "swizzled tiles need 1024-byte alignment");
  static_assert(SETS * MPAD <= A_COL0, "tensor memory");
  static_assert(CORR_RING >= STAGES && CORR_RING >= 2 * SETS + 8, "correction ring too short");
};

// ---------------------------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------------------------
template <int MPAD>
__global__ void __launch_bounds__(kTdThreads, 1)
gemm_tcd_kernel(const GemmParams p, const __grid_constant__ CUtensorMap tmap_a) {
  using G = TdGeometry<MPAD>;
  constexpr int NST = G::STAGES;
  constexpr int NSL = G::SLOTS;
  constexpr int NSE = G::SETS;
  extern __shared__ __align__(128) uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem);          // [32] weights and scales of a stage have landed
  uint64_t* xfull = reinterpret_cast<uint64_t*>(smem + 256);   // [32] activation tile of a stage has landed
  uint64_t* mdone = reinterpret_cast<uint64_t*>(smem + 512);   // [32] the MMAs of a stage have completed
  uint64_t* sfree = reinterpret_cast<uint64_t*>(smem + 768);   // [32] the drain is done with a stage
  uint64_t* afull = reinterpret_cast<uint64_t*>(smem + 1024);  // [4]  A-operand slot written
  uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(smem + 1088);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + 1092);
  volatile int* last_flag = reinterpret_cast<volatile int*>(smem + 1096);
  uint64_t* cfull = reinterpret_cast<uint64_t*>(smem + 1280);  // [32] correction of a k-block written
  uint16_t* sc_sm = reinterpret_cast<uint16_t*>(smem + 2048);  // [16][128] scales of the next k-blocks (drain warps)
  float* corr_sm = reinterpret_cast<float*>(smem + 2048 + 16 * kTdTileN * 2);  // [32][MPAD]
  uint8_t* stage0 = smem + G::FIXED_BYTES;
  const uint32_t stage0_s = smem_u32(stage0);

  // the warp index, broadcast from lane 0 so that the compiler knows it is the same in all lanes (every role branch
  // and loop bound below depends on it: otherwise each warp-wide instruction gets a divergence check)
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
  const int lane = threadIdx.x & 31;
  const uint32_t worker = blockIdx.x;
  const uint32_t U = p.units, P = p.workers, KB = p.kb;
  const uint32_t u0 = stripe_begin32(worker, U, P);
  const uint32_t u1 = stripe_begin32(worker + 1, U, P);
  const uint32_t n_it = u1 - u0;  // k-blocks (= pipeline stages) of this CTA

  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    for (int s = 0; s < NST; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&xfull[s], 1);
      mbar_init(&mdone[s], 1);
      mbar_init(&sfree[s], kTdDrainWarps);
    }
    for (int a = 0; a < NSL; ++a) mbar_init(&afull[a], 4);  // afull[8] at most
    if constexpr (G::BIASED)
      for (int c = 0; c < G::CORR_RING; ++c) mbar_init(&cfull[c], 1);
    *abort_flag = 0;
    *last_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kTdMmaWarp0) {
    tmem_alloc(tmem_base_slot, kTdTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_base_slot;

  if (warp >= kTdProducerWarp0) {
    setmaxnreg_dec<kTdAuxRegs>();
    if (warp < kTdProducerWarp0 + kTdProducers) {
      // ------------------------------- producers --------------------------------------------
      const uint32_t pw = (uint32_t)(warp - kTdProducerWarp0);
      if (lane == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_a) : "memory");
      const uint64_t pol_w = policy_evict_first();
      const uint64_t pol_a = policy_evict_last();
      const uint32_t nb64 = (uint32_t)p.N / kChunkN;
      // weights of (tile, kb): the two 64-column chunks of the tile are adjacent in the packed buffer
      // (super-columns of four chunks, k-blocks one after the other inside a super-column)
      auto weight_src = [&](uint32_t tile, uint32_t kb) -> const uint8_t* {
        const uint32_t nb = tile * 2u;
        const uint32_t sc = nb >> 2, cs = min(4u, nb64 - 4u * sc);
        return p.wq + ((size_t)sc * 4u * KB + (size_t)kb * cs + (nb & 3u)) * (size_t)kChunkBytes;
      };
      // first pass over the ring: weights before the dependency wait, activations after it
      uint32_t it = pw;
      if (lane == 0) {
        for (; it < n_it && it < (uint32_t)NST; it += kTdProducers) {
          const uint32_t u = u0 + it, tile = u / KB, kb = u - tile * KB;
          mbar_expect_tx(&full[it], G::W_BYTES);
          bulk_g2s(stage0 + (size_t)it * G::STAGE_BYTES + G::A_BYTES, weight_src(tile, kb), G::W_BYTES, &full[it], pol_w);
        }
      }
      __syncwarp();
      pdl_wait_prior_grids();
      if (lane == 0) {
        for (it = pw; it < n_it && it < (uint32_t)NST; it += kTdProducers) {
          const uint32_t kb = (u0 + it) % KB;
          mbar_expect_tx(&xfull[it], G::A_BYTES);
          tma_load_3d(stage0 + (size_t)it * G::STAGE_BYTES, &tmap_a, 0, 0, (int)(kb * 2u), &xfull[it], pol_a);
        }
      }
      __syncwarp();
      it = pw + ((min(n_it, (uint32_t)NST) + kTdProducers - 1u - pw) / kTdProducers) * kTdProducers;
      // steady state: a stage is refilled when the drain is done with the k-block that used it (which implies
      // that its codes were converted and its MMAs have completed)
      for (; it < n_it; it += kTdProducers) {
        const uint32_t u = u0 + it, tile = u / KB, kb = u - tile * KB;
        const uint32_t s = it % NST;
        mbar_wait<100>(&sfree[s], ((it / NST) & 1u) ^ 1u, abort_flag, p.status);
        uint8_t* st = stage0 + (size_t)s * G::STAGE_BYTES;
        if (lane == 0) {
          mbar_expect_tx(&full[s], G::W_BYTES);
          bulk_g2s(st + G::A_BYTES, weight_src(tile, kb), G::W_BYTES, &full[s], pol_w);
          mbar_expect_tx(&xfull[s], G::A_BYTES);
          tma_load_3d(st, &tmap_a, 0, 0, (int)(kb * 2u), &xfull[s], pol_a);
        }
        __syncwarp();
      }
    } else if (warp >= kTdMmaWarp0) {
      // ------------------------------- MMA issuers --------------------------------------------
      constexpr uint32_t idesc = instr_desc_f16(128, MPAD);
      const uint32_t mw = (uint32_t)(warp - kTdMmaWarp0);
      for (uint32_t it = mw; it < n_it; it += kTdMmaWarps) {
        const uint32_t s = it % NST, slot = it % NSL, set = it % NSE;
        mbar_wait(&xfull[s], (it / NST) & 1u, abort_flag, p.status);
        if constexpr (G::BIASED) {
          // correction of this k-block: corr[m] = sum_k a[m][k] * (1032 where k % 4 < 2, else 72), with the warp-level
          // MMA (activations as the 16 x 16 operand from the swizzled tile, the constants as the 16 x 8 one)
          const uint32_t a_s = stage0_s + s * G::STAGE_BYTES;
          const uint32_t lrow = ((uint32_t)lane & 7u) + (((uint32_t)lane >> 3) & 1u) * 8u;
          const uint32_t bk = ((uint32_t)lane & 1u) ? kBiasHi : kBiasLo;
#pragma unroll
          for (int blk = 0; blk < MPAD / 16; ++blk) {
            float d[4] = {0.f, 0.f, 0.f, 0.f};
            const uint32_t row = lrow + 16u * blk;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              const uint32_t chunk = 2u * (ks & 3) + ((uint32_t)lane >> 4);
              const uint32_t addr = a_s + (ks >> 2) * G::A_HALF_BYTES + row * 128u + ((chunk ^ (row & 7u)) << 4);
              uint32_t a[4];
              ldmatrix_x4(addr, a);
              mma_16816(d, a, bk, bk);
            }
            if ((lane & 3) == 0) {
              float* dst = corr_sm + (it & (G::CORR_RING - 1)) * MPAD + 16 * blk + (lane >> 2);
              dst[0] = d[0];
              dst[8] = d[2];
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(&cfull[it & (G::CORR_RING - 1)]);
        }
        if (it >= (uint32_t)NSL) {
          // A parity wait only tells the phase before the current one from the current one: before asking for
          // the slot's next filling, make sure that its previous one (k-block it - NSL, issued by another warp)
          // has been consumed, or the wait would fall through on the filling before that.
          const uint32_t jt = it - NSL;
          mbar_wait(&mdone[jt % NST], (jt / NST) & 1u, abort_flag, p.status);
        }
        mbar_wait(&afull[slot], (it / NSL) & 1u, abort_flag, p.status);
        if (it >= (uint32_t)NSE) {
          // the accumulator was last used by k-block it - NSE: the drain must have read it
          const uint32_t jt = it - NSE;
          mbar_wait(&sfree[jt % NST], (jt / NST) & 1u, abort_flag, p.status);
        }
        tc_fence_after_sync();
        if (lane == 0) {
          const uint64_t desc0 = smem_desc_k_sw128(stage0_s + s * G::STAGE_BYTES);
          const uint32_t a_tmem = tmem_base + (uint32_t)(G::A_COL0 + slot * 64);
          const uint32_t d_tmem = tmem_base + set * MPAD;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const uint64_t bdesc = desc0 + (uint64_t)(((ks >> 2) * G::A_HALF_BYTES + (ks & 3) * 32) >> 4);
            tc_mma_ts(d_tmem, a_tmem + ks * 8, bdesc, idesc, ks == 0 ? 0u : 1u);
          }
          tc_commit(&mdone[s]);
        }
        __syncwarp();
      }
    }
  } else if (warp >= kTdDequantWarp0) {
    // --------------------------------- dequantisers -------------------------------------------
    setmaxnreg_inc<kTdDequantRegs>();
    const uint32_t set = (uint32_t)(warp - kTdDequantWarp0) >> 2;
    const uint32_t q = (uint32_t)warp & 3u;              // TMEM lane quarter this warp may access
    const uint32_t n128 = q * 32u + (uint32_t)lane;      // column of the thread inside the tile
    // the thread's 128 codes of a k-block are 64 consecutive bytes: chunk n / 64, then 64 bytes per column
    const uint32_t vec_off = (n128 >> 6) * kChunkBytes + (n128 & 63u) * 64u;
    const uint32_t tmem_lane = tmem_base + ((q * 32u) << 16);
    for (uint32_t it = set; it < n_it; it += kTdSets) {
      const uint32_t s = it % NST, slot = it % NSL;
      mbar_wait(&full[s], (it / NST) & 1u, abort_flag, p.status);
      const uint32_t wbase = stage0_s + s * G::STAGE_BYTES + G::A_BYTES + vec_off;
      uint4 v[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) v[c] = lds128(wbase + (uint32_t)(((c + ((n128 & 7u) >> 1)) & 3u) * 16u));  // slot (c + g/2) % 4
      if (it >= (uint32_t)NSL) {
        // the slot was last read by the MMAs of k-block it - NSL
        const uint32_t jt = it - NSL;
        mbar_wait(&mdone[jt % NST], (jt / NST) & 1u, abort_flag, p.status);
      }
      tc_fence_after_sync();
      const uint32_t a_col = tmem_lane + (uint32_t)(G::A_COL0 + slot * 64);
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        // 64 rows of k = 32 columns of the slot, written with one store
        uint32_t r[32];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const uint32_t w0 = hh == 0 ? v[c].x : v[c].z, w1 = hh == 0 ? v[c].y : v[c].w;
          uint32_t lo[4], hi[4];
          if constexpr (G::BIASED) {
            dequant8_biased(w0, lo);  // rows 64hh + 16c + 0..7, as 1024 + q / 64 + q
            dequant8_biased(w1, hi);  // rows 64hh + 16c + 8..15
          } else {
            dequant8(w0, lo);
            dequant8(w1, hi);
          }
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            r[8 * c + e] = lo[e];
            r[8 * c + 4 + e] = hi[e];
          }
        }
        tc_st_x32(a_col + (uint32_t)(32 * hh), r);  // column = row / 2
      }
      tc_wait_st();
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&afull[slot]);
    }
  } else {
    // --------------------------------- drain / epilogue ----------------------------------------
    setmaxnreg_inc<kTdDrainRegs>();
    const uint32_t q = (uint32_t)warp;
    const uint32_t n128 = q * 32u + (uint32_t)lane;
    const uint32_t n64 = n128 & 63u;
    // position of this column's scale inside the tile's 128 packed scales (runs of 64: 8g + 2j + b)
    const uint32_t spos = (n128 & 64u) + 8u * (n64 & 7u) + 2u * (n64 >> 4) + ((n64 >> 3) & 1u);
    const uint32_t tmem_lane = tmem_base + ((q * 32u) << 16);
    const int tid = (int)threadIdx.x;  // 0..127
    float out[MPAD];
#pragma unroll
    for (int m = 0; m < MPAD; ++m) out[m] = 0.f;
    bool waited_for_prior_grid = false;
    // 64 accumulator columns are read at a time: the k-blocks it = base .. base + DR - 1 of the CTA
    constexpr uint32_t DR = 64 / MPAD;
    static_assert(NSE % DR == 0 && 8 % DR == 0, "drain batches must tile the accumulator ring");
    // The thread's scales, one scalar per k-block, come straight from global memory.  They are fetched sixteen
    // to eight k-blocks ahead, eight at a time, and parked in a column of shared memory that only this thread
    // touches, so that no load latency is ever waited for in the loop.  (pt, pk) = the k-block to fetch next.
    const uint16_t* sq16 = reinterpret_cast<const uint16_t*>(p.sq);
    const uint32_t tile0 = u0 / KB;
    uint32_t pt = tile0, pk = u0 - tile0 * KB, pn = 0;
    auto next_scale = [&]() -> uint16_t {
      uint16_t v = 0;
      if (pn < n_it) {
        const uint32_t gi = !p.grouped ? 0u : (p.group_shift >= 0 ? (pk >> p.group_shift) : (pk / (uint32_t)p.kb_per_group));
        v = __ldg(sq16 + (size_t)gi * p.N + (size_t)pt * kTdTileN + spos);
      }
      ++pn;
      if (++pk == KB) { pk = 0; ++pt; }
      return v;
    };
    {
      uint16_t first[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) first[j] = next_scale();
#pragma unroll
      for (int j = 0; j < 16; ++j) sc_sm[j * kTdTileN + n128] = first[j];
    }
    uint16_t nxt[8];
    uint32_t tile = tile0, kb = u0 - tile0 * KB;  // the k-block whose product is added next
    uint32_t s = 0, sph = 0;                      // ring position and phase of k-block `base`
    for (uint32_t base = 0; base < n_it; base += DR) {
      if ((base & 7u) == 0) {
#pragma unroll
        for (int j = 0; j < 8; ++j) nxt[j] = next_scale();
      }
      const uint32_t nb = min(DR, n_it - base);
      {
        uint32_t s2 = s, ph2 = sph;
#pragma unroll
        for (uint32_t j = 0; j < DR; ++j) {
          if (j < nb) {
            mbar_wait(&mdone[s2], ph2, abort_flag, p.status);
            if constexpr (G::BIASED)
              mbar_wait(&cfull[(base + j) & (G::CORR_RING - 1)], ((base + j) / G::CORR_RING) & 1u, abort_flag, p.status);
          }
          if (++s2 == (uint32_t)NST) { s2 = 0; ph2 ^= 1u; }
        }
      }
      tc_fence_after_sync();
      float acc[64];
      {
        const uint32_t col = tmem_lane + (base % (uint32_t)NSE) * MPAD;
        // two loads of 32 columns (a single 64-column load needs more registers than a 768-thread CTA has per thread)
        float lo[32], hi[32];
        tc_ld_x32(col, lo);
        tc_ld_x32(col + 32u, hi);
#pragma unroll
        for (int e = 0; e < 32; ++e) { acc[e] = lo[e]; acc[32 + e] = hi[e]; }
        tc_wait_ld();
      }
      // the accumulators are in registers: the MMAs of later k-blocks may overwrite them, the stages are free
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) {
        uint32_t s2 = s;
#pragma unroll
        for (uint32_t j = 0; j < DR; ++j) {
          if (j < nb) mbar_arrive(&sfree[s2]);
          if (++s2 == (uint32_t)NST) s2 = 0;
        }
      }
      s += nb;
      if (s >= (uint32_t)NST) { s -= NST; sph ^= 1u; }
      float scj[DR];
#pragma unroll
      for (uint32_t j = 0; j < DR; ++j) scj[j] = __half2float(__ushort_as_half(sc_sm[((base + j) & 15u) * kTdTileN + n128]));

      // add the batch to `out`, segment by segment (a segment = this CTA's k-blocks of one column tile)
      uint32_t j0 = 0;
      while (j0 < nb) {
        const uint32_t to_tile_end = KB - 1u - kb;
        const uint32_t e = j0 + min(nb - 1u - j0, to_tile_end);  // last k-block of the batch that belongs to this segment
        const bool seg_end = (e - j0 == to_tile_end) || (base + e + 1u == n_it);
#pragma unroll
        for (uint32_t j = 0; j < DR; ++j) {
          if (j >= j0 && j <= e) {
            if constexpr (G::BIASED) {
              const float4* cr = reinterpret_cast<const float4*>(corr_sm + ((base + j) & (G::CORR_RING - 1)) * MPAD);
#pragma unroll
              for (int m4 = 0; m4 < MPAD / 4; ++m4) {
                const float4 c4 = cr[m4];  // the same address in every lane: a broadcast
                out[4 * m4 + 0] = fmaf(scj[j], acc[j * MPAD + 4 * m4 + 0] - c4.x, out[4 * m4 + 0]);
                out[4 * m4 + 1] = fmaf(scj[j], acc[j * MPAD + 4 * m4 + 1] - c4.y, out[4 * m4 + 1]);
                out[4 * m4 + 2] = fmaf(scj[j], acc[j * MPAD + 4 * m4 + 2] - c4.z, out[4 * m4 + 2]);
                out[4 * m4 + 3] = fmaf(scj[j], acc[j * MPAD + 4 * m4 + 3] - c4.w, out[4 * m4 + 3]);
              }
            } else {
#pragma unroll
              for (int m = 0; m < MPAD; ++m) out[m] = fmaf(scj[j], acc[j * MPAD + m], out[m]);
            }
          }
        }
        kb += e - j0 + 1u;
        j0 = e + 1u;
        if (!seg_end) continue;
        // ---- the segment ends here: fix-up across the CTAs that share the column tile, store C ----
        if (!waited_for_prior_grid) {
          // first write to C or the workspace: the previous kernel of the stream must be done with them
          pdl_wait_prior_grids();
          waited_for_prior_grid = true;
        }
        const int first_w = (int)stripe_owner32(tile * KB, U, P);
        const int last_w = (int)stripe_owner32((tile + 1) * KB - 1, U, P);
        bool store = true;
        if (last_w > first_w) {
          const int my_slot = 2 * (int)worker + (tile != tile0 ? 1 : 0);
          float* mine = p.partials + (size_t)my_slot * p.slot_floats + n128;
#pragma unroll
          for (int m = 0; m < MPAD; ++m) mine[m * kTdTileN] = out[m];
          named_bar_sync(1, kTdDrainThreads);
          if (tid == 0) {
            const int old = atom_add_acq_rel_gpu(&p.counters[tile], 1);
            const int is_last = (old == last_w - first_w) ? 1 : 0;
            if (is_last) p.counters[tile] = 0;  // everyone has arrived: ready for the next call
            *last_flag = is_last;
          }
          named_bar_sync(1, kTdDrainThreads);
          store = *last_flag != 0;
          if (store) {
            // the last arriver adds every partial of the tile, its own included, in worker order
#pragma unroll
            for (int m = 0; m < MPAD; ++m) out[m] = 0.f;
            for (int w = first_w; w <= last_w; ++w) {
              const int slot = 2 * w + (tile != stripe_begin32((uint32_t)w, U, P) / KB ? 1 : 0);
              const float* src = p.partials + (size_t)slot * p.slot_floats + n128;
              float v[MPAD];
#pragma unroll
              for (int m = 0; m < MPAD; ++m) v[m] = __ldcg(src + m * kTdTileN);
#pragma unroll
              for (int m = 0; m < MPAD; ++m) out[m] += v[m];
            }
          }
          named_bar_sync(1, kTdDrainThreads);  // last_flag may be rewritten by the next segment
        }
        if (store) {
          uint16_t* cptr = p.C + (size_t)tile * kTdTileN + n128;
#pragma unroll
          for (int m = 0; m < MPAD; ++m)
            if (m < p.M) cptr[(size_t)m * p.N] = __half_as_ushort(__float2half_rn(out[m]));
        }
#pragma unroll
        for (int m = 0; m < MPAD; ++m) out[m] = 0.f;
        if (kb == KB) { kb = 0; ++tile; }
      }
      if (((base + DR) & 7u) == 0) {
        // the eight k-blocks whose scales sat in these rows are done: park the next eight
#pragma unroll
        for (int j = 0; j < 8; ++j) sc_sm[((base + DR + 8u + (uint32_t)j) & 15u) * kTdTileN + n128] = nxt[j];
      }
    }
  }

  if (*abort_flag) {
    // a wait gave up: copies may still be in flight towards this CTA's shared memory
    for (int x = 0; x < 1000; ++x) __nanosleep(1000);
  }
  // everybody is done with tensor memory: the owner frees it
  tc_fence_before_sync();
  __syncthreads();
  if (warp == kTdMmaWarp0) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTdTmemCols);
  }
}

template <int MPAD>
cudaError_t launch_tcd(const GemmParams& p, cudaStream_t stream) {
  using G = TdGeometry<MPAD>;
  auto kernel = gemm_tcd_kernel<MPAD>;
  static bool attr_set[64] = {};
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    // the register budget of the warpgroups assumes the launch allocation stated above
    cudaFuncAttributes fa;
    err = cudaFuncGetAttributes(&fa, kernel);
    if (err != cudaSuccess) return err;
    if (fa.numRegs < kTdLaunchRegs) return cudaErrorLaunchOutOfResources;
    err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, G::SMEM_BYTES);
    if (err != cudaSuccess) return err;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  alignas(64) CUtensorMap tmap;
  if (!make_a_tensor_map_3d(&tmap, p.A, p.M, p.K, MPAD)) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.workers);
  cfg.blockDim = dim3(kTdThreads);
  cfg.dynamicSmemBytes = G::SMEM_BYTES;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, p, tmap);
}

}  // namespace

bool tcd_path_supported(int m_slab, int K, int N) {
  return m_slab >= 1 && m_slab <= kTcdMaxSlabM && N % kTdTileN == 0 && K % kTileK == 0;
}

int tcd_mpad(int m_slab) { return m_slab <= 16 ? 16 : (m_slab <= 32 ? 32 : 64); }

size_t tcd_slot_floats(int m_slab) { return (size_t)kTdTileN * tcd_mpad(m_slab); }

cudaError_t launch_gemm_tcd(GemmParams p, int sm_count, cudaStream_t stream) {
  const long long units = (long long)(p.N / kTdTileN) * (p.K / kTileK);
  long long workers = sm_count < kMaxWorkers ? sm_count : kMaxWorkers;
  if (workers > units) workers = units;
  p.ncols = p.N / kTdTileN;
  p.units = (uint32_t)units;
  p.workers = (uint32_t)workers;
  p.split = 0;
  p.cluster = 0;
  const int mpad = tcd_mpad(p.M);
  p.slot_floats = (int)tcd_slot_floats(p.M);
  if (mpad == 16) return launch_tcd<16>(p, stream);
  if (mpad == 32) return launch_tcd<32>(p, stream);
  return launch_tcd<64>(p, stream);
}

}  // namespace marlin_b200
