// W4A16 layer for sm_100a, decode batch sizes (one launch handles up to 16 rows of A), dense and 2:4 sparse.
//
// Structure of one CTA (one per SM, 384 threads, persistent over its share of the work units):
//   warps 8..11   producers.  Per k-block ONE bulk-async copy (cp.async.bulk + mbarrier complete_tx) of
//                 the contiguous packed weights of the column tile, one of the tile's row of group scales,
//                 and one TMA tensor-tile copy per 64-wide half of the A tile (128-byte swizzle, rows beyond M
//                 zero-filled by the hardware) into a ring of shared-memory stages.  Weights carry an L2
//                 evict-first policy (each byte is read once), activations evict-last (re-read by every
//                 tile).  Issuing a bulk copy occupies a warp for a few hundred cycles whatever its size, so
//                 copies are few and large and four warps take the stages round-robin.  The weights of the
//                 first pass over the ring are requested before the programmatic dependency wait.
//   warps 0..7    consumers, arranged as SK groups of NW warps.  Stage number `it` of the CTA is
//                 consumed by group it % SK; inside a group warp wn owns 64 output columns.  A warp
//                 reads its 16-byte weight vectors, turns the 4-bit codes into fp16 with the exponent-bias
//                 trick, and feeds mma.sync.m16n8k16 with the WEIGHTS as the 16-wide operand and the batch
//                 on the 8-wide one, so that batch sizes 1..8 cost one MMA per 256 weights.
//                 Dense layers with up to 8 rows skip the subtraction of the bias trick: the weights enter the MMA as 1024 + q
//                 and 64 + q, one more MMA per 16 rows of k with a constant weight operand collects
//                 sum_k a[k] * (1032 or 72), and the difference is taken when the group closes (five ALU
//                 instructions per eight weights instead of nine).  With 9..16 rows the extra MMAs cost more
//                 than they save, and 2:4 layers cannot use the trick (the correction would depend on the
//                 metadata): both convert exactly.
//                 The group scale is not applied to the weights: each group of k accumulates into `tmp`,
//                 and `acc += s * (tmp - bias)` in fp32 when the group ends.
//   end of a column segment: the groups of the CTA add their tiles through shared memory; then the fix-up
//                 across the CTAs that share the column tile, one of three ways: through the shared memory of
//                 the first CTA of a thread-block cluster (tile-aligned partition, clusters fit in one wave);
//                 or partial tiles to the workspace in fp32 and an arrival counter (acq_rel atomic) that
//                 tells the last CTA to add them in worker order; a segment in the middle of an even stripe
//                 is handled that way by warp group 0 alone while the others go on.  Always the same order
//                 of the fp32 sum; nobody spins on another CTA.
//
// Paper correspondence (Section 3.4): weight streaming and evict-first ("Maximizing Loading
// Bandwidth"), multi-stage pipeline ("Memory Load Pipelining"), warps splitting K with a shared
// memory reduction ("Warp Layout", Algorithm 1), bit-trick dequantisation into fragment layout
// ("Dequantization and Tensor Cores"), scales ("Groups and Instruction Ordering"), stripes and the
// global reduction ("Striped Partitioning").  What differs from the paper's Ampere design is listed
// in the design document of this repository.
#include <cuda.h>
#include <stdlib.h>

#include "device_utils.cuh"
#include "marlin_internal.cuh"

namespace marlin_b200 {
namespace {


// ---------------------------------------------------------------------------------------------
// shared memory map
// ---------------------------------------------------------------------------------------------
constexpr int kBarBytes = 1024;  // full[32] at 0, empty[32] at 256, flags at 512

// Consumer warps per CTA.  Eight everywhere: a sixteen-warp variant of the one-block kernel (batch <= 8)
// raised "unspecified launch failure" on long-K layers, was no faster, and is not built.  The same goes
// for a four-block variant (32 rows of A per launch, the only one whose accumulators spilled): it raised
// that error in two of three timing runs on the 8192 x 8192 layer; batches above 16 rows go to the
// tcgen05 kernel, or through this one as slabs of 16 rows where that kernel does not apply.
constexpr int consumer_warps_for(int /*mb*/) { return 8; }
// Twelve consumer warps (three per scheduler, 152 registers each: the 8-row instances need no more; the 16-row ones
// would spill) hide more of the latency of the conversion -> MMA chains: the loop runs about 10 % faster.  The plan
// takes them where that shows in the launch time (make_dense_plan).
constexpr int kWideConsumerWarps = 12;

// FMT: 0 = dense, 1 = the 2:4 variant, 2 = dense with per-group zero points (W = (q - z) s: the zero-point row of a
// group travels with the stage behind its scale row)
constexpr int kFmtDense = 0, kFmtSparse = 1, kFmtZero = 2;
template <int MB, int NW, int CW, int FMT>
struct Geometry {
  static constexpr bool SP = FMT == kFmtSparse;
  static constexpr bool ZP = FMT == kFmtZero;
  static constexpr int SK = CW / NW;             // groups of warps that split K
  static constexpr int MPAD = MB * 8;
  static constexpr int NT = NW * kChunkN;
  static constexpr int A_HALF_BYTES = MPAD * 128;            // one 64-wide half of the A tile: MPAD rows x 128 B
  static constexpr int A_BYTES = 2 * A_HALF_BYTES;
  static constexpr int CODE_CHUNK = SP ? kSparseCodeChunkBytes : kChunkBytes;  // packed codes of one 64-column chunk
  static constexpr int META_CHUNK = SP ? kSparseMetaChunkBytes : 0;            // 2:4 position metadata of one chunk
  static constexpr int W_BYTES = NW * CODE_CHUNK;
  static constexpr int META_BYTES = NW * META_CHUNK;
  static constexpr int STAGE_BYTES = A_BYTES + W_BYTES + META_BYTES;  // multiple of 1024
  static constexpr int FRAG_F4 = MB * 4;                     // float4 accumulator registers per thread
  static constexpr int TILE_F4 = NW * FRAG_F4 * 32;          // float4s of one partial tile
  static constexpr int RED_BYTES = (SK - 1) * TILE_F4 * 16;  // parked tiles of groups 1 .. SK - 1
  static constexpr int CST_STRIDE = NT + 8;                  // halves
  static constexpr int CST_BYTES = MPAD * CST_STRIDE * 2;
  static constexpr int SC_ROW_BYTES = NT * 2;                // one row of the tile's group scales (or zero points)
  static constexpr int SC_BYTES = (ZP ? 2 : 1) * SC_ROW_BYTES;  // per stage: the scale row, then the zero-point row
  static constexpr int SC_OFF = kBarBytes + RED_BYTES + CST_BYTES;
  static constexpr int ALIGN_SLACK = 1024;                   // the stage ring is placed on a 1024-byte boundary
  // stages: what fits after the fixed areas, each stage bringing its scale row along
  static constexpr int STAGES_FIT = (kSmemBudget - ALIGN_SLACK - SC_OFF - 1023) / (STAGE_BYTES + SC_BYTES);
  static constexpr int STAGES = STAGES_FIT > kMaxStages ? kMaxStages : STAGES_FIT;
  static constexpr int FIXED_BYTES = ((SC_OFF + STAGES * SC_BYTES + 1023) / 1024) * 1024;
  // what the kernel relies on
  static_assert(CW % NW == 0 && SK >= 1, "warp groups");
  static_assert(STAGE_BYTES % 1024 == 0, "swizzled activation tiles need 1024-byte alignment");
  static_assert(FIXED_BYTES + ALIGN_SLACK + STAGES * STAGE_BYTES <= kSmemBudget, "shared memory");
  static_assert(STAGES >= SK && STAGES >= kProducerWarps, "the ring must hold one stage per group and per producer warp");
  static_assert(2 * kMaxStages * 8 <= 512 && kBarBytes >= 512 + 16, "barrier area: full[] at 0, empty[] at 256, flags at 512");
  static_assert(MPAD * NT * 4 == TILE_F4 * 16, "a partial tile is MPAD x NT floats");
  static_assert(TILE_F4 * 4 <= kWsSlotCols * kMaxSlabM, "a partial tile must fit a workspace slot");
  static_assert(CST_BYTES >= MPAD * NT * 2, "output staging tile");
};

// ---------------------------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------------------------
template <int MB, int NW, int CW, int FMT>
__global__ void __launch_bounds__((CW + 4) * 32, 1)
gemm_dense_kernel(const GemmParams p, const __grid_constant__ CUtensorMap tmap_a) {
  using G = Geometry<MB, NW, CW, FMT>;
  constexpr bool SP = G::SP;
  constexpr bool ZP = G::ZP;
  constexpr int SK = G::SK;
  constexpr int kConsumerWarps = CW;
  constexpr int kConsumerThreads = CW * 32;
  // register budget: (CW + 4) * 32 threads share 64K registers; the producer warpgroup keeps 40
  constexpr int kBaseRegs = (65536 / ((CW + 4) * 32)) / 8 * 8;
  constexpr int kConsumerRegs = (kBaseRegs + (kBaseRegs - kProducerRegs) * 4 / CW) / 8 * 8;
  extern __shared__ __align__(128) uint8_t smem_raw[];
  // 128-byte-swizzled TMA tiles need their shared address aligned to the 1024-byte swizzle period
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem);
  uint64_t* empty = reinterpret_cast<uint64_t*>(smem + 256);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + 512);
  volatile int* last_flag = abort_flag + 1;
  float4* red = reinterpret_cast<float4*>(smem + kBarBytes);
  uint16_t* cst = reinterpret_cast<uint16_t*>(smem + kBarBytes + G::RED_BYTES);
  uint8_t* sc_ring = smem + G::SC_OFF;  // [stage][NT] fp16 group scales, copied with the stage
  uint8_t* stage0 = smem + G::FIXED_BYTES;
  const uint32_t stage0_s = smem_u32(stage0);

  // the warp index, broadcast from lane 0 so that the compiler knows it is the same in all lanes (every role branch
  // and loop bound below depends on it: otherwise each warp-wide instruction gets a divergence check)
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
  const int lane = threadIdx.x & 31;
  const uint32_t worker = blockIdx.x;
  const uint32_t U = p.units, P = p.workers, KB = p.kb;
  // split > 0: one k-range of one column tile per CTA instead of an even stripe over all units
  const uint32_t u0 = p.split ? split_begin32(worker, KB, p.split) : stripe_begin32(worker, U, P);
  const uint32_t u1 = p.split ? split_begin32(worker + 1, KB, p.split) : stripe_begin32(worker + 1, U, P);
  const int nstages = p.stages;

  pdl_launch_dependents();
  if ((int)threadIdx.x < nstages) {
    mbar_init(&full[threadIdx.x], 1);
    mbar_init(&empty[threadIdx.x], NW);
  }
  if (threadIdx.x == 0) {
    *abort_flag = 0;
    last_flag[0] = 0;
    last_flag[1] = 0;
  }
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  __syncthreads();

  if (warp >= kConsumerWarps) {
    // ------------------------------- producers --------------------------------------------
    // The third warpgroup gives most of its registers to the two consumer warpgroups.  Its warps
    // take the stages round-robin: issuing a bulk or tensor copy occupies a warp for a few hundred
    // cycles whatever the size of the copy, so several warps issue in parallel.
    const int pw = warp - kConsumerWarps;
    // give the registers away first: the consumers' setmaxnreg.inc retries until they are in the pool
    setmaxnreg_dec<kProducerRegs>();
    if (lane == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_a) : "memory");
    const uint64_t pol_w = policy_evict_first();
    const uint64_t pol_a = policy_evict_last();
    // out-of-range rows of the A box count too; grouped layers bring the scale row of the k-block along
    const uint32_t tx_bytes = G::W_BYTES + G::META_BYTES + G::A_BYTES + (p.grouped ? G::SC_BYTES : 0);  // ZP layers are grouped
    auto scale_src = [&](uint32_t col, uint32_t kb) -> const uint8_t* {
      const uint32_t gi = p.group_shift >= 0 ? (kb >> p.group_shift) : (kb / (uint32_t)p.kb_per_group);
      return p.sq + ((size_t)gi * p.N + (size_t)col * G::NT) * 2;
    };
    const uint32_t nb64 = p.N / kChunkN;
    // weights of (kb, col): super-columns of four chunks, k-blocks contiguous inside a super-column
    auto chunk_index = [&](uint32_t col, uint32_t kb) -> size_t {
      const uint32_t nb = col * NW;
      const uint32_t sc = nb >> 2, cs = min(4u, nb64 - 4u * sc);
      return (size_t)sc * 4u * KB + (size_t)kb * cs + (nb & 3u);
    };
    auto weight_src = [&](uint32_t col, uint32_t kb) -> const uint8_t* {
      return p.wq + chunk_index(col, kb) * G::CODE_CHUNK;
    };
    auto meta_src = [&](uint32_t col, uint32_t kb) -> const uint8_t* {
      return p.meta + chunk_index(col, kb) * G::META_CHUNK;
    };
    // First pass over the ring: the packed weights do not depend on the previous kernel of the
    // stream, so their copies go out before the dependency wait and HBM keeps streaming across the
    // kernel boundary; the A tiles follow once the previous kernel's memory is visible.
    uint32_t u = u0 + pw;
    int s = pw;
#ifdef MARLIN_TEST_HOOKS
    const bool withhold = worker == 0 && pw == 1 && p.status[7] == kTestWithholdMagic;  // stage 1 belongs to producer 1
#else
    constexpr bool withhold = false;
#endif
    if (lane == 0) {
      for (; u < u1 && s < nstages; u += kProducerWarps, s += kProducerWarps) {
        const uint32_t col = u / KB, kb = u - col * KB;
        if (withhold && s == 1) continue;
        mbar_expect_tx(&full[s], tx_bytes);
        bulk_g2s(stage0 + (size_t)s * G::STAGE_BYTES + G::A_BYTES, weight_src(col, kb), G::W_BYTES, &full[s], pol_w);
        if constexpr (SP)
          bulk_g2s(stage0 + (size_t)s * G::STAGE_BYTES + G::A_BYTES + G::W_BYTES, meta_src(col, kb), G::META_BYTES,
                   &full[s], pol_w);
        if (p.grouped) bulk_g2s(sc_ring + (size_t)s * G::SC_BYTES, scale_src(col, kb), G::SC_ROW_BYTES, &full[s], pol_w);
        if constexpr (ZP)
          bulk_g2s(sc_ring + (size_t)s * G::SC_BYTES + G::SC_ROW_BYTES, p.zq + (scale_src(col, kb) - p.sq), G::SC_ROW_BYTES,
                   &full[s], pol_w);
      }
    }
    __syncwarp();
    pdl_wait_prior_grids();
    u = u0 + pw;
    s = pw;
    for (; u < u1 && s < nstages; u += kProducerWarps, s += kProducerWarps) {
      const uint32_t col = u / KB, kb = u - col * KB;
      if (withhold && s == 1) continue;
      if (lane < 2)
        tma_load_2d(stage0 + (size_t)s * G::STAGE_BYTES + lane * G::A_HALF_BYTES, &tmap_a,
                    (int)(kb * kTileK + lane * 64), 0, &full[s], pol_a);
    }
    // steady state: a stage is refilled as soon as its consumers have released it
    uint32_t ph = 1;
    s -= nstages;
    for (; u < u1; u += kProducerWarps) {
      const uint32_t col = u / KB, kb = u - col * KB;
      const uint8_t* wsrc = weight_src(col, kb);
      mbar_wait<200>(&empty[s], ph ^ 1u, abort_flag, p.status);
      uint8_t* st = stage0 + (size_t)s * G::STAGE_BYTES;
      if (lane == 0) {
        mbar_expect_tx(&full[s], tx_bytes);
        bulk_g2s(st + G::A_BYTES, wsrc, G::W_BYTES, &full[s], pol_w);
        if constexpr (SP) bulk_g2s(st + G::A_BYTES + G::W_BYTES, meta_src(col, kb), G::META_BYTES, &full[s], pol_w);
        if (p.grouped) bulk_g2s(sc_ring + (size_t)s * G::SC_BYTES, scale_src(col, kb), G::SC_ROW_BYTES, &full[s], pol_w);
        if constexpr (ZP)
          bulk_g2s(sc_ring + (size_t)s * G::SC_BYTES + G::SC_ROW_BYTES, p.zq + (scale_src(col, kb) - p.sq), G::SC_ROW_BYTES,
                   &full[s], pol_w);
      }
      __syncwarp();
      if (lane < 2) tma_load_2d(st + lane * G::A_HALF_BYTES, &tmap_a, (int)(kb * kTileK + lane * 64), 0, &full[s], pol_a);
      s += kProducerWarps;
      if (s >= nstages) { s -= nstages; ph ^= 1u; }
    }
    if (*abort_flag) {
      // give copies that may still be in flight time to land before the CTA's shared memory goes away
      for (int x = 0; x < 1000; ++x) __nanosleep(1000);
    }
    if (p.cluster) {
      // every thread of every CTA of the cluster takes part in the barriers of the fix-up
      if (p.cluster == 1) cluster_sync_all();
      cluster_sync_all();
    }
    return;
  }

  // --------------------------------- consumers ----------------------------------------------
  setmaxnreg_inc<kConsumerRegs>();
  // From here on this kernel writes C and the workspace, which the previous kernel of the stream
  // may still be using: wait until it has finished and its memory is visible.
  pdl_wait_prior_grids();
  const int grp = warp / NW;
  const int wn = warp % NW;
  const int g = lane >> 2, c = lane & 3;
  const int ctid = threadIdx.x;  // 0..255 among consumers
  int s = grp;                   // this group's first stage is iteration `grp` of the CTA
  uint32_t ph = 0;
  // byte offsets of this thread's two 16-byte A vectors inside a 128-byte row (128B swizzle: chunk ^ row%8)
  const uint32_t a_off0 = (uint32_t)g * 128u + (uint32_t)(((2 * c) ^ g) * 16);
  const uint32_t a_off1 = (uint32_t)g * 128u + (uint32_t)(((2 * c + 1) ^ g) * 16);

  float acc[4 * MB][4];
  float tmp[4 * MB][4];
  // Dense layers, one block of eight batch rows: the weights enter the MMAs as 1024 + q and 64 + q
  // (dequant8_biased), and bias[mb] collects sum_k a[k] * (1032 or 72) of the open group with one more MMA per
  // 16 rows of k whose weight operand is that constant: the same number in every output channel, taken off
  // when the group closes.  With two blocks the MMAs are the larger part of the time and the extra ones cost
  // more than the shorter conversion saves (measured), so those kernels convert exactly, as the 2:4 path must.
  constexpr bool kBiased = !SP && MB == 1;
  float bias[kBiased ? MB : 1][4];
  uint4 cur_raw = make_uint4(0, 0, 0, 0);  // 8 fp16 scales of the open group: columns 16j+g and 16j+8+g, j = 0..3
  // Zero points: sum_k a (q - z) = sum_k a (q - 8) + (8 - z) sum_k a.  asum[mb] collects sum_k a[k][m] of the open group
  // with one more MMA per 16 rows of k whose weight operand is all ones (the same number in every output channel),
  // and the group closes with acc += s (tmp + (8 - z) asum).
  uint4 cur_z = make_uint4(0, 0, 0, 0);    // the 8 zero points of the open group, as fp16 values, same order
  float asum[ZP ? MB : 1][4];

  auto close_group = [&]() {
    const __half2* h2 = reinterpret_cast<const __half2*>(&cur_raw);
    const __half2* z2 = reinterpret_cast<const __half2*>(&cur_z);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 sc2 = __half22float2(h2[j]);
#pragma unroll
      for (int mb = 0; mb < MB; ++mb) {
        const int r = j * MB + mb;
        if constexpr (ZP) {
          const float2 zf = __half22float2(z2[j]);
          tmp[r][0] += (8.f - zf.x) * asum[mb][0];
          tmp[r][1] += (8.f - zf.x) * asum[mb][1];
          tmp[r][2] += (8.f - zf.y) * asum[mb][2];
          tmp[r][3] += (8.f - zf.y) * asum[mb][3];
        }
        if constexpr (!kBiased) {
          acc[r][0] += sc2.x * tmp[r][0];
          acc[r][1] += sc2.x * tmp[r][1];
          acc[r][2] += sc2.y * tmp[r][2];
          acc[r][3] += sc2.y * tmp[r][3];
        } else {
          acc[r][0] += sc2.x * (tmp[r][0] - bias[mb][0]);
          acc[r][1] += sc2.x * (tmp[r][1] - bias[mb][1]);
          acc[r][2] += sc2.y * (tmp[r][2] - bias[mb][2]);
          acc[r][3] += sc2.y * (tmp[r][3] - bias[mb][3]);
        }
        tmp[r][0] = tmp[r][1] = tmp[r][2] = tmp[r][3] = 0.f;
      }
    }
    if constexpr (kBiased) {
#pragma unroll
      for (int mb = 0; mb < MB; ++mb) bias[mb][0] = bias[mb][1] = bias[mb][2] = bias[mb][3] = 0.f;
    }
    if constexpr (ZP) {
#pragma unroll
      for (int mb = 0; mb < MB; ++mb) asum[mb][0] = asum[mb][1] = asum[mb][2] = asum[mb][3] = 0.f;
    }
  };

  // The finished fp16 tile goes from its staging buffer to C with 16-byte row stores, by the first `nthr` consumer
  // threads.  With the fused activation the tile's 16-column blocks hold eight gate and eight up channels: one
  // 16-byte piece of silu(gate) * up per pair of pieces, into a C of half the width.
  auto store_tile = [&](uint32_t col, int nthr) {
    if (!p.swiglu) {
      constexpr int CH = NW * 8;  // 16-byte pieces per row of the tile
      for (int x = ctid; x < p.M * CH; x += nthr) {
        const int m = x / CH, ch = x % CH;
        const uint4 v = *reinterpret_cast<const uint4*>(cst + m * G::CST_STRIDE + ch * 8);
        *reinterpret_cast<uint4*>(p.C + (size_t)m * p.N + (size_t)col * G::NT + ch * 8) = v;
      }
    } else {
      constexpr int CH2 = NW * 4;
      const int ldc = p.N / 2;
      for (int x = ctid; x < p.M * CH2; x += nthr) {
        const int m = x / CH2, c2 = x % CH2;
        const uint4 gate = *reinterpret_cast<const uint4*>(cst + m * G::CST_STRIDE + (2 * c2) * 8);
        const uint4 up = *reinterpret_cast<const uint4*>(cst + m * G::CST_STRIDE + (2 * c2 + 1) * 8);
        *reinterpret_cast<uint4*>(p.C + (size_t)m * ldc + (size_t)col * (G::NT / 2) + c2 * 8) = swiglu8(gate, up);
      }
    }
  };

  uint32_t u = u0;
  uint32_t it0 = 0;  // iteration index of the segment's first unit, relative to u0
  while (u < u1) {
    const uint32_t col = u / KB;
    const uint32_t kb0 = u % KB;
    const uint32_t len = min(KB - kb0, u1 - u);
    const uint16_t* srow = reinterpret_cast<const uint16_t*>(p.sq) + (size_t)col * G::NT + wn * 64 + g * 8;

#pragma unroll
    for (int r = 0; r < 4 * MB; ++r)
#pragma unroll
      for (int x = 0; x < 4; ++x) { acc[r][x] = 0.f; tmp[r][x] = 0.f; }
    if constexpr (kBiased) {
#pragma unroll
      for (int mb = 0; mb < MB; ++mb) bias[mb][0] = bias[mb][1] = bias[mb][2] = bias[mb][3] = 0.f;
    }
    if constexpr (ZP) {
#pragma unroll
      for (int mb = 0; mb < MB; ++mb) asum[mb][0] = asum[mb][1] = asum[mb][2] = asum[mb][3] = 0.f;
    }
    int cur_group = -1;
    if (!p.grouped) cur_raw = __ldg(reinterpret_cast<const uint4*>(srow));

    // iterations of this segment that belong to this group: x = off, off + SK, ...
    const uint32_t off = (grp + SK - (it0 % SK)) % SK;
    for (uint32_t x = off; x < len; x += SK) {
      const uint32_t kb = kb0 + x;
      mbar_wait(&full[s], ph, abort_flag, p.status);
      if (p.grouped) {
        int gi = p.group_shift >= 0 ? (int)(kb >> p.group_shift) : (int)(kb / (uint32_t)p.kb_per_group);
        // with zero points also a long group (one scale per column) is folded into `acc` every 1024 rows of k, so
        // that the offsets carried in `tmp` never cost more than a few of its low bits
        if constexpr (ZP) gi = (gi << 12) | (int)(kb >> 3);
        if (gi != cur_group) {
          if (cur_group >= 0) close_group();
          // the group's scales came with the stage (a read from global memory here would be a cold DRAM
          // access whose latency every warp would wait out once per stage)
          cur_raw = lds128(smem_u32(sc_ring) + (uint32_t)s * G::SC_BYTES + (uint32_t)(wn * 64 + g * 8) * 2);
          if constexpr (ZP)
            cur_z = lds128(smem_u32(sc_ring) + (uint32_t)s * G::SC_BYTES + G::SC_ROW_BYTES + (uint32_t)(wn * 64 + g * 8) * 2);
          cur_group = gi;
        }
      } else {
        // one scale per column: the sums are still folded into `acc` every 1024 rows of k, so that the
        // offsets carried in `tmp` never cost more than a few of its low bits
        const int gi = (int)(kb >> 3);
        if (gi != cur_group) {
          if (cur_group >= 0) close_group();
          cur_group = gi;
        }
      }
      const uint8_t* st = stage0 + (size_t)s * G::STAGE_BYTES;
      const uint32_t st_s = stage0_s + (uint32_t)s * G::STAGE_BYTES;  // the same as a shared-space address
      if constexpr (SP) {
        // 2:4 path (Section 4): the kept codes are the A operand of mma.sp.m16n8k32, the 2-bit positions
        // its metadata; one word of codes = one MMA, and the four 32-row steps of the k-block alternate the
        // sparsity selector so that every lane supplies metadata for half of them.
        const uint32_t cp = st_s + G::A_BYTES + wn * G::CODE_CHUNK + lane * 16;
        const uint32_t mp = st_s + G::A_BYTES + G::W_BYTES + wn * G::META_CHUNK + lane * 16;
        uint32_t Cw[4][4], Mw[4][2];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint4 v = lds128(cp + j * 512);
          Cw[j][0] = v.x; Cw[j][1] = v.y; Cw[j][2] = v.z; Cw[j][3] = v.w;
        }
#pragma unroll
        for (int jh = 0; jh < 2; ++jh) {
          const uint4 v = lds128(mp + jh * 512);
          Mw[2 * jh][0] = v.x; Mw[2 * jh][1] = v.y; Mw[2 * jh + 1][0] = v.z; Mw[2 * jh + 1][1] = v.w;
        }
        // this lane's activations of a 32-row step: four 4-byte words, 8 bytes apart, starting at
        // 32*(c/2) + 4*(c%2) bytes inside the step's 64 bytes (the step's groups of four rows are
        // permuted so that they are)
        const uint32_t b_off = (uint32_t)(32 * (c >> 1) + 4 * (c & 1));
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          uint32_t bf[MB][4];
#pragma unroll
          for (int mb = 0; mb < MB; ++mb) {
            const uint32_t arow = st_s + (t >> 1) * G::A_HALF_BYTES + mb * 1024 + g * 128;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const uint32_t o = (uint32_t)(64 * (t & 1) + 8 * i) + b_off;
              bf[mb][i] = lds32(arow + ((((o >> 4) ^ (uint32_t)g) << 4) | (o & 15u)));
            }
          }
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            uint32_t a[4];
            dequant8(Cw[j][t], a);
#pragma unroll
            for (int mb = 0; mb < MB; ++mb) {
              if (t & 1)
                mma_sp_16832<1>(tmp[j * MB + mb], a, bf[mb], Mw[j][t >> 1]);
              else
                mma_sp_16832<0>(tmp[j * MB + mb], a, bf[mb], Mw[j][t >> 1]);
            }
          }
        }
      } else {
      // lane (g, c) finds its vector in slot (c + g / 2) % 4 of its column's four
      const uint32_t wp = st_s + G::A_BYTES + wn * G::CODE_CHUNK + (uint32_t)((lane & ~3) | ((lane + (lane >> 3)) & 3)) * 16;
      // codes of this lane: columns g (X) and g + 8 (Y) of each 16-column block j, its 32 rows of the k-block
      uint32_t X[4][4], Y[4][4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint4 xv = lds128(wp + (2 * j) * 512);
        const uint4 yv = lds128(wp + (2 * j + 1) * 512);
        X[j][0] = xv.x; X[j][1] = xv.y; X[j][2] = xv.z; X[j][3] = xv.w;
        Y[j][0] = yv.x; Y[j][1] = yv.y; Y[j][2] = yv.z; Y[j][3] = yv.w;
      }
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        uint32_t bf[MB][8];
#pragma unroll
        for (int mb = 0; mb < MB; ++mb) {
          const uint32_t arow = st_s + h * G::A_HALF_BYTES + mb * 1024;
          const uint4 v0 = lds128(arow + a_off0);
          const uint4 v1 = lds128(arow + a_off1);
          bf[mb][0] = v0.x; bf[mb][1] = v0.y; bf[mb][2] = v0.z; bf[mb][3] = v0.w;
          bf[mb][4] = v1.x; bf[mb][5] = v1.y; bf[mb][6] = v1.z; bf[mb][7] = v1.w;
        }
        // one word of X and one of Y feed two MMA steps; consecutive MMAs go to different accumulators
#pragma unroll
        for (int u = 0; u < 2; ++u) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            uint32_t x[4], y[4];
            if constexpr (kBiased) {
              dequant8_biased(X[j][2 * h + u], x);
              dequant8_biased(Y[j][2 * h + u], y);
            } else {
              dequant8(X[j][2 * h + u], x);
              dequant8(Y[j][2 * h + u], y);
            }
            // registers 0, 1 of a fragment are its rows k < 8 (lower nibbles), 2, 3 its rows k >= 8 (upper)
            const uint32_t a0[4] = {x[0], y[0], x[1], y[1]};
            const uint32_t a1[4] = {x[2], y[2], x[3], y[3]};
#pragma unroll
            for (int mb = 0; mb < MB; ++mb) {
              mma_16816(tmp[j * MB + mb], a0, bf[mb][4 * u], bf[mb][4 * u + 1]);
              mma_16816(tmp[j * MB + mb], a1, bf[mb][4 * u + 2], bf[mb][4 * u + 3]);
            }
          }
          if constexpr (kBiased) {
            const uint32_t kc[4] = {kBiasLo, kBiasLo, kBiasHi, kBiasHi};
#pragma unroll
            for (int mb = 0; mb < MB; ++mb) {
              mma_16816(bias[mb], kc, bf[mb][4 * u], bf[mb][4 * u + 1]);
              mma_16816(bias[mb], kc, bf[mb][4 * u + 2], bf[mb][4 * u + 3]);
            }
          }
          if constexpr (ZP) {
            const uint32_t ones[4] = {0x3c003c00u, 0x3c003c00u, 0x3c003c00u, 0x3c003c00u};
#pragma unroll
            for (int mb = 0; mb < MB; ++mb) {
              mma_16816(asum[mb], ones, bf[mb][4 * u], bf[mb][4 * u + 1]);
              mma_16816(asum[mb], ones, bf[mb][4 * u + 2], bf[mb][4 * u + 3]);
            }
          }
        }
      }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[s]);
      s += SK;
      if (s >= nstages) { s -= nstages; ph ^= 1u; }
    }
    if (cur_group >= 0) close_group();

    // ---- reduce the SK groups of this CTA (the last step of Algorithm 1) ----
    // Every group but the first parks its tile in shared memory; after one barrier group 0 adds them to its
    // own in group order (one pass instead of a tree: a barrier costs more here than a few shared loads).
    if (grp > 0) {
      float4* dst = red + (size_t)(grp - 1) * G::TILE_F4 + (size_t)wn * G::FRAG_F4 * 32 + lane;
#pragma unroll
      for (int r = 0; r < 4 * MB; ++r) dst[r * 32] = make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
    }
    named_bar_sync(1, kConsumerThreads);
    if (grp == 0) {
#pragma unroll
      for (int gq = 1; gq < SK; ++gq) {
        const float4* src = red + (size_t)(gq - 1) * G::TILE_F4 + (size_t)wn * G::FRAG_F4 * 32 + lane;
#pragma unroll
        for (int r = 0; r < 4 * MB; ++r) {
          const float4 v = src[r * 32];
          acc[r][0] += v.x; acc[r][1] += v.y; acc[r][2] += v.z; acc[r][3] += v.w;
        }
      }
    }
    named_bar_sync(1, kConsumerThreads);  // `red` may be written again

    // ---- stripe fix-up across CTAs and output ----
    const int first_w = p.split ? (int)(col * p.split) : (int)stripe_owner32(col * KB, U, P);
    const int last_w = p.split ? (int)(col * p.split + p.split - 1) : (int)stripe_owner32((col + 1) * KB - 1, U, P);
    if (u + len < u1) {
      // A segment in the middle of the stripe: group 0 holds the tile and finishes it alone (its L2 round
      // trips take a microsecond or two); the other groups go on with the k-blocks of the next segment.
      if (grp == 0) {
        constexpr int kG0 = NW * 32;
        if (last_w > first_w) {
          const int my_slot = 2 * (int)worker + (col != u0 / KB ? 1 : 0);
          float4* mine = reinterpret_cast<float4*>(p.partials + (size_t)my_slot * p.slot_floats) +
                         (size_t)wn * G::FRAG_F4 * 32 + lane;
#pragma unroll
          for (int r = 0; r < 4 * MB; ++r) mine[r * 32] = make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
          named_bar_sync(2, kG0);
          if (ctid == 0) {
            const int old = atom_add_acq_rel_gpu(&p.counters[col], 1);
            const int is_last = (old == last_w - first_w) ? 1 : 0;
            if (is_last) p.counters[col] = 0;
            last_flag[1] = is_last;
          }
          named_bar_sync(2, kG0);
          if (last_flag[1]) {
            // every thread re-reads its own fragment positions of all partials, in stripe order
            for (int w = first_w; w <= last_w; ++w) {
              const int slot = 2 * w + ((!p.split && col != stripe_begin32(w, U, P) / KB) ? 1 : 0);
              const float4* src = reinterpret_cast<const float4*>(p.partials + (size_t)slot * p.slot_floats) +
                                  (size_t)wn * G::FRAG_F4 * 32 + lane;
#pragma unroll
              for (int r = 0; r < 4 * MB; ++r) {
                const float4 v = ld_cg_f4(src + r * 32);
                if (w == first_w) {
                  acc[r][0] = v.x; acc[r][1] = v.y; acc[r][2] = v.z; acc[r][3] = v.w;
                } else {
                  acc[r][0] += v.x; acc[r][1] += v.y; acc[r][2] += v.z; acc[r][3] += v.w;
                }
              }
            }
          }
        }
        if (last_w == first_w || last_flag[1]) {
#pragma unroll
          for (int r = 0; r < 4 * MB; ++r) {
            const int j = r / MB, mb = r % MB;
            const int n = wn * 64 + 16 * j + g;
            const int m = mb * 8 + 2 * c;
            cst[m * G::CST_STRIDE + n] = __half_as_ushort(__float2half_rn(acc[r][0]));
            cst[(m + 1) * G::CST_STRIDE + n] = __half_as_ushort(__float2half_rn(acc[r][1]));
            cst[m * G::CST_STRIDE + n + 8] = __half_as_ushort(__float2half_rn(acc[r][2]));
            cst[(m + 1) * G::CST_STRIDE + n + 8] = __half_as_ushort(__float2half_rn(acc[r][3]));
          }
          named_bar_sync(2, kG0);
          store_tile(col, kG0);
        }
        named_bar_sync(2, kG0);  // cst and last_flag[1] are free again
      }
      u += len;
      it0 += len;
      continue;
    }
    // ---- the last segment of the stripe: all consumer threads take part ----
    bool tile_in_cst = false;
    if (p.cluster) {
      // The CTAs of this column tile form a thread-block cluster and finish side by side.  The partial tiles
      // go straight into the shared memory of the cluster's first CTA (its stage ring is free by now), which
      // adds them to its own in rank order: the order of the workspace path, without its L2 round trips.
      // (cluster == 2: the launch has room for the partial tiles behind the stage ring, which nobody else touches:
      // no need to wait until the first CTA is done with its ring)
      const int rank = (int)worker - first_w;
      const uint32_t xbuf = p.cluster == 2 ? stage0_s + (uint32_t)nstages * G::STAGE_BYTES : stage0_s;
      if (p.cluster == 1) cluster_sync_all();  // every CTA of the tile is done with its stage ring
      if (rank != 0 && grp == 0) {
        const uint32_t dst = xbuf + (uint32_t)(((rank - 1) * G::TILE_F4 + wn * G::FRAG_F4 * 32 + lane) * 16);
#pragma unroll
        for (int r = 0; r < 4 * MB; ++r) st_cluster_f32x4(dst + (uint32_t)(r * 32 * 16), 0u, acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
      }
      cluster_sync_all();  // the partial tiles have arrived
      if (rank == 0) {
        if (grp == 0) {
          for (int src = 1; src <= last_w - first_w; ++src) {
            const uint32_t from = xbuf + (uint32_t)(((src - 1) * G::TILE_F4 + wn * G::FRAG_F4 * 32 + lane) * 16);
#pragma unroll
            for (int r = 0; r < 4 * MB; ++r) {
              const uint4 v = lds128(from + (uint32_t)(r * 32 * 16));
              acc[r][0] += __uint_as_float(v.x); acc[r][1] += __uint_as_float(v.y);
              acc[r][2] += __uint_as_float(v.z); acc[r][3] += __uint_as_float(v.w);
            }
          }
#pragma unroll
          for (int r = 0; r < 4 * MB; ++r) {
            const int j = r / MB, mb = r % MB;
            const int n = wn * 64 + 16 * j + g;
            const int m = mb * 8 + 2 * c;
            cst[m * G::CST_STRIDE + n] = __half_as_ushort(__float2half_rn(acc[r][0]));
            cst[(m + 1) * G::CST_STRIDE + n] = __half_as_ushort(__float2half_rn(acc[r][1]));
            cst[m * G::CST_STRIDE + n + 8] = __half_as_ushort(__float2half_rn(acc[r][2]));
            cst[(m + 1) * G::CST_STRIDE + n + 8] = __half_as_ushort(__float2half_rn(acc[r][3]));
          }
        }
        tile_in_cst = true;
      }
    } else if (last_w > first_w) {
      // this column tile is shared: publish the partial, count arrivals
      if (grp == 0) {
        const int my_slot = 2 * (int)worker + (col != u0 / KB ? 1 : 0);
        float4* mine = reinterpret_cast<float4*>(p.partials + (size_t)my_slot * p.slot_floats) +
                       (size_t)wn * G::FRAG_F4 * 32 + lane;
#pragma unroll
        for (int r = 0; r < 4 * MB; ++r) mine[r * 32] = make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
      }
      named_bar_sync(1, kConsumerThreads);
      if (ctid == 0) {
        const int old = atom_add_acq_rel_gpu(&p.counters[col], 1);
        const int is_last = (old == last_w - first_w) ? 1 : 0;
        if (is_last) p.counters[col] = 0;  // everyone has arrived: leave the counter ready for the next call
        *last_flag = is_last;
      }
      named_bar_sync(1, kConsumerThreads);
      if (*last_flag) {
        // The last arriver adds every partial of the tile, its own included, in stripe order, so the
        // order of the fp32 sum never depends on who came last.  All consumer threads take part and
        // the loads of several contributors are in flight together.
        constexpr int PER = (G::TILE_F4 + kConsumerThreads - 1) / kConsumerThreads;
        constexpr int BATCH = PER >= 8 ? 1 : (PER >= 4 ? 2 : (PER >= 2 ? 4 : 8));  // contributors whose loads are in flight together
        float4 sum[PER];
        for (int w = first_w; w <= last_w; w += BATCH) {
          float4 v[BATCH][PER];
#pragma unroll
          for (int d = 0; d < BATCH; ++d) {
            const int ww = w + d;
            if (ww <= last_w) {
              const int slot = 2 * ww + ((!p.split && col != stripe_begin32(ww, U, P) / KB) ? 1 : 0);
              const float4* src = reinterpret_cast<const float4*>(p.partials + (size_t)slot * p.slot_floats);
#pragma unroll
              for (int e = 0; e < PER; ++e) {
                const int f = ctid + e * kConsumerThreads;
                if (f < G::TILE_F4) v[d][e] = ld_cg_f4(src + f);
              }
            }
          }
#pragma unroll
          for (int d = 0; d < BATCH; ++d) {
            const int ww = w + d;
            if (ww <= last_w) {
#pragma unroll
              for (int e = 0; e < PER; ++e) {
                if (ww == first_w) {
                  sum[e] = v[d][e];
                } else {
                  sum[e].x += v[d][e].x; sum[e].y += v[d][e].y; sum[e].z += v[d][e].z; sum[e].w += v[d][e].w;
                }
              }
            }
          }
        }
#pragma unroll
        for (int e = 0; e < PER; ++e) {
          const int f = ctid + e * kConsumerThreads;
          if (f < G::TILE_F4) {
            // float4 f of the tile is register r of lane ln of warp w2 (fragment order)
            const int ln = f & 31, r = (f >> 5) % G::FRAG_F4, w2 = f / (32 * G::FRAG_F4);
            const int j = r / MB, mb = r % MB;
            const int n = w2 * 64 + 16 * j + (ln >> 2);
            const int m = mb * 8 + 2 * (ln & 3);
            cst[m * G::CST_STRIDE + n] = __half_as_ushort(__float2half_rn(sum[e].x));
            cst[(m + 1) * G::CST_STRIDE + n] = __half_as_ushort(__float2half_rn(sum[e].y));
            cst[m * G::CST_STRIDE + n + 8] = __half_as_ushort(__float2half_rn(sum[e].z));
            cst[(m + 1) * G::CST_STRIDE + n + 8] = __half_as_ushort(__float2half_rn(sum[e].w));
          }
        }
        tile_in_cst = true;
      }
    } else {
      if (grp == 0) {
#pragma unroll
        for (int r = 0; r < 4 * MB; ++r) {
          const int j = r / MB, mb = r % MB;
          const int n = wn * 64 + 16 * j + g;
          const int m = mb * 8 + 2 * c;
          cst[m * G::CST_STRIDE + n] = __half_as_ushort(__float2half_rn(acc[r][0]));
          cst[(m + 1) * G::CST_STRIDE + n] = __half_as_ushort(__float2half_rn(acc[r][1]));
          cst[m * G::CST_STRIDE + n + 8] = __half_as_ushort(__float2half_rn(acc[r][2]));
          cst[(m + 1) * G::CST_STRIDE + n + 8] = __half_as_ushort(__float2half_rn(acc[r][3]));
        }
      }
      tile_in_cst = true;
    }
    if (tile_in_cst) {
      named_bar_sync(1, kConsumerThreads);
      store_tile(col, kConsumerThreads);
      named_bar_sync(1, kConsumerThreads);  // the tile buffer is free again
    }

    u += len;
    it0 += len;
  }
  if (*abort_flag) {
    // a wait gave up: copies may still be in flight towards this CTA's shared memory
    for (int x = 0; x < 1000; ++x) __nanosleep(1000);
  }
}

// cuTensorMapEncodeTiled through the runtime's driver entry point (no link against libcuda).
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// A[M][K] fp16 row-major as a 2-D tensor (inner K); box = 64 columns x mpad rows, 128-byte swizzle.
}  // namespace

bool make_a_tensor_map(CUtensorMap* map, const void* A, int M, int K, int mpad) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
  const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)mpad};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(A), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_a_tensor_map_3d(CUtensorMap* map, const void* A, int M, int K, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {64, (cuuint64_t)M, (cuuint64_t)(K / 64)};
  const cuuint64_t strides[2] = {(cuuint64_t)K * 2, 128};
  const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 2};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(A), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {

template <int MB, int NW, int FMT, int CW = consumer_warps_for(MB)>
cudaError_t launch_one(const DensePlan& plan, const GemmParams& p, cudaStream_t stream) {
  constexpr size_t G_TILE_BYTES = (size_t)Geometry<MB, NW, CW, FMT>::TILE_F4 * 16;
  auto kernel = gemm_dense_kernel<MB, NW, CW, FMT>;
  static bool attr_set[64] = {};  // per device
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
    if (err != cudaSuccess) return err;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  alignas(64) CUtensorMap tmap;
  if (!make_a_tensor_map(&tmap, p.A, p.M, p.K, MB * 8)) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(plan.workers);
  cfg.blockDim = dim3((CW + 4) * 32);
  cfg.dynamicSmemBytes = plan.smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  GemmParams q = p;
  q.cluster = 0;
  const int S = plan.split;
  const char* e = getenv("MARLIN_B200_CLUSTER");  // tuning knob: 0 = fix-up through the workspace
  if (S >= 2 && S <= 8 && (size_t)(S - 1) * G_TILE_BYTES <= (size_t)plan.stages * plan.stage_bytes && !(e && atoi(e) == 0)) {
    // the S CTAs of a column tile as one thread-block cluster, if all clusters of the grid fit on the device
    // at once (a GPC holds only so many clusters of a size; a second wave would cost more than it saves)
    static int max_clusters[64][9] = {};  // per device and cluster size: clusters resident at once (0 unknown, -1 none)
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
    const int ok = (nmax > 0 && (long long)nmax * S >= plan.workers) ? 1 : -1;  // all clusters of THIS grid at once
    cfg.numAttrs = ok > 0 ? 2 : 1;
    q.cluster = ok > 0 ? 1u : 0u;
    // room behind the ring for the S - 1 partial tiles: the exchange then needs one cluster barrier instead of two
    const char* x = getenv("MARLIN_B200_XBUF");  // tuning knob: 0 = partial tiles into the first CTA's ring
    if (ok > 0 && (size_t)plan.smem_bytes + (size_t)(S - 1) * G_TILE_BYTES <= (size_t)kSmemBudget && !(x && atoi(x) == 0)) {
      cfg.dynamicSmemBytes = plan.smem_bytes + (S - 1) * G_TILE_BYTES;
      q.cluster = 2u;
    }
  }
  return cudaLaunchKernelEx(&cfg, kernel, q, tmap);
}

template <int MB, int NW, int FMT, int CW = consumer_warps_for(MB)>
void fill_geometry(DensePlan* plan) {
  using G = Geometry<MB, NW, CW, FMT>;
  plan->cw = CW;
  plan->stage_bytes = G::STAGE_BYTES;
  int stages = G::STAGES;
  if (const char* e = getenv("MARLIN_B200_STAGES")) { int v = atoi(e); if (v >= 2 && v < stages) stages = v; }
  // The ring length is a multiple of the number of warp groups and of the number of producer warps, so that a
  // stage is always consumed by the same group and refilled by the same producer warp.  Every thread then waits
  // on a given barrier for consecutive fillings in its own program order.  Without this, stage s would pass from
  // group to group between ring passes, and a group running more than a ring pass ahead of another (group 0 alone
  // finishes segments in the middle of a stripe) could ask for the filling after next of a barrier: a parity wait
  // cannot tell that from the last completed one and falls through, after which the stage's transaction counts
  // no longer add up.
  constexpr int kRingUnit = (G::SK % kProducerWarps == 0) ? G::SK
                            : (kProducerWarps % G::SK == 0) ? kProducerWarps
                                                            : G::SK * kProducerWarps / (G::SK % 2 == 0 ? 2 : 1);
  static_assert(kRingUnit % G::SK == 0 && kRingUnit % kProducerWarps == 0, "ring unit must be a common multiple");
  stages -= stages % kRingUnit;
  plan->stages = stages;
  plan->smem_bytes = G::FIXED_BYTES + G::ALIGN_SLACK + stages * G::STAGE_BYTES;
}

template <int MB, int NW, int CW>
void fill_geometry_fmt(int fmt, DensePlan* plan) {
  if (fmt == kFmtSparse) fill_geometry<MB, NW, kFmtSparse, CW>(plan);
  else if (fmt == kFmtZero) fill_geometry<MB, NW, kFmtZero, CW>(plan);
  else fill_geometry<MB, NW, kFmtDense, CW>(plan);
}

template <int MB, int NW, int CW>
cudaError_t launch_one_fmt(int fmt, const DensePlan& plan, const GemmParams& p, cudaStream_t stream) {
  if (fmt == kFmtSparse) return launch_one<MB, NW, kFmtSparse, CW>(plan, p, stream);
  if (fmt == kFmtZero) return launch_one<MB, NW, kFmtZero, CW>(plan, p, stream);
  return launch_one<MB, NW, kFmtDense, CW>(plan, p, stream);
}

}  // namespace


bool make_dense_plan(int m_slab, int K, int N, int sm_count, int fmt, DensePlan* plan) {
  if (m_slab < 1 || m_slab > kMaxSlabM || K < kTileK || K % kTileK || N < kChunkN || N % kChunkN) return false;
  if (sm_count < 1) return false;
  int mb = m_slab <= 8 ? 1 : 2;
  const int kb = K / kTileK;
  const long long max_workers = sm_count < kMaxWorkers ? sm_count : kMaxWorkers;
  // Partition (Section 3.4 "Striped Partitioning", adapted).  Two forms.  Tile-aligned: every column tile
  // is cut into S equal k-ranges, one per CTA, so that all CTAs do the same work and run the fix-up once
  // (S = 1: not at all), with the tile width (64, 128 or 256 columns) that suits the shape.  Even stripes
  // over all units (the paper's form, 128-column tiles): every SM is busy to the end, but a CTA whose
  // stripe crosses a tile boundary pays the fix-up twice and finishes microseconds after the others.
  // A cost in microseconds picks between them: a least-squares fit (relative error) to the launch times measured
  // on B200 for every candidate on 36 layer shapes (K, N from 2048 to 28672), at one row and at sixteen.  Up to
  // eight rows: 2.33 fixed, the chunks of the longest CTA at 0.121 (64-column tiles), 0.099 (128 columns; 0.096
  // with twelve consumer warps) or 0.105 (256 columns) each, the cluster fix-up at 0 / 0.36 / 0.68 by tile width
  // plus 0.137 per CTA of the tile (1.11 more through the workspace, above eight CTAs), 4.14 for the late finishers
  // of even stripes: the pick is within 3 % of the fastest candidate on all 36 shapes (0.1 % on average).  Sixteen
  // rows (twice the MMAs per chunk, a ring of fewer and larger stages) have constants of their own and leave out
  // split 256-column tiles, whose times the linear model does not follow (0.3 % on average, at most 5 %).
  int forced_nw = 0;
  if (const char* e = getenv("MARLIN_B200_NW")) { int v = atoi(e); if (v == 1 || v == 2 || v == 4) forced_nw = v; }
  bool allow_split = true;
  if (const char* e = getenv("MARLIN_B200_SPLIT")) allow_split = atoi(e) != 0;
  int want_cw = 0;  // MARLIN_B200_CW: tuning knob, 8 or 12
  if (const char* e = getenv("MARLIN_B200_CW")) want_cw = atoi(e);
  // twelve consumer warps: 128-column tiles from 16 stages per CTA on (see kWideConsumerWarps)
  auto wide_pays = [&](int nw_, long long n) { return mb == 1 && nw_ == 2 && n >= 16 && fmt != kFmtSparse; };
  auto chunk_us = [&](int nw_, long long n) {
    if (mb != 1) return nw_ == 1 ? 0.1536 : nw_ == 4 ? 0.1424 : 0.1303;
    const bool wide = want_cw == kWideConsumerWarps || (want_cw != consumer_warps_for(mb) && wide_pays(nw_, n));
    return nw_ == 1 ? 0.1213 : nw_ == 4 ? 0.1051 : (wide ? 0.0964 : 0.0991);
  };
  const double base_us = mb == 1 ? 2.33 : 2.55, even_us = mb == 1 ? 4.14 : 4.62;
  auto fixup_us = [&](int nw_, long long S) {
    if (S <= 1) return 0.0;
    if (mb == 1) return (nw_ == 1 ? 0.0 : nw_ == 2 ? 0.36 : 0.68) + 0.137 * (double)S + (S > 8 ? 1.11 : 0.0);
    return (nw_ == 1 ? -0.34 : nw_ == 2 ? 0.0 : 0.89) + 0.268 * (double)S + (S > 8 ? 0.51 : 0.0);
  };
  int even_nw = forced_nw ? forced_nw : 2;
  while (even_nw > 1 && N % (kChunkN * even_nw)) even_nw >>= 1;
  const long long even_units = (long long)(N / (kChunkN * even_nw)) * kb;
  const long long even_workers = even_units < max_workers ? even_units : max_workers;
  const long long even_n = (even_units + even_workers - 1) / even_workers;
  double best = base_us + even_us + chunk_us(even_nw, even_n) * (double)(even_n * even_nw);
  int nw = even_nw, split = 0;
  for (int cand = 1; cand <= 4 && allow_split; cand *= 2) {
    if (forced_nw && cand != forced_nw) continue;
    if (N % (kChunkN * cand)) continue;
    const long long ncols = N / (kChunkN * cand);
    long long S = max_workers / ncols;
    if (S > kb) S = kb;
    if (S < 1) continue;
    const long long stages_per_cta = (kb + S - 1) / S;
    if (mb != 1 && cand == 4 && S > 1 && !forced_nw) continue;
    const double cost = base_us + chunk_us(cand, stages_per_cta) * (double)(stages_per_cta * cand) + fixup_us(cand, S);
    if (cost < best) { nw = cand; split = (int)S; best = cost; }
  }
  plan->mb = mb;
  plan->nw = nw;
  plan->kb = kb;
  plan->ncols = N / (kChunkN * nw);
  plan->units = (long long)plan->ncols * plan->kb;
  plan->split = split;
  long long workers = split ? (long long)split * plan->ncols : max_workers;
  if (workers > plan->units) workers = plan->units;
  plan->workers = (int)workers;
  // Consumer warps: twelve for 128-column tiles (nw = 2) from 16 stages per CTA on.  Measured on B200 over 42 layer
  // shapes (K, N from 2048 to 28672, one row): with 128-column tiles twelve warps are 5.5-7.7 % faster at every
  // shape from 16 stages per CTA up; with 64-column tiles they are 3-5 % slower (the ring, capped at 32 stages, holds
  // only two rounds of twelve stages, too few to cover the refill latency); with 256-column tiles it makes no
  // difference; the 2:4 instance gains nothing.
  int cw = consumer_warps_for(mb);
  if (mb == 1) {
    const long long n = split ? (kb + split - 1) / split : (plan->units + workers - 1) / workers;
    if (want_cw == kWideConsumerWarps || (want_cw != consumer_warps_for(mb) && wide_pays(nw, n))) cw = kWideConsumerWarps;
  }
  for (;;) {
    if (cw == kWideConsumerWarps) {
      if (nw == 1) fill_geometry_fmt<1, 1, kWideConsumerWarps>(fmt, plan);
      else if (nw == 2) fill_geometry_fmt<1, 2, kWideConsumerWarps>(fmt, plan);
      else fill_geometry_fmt<1, 4, kWideConsumerWarps>(fmt, plan);
    } else if (mb == 1) {
      if (nw == 1) fill_geometry_fmt<1, 1, consumer_warps_for(1)>(fmt, plan);
      else if (nw == 2) fill_geometry_fmt<1, 2, consumer_warps_for(1)>(fmt, plan);
      else fill_geometry_fmt<1, 4, consumer_warps_for(1)>(fmt, plan);
    } else {
      if (nw == 1) fill_geometry_fmt<2, 1, consumer_warps_for(2)>(fmt, plan);
      else if (nw == 2) fill_geometry_fmt<2, 2, consumer_warps_for(2)>(fmt, plan);
      else fill_geometry_fmt<2, 4, consumer_warps_for(2)>(fmt, plan);
    }
    // the ring must hold one stage per group of warps and per producer warp
    if (plan->stages >= plan->cw / nw && plan->stages >= kProducerWarps) return true;
    if (cw == consumer_warps_for(mb)) return false;
    cw = consumer_warps_for(mb);  // a ring too short for twelve warps (MARLIN_B200_STAGES): eight
  }
}

cudaError_t launch_gemm_dense(const DensePlan& plan, const GemmParams& p, int fmt, cudaStream_t stream) {
  if (plan.mb == 1 && plan.cw == kWideConsumerWarps) {
    if (plan.nw == 1) return launch_one_fmt<1, 1, kWideConsumerWarps>(fmt, plan, p, stream);
    if (plan.nw == 2) return launch_one_fmt<1, 2, kWideConsumerWarps>(fmt, plan, p, stream);
    if (plan.nw == 4) return launch_one_fmt<1, 4, kWideConsumerWarps>(fmt, plan, p, stream);
  } else if (plan.mb == 1 && plan.cw == consumer_warps_for(1)) {
    if (plan.nw == 1) return launch_one_fmt<1, 1, consumer_warps_for(1)>(fmt, plan, p, stream);
    if (plan.nw == 2) return launch_one_fmt<1, 2, consumer_warps_for(1)>(fmt, plan, p, stream);
    if (plan.nw == 4) return launch_one_fmt<1, 4, consumer_warps_for(1)>(fmt, plan, p, stream);
  } else if (plan.mb == 2 && plan.cw == consumer_warps_for(2)) {
    if (plan.nw == 1) return launch_one_fmt<2, 1, consumer_warps_for(2)>(fmt, plan, p, stream);
    if (plan.nw == 2) return launch_one_fmt<2, 2, consumer_warps_for(2)>(fmt, plan, p, stream);
    if (plan.nw == 4) return launch_one_fmt<2, 4, consumer_warps_for(2)>(fmt, plan, p, stream);
  }
  return cudaErrorInvalidValue;
}

}  // namespace marlin_b200
