// Dense W4A16 layer for sm_100a, decode batch sizes (one launch handles up to 32 rows of A).
//
// Structure of one CTA (one per SM, persistent over its stripe of work units):
//   warp 8        producer: one elected lane issues bulk-async copies (cp.async.bulk + mbarrier
//                 complete_tx) of the packed weight chunks, the group scales and the A rows of one
//                 k-block into a ring of shared-memory stages; weights carry an L2 evict-first policy
//                 (each byte is read once), activations evict-last (re-read by every column tile).
//   warps 0..7    consumers, arranged as SK groups of NW warps.  Stage number `it` of the CTA is
//                 consumed by group it % SK; inside a group warp wn owns 64 output columns.  A warp
//                 reads its 16-byte weight vectors, converts the 4-bit codes to fp16 (q - 8) with the
//                 exponent-bias trick, and feeds mma.sync.m16n8k16 with the WEIGHTS as the 16-wide
//                 operand and the batch on the 8-wide one, so that batch sizes 1..8 cost one MMA per
//                 256 weights.  The group scale is not applied to the weights: each group of k
//                 accumulates into `tmp`, and `acc += s * tmp` in fp32 when the group ends.
//   end of a column segment: tree reduction of the SK groups through shared memory, then the stripe
//                 fix-up across CTAs: partial tiles go to the workspace in fp32, an arrival counter
//                 tells the last CTA of a column tile to add them in stripe order and write fp16 C.
//                 Nobody spins on another CTA.
//
// Paper correspondence (Section 3.4): weight streaming and evict-first ("Maximizing Loading
// Bandwidth"), multi-stage pipeline ("Memory Load Pipelining"), warps splitting K with a shared
// memory reduction ("Warp Layout", Algorithm 1), bit-trick dequantisation into fragment layout
// ("Dequantization and Tensor Cores"), scales ("Groups and Instruction Ordering"), stripes and the
// global reduction ("Striped Partitioning").  What differs from the paper's Ampere design is listed
// in the design document of this repository.
#include "marlin_internal.cuh"

namespace marlin_b200 {
namespace {

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait.  After kWaitLimitNs without completion the CTA-wide abort flag and the status word
// are set; from then on every wait of the CTA returns at once, so all warps run to the end of the
// kernel through their normal control flow (no barrier is left unattended) and the host sees
// MARLIN_ERR_DEVICE_TIMEOUT instead of a hang.
constexpr uint64_t kWaitLimitNs = 2000000000ull;
__device__ __forceinline__ void mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status) {
  if (mbar_try_wait(bar, parity)) return;
  uint32_t spins = 0;
  uint64_t t0 = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 255u) == 0) {
      if (*abort_flag) return;
      uint64_t now = global_timer_ns();
      if (t0 == 0) t0 = now;
      if (now - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        atomicExch(status, (int)MARLIN_ERR_DEVICE_TIMEOUT);
        return;
      }
    }
  }
}

__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
// global -> shared bulk copy; dst, src 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(pol)
      : "memory");
}
__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

template <int LUT>
__device__ __forceinline__ uint32_t lop3(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t r;
  asm("lop3.b32 %0, %1, %2, %3, %4;" : "=r"(r) : "r"(a), "r"(b), "r"(c), "n"(LUT));
  return r;
}
__device__ __forceinline__ uint32_t hsub2_u32(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("sub.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}
__device__ __forceinline__ uint32_t hfma2_u32(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t r;
  asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
  return r;
}

// Eight 4-bit codes of one word -> four registers of two fp16 values (q - 8), in the order of the
// m16n8k16 A fragment.  A code OR'ed under 0x6400 is the fp16 number 1024 + q (1024 + 16 q for the
// upper nibble of a byte); subtracting 1032, or multiplying by 1/16 and subtracting 72, leaves q - 8
// exactly (Section 3.4, "Dequantization and Tensor Cores").
__device__ __forceinline__ void dequant8(uint32_t w, uint32_t (&a)[4]) {
  constexpr uint32_t LO = 0x000f000fu, HI = 0x00f000f0u, EX = 0x64006400u;
  constexpr uint32_t SUB = 0x64086408u;  // {1032, 1032}
  constexpr uint32_t MUL = 0x2c002c00u;  // {1/16, 1/16}
  constexpr uint32_t ADD = 0xd480d480u;  // {-72, -72}
  uint32_t w2 = w >> 8;
  a[0] = hsub2_u32(lop3<0xea>(w, LO, EX), SUB);
  a[1] = hfma2_u32(lop3<0xea>(w, HI, EX), MUL, ADD);
  a[2] = hsub2_u32(lop3<0xea>(w2, LO, EX), SUB);
  a[3] = hfma2_u32(lop3<0xea>(w2, HI, EX), MUL, ADD);
}

__device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ float4 ld_cg_f4(const float4* p) { return __ldcg(p); }

// ---------------------------------------------------------------------------------------------
// shared memory map
// ---------------------------------------------------------------------------------------------
constexpr int kBarBytes = 1024;  // full[32], empty[32], flags
constexpr int kARowBytes = kTileK * 2 + 16;  // 272: rows 16 bytes apart modulo 128 -> conflict-free 16-byte reads

template <int MB, int NW>
struct Geometry {
  static constexpr int SK = kConsumerWarps / NW;
  static constexpr int MPAD = MB * 8;
  static constexpr int NT = NW * 64;
  static constexpr int W_BYTES = NW * kChunkBytes;
  static constexpr int S_BYTES = NW * 128;
  static constexpr int A_OFF = W_BYTES + S_BYTES;
  static constexpr int FRAG_F4 = MB * 4;                     // float4 accumulator registers per thread
  static constexpr int TILE_FLOATS = NW * 32 * FRAG_F4 * 4;  // one partial tile
  static constexpr int RED_BYTES = (SK / 2) * TILE_FLOATS * 4;
  static constexpr int CST_STRIDE = NT + 8;                  // halves
  static constexpr int CST_BYTES = ((MPAD * CST_STRIDE * 2 + 127) / 128) * 128;
  static constexpr int STAGE_BYTES = ((A_OFF + MPAD * kARowBytes + 127) / 128) * 128;
  static constexpr int FIXED_BYTES = kBarBytes + RED_BYTES + CST_BYTES;
};

// ---------------------------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------------------------
template <int MB, int NW>
__global__ void __launch_bounds__(kGemmThreads, 1) gemm_dense_kernel(const GemmParams p) {
  using G = Geometry<MB, NW>;
  constexpr int SK = G::SK;
  extern __shared__ __align__(128) uint8_t smem[];
  uint64_t* full = reinterpret_cast<uint64_t*>(smem);
  uint64_t* empty = full + kMaxStages;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + 2 * kMaxStages * 8);
  volatile int* last_flag = abort_flag + 1;
  float4* red = reinterpret_cast<float4*>(smem + kBarBytes);
  uint16_t* cst = reinterpret_cast<uint16_t*>(smem + kBarBytes + G::RED_BYTES);
  uint8_t* stage0 = smem + G::FIXED_BYTES;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int worker = blockIdx.x;
  const long long U = p.units, P = p.workers;
  const long long u0 = stripe_begin(worker, U, P), u1 = stripe_begin(worker + 1, U, P);
  const int KB = p.kb;
  const int nstages = p.stages;

  if (threadIdx.x == 0) {
    for (int s = 0; s < nstages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], NW);
    }
    *abort_flag = 0;
    *last_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // rows of the A tile at or beyond M are never copied; give them a defined value once
  for (int s = 0; s < nstages; ++s) {
    uint4* arows = reinterpret_cast<uint4*>(stage0 + (size_t)s * G::STAGE_BYTES + G::A_OFF);
    for (int x = threadIdx.x; x < G::MPAD * kARowBytes / 16; x += kGemmThreads) arows[x] = make_uint4(0, 0, 0, 0);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();

  if (warp == kConsumerWarps) {
    // ------------------------------- producer ---------------------------------------------
    const uint64_t pol_w = policy_evict_first();
    const uint64_t pol_a = policy_evict_last();
    const uint32_t tx_bytes = G::W_BYTES + (p.grouped ? G::S_BYTES : 0) + p.M * (kTileK * 2);
    const int nb64 = p.N / 64;
    int s = 0;
    uint32_t ph = 0;
    int col = (int)(u0 / KB), kb = (int)(u0 % KB);
    for (long long u = u0; u < u1; ++u) {
      mbar_wait(&empty[s], ph ^ 1u, abort_flag, p.status);
      uint8_t* st = stage0 + (size_t)s * G::STAGE_BYTES;
      if (lane == 0) mbar_expect_tx(&full[s], tx_bytes);
      __syncwarp();
      if (lane == 0)
        bulk_g2s(st, p.wq + ((size_t)kb * nb64 + (size_t)col * NW) * kChunkBytes, G::W_BYTES, &full[s], pol_w);
      if (lane == 1 && p.grouped)
        bulk_g2s(st + G::W_BYTES, p.sq + ((size_t)(kb / p.kb_per_group) * p.N + (size_t)col * G::NT) * 2, G::S_BYTES,
                 &full[s], pol_w);
      for (int m = lane; m < p.M; m += 32)
        bulk_g2s(st + G::A_OFF + m * kARowBytes, p.A + (size_t)m * p.K + (size_t)kb * kTileK, kTileK * 2, &full[s],
                 pol_a);
      if (++s == nstages) { s = 0; ph ^= 1u; }
      if (++kb == KB) { kb = 0; ++col; }
    }
    if (*abort_flag) {
      // give copies that may still be in flight time to land before the CTA's shared memory goes away
      for (int x = 0; x < 1000; ++x) __nanosleep(1000);
    }
    return;
  }

  // --------------------------------- consumers ----------------------------------------------
  const int grp = warp / NW;
  const int wn = warp % NW;
  const int g = lane >> 2, c = lane & 3;
  int s = grp;  // this group's first stage is iteration `grp` of the CTA
  uint32_t ph = 0;

  float acc[4 * MB][4];
  float tmp[4 * MB][4];
  float cur_s[8];

  long long u = u0;
  long long it0 = 0;  // iteration index of the segment's first unit, relative to u0
  while (u < u1) {
    const int col = (int)(u / KB);
    const int kb0 = (int)(u % KB);
    const int len = (int)min((long long)(KB - kb0), u1 - u);

#pragma unroll
    for (int r = 0; r < 4 * MB; ++r)
#pragma unroll
      for (int x = 0; x < 4; ++x) { acc[r][x] = 0.f; tmp[r][x] = 0.f; }
    int cur_group = -1;
    if (!p.grouped) {
      const uint4 sv = *reinterpret_cast<const uint4*>(p.sq + ((size_t)col * G::NT + wn * 64 + g * 8) * 2);
      const __half2* h2 = reinterpret_cast<const __half2*>(&sv);
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        float2 f = __half22float2(h2[x]);
        cur_s[2 * x] = f.x;
        cur_s[2 * x + 1] = f.y;
      }
      cur_group = 0;
    }

    // first iteration of this segment that belongs to this group
    int off = (int)((grp - (it0 % SK) + SK) % SK);
    for (int x = off; x < len; x += SK) {
      const int kb = kb0 + x;
      mbar_wait(&full[s], ph, abort_flag, p.status);
      const uint8_t* st = stage0 + (size_t)s * G::STAGE_BYTES;

      if (p.grouped) {
        const int gi = kb / p.kb_per_group;
        if (gi != cur_group) {
          if (cur_group >= 0) {
#pragma unroll
            for (int r = 0; r < 4 * MB; ++r) {
              const int j = r / MB;
              acc[r][0] += cur_s[2 * j] * tmp[r][0];
              acc[r][1] += cur_s[2 * j] * tmp[r][1];
              acc[r][2] += cur_s[2 * j + 1] * tmp[r][2];
              acc[r][3] += cur_s[2 * j + 1] * tmp[r][3];
              tmp[r][0] = tmp[r][1] = tmp[r][2] = tmp[r][3] = 0.f;
            }
          }
          const uint4 sv = *reinterpret_cast<const uint4*>(st + G::W_BYTES + wn * 128 + g * 16);
          const __half2* h2 = reinterpret_cast<const __half2*>(&sv);
#pragma unroll
          for (int y = 0; y < 4; ++y) {
            float2 f = __half22float2(h2[y]);
            cur_s[2 * y] = f.x;
            cur_s[2 * y + 1] = f.y;
          }
          cur_group = gi;
        }
      }

      const uint4* wp = reinterpret_cast<const uint4*>(st + wn * kChunkBytes) + lane;
      const uint8_t* ap = st + G::A_OFF + g * kARowBytes + c * 32;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        uint32_t bf[MB][8];
#pragma unroll
        for (int mb = 0; mb < MB; ++mb) {
          const uint4 v0 = *reinterpret_cast<const uint4*>(ap + mb * 8 * kARowBytes + h * 128);
          const uint4 v1 = *reinterpret_cast<const uint4*>(ap + mb * 8 * kARowBytes + h * 128 + 16);
          bf[mb][0] = v0.x; bf[mb][1] = v0.y; bf[mb][2] = v0.z; bf[mb][3] = v0.w;
          bf[mb][4] = v1.x; bf[mb][5] = v1.y; bf[mb][6] = v1.z; bf[mb][7] = v1.w;
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint4 wv = wp[(h * 4 + j) * 32];
          const uint32_t ww[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            uint32_t a[4];
            dequant8(ww[t], a);
#pragma unroll
            for (int mb = 0; mb < MB; ++mb) mma_16816(tmp[j * MB + mb], a, bf[mb][2 * t], bf[mb][2 * t + 1]);
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[s]);
      s += SK;
      if (s >= nstages) { s -= nstages; ph ^= 1u; }
    }
    // close the open scale group
    if (cur_group >= 0) {
#pragma unroll
      for (int r = 0; r < 4 * MB; ++r) {
        const int j = r / MB;
        acc[r][0] += cur_s[2 * j] * tmp[r][0];
        acc[r][1] += cur_s[2 * j] * tmp[r][1];
        acc[r][2] += cur_s[2 * j + 1] * tmp[r][2];
        acc[r][3] += cur_s[2 * j + 1] * tmp[r][3];
      }
    }

    // ---- reduce the SK groups of this CTA (Algorithm 1's final step, as a tree) ----
    if (SK > 1) {
#pragma unroll
      for (int half = SK / 2; half >= 1; half >>= 1) {
        if (grp >= half && grp < 2 * half) {
          float4* dst = red + (size_t)(grp - half) * (G::TILE_FLOATS / 4) + (size_t)wn * G::FRAG_F4 * 32 + lane;
#pragma unroll
          for (int r = 0; r < 4 * MB; ++r) dst[r * 32] = make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
        }
        named_bar_sync(1, kConsumerWarps * 32);
        if (grp < half) {
          const float4* src = red + (size_t)grp * (G::TILE_FLOATS / 4) + (size_t)wn * G::FRAG_F4 * 32 + lane;
#pragma unroll
          for (int r = 0; r < 4 * MB; ++r) {
            const float4 v = src[r * 32];
            acc[r][0] += v.x; acc[r][1] += v.y; acc[r][2] += v.z; acc[r][3] += v.w;
          }
        }
        named_bar_sync(1, kConsumerWarps * 32);
      }
    }

    // ---- stripe fix-up and output, by group 0 ----
    if (grp == 0) {
      const int first_w = stripe_owner((long long)col * KB, U, P);
      const int last_w = stripe_owner((long long)(col + 1) * KB - 1, U, P);
      bool write_out = true;
      if (last_w > first_w) {
        const int my_slot = 2 * worker + (col != (int)(u0 / KB) ? 1 : 0);
        float4* mine = reinterpret_cast<float4*>(p.partials + (size_t)my_slot * p.slot_floats) +
                       (size_t)wn * G::FRAG_F4 * 32 + lane;
#pragma unroll
        for (int r = 0; r < 4 * MB; ++r) mine[r * 32] = make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
        __threadfence();
        named_bar_sync(2, NW * 32);
        if (warp == 0 && lane == 0) {
          const int old = atomicAdd(&p.counters[col], 1);
          const int is_last = (old == last_w - first_w) ? 1 : 0;
          if (is_last) p.counters[col] = 0;  // everyone has arrived: leave the counter ready for the next call
          *last_flag = is_last;
        }
        named_bar_sync(2, NW * 32);
        write_out = (*last_flag != 0);
        if (write_out) {
          // The last arriver adds every partial of the column tile, its own included, in stripe
          // order from the workspace: the order of the fp32 sum never depends on who came last.
          __threadfence();
          for (int w = first_w; w <= last_w; ++w) {
            const int wcol0 = (int)(stripe_begin(w, U, P) / KB);
            const int slot = 2 * w + (col != wcol0 ? 1 : 0);
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
      if (write_out) {
        // fragments -> fp16 tile in shared memory -> 16-byte row stores
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
      named_bar_sync(2, NW * 32);
      if (write_out) {
        constexpr int CH = NW * 8;  // 16-byte chunks per row
        for (int x = warp * 32 + lane; x < p.M * CH; x += NW * 32) {
          const int m = x / CH, ch = x % CH;
          const uint4 v = *reinterpret_cast<const uint4*>(cst + m * G::CST_STRIDE + ch * 8);
          *reinterpret_cast<uint4*>(p.C + (size_t)m * p.N + (size_t)col * G::NT + ch * 8) = v;
        }
      }
      named_bar_sync(2, NW * 32);
    }

    u += len;
    it0 += len;
  }
}

template <int MB, int NW>
cudaError_t launch_one(const DensePlan& plan, const GemmParams& p, cudaStream_t stream) {
  auto kernel = gemm_dense_kernel<MB, NW>;
  static bool attr_set[16] = {};  // per device
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 16 && !attr_set[dev]) {
    err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
    if (err != cudaSuccess) return err;
    attr_set[dev] = true;
  } else if (dev >= 16) {
    err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
    if (err != cudaSuccess) return err;
  }
  kernel<<<plan.workers, kGemmThreads, plan.smem_bytes, stream>>>(p);
  return cudaGetLastError();
}

template <int MB, int NW>
void fill_geometry(DensePlan* plan) {
  using G = Geometry<MB, NW>;
  plan->stage_bytes = G::STAGE_BYTES;
  int stages = (kSmemBudget - G::FIXED_BYTES) / G::STAGE_BYTES;
  if (stages > kMaxStages) stages = kMaxStages;
  plan->stages = stages;
  plan->smem_bytes = G::FIXED_BYTES + stages * G::STAGE_BYTES;
}

}  // namespace

#define MARLIN_DISPATCH(MBV, NWV, STMT)         \
  if (plan_mb == MBV && plan_nw == NWV) { STMT; }

bool make_dense_plan(int m_slab, int K, int N, int sm_count, DensePlan* plan) {
  if (m_slab < 1 || m_slab > kMaxSlabM || K < kTileK || K % kTileK || N < kChunkN || N % kChunkN) return false;
  if (sm_count < 1) return false;
  int mb = m_slab <= 8 ? 1 : (m_slab <= 16 ? 2 : 4);
  int nw = m_slab <= 8 ? 1 : (m_slab <= 16 ? 2 : 4);
  while (nw > 1 && N % (64 * nw)) nw >>= 1;
  plan->mb = mb;
  plan->nw = nw;
  plan->kb = K / kTileK;
  plan->ncols = N / (64 * nw);
  plan->units = (long long)plan->ncols * plan->kb;
  long long workers = sm_count < kMaxWorkers ? sm_count : kMaxWorkers;
  if (workers > plan->units) workers = plan->units;
  plan->workers = (int)workers;
  const int plan_mb = mb, plan_nw = nw;
  MARLIN_DISPATCH(1, 1, (fill_geometry<1, 1>(plan)))
  MARLIN_DISPATCH(1, 2, (fill_geometry<1, 2>(plan)))
  MARLIN_DISPATCH(1, 4, (fill_geometry<1, 4>(plan)))
  MARLIN_DISPATCH(2, 1, (fill_geometry<2, 1>(plan)))
  MARLIN_DISPATCH(2, 2, (fill_geometry<2, 2>(plan)))
  MARLIN_DISPATCH(2, 4, (fill_geometry<2, 4>(plan)))
  MARLIN_DISPATCH(4, 1, (fill_geometry<4, 1>(plan)))
  MARLIN_DISPATCH(4, 2, (fill_geometry<4, 2>(plan)))
  MARLIN_DISPATCH(4, 4, (fill_geometry<4, 4>(plan)))
  return plan->stages >= kConsumerWarps / nw && plan->stages >= 2;
}

cudaError_t launch_gemm_dense(const DensePlan& plan, const GemmParams& p, cudaStream_t stream) {
  const int plan_mb = plan.mb, plan_nw = plan.nw;
  MARLIN_DISPATCH(1, 1, return (launch_one<1, 1>(plan, p, stream)))
  MARLIN_DISPATCH(1, 2, return (launch_one<1, 2>(plan, p, stream)))
  MARLIN_DISPATCH(1, 4, return (launch_one<1, 4>(plan, p, stream)))
  MARLIN_DISPATCH(2, 1, return (launch_one<2, 1>(plan, p, stream)))
  MARLIN_DISPATCH(2, 2, return (launch_one<2, 2>(plan, p, stream)))
  MARLIN_DISPATCH(2, 4, return (launch_one<2, 4>(plan, p, stream)))
  MARLIN_DISPATCH(4, 1, return (launch_one<4, 1>(plan, p, stream)))
  MARLIN_DISPATCH(4, 2, return (launch_one<4, 2>(plan, p, stream)))
  MARLIN_DISPATCH(4, 4, return (launch_one<4, 4>(plan, p, stream)))
  return cudaErrorInvalidValue;
}

}  // namespace marlin_b200
