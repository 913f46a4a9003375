// Device-side helpers shared by the GEMM kernels of libmarlin_b200: PTX wrappers for mbarriers,
// bulk and tensor copies, programmatic dependent launch, register re-allocation, and the int4 -> fp16
// conversion.  sm_100a only.
#pragma once

#include <cuda.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "marlin_b200.h"

namespace marlin_b200 {

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
#ifndef MARLIN_WAIT_LIMIT_NS
#define MARLIN_WAIT_LIMIT_NS 2000000000ull  // a test build of the library shortens this to milliseconds
#endif
constexpr uint64_t kWaitLimitNs = MARLIN_WAIT_LIMIT_NS;
// Test builds only (-DMARLIN_TEST_HOOKS): when word 7 of the workspace's status area holds this value, worker 0
// leaves out the copies of its second pipeline stage, so that the waits on that stage run into their limit and
// the time-out path can be exercised without any fault.  The product library is built without the hooks.
constexpr int kTestWithholdMagic = 0x57495448;
// BACKOFF_NS > 0: sleep between polls.  The copy-issuing warps use it: their waits are long and not urgent,
// and a warp that polls flat out takes issue slots from the compute warps of its scheduler.
template <int BACKOFF_NS = 0>
__device__ __forceinline__ void mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status) {
  if (mbar_try_wait(bar, parity)) return;
  uint32_t spins = 0;
  uint64_t t0 = 0;
  while (!mbar_try_wait(bar, parity)) {
    if (BACKOFF_NS > 0) __nanosleep(BACKOFF_NS);
    if ((++spins & 255u) == 0) {
      if (*abort_flag) return;
      uint64_t now = global_timer_ns();
      if (t0 == 0) t0 = now;
      if (now > t0 && now - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        // the first wait that gives up leaves a record behind the status word: who waited, on what, how long
        if (atomicCAS(status, 0, (int)MARLIN_ERR_DEVICE_TIMEOUT) == 0) {
          status[1] = (int)blockIdx.x;
          status[2] = (int)threadIdx.x;
          status[3] = (int)(smem_u32(bar) & 1023u);
          status[4] = (int)parity;
          status[5] = (int)spins;
          status[6] = (int)((now - t0) >> 10);
        }
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
__device__ __forceinline__ uint64_t policy_evict_normal() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
// global -> shared bulk copy; dst, src 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(pol)
      : "memory");
}
// One box of a 2-D tensor map -> shared memory (no multicast: every CTA fetches its own copy).
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar,
                                            uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(pol)
      : "memory");
}
// One box of a 3-D tensor map -> shared memory
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, int x, int y, int z, uint64_t* bar,
                                            uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3, %4}], [%5], %6;"
      ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar)), "l"(pol)
      : "memory");
}
__device__ __forceinline__ int atom_add_acq_rel_gpu(int* addr, int v) {
  int old;
  asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(addr), "r"(v) : "memory");
  return old;
}
__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// Thread-block cluster: hardware barrier over all threads of all CTAs of the cluster (release / acquire), and
// a 16-byte store into the shared memory of the CTA with rank `cta` at the address that `local_addr` has here.
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void st_cluster_f32x4(uint32_t local_addr, uint32_t cta, float a, float b, float c, float d) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(cta));
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(remote), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
// 16-byte load from the shared memory of the CTA with rank `cta`, at the address `local_addr` has here
__device__ __forceinline__ float4 ld_cluster_f32x4(uint32_t local_addr, uint32_t cta) {
  uint32_t remote;
  float4 v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(cta));
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(remote) : "memory");
  return v;
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
__device__ __forceinline__ uint32_t hadd2_u32(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("add.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
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

// The same with a per-group zero point z in place of 8 (W = (q - z) * s): the subtrahends become registers,
// sub_lo = {1024 + z, 1024 + z} and add_hi = {-(64 + z), -(64 + z)}; the instruction count is unchanged.
__device__ __forceinline__ void dequant8_zp(uint32_t w, uint32_t (&a)[4], uint32_t sub_lo, uint32_t add_hi) {
  constexpr uint32_t LO = 0x000f000fu, HI = 0x00f000f0u, EX = 0x64006400u;
  constexpr uint32_t MUL = 0x2c002c00u;  // {1/16, 1/16}
  uint32_t w2 = w >> 8;
  a[0] = hsub2_u32(lop3<0xea>(w, LO, EX), sub_lo);
  a[1] = hfma2_u32(lop3<0xea>(w, HI, EX), MUL, add_hi);
  a[2] = hsub2_u32(lop3<0xea>(w2, LO, EX), sub_lo);
  a[3] = hfma2_u32(lop3<0xea>(w2, HI, EX), MUL, add_hi);
}

// The same eight codes WITHOUT the subtraction: a[0], a[2] = 1024 + q (lower nibbles under 0x6400), a[1],
// a[3] = 64 + q (upper nibbles under 0x5400, whose unit in the last place is 1/16).  Five instructions
// instead of nine.  The caller carries the offsets through the product and removes
// sum_k a[k] * (1032 or 72) afterwards (kBiasLo, kBiasHi: offset + 8 as fp16 pairs).
constexpr uint32_t kBiasLo = 0x64086408u;  // {1032, 1032}
constexpr uint32_t kBiasHi = 0x54805480u;  // {72, 72}
__device__ __forceinline__ void dequant8_biased(uint32_t w, uint32_t (&a)[4]) {
  constexpr uint32_t LO = 0x000f000fu, HI = 0x00f000f0u, EXL = 0x64006400u, EXH = 0x54005400u;
  uint32_t w2 = w >> 8;
  a[0] = lop3<0xea>(w, LO, EXL);
  a[1] = lop3<0xea>(w, HI, EXH);
  a[2] = lop3<0xea>(w2, LO, EXL);
  a[3] = lop3<0xea>(w2, HI, EXH);
}

__device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// four 8 x 8 matrices of 16-bit elements from shared memory: lanes 8i .. 8i + 7 give the row addresses of matrix i,
// register i of every lane receives its two elements of matrix i (the m16n8k16 operand order)
__device__ __forceinline__ void ldmatrix_x4(uint32_t saddr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(saddr));
}

// 2:4 sparse MMA: A = 16 x 32 with 16 stored values per row (the usual 16 x 16 A fragment), B = 32 x 8,
// E = metadata word of the lanes the selector names (lane % 4 in {0, 1} for selector 0, {2, 3} for 1):
// nibble x of that lane's word = positions (first | second << 2) of the two kept values of row
// g + 8*(x / 4) in group 4*(lane % 2) + x % 4 of four consecutive rows of B.  (Layout confirmed on B200
// with one-hot probes.)
template <int SEL>
__device__ __forceinline__ void mma_sp_16832(float (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[4], uint32_t e) {
  asm("mma.sp::ordered_metadata.sync.aligned.m16n8k32.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
      "{%8,%9,%10,%11}, {%0,%1,%2,%3}, %12, %13;"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]), "r"(b[2]), "r"(b[3]), "r"(e), "n"(SEL));
}

// Explicit shared-space loads from a 32-bit shared address (the stage ring is addressed through a pointer
// that is re-aligned at run time, which can hide the address space from the compiler).
// silu(gate) * up for eight fp16 pairs: fp16 -> fp32, g / (1 + exp(-g)) * u in fp32, one rounding to fp16
__device__ __forceinline__ uint32_t swiglu2(uint32_t gate, uint32_t up) {
  const float2 g = __half22float2(*reinterpret_cast<const __half2*>(&gate));
  const float2 u = __half22float2(*reinterpret_cast<const __half2*>(&up));
  const float y0 = __fdividef(g.x, 1.f + __expf(-g.x)) * u.x;
  const float y1 = __fdividef(g.y, 1.f + __expf(-g.y)) * u.y;
  const __half2 r = __floats2half2_rn(y0, y1);
  return *reinterpret_cast<const uint32_t*>(&r);
}
__device__ __forceinline__ uint4 swiglu8(uint4 gate, uint4 up) {
  return make_uint4(swiglu2(gate.x, up.x), swiglu2(gate.y, up.y), swiglu2(gate.z, up.z), swiglu2(gate.w, up.w));
}
__device__ __forceinline__ uint4 lds128(uint32_t saddr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(saddr));
  return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t saddr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(saddr));
  return v;
}
__device__ __forceinline__ uint32_t lds16(uint32_t saddr) {
  uint16_t v;
  asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(saddr));
  return v;
}

// Register re-allocation between warpgroups (all four warps of a warpgroup execute it together).
template <int N>
__device__ __forceinline__ void setmaxnreg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N>
__device__ __forceinline__ void setmaxnreg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

// Programmatic dependent launch: let the next kernel of the stream start its prologue while this
// one drains, and wait for the previous kernel's memory before touching anything it may have written.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait_prior_grids() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ float4 ld_cg_f4(const float4* p) { return __ldcg(p); }

// tensor maps are built through the runtime's driver entry point (no link against libcuda)
bool make_a_tensor_map(CUtensorMap* map, const void* A, int M, int K, int box_rows);
// A[M][K] as a 3-D tensor (64 columns, M rows, K / 64 column blocks): one box of 64 x box_rows x 2 brings both
// 64-wide halves of a 128-row k-block, each as a 128-byte-swizzled tile of box_rows rows, one after the other
bool make_a_tensor_map_3d(CUtensorMap* map, const void* A, int M, int K, int box_rows);

}  // namespace marlin_b200
