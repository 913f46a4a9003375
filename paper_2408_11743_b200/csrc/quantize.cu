// Data-free quantiser in front of marlin_pack: fp16 weights -> 4-bit codes and fp16 group scales, round to nearest
// with a per-group search for the clipping threshold (Section 3.5 (a): group scales picked by searching for the
// best group-wise clipping thresholds; the grid is the symmetric one of Section 3.4, W ~ (q - 8) * s).
//
// Per group of G consecutive rows of one column:
//   a   = max |w|
//   r_t = 1 - t / n_grid,  t = 0 .. n_candidates - 1         (t = 0: no clipping)
//   s_t = fp16((a * r_t) * (2 / 15))                          (15 steps across [-a r, a r]; never zero)
//   q_i = clamp(round_half_even(w_i * (1 / s_t)), -8, 7) + 8
//   e_t = sum_i (w_i - (q_i - 8) s_t)^2, summed in the order i = 0 .. G - 1
// and the first candidate with the least e_t wins.  Codes and the winner are integers decided by fp32 arithmetic,
// so every operation is spelled out with its rounding (single IEEE operations, fused multiply-add where written):
// the same inputs give the same codes on every run and on any implementation that follows these lines.
//
// One thread owns one (group, column): its sums run in a fixed order and neighbouring threads read neighbouring
// columns (coalesced).  Groups of 32, 64 or 128 rows are held in registers; longer groups are re-read once per
// candidate from the L1/L2.  This is an offline step bounded by the arithmetic of the search (about 10 operations
// per weight and candidate), not by DRAM.
#include "marlin_internal.cuh"

namespace marlin_b200 {
namespace {

__device__ __forceinline__ float load_w(const uint16_t* p) { return __half2float(__ushort_as_half(__ldg(p))); }

__device__ __forceinline__ float quantise_one(float w, float inv) {
  float q = rintf(__fmul_rn(w, inv));  // round half to even
  return fminf(fmaxf(q, -8.f), 7.f);
}

__global__ void __launch_bounds__(128)
quantize_rtn_kernel(const uint16_t* __restrict__ W, uint32_t* __restrict__ q_kpacked, uint16_t* __restrict__ scales, int K,
                    int N, int G, int n_grid, int n_candidates) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  const int g = blockIdx.y;
  if (n >= N) return;
  const uint16_t* w = W + (size_t)g * G * N + n;
  float a = 0.f;
  for (int i = 0; i < G; ++i) a = fmaxf(a, fabsf(load_w(w + (size_t)i * N)));
  const float two_fifteenths = __fdiv_rn(2.f, 15.f);
  float best_err = __int_as_float(0x7f800000);  // +inf
  uint16_t best_s = 1;
  for (int t = 0; t < n_candidates; ++t) {
    const float r = __fsub_rn(1.f, __fdiv_rn((float)t, (float)n_grid));
    const float s32 = __fmul_rn(__fmul_rn(a, r), two_fifteenths);
    uint16_t sh = __half_as_ushort(__float2half_rn(s32));
    if (sh == 0) sh = 1;  // a scale that rounds to zero: the smallest positive fp16
    const float s = __half2float(__ushort_as_half(sh));
    const float inv = __fdiv_rn(1.f, s);
    float err = 0.f;
    for (int i = 0; i < G; ++i) {
      const float wi = load_w(w + (size_t)i * N);
      const float q = quantise_one(wi, inv);
      const float d = __fmaf_rn(-q, s, wi);
      err = __fmaf_rn(d, d, err);
    }
    if (err < best_err) {
      best_err = err;
      best_s = sh;
    }
  }
  const float s = __half2float(__ushort_as_half(best_s));
  const float inv = __fdiv_rn(1.f, s);
  scales[(size_t)g * N + n] = best_s;
  // canonical code words: nibble j of word (k / 8, n) = code of row 8 * (k / 8) + j
  for (int i8 = 0; i8 < G / 8; ++i8) {
    uint32_t word = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float wi = load_w(w + (size_t)(8 * i8 + j) * N);
      const int q = (int)quantise_one(wi, inv) + 8;
      word |= (uint32_t)q << (4 * j);
    }
    q_kpacked[((size_t)g * (G / 8) + i8) * N + n] = word;
  }
}

// The same for groups of 32, 64 or 128 rows with the group held in registers: one read of W, then arithmetic only
// (the operations and their order are those of the kernel above, so the outputs are the same bit for bit).
template <int GC>
__global__ void __launch_bounds__(128)
quantize_rtn_cached_kernel(const uint16_t* __restrict__ W, uint32_t* __restrict__ q_kpacked, uint16_t* __restrict__ scales,
                           int K, int N, int n_grid, int n_candidates) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  const int g = blockIdx.y;
  if (n >= N) return;
  const uint16_t* wp = W + (size_t)g * GC * N + n;
  float w[GC];
#pragma unroll
  for (int i = 0; i < GC; ++i) w[i] = load_w(wp + (size_t)i * N);
  float a = 0.f;
#pragma unroll
  for (int i = 0; i < GC; ++i) a = fmaxf(a, fabsf(w[i]));
  const float two_fifteenths = __fdiv_rn(2.f, 15.f);
  float best_err = __int_as_float(0x7f800000);
  uint16_t best_s = 1;
#pragma unroll 1
  for (int t = 0; t < n_candidates; ++t) {
    const float r = __fsub_rn(1.f, __fdiv_rn((float)t, (float)n_grid));
    const float s32 = __fmul_rn(__fmul_rn(a, r), two_fifteenths);
    uint16_t sh = __half_as_ushort(__float2half_rn(s32));
    if (sh == 0) sh = 1;
    const float s = __half2float(__ushort_as_half(sh));
    const float inv = __fdiv_rn(1.f, s);
    float err = 0.f;
#pragma unroll
    for (int i = 0; i < GC; ++i) {
      const float q = quantise_one(w[i], inv);
      const float d = __fmaf_rn(-q, s, w[i]);
      err = __fmaf_rn(d, d, err);
    }
    if (err < best_err) {
      best_err = err;
      best_s = sh;
    }
  }
  const float s = __half2float(__ushort_as_half(best_s));
  const float inv = __fdiv_rn(1.f, s);
  scales[(size_t)g * N + n] = best_s;
#pragma unroll
  for (int i8 = 0; i8 < GC / 8; ++i8) {
    uint32_t word = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) word |= (uint32_t)((int)quantise_one(w[8 * i8 + j], inv) + 8) << (4 * j);
    q_kpacked[((size_t)g * (GC / 8) + i8) * N + n] = word;
  }
}

}  // namespace

cudaError_t launch_quantize_rtn(const uint16_t* W, uint32_t* q_kpacked, uint16_t* scales, int K, int N, int G, int n_grid,
                                int n_candidates, cudaStream_t stream) {
  const int threads = N % 128 == 0 ? 128 : 64;
  dim3 grid((unsigned)(N / threads), (unsigned)(K / G));
  if (G == 128)
    quantize_rtn_cached_kernel<128><<<grid, threads, 0, stream>>>(W, q_kpacked, scales, K, N, n_grid, n_candidates);
  else if (G == 64)
    quantize_rtn_cached_kernel<64><<<grid, threads, 0, stream>>>(W, q_kpacked, scales, K, N, n_grid, n_candidates);
  else if (G == 32)
    quantize_rtn_cached_kernel<32><<<grid, threads, 0, stream>>>(W, q_kpacked, scales, K, N, n_grid, n_candidates);
  else
    quantize_rtn_kernel<<<grid, threads, 0, stream>>>(W, q_kpacked, scales, K, N, G, n_grid, n_candidates);
  return cudaGetLastError();
}

}  // namespace marlin_b200
