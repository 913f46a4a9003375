// Offline re-layout of the dense W4A16 weights and scales (and its inverse).
//
// The paper reshuffles the static weight matrix once so that every thread's 16-byte load holds
// exactly the codes of its tensor-core fragments and so that a tile is one contiguous run of memory
// (Section 3.4, "Maximizing Loading Bandwidth" and "Dequantization and Tensor Cores").  The order
// used here is this library's own:
//
//   One 4096-byte chunk holds the codes of 128 rows (k-block kb = k / 128) x 64 columns (nb = n / 64).
//   Chunks are ordered by "super-columns" of four chunks (256 columns): inside super-column sc = nb / 4
//   the k-blocks follow one another, each with its cs chunks side by side (cs = 4, or the 1..3 chunks
//   left over in the last super-column when N is not a multiple of 256):
//     chunk index = sc * 4 * (K/128) + kb * cs + (nb % 4)
//   so the weights a CTA streams for a 256-column tile are one contiguous run of memory, k-block after
//   k-block, and one k-block of a tile is a single 16 KB bulk copy.
//   word index = ((chunk index * 8 + i) * 32 + lane) * 4 + t
//     i    = 4*h + j                         h: which 64-row half of the k-block, j: which 16 columns
//     lane = 4*g + c                         the consuming thread; g = lane / 4, c = lane % 4
//     t    = 0..3                            which 16-row MMA step inside the half
//   nibble p of the word (bits 4p..4p+3): with r = p % 4,
//     column n = 64*nb + 16*j + g + 8*(r & 1)
//     row    k = 128*kb + 64*h + 16*c + 4*t + 2*(r >> 1) + (p >> 2)
//   so the nibble pairs (0,4) (1,5) (2,6) (3,7) are the four 2 x fp16 registers of the m16n8k16
//   A-operand fragment with the weights transposed onto the 16-wide side, and thread c owns 16
//   consecutive rows of k inside each 64-row half (the order of k inside an MMA step is free as long
//   as both operands agree).
//
//   scales: inside every run of 64 columns, position 8*g + 2*j + b holds column 16*j + 8*b + g,
//   so that the 8 scales a thread needs are one 16-byte load.
#include "marlin_internal.cuh"

namespace marlin_b200 {
namespace {

__device__ __forceinline__ void decode_position(int p, int g, int c, int t, int h, int j, int kb, int nb, int* k,
                                                int* n) {
  int r = p & 3;
  *n = 64 * nb + 16 * j + g + 8 * (r & 1);
  *k = 128 * kb + 64 * h + 16 * c + 4 * t + 2 * (r >> 1) + (p >> 2);
}

// chunk index <-> (kb, nb)
__device__ __forceinline__ long long chunk_index(int kb, int nb, int KB, int nb64) {
  int sc = nb >> 2;
  int cs = min(4, nb64 - 4 * sc);
  return (long long)sc * 4 * KB + (long long)kb * cs + (nb & 3);
}
__device__ __forceinline__ void chunk_coords(long long chunk, int KB, int nb64, int* kb, int* nb) {
  long long full = (long long)(nb64 >> 2) * 4 * KB;  // chunks in complete super-columns
  if (chunk < full) {
    int sc = (int)(chunk / (4 * KB));
    int rem = (int)(chunk % (4 * KB));
    *kb = rem >> 2;
    *nb = 4 * sc + (rem & 3);
  } else {
    int cs = nb64 & 3;
    int rem = (int)(chunk - full);
    *kb = rem / cs;
    *nb = 4 * (nb64 >> 2) + rem % cs;
  }
}

__global__ void pack_weights_kernel(const uint32_t* __restrict__ q, uint32_t* __restrict__ wq, int K, int N) {
  long long total = (long long)K * N / 8;
  for (long long wi = blockIdx.x * (long long)blockDim.x + threadIdx.x; wi < total;
       wi += (long long)gridDim.x * blockDim.x) {
    int t = (int)(wi & 3);
    int lane = (int)((wi >> 2) & 31);
    int i = (int)((wi >> 7) & 7);
    int nb64 = N / 64;
    int kb, nb;
    chunk_coords(wi >> 10, K / 128, nb64, &kb, &nb);
    int g = lane >> 2, c = lane & 3, h = i >> 2, j = i & 3;
    uint32_t out = 0;
#pragma unroll
    for (int p = 0; p < 8; ++p) {
      int k, n;
      decode_position(p, g, c, t, h, j, kb, nb, &k, &n);
      uint32_t code = (q[(size_t)(k >> 3) * N + n] >> (4 * (k & 7))) & 15u;
      out |= code << (4 * p);
    }
    wq[wi] = out;
  }
}

__global__ void unpack_weights_kernel(const uint32_t* __restrict__ wq, uint32_t* __restrict__ q, int K, int N) {
  long long total = (long long)K * N / 8;
  int nb64 = N / 64;
  for (long long qi = blockIdx.x * (long long)blockDim.x + threadIdx.x; qi < total;
       qi += (long long)gridDim.x * blockDim.x) {
    int n = (int)(qi % N);
    int k8 = (int)(qi / N);
    int nb = n >> 6, j = (n >> 4) & 3, row = n & 15;
    int g = row & 7, rbit0 = row >> 3;
    uint32_t out = 0;
#pragma unroll
    for (int jn = 0; jn < 8; ++jn) {
      int k = 8 * k8 + jn;
      int kb = k >> 7, h = (k >> 6) & 1, c = (k >> 4) & 3, t = (k >> 2) & 3, e = k & 3;
      int p = (rbit0 | ((e >> 1) << 1)) + 4 * (e & 1);
      int lane = 4 * g + c, i = 4 * h + j;
      long long wi = ((chunk_index(kb, nb, K / 128, nb64) * 8 + i) * 32 + lane) * 4 + t;
      uint32_t code = (wq[wi] >> (4 * p)) & 15u;
      out |= code << (4 * jn);
    }
    q[qi] = out;
  }
}

__global__ void permute_scales_kernel(const uint16_t* __restrict__ in, uint16_t* __restrict__ out, long long total,
                                      bool inverse) {
  for (long long x = blockIdx.x * (long long)blockDim.x + threadIdx.x; x < total;
       x += (long long)gridDim.x * blockDim.x) {
    long long base = x & ~63LL;
    int pos = (int)(x & 63);  // packed position inside the run of 64
    int g = pos >> 3, j = (pos >> 1) & 3, b = pos & 1;
    long long canon = base + 16 * j + 8 * b + g;
    if (inverse)
      out[canon] = in[x];
    else
      out[x] = in[canon];
  }
}

}  // namespace

cudaError_t launch_pack_dense(uint32_t* q, uint16_t* s, uint32_t* wq, uint16_t* sq, int K, int N, int G, bool inverse,
                              cudaStream_t stream) {
  long long words = (long long)K * N / 8;
  int threads = 256;
  int blocks = (int)((words + threads - 1) / threads);
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (!inverse)
    pack_weights_kernel<<<blocks, threads, 0, stream>>>(q, wq, K, N);
  else
    unpack_weights_kernel<<<blocks, threads, 0, stream>>>(wq, q, K, N);
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  long long ns = (long long)(K / G) * N;
  int sblocks = (int)((ns + threads - 1) / threads);
  if (sblocks > 148 * 16) sblocks = 148 * 16;
  if (!inverse)
    permute_scales_kernel<<<sblocks, threads, 0, stream>>>(s, sq, ns, false);
  else
    permute_scales_kernel<<<sblocks, threads, 0, stream>>>(sq, s, ns, true);
  return cudaGetLastError();
}

}  // namespace marlin_b200
