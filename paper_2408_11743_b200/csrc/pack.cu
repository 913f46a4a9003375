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
//   Inside a chunk, 16-byte vector number v = (2*j + b) * 32 + 4*g + slot holds 32 codes of ONE column:
//     column n = 64*nb + 16*j + 8*b + g        (g = 0..7; slot = (c + g/2) % 4, c = 0..3)
//     rows   k = 128*kb + {16*c .. 16*c + 15} and 128*kb + 64 + {16*c .. 16*c + 15}
//   (the four vectors of a column are rotated by g/2 so that the threads of the tcgen05 kernel, one column each
//   and 64 bytes apart, hit different banks when they all read their vector of the same c)
//   word w of the vector (w = 2*h + u) holds rows 128*kb + 64*h + 16*c + 8*u + o, o = 0..7, with
//   row offset o in nibble (o >> 1) + 4*(o & 1): one AND+OR pulls out the two codes of rows (2i, 2i+1).
//   Two readers use this order:
//     - the warp-level MMA kernel: lane (g, c) reads the vectors (slot as above) of columns g and g + 8 of a 16-column
//       block; one word of each gives the A-operand registers of two m16n8k16 steps (weights on the
//       16-wide side), and the lane's activations for its rows are 16 contiguous fp16 per 64-row half;
//     - the tcgen05 kernel: a thread owns one column and reads its four vectors (c = 0..3), i.e. all
//       128 rows of the k-block, dequantises and stores them to tensor memory in row order.
//   scales: inside every run of 64 columns, position 8*g + 2*j + b holds column 16*j + 8*b + g,
//   so that the 8 scales a thread needs are one 16-byte load.  Groups of 128 rows and more keep the row order
//   [K/G][N].  Groups of 64 or 32 rows (N a multiple of 256) are stored per k-block and 256-column tile,
//   [K/128][N/256][128/G][256], so that the two or four rows a k-block needs are one contiguous copy.
#include "marlin_internal.cuh"

namespace marlin_b200 {
namespace {

// word `wi` (0..1023) of chunk (kb, nb), nibble p -> matrix position
__device__ __forceinline__ void decode_position(int wi, int p, int kb, int nb, int* k, int* n) {
  int w = wi & 3, lane = (wi >> 2) & 31, i = wi >> 7;
  int g = lane >> 2, c = ((lane & 3) - (g >> 1)) & 3, j = i >> 1, b = i & 1;  // slot = (c + g/2) % 4
  int o = 2 * (p & 3) + (p >> 2);
  *n = 64 * nb + 16 * j + 8 * b + g;
  *k = 128 * kb + 64 * (w >> 1) + 16 * c + 8 * (w & 1) + o;
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
    int nb64 = N / 64;
    int kb, nb;
    chunk_coords(wi >> 10, K / 128, nb64, &kb, &nb);
    uint32_t out = 0;
#pragma unroll
    for (int p = 0; p < 8; ++p) {
      int k, n;
      decode_position((int)(wi & 1023), p, kb, nb, &k, &n);
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
    int nb = n >> 6, j = (n >> 4) & 3, b = (n >> 3) & 1, g = n & 7;
    uint32_t out = 0;
#pragma unroll
    for (int jn = 0; jn < 8; ++jn) {
      int k = 8 * k8 + jn;
      int kb = k >> 7, h = (k >> 6) & 1, c = (k >> 4) & 3, u = (k >> 3) & 1, o = k & 7;
      int p = (o >> 1) + 4 * (o & 1);
      int lane = 4 * g + ((c + (g >> 1)) & 3), i = 2 * j + b, w = 2 * h + u;
      long long wi = ((chunk_index(kb, nb, K / 128, nb64) * 8 + i) * 32 + lane) * 4 + w;
      uint32_t code = (wq[wi] >> (4 * p)) & 15u;
      out |= code << (4 * jn);
    }
    q[qi] = out;
  }
}

__global__ void permute_scales_kernel(const uint16_t* __restrict__ in, uint16_t* __restrict__ out, long long total,
                                      int N, int sub, bool inverse) {
  for (long long x = blockIdx.x * (long long)blockDim.x + threadIdx.x; x < total;
       x += (long long)gridDim.x * blockDim.x) {
    // x = packed position
    const int pos = (int)(x & 63);  // packed position inside the run of 64
    const int g = pos >> 3, j = (pos >> 1) & 3, b = pos & 1;
    const int c64 = 16 * j + 8 * b + g;  // column inside the run
    long long canon;
    if (sub == 1) {
      canon = (x & ~63LL) + c64;
    } else {
      // packed [kb][tile][r][256]  <->  canonical row kb * sub + r, column 256 * tile + ...
      const long long rec = x >> 8;  // (kb * NT + tile) * sub + r
      const int r = (int)(rec % sub);
      const long long kt = rec / sub;
      const int NT = N / 256;
      const long long kb = kt / NT, tile = kt % NT;
      canon = (kb * sub + r) * (long long)N + tile * 256 + (x & 192) + c64;
    }
    if (inverse)
      out[canon] = in[x];
    else
      out[x] = in[canon];
  }
}

// zero points: the same permutation, uint8 codes on the canonical side and fp16 values on the packed side
__global__ void permute_zeros_kernel(uint8_t* __restrict__ z, uint16_t* __restrict__ zq, long long total, int N, int sub,
                                     bool inverse) {
  for (long long x = blockIdx.x * (long long)blockDim.x + threadIdx.x; x < total;
       x += (long long)gridDim.x * blockDim.x) {
    const int pos = (int)(x & 63);
    const int g = pos >> 3, j = (pos >> 1) & 3, b = pos & 1;
    const int c64 = 16 * j + 8 * b + g;
    long long canon;
    if (sub == 1) {
      canon = (x & ~63LL) + c64;
    } else {
      const long long rec = x >> 8;
      const int r = (int)(rec % sub);
      const long long kt = rec / sub;
      const int NT = N / 256;
      const long long kb = kt / NT, tile = kt % NT;
      canon = (kb * sub + r) * (long long)N + tile * 256 + (x & 192) + c64;
    }
    if (inverse)
      z[canon] = (uint8_t)__half2float(__ushort_as_half(zq[x]));
    else
      zq[x] = __half_as_ushort(__float2half_rn((float)z[canon]));
  }
}

// out[row][n], n = 16 b + r: r < 8 -> gate[row][8 b + r], else up[row][8 b + r - 8]
template <typename T>
__global__ void interleave_gate_up_kernel(const T* __restrict__ gate, const T* __restrict__ up, T* __restrict__ out,
                                          long long rows, int I) {
  const long long total = rows * 2 * I;
  for (long long x = blockIdx.x * (long long)blockDim.x + threadIdx.x; x < total; x += (long long)gridDim.x * blockDim.x) {
    const long long row = x / (2 * I);
    const int n = (int)(x % (2 * I));
    const int b = n >> 4, r = n & 15;
    out[x] = r < 8 ? gate[row * I + 8 * b + r] : up[row * I + 8 * b + r - 8];
  }
}

// 8-bit codes: one thread per 16-byte vector of the packed buffer = rows 128 kb + 16 c + 0..15 of column 256 T + n
__global__ void pack_w8_kernel(uint8_t* __restrict__ q8, uint8_t* __restrict__ wq, int K, int N, bool inverse) {
  const long long vecs = (long long)K * N / 16;
  const int KB = K / 128;
  for (long long v = blockIdx.x * (long long)blockDim.x + threadIdx.x; v < vecs; v += (long long)gridDim.x * blockDim.x) {
    const int n = (int)(v & 255);
    const int c = (int)((v >> 8) & 7);
    const long long rec = v >> 11;  // T * KB + kb
    const int kb = (int)(rec % KB);
    const long long T = rec / KB;
    uint8_t* canon = q8 + ((size_t)kb * 128 + 16 * c) * N + T * 256 + n;
    uint8_t* packed = wq + v * 16;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      if (inverse)
        canon[(size_t)j * N] = packed[j];
      else
        packed[j] = canon[(size_t)j * N];
    }
  }
}

}  // namespace

cudaError_t launch_pack_w8(uint8_t* q8, uint8_t* wq, int K, int N, bool inverse, cudaStream_t stream) {
  const long long vecs = (long long)K * N / 16;
  const int threads = 256;
  int blocks = (int)((vecs + threads - 1) / threads);
  if (blocks > 148 * 16) blocks = 148 * 16;
  pack_w8_kernel<<<blocks, threads, 0, stream>>>(q8, wq, K, N, inverse);
  return cudaGetLastError();
}

cudaError_t launch_interleave_gate_up(const uint32_t* q_gate, const uint16_t* s_gate, const uint32_t* q_up, const uint16_t* s_up,
                                      uint32_t* q_out, uint16_t* s_out, int K, int I, int G, cudaStream_t stream) {
  const int threads = 256;
  const long long qrows = K / 8, srows = K / G;
  int blocks = (int)((qrows * 2 * I + threads - 1) / threads);
  if (blocks > 148 * 16) blocks = 148 * 16;
  interleave_gate_up_kernel<uint32_t><<<blocks, threads, 0, stream>>>(q_gate, q_up, q_out, qrows, I);
  blocks = (int)((srows * 2 * I + threads - 1) / threads);
  if (blocks > 148 * 16) blocks = 148 * 16;
  interleave_gate_up_kernel<uint16_t><<<blocks, threads, 0, stream>>>(s_gate, s_up, s_out, srows, I);
  return cudaGetLastError();
}

cudaError_t launch_permute_zeros(uint8_t* z, uint16_t* zq, int K, int N, int G, bool inverse, cudaStream_t stream) {
  const long long ns = (long long)(K / G) * N;
  const int sub = G >= kTileK ? 1 : kTileK / G;
  const int threads = 256;
  int blocks = (int)((ns + threads - 1) / threads);
  if (blocks > 148 * 16) blocks = 148 * 16;
  permute_zeros_kernel<<<blocks, threads, 0, stream>>>(z, zq, ns, N, sub, inverse);
  return cudaGetLastError();
}

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
  return launch_permute_scales(s, sq, K, N, G, inverse, stream);
}

cudaError_t launch_permute_scales(uint16_t* s, uint16_t* sq, int K, int N, int G, bool inverse, cudaStream_t stream) {
  const int threads = 256;
  const long long ns = (long long)(K / G) * N;
  const int sub = G < kTileK ? kTileK / G : 1;
  int sblocks = (int)((ns + threads - 1) / threads);
  if (sblocks > 148 * 16) sblocks = 148 * 16;
  if (!inverse)
    permute_scales_kernel<<<sblocks, threads, 0, stream>>>(s, sq, ns, N, sub, false);
  else
    permute_scales_kernel<<<sblocks, threads, 0, stream>>>(sq, s, ns, N, sub, true);
  return cudaGetLastError();
}

}  // namespace marlin_b200
