// Offline re-layout of the 2:4 sparse W4A16 weights: kept codes, 2-bit position metadata and scales
// (Section 4, "Quantized non-zero values" and "Metadata indices": both structures are reshuffled once so
// that every thread's loads are contiguous and the metadata lands in the lanes the sparse MMA reads).
//
// Per chunk (128 rows of the ORIGINAL K = 64 kept rows, 64 columns), ordered like the dense chunks
// (super-columns of four):
//   codes, 2048 bytes: 16-byte vector j*32 + lane (lane = 4g + c) holds words t = 0..3, one per 32-row
//     step of the k-block = one mma.sp.m16n8k32; nibble p of a word (r = p % 4, e = p / 4) is kept value
//     e (first or second) of
//       column 64*nb + 16*j + g + 8*(r & 1)
//       group  gamma = c + 4*(r >> 1) of the step's eight groups of four rows, where MMA group gamma
//              stands for the actual group Gamma(gamma) = 4*(gamma % 2) + gamma / 2 of the step
//     (the permutation of groups makes a lane's activations four words 8 bytes apart);
//   metadata, 1024 bytes: 16-byte vector (j/2)*32 + lane, word (j % 2)*2 + w: the word lane (g, c)
//     supplies for step t = c/2 + 2*w (selector t % 2): nibble x = positions (first | second << 2) of
//     the kept values of column 64*nb + 16*j + g + 8*(x / 4) in MMA group 4*(c % 2) + x % 4.
//   scales: as in the dense layout, one row per scale group of the original K.
//
// Layers whose N is a multiple of 256 use the WIDE layout instead, which the tcgen05 kernel reads (thread = one
// output channel = one tensor-memory lane).  Per 256-column tile T and k-block kb, records in the order T * K/128 + kb:
//   codes, 8192 bytes: 16-byte vector c * 256 + n (c = 0, 1; n = column inside the tile) holds kept values
//     32c .. 32c + 31 of column 256T + n (kept value e of the k-block = kept row 64kb + e); word w holds kept values
//     32c + 8w + o, o = 0..7, in nibble (o >> 1) + 4(o & 1), so that one AND+OR yields the pair (2i, 2i + 1) = the two
//     kept values of one group of four rows;
//   metadata, 4096 bytes: 16-byte vector 128t + L (t = 128-channel half of the tile, L = tensor-memory lane) holds the
//     four words lane L feeds to the four tcgen05.mma.sp steps i = 0..3 (32 rows of k each).  With L = 16a + 8h + r:
//     bits 0-15 describe column 256T + 128t + 16a + r, bits 16-31 column 256T + 128t + 16a + 8 + r, each with four
//     4-bit entries (first | second << 2) for the groups 8i + 4h + 0..3 of the k-block's 32 groups of four rows.
#include "marlin_internal.cuh"

namespace marlin_b200 {
namespace {

__device__ __forceinline__ long long sp_chunk_index(int kb, int nb, int KB, int nb64) {
  int sc = nb >> 2;
  int cs = min(4, nb64 - 4 * sc);
  return (long long)sc * 4 * KB + (long long)kb * cs + (nb & 3);
}
__device__ __forceinline__ void sp_chunk_coords(long long chunk, int KB, int nb64, int* kb, int* nb) {
  long long full = (long long)(nb64 >> 2) * 4 * KB;
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
__device__ __forceinline__ int actual_group(int gamma) { return 4 * (gamma & 1) + (gamma >> 1); }
__device__ __forceinline__ int mma_group(int Gamma) { return 2 * (Gamma & 3) + (Gamma >> 2); }

// codes: one thread per packed word
__global__ void pack_sparse_codes_kernel(const uint32_t* __restrict__ qc, uint32_t* __restrict__ wq, int K, int N) {
  const long long total = (long long)K * N / 16;
  const int KB = K / 128, nb64 = N / 64;
  for (long long wi = blockIdx.x * (long long)blockDim.x + threadIdx.x; wi < total;
       wi += (long long)gridDim.x * blockDim.x) {
    int kb, nb;
    sp_chunk_coords(wi >> 9, KB, nb64, &kb, &nb);
    const int in = (int)(wi & 511);
    const int t = in & 3, lane = (in >> 2) & 31, j = in >> 7;
    const int g = lane >> 2, c = lane & 3;
    uint32_t out = 0;
#pragma unroll
    for (int p = 0; p < 8; ++p) {
      const int r = p & 3, e = p >> 2;
      const int n = 64 * nb + 16 * j + g + 8 * (r & 1);
      const int gamma = c + 4 * (r >> 1);
      const int T = 2 * (32 * kb + 8 * t + actual_group(gamma)) + e;  // kept-value row
      const uint32_t code = (qc[(size_t)(T >> 3) * N + n] >> (4 * (T & 7))) & 15u;
      out |= code << (4 * p);
    }
    wq[wi] = out;
  }
}

// metadata: one thread per packed word
__global__ void pack_sparse_meta_kernel(const uint8_t* __restrict__ idx, uint32_t* __restrict__ meta, int K, int N) {
  const long long total = (long long)K * N / 32;
  const int KB = K / 128, nb64 = N / 64;
  for (long long wi = blockIdx.x * (long long)blockDim.x + threadIdx.x; wi < total;
       wi += (long long)gridDim.x * blockDim.x) {
    int kb, nb;
    sp_chunk_coords(wi >> 8, KB, nb64, &kb, &nb);
    const int in = (int)(wi & 255);
    const int q = in & 3, lane = (in >> 2) & 31, jh = in >> 7;
    const int j = 2 * jh + (q >> 1), w = q & 1;
    const int g = lane >> 2, c = lane & 3;
    const int t = (c >> 1) + 2 * w;
    uint32_t out = 0;
#pragma unroll
    for (int x = 0; x < 8; ++x) {
      const int n = 64 * nb + 16 * j + g + 8 * (x >> 2);
      const int gamma = 4 * (c & 1) + (x & 3);
      const long long G2 = 2LL * (32 * kb + 8 * t + actual_group(gamma));
      const uint32_t i0 = idx[(size_t)G2 * N + n] & 3u, i1 = idx[(size_t)(G2 + 1) * N + n] & 3u;
      out |= (i0 | (i1 << 2)) << (4 * x);
    }
    meta[wi] = out;
  }
}

// inverse: one thread per canonical word of kept codes
__global__ void unpack_sparse_codes_kernel(const uint32_t* __restrict__ wq, uint32_t* __restrict__ qc, int K, int N) {
  const long long total = (long long)K * N / 16;
  const int KB = K / 128, nb64 = N / 64;
  for (long long qi = blockIdx.x * (long long)blockDim.x + threadIdx.x; qi < total;
       qi += (long long)gridDim.x * blockDim.x) {
    const int n = (int)(qi % N);
    const int T8 = (int)(qi / N);
    const int nb = n >> 6, j = (n >> 4) & 3, row = n & 15, g = row & 7, rlo = row >> 3;
    uint32_t out = 0;
#pragma unroll
    for (int jn = 0; jn < 8; ++jn) {
      const int T = 8 * T8 + jn;
      const int e = T & 1, Gabs = T >> 1;
      const int kb = Gabs >> 5, t = (Gabs >> 3) & 3, gamma = mma_group(Gabs & 7);
      const int c = gamma & 3, r = rlo + 2 * (gamma >> 2), p = r + 4 * e;
      const long long wi = sp_chunk_index(kb, nb, KB, nb64) * 512 + (j * 32 + 4 * g + c) * 4 + t;
      out |= ((wq[wi] >> (4 * p)) & 15u) << (4 * jn);
    }
    qc[qi] = out;
  }
}

// inverse: one thread per (group of four original rows, column): writes the two position bytes
__global__ void unpack_sparse_meta_kernel(const uint32_t* __restrict__ meta, uint8_t* __restrict__ idx, int K, int N) {
  const long long total = (long long)(K / 4) * N;
  const int KB = K / 128, nb64 = N / 64;
  for (long long x0 = blockIdx.x * (long long)blockDim.x + threadIdx.x; x0 < total;
       x0 += (long long)gridDim.x * blockDim.x) {
    const int n = (int)(x0 % N);
    const int Gabs = (int)(x0 / N);
    const int nb = n >> 6, j = (n >> 4) & 3, row = n & 15, g = row & 7, rlo = row >> 3;
    const int kb = Gabs >> 5, t = (Gabs >> 3) & 3, gamma = mma_group(Gabs & 7);
    const int c = (gamma >> 2) + 2 * (t & 1), w = t >> 1;
    const int x = (gamma & 3) + 4 * rlo;
    const long long wi = sp_chunk_index(kb, nb, KB, nb64) * 256 + ((j >> 1) * 32 + 4 * g + c) * 4 + (j & 1) * 2 + w;
    const uint32_t nib = (meta[wi] >> (4 * x)) & 15u;
    idx[(size_t)(2LL * Gabs) * N + n] = (uint8_t)(nib & 3u);
    idx[(size_t)(2LL * Gabs + 1) * N + n] = (uint8_t)(nib >> 2);
  }
}

// ---- the wide layout (N % 256 == 0) ----------------------------------------------------------------
__device__ __forceinline__ uint32_t permute_nibbles(uint32_t x, bool inverse) {
  // forward: value o (nibble o of x) goes to nibble (o >> 1) + 4(o & 1); inverse: the other way round
  uint32_t out = 0;
#pragma unroll
  for (int o = 0; o < 8; ++o) {
    const int pnib = (o >> 1) + 4 * (o & 1);
    if (!inverse)
      out |= ((x >> (4 * o)) & 15u) << (4 * pnib);
    else
      out |= ((x >> (4 * pnib)) & 15u) << (4 * o);
  }
  return out;
}

// codes: one thread per word, both directions (a packed word is a nibble permutation of one canonical word)
__global__ void wide_sparse_codes_kernel(const uint32_t* __restrict__ src, uint32_t* __restrict__ dst, int K, int N,
                                         bool inverse) {
  const long long total = (long long)K * N / 16;
  const int KB = K / 128;
  for (long long wi = blockIdx.x * (long long)blockDim.x + threadIdx.x; wi < total;
       wi += (long long)gridDim.x * blockDim.x) {
    // wi indexes the PACKED words: record (T, kb), vector (c, n), word w
    const long long rec = wi >> 11;
    const int in = (int)(wi & 2047);
    const int w = in & 3, vec = in >> 2, c = vec >> 8, n = vec & 255;
    const int T = (int)(rec / KB), kb = (int)(rec % KB);
    const long long canon = (long long)(8 * kb + 4 * c + w) * N + 256 * T + n;  // canonical word: kept rows 8 * (..) + 0..7
    if (!inverse)
      dst[wi] = permute_nibbles(src[canon], false);
    else
      dst[canon] = permute_nibbles(src[wi], true);
  }
}

// metadata: one thread per packed word
__global__ void wide_sparse_meta_pack_kernel(const uint8_t* __restrict__ idx, uint32_t* __restrict__ meta, int K, int N) {
  const long long total = (long long)K * N / 32;
  const int KB = K / 128;
  for (long long wi = blockIdx.x * (long long)blockDim.x + threadIdx.x; wi < total;
       wi += (long long)gridDim.x * blockDim.x) {
    const long long rec = wi >> 10;
    const int in = (int)(wi & 1023);
    const int i = in & 3, vec = in >> 2, t = vec >> 7, L = vec & 127;
    const int a = L >> 4, h = (L >> 3) & 1, r = L & 7;
    const int T = (int)(rec / KB), kb = (int)(rec % KB);
    uint32_t out = 0;
#pragma unroll
    for (int hw = 0; hw < 2; ++hw) {
      const int col = 256 * T + 128 * t + 16 * a + 8 * hw + r;
#pragma unroll
      for (int gq = 0; gq < 4; ++gq) {
        const long long g2 = 2LL * (32 * kb + 8 * i + 4 * h + gq);
        const uint32_t i0 = idx[(size_t)g2 * N + col] & 3u, i1 = idx[(size_t)(g2 + 1) * N + col] & 3u;
        out |= (i0 | (i1 << 2)) << (16 * hw + 4 * gq);
      }
    }
    meta[wi] = out;
  }
}

// inverse: one thread per (group of four original rows, column): writes the two position bytes
__global__ void wide_sparse_meta_unpack_kernel(const uint32_t* __restrict__ meta, uint8_t* __restrict__ idx, int K, int N) {
  const long long total = (long long)(K / 4) * N;
  const int KB = K / 128;
  for (long long x0 = blockIdx.x * (long long)blockDim.x + threadIdx.x; x0 < total;
       x0 += (long long)gridDim.x * blockDim.x) {
    const int col = (int)(x0 % N);
    const int Gabs = (int)(x0 / N);
    const int kb = Gabs >> 5, G = Gabs & 31;
    const int i = G >> 3, h = (G >> 2) & 1, gq = G & 3;
    const int T = col >> 8, n = col & 255, t = n >> 7, m = n & 127;
    const int a = m >> 4, hw = (m >> 3) & 1, r = m & 7;
    const int L = 16 * a + 8 * h + r;
    const long long wi = ((long long)T * KB + kb) * 1024 + (128 * t + L) * 4 + i;
    const uint32_t nib = (meta[wi] >> (16 * hw + 4 * gq)) & 15u;
    idx[(size_t)(2LL * Gabs) * N + col] = (uint8_t)(nib & 3u);
    idx[(size_t)(2LL * Gabs + 1) * N + col] = (uint8_t)(nib >> 2);
  }
}

int grid_for(long long items, int threads) {
  long long b = (items + threads - 1) / threads;
  return (int)(b > 148 * 16 ? 148 * 16 : (b < 1 ? 1 : b));
}

}  // namespace

cudaError_t launch_pack_sparse24(uint32_t* qc, uint8_t* idx, uint16_t* s, uint32_t* wq, uint32_t* meta, uint16_t* sq, int K,
                                 int N, int G, bool inverse, cudaStream_t stream) {
  const int threads = 256;
  const long long code_words = (long long)K * N / 16, meta_words = (long long)K * N / 32;
  if (N % 256 == 0) {
    // the wide layout of the tcgen05 kernel
    if (!inverse) {
      wide_sparse_codes_kernel<<<grid_for(code_words, threads), threads, 0, stream>>>(qc, wq, K, N, false);
      wide_sparse_meta_pack_kernel<<<grid_for(meta_words, threads), threads, 0, stream>>>(idx, meta, K, N);
      if (launch_permute_scales(s, sq, K, N, G, false, stream) != cudaSuccess) return cudaGetLastError();
    } else {
      wide_sparse_codes_kernel<<<grid_for(code_words, threads), threads, 0, stream>>>(wq, qc, K, N, true);
      wide_sparse_meta_unpack_kernel<<<grid_for((long long)(K / 4) * N, threads), threads, 0, stream>>>(meta, idx, K, N);
      if (launch_permute_scales(s, sq, K, N, G, true, stream) != cudaSuccess) return cudaGetLastError();
    }
    return cudaGetLastError();
  }
  if (!inverse) {
    pack_sparse_codes_kernel<<<grid_for(code_words, threads), threads, 0, stream>>>(qc, wq, K, N);
    pack_sparse_meta_kernel<<<grid_for(meta_words, threads), threads, 0, stream>>>(idx, meta, K, N);
    if (launch_permute_scales(s, sq, K, N, G, false, stream) != cudaSuccess) return cudaGetLastError();
  } else {
    unpack_sparse_codes_kernel<<<grid_for(code_words, threads), threads, 0, stream>>>(wq, qc, K, N);
    unpack_sparse_meta_kernel<<<grid_for((long long)(K / 4) * N, threads), threads, 0, stream>>>(meta, idx, K, N);
    if (launch_permute_scales(s, sq, K, N, G, true, stream) != cudaSuccess) return cudaGetLastError();
  }
  return cudaGetLastError();
}

}  // namespace marlin_b200
