// Internal declarations shared by the translation units of libmarlin_b200 (sm_100a only).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "marlin_b200.h"

namespace marlin_b200 {

// ---- fixed geometry of the packed layouts ----------------------------------------------------
// One "chunk" is the 64-column x 128-row block of weights a consumer warp turns into tensor-core
// fragments: 8 x 32 lanes x 16 bytes = 4096 bytes (dense).  A pipeline stage holds NW chunks that
// are adjacent in the packed buffer (the same 128 rows, NW*64 consecutive columns).
constexpr int kTileK = 128;           // rows of W per k-block
constexpr int kChunkN = 64;           // columns of W per chunk
constexpr int kChunkBytes = 4096;     // dense chunk
constexpr int kSparseCodeChunkBytes = 2048;  // 2:4 chunk: 64 kept codes per column
constexpr int kSparseMetaChunkBytes = 1024;  // 2:4 chunk: 2-bit positions of the kept codes
constexpr int kProducerWarps = 4;     // the warps of the third warpgroup that issue copies
// The last warpgroup of a CTA issues the copies; it shrinks to kProducerRegs registers per thread
// (setmaxnreg) and the consumer warpgroups share what that frees.
constexpr int kProducerRegs = 40;
constexpr int kMaxStages = 32;
constexpr int kMaxWorkers = 160;      // grid size cap (a B200 has 148 SMs)
constexpr int kMaxSlabM = 16;         // rows of A handled by one launch of the mma.sync kernel
constexpr int kTcMaxSlabM = 128;      // rows of A handled by one launch of the tcgen05 kernel with in-loop scales
constexpr int kTcdMaxSlabM = 64;      // rows of A handled by one launch of the tcgen05 kernel with deferred scales
constexpr int kSmemBudget = 227 * 1024;

// workspace layout (bytes)
constexpr size_t kWsStatusOff = 0;
constexpr size_t kWsCounterOff = 256;
constexpr int kWsMaxCounters = 1024;  // N / 64 <= 1024
constexpr size_t kWsPartialOff = 8192;
constexpr int kWsSlotCols = 256;      // widest column tile

struct DensePlan {
  int mb;          // 8-row blocks of A per launch (1, 2 or 4)
  int nw;          // chunks per stage; column tile = 64 * nw
  int cw;          // consumer warps of the CTA (8 or 12)
  int kb;          // K / 128
  int ncols;       // N / (64 * nw)
  long long units; // ncols * kb
  int workers;     // CTAs
  int split;       // 0: even stripes; S > 0: S k-ranges per column tile, one per CTA
  int stages;
  int stage_bytes;
  int smem_bytes;
};

// Chooses tile width, worker count and pipeline depth for one slab of m_slab <= 32 rows.
// Pure host arithmetic.  Returns false on an unsupported shape.
// fmt: 0 dense, 1 the 2:4 variant, 2 dense with zero points (the stage then carries a zero-point row)
bool make_dense_plan(int m_slab, int K, int N, int sm_count, int fmt, DensePlan* plan);

struct GemmParams {
  const uint16_t* A;
  const uint8_t* wq;
  const uint8_t* sq;
  const uint8_t* meta;   // 2:4 variant only
  const uint8_t* zq;     // packed zero points (fp16 values 0..15 in the order of the packed scales), or nullptr: z = 8
  uint16_t* C;
  int M, K, N;
  uint32_t kb;       // K / 128
  int kb_per_group;  // group_size / 128 (1 for groups of 64 or 32 rows)
  int sub_groups;    // scale groups per 128-row k-block: 1, or 2 / 4 for groups of 64 / 32 rows (tcgen05 kernel only)
  int group_shift;   // log2(kb_per_group) if it is a power of two, else -1
  int grouped;       // 0: one scale per column (group_size == K)
  int ncols;
  uint32_t units;
  uint32_t workers;
  int stages;
  int stage_bytes;
  int* status;
  int* counters;
  float* partials;   // warp-MMA kernel: partial-tile slots
  float* tc_tiles;   // tcgen05 kernel: one fp32 accumulation tile per 256-column tile
  int slot_floats;   // floats per partial-tile slot
  int swiglu;        // 1: the columns come in blocks of 16 (eight gate channels, then the same eight up channels) and the
                     // kernel stores silu(gate) * up, N / 2 columns per row of C
  uint32_t cluster;  // tcgen05 kernel: 1 = launched as thread-block clusters of `split` CTAs (the CTAs of one column tile)
  uint32_t slabs;    // tcgen05 kernel: slabs of 128 batch rows in this launch (1 up to 128 rows); virtual column tile
                     // v = column tile v / slabs of W, batch rows 128 * (v % slabs) ..
  uint32_t whole;    // tcgen05 kernel: 1 = worker w owns the virtual column tiles [w * ncols / P, (w + 1) * ncols / P) whole
  uint32_t split;    // tcgen05 kernel: 0 = even stripes over all units; S > 0 = every column tile is cut into S
                     // k-ranges and worker w owns range w % S of tile w / S (one segment per CTA)
};

cudaError_t launch_gemm_dense(const DensePlan& plan, const GemmParams& p, int fmt, cudaStream_t stream);
cudaError_t launch_pack_sparse24(uint32_t* qc, uint8_t* idx, uint16_t* s, uint32_t* wq, uint32_t* meta, uint16_t* sq, int K,
                                 int N, int G, bool inverse, cudaStream_t stream);

// tcgen05 kernel (gemm_dense_tc.cu): 256-column tiles, up to 128 rows of A per launch.
bool tc_path_supported(int m_slab, int K, int N);
int tc_mpad(int m_slab);  // rows of A padded to the MMA's N: 32, 64 or 128
int tc_max_rows(int K, int N, int sm_count);      // most rows one launch takes (a multiple of 128)
size_t tc_fixup_tiles(int M, int N, int workers); // fp32 accumulation tiles (256 columns x padded rows) the fix-up needs
// fills the plan fields of `p` (ncols, units, workers) itself; sparse24: the 2:4 instances (tcgen05.mma.sp), which read
// the wide 2:4 layout (N a multiple of 256)
// w8: the instances for 8-bit codes (N a multiple of 256)
cudaError_t launch_gemm_dense_tc(GemmParams p, int sm_count, bool sparse24, cudaStream_t stream, bool w8 = false);
// 8-bit codes uint8 [K][N] <-> packed [N/256][K/128][8 vectors][256 columns][16 bytes]
cudaError_t launch_pack_w8(uint8_t* q8, uint8_t* wq, int K, int N, bool inverse, cudaStream_t stream);
// tcgen05 kernel with deferred scales (gemm_tcd.cu): 128-column tiles, up to 64 rows of A per launch.
bool tcd_path_supported(int m_slab, int K, int N);
int tcd_mpad(int m_slab);            // rows of A padded to the MMA's N: 16, 32 or 64
size_t tcd_slot_floats(int m_slab);  // floats of one partial-tile slot of the fix-up
// fills the plan fields of `p` (ncols, units, workers, slot_floats) itself
cudaError_t launch_gemm_tcd(GemmParams p, int sm_count, cudaStream_t stream);
// inverse == false: (q, s) canonical inputs -> (wq, sq) packed outputs; inverse == true: the other way round.
cudaError_t launch_pack_dense(uint32_t* q, uint16_t* s, uint32_t* wq, uint16_t* sq, int K, int N, int G, bool inverse,
                              cudaStream_t stream);
// round-to-nearest quantiser with clipping search (quantize.cu): W fp16 [K][N] -> canonical codes and scales
cudaError_t launch_quantize_rtn(const uint16_t* W, uint32_t* q_kpacked, uint16_t* scales, int K, int N, int G, int n_grid,
                                int n_candidates, cudaStream_t stream);
// gate and up projections side by side in blocks of 16 columns (8 gate, 8 up), canonical codes and scales
cudaError_t launch_interleave_gate_up(const uint32_t* q_gate, const uint16_t* s_gate, const uint32_t* q_up, const uint16_t* s_up,
                                      uint32_t* q_out, uint16_t* s_out, int K, int I, int G, cudaStream_t stream);
// canonical zero points uint8 [K/G][N] (0..15) <-> fp16 values in the packed order of the scales
cudaError_t launch_permute_zeros(uint8_t* z, uint16_t* zq, int K, int N, int G, bool inverse, cudaStream_t stream);
// canonical scales [K/G][N] <-> packed order (shared by the dense and the 2:4 pack)
cudaError_t launch_permute_scales(uint16_t* s, uint16_t* sq, int K, int N, int G, bool inverse, cudaStream_t stream);

// ---- the stripe partition (host and device use the same two formulas) ------------------------
// worker w of P owns units [w*U/P, (w+1)*U/P); the owner of unit x is floor(((x+1)*P - 1) / U).
__host__ __device__ inline long long stripe_begin(long long w, long long U, long long P) { return (w * U) / P; }
__host__ __device__ inline int stripe_owner(long long x, long long U, long long P) {
  return (int)(((x + 1) * P - 1) / U);
}
// the same in 32-bit arithmetic for the device (U * P < 2^32 is checked on the host)
__device__ inline uint32_t stripe_begin32(uint32_t w, uint32_t U, uint32_t P) { return (w * U) / P; }
__device__ inline uint32_t stripe_owner32(uint32_t x, uint32_t U, uint32_t P) { return ((x + 1) * P - 1) / U; }
// The tile-aligned variant of the partition: tile t = w / S, k-range r = w % S covers k-blocks
// [r * KB / S, (r + 1) * KB / S) of the tile (S <= KB, so no range is empty).
__device__ inline uint32_t split_begin32(uint32_t w, uint32_t KB, uint32_t S) {
  const uint32_t t = w / S, r = w - t * S;
  return t * KB + (r * KB) / S;
}

}  // namespace marlin_b200
