// C-ABI entry points of libmarlin_b200: argument validation, planning, launches.
#include <stdlib.h>

#include "marlin_internal.cuh"

using namespace marlin_b200;

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// group_size -> normalised G, or 0 if unsupported: K itself (one scale per column, also written -1), a multiple of
// 128 that divides K, or 64 / 32 on layers whose N is a multiple of 256 (those run on the tcgen05 kernel alone).
int normalise_group(int K, int N, int group_size) {
  if (K <= 0) return 0;
  if (group_size == -1 || group_size == K) return K;
  if (group_size == 64 || group_size == 32) return (N % 256 == 0) ? group_size : 0;
  if (group_size <= 0 || group_size % kTileK || K % group_size) return 0;
  return group_size;
}

bool shape_ok(int K, int N) {
  // the device's 32-bit stripe arithmetic needs (N/64) * (K/128) * workers < 2^32
  return K >= kTileK && K % kTileK == 0 && K <= (1 << 20) && N >= kChunkN && N % kChunkN == 0 &&
         N / kChunkN <= kWsMaxCounters;
}

struct DeviceInfo {
  int sm_count;
  int cc_major;
};

// Queried once per device and cached (a few attribute reads; no allocation).
int device_info(DeviceInfo* out) {
  static DeviceInfo cache[64];
  static bool known[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MARLIN_ERR_CUDA;
  if (dev >= 0 && dev < 64 && known[dev]) {
    *out = cache[dev];
    return MARLIN_OK;
  }
  DeviceInfo info;
  if (cudaDeviceGetAttribute(&info.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&info.cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return MARLIN_ERR_CUDA;
  if (dev >= 0 && dev < 64) {
    cache[dev] = info;
    known[dev] = true;
  }
  *out = info;
  return MARLIN_OK;
}

// Batch size from which the tcgen05 kernel takes over from the warp-level MMA kernel.
int tc_min_m() {
  static int v = -1;
  if (v < 0) {
    const char* e = getenv("MARLIN_B200_TC_MIN_M");  // tuning knob; default below
    v = e ? atoi(e) : 17;
    if (v < 1) v = 1;
  }
  return v;
}

// The tcgen05 kernel with deferred scales and 128-column tiles (gemm_tcd.cu) takes the layers whose N is a
// multiple of 128 but not of 256 at batch sizes above 16.  MARLIN_B200_TCD (tuning knob): 0 switches it off
// (slabs of 16 rows through the warp-level kernel instead), 1 makes it take every batch size on every layer
// whose N is a multiple of 128 (64 rows per launch).
int tcd_mode() {
  const char* e = getenv("MARLIN_B200_TCD");  // read at every call, like the other tuning knobs
  return !e ? 2 : (atoi(e) == 0 ? 0 : 1);     // 0 off, 1 everywhere, 2 default
}

}  // namespace

extern "C" {

const char* marlin_status_string(int status) {
  switch (status) {
    case MARLIN_OK: return "ok";
    case MARLIN_ERR_NULL: return "null pointer";
    case MARLIN_ERR_SHAPE: return "unsupported shape";
    case MARLIN_ERR_GROUP: return "unsupported group size";
    case MARLIN_ERR_ALIGN: return "pointer not 16-byte aligned";
    case MARLIN_ERR_WORKSPACE: return "workspace too small";
    case MARLIN_ERR_ARCH: return "device is not sm_100";
    case MARLIN_ERR_CUDA: return "CUDA error";
    case MARLIN_ERR_DEVICE_TIMEOUT: return "bounded wait expired inside a kernel";
    default: return "unknown status";
  }
}

size_t marlin_packed_weight_bytes(int K, int N, int sparse24) {
  if (!shape_ok(K, N)) return 0;
  return (size_t)K * N / (sparse24 ? 4 : 2);
}

size_t marlin_packed_scale_bytes(int K, int N, int group_size) {
  int G = normalise_group(K, N, group_size);
  if (!shape_ok(K, N) || !G) return 0;
  return (size_t)2 * (K / G) * N;
}

size_t marlin_packed_meta_bytes(int K, int N) {
  if (!shape_ok(K, N)) return 0;
  return (size_t)K * N / 8;
}

// Workspace map: [status word, counters: 8192 bytes][partial-tile slots of the warp-MMA kernel and of the tcgen05
// kernel with deferred scales: a region of FIXED size][fp32 accumulation tiles of the tcgen05 kernel].
// The counters and the accumulation tiles are zero at rest and every kernel leaves them that way; the slots are
// written before they are read in every call and keep what the last call left.  Both boundaries are the same for
// every layer, batch size and buffer size, so one buffer may serve calls on different layers one after the other:
// the slots of one call never fall into the accumulation tiles of another.
// two slots per worker, each the widest partial tile: 16 rows x 256 columns (warp-level kernel) or 64 rows x 128
// columns (deferred scales)
constexpr size_t kWsSlotFloats = (size_t)kWsSlotCols * kMaxSlabM > (size_t)128 * kTcdMaxSlabM ? (size_t)kWsSlotCols * kMaxSlabM
                                                                                                : (size_t)128 * kTcdMaxSlabM;
constexpr size_t kWsSlotRegionBytes = (size_t)2 * kMaxWorkers * kWsSlotFloats * sizeof(float);
constexpr size_t kWsTcOff = kWsPartialOff + kWsSlotRegionBytes;
// what the warp-level kernel alone needs: counters and its own slots
constexpr size_t kWarpOnlyWsBytes = kWsPartialOff + (size_t)2 * kMaxWorkers * kWsSlotCols * kMaxSlabM * sizeof(float);
// sparse24: 2:4 layers on the wide layout run on the tcgen05 kernel at every batch size
static size_t tc_tile_bytes(int max_M, int N, bool sparse24) {
  if ((!sparse24 && max_M < tc_min_m()) || N % 256) return 0;
  // one tile of 256 columns x padded rows per column tile; above 128 rows per worker at most (one launch takes all rows)
  return tc_fixup_tiles(max_M, N, kMaxWorkers) * 256 * (size_t)tc_mpad(max_M < kTcMaxSlabM ? max_M : kTcMaxSlabM) *
         sizeof(float);
}
static size_t workspace_bytes_for(int max_M, int K, int N, bool sparse24) {
  (void)K;
  return kWsTcOff + tc_tile_bytes(max_M, N, sparse24);
}

size_t marlin_workspace_bytes(int max_M, int K, int N) {
  if (max_M < 1 || !shape_ok(K, N)) return 0;
  // the larger of what a dense and a 2:4 layer of this shape need (the query does not know which it will be)
  const size_t d = workspace_bytes_for(max_M, K, N, false), sp = workspace_bytes_for(max_M, K, N, true);
  return d > sp ? d : sp;
}

int marlin_pack(const uint32_t* q_kpacked, const void* scales, void* w_packed, void* s_packed, int K, int N,
                int group_size, marlin_stream stream) {
  if (!q_kpacked || !scales || !w_packed || !s_packed) return MARLIN_ERR_NULL;
  if (!shape_ok(K, N)) return MARLIN_ERR_SHAPE;
  int G = normalise_group(K, N, group_size);
  if (!G) return MARLIN_ERR_GROUP;
  if (!aligned16(q_kpacked) || !aligned16(scales) || !aligned16(w_packed) || !aligned16(s_packed))
    return MARLIN_ERR_ALIGN;
  cudaError_t err = launch_pack_dense(const_cast<uint32_t*>(q_kpacked),
                                      static_cast<uint16_t*>(const_cast<void*>(scales)),
                                      static_cast<uint32_t*>(w_packed), static_cast<uint16_t*>(s_packed), K, N, G,
                                      false, static_cast<cudaStream_t>(stream));
  return err == cudaSuccess ? MARLIN_OK : MARLIN_ERR_CUDA;
}

int marlin_quantize_rtn(const void* W, uint32_t* q_kpacked, void* scales, int K, int N, int group_size, int n_grid,
                        int n_candidates, marlin_stream stream) {
  if (!W || !q_kpacked || !scales) return MARLIN_ERR_NULL;
  if (!shape_ok(K, N)) return MARLIN_ERR_SHAPE;
  int G = normalise_group(K, N, group_size);
  if (!G) return MARLIN_ERR_GROUP;
  if (n_grid < 1 || n_candidates < 1 || n_candidates > n_grid) return MARLIN_ERR_SHAPE;
  if (!aligned16(W) || !aligned16(q_kpacked) || !aligned16(scales)) return MARLIN_ERR_ALIGN;
  if ((long long)(K / G) > 65535) return MARLIN_ERR_SHAPE;  // one grid row per group
  cudaError_t err = launch_quantize_rtn(static_cast<const uint16_t*>(W), q_kpacked, static_cast<uint16_t*>(scales), K, N, G,
                                        n_grid, n_candidates, static_cast<cudaStream_t>(stream));
  return err == cudaSuccess ? MARLIN_OK : MARLIN_ERR_CUDA;
}

int marlin_pack_zeros(const uint8_t* zeros, void* z_packed, int K, int N, int group_size, marlin_stream stream) {
  if (!zeros || !z_packed) return MARLIN_ERR_NULL;
  if (!shape_ok(K, N)) return MARLIN_ERR_SHAPE;
  int G = normalise_group(K, N, group_size);
  if (!G) return MARLIN_ERR_GROUP;
  if (!aligned16(zeros) || !aligned16(z_packed)) return MARLIN_ERR_ALIGN;
  cudaError_t err = launch_permute_zeros(const_cast<uint8_t*>(zeros), static_cast<uint16_t*>(z_packed), K, N, G, false,
                                         static_cast<cudaStream_t>(stream));
  return err == cudaSuccess ? MARLIN_OK : MARLIN_ERR_CUDA;
}

int marlin_unpack_zeros(const void* z_packed, uint8_t* zeros, int K, int N, int group_size, marlin_stream stream) {
  if (!zeros || !z_packed) return MARLIN_ERR_NULL;
  if (!shape_ok(K, N)) return MARLIN_ERR_SHAPE;
  int G = normalise_group(K, N, group_size);
  if (!G) return MARLIN_ERR_GROUP;
  if (!aligned16(zeros) || !aligned16(z_packed)) return MARLIN_ERR_ALIGN;
  cudaError_t err = launch_permute_zeros(zeros, static_cast<uint16_t*>(const_cast<void*>(z_packed)), K, N, G, true,
                                         static_cast<cudaStream_t>(stream));
  return err == cudaSuccess ? MARLIN_OK : MARLIN_ERR_CUDA;
}

int marlin_unpack(const void* w_packed, const void* s_packed, uint32_t* q_kpacked, void* scales, int K, int N,
                  int group_size, marlin_stream stream) {
  if (!q_kpacked || !scales || !w_packed || !s_packed) return MARLIN_ERR_NULL;
  if (!shape_ok(K, N)) return MARLIN_ERR_SHAPE;
  int G = normalise_group(K, N, group_size);
  if (!G) return MARLIN_ERR_GROUP;
  if (!aligned16(q_kpacked) || !aligned16(scales) || !aligned16(w_packed) || !aligned16(s_packed))
    return MARLIN_ERR_ALIGN;
  cudaError_t err = launch_pack_dense(q_kpacked, static_cast<uint16_t*>(scales),
                                      static_cast<uint32_t*>(const_cast<void*>(w_packed)),
                                      static_cast<uint16_t*>(const_cast<void*>(s_packed)), K, N, G, true,
                                      static_cast<cudaStream_t>(stream));
  return err == cudaSuccess ? MARLIN_OK : MARLIN_ERR_CUDA;
}

// Shared body of marlin_gemm and marlin_gemm_sparse24 (meta_packed == nullptr: dense).
static int gemm_common(const void* A, const void* w_packed, const void* meta_packed, const void* s_packed, void* C, int M,
                       int K, int N, int group_size, void* workspace, size_t workspace_bytes, marlin_stream stream,
                       bool sparse24, const void* z_packed = nullptr, bool swiglu = false, bool w8 = false,
                       bool warp_kernel_only = false) {
  if (!A || !w_packed || !s_packed || !C || !workspace || (sparse24 && !meta_packed)) return MARLIN_ERR_NULL;
  // layers with zero points: the warp-level kernel up to 16 rows (and in slabs where N is not a multiple of 256), the
  // tcgen05 kernel above
  const bool zero_points = z_packed != nullptr;
  if (zero_points && !aligned16(z_packed)) return MARLIN_ERR_ALIGN;
  if (w8 && N % 256) return MARLIN_ERR_SHAPE;  // 8-bit codes: the tcgen05 kernel alone, at every batch size
  if (M < 1 || !shape_ok(K, N)) return MARLIN_ERR_SHAPE;
  int G = normalise_group(K, N, group_size);
  if (!G) return MARLIN_ERR_GROUP;
  if (!aligned16(A) || !aligned16(w_packed) || !aligned16(s_packed) || !aligned16(C) || !aligned16(workspace) ||
      (sparse24 && !aligned16(meta_packed)))
    return MARLIN_ERR_ALIGN;
  // (warp_kernel_only: the built-in array of marlin_gemm_static_ws, which holds the counters and the slots of the
  // warp-level kernel and nothing else; its caller has checked that this kernel serves the call)
  if (workspace_bytes < (warp_kernel_only ? kWarpOnlyWsBytes : workspace_bytes_for(M, K, N, sparse24 || G < kTileK || zero_points || w8)))
    return MARLIN_ERR_WORKSPACE;
  DeviceInfo info;
  int st = device_info(&info);
  if (st != MARLIN_OK) return st;
  if (info.cc_major != 10) return MARLIN_ERR_ARCH;

  uint8_t* ws = static_cast<uint8_t*>(workspace);
  int m0 = 0;
  while (m0 < M) {
    const int rem = M - m0;
    // Which kernel takes the next rows.  Up to 16: the warp-level kernel.  Above: the tcgen05 kernel with
    // in-loop scales (N a multiple of 256; all rows in one launch, slabs of 128 rows sharing its stripes), or the
    // one with deferred scales (64 rows per launch, N a multiple of 128).  What none of them serves (2:4 layers, other N) goes through the warp-level
    // kernel in slabs of 16 rows.
    const int tmode = tcd_mode();
    // 2:4 layers whose N is a multiple of 256 are packed in the wide layout, which only the tcgen05 kernel reads:
    // it takes every batch size there
    const bool tc_ok = tc_path_supported(1, K, N);
    // groups of 64 or 32 rows likewise (accepted only where N is a multiple of 256)
    const bool small_groups = G < kTileK || w8;
    // (the kernel with deferred scales has no fused activation: those layers go through the warp-level kernel then)
    const bool use_tcd = !warp_kernel_only && !swiglu && !sparse24 && !small_groups && !zero_points &&
                         tcd_path_supported(1, K, N) && (tmode == 1 || (tmode == 2 && rem >= tc_min_m() && !tc_ok));
    const bool use_tc = !warp_kernel_only && !use_tcd && tc_ok && (sparse24 || small_groups || rem >= tc_min_m());
    const int m_slab = use_tcd ? (rem < kTcdMaxSlabM ? rem : kTcdMaxSlabM)
                               : use_tc ? (rem < tc_max_rows(K, N, info.sm_count) ? rem : tc_max_rows(K, N, info.sm_count))
                                        : (rem < kMaxSlabM ? rem : kMaxSlabM);
    GemmParams p;
    p.A = static_cast<const uint16_t*>(A) + (size_t)m0 * K;
    p.wq = static_cast<const uint8_t*>(w_packed);
    p.sq = static_cast<const uint8_t*>(s_packed);
    p.meta = static_cast<const uint8_t*>(meta_packed);
    p.zq = static_cast<const uint8_t*>(z_packed);
    p.C = static_cast<uint16_t*>(C) + (size_t)m0 * (swiglu ? N / 2 : N);
    p.swiglu = swiglu ? 1 : 0;
    p.M = m_slab;
    p.K = K;
    p.N = N;
    p.kb = (uint32_t)(K / kTileK);
    p.kb_per_group = G >= kTileK ? G / kTileK : 1;
    p.sub_groups = G >= kTileK ? 1 : kTileK / G;
    p.group_shift = -1;
    for (int sh = 0; sh < 31; ++sh)
      if ((1 << sh) == p.kb_per_group) p.group_shift = sh;
    p.grouped = (G != K || zero_points) ? 1 : 0;  // zero points travel with the scale rows of the in-loop path
    p.status = reinterpret_cast<int*>(ws + kWsStatusOff);
    p.counters = reinterpret_cast<int*>(ws + kWsCounterOff);
    p.partials = reinterpret_cast<float*>(ws + kWsPartialOff);
    p.tc_tiles = use_tc ? reinterpret_cast<float*>(ws + kWsTcOff) : nullptr;
    p.split = 0;
    p.whole = 0;
    p.slabs = 1;
    p.cluster = 0;
    p.slot_floats = kWsSlotCols * kMaxSlabM;
    if (use_tcd) {
      if (launch_gemm_tcd(p, info.sm_count, static_cast<cudaStream_t>(stream)) != cudaSuccess) return MARLIN_ERR_CUDA;
    } else if (use_tc) {
      if (launch_gemm_dense_tc(p, info.sm_count, sparse24, static_cast<cudaStream_t>(stream), w8) != cudaSuccess)
        return MARLIN_ERR_CUDA;
    } else {
      DensePlan plan;
      const int fmt = sparse24 ? 1 : (zero_points ? 2 : 0);
      if (!make_dense_plan(m_slab, K, N, info.sm_count, fmt, &plan)) return MARLIN_ERR_SHAPE;
      p.ncols = plan.ncols;
      p.units = (uint32_t)plan.units;
      p.workers = (uint32_t)plan.workers;
      p.split = (uint32_t)plan.split;
      p.stages = plan.stages;
      p.stage_bytes = plan.stage_bytes;
      if (launch_gemm_dense(plan, p, fmt, static_cast<cudaStream_t>(stream)) != cudaSuccess) return MARLIN_ERR_CUDA;
    }
    m0 += m_slab;
  }
  return MARLIN_OK;
}

int marlin_gemm(const void* A, const void* w_packed, const void* s_packed, void* C, int M, int K, int N,
                int group_size, void* workspace, size_t workspace_bytes, marlin_stream stream) {
  return gemm_common(A, w_packed, nullptr, s_packed, C, M, K, N, group_size, workspace, workspace_bytes, stream, false);
}

int marlin_gemm_swiglu(const void* A, const void* w_packed, const void* s_packed, void* H, int M, int K, int N,
                       int group_size, void* workspace, size_t workspace_bytes, marlin_stream stream) {
  return gemm_common(A, w_packed, nullptr, s_packed, H, M, K, N, group_size, workspace, workspace_bytes, stream, false,
                     nullptr, true);
}

int marlin_interleave_gate_up(const uint32_t* q_gate, const void* s_gate, const uint32_t* q_up, const void* s_up,
                              uint32_t* q_out, void* s_out, int K, int I, int group_size, marlin_stream stream) {
  if (!q_gate || !s_gate || !q_up || !s_up || !q_out || !s_out) return MARLIN_ERR_NULL;
  if (I < 32 || I % 32 || !shape_ok(K, 2 * I)) return MARLIN_ERR_SHAPE;
  int G = normalise_group(K, 2 * I, group_size);
  if (!G) return MARLIN_ERR_GROUP;
  if (!aligned16(q_gate) || !aligned16(s_gate) || !aligned16(q_up) || !aligned16(s_up) || !aligned16(q_out) ||
      !aligned16(s_out))
    return MARLIN_ERR_ALIGN;
  cudaError_t err = launch_interleave_gate_up(q_gate, static_cast<const uint16_t*>(s_gate), q_up,
                                              static_cast<const uint16_t*>(s_up), q_out, static_cast<uint16_t*>(s_out), K, I,
                                              G, static_cast<cudaStream_t>(stream));
  return err == cudaSuccess ? MARLIN_OK : MARLIN_ERR_CUDA;
}

int marlin_mlp_swiglu(const void* A, const void* w_gate_up, const void* s_gate_up, const void* w_down, const void* s_down,
                      void* H, void* C, int M, int K, int I, int N, int group_size, void* workspace, size_t workspace_bytes,
                      marlin_stream stream) {
  // two launches: gate_up with the activation fused into its epilogue, then down; the second starts under
  // programmatic dependent launch and prefetches its weights while the first finishes
  int st = marlin_gemm_swiglu(A, w_gate_up, s_gate_up, H, M, K, 2 * I, group_size, workspace, workspace_bytes, stream);
  if (st != MARLIN_OK) return st;
  return marlin_gemm(H, w_down, s_down, C, M, I, N, group_size, workspace, workspace_bytes, stream);
}

size_t marlin_packed_weight_bytes_w8(int K, int N) {
  if (!shape_ok(K, N) || N % 256) return 0;
  return (size_t)K * N;
}

int marlin_pack_w8(const uint8_t* q8, const void* scales, void* w_packed, void* s_packed, int K, int N, int group_size,
                   marlin_stream stream) {
  if (!q8 || !scales || !w_packed || !s_packed) return MARLIN_ERR_NULL;
  if (!shape_ok(K, N) || N % 256) return MARLIN_ERR_SHAPE;
  int G = normalise_group(K, N, group_size);
  if (!G) return MARLIN_ERR_GROUP;
  if (!aligned16(q8) || !aligned16(scales) || !aligned16(w_packed) || !aligned16(s_packed)) return MARLIN_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (launch_pack_w8(const_cast<uint8_t*>(q8), static_cast<uint8_t*>(w_packed), K, N, false, st) != cudaSuccess)
    return MARLIN_ERR_CUDA;
  cudaError_t err = launch_permute_scales(static_cast<uint16_t*>(const_cast<void*>(scales)), static_cast<uint16_t*>(s_packed),
                                          K, N, G, false, st);
  return err == cudaSuccess ? MARLIN_OK : MARLIN_ERR_CUDA;
}

int marlin_unpack_w8(const void* w_packed, const void* s_packed, uint8_t* q8, void* scales, int K, int N, int group_size,
                     marlin_stream stream) {
  if (!q8 || !scales || !w_packed || !s_packed) return MARLIN_ERR_NULL;
  if (!shape_ok(K, N) || N % 256) return MARLIN_ERR_SHAPE;
  int G = normalise_group(K, N, group_size);
  if (!G) return MARLIN_ERR_GROUP;
  if (!aligned16(q8) || !aligned16(scales) || !aligned16(w_packed) || !aligned16(s_packed)) return MARLIN_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (launch_pack_w8(q8, static_cast<uint8_t*>(const_cast<void*>(w_packed)), K, N, true, st) != cudaSuccess)
    return MARLIN_ERR_CUDA;
  cudaError_t err = launch_permute_scales(static_cast<uint16_t*>(scales), static_cast<uint16_t*>(const_cast<void*>(s_packed)),
                                          K, N, G, true, st);
  return err == cudaSuccess ? MARLIN_OK : MARLIN_ERR_CUDA;
}

int marlin_gemm_w8(const void* A, const void* w_packed, const void* s_packed, void* C, int M, int K, int N, int group_size,
                   void* workspace, size_t workspace_bytes, marlin_stream stream) {
  return gemm_common(A, w_packed, nullptr, s_packed, C, M, K, N, group_size, workspace, workspace_bytes, stream, false,
                     nullptr, false, true);
}

int marlin_gemm_zp(const void* A, const void* w_packed, const void* s_packed, const void* z_packed, void* C, int M, int K,
                   int N, int group_size, void* workspace, size_t workspace_bytes, marlin_stream stream) {
  if (!z_packed) return MARLIN_ERR_NULL;
  return gemm_common(A, w_packed, nullptr, s_packed, C, M, K, N, group_size, workspace, workspace_bytes, stream, false,
                     z_packed);
}

// ---- the variant with a built-in workspace ------------------------------------------------------
// Scratch for marlin_gemm_static_ws: the workspace of one layer call with M <= MARLIN_STATIC_WS_MAX_M,
// as a file-scope device array.  In host code the name `g_static_workspace` is only a handle for
// cudaGetSymbolAddress; the kernels get the device address that call returns.
static_assert(MARLIN_STATIC_WS_MAX_M <= kMaxSlabM, "the built-in workspace serves the warp-level kernel alone");
constexpr size_t kStaticWsBytes = kWarpOnlyWsBytes;
static __device__ __align__(256) unsigned char g_static_workspace[kStaticWsBytes];

int marlin_gemm_static_ws(const void* A, const void* w_packed, const void* s_packed, void* C, int M, int K, int N,
                          int group_size, marlin_stream stream) {
  // the argument checks of marlin_gemm first: nothing is queued for a call that is going to be refused
  if (!A || !w_packed || !s_packed || !C) return MARLIN_ERR_NULL;
  if (M < 1 || M > MARLIN_STATIC_WS_MAX_M || !shape_ok(K, N)) return MARLIN_ERR_SHAPE;
  const int Gs = normalise_group(K, N, group_size);
  if (!Gs || Gs < kTileK) return MARLIN_ERR_GROUP;  // groups of 64 / 32 rows need the tcgen05 kernel's share of a workspace
  if (!aligned16(A) || !aligned16(w_packed) || !aligned16(s_packed) || !aligned16(C)) return MARLIN_ERR_ALIGN;
  DeviceInfo info;
  int st = device_info(&info);
  if (st != MARLIN_OK) return st;
  if (info.cc_major != 10) return MARLIN_ERR_ARCH;
  static void* device_address[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return MARLIN_ERR_CUDA;
  if (!device_address[dev]) {
    // once per device, with that device current: where the array lives on this GPU
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_workspace) != cudaSuccess || !ptr) return MARLIN_ERR_CUDA;
    device_address[dev] = ptr;
  }
  uint8_t* ws = static_cast<uint8_t*>(device_address[dev]);
  // the array keeps whatever the last call left: the arrival counters must start at zero (the partial-tile
  // slots behind them are written before they are read; the status word is left alone)
  if (cudaMemsetAsync(ws + kWsCounterOff, 0, kWsPartialOff - kWsCounterOff, static_cast<cudaStream_t>(stream)) !=
      cudaSuccess)
    return MARLIN_ERR_CUDA;
  return gemm_common(A, w_packed, nullptr, s_packed, C, M, K, N, group_size, ws, kStaticWsBytes, stream, false, nullptr,
                     false, false, true);
}

int marlin_pack_sparse24(const uint32_t* qc_kpacked, const uint8_t* idx, const void* scales, void* w_packed,
                         void* meta_packed, void* s_packed, int K, int N, int group_size, marlin_stream stream) {
  if (!qc_kpacked || !idx || !scales || !w_packed || !meta_packed || !s_packed) return MARLIN_ERR_NULL;
  if (!shape_ok(K, N)) return MARLIN_ERR_SHAPE;
  int G = normalise_group(K, N, group_size);
  if (!G) return MARLIN_ERR_GROUP;
  if (!aligned16(qc_kpacked) || !aligned16(idx) || !aligned16(scales) || !aligned16(w_packed) ||
      !aligned16(meta_packed) || !aligned16(s_packed))
    return MARLIN_ERR_ALIGN;
  cudaError_t err = launch_pack_sparse24(
      const_cast<uint32_t*>(qc_kpacked), const_cast<uint8_t*>(idx), static_cast<uint16_t*>(const_cast<void*>(scales)),
      static_cast<uint32_t*>(w_packed), static_cast<uint32_t*>(meta_packed), static_cast<uint16_t*>(s_packed), K, N, G,
      false, static_cast<cudaStream_t>(stream));
  return err == cudaSuccess ? MARLIN_OK : MARLIN_ERR_CUDA;
}

int marlin_unpack_sparse24(const void* w_packed, const void* meta_packed, const void* s_packed, uint32_t* qc_kpacked,
                           uint8_t* idx, void* scales, int K, int N, int group_size, marlin_stream stream) {
  if (!qc_kpacked || !idx || !scales || !w_packed || !meta_packed || !s_packed) return MARLIN_ERR_NULL;
  if (!shape_ok(K, N)) return MARLIN_ERR_SHAPE;
  int G = normalise_group(K, N, group_size);
  if (!G) return MARLIN_ERR_GROUP;
  if (!aligned16(qc_kpacked) || !aligned16(idx) || !aligned16(scales) || !aligned16(w_packed) ||
      !aligned16(meta_packed) || !aligned16(s_packed))
    return MARLIN_ERR_ALIGN;
  cudaError_t err = launch_pack_sparse24(
      qc_kpacked, idx, static_cast<uint16_t*>(scales), static_cast<uint32_t*>(const_cast<void*>(w_packed)),
      static_cast<uint32_t*>(const_cast<void*>(meta_packed)), static_cast<uint16_t*>(const_cast<void*>(s_packed)), K, N,
      G, true, static_cast<cudaStream_t>(stream));
  return err == cudaSuccess ? MARLIN_OK : MARLIN_ERR_CUDA;
}

int marlin_gemm_sparse24(const void* A, const void* w_packed, const void* meta_packed, const void* s_packed, void* C,
                         int M, int K, int N, int group_size, void* workspace, size_t workspace_bytes,
                         marlin_stream stream) {
  return gemm_common(A, w_packed, meta_packed, s_packed, C, M, K, N, group_size, workspace, workspace_bytes, stream,
                     true);
}

int marlin_read_status(const void* workspace, marlin_stream stream) {
  if (!workspace) return MARLIN_ERR_NULL;
  int host_status = 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(&host_status, static_cast<const uint8_t*>(workspace) + kWsStatusOff, sizeof(int),
                      cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return MARLIN_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return MARLIN_ERR_CUDA;
  return host_status;
}

int marlin_plan_stripes(int M, int K, int N, int sm_count, int* n_tile, int* workers, int64_t* bounds, int cap) {
  if (!n_tile || !workers || !bounds) return MARLIN_ERR_NULL;
  if (M < 1 || !shape_ok(K, N)) return MARLIN_ERR_SHAPE;
  DensePlan plan;
  const int m_slab = M < kMaxSlabM ? M : kMaxSlabM;
  if (!make_dense_plan(m_slab, K, N, sm_count, false, &plan)) return MARLIN_ERR_SHAPE;
  if (cap < plan.workers + 1) return MARLIN_ERR_SHAPE;
  *n_tile = plan.nw * kChunkN;
  *workers = plan.workers;
  for (int w = 0; w <= plan.workers; ++w) {
    if (plan.split) {
      const long long t = w / plan.split, r = w % plan.split;
      bounds[w] = t * plan.kb + (r * plan.kb) / plan.split;
    } else {
      bounds[w] = stripe_begin(w, plan.units, plan.workers);
    }
  }
  return MARLIN_OK;
}

}  // extern "C"
