/*
 * marlin_b200 -- W4A16 linear layer for NVIDIA B200 (sm_100a), C ABI.
 *
 *     C[M x N] (fp16) = A[M x K] (fp16) . dequant(Wq[K x N] int4, fp16 scales),  fp32 accumulation
 *     dequant:  W[k][n] = (Q[k][n] - 8) * S[k / G][n],  Q in 0..15
 *
 * The operation is the mixed-precision layer of the MARLIN paper (arxiv 2408.11743), Section 3.4
 * "Kernel Design": A in fp16, B a K x N INT4 matrix, symmetrically quantised, with one fp16 scale per
 * output column or per G consecutive weights of a column (ceil(K/G) * N scales).  The 2:4 variant is
 * Section 4 ("The Sparse-MARLIN Kernel"): groups of four along K, two values kept, 2-bit positions.
 *
 * General rules
 *   - Every pointer named *device* is a CUDA device pointer owned by the caller, 16-byte aligned,
 *     valid on the current device until the work queued on `stream` has finished.  Host pointers
 *     are said to be host pointers.  Buffers of one call must not overlap.
 *   - Calls are asynchronous on `stream`; nothing synchronises, nothing is allocated, nothing throws.
 *     Every function that can fail returns a marlin_status; 0 is success.
 *   - There is no CPU path and no other-architecture path: on a device that is not compute
 *     capability 10.x the calls return MARLIN_ERR_ARCH.
 *   - Shapes: K % 128 == 0, K <= 2^20, N % 64 == 0, N <= 65536, M >= 1 (any number of rows: a call splits
 *     them over as many launches as it needs).  group_size is a multiple of 128 that divides K, or K itself
 *     (also written -1): one scale per column; on layers whose N is a multiple of 256 also 64 or 32 (Section 2.3,
 *     group quantization with smaller groups; other values return MARLIN_ERR_GROUP).
 *   - The packed device layout is opaque (the design notes of this repository describe it); only marlin_pack* writes it and
 *     only marlin_unpack* / marlin_gemm* read it.
 */
#ifndef MARLIN_B200_H_
#define MARLIN_B200_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define MARLIN_API __attribute__((visibility("default")))
#else
#define MARLIN_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  MARLIN_OK = 0,
  MARLIN_ERR_NULL = 1,           /* a required pointer is NULL                                  */
  MARLIN_ERR_SHAPE = 2,          /* M, K or N out of range or not a multiple of the tile sizes  */
  MARLIN_ERR_GROUP = 3,          /* group_size not supported for this K                         */
  MARLIN_ERR_ALIGN = 4,          /* a device pointer is not 16-byte aligned                     */
  MARLIN_ERR_WORKSPACE = 5,      /* workspace smaller than marlin_workspace_bytes()             */
  MARLIN_ERR_ARCH = 6,           /* current device is not sm_100                                */
  MARLIN_ERR_CUDA = 7,           /* a CUDA runtime call or the launch failed                    */
  MARLIN_ERR_DEVICE_TIMEOUT = 8  /* a bounded wait inside a kernel expired (see marlin_read_status) */
} marlin_status;

/* A CUDA stream handle (cudaStream_t) passed as an opaque pointer; NULL is the default stream. */
typedef void* marlin_stream;

MARLIN_API const char* marlin_status_string(int status);

/* ---- sizes (host arithmetic only; valid without a GPU) ------------------------------------- */

/* Bytes of the packed weight buffer: K*N/2 dense; K*N/4 when sparse24 != 0.  0 on a bad shape. */
MARLIN_API size_t marlin_packed_weight_bytes(int K, int N, int sparse24);
/* Bytes of the packed scale buffer: 2 * (K/G) * N.  0 on a bad shape or group size. */
MARLIN_API size_t marlin_packed_scale_bytes(int K, int N, int group_size);
/* Bytes of the packed 2:4 metadata buffer: K*N/8 (2 bits per kept value). */
MARLIN_API size_t marlin_packed_meta_bytes(int K, int N);
/* Bytes of the workspace marlin_gemm* needs for any M <= max_M on this K x N layer.
 * The workspace holds a status word, per-column-tile arrival counters and the fp32 partial tiles
 * of the stripe fix-up (the global reduction of Section 3.4 "Striped Partitioning"): a part of fixed size
 * (10.5 MB) and one that grows with N and with max_M up to 128 rows and, above, with the number of
 * (column tile, 128-row slab) pairs up to the number of CTAs (at most 20 MB more).
 * The caller zeroes it ONCE after allocation (cudaMemset); every call leaves the counters zero.
 * One workspace must not be used by two calls that can run at the same time.  It may serve calls on
 * different layers, formats and batch sizes one after the other (one stream, or ordered by events) if it
 * has the largest of their sizes: the parts lie at the same offsets for every call. */
MARLIN_API size_t marlin_workspace_bytes(int max_M, int K, int N);

/* ---- offline quantiser (Section 3.5 (a): group scales picked by a search over group-wise clipping
 *      thresholds; here without calibration data: round to nearest, least squared weight error) ------ */

/* fp16 weights -> canonical 4-bit codes and fp16 group scales, the inputs of marlin_pack.
 *   W             device, fp16 [K][N] row-major, finite values
 *   q_kpacked     device, out, uint32 [K/8][N]: nibble j of word (kb, n) = code of row 8*kb + j, codes 0..15 = q
 *   scales        device, out, fp16 [K/G][N]
 *   n_grid, n_candidates   1 <= n_candidates <= n_grid: candidate t = 0 .. n_candidates-1 clips the group's range
 *                 to r_t = 1 - t / n_grid of its largest magnitude a (n_candidates = 1: plain round to nearest)
 * Per group of G rows of a column: s_t = fp16(2 a r_t / 15) (never zero: at least the smallest positive fp16),
 * q_i = clamp(round_half_even(w_i / s_t), -8, 7) + 8, and the candidate with the least sum of squared errors
 * (w_i - (q_i - 8) s_t)^2 wins, the first one on ties.  All of it in fp32 with a fixed order of operations (see
 * csrc/quantize.cu), so the outputs are reproducible bit for bit.  Shapes and group sizes as for marlin_pack;
 * pointers 16-byte aligned; errors are returned before anything is queued. */
MARLIN_API int marlin_quantize_rtn(const void* W, uint32_t* q_kpacked, void* scales, int K, int N, int group_size,
                        int n_grid, int n_candidates, marlin_stream stream);

/* ---- offline re-layout (Section 3.4 "Maximizing Loading Bandwidth", "Dequantization and Tensor
 *      Cores": weights are static, so they are reshuffled once into the order the kernel streams) -- */

/* Dense pack.
 *   q_kpacked  device, uint32 [K/8][N]: canonical codes, nibble j of word (kb, n) = Q[8*kb + j][n]
 *   scales     device, fp16   [K/G][N] row-major
 *   w_packed   device, out, marlin_packed_weight_bytes(K, N, 0) bytes
 *   s_packed   device, out, marlin_packed_scale_bytes(K, N, G) bytes
 * Integer-only permutation; unpack(pack(x)) == x bit for bit. */
MARLIN_API int marlin_pack(const uint32_t* q_kpacked, const void* scales, void* w_packed, void* s_packed,
                int K, int N, int group_size, marlin_stream stream);

/* Inverse of marlin_pack: writes the canonical forms back. */
MARLIN_API int marlin_unpack(const void* w_packed, const void* s_packed, uint32_t* q_kpacked, void* scales,
                  int K, int N, int group_size, marlin_stream stream);

/* Zero points for layers quantised asymmetrically, W = (q - z) * s with one integer z in 0..15 per scale group
 * (Section 2.3 "uniform quantization": a zero point and a scale per group; the integer form is the one of the
 * activation-aware format the paper names in Section 6).  Codes and scales go through marlin_pack as usual.
 *   zeros      device, uint8 [K/G][N] row-major, values 0..15
 *   z_packed   device, out, marlin_packed_scale_bytes(K, N, G) bytes (fp16 values in the order of the packed scales)
 * Shapes and group sizes as for marlin_pack. */
MARLIN_API int marlin_pack_zeros(const uint8_t* zeros, void* z_packed, int K, int N, int group_size, marlin_stream stream);
MARLIN_API int marlin_unpack_zeros(const void* z_packed, uint8_t* zeros, int K, int N, int group_size, marlin_stream stream);

/* ---- the layer (Section 3.4, all paragraphs: weight streaming, dequantisation, tensor-core
 *      product, striped partition with global reduction) ----------------------------------------- */

/* C = A . dequant(W).
 *   A          device, fp16 [M][K] row-major
 *   w_packed, s_packed   device, from marlin_pack with the same K, N, group_size
 *   C          device, out, fp16 [M][N] row-major, every element written
 *   workspace  device, at least marlin_workspace_bytes(M, K, N) bytes, zeroed once by the caller
 * Accumulation is fp32 (also across stripes) and the result is rounded to fp16 once (nearest even).  The
 * weights reach the tensor cores as exact integers q - 8 (warp-level kernel, up to 16 rows: scales applied to
 * the fp32 sums per group) or as fp16((q - 8) * s) (tcgen05 kernel with in-loop scales, from 17 rows: one more
 * rounding of 2^-11 per weight, as in the paper's kernel).
 * Up to 16 rows the warp-level kernel runs and the same inputs give the same bits on every call.
 * From 17 rows a tcgen05 kernel takes over.  Where N is a multiple of 256 one launch takes all rows: above
 * 128 rows the layer is replicated in the numbering of the work units, once per slab of 128 rows (Section 3.4,
 * last paragraph), and the stripes of the CTAs run over (column tile, slab, k-block), so the weights come from
 * DRAM once and from the L2 after that.  Where N is a multiple of 128 only, 64 rows per launch; any other N goes
 * through the warp-level kernel in slabs of 16 rows.  Groups of 64 or 32 rows run on the tcgen05 kernel at
 * every batch size.  Where the 256-column tcgen05 kernel adds the partial sums of a column tile shared by
 * several CTAs through the L2 (up to 32 rows, above 128 rows, or shapes whose CTAs do not fit as one wave of
 * thread-block clusters) the fp32 additions happen in arrival order, so the last bit of an fp16 result can
 * differ between two calls; everywhere else the order is fixed.
 * Errors: argument checks return before anything is queued.  A kernel whose bounded waits expire
 * sets the workspace status word; read it with marlin_read_status. */
MARLIN_API int marlin_gemm(const void* A, const void* w_packed, const void* s_packed, void* C,
                int M, int K, int N, int group_size,
                void* workspace, size_t workspace_bytes, marlin_stream stream);


/* ---- the gated MLP of a decoder layer as a chain of two launches (Section 5.1 names the per-kernel overheads on
 *      real layer shapes; fusing the activation removes one launch and the round trip of the wide intermediate) -- */

/* Gate and up projections of one MLP side by side, in the column order the fused epilogue expects: output column
 * n = 16 b + r holds gate channel 8 b + r for r < 8 and up channel 8 b + r - 8 otherwise.
 *   q_gate, q_up   device, uint32 [K/8][I] canonical codes;   s_gate, s_up   device, fp16 [K/G][I]
 *   q_out          device, out, uint32 [K/8][2 I];            s_out          device, out, fp16 [K/G][2 I]
 * Feed q_out, s_out to marlin_pack with N = 2 I.  I % 32 == 0. */
MARLIN_API int marlin_interleave_gate_up(const uint32_t* q_gate, const void* s_gate, const uint32_t* q_up, const void* s_up,
                              uint32_t* q_out, void* s_out, int K, int I, int group_size, marlin_stream stream);

/* marlin_gemm on such a layer (N = 2 I columns) with the activation fused into the epilogue:
 *   H[m][c] = fp16( silu(g) * u ),  g = fp16(A . W)[m][gate channel c],  u = fp16(A . W)[m][up channel c],
 * silu(g) = g / (1 + exp(-g)) in fp32.  H is device, out, fp16 [M][N/2] row-major.  Everything else as marlin_gemm
 * (the product is rounded to fp16 before the activation, as it would be if H were computed from a stored C). */
MARLIN_API int marlin_gemm_swiglu(const void* A, const void* w_packed, const void* s_packed, void* H, int M, int K, int N,
                       int group_size, void* workspace, size_t workspace_bytes, marlin_stream stream);

/* C = (silu(A . W_gate) * (A . W_up)) . W_down: marlin_gemm_swiglu into H (device scratch, fp16 [M][I]), then
 * marlin_gemm of H with the down projection (I x N).  One workspace serves both launches (they run one after the
 * other on `stream`): at least max(marlin_workspace_bytes(M, K, 2 I), marlin_workspace_bytes(M, I, N)) bytes. */
MARLIN_API int marlin_mlp_swiglu(const void* A, const void* w_gate_up, const void* s_gate_up, const void* w_down,
                      const void* s_down, void* H, void* C, int M, int K, int I, int N, int group_size,
                      void* workspace, size_t workspace_bytes, marlin_stream stream);

/* ---- 8-bit weights (Section 6 names other formats the approach extends to): W = (q - 128) * s, q in 0..255 ------ */

/* q8: device, uint8 [K][N] row-major codes; scales as for marlin_pack.  w_packed: marlin_packed_weight_bytes_w8(K, N)
 * = K * N bytes.  N % 256 == 0 (these layers run on the tcgen05 kernel at every batch size).  Integer-only
 * permutation; marlin_unpack_w8 is its inverse bit for bit. */
MARLIN_API size_t marlin_packed_weight_bytes_w8(int K, int N);
MARLIN_API int marlin_pack_w8(const uint8_t* q8, const void* scales, void* w_packed, void* s_packed, int K, int N,
                   int group_size, marlin_stream stream);
MARLIN_API int marlin_unpack_w8(const void* w_packed, const void* s_packed, uint8_t* q8, void* scales, int K, int N,
                     int group_size, marlin_stream stream);
/* C = A . W as marlin_gemm; the conversion places a code byte under the exponent of 1024 and subtracts 1152 (the
 * 8-bit form of the exponent trick of Section 3.4 "Dequantization and Tensor Cores"), scales in the loop. */
MARLIN_API int marlin_gemm_w8(const void* A, const void* w_packed, const void* s_packed, void* C, int M, int K, int N,
                   int group_size, void* workspace, size_t workspace_bytes, marlin_stream stream);

/* The layer with zero points: C = A . W, W[k][n] = (q[k][n] - z[k/G][n]) * s[k/G][n].  Arguments as marlin_gemm, plus
 * z_packed from marlin_pack_zeros.  Up to 16 rows (and in slabs of 16 rows where N is not a multiple of 256) the
 * warp-level kernel runs: the weights enter the MMAs as for the symmetric layer and one more MMA per 16 rows of k,
 * with an all-ones weight operand, gives sum_k a[k][m] per group, so that the group closes with
 * s * (sum_k a (q - 8) + (8 - z) sum_k a).  Above, the tcgen05 kernel, where the zero point replaces the constant 8
 * inside the conversion (the subtrahend of the exponent trick of Section 3.4 "Dequantization and Tensor Cores"
 * becomes 1024 + z): no extra instruction per weight.  workspace: marlin_workspace_bytes(M, K, N). */
MARLIN_API int marlin_gemm_zp(const void* A, const void* w_packed, const void* s_packed, const void* z_packed, void* C,
                   int M, int K, int N, int group_size, void* workspace, size_t workspace_bytes,
                   marlin_stream stream);

/* The same layer for callers that cannot allocate device memory or carry a workspace pointer
 * around: for example a plug-in that runs inside another framework's pre-captured execution plan,
 * or a constrained runtime where cudaMalloc is forbidden after start-up.  (The paper has no
 * counterpart; this is a convenience of this library.)
 *
 * Works like marlin_gemm, but the fix-up workspace is a fixed array inside the library's device
 * image (about 5 MB, held by every GPU that loads the library until the process exits), so only
 * M <= MARLIN_STATIC_WS_MAX_M is accepted; larger M returns MARLIN_ERR_SHAPE.  The call allocates
 * nothing: no cudaMalloc, no cudaFree, no library routine that allocates.
 *
 * The first call on each device looks up the device address of that array (with that device
 * current) and remembers it; make this first call outside any stream capture.  Every call clears
 * the arrival counters of the array on `stream` before the kernels run (the array keeps whatever
 * the previous call left), and all calls on one device share the one array: two such calls that
 * can overlap on the GPU (two streams, or two host threads) race with each other and must be
 * serialised by the caller.
 * Errors: the argument checks of marlin_gemm, made before anything is queued; MARLIN_ERR_CUDA if
 * the address lookup or the clearing fails.  The array's status word is private to the library:
 * a bounded wait that expires inside a kernel of this entry point is NOT reported to the caller
 * (use marlin_gemm with a workspace of your own and marlin_read_status where that matters). */
#define MARLIN_STATIC_WS_MAX_M 16
MARLIN_API int marlin_gemm_static_ws(const void* A, const void* w_packed, const void* s_packed, void* C,
                                     int M, int K, int N, int group_size, marlin_stream stream);

/* ---- 2:4 structured-sparse variant (Section 4: values structure + metadata indices) ------------ */

/* Pack the compressed form.
 *   qc_kpacked device, uint32 [K/16][N]: kept codes Qc[K/2][N], nibble j of word (r, n) = Qc[8r+j][n]
 *   idx        device, uint8  [K/2][N]: position 0..3 of kept value t inside group t/2 of four rows
 *              along K; idx[2u][n] < idx[2u+1][n]
 *   scales     device, fp16 [K/G][N], groups over the ORIGINAL K
 *   outputs    w_packed (K*N/4 bytes), meta_packed (K*N/8 bytes), s_packed (2*(K/G)*N bytes) */
MARLIN_API int marlin_pack_sparse24(const uint32_t* qc_kpacked, const uint8_t* idx, const void* scales,
                         void* w_packed, void* meta_packed, void* s_packed,
                         int K, int N, int group_size, marlin_stream stream);

MARLIN_API int marlin_unpack_sparse24(const void* w_packed, const void* meta_packed, const void* s_packed,
                           uint32_t* qc_kpacked, uint8_t* idx, void* scales,
                           int K, int N, int group_size, marlin_stream stream);

/* C = A . dequant(expand(W)) with the pruned positions contributing zero.  Layers whose N is a multiple of 256
 * run on the sparse tcgen05 instruction (tcgen05.mma.sp) at every batch size, all rows in one launch (slabs of
 * 128 rows as in marlin_gemm), reading the compressed weights from DRAM once; other N on the warp-level sparse
 * MMA in slabs of 16 rows. */
MARLIN_API int marlin_gemm_sparse24(const void* A, const void* w_packed, const void* meta_packed,
                         const void* s_packed, void* C, int M, int K, int N, int group_size,
                         void* workspace, size_t workspace_bytes, marlin_stream stream);

/* Synchronises `stream`, then returns the device-side status word of `workspace`
 * (MARLIN_OK, or MARLIN_ERR_DEVICE_TIMEOUT if a kernel gave up a bounded wait), or
 * MARLIN_ERR_CUDA if the stream reports an error.  The status word is sticky until the
 * workspace is zeroed again. */
MARLIN_API int marlin_read_status(const void* workspace, marlin_stream stream);

/* ---- host-side planning, exposed for inspection and tests (no GPU needed) ----------------------- */

/* The partition of Section 3.4 "Striped Partitioning" as the warp-level kernel uses it for this shape:
 * the (column tile, 128-row k-block) units of the weight matrix are numbered column tile by column tile,
 * top to bottom, and worker i of `workers` owns units [bounds[i], bounds[i+1]).  Two forms: where the
 * column tiles divide the SMs well, every tile is cut into the same number of equal k-ranges, one per
 * worker (no stripe crosses a tile boundary); otherwise the units are cut into `workers` even stripes,
 * the paper's form.  Fills n_tile (columns per tile: 64, 128 or 256), workers (<= sm_count) and
 * bounds[0..workers] (host pointers; `cap` entries available in bounds).
 * Returns MARLIN_ERR_SHAPE if cap is too small or the shape is invalid. */
MARLIN_API int marlin_plan_stripes(int M, int K, int N, int sm_count, int* n_tile, int* workers,
                        int64_t* bounds, int cap);

#ifdef __cplusplus
}
#endif
#endif /* MARLIN_B200_H_ */
