/*
 * CPU oracle for the W4A16 linear layer of the MARLIN paper (arxiv 2408.11743).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition of what the
 * GPU library must compute.  It shares no code, table or constant with the CUDA
 * path and is never called by it.  Only the test-suite, the smoke check and the
 * benchmark's CPU-baseline leg may load it.
 *
 * What it computes (Section 3.4 "Kernel Design", first paragraph: A is fp16 M x K,
 * B is K x N INT4, symmetrically quantised, one fp16 scale per column or per G
 * consecutive weights of a column):
 *
 *   O1  unpack      Q[k][n] = (q_kpacked[k/8][n] >> 4*(k%8)) & 15
 *   O2  dequantise  W[k][n] = (Q[k][n] - 8) * S[k/G][n]          (fp64, exact)
 *   O3  product     Y[m][n] = sum_{k ascending} A[m][k] * W[k][n] (fp64)
 *   O4  round       C[m][n] = fp16 round-to-nearest-even of Y[m][n]
 *
 * The "- 8" is the symmetric zero point the paper fuses into its conversion
 * ("Dequantization and Tensor Cores", Section 3.4).  Groups run along K
 * (Section 2.3, "partitioning v into groups").
 *
 * 2:4 variant (Section 2.2 "Modern Tensor Core Units"; Section 4 "Quantized
 * non-zero values", "Metadata indices"): the weight matrix is split into groups
 * of four along K; two entries per group are kept.  The compressed input holds
 * the kept values Qc[K/2][N] and their positions idx[K/2][N] in 0..3.  The oracle
 * expands to the dense K x N matrix with zeros (code 8) at pruned positions and
 * then applies O2-O4 unchanged.
 *
 * Every function is plain loops; OpenMP only distributes independent output
 * columns over threads, it never changes the order of any sum.
 *
 * Parity pins (tests/test_oracle_pins.py): fp16 conversion against all 65536
 * bit patterns and numpy; product against exact rational arithmetic on tiny
 * shapes and against numpy's fp64 matmul; closed forms; sparse == dense with
 * zeros.  Summation-order effects on C are parity unpinned beyond the tolerance
 * (any order within the stated tolerance is a correct result).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_ERR_ARG 1
#define ORACLE_ERR_ALLOC 2
#define ORACLE_ERR_INDEX 3

/* ---- fp16 <-> fp64 ------------------------------------------------------- */

/* IEEE binary16 bits -> double, exact. */
double oracle_f16_to_f64(uint16_t h) {
  int sign = (h >> 15) & 1;
  int e = (h >> 10) & 31;
  int f = h & 1023;
  double v;
  if (e == 31) {
    v = f ? NAN : INFINITY;
  } else if (e == 0) {
    v = ldexp((double)f, -24); /* subnormal: f * 2^-24 */
  } else {
    v = ldexp((double)(1024 + f), e - 25); /* (1 + f/1024) * 2^(e-15) */
  }
  return sign ? -v : v;
}

/* double -> IEEE binary16 bits, round to nearest, ties to even, directly from
 * the double (no float intermediate).  Overflow gives +-inf. */
uint16_t oracle_f64_to_f16(double x) {
  uint16_t sign = signbit(x) ? 0x8000u : 0u;
  if (isnan(x)) return (uint16_t)(sign | 0x7e00u);
  double a = fabs(x);
  if (isinf(a)) return (uint16_t)(sign | 0x7c00u);
  if (a == 0.0) return sign;
  int ex;
  (void)frexp(a, &ex); /* a = m * 2^ex, m in [0.5, 1) => floor(log2 a) = ex-1 */
  int e = ex - 1;
  if (e < -14) e = -14;             /* subnormal range shares the quantum 2^-24 */
  double q = ldexp(a, 10 - e);      /* a / 2^(e-10): exact power-of-two scaling  */
  double fl = floor(q);
  double d = q - fl;                /* exact: q has at most 53 significant bits  */
  if (d > 0.5 || (d == 0.5 && fmod(fl, 2.0) == 1.0)) fl += 1.0;
  /* fl is now an integer in [0, 2048] */
  if (fl == 2048.0) { fl = 1024.0; e += 1; }
  if (e > 15) return (uint16_t)(sign | 0x7c00u);
  uint32_t n = (uint32_t)fl;
  if (n < 1024u) return (uint16_t)(sign | n);        /* subnormal or zero   */
  return (uint16_t)(sign | ((uint32_t)(e + 15) << 10) | (n - 1024u));
}

void oracle_f64_to_f16_array(const double* x, uint16_t* out, int64_t n) {
  for (int64_t i = 0; i < n; ++i) out[i] = oracle_f64_to_f16(x[i]);
}

void oracle_f16_to_f64_array(const uint16_t* h, double* out, int64_t n) {
  for (int64_t i = 0; i < n; ++i) out[i] = oracle_f16_to_f64(h[i]);
}

/* ---- O1: canonical K-packed words <-> one code per byte ------------------- */

/* q_kpacked is [K/8][N] uint32; nibble j of word (kb, n) is Q[8*kb + j][n]. */
int oracle_unpack_q(const uint32_t* q_kpacked, int K, int N, uint8_t* Q) {
  if (!q_kpacked || !Q || K <= 0 || N <= 0 || K % 8) return ORACLE_ERR_ARG;
  for (int k = 0; k < K; ++k)
    for (int n = 0; n < N; ++n)
      Q[(size_t)k * N + n] = (uint8_t)((q_kpacked[(size_t)(k / 8) * N + n] >> (4 * (k % 8))) & 15u);
  return ORACLE_OK;
}

int oracle_pack_q(const uint8_t* Q, int K, int N, uint32_t* q_kpacked) {
  if (!q_kpacked || !Q || K <= 0 || N <= 0 || K % 8) return ORACLE_ERR_ARG;
  memset(q_kpacked, 0, (size_t)(K / 8) * N * sizeof(uint32_t));
  for (int k = 0; k < K; ++k)
    for (int n = 0; n < N; ++n) {
      if (Q[(size_t)k * N + n] > 15) return ORACLE_ERR_ARG;
      q_kpacked[(size_t)(k / 8) * N + n] |= (uint32_t)Q[(size_t)k * N + n] << (4 * (k % 8));
    }
  return ORACLE_OK;
}

/* ---- O2: dequantise ------------------------------------------------------- */

/* W[k][n] = (Q[k][n] - 8) * S[k/G][n] in fp64; S is [K/G][N] fp16 bits. */
int oracle_dequant(const uint8_t* Q, const uint16_t* S, int K, int N, int G, double* W) {
  if (!Q || !S || !W || K <= 0 || N <= 0 || G <= 0 || K % G) return ORACLE_ERR_ARG;
  for (int k = 0; k < K; ++k)
    for (int n = 0; n < N; ++n)
      W[(size_t)k * N + n] =
          ((double)Q[(size_t)k * N + n] - 8.0) * oracle_f16_to_f64(S[(size_t)(k / G) * N + n]);
  return ORACLE_OK;
}

/* ---- O2..O4 from unpacked codes ------------------------------------------- */

/* C[m][n] = fp16( sum_k A[m][k] * (Q[k][n]-8) * S[k/G][n] ), Q one code per byte. */
static int gemm_from_codes(const uint16_t* A, const uint8_t* Q, const uint16_t* S,
                           int M, int K, int N, int G, uint16_t* C) {
  double* Ad = (double*)malloc((size_t)M * K * sizeof(double));
  if (!Ad) return ORACLE_ERR_ALLOC;
  for (size_t i = 0; i < (size_t)M * K; ++i) Ad[i] = oracle_f16_to_f64(A[i]);
  int err = ORACLE_OK;
#pragma omp parallel
  {
    double* wcol = (double*)malloc((size_t)K * sizeof(double));
    if (!wcol) {
#pragma omp atomic write
      err = ORACLE_ERR_ALLOC;
    }
#pragma omp for schedule(static)
    for (int n = 0; n < N; ++n) {
      if (!wcol) continue;
      /* O2 for column n */
      for (int k = 0; k < K; ++k)
        wcol[k] = ((double)Q[(size_t)k * N + n] - 8.0) * oracle_f16_to_f64(S[(size_t)(k / G) * N + n]);
      /* O3 + O4 for every row m, k ascending */
      for (int m = 0; m < M; ++m) {
        const double* a = Ad + (size_t)m * K;
        double y = 0.0;
        for (int k = 0; k < K; ++k) y += a[k] * wcol[k];
        C[(size_t)m * N + n] = oracle_f64_to_f16(y);
      }
    }
    free(wcol);
  }
  free(Ad);
  return err;
}

/* Full dense pipeline O1..O4.
 *   A          [M][K]   fp16 bits, row-major
 *   q_kpacked  [K/8][N] uint32 (canonical, see oracle_unpack_q)
 *   S          [K/G][N] fp16 bits; G == K means one scale per output column
 *   C          [M][N]   fp16 bits (output) */
int oracle_gemm(const uint16_t* A, const uint32_t* q_kpacked, const uint16_t* S,
                int M, int K, int N, int G, uint16_t* C) {
  if (!A || !q_kpacked || !S || !C) return ORACLE_ERR_ARG;
  if (M <= 0 || K <= 0 || N <= 0 || G <= 0 || K % 8 || K % G) return ORACLE_ERR_ARG;
  uint8_t* Q = (uint8_t*)malloc((size_t)K * N);
  if (!Q) return ORACLE_ERR_ALLOC;
  int err = oracle_unpack_q(q_kpacked, K, N, Q);
  if (!err) err = gemm_from_codes(A, Q, S, M, K, N, G, C);
  free(Q);
  return err;
}

/* Same result for a list of single outputs (m_i, n_i), each computed from the
 * packed inputs on its own: used at sizes where the full product is too slow. */
int oracle_gemm_samples(const uint16_t* A, const uint32_t* q_kpacked, const uint16_t* S,
                        int M, int K, int N, int G, const int32_t* ms, const int32_t* ns,
                        int count, uint16_t* out) {
  if (!A || !q_kpacked || !S || !ms || !ns || !out) return ORACLE_ERR_ARG;
  if (M <= 0 || K <= 0 || N <= 0 || G <= 0 || K % 8 || K % G || count < 0) return ORACLE_ERR_ARG;
  int err = ORACLE_OK;
#pragma omp parallel for schedule(static)
  for (int i = 0; i < count; ++i) {
    int m = ms[i], n = ns[i];
    if (m < 0 || m >= M || n < 0 || n >= N) {
#pragma omp atomic write
      err = ORACLE_ERR_INDEX;
      continue;
    }
    double y = 0.0;
    for (int k = 0; k < K; ++k) {
      unsigned q = (q_kpacked[(size_t)(k / 8) * N + n] >> (4 * (k % 8))) & 15u;
      double w = ((double)q - 8.0) * oracle_f16_to_f64(S[(size_t)(k / G) * N + n]);
      y += oracle_f16_to_f64(A[(size_t)m * K + k]) * w;
    }
    out[i] = oracle_f64_to_f16(y);
  }
  return err;
}

/* ---- 2:4 variant ----------------------------------------------------------- */

/* Expand the compressed form to dense codes.
 *   qc_kpacked [K/2/8][N] uint32: nibble j of word (r, n) is Qc[8r + j][n]
 *   idx        [K/2][N]   uint8, 0..3: position of kept value Qc[t][n] inside
 *              its group of four, idx[2u][n] < idx[2u+1][n]
 *   Q          [K][N]     output, code 8 (value 0) at pruned positions
 * Kept value 2u+j of column n lands at row 4u + idx[2u+j][n]. */
int oracle_sparse24_expand(const uint32_t* qc_kpacked, const uint8_t* idx, int K, int N, uint8_t* Q) {
  if (!qc_kpacked || !idx || !Q || K <= 0 || N <= 0 || K % 16) return ORACLE_ERR_ARG;
  int Kc = K / 2;
  memset(Q, 8, (size_t)K * N);
  for (int u = 0; u < K / 4; ++u)
    for (int n = 0; n < N; ++n) {
      int i0 = idx[(size_t)(2 * u) * N + n], i1 = idx[(size_t)(2 * u + 1) * N + n];
      if (i0 > 3 || i1 > 3 || i0 >= i1) return ORACLE_ERR_INDEX;
      for (int j = 0; j < 2; ++j) {
        int t = 2 * u + j;
        if (t >= Kc) return ORACLE_ERR_INDEX;
        uint8_t q = (uint8_t)((qc_kpacked[(size_t)(t / 8) * N + n] >> (4 * (t % 8))) & 15u);
        Q[(size_t)(4 * u + (j ? i1 : i0)) * N + n] = q;
      }
    }
  return ORACLE_OK;
}

/* 2:4 pipeline: expand, then O2..O4 with scale groups over the ORIGINAL K. */
int oracle_gemm_sparse24(const uint16_t* A, const uint32_t* qc_kpacked, const uint8_t* idx,
                         const uint16_t* S, int M, int K, int N, int G, uint16_t* C) {
  if (!A || !qc_kpacked || !idx || !S || !C) return ORACLE_ERR_ARG;
  if (M <= 0 || K <= 0 || N <= 0 || G <= 0 || K % 16 || K % G) return ORACLE_ERR_ARG;
  uint8_t* Q = (uint8_t*)malloc((size_t)K * N);
  if (!Q) return ORACLE_ERR_ALLOC;
  int err = oracle_sparse24_expand(qc_kpacked, idx, K, N, Q);
  if (!err) err = gemm_from_codes(A, Q, S, M, K, N, G, C);
  free(Q);
  return err;
}

/* Acceptance test of the build: |C - C_ref| <= rel * (|C_ref| + rms(C_ref)),
 * rms over the whole reference.  Returns the number of failing elements and
 * writes the worst ratio error/allowance.  Non-finite C where C_ref is finite
 * fails. */
int64_t oracle_check_tolerance(const uint16_t* C, const uint16_t* C_ref, int64_t count, double rel,
                               double* worst_ratio, double* rms_out) {
  double ss = 0.0;
  for (int64_t i = 0; i < count; ++i) {
    double r = oracle_f16_to_f64(C_ref[i]);
    ss += r * r;
  }
  double rms = count ? sqrt(ss / (double)count) : 0.0;
  double worst = 0.0;
  int64_t bad = 0;
  for (int64_t i = 0; i < count; ++i) {
    double r = oracle_f16_to_f64(C_ref[i]), c = oracle_f16_to_f64(C[i]);
    if (!isfinite(r)) {
      if (!(isnan(r) ? isnan(c) : c == r)) ++bad;
      continue;
    }
    if (!isfinite(c)) { ++bad; worst = INFINITY; continue; }
    double allow = rel * (fabs(r) + rms);
    double e = fabs(c - r);
    if (e > allow) ++bad;
    double ratio = allow > 0.0 ? e / allow : (e > 0.0 ? INFINITY : 0.0);
    if (ratio > worst) worst = ratio;
  }
  if (worst_ratio) *worst_ratio = worst;
  if (rms_out) *rms_out = rms;
  return bad;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
