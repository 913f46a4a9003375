/* CPU oracle of the data-free quantiser front end -- TEST INFRASTRUCTURE ONLY.
 *
 * Section 3.5 (a): the group scales are picked by searching, per group, for the clipping threshold that gives the
 * least quantisation error (in the manner of activation-aware weight quantisation, but without activations:
 * round-to-nearest onto the symmetric 4-bit grid of Section 3.4, W ~ (q - 8) * s with q in 0..15).
 *
 * The paper gives no more than that sentence; the reading taken here, step by step, for every group g of G
 * consecutive rows of one column n (w_i = W[g*G + i][n], i = 0..G-1):
 *   Q1  a = max_i |w_i|.
 *   Q2  Candidate t = 0 .. n_candidates-1 shrinks the range by r_t = 1 - t / n_grid (t = 0: no clipping).  The grid
 *       -8..7 is centred on -0.5, so a symmetric range [-a r, a r] maps to 15 steps: s_t = 2 a r_t / 15, stored as fp16
 *       (a scale that rounds to zero becomes the smallest positive fp16).
 *   Q3  q_i = clamp(round_half_even(w_i / s_t), -8, 7) + 8.
 *   Q4  e_t = sum_i (w_i - (q_i - 8) s_t)^2; the candidate with the least e_t wins, the first one on ties.
 * These steps decide integers (codes, the winning candidate), so they are taken in the precision of the kernel under
 * test, fp32, in a fixed order (stated at each line below); every fp32 operation here is a single IEEE operation
 * (compile with -ffp-contract=off), fmaf is the correctly rounded fused multiply-add.
 * Inputs must be finite.  No blocking, no vectorisation; OpenMP only over independent columns.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

static float f16_to_f32(uint16_t h) {
  const int sign = h >> 15, e = (h >> 10) & 31, m = h & 1023;
  double v;
  if (e == 0) v = ldexp((double)m, -24);
  else if (e == 31) v = m ? NAN : INFINITY;
  else v = ldexp((double)(1024 + m), e - 25);
  return (float)(sign ? -v : v); /* every fp16 value is exactly representable in fp32 */
}

/* fp32 -> fp16, round to nearest even (finite, non-negative inputs below 65520 are all this file needs) */
static uint16_t f32_to_f16_rn(float x) {
  if (!(x > 0.0f)) return 0;
  int e;
  const double fr = frexp((double)x, &e); /* x = fr * 2^e, 0.5 <= fr < 1 */
  int ex = e - 1;                         /* x = (2 fr) * 2^ex, 1 <= 2 fr < 2 */
  if (ex < -14) ex = -14;                 /* subnormal range: fixed exponent */
  const double scaled = ldexp((double)x, 10 - ex); /* in units of the fp16 ulp at this exponent */
  double r = nearbyint(scaled);                     /* default rounding mode: half to even */
  if (ex == -14 && r < 1024.0) return (uint16_t)r;  /* subnormal (or zero) */
  if (r >= 2048.0) { r /= 2.0; ex += 1; }
  if (ex > 15) return 0x7C00;
  return (uint16_t)(((ex + 15) << 10) | ((int)r - 1024));
}

/* W fp16 bits [K][N] row-major -> codes Q [K][N] (0..15), scales fp16 bits [K/G][N], chosen candidate [K/G][N] */
int oracle_quantize_rtn(const uint16_t* W, int K, int N, int G, int n_grid, int n_candidates, uint8_t* Q, uint16_t* S,
                        int32_t* chosen) {
  if (K <= 0 || N <= 0 || G <= 0 || K % G || n_grid < 1 || n_candidates < 1 || n_candidates > n_grid) return 1;
  const float two_fifteenths = 2.0f / 15.0f; /* one fp32 division of exact constants */
#pragma omp parallel for schedule(static)
  for (int n = 0; n < N; ++n) {
    for (int g = 0; g < K / G; ++g) {
      const uint16_t* w = W + (size_t)g * G * N + n; /* stride N */
      /* Q1 */
      float a = 0.0f;
      for (int i = 0; i < G; ++i) {
        const float v = fabsf(f16_to_f32(w[(size_t)i * N]));
        if (v > a) a = v;
      }
      float best_err = INFINITY;
      uint16_t best_s = 0;
      int best_t = -1;
      for (int t = 0; t < n_candidates; ++t) {
        /* Q2: r = 1 - t / n_grid, s = (a * r) * (2 / 15), each operation rounded to fp32, then to fp16 */
        const float r = 1.0f - (float)t / (float)n_grid;
        const float s32 = (a * r) * two_fifteenths;
        uint16_t sh = f32_to_f16_rn(s32);
        if (sh == 0) sh = 1;
        const float s = f16_to_f32(sh);
        const float inv = 1.0f / s;
        /* Q3, Q4 in the order i = 0 .. G-1 */
        float err = 0.0f;
        for (int i = 0; i < G; ++i) {
          const float wi = f16_to_f32(w[(size_t)i * N]);
          float qf = rintf(wi * inv);
          if (qf < -8.0f) qf = -8.0f;
          if (qf > 7.0f) qf = 7.0f;
          const float d = fmaf(-qf, s, wi);
          err = fmaf(d, d, err);
        }
        if (err < best_err) {
          best_err = err;
          best_s = sh;
          best_t = t;
        }
      }
      const float s = f16_to_f32(best_s);
      const float inv = 1.0f / s;
      for (int i = 0; i < G; ++i) {
        const float wi = f16_to_f32(w[(size_t)i * N]);
        float qf = rintf(wi * inv);
        if (qf < -8.0f) qf = -8.0f;
        if (qf > 7.0f) qf = 7.0f;
        Q[((size_t)g * G + i) * N + n] = (uint8_t)((int)qf + 8);
      }
      S[(size_t)g * N + n] = best_s;
      if (chosen) chosen[(size_t)g * N + n] = best_t;
    }
  }
  return 0;
}
