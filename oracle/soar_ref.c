/*
 * SOAR reference oracle (CPU, plain C).  TEST INFRASTRUCTURE ONLY.
 *
 * A slow, direct restatement of the SOAR paper's NVFP4 weight quantizer:
 * Sec. 3.1 (Eq. 1-3, the NVFP4 format and the max-based rule), Sec. 3.2
 * (Eq. 4-6, CJSO), Sec. 3.3 (Eq. 7-8, DSS), Appendix B.3 (the candidate grids)
 * and Algorithm 1 (the loop).  Steps run in the algorithm's order with no
 * blocking, fusion or reuse: every candidate pair re-rounds the whole block and
 * sums its squared error term by term.
 *
 * Optional column weights (Sec. 5, "Discussions and Future Works": the output
 * distortion ||(W - What) X||^2, taken here in its diagonal form): with h_j >= 0
 * per input column the objective is sum_ij h_j (W_ij - What_ij)^2, and every
 * per-element term of Eq. 4-8 carries its column's h_j.  Without weights h_j = 1
 * and the arithmetic is the unweighted one, operation for operation.
 *
 * Arithmetic convention.  Every quantity that feeds a discrete decision (a
 * rounding to the E2M1 grid, a projection to E4M3) is a fixed sequence of IEEE
 * binary32 round-to-nearest operations, written out where it happens; every sum
 * and every error is binary64.  Compile with -ffp-contract=off and without
 * fast-math so that the binary32 steps round exactly as written.
 *
 * Nothing here is shared with the CUDA library: no header, table or helper.
 * Only tests, the smoke check and the CPU-baseline leg of the benchmark may
 * load this file's shared object.
 *
 * Pins (see the CPU tests): E2M1 grid and E4M3 range from Sec. 3.1; rounding
 * against an independent library cast; Eq. 5/6 against brute-force minimisation;
 * the Eq. 8 argmin against a separate NumPy enumeration; grid-aligned tensors
 * against their closed-form result; the weighted form against weighted least
 * squares, constant weights and zero-weight columns; the MXFP4 mode (end of this file)
 * against the format's definition, a NumPy restatement and a brute-force argmin, its
 * candidate rule being a reading the paper does not fix.  Parity unpinned: the early-stop trajectory
 * and the iteration-to-iteration path (the paper prints no numbers for them);
 * those rest on agreement between this file and the NumPy restatement.
 */
#include <float.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#if defined(FLT_EVAL_METHOD) && FLT_EVAL_METHOD != 0
#error "binary32 expressions must be evaluated in binary32 (FLT_EVAL_METHOD == 0)"
#endif

#define REF_BLOCK 16          /* Sec. 3.1: one E4M3 scale per 16 elements        */
#define REF_MAX_BETA 512
#define REF_MAX_DQ 16

/* status bits reported by soar_ref_quantize */
#define REF_STATUS_ZERO_TENSOR 1
#define REF_STATUS_NONFINITE 2
#define REF_STATUS_RANGE 4
#define REF_STATUS_BAD_WEIGHT 16   /* a column weight that is negative, not finite, or outside {0} u [2^-20, 2^20] */

typedef struct soar_ref_cfg {
  int32_t max_iters;      /* T of Algorithm 1; 0 = max-based NVFP4 only (Eq. 1-3) */
  float early_stop_rel;   /* Sec. 4.1: stop when the relative MSE gain is below   */
  int32_t n_dq;           /* E4M3 dequantization candidates per block (App. B.3)  */
  int32_t n_beta;         /* multipliers for the quantization scale (App. B.3)    */
  int32_t beta_step_pct;  /* grid step in hundredths (App. B.3: 0.01)             */
  int32_t flags;          /* REF_FLAG_* : the paper's stand-alone arms (Sec. 3.2, 3.3) */
} soar_ref_cfg;

/* Sec. 3.2 alone ("Refinement Scheme"): one block scale plays both roles, so a candidate's
 * quantization scale is its own E4M3 dequantization value (times beta) instead of the
 * unrounded Eq. 6 solution. */
#define REF_FLAG_COUPLED_SCALE 1
/* Sec. 3.3 alone ((i),(ii)): the search runs around the max-based start, so Eq. 5 is
 * skipped (alpha stays Eq. 1's) ... */
#define REF_FLAG_KEEP_ALPHA 2
/* ... and Eq. 6 is skipped (the candidate sets are centred on the stored scale). */
#define REF_FLAG_KEEP_BLOCK_SCALE 4

/* ------------------------------------------------------------------ formats */

/* bf16 bit pattern -> binary32 (exact). */
float soar_ref_bf16_to_f32(uint16_t h) {
  uint32_t u = ((uint32_t)h) << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

/* Eq. 2 evaluated literally on a magnitude x >= 0, with round-half-to-even for
 * the nearest-integer bracket and saturation at M_FP4 = 6 above the last
 * branch.  Returns a value of the E2M1 grid {0,.5,1,1.5,2,3,4,6}. */
double soar_ref_e2m1_round(double x) {
  if (x < 2.0) return 0.5 * nearbyint(2.0 * x);
  if (x < 4.0) return nearbyint(x);
  if (x <= 6.0) return 2.0 * nearbyint(0.5 * x);
  return 6.0;
}

/* E2M1 magnitude value -> 3-bit code (0,.5,1,1.5,2,3,4,6 -> 0..7). */
int soar_ref_e2m1_code(double m) {
  if (m == 0.0) return 0;
  if (m == 0.5) return 1;
  if (m == 1.0) return 2;
  if (m == 1.5) return 3;
  if (m == 2.0) return 4;
  if (m == 3.0) return 5;
  if (m == 4.0) return 6;
  return 7;
}

/* FP8 E4M3 (4 exponent bits, bias 7, 3 mantissa bits, no infinity, max 448)
 * positive code 0x00..0x7E -> value. */
float soar_ref_e4m3_decode(uint8_t c) {
  int e = (c >> 3) & 0xF;
  int f = c & 7;
  if (e == 0) return (float)ldexp((double)f, -9);         /* subnormal: f/8 * 2^-6 */
  return (float)ldexp(8.0 + (double)f, e - 7 - 3);
}

/* Projection of a non-negative scale onto E4M3 (Eq. 16): round to nearest,
 * ties to even, subnormals included, clipped to M_FP8 = 448. Returns the code. */
uint8_t soar_ref_e4m3_encode(float v) {
  double d = (double)v;
  if (!(d > 0.0)) return 0;
  if (d >= 448.0) return 0x7E;
  if (d < ldexp(1.0, -6)) {
    int q = (int)nearbyint(ldexp(d, 9));                  /* steps of 2^-9          */
    return (uint8_t)q;                                    /* q == 8 is 2^-6 = 0x08  */
  }
  int e;
  (void)frexp(d, &e);                                     /* d = m*2^e, m in [.5,1) */
  e -= 1;                                                 /* 2^e <= d < 2^(e+1)     */
  int q = (int)nearbyint(ldexp(d, 3 - e));                /* in [8,16]              */
  if (q == 16) { q = 8; e += 1; }
  return (uint8_t)(((e + 7) << 3) | (q - 8));
}

/* ------------------------------------------------------- block-level steps */

/* Re-rounding of one block under scales (alpha, dq) (Eq. 2; Algorithm 1 "Compute
 * FP4 assignment"): s = fl32(alpha*dq), r = fl32(1/s), x_j = fl32(|W_j|*r),
 * m_j = E2M1 rounding of x_j.  Writes magnitudes m[16]; returns through A, B the
 * binary64 sums  A = sum h_j |W_j| m_j,  B = sum h_j m_j^2  (the block's terms of Eq. 5/6;
 * W_j and Q_j share a sign, so W_j Q_j = |W_j| m_j).  h points at the block's 16 column
 * weights, or is NULL for h_j = 1.  Each product is exact in binary64 (24 + 8 + 2 and
 * 24 + 4 significant bits); the sums run in element order. */
void soar_ref_round_block_w(const uint16_t* w, const float* h, float alpha, float dq, double* m,
                            double* A, double* B) {
  float s = alpha * dq;
  float r = 1.0f / s;
  double a = 0.0, b = 0.0;
  for (int j = 0; j < REF_BLOCK; ++j) {
    float mag = fabsf(soar_ref_bf16_to_f32(w[j]));
    float x = mag * r;
    double mj = soar_ref_e2m1_round((double)x);
    double hj = h ? (double)h[j] : 1.0;
    m[j] = mj;
    a += (hj * (double)mag) * mj;
    b += hj * (mj * mj);
  }
  *A = a;
  *B = b;
}

void soar_ref_round_block(const uint16_t* w, float alpha, float dq, double* m,
                          double* A, double* B) {
  soar_ref_round_block_w(w, NULL, alpha, dq, m, A, B);
}

/* Block reconstruction error of Eq. 8 for magnitudes m and dequantization scale
 * code d under global scale alpha:  sum_j h_j (|W_j| - m_j * alpha*value(d))^2
 * (h == NULL: h_j = 1). */
double soar_ref_block_error_w(const uint16_t* w, const float* h, const double* m, float alpha,
                              uint8_t d) {
  double s = (double)alpha * (double)soar_ref_e4m3_decode(d);
  double L = 0.0;
  for (int j = 0; j < REF_BLOCK; ++j) {
    double mag = fabs((double)soar_ref_bf16_to_f32(w[j]));
    double hj = h ? (double)h[j] : 1.0;
    double e = mag - m[j] * s;
    L += hj * (e * e);
  }
  return L;
}

double soar_ref_block_error(const uint16_t* w, const double* m, float alpha, uint8_t d) {
  return soar_ref_block_error_w(w, NULL, m, alpha, d);
}

/* Eq. 6 / Algorithm 1 "Update block-wise scale": A/(alpha*B) as binary32 steps.
 * B == 0 (every code zero) keeps the current stored scale. */
float soar_ref_block_scale(double A, double B, float alpha, uint8_t d_cur) {
  if (!(B > 0.0)) return soar_ref_e4m3_decode(d_cur);
  float den = alpha * (float)B;
  float q = (float)A / den;
  return q;
}

/* App. B.3 / Algorithm 1 "Find dequantization candidates": E4M3 codes around
 * the analytic scale.  n == 1: nearest code.  n >= 2: with c_f the largest code
 * whose value is <= center, codes c_f-(n/2-1) .. c_f+n/2.  Clipped to the
 * positive finite range [0x01,0x7E], duplicates dropped, ascending. Returns count. */
int soar_ref_dq_candidates(float center, int n, uint8_t* out) {
  int lo, hi;
  if (n <= 1) {
    lo = hi = soar_ref_e4m3_encode(center);
  } else {
    int cf = 0;
    for (int c = 0x7E; c >= 0; --c) {
      if (soar_ref_e4m3_decode((uint8_t)c) <= center) { cf = c; break; }
    }
    lo = cf - (n / 2 - 1);
    hi = cf + n / 2;
  }
  int cnt = 0;
  for (int c = lo; c <= hi; ++c) {
    int cc = c < 1 ? 1 : (c > 0x7E ? 0x7E : c);
    if (cnt > 0 && out[cnt - 1] == (uint8_t)cc) continue;
    out[cnt++] = (uint8_t)cc;
  }
  return cnt;
}

/* App. B.3 / Algorithm 1 "Construct quantization scale search space":
 * beta_k = (100 + (k - floor(n/2))*step)/100 rounded once to binary32. */
float soar_ref_beta(int k, int n_beta, int step_pct) {
  double b = (100.0 + (double)((k - n_beta / 2) * step_pct)) / 100.0;
  return (float)b;
}

/* One block's DSS (Eq. 8; Algorithm 1 "Evaluate" and "Select"): scan beta
 * ascending, then dequantization candidates ascending, strict '<' so the first
 * minimum wins.  Returns the winner through dq_out/d_out/L_out and, through
 * gap_rel, the relative gap to the best candidate whose outcome (16 magnitudes,
 * scale code) differs from the winner's (1e300 if there is none). */
static void dss_block(const uint16_t* w, const float* h, float alpha, float center,
                      const soar_ref_cfg* cfg,
                      float* dq_out, uint8_t* d_out, double* L_out, double* A_out,
                      double* B_out, double* gap_rel) {
  uint8_t dc[REF_MAX_DQ];
  int nd = soar_ref_dq_candidates(center, cfg->n_dq, dc);
  int nb = cfg->n_beta;
  const int coupled = (cfg->flags & REF_FLAG_COUPLED_SCALE) != 0;
  /* one entry per candidate pair (k, d); without coupling the codes of a beta are the same
   * for every d and are simply made again */
  static _Thread_local double mk[REF_MAX_BETA][REF_MAX_DQ][REF_BLOCK];
  static _Thread_local double Lk[REF_MAX_BETA][REF_MAX_DQ];
  static _Thread_local double Ak[REF_MAX_BETA][REF_MAX_DQ], Bk[REF_MAX_BETA][REF_MAX_DQ];
  static _Thread_local float dqk[REF_MAX_BETA][REF_MAX_DQ];
  double best = 0.0;
  int bk = -1, bd = -1;
  for (int k = 0; k < nb; ++k) {
    float beta = soar_ref_beta(k, nb, cfg->beta_step_pct);
    for (int d = 0; d < nd; ++d) {
      float dq = (coupled ? soar_ref_e4m3_decode(dc[d]) : center) * beta;
      dqk[k][d] = dq;
      soar_ref_round_block_w(w, h, alpha, dq, mk[k][d], &Ak[k][d], &Bk[k][d]);
      double L = soar_ref_block_error_w(w, h, mk[k][d], alpha, dc[d]);
      Lk[k][d] = L;
      if (bk < 0 || L < best) { best = L; bk = k; bd = d; }
    }
  }
  double second = 1e300;
  for (int k = 0; k < nb; ++k) {
    for (int d = 0; d < nd; ++d) {
      int same_codes = memcmp(mk[k][d], mk[bk][bd], sizeof(mk[k][d])) == 0;
      if (same_codes && dc[d] == dc[bd]) continue;
      if (Lk[k][d] < second) second = Lk[k][d];
    }
  }
  *dq_out = dqk[bk][bd];
  *d_out = dc[bd];
  *L_out = best;
  *A_out = Ak[bk][bd];
  *B_out = Bk[bk][bd];
  if (second >= 1e300) *gap_rel = 1e300;
  else if (best > 0.0) *gap_rel = (second - best) / best;
  else *gap_rel = (second > 0.0) ? 1e300 : 0.0;
}

/* ------------------------------------------------------------- whole tensor */

/*
 * SOAR on one bf16 matrix W[rows][ld] (cols used, cols % 16 == 0), Algorithm 1.
 *
 *   out_packed  rows*cols/2 bytes: code(2j) | code(2j+1)<<4, code = sign<<3 | magnitude code
 *   out_scales  rows*cols/16 bytes: E4M3 dequantization scale per block, row-major
 *   out_alpha   the FP32 global scale
 *   trace_alpha [max_iters+1]: alpha^(0), then the alpha used by each executed iteration
 *   trace_sse   [max_iters+1]: error of the initial state, then after each executed iteration
 *   tie_flags   per block (may be NULL): 1 if in any executed iteration the best two
 *               distinct candidate outcomes were closer than tie_rel (relative)
 *   out_sumsq   sum of h_j W^2 (may be NULL)
 *   h           cols column weights (Sec. 5 in diagonal form), or NULL for h_j = 1; the
 *               initialization (Eq. 1) does not depend on them
 * Returns status bits; *iters_run = executed iterations.
 */
int soar_ref_quantize_weighted(const uint16_t* W, int64_t rows, int64_t cols, int64_t ld,
                               const float* h, const soar_ref_cfg* cfg, uint8_t* out_packed,
                               uint8_t* out_scales, float* out_alpha, int32_t* iters_run,
                               double* trace_alpha, double* trace_sse, uint8_t* tie_flags,
                               double tie_rel, double* out_sumsq) {
  const int64_t nbc = cols / REF_BLOCK;
  const int64_t nblk = rows * nbc;
  int status = 0;
  *iters_run = 0;

  /* Eq. 1: tensor-wide maximum magnitude. */
  float amax = 0.0f;
  double sumsq = 0.0;
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t c = 0; c < cols; ++c) {
      float v = fabsf(soar_ref_bf16_to_f32(W[r * ld + c]));
      if (!(v <= 3.4e38f)) status |= REF_STATUS_NONFINITE;
      if (v > amax) amax = v;
      sumsq += (h ? (double)h[c] : 1.0) * ((double)v * (double)v);
    }
  if (h)
    for (int64_t c = 0; c < cols; ++c) {
      float hv = h[c];
      if (!(hv == 0.0f || (hv >= 0x1p-20f && hv <= 0x1p20f))) status |= REF_STATUS_BAD_WEIGHT;
    }
  if (out_sumsq) *out_sumsq = sumsq;
  if (tie_flags) memset(tie_flags, 0, (size_t)nblk);
  if (status & (REF_STATUS_NONFINITE | REF_STATUS_BAD_WEIGHT)) return status;
  if (amax == 0.0f) {
    /* all-zero tensor: alpha = 1, zero scales, codes carry only the input's sign bit */
    for (int64_t r = 0; r < rows; ++r)
      for (int64_t c = 0; c < cols; c += 2) {
        int lo = (W[r * ld + c] >> 15) << 3, hi = (W[r * ld + c + 1] >> 15) << 3;
        out_packed[(r * cols + c) / 2] = (uint8_t)(lo | (hi << 4));
      }
    memset(out_scales, 0, (size_t)nblk);
    *out_alpha = 1.0f;
    trace_alpha[0] = 1.0;
    trace_sse[0] = 0.0;
    return status | REF_STATUS_ZERO_TENSOR;
  }
  if (!(amax >= 0x1p-100f && amax <= 0x1p100f)) return status | REF_STATUS_RANGE;

  /* Eq. 1 and Algorithm 1 "Initialization": alpha0 = amax/(6*448); per block
   * dd0 = E4M3(bmax/(6*alpha0)), dq0 = dd0.  A non-zero block whose scale would
   * round to zero takes the smallest positive code. */
  float alpha0v = amax / 2688.0f;
  float alpha = alpha0v;
  float six_alpha = alpha * 6.0f;
  float* dq = (float*)malloc(sizeof(float) * (size_t)nblk);
  uint8_t* dd = (uint8_t*)malloc((size_t)nblk);
  double* rowA = (double*)malloc(sizeof(double) * (size_t)rows);
  double* rowB = (double*)malloc(sizeof(double) * (size_t)rows);
  double* rowL = (double*)malloc(sizeof(double) * (size_t)rows);

#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r) {
    double sL = 0.0;
    for (int64_t b = 0; b < nbc; ++b) {
      const uint16_t* w = W + r * ld + b * REF_BLOCK;
      float bmax = 0.0f;
      for (int j = 0; j < REF_BLOCK; ++j) {
        float v = fabsf(soar_ref_bf16_to_f32(w[j]));
        if (v > bmax) bmax = v;
      }
      int64_t i = r * nbc + b;
      if (bmax == 0.0f) { dd[i] = 0; dq[i] = 0.0f; continue; }
      float t = bmax / six_alpha;
      uint8_t c = soar_ref_e4m3_encode(t);
      if (c == 0) c = 1;
      dd[i] = c;
      dq[i] = soar_ref_e4m3_decode(c);
      double m[REF_BLOCK], A, B;
      const float* hb = h ? h + b * REF_BLOCK : NULL;
      soar_ref_round_block_w(w, hb, alpha, dq[i], m, &A, &B);
      sL += soar_ref_block_error_w(w, hb, m, alpha, c);
    }
    rowL[r] = sL;
  }
  double sse = 0.0;
  for (int64_t r = 0; r < rows; ++r) sse += rowL[r];
  trace_alpha[0] = (double)alpha;
  trace_sse[0] = sse;

  /* Algorithm 1 main loop. */
  for (int t = 0; t < cfg->max_iters; ++t) {
    /* "Compute FP4 assignment" under (alpha^t, dq^t) and the tensor sums of Eq. 5
     * with the stored E4M3 scales dd^t. */
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
      double sA = 0.0, sB = 0.0;
      for (int64_t b = 0; b < nbc; ++b) {
        int64_t i = r * nbc + b;
        if (dd[i] == 0) continue;
        double m[REF_BLOCK], A, B;
        soar_ref_round_block_w(W + r * ld + b * REF_BLOCK, h ? h + b * REF_BLOCK : NULL, alpha,
                               dq[i], m, &A, &B);
        double v = (double)soar_ref_e4m3_decode(dd[i]);
        sA += A * v;
        sB += B * v * v;
      }
      rowA[r] = sA;
      rowB[r] = sB;
    }
    double num = 0.0, den = 0.0;
    for (int64_t r = 0; r < rows; ++r) { num += rowA[r]; den += rowB[r]; }
    /* Eq. 5: alpha^(t+1); one rounding of the binary64 quotient. A zero
     * denominator (every code zero) keeps alpha. */
    float alpha_new = (den > 0.0) ? (float)(num / den) : alpha;
    if (cfg->flags & REF_FLAG_KEEP_ALPHA) alpha_new = alpha;      /* Sec. 3.3 alone: alpha stays Eq. 1's */

    /* Eq. 6 with the same codes and the new alpha, then DSS per block. */
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < rows; ++r) {
      double sL = 0.0;
      for (int64_t b = 0; b < nbc; ++b) {
        int64_t i = r * nbc + b;
        if (dd[i] == 0) continue;
        const uint16_t* w = W + r * ld + b * REF_BLOCK;
        const float* hb = h ? h + b * REF_BLOCK : NULL;
        double m[REF_BLOCK], A, B;
        soar_ref_round_block_w(w, hb, alpha, dq[i], m, &A, &B);
        float center = (cfg->flags & REF_FLAG_KEEP_BLOCK_SCALE)
                           ? soar_ref_e4m3_decode(dd[i])                  /* Sec. 3.3 alone: around the stored scale */
                           : soar_ref_block_scale(A, B, alpha_new, dd[i]);
        float ndq;
        uint8_t nd;
        double L, wA, wB, gap;
        dss_block(w, hb, alpha_new, center, cfg, &ndq, &nd, &L, &wA, &wB, &gap);
        dq[i] = ndq;
        dd[i] = nd;
        sL += L;
        if (tie_flags && gap < tie_rel) tie_flags[i] = 1;
      }
      rowL[r] = sL;
    }
    alpha = alpha_new;
    double sse_new = 0.0;
    for (int64_t r = 0; r < rows; ++r) sse_new += rowL[r];
    trace_alpha[t + 1] = (double)alpha;
    trace_sse[t + 1] = sse_new;
    *iters_run = t + 1;
    /* Sec. 4.1: early stop on the relative MSE improvement. */
    int stop = 0;
    if (cfg->early_stop_rel > 0.0f) {
      if (sse == 0.0) stop = 1;
      else if ((sse - sse_new) / sse < (double)cfg->early_stop_rel) stop = 1;
    }
    sse = sse_new;
    if (stop) break;
  }

  /* Algorithm 1 "Reconstruction": codes from (alpha, dq), stored scale dd. */
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r) {
    for (int64_t b = 0; b < nbc; ++b) {
      int64_t i = r * nbc + b;
      const uint16_t* w = W + r * ld + b * REF_BLOCK;
      double m[REF_BLOCK], A, B;
      if (dd[i] == 0) memset(m, 0, sizeof(m));
      else soar_ref_round_block(w, alpha, dq[i], m, &A, &B);
      for (int j = 0; j < REF_BLOCK; j += 2) {
        int lo = soar_ref_e2m1_code(m[j]) | ((w[j] >> 15) << 3);
        int hi = soar_ref_e2m1_code(m[j + 1]) | ((w[j + 1] >> 15) << 3);
        out_packed[(r * cols + b * REF_BLOCK + j) / 2] = (uint8_t)(lo | (hi << 4));
      }
      out_scales[i] = dd[i];
    }
  }
  *out_alpha = alpha;
  free(dq); free(dd); free(rowA); free(rowB); free(rowL);
  return status;
}

/* Algorithm 1 as the paper states it: every h_j = 1. */
int soar_ref_quantize(const uint16_t* W, int64_t rows, int64_t cols, int64_t ld,
                      const soar_ref_cfg* cfg, uint8_t* out_packed, uint8_t* out_scales,
                      float* out_alpha, int32_t* iters_run, double* trace_alpha,
                      double* trace_sse, uint8_t* tie_flags, double tie_rel,
                      double* out_sumsq) {
  return soar_ref_quantize_weighted(W, rows, cols, ld, NULL, cfg, out_packed, out_scales, out_alpha,
                                    iters_run, trace_alpha, trace_sse, tie_flags, tie_rel, out_sumsq);
}

/* Eq. 3 + Eq. 4 on stored outputs: sum h_j (W - Q*alpha*value(d))^2 and sum h_j W^2,
 * element by element in binary64 (h == NULL: h_j = 1). */
void soar_ref_dequant_error_weighted(const uint16_t* W, int64_t rows, int64_t cols, int64_t ld,
                                     const float* h, const uint8_t* packed, const uint8_t* scales,
                                     float alpha, double* out_sse, double* out_sumsq) {
  static const double grid[8] = {0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0};
  const int64_t nbc = cols / REF_BLOCK;
  double sse = 0.0, ss = 0.0;
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t c = 0; c < cols; ++c) {
      double w = (double)soar_ref_bf16_to_f32(W[r * ld + c]);
      uint8_t byte = packed[(r * cols + c) / 2];
      int code = (c & 1) ? (byte >> 4) : (byte & 0xF);
      double q = grid[code & 7] * ((code & 8) ? -1.0 : 1.0);
      double s = (double)alpha * (double)soar_ref_e4m3_decode(scales[r * nbc + c / REF_BLOCK]);
      double hj = h ? (double)h[c] : 1.0;
      double e = w - q * s;
      sse += hj * (e * e);
      ss += hj * (w * w);
    }
  *out_sse = sse;
  *out_sumsq = ss;
}

void soar_ref_dequant_error(const uint16_t* W, int64_t rows, int64_t cols, int64_t ld,
                            const uint8_t* packed, const uint8_t* scales, float alpha,
                            double* out_sse, double* out_sumsq) {
  soar_ref_dequant_error_weighted(W, rows, cols, ld, NULL, packed, scales, alpha, out_sse, out_sumsq);
}

int soar_ref_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ------------------------------------------------------------------ MXFP4
 *
 * Sec. 4.3 "DSS on MXFP4" applies the decoupled search of Sec. 3.3 to the other microscaling
 * format: E2M1 elements in blocks of 32 with one shared power-of-two scale (an E8M0 byte,
 * value 2^(code - 127)) and no tensor-wide scale.  The paper reports results and no
 * procedure, so what follows is a reading (parity unpinned by the paper; pinned by the
 * CPU tests against a separate NumPy restatement, brute force and the format's definition):
 *
 *   plain MXFP4   the format's own rule: shared exponent floor(log2 bmax) - 2 (2 is the
 *                 exponent of E2M1's largest value, 6 = 1.5 * 2^2), elements rounded to nearest
 *                 (ties to even) and saturated at 6.
 *   with DSS      Sec. 3.3 (i)-(ii) with alpha = 1: the high-precision scale is Eq. 1's
 *                 max-based one, D* = fl32(bmax / 6); dequantization candidates are the n_dq
 *                 E8M0 values around D* (App. B.3's rule on powers of two: with c_f the largest
 *                 code whose value is <= D*, codes c_f-(n/2-1) .. c_f+n/2; n = 1: the nearer of
 *                 c_f, c_f+1, the lower one on a tie), quantization candidates D* * beta_k on
 *                 App. B.3's multiplier grid; every pair is scored by Eq. 8 and the first
 *                 minimum in (beta, code) order is kept.  For n_dq = 2 the plain rule's
 *                 exponent is always one of the two candidates.
 *
 * Blocks whose largest magnitude is below 2^-120 (or zero) are stored as zero blocks: scale
 * code 0 and zero codes (their sign bits kept).
 */
#define REF_MX_BLOCK 32

double soar_ref_e8m0_decode(uint8_t code) { return ldexp(1.0, (int)code - 127); }

/* Largest e with 2^e <= v, for finite v > 0. */
static int mx_floor_log2(float v) {
  int e;
  (void)frexpf(v, &e);          /* v = m * 2^e, m in [0.5, 1) */
  return e - 1;
}

/* The plain rule's scale code for a block maximum. */
uint8_t soar_ref_mx_plain_code(float bmax) {
  int c = mx_floor_log2(bmax) - 2 + 127;
  return (uint8_t)(c < 0 ? 0 : (c > 254 ? 254 : c));
}

/* E8M0 codes around a positive scale; returns how many (ascending, clipped to [0, 254],
 * duplicates dropped). */
int soar_ref_mx_candidates(float center, int n, uint8_t* out) {
  int cf = mx_floor_log2(center) + 127;
  int lo, hi;
  if (n <= 1) {
    double mid = 1.5 * ldexp(1.0, cf - 127);
    lo = hi = ((double)center > mid) ? cf + 1 : cf;
  } else {
    lo = cf - (n / 2 - 1);
    hi = cf + n / 2;
  }
  int cnt = 0;
  for (int c = lo; c <= hi; ++c) {
    int cc = c < 0 ? 0 : (c > 254 ? 254 : c);
    if (cnt > 0 && out[cnt - 1] == (uint8_t)cc) continue;
    out[cnt++] = (uint8_t)cc;
  }
  return cnt;
}

/* Eq. 2 for a block of 32 under quantization scale dq (alpha = 1): r = fl32(1/dq),
 * x_j = fl32(|W_j| * r), m_j = E2M1 rounding of x_j. */
void soar_ref_mx_round_block(const uint16_t* w, float dq, double* m) {
  float r = 1.0f / dq;
  for (int j = 0; j < REF_MX_BLOCK; ++j) {
    float x = fabsf(soar_ref_bf16_to_f32(w[j])) * r;
    m[j] = soar_ref_e2m1_round((double)x);
  }
}

/* Eq. 8's error of a block of 32 for magnitudes m and scale code d: sum (|W_j| - m_j 2^(d-127))^2. */
double soar_ref_mx_block_error(const uint16_t* w, const double* m, uint8_t d) {
  double s = soar_ref_e8m0_decode(d), L = 0.0;
  for (int j = 0; j < REF_MX_BLOCK; ++j) {
    double e = fabs((double)soar_ref_bf16_to_f32(w[j])) - m[j] * s;
    L += e * e;
  }
  return L;
}

/*
 * MXFP4 quantization of W[rows][ld] (cols used, cols % 32 == 0).  n_beta == 0: the plain rule;
 * otherwise the search above with n_dq codes and n_beta multipliers of step step_pct/100.
 *   out_packed  rows*cols/2 bytes, nibble layout as soar_ref_quantize
 *   out_scales  rows*cols/32 E8M0 bytes, row-major
 *   out_sse     sum (W - What)^2;  out_sumsq  sum W^2 (may be NULL)
 *   tie_flags   per block (may be NULL): 1 if the best two distinct outcomes were closer than tie_rel
 * Returns status bits (REF_STATUS_NONFINITE, REF_STATUS_ZERO_TENSOR).
 */
int soar_ref_mx_quantize(const uint16_t* W, int64_t rows, int64_t cols, int64_t ld, int n_dq, int n_beta,
                         int step_pct, uint8_t* out_packed, uint8_t* out_scales, double* out_sse,
                         double* out_sumsq, uint8_t* tie_flags, double tie_rel) {
  const int64_t nbc = cols / REF_MX_BLOCK;
  int status = 0;
  double sumsq = 0.0;
  float amax = 0.0f;
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t c = 0; c < cols; ++c) {
      float v = fabsf(soar_ref_bf16_to_f32(W[r * ld + c]));
      if (!(v <= 3.4e38f)) status |= REF_STATUS_NONFINITE;
      if (v > amax) amax = v;
      sumsq += (double)v * (double)v;
    }
  if (out_sumsq) *out_sumsq = sumsq;
  *out_sse = 0.0;
  if (status) return status;
  if (amax == 0.0f) status |= REF_STATUS_ZERO_TENSOR;
  double* rowL = (double*)calloc((size_t)rows, sizeof(double));
#ifdef _OPENMP
#pragma omp parallel for schedule(static)
#endif
  for (int64_t r = 0; r < rows; ++r) {
    static _Thread_local double mk[REF_MAX_BETA][REF_MX_BLOCK];
    static _Thread_local double Lk[REF_MAX_BETA][REF_MAX_DQ];
    double acc = 0.0;
    for (int64_t b = 0; b < nbc; ++b) {
      const uint16_t* w = W + r * ld + b * REF_MX_BLOCK;
      float bmax = 0.0f;
      for (int j = 0; j < REF_MX_BLOCK; ++j) {
        float v = fabsf(soar_ref_bf16_to_f32(w[j]));
        if (v > bmax) bmax = v;
      }
      double m[REF_MX_BLOCK];
      uint8_t code = 0;
      if (tie_flags) tie_flags[r * nbc + b] = 0;
      if (bmax < 0x1p-120f) {
        for (int j = 0; j < REF_MX_BLOCK; ++j) m[j] = 0.0;
      } else if (n_beta == 0) {
        code = soar_ref_mx_plain_code(bmax);
        soar_ref_mx_round_block(w, (float)soar_ref_e8m0_decode(code), m);
      } else {
        float center = bmax / 6.0f;
        uint8_t dc[REF_MAX_DQ];
        int nd = soar_ref_mx_candidates(center, n_dq, dc);
        double best = 0.0;
        int bk = -1, bd = -1;
        for (int k = 0; k < n_beta; ++k) {
          float dq = center * soar_ref_beta(k, n_beta, step_pct);
          soar_ref_mx_round_block(w, dq, mk[k]);
          for (int d = 0; d < nd; ++d) {
            double L = soar_ref_mx_block_error(w, mk[k], dc[d]);
            Lk[k][d] = L;
            if (bk < 0 || L < best) { best = L; bk = k; bd = d; }
          }
        }
        double second = 1e300;
        for (int k = 0; k < n_beta; ++k)
          for (int d = 0; d < nd; ++d) {
            if (dc[d] == dc[bd] && memcmp(mk[k], mk[bk], sizeof(mk[k])) == 0) continue;
            if (Lk[k][d] < second) second = Lk[k][d];
          }
        if (tie_flags && second < 1e300) {
          double gap = best > 0.0 ? (second - best) / best : (second > 0.0 ? 1e300 : 0.0);
          if (gap < tie_rel) tie_flags[r * nbc + b] = 1;
        }
        code = dc[bd];
        memcpy(m, mk[bk], sizeof(m));
      }
      acc += soar_ref_mx_block_error(w, m, code);
      for (int j = 0; j < REF_MX_BLOCK; j += 2) {
        int lo = soar_ref_e2m1_code(m[j]) | ((w[j] >> 15) << 3);
        int hi = soar_ref_e2m1_code(m[j + 1]) | ((w[j + 1] >> 15) << 3);
        out_packed[(r * cols + b * REF_MX_BLOCK + j) / 2] = (uint8_t)(lo | (hi << 4));
      }
      out_scales[r * nbc + b] = code;
    }
    rowL[r] = acc;
  }
  double sse = 0.0;
  for (int64_t r = 0; r < rows; ++r) sse += rowL[r];
  free(rowL);
  *out_sse = sse;
  return status;
}
