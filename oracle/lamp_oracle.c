/*
 * LampAttention forward pass -- CPU oracle (TEST INFRASTRUCTURE, not a product path).
 *
 * A plain, slow, step-by-step restatement of Algorithm 1 of the paper
 * ("LampAttention: Look-Ahead Mixed-Precision FlashAttention"), with the number
 * formats of Section 3.3 emulated exactly and the simulation rules of Section 4.1
 * (recursive round(c + a*b) accumulation, correctly rounded exponentials,
 * tiles 128 x 64 with N_k = 4 key sub-blocks).
 *
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call this
 * file.  It shares no code, header, table or constant with the CUDA library and
 * never includes or links anything from it.
 *
 * Every decision-path quantity is a deterministic function of the input bits:
 * IEEE single/double operations in a stated order (the file is compiled with
 * -ffp-contract=off so that no multiply-add is fused unless fma()/fmaf() is
 * written), exact sums, or library exp()/log() in double.
 *
 * Readings of the paper this file takes where the paper is silent or ambiguous
 * (each is listed, with the alternative, in the design notes of the repository):
 *   - rounding is round-to-nearest-even onto the real 8/16-bit grids, including
 *     their subnormals; overflow saturates to +-448 (Sec. 3.3 only prevents it);
 *   - the softmax scale is folded into Q once, in fp32 (Sec. 3.3 wants the 1/sqrt(d) scaling in
 *     place before the accumulation starts);
 *   - a warp owns b_q = 32 query rows (Sec. 4.1 gives only b_q N_q = 128);
 *   - 16-bit logits are a sequential fp64 fma chain, rounded once to e4m11 (optional mode: the
 *     per-step e4m11 recursion instead);
 *   - among equally small stage-2 recompute sets the smallest bitmask wins;
 *   - (optional mode) the compact layout's branch recomputes the remaining 8-bit sub-blocks of a
 *     tile with two or more marked sub-blocks exactly like stage-2 recomputations.
 * Parity unpinned (no value in the paper fixes them): b_q = 32, the stage-2
 * tie-break, the 16-bit accumulation rounding, the truncated-maximum shift.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define BQ 32          /* query rows per warp (group)            Alg. 1: the work of one warp */
#define BQM 64         /* the largest group size on offer (group_rows = 64); sizes of the per-unit arrays */
#define BK 16          /* keys per sub-block                     Sec. 4.1: 64 / N_k   */
#define NK 4           /* sub-blocks per key tile                Sec. 4.1             */
#define TK (BK * NK)   /* keys per tile                                                 */

#define LAMP_FORCE_16BIT 1u
#define LAMP_FORCE_8BIT  2u
#define LAMP_NO_STAGE1   4u
#define LAMP_COMPACT_BRANCH 16u  /* Sec. 3.3 "Register layout": the compact layout's branch (see below) */
#define LAMP_SR_E4M3     64u     /* stochastic rounding in the 8-bit accumulation (Sec. 3.3, last sentence of the
                                    paragraph on formats), see lamp_oracle_sr_e4m3 */
#define LAMP_H16_SEQ     32u     /* 16-bit logits by per-step e4m11 accumulation (the other reading, see logit16) */

typedef struct {
  int32_t batch, heads_q, heads_kv, seqlen, head_dim;
  int32_t causal, window;
  float scale, tau, delta;
  uint32_t flags;
  uint32_t sr_seed;      /* seed of the counter-based generator of LAMP_SR_E4M3 */
  int32_t group_rows;    /* b_q: query rows that decide together (a "warp" of Alg. 1); 0 = 32.  Sec. 4.1 fixes only
                            b_q N_q = 128; 16 is the other instance offered, to bracket that reading */
} lamp_oracle_params;

typedef struct {
  uint64_t subblocks_active, stage1_flagged, stage2_flagged;
  uint64_t hist_flagged_per_tile[5];
  uint64_t sat_e4m3, sat_e4m11, exp16_gt1, big_rowsum;
} lamp_oracle_stats;

/* ------------------------------------------------------------------ formats */

static float bf16_to_float(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

/* Round |x| to the nearest multiple of the local quantum 2^(max(e, emin) - mbits),
 * e = floor(log2 |x|), ties to even, then saturate at vmax.  With emin = -6 and
 * mbits = 3 this is the e4m3 grid of Sec. 3.3 (max 448, subnormal quantum 2^-9);
 * mbits = 11 gives e4m11 (same exponent field, subnormal quantum 2^-17). */
static double rne_grid(double x, int emin, int mbits, double vmax) {
  if (x == 0.0 || isnan(x)) return x;
  double a = fabs(x);
  if (isinf(a)) return copysign(vmax, x);
  int e;
  frexp(a, &e);           /* a = m * 2^e, m in [0.5, 1)  =>  floor(log2 a) = e - 1 */
  e -= 1;
  if (e < emin) e = emin;
  double q = ldexp(1.0, e - mbits);
  double r = nearbyint(a / q) * q;   /* default rounding mode: nearest, ties to even */
  if (r > vmax) r = vmax;
  return copysign(r, x);
}

float lamp_oracle_rne_e4m3(float x) { return (float)rne_grid((double)x, -6, 3, 448.0); }
float lamp_oracle_rne_e4m11(double x) { return (float)rne_grid(x, -6, 11, 448.0); }

/* Drop the low 8 mantissa bits of an e4m11 value (toward zero): Sec. 3.3,
 * the running maxima reach the 8-bit shift by truncation of their low mantissa bits. */
float lamp_oracle_trunc_e4m3(float x) {
  if (x == 0.0f || isinf(x)) return x;
  double a = fabs((double)x);
  int e;
  frexp(a, &e);
  e -= 1;
  if (e < -6) e = -6;
  double q = ldexp(1.0, e - 3);
  return (float)copysign(floor(a / q) * q, (double)x);
}

/* e4m3 byte of a value already on the grid; -0 is stored as +0. */
uint8_t lamp_oracle_enc_e4m3(float v) {
  double a = fabs((double)v);
  if (a == 0.0) return 0;
  uint8_t s = v < 0 ? 0x80 : 0;
  if (a < ldexp(1.0, -6)) return s | (uint8_t)(a / ldexp(1.0, -9));
  int e;
  double m = frexp(a, &e);  /* m in [0.5,1) */
  e -= 1;
  int mant = (int)((m * 2.0 - 1.0) * 8.0);
  return s | (uint8_t)(((e + 7) << 3) | mant);
}

float lamp_oracle_dec_e4m3(uint8_t b) {
  int E = (b >> 3) & 15, M = b & 7;
  double v = E ? ldexp(1.0 + M / 8.0, E - 7) : ldexp(M / 8.0, -6);
  return (float)((b & 0x80) ? -v : v);
}

/* Round to nbits significant bits, ties to even (no exponent limits). */
static double rne_sig(double x, int nbits) {
  if (x == 0.0 || isnan(x) || isinf(x)) return x;
  int e;
  frexp(fabs(x), &e);
  double q = ldexp(1.0, e - nbits);
  return copysign(nearbyint(fabs(x) / q) * q, x);
}

/* Unsigned shift format ue5m3 (Sec. 3.3: range up to 896), exponent bias 15. */
uint8_t lamp_oracle_enc_ue5m3(float s) {
  if (s == 0.0f) return 0;
  int e;
  double m = frexp((double)s, &e);
  e -= 1;
  return (uint8_t)(((e + 15) << 3) | (int)((m * 2.0 - 1.0) * 8.0));
}

float lamp_oracle_dec_ue5m3(uint8_t p) {
  int E = p >> 3, M = p & 7;
  return (float)(E ? ldexp(1.0 + M / 8.0, E - 15) : ldexp(M / 8.0, -14));
}

/* Exponential format: ue5m3 with the bias that maps 0xF8 to 1.0 (Sec. 3.3):
 * value = 2^(E-31) (1 + M/8) for E >= 1, 2^-30 M/8 for E = 0. */
double lamp_oracle_dec_exp8(uint8_t b) {
  int E = b >> 3, M = b & 7;
  return E ? ldexp(1.0 + M / 8.0, E - 31) : ldexp(M / 8.0, -30);
}

/* Correctly rounded exp(-s) on the 8-bit exponential grid, as its byte. */
static uint8_t exp8_byte(double s) {
  double v = exp(-s);
  double r = rne_grid(v, -30, 3, 1.0);
  if (r == 0.0) return 0;
  if (r < ldexp(1.0, -30)) return (uint8_t)(r / ldexp(1.0, -33));
  int e;
  double m = frexp(r, &e);
  e -= 1;
  return (uint8_t)(((e + 31) << 3) | (int)((m * 2.0 - 1.0) * 8.0));
}

/* The 256-entry table of Sec. 3.3: index = shift byte (ue5m3), entry = exp byte. */
uint8_t lamp_oracle_lut8(uint8_t p) { return exp8_byte((double)lamp_oracle_dec_ue5m3(p)); }

static uint8_t g_lut8[256];   /* the table itself, filled before any unit runs */

/* 16-bit exponential (ue5m11 with the same bias idea): exp(a) correctly rounded
 * to 12 significant bits, subnormal quantum 2^-41 below 2^-30, no upper clamp. */
float lamp_oracle_exp16(float a) {
  double v = exp((double)a);
  double r;
  if (v < ldexp(1.0, -30)) r = nearbyint(v / ldexp(1.0, -41)) * ldexp(1.0, -41);
  else r = rne_sig(v, 12);
  return (float)r;   /* 12 significant bits: exact in fp32 unless it overflows to inf */
}

void lamp_oracle_exp16_array(const float* in, float* out, size_t n) {
  for (size_t i = 0; i < n; ++i) out[i] = lamp_oracle_exp16(in[i]);
}

/* --------------------------------------------------------- stage 2 (eq. 8) */

/* xi[theta][j]: per sub-block, per query sum of (omega_hat - e) e  (0 for sub-blocks
 * that are not free).  Returns the recompute set as a bitmask over theta: the
 * smallest set (then the smallest bitmask) whose removal makes every query's kept
 * sum <= tau * omega_hat^2.  The stage-2 step of Algorithm 1 (solve the block-LAMP problem). */
static uint32_t stage2_rows(const double* xi, int ld, int nrows, const float* omega_hat, float tau,
                            uint32_t free_mask) {
  for (int size = 0; size <= NK; ++size) {
    for (uint32_t r = 0; r < (1u << NK); ++r) {
      if ((r & ~free_mask) != 0 || __builtin_popcount(r) != size) continue;
      int ok = 1;
      for (int j = 0; j < nrows && ok; ++j) {
        /* a row whose omega_hat has overflowed (or is 0 * inf) states no constraint: eq. (8) has no meaning for it */
        if (!isfinite(omega_hat[j])) continue;
        double kept = 0.0;
        for (int th = 0; th < NK; ++th)
          if (((free_mask & ~r) >> th) & 1u) kept += xi[th * ld + j];
        double rhs = ((double)tau * (double)omega_hat[j]) * (double)omega_hat[j];
        if (!(kept <= rhs)) ok = 0;
      }
      if (ok) return r;
    }
  }
  return free_mask;
}
uint32_t lamp_oracle_stage2(const double xi[NK][BQ], const float* omega_hat, float tau,
                            uint32_t free_mask) {
  return stage2_rows(&xi[0][0], BQ, BQ, omega_hat, tau, free_mask);
}

float lamp_oracle_chain16(const float* a, const float* b, int n);
float lamp_oracle_sr_e4m3(float t, uint32_t u20);
uint32_t lamp_oracle_sr_bits(uint32_t seed, uint32_t bh, uint32_t j, uint32_t i, uint32_t kk);

/* A 16-bit logit (the high-precision recomputation of a sub-block in Alg. 1).
 * Default reading: the exact dot product as a sequential fp64 fma chain over the channels, times the
 * scale, rounded once to e4m11 (Sec. 3.3 names e4m11 as the 16-bit accumulation format; taken as
 * the format of the result).
 * LAMP_H16_SEQ, the other reading: the same recursion as the 8-bit pass (Sec. 4.1, round(c + a*b) with
 * the multiplication and addition in fp32), every partial sum rounded to e4m11, on the pre-scaled query. */
static float logit16(const lamp_oracle_params* p, const uint16_t* krow, const uint16_t* qrow,
                     const float* qsrow, int D) {
  if (p->flags & LAMP_H16_SEQ) {
    float kf[256];
    for (int kk = 0; kk < D; ++kk) kf[kk] = bf16_to_float(krow[kk]);
    return lamp_oracle_chain16(kf, qsrow, D);
  }
  double acc = 0.0;
  for (int kk = 0; kk < D; ++kk)
    acc = fma((double)bf16_to_float(krow[kk]), (double)bf16_to_float(qrow[kk]), acc);
  return lamp_oracle_rne_e4m11((double)p->scale * acc);
}

/* ---------------------------------------------------------------- checksum */

static uint64_t mix64(uint64_t x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}

/* ------------------------------------------------------------------ a unit */

/* Sum of one query's 64 exponentials, exact: every term is a multiple of 2^-41, so
 * the sum is taken in integer units of 2^-41.  (Terms of 2^40 or more can only come
 * from a recomputed logit far above the running maximum; then a plain double sum is
 * used and the event is reported.)  *big is set when the sum reaches 2^12, beyond
 * which a double no longer holds it exactly. */
static double exact_rowsum(const float Ef[TK][BQM], int j, int* big) {
  unsigned __int128 acc = 0;
  int huge = 0;
  double plain = 0.0;
  for (int i = 0; i < TK; ++i) {
    double e = (double)Ef[i][j];
    plain += e;
    if (!(e < 1099511627776.0)) huge = 1;
    else acc += (unsigned __int128)ldexp(e, 41);
  }
  double R = huge ? plain : ldexp((double)acc, -41);
  if (!(R < 4096.0)) *big = 1;
  return R;
}

static int pair_valid(const lamp_oracle_params* p, int64_t i, int64_t j) {
  if (i >= p->seqlen || j >= p->seqlen) return 0;   /* the last group / tile of a ragged sequence */
  if (p->causal && i > j) return 0;
  if (p->window > 0 && j - i >= p->window) return 0;
  return 1;
}

/* One unit = (batch b, query head h, group g of 32 query rows): Algorithm 1's
 * per-warp body over all key tiles in ascending order.
 * out [32][D], lse [32], flags [ceil(N/64)], checks [ceil(N/64)][2] (or NULL),
 * y8 / e8 [32][N] bytes (or NULL).                                              */
static void oracle_unit(const uint16_t* q, const uint16_t* k, const uint16_t* v,
                        const lamp_oracle_params* p, int b, int h, int g, float* out,
                        float* lse, uint8_t* flags, uint64_t* checks, uint8_t* y8d,
                        uint8_t* e8d, lamp_oracle_stats* st) {
  const int D = p->head_dim, N = p->seqlen;
  const int hk = h / (p->heads_q / p->heads_kv);
  const int bq = p->group_rows ? p->group_rows : BQ;   /* rows bq .. BQM-1 of the arrays below do not exist */
  const int bqo = bq > BQ ? BQM : BQ;                  /* rows per unit in the output arrays */
  const uint16_t* Q = q + ((int64_t)(b * p->heads_q + h) * N + (int64_t)g * bq) * D;
  const uint16_t* K = k + (int64_t)(b * p->heads_kv + hk) * N * D;
  const uint16_t* V = v + (int64_t)(b * p->heads_kv + hk) * N * D;
  const int ntiles = (N + TK - 1) / TK;
  const int64_t j0 = (int64_t)g * bq;

  float* qs = (float*)malloc(sizeof(float) * BQM * D);
  double* O = (double*)calloc((size_t)BQM * D, sizeof(double));
  float mu[BQM], omega[BQM];
  for (int j = 0; j < BQM; ++j) {
    mu[j] = -INFINITY;
    omega[j] = 0.0f;
    for (int c = 0; c < D; ++c) qs[j * D + c] = (j < bq && j0 + j < N) ? bf16_to_float(Q[j * D + c]) * p->scale : 0.0f;
  }
  if (y8d) memset(y8d, 0x7F, (size_t)bqo * N);
  if (e8d) memset(e8d, 0xFF, (size_t)bqo * N);

  float Y8[TK][BQM], Y16[TK][BQM], Ef[TK][BQM];
  uint8_t E8[TK][BQM], val[TK][BQM];

  for (int t = 0; t < ntiles; ++t) {
    const int64_t i0 = (int64_t)t * TK;
    flags[t] = 0;
    if (checks) checks[2 * t] = checks[2 * t + 1] = 0;
    int active[NK] = {0, 0, 0, 0}, any = 0;
    for (int i = 0; i < TK; ++i)
      for (int j = 0; j < BQM; ++j) {
        val[i][j] = (uint8_t)(j < bq && pair_valid(p, i0 + i, j0 + j));
        if (val[i][j]) active[i / BK] = 1, any = 1;
      }
    if (!any) continue;

    /* Alg. 1, low-precision accumulation of Y; Sec. 4.1: round(c + a*b), fp32 fma. */
    for (int i = 0; i < TK; ++i)
      for (int j = 0; j < BQM; ++j) {
        float c = 0.0f;
        if (!val[i][j]) { Y8[i][j] = 0.0f; continue; }   /* never used, and may lie past the tensors */
        for (int kk = 0; kk < D; ++kk)
          {
            float tkk = fmaf(bf16_to_float(K[(i0 + i) * D + kk]), qs[j * D + kk], c);
            if (p->flags & LAMP_SR_E4M3)
              c = lamp_oracle_sr_e4m3(tkk, lamp_oracle_sr_bits(p->sr_seed, (uint32_t)(b * p->heads_q + h),
                                                               (uint32_t)(j0 + j), (uint32_t)(i0 + i), (uint32_t)kk));
            else
              c = lamp_oracle_rne_e4m3(tkk);
          }
        Y8[i][j] = c;
      }

    /* maximum low-precision logit per sub-block and query (the C matrix of Sec. 3.1) */
    float cm8[NK][BQM];
    for (int th = 0; th < NK; ++th)
      for (int j = 0; j < BQM; ++j) {
        float m = -INFINITY;
        for (int i = th * BK; i < (th + 1) * BK; ++i)
          if (val[i][j] && Y8[i][j] > m) m = Y8[i][j];
        cm8[th][j] = m;
        if (m == 448.0f) st->sat_e4m3++;
      }

    /* threats T_theta against the maxima at tile start, then the visiting order */
    float T[NK];
    int order[NK], nact = 0;
    for (int th = 0; th < NK; ++th) {
      T[th] = -INFINITY;
      for (int j = 0; j < BQM; ++j)
        if (cm8[th][j] > -INFINITY) {
          float d = cm8[th][j] - mu[j];
          if (d > T[th]) T[th] = d;
        }
      if (active[th]) order[nact++] = th;
    }
    for (int a = 1; a < nact; ++a) {           /* stable insertion sort, T descending */
      int x = order[a], c = a - 1;
      while (c >= 0 && T[order[c]] < T[x]) { order[c + 1] = order[c]; --c; }
      order[c + 1] = x;
    }

    /* stage 1: eq. (7) on the running maxima, sub-blocks in threat order */
    float muh[BQM];
    memcpy(muh, mu, sizeof(mu));
    uint32_t Theta = 0;
    const int skip1 = (p->flags & (LAMP_FORCE_8BIT | LAMP_NO_STAGE1)) != 0;
    for (int a = 0; a < nact; ++a) {
      const int th = order[a];
      int pass = 1;
      if (p->flags & LAMP_FORCE_16BIT) pass = 0;
      else if (!skip1)
        for (int j = 0; j < BQM; ++j) {
          if (!(cm8[th][j] > -INFINITY)) continue;
          if (isinf(muh[j])) { pass = 0; break; }
          float margin = fabsf(muh[j]) * p->delta;
          float rhs = cm8[th][j] + margin;
          if (!(muh[j] > rhs)) { pass = 0; break; }
        }
      if (pass) continue;
      Theta |= 1u << th;
      for (int i = th * BK; i < (th + 1) * BK; ++i)
        for (int j = 0; j < BQM; ++j) {
          if (!val[i][j]) continue;
          Y16[i][j] = logit16(p, K + (size_t)(i0 + i) * D, Q + (size_t)j * D, qs + (size_t)j * D, D);
          if (fabsf(Y16[i][j]) == 448.0f) st->sat_e4m11++;
          if (Y16[i][j] > muh[j]) muh[j] = Y16[i][j];
        }
    }
    if (skip1)
      for (int j = 0; j < BQM; ++j)
        for (int th = 0; th < NK; ++th)
          if (cm8[th][j] > muh[j]) muh[j] = cm8[th][j];

    /* exponentials: 8-bit through the table, 16-bit correctly rounded */
    for (int i = 0; i < TK; ++i)
      for (int j = 0; j < BQM; ++j) {
        Ef[i][j] = 0.0f;
        E8[i][j] = 0xFF;
        if (!val[i][j]) continue;
        if ((Theta >> (i / BK)) & 1u) {
          float d = Y16[i][j] - muh[j];
          Ef[i][j] = lamp_oracle_exp16((float)rne_sig((double)d, 12));
          if (Ef[i][j] > 1.0f) st->exp16_gt1++;
        } else {
          float s = lamp_oracle_trunc_e4m3(muh[j]) - Y8[i][j];
          uint8_t pb = lamp_oracle_enc_ue5m3((float)rne_sig((double)s, 4));
          E8[i][j] = g_lut8[pb];
          Ef[i][j] = (float)lamp_oracle_dec_exp8(E8[i][j]);
        }
      }

    /* lambda_hat (high precision), exact row sums, omega_hat */
    float lam[BQM], omh[BQM];
    for (int j = 0; j < BQM; ++j) {
      float d = mu[j] - muh[j];
      lam[j] = isinf(mu[j]) ? 0.0f : (float)exp((double)d);
    }
    int bigrow = 0;
    for (int j = 0; j < BQM; ++j)
      omh[j] = (float)((double)lam[j] * (double)omega[j] + exact_rowsum(Ef, j, &bigrow));

    /* stage 2: block-LAMP problem, eq. (8) */
    uint32_t freem = 0, Rset = 0;
    for (int th = 0; th < NK; ++th)
      if (active[th] && !((Theta >> th) & 1u)) freem |= 1u << th;
    if (!(p->flags & (LAMP_FORCE_8BIT | LAMP_FORCE_16BIT)) && freem) {
      double xi[NK][BQM];
      for (int th = 0; th < NK; ++th)
        for (int j = 0; j < BQM; ++j) {
          double s = 0.0;
          if ((freem >> th) & 1u)
            for (int i = th * BK; i < (th + 1) * BK; ++i)
              if (val[i][j]) s += ((double)omh[j] - (double)Ef[i][j]) * (double)Ef[i][j];
          xi[th][j] = s;
        }
      Rset = stage2_rows(&xi[0][0], BQM, BQM, omh, p->tau, freem);
    }
    /* Compact register layout (Sec. 3.3, "Register layout"): when the two stages mark two or more
     * sub-blocks of the tile, the update of O falls back to 16 bits for the whole tile.  Reading taken
     * here: the sub-blocks still held in 8 bits join the stage-2 set and are recomputed under the rule
     * of Alg. 1's stage-2 recomputation (running maxima unchanged). */
    if ((p->flags & LAMP_COMPACT_BRANCH) && __builtin_popcount(Theta | Rset) >= 2) Rset = freem;

    /* dumps and checksums refer to the 8-bit pass before any stage-2 replacement */
    for (int i = 0; i < TK; ++i)
      for (int j = 0; j < BQM; ++j) {
        if (!val[i][j]) continue;
        uint8_t yb = lamp_oracle_enc_e4m3(Y8[i][j]);
        if (y8d) y8d[(size_t)j * N + i0 + i] = yb;
        if (e8d) e8d[(size_t)j * N + i0 + i] = E8[i][j];
        if (checks) {
          uint64_t idx = (uint64_t)(i * bqo + j) << 8;
          checks[2 * t] += mix64(idx | yb);
          checks[2 * t + 1] += mix64(idx | E8[i][j]);
        }
      }

    /* stage-2 recomputation with the maxima unchanged (Alg. 1) */
    for (int th = 0; th < NK; ++th) {
      if (!((Rset >> th) & 1u)) continue;
      for (int i = th * BK; i < (th + 1) * BK; ++i)
        for (int j = 0; j < BQM; ++j) {
          if (!val[i][j]) continue;
          float y = logit16(p, K + (size_t)(i0 + i) * D, Q + (size_t)j * D, qs + (size_t)j * D, D);
          if (fabsf(y) == 448.0f) st->sat_e4m11++;
          float d = y - muh[j];
          Ef[i][j] = lamp_oracle_exp16((float)rne_sig((double)d, 12));
          if (Ef[i][j] > 1.0f) st->exp16_gt1++;
        }
    }

    /* state update and P V (fp64 here) */
    float omn[BQM];
    for (int j = 0; j < BQM; ++j)
      omn[j] = (float)((double)lam[j] * (double)omega[j] + exact_rowsum(Ef, j, &bigrow));
    if (bigrow) st->big_rowsum++;
    for (int j = 0; j < BQM; ++j) {
      mu[j] = muh[j];
      omega[j] = omn[j];
      for (int c = 0; c < D; ++c) O[j * D + c] *= (double)lam[j];
      for (int i = 0; i < TK; ++i) {
        if (Ef[i][j] == 0.0f) continue;
        const double e = (double)Ef[i][j];
        for (int c = 0; c < D; ++c) O[j * D + c] += e * (double)bf16_to_float(V[(i0 + i) * D + c]);
      }
    }

    flags[t] = (uint8_t)(Theta | (Rset << 4));
    int nact_sb = 0;
    for (int th = 0; th < NK; ++th) nact_sb += active[th];
    st->subblocks_active += (uint64_t)nact_sb;
    st->stage1_flagged += (uint64_t)__builtin_popcount(Theta);
    st->stage2_flagged += (uint64_t)__builtin_popcount(Rset);
    st->hist_flagged_per_tile[__builtin_popcount(Theta | Rset)]++;
  }

  for (int j = 0; j < bqo; ++j) {
    if (j >= bq || j0 + j >= N) {   /* rows that do not exist: past the group, or past a ragged sequence */
      for (int c = 0; c < D; ++c) out[j * D + c] = 0.0f;
      lse[j] = 0.0f;
      continue;
    }
    for (int c = 0; c < D; ++c) out[j * D + c] = (float)(O[j * D + c] / (double)omega[j]);
    lse[j] = (float)((double)mu[j] + log((double)omega[j]));
  }
  free(qs);
  free(O);
}

/* ------------------------------------------------------------ entry points */

static void stats_add(lamp_oracle_stats* a, const lamp_oracle_stats* b) {
  uint64_t* x = (uint64_t*)a;
  const uint64_t* y = (const uint64_t*)b;
  for (size_t i = 0; i < sizeof(*a) / 8; ++i) x[i] += y[i];
}

/* Run the listed units.  q, k, v: host, bf16 bit patterns, contiguous
 * [B, H, N, D].  units: n_units triples (b, h, g).  Outputs are per unit:
 * out [n][32][D] fp32, lse [n][32], flags [n][ceil(N/64)] (bits 0-3 stage-1 set,
 * bits 4-7 stage-2 set), checks [n][ceil(N/64)][2] or NULL, y8 / e8 [n][32][N] or NULL.
 * N need not be a multiple of the tile sizes: rows and keys past N do not exist (rows past N of the
 * last group come back as zeros).
 * Returns 0, or -1 on an unsupported shape. */
int lamp_oracle_units(const uint16_t* q, const uint16_t* k, const uint16_t* v,
                      const lamp_oracle_params* p, int64_t n_units, const int32_t* units,
                      float* out, float* lse, uint8_t* flags, uint64_t* checks, uint8_t* y8,
                      uint8_t* e8, lamp_oracle_stats* stats) {
  if (p->seqlen <= 0 || p->heads_q % p->heads_kv || p->head_dim <= 0 || p->head_dim > 256 ||
      (p->group_rows != 0 && p->group_rows != 16 && p->group_rows != 32 && p->group_rows != 64) ||
      p->delta < 0.0f || (p->window > 0 && !p->causal))
    return -1;
  const int N = p->seqlen, D = p->head_dim, nt = (N + TK - 1) / TK;
  const int bqo = p->group_rows > BQ ? BQM : BQ;   /* rows per unit in out, lse, y8, e8 */
  lamp_oracle_stats total;
  memset(&total, 0, sizeof(total));
  for (int i = 0; i < 256; ++i) g_lut8[i] = lamp_oracle_lut8((uint8_t)i);
#pragma omp parallel
  {
    lamp_oracle_stats mine;
    memset(&mine, 0, sizeof(mine));
#pragma omp for schedule(dynamic, 1)
    for (int64_t u = 0; u < n_units; ++u)
      oracle_unit(q, k, v, p, units[3 * u], units[3 * u + 1], units[3 * u + 2],
                  out + (size_t)u * bqo * D, lse + (size_t)u * bqo, flags + (size_t)u * nt,
                  checks ? checks + (size_t)u * nt * 2 : NULL, y8 ? y8 + (size_t)u * bqo * N : NULL,
                  e8 ? e8 + (size_t)u * bqo * N : NULL, &mine);
#pragma omp critical
    stats_add(&total, &mine);
  }
  if (stats) *stats = total;
  return 0;
}

/* The rounding of Sec. 3.3 over an array (for checking a device's rounding routine in bulk). */
void lamp_oracle_rne_e4m3_array(const float* in, float* out, int64_t n) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) out[i] = lamp_oracle_rne_e4m3(in[i]);
}

/* Stochastic rounding onto the e4m3 grid (Sec. 3.3 proposes it against swamping; the paper does not
 * specify it further).  Reading taken here, in integer arithmetic so that any two implementations agree
 * bit for bit: with u a uniform 20-bit integer, the magnitude's fp32 bit pattern plus u, with the 20
 * mantissa bits below e4m3's three cleared, is the result: the value goes up to the next grid point
 * with probability (distance from the lower one) / (spacing), exactly, in units of 2^-20.  Below 2^-6
 * (the subnormal range, fixed spacing 2^-9) the magnitude is first moved into [2^-6, 2^-5), whose
 * spacing is 2^-9, by one fp32 addition, and moved back afterwards.  Magnitudes beyond 448 saturate. */
float lamp_oracle_sr_e4m3(float t, uint32_t u20) {
  float a = fabsf(t);
  float off = a < 0.015625f ? 0.015625f : 0.0f;
  float s = a + off;
  uint32_t bits;
  memcpy(&bits, &s, 4);
  bits = (bits + (u20 & 0xFFFFFu)) & 0xFFF00000u;
  float r;
  memcpy(&r, &bits, 4);
  r = r - off;
  if (r > 448.0f) r = 448.0f;
  return copysignf(r, t);
}

/* The 20 random bits of one accumulation step: a counter-based generator (a 32-bit integer hash of
 * the step's coordinates: batch * heads + head, absolute query row, absolute key, channel), so that
 * every implementation draws the same bits whatever its order of evaluation. */
uint32_t lamp_oracle_sr_bits(uint32_t seed, uint32_t bh, uint32_t j, uint32_t i, uint32_t kk) {
  uint32_t x = seed ^ (bh * 0x27D4EB2Fu) ^ (j * 0x85EBCA77u) ^ (i * 0x9E3779B1u) ^ (kk * 0xC2B2AE3Du);
  x ^= x >> 16; x *= 0x7FEB352Du;
  x ^= x >> 15; x *= 0x846CA68Bu;
  x ^= x >> 16;
  return x >> 12;
}

/* The same recursion on the 16-bit grid: c <- RNE_e4m11(fmaf(a[t], b[t], c)), t ascending, c0 = +0
 * (the fp32 result of the fused multiply-add is exact in double, so one rounding follows it). */
float lamp_oracle_chain16(const float* a, const float* b, int n) {
  float c = 0.0f;
  for (int t = 0; t < n; ++t) c = lamp_oracle_rne_e4m11((double)fmaf(a[t], b[t], c));
  return c;
}

/* One low-precision dot product on its own (for the accumulation-order pins):
 * c <- RNE_e4m3(fmaf(a[t], b[t], c)), t ascending, c0 = +0. */
float lamp_oracle_chain8(const float* a, const float* b, int n) {
  float c = 0.0f;
  for (int t = 0; t < n; ++t) c = lamp_oracle_rne_e4m3(fmaf(a[t], b[t], c));
  return c;
}
