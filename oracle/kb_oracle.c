/*
 * kb_oracle.c -- plain CPU oracle for the candidate screen, the timing
 * adjudication and the survivor selection.
 *
 * THIS IS TEST INFRASTRUCTURE.  It exists so that the CUDA library can be
 * checked element by element against something slow and obviously correct.
 * It shares no code, header, table or helper with the CUDA path and is never
 * linked into, imported by or called from the product.
 *
 * Everything is the definition written out: one loop per definition, in the
 * order the definition states, no blocking, no fusion, no reordering.
 * All floating point is IEEE-754 binary32, round-to-nearest-even (binary64 in
 * kbo_screen_f64, the gate for double-precision tensors).  Build with
 *     gcc -O2 -std=c99 -ffp-contract=off -fPIC -shared
 * (no -ffast-math, no FTZ/DAZ) so that no multiply-add is fused and
 * subnormals are honoured.
 *
 * What the paper fixes and what is a reading of it:
 *   - The gate is the Verifier's "checks output correctness against the
 *     reference" (Sec. 3.4, Evaluation Plane) = the correctness indicator
 *     K(p) "passes task and numerical tests" (Sec. 3.1).  The paper prints no
 *     tolerance formula; the reading used here is the asymmetric
 *     |c - r| <= atol + rtol*|r| test, NaN never matching (see kbo_screen).
 *   - "Adjudicated latency" (Algorithm 1) is read as the median of the
 *     repeated timings, reported with the inter-quartile range; ranking under
 *     noise (Appendix, Relative Variability Metrics) is supported by pairwise
 *     doubled Mann-Whitney win counts (see kbo_quantiles, kbo_wins).
 *   - The promotion decision (Sec. 3.2; Sec. 3.4 "ranks candidates ... with
 *     deterministic tie-breaking ... promotes the top fraction") is
 *     kbo_select.
 *
 * Pins: every function here is pinned by the CPU tests (worked examples
 * stored under tests/golden, numpy/scipy special cases, brute force over small
 * alphabets, invariants).  Nothing in this file is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* dtype codes of this oracle's own interface */
enum { KBO_F32 = 0, KBO_F16 = 1, KBO_BF16 = 2, KBO_F8E4M3 = 3, KBO_F8E5M2 = 4 };

/* mask kinds */
enum { KBO_MASK_NONE = 0, KBO_MASK_STRIDED = 1, KBO_MASK_BITMAP = 2 };

typedef struct {
  uint64_t mismatch_count;
  uint64_t nan_count;
  uint64_t inf_count;
  int64_t argmax_idx;
  float max_abs_err;
  float max_rel_err;
  uint32_t pass;
  uint32_t reserved;
} kbo_screen_result;

static float bits_to_float(uint32_t u) {
  float f;
  memcpy(&f, &u, sizeof f);
  return f;
}

static uint32_t float_to_bits(float f) {
  uint32_t u;
  memcpy(&u, &f, sizeof u);
  return u;
}

/* Classification by bit pattern, so that no compiler flag can change it. */
static int is_nan32(float f) {
  uint32_t u = float_to_bits(f) & 0x7FFFFFFFu;
  return u > 0x7F800000u;
}
static int is_inf32(float f) {
  uint32_t u = float_to_bits(f) & 0x7FFFFFFFu;
  return u == 0x7F800000u;
}
static int is_finite32(float f) {
  uint32_t u = float_to_bits(f) & 0x7FFFFFFFu;
  return u < 0x7F800000u;
}

/* binary16 -> binary32, exact (every binary16 value is a binary32 value). */
float kbo_decode_f16(uint16_t h) {
  uint32_t sign = (uint32_t)(h >> 15) & 1u;
  uint32_t expo = (uint32_t)(h >> 10) & 0x1Fu;
  uint32_t frac = (uint32_t)h & 0x3FFu;
  float mag;
  if (expo == 0x1Fu) {
    /* Inf or NaN: keep the payload in the top fraction bits */
    return bits_to_float((sign << 31) | 0x7F800000u | (frac << 13));
  }
  if (expo == 0) {
    /* zero or subnormal: frac * 2^-24, exact */
    mag = ldexpf((float)frac, -24);
  } else {
    /* normal: (1024 + frac) * 2^(expo - 25), exact */
    mag = ldexpf((float)(1024u + frac), (int)expo - 25);
  }
  return sign ? -mag : mag;
}

/* bfloat16 -> binary32: the 16 bits are the top half of the binary32 word. */
float kbo_decode_bf16(uint16_t b) { return bits_to_float((uint32_t)b << 16); }

/* 8-bit float, 4 exponent bits (bias 7), 3 fraction bits, the "fn" flavour: no
 * infinities, the only NaN is S.1111.111, S.1111.110 is the largest finite (448). */
float kbo_decode_f8e4m3(uint8_t v) {
  uint32_t sign = (uint32_t)(v >> 7) & 1u;
  uint32_t expo = (uint32_t)(v >> 3) & 0xFu;
  uint32_t frac = (uint32_t)v & 0x7u;
  float mag;
  if (expo == 0xFu && frac == 0x7u) return bits_to_float((sign << 31) | 0x7FC00000u);
  if (expo == 0)
    mag = ldexpf((float)frac, -9);                      /* subnormal: frac * 2^-3 * 2^-6 */
  else
    mag = ldexpf((float)(8u + frac), (int)expo - 10);   /* (1 + frac/8) * 2^(expo-7) */
  return sign ? -mag : mag;
}

/* 8-bit float, 5 exponent bits (bias 15), 2 fraction bits, IEEE-like: the top half
 * of a binary16. */
float kbo_decode_f8e5m2(uint8_t v) { return kbo_decode_f16((uint16_t)((uint16_t)v << 8)); }

static float load_as_f32(const void* base, uint64_t i, int dtype) {
  if (dtype == KBO_F32) return ((const float*)base)[i];
  if (dtype == KBO_F16) return kbo_decode_f16(((const uint16_t*)base)[i]);
  if (dtype == KBO_BF16) return kbo_decode_bf16(((const uint16_t*)base)[i]);
  if (dtype == KBO_F8E4M3) return kbo_decode_f8e4m3(((const uint8_t*)base)[i]);
  return kbo_decode_f8e5m2(((const uint8_t*)base)[i]);
}

/* Is element i selected by the fidelity mask?  A mask selects whole tiles of
 * 2^log2_tile consecutive elements. */
static int selected(uint64_t i, int mask_kind, uint32_t log2_tile, uint32_t stride, uint32_t phase,
                    const uint64_t* bits) {
  uint64_t tile;
  if (mask_kind == KBO_MASK_NONE) return 1;
  tile = i >> log2_tile;
  if (mask_kind == KBO_MASK_STRIDED) return (tile % stride) == phase;
  return (int)((bits[tile >> 6] >> (tile & 63u)) & 1u);
}

/*
 * The correctness gate for ONE candidate (Sec. 3.1 K(p); Sec. 3.4 Verifier).
 * For every selected element i, ascending:
 *   1. d = |c - r|
 *   2. tol = atol + (rtol * |r|)            product rounded, then sum rounded
 *   3. match = (c == r) || (isfinite(d) && d <= tol)
 *   4. counts of mismatches, of NaN candidates, of +-Inf candidates
 *   5. max_abs_err / argmax over finite d, first index wins ties, the first
 *      finite-d element initialises with its own d
 *   6. max_rel_err = max d/|r| over finite d and r != 0, starting from 0
 *   7. pass = no mismatch
 * Returns 0, or -1 on a bad argument.
 */
int kbo_screen(const void* ref, const void* cand, uint64_t N, int dtype, float atol, float rtol,
               int mask_kind, uint32_t log2_tile, uint32_t stride, uint32_t phase,
               const uint64_t* bits, kbo_screen_result* out) {
  uint64_t i;
  uint64_t mism = 0, nans = 0, infs = 0;
  int have_abs = 0;
  float max_abs = 0.0f, max_rel = 0.0f;
  int64_t argmax = -1;
  if (!ref || !cand || !out || N == 0) return -1;
  if (dtype < KBO_F32 || dtype > KBO_F8E5M2) return -1;
  if (mask_kind == KBO_MASK_STRIDED && (stride == 0 || phase >= stride)) return -1;
  if (mask_kind == KBO_MASK_BITMAP && !bits) return -1;

  for (i = 0; i < N; ++i) {
    float r, c, d, prod, tol;
    int match;
    if (!selected(i, mask_kind, log2_tile, stride, phase, bits)) continue;
    r = load_as_f32(ref, i, dtype);
    c = load_as_f32(cand, i, dtype);
    d = fabsf(c - r);
    prod = rtol * fabsf(r);
    tol = atol + prod;
    match = (c == r) || (is_finite32(d) && d <= tol);
    if (!match) ++mism;
    if (is_nan32(c)) ++nans;
    if (is_inf32(c)) ++infs;
    if (is_finite32(d)) {
      if (!have_abs || d > max_abs) {
        max_abs = d;
        argmax = (int64_t)i;
        have_abs = 1;
      }
      if (r != 0.0f) {
        float q = d / fabsf(r);
        if (q > max_rel) max_rel = q;
      }
    }
  }
  out->mismatch_count = mism;
  out->nan_count = nans;
  out->inf_count = infs;
  out->argmax_idx = have_abs ? argmax : -1;
  out->max_abs_err = have_abs ? max_abs : 0.0f;
  out->max_rel_err = max_rel;
  out->pass = (mism == 0) ? 1u : 0u;
  out->reserved = 0;
  return 0;
}

/* ---- the gate for binary64 tensors ---------------------------------------- */

typedef struct {
  uint64_t mismatch_count;
  uint64_t nan_count;
  uint64_t inf_count;
  int64_t argmax_idx;
  double max_abs_err;
  double max_rel_err;
  uint32_t pass;
  uint32_t reserved;
} kbo_screen_result_f64;

static uint64_t double_to_bits(double f) {
  uint64_t u;
  memcpy(&u, &f, sizeof u);
  return u;
}
static int is_nan64(double f) { return (double_to_bits(f) & 0x7FFFFFFFFFFFFFFFull) > 0x7FF0000000000000ull; }
static int is_inf64(double f) { return (double_to_bits(f) & 0x7FFFFFFFFFFFFFFFull) == 0x7FF0000000000000ull; }
static int is_finite64(double f) { return (double_to_bits(f) & 0x7FFFFFFFFFFFFFFFull) < 0x7FF0000000000000ull; }

/*
 * The same gate as kbo_screen (Sec. 3.1 K(p); Sec. 3.4 Verifier) for a reference and a
 * candidate stored in binary64.  The seven steps are those of kbo_screen with every
 * operation in binary64: a double-precision output is judged in its own precision, and the
 * record carries the two errors as doubles.
 */
int kbo_screen_f64(const double* ref, const double* cand, uint64_t N, double atol, double rtol,
                   int mask_kind, uint32_t log2_tile, uint32_t stride, uint32_t phase,
                   const uint64_t* bits, kbo_screen_result_f64* out) {
  uint64_t i;
  uint64_t mism = 0, nans = 0, infs = 0;
  int have_abs = 0;
  double max_abs = 0.0, max_rel = 0.0;
  int64_t argmax = -1;
  if (!ref || !cand || !out || N == 0) return -1;
  if (mask_kind == KBO_MASK_STRIDED && (stride == 0 || phase >= stride)) return -1;
  if (mask_kind == KBO_MASK_BITMAP && !bits) return -1;

  for (i = 0; i < N; ++i) {
    double r, c, d, prod, tol;
    int match;
    if (!selected(i, mask_kind, log2_tile, stride, phase, bits)) continue;
    r = ref[i];
    c = cand[i];
    d = fabs(c - r);
    prod = rtol * fabs(r);
    tol = atol + prod;
    match = (c == r) || (is_finite64(d) && d <= tol);
    if (!match) ++mism;
    if (is_nan64(c)) ++nans;
    if (is_inf64(c)) ++infs;
    if (is_finite64(d)) {
      if (!have_abs || d > max_abs) {
        max_abs = d;
        argmax = (int64_t)i;
        have_abs = 1;
      }
      if (r != 0.0) {
        double q = d / fabs(r);
        if (q > max_rel) max_rel = q;
      }
    }
  }
  out->mismatch_count = mism;
  out->nan_count = nans;
  out->inf_count = infs;
  out->argmax_idx = have_abs ? argmax : -1;
  out->max_abs_err = have_abs ? max_abs : 0.0;
  out->max_rel_err = max_rel;
  out->pass = (mism == 0) ? 1u : 0u;
  out->reserved = 0;
  return 0;
}

/* Ascending order of timings as a TOTAL order, so that the sorted row (and with it
 * the sign of a quantile that is zero) is unique: by value, and where two values are
 * equal but differ in sign (-0 and +0, the only such pair) the negative zero first. */
static int cmp_float_asc(const void* pa, const void* pb) {
  float a = *(const float*)pa, b = *(const float*)pb;
  if (a > b) return 1;
  if (a < b) return -1;
  {
    int sa = (int)(float_to_bits(a) >> 31), sb = (int)(float_to_bits(b) >> 31);
    return sb - sa; /* a negative (sa = 1), b positive (sb = 0): a first */
  }
}

/*
 * Quartiles of one row of S timings (Algorithm 1, "adjudicated latency"):
 * copy, sort ascending, then for j = 1, 2, 3 the type-7 (linear) quantile
 *   pos = j*(S-1); lo = pos/4; rem = pos%4; hi = min(lo+1, S-1)
 *   Q_j = x_lo                                   if rem == 0
 *       = x_lo + ((rem*0.25f) * (x_hi - x_lo))   otherwise, each op rounded.
 * out4 = {Q1, median = Q2, Q3, iqr = Q3 - Q1}.  `sorted` (S floats, may be
 * NULL) receives the sorted copy.
 * Returns 0; -1 on a bad argument; -2 if a timing is NaN or +-Inf.
 */
int kbo_quantiles(const float* row, uint32_t S, float* out4, float* sorted) {
  float* x;
  float q[4];
  uint32_t j, i;
  if (!row || !out4 || S == 0) return -1;
  for (i = 0; i < S; ++i)
    if (!is_finite32(row[i])) return -2;
  x = (float*)malloc((size_t)S * sizeof(float));
  if (!x) return -1;
  memcpy(x, row, (size_t)S * sizeof(float));
  qsort(x, S, sizeof(float), cmp_float_asc);
  for (j = 1; j <= 3; ++j) {
    uint64_t pos = (uint64_t)j * (uint64_t)(S - 1);
    uint64_t lo = pos / 4u;
    uint32_t rem = (uint32_t)(pos % 4u);
    uint64_t hi = (lo + 1 < (uint64_t)S) ? lo + 1 : (uint64_t)S - 1;
    if (rem == 0) {
      q[j] = x[lo];
    } else {
      float w = (float)rem * 0.25f;
      float diff = x[hi] - x[lo];
      float step = w * diff;
      q[j] = x[lo] + step;
    }
  }
  out4[0] = q[1];
  out4[1] = q[2];
  out4[2] = q[3];
  out4[3] = q[3] - q[1];
  if (sorted) memcpy(sorted, x, (size_t)S * sizeof(float));
  free(x);
  return 0;
}

/*
 * Win count of row a over row b: twice the Mann-Whitney U statistic of
 * "a is faster (smaller) than b", ties counted once:
 *   W = sum_i sum_j ( 2*[a_i < b_j] + [a_i == b_j] )
 * by the literal double loop over the rows as given (unsorted).
 */
uint64_t kbo_wins_pair(const float* a, const float* b, uint32_t S) {
  uint64_t w = 0;
  uint32_t i, j;
  for (i = 0; i < S; ++i) {
    for (j = 0; j < S; ++j) {
      if (a[i] < b[j]) w += 2;
      if (a[i] == b[j]) w += 1;
    }
  }
  return w;
}

/*
 * Full adjudication of timings[K][S]: median[K], iqr[K], W[K][K] (uint32,
 * row-major).  Any output may be NULL.  Returns 0; -1 bad argument; -2 if any
 * timing is non-finite (outputs then unspecified).
 */
int kbo_adjudicate(const float* timings, uint32_t K, uint32_t S, float* median, float* iqr,
                   uint32_t* wins) {
  uint32_t a, b;
  uint64_t t;
  if (!timings || K == 0 || S == 0) return -1;
  for (t = 0; t < (uint64_t)K * S; ++t)
    if (!is_finite32(timings[t])) return -2;
  if (median || iqr) {
    for (a = 0; a < K; ++a) {
      float q[4];
      int rc = kbo_quantiles(timings + (size_t)a * S, S, q, NULL);
      if (rc != 0) return rc;
      if (median) median[a] = q[1];
      if (iqr) iqr[a] = q[3];
    }
  }
  if (wins) {
    for (a = 0; a < K; ++a)
      for (b = 0; b < K; ++b)
        wins[(size_t)a * K + b] =
            (uint32_t)kbo_wins_pair(timings + (size_t)a * S, timings + (size_t)b * S, S);
  }
  return 0;
}

/* Rows [a0, a1) of W only -- lets a caller spread the literal double loop over
 * several host threads, or time a bounded sample of it. */
int kbo_wins_rows(const float* timings, uint32_t K, uint32_t S, uint32_t a0, uint32_t a1,
                  uint32_t* wins_rows /* [(a1-a0)][K] */) {
  uint32_t a, b;
  if (!timings || !wins_rows || K == 0 || S == 0 || a0 > a1 || a1 > K) return -1;
  for (a = a0; a < a1; ++a)
    for (b = 0; b < K; ++b)
      wins_rows[(size_t)(a - a0) * K + b] =
          (uint32_t)kbo_wins_pair(timings + (size_t)a * S, timings + (size_t)b * S, S);
  return 0;
}

/*
 * Promotion decision (Sec. 3.2; Sec. 3.4 scheduler).  Eligible = pass == 1.
 * policy 0: order by (max_rel_err asc, median asc, index asc);
 * policy 1: order by (median asc, index asc).
 * The first n = min(budget, #eligible) indices go to survivors[0..n) in rank
 * order, survivors[n..budget) = -1, *n_out = n.
 * Written as a selection sort on the candidate list: find the best remaining
 * candidate, emit it, repeat.
 */
int kbo_select(const kbo_screen_result* screen, const float* median, uint32_t K, int policy,
               uint32_t budget, int32_t* survivors, uint32_t* n_out) {
  uint8_t* taken;
  uint32_t n = 0, k, slot;
  if (!screen || !median || !survivors || !n_out || K == 0 || budget == 0) return -1;
  if (policy != 0 && policy != 1) return -1;
  taken = (uint8_t*)calloc(K, 1);
  if (!taken) return -1;
  for (slot = 0; slot < budget; ++slot) {
    int64_t best = -1;
    for (k = 0; k < K; ++k) {
      int better;
      if (taken[k] || screen[k].pass != 1u) continue;
      if (best < 0) {
        best = k;
        continue;
      }
      better = 0;
      if (policy == 0) {
        if (screen[k].max_rel_err < screen[best].max_rel_err)
          better = 1;
        else if (screen[k].max_rel_err == screen[best].max_rel_err && median[k] < median[best])
          better = 1;
      } else {
        if (median[k] < median[best]) better = 1;
      }
      /* equal keys: the lower index (already held in best) stays */
      if (better) best = k;
    }
    if (best < 0) break;
    taken[best] = 1;
    survivors[n++] = (int32_t)best;
  }
  for (slot = n; slot < budget; ++slot) survivors[slot] = -1;
  *n_out = n;
  free(taken);
  return 0;
}

/* ------------------------------------------------------------------------
 * Scheduler-side statistics on top of the three calls above.
 * ------------------------------------------------------------------------ */

/*
 * Runtime score of one candidate (Sec. 3.1, Eq. 2):
 *   S(p, r) = 1e6 / max(1, latency_us) + gamma(r),  gamma(r) = alpha*r + beta*b_r
 * with the latency taken as the adjudicated (median) latency, given in
 * milliseconds.  Every operation is a binary32 operation in the order written:
 *   l_us = median_ms * 1000;  m = max(1, l_us);  base = 1e6 / m;
 *   gamma = (alpha * r) + (beta * b_r);  score = base + gamma.
 */
float kbo_score(float median_ms, uint32_t rung, uint32_t rung_budget, float alpha, float beta) {
  float l_us = median_ms * 1000.0f;
  float m = (l_us > 1.0f) ? l_us : 1.0f;
  float base = 1.0e6f / m;
  float ga = alpha * (float)rung;
  float gb = beta * (float)rung_budget;
  float gamma = ga + gb;
  return base + gamma;
}

/*
 * Promotion by runtime score (Sec. 3.4: "ranks candidates by s(c,r) with
 * deterministic tie-breaking ... promotes the top fraction"): eligible =
 * pass == 1, order by (score descending, index ascending).  scores[K] (may be
 * NULL) receives every candidate's score, eligible or not.
 */
int kbo_select_by_score(const kbo_screen_result* screen, const float* median, uint32_t K,
                        uint32_t rung, uint32_t rung_budget, float alpha, float beta,
                        uint32_t budget, float* scores, int32_t* survivors, uint32_t* n_out) {
  uint8_t* taken;
  float* sc;
  uint32_t n = 0, k, slot;
  if (!screen || !median || !survivors || !n_out || K == 0 || budget == 0) return -1;
  taken = (uint8_t*)calloc(K, 1);
  sc = (float*)malloc((size_t)K * sizeof(float));
  if (!taken || !sc) return -1;
  for (k = 0; k < K; ++k) {
    sc[k] = kbo_score(median[k], rung, rung_budget, alpha, beta);
    if (scores) scores[k] = sc[k];
  }
  for (slot = 0; slot < budget; ++slot) {
    int64_t best = -1;
    for (k = 0; k < K; ++k) {
      if (taken[k] || screen[k].pass != 1u) continue;
      if (best < 0 || sc[k] > sc[best]) best = k;   /* equal scores: the lower index stays */
    }
    if (best < 0) break;
    taken[best] = 1;
    survivors[n++] = (int32_t)best;
  }
  for (slot = n; slot < budget; ++slot) survivors[slot] = -1;
  *n_out = n;
  free(taken);
  free(sc);
  return 0;
}

/*
 * Tail ratios of one row (Appendix, Relative Variability Metrics: p90/p50,
 * p95/p50, p99/p50).  Percentile q in {50, 90, 95, 99} of the sorted row by
 * the linear (type-7) rule with integer position arithmetic:
 *   pos = q*(S-1); lo = pos/100; rem = pos%100; hi = min(lo+1, S-1)
 *   P_q = x_lo                                          if rem == 0
 *       = x_lo + (((float)rem / 100.0f) * (x_hi - x_lo))   otherwise,
 * each operation rounded; out3 = {P90/P50, P95/P50, P99/P50} (rounded
 * divisions).  Returns 0; -1 bad argument; -2 non-finite timing.
 */
int kbo_tail_ratios(const float* row, uint32_t S, float* out3) {
  static const uint32_t qs[4] = {50u, 90u, 95u, 99u};
  float p[4];
  float* x;
  uint32_t i, t;
  if (!row || !out3 || S == 0) return -1;
  for (i = 0; i < S; ++i)
    if (!is_finite32(row[i])) return -2;
  x = (float*)malloc((size_t)S * sizeof(float));
  if (!x) return -1;
  memcpy(x, row, (size_t)S * sizeof(float));
  qsort(x, S, sizeof(float), cmp_float_asc);
  for (t = 0; t < 4; ++t) {
    uint64_t pos = (uint64_t)qs[t] * (uint64_t)(S - 1);
    uint64_t lo = pos / 100u;
    uint32_t rem = (uint32_t)(pos % 100u);
    uint64_t hi = (lo + 1 < (uint64_t)S) ? lo + 1 : (uint64_t)S - 1;
    if (rem == 0) {
      p[t] = x[lo];
    } else {
      float w = (float)rem / 100.0f;
      float diff = x[hi] - x[lo];
      float step = w * diff;
      p[t] = x[lo] + step;
    }
  }
  out3[0] = p[1] / p[0];
  out3[1] = p[2] / p[0];
  out3[2] = p[3] / p[0];
  free(x);
  return 0;
}

/*
 * Copeland counts from the win matrix: candidate a "beats" b when it wins more
 * than half of the doubled sample pairs, W[a][b] > S*S, and ties with b when
 * W[a][b] == S*S.  beats[a], ties[a] (may be NULL) count opponents b != a.
 * A ranking by beats is stable under timing noise in the sense of the
 * appendix: it only uses the order of samples.
 */
int kbo_copeland(const uint32_t* wins, uint32_t K, uint32_t S, uint32_t* beats, uint32_t* ties) {
  uint32_t a, b;
  uint64_t half = (uint64_t)S * S;
  if (!wins || !beats || K == 0 || S == 0) return -1;
  for (a = 0; a < K; ++a) {
    uint32_t nb = 0, nt = 0;
    for (b = 0; b < K; ++b) {
      uint64_t w = wins[(size_t)a * K + b];
      if (b == a) continue;
      if (w > half) ++nb;
      if (w == half) ++nt;
    }
    beats[a] = nb;
    if (ties) ties[a] = nt;
  }
  return 0;
}

/*
 * Re-measure-and-confirm adjudication.  The paper's only description of
 * "stability adjudication" is a commented-out passage of Sec. 3: when a
 * candidate's score change exceeds a configurable threshold, it is measured
 * again at the same fidelity and reverted if the improvement is not confirmed.
 * Reading (binary32, operations as written), per candidate k with the
 * incumbent's score prev, the first score s1 and the re-measured score s2:
 *   flagged   = (s1 - prev) > (threshold * prev)
 *   confirmed = (s2 - prev) > (threshold * prev)
 *   status = 0, score = s1            if not flagged            (no re-measurement needed)
 *   status = 1, score = min(s1, s2)   if flagged and confirmed  (the cautious of the two)
 *   status = 2, score = prev          if flagged, not confirmed (reverted)
 */
int kbo_confirm(const float* s1, const float* s2, const float* prev, uint32_t K, float threshold,
                uint32_t* status, float* score) {
  uint32_t k;
  if (!s1 || !s2 || !prev || !status || !score || K == 0) return -1;
  for (k = 0; k < K; ++k) {
    float bar = threshold * prev[k];
    float d1 = s1[k] - prev[k];
    float d2 = s2[k] - prev[k];
    int flagged = d1 > bar;
    int confirmed = d2 > bar;
    if (!flagged) {
      status[k] = 0u;
      score[k] = s1[k];
    } else if (confirmed) {
      status[k] = 1u;
      score[k] = (s2[k] < s1[k]) ? s2[k] : s1[k];
    } else {
      status[k] = 2u;
      score[k] = prev[k];
    }
  }
  return 0;
}

/*
 * Adjudication with a different number of timings per candidate (a candidate
 * may have been measured at another fidelity, Sec. 3.2 "Fidelity level").
 * Row k is timings[offsets[k] .. offsets[k+1]), S_k = its length >= 1.
 * median/iqr as in kbo_quantiles on each row; the win count is the same double
 * loop, so that W[a][b] + W[b][a] = 2*S_a*S_b and W[a][a] = S_a*S_a.
 * Returns 0; -1 bad argument; -2 non-finite timing.
 */
int kbo_adjudicate_ragged(const float* timings, const uint32_t* offsets, uint32_t K, float* median,
                          float* iqr, uint32_t* wins) {
  uint32_t a, b, i, j;
  if (!timings || !offsets || K == 0) return -1;
  for (a = 0; a < K; ++a)
    if (offsets[a + 1] <= offsets[a]) return -1;
  for (i = offsets[0]; i < offsets[K]; ++i)
    if (!is_finite32(timings[i])) return -2;
  for (a = 0; a < K; ++a) {
    float q[4];
    int rc = kbo_quantiles(timings + offsets[a], offsets[a + 1] - offsets[a], q, NULL);
    if (rc != 0) return rc;
    if (median) median[a] = q[1];
    if (iqr) iqr[a] = q[3];
  }
  if (wins) {
    for (a = 0; a < K; ++a)
      for (b = 0; b < K; ++b) {
        uint64_t w = 0;
        for (i = offsets[a]; i < offsets[a + 1]; ++i)
          for (j = offsets[b]; j < offsets[b + 1]; ++j) {
            if (timings[i] < timings[j]) w += 2;
            if (timings[i] == timings[j]) w += 1;
          }
        wins[(size_t)a * K + b] = (uint32_t)w;
      }
  }
  return 0;
}

/*
 * The gate over an element range split into R consecutive parts (Sec. 3.1 K(p); the paper
 * runs on one GPU, this is the definition carried over a partition of the index set): the
 * record of the whole range from the records of the parts.  parts[r*K + k] is candidate k's
 * record over part r, whose first element has global index first[r] (ascending in r).
 *   counts add; the largest error wins, the earlier part on ties (its indices are lower),
 *   with its index moved to global numbering; the largest relative error is the maximum;
 *   pass = no mismatch anywhere.  A part without a finite difference (argmax_idx = -1)
 *   contributes no error.
 * Returns 0, or -1 on a bad argument.
 */
int kbo_merge_ranges(const kbo_screen_result* parts, uint32_t R, uint32_t K, const uint64_t* first,
                     kbo_screen_result* out) {
  uint32_t r, k;
  if (!parts || !first || !out || R == 0 || K == 0) return -1;
  for (r = 1; r < R; ++r)
    if (first[r] <= first[r - 1]) return -1;
  for (k = 0; k < K; ++k) {
    kbo_screen_result m;
    int have = 0;
    memset(&m, 0, sizeof m);
    m.argmax_idx = -1;
    for (r = 0; r < R; ++r) {
      const kbo_screen_result* p = &parts[(size_t)r * K + k];
      m.mismatch_count += p->mismatch_count;
      m.nan_count += p->nan_count;
      m.inf_count += p->inf_count;
      if (p->argmax_idx >= 0 && (!have || p->max_abs_err > m.max_abs_err)) {
        have = 1;
        m.max_abs_err = p->max_abs_err;
        m.argmax_idx = p->argmax_idx + (int64_t)first[r];
      }
      if (p->max_rel_err > m.max_rel_err) m.max_rel_err = p->max_rel_err;
    }
    m.pass = (m.mismatch_count == 0) ? 1u : 0u;
    out[k] = m;
  }
  return 0;
}
