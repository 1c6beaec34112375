/* Runs every oracle routine on exactly-sized heap buffers at awkward sizes, for a build with
 * -fsanitize=address,undefined: a read or write past a buffer, a misaligned access, a signed
 * overflow or an out-of-range shift in the oracle ends the program with a report.  It also
 * checks a few identities that hold for any input, so that the calls cannot be optimised away.
 * Test infrastructure only (it includes the oracle's source). */
#include "../oracle/kb_oracle.c"

#include <stdio.h>

static uint64_t rng_state = 0x9E3779B97F4A7C15ull;
static uint32_t rnd(void) {
  rng_state = rng_state * 6364136223846793005ull + 1442695040888963407ull;
  return (uint32_t)(rng_state >> 33);
}

static int fail(const char* what, long a, long b) {
  fprintf(stderr, "oracle_sanitize_driver: %s (%ld, %ld)\n", what, a, b);
  return 1;
}

/* every byte pattern is a legal element of every storage type, NaN and Inf included */
static int run_screen(void) {
  static const uint64_t sizes[] = {1, 7, 8, 9, 63, 64, 65, 4095, 4096, 4097, 12289};
  static const int dtypes[] = {KBO_F32, KBO_F16, KBO_BF16, KBO_F8E4M3, KBO_F8E5M2};
  static const int esize[] = {4, 2, 2, 1, 1};
  size_t si, di;
  for (si = 0; si < sizeof sizes / sizeof sizes[0]; ++si)
    for (di = 0; di < 5; ++di) {
      const uint64_t N = sizes[si];
      const size_t bytes = (size_t)N * (size_t)esize[di];
      uint8_t* r = (uint8_t*)malloc(bytes);
      uint8_t* c = (uint8_t*)malloc(bytes);
      const uint32_t log2_tile = 3;
      const uint64_t ntiles = (N + 7) >> 3;
      uint64_t* bits = (uint64_t*)calloc((size_t)((ntiles + 63) / 64), 8);
      kbo_screen_result all, strided, bitmap, same;
      size_t i;
      uint64_t t;
      if (!r || !c || !bits) return fail("malloc", (long)N, (long)di);
      for (i = 0; i < bytes; ++i) {
        r[i] = (uint8_t)rnd();
        c[i] = (rnd() & 3u) ? r[i] : (uint8_t)rnd();
      }
      for (t = 0; t < ntiles; t += 2) bits[t >> 6] |= 1ull << (t & 63u);     /* even tiles */
      if (kbo_screen(r, c, N, dtypes[di], 1e-2f, 1.6e-2f, KBO_MASK_NONE, 0, 0, 0, NULL, &all)) return fail("screen", (long)N, (long)di);
      if (kbo_screen(r, c, N, dtypes[di], 1e-2f, 1.6e-2f, KBO_MASK_STRIDED, log2_tile, 2, 0, NULL, &strided)) return fail("strided", (long)N, (long)di);
      if (kbo_screen(r, c, N, dtypes[di], 1e-2f, 1.6e-2f, KBO_MASK_BITMAP, log2_tile, 0, 0, bits, &bitmap)) return fail("bitmap", (long)N, (long)di);
      if (kbo_screen(r, r, N, dtypes[di], 0.0f, 0.0f, KBO_MASK_NONE, 0, 0, 0, NULL, &same)) return fail("same", (long)N, (long)di);
      /* the two masks name the same elements; a subset cannot count more */
      if (strided.mismatch_count != bitmap.mismatch_count || strided.argmax_idx != bitmap.argmax_idx ||
          strided.nan_count != bitmap.nan_count || strided.inf_count != bitmap.inf_count)
        return fail("strided and bitmap masks disagree", (long)N, (long)di);
      if (strided.mismatch_count > all.mismatch_count) return fail("subset counts more", (long)N, (long)di);
      /* a tensor against itself mismatches exactly where it holds NaN */
      if (same.mismatch_count != same.nan_count) return fail("self comparison", (long)N, (long)di);
      free(r);
      free(c);
      free(bits);
    }
  return 0;
}

static int run_screen_f64(void) {
  static const uint64_t sizes[] = {1, 7, 9, 4097};
  size_t si;
  for (si = 0; si < sizeof sizes / sizeof sizes[0]; ++si) {
    const uint64_t N = sizes[si];
    double* r = (double*)malloc((size_t)N * 8);
    double* c = (double*)malloc((size_t)N * 8);
    kbo_screen_result_f64 out;
    uint64_t i;
    if (!r || !c) return fail("malloc", (long)N, 0);
    for (i = 0; i < N; ++i) {
      r[i] = (double)(int32_t)rnd() / 65536.0;
      c[i] = (rnd() & 1u) ? r[i] : r[i] * (1.0 + 1e-9);
    }
    if (kbo_screen_f64(r, c, N, 1e-12, 1e-6, KBO_MASK_NONE, 0, 0, 0, NULL, &out)) return fail("screen_f64", (long)N, 0);
    if (out.mismatch_count != 0) return fail("screen_f64 tolerance", (long)N, 0);
    free(r);
    free(c);
  }
  return 0;
}

static float timing(void) { return 0.5f + (float)(rnd() % 64u) * 0.03125f; }   /* many ties */

static int run_adjudicate(void) {
  static const uint32_t Ks[] = {1, 2, 3, 33};
  static const uint32_t Ss[] = {1, 2, 3, 4, 5, 31, 32, 33, 100};
  size_t ki, si;
  for (ki = 0; ki < sizeof Ks / sizeof Ks[0]; ++ki)
    for (si = 0; si < sizeof Ss / sizeof Ss[0]; ++si) {
      const uint32_t K = Ks[ki], S = Ss[si];
      float* t = (float*)malloc((size_t)K * S * 4);
      float* med = (float*)malloc((size_t)K * 4);
      float* iqr = (float*)malloc((size_t)K * 4);
      float* ratios = (float*)malloc(3 * 4);
      float* sorted = (float*)malloc((size_t)S * 4);
      uint32_t* wins = (uint32_t*)malloc((size_t)K * K * 4);
      uint32_t* rows = (uint32_t*)malloc((size_t)K * K * 4);
      uint32_t* beats = (uint32_t*)malloc((size_t)K * 4);
      uint32_t* ties = (uint32_t*)malloc((size_t)K * 4);
      uint32_t* offsets = (uint32_t*)malloc((size_t)(K + 1) * 4);
      float q[4];
      uint32_t a, b, i;
      if (!t || !med || !iqr || !ratios || !sorted || !wins || !rows || !beats || !ties || !offsets)
        return fail("malloc", (long)K, (long)S);
      for (i = 0; i < K * S; ++i) t[i] = timing();
      if (kbo_adjudicate(t, K, S, med, iqr, wins)) return fail("adjudicate", (long)K, (long)S);
      if (kbo_wins_rows(t, K, S, 0, K, rows)) return fail("wins_rows", (long)K, (long)S);
      for (a = 0; a < K; ++a) {
        if (kbo_quantiles(t + (size_t)a * S, S, q, sorted)) return fail("quantiles", (long)K, (long)S);
        if (q[1] != med[a] || q[3] != iqr[a]) return fail("quantiles against adjudicate", (long)a, (long)S);
        for (i = 1; i < S; ++i)
          if (sorted[i - 1] > sorted[i]) return fail("not sorted", (long)a, (long)i);
        if (kbo_tail_ratios(t + (size_t)a * S, S, ratios)) return fail("tail_ratios", (long)K, (long)S);
        if (!(ratios[0] >= 1.0f && ratios[1] >= ratios[0] && ratios[2] >= ratios[1]))
          return fail("tail ratios not ordered", (long)a, (long)S);
        for (b = 0; b < K; ++b) {
          if (wins[(size_t)a * K + b] != rows[(size_t)a * K + b]) return fail("wins rows", (long)a, (long)b);
          if (wins[(size_t)a * K + b] + wins[(size_t)b * K + a] != 2u * S * S) return fail("wins pair sum", (long)a, (long)b);
        }
      }
      if (kbo_copeland(wins, K, S, beats, ties)) return fail("copeland", (long)K, (long)S);
      for (a = 0; a < K; ++a)
        if (beats[a] + ties[a] > K - 1) return fail("copeland counts", (long)a, (long)K);
      /* the same rows through the ragged entry point (every row of length S) */
      for (a = 0; a <= K; ++a) offsets[a] = a * S;
      if (kbo_adjudicate_ragged(t, offsets, K, iqr, med, rows)) return fail("ragged", (long)K, (long)S);
      for (i = 0; i < K * K; ++i)
        if (rows[i] != wins[i]) return fail("ragged wins", (long)i, (long)S);
      free(t); free(med); free(iqr); free(ratios); free(sorted); free(wins); free(rows);
      free(beats); free(ties); free(offsets);
    }
  return 0;
}

static int run_ragged_and_select(void) {
  const uint32_t K = 9;
  uint32_t offsets[10], total = 0, a, i, n = 0;
  float *t, med[9], iqr[9], scores[9], prev[9], s2[9], conf_score[9];
  uint32_t wins[81], status[9];
  kbo_screen_result rec[9];
  int32_t* surv;
  for (a = 0; a < K; ++a) {
    offsets[a] = total;
    total += 1u + (a * 7u) % 13u;           /* lengths 1..13, among them 1 */
  }
  offsets[K] = total;
  t = (float*)malloc((size_t)total * 4);
  if (!t) return fail("malloc", (long)total, 0);
  for (i = 0; i < total; ++i) t[i] = timing();
  if (kbo_adjudicate_ragged(t, offsets, K, med, iqr, wins)) return fail("ragged", (long)K, 0);
  for (a = 0; a < K; ++a) {
    const uint32_t sa = offsets[a + 1] - offsets[a];
    uint32_t b;
    if (wins[a * K + a] != sa * sa) return fail("ragged diagonal", (long)a, (long)sa);
    for (b = 0; b < K; ++b)
      if (wins[a * K + b] + wins[b * K + a] != 2u * sa * (offsets[b + 1] - offsets[b]))
        return fail("ragged pair sum", (long)a, (long)b);
    memset(&rec[a], 0, sizeof rec[a]);
    rec[a].pass = (a % 3u) != 1u;
    rec[a].mismatch_count = rec[a].pass ? 0u : 5u;
    rec[a].max_rel_err = (float)(a % 4u) * 0.001f;
    rec[a].argmax_idx = (int64_t)a;
    prev[a] = med[a] * 1.05f;
    s2[a] = med[a] * ((a & 1u) ? 1.2f : 1.0f);
  }
  for (i = 1; i <= K + 2; ++i) {          /* budgets below, at and above the number eligible */
    int policy;
    surv = (int32_t*)malloc((size_t)i * 4);
    if (!surv) return fail("malloc", (long)i, 0);
    for (policy = 0; policy < 2; ++policy) {
      uint32_t j;
      if (kbo_select(rec, med, K, policy, i, surv, &n)) return fail("select", (long)i, policy);
      if (n != (i < 6u ? i : 6u)) return fail("select count", (long)i, (long)n);
      for (j = 0; j < i; ++j)
        if ((j < n) != (surv[j] >= 0)) return fail("select padding", (long)i, (long)j);
    }
    if (kbo_select_by_score(rec, med, K, 2, 8, 0.02f, 0.01f, i, scores, surv, &n)) return fail("select_by_score", (long)i, 0);
    if (n != (i < 6u ? i : 6u)) return fail("select_by_score count", (long)i, (long)n);
    free(surv);
  }
  if (kbo_confirm(med, s2, prev, K, 0.97f, status, conf_score)) return fail("confirm", (long)K, 0);
  for (a = 0; a < K; ++a)
    if (status[a] > 2u) return fail("confirm status", (long)a, (long)status[a]);
  if (!(kbo_score(1.0f, 1, 8, 0.02f, 0.01f) > kbo_score(2.0f, 1, 8, 0.02f, 0.01f)))
    return fail("score not decreasing in time", 0, 0);
  free(t);
  /* a range in three parts: the merged records are those of the whole range */
  {
    const uint64_t N = 3000, cuts[4] = {0, 1, 1500, 3000};
    const uint64_t first[3] = {0, 1, 1500};
    float* r = (float*)malloc((size_t)N * 4);
    float* c = (float*)malloc((size_t)N * 4);
    kbo_screen_result* parts = (kbo_screen_result*)malloc(3 * sizeof(kbo_screen_result));
    kbo_screen_result whole, merged;
    uint64_t j;
    if (!r || !c || !parts) return fail("malloc", (long)N, 0);
    for (j = 0; j < N; ++j) {
      r[j] = timing();
      c[j] = (rnd() & 7u) ? r[j] : r[j] + 0.125f;
    }
    for (j = 0; j < 3; ++j)
      if (kbo_screen(r + cuts[j], c + cuts[j], cuts[j + 1] - cuts[j], KBO_F32, 1e-2f, 1e-2f, KBO_MASK_NONE, 0, 0,
                     0, NULL, &parts[j]))
        return fail("screen part", (long)j, 0);
    if (kbo_screen(r, c, N, KBO_F32, 1e-2f, 1e-2f, KBO_MASK_NONE, 0, 0, 0, NULL, &whole)) return fail("screen whole", 0, 0);
    if (kbo_merge_ranges(parts, 3, 1, first, &merged)) return fail("merge_ranges", 0, 0);
    if (merged.mismatch_count != whole.mismatch_count || merged.argmax_idx != whole.argmax_idx ||
        merged.max_abs_err != whole.max_abs_err || merged.max_rel_err != whole.max_rel_err ||
        merged.pass != whole.pass)
      return fail("merged parts differ from the whole", (long)merged.argmax_idx, (long)whole.argmax_idx);
    free(r);
    free(c);
    free(parts);
  }
  return 0;
}

int main(void) {
#ifdef KBO_SAN_SELFCHECK
  /* proves that the build would notice: the oracle is told of one element more than the
   * (host) buffers hold, and the program must end with a report instead of "ok" */
  {
    float* r = (float*)calloc(8, 4);
    float* c = (float*)calloc(8, 4);
    kbo_screen_result out;
    if (!r || !c) return 1;
    kbo_screen(r, c, 9, KBO_F32, 0.0f, 0.0f, KBO_MASK_NONE, 0, 0, 0, NULL, &out);
    free(r);
    free(c);
  }
#endif
  if (run_screen() || run_screen_f64() || run_adjudicate() || run_ragged_and_select()) return 1;
  puts("oracle_sanitize_driver: ok");
  return 0;
}
