// Promotion decision (Sec. 3.2 "Promotion decision"; Sec. 3.4 scheduler;
// Algorithm 1, D): rank the candidates that passed the gate by a
// lexicographic key with the candidate index as the final tie-break, and emit
// the first `budget` of them in rank order.
//
// Every key is distinct (the index is part of it), so the rank of a candidate
// is the number of eligible candidates with a smaller key: one thread per
// candidate counts them against tiles of keys staged in shared memory.  No
// sort, no scratch memory, no dependence on scheduling.
#pragma once

#include "kb_common.cuh"

namespace kb {

constexpr int kSelectThreads = 256;

// Order-preserving map of a finite-or-infinite float to uint32 (-0 == +0).
__device__ __forceinline__ unsigned int ordered_bits(float x) {
  const unsigned int u = __float_as_uint(x + 0.0f);   // -0 -> +0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ unsigned long long select_key(const kb_screen_result& r, float med,
                                                         int policy, bool* eligible) {
  *eligible = (r.pass == 1u);
  const unsigned long long hi = (policy == KB_SELECT_ERR_THEN_TIME) ? ordered_bits(r.max_rel_err) : 0u;
  return (hi << 32) | ordered_bits(med);
}

__global__ void __launch_bounds__(kSelectThreads) select_kernel(
    const kb_screen_result* __restrict__ screen, const float* __restrict__ median, unsigned int K,
    int policy, unsigned int budget, int* __restrict__ survivors, unsigned int* __restrict__ n_out) {
  __shared__ unsigned long long skey[kSelectThreads];
  __shared__ unsigned char selig[kSelectThreads];
  const unsigned int k = blockIdx.x * kSelectThreads + threadIdx.x;
  bool mine_ok = false;
  unsigned long long mine = 0ull;
  if (k < K) mine = select_key(screen[k], median[k], policy, &mine_ok);
  unsigned int rank = 0, n_elig = 0;
  for (unsigned int base = 0; base < K; base += kSelectThreads) {
    const unsigned int m = base + threadIdx.x;
    bool ok = false;
    unsigned long long key = 0ull;
    if (m < K) key = select_key(screen[m], median[m], policy, &ok);
    __syncthreads();
    skey[threadIdx.x] = key;
    selig[threadIdx.x] = ok ? 1 : 0;
    __syncthreads();
    const unsigned int lim = min((unsigned int)kSelectThreads, K - base);
    for (unsigned int t = 0; t < lim; ++t) {
      if (!selig[t]) continue;
      ++n_elig;
      const unsigned long long other = skey[t];
      const unsigned int mi = base + t;
      rank += (other < mine || (other == mine && mi < k)) ? 1u : 0u;
    }
  }
  const unsigned int n = n_elig < budget ? n_elig : budget;
  if (k < K && mine_ok && rank < budget) survivors[rank] = (int)k;
  // unused slots and the count: every thread knows n
  const unsigned long long gtid = (unsigned long long)blockIdx.x * kSelectThreads + threadIdx.x;
  const unsigned long long gsz = (unsigned long long)gridDim.x * kSelectThreads;
  for (unsigned long long slot = n + gtid; slot < budget; slot += gsz) survivors[slot] = -1;
  if (gtid == 0) *n_out = n;
}

// ---------------------------------------------------------------------------
// Runtime score (Sec. 3.1, Eq. 2) and promotion by it: (score descending, index ascending).
// ---------------------------------------------------------------------------
__device__ __forceinline__ float runtime_score(float median_ms, float gamma) {
  const float l_us = __fmul_rn(median_ms, 1000.0f);
  const float m = l_us > 1.0f ? l_us : 1.0f;
  return __fadd_rn(__fdiv_rn(1.0e6f, m), gamma);
}

__global__ void __launch_bounds__(kSelectThreads) select_by_score_kernel(
    const kb_screen_result* __restrict__ screen, const float* __restrict__ median, unsigned int K,
    float gamma, unsigned int budget, float* __restrict__ score_out, int* __restrict__ survivors,
    unsigned int* __restrict__ n_out) {
  __shared__ unsigned int skey[kSelectThreads];
  __shared__ unsigned char selig[kSelectThreads];
  const unsigned int k = blockIdx.x * kSelectThreads + threadIdx.x;
  bool mine_ok = false;
  unsigned int mine = 0u;   // descending score = ascending complement of the ordered bits
  if (k < K) {
    const float sc = runtime_score(median[k], gamma);
    if (score_out) score_out[k] = sc;
    mine = ~ordered_bits(sc);
    mine_ok = screen[k].pass == 1u;
  }
  unsigned int rank = 0, n_elig = 0;
  for (unsigned int base = 0; base < K; base += kSelectThreads) {
    const unsigned int m = base + threadIdx.x;
    bool ok = false;
    unsigned int key = 0u;
    if (m < K) {
      key = ~ordered_bits(runtime_score(median[m], gamma));
      ok = screen[m].pass == 1u;
    }
    __syncthreads();
    skey[threadIdx.x] = key;
    selig[threadIdx.x] = ok ? 1 : 0;
    __syncthreads();
    const unsigned int lim = min((unsigned int)kSelectThreads, K - base);
    for (unsigned int t = 0; t < lim; ++t) {
      if (!selig[t]) continue;
      ++n_elig;
      const unsigned int other = skey[t];
      const unsigned int mi = base + t;
      rank += (other < mine || (other == mine && mi < k)) ? 1u : 0u;
    }
  }
  const unsigned int n = n_elig < budget ? n_elig : budget;
  if (k < K && mine_ok && rank < budget) survivors[rank] = (int)k;
  const unsigned long long gtid = (unsigned long long)blockIdx.x * kSelectThreads + threadIdx.x;
  const unsigned long long gsz = (unsigned long long)gridDim.x * kSelectThreads;
  for (unsigned long long slot = n + gtid; slot < budget; slot += gsz) survivors[slot] = -1;
  if (gtid == 0) *n_out = n;
}

// Copeland counts: one warp per row of the win matrix.
__global__ void __launch_bounds__(256) copeland_kernel(const unsigned int* __restrict__ wins,
                                                       unsigned int K, unsigned int S,
                                                       unsigned int* __restrict__ beats,
                                                       unsigned int* __restrict__ ties) {
  const unsigned int a = blockIdx.x * 8 + (threadIdx.x >> 5);
  const unsigned int lane = threadIdx.x & 31;
  if (a >= K) return;
  const unsigned int half = S * S;
  unsigned int nb = 0, nt = 0;
  for (unsigned int b = lane; b < K; b += 32) {
    if (b == a) continue;
    const unsigned int w = wins[(size_t)a * K + b];
    nb += w > half ? 1u : 0u;
    nt += w == half ? 1u : 0u;
  }
  nb = warp_add_u32(nb);
  nt = warp_add_u32(nt);
  if (lane == 0) {
    beats[a] = nb;
    if (ties) ties[a] = nt;
  }
}

// Re-measure-and-confirm rule, one thread per candidate.
__global__ void confirm_kernel(const float* __restrict__ s1, const float* __restrict__ s2,
                               const float* __restrict__ prev, unsigned int K, float threshold,
                               unsigned int* __restrict__ status, float* __restrict__ score) {
  const unsigned int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= K) return;
  const float p = prev[k], a = s1[k], b = s2[k];
  const float bar = __fmul_rn(threshold, p);
  const bool flagged = __fsub_rn(a, p) > bar;
  const bool confirmed = __fsub_rn(b, p) > bar;
  unsigned int st;
  float sc;
  if (!flagged) {
    st = 0u;
    sc = a;
  } else if (confirmed) {
    st = 1u;
    sc = b < a ? b : a;
  } else {
    st = 2u;
    sc = p;
  }
  status[k] = st;
  score[k] = sc;
}

// ---------------------------------------------------------------------------
// Records of a whole element range from the records of its R consecutive parts
// (kb_merge_ranges): one thread per candidate walks the parts in order.
// ---------------------------------------------------------------------------
constexpr int kMergeMaxParts = 64;
struct RangeFirsts {
  unsigned long long first[kMergeMaxParts];
};

__global__ void merge_ranges_kernel(const kb_screen_result* __restrict__ parts, unsigned int R,
                                    unsigned int K, const RangeFirsts f,
                                    kb_screen_result* __restrict__ out) {
  const unsigned int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= K) return;
  kb_screen_result m;
  m.mismatch_count = m.nan_count = m.inf_count = 0ull;
  m.argmax_idx = -1;
  m.max_abs_err = 0.0f;
  m.max_rel_err = 0.0f;
  m.reserved = 0u;
  bool have = false;
  for (unsigned int r = 0; r < R; ++r) {
    const kb_screen_result p = parts[(size_t)r * K + k];
    m.mismatch_count += p.mismatch_count;
    m.nan_count += p.nan_count;
    m.inf_count += p.inf_count;
    // errors are non-negative and finite: their order is the order of their bit patterns
    if (p.argmax_idx >= 0 && (!have || __float_as_uint(p.max_abs_err) > __float_as_uint(m.max_abs_err))) {
      have = true;
      m.max_abs_err = p.max_abs_err;
      m.argmax_idx = p.argmax_idx + (long long)f.first[r];
    }
    if (__float_as_uint(p.max_rel_err) > __float_as_uint(m.max_rel_err)) m.max_rel_err = p.max_rel_err;
  }
  m.pass = m.mismatch_count == 0ull ? 1u : 0u;
  out[k] = m;
}

}  // namespace kb
