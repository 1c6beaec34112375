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

}  // namespace kb
