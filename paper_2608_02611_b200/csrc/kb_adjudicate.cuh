// Stability adjudication kernels (Algorithm 1 "adjudicated latency"; Sec. 1
// contribution 1; Appendix "Relative Variability Metrics").
//
// rows_kernel         one CTA per candidate: sort its S timings in shared
//                     memory (bitonic), take the type-7 quartiles with the
//                     operation order fixed, write median and IQR.
// wins_rank_kernel    the same integers from the SORTED rows: for a sample x of
//                     row a, lb = #{b_j < x} and ub = #{b_j <= x}; W[b][a] =
//                     sum_x (lb + ub), W[a][b] = 2*S*S - that.  A warp takes a
//                     pair of rows, each lane a contiguous run of a's samples:
//                     one binary search, then a merge walk.  O(K^2 (S + 32 log S))
//                     instead of O(K^2 S^2); the default when a
//                     block of 8 sorted rows fits shared memory (S <= 4096).
// wins_merge_kernel   the same integers again, for many candidates with short rows: a warp
//                     walks one a row against 32 b rows, one per lane (see below).
// wins_kernel         pairwise doubled Mann-Whitney counts by direct comparison.  A CTA takes a
//                     block of 8 "a" rows x 8 "b" rows and a chunk of samples
//                     of each; the a-chunk is staged in shared memory, each
//                     warp owns one b row and each lane keeps up to 8 of its
//                     samples in registers.  Per sample pair the work is two
//                     compares and two predicated increments.
//                     When a pair's samples fit one chunk each entry has a
//                     single writer (plain stores); otherwise partial counts
//                     are merged with integer atomics into a zeroed matrix.
//                     The mirrored entry W[b][a] = 2*S*S - W[a][b] is written by
//                     the same warp (the complement is additive over chunks).
#pragma once

#include "kb_common.cuh"

namespace kb {

constexpr int kRowsThreads = 256;

// Load one row into shared memory (padded with +Inf to P, a power of two), flag
// non-finite timings, sort ascending (bitonic network).  The order is total, so that the
// sorted row is unique: by value, and -0 before +0 (the only equal values whose bits differ;
// as signed integers the bits of -0 lie below those of +0).
__device__ __forceinline__ void load_and_sort_row(const float* __restrict__ row, unsigned int S,
                                                  unsigned int P, float* xs, unsigned int* status) {
  const float inf = __uint_as_float(0x7F800000u);
  bool nonfinite = false;
  for (unsigned int i = threadIdx.x; i < P; i += kRowsThreads) {
    float v = inf;   // padding sorts to the end
    if (i < S) {
      v = row[i];
      if (!(fabsf(v) <= 3.402823466e38f)) nonfinite = true;
    }
    xs[i] = v;
  }
  if (nonfinite) set_status(status, (unsigned int)KB_ERR_NONFINITE);
  __syncthreads();
  for (unsigned int size = 2; size <= P; size <<= 1) {
    for (unsigned int stride = size >> 1; stride > 0; stride >>= 1) {
      for (unsigned int t = threadIdx.x; t < (P >> 1); t += kRowsThreads) {
        const unsigned int lo = 2 * t - (t & (stride - 1));
        const unsigned int hi = lo + stride;
        const bool up = (lo & size) == 0;
        const float a = xs[lo], b = xs[hi];
        const bool gt = (a > b) || (a == b && __float_as_int(a) > __float_as_int(b));
        if (gt == up) {
          xs[lo] = b;
          xs[hi] = a;
        }
      }
      __syncthreads();
    }
  }
}

__global__ void __launch_bounds__(kRowsThreads) rows_kernel(const float* __restrict__ timings,
                                                            unsigned int S, unsigned int P /*pow2 >= S*/,
                                                            float* __restrict__ median,
                                                            float* __restrict__ iqr,
                                                            float* __restrict__ sorted_out /*[K][S] or NULL*/,
                                                            unsigned int* status) {
  extern __shared__ float xs[];
  const unsigned int k = blockIdx.x;
  load_and_sort_row(timings + (size_t)k * S, S, P, xs, status);
  if (sorted_out) {
    for (unsigned int i = threadIdx.x; i < S; i += kRowsThreads) sorted_out[(size_t)k * S + i] = xs[i];
  }
  if (threadIdx.x == 0) {
    float q[4];
#pragma unroll
    for (unsigned int j = 1; j <= 3; ++j) {
      const unsigned long long pos = (unsigned long long)j * (S - 1);
      const unsigned int lo = (unsigned int)(pos >> 2);
      const unsigned int rem = (unsigned int)(pos & 3ull);
      const unsigned int hi = (lo + 1 < S) ? lo + 1 : S - 1;
      if (rem == 0) {
        q[j] = xs[lo];
      } else {
        const float w = (float)rem * 0.25f;
        q[j] = __fadd_rn(xs[lo], __fmul_rn(w, __fsub_rn(xs[hi], xs[lo])));
      }
    }
    if (median) median[k] = q[2];
    if (iqr) iqr[k] = __fsub_rn(q[3], q[1]);
  }
}

// Tail ratios P90/P50, P95/P50, P99/P50 of every row (Appendix "Relative Variability
// Metrics"): the same sort, percentiles by the linear rule with q*(S-1)/100 positions.
__global__ void __launch_bounds__(kRowsThreads) tails_kernel(const float* __restrict__ timings,
                                                             unsigned int S, unsigned int P,
                                                             float* __restrict__ ratios /*[K][3]*/,
                                                             unsigned int* status) {
  extern __shared__ float xs[];
  const unsigned int k = blockIdx.x;
  load_and_sort_row(timings + (size_t)k * S, S, P, xs, status);
  if (threadIdx.x == 0) {
    const unsigned int qs[4] = {50u, 90u, 95u, 99u};
    float pq[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const unsigned long long pos = (unsigned long long)qs[t] * (S - 1);
      const unsigned int lo = (unsigned int)(pos / 100ull);
      const unsigned int rem = (unsigned int)(pos % 100ull);
      const unsigned int hi = (lo + 1 < S) ? lo + 1 : S - 1;
      if (rem == 0) {
        pq[t] = xs[lo];
      } else {
        const float w = __fdiv_rn((float)rem, 100.0f);
        pq[t] = __fadd_rn(xs[lo], __fmul_rn(w, __fsub_rn(xs[hi], xs[lo])));
      }
    }
    ratios[(size_t)k * 3 + 0] = __fdiv_rn(pq[1], pq[0]);
    ratios[(size_t)k * 3 + 1] = __fdiv_rn(pq[2], pq[0]);
    ratios[(size_t)k * 3 + 2] = __fdiv_rn(pq[3], pq[0]);
  }
}

// ---------------------------------------------------------------------------
constexpr int kWinsThreads = 256;
constexpr int kWinsRowsPerBlock = 8;    // a rows per CTA = b rows per CTA = warps
constexpr int kWinsMaxR = 8;            // b samples per lane

struct WinsParams {
  const float* timings;
  unsigned int* wins;
  unsigned int K, S;
  unsigned int KB;      // ceil(K / 8) blocks of 8 rows
  unsigned int npairs;  // KB*(KB+1)/2 block pairs, diagonal included
  unsigned int TA;      // a rows per CTA (1, 2, 4 or 8); 8/TA CTAs share one block pair
  unsigned int nj, JC;  // b-sample chunks and their length (JC = 32*R)
  unsigned int ni, IC;  // a-sample chunks and their length (multiple of 4)
  unsigned int direct;  // 1: each entry has one writer (ni == nj == 1): plain stores, no zeroing
};

// cnt += [a < b] + [a <= b]  (= 2*[a<b] + [a==b]); NaN padding compares false.
// Two compares into predicates and two predicated increments: measured twice as fast as
// compare-to-mask (`set`) plus a three-input add, which costs five machine instructions.
__device__ __forceinline__ void count_pair(unsigned int& cnt, float a, float b) {
  asm("{\n.reg .pred p, q;\nsetp.lt.f32 p, %1, %2;\nsetp.le.f32 q, %1, %2;\n@p add.u32 %0, %0, 1;\n@q add.u32 %0, %0, 1;\n}"
      : "+r"(cnt)
      : "f"(a), "f"(b));
}

// Register-only probe of the direct win count's instruction mix (no paper counterpart): every
// thread runs count_pair on values that never leave its registers, 8 b-values against a
// stream of a-values, as wins_kernel<8> does between two shared-memory reads.  The rate it
// reaches is the measured ceiling for "sample pairs per second" of that kernel on this GPU at
// the clock it holds.  The result is stored only if it has a value it cannot have, which is
// enough to keep the loop alive.
__global__ void __launch_bounds__(256) alu_probe_kernel(unsigned int iters, float seed,
                                                        unsigned int* __restrict__ sink) {
  float b[8];
  unsigned int cnt[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    b[i] = seed + 0.37f * (float)i + 0.001f * (float)threadIdx.x;
    cnt[i] = 0u;
  }
  float a = 0.5f * seed + 0.01f * (float)(threadIdx.x & 31);
  for (unsigned int it = 0; it < iters; ++it) {
#pragma unroll
    for (int u = 0; u < 16; ++u) {
#pragma unroll
      for (int i = 0; i < 8; ++i) count_pair(cnt[i], a, b[i]);
      a = fmaf(a, 1.0000001f, 0.03125f);   // one more instruction per 8 pairs keeps a moving
      if (a > 4.0f * seed) a -= 4.0f * seed;
    }
  }
  unsigned int tot = 0u;
#pragma unroll
  for (int i = 0; i < 8; ++i) tot += cnt[i];
  if (tot == 0xFFFFFFFFu) *sink = tot;   // 2 * 16 * 8 * iters < 2^32 - 1: never taken
}

template <int R>
__global__ void __launch_bounds__(kWinsThreads) wins_kernel(const WinsParams p) {
  extern __shared__ float as[];   // [TA][IC]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned int item = blockIdx.x;
  const unsigned int ic = item % p.ni;
  item /= p.ni;
  const unsigned int jc = item % p.nj;
  item /= p.nj;
  const unsigned int nsub = kWinsRowsPerBlock / p.TA;
  const unsigned int sub = item % nsub;
  const unsigned int pair = item / nsub;
  // block pair index -> (Ab <= Bb): row-major upper triangle
  unsigned int Ab = 0, rem = pair;
  while (rem >= p.KB - Ab) {
    rem -= p.KB - Ab;
    ++Ab;
  }
  const unsigned int Bb = Ab + rem;
  const float qnan = __uint_as_float(0x7FC00000u);

  // stage the a-chunk: TA rows from Ab*8 + sub*TA, samples ic*IC .. +IC
  const unsigned int a0 = Ab * kWinsRowsPerBlock + sub * p.TA;
  const unsigned int i0 = ic * p.IC;
  for (unsigned int t = threadIdx.x; t < p.TA * p.IC; t += kWinsThreads) {
    const unsigned int rr = t / p.IC, ii = t % p.IC;
    const unsigned int a = a0 + rr, i = i0 + ii;
    as[t] = (a < p.K && i < p.S) ? p.timings[(size_t)a * p.S + i] : qnan;
  }
  // this warp's b row, this lane's samples
  const unsigned int b = Bb * kWinsRowsPerBlock + warp;
  const unsigned int j0 = jc * p.JC;
  float bv[R];
#pragma unroll
  for (int m = 0; m < R; ++m) {
    const unsigned int j = j0 + lane + 32 * m;
    bv[m] = (b < p.K && j < p.S) ? p.timings[(size_t)b * p.S + j] : qnan;
  }
  __syncthreads();
  if (b >= p.K) return;
  const unsigned int ilen = min(p.IC, p.S - i0);
  const unsigned int jlen = min(p.JC, p.S - j0);

  for (unsigned int rr = 0; rr < p.TA; ++rr) {
    const unsigned int a = a0 + rr;
    if (a >= p.K) break;
    unsigned int cnt[R];
#pragma unroll
    for (int m = 0; m < R; ++m) cnt[m] = 0u;
    const float4* arow = reinterpret_cast<const float4*>(as + (size_t)rr * p.IC);
    const unsigned int n4 = p.IC >> 2;
#pragma unroll 2
    for (unsigned int i = 0; i < n4; ++i) {
      const float4 a4 = arow[i];
#pragma unroll
      for (int m = 0; m < R; ++m) {
        count_pair(cnt[m], a4.x, bv[m]);
        count_pair(cnt[m], a4.y, bv[m]);
        count_pair(cnt[m], a4.z, bv[m]);
        count_pair(cnt[m], a4.w, bv[m]);
      }
    }
    unsigned int total = 0u;
#pragma unroll
    for (int m = 0; m < R; ++m) total += cnt[m];
    total = warp_add_u32(total);
    if (lane == 0) {
      // W[b][a] = 2*S*S - W[a][b]; over chunks the complement is additive as well
      const unsigned int mirror = 2u * ilen * jlen - total;
      unsigned int* wab = &p.wins[(size_t)a * p.K + b];
      unsigned int* wba = &p.wins[(size_t)b * p.K + a];
      if (p.direct) {
        *wab = total;
        if (Ab != Bb) *wba = mirror;
      } else {
        if (total) atomicAdd(wab, total);
        if (Ab != Bb && mirror) atomicAdd(wba, mirror);
      }
    }
  }
}

// ---------------------------------------------------------------------------
struct WinsRankParams {
  const float* sorted;   // [K][S], each row ascending
  unsigned int* wins;
  unsigned int K, S, P;  // P: smallest power of two > S
  unsigned int KB, TA;   // blocks of 8 rows; a rows per CTA
};

__global__ void __launch_bounds__(kWinsThreads) wins_rank_kernel(const WinsRankParams p) {
  extern __shared__ float bs[];   // [8][S] sorted b rows
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const unsigned int nsub = kWinsRowsPerBlock / p.TA;
  const unsigned int sub = blockIdx.x % nsub;
  const unsigned int pair = blockIdx.x / nsub;
  unsigned int Ab = 0, rem = pair;
  while (rem >= p.KB - Ab) {
    rem -= p.KB - Ab;
    ++Ab;
  }
  const unsigned int Bb = Ab + rem;
  const unsigned int b0 = Bb * kWinsRowsPerBlock;
  const unsigned int nb = min((unsigned int)kWinsRowsPerBlock, p.K - b0);
  for (unsigned int t = threadIdx.x; t < nb * p.S; t += kWinsThreads) bs[t] = p.sorted[(size_t)b0 * p.S + t];
  __syncthreads();
  const unsigned int b = b0 + warp;
  if (b >= p.K) return;
  const float* brow = bs + (size_t)warp * p.S;
  const unsigned int a0 = Ab * kWinsRowsPerBlock + sub * p.TA;
  for (unsigned int rr = 0; rr < p.TA; ++rr) {
    const unsigned int a = a0 + rr;
    if (a >= p.K) break;
    const float* arow = p.sorted + (size_t)a * p.S;
    // Each lane takes a contiguous run of a's sorted samples: one binary search for the
    // first, then both rows are walked in step (a merge), since lb and ub only grow.
    const unsigned int L = (p.S + 31) / 32;
    const unsigned int i0 = lane * L;
    const unsigned int i1 = min(i0 + L, p.S);
    unsigned int sum = 0u;
    if (i0 < i1) {
      const float x0 = arow[i0];
      unsigned int lb = 0u;                       // number of b samples < x
      for (unsigned int step = p.P >> 1; step > 0; step >>= 1) {
        const unsigned int nxt = lb + step;
        if (nxt <= p.S && brow[nxt - 1] < x0) lb = nxt;
      }
      unsigned int ub = lb;                       // number of b samples <= x
      for (unsigned int i = i0; i < i1; ++i) {
        const float x = arow[i];
        while (lb < p.S && brow[lb] < x) ++lb;
        if (ub < lb) ub = lb;
        while (ub < p.S && brow[ub] <= x) ++ub;
        sum += lb + ub;
      }
    }
    sum = warp_add_u32(sum);
    if (lane == 0) {
      p.wins[(size_t)a * p.K + b] = 2u * p.S * p.S - sum;
      if (Ab != Bb) p.wins[(size_t)b * p.K + a] = sum;
    }
  }
}

// ---------------------------------------------------------------------------
// The same integers by a lane-per-row merge, for many candidates with short rows.  A CTA
// stages a tile of 32 sorted b rows and 8 sorted a rows in shared memory (odd row stride,
// every row closed by +Inf); warp w walks a row w against the 32 b rows at once, lane l
// against b row l, with three pointers that only grow: i over a's samples, jl = #{b < a_i},
// ju = #{b <= a_i}.  At most 3S steps of a dozen instructions serve 32 row pairs, against a
// binary search and a walk per pair and lane in wins_rank_kernel.  Tiles (TA <= TB) of 32 x 32
// rows; the mirrored entry comes from W[a][b] + W[b][a] = 2*S*S.
// ---------------------------------------------------------------------------
constexpr int kMergeTile = 32;    // b rows per CTA (one per lane) and rows per tile
constexpr int kMergeARows = 8;    // a rows per CTA (one per warp)
struct WinsMergeParams {
  const float* sorted;   // [K][S] rows sorted ascending
  unsigned int* wins;
  unsigned int K, S, stride, nT;   // stride: odd, > S; nT: tiles of 32 rows
};

__global__ void __launch_bounds__(256) wins_merge_kernel(const WinsMergeParams p) {
  extern __shared__ float ms[];   // [32][stride] b rows, then [8][stride] a rows
  float* Bs = ms;
  float* As = ms + (size_t)kMergeTile * p.stride;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const unsigned int nsub = kMergeTile / kMergeARows;
  const unsigned int sub = blockIdx.x % nsub;
  unsigned int TA = 0, rem = blockIdx.x / nsub;
  while (rem >= p.nT - TA) {
    rem -= p.nT - TA;
    ++TA;
  }
  const unsigned int TB = TA + rem;
  const unsigned int b0 = TB * kMergeTile;
  const unsigned int a0 = TA * kMergeTile + sub * kMergeARows;
  const float inf = __uint_as_float(0x7F800000u);
  // stage the rows; rows past K and the closing element of every row are +Inf
  for (unsigned int r = warp; r < kMergeTile + kMergeARows; r += 8) {
    const bool is_b = r < kMergeTile;
    const unsigned int row = is_b ? b0 + r : a0 + (r - kMergeTile);
    float* dst = (is_b ? Bs + (size_t)r * p.stride : As + (size_t)(r - kMergeTile) * p.stride);
    const float* src = p.sorted + (size_t)row * p.S;
    for (unsigned int j = lane; j <= p.S; j += 32) {
      float v = inf;
      if (row < p.K && j < p.S) {
        v = src[j];
        // A non-finite timing voids the call (rows_kernel has set KB_ERR_NONFINITE); here it
        // must only not reach the closing +Inf's role: the walk below stops at the first value
        // that is above every sample, so no staged sample may be +Inf or NaN.
        if (!(fabsf(v) <= 3.402823466e38f)) v = 3.402823466e38f;
      }
      dst[j] = v;
    }
  }
  __syncthreads();
  const unsigned int a = a0 + warp, b = b0 + lane;
  if (a >= p.K) return;   // the whole warp
  const float* ar = As + (size_t)warp * p.stride;
  const float* br = Bs + (size_t)lane * p.stride;
  const bool live = b < p.K;
  // The three current values live in registers; a step reloads only the one whose pointer moved.
  // Pointers are byte addresses in shared memory, so that a step is 16 instructions: the sum of
  // the two b pointers is accumulated as it stands and rebased at the end.
  const unsigned int a_end = smem_u32(ar) + 4u * p.S;
  const unsigned int b_base = smem_u32(br);
  unsigned int ia = live ? smem_u32(ar) : a_end, il = b_base, iu = b_base, sum = 0u;
  float x = ar[0], yl = br[0], yu = yl;
  while (__any_sync(0xFFFFFFFFu, ia < a_end)) {
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      asm volatile(
          "{\n"
          ".reg .pred on, pl, pu, tk;\n"
          ".reg .u32 ad;\n"
          ".reg .f32 v;\n"
          "setp.lt.u32 on, %0, %7;\n"              // rows left in a?
          "setp.lt.and.f32 pl, %4, %3, on;\n"      // b[jl] <  x: the closing +Inf stops both pointers
          "setp.le.and.f32 pu, %5, %3, on;\n"      // b[ju] <= x
          "and.pred pu, pu, !pl;\n"
          "or.pred tk, pl, pu;\n"
          "and.pred tk, on, !tk;\n"                // neither moves: x is counted
          "@pl add.u32 %1, %1, 4;\n"
          "@pu add.u32 %2, %2, 4;\n"
          "@tk add.u32 %6, %6, %1;\n"
          "@tk add.u32 %6, %6, %2;\n"
          "@tk add.u32 %0, %0, 4;\n"
          "selp.u32 ad, %1, %2, pl;\n"
          "selp.u32 ad, %0, ad, tk;\n"
          "ld.shared.f32 v, [ad];\n"               // a[S] = +Inf is loaded but never used
          "@pl mov.f32 %4, v;\n"
          "@pu mov.f32 %5, v;\n"
          "@tk mov.f32 %3, v;\n"
          "}\n"
          : "+r"(ia), "+r"(il), "+r"(iu), "+f"(x), "+f"(yl), "+f"(yu), "+r"(sum)
          : "r"(a_end)
          : "memory");
    }
  }
  const unsigned int acc = (sum - 2u * p.S * b_base) >> 2;
  if (!live) return;
  // acc = sum over a's samples of (#{b < x} + #{b <= x}) = W[b][a]
  if (TA == TB) {
    p.wins[(size_t)b * p.K + a] = acc;   // a diagonal tile computes every ordered pair itself
  } else {
    p.wins[(size_t)a * p.K + b] = 2u * p.S * p.S - acc;
    p.wins[(size_t)b * p.K + a] = acc;
  }
}

// ---------------------------------------------------------------------------
// Rows of different lengths: row k = timings[offsets[k] .. offsets[k+1]).
// ---------------------------------------------------------------------------

// Sort + quartiles per row; a row longer than S_max or empty marks the call invalid.
__global__ void __launch_bounds__(kRowsThreads) rows_ragged_kernel(
    const float* __restrict__ timings, const unsigned int* __restrict__ offsets, unsigned int S_max,
    float* __restrict__ median, float* __restrict__ iqr, float* __restrict__ sorted_out,
    unsigned int* status) {
  extern __shared__ float xs[];
  const unsigned int k = blockIdx.x;
  const unsigned int o0 = offsets[k], o1 = offsets[k + 1];
  if (o1 <= o0 || o1 - o0 > S_max) {
    if (threadIdx.x == 0) set_status(status, (unsigned int)KB_ERR_INVALID_ARG);
    return;
  }
  const unsigned int S = o1 - o0;
  unsigned int P = 1;
  while (P < S) P <<= 1;
  load_and_sort_row(timings + o0, S, P, xs, status);
  if (sorted_out) {
    for (unsigned int i = threadIdx.x; i < S; i += kRowsThreads) sorted_out[o0 + i] = xs[i];
  }
  if (threadIdx.x == 0) {
    float q[4];
#pragma unroll
    for (unsigned int j = 1; j <= 3; ++j) {
      const unsigned long long pos = (unsigned long long)j * (S - 1);
      const unsigned int lo = (unsigned int)(pos >> 2);
      const unsigned int rem = (unsigned int)(pos & 3ull);
      const unsigned int hi = (lo + 1 < S) ? lo + 1 : S - 1;
      if (rem == 0) {
        q[j] = xs[lo];
      } else {
        const float w = (float)rem * 0.25f;
        q[j] = __fadd_rn(xs[lo], __fmul_rn(w, __fsub_rn(xs[hi], xs[lo])));
      }
    }
    if (median) median[k] = q[2];
    if (iqr) iqr[k] = __fsub_rn(q[3], q[1]);
  }
}

struct WinsRaggedParams {
  const float* sorted;            // rows ascending, at the offsets of the input
  const unsigned int* offsets;    // [K+1]
  unsigned int* wins;
  unsigned int K, S_max, KB, TA;
};

// As wins_rank_kernel, with per-row lengths: W[b][a] = sum over a's samples of (lb + ub) in
// row b, W[a][b] = 2*S_a*S_b - that.
__global__ void __launch_bounds__(kWinsThreads) wins_ragged_kernel(const WinsRaggedParams p) {
  extern __shared__ float bs[];   // [8][S_max]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const unsigned int nsub = kWinsRowsPerBlock / p.TA;
  const unsigned int sub = blockIdx.x % nsub;
  const unsigned int pair = blockIdx.x / nsub;
  unsigned int Ab = 0, rem = pair;
  while (rem >= p.KB - Ab) {
    rem -= p.KB - Ab;
    ++Ab;
  }
  const unsigned int Bb = Ab + rem;
  const unsigned int b = Bb * kWinsRowsPerBlock + warp;
  unsigned int Sb = 0, ob = 0;
  bool bad = false;
  if (b < p.K) {
    ob = p.offsets[b];
    const unsigned int oe = p.offsets[b + 1];
    bad = oe <= ob || oe - ob > p.S_max;
    Sb = bad ? 0u : oe - ob;
    for (unsigned int i = lane; i < Sb; i += 32) bs[(size_t)warp * p.S_max + i] = p.sorted[ob + i];
  }
  __syncthreads();
  if (b >= p.K || bad) return;
  const float* brow = bs + (size_t)warp * p.S_max;
  unsigned int P = 1;
  while (P <= Sb) P <<= 1;
  const unsigned int a0 = Ab * kWinsRowsPerBlock + sub * p.TA;
  for (unsigned int rr = 0; rr < p.TA; ++rr) {
    const unsigned int a = a0 + rr;
    if (a >= p.K) break;
    const unsigned int oa = p.offsets[a], oae = p.offsets[a + 1];
    if (oae <= oa || oae - oa > p.S_max) continue;
    const unsigned int Sa = oae - oa;
    const float* arow = p.sorted + oa;
    const unsigned int L = (Sa + 31) / 32;
    const unsigned int i0 = lane * L;
    const unsigned int i1 = min(i0 + L, Sa);
    unsigned int sum = 0u;
    if (i0 < i1) {
      const float x0 = arow[i0];
      unsigned int lb = 0u;
      for (unsigned int step = P >> 1; step > 0; step >>= 1) {
        const unsigned int nxt = lb + step;
        if (nxt <= Sb && brow[nxt - 1] < x0) lb = nxt;
      }
      unsigned int ub = lb;
      for (unsigned int i = i0; i < i1; ++i) {
        const float x = arow[i];
        while (lb < Sb && brow[lb] < x) ++lb;
        if (ub < lb) ub = lb;
        while (ub < Sb && brow[ub] <= x) ++ub;
        sum += lb + ub;
      }
    }
    sum = warp_add_u32(sum);
    if (lane == 0) {
      p.wins[(size_t)a * p.K + b] = 2u * Sa * Sb - sum;
      if (Ab != Bb) p.wins[(size_t)b * p.K + a] = sum;
    }
  }
}

}  // namespace kb
