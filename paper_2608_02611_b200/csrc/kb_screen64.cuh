// The correctness gate (Sec. 3.1 K(p); Sec. 3.4 Verifier) for binary64 tensors: every
// operation of the gate in binary64, errors reported as doubles.
//
// Same plan as the 16/32-bit path: a producer lane feeds a ring of shared-memory stages
// with 1-D bulk copies (reference half-tile, then the same half-tile of every candidate of
// the chunk), 256 consumer threads keep their 8 reference elements in registers and run a
// filter over each candidate stage; only warps whose filter fires take the exact path.
// What differs:
//   - a stage is 2048 elements (16 KB); a 4096-element mask tile is two of them;
//   - the (error, index) record does not fit one 64-bit word, so new maxima go straight
//     to the global accumulator with a 128-bit compare-and-swap (a rare event once the
//     thresholds are seeded), and only the counts are kept in shared memory;
//   - the other CTAs' maxima come back by reading that accumulator once per stage (the
//     pair as one unit, through a 128-bit compare-and-swap that changes nothing).
#pragma once

#include "kb_screen.cuh"

namespace kb {

constexpr int kTile64 = 2048;     // elements per stage
constexpr int kEPT64 = 8;         // elements per consumer thread per stage
constexpr int kMaxKC64 = 64;      // candidates per chunk
constexpr uint32_t kTileBytes64 = kTile64 * 8;
constexpr double kDblMax = 1.7976931348623157e308;

// hi = bits(|c - r|) + 1 (0: no finite difference seen), lo = 0xFFFFFFFF - index: a larger
// pair (hi first) is a larger error and, at equal error, a lower index.
struct alignas(16) Key128 {
  unsigned long long lo, hi;
};
struct alignas(16) Acc64 {
  Key128 key;
  unsigned long long mism, nan, inf;
  unsigned long long rel;   // bits of the max relative error (a non-negative double)
};
static_assert(sizeof(Acc64) == 48, "Acc64 layout");

// Raise the accumulator's record to (hi, lo) if that is larger.  Lock-free: a failed swap
// means another thread raised the record, so the loop ends after at most as many rounds as
// there are writers; the cap only guards against the impossible.
__device__ __forceinline__ void merge_key(Acc64* a, unsigned long long hi, unsigned long long lo) {
  Key128 cur;
  cur.hi = *reinterpret_cast<volatile unsigned long long*>(&a->key.hi);
  cur.lo = *reinterpret_cast<volatile unsigned long long*>(&a->key.lo);
  for (int it = 0; it < (1 << 20); ++it) {
    if (!(hi > cur.hi || (hi == cur.hi && lo > cur.lo))) return;
    Key128 mine;
    mine.lo = lo;
    mine.hi = hi;
    const Key128 old = atomicCAS(&a->key, cur, mine);
    if (old.hi == cur.hi && old.lo == cur.lo) return;
    cur = old;
  }
}

__device__ __forceinline__ void unpack_record64(const Acc64& a, kb_screen_result_f64* dst) {
  kb_screen_result_f64 r;
  r.mismatch_count = a.mism;
  r.nan_count = a.nan;
  r.inf_count = a.inf;
  if (a.key.hi == 0ull) {
    r.argmax_idx = -1;
    r.max_abs_err = 0.0;
  } else {
    r.max_abs_err = __longlong_as_double((long long)(a.key.hi - 1ull));
    r.argmax_idx = (int64_t)(0xFFFFFFFFull - a.key.lo);
  }
  r.max_rel_err = __longlong_as_double((long long)a.rel);
  r.pass = a.mism == 0ull ? 1u : 0u;
  r.reserved = 0u;
  *dst = r;
}

// ---------------------------------------------------------------------------
// Every element by the definition (plain loads): leading tiles, ragged tail, fine masks.
// ---------------------------------------------------------------------------
struct ExactAcc64 {
  unsigned int n_mis = 0, n_nan = 0, n_inf = 0;
  unsigned long long bd = 0ull, bi = 0ull, qb = 0ull;   // best (bits(d)+1, inverted index), rel bits

  __device__ __forceinline__ void add(double r, double c, unsigned long long i, double atol, double rtol) {
    const double ad = fabs(__dsub_rn(c, r));
    const double ar = fabs(r);
    const double tol = __dadd_rn(atol, __dmul_rn(rtol, ar));
    const bool fin = ad <= kDblMax;
    const bool match = (c == r) || (fin && ad <= tol);
    n_mis += match ? 0u : 1u;
    n_nan += (c != c) ? 1u : 0u;
    n_inf += (fabs(c) == __longlong_as_double(0x7FF0000000000000ll)) ? 1u : 0u;
    if (fin) {
      const unsigned long long hi = (unsigned long long)__double_as_longlong(ad) + 1ull;
      const unsigned long long lo = 0xFFFFFFFFull - i;
      if (hi > bd || (hi == bd && lo > bi)) {
        bd = hi;
        bi = lo;
      }
      if (ar > 0.0 && ar <= kDblMax) {
        const unsigned long long q = (unsigned long long)__double_as_longlong(__ddiv_rn(ad, ar));
        qb = q > qb ? q : qb;
      }
    }
  }
  __device__ __forceinline__ void commit(Acc64* a) {
    n_mis = warp_add_u32(n_mis);
    n_nan = warp_add_u32(n_nan);
    n_inf = warp_add_u32(n_inf);
    const unsigned long long hmax = warp_max_u64(bd);
    const unsigned int lmax = warp_max_u32(bd == hmax ? (unsigned int)bi : 0u);
    qb = warp_max_u64(qb);
    if ((threadIdx.x & 31) == 0) {
      if (n_mis) atomicAdd(&a->mism, (unsigned long long)n_mis);
      if (n_nan) atomicAdd(&a->nan, (unsigned long long)n_nan);
      if (n_inf) atomicAdd(&a->inf, (unsigned long long)n_inf);
      if (hmax) merge_key(a, hmax, (unsigned long long)lmax);
      if (qb) atomicMax(&a->rel, qb);
    }
  }
};

__global__ void __launch_bounds__(256) screen_generic64_kernel(const double* __restrict__ ref,
                                                               const void* const* __restrict__ cands,
                                                               Acc64* __restrict__ acc,
                                                               unsigned long long e0,
                                                               unsigned long long e1, double atol,
                                                               double rtol, MaskDev mask) {
  const unsigned int k = blockIdx.y;
  const double* cand = reinterpret_cast<const double*>(cands[k]);
  ExactAcc64 x;
  const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
  for (unsigned long long i = e0 + (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < e1;
       i += stride) {
    if (!mask_selected(mask, i)) continue;
    x.add(ref[i], cand[i], i, atol, rtol);
  }
  x.commit(&acc[k]);
}

// The first `nscout` 4096-element tiles (of the list, or tiles 0..nscout-1), exactly; their
// maxima seed the streaming kernel's thresholds.  grid = (nscout * 4, K).
__global__ void __launch_bounds__(256) screen_scout64_kernel(const double* __restrict__ ref,
                                                             const void* const* __restrict__ cands,
                                                             Acc64* __restrict__ acc,
                                                             const uint32_t* __restrict__ tile_list,
                                                             double atol, double rtol) {
  const unsigned int k = blockIdx.y;
  const unsigned int slot = blockIdx.x / 4;
  const unsigned long long tile = tile_list ? tile_list[slot] : slot;
  const unsigned long long base = tile * kTile + (blockIdx.x % 4) * 1024ull;
  const double* cand = reinterpret_cast<const double*>(cands[k]);
  ExactAcc64 x;
#pragma unroll
  for (unsigned int j = 0; j < 4; ++j) {
    const unsigned long long i = base + j * 256 + threadIdx.x;
    x.add(ref[i], cand[i], i, atol, rtol);
  }
  x.commit(&acc[k]);
}

__global__ void screen_prep64_kernel(const PtrChunk chunk, const void** table, Acc64* acc,
                                     unsigned int* done, unsigned int offset, unsigned int count) {
  const unsigned int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) {
    table[offset + i] = chunk.p[i];
    Acc64 z;
    z.key.lo = z.key.hi = 0ull;
    z.mism = z.nan = z.inf = z.rel = 0ull;
    acc[offset + i] = z;
  }
  if (i == 0) {
    done[0] = 0u;   // ticket counter
    done[1] = 0u;   // work counter (64 bits)
    done[2] = 0u;
  }
}

__global__ void screen_finalize64_kernel(const Acc64* __restrict__ acc,
                                         kb_screen_result_f64* __restrict__ out, unsigned int K) {
  const unsigned int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k < K) unpack_record64(acc[k], &out[k]);
}

// ---------------------------------------------------------------------------
// The streaming kernel.
// ---------------------------------------------------------------------------
struct Stream64Params {
  const double* ref;
  const void* const* cands;
  Acc64* acc;
  const uint32_t* tile_list;    // selected 4096-element tiles, ascending; NULL: tile = slot
  uint32_t nhalf;               // stages (half tiles) to visit per candidate
  uint32_t half0;               // first half-tile slot (earlier ones were scouted)
  uint32_t K, KC, nchunks;
  uint32_t stages;
  double atol, rtol;
  unsigned int* status;
  unsigned int* done;
  unsigned long long* sched;
  kb_screen_result_f64* out;
};

// Items of the binary64 kernel: chunk-major over half tiles (a stage holds 2048 doubles, half a
// kernel tile); the consumers read the item number itself.
struct HalfTileItemMap {
  uint32_t nhalf, half0, KC, K;
  const uint32_t* tile_list;          // NULL: tile = slot / 2
  __device__ __forceinline__ void locate(unsigned long long item, uint32_t& chunk, uint32_t& k0, int& kc,
                                         size_t& off, unsigned long long& id) const {
    chunk = (uint32_t)(item / nhalf);
    const uint32_t slot = half0 + (uint32_t)(item % nhalf);
    k0 = chunk * KC;
    kc = (int)min(KC, K - k0);
    const uint32_t tile = tile_list ? tile_list[slot >> 1] : (slot >> 1);
    off = ((size_t)tile * kTile + (size_t)(slot & 1u) * kTile64) * 8;
    id = item;
  }
};

struct Stream64Smem {
  unsigned char* buf;
  uint64_t* full;
  uint64_t* empty;
  uint64_t* sync_bar;
  unsigned long long* item_id;
  unsigned long long* cnt;      // [3][kMaxKC64]
  const void** ptrs;            // [kMaxKC64]
  long long* thr;               // [kMaxKC64][kWarps][2]: bits of {th, rel}; th = -1.0: none yet
  volatile unsigned int* abort_flag;
};

__host__ __device__ inline size_t stream64_smem_bytes(uint32_t stages) {
  size_t b = (size_t)stages * kTileBytes64;
  b += 3 * (size_t)stages * 8 + 8;
  b += 3 * (size_t)kMaxKC64 * 8 + (size_t)kMaxKC64 * 8;
  b += (size_t)kMaxKC64 * kWarps * 16;
  b += 16;
  return b + 128;
}

constexpr long long kThNone = (long long)0xBFF0000000000000ull;   // bits of -1.0

// The filter, per element, with ad = |c - r|, th = the warp's threshold on errors and rel =
// the running max of ad/|r|: nothing about the element can change the record if
//   ad <= th,   ad - rel*|r| <= 0 (one fused multiply-add: its single rounding keeps the
//   sign, so ad/|r| cannot round above rel),   ad <= atol + rtol*|r|,
// and no NaN is involved (every comparison is written so that a NaN fires).
__global__ void __maxnreg__(160) screen_stream64_kernel(const Stream64Params p) {
  extern __shared__ unsigned char smem_raw[];
  Stream64Smem s;
  {
    uintptr_t base = (reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127;
    unsigned char* q = reinterpret_cast<unsigned char*>(base);
    s.buf = q;
    q += (size_t)p.stages * kTileBytes64;
    s.full = reinterpret_cast<uint64_t*>(q);
    q += (size_t)p.stages * 8;
    s.empty = reinterpret_cast<uint64_t*>(q);
    q += (size_t)p.stages * 8;
    s.sync_bar = reinterpret_cast<uint64_t*>(q);
    q += 8;
    s.item_id = reinterpret_cast<unsigned long long*>(q);
    q += (size_t)p.stages * 8;
    s.cnt = reinterpret_cast<unsigned long long*>(q);
    q += 3 * (size_t)kMaxKC64 * 8;
    s.ptrs = reinterpret_cast<const void**>(q);
    q += (size_t)kMaxKC64 * 8;
    s.thr = reinterpret_cast<long long*>(q);
    q += (size_t)kMaxKC64 * kWarps * 16;
    s.abort_flag = reinterpret_cast<volatile unsigned int*>(q);
  }
  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;
  const uint32_t stages = p.stages;

  if (tid == 0) {
    for (uint32_t i = 0; i < stages; ++i) {
      mbar_init(&s.full[i], 1);
      mbar_init(&s.empty[i], kWarps);
    }
    mbar_init(s.sync_bar, kWarps);
    *s.abort_flag = 0u;
    mbar_fence_init();
  }
  for (int i = tid; i < 3 * kMaxKC64; i += kStreamThreads) s.cnt[i] = 0ull;
  for (int i = tid; i < kMaxKC64 * kWarps; i += kStreamThreads) {
    s.thr[2 * i] = kThNone;
    s.thr[2 * i + 1] = 0ll;
  }
  __syncthreads();

  const unsigned long long nitems = (unsigned long long)p.nchunks * p.nhalf;

  if (warp == kWarps) {
    // ------------------------------ producer ------------------------------
    const RingProducerView ring{s.buf, s.full, s.empty, s.item_id, s.ptrs, s.abort_flag};
    const HalfTileItemMap map{p.nhalf, p.half0, p.KC, p.K, p.tile_list};
    ring_producer(ring, map, lane, stages, kTileBytes64, nitems, p.sched, p.ref, p.cands, p.nchunks > 1, p.status);
  } else {
    // ------------------------------ consumers -----------------------------
    uint32_t stage = 0, phase = 0;
    int cur_chunk = -1;
    int cur_kc = 0;
    uint32_t cur_k0 = 0;
    bool ok = true;

    uint32_t sync_phase = 0;
    auto consumers_barrier = [&]() -> bool {
      __syncwarp();
      if (lane == 0) mbar_arrive(s.sync_bar);
      const bool done = mbar_wait_bounded(s.sync_bar, sync_phase, s.abort_flag, p.status);
      sync_phase ^= 1u;
      return done;
    };
    auto flush = [&]() -> bool {
      if (!consumers_barrier()) return false;
      for (int i = tid; i < cur_kc; i += kConsumers) {
        Acc64* a = &p.acc[cur_k0 + i];
        unsigned long long v;
        if ((v = s.cnt[i]) != 0ull) atomicAdd(&a->mism, v);
        if ((v = s.cnt[kMaxKC64 + i]) != 0ull) atomicAdd(&a->nan, v);
        if ((v = s.cnt[2 * kMaxKC64 + i]) != 0ull) atomicAdd(&a->inf, v);
        s.cnt[i] = 0ull;
        s.cnt[kMaxKC64 + i] = 0ull;
        s.cnt[2 * kMaxKC64 + i] = 0ull;
      }
      for (int i = tid; i < kMaxKC64 * kWarps; i += kConsumers) {
        s.thr[2 * i] = kThNone;
        s.thr[2 * i + 1] = 0ll;
      }
      return consumers_barrier();
    };

    // What the other CTAs have recorded comes back by reading the global accumulator:
    // lane (warp, lane) owns candidate warp + 8*lane of the chunk.  The (error, index)
    // pair is read as one unit with a 128-bit compare-and-swap that changes nothing.  A
    // value read at one stage is applied at the next (the round trip to L2 is then
    // hidden), except on a chunk's first stage.  An error equal to one recorded at a lower
    // index, or strictly below one recorded anywhere, can never become the maximum.
    const int xkk = warp + kWarps * lane;
    unsigned long long xk = 0ull, xl = 0ull, xr = 0ull, xr_applied = 0ull;
    long long xlim_applied = -1ll;
    unsigned long long prev_base = 0ull;
    auto exchange_issue = [&]() {
      if (xkk < cur_kc) {
        Acc64* a = &p.acc[cur_k0 + xkk];
        Key128 zero;
        zero.lo = zero.hi = 0ull;
        const Key128 cur = atomicCAS(&a->key, zero, zero);
        xk = cur.hi;
        xl = cur.lo;
        xr = *reinterpret_cast<const volatile unsigned long long*>(&a->rel);
      }
    };
    // `safe_base`: every element any warp of this CTA may still look at has an index >= it.
    auto exchange_apply = [&](unsigned long long safe_base) {
      if (xkk < cur_kc) {
        long long* row = &s.thr[(size_t)xkk * kWarps * 2];
        if (xr > xr_applied) {
          xr_applied = xr;
#pragma unroll
          for (int w2 = 0; w2 < kWarps; ++w2) atomicMax(row + 2 * w2 + 1, (long long)xr);
        }
        if (xk != 0ull) {
          const long long db = (long long)(xk - 1ull);
          const unsigned long long gidx = 0xFFFFFFFFull - xl;
          const long long lim = gidx < safe_base ? db : db - 1;
          if (lim > xlim_applied) {
            xlim_applied = lim;
#pragma unroll
            for (int w2 = 0; w2 < kWarps; ++w2) atomicMax(row + 2 * w2, lim);
          }
        }
      }
      __syncwarp();
    };

    for (;;) {
      if (!mbar_wait_bounded(&s.full[stage], phase, s.abort_flag, p.status)) {
        ok = false;
        break;
      }
      const unsigned long long item = *reinterpret_cast<volatile unsigned long long*>(&s.item_id[stage]);
      if (item == kNoItem) break;
      const uint32_t chunk = (uint32_t)(item / p.nhalf);
      const uint32_t slot = p.half0 + (uint32_t)(item % p.nhalf);
      const uint32_t tile = p.tile_list ? p.tile_list[slot >> 1] : (slot >> 1);
      const bool first_of_chunk = (int)chunk != cur_chunk;
      if (first_of_chunk) {
        if (cur_chunk >= 0 && !flush()) {
          ok = false;
          break;
        }
        cur_chunk = (int)chunk;
        cur_k0 = chunk * p.KC;
        cur_kc = (int)min(p.KC, p.K - cur_k0);
        xk = xl = xr = xr_applied = 0ull;
        xlim_applied = -1ll;
      }
      const unsigned long long elem_base =
          (unsigned long long)tile * kTile + (unsigned long long)(slot & 1u) * kTile64;

      // The slowest warp may still be up to (ring depth - 1) stages back, inside the previous
      // item if items are at least that long: only what lies below the previous item's
      // elements is "earlier" for every warp.  (On a chunk's first item the flush barrier has
      // just lined the warps up.)
      if (!first_of_chunk) exchange_apply((uint32_t)cur_kc + 1u >= stages ? prev_base : 0ull);
      prev_base = elem_base;
      exchange_issue();

      // ---- reference stage: 8 elements per thread stay in registers ----
      double r[kEPT64];
      bool extreme = false;   // 0 < |r| < 2^-960: the filter's multiply-add could underflow to
                              // zero and lose its sign; such threads go exact
      {
        const double2* src = reinterpret_cast<const double2*>(s.buf + (size_t)stage * kTileBytes64);
#pragma unroll
        for (int j = 0; j < kEPT64 / 2; ++j) {
          const double2 v = src[tid + kConsumers * j];
          r[2 * j] = v.x;
          r[2 * j + 1] = v.y;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&s.empty[stage]);
        if (++stage == stages) {
          stage = 0;
          phase ^= 1u;
        }
#pragma unroll
        for (int e = 0; e < kEPT64; ++e) {
          const double ar = fabs(r[e]);
          extreme |= (ar > 0.0 && ar < 1.0261342003245941e-289);   // 2^-960
        }
      }
      if (first_of_chunk) exchange_apply(elem_base);

      for (int kk = 0; kk < cur_kc; ++kk) {
        const volatile long long* tw = &s.thr[((size_t)kk * kWarps + warp) * 2];
        const double th = __longlong_as_double(tw[0]);
        const double rel = __longlong_as_double(tw[1]);
        if (!mbar_wait_bounded(&s.full[stage], phase, s.abort_flag, p.status)) {
          ok = false;
          break;
        }
        double c[kEPT64];
        {
          const double2* src = reinterpret_cast<const double2*>(s.buf + (size_t)stage * kTileBytes64);
#pragma unroll
          for (int j = 0; j < kEPT64 / 2; ++j) {
            const double2 v = src[tid + kConsumers * j];
            c[2 * j] = v.x;
            c[2 * j + 1] = v.y;
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&s.empty[stage]);
        if (++stage == stages) {
          stage = 0;
          phase ^= 1u;
        }

        bool bad = false, trig = extreme;
#pragma unroll
        for (int e = 0; e < kEPT64; ++e) {
          const double ad = fabs(__dsub_rn(c[e], r[e]));
          const double ar = fabs(r[e]);
          const double tol = __dadd_rn(p.atol, __dmul_rn(p.rtol, ar));
          bad |= !(ad <= tol);
          trig |= (ad > th) || !(__fma_rn(-rel, ar, ad) <= 0.0);
        }
        // Every vote below is reached by all 32 lanes.
        if (!__any_sync(0xFFFFFFFFu, trig || bad)) continue;
        // Threads that saw an element out of tolerance count their finite mismatches here; a
        // NaN or Inf difference sends them down the exact path.
        unsigned int mis_fast = 0u;
        if (bad) {
          bool nonfin = false;
#pragma unroll
          for (int e = 0; e < kEPT64; ++e) {
            const double ad = fabs(__dsub_rn(c[e], r[e]));
            const double tol = __dadd_rn(p.atol, __dmul_rn(p.rtol, fabs(r[e])));
            const bool fin = ad <= kDblMax;
            nonfin |= !fin;
            mis_fast += (ad > tol && fin) ? 1u : 0u;   // (c == r gives ad = 0 <= tol)
          }
          trig = trig || nonfin;
        }
        if (!__any_sync(0xFFFFFFFFu, trig)) {
          const unsigned int tot = warp_add_u32(mis_fast);
          if (lane == 0 && tot) atomicAdd(&s.cnt[kk], (unsigned long long)tot);
          continue;
        }

        // ---- exact path ----
        unsigned int n_mis = 0, n_nan = 0, n_inf = 0;
        unsigned long long qb = 0ull, bd = 0ull;
        unsigned int bi = 0u;
        if (trig) {
          double m = -1.0;
          int mi = 0;
#pragma unroll
          for (int e = 0; e < kEPT64; ++e) {
            const double ad = fabs(__dsub_rn(c[e], r[e]));
            const double ar = fabs(r[e]);
            const double t = __fma_rn(-rel, ar, ad);
            const double tol = __dadd_rn(p.atol, __dmul_rn(p.rtol, ar));
            const bool fin = ad <= kDblMax;
            if (fin && ad > m) {
              m = ad;
              mi = e;
            }
            const bool hot = !(t <= 0.0) || !fin || extreme || !(ad <= tol);
            if (hot) {
              const bool match = (c[e] == r[e]) || (fin && ad <= tol);
              n_mis += match ? 0u : 1u;
              n_nan += (c[e] != c[e]) ? 1u : 0u;
              n_inf += (fabs(c[e]) == __longlong_as_double(0x7FF0000000000000ll)) ? 1u : 0u;
              if (fin && ar > 0.0 && ar <= kDblMax && (extreme || t > 0.0)) {
                const unsigned long long q = (unsigned long long)__double_as_longlong(__ddiv_rn(ad, ar));
                qb = q > qb ? q : qb;
              }
            }
          }
          if (m > th) {
            const unsigned long long idx =
                elem_base + (unsigned long long)((tid + kConsumers * (mi >> 1)) * 2 + (mi & 1));
            bd = (unsigned long long)__double_as_longlong(m) + 1ull;
            bi = 0xFFFFFFFFu - (unsigned int)idx;
          }
        }
        if (!trig) n_mis = mis_fast;
        n_mis = warp_add_u32(n_mis);
        n_nan = warp_add_u32(n_nan);
        n_inf = warp_add_u32(n_inf);
        const unsigned long long hmax = warp_max_u64(bd);
        const unsigned int lmax = warp_max_u32(bd == hmax ? bi : 0u);
        qb = warp_max_u64(qb);
        if (lane == 0) {
          if (n_mis) atomicAdd(&s.cnt[kk], (unsigned long long)n_mis);
          if (n_nan) atomicAdd(&s.cnt[kMaxKC64 + kk], (unsigned long long)n_nan);
          if (n_inf) atomicAdd(&s.cnt[2 * kMaxKC64 + kk], (unsigned long long)n_inf);
          long long* row = &s.thr[(size_t)kk * kWarps * 2];
          Acc64* a = &p.acc[cur_k0 + kk];
          if (hmax != 0ull) {
            merge_key(a, hmax, (unsigned long long)lmax);
            // what this warp meets later with an error <= this one loses the index tie; for
            // the other warps (same stage, other indices) only strictly smaller errors do
            const long long db = (long long)(hmax - 1ull);
#pragma unroll
            for (int w2 = 0; w2 < kWarps; ++w2) {
              const long long lim = (w2 == warp) ? db : db - 1;
              if (lim >= 0) atomicMax(row + 2 * w2, lim);
            }
          }
          if (qb > (unsigned long long)__double_as_longlong(rel)) {
            atomicMax(&a->rel, qb);
#pragma unroll
            for (int w2 = 0; w2 < kWarps; ++w2) atomicMax(row + 2 * w2 + 1, (long long)qb);
          }
        }
        __syncwarp();
      }
      if (!ok) break;
    }
    if (ok && cur_chunk >= 0) flush();
  }
  // ---- the last CTA to get here unpacks all K records ----
  __shared__ unsigned int s_ticket;
  __threadfence();
  __syncthreads();
  if (tid == 0) s_ticket = atomicAdd(p.done, 1u);
  __syncthreads();
  if (s_ticket == gridDim.x - 1) {
    __threadfence();
    for (unsigned int k = tid; k < p.K; k += kStreamThreads) {
      Acc64 a;
      a.key.lo = __ldcg(&p.acc[k].key.lo);
      a.key.hi = __ldcg(&p.acc[k].key.hi);
      a.mism = __ldcg(&p.acc[k].mism);
      a.nan = __ldcg(&p.acc[k].nan);
      a.inf = __ldcg(&p.acc[k].inf);
      a.rel = __ldcg(&p.acc[k].rel);
      unpack_record64(a, &p.out[k]);
    }
  }
}

}  // namespace kb
