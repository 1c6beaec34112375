// The correctness gate's streaming kernel for 8-bit floats, used for e4m3 (Sec. 3.1 K(p);
// Sec. 3.4 Verifier).  Same plan as screen_stream_kernel -- work items drawn from a global
// counter, one producer lane feeding a ring of shared-memory stages with 1-D bulk copies,
// thresholds exchanged between CTAs, integer merges, the last CTA unpacks -- with what a
// byte per element changes:
//
//  * 128 consumer threads per CTA, 32 elements (two 16-byte words) per thread and 4 KB
//    stage: the per-stage work (barrier wait and arrive, threshold read, vote) is paid half
//    as often per element as with 16 elements per thread.
//  * A PACKED HALF-PRECISION PRE-FILTER in front of the binary32 filter.  Every value of
//    either 8-bit format is a binary16 value, so pairs are widened exactly by one conversion;
//    with s = sign(r), |c - r| = |s*c - |r||, so the reference is kept as |r| (f16x2) and the
//    sign flip is one XOR on the raw bytes.  Per pair: d = s*c - |r| (rounded to binary16),
//    a = |d|, t = fma(-rel16, |r|, a), two maxima.  rel16 and th16 are the running maxima
//    rounded DOWN to binary16.  A thread is certainly clean if a <= th16 and t <= 0 for all
//    its elements and nothing is NaN:
//      - where the subtraction is exact in binary16 (always, unless the two exponents differ
//        by 7 or more: the difference of two 4-bit significands g binades apart has at most
//        g + 5 bits), a = |c - r| exactly, the fused multiply-add rounds once and keeps its
//        sign, and rel16 <= rel, th16 <= th give |c - r| <= th and |c - r| - rel*|r| <= 0: the
//        binary32 filter's conditions (b) and (c);
//      - where it is not exact, one magnitude is more than 64 times the other, so
//        |c - r| >= (63/64) * max(|c|, |r|) and t >= |r| * (63/64 - 1/1024 - rel16) > 0
//        (or, for |c| >> |r|, far above rel16*|r|) as long as rel16 <= 1/2: condition (c)
//        fails and the thread is not declared clean.  The pre-filter is therefore used only
//        with a lean bound of at most 1/2 (rtol <= 1/2); beyond the bound rel is clamped to it,
//        as in the binary32 filter (a clean element then matches, since |c - r| <= rtol_lean*|r|
//        <= tol, and its quotient stays below the real, larger maximum);
//      - the fused multiply-add must not round a positive t to zero.  In e4m3 every |c - r| and
//        every |r| is a multiple of 2^-9, rel16 a multiple of 2^(e-10) with e its exponent, so the
//        exact t is a multiple of 2^(e-19): for rel16 >= 2^-5 (or rel16 = 0, t = a) that is a
//        multiple of 2^-24, which binary16 holds exactly down to its smallest subnormal.  The
//        pre-filter is skipped for 0 < rel < 2^-5 (8-bit formats cannot produce so small a
//        largest relative error from a real difference).  e5m2 goes down to 2^-16 with two
//        fraction bits: products with its tiny values would need a guard that flags most warps
//        on data that has any, so e5m2 stays with screen_stream_kernel.
//    A warp none of whose threads is flagged has finished the step; otherwise the whole warp
//    runs the binary32 step of screen_stream_kernel on its two 16-element groups.
//  * The thresholds a warp reads decide which vote it takes next (pre-filter or binary32
//    step), so lane 0's copy is broadcast to the warp, and a wait that gives up does so for the
//    whole warp.
//  * No sharp instantiation and no count of fruitless second looks.
#pragma once

#include "kb_screen.cuh"

namespace kb {

constexpr int kCons8 = 128;            // consumer threads per CTA (4 warps)
constexpr int kWarps8 = kCons8 / 32;
constexpr int kThreads8 = kCons8 + 32;
constexpr int kGroups8 = 2;            // 16-byte words (groups of 16 elements) per thread and tile

__host__ __device__ inline size_t stream8_smem_bytes(uint32_t stages) {
  size_t b = (size_t)stages * kTile;
  b += (size_t)kMaxKC * 16;
  b += 3 * (size_t)stages * 8 + 8;
  b += 3 * (size_t)kMaxKC * 8 + (size_t)kMaxKC * 8 + (size_t)kMaxKC * 8 + (size_t)kMaxKC * 4;
  b += (size_t)kMaxKC * kWarps8 * 8;
  b += 16;
  return b + 128;  // alignment slack
}

template <int DT>
__global__ void __maxnreg__(96) screen_stream8_kernel(const StreamParams p) {
  using E = Elem<DT>;
  static_assert(E::kBytes == 1 && E::kVec == 16, "the 8-bit formats only");
  constexpr bool SHARP = false;
  constexpr bool kPrefilter = DT == KB_F8E4M3;   // see the head of this file
  constexpr int VEC = 16;
  constexpr uint32_t TILE_BYTES = kTile;
  constexpr int kConsumers = kCons8;      // (shadow the 16-bit kernel's constants)
  constexpr int kWarps = kWarps8;
  constexpr int kStreamThreads = kThreads8;
  const float kInf = __uint_as_float(0x7F800000u);
  const float kFltMax = 3.402823466e38f;

  extern __shared__ unsigned char smem_raw[];
  StreamSmem s;
  {
    uintptr_t base = (reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127;
    unsigned char* q = reinterpret_cast<unsigned char*>(base);
    s.buf = q;
    q += (size_t)p.stages * TILE_BYTES;
    s.xg = reinterpret_cast<uint4*>(q);
    q += (size_t)kMaxKC * 16;
    s.full = reinterpret_cast<uint64_t*>(q);
    q += (size_t)p.stages * 8;
    s.empty = reinterpret_cast<uint64_t*>(q);
    q += (size_t)p.stages * 8;
    s.sync_bar = reinterpret_cast<uint64_t*>(q);
    q += 8;
    s.item_id = reinterpret_cast<unsigned long long*>(q);
    q += (size_t)p.stages * 8;
    s.cnt = reinterpret_cast<unsigned long long*>(q);
    q += 3 * (size_t)kMaxKC * 8;
    s.key = reinterpret_cast<unsigned long long*>(q);
    q += (size_t)kMaxKC * 8;
    s.ptrs = reinterpret_cast<const void**>(q);
    q += (size_t)kMaxKC * 8;
    s.thr2 = reinterpret_cast<float2*>(q);
    q += (size_t)kMaxKC * kWarps * 8;
    s.rel = reinterpret_cast<unsigned int*>(q);
    q += (size_t)kMaxKC * 4;
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
  for (int i = tid; i < kMaxKC; i += kStreamThreads) {
    s.cnt[i] = 0ull;
    s.cnt[kMaxKC + i] = 0ull;
    s.cnt[2 * kMaxKC + i] = 0ull;
    s.key[i] = 0ull;
    s.rel[i] = 0u;
    s.xg[i] = make_uint4(0u, 0u, 0u, 0u);
  }
  for (int i = tid; i < kMaxKC * kWarps; i += kStreamThreads) s.thr2[i] = make_float2(-1.0f, 0.0f);
  __syncthreads();

  // Work items (chunk, tile), chunk-major, are drawn from a global counter: a CTA gets
  // ascending items (so ascending tiles inside a chunk, which the index tie-break needs),
  // the CTAs that run together work on neighbouring tiles, and the tail is one item long.
  const uint32_t K_eff = p.K_dev ? min(*p.K_dev, p.K) : p.K;
  const uint32_t nchunks_eff = (K_eff + p.KC - 1) / p.KC;
  const unsigned long long nitems = (unsigned long long)nchunks_eff * p.ntiles;

  if (warp == kWarps) {
    // ------------------------------ producer ------------------------------
    const RingProducerView ring{s.buf, s.full, s.empty, s.item_id, s.ptrs, s.abort_flag};
    const TileItemMap map{p.ntiles, p.slot0, p.KC, K_eff, p.tile_list, TILE_BYTES};
    ring_producer(ring, map, lane, stages, TILE_BYTES, nitems, p.sched, p.ref, p.cands, p.nchunks > 1, p.status);
  } else {
    // ------------------------------ consumers -----------------------------
    uint32_t stage = 0, phase = 0;
    int cur_chunk = -1;
    int cur_kc = 0;
    uint32_t cur_k0 = 0;
    bool ok = true;

    // Consumer-wide barrier whose wait is bounded (a timed-out warp raises the abort flag,
    // which releases everyone else's waits as well).
    uint32_t sync_phase = 0;
    auto consumers_barrier = [&]() -> bool {
      __syncwarp();
      if (lane == 0) mbar_arrive(s.sync_bar);
      const bool done = mbar_wait_bounded(s.sync_bar, sync_phase, s.abort_flag, p.status);
      sync_phase ^= 1u;
      return done;
    };
    // Move the chunk's shared-memory accumulators to global memory and reset them.
    auto flush = [&]() -> bool {
      cp_async_wait_all();   // this thread's last fetch has landed before the slots are cleared
      if (!consumers_barrier()) return false;
      for (int i = tid; i < cur_kc; i += kConsumers) {
        Acc* a = &p.acc[cur_k0 + i];
        unsigned long long v;
        if ((v = s.cnt[i]) != 0ull) atomicAdd(&a->mism, v);
        if ((v = s.cnt[kMaxKC + i]) != 0ull) atomicAdd(&a->nan, v);
        if ((v = s.cnt[2 * kMaxKC + i]) != 0ull) atomicAdd(&a->inf, v);
        if ((v = s.key[i]) != 0ull) atomicMax(&a->key, v);
        unsigned int r = s.rel[i];
        if (r != 0u) atomicMax(&a->rel, r);
        s.cnt[i] = 0ull;
        s.cnt[kMaxKC + i] = 0ull;
        s.cnt[2 * kMaxKC + i] = 0ull;
        s.key[i] = 0ull;
        s.rel[i] = 0u;
      }
      for (int i = tid; i < kMaxKC; i += kConsumers) s.xg[i] = make_uint4(0u, 0u, 0u, 0u);
      for (int i = tid; i < kMaxKC * kWarps; i += kConsumers) s.thr2[i] = make_float2(-1.0f, 0.0f);
      return consumers_barrier();
    };

    // Exchange of running maxima with the other CTAs.  Every merge is a maximum, so the
    // exchange needs no ordering: lane (warp, lane) owns candidate warp + 8*lane of the
    // chunk, pushes this CTA's maxima with atomicMax (no return value) and fetches the
    // global (key, rel) block with an asynchronous copy into shared memory.  What comes
    // back is applied one tile later (the round trip to L2 is then hidden and no register
    // waits for it), except on a chunk's first tile, where the scout's seeds are wanted at once.
    const int xkk = warp + kWarps * lane;
    bool xpending = false;
    auto exchange_issue = [&]() {
      if (xkk < cur_kc) {
        const unsigned long long mk = *reinterpret_cast<volatile unsigned long long*>(&s.key[xkk]);
        const unsigned int mr = *reinterpret_cast<volatile unsigned int*>(&s.rel[xkk]);
        Acc* a = &p.acc[cur_k0 + xkk];
        // push only what exceeds the last fetched global values (maxima only grow): once the
        // maxima have settled nobody writes, and the accumulator's line is only read
        const volatile uint4* slot = &s.xg[xkk];
        const unsigned long long seen_k = ((unsigned long long)slot->y << 32) | slot->x;
        if (mk > seen_k) atomicMax(&a->key, mk);
        if (mr > slot->z) atomicMax(&a->rel, mr);
        cp_async16(&s.xg[xkk], &a->key);
      }
      cp_async_commit();
    };
    // `safe_base`: every element any warp of this CTA may still look at has an index >= it
    // (warps drift apart by less than the ring depth, i.e. by less than one work item).
    auto exchange_apply = [&](unsigned long long safe_base) {
      cp_async_wait_all();
      if (xkk < cur_kc) {
        const volatile uint4* slot = &s.xg[xkk];
        const unsigned long long gk0 = ((unsigned long long)slot->y << 32) | slot->x;
        const unsigned int gr = slot->z;
        const unsigned long long mk = *reinterpret_cast<volatile unsigned long long*>(&s.key[xkk]);
        int* row = reinterpret_cast<int*>(&s.thr2[xkk * kWarps]);
        if (gr > *reinterpret_cast<volatile unsigned int*>(&s.rel[xkk])) {
          atomicMax(&s.rel[xkk], gr);
#pragma unroll
          for (int w2 = 0; w2 < kWarps; ++w2) atomicMax(row + 2 * w2 + 1, (int)gr);
        }
        const unsigned long long gk = gk0 > mk ? gk0 : mk;
        if (gk != 0ull) {
          // An error equal to one recorded at a lower index, or strictly below one
          // recorded anywhere, can never become the maximum.
          const unsigned int db = (unsigned int)((gk - 1ull) >> 32);
          const unsigned long long gidx = 0xFFFFFFFFull - ((gk - 1ull) & 0xFFFFFFFFull);
          const int lim = gidx < safe_base ? (int)db : (int)db - 1;   // db == 0: -1 is below every float >= -1
          if (lim >= 0) {
#pragma unroll
            for (int w2 = 0; w2 < kWarps; ++w2) atomicMax(row + 2 * w2, lim);
          }
        }
      }
      __syncwarp();
    };
    uint32_t prev_tile = 0;

    for (;;) {
      // the next stage holds a reference tile and names its work item (or the end)
      if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(&s.full[stage], phase, s.abort_flag, p.status))) {
        ok = false;
        break;
      }
      const unsigned long long item = *reinterpret_cast<volatile unsigned long long*>(&s.item_id[stage]);
      if (item == kNoItem) break;
      const uint32_t chunk = (uint32_t)(item >> 32);
      const uint32_t slot = p.slot0 + (uint32_t)item;
      const uint32_t tile = p.tile_list ? p.tile_list[slot] : slot;
      const bool first_of_chunk = (int)chunk != cur_chunk;
      if (first_of_chunk) {
        xpending = false;
        if (cur_chunk >= 0 && !flush()) {
          ok = false;
          break;
        }
        cur_chunk = (int)chunk;
        cur_k0 = chunk * p.KC;
        cur_kc = (int)min(p.KC, K_eff - cur_k0);
      }
      const unsigned long long tile_base = (unsigned long long)tile * kTile;

      // Not all warps are in this item yet: the slowest may still be up to (ring depth - 1)
      // stages back, inside the previous item if items are at least that long, so only what
      // lies below the previous item's tile is "earlier" for everyone.  (On a chunk's first
      // item the flush barrier has just lined the warps up.)
      if (xpending)
        exchange_apply((uint32_t)cur_kc + 1u >= stages ? (unsigned long long)prev_tile * kTile : 0ull);
      prev_tile = tile;
      exchange_issue();
      xpending = !first_of_chunk;

      // ---- reference tile: 32 elements per thread stay in registers, as raw bytes (for the
      // binary32 step and for the sign flip) and as |r| in packed binary16 (for the pre-filter) ----
      uint4 rw[kGroups8];
      unsigned int ar2[kGroups8 * 8];
      {
        const uint4* src = reinterpret_cast<const uint4*>(s.buf + (size_t)stage * TILE_BYTES);
#pragma unroll
        for (int g = 0; g < kGroups8; ++g) rw[g] = src[tid + kConsumers * g];
        __syncwarp();
        if (lane == 0) mbar_arrive(&s.empty[stage]);
        if (++stage == stages) {
          stage = 0;
          phase ^= 1u;
        }
        const unsigned int* rwords = reinterpret_cast<const unsigned int*>(rw);
#pragma unroll
        for (int i = 0; i < kGroups8 * 4; ++i) E::widen4(rwords[i] & 0x7F7F7F7Fu, ar2[2 * i], ar2[2 * i + 1]);
      }
      if (first_of_chunk) exchange_apply(tile_base);

      // ---- the candidates of this chunk against the tile in registers ----
      for (int kk = 0; kk < cur_kc; ++kk) {
        // The thresholds decide which of two votes this warp takes next (pre-filter or binary32
        // step), so every lane must hold the SAME pair: other warps update the slot with atomics
        // at any time, and lanes that are not converged at this load (lane 0 has just arrived on
        // a barrier by itself) could read different values.  Lane 0's copy is broadcast.
        const unsigned long long trw = __shfl_sync(
            0xFFFFFFFFu, *reinterpret_cast<volatile unsigned long long*>(&s.thr2[kk * kWarps + warp]), 0);
        const float th = __uint_as_float((unsigned int)trw);
        const float rel = __uint_as_float((unsigned int)(trw >> 32));
        // (a wait that gave up in one lane gives up for the warp: no lane is left behind at a vote)
        if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(&s.full[stage], phase, s.abort_flag, p.status))) {
          ok = false;
          break;
        }
        const uint4* src = reinterpret_cast<const uint4*>(s.buf + (size_t)stage * TILE_BYTES);
        uint4 w8[kGroups8];
#pragma unroll
        for (int g = 0; g < kGroups8; ++g) w8[g] = src[tid + kConsumers * g];
        __syncwarp();
        if (lane == 0) mbar_arrive(&s.empty[stage]);
        if (++stage == stages) {
          stage = 0;
          phase ^= 1u;
        }

        // ---- the packed half-precision pre-filter (see the head of this file) ----
        // (with the relative error clamped to the lean bound, as in the binary32 filter: beyond
        // it a clean thread's elements still match and cannot raise the larger real maximum)
        const float rel_l0 = fminf(rel, p.rtol_lean);
        if (kPrefilter && p.rtol_lean >= 0.0f && p.rtol_lean <= 0.5f &&
            (rel_l0 == 0.0f || rel_l0 >= 0.03125f)) {
          const unsigned int* cw = reinterpret_cast<const unsigned int*>(w8);
          const unsigned int* rwords = reinterpret_cast<const unsigned int*>(rw);
          // running maxima rounded toward zero (down: both are >= 0, or th is -1 "none")
          unsigned short th16, nrel16;
          asm("cvt.rz.f16.f32 %0, %1;" : "=h"(th16) : "f"(th));
          asm("cvt.rz.f16.f32 %0, %1;" : "=h"(nrel16) : "f"(rel_l0));
          const unsigned int nrel2 = (((unsigned int)nrel16 << 16) | nrel16) ^ 0x80008000u;   // -rel16 twice
          unsigned int mabs2 = 0u, mrel2 = 0u;
#pragma unroll
          for (int i = 0; i < kGroups8 * 4; ++i) {
            // four candidate bytes with the reference's signs flipped in (s*c), widened pairwise
            const unsigned int x = cw[i] ^ (rwords[i] & 0x80808080u);
            unsigned int c2a, c2b;
            E::widen4(x, c2a, c2b);
            unsigned int da, db, ta, tb;
            asm("sub.rn.f16x2 %0, %1, %2;" : "=r"(da) : "r"(c2a), "r"(ar2[2 * i]));
            asm("sub.rn.f16x2 %0, %1, %2;" : "=r"(db) : "r"(c2b), "r"(ar2[2 * i + 1]));
            asm("abs.f16x2 %0, %0;" : "+r"(da));
            asm("abs.f16x2 %0, %0;" : "+r"(db));
            asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(ta) : "r"(nrel2), "r"(ar2[2 * i]), "r"(da));
            asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(tb) : "r"(nrel2), "r"(ar2[2 * i + 1]), "r"(db));
            asm("max.NaN.f16x2 %0, %0, %1;" : "+r"(mabs2) : "r"(da));
            asm("max.NaN.f16x2 %0, %0, %1;" : "+r"(mabs2) : "r"(db));
            asm("max.NaN.f16x2 %0, %0, %1;" : "+r"(mrel2) : "r"(ta));
            asm("max.NaN.f16x2 %0, %0, %1;" : "+r"(mrel2) : "r"(tb));
          }
          // flagged: an error above th16, a positive or NaN t in either half
          const __half2 ma = *reinterpret_cast<const __half2*>(&mabs2);
          const __half2 mr = *reinterpret_cast<const __half2*>(&mrel2);
          const float thf = __half2float(*reinterpret_cast<const __half*>(&th16));
          const float ma_hi = fmaxf(__low2float(ma), __high2float(ma));
          const float mr_hi = max2_nan(__low2float(mr), __high2float(mr));
          const bool flagged = !(ma_hi <= thf) || !(mr_hi <= 0.0f);
          if (!__any_sync(0xFFFFFFFFu, flagged)) continue;
        }

        // ---- the binary32 step of screen_stream_kernel on each group of 16 elements ----
#pragma unroll 1
        for (int g = 0; g < kGroups8; ++g) {
        float r[16];
        E::decode(g ? rw[1] : rw[0], r);     // (selects, not indexing: the words stay in registers)
        const uint4 wg = g ? w8[1] : w8[0];
        const unsigned int* words = reinterpret_cast<const unsigned int*>(&wg);
        constexpr int kEPT = 16;
        const bool extreme = false;   // no 8-bit value lies in (0, 2^-100)
        const bool has_lean = p.rtol_lean >= 0.0f;
        const bool lean = rel <= p.rtol_lean;
        const float rel_f = (has_lean && !lean) ? p.rtol_lean : rel;
        float mabs = 0.0f, mrel = 0.0f;
        // g = (ulp(rel)/2)*(1 - 2^-20), or 0 where that would be subnormal
        auto half_ulp_of_rel = [&]() -> float {
          const unsigned int rb = __float_as_uint(rel);
          return rb >= (30u << 23)
                     ? __uint_as_float((rb & 0x7F800000u) - (24u << 23)) * 0.99999904632568359375f
                     : 0.0f;
        };
        const bool sharp = SHARP && lean;
        if (!SHARP || !sharp) {
#pragma unroll
          for (int e = 0; e < kEPT; e += 2) {
            float d0, d1;
            E::pair_diff(words, e, r[e], r[e + 1], d0, d1);
            const float t0 = fmaf(-rel_f, fabsf(r[e]), fabsf(d0));
            const float t1 = fmaf(-rel_f, fabsf(r[e + 1]), fabsf(d1));
            mabs = max3(mabs, fabsf(d0), fabsf(d1));
            mrel = max3_nan(mrel, t0, t1);
          }
        } else {
          const float g = half_ulp_of_rel();
#pragma unroll
          for (int e = 0; e < kEPT; e += 2) {
            float d0, d1;
            E::pair_diff(words, e, r[e], r[e + 1], d0, d1);
            const float ar0 = fabsf(r[e]), ar1 = fabsf(r[e + 1]);
            const float t0 = fmaf(-rel, ar0, fabsf(d0)), t1 = fmaf(-rel, ar1, fabsf(d1));
            // t <= 0: fine as before.  A normal t > 0 with t - g*|r| <= 0: the quotient still rounds
            // to at most rel.  A tiny positive t, NaN or Inf stay positive or NaN: the exact path.
            const float v0 = t0 >= 7.888609052e-31f ? fmaf(-g, ar0, t0) : t0;
            const float v1 = t1 >= 7.888609052e-31f ? fmaf(-g, ar1, t1) : t1;
            mabs = max3(mabs, fabsf(d0), fabsf(d1));
            mrel = max3_nan(mrel, v0, v1);
          }
        }
        // A thread whose (c) fails, or (no lean bound) whose largest error exceeds atol, looks
        // again element by element below before its warp is sent down the exact path.
        // A thread whose (c) fails, or (no lean bound) whose largest error exceeds atol, looks
        // again element by element below before its warp is sent down the exact path.
        const bool bad = !(mrel <= 0.0f) || (!has_lean && mabs > p.atol);
        bool trig = (mabs > th) || extreme;
        (void)extreme;
        // Every vote below is reached by all 32 lanes: no warp-synchronous call sits under a
        // condition that could differ between lanes.
        if (!__any_sync(0xFFFFFFFFu, trig || bad)) continue;
        // Threads that saw an element out of tolerance count their finite mismatches here, so
        // that a failing candidate does not send every step down the exact path; a NaN or Inf
        // difference still does.
        unsigned int mis_fast = 0u;
        if (bad && lean) {
          // The second look while lean: the warp goes on to the exact path only for a NaN or Inf
          // difference or a quotient that can round above rel.  That test is sharper than (c):
          // with t = fl(ad - rel*|r|) > 0 the quotient still rounds to at most rel while
          // ad/|r| < rel + ulp(rel)/2, which t <= g*|r| with g = (ulp(rel)/2)*(1 - 2^-20)
          // guarantees for a normal t (t carries a relative error of 2^-24 at most).  So elements
          // whose quotient was rounded DOWN to the running maximum (every element of the same
          // significand class, if the maximum comes from one-ulp differences) stop here instead
          // of taking the exact path each time.  Such an element is within tolerance as well:
          // ad < (rel + ulp(rel)/2)*|r| < rtol*(1 - 2^-21)*|r| <= RN(rtol*|r|) <= tol.
          const float g = half_ulp_of_rel();
          // (A failure that is large against the thread's errors is a real new maximum: no
          // need to look.  An element of the kind above fails by 2^-24 of its error at most.
          // In the sharp instantiation the look has been taken already.)
          bool again = sharp || !(mrel <= mabs * 9.5367431640625e-07f);
          if (!again) {
#pragma unroll
          for (int e = 0; e < kEPT; e += 2) {
            float d0, d1;
            E::pair_diff(words, e, r[e], r[e + 1], d0, d1);
            const float ar0 = fabsf(r[e]), ar1 = fabsf(r[e + 1]);
            const float t0 = fmaf(-rel, ar0, fabsf(d0)), t1 = fmaf(-rel, ar1, fabsf(d1));
            // (a NaN or Inf difference makes t NaN or Inf: neither clause holds)
            const bool c0 = (t0 <= 0.0f) || (t0 >= 7.888609052e-31f && fmaf(-g, ar0, t0) <= 0.0f);
            const bool c1 = (t1 <= 0.0f) || (t1 >= 7.888609052e-31f && fmaf(-g, ar1, t1) <= 0.0f);
            again |= !c0 || !c1;
          }
          }
          trig = trig || again;
        } else if (bad) {
          // The second look beyond the lean bound: finite mismatches are counted here, so that
          // a failing candidate does not send every step down the exact path; a NaN or Inf
          // difference, or a failure of the real (c), still does.
          bool again = false;
#pragma unroll
          for (int e = 0; e < kEPT; e += 2) {
            float d0, d1;
            E::pair_diff(words, e, r[e], r[e + 1], d0, d1);
            const float a0 = fabsf(d0), a1 = fabsf(d1);
            const float tol0 = __fadd_rn(p.atol, __fmul_rn(p.rtol, fabsf(r[e])));
            const float tol1 = __fadd_rn(p.atol, __fmul_rn(p.rtol, fabsf(r[e + 1])));
            const bool f0 = a0 <= kFltMax, f1 = a1 <= kFltMax;
            again |= !f0 || !f1;
            again |= !(fmaf(-rel, fabsf(r[e]), a0) <= 0.0f) || !(fmaf(-rel, fabsf(r[e + 1]), a1) <= 0.0f);
            mis_fast += ((a0 > tol0) && f0) ? 1u : 0u;   // (c == r would give a0 = 0 <= tol0)
            mis_fast += ((a1 > tol1) && f1) ? 1u : 0u;
          }
          trig = trig || again;
        }
        if (!__any_sync(0xFFFFFFFFu, trig)) {
          const unsigned int tot = warp_add_u32(mis_fast);
          if (lane == 0 && tot) atomicAdd(&s.cnt[kk], (unsigned long long)tot);
          continue;
        }

        // ---- exact path.  A triggered thread finds its largest finite error (first
        // index on ties) with a running compare, and evaluates by the definition the
        // elements that fail the tolerance / relative-error filter or are not finite. ----
        unsigned int n_mis = 0, n_nan = 0, n_inf = 0, qb = 0u;
        unsigned long long best = 0ull;
        if (trig) {
          float c[kEPT];
          E::decode(wg, c);
          float m = -1.0f;
          int mi = 0;
#pragma unroll
          for (int e = 0; e < kEPT; ++e) {
            const float ad = fabsf(__fsub_rn(c[e], r[e]));
            const float ar = fabsf(r[e]);
            const float t = fmaf(-rel, ar, ad);
            const bool fin = ad <= kFltMax;
            if (fin && ad > m) {
              m = ad;
              mi = e;
            }
            bool hot = !(t <= 0.0f) || !fin || extreme;
            if (!lean) hot = hot || !(ad <= __fadd_rn(p.atol, __fmul_rn(p.rtol, ar)));
            if (hot) {
              const float tol = __fadd_rn(p.atol, __fmul_rn(p.rtol, ar));
              const bool match = (c[e] == r[e]) || (fin && ad <= tol);
              n_mis += match ? 0u : 1u;
              n_nan += (c[e] != c[e]) ? 1u : 0u;
              n_inf += (fabsf(c[e]) == kInf) ? 1u : 0u;
              if (fin && ar > 0.0f && ar <= kFltMax && (extreme || t > 0.0f)) {
                const unsigned int q = __float_as_uint(__fdiv_rn(ad, ar));
                qb = q > qb ? q : qb;
              }
            }
          }
          if (m > th) {
            const unsigned long long idx =
                tile_base + (unsigned long long)((tid + kConsumers * g) * VEC + mi);
            best = pack_key(m, idx);
          }
        }
        if (!trig) n_mis = mis_fast;   // lanes that did not take the exact path keep their fast count
        n_mis = warp_add_u32(n_mis);
        n_nan = warp_add_u32(n_nan);
        n_inf = warp_add_u32(n_inf);
        best = warp_max_u64(best);
        qb = warp_max_u32(qb);
        if (lane == 0) {
          if (n_mis) atomicAdd(&s.cnt[kk], (unsigned long long)n_mis);
          if (n_nan) atomicAdd(&s.cnt[kMaxKC + kk], (unsigned long long)n_nan);
          if (n_inf) atomicAdd(&s.cnt[2 * kMaxKC + kk], (unsigned long long)n_inf);
          int* row = reinterpret_cast<int*>(&s.thr2[kk * kWarps]);
          if (best != 0ull) {
            atomicMax(&s.key[kk], best);
            // what this warp meets in later tiles with an error <= this one loses the index
            // tie; for the other warps (same tile, other indices) only strictly smaller errors do
            const int db = (int)(unsigned int)((best - 1ull) >> 32);
#pragma unroll
            for (int w2 = 0; w2 < kWarps; ++w2) {
              const int lim = (w2 == warp) ? db : db - 1;
              if (lim >= 0) atomicMax(row + 2 * w2, lim);
            }
          }
          if (qb > __float_as_uint(rel)) {
            atomicMax(&s.rel[kk], qb);
#pragma unroll
            for (int w2 = 0; w2 < kWarps; ++w2) atomicMax(row + 2 * w2 + 1, (int)qb);
          }
        }
        __syncwarp();
        }   // groups
      }
      if (!ok) break;
    }
    if (ok && cur_chunk >= 0) flush();
  }
  // ---- the last CTA to get here unpacks all K records (saves a launch) ----
  __shared__ unsigned int s_ticket;
  __threadfence();
  __syncthreads();
  if (tid == 0) s_ticket = atomicAdd(p.done, 1u);
  __syncthreads();
  if (s_ticket == gridDim.x - 1) {
    __threadfence();
    for (unsigned int k = tid; k < p.K; k += kStreamThreads) {
      if (k >= K_eff) {
        write_absent_record(&p.out[k]);
        continue;
      }
      Acc a;
      a.mism = __ldcg(&p.acc[k].mism);
      a.nan = __ldcg(&p.acc[k].nan);
      a.inf = __ldcg(&p.acc[k].inf);
      a.key = __ldcg(&p.acc[k].key);
      a.rel = __ldcg(&p.acc[k].rel);
      unpack_record(a, &p.out[k]);
    }
  }
}


}  // namespace kb
