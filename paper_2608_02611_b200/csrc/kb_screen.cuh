// Correctness gate kernels (Sec. 3.1 K(p); Sec. 3.4 Verifier): compare K
// candidate tensors with one reference.
//
// screen_stream_kernel  the bandwidth-bound path.  CTAs draw work items
//   (candidate chunk, 4096-element tile) from a global counter, in ascending
//   order.  One producer lane feeds a ring of shared-memory stages with 1-D
//   bulk copies (TMA, each CTA its own): first the reference tile, then the same
//   tile of each candidate of the chunk.  256 consumer threads keep their 16
//   reference elements in registers for the whole item and run a branch-free
//   filter over each candidate stage; only warps whose filter fires take the
//   exact path.  Merges are integer adds and integer maxima on packed keys, so
//   the result does not depend on order.  The last CTA to finish unpacks the
//   K records.
// screen_lead_kernel    classifies a few leading tiles exactly before the
//   streaming kernel starts (their maxima seed its thresholds), and the ragged
//   tail past the last full tile; it also does the call's housekeeping (pointer
//   table from its own arguments, zeroing of the accumulators the NEXT call
//   will use), so that a call of up to 480 candidates is two launches.
// screen_generic_kernel plain loads, every element classified exactly; used
//   for masks finer than a kernel tile.
// Accumulators and counters exist twice: a call works on one set while its
//   lead kernel zeroes the other for the call after it, so no call needs a
//   zeroing launch and the streaming kernel's epilogue stays a plain unpack.
// screen_small_kernel / screen_multi_kernel  the latency regime: one launch
//   for a small problem / for several small problems of different shapes.
// screen_prep_kernel / screen_prep_indexed_kernel  pointer table, zeroed
//   accumulators and counters (the indexed form also validates a selection
//   that lives on the device).
// screen_finalize_kernel  unpacks the accumulators when no streaming launch did.
#pragma once

#include "kb_common.cuh"
#include "kb_ring.cuh"

namespace kb {

constexpr int kTile = 4096;       // elements per kernel tile
constexpr int kConsumers = 256;   // consumer threads per CTA (8 warps)
constexpr int kStreamThreads = kConsumers + 32;
constexpr int kEPT = 16;          // elements per consumer thread per tile
constexpr int kMaxKC = 128;       // candidates per chunk (shared-memory accumulators)
constexpr int kWarps = kConsumers / 32;

struct StreamParams {
  const void* ref;
  const void* const* cands;     // device table of K pointers
  Acc* acc;                     // [K], zeroed by the caller
  const uint32_t* tile_list;    // selected full tiles, ascending; NULL: tile = slot
  uint32_t ntiles;              // number of full tiles to visit
  uint32_t slot0;               // first slot of the tile list / first tile (earlier ones were scouted)
  uint32_t K, KC, nchunks;
  const unsigned int* K_dev;    // optional: the number of candidates actually present (<= K)
  uint32_t stages;
  float atol, rtol;
  float rtol_lean;              // rtol*(1-2^-20) rounded down, or -1: see the lean filter below
  unsigned int* status;
  unsigned int* done;           // zeroed ticket counter: the last CTA to finish unpacks the records
  unsigned long long* sched;    // zeroed work counter: CTAs draw items from it
  kb_screen_result* out;        // [K]
};

struct MaskDev {
  int kind;                     // 0 none, 1 strided, 2 bitmap
  uint32_t log2_tile, stride, phase;
  const unsigned long long* bits;
};

__device__ __forceinline__ bool mask_selected(const MaskDev& m, unsigned long long i) {
  if (m.kind == 0) return true;
  unsigned long long t = i >> m.log2_tile;
  if (m.kind == 1) return (t % m.stride) == m.phase;
  return (m.bits[t >> 6] >> (t & 63ull)) & 1ull;
}


// K pointers travel to the device table through kernel arguments (no staging
// buffer whose reuse would have to be fenced).
constexpr int kPtrsPerLaunch = 480;
struct PtrChunk {
  const void* p[kPtrsPerLaunch];
};
// accumulator -> public record
__device__ __forceinline__ void unpack_record(const Acc& a, kb_screen_result* dst) {
  kb_screen_result r;
  r.mismatch_count = a.mism;
  r.nan_count = a.nan;
  r.inf_count = a.inf;
  if (a.key == 0ull) {
    r.argmax_idx = -1;
    r.max_abs_err = 0.0f;
  } else {
    const unsigned long long kv = a.key - 1ull;
    r.max_abs_err = __uint_as_float((unsigned int)(kv >> 32));
    r.argmax_idx = (int64_t)(0xFFFFFFFFu - (unsigned int)kv);
  }
  r.max_rel_err = __uint_as_float(a.rel);
  r.pass = a.mism == 0ull ? 1u : 0u;
  r.reserved = 0u;
  *dst = r;
}

__device__ __forceinline__ void clear_acc(Acc* a) {
  Acc z;
  z.mism = z.nan = z.inf = z.spare = z.key = 0ull;
  z.rel = z.pad = 0u;
  *a = z;
}

// record of a candidate slot that holds no candidate (indexed screening with fewer
// survivors than slots): nothing counted, no index, not passed
__device__ __forceinline__ void write_absent_record(kb_screen_result* dst) {
  kb_screen_result r;
  r.mismatch_count = r.nan_count = r.inf_count = 0ull;
  r.argmax_idx = -1;
  r.max_abs_err = r.max_rel_err = 0.0f;
  r.pass = 0u;
  r.reserved = 0u;
  *dst = r;
}

// three-input maxima (one instruction on sm_100); the .NaN form returns NaN if any input is NaN
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float max3_nan(float a, float b, float c) {
  float d;
  asm("max.NaN.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float max2_nan(float a, float b) {
  float d;
  asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
  return d;
}

// Shared-memory carve-up (dynamic): stage buffers first (128-byte aligned).
struct StreamSmem {
  unsigned char* buf;
  uint4* xg;                 // [kMaxKC] landing slots of the global (key, rel) blocks (exchange)
  uint64_t* full;
  uint64_t* empty;
  uint64_t* sync_bar;        // consumer-wide barrier with a bounded wait (flush)
  unsigned long long* item_id;   // [stages] (chunk << 32 | position) of the work item whose reference
                                 // tile a stage holds; all ones: no more work
  unsigned long long* cnt;   // [4][kMaxKC] mism, nan, inf; fruitless second looks (plain instantiation)
  unsigned long long* key;   // [kMaxKC]
  const void** ptrs;         // [kMaxKC] candidate pointers of the current chunk (producer only)
  unsigned int* rel;         // [kMaxKC] bits of the running max relative error (CTA-wide)
  float2* thr2;              // [kMaxKC][kWarps] per warp: x = errors <= x cannot become the maximum
                             // (-1: none), y = the running max relative error (copy of rel)
  volatile unsigned int* abort_flag;
};

__host__ __device__ inline size_t stream_smem_bytes(uint32_t stages, uint32_t tile_bytes) {
  size_t b = (size_t)stages * tile_bytes;
  b += (size_t)kMaxKC * 16;
  b += 3 * (size_t)stages * 8 + 8;
  b += 4 * (size_t)kMaxKC * 8 + (size_t)kMaxKC * 8 + (size_t)kMaxKC * 8 + (size_t)kMaxKC * 4;
  b += (size_t)kMaxKC * kWarps * 8;
  b += 16;
  return b + 128;  // alignment slack
}

// The filter.  Per (tile, candidate) step a thread looks at its 16 elements and
// decides, without branches, whether anything about them could change the
// candidate's record; only then does its warp take the exact path.  With
//   ad = |c - r|,  rel = the CTA's running max of ad/|r|,  th = the warp's running max of ad,
// nothing can change if for every element
//   (b) ad <= th                          (an equal error in a later tile loses the index tie)
//   (c) ad - rel*|r| <= 0 as a real number (then ad/|r| cannot round above rel)
//   (a) ad <= atol + rtol*|r|              (match)
// and no NaN is involved.  (c) is one fused multiply-add, whose single rounding
// keeps the sign; a NaN-propagating max carries any NaN (a NaN or Inf candidate,
// Inf - Inf) to the decision.  While rel <= rtol*(1-2^-20), (c) implies (a):
// ad <= rel*|r| <= RN(rtol*|r|) <= tol ("lean").  Beyond that the same loop runs with rel
// clamped to that bound, and only threads for which it fails compare element by element.
//
// Instantiations (MODE, below).  SHARP = false is the filter above with a second look for threads whose
// (c) fails.  SHARP = true applies the second look's sharper test to every element in the main
// loop (two dependent fused multiply-adds instead of one): a quarter more instructions per
// step, but no second looks.  It pays when many elements have a quotient that was rounded DOWN
// to the running maximum (one-ulp differences everywhere whose largest quotient is inexact):
// the plain kernel then takes a second look on nearly every step.  The plain kernel counts its
// fruitless second looks per candidate (they travel in the accumulator's spare word); the lead
// kernels of the following calls add them up and publish their share of all warp steps to the
// host, which picks the instantiation from it.  The records do not depend on the choice.
//
// MODE 0: plain, 1: sharp, 2: plain, launched as a programmatic dependent of the lead kernel
// (its CTAs are set up while the lead kernel still runs, and wait for it below), 3: "by
// definition": the plain loop while a candidate is lean, and beyond the lean bound a loop that
// tests every element against its own tolerance and the real running maximum, so that elements
// that pass by atol alone (candidates that differ from the reference by absolute noise, where
// the reference has values near zero) do not send their thread to a second look every step.
// The plain instantiations count such fruitless looks beside the lean ones; the host picks 3
// from that report the way it picks 1.  Mode 3 waits for the lead kernel like mode 2.
template <int DT, int MODE>
__global__ void __maxnreg__(72) screen_stream_kernel(const StreamParams p) {
  constexpr bool SHARP = MODE == 1;
  constexpr bool BYDEF = MODE == 3;
  constexpr bool PLAIN = MODE == 0 || MODE == 2;
  using E = Elem<DT>;
  constexpr int VEC = E::kVec;
  constexpr int NV = kEPT / VEC;
  constexpr uint32_t TILE_BYTES = kTile * E::kBytes;
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
    q += 4 * (size_t)kMaxKC * 8;
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
    s.cnt[3 * kMaxKC + i] = 0ull;
    s.key[i] = 0ull;
    s.rel[i] = 0u;
    s.xg[i] = make_uint4(0u, 0u, 0u, 0u);
  }
  for (int i = tid; i < kMaxKC * kWarps; i += kStreamThreads) s.thr2[i] = make_float2(-1.0f, 0.0f);
  __syncthreads();
  // everything the lead kernel wrote (pointer table, seeds, zeroed counters) is read below
  if constexpr (MODE == 2 || MODE == 3) asm volatile("griddepcontrol.wait;" ::: "memory");

  // Work items (chunk, tile), chunk-major, are drawn from a global counter: a CTA gets
  // ascending items (so ascending tiles inside a chunk, which the index tie-break needs),
  // the CTAs that run together work on neighbouring tiles, and the tail is one item long.
  const uint32_t K_eff = p.K_dev ? min(*p.K_dev, p.K) : p.K;
  const uint32_t nchunks_eff = (K_eff + p.KC - 1) / p.KC;
  const unsigned long long nitems = (unsigned long long)nchunks_eff * p.ntiles;
  constexpr unsigned long long kNoItem = ~0ull;

  if (warp == kWarps) {
    // ------------------------------ producer ------------------------------
    // (ring_producer of kb_ring.cuh with TileItemMap written in: this kernel's consumer loop is
    // compiled measurably slower when the producer branch is the shared routine)
    const uint64_t pol_first = l2_policy_evict_first();
    const uint64_t pol_last = l2_policy_evict_last();
    uint32_t stage = 0, phase = 0;   // phase of the ring pass being filled
    unsigned long long issued = 0;
    bool ok = true;
    int cur_chunk = -1;
    unsigned long long next_item = 0ull;
    if (lane == 0) next_item = atomicAdd(p.sched, 1ull);
    for (;;) {
      const unsigned long long item = __shfl_sync(0xFFFFFFFFu, next_item, 0);
      if (item >= nitems) break;
      if (lane == 0) next_item = atomicAdd(p.sched, 1ull);   // drawn one item ahead: latency hidden
      const uint32_t chunk = (uint32_t)(item / p.ntiles);
      const uint32_t slot = p.slot0 + (uint32_t)(item % p.ntiles);
      const uint32_t k0 = chunk * p.KC;
      const int kc = (int)min(p.KC, K_eff - k0);
      if ((int)chunk != cur_chunk) {
        // the chunk's candidate pointers go to shared memory once (whole warp)
        cur_chunk = (int)chunk;
        __syncwarp();
        for (int i = lane; i < kc; i += 32) s.ptrs[i] = p.cands[k0 + i];
        __syncwarp();
      }
      if (lane == 0) {
        const uint32_t tile = p.tile_list ? p.tile_list[slot] : slot;
        const size_t off = (size_t)tile * TILE_BYTES;
        for (int kk = -1; kk < kc; ++kk) {
          if (!mbar_wait_bounded(&s.empty[stage], phase ^ 1u, s.abort_flag, p.status)) {
            ok = false;
            break;
          }
          // (chunk, position in the visit order), visible to the consumers with the phase
          if (kk < 0) s.item_id[stage] = ((unsigned long long)chunk << 32) | (unsigned long long)(slot - p.slot0);
          const unsigned char* src =
              reinterpret_cast<const unsigned char*>(kk < 0 ? p.ref : s.ptrs[kk]) + off;
          mbar_arrive_expect_tx(&s.full[stage], TILE_BYTES);
          bulk_g2s(s.buf + (size_t)stage * TILE_BYTES, src, TILE_BYTES, &s.full[stage],
                   (kk < 0 && p.nchunks > 1) ? pol_last : pol_first);
          ++issued;
          if (++stage == stages) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
      ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
      if (!ok) break;
    }
    if (lane == 0 && ok) {
      // no more work: an empty stage that carries the end marker
      if (mbar_wait_bounded(&s.empty[stage], phase ^ 1u, s.abort_flag, p.status)) {
        s.item_id[stage] = kNoItem;
        mbar_arrive(&s.full[stage]);
      } else {
        ok = false;
      }
    }
    if (lane == 0 && !ok) {
      // Gave up: let every copy already issued land before the CTA may exit.
      const unsigned long long back = issued < stages ? issued : stages;
      for (unsigned long long m = issued - back; m < issued; ++m) {
        uint64_t* bar = &s.full[m % stages];
        const uint32_t par = (uint32_t)((m / stages) & 1ull);
        const unsigned long long t0 = global_ns();
        while (!mbar_try_wait(bar, par)) {
          if (global_ns() - t0 > 1000000000ull) break;
        }
      }
    }
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
        if (PLAIN && (v = s.cnt[3 * kMaxKC + i]) != 0ull) atomicAdd(&a->spare, v);
        s.cnt[3 * kMaxKC + i] = 0ull;
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
      if (!mbar_wait_bounded(&s.full[stage], phase, s.abort_flag, p.status)) {
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

      // ---- reference tile: 16 elements per thread stay in registers ----
      float r[kEPT];
      bool extreme = false;   // 0 < |r| < 2^-100: the fused multiply-add of the filter could
                              // underflow to zero and lose its sign; such threads go exact
      float rlim = 0.0f;      // (by definition only: extreme in a step iff 0 < rel_f < rlim)
      {
        const uint4* src = reinterpret_cast<const uint4*>(s.buf + (size_t)stage * TILE_BYTES);
        uint4 w[NV];
#pragma unroll
        for (int j = 0; j < NV; ++j) w[j] = src[tid + kConsumers * j];
        __syncwarp();
        if (lane == 0) mbar_arrive(&s.empty[stage]);
        if (++stage == stages) {
          stage = 0;
          phase ^= 1u;
        }
#pragma unroll
        for (int j = 0; j < NV; ++j) E::decode(w[j], &r[j * VEC]);
        // (binary16 and e5m2 have no value in (0, 2^-100): their smallest are 2^-24 and 2^-16)
        if constexpr (DT != KB_F16 && DT != KB_F8E5M2) {
          if constexpr (BYDEF) {
            // By definition: the same danger, judged per step.  The fused multiply-add can only
            // mislead if rel_f*|r| < 2^-125 (see above), so with the thread's smallest non-zero
            // magnitude m the thread is extreme in a step iff 0 < rel_f < 2^-124/m.  Outputs
            // with long tails of tiny values (a softmax over widely spread logits) then leave
            // the filter only while the running maximum is still tiny itself.
            unsigned int umin = 0xFFFFFFFFu;
#pragma unroll
            for (int e = 0; e < kEPT; ++e) umin = min(umin, (__float_as_uint(r[e]) & 0x7FFFFFFFu) - 1u);
            if (umin < 0x0D800000u - 1u) rlim = __fdiv_ru(4.70197740328915e-38f, __uint_as_float(umin + 1u));
          } else {
#pragma unroll
            for (int e = 0; e < kEPT; ++e)   // 0 < |r| < 2^-100 on the bit pattern (zero wraps to the top)
              extreme |= ((__float_as_uint(r[e]) & 0x7FFFFFFFu) - 1u) < (0x0D800000u - 1u);
          }
        }
      }
      if (first_of_chunk) exchange_apply(tile_base);

      // ---- the candidates of this chunk against the tile in registers ----
      for (int kk = 0; kk < cur_kc; ++kk) {
        const unsigned long long trw =
            *reinterpret_cast<volatile unsigned long long*>(&s.thr2[kk * kWarps + warp]);
        const float th = __uint_as_float((unsigned int)trw);
        const float rel = __uint_as_float((unsigned int)(trw >> 32));
        if (!mbar_wait_bounded(&s.full[stage], phase, s.abort_flag, p.status)) {
          ok = false;
          break;
        }
        const uint4* src = reinterpret_cast<const uint4*>(s.buf + (size_t)stage * TILE_BYTES);
        uint4 w[NV];
#pragma unroll
        for (int j = 0; j < NV; ++j) w[j] = src[tid + kConsumers * j];
        __syncwarp();
        if (lane == 0) mbar_arrive(&s.empty[stage]);
        if (++stage == stages) {
          stage = 0;
          phase ^= 1u;
        }
        const unsigned int* words = reinterpret_cast<const unsigned int*>(w);

        // One loop for every case: (b) on the largest error, (c) with rel_f = min(rel, rtol_lean).
        //   rel <= rtol_lean ("lean"): rel_f = rel; (c) implies (a).
        //   rel  > rtol_lean: (c) with the smaller rel_f still implies both (a) and the real (c)
        //     (a thread for which it fails holds an element whose relative error exceeds rtol: a
        //     mismatch, or one that passes by atol).
        //   no lean bound (rtol < 2^-20): rel_f = rel, and (a) is pre-tested per thread on the
        //     largest error against atol alone.
        const bool has_lean = p.rtol_lean >= 0.0f;
        const bool lean = rel <= p.rtol_lean;
        const float rel_f = (has_lean && !lean) ? p.rtol_lean : rel;
        const bool ext = BYDEF ? (rel_f > 0.0f && rel_f < rlim) : extreme;
        float mabs = 0.0f, mrel = 0.0f;
        // g = (ulp(rel)/2)*(1 - 2^-20), or 0 where that would be subnormal
        auto half_ulp_of_rel = [&]() -> float {
          const unsigned int rb = __float_as_uint(rel);
          return rb >= (30u << 23)
                     ? __uint_as_float((rb & 0x7F800000u) - (24u << 23)) * 0.99999904632568359375f
                     : 0.0f;
        };
        const bool sharp = SHARP && lean;
        float mtol = -kInf;   // (by definition only) largest |d| - rtol_lean*|r| of the thread
        if (BYDEF && has_lean && !lean) {
          // Beyond the lean bound: no quotient above the REAL running maximum (t <= 0 as in the
          // lean form) and every element within tolerance by a sufficient test,
          //   RN(|d| - rtol_lean*|r|) <= atol*(1 - 2^-20)   =>   |d| <= RN(atol + RN(rtol*|r|)):
          // the left side is one fused multiply-add, so |d| <= atol_d*(1 + 2^-24) + rtol_lean*|r|
          // <= (atol + rtol*|r|)*(1 - 2^-21), below the definition's twice-rounded tolerance
          // (rtol_lean*|r| >= 2^-124 is normal for every non-zero |r| of a thread that is not
          // extreme in this step; |r| = 0 leaves |d| <= atol_d).  NaN and Inf differences make it NaN or
          // Inf.  An element within 2^-20 of its tolerance is flagged and settled by the second look.
#pragma unroll
          for (int e = 0; e < kEPT; e += 2) {
            float d0, d1;
            E::pair_diff(words, e, r[e], r[e + 1], d0, d1);
            const float ar0 = fabsf(r[e]), ar1 = fabsf(r[e + 1]);
            const float u0 = fmaf(-p.rtol_lean, ar0, fabsf(d0)), u1 = fmaf(-p.rtol_lean, ar1, fabsf(d1));
            const float t0 = fmaf(-rel, ar0, fabsf(d0)), t1 = fmaf(-rel, ar1, fabsf(d1));
            mabs = max3(mabs, fabsf(d0), fabsf(d1));
            mtol = max3_nan(mtol, u0, u1);
            mrel = max3_nan(mrel, t0, t1);
          }
          // (folded into the relative test's flag: positive, or NaN, when some element may be out of tolerance)
          mrel = max2_nan(mrel, __fsub_rn(mtol, p.atol * 0.99999904632568359375f));
        } else if (!SHARP || !sharp) {
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
        // (by definition: an extreme thread takes the second look, which tests its tiny elements
        // with both operands scaled by 2^64 so that the fused multiply-add cannot underflow.  A
        // tiny element whose quotient is fine also matches, given atol >= 2^-124: its error is
        // at most rel_f*|r| < 2^-124.  Without such an atol the thread goes exact as elsewhere.)
        const bool ext_look = BYDEF && ext && p.atol >= 4.70197740328915e-38f;
        const bool bad = !(mrel <= 0.0f) || (!has_lean && mabs > p.atol) || ext_look;
        bool trig = (mabs > th) || (ext && !ext_look);
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
          bool again = sharp || (!BYDEF && !(mrel <= mabs * 9.5367431640625e-07f));
          if (!again) {
#pragma unroll
          for (int e = 0; e < kEPT; e += 2) {
            float d0, d1;
            E::pair_diff(words, e, r[e], r[e + 1], d0, d1);
            float ar0 = fabsf(r[e]), ar1 = fabsf(r[e + 1]);
            float a0 = fabsf(d0), a1 = fabsf(d1);
            if constexpr (BYDEF) {   // magnitudes below 2^-64 and their errors times 2^64 (exact)
              const float s0 = (ar0 > 0.0f && ar0 < 5.421010862427522e-20f) ? 18446744073709551616.0f : 1.0f;
              const float s1 = (ar1 > 0.0f && ar1 < 5.421010862427522e-20f) ? 18446744073709551616.0f : 1.0f;
              ar0 *= s0, a0 *= s0, ar1 *= s1, a1 *= s1;
            }
            const float t0 = fmaf(-rel, ar0, a0), t1 = fmaf(-rel, ar1, a1);
            // (a NaN or Inf difference makes t NaN or Inf: neither clause holds)
            // (by definition only: a zero reference has no quotient, its element only has to be
            // within atol.  In the other instantiations such an element goes to the exact path;
            // the clause is kept out of them because it changes how the compiler lays out their
            // main loop.)
            const bool c0 = (t0 <= 0.0f) || (t0 >= 7.888609052e-31f && fmaf(-g, ar0, t0) <= 0.0f) ||
                            (BYDEF && ar0 == 0.0f && a0 <= p.atol);
            const bool c1 = (t1 <= 0.0f) || (t1 >= 7.888609052e-31f && fmaf(-g, ar1, t1) <= 0.0f) ||
                            (BYDEF && ar1 == 0.0f && a1 <= p.atol);
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
            // (by definition only: a zero reference has no quotient; magnitudes below 2^-64 and
            // their errors are scaled by 2^64, which is exact, so that the product cannot underflow)
            if constexpr (BYDEF) {
              const float q0 = fabsf(r[e]), q1 = fabsf(r[e + 1]);
              const float s0 = q0 < 5.421010862427522e-20f ? 18446744073709551616.0f : 1.0f;
              const float s1 = q1 < 5.421010862427522e-20f ? 18446744073709551616.0f : 1.0f;
              again |= (q0 > 0.0f && !(fmaf(-rel, q0 * s0, a0 * s0) <= 0.0f)) ||
                       (q1 > 0.0f && !(fmaf(-rel, q1 * s1, a1 * s1) <= 0.0f));
            } else {
              again |= !(fmaf(-rel, fabsf(r[e]), a0) <= 0.0f) || !(fmaf(-rel, fabsf(r[e + 1]), a1) <= 0.0f);
            }
            mis_fast += ((a0 > tol0) && f0) ? 1u : 0u;   // (c == r would give a0 = 0 <= tol0)
            mis_fast += ((a1 > tol1) && f1) ? 1u : 0u;
          }
          trig = trig || again;
        }
        if (!__any_sync(0xFFFFFFFFu, trig)) {
          const unsigned int tot = warp_add_u32(mis_fast);
          if (lane == 0 && tot) atomicAdd(&s.cnt[kk], (unsigned long long)tot);
          // (some lane was `bad`, or the step would have ended above: while lean that lane took
          // a second look, and it found nothing)
          // (32-bit add on the low word of the 64-bit slot; flush() moves it to the accumulator)
          // (low word: looks taken while lean; high word: looks beyond the lean bound that found
          // no mismatch either, i.e. the thread's elements pass by atol)
          if (PLAIN && lane == 0 && (lean || tot == 0u))
            atomicAdd(reinterpret_cast<unsigned int*>(&s.cnt[3 * kMaxKC + kk]) + (lean ? 0 : 1), 1u);
          continue;
        }

        // ---- exact path.  A triggered thread finds its largest finite error (first
        // index on ties) with a running compare, and evaluates by the definition the
        // elements that fail the tolerance / relative-error filter or are not finite. ----
        unsigned int n_mis = 0, n_nan = 0, n_inf = 0, qb = 0u;
        unsigned long long best = 0ull;
        if (trig) {
          float c[kEPT];
#pragma unroll
          for (int j = 0; j < NV; ++j) E::decode(w[j], &c[j * VEC]);
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
            // (by definition: only the elements the danger is about, rel_f*|r| < 2^-124, are
            // evaluated unconditionally; the thread's other elements have a reliable t)
            const bool ext_e = BYDEF ? (ext && ar * rel_f < 4.70197740328915e-38f) : ext;
            bool hot = !(t <= 0.0f) || !fin || ext_e;
            if (!lean) hot = hot || !(ad <= __fadd_rn(p.atol, __fmul_rn(p.rtol, ar)));
            if (hot) {
              const float tol = __fadd_rn(p.atol, __fmul_rn(p.rtol, ar));
              const bool match = (c[e] == r[e]) || (fin && ad <= tol);
              n_mis += match ? 0u : 1u;
              n_nan += (c[e] != c[e]) ? 1u : 0u;
              n_inf += (fabsf(c[e]) == kInf) ? 1u : 0u;
              if (fin && ar > 0.0f && ar <= kFltMax && (ext_e || t > 0.0f)) {
                const unsigned int q = __float_as_uint(__fdiv_rn(ad, ar));
                qb = q > qb ? q : qb;
              }
            }
          }
          if (m > th) {
            const unsigned long long idx =
                tile_base + (unsigned long long)((tid + kConsumers * (mi / VEC)) * VEC + (mi % VEC));
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
          } else if (PLAIN && best == 0ull && (n_mis | n_nan | n_inf) == 0u) {
            // an exact path that changed nothing (typically a zero reference under a non-zero
            // candidate within atol, which has no quotient): reported with the fruitless looks
            // beyond the lean bound, since the by-definition instantiation settles those earlier
            atomicAdd(reinterpret_cast<unsigned int*>(&s.cnt[3 * kMaxKC + kk]) + 1, 1u);
          }
        }
        __syncwarp();
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

// ---------------------------------------------------------------------------
// Plain-load kernels: every selected element classified by the definition.
// ---------------------------------------------------------------------------
struct ExactAcc {
  unsigned int n_mis = 0, n_nan = 0, n_inf = 0, qb = 0;
  unsigned long long best = 0ull;

  __device__ __forceinline__ void add(float r, float c, unsigned long long i, float atol, float rtol) {
    const float ad = fabsf(__fsub_rn(c, r));
    const float tolc = tol_clamped(r, atol, rtol);
    const bool match = (c == r) || (ad <= tolc);
    n_mis += match ? 0u : 1u;
    n_nan += (c != c) ? 1u : 0u;
    n_inf += (fabsf(c) == __uint_as_float(0x7F800000u)) ? 1u : 0u;
    if (is_finite_nonneg(ad)) {
      const unsigned long long kv = pack_key(ad, i);
      best = kv > best ? kv : best;
      const float ar = fabsf(r);
      if (ar > 0.0f && is_finite_nonneg(ar)) {
        const unsigned int q = __float_as_uint(__fdiv_rn(ad, ar));
        qb = q > qb ? q : qb;
      }
    }
  }
  // warp-level merge, then one set of atomics per warp (a warp sees < 2^32 elements)
  __device__ __forceinline__ void commit(Acc* a) {
    n_mis = warp_add_u32(n_mis);
    n_nan = warp_add_u32(n_nan);
    n_inf = warp_add_u32(n_inf);
    best = warp_max_u64(best);
    qb = warp_max_u32(qb);
    if ((threadIdx.x & 31) == 0) {
      if (n_mis) atomicAdd(&a->mism, (unsigned long long)n_mis);
      if (n_nan) atomicAdd(&a->nan, (unsigned long long)n_nan);
      if (n_inf) atomicAdd(&a->inf, (unsigned long long)n_inf);
      if (best) atomicMax(&a->key, best);
      if (qb) atomicMax(&a->rel, qb);
    }
  }
};

// Elements [e0, e1) of every candidate under an arbitrary mask.  grid = (blocks, K).
// Used for the ragged tail and for masks finer than a kernel tile.
template <int DT>
__global__ void __launch_bounds__(256) screen_generic_kernel(const void* __restrict__ ref,
                                                             const void* const* __restrict__ cands,
                                                             Acc* __restrict__ acc,
                                                             unsigned long long e0,
                                                             unsigned long long e1, float atol,
                                                             float rtol, MaskDev mask,
                                                             const unsigned int* __restrict__ count) {
  using E = Elem<DT>;
  const unsigned int k = blockIdx.y;
  if (count && k >= *count) return;
  const void* cand = cands[k];
  ExactAcc x;
  const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
  for (unsigned long long i = e0 + (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < e1;
       i += stride) {
    if (!mask_selected(mask, i)) continue;
    x.add(E::load(ref, i), E::load(cand, i), i, atol, rtol);
  }
  x.commit(&acc[k]);
}

// Lead kernel: (1) the first `nscout` full tiles (of the list, or tiles 0..nscout-1) of every
// candidate, classified exactly before the streaming kernel starts: their maxima seed the
// streaming kernel's thresholds, so that its first tile does not have to discover them;
// (2) the ragged tail [tail0, N) past the last full tile, under the mask; (3) housekeeping by
// the blocks with blockIdx.x == 0: candidate k's pointer goes from the kernel's arguments to
// the device table the streaming kernel reads (when `from_args`), and the accumulators and
// counters of the OTHER set -- the one the next call will work on -- are zeroed (nobody else
// touches them during this call).  A block takes per_block elements of one candidate (1024,
// or a whole kernel tile when there are many candidates) and issues one set of atomics.
// grid = (max(1, nscout * (4096 / per_block) + ceil((N - tail0) / per_block)), K).
constexpr unsigned int kScoutPerBlock = 1024;
// four consecutive elements starting at element i (i a multiple of 4, p 16-byte aligned)
template <int DT>
__device__ __forceinline__ void load4(const void* p, unsigned long long i, float* out) {
  using E = Elem<DT>;
  uint4 w = make_uint4(0u, 0u, 0u, 0u);
  const char* at = reinterpret_cast<const char*>(p) + i * E::kBytes;
  if (E::kBytes == 4) {
    w = *reinterpret_cast<const uint4*>(at);
  } else if (E::kBytes == 2) {
    const uint2 v = *reinterpret_cast<const uint2*>(at);
    w.x = v.x;
    w.y = v.y;
  } else {
    w.x = *reinterpret_cast<const unsigned int*>(at);
  }
  float o[E::kVec];
  E::decode(w, o);
#pragma unroll
  for (int j = 0; j < 4; ++j) out[j] = o[j];
}
struct LeadParams {
  const void* ref;
  const void** table;           // device pointer table [K]
  Acc* acc;                     // this call's accumulators (zero on entry)
  Acc* acc_next;                // the other set: entries [0, n_clear) are zeroed here
  unsigned int* counters_next;  // the other set's ticket and work counters (3 words)
  const uint32_t* tile_list;
  unsigned int nscout, n_clear, from_args;
  unsigned long long tail0, N;
  float atol, rtol;
  MaskDev mask;
  const unsigned int* count;
  // Fruitless second looks of earlier plain streaming launches, on their way to the host: the
  // spare words of the accumulators cleared here (the previous call's) are added to looks_sum;
  // looks_pub, which the previous lead kernel filled the same way (the call before that), is
  // published as 64 * looks / pub_steps (capped at 64) in host-visible memory (if that call had a
  // plain streaming launch: pub_steps > 0) and reset.
  unsigned long long* looks_sum;
  unsigned long long* looks_pub;
  unsigned int* hint;
  float pub_steps;
  unsigned int per_block;       // elements one block classifies: kScoutPerBlock or kTile
};
template <int DT>
__global__ void __launch_bounds__(256) screen_lead_kernel(const LeadParams p, const __grid_constant__ PtrChunk chunk_ptrs) {
  using E = Elem<DT>;
  // elements per block: kScoutPerBlock, or a whole kernel tile when the call has so many
  // candidates that the smaller blocks would queue up in many waves
  const unsigned int per_block = p.per_block;
  const unsigned int kBlocksPerTile = kTile / per_block;
  const unsigned int k = blockIdx.y;
  // a streaming kernel launched as a programmatic dependent may be set up from here on (it
  // waits for this grid to finish before it reads anything); no effect otherwise
  asm volatile("griddepcontrol.launch_dependents;");
  if (blockIdx.x == 0) {
    if (threadIdx.x == 0 && p.from_args) p.table[k] = chunk_ptrs.p[k];
    unsigned long long looks = 0ull;
    for (unsigned int j = k + gridDim.y * threadIdx.x; j < p.n_clear; j += gridDim.y * 256u) {
      looks += p.acc_next[j].spare;
      clear_acc(&p.acc_next[j]);
    }
    if (looks && p.looks_sum) atomicAdd(p.looks_sum, looks);
    if (k == 0 && threadIdx.x < 3) p.counters_next[threadIdx.x] = 0u;
    if (k == 0 && threadIdx.x == 32 && p.hint) {
      // (only plain launches report: the word keeps the last report until the host takes it)
      if (p.pub_steps > 0.0f) {
        // byte 0: looks taken while lean, byte 1: fruitless looks beyond the lean bound, each as
        // 64ths of the call's warp steps
        const unsigned long long looks = *p.looks_pub;
        const unsigned int lean_share = (unsigned int)fminf(64.0f * (float)(looks & 0xFFFFFFFFull) / p.pub_steps, 64.0f);
        const unsigned int atol_share = (unsigned int)fminf(64.0f * (float)(looks >> 32) / p.pub_steps, 64.0f);
        *reinterpret_cast<volatile unsigned int*>(p.hint) = lean_share | (atol_share << 8);
      }
      *p.looks_pub = 0ull;
    }
  }
  if (p.count && k >= *p.count) return;
  __shared__ unsigned int s_cnt[3];
  __shared__ unsigned int s_rel;
  __shared__ unsigned long long s_key;
  if (threadIdx.x == 0) {
    s_cnt[0] = s_cnt[1] = s_cnt[2] = 0u;
    s_rel = 0u;
    s_key = 0ull;
  }
  __syncthreads();
  const void* cand = p.from_args ? chunk_ptrs.p[k] : p.table[k];
  ExactAcc x;
  if (blockIdx.x < p.nscout * kBlocksPerTile) {
    const unsigned int slot = blockIdx.x / kBlocksPerTile;
    const unsigned long long tile = p.tile_list ? p.tile_list[slot] : slot;
    const unsigned long long base = tile * kTile + (blockIdx.x % kBlocksPerTile) * per_block;
    // four consecutive elements per thread and step (one vector load each from the reference
    // and the candidate); the running maxima stay plain floats, and the quotient is only
    // formed where it can exceed the thread's largest so far
    float bad = -1.0f, qf = 0.0f;
    unsigned int bi = 0u;
    for (unsigned int j0 = 0; j0 < per_block / 1024; ++j0) {
      const unsigned long long i0 = base + ((unsigned long long)j0 * 256 + threadIdx.x) * 4;
      float rv[4], cv[4];
      load4<DT>(p.ref, i0, rv);
      load4<DT>(cand, i0, cv);
#pragma unroll
      for (unsigned int j = 0; j < 4; ++j) {
        const float r = rv[j], c = cv[j];
        const float ad = fabsf(__fsub_rn(c, r));
        const bool match = (c == r) || (ad <= tol_clamped(r, p.atol, p.rtol));
        x.n_mis += match ? 0u : 1u;
        x.n_nan += (c != c) ? 1u : 0u;
        x.n_inf += (fabsf(c) == __uint_as_float(0x7F800000u)) ? 1u : 0u;
        if (is_finite_nonneg(ad)) {
          if (ad > bad) {          // indices rise within a thread: the first of equal maxima stays
            bad = ad;
            bi = (unsigned int)(i0 + j);
          }
          const float ar = fabsf(r);
          // RD(qf * ar) >= ad  =>  ad / ar <= qf  =>  RN(ad / ar) <= qf: nothing to gain
          if (ar > 0.0f && is_finite_nonneg(ar) && !(__fmul_rd(qf, ar) >= ad))
            qf = fmaxf(qf, __fdiv_rn(ad, ar));
        }
      }
    }
    if (bad >= 0.0f) x.best = pack_key(bad, bi);
    x.qb = __float_as_uint(qf);
  } else {
    const unsigned long long base =
        p.tail0 + (unsigned long long)(blockIdx.x - p.nscout * kBlocksPerTile) * per_block;
    for (unsigned int j = 0; j < per_block / 256; ++j) {
      const unsigned long long i = base + j * 256 + threadIdx.x;
      if (i < p.N && mask_selected(p.mask, i)) x.add(E::load(p.ref, i), E::load(cand, i), i, p.atol, p.rtol);
    }
  }
  // block-level merge in shared memory, then one set of global atomics
  x.n_mis = warp_add_u32(x.n_mis);
  x.n_nan = warp_add_u32(x.n_nan);
  x.n_inf = warp_add_u32(x.n_inf);
  x.best = warp_max_u64(x.best);
  x.qb = warp_max_u32(x.qb);
  if ((threadIdx.x & 31) == 0) {
    if (x.n_mis) atomicAdd(&s_cnt[0], x.n_mis);
    if (x.n_nan) atomicAdd(&s_cnt[1], x.n_nan);
    if (x.n_inf) atomicAdd(&s_cnt[2], x.n_inf);
    if (x.best) atomicMax(&s_key, x.best);
    if (x.qb) atomicMax(&s_rel, x.qb);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    Acc* a = &p.acc[k];
    if (s_cnt[0]) atomicAdd(&a->mism, (unsigned long long)s_cnt[0]);
    if (s_cnt[1]) atomicAdd(&a->nan, (unsigned long long)s_cnt[1]);
    if (s_cnt[2]) atomicAdd(&a->inf, (unsigned long long)s_cnt[2]);
    if (s_key) atomicMax(&a->key, s_key);
    if (s_rel) atomicMax(&a->rel, s_rel);
  }
}

// ---------------------------------------------------------------------------
// Small problems (the latency-bound regime: a few candidates of at most a few hundred
// thousand elements, e.g. 21 candidates of a 2048-element mat-vec output): ONE launch.
// Candidate pointers travel as kernel arguments; block (bx, k) classifies 1024 elements
// exactly and writes a partial record; the last block of candidate k to finish (a
// self-resetting ticket per candidate) merges the partials and writes the result.
// Nothing has to be zeroed beforehand and no atomics touch the accumulators.
// ---------------------------------------------------------------------------
constexpr unsigned int kSmallPerBlock = 1024;
struct SmallParams {
  const void* ref;
  Acc* partials;            // [K][nb]
  unsigned int* tickets;    // [K], zero between launches
  kb_screen_result* out;    // [K]
  unsigned long long N;
  unsigned int nb;
  float atol, rtol;
  MaskDev mask;
};

// One block's share of a small problem: classify elements [base, base+4096) of one candidate
// exactly, store the partial record, and -- if this block is the candidate's last to finish --
// merge the nb partials and write the candidate's result.
template <int DT>
__device__ __forceinline__ void small_block(const void* ref, const void* cand, unsigned long long N,
                                            unsigned long long base, const MaskDev& mask, float atol,
                                            float rtol, Acc* partials /*[nb] of this candidate*/,
                                            unsigned int bx, unsigned int nb, unsigned int* ticket,
                                            kb_screen_result* out) {
  using E = Elem<DT>;
  __shared__ unsigned int s_cnt[3];
  __shared__ unsigned int s_rel;
  __shared__ unsigned long long s_key;
  __shared__ unsigned int s_ticket;
  if (threadIdx.x == 0) {
    s_cnt[0] = s_cnt[1] = s_cnt[2] = 0u;
    s_rel = 0u;
    s_key = 0ull;
  }
  __syncthreads();
  ExactAcc x;
  {
    // all loads first (one round trip to memory instead of one per unrolled group), then the
    // arithmetic
    constexpr unsigned int kPer = kSmallPerBlock / 256;
    float rv[kPer], cv[kPer];
    unsigned int sel = 0u;
#pragma unroll
    for (unsigned int j = 0; j < kPer; ++j) {
      const unsigned long long i = base + j * 256 + threadIdx.x;
      const bool on = i < N && mask_selected(mask, i);
      sel |= on ? (1u << j) : 0u;
      rv[j] = on ? E::load(ref, i) : 0.0f;
      cv[j] = on ? E::load(cand, i) : 0.0f;
    }
#pragma unroll
    for (unsigned int j = 0; j < kPer; ++j)
      if (sel & (1u << j)) x.add(rv[j], cv[j], base + j * 256 + threadIdx.x, atol, rtol);
  }
  x.n_mis = warp_add_u32(x.n_mis);
  x.n_nan = warp_add_u32(x.n_nan);
  x.n_inf = warp_add_u32(x.n_inf);
  x.best = warp_max_u64(x.best);
  x.qb = warp_max_u32(x.qb);
  if ((threadIdx.x & 31) == 0) {
    if (x.n_mis) atomicAdd(&s_cnt[0], x.n_mis);
    if (x.n_nan) atomicAdd(&s_cnt[1], x.n_nan);
    if (x.n_inf) atomicAdd(&s_cnt[2], x.n_inf);
    if (x.best) atomicMax(&s_key, x.best);
    if (x.qb) atomicMax(&s_rel, x.qb);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    Acc a;
    a.mism = s_cnt[0];
    a.nan = s_cnt[1];
    a.inf = s_cnt[2];
    a.key = s_key;
    a.rel = s_rel;
    a.pad = 0u;
    a.spare = 0ull;
    partials[bx] = a;
    __threadfence();
    s_ticket = atomicAdd(ticket, 1u);
  }
  __syncthreads();
  if (s_ticket != nb - 1) return;
  // last block of this candidate: merge the partial records (warp 0 is enough)
  __threadfence();
  if (threadIdx.x < 32) {
    unsigned long long mism = 0ull, nan = 0ull, inf = 0ull, key = 0ull;
    unsigned int rel = 0u;
    for (unsigned int b = threadIdx.x; b < nb; b += 32) {
      const Acc* q = &partials[b];
      mism += __ldcg(&q->mism);
      nan += __ldcg(&q->nan);
      inf += __ldcg(&q->inf);
      const unsigned long long kv = __ldcg(&q->key);
      key = kv > key ? kv : key;
      const unsigned int rv = __ldcg(&q->rel);
      rel = rv > rel ? rv : rel;
    }
    // each partial count is <= 1024 and nb <= 8192: the 32-bit adds below cannot overflow
    const unsigned long long tm = warp_add_u32((unsigned int)mism);
    const unsigned long long tn = warp_add_u32((unsigned int)nan);
    const unsigned long long ti = warp_add_u32((unsigned int)inf);
    key = warp_max_u64(key);
    rel = warp_max_u32(rel);
    if (threadIdx.x == 0) {
      Acc a;
      a.mism = tm;
      a.nan = tn;
      a.inf = ti;
      a.key = key;
      a.rel = rel;
      a.pad = 0u;
      a.spare = 0ull;
      unpack_record(a, out);
      *ticket = 0u;   // ready for the next launch
    }
  }
}

template <int DT>
__global__ void __launch_bounds__(256) screen_small_kernel(const SmallParams p, const PtrChunk cands) {
  // Launched as a programmatic dependent of whatever precedes it in the stream (back-to-back
  // calls: the next launch is set up while this one runs): let the next one be scheduled, then
  // wait until the previous grid has finished and its writes are visible.  No effect when the
  // launch carries no such attribute.
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const unsigned int k = blockIdx.y;
  small_block<DT>(p.ref, cands.p[k], p.N, (unsigned long long)blockIdx.x * kSmallPerBlock, p.mask,
                  p.atol, p.rtol, p.partials + (size_t)k * p.nb, blockIdx.x, p.nb, &p.tickets[k],
                  &p.out[k]);
}

// Several (reference, candidates) groups of different sizes in ONE launch (the paper's
// fidelity includes the set of input shapes, Sec. 3.2): every candidate of every group is a
// "row"; blocks are numbered row-major over the rows' 4096-element blocks.  Everything the
// kernel needs travels as kernel arguments.
constexpr int kMultiMaxGroups = 64;
constexpr int kMultiMaxRows = 1024;
struct MultiParams {
  const void* ref[kMultiMaxGroups];
  unsigned long long N[kMultiMaxGroups];
  const void* cand[kMultiMaxRows];
  unsigned int first_block[kMultiMaxRows + 1];   // prefix sums of the rows' block counts
  unsigned char group[kMultiMaxRows];
  Acc* partials;
  unsigned int* tickets;
  kb_screen_result* out;
  unsigned int rows;
  float atol, rtol;
};

template <int DT>
__global__ void __launch_bounds__(256) screen_multi_kernel(const __grid_constant__ MultiParams p) {
  // row of this block: the last row whose first block is <= blockIdx.x
  unsigned int lo = 0, hi = p.rows;
  while (hi - lo > 1) {
    const unsigned int mid = (lo + hi) >> 1;
    if (p.first_block[mid] <= blockIdx.x) lo = mid; else hi = mid;
  }
  const unsigned int row = lo;
  const unsigned int g = p.group[row];
  const unsigned int bx = blockIdx.x - p.first_block[row];
  const unsigned int nb = p.first_block[row + 1] - p.first_block[row];
  MaskDev none;
  none.kind = 0;
  none.log2_tile = 0;
  none.stride = 1;
  none.phase = 0;
  none.bits = nullptr;
  small_block<DT>(p.ref[g], p.cand[row], p.N[g], (unsigned long long)bx * kSmallPerBlock, none, p.atol,
                  p.rtol, p.partials + p.first_block[row], bx, nb, &p.tickets[row], &p.out[row]);
}

__global__ void screen_finalize_kernel(const Acc* __restrict__ acc, kb_screen_result* __restrict__ out,
                                       unsigned int K, const unsigned int* __restrict__ count) {
  const unsigned int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= K) return;
  if (count && k >= *count)
    write_absent_record(&out[k]);
  else
    unpack_record(acc[k], &out[k]);
}

// Candidate pointers of a call with more than kPtrsPerLaunch candidates go to the device table.
__global__ void screen_prep_kernel(const PtrChunk chunk, const void** table, unsigned int offset,
                                   unsigned int count) {
  const unsigned int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) table[offset + i] = chunk.p[i];
}

// Indexed screening: candidate slot j holds table[index[j]] for j < *count.  Builds the
// slot pointer table on the device, zeroes accumulators and counters, and validates what
// the host cannot see: an index outside [0, K_all), a null or misaligned pointer, or a
// count above the slots makes the whole call a no-op (effective count 0) and sets the
// device status, so that no later kernel ever touches a bad address.
__global__ void screen_prep_indexed_kernel(const void* const* __restrict__ all, unsigned int K_all,
                                           const int* __restrict__ index,
                                           const unsigned int* __restrict__ count, unsigned int Kmax,
                                           const void** table, Acc* acc, unsigned int* counters,
                                           unsigned int* eff_count, unsigned int* status) {
  // single block: Kmax <= 1024 slots
  __shared__ unsigned int s_bad;
  if (threadIdx.x == 0) s_bad = 0u;
  __syncthreads();
  const unsigned int n = *count;
  if (n > Kmax && threadIdx.x == 0) s_bad = 1u;
  for (unsigned int j = threadIdx.x; j < Kmax; j += blockDim.x) {
    const void* ptr = nullptr;
    if (j < n && n <= Kmax) {
      const int ix = index[j];
      if (ix < 0 || (unsigned int)ix >= K_all) {
        atomicOr(&s_bad, 1u);
      } else {
        ptr = all[ix];
        if (!ptr || (reinterpret_cast<uintptr_t>(ptr) & 15u)) atomicOr(&s_bad, 2u);
      }
    }
    table[j] = ptr;
    Acc z;
    z.mism = z.nan = z.inf = z.spare = z.key = 0ull;
    z.rel = z.pad = 0u;
    acc[j] = z;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    counters[0] = 0u;   // ticket counter
    counters[1] = 0u;   // work counter (64 bits)
    counters[2] = 0u;
    *eff_count = s_bad ? 0u : n;   // effective number of candidates
    if (s_bad) set_status(status, (unsigned int)((s_bad & 2u) ? KB_ERR_ALIGNMENT : KB_ERR_INVALID_ARG));
  }
}

}  // namespace kb
