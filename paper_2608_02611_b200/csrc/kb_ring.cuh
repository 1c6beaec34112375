// The producer half of the streaming gates (Sec. 3.1 K(p); Sec. 3.4 Verifier: K candidate
// tensors against one reference), shared by the 32/16-bit, the e4m3 and the binary64 kernel.
//
// One warp per CTA runs it.  Work items are drawn from a global counter, one ahead of use.
// An item is a reference block followed by the same block of each candidate of a chunk; each
// block goes to the next stage of a shared-memory ring with a 1-D bulk copy that completes on
// the stage's "full" barrier, after the stage's "empty" barrier says the consumers are done
// with what it held.  The stage that takes a reference block also names the item for the
// consumers.  A stage with the end marker and no copy closes the stream.  Every wait is
// bounded; when one gives up, the abort flag releases the consumers and the producer lets the
// copies it has in flight land before the CTA may exit.
//
// What differs between the kernels is how an item number maps to (chunk, block) and where a
// block lies in a tensor: the Map argument.
//   void locate(item, chunk, k0, kc, off, id)   the item's chunk, the chunk's first candidate
//        and number of candidates, the byte offset of the item's block in every tensor, and
//        the word the consumers read to learn which item a stage starts
#pragma once

#include "kb_common.cuh"

namespace kb {

constexpr unsigned long long kNoItem = ~0ull;   // end marker in a stage's item word

struct RingProducerView {
  unsigned char* buf;                 // [stages][block_bytes]
  uint64_t* full;                     // [stages]
  uint64_t* empty;                    // [stages]
  unsigned long long* item_id;        // [stages]
  const void** ptrs;                  // candidate pointers of the current chunk
  volatile unsigned int* abort_flag;
};

template <class Map>
__device__ __forceinline__ void ring_producer(const RingProducerView s, const Map map, const int lane,
                                              const uint32_t stages, const uint32_t block_bytes,
                                              const unsigned long long nitems,
                                              unsigned long long* sched, const void* ref,
                                              const void* const* cands, const bool ref_is_reused,
                                              unsigned int* status) {
  const uint64_t pol_first = l2_policy_evict_first();
  const uint64_t pol_last = l2_policy_evict_last();
  uint32_t stage = 0, phase = 0;   // phase of the ring pass being filled
  unsigned long long issued = 0;
  bool ok = true;
  int cur_chunk = -1;
  unsigned long long next_item = 0ull;
  if (lane == 0) next_item = atomicAdd(sched, 1ull);
  for (;;) {
    const unsigned long long item = __shfl_sync(0xFFFFFFFFu, next_item, 0);
    if (item >= nitems) break;
    if (lane == 0) next_item = atomicAdd(sched, 1ull);   // drawn one item ahead: latency hidden
    uint32_t chunk, k0;
    int kc;
    size_t off;
    unsigned long long id;
    map.locate(item, chunk, k0, kc, off, id);
    if ((int)chunk != cur_chunk) {
      // the chunk's candidate pointers go to shared memory once (whole warp)
      cur_chunk = (int)chunk;
      __syncwarp();
      for (int i = lane; i < kc; i += 32) s.ptrs[i] = cands[k0 + i];
      __syncwarp();
    }
    if (lane == 0) {
      for (int kk = -1; kk < kc; ++kk) {
        if (!mbar_wait_bounded(&s.empty[stage], phase ^ 1u, s.abort_flag, status)) {
          ok = false;
          break;
        }
        // the item's name becomes visible to the consumers with the phase
        if (kk < 0) s.item_id[stage] = id;
        const unsigned char* src = reinterpret_cast<const unsigned char*>(kk < 0 ? ref : s.ptrs[kk]) + off;
        mbar_arrive_expect_tx(&s.full[stage], block_bytes);
        bulk_g2s(s.buf + (size_t)stage * block_bytes, src, block_bytes, &s.full[stage],
                 (kk < 0 && ref_is_reused) ? pol_last : pol_first);
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
    if (mbar_wait_bounded(&s.empty[stage], phase ^ 1u, s.abort_flag, status)) {
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
}

// Items of the 32/16/8-bit kernels: chunk-major over the tiles a launch visits; a block is one
// kernel tile.
struct TileItemMap {
  uint32_t ntiles, slot0, KC, K_eff;
  const uint32_t* tile_list;          // NULL: tile = slot
  uint32_t tile_bytes;
  __device__ __forceinline__ void locate(unsigned long long item, uint32_t& chunk, uint32_t& k0, int& kc,
                                         size_t& off, unsigned long long& id) const {
    chunk = (uint32_t)(item / ntiles);
    const uint32_t pos = (uint32_t)(item % ntiles);
    const uint32_t slot = slot0 + pos;
    k0 = chunk * KC;
    kc = (int)min(KC, K_eff - k0);
    const uint32_t tile = tile_list ? tile_list[slot] : slot;
    off = (size_t)tile * tile_bytes;
    id = ((unsigned long long)chunk << 32) | (unsigned long long)pos;   // (chunk, position in the visit order)
  }
};

}  // namespace kb
