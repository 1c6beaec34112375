// Shared device helpers of the kb library: element decoding, packed
// accumulator keys, mbarrier / bulk-copy wrappers with bounded waits.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/kb_hooks.h"

namespace kb {

// ---- per-candidate accumulator in global memory (order-independent merges) --
// counts: integer add.  key: integer max of ((bits(d) << 32) | (0xFFFFFFFF - idx)) + 1,
// so a larger key is a larger |c - r| and, at equal error, a lower index;
// 0 means "no finite difference seen".  rel: integer max of the bits of a
// non-negative float (monotone, +Inf included).
struct alignas(16) Acc {
  unsigned long long mism;
  unsigned long long nan;
  unsigned long long inf;
  unsigned long long spare;
  // the two maxima share one aligned 16-byte block, so that one asynchronous 16-byte copy
  // brings both into shared memory
  unsigned long long key;
  unsigned int rel;
  unsigned int pad;
};
static_assert(sizeof(Acc) == 48, "Acc layout");

__device__ __forceinline__ unsigned long long pack_key(float d, unsigned long long idx) {
  return (((unsigned long long)__float_as_uint(d) << 32) |
          (unsigned long long)(0xFFFFFFFFu - (unsigned int)idx)) + 1ull;
}

// ---- element decoding to binary32 (exact for all three formats) ------------
template <int DT> struct Elem;
template <> struct Elem<KB_F32> {
  static constexpr int kBytes = 4;
  static constexpr int kVec = 4;  // elements per 16-byte vector
  __device__ __forceinline__ static void decode(const uint4& w, float* out) {
    out[0] = __uint_as_float(w.x);
    out[1] = __uint_as_float(w.y);
    out[2] = __uint_as_float(w.z);
    out[3] = __uint_as_float(w.w);
  }
  __device__ __forceinline__ static float load(const void* p, unsigned long long i) {
    return reinterpret_cast<const float*>(p)[i];
  }
  // d0 = c[e] - r0, d1 = c[e+1] - r1 for the even element e of a thread's raw words
  __device__ __forceinline__ static void pair_diff(const unsigned int* words, int e, float r0, float r1,
                                                   float& d0, float& d1) {
    d0 = __fsub_rn(__uint_as_float(words[e]), r0);
    d1 = __fsub_rn(__uint_as_float(words[e + 1]), r1);
  }
};
template <> struct Elem<KB_BF16> {
  static constexpr int kBytes = 2;
  static constexpr int kVec = 8;
  __device__ __forceinline__ static void decode(const uint4& w, float* out) {
    out[0] = __uint_as_float(w.x << 16);
    out[1] = __uint_as_float(w.x & 0xFFFF0000u);
    out[2] = __uint_as_float(w.y << 16);
    out[3] = __uint_as_float(w.y & 0xFFFF0000u);
    out[4] = __uint_as_float(w.z << 16);
    out[5] = __uint_as_float(w.z & 0xFFFF0000u);
    out[6] = __uint_as_float(w.w << 16);
    out[7] = __uint_as_float(w.w & 0xFFFF0000u);
  }
  __device__ __forceinline__ static float load(const void* p, unsigned long long i) {
    return __uint_as_float((unsigned int)reinterpret_cast<const unsigned short*>(p)[i] << 16);
  }
  // Mixed-precision subtract: the bf16 operand is widened exactly and the
  // difference rounded once, i.e. the same value as decode + fp32 subtract,
  // without a separate decode instruction.
  __device__ __forceinline__ static void pair_diff(const unsigned int* words, int e, float r0, float r1,
                                                   float& d0, float& d1) {
    asm("{\n.reg .b16 lo, hi;\nmov.b32 {lo, hi}, %2;\nsub.rn.f32.bf16 %0, lo, %3;\nsub.rn.f32.bf16 %1, hi, %4;\n}"
        : "=f"(d0), "=f"(d1)
        : "r"(words[e >> 1]), "f"(r0), "f"(r1));
  }
};
template <> struct Elem<KB_F16> {
  static constexpr int kBytes = 2;
  static constexpr int kVec = 8;
  __device__ __forceinline__ static void decode(const uint4& w, float* out) {
    const __half2* h = reinterpret_cast<const __half2*>(&w);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 f = __half22float2(h[i]);
      out[2 * i] = f.x;
      out[2 * i + 1] = f.y;
    }
  }
  __device__ __forceinline__ static float load(const void* p, unsigned long long i) {
    return __half2float(reinterpret_cast<const __half*>(p)[i]);
  }
  __device__ __forceinline__ static void pair_diff(const unsigned int* words, int e, float r0, float r1,
                                                   float& d0, float& d1) {
    asm("{\n.reg .b16 lo, hi;\nmov.b32 {lo, hi}, %2;\nsub.rn.f32.f16 %0, lo, %3;\nsub.rn.f32.f16 %1, hi, %4;\n}"
        : "=f"(d0), "=f"(d1)
        : "r"(words[e >> 1]), "f"(r0), "f"(r1));
  }
};

// The two 8-bit formats: 16 elements per 16-byte vector.  Pairs of bytes are widened to
// f16x2 by one hardware conversion (exact: every fp8 value is an fp16 value), then the
// mixed-precision subtract does the rest.
template <bool E5M2> struct ElemF8 {
  static constexpr int kBytes = 1;
  static constexpr int kVec = 16;
  __device__ __forceinline__ static unsigned int widen2(unsigned short pr) {
    unsigned int h2;
    if (E5M2)
      asm("cvt.rn.f16x2.e5m2x2 %0, %1;" : "=r"(h2) : "h"(pr));
    else
      asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(pr));
    return h2;
  }
  // four bytes -> two f16x2 words (bytes 0,1 and bytes 2,3), without shifting the halves out first
  __device__ __forceinline__ static void widen4(unsigned int w, unsigned int& lo2, unsigned int& hi2) {
    if (E5M2)
      asm("{\n.reg .b16 lo, hi;\nmov.b32 {lo, hi}, %2;\ncvt.rn.f16x2.e5m2x2 %0, lo;\ncvt.rn.f16x2.e5m2x2 %1, hi;\n}"
          : "=r"(lo2), "=r"(hi2)
          : "r"(w));
    else
      asm("{\n.reg .b16 lo, hi;\nmov.b32 {lo, hi}, %2;\ncvt.rn.f16x2.e4m3x2 %0, lo;\ncvt.rn.f16x2.e4m3x2 %1, hi;\n}"
          : "=r"(lo2), "=r"(hi2)
          : "r"(w));
  }
  __device__ __forceinline__ static void decode(const uint4& w, float* out) {
    const unsigned int* u = reinterpret_cast<const unsigned int*>(&w);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const unsigned int h2 = widen2((unsigned short)(u[i >> 1] >> (16 * (i & 1))));
      const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&h2));
      out[2 * i] = f.x;
      out[2 * i + 1] = f.y;
    }
  }
  __device__ __forceinline__ static float load(const void* p, unsigned long long i) {
    const unsigned int h2 = widen2((unsigned short)reinterpret_cast<const unsigned char*>(p)[i]);
    return __low2float(*reinterpret_cast<const __half2*>(&h2));
  }
  __device__ __forceinline__ static void pair_diff(const unsigned int* words, int e, float r0, float r1,
                                                   float& d0, float& d1) {
    // e5m2 is the high byte of binary16: a byte permute widens a pair (no conversion, no shift)
    const unsigned int h2 = E5M2 ? __byte_perm(words[e >> 2], 0u, ((e >> 1) & 1) ? 0x3424u : 0x1404u)
                                 : widen2((unsigned short)(words[e >> 2] >> (16 * ((e >> 1) & 1))));
    asm("{\n.reg .b16 lo, hi;\nmov.b32 {lo, hi}, %2;\nsub.rn.f32.f16 %0, lo, %3;\nsub.rn.f32.f16 %1, hi, %4;\n}"
        : "=f"(d0), "=f"(d1)
        : "r"(h2), "f"(r0), "f"(r1));
  }
};
template <> struct Elem<KB_F8E4M3> : ElemF8<false> {};
template <> struct Elem<KB_F8E5M2> : ElemF8<true> {};

// ---- the gate on one element, written out (used by every slow path) --------
// tol_c = min(atol + rtol*|r|, FLT_MAX): then  |c-r| <= tol_c  <=>  d finite and d <= tol.
__device__ __forceinline__ float tol_clamped(float r, float atol, float rtol) {
  return fminf(__fadd_rn(atol, __fmul_rn(rtol, fabsf(r))), 3.402823466e38f);
}
__device__ __forceinline__ bool is_finite_nonneg(float ad) { return ad <= 3.402823466e38f; }

// ---- device status word -----------------------------------------------------
__device__ __forceinline__ void set_status(unsigned int* status, unsigned int code) {
  atomicCAS(status, 0u, code);
}

// ---- mbarrier + bulk copy (TMA, 1-D, each CTA fetches its own tiles) --------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: polls until the phase with `parity` completes, the CTA-wide
// abort flag is raised, or `limit_ns` (2 s unless stated) pass.  Returns false when it gave
// up; it then raises the abort flag and records KB_ERR_DEVICE_TIMEOUT.  Never traps.
constexpr unsigned long long kWaitLimitNs = 2000000000ull;
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity,
                                                  volatile unsigned int* abort_flag,
                                                  unsigned int* status,
                                                  unsigned long long limit_ns = kWaitLimitNs) {
  if (mbar_try_wait(bar, parity)) return true;
  unsigned long long t0 = 0;
  unsigned int polls = 0;
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if ((++polls & 1023u) == 0) {
      unsigned long long now = global_ns();
      if (t0 == 0) t0 = now;
      if (now - t0 > limit_ns) {
        *abort_flag = 1u;
        set_status(status, (unsigned int)KB_ERR_DEVICE_TIMEOUT);
        return false;
      }
    }
  }
}
// Self-test of the wait above (kb_ctx_selftest_wait): one warp waits on a barrier that nothing
// completes.  No copy is in flight, so giving up leaves nothing behind; the kernel returns
// normally with KB_ERR_DEVICE_TIMEOUT in the status word.
__global__ void wait_selftest_kernel(unsigned int* status, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  __shared__ unsigned int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0u;
    mbar_fence_init();
  }
  __syncwarp();
  mbar_wait_bounded(&bar, 0u, &abort_flag, status, limit_ns);
}

__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
// 1-D bulk copy global -> this CTA's shared memory, completion on an mbarrier.
// dst, src 16-byte aligned; bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src_gmem, uint32_t bytes,
                                         uint64_t* bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1], %2, [%3], %4;" ::"r"(smem_u32(dst_smem)),
      "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}

// 16-byte asynchronous copy global -> shared that bypasses L1 (the source is updated by other
// CTAs' atomics) and needs no register for the data.
__device__ __forceinline__ void cp_async16(void* dst_smem, const void* src_gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst_smem)), "l"(src_gmem)
               : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ unsigned int warp_max_u32(unsigned int v) {
  return __reduce_max_sync(0xFFFFFFFFu, v);
}
__device__ __forceinline__ unsigned int warp_add_u32(unsigned int v) {
  return __reduce_add_sync(0xFFFFFFFFu, v);
}
__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
  unsigned int hi = (unsigned int)(v >> 32);
  unsigned int hmax = warp_max_u32(hi);
  unsigned int lo = (hi == hmax) ? (unsigned int)v : 0u;
  unsigned int lmax = warp_max_u32(lo);
  return ((unsigned long long)hmax << 32) | lmax;
}

}  // namespace kb
