// Host side of the kb C ABI: argument validation (the shape/dtype part of
// the policy check, Sec. 3.2), workspace management and kernel dispatch.
// Declarations and their contracts are in include/kb.h.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <cmath>
#include <mutex>
#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "kb_adjudicate.cuh"
#include "kb_common.cuh"
#include "kb_screen.cuh"
#include "kb_screen8.cuh"
#include "kb_screen64.cuh"
#include "kb_select.cuh"

using namespace kb;

struct kb_ctx {
  int device = 0;
  int sm_count = 0;
  // Workspace for ws_cap_K candidates: [accumulators, set 0 | accumulators, set 1 | pointer table |
  // accumulators of the binary64 gate]; no offset depends on a call's K.
  unsigned char* ws = nullptr;
  size_t ws_bytes = 0;
  uint32_t ws_cap_K = 0;
  bool ws_fixed = false;            // the workspace is not ours to grow or free (kb_screen_static)
  // The binary32 gate keeps two sets of accumulators and counters.  A call works on set
  // `ws_parity`, which is zero on entry, and its lead kernel zeroes the other set (as far as the
  // last call on it got: `used_K`) for the next call.  `ws_dirty`: that may not hold (fresh
  // memory, a call that failed half-way or ran out of time, a call captured into a graph, a path
  // without a lead launch): the next call zeroes both sets with memsets first.
  int ws_parity = 0;
  uint32_t used_K[2] = {0, 0};
  bool ws_dirty = true;
  // Choice between the instantiations of the streaming kernel.  The plain one reports, in a
  // host-visible word, the share of its warp steps that took a fruitless second look: one byte
  // for looks taken while the candidate was lean, one for looks (and exact paths) beyond the lean
  // bound that changed nothing.  When the last report says a quarter or more, the next calls use
  // the sharp instantiation (first byte) or the by-definition one (second byte), and every so
  // often one of them probes the plain one again.
  unsigned int* h_hint = nullptr;   // pinned, mapped
  unsigned int* d_hint = nullptr;   // its device address
  int filter_mode = 0;              // 0 automatic, 1 plain, 2 sharp, 3 by definition
  int alt_mode = 1;                 // the instantiation the automatic choice currently alternates with: 1 or 3
  int sharp_left = 0;
  bool sharp_probe_next = false, sharp_probed = false;
  int last_mode = 0;                // instantiation of the last streaming launch: 0 plain, 1 sharp, 3 by definition
  float call_steps = 0.0f;          // warp steps of the current call's plain streaming launch (0: none)
  float steps_hist[2] = {0.0f, 0.0f};   // the same for the last call on each accumulator set
  // [0] status, [1..3] counters of the binary64 gate, [4] effective K of an indexed call,
  // [8..10] and [16..18] the two counter sets of the binary32 gate, [20..23] two 64-bit sums of
  // fruitless second looks on their way to the host, [60] probe sink
  unsigned int* d_status = nullptr;
  uint32_t forced_grid = 0;
  unsigned char* small_ws = nullptr; // single-launch path: [tickets 4 KB | partial records 384 KB]
  bool small_on = true;
  int wins_algo = 0;                // 0 auto, 1 direct comparison, 2 binary search on sorted rows,
                                    // 3 lane-per-row merge of sorted rows
  float* srt = nullptr;             // [K][S] sorted timings (binary-search win count)
  size_t srt_bytes = 0;
  char err[512] = {0};
  // staging owned for kb_screen_host
  unsigned char* st_ref = nullptr;
  size_t st_ref_bytes = 0;
  unsigned char* st_batch[2] = {nullptr, nullptr};
  size_t st_batch_bytes[2] = {0, 0};
  kb_screen_result* st_out = nullptr;
  size_t st_out_bytes = 0;
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_copied[2] = {nullptr, nullptr};
  cudaEvent_t ev_done[2] = {nullptr, nullptr};
  uint32_t skip_allocs = 0;         // test hook: let this many device allocations through, ...
  uint32_t fail_allocs = 0;         // ... then refuse this many
  // Every buffer the context owns sits between two 256-byte guard bands filled with kGuardByte;
  // kb_ctx_check_guards counts the band bytes that no longer hold it (an out-of-bounds write).
  struct Guarded { unsigned char* raw; size_t bytes; };
  std::vector<Guarded> guarded;
  // instrumentation
  uint64_t launches = 0;
  bool timing = false;
  bool dependent_launch = true;     // streaming kernel as a programmatic dependent of the lead kernel
  static constexpr int kTimers = 2, kPool = 256;
  cudaEvent_t tm_beg[kTimers][kPool] = {};
  cudaEvent_t tm_end[kTimers][kPool] = {};
  uint32_t tm_used[kTimers] = {0, 0};
};

struct kb_mask {
  kb_ctx* ctx = nullptr;
  uint64_t N = 0;
  uint32_t log2_tile = 0;
  int kind = 0;                    // 1 strided, 2 bitmap
  uint32_t stride = 1, phase = 0;
  unsigned long long* d_bits = nullptr;
  uint32_t* d_tiles = nullptr;     // selected FULL kernel tiles (log2_tile >= 12 only)
  uint32_t n_tiles = 0;
  bool coarse = false;             // log2_tile >= 12: the streaming kernel can skip tiles
  uint64_t n_selected = 0;
};

namespace {

thread_local char g_create_err[256] = {0};

kb_status fail(kb_ctx* ctx, kb_status st, const char* fmt, ...) {
  if (ctx) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(ctx->err, sizeof ctx->err, fmt, ap);
    va_end(ap);
  }
  return st;
}

struct DeviceGuard {
  int prev = -1;
  bool changed = false;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) changed = cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() {
    if (changed) cudaSetDevice(prev);
  }
};

#define KB_CUDA(ctx, call)                                                              \
  do {                                                                                  \
    cudaError_t e_ = (call);                                                            \
    if (e_ != cudaSuccess)                                                              \
      return fail((ctx), KB_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_));  \
  } while (0)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int elem_bytes(kb_dtype dt) { return dt == KB_F32 ? 4 : (dt == KB_F8E4M3 || dt == KB_F8E5M2) ? 1 : 2; }
inline bool known_dtype(int dt) { return dt >= KB_F32 && dt <= KB_F8E5M2; }
constexpr size_t kSmallTicketBytes = 4096;
constexpr size_t kSmallMaxPartials = 8192;
constexpr size_t kSmallWsBytes = kSmallTicketBytes + kSmallMaxPartials * sizeof(Acc);

// A named range around an entry point's host work, for a timeline tool that is attached
// (the header-only NVTX v3 calls do nothing otherwise).
struct TraceRange {
  explicit TraceRange(const char* name) { nvtxRangePushA(name); }
  ~TraceRange() { nvtxRangePop(); }
  TraceRange(const TraceRange&) = delete;
  TraceRange& operator=(const TraceRange&) = delete;
};

// Event pair around one launch of an instrumented kernel (no-op unless timing is on).
struct ScopedTimer {
  kb_ctx* ctx;
  cudaStream_t st;
  int which, slot = -1;
  ScopedTimer(kb_ctx* c, int w, cudaStream_t s) : ctx(c), st(s), which(w) {
    if (!ctx->timing) return;
    slot = (int)(ctx->tm_used[which] % kb_ctx::kPool);
    cudaEventRecord(ctx->tm_beg[which][slot], st);
  }
  ~ScopedTimer() {
    if (slot < 0) return;
    cudaEventRecord(ctx->tm_end[which][slot], st);
    ++ctx->tm_used[which];
  }
};

// Every device allocation of a context goes through here: a test can make it fail
// (kb_ctx_fail_next_allocs) without exhausting a GPU's memory, and every buffer gets guard
// bands (compute-sanitizer's stand-in for out-of-bounds writes; see kb_ctx_check_guards).
constexpr size_t kGuardBytes = 256;
constexpr int kGuardByte = 0xA5;
cudaError_t ctx_malloc(kb_ctx* ctx, void** p, size_t bytes) {
  *p = nullptr;
  if (ctx->skip_allocs) {
    --ctx->skip_allocs;
  } else if (ctx->fail_allocs) {
    --ctx->fail_allocs;
    return cudaErrorMemoryAllocation;
  }
  unsigned char* raw = nullptr;
  const size_t body = round_up(bytes, 256);
  cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&raw), body + 2 * kGuardBytes);
  if (e == cudaSuccess) e = cudaMemset(raw, kGuardByte, kGuardBytes);
  if (e == cudaSuccess) e = cudaMemset(raw + kGuardBytes + body, kGuardByte, kGuardBytes);
  if (e != cudaSuccess) {
    if (raw) cudaFree(raw);
    cudaGetLastError();
    return e;
  }
  ctx->guarded.push_back({raw, body});
  *p = raw + kGuardBytes;
  return cudaSuccess;
}
void ctx_free(kb_ctx* ctx, void* p) {
  if (!p) return;
  unsigned char* raw = static_cast<unsigned char*>(p) - kGuardBytes;
  for (size_t i = 0; i < ctx->guarded.size(); ++i)
    if (ctx->guarded[i].raw == raw) {
      ctx->guarded.erase(ctx->guarded.begin() + (long)i);
      break;
    }
  cudaFree(raw);   // waits for enqueued work that still uses the buffer
}

// Grow *buf to at least `need` bytes.  The new buffer is allocated BEFORE the old one is
// released, and pointer and size change together: after a failure the context still holds
// its old, valid (pointer, size) pair and a later, smaller call works as before.
template <typename T>
kb_status ensure_buf(kb_ctx* ctx, T** buf, size_t* have, size_t need, const char* what = "device staging") {
  if (need <= *have) return KB_OK;
  void* fresh = nullptr;
  if (ctx_malloc(ctx, &fresh, need) != cudaSuccess)
    return fail(ctx, KB_ERR_WORKSPACE, "cannot allocate %zu bytes of %s", need, what);
  ctx_free(ctx, *buf);
  *buf = static_cast<T*>(fresh);
  *have = need;
  return KB_OK;
}

static_assert(sizeof(Acc) == sizeof(Acc64), "one region size serves both gates");
inline size_t ws_region(uint32_t cap_K) { return round_up((size_t)cap_K * sizeof(Acc), 256); }
inline size_t ws_table_offset(uint32_t cap_K) { return 2 * ws_region(cap_K); }
inline size_t ws_acc64_offset(uint32_t cap_K) {
  return 2 * ws_region(cap_K) + round_up((size_t)cap_K * sizeof(void*), 256);
}
inline unsigned int* counter_set(kb_ctx* ctx, int set) { return ctx->d_status + 8 + 8 * set; }
kb_status ensure_ws(kb_ctx* ctx, uint32_t K) {
  if (K <= ctx->ws_cap_K) return KB_OK;
  if (ctx->ws_fixed)
    return fail(ctx, KB_ERR_WORKSPACE, "the fixed scratch holds %u candidates, %u asked for", ctx->ws_cap_K, K);
  const uint32_t cap = K < 32768u ? 2u * K : 65535u;
  const kb_status rc =
      ensure_buf(ctx, &ctx->ws, &ctx->ws_bytes, ws_acc64_offset(cap) + ws_region(cap), "device workspace");
  if (rc != KB_OK) return rc;
  ctx->ws_cap_K = cap;
  ctx->ws_dirty = true;   // fresh memory
  return KB_OK;
}

// ring depth by stage size: 3 CTAs/SM must fit ~75 KB each
inline uint32_t stream_stages(uint32_t tile_bytes) { return tile_bytes >= 16384 ? 3 : tile_bytes >= 8192 ? 7 : 10; }

constexpr int kSharpCalls = 32, kSharpGrace = 4;
#ifndef KB8_STAGES
#define KB8_STAGES 7
#endif
// e4m3 kernel: stages of 4 KB, CTAs of 160 threads, four resident per SM at 96 registers
constexpr uint32_t kStages8 = KB8_STAGES, kCtas8 = 4;
template <int DT>
kb_status launch_stream(kb_ctx* ctx, StreamParams& sp, cudaStream_t st, bool behind_lead = false) {
  const uint32_t tile_bytes = kTile * Elem<DT>::kBytes;
  constexpr bool k8 = DT == KB_F8E4M3;           // e4m3 has a kernel of its own (kb_screen8.cuh)
  sp.stages = k8 ? kStages8 : stream_stages(tile_bytes);
  const size_t smem = k8 ? stream8_smem_bytes(sp.stages) : stream_smem_bytes(sp.stages, tile_bytes);
  const unsigned long long nitems = (unsigned long long)sp.nchunks * sp.ntiles;
  unsigned long long grid = ctx->forced_grid ? ctx->forced_grid : (k8 ? (unsigned long long)kCtas8 : 3ull) * ctx->sm_count;
  if (grid > nitems) grid = nitems;
  // which instantiation: what the last finished plain call on this context reported
  // Plain until a plain launch reports that a quarter of its warp steps took a fruitless
  // second look; then sharp for kSharpCalls launches, one plain launch as a probe, sharp again
  // for the kSharpGrace launches its report needs to arrive, and the report decides.
  bool sharp = ctx->filter_mode >= 2 && !k8;     // "sharp": not the plain instantiation
  if (ctx->filter_mode == 2) ctx->alt_mode = 1;
  if (ctx->filter_mode == 3) ctx->alt_mode = 3;
  if (ctx->filter_mode == 0 && ctx->h_hint && !k8) {
    volatile unsigned int* hint = reinterpret_cast<volatile unsigned int*>(ctx->h_hint);
    if (ctx->sharp_left > 0) {
      sharp = true;
      if (--ctx->sharp_left == 0 && !ctx->sharp_probed) {
        ctx->sharp_probe_next = true;          // the next launch is the probe
      } else if (ctx->sharp_left == 0) {
        ctx->sharp_probed = false;             // the grace period is over: the report decides below
      }
    } else if (ctx->sharp_probe_next) {
      ctx->sharp_probe_next = false;
      ctx->sharp_probed = true;
      ctx->sharp_left = kSharpGrace;
      *hint = 0u;
    } else {
      // byte 0: second looks taken while lean, byte 1: fruitless looks beyond the lean bound,
      // in 64ths of the reporting call's warp steps; a quarter of the steps decides
      const unsigned int h = *hint;
      const unsigned int lean_share = h & 0xFFu, atol_share = (h >> 8) & 0xFFu;
      if (lean_share >= 16u || atol_share >= 16u) {
        sharp = true;
        ctx->alt_mode = atol_share > lean_share ? 3 : 1;
        ctx->sharp_left = kSharpCalls - 1;
        ctx->sharp_probed = false;
        *hint = 0u;                            // the next plain launch reports afresh
      }
    }
  }
  const int alt = ctx->alt_mode;
  ctx->last_mode = sharp ? alt : 0;
  // warp steps of this launch if it counts its fruitless second looks (see LeadParams)
  ctx->call_steps = (sharp || k8) ? 0.0f : (float)sp.ntiles * (float)sp.K * (float)kWarps;
  {
    ScopedTimer tm(ctx, KB_TIMER_SCREEN_STREAM, st);
    if constexpr (k8) {
      screen_stream8_kernel<DT><<<(unsigned int)grid, kThreads8, smem, st>>>(sp);
    } else {
      const bool dependent = behind_lead && ctx->dependent_launch;
      if (sharp && alt == 1) {
        screen_stream_kernel<DT, 1><<<(unsigned int)grid, kStreamThreads, smem, st>>>(sp);
      } else if (dependent) {
        // launch and set-up overlap the lead kernel (about 3 us per call)
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned int)grid);
        cfg.blockDim = dim3(kStreamThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (sharp)
          KB_CUDA(ctx, cudaLaunchKernelEx(&cfg, screen_stream_kernel<DT, 3>, sp));
        else
          KB_CUDA(ctx, cudaLaunchKernelEx(&cfg, screen_stream_kernel<DT, 2>, sp));
      } else if (sharp) {
        screen_stream_kernel<DT, 3><<<(unsigned int)grid, kStreamThreads, smem, st>>>(sp);
      } else {
        screen_stream_kernel<DT, 0><<<(unsigned int)grid, kStreamThreads, smem, st>>>(sp);
      }
    }
  }
  ++ctx->launches;
  KB_CUDA(ctx, cudaGetLastError());
  return KB_OK;
}

template <int DT>
kb_status launch_generic(kb_ctx* ctx, const void* ref, const void* const* tab, Acc* acc, uint32_t K,
                         uint64_t e0, uint64_t e1, float atol, float rtol, const MaskDev& md,
                         const unsigned int* count, cudaStream_t st) {
  if (e1 <= e0) return KB_OK;
  const uint64_t len = e1 - e0;
  uint64_t bx = (len + 255) / 256;
  const uint64_t cap = (uint64_t)ctx->sm_count * 8;
  if (bx > cap) bx = cap;
  dim3 grid((unsigned int)bx, K);
  screen_generic_kernel<DT><<<grid, 256, 0, st>>>(ref, tab, acc, e0, e1, atol, rtol, md, count);
  ++ctx->launches;
  KB_CUDA(ctx, cudaGetLastError());
  return KB_OK;
}

template <int DT>
kb_status set_stream_attr(kb_ctx* ctx) {
  if constexpr (DT == KB_F8E4M3) {
    KB_CUDA(ctx, cudaFuncSetAttribute(screen_stream8_kernel<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)stream8_smem_bytes(kStages8)));
    KB_CUDA(ctx, cudaFuncSetAttribute(screen_stream8_kernel<DT>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                      (int)cudaSharedmemCarveoutMaxShared));
  } else {
    const uint32_t tile_bytes = kTile * Elem<DT>::kBytes;
    const size_t smem = stream_smem_bytes(stream_stages(tile_bytes), tile_bytes);
    KB_CUDA(ctx, cudaFuncSetAttribute(screen_stream_kernel<DT, 0>,
                                      cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    KB_CUDA(ctx, cudaFuncSetAttribute(screen_stream_kernel<DT, 0>,
                                      cudaFuncAttributePreferredSharedMemoryCarveout,
                                      (int)cudaSharedmemCarveoutMaxShared));
    KB_CUDA(ctx, cudaFuncSetAttribute(screen_stream_kernel<DT, 1>,
                                      cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    KB_CUDA(ctx, cudaFuncSetAttribute(screen_stream_kernel<DT, 1>,
                                      cudaFuncAttributePreferredSharedMemoryCarveout,
                                      (int)cudaSharedmemCarveoutMaxShared));
    KB_CUDA(ctx, cudaFuncSetAttribute(screen_stream_kernel<DT, 2>,
                                      cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    KB_CUDA(ctx, cudaFuncSetAttribute(screen_stream_kernel<DT, 2>,
                                      cudaFuncAttributePreferredSharedMemoryCarveout,
                                      (int)cudaSharedmemCarveoutMaxShared));
    KB_CUDA(ctx, cudaFuncSetAttribute(screen_stream_kernel<DT, 3>,
                                      cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    KB_CUDA(ctx, cudaFuncSetAttribute(screen_stream_kernel<DT, 3>,
                                      cudaFuncAttributePreferredSharedMemoryCarveout,
                                      (int)cudaSharedmemCarveoutMaxShared));
  }
  return KB_OK;
}

constexpr uint32_t kStages64 = 12;
kb_status set_stream64_attr(kb_ctx* ctx) {
  KB_CUDA(ctx, cudaFuncSetAttribute(screen_stream64_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)stream64_smem_bytes(kStages64)));
  KB_CUDA(ctx, cudaFuncSetAttribute(screen_stream64_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                    (int)cudaSharedmemCarveoutMaxShared));
  return KB_OK;
}

constexpr uint32_t kMergeMaxS = 1024;   // 40 rows of S + 2 floats in shared memory: 164 KB

template <int R>
void launch_wins(const WinsParams& wp, unsigned int grid, size_t smem, cudaStream_t st) {
  wins_kernel<R><<<grid, kWinsThreads, smem, st>>>(wp);
}

}  // namespace

// ---------------------------------------------------------------------------
// context
// ---------------------------------------------------------------------------

extern "C" kb_status kb_ctx_create(int device, kb_ctx** out) {
  if (!out) {
    snprintf(g_create_err, sizeof g_create_err, "kb_ctx_create: out is NULL");
    return KB_ERR_INVALID_ARG;
  }
  *out = nullptr;
  int ndev = 0;
  cudaError_t e = cudaGetDeviceCount(&ndev);
  if (e != cudaSuccess || device < 0 || device >= ndev) {
    snprintf(g_create_err, sizeof g_create_err, "kb_ctx_create: no CUDA device %d (%s)", device,
             e != cudaSuccess ? cudaGetErrorString(e) : "out of range");
    cudaGetLastError();
    return e != cudaSuccess ? KB_ERR_CUDA : KB_ERR_INVALID_ARG;
  }
  kb_ctx* ctx = new (std::nothrow) kb_ctx();
  if (!ctx) return KB_ERR_WORKSPACE;
  ctx->device = device;
  DeviceGuard g(device);
  cudaDeviceProp prop;
  kb_status st = KB_OK;
  auto bail = [&](kb_status s) {
    snprintf(g_create_err, sizeof g_create_err, "kb_ctx_create: %s", ctx->err);
    kb_ctx_destroy(ctx);
    return s;
  };
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) {
    fail(ctx, KB_ERR_CUDA, "cudaGetDeviceProperties failed");
    return bail(KB_ERR_CUDA);
  }
  ctx->sm_count = prop.multiProcessorCount;
  if (ctx_malloc(ctx, reinterpret_cast<void**>(&ctx->d_status), 256) != cudaSuccess ||
      cudaMemset(ctx->d_status, 0, 256) != cudaSuccess) {
    fail(ctx, KB_ERR_WORKSPACE, "cannot allocate the device status word");
    return bail(KB_ERR_WORKSPACE);
  }
  if (ctx_malloc(ctx, reinterpret_cast<void**>(&ctx->small_ws), kSmallWsBytes) != cudaSuccess ||
      cudaMemset(ctx->small_ws, 0, kSmallWsBytes) != cudaSuccess) {
    fail(ctx, KB_ERR_WORKSPACE, "cannot allocate the small-problem workspace");
    return bail(KB_ERR_WORKSPACE);
  }
  // the hint word is optional: without it the plain instantiation always runs
  if (cudaHostAlloc(reinterpret_cast<void**>(&ctx->h_hint), 64, cudaHostAllocMapped) == cudaSuccess) {
    memset(ctx->h_hint, 0, 64);
    if (cudaHostGetDevicePointer(reinterpret_cast<void**>(&ctx->d_hint), ctx->h_hint, 0) != cudaSuccess) {
      cudaFreeHost(ctx->h_hint);
      ctx->h_hint = nullptr;
      ctx->d_hint = nullptr;
    }
  } else {
    ctx->h_hint = nullptr;
  }
  cudaGetLastError();
  if ((st = set_stream_attr<KB_F32>(ctx)) != KB_OK) return bail(st);
  if ((st = set_stream_attr<KB_F16>(ctx)) != KB_OK) return bail(st);
  if ((st = set_stream_attr<KB_BF16>(ctx)) != KB_OK) return bail(st);
  if ((st = set_stream_attr<KB_F8E4M3>(ctx)) != KB_OK) return bail(st);
  if ((st = set_stream_attr<KB_F8E5M2>(ctx)) != KB_OK) return bail(st);
  if ((st = set_stream64_attr(ctx)) != KB_OK) return bail(st);
  if (cudaFuncSetAttribute(rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)(KB_MAX_S * sizeof(float))) != cudaSuccess) {
    fail(ctx, KB_ERR_CUDA, "cannot raise the shared-memory limit of the row kernel");
    return bail(KB_ERR_CUDA);
  }
  if (cudaFuncSetAttribute(wins_merge_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)((kMergeTile + kMergeARows) * ((kMergeMaxS + 1) | 1u) * sizeof(float))) != cudaSuccess) {
    fail(ctx, KB_ERR_CUDA, "cannot raise the shared-memory limit of the merge win-count kernel");
    return bail(KB_ERR_CUDA);
  }
  if (cudaFuncSetAttribute(tails_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)(KB_MAX_S * sizeof(float))) != cudaSuccess) {
    fail(ctx, KB_ERR_CUDA, "cannot raise the shared-memory limit of the tail-ratio kernel");
    return bail(KB_ERR_CUDA);
  }
  if (cudaFuncSetAttribute(wins_ragged_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kWinsRowsPerBlock * 4096 * (int)sizeof(float)) != cudaSuccess) {
    fail(ctx, KB_ERR_CUDA, "cannot raise the shared-memory limit of the ragged win-count kernel");
    return bail(KB_ERR_CUDA);
  }
  if (cudaFuncSetAttribute(wins_rank_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kWinsRowsPerBlock * 4096 * (int)sizeof(float)) != cudaSuccess) {
    fail(ctx, KB_ERR_CUDA, "cannot raise the shared-memory limit of the win-count kernel");
    return bail(KB_ERR_CUDA);
  }
  *out = ctx;
  return KB_OK;
}

extern "C" kb_status kb_ctx_destroy(kb_ctx* ctx) {
  if (!ctx) return KB_OK;
  DeviceGuard g(ctx->device);
  cudaDeviceSynchronize();
  if (!ctx->ws_fixed) ctx_free(ctx, ctx->ws);
  ctx_free(ctx, ctx->d_status);
  ctx_free(ctx, ctx->st_ref);
  ctx_free(ctx, ctx->srt);
  ctx_free(ctx, ctx->small_ws);
  for (int i = 0; i < 2; ++i) {
    ctx_free(ctx, ctx->st_batch[i]);
    if (ctx->ev_copied[i]) cudaEventDestroy(ctx->ev_copied[i]);
    if (ctx->ev_done[i]) cudaEventDestroy(ctx->ev_done[i]);
  }
  ctx_free(ctx, ctx->st_out);
  if (ctx->h_hint) cudaFreeHost(ctx->h_hint);
  if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
  for (int t = 0; t < kb_ctx::kTimers; ++t)
    for (int i = 0; i < kb_ctx::kPool; ++i) {
      if (ctx->tm_beg[t][i]) cudaEventDestroy(ctx->tm_beg[t][i]);
      if (ctx->tm_end[t][i]) cudaEventDestroy(ctx->tm_end[t][i]);
    }
  cudaGetLastError();
  delete ctx;
  return KB_OK;
}

extern "C" const char* kb_last_error(const kb_ctx* ctx) { return ctx ? ctx->err : g_create_err; }

extern "C" kb_status kb_ctx_poll(kb_ctx* ctx, void* stream, kb_status* device_status) {
  if (!ctx || !device_status) return KB_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  unsigned int word = 0;
  KB_CUDA(ctx, cudaMemcpyAsync(&word, ctx->d_status, sizeof word, cudaMemcpyDeviceToHost, st));
  KB_CUDA(ctx, cudaMemsetAsync(ctx->d_status, 0, sizeof word, st));
  KB_CUDA(ctx, cudaStreamSynchronize(st));
  *device_status = (kb_status)word;
  if (word != 0u) ctx->ws_dirty = true;   // a call may have been cut short: take nothing on trust
  return KB_OK;
}

extern "C" kb_status kb_ctx_set_grid(kb_ctx* ctx, uint32_t blocks) {
  if (!ctx) return KB_ERR_INVALID_ARG;
  ctx->forced_grid = blocks;
  return KB_OK;
}

extern "C" kb_status kb_ctx_set_filter(kb_ctx* ctx, int mode) {
  if (!ctx || mode < 0 || mode > 3) return KB_ERR_INVALID_ARG;
  ctx->filter_mode = mode;
  ctx->sharp_left = 0;
  ctx->sharp_probe_next = ctx->sharp_probed = false;
  if (ctx->h_hint) *reinterpret_cast<volatile unsigned int*>(ctx->h_hint) = 0u;
  return KB_OK;
}

extern "C" kb_status kb_ctx_last_filter(const kb_ctx* ctx, int* mode) {
  if (!ctx || !mode) return KB_ERR_INVALID_ARG;
  *mode = ctx->last_mode;
  return KB_OK;
}

extern "C" kb_status kb_ctx_set_dependent_launch(kb_ctx* ctx, int on) {
  if (!ctx) return KB_ERR_INVALID_ARG;
  ctx->dependent_launch = on != 0;
  return KB_OK;
}

extern "C" kb_status kb_ctx_set_small_path(kb_ctx* ctx, int on) {
  if (!ctx) return KB_ERR_INVALID_ARG;
  ctx->small_on = on != 0;
  return KB_OK;
}

extern "C" kb_status kb_ctx_fail_next_allocs(kb_ctx* ctx, uint32_t skip, uint32_t n) {
  if (!ctx) return KB_ERR_INVALID_ARG;
  ctx->skip_allocs = n ? skip : 0;
  ctx->fail_allocs = n;
  return KB_OK;
}

extern "C" kb_status kb_ctx_check_guards(kb_ctx* ctx, void* stream, uint32_t* n_buffers, uint32_t* n_bad_bytes) {
  if (!ctx || !n_buffers || !n_bad_bytes) return KB_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  KB_CUDA(ctx, cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream)));
  uint32_t bad = 0;
  unsigned char band[2 * kGuardBytes];
  for (const kb_ctx::Guarded& gb : ctx->guarded) {
    KB_CUDA(ctx, cudaMemcpy(band, gb.raw, kGuardBytes, cudaMemcpyDeviceToHost));
    KB_CUDA(ctx, cudaMemcpy(band + kGuardBytes, gb.raw + kGuardBytes + gb.bytes, kGuardBytes, cudaMemcpyDeviceToHost));
    for (size_t i = 0; i < 2 * kGuardBytes; ++i) bad += band[i] != (unsigned char)kGuardByte;
  }
  *n_buffers = (uint32_t)ctx->guarded.size();
  *n_bad_bytes = bad;
  return KB_OK;
}

extern "C" kb_status kb_ctx_selftest_wait(kb_ctx* ctx, uint64_t limit_ns, void* stream) {
  if (!ctx) return KB_ERR_INVALID_ARG;
  if (limit_ns < 1000ull || limit_ns > 100000000ull)
    return fail(ctx, KB_ERR_INVALID_ARG, "kb_ctx_selftest_wait: limit outside [1 us, 100 ms]");
  DeviceGuard g(ctx->device);
  wait_selftest_kernel<<<1, 32, 0, reinterpret_cast<cudaStream_t>(stream)>>>(ctx->d_status, limit_ns);
  ++ctx->launches;
  KB_CUDA(ctx, cudaGetLastError());
  return KB_OK;
}

extern "C" kb_status kb_ctx_set_wins_algo(kb_ctx* ctx, int algo) {
  if (!ctx || algo < 0 || algo > 3) return KB_ERR_INVALID_ARG;
  ctx->wins_algo = algo;
  return KB_OK;
}

extern "C" kb_status kb_ctx_enable_timing(kb_ctx* ctx, int on) {
  if (!ctx) return KB_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (on && !ctx->tm_beg[0][0]) {
    for (int t = 0; t < kb_ctx::kTimers; ++t)
      for (int i = 0; i < kb_ctx::kPool; ++i) {
        KB_CUDA(ctx, cudaEventCreate(&ctx->tm_beg[t][i]));
        KB_CUDA(ctx, cudaEventCreate(&ctx->tm_end[t][i]));
      }
  }
  ctx->timing = on != 0;
  if (on == 1) ctx->tm_used[0] = ctx->tm_used[1] = 0;
  return KB_OK;
}

extern "C" kb_status kb_ctx_read_timer(kb_ctx* ctx, kb_timer which, float* h_ms, uint32_t cap,
                                       uint32_t* n) {
  if (!ctx || !h_ms || !n || (int)which < 0 || (int)which >= kb_ctx::kTimers) return KB_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  const uint32_t used = ctx->tm_used[which];
  uint32_t have = used < (uint32_t)kb_ctx::kPool ? used : (uint32_t)kb_ctx::kPool;
  if (have > cap) have = cap;
  for (uint32_t i = 0; i < have; ++i) {
    const uint32_t slot = (used - have + i) % kb_ctx::kPool;
    KB_CUDA(ctx, cudaEventSynchronize(ctx->tm_end[which][slot]));
    KB_CUDA(ctx, cudaEventElapsedTime(&h_ms[i], ctx->tm_beg[which][slot], ctx->tm_end[which][slot]));
  }
  *n = have;
  ctx->tm_used[which] = 0;
  return KB_OK;
}

extern "C" kb_status kb_alu_probe(kb_ctx* ctx, uint32_t iters, double* pairs_per_s, void* stream) {
  if (!ctx) return KB_ERR_INVALID_ARG;
  if (!pairs_per_s || iters == 0) return fail(ctx, KB_ERR_INVALID_ARG, "kb_alu_probe: null pointer or iters = 0");
  DeviceGuard g(ctx->device);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const unsigned int blocks = (unsigned int)ctx->sm_count * 8u, threads = 256u;
  if (iters > (1u << 23)) return fail(ctx, KB_ERR_INVALID_ARG, "kb_alu_probe: iters above 2^23");
  unsigned int* sink = ctx->d_status + 60;   // a spare status word; never written in practice
  struct Events {   // released on every path
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    ~Events() {
      if (e0) cudaEventDestroy(e0);
      if (e1) cudaEventDestroy(e1);
    }
  } ev;
  KB_CUDA(ctx, cudaEventCreate(&ev.e0));
  KB_CUDA(ctx, cudaEventCreate(&ev.e1));
  alu_probe_kernel<<<blocks, threads, 0, st>>>(iters / 8 + 1, 1.5f, sink);   // warm-up
  KB_CUDA(ctx, cudaEventRecord(ev.e0, st));
  alu_probe_kernel<<<blocks, threads, 0, st>>>(iters, 1.5f, sink);
  KB_CUDA(ctx, cudaEventRecord(ev.e1, st));
  ctx->launches += 2;
  KB_CUDA(ctx, cudaGetLastError());
  KB_CUDA(ctx, cudaEventSynchronize(ev.e1));
  float ms = 0.0f;
  KB_CUDA(ctx, cudaEventElapsedTime(&ms, ev.e0, ev.e1));
  if (!(ms > 0.0f)) return fail(ctx, KB_ERR_CUDA, "kb_alu_probe: the probe took no measurable time");
  *pairs_per_s = (double)blocks * threads * (double)iters * 16.0 * 8.0 / ((double)ms * 1e-3);
  return KB_OK;
}

extern "C" kb_status kb_ctx_launch_count(const kb_ctx* ctx, uint64_t* n) {
  if (!ctx || !n) return KB_ERR_INVALID_ARG;
  *n = ctx->launches;
  return KB_OK;
}

// ---------------------------------------------------------------------------
// masks
// ---------------------------------------------------------------------------

namespace {

kb_status mask_finish(kb_ctx* ctx, kb_mask* m, const uint64_t* host_bits, kb_mask** out) {
  const uint64_t tile = 1ull << m->log2_tile;
  const uint64_t nt = (m->N + tile - 1) >> m->log2_tile;
  auto sel = [&](uint64_t t) -> bool {
    if (m->kind == 1) return (t % m->stride) == m->phase;
    return (host_bits[t >> 6] >> (t & 63)) & 1ull;
  };
  auto tile_len = [&](uint64_t t) -> uint64_t {
    const uint64_t b = t << m->log2_tile;
    return (m->N - b < tile) ? m->N - b : tile;
  };
  m->coarse = m->log2_tile >= 12;
  uint64_t nsel = 0;
  if (m->kind == 1) {
    const uint64_t cnt = nt > m->phase ? (nt - 1 - m->phase) / m->stride + 1 : 0;
    nsel = cnt * tile;
    if (cnt && sel(nt - 1)) nsel -= tile - tile_len(nt - 1);
  } else {
    for (uint64_t t = 0; t < nt; ++t)
      if (sel(t)) nsel += tile_len(t);
  }
  m->n_selected = nsel;
  DeviceGuard g(ctx->device);
  if (m->kind == 2) {
    const size_t words = (size_t)((nt + 63) / 64);
    if (cudaMalloc(&m->d_bits, words * 8) != cudaSuccess) {
      cudaGetLastError();
      delete m;
      return fail(ctx, KB_ERR_WORKSPACE, "cannot allocate the mask bitmap");
    }
    if (cudaMemcpy(m->d_bits, host_bits, words * 8, cudaMemcpyHostToDevice) != cudaSuccess) {
      cudaFree(m->d_bits);
      delete m;
      return fail(ctx, KB_ERR_CUDA, "mask bitmap upload failed");
    }
  }
  if (m->coarse) {
    // list of selected FULL kernel tiles, ascending (the ragged tail goes to the generic kernel)
    const uint32_t per = 1u << (m->log2_tile - 12);
    const uint64_t nfull = m->N / kTile;
    std::vector<uint32_t> tiles;
    for (uint64_t t = 0; t < nt; ++t) {
      if (!sel(t)) continue;
      for (uint32_t w = 0; w < per; ++w) {
        const uint64_t kt = t * per + w;
        if (kt < nfull) tiles.push_back((uint32_t)kt);
      }
    }
    m->n_tiles = (uint32_t)tiles.size();
    if (m->n_tiles) {
      if (cudaMalloc(&m->d_tiles, tiles.size() * 4) != cudaSuccess ||
          cudaMemcpy(m->d_tiles, tiles.data(), tiles.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess) {
        cudaGetLastError();
        if (m->d_tiles) cudaFree(m->d_tiles);
        if (m->d_bits) cudaFree(m->d_bits);
        delete m;
        return fail(ctx, KB_ERR_WORKSPACE, "cannot build the mask tile list");
      }
    }
  }
  *out = m;
  return KB_OK;
}

}  // namespace

extern "C" kb_status kb_mask_create_strided(kb_ctx* ctx, uint64_t N, uint32_t log2_tile,
                                            uint32_t stride, uint32_t phase, kb_mask** out) {
  if (!ctx || !out) return KB_ERR_INVALID_ARG;
  *out = nullptr;
  if (N == 0 || N > KB_MAX_N || log2_tile > 31 || stride == 0 || phase >= stride)
    return fail(ctx, KB_ERR_INVALID_ARG, "kb_mask_create_strided: bad N, log2_tile, stride or phase");
  kb_mask* m = new (std::nothrow) kb_mask();
  if (!m) return fail(ctx, KB_ERR_WORKSPACE, "out of host memory");
  m->ctx = ctx;
  m->N = N;
  m->log2_tile = log2_tile;
  m->kind = 1;
  m->stride = stride;
  m->phase = phase;
  return mask_finish(ctx, m, nullptr, out);
}

extern "C" kb_status kb_mask_create_bitmap(kb_ctx* ctx, uint64_t N, uint32_t log2_tile,
                                           const uint64_t* host_bits, kb_mask** out) {
  if (!ctx || !out) return KB_ERR_INVALID_ARG;
  *out = nullptr;
  if (N == 0 || N > KB_MAX_N || log2_tile > 31 || !host_bits)
    return fail(ctx, KB_ERR_INVALID_ARG, "kb_mask_create_bitmap: bad N, log2_tile or bitmap");
  kb_mask* m = new (std::nothrow) kb_mask();
  if (!m) return fail(ctx, KB_ERR_WORKSPACE, "out of host memory");
  m->ctx = ctx;
  m->N = N;
  m->log2_tile = log2_tile;
  m->kind = 2;
  return mask_finish(ctx, m, host_bits, out);
}

extern "C" kb_status kb_mask_count(const kb_mask* mask, uint64_t* n_selected) {
  if (!mask || !n_selected) return KB_ERR_INVALID_ARG;
  *n_selected = mask->n_selected;
  return KB_OK;
}

extern "C" kb_status kb_mask_destroy(kb_mask* m) {
  if (!m) return KB_OK;
  DeviceGuard g(m->ctx->device);
  if (m->d_bits) cudaFree(m->d_bits);
  if (m->d_tiles) cudaFree(m->d_tiles);
  cudaGetLastError();
  delete m;
  return KB_OK;
}

// ---------------------------------------------------------------------------
// kb_screen
// ---------------------------------------------------------------------------

namespace {

kb_status validate_screen(kb_ctx* ctx, const void* ref, const void* const* cands, uint32_t K,
                          uint64_t N, kb_dtype dtype, float atol, float rtol, const kb_mask* mask,
                          const void* out, bool device_ptrs) {
  if (!ctx) return KB_ERR_INVALID_ARG;
  if (!ref || !cands || !out) return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen: null pointer");
  if (K == 0 || K > KB_MAX_K) return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen: K=%u outside [1, %u]", K, KB_MAX_K);
  if (N == 0 || N > KB_MAX_N) return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen: N outside [1, 2^32]");
  if (!known_dtype((int)dtype))
    return fail(ctx, KB_ERR_UNSUPPORTED, "kb_screen: unknown dtype %d", (int)dtype);
  if (!(atol >= 0.0f) || !(rtol >= 0.0f) || std::isinf(atol) || std::isinf(rtol))
    return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen: atol and rtol must be finite and >= 0");
  if (mask && (mask->N != N || mask->ctx != ctx))
    return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen: the mask was created for another N or context");
  if (device_ptrs) {
    if (!aligned16(ref)) return fail(ctx, KB_ERR_ALIGNMENT, "kb_screen: reference not 16-byte aligned");
    if ((reinterpret_cast<uintptr_t>(out) & 7u) != 0)
      return fail(ctx, KB_ERR_ALIGNMENT, "kb_screen: output not 8-byte aligned");
  }
  for (uint32_t k = 0; k < K; ++k) {
    if (!cands[k]) return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen: candidate %u is NULL", k);
    if (device_ptrs && !aligned16(cands[k]))
      return fail(ctx, KB_ERR_ALIGNMENT, "kb_screen: candidate %u not 16-byte aligned", k);
  }
  return KB_OK;
}

// A selection of candidates that lives on the device (kb_screen_indexed).
struct IndexedSel {
  const void* const* d_table;
  uint32_t K_all;
  const int32_t* d_index;
  const uint32_t* d_count;
};

template <int DT>
kb_status screen_impl(kb_ctx* ctx, const void* d_ref, const void* const* h_cands, uint32_t K,
                      uint64_t N, float atol, float rtol, const kb_mask* mask,
                      kb_screen_result* d_out, cudaStream_t st, const IndexedSel* sel = nullptr) {
  // Latency-bound sizes: everything in one launch (pointers as kernel arguments).
  const uint64_t nb_small = (N + kSmallPerBlock - 1) / kSmallPerBlock;
  if (!sel && ctx->small_ws && ctx->small_on && K <= (uint32_t)kPtrsPerLaunch && (uint64_t)K * N <= (1ull << 22) &&
      (uint64_t)K * nb_small <= kSmallMaxPartials) {
    SmallParams sm;
    sm.ref = d_ref;
    sm.tickets = reinterpret_cast<unsigned int*>(ctx->small_ws);
    sm.partials = reinterpret_cast<Acc*>(ctx->small_ws + kSmallTicketBytes);
    sm.out = d_out;
    sm.N = N;
    sm.nb = (unsigned int)nb_small;
    sm.atol = atol;
    sm.rtol = rtol;
    sm.mask.kind = mask ? mask->kind : 0;
    sm.mask.log2_tile = mask ? mask->log2_tile : 0;
    sm.mask.stride = mask ? mask->stride : 1;
    sm.mask.phase = mask ? mask->phase : 0;
    sm.mask.bits = mask ? mask->d_bits : nullptr;
    PtrChunk ch;
    memcpy(ch.p, h_cands, K * sizeof(void*));
    dim3 grid((unsigned int)nb_small, K);
    cudaStreamCaptureStatus cap_small = cudaStreamCaptureStatusNone;
    if (ctx->dependent_launch && cudaStreamIsCapturing(st, &cap_small) == cudaSuccess &&
        cap_small == cudaStreamCaptureStatusNone) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = grid;
      cfg.blockDim = dim3(256);
      cfg.stream = st;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[0].val.programmaticStreamSerializationAllowed = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      KB_CUDA(ctx, cudaLaunchKernelEx(&cfg, screen_small_kernel<DT>, sm, ch));
    } else {
      screen_small_kernel<DT><<<grid, 256, 0, st>>>(sm, ch);
    }
    ++ctx->launches;
    KB_CUDA(ctx, cudaGetLastError());
    return KB_OK;
  }
  kb_status rc = ensure_ws(ctx, K);
  if (rc != KB_OK) return rc;
  const void** table = reinterpret_cast<const void**>(ctx->ws + ws_table_offset(ctx->ws_cap_K));

  // Two sets of accumulators and counters: this call's (zero on entry) and the one its lead
  // kernel zeroes for the next call.  Whatever may have broken that is repaired with memsets.
  // A call that is being captured into a graph takes nothing on trust (the graph may be
  // replayed in any state) and leaves the workspace marked dirty for the calls after it.
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) {
    cudaGetLastError();
    cap = cudaStreamCaptureStatusActive;
  }
  const bool capturing = cap != cudaStreamCaptureStatusNone;
  if (capturing || ctx->ws_dirty) {
    KB_CUDA(ctx, cudaMemsetAsync(ctx->ws, 0, 2 * ws_region(ctx->ws_cap_K), st));
    KB_CUDA(ctx, cudaMemsetAsync(counter_set(ctx, 0), 0, 16 * sizeof(unsigned int), st));   // both sets, the sums
    ctx->used_K[0] = ctx->used_K[1] = 0;
    ctx->steps_hist[0] = ctx->steps_hist[1] = 0.0f;
  }
  const int set = ctx->ws_parity;
  Acc* acc = reinterpret_cast<Acc*>(ctx->ws + (size_t)set * ws_region(ctx->ws_cap_K));
  Acc* acc_next = reinterpret_cast<Acc*>(ctx->ws + (size_t)(set ^ 1) * ws_region(ctx->ws_cap_K));
  unsigned int* counters = counter_set(ctx, set);
  ctx->ws_dirty = true;      // until every launch of this call has been enqueued
  bool lead_ran = false;
  ctx->call_steps = 0.0f;
  auto finished = [&]() {
    ctx->steps_hist[set] = ctx->call_steps;
    // the lead kernel has cleaned the other set; without one (or under capture) the next call memsets
    if (lead_ran && !capturing) {
      ctx->used_K[set] = K;
      ctx->used_K[set ^ 1] = 0;
      ctx->ws_parity = set ^ 1;
      ctx->ws_dirty = false;
    }
    return KB_OK;
  };

  // Candidate pointers: up to kPtrsPerLaunch travel in the lead kernel's own arguments (it puts
  // them into the device table); more, or a selection that lives on the device, take a launch.
  const bool fine_mask = mask && !mask->coarse;
  const bool by_args = !sel && !fine_mask && K <= (uint32_t)kPtrsPerLaunch;
  static thread_local PtrChunk chunk;   // 3.8 KB: kept off the stack
  if (by_args) memcpy(chunk.p, h_cands, K * sizeof(void*));

  // with a device-resident selection the later kernels read the effective candidate count
  unsigned int* eff_count = ctx->d_status + 4;
  const unsigned int* count = sel ? eff_count : nullptr;
  if (sel) {
    screen_prep_indexed_kernel<<<1, 256, 0, st>>>(sel->d_table, sel->K_all, sel->d_index, sel->d_count, K,
                                                  table, acc, counters, eff_count, ctx->d_status);
    ++ctx->launches;
    KB_CUDA(ctx, cudaGetLastError());
  }
  for (uint32_t off = 0; !sel && !by_args && off < K; off += kPtrsPerLaunch) {
    PtrChunk ch;
    const uint32_t cnt = (K - off < (uint32_t)kPtrsPerLaunch) ? K - off : (uint32_t)kPtrsPerLaunch;
    memcpy(ch.p, h_cands + off, cnt * sizeof(void*));
    screen_prep_kernel<<<(cnt + 127) / 128, 128, 0, st>>>(ch, table, off, cnt);
    ++ctx->launches;
    KB_CUDA(ctx, cudaGetLastError());
  }

  MaskDev md;
  md.kind = mask ? mask->kind : 0;
  md.log2_tile = mask ? mask->log2_tile : 0;
  md.stride = mask ? mask->stride : 1;
  md.phase = mask ? mask->phase : 0;
  md.bits = mask ? mask->d_bits : nullptr;

  if (fine_mask) {
    // finer than a kernel tile: every sector is touched anyway
    rc = launch_generic<DT>(ctx, d_ref, table, acc, K, 0, N, atol, rtol, md, count, st);
    if (rc != KB_OK) return rc;
  } else {
    const uint64_t nfull = N / kTile;
    StreamParams sp;
    sp.ref = d_ref;
    sp.cands = table;
    sp.acc = acc;
    sp.tile_list = mask ? mask->d_tiles : nullptr;
    sp.ntiles = mask ? mask->n_tiles : (uint32_t)nfull;
    sp.K = K;
    sp.K_dev = count;
    sp.atol = atol;
    sp.rtol = rtol;
    sp.rtol_lean = -1.0f;
    if (rtol >= 9.5367431640625e-07f) {   // 2^-20
      const double v = (double)rtol * (1.0 - 9.5367431640625e-07);
      float f = (float)v;
      if ((double)f > v) f = std::nextafterf(f, 0.0f);
      sp.rtol_lean = f;
    }
    sp.status = ctx->d_status;
    // Lead launch: a few leading tiles scouted exactly (about 1% of the work at most; the
    // streaming kernel starts behind them with its thresholds seeded), the ragged tail
    // (elements past the last full kernel tile) and the call's housekeeping.
    uint32_t nscout = 0;
    if (sp.ntiles >= 2) {
      nscout = sp.ntiles / 128;
      if (nscout < 1) nscout = 1;
      if (nscout > 8) nscout = 8;
    }
    const uint64_t tail0 = nfull * kTile;
    // small blocks spread a few candidates over the machine; with many candidates they would
    // only queue up, so each block then takes a whole kernel tile
    unsigned int per_block = kScoutPerBlock;
    if ((uint64_t)K * (nscout * (kTile / kScoutPerBlock) + 1u) > 32ull * ctx->sm_count) per_block = kTile;
    const unsigned int tail_blocks = (unsigned int)((N - tail0 + per_block - 1) / per_block);
    const unsigned int lead_blocks = nscout * (kTile / per_block) + tail_blocks;
    {
      LeadParams lp;
      lp.ref = d_ref;
      lp.table = table;
      lp.acc = acc;
      lp.acc_next = acc_next;
      lp.counters_next = counter_set(ctx, set ^ 1);
      lp.tile_list = sp.tile_list;
      lp.nscout = nscout;
      lp.n_clear = ctx->used_K[set ^ 1];
      lp.from_args = by_args ? 1u : 0u;
      lp.tail0 = tail0;
      lp.N = N;
      lp.atol = atol;
      lp.rtol = rtol;
      lp.mask = md;
      lp.count = count;
      // This call (set `set`) clears the previous call's accumulators (set ^ 1) and adds their
      // looks to sum[set]; sum[set ^ 1] holds the looks of the call before that (the last one on
      // `set`), added up by the previous lead kernel, and goes out with that call's steps.
      unsigned long long* sums = reinterpret_cast<unsigned long long*>(ctx->d_status + 20);
      lp.looks_sum = ctx->d_hint ? sums + set : nullptr;
      lp.looks_pub = sums + (set ^ 1);
      lp.hint = ctx->d_hint;
      lp.pub_steps = ctx->steps_hist[set];
      lp.per_block = per_block;
      screen_lead_kernel<DT><<<dim3(lead_blocks ? lead_blocks : 1u, K), 256, 0, st>>>(lp, chunk);
      ++ctx->launches;
      KB_CUDA(ctx, cudaGetLastError());
      lead_ran = true;
    }
    sp.slot0 = nscout;
    sp.ntiles -= nscout;
    if (sp.ntiles) {
      // chunk the candidates: shared-memory accumulators hold kMaxKC of them, and
      // small tensors need more, smaller items to fill the machine
      uint32_t nchunks = (K + kMaxKC - 1) / kMaxKC;
      const uint64_t grid =
          ctx->forced_grid ? ctx->forced_grid : (DT == KB_F8E4M3 ? (unsigned long long)kCtas8 : 3ull) * ctx->sm_count;
      const uint64_t want_items = 8 * grid;
      if ((uint64_t)nchunks * sp.ntiles < want_items) {
        uint64_t nc = (want_items + sp.ntiles - 1) / sp.ntiles;
        const uint64_t max_nc = (K + 7) / 8;           // at least 8 candidates per chunk
        if (nc > max_nc) nc = max_nc;
        if (nc > nchunks) nchunks = (uint32_t)nc;
      }
      sp.KC = (K + nchunks - 1) / nchunks;
      sp.nchunks = (K + sp.KC - 1) / sp.KC;
      sp.done = counters;
      sp.sched = reinterpret_cast<unsigned long long*>(counters + 2);
      sp.out = d_out;
      rc = launch_stream<DT>(ctx, sp, st, lead_ran && !capturing);
      return rc == KB_OK ? finished() : rc;
    }
  }
  screen_finalize_kernel<<<(K + 127) / 128, 128, 0, st>>>(acc, d_out, K, count);
  ++ctx->launches;
  KB_CUDA(ctx, cudaGetLastError());
  return finished();
}

kb_status screen_dispatch(kb_ctx* ctx, const void* d_ref, const void* const* h_cands, uint32_t K,
                          uint64_t N, kb_dtype dtype, float atol, float rtol, const kb_mask* mask,
                          kb_screen_result* d_out, cudaStream_t st, const IndexedSel* sel = nullptr) {
  switch (dtype) {
    case KB_F32: return screen_impl<KB_F32>(ctx, d_ref, h_cands, K, N, atol, rtol, mask, d_out, st, sel);
    case KB_F16: return screen_impl<KB_F16>(ctx, d_ref, h_cands, K, N, atol, rtol, mask, d_out, st, sel);
    case KB_F8E4M3: return screen_impl<KB_F8E4M3>(ctx, d_ref, h_cands, K, N, atol, rtol, mask, d_out, st, sel);
    case KB_F8E5M2: return screen_impl<KB_F8E5M2>(ctx, d_ref, h_cands, K, N, atol, rtol, mask, d_out, st, sel);
    default: return screen_impl<KB_BF16>(ctx, d_ref, h_cands, K, N, atol, rtol, mask, d_out, st, sel);
  }
}

}  // namespace

extern "C" kb_status kb_screen(kb_ctx* ctx, const void* d_ref, const void* const* h_cands, uint32_t K,
                               uint64_t N, kb_dtype dtype, float atol, float rtol,
                               const kb_mask* mask, kb_screen_result* d_out, void* stream) {
  TraceRange trace("kb_screen");
  kb_status rc = validate_screen(ctx, d_ref, h_cands, K, N, dtype, atol, rtol, mask, d_out, true);
  if (rc != KB_OK) return rc;
  DeviceGuard g(ctx->device);
  return screen_dispatch(ctx, d_ref, h_cands, K, N, dtype, atol, rtol, mask, d_out,
                         reinterpret_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------------------
// kb_screen_f64: the gate in binary64
// ---------------------------------------------------------------------------
extern "C" kb_status kb_merge_ranges(kb_ctx* ctx, const kb_screen_result* d_parts, uint32_t R, uint32_t K,
                                     const uint64_t* h_first, kb_screen_result* d_out, void* stream) {
  TraceRange trace("kb_merge_ranges");
  if (!ctx) return KB_ERR_INVALID_ARG;
  if (!d_parts || !h_first || !d_out) return fail(ctx, KB_ERR_INVALID_ARG, "kb_merge_ranges: null pointer");
  if (R == 0 || R > (uint32_t)kMergeMaxParts)
    return fail(ctx, KB_ERR_INVALID_ARG, "kb_merge_ranges: R=%u outside [1, %d]", R, kMergeMaxParts);
  if (K == 0 || K > KB_MAX_K) return fail(ctx, KB_ERR_INVALID_ARG, "kb_merge_ranges: K=%u outside [1, %u]", K, KB_MAX_K);
  if ((reinterpret_cast<uintptr_t>(d_parts) & 7u) || (reinterpret_cast<uintptr_t>(d_out) & 7u))
    return fail(ctx, KB_ERR_ALIGNMENT, "kb_merge_ranges: records not 8-byte aligned");
  RangeFirsts f;
  for (uint32_t r = 0; r < (uint32_t)kMergeMaxParts; ++r) f.first[r] = 0ull;
  for (uint32_t r = 0; r < R; ++r) {
    if (r && h_first[r] <= h_first[r - 1])
      return fail(ctx, KB_ERR_INVALID_ARG, "kb_merge_ranges: the parts' first indices must ascend (part %u)", r);
    if (h_first[r] >= KB_MAX_N)
      return fail(ctx, KB_ERR_INVALID_ARG, "kb_merge_ranges: first index of part %u beyond the element limit", r);
    f.first[r] = h_first[r];
  }
  DeviceGuard g(ctx->device);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  merge_ranges_kernel<<<(K + 127) / 128, 128, 0, st>>>(d_parts, R, K, f, d_out);
  ++ctx->launches;
  KB_CUDA(ctx, cudaGetLastError());
  return KB_OK;
}

extern "C" kb_status kb_screen_f64(kb_ctx* ctx, const double* d_ref, const double* const* h_cands,
                                   uint32_t K, uint64_t N, double atol, double rtol,
                                   const kb_mask* mask, kb_screen_result_f64* d_out, void* stream) {
  TraceRange trace("kb_screen_f64");
  if (!ctx) return KB_ERR_INVALID_ARG;
  if (!d_ref || !h_cands || !d_out) return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen_f64: null pointer");
  if (K == 0 || K > KB_MAX_K) return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen_f64: K=%u outside [1, %u]", K, KB_MAX_K);
  if (N == 0 || N > KB_MAX_N) return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen_f64: N outside [1, 2^32]");
  if (!(atol >= 0.0) || !(rtol >= 0.0) || std::isinf(atol) || std::isinf(rtol))
    return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen_f64: atol and rtol must be finite and >= 0");
  if (mask && (mask->N != N || mask->ctx != ctx))
    return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen_f64: the mask was created for another N or context");
  if (!aligned16(d_ref)) return fail(ctx, KB_ERR_ALIGNMENT, "kb_screen_f64: reference not 16-byte aligned");
  if ((reinterpret_cast<uintptr_t>(d_out) & 7u) != 0)
    return fail(ctx, KB_ERR_ALIGNMENT, "kb_screen_f64: output not 8-byte aligned");
  for (uint32_t k = 0; k < K; ++k) {
    if (!h_cands[k]) return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen_f64: candidate %u is NULL", k);
    if (!aligned16(h_cands[k]))
      return fail(ctx, KB_ERR_ALIGNMENT, "kb_screen_f64: candidate %u not 16-byte aligned", k);
  }
  DeviceGuard g(ctx->device);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  kb_status rc = ensure_ws(ctx, K);
  if (rc != KB_OK) return rc;
  // its own accumulator region and counters, zeroed by its prep kernel: independent of the
  // binary32 gate's two sets
  Acc64* acc = reinterpret_cast<Acc64*>(ctx->ws + ws_acc64_offset(ctx->ws_cap_K));
  const void** table = reinterpret_cast<const void**>(ctx->ws + ws_table_offset(ctx->ws_cap_K));
  for (uint32_t off = 0; off < K; off += kPtrsPerLaunch) {
    PtrChunk ch;
    const uint32_t cnt = (K - off < (uint32_t)kPtrsPerLaunch) ? K - off : (uint32_t)kPtrsPerLaunch;
    memcpy(ch.p, h_cands + off, cnt * sizeof(void*));
    screen_prep64_kernel<<<(cnt + 127) / 128, 128, 0, st>>>(ch, table, acc, ctx->d_status + 1, off, cnt);
    ++ctx->launches;
    KB_CUDA(ctx, cudaGetLastError());
  }
  MaskDev md;
  md.kind = mask ? mask->kind : 0;
  md.log2_tile = mask ? mask->log2_tile : 0;
  md.stride = mask ? mask->stride : 1;
  md.phase = mask ? mask->phase : 0;
  md.bits = mask ? mask->d_bits : nullptr;
  auto generic = [&](uint64_t e0, uint64_t e1) -> kb_status {
    if (e1 <= e0) return KB_OK;
    uint64_t bx = (e1 - e0 + 255) / 256;
    const uint64_t cap = (uint64_t)ctx->sm_count * 8;
    if (bx > cap) bx = cap;
    dim3 grid((unsigned int)bx, K);
    screen_generic64_kernel<<<grid, 256, 0, st>>>(d_ref, table, acc, e0, e1, atol, rtol, md);
    ++ctx->launches;
    KB_CUDA(ctx, cudaGetLastError());
    return KB_OK;
  };
  if (mask && !mask->coarse) {
    if ((rc = generic(0, N)) != KB_OK) return rc;
  } else {
    const uint64_t nfull = N / kTile;
    uint32_t ntiles = mask ? mask->n_tiles : (uint32_t)nfull;
    const uint32_t* tile_list = mask ? mask->d_tiles : nullptr;
    uint32_t nscout = 0;
    if (ntiles >= 2) {
      nscout = ntiles / 128;
      if (nscout < 1) nscout = 1;
      if (nscout > 8) nscout = 8;
      dim3 sg(nscout * 4, K);
      screen_scout64_kernel<<<sg, 256, 0, st>>>(d_ref, table, acc, tile_list, atol, rtol);
      ++ctx->launches;
      KB_CUDA(ctx, cudaGetLastError());
    }
    if ((rc = generic(nfull * kTile, N)) != KB_OK) return rc;
    ntiles -= nscout;
    if (ntiles) {
      Stream64Params sp;
      sp.ref = d_ref;
      sp.cands = table;
      sp.acc = acc;
      sp.tile_list = tile_list;
      sp.nhalf = 2 * ntiles;
      sp.half0 = 2 * nscout;
      sp.K = K;
      uint32_t nchunks = (K + kMaxKC64 - 1) / kMaxKC64;
      const uint64_t grid_want = ctx->forced_grid ? ctx->forced_grid : 1ull * ctx->sm_count;
      const uint64_t want_items = 8 * grid_want;
      if ((uint64_t)nchunks * sp.nhalf < want_items) {
        uint64_t nc = (want_items + sp.nhalf - 1) / sp.nhalf;
        const uint64_t max_nc = (K + 7) / 8;
        if (nc > max_nc) nc = max_nc;
        if (nc > nchunks) nchunks = (uint32_t)nc;
      }
      sp.KC = (K + nchunks - 1) / nchunks;
      sp.nchunks = (K + sp.KC - 1) / sp.KC;
      sp.stages = kStages64;
      sp.atol = atol;
      sp.rtol = rtol;
      sp.status = ctx->d_status;
      sp.done = ctx->d_status + 1;
      sp.sched = reinterpret_cast<unsigned long long*>(ctx->d_status + 2);
      sp.out = d_out;
      const unsigned long long nitems = (unsigned long long)sp.nchunks * sp.nhalf;
      unsigned long long grid = grid_want;
      if (grid > nitems) grid = nitems;
      {
        ScopedTimer tm(ctx, KB_TIMER_SCREEN_STREAM, st);
        screen_stream64_kernel<<<(unsigned int)grid, kStreamThreads, stream64_smem_bytes(kStages64), st>>>(sp);
      }
      ++ctx->launches;
      KB_CUDA(ctx, cudaGetLastError());
      return KB_OK;
    }
  }
  screen_finalize64_kernel<<<(K + 127) / 128, 128, 0, st>>>(acc, d_out, K);
  ++ctx->launches;
  KB_CUDA(ctx, cudaGetLastError());
  return KB_OK;
}

extern "C" kb_status kb_screen_indexed(kb_ctx* ctx, const void* d_ref, const void* const* d_table,
                                       uint32_t K_all, const int32_t* d_index,
                                       const uint32_t* d_count, uint32_t Kmax, uint64_t N,
                                       kb_dtype dtype, float atol, float rtol, const kb_mask* mask,
                                       kb_screen_result* d_out, void* stream) {
  TraceRange trace("kb_screen_indexed");
  if (!ctx) return KB_ERR_INVALID_ARG;
  if (!d_ref || !d_table || !d_index || !d_count || !d_out)
    return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen_indexed: null pointer");
  if (Kmax == 0 || Kmax > 1024) return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen_indexed: Kmax=%u outside [1, 1024]", Kmax);
  if (K_all == 0) return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen_indexed: K_all is 0");
  if (N == 0 || N > KB_MAX_N) return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen_indexed: N outside [1, 2^32]");
  if (!known_dtype((int)dtype))
    return fail(ctx, KB_ERR_UNSUPPORTED, "kb_screen_indexed: unknown dtype %d", (int)dtype);
  if (!(atol >= 0.0f) || !(rtol >= 0.0f) || std::isinf(atol) || std::isinf(rtol))
    return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen_indexed: atol and rtol must be finite and >= 0");
  if (mask && (mask->N != N || mask->ctx != ctx))
    return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen_indexed: the mask was created for another N or context");
  if (!aligned16(d_ref)) return fail(ctx, KB_ERR_ALIGNMENT, "kb_screen_indexed: reference not 16-byte aligned");
  if ((reinterpret_cast<uintptr_t>(d_out) & 7u) != 0)
    return fail(ctx, KB_ERR_ALIGNMENT, "kb_screen_indexed: output not 8-byte aligned");
  DeviceGuard g(ctx->device);
  IndexedSel sel{d_table, K_all, d_index, d_count};
  return screen_dispatch(ctx, d_ref, nullptr, Kmax, N, dtype, atol, rtol, mask, d_out,
                         reinterpret_cast<cudaStream_t>(stream), &sel);
}

extern "C" kb_status kb_screen_multi(kb_ctx* ctx, uint32_t G, const void* const* h_refs,
                                     const void* const* h_cands, const uint32_t* h_K,
                                     const uint64_t* h_N, kb_dtype dtype, float atol, float rtol,
                                     kb_screen_result* d_out, void* stream) {
  TraceRange trace("kb_screen_multi");
  if (!ctx) return KB_ERR_INVALID_ARG;
  if (!h_refs || !h_cands || !h_K || !h_N || !d_out)
    return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen_multi: null pointer");
  if (G == 0 || G > (uint32_t)kMultiMaxGroups)
    return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen_multi: G=%u outside [1, %d]", G, kMultiMaxGroups);
  if (!known_dtype((int)dtype))
    return fail(ctx, KB_ERR_UNSUPPORTED, "kb_screen_multi: unknown dtype %d", (int)dtype);
  if (!(atol >= 0.0f) || !(rtol >= 0.0f) || std::isinf(atol) || std::isinf(rtol))
    return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen_multi: atol and rtol must be finite and >= 0");
  if ((reinterpret_cast<uintptr_t>(d_out) & 7u) != 0)
    return fail(ctx, KB_ERR_ALIGNMENT, "kb_screen_multi: output not 8-byte aligned");
  if (!ctx->small_ws) return fail(ctx, KB_ERR_WORKSPACE, "kb_screen_multi: this context has no small-problem workspace");
  static thread_local MultiParams mp;   // 12 KB: kept off the stack
  uint32_t rows = 0;
  uint64_t blocks = 0;
  for (uint32_t g = 0; g < G; ++g) {
    if (!h_refs[g] || h_K[g] == 0 || h_N[g] == 0 || h_N[g] > KB_MAX_N)
      return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen_multi: group %u has a null reference, K = 0 or a bad N", g);
    if (!aligned16(h_refs[g])) return fail(ctx, KB_ERR_ALIGNMENT, "kb_screen_multi: reference %u not 16-byte aligned", g);
    mp.ref[g] = h_refs[g];
    mp.N[g] = h_N[g];
    const uint64_t nb = (h_N[g] + kSmallPerBlock - 1) / kSmallPerBlock;
    for (uint32_t k = 0; k < h_K[g]; ++k) {
      if (rows >= (uint32_t)kMultiMaxRows || blocks + nb > kSmallMaxPartials)
        return fail(ctx, KB_ERR_UNSUPPORTED,
                    "kb_screen_multi: more than %d candidates or %zu blocks of 1024 elements; "
                    "call kb_screen per group", kMultiMaxRows, kSmallMaxPartials);
      const void* c = h_cands[rows];
      if (!c) return fail(ctx, KB_ERR_INVALID_ARG, "kb_screen_multi: candidate %u is NULL", rows);
      if (!aligned16(c)) return fail(ctx, KB_ERR_ALIGNMENT, "kb_screen_multi: candidate %u not 16-byte aligned", rows);
      mp.cand[rows] = c;
      mp.group[rows] = (unsigned char)g;
      mp.first_block[rows] = (unsigned int)blocks;
      blocks += nb;
      ++rows;
    }
  }
  mp.first_block[rows] = (unsigned int)blocks;
  mp.rows = rows;
  mp.tickets = reinterpret_cast<unsigned int*>(ctx->small_ws);
  mp.partials = reinterpret_cast<Acc*>(ctx->small_ws + kSmallTicketBytes);
  mp.out = d_out;
  mp.atol = atol;
  mp.rtol = rtol;
  DeviceGuard gd(ctx->device);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  switch (dtype) {
    case KB_F32: screen_multi_kernel<KB_F32><<<(unsigned int)blocks, 256, 0, st>>>(mp); break;
    case KB_F16: screen_multi_kernel<KB_F16><<<(unsigned int)blocks, 256, 0, st>>>(mp); break;
    case KB_F8E4M3: screen_multi_kernel<KB_F8E4M3><<<(unsigned int)blocks, 256, 0, st>>>(mp); break;
    case KB_F8E5M2: screen_multi_kernel<KB_F8E5M2><<<(unsigned int)blocks, 256, 0, st>>>(mp); break;
    default: screen_multi_kernel<KB_BF16><<<(unsigned int)blocks, 256, 0, st>>>(mp); break;
  }
  ++ctx->launches;
  KB_CUDA(ctx, cudaGetLastError());
  return KB_OK;
}

// ---------------------------------------------------------------------------
// kb_screen_static: the gate without any allocation
// ---------------------------------------------------------------------------

// Scratch of the allocation-free entry point: [status words and counters 256 B | two sets of
// accumulators | pointer table].  In host code this name is only a handle for cudaGetSymbolAddress; it is not a
// device address and must never be passed to a kernel as it stands.
static __device__ __align__(256) unsigned char g_static_scratch[KB_STATIC_SCRATCH_BYTES];
static_assert(KB_STATIC_SCRATCH_BYTES == 256 + 2 * KB_STATIC_MAX_K * sizeof(Acc) + KB_STATIC_MAX_K * sizeof(void*),
              "the header's scratch size must match the accumulator layout");

namespace {

constexpr int kStaticMaxDevices = 64;
struct StaticSlot {
  bool ready = false;
  kb_ctx ctx;   // a host-side view over the static array; owns nothing, is never destroyed
};
StaticSlot g_static_slot[kStaticMaxDevices];
std::mutex g_static_mutex;

// Once per device, with that device current: resolve the array's device address, read the
// SM count, raise the kernels' shared-memory limits.  None of these allocates.
// (the caller holds g_static_mutex)
kb_status static_setup(int device, kb_ctx** out) {
  StaticSlot& slot = g_static_slot[device];
  if (!slot.ready) {
    kb_ctx* ctx = &slot.ctx;
    ctx->device = device;
    unsigned char* base = nullptr;
    KB_CUDA(ctx, cudaGetSymbolAddress(reinterpret_cast<void**>(&base), g_static_scratch));
    int sms = 0;
    KB_CUDA(ctx, cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    ctx->sm_count = sms;
    ctx->d_status = reinterpret_cast<unsigned int*>(base);
    ctx->ws = base + 256;
    ctx->ws_bytes = KB_STATIC_SCRATCH_BYTES - 256;   // ensure_ws never grows it: K is capped
    ctx->ws_cap_K = KB_STATIC_MAX_K;
    ctx->ws_fixed = true;
    kb_status st;
    if ((st = set_stream_attr<KB_F32>(ctx)) != KB_OK) return st;
    if ((st = set_stream_attr<KB_F16>(ctx)) != KB_OK) return st;
    if ((st = set_stream_attr<KB_BF16>(ctx)) != KB_OK) return st;
    if ((st = set_stream_attr<KB_F8E4M3>(ctx)) != KB_OK) return st;
    if ((st = set_stream_attr<KB_F8E5M2>(ctx)) != KB_OK) return st;
    slot.ready = true;
  }
  *out = &slot.ctx;
  return KB_OK;
}

}  // namespace

extern "C" kb_status kb_screen_static(const void* d_ref, const void* const* h_cands, uint32_t K,
                                      uint64_t N, kb_dtype dtype, float atol, float rtol,
                                      kb_screen_result* d_out, void* stream) {
  TraceRange trace("kb_screen_static");
  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kStaticMaxDevices) {
    cudaGetLastError();
    snprintf(g_create_err, sizeof g_create_err, "kb_screen_static: no usable current CUDA device");
    return KB_ERR_CUDA;
  }
  if (K > KB_STATIC_MAX_K) {
    snprintf(g_create_err, sizeof g_create_err,
             "kb_screen_static: K=%u exceeds the %u candidates the static scratch holds "
             "(use kb_screen, which may allocate)", K, KB_STATIC_MAX_K);
    return KB_ERR_WORKSPACE;
  }
  // One host thread at a time validates and enqueues: all callers on a device share the
  // slot's error text and launch counter as well as the scratch array.
  std::lock_guard<std::mutex> lock(g_static_mutex);
  kb_ctx* ctx = nullptr;
  kb_status rc = static_setup(device, &ctx);
  if (rc == KB_OK) rc = validate_screen(ctx, d_ref, h_cands, K, N, dtype, atol, rtol, nullptr, d_out, true);
  if (rc == KB_OK) {
    // The array is shared by every caller on the device and keeps what the last call left:
    // nothing is taken on trust, the part this call uses is cleared first.
    ctx->ws_dirty = true;
  }
  if (rc == KB_OK)
    rc = screen_dispatch(ctx, d_ref, h_cands, K, N, dtype, atol, rtol, nullptr, d_out,
                         reinterpret_cast<cudaStream_t>(stream));
  if (rc != KB_OK) snprintf(g_create_err, sizeof g_create_err, "%.250s", g_static_slot[device].ctx.err);
  return rc;
}

extern "C" kb_status kb_static_scratch_read(void* h_dst, uint32_t bytes) {
  if (!h_dst || bytes > KB_STATIC_SCRATCH_BYTES) return KB_ERR_INVALID_ARG;
  if (cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpyFromSymbol(h_dst, g_static_scratch, bytes, 0, cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return KB_ERR_CUDA;
  }
  return KB_OK;
}

extern "C" kb_status kb_screen_host(kb_ctx* ctx, const void* h_ref, const void* const* h_cands_host,
                                    uint32_t K, uint64_t N, kb_dtype dtype, float atol, float rtol,
                                    const kb_mask* mask, kb_screen_result* h_out, void* stream) {
  TraceRange trace("kb_screen_host");
  kb_status rc = validate_screen(ctx, h_ref, h_cands_host, K, N, dtype, atol, rtol, mask, h_out, false);
  if (rc != KB_OK) return rc;
  DeviceGuard g(ctx->device);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const size_t bytes = (size_t)N * elem_bytes(dtype);
  const size_t pitch = round_up(bytes, 256);
  // batch size: about 512 MiB of candidates per batch, two batches in flight
  uint32_t B = (uint32_t)((512ull << 20) / pitch);
  if (B < 1) B = 1;
  if (B > K) B = K;
  if (!ctx->copy_stream) {
    KB_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking));
    for (int i = 0; i < 2; ++i) {
      KB_CUDA(ctx, cudaEventCreateWithFlags(&ctx->ev_copied[i], cudaEventDisableTiming));
      KB_CUDA(ctx, cudaEventCreateWithFlags(&ctx->ev_done[i], cudaEventDisableTiming));
    }
  }
  if ((rc = ensure_buf(ctx, &ctx->st_ref, &ctx->st_ref_bytes, pitch)) != KB_OK) return rc;
  for (int i = 0; i < 2; ++i)
    if ((rc = ensure_buf(ctx, &ctx->st_batch[i], &ctx->st_batch_bytes[i], (size_t)B * pitch)) != KB_OK) return rc;
  if ((rc = ensure_buf(ctx, &ctx->st_out, &ctx->st_out_bytes, (size_t)K * sizeof(kb_screen_result))) != KB_OK)
    return rc;

  // order the copy stream after work already enqueued on the caller's stream
  KB_CUDA(ctx, cudaEventRecord(ctx->ev_done[0], st));
  KB_CUDA(ctx, cudaEventRecord(ctx->ev_done[1], st));
  KB_CUDA(ctx, cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_done[0], 0));
  KB_CUDA(ctx, cudaMemcpyAsync(ctx->st_ref, h_ref, bytes, cudaMemcpyHostToDevice, ctx->copy_stream));
  std::vector<const void*> ptrs(B);
  int buf = 0;
  for (uint32_t k0 = 0; k0 < K; k0 += B, buf ^= 1) {
    const uint32_t nb = (K - k0 < B) ? K - k0 : B;
    KB_CUDA(ctx, cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_done[buf], 0));
    for (uint32_t i = 0; i < nb; ++i) {
      unsigned char* dst = ctx->st_batch[buf] + (size_t)i * pitch;
      KB_CUDA(ctx, cudaMemcpyAsync(dst, h_cands_host[k0 + i], bytes, cudaMemcpyHostToDevice, ctx->copy_stream));
      ptrs[i] = dst;
    }
    KB_CUDA(ctx, cudaEventRecord(ctx->ev_copied[buf], ctx->copy_stream));
    KB_CUDA(ctx, cudaStreamWaitEvent(st, ctx->ev_copied[buf], 0));
    rc = screen_dispatch(ctx, ctx->st_ref, ptrs.data(), nb, N, dtype, atol, rtol, mask, ctx->st_out + k0, st);
    if (rc != KB_OK) return rc;
    KB_CUDA(ctx, cudaEventRecord(ctx->ev_done[buf], st));
  }
  KB_CUDA(ctx, cudaMemcpyAsync(h_out, ctx->st_out, (size_t)K * sizeof(kb_screen_result),
                               cudaMemcpyDeviceToHost, st));
  KB_CUDA(ctx, cudaStreamSynchronize(st));
  return KB_OK;
}

// ---------------------------------------------------------------------------
// kb_adjudicate
// ---------------------------------------------------------------------------

extern "C" kb_status kb_adjudicate(kb_ctx* ctx, const float* d_timings, uint32_t K, uint32_t S,
                                   float* d_median, float* d_iqr, uint32_t* d_wins, void* stream) {
  TraceRange trace("kb_adjudicate");
  if (!ctx) return KB_ERR_INVALID_ARG;
  if (!d_timings) return fail(ctx, KB_ERR_INVALID_ARG, "kb_adjudicate: timings is NULL");
  if (K == 0 || K > KB_MAX_K) return fail(ctx, KB_ERR_INVALID_ARG, "kb_adjudicate: K=%u outside [1, %u]", K, KB_MAX_K);
  if (S == 0 || S > KB_MAX_S) return fail(ctx, KB_ERR_INVALID_ARG, "kb_adjudicate: S=%u outside [1, %u]", S, KB_MAX_S);
  if ((reinterpret_cast<uintptr_t>(d_timings) & 3u) || (reinterpret_cast<uintptr_t>(d_median) & 3u) ||
      (reinterpret_cast<uintptr_t>(d_iqr) & 3u) || (reinterpret_cast<uintptr_t>(d_wins) & 3u))
    return fail(ctx, KB_ERR_ALIGNMENT, "kb_adjudicate: a pointer is not 4-byte aligned");
  DeviceGuard g(ctx->device);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);

  // which win-count algorithm
  bool rank = d_wins && S <= 4096 && ctx->wins_algo != 1;
  if (ctx->wins_algo == 2 && d_wins && S > 4096)
    return fail(ctx, KB_ERR_UNSUPPORTED, "kb_adjudicate: the binary-search win count needs S <= 4096");
  if (ctx->wins_algo == 3 && d_wins && S > kMergeMaxS)
    return fail(ctx, KB_ERR_UNSUPPORTED, "kb_adjudicate: the merge win count needs S <= %u", kMergeMaxS);
  if (rank && ensure_buf(ctx, &ctx->srt, &ctx->srt_bytes, (size_t)K * S * sizeof(float), "sorted timings") != KB_OK) {
    if (ctx->wins_algo >= 2) return KB_ERR_WORKSPACE;
    rank = false;     // no room for the sorted copy: count by direct comparison
  }
  // rows: sort + quartiles (also the place where non-finite timings are caught)
  unsigned int P = 1;
  while (P < S) P <<= 1;
  rows_kernel<<<K, kRowsThreads, (size_t)P * sizeof(float), st>>>(d_timings, S, P, d_median, d_iqr,
                                                                   rank ? ctx->srt : nullptr,
                                                                   ctx->d_status);
  ++ctx->launches;
  KB_CUDA(ctx, cudaGetLastError());
  if (!d_wins) return KB_OK;

  // many candidates with short rows: one warp walks a row against 32 rows at once
  const unsigned int nT = (K + kMergeTile - 1) / kMergeTile;
  if (rank && S <= kMergeMaxS && (ctx->wins_algo == 3 || (ctx->wins_algo == 0 && nT >= 8))) {
    WinsMergeParams mp;
    mp.sorted = ctx->srt;
    mp.wins = d_wins;
    mp.K = K;
    mp.S = S;
    mp.stride = (S + 1) | 1u;
    mp.nT = nT;
    const unsigned long long grid_m = (unsigned long long)nT * (nT + 1) / 2 * (kMergeTile / kMergeARows);
    if (grid_m > 0x7FFFFFFFull) return fail(ctx, KB_ERR_UNSUPPORTED, "kb_adjudicate: K too large for one launch");
    {
      ScopedTimer tm(ctx, KB_TIMER_WINS, st);
      wins_merge_kernel<<<(unsigned int)grid_m, 256,
                          (size_t)(kMergeTile + kMergeARows) * mp.stride * sizeof(float), st>>>(mp);
    }
    ++ctx->launches;
    KB_CUDA(ctx, cudaGetLastError());
    return KB_OK;
  }

  if (rank) {
    WinsRankParams rp;
    rp.sorted = ctx->srt;
    rp.wins = d_wins;
    rp.K = K;
    rp.S = S;
    rp.P = 1;
    while (rp.P <= S) rp.P <<= 1;
    rp.KB = (K + kWinsRowsPerBlock - 1) / kWinsRowsPerBlock;
    const unsigned long long npairs_r = (unsigned long long)rp.KB * (rp.KB + 1) / 2;
    rp.TA = kWinsRowsPerBlock;
    while (npairs_r * (kWinsRowsPerBlock / rp.TA) < 8ull * ctx->sm_count && rp.TA > 1) rp.TA /= 2;
    const unsigned long long grid_r = npairs_r * (kWinsRowsPerBlock / rp.TA);
    if (grid_r > 0x7FFFFFFFull) return fail(ctx, KB_ERR_UNSUPPORTED, "kb_adjudicate: K too large for one launch");
    {
      ScopedTimer tm(ctx, KB_TIMER_WINS, st);
      wins_rank_kernel<<<(unsigned int)grid_r, kWinsThreads,
                         (size_t)kWinsRowsPerBlock * S * sizeof(float), st>>>(rp);
    }
    ++ctx->launches;
    KB_CUDA(ctx, cudaGetLastError());
    return KB_OK;
  }

  WinsParams wp;
  wp.timings = d_timings;
  wp.wins = d_wins;
  wp.K = K;
  wp.S = S;
  wp.KB = (K + kWinsRowsPerBlock - 1) / kWinsRowsPerBlock;
  const unsigned long long npairs = (unsigned long long)wp.KB * (wp.KB + 1) / 2;
  wp.npairs = (unsigned int)npairs;
  wp.nj = (S + 32 * kWinsMaxR - 1) / (32 * kWinsMaxR);
  const unsigned int per_chunk = (S + wp.nj - 1) / wp.nj;
  const int R = (int)((per_chunk + 31) / 32);
  wp.JC = 32u * R;
  wp.IC = (unsigned int)round_up(S < 1024 ? S : 1024, 4);
  wp.ni = (S + wp.IC - 1) / wp.IC;
  // small problems: fewer a rows per CTA, then shorter a chunks, until the machine is filled
  wp.TA = kWinsRowsPerBlock;
  auto items = [&]() { return npairs * (kWinsRowsPerBlock / wp.TA) * wp.nj * wp.ni; };
  while (items() < 2ull * ctx->sm_count && wp.TA > 1) wp.TA /= 2;
  while (items() < (unsigned long long)ctx->sm_count && wp.IC > 256) {
    wp.IC = (unsigned int)round_up((wp.IC + 1) / 2, 4);
    wp.ni = (S + wp.IC - 1) / wp.IC;
  }
  wp.direct = (wp.ni == 1 && wp.nj == 1) ? 1u : 0u;
  if (items() > 0x7FFFFFFFull) return fail(ctx, KB_ERR_UNSUPPORTED, "kb_adjudicate: K*S too large for one launch");
  if (!wp.direct) KB_CUDA(ctx, cudaMemsetAsync(d_wins, 0, (size_t)K * K * sizeof(uint32_t), st));
  const size_t smem = (size_t)wp.TA * wp.IC * sizeof(float);
  const unsigned int grid = (unsigned int)items();
  {
    ScopedTimer tm(ctx, KB_TIMER_WINS, st);
    switch (R) {
      case 1: launch_wins<1>(wp, grid, smem, st); break;
      case 2: launch_wins<2>(wp, grid, smem, st); break;
      case 3: launch_wins<3>(wp, grid, smem, st); break;
      case 4: launch_wins<4>(wp, grid, smem, st); break;
      case 5: launch_wins<5>(wp, grid, smem, st); break;
      case 6: launch_wins<6>(wp, grid, smem, st); break;
      case 7: launch_wins<7>(wp, grid, smem, st); break;
      default: launch_wins<8>(wp, grid, smem, st); break;
    }
  }
  ++ctx->launches;
  KB_CUDA(ctx, cudaGetLastError());
  return KB_OK;
}

// ---------------------------------------------------------------------------
// kb_select
// ---------------------------------------------------------------------------

extern "C" kb_status kb_select(kb_ctx* ctx, const kb_screen_result* d_screen, const float* d_median,
                               uint32_t K, kb_select_policy policy, uint32_t budget,
                               int32_t* d_survivors, uint32_t* d_n_survivors, void* stream) {
  TraceRange trace("kb_select");
  if (!ctx) return KB_ERR_INVALID_ARG;
  if (!d_screen || !d_median || !d_survivors || !d_n_survivors)
    return fail(ctx, KB_ERR_INVALID_ARG, "kb_select: null pointer");
  if (K == 0 || K > KB_MAX_K) return fail(ctx, KB_ERR_INVALID_ARG, "kb_select: K=%u outside [1, %u]", K, KB_MAX_K);
  if (budget == 0) return fail(ctx, KB_ERR_INVALID_ARG, "kb_select: budget must be >= 1");
  if (policy != KB_SELECT_ERR_THEN_TIME && policy != KB_SELECT_TIME)
    return fail(ctx, KB_ERR_UNSUPPORTED, "kb_select: unknown policy %d", (int)policy);
  DeviceGuard g(ctx->device);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  select_kernel<<<(K + kSelectThreads - 1) / kSelectThreads, kSelectThreads, 0, st>>>(
      d_screen, d_median, K, (int)policy, budget, d_survivors, d_n_survivors);
  ++ctx->launches;
  KB_CUDA(ctx, cudaGetLastError());
  return KB_OK;
}

// ---------------------------------------------------------------------------
// scheduler-side statistics
// ---------------------------------------------------------------------------

extern "C" kb_status kb_select_by_score(kb_ctx* ctx, const kb_screen_result* d_screen,
                                        const float* d_median, uint32_t K, uint32_t rung,
                                        uint32_t rung_budget, float alpha, float beta,
                                        uint32_t budget, float* d_score, int32_t* d_survivors,
                                        uint32_t* d_n_survivors, void* stream) {
  TraceRange trace("kb_select_by_score");
  if (!ctx) return KB_ERR_INVALID_ARG;
  if (!d_screen || !d_median || !d_survivors || !d_n_survivors)
    return fail(ctx, KB_ERR_INVALID_ARG, "kb_select_by_score: null pointer");
  if (K == 0 || K > KB_MAX_K) return fail(ctx, KB_ERR_INVALID_ARG, "kb_select_by_score: K=%u outside [1, %u]", K, KB_MAX_K);
  if (budget == 0) return fail(ctx, KB_ERR_INVALID_ARG, "kb_select_by_score: budget must be >= 1");
  if (!std::isfinite(alpha) || !std::isfinite(beta))
    return fail(ctx, KB_ERR_INVALID_ARG, "kb_select_by_score: alpha and beta must be finite");
  DeviceGuard g(ctx->device);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  // gamma(r) = (alpha*r) + (beta*b_r), each operation in binary32 (host floats are IEEE binary32)
  volatile float ga = alpha * (float)rung;
  volatile float gb = beta * (float)rung_budget;
  const float gamma = ga + gb;
  select_by_score_kernel<<<(K + kSelectThreads - 1) / kSelectThreads, kSelectThreads, 0, st>>>(
      d_screen, d_median, K, gamma, budget, d_score, d_survivors, d_n_survivors);
  ++ctx->launches;
  KB_CUDA(ctx, cudaGetLastError());
  return KB_OK;
}

extern "C" kb_status kb_tail_ratios(kb_ctx* ctx, const float* d_timings, uint32_t K, uint32_t S,
                                    float* d_ratios, void* stream) {
  TraceRange trace("kb_tail_ratios");
  if (!ctx) return KB_ERR_INVALID_ARG;
  if (!d_timings || !d_ratios) return fail(ctx, KB_ERR_INVALID_ARG, "kb_tail_ratios: null pointer");
  if (K == 0 || K > KB_MAX_K) return fail(ctx, KB_ERR_INVALID_ARG, "kb_tail_ratios: K=%u outside [1, %u]", K, KB_MAX_K);
  if (S == 0 || S > KB_MAX_S) return fail(ctx, KB_ERR_INVALID_ARG, "kb_tail_ratios: S=%u outside [1, %u]", S, KB_MAX_S);
  DeviceGuard g(ctx->device);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  unsigned int P = 1;
  while (P < S) P <<= 1;
  tails_kernel<<<K, kRowsThreads, (size_t)P * sizeof(float), st>>>(d_timings, S, P, d_ratios, ctx->d_status);
  ++ctx->launches;
  KB_CUDA(ctx, cudaGetLastError());
  return KB_OK;
}

extern "C" kb_status kb_copeland(kb_ctx* ctx, const uint32_t* d_wins, uint32_t K, uint32_t S,
                                 uint32_t* d_beats, uint32_t* d_ties, void* stream) {
  TraceRange trace("kb_copeland");
  if (!ctx) return KB_ERR_INVALID_ARG;
  if (!d_wins || !d_beats) return fail(ctx, KB_ERR_INVALID_ARG, "kb_copeland: null pointer");
  if (K == 0 || K > KB_MAX_K) return fail(ctx, KB_ERR_INVALID_ARG, "kb_copeland: K=%u outside [1, %u]", K, KB_MAX_K);
  if (S == 0 || S > KB_MAX_S) return fail(ctx, KB_ERR_INVALID_ARG, "kb_copeland: S=%u outside [1, %u]", S, KB_MAX_S);
  DeviceGuard g(ctx->device);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  copeland_kernel<<<(K + 7) / 8, 256, 0, st>>>(d_wins, K, S, d_beats, d_ties);
  ++ctx->launches;
  KB_CUDA(ctx, cudaGetLastError());
  return KB_OK;
}

extern "C" kb_status kb_confirm(kb_ctx* ctx, const float* d_first, const float* d_second,
                                const float* d_prev, uint32_t K, float threshold,
                                uint32_t* d_status, float* d_score, void* stream) {
  TraceRange trace("kb_confirm");
  if (!ctx) return KB_ERR_INVALID_ARG;
  if (!d_first || !d_second || !d_prev || !d_status || !d_score)
    return fail(ctx, KB_ERR_INVALID_ARG, "kb_confirm: null pointer");
  if (K == 0 || K > KB_MAX_K) return fail(ctx, KB_ERR_INVALID_ARG, "kb_confirm: K=%u outside [1, %u]", K, KB_MAX_K);
  if (!std::isfinite(threshold)) return fail(ctx, KB_ERR_INVALID_ARG, "kb_confirm: threshold must be finite");
  DeviceGuard g(ctx->device);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  confirm_kernel<<<(K + 255) / 256, 256, 0, st>>>(d_first, d_second, d_prev, K, threshold, d_status, d_score);
  ++ctx->launches;
  KB_CUDA(ctx, cudaGetLastError());
  return KB_OK;
}

extern "C" kb_status kb_adjudicate_ragged(kb_ctx* ctx, const float* d_timings,
                                          const uint32_t* d_offsets, uint32_t K, uint32_t S_max,
                                          uint64_t total, float* d_median, float* d_iqr,
                                          uint32_t* d_wins, void* stream) {
  TraceRange trace("kb_adjudicate_ragged");
  if (!ctx) return KB_ERR_INVALID_ARG;
  if (!d_timings || !d_offsets) return fail(ctx, KB_ERR_INVALID_ARG, "kb_adjudicate_ragged: null pointer");
  if (K == 0 || K > KB_MAX_K) return fail(ctx, KB_ERR_INVALID_ARG, "kb_adjudicate_ragged: K=%u outside [1, %u]", K, KB_MAX_K);
  if (S_max == 0 || S_max > 4096) return fail(ctx, KB_ERR_INVALID_ARG, "kb_adjudicate_ragged: S_max=%u outside [1, 4096]", S_max);
  if (total == 0 || total > (uint64_t)K * S_max)
    return fail(ctx, KB_ERR_INVALID_ARG, "kb_adjudicate_ragged: total sample count outside [1, K*S_max]");
  DeviceGuard g(ctx->device);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  float* srt = nullptr;
  if (d_wins) {
    kb_status rc = ensure_buf(ctx, &ctx->srt, &ctx->srt_bytes, (size_t)total * sizeof(float), "sorted timings");
    if (rc != KB_OK) return rc;
    srt = ctx->srt;
  }
  unsigned int P = 1;
  while (P < S_max) P <<= 1;
  rows_ragged_kernel<<<K, kRowsThreads, (size_t)P * sizeof(float), st>>>(d_timings, d_offsets, S_max, d_median,
                                                                          d_iqr, srt, ctx->d_status);
  ++ctx->launches;
  KB_CUDA(ctx, cudaGetLastError());
  if (!d_wins) return KB_OK;
  WinsRaggedParams rp;
  rp.sorted = srt;
  rp.offsets = d_offsets;
  rp.wins = d_wins;
  rp.K = K;
  rp.S_max = S_max;
  rp.KB = (K + kWinsRowsPerBlock - 1) / kWinsRowsPerBlock;
  const unsigned long long npairs = (unsigned long long)rp.KB * (rp.KB + 1) / 2;
  rp.TA = kWinsRowsPerBlock;
  while (npairs * (kWinsRowsPerBlock / rp.TA) < 8ull * ctx->sm_count && rp.TA > 1) rp.TA /= 2;
  const unsigned long long grid = npairs * (kWinsRowsPerBlock / rp.TA);
  if (grid > 0x7FFFFFFFull) return fail(ctx, KB_ERR_UNSUPPORTED, "kb_adjudicate_ragged: K too large for one launch");
  {
    ScopedTimer tm(ctx, KB_TIMER_WINS, st);
    wins_ragged_kernel<<<(unsigned int)grid, kWinsThreads, (size_t)kWinsRowsPerBlock * S_max * sizeof(float), st>>>(rp);
  }
  ++ctx->launches;
  KB_CUDA(ctx, cudaGetLastError());
  return KB_OK;
}
