/*
 * kb_hooks.h -- test, tuning and instrumentation hooks of the kb library.
 *
 * None of these is part of the method (the paper has no counterpart for any of
 * them): they force a dispatch path or a grid size so that tests can show that
 * results do not depend on it, time the two dominant kernels with CUDA events
 * for the benchmark, count launches, and exercise failure paths (a device-side
 * wait that runs out, a workspace allocation that fails) without faulting a GPU.
 * A user of the library needs only kb.h.
 */
#ifndef KB_HOOKS_H_
#define KB_HOOKS_H_

#include "kb.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Test/tuning hook: force the number of thread blocks of the streaming screen
 * kernel (0 = automatic).  Results do not depend on it. */
kb_status kb_ctx_set_grid(kb_ctx* ctx, uint32_t blocks);

/* Test/tuning hook: small problems (K <= 480 and K*N <= 2^22 elements) are
 * screened by a single-launch kernel; on = 0 sends them down the general
 * (streaming) path instead.  Results do not depend on it. */
kb_status kb_ctx_set_small_path(kb_ctx* ctx, int on);

/* Test/tuning hook: the streaming screen kernel is launched as a programmatic dependent of the
 * lead kernel in front of it (its CTAs are set up while the lead kernel still runs and wait
 * for it before they read anything); on = 0 launches it in plain stream order.  Never used
 * while the stream is being captured into a graph.  Results do not depend on it. */
kb_status kb_ctx_set_dependent_launch(kb_ctx* ctx, int on);

/* Test/tuning hook: which instantiation of the streaming screen kernel runs.  0 = automatic:
 * the plain one, until a call reports that a quarter of its steps took a second look that
 * found nothing.  If those looks came while the candidate was lean (many elements whose
 * quotient was rounded down to the largest relative error, e.g. dense one-ulp differences)
 * the next 32 calls use the SHARP instantiation, which applies the sharper test to every
 * element; if they came beyond the lean bound (elements that pass by atol alone, e.g.
 * candidates that differ by absolute noise where the reference is near zero) they use the BY
 * DEFINITION instantiation, which there tests every element against its own tolerance.  A
 * plain call every 32 calls checks whether the report still holds.
 * 1 = always plain, 2 = always sharp, 3 = always by definition.  Results do not depend on it. */
kb_status kb_ctx_set_filter(kb_ctx* ctx, int mode);
/* The instantiation of this context's last streaming launch (HOST out): 0 plain, 1 sharp,
 * 3 by definition. */
kb_status kb_ctx_last_filter(const kb_ctx* ctx, int* mode);

/* ---- instrumentation (used by the benchmark) ------------------------------ */

typedef enum {
  KB_TIMER_SCREEN_STREAM = 0, /* the streaming screen kernel */
  KB_TIMER_WINS = 1           /* the pairwise win-count kernel */
} kb_timer;

/* With timing on, every launch of the two kernels above is bracketed by a pair
 * of CUDA events recorded on the launching stream (taken from a ctx-owned
 * pool of 256 pairs per timer, created at the first call with on != 0; older launches are
 * overwritten).  on = 1 starts a new record, on = 0 stops recording and keeps the record,
 * on = 2 goes on recording into the kept record (to time a subset of a sequence of calls). */
kb_status kb_ctx_enable_timing(kb_ctx* ctx, int on);
/* Wait for the recorded launches of `which` since the last read, write their
 * durations in milliseconds (oldest first, at most `cap`) to h_ms (HOST) and
 * their number to *n (HOST); the record is then cleared. */
kb_status kb_ctx_read_timer(kb_ctx* ctx, kb_timer which, float* h_ms, uint32_t cap, uint32_t* n);
/* Register-only probe of the instruction mix of the direct win count (two compares and two
 * predicated increments per sample pair, values held in registers): runs it on every SM for
 * `iters` (<= 2^23) rounds of 128 sample pairs per thread, times it with CUDA events on
 * `stream`, and writes the rate in sample pairs per second to *pairs_per_s (HOST).  This is
 * the measured ceiling the direct win-count kernel is compared with.  Synchronous. */
kb_status kb_alu_probe(kb_ctx* ctx, uint32_t iters, double* pairs_per_s, void* stream);
/* Choose how kb_adjudicate counts wins: 0 = automatic (on the sorted rows when they fit shared
 * memory: a lane-per-row merge for K >= 225 and S <= 1024, else a binary search and walk per
 * row pair for S <= 4096; direct comparison beyond), 1 = always direct comparison of all
 * sample pairs, 2 = always binary search (S <= 4096 only), 3 = always the lane-per-row merge
 * (S <= 1024 only).  The integers produced are identical. */
kb_status kb_ctx_set_wins_algo(kb_ctx* ctx, int algo);
/* Number of kernels this context has launched since it was created (HOST out). */
kb_status kb_ctx_launch_count(const kb_ctx* ctx, uint64_t* n);

/* ---- failure paths, exercised without a GPU fault -------------------------- */

/* Let the next `skip` device allocations of this context through, then make the `n` after
 * them fail as if the device were out of memory (the allocator is not called for those).
 * Lets a test check that a failed workspace growth leaves the context usable.  n = 0
 * switches the hook off. */
kb_status kb_ctx_fail_next_allocs(kb_ctx* ctx, uint32_t skip, uint32_t n);

/* Every device buffer a context owns (status words, accumulator workspace, sorted timings,
 * single-launch workspace, host-path staging) is allocated between two 256-byte guard bands
 * holding a fixed byte pattern.  Synchronises `stream`, reads all bands back and writes the
 * number of buffers checked to *n_buffers and the number of band bytes that no longer hold
 * the pattern to *n_bad_bytes (HOST pointers): a kernel of the library that wrote outside
 * its workspace shows up here.  (The tests put the same bands around the caller-owned
 * outputs.) */
kb_status kb_ctx_check_guards(kb_ctx* ctx, void* stream, uint32_t* n_buffers, uint32_t* n_bad_bytes);

/* Copy the first `bytes` (<= KB_STATIC_SCRATCH_BYTES) of kb_screen_static's scratch array on
 * the current device to h_dst (HOST), after synchronising the device: lets a test see that a
 * call left everything beyond the part it uses untouched.  Allocates nothing. */
kb_status kb_static_scratch_read(void* h_dst, uint32_t bytes);

/* Self-test of the bounded device-side wait every streaming kernel uses: launches ONE warp
 * that waits, with the library's own wait routine and a limit of `limit_ns` nanoseconds
 * (1,000 <= limit_ns <= 100,000,000), on a barrier that nothing will ever complete.  No copy
 * is in flight and no other thread waits.  The wait gives up after the limit, records
 * KB_ERR_DEVICE_TIMEOUT in the context's device status word and the kernel returns normally;
 * kb_ctx_poll then reports and clears it.  Asynchronous on `stream`. */
kb_status kb_ctx_selftest_wait(kb_ctx* ctx, uint64_t limit_ns, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* KB_HOOKS_H_ */
