/*
 * kb.h -- C ABI of the candidate screen, timing adjudication and survivor
 * selection used inside a multi-fidelity kernel-search evaluation loop
 * (KernelBrain, arxiv 2608.02611).
 *
 * The library covers the data-parallel interior of the paper's Evaluation
 * Plane (Sec. 3.4) and of the scheduler's promote/prune step:
 *
 *   kb_screen      the Verifier's "output correctness against the reference"
 *                  check (Sec. 3.4, Evaluation Plane; the correctness
 *                  indicator K(p) of Sec. 3.1), for K candidates at once,
 *                  optionally on a fidelity-dependent subset of tiles
 *                  (low-cost screening, Abstract / Sec. 3.3 Observation 2);
 *   kb_adjudicate  the reduction of repeated, noisy timings to an
 *                  "adjudicated latency" (Algorithm 1, the step that scores a
 *                  candidate from it; Sec. 1 contribution 1
 *                  "stability adjudication"; Appendix "Relative Variability
 *                  Metrics"), as median + IQR per candidate plus a K x K
 *                  matrix of doubled Mann-Whitney win counts;
 *   kb_select      the promotion decision D (Sec. 3.2 "Promotion decision",
 *                  Sec. 3.4 "Adaptive Resource Allocation": rank with
 *                  deterministic tie-breaking, promote the top part).
 *
 * Conventions (all entry points)
 *   - Plain C99 types only.  Every pointer is marked HOST or DEVICE below.
 *   - Ownership: the caller owns every input and output buffer.  The library
 *     owns kb_ctx (a device workspace that grows on demand with cudaMalloc
 *     and is released by kb_ctx_destroy) and kb_mask.
 *   - Asynchrony: kb_screen / kb_adjudicate / kb_select enqueue work on
 *     `stream` (a cudaStream_t passed as void*; NULL = the default stream) and
 *     return without synchronising.  Outputs are valid once the stream has
 *     been synchronised.  Host arrays passed in (h_cands) are consumed before
 *     the call returns.  One kb_ctx must not be used from two streams or two
 *     host threads at the same time.
 *   - Errors: a kb_status is returned; nothing aborts or throws.  Argument
 *     errors are detected before any launch and leave the outputs untouched.
 *     Conditions only the device can see (a non-finite timing, a bounded wait
 *     that ran out) are recorded in a ctx-owned device status word that
 *     kb_ctx_poll reads back.
 *   - Determinism: every output is a pure function of the inputs; it does not
 *     depend on grid size, scheduling or call history.
 *   - Arithmetic: IEEE-754 binary32 (binary64 in kb_screen_f64),
 *     round-to-nearest-even, no fused multiply-add, subnormals honoured.
 */
#ifndef KB_H_
#define KB_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  KB_OK = 0,
  KB_ERR_INVALID_ARG = 1,   /* null pointer, zero size, out-of-range value        */
  KB_ERR_ALIGNMENT = 2,     /* a tensor pointer is not 16-byte aligned            */
  KB_ERR_UNSUPPORTED = 3,   /* unknown dtype / policy                             */
  KB_ERR_WORKSPACE = 4,     /* the device workspace could not be grown            */
  KB_ERR_CUDA = 5,          /* a CUDA runtime call failed (see kb_last_error)     */
  KB_ERR_NONFINITE = 6,     /* device status: a timing was NaN or +-Inf           */
  KB_ERR_DEVICE_TIMEOUT = 7 /* device status: a bounded device-side wait ran out  */
} kb_status;

typedef enum {
  KB_F32 = 0,
  KB_F16 = 1,
  KB_BF16 = 2,
  KB_F8E4M3 = 3, /* 8-bit float, 4 exponent / 3 fraction bits, "fn": no Inf, one NaN (S.1111.111) */
  KB_F8E5M2 = 4  /* 8-bit float, 5 exponent / 2 fraction bits, IEEE-like                         */
} kb_dtype;

/* One record per candidate; 48 bytes, 8-byte aligned.
 * With r = ref[i], c = cand[i] decoded exactly to binary32 and, over the
 * selected elements i in ascending order,
 *     d     = |c - r|                       (one rounding)
 *     tol   = atol + (rtol * |r|)           (product rounded, then sum rounded)
 *     match = (c == r) || (isfinite(d) && d <= tol)      (NaN never matches)
 * the fields are: */
typedef struct {
  uint64_t mismatch_count; /* selected elements with match == false                 */
  uint64_t nan_count;      /* selected elements whose CANDIDATE value is NaN        */
  uint64_t inf_count;      /* selected elements whose CANDIDATE value is +-Inf      */
  int64_t argmax_idx;      /* flat index in the FULL tensor of max_abs_err, lowest
                              index on ties; -1 if no selected element has finite d */
  float max_abs_err;       /* max of d over selected elements with finite d; 0 if none */
  float max_rel_err;       /* max of d/|r| (correctly rounded) over selected elements
                              with finite d and r != 0; 0 if none; may be +Inf      */
  uint32_t pass;           /* 1 iff mismatch_count == 0                             */
  uint32_t reserved;       /* 0                                                     */
} kb_screen_result;

typedef struct kb_ctx kb_ctx;   /* device workspace + status word; bound to one device */
typedef struct kb_mask kb_mask; /* immutable fidelity mask; owns a device tile list    */

/* Limits checked at the boundary. */
#define KB_MAX_K 65535u         /* candidates per call                               */
#define KB_MAX_N 4294967296ull  /* elements per tensor (2^32)                        */
#define KB_MAX_S 32768u         /* timings per candidate (2*S*S must fit uint32)     */

/* ---- context ----------------------------------------------------------- */

/* Create a context on CUDA device `device`.  HOST out pointer. */
kb_status kb_ctx_create(int device, kb_ctx** out);
/* Synchronises the device, frees the workspace.  NULL is accepted. */
kb_status kb_ctx_destroy(kb_ctx* ctx);
/* Text of the last error recorded on this context (ctx-owned, valid until the
 * next call on the context); with ctx == NULL, the text of the last failed
 * kb_ctx_create on this thread. */
const char* kb_last_error(const kb_ctx* ctx);
/* (Takes the stream it synchronises, since the library keeps no stream of its own.)
 * Synchronise `stream`, read the device status word into *device_status
 * (KB_OK, KB_ERR_NONFINITE or KB_ERR_DEVICE_TIMEOUT; HOST pointer) and clear
 * it.  Returns KB_OK unless the read itself failed. */
kb_status kb_ctx_poll(kb_ctx* ctx, void* stream, kb_status* device_status);
/* Test, tuning and instrumentation hooks (forced grid sizes and dispatch paths,
 * CUDA-event timers, launch counter, self-tests) are declared in kb_hooks.h. */

/* ---- fidelity masks (Sec. 3.2 "Fidelity level", rendered on elements) --- */

/* A mask selects whole tiles of 2^log2_tile consecutive elements: element i is
 * selected iff tile (i >> log2_tile) is selected; the last tile may be
 * partial.  log2_tile <= 31.  Tiles of >= 4096 elements let a lower tier skip
 * DRAM traffic; smaller tiles are legal but every sector is still fetched. */

/* Strided mask: tile t selected iff (t % stride) == phase; stride >= 1,
 * phase < stride. */
kb_status kb_mask_create_strided(kb_ctx* ctx, uint64_t N, uint32_t log2_tile, uint32_t stride,
                                 uint32_t phase, kb_mask** out);
/* Bitmap mask: tile t selected iff bit (t & 63) of host_bits[t >> 6] is set.
 * HOST pointer to ceil(ntiles/64) words, consumed before return. */
kb_status kb_mask_create_bitmap(kb_ctx* ctx, uint64_t N, uint32_t log2_tile,
                                const uint64_t* host_bits, kb_mask** out);
/* Number of selected elements (HOST out). */
kb_status kb_mask_count(const kb_mask* mask, uint64_t* n_selected);
kb_status kb_mask_destroy(kb_mask* mask);

/* ---- correctness gate (Sec. 3.1 K(p); Sec. 3.2 policy check, output-shape
 *      and dtype constraints; Sec. 3.4 Verifier) --------------------------- */

/* Compare K candidates with one reference.
 *   d_ref    DEVICE, N elements of `dtype`, 16-byte aligned.
 *   h_cands  HOST array of K DEVICE pointers, each N elements of `dtype`,
 *            16-byte aligned.  All tensors share one dtype and one N: that is
 *            the shape/dtype part of the policy check.
 *   atol, rtol  finite and >= 0.
 *   mask     NULL = every element; else a mask created for the same N.
 *   d_out    DEVICE, K records, 8-byte aligned; fully overwritten.
 * 1 <= K <= KB_MAX_K, 1 <= N <= KB_MAX_N. */
kb_status kb_screen(kb_ctx* ctx, const void* d_ref, const void* const* h_cands, uint32_t K,
                    uint64_t N, kb_dtype dtype, float atol, float rtol, const kb_mask* mask,
                    kb_screen_result* d_out, void* stream);

/* Same operation with every tensor in HOST memory (pinned memory gives the
 * best transfer rate; pageable works).  The reference and the candidates are
 * copied to ctx-owned device staging in batches of candidates so that copies
 * overlap the kernel, and the K records are copied back to h_out (HOST).
 * Synchronous: returns when h_out is complete.  `stream` orders the work. */
kb_status kb_screen_host(kb_ctx* ctx, const void* h_ref, const void* const* h_cands_host,
                         uint32_t K, uint64_t N, kb_dtype dtype, float atol, float rtol,
                         const kb_mask* mask, kb_screen_result* h_out, void* stream);

/* The same gate on a selection that lives on the device (tier chaining without
 * a host round trip, e.g. kb_select's output feeding the next tier's screen;
 * the whole sequence can be recorded in one CUDA graph).  Slot j of the call
 * is candidate d_table[d_index[j]] for j < *d_count; slots j >= *d_count hold
 * no candidate and get the record {counts 0, argmax_idx -1, errors 0, pass 0}.
 *   d_table  DEVICE array of K_all DEVICE pointers (N elements of dtype each).
 *   d_index  DEVICE int32 [Kmax] (kb_select's d_survivors fits as it is).
 *   d_count  DEVICE uint32 (kb_select's d_n_survivors).
 *   d_out    DEVICE [Kmax] records.   1 <= Kmax <= 1024.
 * What the host cannot check is checked on the device before any tensor is
 * touched: an index outside [0, K_all), a null or misaligned pointer, or
 * *d_count > Kmax turns the call into a no-op (all slots "no candidate") and
 * sets the device status to KB_ERR_INVALID_ARG / KB_ERR_ALIGNMENT. */
kb_status kb_screen_indexed(kb_ctx* ctx, const void* d_ref, const void* const* d_table,
                            uint32_t K_all, const int32_t* d_index, const uint32_t* d_count,
                            uint32_t Kmax, uint64_t N, kb_dtype dtype, float atol, float rtol,
                            const kb_mask* mask, kb_screen_result* d_out, void* stream);

/* Several shapes in one launch (the fidelity level includes the set of input
 * shapes, Sec. 3.2): G groups, group g with one reference of h_N[g] elements
 * and h_K[g] candidates of that size; all of one dtype.  Meant for the
 * latency-bound regime of many small tensors (e.g. 21 candidates of a 512-,
 * 1024- and 2048-element output): one kernel launch for everything.
 *   h_refs   HOST array of G DEVICE pointers.
 *   h_cands  HOST array of sum(h_K) DEVICE pointers, group after group.
 *   d_out    DEVICE records in the order of h_cands.
 * 1 <= G <= 64, sum(h_K) <= 1024, and the tensors together at most 8192
 * blocks of 1024 elements (sum over candidates of ceil(N_g / 1024)); no mask.
 * Larger jobs: call kb_screen per group. */
kb_status kb_screen_multi(kb_ctx* ctx, uint32_t G, const void* const* h_refs,
                          const void* const* h_cands, const uint32_t* h_K, const uint64_t* h_N,
                          kb_dtype dtype, float atol, float rtol, kb_screen_result* d_out,
                          void* stream);

/* The gate over an element range cut into R consecutive parts (the definition of Sec. 3.1
 * K(p) carried over a partition of the index set; used when the ELEMENTS of a few large
 * tensors, not the candidates, are spread over several GPUs): the records of the whole range
 * from the records of its parts.  Counts add; the largest error wins and the earlier part
 * keeps it on a tie (its indices are lower), with argmax_idx moved to global numbering; the
 * largest relative error is the maximum; pass = no mismatch anywhere.  A part that saw no
 * finite difference (argmax_idx = -1) contributes no error.
 *   d_parts  DEVICE [R][K] records, part after part; part r covers the elements from global
 *            index h_first[r] on (the parts' own records number their elements from 0).
 *   h_first  HOST array of R strictly ascending indices.
 *   d_out    DEVICE [K] records (8-byte aligned); may not overlap d_parts.
 * 1 <= R <= 64, 1 <= K <= KB_MAX_K.  Asynchronous on `stream`; no allocation. */
kb_status kb_merge_ranges(kb_ctx* ctx, const kb_screen_result* d_parts, uint32_t R, uint32_t K,
                          const uint64_t* h_first, kb_screen_result* d_out, void* stream);

/* ---- the gate for double-precision tensors (Sec. 3.1 K(p); Sec. 3.4 Verifier) ----
 * The same gate with the reference and the candidates stored in binary64 and
 * EVERY operation of the record (d, tol, the comparison, d/|r|) in binary64,
 * round-to-nearest-even, no fused multiply-add: a double-precision output is
 * judged in its own precision.  56 bytes per record, 8-byte aligned; field
 * meanings as in kb_screen_result. */
typedef struct {
  uint64_t mismatch_count;
  uint64_t nan_count;
  uint64_t inf_count;
  int64_t argmax_idx;
  double max_abs_err;
  double max_rel_err;
  uint32_t pass;
  uint32_t reserved;
} kb_screen_result_f64;

/* Arguments as for kb_screen (DEVICE d_ref, HOST array of K DEVICE pointers, all
 * 16-byte aligned; atol, rtol finite and >= 0; mask NULL or created for the
 * same N; DEVICE d_out of K records, fully overwritten).  Asynchronous on
 * `stream`.  1 <= K <= KB_MAX_K, 1 <= N <= KB_MAX_N.  Errors as for kb_screen. */
kb_status kb_screen_f64(kb_ctx* ctx, const double* d_ref, const double* const* h_cands, uint32_t K,
                        uint64_t N, double atol, double rtol, const kb_mask* mask,
                        kb_screen_result_f64* d_out, void* stream);

/* ---- the same gate for callers that must not allocate ----------------------
 * (The paper has no counterpart; this entry point exists for integration.)
 *
 * Some hosts of this library cannot let it call cudaMalloc: a serving loop that
 * has promised its users no allocation after start-up; a framework whose own
 * allocator has already claimed nearly all device memory, so that a driver
 * allocation from a third party may simply fail; a process whose allocations
 * are all audited and pre-approved.  kb_screen_static does what kb_screen does
 * with mask == NULL, but creates no context and allocates nothing, neither on
 * the device nor through any library: the per-candidate accumulators and the
 * candidate pointer table live in a fixed array inside the library's device
 * image (KB_STATIC_SCRATCH_BYTES, held by every GPU that loads the library
 * until the process exits).
 *
 *   - The call works on the CURRENT device; `stream` must belong to it.
 *   - 1 <= K <= KB_STATIC_MAX_K; larger K is refused with KB_ERR_WORKSPACE and
 *     a message readable through kb_last_error(NULL).  Other argument rules are
 *     those of kb_screen; there is no fidelity mask.
 *   - The first call on a device looks up the address of the array and sets
 *     kernel attributes.  Make that first call before any stream capture
 *     begins.
 *   - All calls on one device share the one array, which keeps what the last
 *     call left in it; each call clears the part it uses before use.  Two
 *     calls that overlap on the GPU (different streams, or one stream and a
 *     graph replay) race on it and give wrong records: order them.
 *   - Host threads: calls on one device are serialised by a lock inside the library for
 *     as long as they validate and enqueue, so two host threads may call it; they still
 *     have to order their work on the GPU (previous point).  kb_last_error(NULL) is per
 *     thread.
 *   - Asynchronous like kb_screen; d_out is valid after `stream` synchronises.
 *     A device-side wait that ran out cannot be polled through this entry point
 *     (there is no context); use kb_screen + kb_ctx_poll where that matters. */
#define KB_STATIC_MAX_K 1024u
#define KB_STATIC_SCRATCH_BYTES (256u + 2u * 1024u * 48u + 1024u * 8u)
kb_status kb_screen_static(const void* d_ref, const void* const* h_cands, uint32_t K, uint64_t N,
                           kb_dtype dtype, float atol, float rtol, kb_screen_result* d_out,
                           void* stream);

/* ---- stability adjudication (Algorithm 1 "adjudicated latency"; Sec. 1
 *      contribution 1; Appendix "Relative Variability Metrics") ------------ */

/* d_timings  DEVICE, [K][S] row-major binary32 milliseconds, all finite
 *            (otherwise the device status becomes KB_ERR_NONFINITE and the
 *            outputs are unspecified).
 * d_median   DEVICE [K]: type-7 (linear) quantile at 1/2 of the sorted row:
 *            pos = j*(S-1), lo = pos/4, rem = pos%4, hi = min(lo+1, S-1),
 *            Q_j = x_lo if rem == 0 else x_lo + ((rem*0.25f) * (x_hi - x_lo)),
 *            each operation rounded.  median = Q_2.
 * d_iqr      DEVICE [K]: Q_3 - Q_1 (rounded).
 * d_wins     DEVICE [K][K] row-major uint32:
 *            W[a][b] = sum_i sum_j ( 2*[t_a,i < t_b,j] + [t_a,i == t_b,j] ),
 *            i.e. twice the Mann-Whitney U of "a faster than b" with ties
 *            counted once; W[a][b] + W[b][a] = 2*S*S and W[a][a] = S*S.
 * Any of the three outputs may be NULL to skip it.
 * 1 <= K <= KB_MAX_K, 1 <= S <= KB_MAX_S. */
kb_status kb_adjudicate(kb_ctx* ctx, const float* d_timings, uint32_t K, uint32_t S,
                        float* d_median, float* d_iqr, uint32_t* d_wins, void* stream);

/* The same with a different number of timings per candidate (candidates
 * measured at different fidelities): row k is d_timings[d_offsets[k] ..
 * d_offsets[k+1]), S_k = its length.  Median and IQR per row as above;
 * W[a][b] by the same double sum, so W[a][b] + W[b][a] = 2*S_a*S_b and
 * W[a][a] = S_a*S_a.
 *   d_offsets  DEVICE uint32 [K+1], ascending.
 *   S_max      an upper bound of every S_k, 1 <= S_max <= 4096.  A row that is
 *              empty or longer than S_max sets the device status to
 *              KB_ERR_INVALID_ARG; its outputs are then unspecified. */
kb_status kb_adjudicate_ragged(kb_ctx* ctx, const float* d_timings, const uint32_t* d_offsets,
                               uint32_t K, uint32_t S_max, uint64_t total, float* d_median,
                               float* d_iqr, uint32_t* d_wins, void* stream);

/* ---- promotion decision (Sec. 3.2; Sec. 3.4 scheduler; Algorithm 1, D) --- */

typedef enum {
  KB_SELECT_ERR_THEN_TIME = 0, /* key (max_rel_err asc, median asc, index asc) */
  KB_SELECT_TIME = 1           /* key (median asc, index asc)                   */
} kb_select_policy;

/* (The policies below read only the gate's records and the medians, so those are the
 * statistics this call takes; a ranking over the win matrix is kb_copeland.)
 * Eligible candidates are those with pass == 1 (failed candidates are never
 * promoted).  They are ordered by the policy's key, floats compared as values
 * (none is NaN), ties broken by the lower candidate index; the first
 * n = min(budget, #eligible) indices are written to d_survivors IN RANK ORDER
 * and n to *d_n_survivors.  Entries d_survivors[n..budget) are set to -1.
 *   d_screen     DEVICE [K] records from kb_screen.
 *   d_median     DEVICE [K] from kb_adjudicate.
 *   d_survivors  DEVICE [budget] int32.   d_n_survivors  DEVICE uint32.
 * 1 <= K <= KB_MAX_K, budget >= 1. */
kb_status kb_select(kb_ctx* ctx, const kb_screen_result* d_screen, const float* d_median,
                    uint32_t K, kb_select_policy policy, uint32_t budget, int32_t* d_survivors,
                    uint32_t* d_n_survivors, void* stream);

/* ---- scheduler-side statistics ------------------------------------------- */

/* Runtime score and promotion by it (Sec. 3.1, Eq. 2; Sec. 3.4 scheduler):
 *     S(p, r) = 1e6 / max(1, latency_us) + gamma(r),   gamma(r) = alpha*r + beta*b_r
 * with latency = the adjudicated (median) latency, given in milliseconds; every
 * operation in binary32 in this order: l = median*1000; m = max(1, l);
 * base = 1e6/m; gamma = (alpha*rung) + (beta*rung_budget); score = base + gamma.
 * Eligible = pass == 1; order by (score descending, index ascending); the first
 * n = min(budget, #eligible) indices go to d_survivors in rank order, the rest
 * is -1, n to *d_n_survivors.
 *   d_score  DEVICE [K] float, every candidate's score (eligible or not); may be NULL.
 * Other arguments as for kb_select. */
kb_status kb_select_by_score(kb_ctx* ctx, const kb_screen_result* d_screen, const float* d_median,
                             uint32_t K, uint32_t rung, uint32_t rung_budget, float alpha,
                             float beta, uint32_t budget, float* d_score, int32_t* d_survivors,
                             uint32_t* d_n_survivors, void* stream);

/* Tail ratios per candidate (Appendix "Relative Variability Metrics"):
 * d_ratios DEVICE [K][3] = {P90/P50, P95/P50, P99/P50} of each row of
 * d_timings [K][S], with P_q the linear (type-7) percentile of the sorted row:
 *   pos = q*(S-1); lo = pos/100; rem = pos%100; hi = min(lo+1, S-1);
 *   P_q = x_lo if rem == 0 else x_lo + (((float)rem / 100.0f) * (x_hi - x_lo)),
 * each operation (and the final divisions) rounded.  Non-finite timings set
 * KB_ERR_NONFINITE in the device status.  1 <= S <= KB_MAX_S. */
kb_status kb_tail_ratios(kb_ctx* ctx, const float* d_timings, uint32_t K, uint32_t S,
                         float* d_ratios, void* stream);

/* Copeland counts from a win matrix of kb_adjudicate (a ranking that uses only
 * the order of samples, Appendix "Relative Variability Metrics"):
 *   d_beats[a] = #{b != a : W[a][b] >  S*S},  d_ties[a] = #{b != a : W[a][b] == S*S}
 * DEVICE [K] uint32 each; d_ties may be NULL. */
kb_status kb_copeland(kb_ctx* ctx, const uint32_t* d_wins, uint32_t K, uint32_t S,
                      uint32_t* d_beats, uint32_t* d_ties, void* stream);

/* Re-measure and confirm (the paper's only description of stability
 * adjudication, a commented-out passage of Sec. 3: a candidate whose score
 * change exceeds a threshold is measured again at the same fidelity and
 * reverted if the improvement is not confirmed).  Per candidate, in binary32:
 *   flagged   = (first - prev)  > (threshold * prev)
 *   confirmed = (second - prev) > (threshold * prev)
 *   not flagged:            status 0, score = first
 *   flagged and confirmed:  status 1, score = min(first, second)
 *   flagged, not confirmed: status 2, score = prev
 * All arrays DEVICE [K]; d_status uint32, the others float. */
kb_status kb_confirm(kb_ctx* ctx, const float* d_first, const float* d_second, const float* d_prev,
                     uint32_t K, float threshold, uint32_t* d_status, float* d_score, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* KB_H_ */
