/* ralm.h -- C ABI of the exact dense retrieval library for sm_100a (NVIDIA B200).
 *
 * The library implements the retrieval calls of RaLMSpec's serving loop (Algorithm 1):
 *
 *   C.retrieve(q_1..q_s)      -> ralm_search        batched verification retrieval with an
 *                                                   exact dense retriever (Algorithm 1,
 *                                                   batched verification step; Section 3,
 *                                                   "Batched verification")
 *   Q.retrieve(q_i)           -> ralm_cache_search  speculative retrieval from a request's
 *                                                   local cache, ranked with the retriever's
 *                                                   own metric (Algorithm 1, speculative
 *                                                   retrieval step; Section 3, "Speculative
 *                                                   retrieval"; Fig. 3)
 *   m = argmin_i d^_i != d_i  -> ralm_verify        first mis-speculated position
 *                                                   (Algorithm 1, verification step; toy
 *                                                   example of Section 3)
 *
 * Conventions
 *   - Every call returns a ralm_status_t; nothing throws, aborts or prints.
 *   - Argument errors are detected on the host before any launch.
 *   - Calls taking a `stream` (a cudaStream_t passed as void*, NULL = default stream) only
 *     enqueue work; outputs are valid once the stream has reached that point.
 *   - All fp16 data is IEEE binary16 and must be finite.
 *   - Ranking is a total order: inner product (score descending, id ascending); L2
 *     (squared distance ascending, id ascending). L2 scores are SQUARED distances.
 *   - When fewer than k rows qualify, trailing slots hold id -1 and score -inf (inner
 *     product) or +inf (L2).
 *   - Scores are accumulated in fp32.
 *   - One index may be used from one stream at a time (its workspace is shared by calls).
 *   - Device-side anomalies (an out-of-range cache id, a wait that ran out, a candidate list
 *     asked to hold more than its capacity: RALM_ERR_INTERNAL, a defect of the library, the
 *     results of that search are then not to be trusted) set a sticky status word that
 *     ralm_device_status reads.
 */
#ifndef RALM_H_
#define RALM_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ralm_index ralm_index_t; /* opaque */

typedef enum { RALM_IP = 0, RALM_L2 = 1 } ralm_metric_t;

typedef enum {
    RALM_OK = 0,
    RALM_ERR_INVALID_ARG = 1,
    RALM_ERR_OOM = 2,
    RALM_ERR_CUDA = 3,
    RALM_ERR_TIMEOUT = 4,
    RALM_ERR_UNSUPPORTED = 5,
    RALM_ERR_BAD_CACHE_ID = 6,
    RALM_ERR_STATIC_LIMIT = 7,
    RALM_ERR_INTERNAL = 8
} ralm_status_t;

/* Limits checked by the host side. */
#define RALM_MAX_K 1024       /* neighbours per query (the KNN-LM evaluation's largest k) */
#define RALM_MAX_D 4096       /* vector dimension */
#define RALM_MAX_QUERIES 4096 /* queries per ralm_search call */
#define RALM_MAX_CACHE 4096   /* cache slots per request */
#define RALM_MAX_CACHE_KEYS (1 << 20) /* R * q * (C rounded up to a power of two) per call */

/* Create an index over a corpus that is already resident in device memory.
 *   corpus  DEVICE pointer, fp16 [N][d] row-major, 16-byte aligned, d % 8 == 0,
 *           8 <= d <= RALM_MAX_D, 0 <= N < 2^31. BORROWED: never copied; the caller keeps it
 *           alive and unmodified until ralm_index_destroy. May be NULL only when N == 0.
 *   metric  RALM_IP (QA dense retriever) or RALM_L2 (KNN-LM datastore).
 *   max_s   largest number of queries a later ralm_search will pass (1..RALM_MAX_QUERIES).
 *   max_k   largest k a later call will pass (1..RALM_MAX_K).
 *   out     receives the handle (host memory owned by the library).
 * Allocates the per-index device workspace on the current device: partial top-k lists, staging
 * buffers, a status word; for L2 the squared norm of every row (4 N bytes, computed here in one
 * pass over the corpus); for max_k > 256 spilled candidate lists (about 19 MB at k = 1024); for
 * max_s >= 9 the candidate lists of the large-batch scan (about 300 KB per query, 155 MB at 512
 * queries; twice that for max_k > 64). Synchronous.
 * Errors: INVALID_ARG (null pointer, misaligned corpus, bad sizes), OOM, CUDA,
 * UNSUPPORTED (device is not compute capability 10.x). */
ralm_status_t ralm_index_create(const void *corpus, int64_t N, int32_t d, ralm_metric_t metric,
                                int32_t max_s, int32_t max_k, ralm_index_t **out);

/* Free the workspace and the handle. The corpus is untouched. NULL is accepted. */
ralm_status_t ralm_index_destroy(ralm_index_t *idx);

/* C.retrieve(q_1..q_s): exact top-k of s queries over the whole corpus, one stream of the
 * corpus from HBM per pass (up to 32 queries on the small-batch scan, up to 512 on the
 * large-batch scan, which takes over from 9 queries on large corpora, 17 for inner product with k == 1).
 *   queries DEVICE fp16 [s][d], 16-byte aligned.     0 <= s <= max_s
 *   ids     DEVICE int64 [s][k]  (written)           1 <= k <= max_k
 *   scores  DEVICE fp32  [s][k]  (written)
 * Asynchronous on `stream`. s == 0 is a no-op. */
ralm_status_t ralm_search(ralm_index_t *idx, const void *queries, int32_t s, int32_t k,
                          int64_t *ids, float *scores, void *stream);

/* Same as ralm_search with HOST buffers: copies the queries to the device, searches, copies
 * ids and scores back, and returns after the results are in host memory (synchronises
 * `stream`). Pinned host memory makes the copies asynchronous up to that point. */
ralm_status_t ralm_search_host(ralm_index_t *idx, const void *queries_host, int32_t s,
                               int32_t k, int64_t *ids_host, float *scores_host, void *stream);

/* Limits of ralm_search_static (below). */
#define RALM_STATIC_MAX_S 8        /* queries per call */
#define RALM_STATIC_MAX_K 32       /* neighbours per query */
#define RALM_STATIC_MAX_BLOCKS 160 /* scan CTAs whose partial lists the scratch can hold */

/* ralm_search for callers that must not allocate. (The paper has no counterpart: this entry
 * point exists for the way the library gets embedded, not for the method.)
 *
 * Who needs it: code that runs where device allocation is off the table -- a serving process
 * whose memory pool has already claimed the whole GPU and hands out no more, a real-time or
 * safety-certified host loop that forbids allocator calls after start-up, or a plug-in that
 * is handed buffers by its host application and has no right to create its own.
 * ralm_index_create calls cudaMalloc for its workspace, so those callers cannot use it.
 *
 * This call needs no index and calls no cudaMalloc, cudaFree or any other allocating routine.
 * The scan's scratch (per-CTA partial top-k lists) is a fixed array inside the library image:
 * RALM_STATIC_MAX_BLOCKS * RALM_STATIC_MAX_S * RALM_STATIC_MAX_K * 8 bytes = 320 KiB (plus a
 * 256-byte status block), held by every GPU that loads the library until the process exits.
 *
 *   corpus, N, d, metric   as for ralm_index_create (DEVICE fp16 [N][d], borrowed for the call),
 *                          except that two tiles of 16 rows must fit in shared memory next to
 *                          the queries: d up to about 2800. (An index serves longer rows on its
 *                          large-batch scan, whose workspace this call does not have.)
 *   queries                DEVICE fp16 [s][d], 16-byte aligned, 0 <= s <= RALM_STATIC_MAX_S
 *   ids, scores            DEVICE int64 [s][k] / fp32 [s][k] (written), 1 <= k <= RALM_STATIC_MAX_K
 *   device_status          DEVICE int32, may be NULL: zeroed by the call (also when s == 0), then
 *                          set to a ralm_status_t value if a device-side wait ran out. With NULL
 *                          the library keeps that word in its own scratch and nobody reads it:
 *                          pass a status word if a time-out must be seen.
 * Results are identical to ralm_search's.
 * Errors: RALM_ERR_STATIC_LIMIT when s or k exceeds the limits above (nothing is launched);
 * UNSUPPORTED for rows longer than the limit above or a device that is not compute capability
 * 10.x; INVALID_ARG, CUDA as elsewhere.
 *
 * The first call on each device looks up the scratch's device address and the device's
 * properties (with that device current); make that first call before any stream capture.
 * Every call on a device shares the one scratch array, which keeps the previous call's
 * contents: the call clears what must start at zero itself, but two calls whose GPU work
 * overlaps (different streams, different threads) race on it -- serialise them.
 * Asynchronous on `stream`. */
ralm_status_t ralm_search_static(const void *corpus, int64_t N, int32_t d, ralm_metric_t metric,
                                 const void *queries, int32_t s, int32_t k, int64_t *ids,
                                 float *scores, int32_t *device_status, void *stream);

/* Q.retrieve for R requests at once: request r owns C cache slots holding corpus ids
 * (-1 = empty slot; the cache is a set, a repeated id counts once) and q queries; each
 * query is ranked against that request's cached rows only, with the index's metric and the
 * same total order as ralm_search.
 *   cache_ids DEVICE int64 [R][C]       queries DEVICE fp16 [R][q][d], 16-byte aligned
 *   ids       DEVICE int64 [R][q][k]    scores  DEVICE fp32 [R][q][k]
 *   1 <= C <= RALM_MAX_CACHE, 1 <= q, 1 <= k <= max_k,
 *   R * q * pow2ceil(C) <= RALM_MAX_CACHE_KEYS. R == 0 is a no-op.
 * An id outside [-1, N) is skipped and sets RALM_ERR_BAD_CACHE_ID in the status word.
 * Asynchronous on `stream`. */
ralm_status_t ralm_cache_search(ralm_index_t *idx, const int64_t *cache_ids, int32_t R,
                                int32_t C, const void *queries, int32_t q, int32_t k,
                                int64_t *ids, float *scores, void *stream);

/* Verification: first_mismatch[r] = the smallest step i in [0, stride) at which any of the
 * first cmp_k speculated ids differs from the retrieved ones, or `stride` if every step
 * matches (0-based; Algorithm 1's "m <= s" becomes first_mismatch < stride).
 *   speculated_ids DEVICE int64 [R][stride][cmp_k]
 *   retrieved_ids  DEVICE int64 [R][stride][ld]   (ld = k of the search that produced them)
 *   first_mismatch DEVICE int32 [R] (written)
 *   `stride` is the speculation stride s of the paper, not a memory pitch.
 *   1 <= cmp_k <= ld; cmp_k == 1 compares the top-ranked document only.
 * Needs no index. Asynchronous on `stream`. R == 0 or stride == 0 are accepted. */
ralm_status_t ralm_verify(const int64_t *speculated_ids, const int64_t *retrieved_ids, int32_t R,
                          int32_t stride, int32_t ld, int32_t cmp_k, int32_t *first_mismatch,
                          void *stream);

/* Cache update after a verification step (Section 3, "Speculative retrieval": the local cache is
 * populated with the documents retrieved during verification, the top-ranked one per query or
 * the first `top` of them (top-k update, prefetching; Fig. 3); Section 5.3: for KNN-LM the next n
 * entries after each retrieved item go in instead of the items themselves).
 * Request r's cache is a set of corpus ids in C slots (-1 = empty) used as a ring: a new id is
 * written at cursor[r], which then advances modulo C, so a full cache drops its oldest entry
 * (the paper does not name an eviction rule; first-in first-out is this library's). For request r,
 * in this order: steps i = 0 .. steps[r]-1, ranks j = 0 .. top-1, id = retrieved_ids[r][i][j]
 * (negative ids are skipped); candidates are id itself (next_n == 0) or id+1 .. id+next_n
 * (next_n > 0), cut at N; a candidate already in the cache is skipped, any other is inserted.
 *   cache_ids     DEVICE int64 [R][C] (read and written)   1 <= C <= RALM_MAX_CACHE
 *   cursor        DEVICE int32 [R] (read and written), values in [0, C)
 *   retrieved_ids DEVICE int64 [R][stride][ld], 1 <= top <= ld
 *   steps         DEVICE int32 [R] or NULL (= stride for every request); values are clamped to
 *                 [0, stride]. Passing min(first_mismatch + 1, stride) inserts what was confirmed
 *                 plus the correcting document.
 *   N             number of corpus rows (candidates >= N are never inserted)
 * Needs no index. Asynchronous on `stream`. R == 0 or stride == 0 are no-ops. */
ralm_status_t ralm_cache_update(int64_t *cache_ids, int32_t *cursor, int32_t R, int32_t C,
                                const int64_t *retrieved_ids, int32_t stride, int32_t ld, int32_t top,
                                const int32_t *steps, int32_t next_n, int64_t N, void *stream);

/* Synchronise `stream`, read and clear the index's sticky device status word. Returns
 * RALM_OK, RALM_ERR_TIMEOUT, RALM_ERR_BAD_CACHE_ID, RALM_ERR_INTERNAL, or RALM_ERR_CUDA if the
 * stream itself reports an error. */
ralm_status_t ralm_device_status(ralm_index_t *idx, void *stream);

/* Pin the scan variant used by ralm_search on this index (benchmarking aid).
 *   0 = automatic, 1 = FMA scan (fp32 FMAs, d <= 1024, 4 queries per pass), 2 = warp-MMA scan
 *   (8 queries per pass, 16 for larger batches, 32 for inner product; for L2 the tensor-core
 *   value only filters and the ranked distance is the direct sum of squared differences), 3 = tcgen05 scan (up to 512 queries per pass, k <= 256,
 *   d >= 64; pairs of CTAs share each MMA; for L2 the tensor-core value again only filters,
 *   and the corpus must be large enough to scan a sample first, about 600 K rows), 4 = tcgen05
 *   scan with single CTAs. Automatic: warp-MMA up to 16 queries (inner product, k == 1; up to 8
 *   for k > 1; 32 on corpora too small for a sample launch, about 600 K rows) or 8 (L2), the
 *   tcgen05 scan beyond that where it applies.
 * UNSUPPORTED if the variant cannot serve the index's metric or dimension. The environment
 * variable RALM_FORCE_VARIANT=<1..4> applies the same pin to every index at creation. */
ralm_status_t ralm_index_set_variant(ralm_index_t *idx, int32_t variant);

/* Optional: build a one-byte-per-element copy of the corpus (E5M2, N * d bytes, plus one fp32
 * bound per row) that ralm_search then streams instead of the fp16 rows for batches of up to 8
 * queries (any k the index allows) and of 9..16 queries with k == 1 (k <= 64 when forced), under
 * the automatic variant (other shapes take the fp16 scans). The copy only
 * FILTERS: by the Cauchy-Schwarz inequality the inner product with the rounded row is within
 * |q| * |x - x8| of the true one, which bounds the score (inner product) or, with the rows' stored
 * squared norms, the squared distance (L2) from the right side; a (row, query) pair whose bound
 * cannot reach the value that k rows are already known to reach is dropped, and every other pair
 * is scored again from the fp16 row (L2: in the direct sum-of-squared-differences form), which is
 * the value that is ranked and returned. Results are those of the fp16
 * scan (what the paper's exact dense retriever returns, Section 5.1; the KNN-LM datastore's
 * neighbours and distances, Section 5.3); the bytes streamed per batch drop to about half. The
 * copy is used on corpora large enough for the sample phase that
 * gives the filter its thresholds (about 2.4 M rows); smaller ones keep the fp16 scan unless
 * `force` is non-zero (a testing aid: correct, but slow without thresholds to start from).
 * One pass over the corpus on the default stream, synchronous; allocates device memory.
 * Errors: UNSUPPORTED for d % 16 != 0; OOM. Calling it again only updates `force`. */
ralm_status_t ralm_index_enable_q8(ralm_index_t *idx, int32_t force);

/* Override the scan kernel's launch shape on this index (benchmarking aid; 0 keeps the
 * library's choice): consumer warps per CTA (1..8), shared-memory stages per consumer warp,
 * rows per tile of the FMA scan (rounded down to its group size; the warp-MMA scan always
 * uses 16). Values that do not fit in shared memory are reduced. Results do not depend on it. */
ralm_status_t ralm_index_set_tuning(ralm_index_t *idx, int32_t consumer_warps, int32_t ring_depth,
                                    int32_t tile_rows);

/* Number of kernels the library launched on behalf of this index since creation. */
int64_t ralm_index_launch_count(const ralm_index_t *idx);

/* Time every scan-kernel launch of this index with a pair of CUDA events recorded on the
 * caller's stream directly around the launch (measurement aid; off by default). */
ralm_status_t ralm_index_set_timing(ralm_index_t *idx, int32_t enabled);

/* Wait for the scan launches timed since the last read, return the sum of their durations in
 * milliseconds and how many there were, and forget them. HOST pointers. */
ralm_status_t ralm_index_read_timing(ralm_index_t *idx, double *total_ms, int64_t *launches);

/* As ralm_index_read_timing, but the durations one by one, in the order of the passes:
 * ms[0 .. *count) (HOST array of `capacity` doubles; passes beyond it are dropped). */
ralm_status_t ralm_index_read_timing_list(ralm_index_t *idx, double *ms, int64_t capacity, int64_t *count);

/* What the most recent ralm_search / ralm_search_host on this index ran (measurement aid; HOST
 * pointers). kernel: 0 = no search yet, 1 = FMA scan, 2 = warp-MMA scan, 3 = tcgen05 scan with CTA
 * pairs, 4 = tcgen05 scan with single CTAs, 5 = 8-bit scan. passes: passes over the corpus (each
 * serves one slice of the batch). phases: 1 = one launch per pass; 2 = a sample of the rows is
 * scanned first (in fp16) and the main launch covers the other rows; 3 = the sample launch only
 * yields thresholds and the main launch scans every row, the sample's again (the tcgen05 scan;
 * the other scans for k >= 128). sample_rows: rows of that sample (0 without one). */
ralm_status_t ralm_index_last_dispatch(const ralm_index_t *idx, int32_t *kernel, int32_t *passes,
                                       int32_t *phases, int64_t *sample_rows);

/* ---- Optimal speculation stride scheduler (OS^3): host arithmetic, no device work ---------
 * Section 4 ("Optimal speculation stride scheduler") and Appendix A.2. `a` is the latency of one
 * speculation step, `b` of one verification step (any one unit, e.g. the milliseconds that CUDA
 * events around ralm_cache_search and ralm_search report), gamma the probability that one
 * speculated document matches.
 *
 * ralm_os3_expected_verified: (1 - gamma^s) / (1 - gamma), the expected number of documents one
 *   verification step of stride s confirms (Appendix A.2); s for gamma = 1, 0 for s <= 0.
 * ralm_os3_objective: expected verified documents per unit time for stride s. Synchronous
 *   verification: latency s a + b. Asynchronous (async_verify != 0): with probability gamma^s
 *   the latency is (s - 1) a + max(a, b), otherwise s a + b.
 * ralm_os3_gamma: the windowed estimate sum(M) / (sum(M) + #{t : M(t) < s(t)}) over the last w
 *   verification steps, truncated at gamma_max (the evaluation uses w = 5, gamma_max = 0.6).
 *   matched[t] = the first_mismatch value ralm_verify returned for a step of stride strides[t]
 *   (HOST arrays, 0 <= matched[t] <= strides[t], strides[t] >= 1). No history (w = 0) gives 0.
 * ralm_os3_stride: the stride in 1..s_max that maximises the objective for the estimated gamma
 *   (the smaller stride on ties). With no history this is 1, where the scheduler starts.
 * Errors: INVALID_ARG for null pointers, negative latencies, values out of the stated ranges. */
double ralm_os3_expected_verified(double gamma, int32_t s);
double ralm_os3_objective(double gamma, double a, double b, int32_t s, int32_t async_verify);
ralm_status_t ralm_os3_gamma(const int32_t *matched, const int32_t *strides, int32_t w, double gamma_max,
                             double *gamma_out);
ralm_status_t ralm_os3_stride(const int32_t *matched, const int32_t *strides, int32_t w, double gamma_max,
                              double a, double b, int32_t s_max, int32_t async_verify, int32_t *s_out);

/* Row-sharded retrieval (a corpus split by rows over several indexes, on one GPU or one per
 * GPU): every shard answers the same batch with ralm_search over its own rows; this call merges
 * the G answers into the answer of C.retrieve over the whole corpus (Algorithm 1, batched
 * verification step), with the same total order, so the result equals the unsharded search.
 *   ids        DEVICE int64 [G][s][k]  shard-local row ids as ralm_search wrote them (-1 = padding)
 *   scores     DEVICE fp32  [G][s][k]
 *   row_offset DEVICE int64 [G]        global id of each shard's first row
 *   out_ids    DEVICE int64 [s][k], out_scores DEVICE fp32 [s][k] (written)
 *   G >= 1, 1 <= k <= RALM_MAX_K; global ids must stay below 2^32. s == 0 is a no-op.
 * Between GPUs the [G][s][k] arrays are what an all-gather of each rank's [s][k] answer
 * produces: G * s * k * 12 bytes in all. Needs no index. Asynchronous on `stream`. */
ralm_status_t ralm_merge_lists(const int64_t *ids, const float *scores, const int64_t *row_offset, int32_t G,
                               int32_t s, int32_t k, ralm_metric_t metric, int64_t *out_ids, float *out_scores,
                               void *stream);

/* Testing aids for the failure paths (neither is needed in normal use).
 *
 * ralm_debug_fail_allocation: the nth device allocation the library makes from now on (1 = the
 *   next one) fails as if the device were out of memory; 0 switches the injection off. Lets a
 *   test see ralm_index_create return RALM_ERR_OOM and give back what it had already allocated.
 *   Process-wide; not for concurrent use with real work.
 * ralm_selftest_wait_timeout: runs the library's bounded wait on a barrier that nothing ever
 *   completes, with a limit of `limit_cycles` SM clock cycles (1 .. 2e9). The kernel must return
 *   by itself and set *device_status (DEVICE int32, zeroed by the caller) to RALM_ERR_TIMEOUT,
 *   which is how every pipeline wait of the scan kernels ends when its partner never arrives.
 *   Asynchronous on `stream`. */
ralm_status_t ralm_debug_fail_allocation(int32_t nth);
ralm_status_t ralm_selftest_wait_timeout(int64_t limit_cycles, int32_t *device_status, void *stream);

/* Static description of a status code. */
const char *ralm_status_string(ralm_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* RALM_H_ */
