/*
 * sloweave — C ABI of the B200 (sm_100a) mixed prefill-chunk + decode attention iteration and of the
 * SLOWeave chunk controller.
 *
 * One serving iteration decodes one token for every active request and optionally processes one
 * prefill chunk (Sec. 4.1); the controller admits the largest chunk whose predicted iteration cost still
 * meets the earliest next-token deadline (Sec. 3.1-3.2, Eq. (1), Algorithm 1).  The paper leaves the
 * attention kernels and the paged KV layout untouched (Sec. 1, Sec. 5.1, Table 1), so the attention itself
 * is textbook scaled-dot-product attention over a paged bf16 KV cache.
 *
 * Conventions
 *   - Plain C99 types; no exceptions cross the boundary; every call returns an sw_status.
 *   - "device" pointers are CUDA device memory owned by the caller; the library never frees them and
 *     allocates no device memory after sw_create (sw_create itself allocates none either: all scratch is
 *     the caller's workspace).
 *   - `stream` is a cudaStream_t passed as void*.  Launching calls are asynchronous on that stream.
 *     One sw_ctx serves one stream at a time (its scratch and counters are shared by its launches).
 *   - A context belongs to the device it was created on.  Launching calls (sw_kv_append, sw_mixed_attn_run,
 *     sw_mixed_iteration_run, sw_mixed_iteration_host, the cost probes) require that device to be the caller's
 *     current CUDA device and return SW_ERR_INVALID_ARG otherwise; no call changes the current device
 *     (sw_create sets `device` for its own set-up and restores the caller's).
 *   - bf16 tensors are dense, row-major, innermost index last.  The pool, q, k_new, v_new and out must start
 *     on a 16-byte boundary (the copy engine reads and writes them through tensor maps); a call given a
 *     pointer that does not returns SW_ERR_INVALID_ARG and launches nothing.
 *   - KV pool layout (elements, bf16):  [num_pages][2 (0 = K, 1 = V)][num_kv_heads][page_size][head_dim].
 *     The pool must hold finite values everywhere a page list can reach (initialise it with zeros): the
 *     unwritten slots of a partly filled last page are read and multiplied by a zero weight.
 *   - Row order of q / k_new / v_new / out: rows 0..C-1 are the prefill chunk tokens (chunk token j has
 *     absolute position P + j), rows C..C+n-1 are the decode tokens of requests 0..n-1.
 *   - Query head h reads KV head floor(h / (num_q_heads / num_kv_heads)).
 */
#ifndef SLOWEAVE_SW_H
#define SLOWEAVE_SW_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SW_OK = 0,
    SW_ERR_INVALID_ARG = 1,    /* null pointer, negative size, inconsistent arguments */
    SW_ERR_OUT_OF_RANGE = 2,   /* page id / length / chunk outside pool, prompt or table grid */
    SW_ERR_UNSUPPORTED = 3,    /* head_dim, page_size, GQA ratio or device architecture not supported */
    SW_ERR_WORKSPACE = 4,      /* caller's workspace too small or misaligned */
    SW_ERR_CUDA = 5,           /* a CUDA runtime / driver call failed; see sw_last_error() */
    SW_ERR_DEVICE_TIMEOUT = 6, /* a bounded device-side wait gave up */
    SW_ERR_NOT_MONOTONE = 7    /* cost table not nondecreasing and make_monotone == 0 */
} sw_status;

typedef struct sw_ctx sw_ctx;               /* opaque; owns tensor-map cache and pointers into the workspace */
typedef struct sw_cost_table sw_cost_table; /* opaque host object */

/* Attention shape and pool geometry.  Supported: head_dim 64 or 128; page_size 16;
 * num_q_heads / num_kv_heads in {1, 2, 4, 8}; num_pages <= 2^30 and 2 * num_pages * num_kv_heads < 2^31
 * (the copy engine addresses a page's K or V of one head by a 32-bit block index). */
typedef struct {
    int32_t num_q_heads, num_kv_heads, head_dim, page_size;
    int64_t num_pages; /* pages in every pool passed to this context */
    float sm_scale;    /* softmax scale; <= 0 selects 1/sqrt(head_dim) */
} sw_layout;

/* One mixed iteration (Sec. 4.1): one prefill chunk of C tokens at cached-prefix offset P of one prompt,
 * plus the next token of each of n active decodes.  Pointers are DEVICE pointers. */
typedef struct {
    int32_t prefix_len;               /* P >= 0 */
    int32_t chunk_len;                /* C >= 0; 0 = decode-only iteration */
    const int32_t* prefill_pages;     /* [num_prefill_pages] page ids of the prompt, in order */
    int32_t num_prefill_pages;        /* >= ceil((P + C) / page_size) */
    int32_t num_decode;               /* n >= 0; 0 = prefill-only iteration */
    const int32_t* decode_kv_len;     /* [n] keys attended by request i, INCLUDING the token appended now */
    const int32_t* decode_page_indptr;/* [n+1] CSR offsets into decode_pages */
    const int32_t* decode_pages;      /* [indptr[n]] page ids */
    /* Several prefill chunks in one iteration (Sec. 3.3, "Prefill batching"): with num_chunks > 0 the three arrays
     * below, which are HOST arrays, replace prefix_len / chunk_len.  Chunk j has chunk_lens[j] tokens at prefix
     * chunk_prefix_lens[j] of its own prompt; its rows follow those of chunk j-1 in q / k_new / v_new / out (C is then
     * the sum of the chunk lengths), and its prompt's page list is
     * prefill_pages[chunk_page_indptr[j] .. chunk_page_indptr[j+1]) with chunk_page_indptr[num_chunks] ==
     * num_prefill_pages.  At most SW_MAX_CHUNKS chunks; list the longest first (they are scheduled in this order).
     * num_chunks == 0 (all three pointers ignored) is the single chunk described by prefix_len / chunk_len. */
    int32_t num_chunks;
    const int32_t* chunk_prefix_lens;
    const int32_t* chunk_lens;
    const int32_t* chunk_page_indptr;
} sw_batch;
#define SW_MAX_CHUNKS 8

/* ---- context -------------------------------------------------------------------------------------- */

/* Bytes of device workspace a context needs for iterations of at most max_chunk chunk tokens and
 * max_decode decode requests (split-KV partial results, tickets, counters, status words, and staging for
 * sw_mixed_iteration_host with at most max_pages page-table entries).  Returns 0 on invalid arguments. */
size_t sw_workspace_bytes(const sw_layout* layout, int32_t max_chunk, int32_t max_decode, int64_t max_pages);

/* Create a context on CUDA device `device`.  `workspace` is device memory of at least
 * sw_workspace_bytes(...) bytes, 256-byte aligned, owned by the caller and kept alive until sw_destroy.
 * Its contents are initialised here (synchronously).  Fails with SW_ERR_UNSUPPORTED on a device that is not
 * compute capability 10.x or on an unsupported shape. */
sw_status sw_create(const sw_layout* layout, int device, void* workspace, size_t workspace_bytes,
                    int32_t max_chunk, int32_t max_decode, int64_t max_pages, sw_ctx** out);
void sw_destroy(sw_ctx* ctx);

/* ---- the hot path ----------------------------------------------------------------------------------- */

/* KV manager step (Table 1): write this iteration's new K/V rows into the pool.  k_new / v_new are device
 * bf16 [C+n][num_kv_heads][head_dim].  Chunk row j goes to position P+j of the prompt's page list, decode row
 * i to position decode_kv_len[i]-1 of request i's list.  One kernel launch, asynchronous.  Page ids or
 * positions outside their list / the pool are skipped and reported by sw_check_status.  (The attention calls
 * below report a page id outside the pool the same way and read page 0 in its place; their output for the
 * affected rows is then meaningless.) */
sw_status sw_kv_append(sw_ctx* ctx, void* kv_pool, const sw_batch* batch, const void* k_new, const void* v_new,
                       void* stream);

/* Executor step (Sec. 4.1; Fig. 1 card 4): attention of the whole mixed iteration in ONE kernel launch —
 * chunk-prefill tiles on the tensor cores (chunk row j attends keys 0..P+j inclusive), split-KV decode
 * units and their combine.  q, out: device bf16 [C+n][num_q_heads][head_dim].  lse: device fp32
 * [C+n][num_q_heads] (natural-log sum-exp of the scaled scores) or NULL.  The K/V of this iteration's rows
 * must already be in the pool (call sw_kv_append first on the same stream).  Asynchronous. */
sw_status sw_mixed_attn_run(sw_ctx* ctx, const void* kv_pool, const sw_batch* batch, const void* q, void* out,
                            float* lse, void* stream);

/* KV manager step and executor step of one iteration in ONE kernel launch: what sw_kv_append followed by
 * sw_mixed_attn_run computes, without the second launch and the gap between the two.  Every CTA of the persistent
 * grid first writes its share of the k_new / v_new rows into the pool; the chunk-prefill tiles that reach into the
 * chunk's own keys and the decode units that reach a request's last page wait (bounded) until every CTA has done so.
 * Arguments as for the two calls.  Contract beyond theirs: no page of a decode request other than its last, and no
 * page below the chunk's first row, is written by this call (true of any page table in which requests own their
 * pages, shared prompt prefixes included).  Asynchronous.
 * The waits need every CTA of the persistent grid to be resident at once.  sw_create checks that (occupancy of the
 * kernel times the SM count against the grid); on a device where it does not hold this call issues the append as a
 * launch of its own before the attention launch, with the same results. */
sw_status sw_mixed_iteration_run(sw_ctx* ctx, void* kv_pool, const sw_batch* batch, const void* k_new, const void* v_new,
                                 const void* q, void* out, float* lse, void* stream);

/* The same iteration from HOST buffers: copies q / k_new / v_new and the page tables to the device (into the
 * workspace), runs sw_mixed_iteration_run, copies `out` (and lse if non-NULL) back and waits.
 * All pointers inside `h_batch` and h_q / h_k_new / h_v_new / h_out / h_lse are HOST pointers (pinned memory
 * makes the copies asynchronous); kv_pool stays a device pointer. */
sw_status sw_mixed_iteration_host(sw_ctx* ctx, void* kv_pool, const sw_batch* h_batch, const void* h_q,
                                  const void* h_k_new, const void* h_v_new, void* h_out, float* h_lse,
                                  void* stream);

/* Profiler step (Sec. 5.1; Sec. 6.4): time the attention of one iteration over a stack of `layers` pools
 * (kv_pools: HOST array of `layers` device pool pointers, used round-robin so that successive launches do
 * not hit the same cache lines).  Runs `warmup` untimed and `reps` timed iterations of `layers` launches
 * each, timed with CUDA events on `stream`; synchronous.  Returns per-ITERATION nanoseconds: median,
 * nearest-rank 99th percentile, and (if samples_ns != NULL) all `reps` samples in run order. */
sw_status sw_cost_probe(sw_ctx* ctx, void* const* kv_pools, int32_t layers, const sw_batch* batch, const void* q,
                        void* out, int32_t warmup, int32_t reps, int64_t* p50_ns, int64_t* p99_ns,
                        int64_t* samples_ns, void* stream);

/* The same measurement for a runtime whose iteration is sw_mixed_iteration_run: every timed launch also appends
 * k_new / v_new (device bf16 [C+n][num_kv_heads][head_dim]) to its pool, so the table holds the cost of what the
 * executor really launches.  The probed pools are written at the batch's append positions. */
sw_status sw_cost_probe_iteration(sw_ctx* ctx, void* const* kv_pools, int32_t layers, const sw_batch* batch,
                                  const void* k_new, const void* v_new, const void* q, void* out, int32_t warmup,
                                  int32_t reps, int64_t* p50_ns, int64_t* p99_ns, int64_t* samples_ns, void* stream);

/* (No counterpart in the paper.)  Decode-only attention for callers that cannot allocate device memory at all — for
 * example a plugin or a real-time serving loop that runs inside someone else's memory pool, where cudaMalloc is
 * forbidden or would synchronise the device, so neither a context nor a workspace can be created.  It computes what
 * sw_mixed_attn_run computes for an iteration with chunk_len == 0 (q, out: device bf16 [n][num_q_heads][head_dim],
 * lse: device fp32 [n][num_q_heads] or NULL; batch pointers are device pointers), but keeps its counters, tickets
 * and split-KV partial results in a fixed array of SW_STATIC_SCRATCH_BYTES that is part of the library image: every
 * GPU that loads the library holds that array until the process exits.  It calls no cudaMalloc / cudaFree and no
 * allocating library routine.
 * Limits: chunk_len must be 0, num_decode <= SW_STATIC_MAX_DECODE, num_kv_heads <= 8; anything larger is refused with
 * SW_ERR_WORKSPACE (SW_ERR_UNSUPPORTED for a prefill chunk).
 * `device` must be the caller's current CUDA device (cudaSetDevice before the call); the call changes no device and
 * refuses with SW_ERR_INVALID_ARG when another device is current.
 * The first call on a device looks up the array's device address, the device properties and the kernel attributes;
 * make that first call outside any stream capture.  All calls share the one array: it is cleared where it must start
 * at zero at the beginning of every call (on `stream`), so calls must not overlap on the GPU — issue them on one
 * stream, or order them yourself; overlapping calls race on the scratch.  Not thread-safe for concurrent first calls.
 * Asynchronous on `stream`; device-side problems are not reported by this variant (a page id outside the pool is
 * never fetched: page 0 is read in its place). */
#define SW_STATIC_MAX_DECODE 128
#define SW_STATIC_SCRATCH_BYTES (7u * 1024u * 1024u)
sw_status sw_decode_attn_static(const sw_layout* layout, int device, const void* kv_pool, const sw_batch* batch,
                                const void* q, void* out, float* lse, void* stream);

/* Wait for `stream` and read the device status words: *code is 0 or the first device-detected problem as an
 * sw_status (bad page id / length → SW_ERR_OUT_OF_RANGE, bounded wait expired → SW_ERR_DEVICE_TIMEOUT),
 * *detail an implementation-defined locator.  The words are cleared; after a reported problem the context's
 * work counters and tickets are cleared too, so the next launch starts clean.  Returns *code as status. */
sw_status sw_check_status(sw_ctx* ctx, void* stream, int32_t* code, int32_t* detail);

/* Self-test of the failure path (no counterpart in the paper): launches one warp that waits on a barrier nothing will
 * ever complete.  Every device-side wait of this library is bounded; this one gives up after `budget_cycles` SM cycles
 * (at most 4e9), records SW_ERR_DEVICE_TIMEOUT in the status words and ends normally — the context stays usable and
 * sw_check_status then returns SW_ERR_DEVICE_TIMEOUT once.  Asynchronous on `stream`. */
sw_status sw_selftest_wait_timeout(sw_ctx* ctx, int64_t budget_cycles, void* stream);

/* ---- the controller (host only; no CUDA) ---------------------------------------------------------- */

/* Cost table T^(n, ctx, prefix, c) in integer nanoseconds (Sec. 5.1: lookup table indexed by decode batch
 * size, total cached context and candidate prefill tokens; a prefix-length axis is added).  Grids are
 * strictly increasing; cost_ns is [nn][nc][np][nk].  make_monotone != 0 applies the cumulative maximum
 * along the chunk axis (Sec. 5.1) and along the other axes (T is nondecreasing in every argument);
 * make_monotone == 0 requires the input to be nondecreasing already (else SW_ERR_NOT_MONOTONE).
 * interp != 0 selects integer-linear interpolation (rounded up) along the chunk axis (Sec. 6.4); otherwise
 * every coordinate is rounded up to the next grid point. */
sw_status sw_cost_table_create(const int32_t* n_grid, int32_t nn, const int64_t* ctx_grid, int32_t nc,
                               const int32_t* prefix_grid, int32_t np, const int32_t* chunk_grid, int32_t nk,
                               const int64_t* cost_ns, int make_monotone, int interp, sw_cost_table** out);
void sw_cost_table_destroy(sw_cost_table* table);
/* Predicted duration; a chunk beyond the last grid point yields INT64_MAX (infeasible); n / ctx / prefix
 * beyond their grids yield SW_ERR_OUT_OF_RANGE. */
sw_status sw_cost_table_lookup(const sw_cost_table* table, int64_t n, int64_t ctx, int64_t prefix, int64_t c,
                               int64_t* cost_ns);

typedef struct {
    int64_t margin_abs_ns; /* delta = margin_abs_ns + ceil(T^ * margin_ppm / 1e6)  (Sec. 3.3, prediction error) */
    int32_t margin_ppm;
    int32_t c_max;         /* C_max, the cap also used when no decode is active (Sec. 3.1) */
    int32_t chunk_quantum; /* 1 = any integer chunk; q > 1 restricts to multiples of q that are <= L */
} sw_chooser_params;

#define SW_F_NO_PREFILL 1        /* nothing pending: chunk = 0 */
#define SW_F_NO_DECODE 2         /* no active decode: chunk = L without consulting the table */
#define SW_F_DECODE_INFEASIBLE 4 /* even the decode-only iteration misses the earliest deadline */
#define SW_F_CAPPED 8            /* c_max < remaining */

typedef struct {
    int32_t chunk;        /* chosen c* */
    int32_t flags;        /* SW_F_* */
    int64_t budget_ns;    /* B = max(0, min_i d_i - now) */
    int64_t predicted_ns; /* T^ + delta at the chosen chunk (INT64_MAX never; 0 when no table query was made) */
    int32_t queries;      /* table reads made by the bisection */
} sw_choice;

/* Several prefills in one iteration by first fit (Sec. 3.3, "Prefill batching").  The pending requests are given
 * oldest first (HOST arrays prefix_lens / remaining_prefill, num_pending entries; at most SW_MAX_CHUNKS are looked at).
 * With t tokens admitted so far and S the sum of the admitted requests' prefix lengths, request j may add c tokens if
 * T^(n, ctx, S + prefix_lens[j], t + c) + delta <= B: the prediction for the total number of prefill tokens at the
 * summed prefix bounds the arithmetic and the K/V traffic of the separate chunks from above.  A request that fits
 * whole (L_j = min(C_max - t, remaining_j) tokens) is followed by the next; the first one that does not is cut by the
 * bisection of Algorithm 1 and ends the list, so the search stays logarithmic.  Without active decodes requests are
 * admitted whole up to C_max tokens.  chunks receives the admitted lengths (room for SW_MAX_CHUNKS), *num_chunks their
 * count; out->chunk is their sum, out->predicted_ns the prediction for the admitted list.  With one pending request
 * the result equals sw_choose_chunk's. */
sw_status sw_choose_chunks(const sw_cost_table* table, const sw_chooser_params* params, int64_t now_ns,
                           const int64_t* deadlines_ns, int32_t n_active, int64_t total_ctx, const int32_t* prefix_lens,
                           const int32_t* remaining_prefill, int32_t num_pending, int32_t* chunks, int32_t* num_chunks,
                           sw_choice* out);

/* ---- telemetry (host only; no CUDA) --------------------------------------------------------------- */

/* Residual table of the online feedback loop (Table 1 "Telemetry"; Sec. 3.3 "Prediction error"; Sec. 5.1).  Every
 * iteration's predicted and observed duration is recorded; the one-sided residual max(0, observed - predicted) goes
 * into the bucket of its (decode count n, chunk c).  n_edges / c_edges are strictly increasing UPPER edges: a value
 * falls into the first bucket whose edge is >= it, values beyond the last edge into the last bucket.  A bucket keeps
 * its most recent `window` residuals. */
typedef struct sw_telemetry sw_telemetry;
typedef struct {
    int64_t records;         /* iterations recorded */
    int64_t fallbacks;       /* of those, iterations the caller marked as decode-only fallbacks */
    int64_t deadline_misses; /* of those, iterations recorded with a negative deadline slack */
    int64_t max_residual_ns; /* largest residual seen */
} sw_telemetry_totals;
sw_status sw_telemetry_create(const int32_t* n_edges, int32_t num_n, const int32_t* c_edges, int32_t num_c, int32_t window,
                              sw_telemetry** out);
void sw_telemetry_destroy(sw_telemetry* t);
/* slack_ns = earliest deadline - end of the iteration (negative = a missed deadline); fallback != 0 marks an
 * iteration that ran decode-only because sw_telemetry_exceeds said so. */
sw_status sw_telemetry_record(sw_telemetry* t, int32_t n, int32_t c, int64_t predicted_ns, int64_t observed_ns,
                              int64_t slack_ns, int32_t fallback);
/* The margin delta(n, c) to reserve (Sec. 3.3): the nearest-rank percentile (percentile_ppm of 1e6, e.g. 990000) of a
 * bucket's residuals, floor_ns for a bucket with fewer than min_samples of them, maximised over all buckets at or
 * below the bucket of (n, c) in both coordinates so that the margin is nondecreasing in n and in c (the feasibility
 * test of Algorithm 1 has to stay monotone).  Pass the result as sw_chooser_params.margin_abs_ns. */
sw_status sw_telemetry_margin(const sw_telemetry* t, int32_t n, int32_t c, int32_t percentile_ppm, int32_t min_samples,
                              int64_t floor_ns, int64_t* margin_ns);
/* Fallback signal (Sec. 5.1): *exceeds = 1 when that margin (with floor 0) is larger than configured_margin_ns; the
 * scheduler then runs the iteration decode-only. */
sw_status sw_telemetry_exceeds(const sw_telemetry* t, int32_t n, int32_t c, int32_t percentile_ppm, int32_t min_samples,
                               int64_t configured_margin_ns, int32_t* exceeds);
/* Forgets every residual (the totals stay): to be called when the cost table the predictions come from is replaced
 * (re-profiling, Sec. 5.1), since residuals against the old table say nothing about the new one. */
sw_status sw_telemetry_reset(sw_telemetry* t);
sw_status sw_telemetry_get_totals(const sw_telemetry* t, sw_telemetry_totals* out);

/* The chunk decision of one iteration (Sec. 3.1-3.2, Eq. (1), Algorithm 1): the largest chunk c <= min(C_max,
 * remaining_prefill) whose predicted cost T^(n_active, total_ctx, prefix_len, c) + delta still ends before the
 * earliest of the active decodes' next-token deadlines.  deadlines_ns are absolute deadlines d_i = l_i + D_i (HOST
 * array, n_active entries), so the budget is B = max(0, min_i d_i - now_ns).  Nothing pending (remaining_prefill == 0)
 * gives 0; no active decode gives the capped remainder without a table.  The cost is nondecreasing in c, so the
 * answer is found by bisection (Proposition 1); this implementation bisects over the points of the table's chunk
 * grid and closes the last stretch in closed form, which needs at most ceil(log2(candidates + 1)) table reads.
 * The decode-only cost (c = 0), which decides SW_F_DECODE_INFEASIBLE, is read at prefix 0: an iteration without
 * prefill tokens processes no prompt. */
sw_status sw_choose_chunk(const sw_cost_table* table, const sw_chooser_params* params, int64_t now_ns,
                          const int64_t* deadlines_ns, int32_t n_active, int64_t total_ctx, int32_t prefix_len,
                          int32_t remaining_prefill, sw_choice* out);

/* Thread-local text describing the last non-OK status returned on this thread ("" if none). */
const char* sw_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SLOWEAVE_SW_H */
