/*
 * oilbird.h - C-ABI of the B200-native semantic draft pool.
 *
 * The library implements the nearest-neighbour lookup of Oilbird's semantic draft
 * source (paper Section 4, "(i) Store" and "(ii) Retrieve"; Eq. 1-3; Algorithm 1):
 * a pool keyed by the verifier's hidden state at every committed token is searched
 * with the state at the current position, the top-k past positions are selected and
 * the token continuation behind each one is copied out as a draft chain.
 *
 * Conventions
 *   - Every function returns OILBIRD_OK (0) or a negative OILBIRD_E* code; nothing
 *     throws or aborts.  oilbird_strerror() names a code.
 *   - "dev" pointers are CUDA device pointers on the pool's device, "host" pointers
 *     are ordinary host memory.  The caller owns every buffer it passes in; the pool
 *     owns the keys, tokens, trace table and its scratch.
 *   - bf16 data is passed as raw 16-bit patterns (void* / uint16_t).
 *   - `cuda_stream` is a cudaStream_t (NULL = the default stream).  append and query
 *     only enqueue work; they never synchronise.  The row count is tracked on the
 *     host at enqueue time, so rows are visible to every query enqueued after their
 *     append on the same stream.  Using different streams for append and query is
 *     the caller's synchronisation problem.  One host thread per pool at a time.
 *   - There is no CPU fallback: without a CUDA device create() fails.
 *   - Alignment: bf16 matrices passed in (states, q, and the keys of
 *     oilbird_query_static) must start on a 16-byte boundary, int32 / float arrays on a
 *     4-byte boundary, exclude_tag on an 8-byte boundary; rows are then aligned by
 *     themselves because d is a multiple of 8.  The kernels read them with vector loads, so a
 *     misaligned pointer is refused with OILBIRD_EINVAL before anything is launched.
 */
#ifndef OILBIRD_H_
#define OILBIRD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define OILBIRD_OK         0
#define OILBIRD_EINVAL    (-1)  /* bad argument (null pointer, size out of range, ...) */
#define OILBIRD_ECAPACITY (-2)  /* rows or traces would exceed what create() sized     */
#define OILBIRD_ENOMEM    (-3)  /* device or host allocation failed                    */
#define OILBIRD_ECUDA     (-4)  /* a CUDA call failed; see oilbird_last_cuda_error()   */
#define OILBIRD_ESTALL    (-5)  /* a bounded device-side wait gave up (status only)    */
#define OILBIRD_EGUARD    (-6)  /* oilbird_pool_check_guards found sentinel bytes changed */

#define OILBIRD_MAX_NQ        256   /* queries per call                                */
#define OILBIRD_MAX_K         128   /* neighbours per query                            */
#define OILBIRD_MAX_CONT_LEN  128   /* tokens per continuation                         */
#define OILBIRD_MAX_TIERS     4

/* pool flags (oilbird_pool_config.flags) */
#define OILBIRD_KEYS_E4M3  1u   /* keys are stored as FP8 E4M3 codes with one fp32 scale
                                   per row instead of bf16 (see "8-bit keys" below)     */
#define OILBIRD_DEBUG_GUARDS 2u /* debugging aid: every array of the pool's allocation is
                                   followed by sentinel bytes (from its last byte to the
                                   next array, at least 256) that no kernel may touch;
                                   see oilbird_pool_check_guards                        */

/* append flags */
#define OILBIRD_NEW_TRACE  1u   /* the rows open a new trace (a finished request)      */
#define OILBIRD_EVICT_TO_FIT 2u /* bounded store: if the rows (or the new trace) do not fit,
                                   the fewest oldest traces are evicted first, as by
                                   oilbird_pool_evict_oldest (never the trace being extended);
                                   OILBIRD_ECAPACITY only if that cannot make room        */

/* depth modes (Eq. 3 and the fixed-span variant of the batched harness) */
#define OILBIRD_DEPTH_FIXED   0  /* every neighbour copies cont_len tokens             */
#define OILBIRD_DEPTH_TIERED  1  /* D(s): first tier whose floor the score reaches     */
#define OILBIRD_DEPTH_RANKED  2  /* by rank (Section 6, "Retrieval granularity", the arm
                                    the paper compares D(s) with; it gives no schedule, this
                                    is the library's reading): neighbour j, best first from
                                    0, copies tier_depth[j] tokens, the last entry from
                                    j = n_tiers - 1 on; tier_thr is not looked at         */

/* which scoring kernel runs */
#define OILBIRD_PATH_AUTO    0   /* chosen from nq, the pool's size and its key format  */
#define OILBIRD_PATH_GEMV    1   /* CUDA-core scan (single-request decode)             */
#define OILBIRD_PATH_TENSOR  2   /* tcgen05 tensor-core scan (batched queries)         */
#define OILBIRD_PATH_MMA     3   /* warp-level tensor-core scan (small batches):
                                    d a multiple of 128 (256 for 8-bit keys), k <= 64   */

typedef struct oilbird_pool oilbird_pool_t;   /* opaque */

/*
 * Pool geometry, fixed at creation (Eq. 1: one record (x_i, h_i) per committed
 * generated position, the state stored L2-normalised in 16-bit floating point).
 */
typedef struct {
  int32_t  d;              /* key width d_model; a multiple of 8, 8..16384              */
  int64_t  capacity_rows;  /* rows the pool can hold; arrays are never reallocated      */
  int32_t  max_traces;     /* trace-table capacity; 0 = min(capacity_rows, 1<<20)       */
  int32_t  max_nq;         /* largest nq a query will use (<= OILBIRD_MAX_NQ); 0 = 256  */
  int32_t  max_k;          /* largest k (<= OILBIRD_MAX_K); 0 = 64                      */
  int32_t  max_append;     /* largest n of the *_host append variant; 0 = 4096          */
  int32_t  device;         /* CUDA ordinal                                              */
  uint32_t flags;          /* 0, OILBIRD_KEYS_E4M3, OILBIRD_DEBUG_GUARDS                */
  void*    arena;          /* dev, optional: caller-provided memory (256-B aligned) of  */
  size_t   arena_bytes;    /*   at least oilbird_pool_arena_bytes(); NULL = cudaMalloc  */
} oilbird_pool_config;

/*
 * Retrieval parameters (Algorithm 1's Require line; Eq. 2; Eq. 3).
 * oilbird_query_params_default() fills in the values the paper deploys.
 */
typedef struct {
  int32_t  k;                               /* neighbours, paper: 8                     */
  float    theta;                           /* firing floor on the best score, 0.8      */
  int32_t  offset;                          /* copy starts at row idx+offset, paper: 2  */
  int32_t  depth_mode;                      /* OILBIRD_DEPTH_*                          */
  int32_t  cont_len;                        /* L: row length of cont_tok and the cap on
                                               every depth; the fixed depth itself      */
  int32_t  n_tiers;                         /* tiers of D(s), tested in order           */
  float    tier_thr[OILBIRD_MAX_TIERS];     /* paper: 0.90, 0.82                        */
  int32_t  tier_depth[OILBIRD_MAX_TIERS];   /* paper: 48, 8 (0 below every tier)        */
  const uint64_t* exclude_tag;              /* dev [nq] or NULL: rows of traces whose
                                               tag equals a non-zero entry are skipped
                                               (a request must not draft from a stored
                                               copy of its own prompt's trace).  A
                                               DEVICE pointer on purpose, like q: the
                                               scan reads it, and a host pointer would
                                               cost a copy and a staging buffer on the
                                               latency path; the *_host entry points
                                               take a host pointer and upload it with
                                               the queries                              */
  int32_t  path;                            /* OILBIRD_PATH_*                           */
} oilbird_query_params;

/* Query results.  All five arrays are written on every call. */
typedef struct {
  int32_t* idx;       /* [nq,k]   pool row of each neighbour, best first (score
                                  descending, lower row first among equal scores);
                                  -1 where fewer than k rows were eligible             */
  float*   score;     /* [nq,k]   cosine similarity; -INF where idx == -1              */
  int32_t* fired;     /* [nq]     1 iff the best score >= theta (Eq. 2)                */
  int32_t* cont_len;  /* [nq,k]   tokens copied for each neighbour (0 if not fired)    */
  int32_t* cont_tok;  /* [nq,k,L] the continuation, padded with -1                     */
} oilbird_query_out;

/* Counters accumulated on the device since create()/reset(). */
typedef struct {
  int64_t degenerate_rows;     /* appended rows that were all zero or held NaN/Inf and
                                  were therefore stored as zero keys                   */
  int64_t nonfinite_queries;   /* queries holding NaN/Inf (they return no neighbours)  */
  int32_t stalled;             /* non-zero if a bounded device-side wait ever gave up  */
  int32_t reserved;
} oilbird_pool_stats;

void   oilbird_query_params_default(oilbird_query_params* p);
size_t oilbird_pool_arena_bytes(const oilbird_pool_config* cfg);

/*
 * Lifecycle.  create() validates cfg, allocates (or carves the arena) and sets the
 * pool empty.  reset() empties it (rows = traces = 0, counters cleared) in stream
 * order without freeing anything.  destroy() synchronises the device and frees.
 *
 * Module loading and programmatic launches.  create loads all of the library's kernels and
 * sets their attributes before anything is launched, so that a query's first call does
 * nothing a later call does not do.  The kernels of a step can be chained with programmatic
 * stream serialization (a kernel is set up on the GPU while its predecessor still runs:
 * about 6 us per step on a 90 us step).  The library does that only when the process loads
 * CUDA modules eagerly (CUDA_MODULE_LOADING=EAGER in the environment before CUDA is
 * initialised; the Python binding, bench.py and the tests set it) and only for scans short
 * enough to gain from it (pools up to 4 GB of keys); in every other case, lazy loading (the
 * CUDA default) included, its launches are plain ones, and nothing needs to be set for the
 * library to be safe.  Reason: with lazy loading and chained launches the first steps of a
 * process were seen to dead-lock now and then on the largest configuration; the mechanism
 * inside the driver was not established, so the combination is simply not used.  A chained
 * kernel releases its successor only after its own predecessor has finished: at most two of
 * the library's grids are on the GPU at a time.
 */
int oilbird_pool_create (oilbird_pool_t** out, const oilbird_pool_config* cfg);
int oilbird_pool_reset  (oilbird_pool_t* pool, void* cuda_stream);
int oilbird_pool_destroy(oilbird_pool_t* pool);

/*
 * Store (Eq. 1; last line of Algorithm 1: a finished request's trace joins the pool).
 * Appends n rows: key = bf16(x / ||x||_2) (norm and scaling in double precision, one
 * rounding to float and one to bf16, round-to-nearest-even), token, trace
 * membership.  With OILBIRD_NEW_TRACE the rows open a new trace carrying trace_tag
 * (0 = never excluded); otherwise they extend the newest trace and trace_tag is
 * ignored.  The first append to an empty pool always opens a trace.  n = 0 is legal.
 * states: dev [n,d] bf16 row-major; tokens: dev [n] int32.
 * Errors: EINVAL (null pointers, n < 0), ECAPACITY (rows or traces exhausted;
 * nothing is appended).
 */
int oilbird_pool_append(oilbird_pool_t* pool, const void* states_bf16, const int32_t* tokens,
                        int64_t n, uint64_t trace_tag, uint32_t flags, void* cuda_stream);

/*
 * Retrieve (Algorithm 1: the cosine of the query state with every stored state, top-k,
 * the theta test, the depth D(s_i) and the copy that starts two rows on; Eq. 2; Eq. 3).
 * For each of the nq query states: L2-normalise and round to bf16 (as a key is),
 * score every stored row by the dot product of the two bf16 vectors accumulated in
 * fp32, keep the k best by (score descending, row ascending), set fired, give each
 * neighbour its depth (cont_len, or D(score); 0 if not fired) and copy
 * min(depth, trace_end - (idx+offset)) tokens starting at row idx+offset of the
 * token stream, never past the end of the trace that holds idx.
 * q: dev [nq,d] bf16 row-major.  out: dev arrays as described above.
 * Errors: EINVAL (nq, k, cont_len, n_tiers out of range for this pool; null
 * pointers).  An empty pool is legal and yields idx = -1 everywhere.
 */
int oilbird_pool_query(oilbird_pool_t* pool, const void* q_bf16, int32_t nq,
                       const oilbird_query_params* params, const oilbird_query_out* out,
                       void* cuda_stream);

/*
 * Fire / depth / copy alone (Eq. 2's condition and Eq. 3) for neighbours the caller
 * already holds: idx dev [nq,k] (best first; -1 = none), score dev [nq,k].
 * Writes out->fired, out->cont_len, out->cont_tok; out->idx / out->score are not
 * touched and may be NULL.
 */
int oilbird_pool_gather(oilbird_pool_t* pool, const int32_t* idx, const float* score,
                        int32_t nq, const oilbird_query_params* params,
                        const oilbird_query_out* out, void* cuda_stream);

/*
 * Eviction, for a bounded store (the paper's Limitations section names eviction as one way
 * to keep the store bounded and defines no policy).  Drops the n_traces oldest traces
 * (all of them if there are fewer) with their rows and moves the rest to the front: the
 * pool afterwards is exactly the pool that the remaining traces alone would have built,
 * rows and traces renumbered from zero, so row numbers returned by earlier queries are
 * stale.  The global positions given to oilbird_pool_append_global are kept.  The live rows
 * are read and written once (a cooperative kernel on cuda_stream); the call also waits for
 * earlier work on cuda_stream when it publishes the renumbered trace table.
 * *rows_dropped (may be NULL) receives the number of rows removed.
 */
int oilbird_pool_evict_oldest(oilbird_pool_t* pool, int32_t n_traces, int64_t* rows_dropped,
                              void* cuda_stream);

/*
 * One serving step with DEVICE buffers: oilbird_pool_append (the n rows committed since
 * the last step; n may be 0) followed by oilbird_pool_query, in one call, with the same
 * arguments, results and error codes as the two calls (Algorithm 1 runs once per decoding
 * step: the accepted tokens' states are stored, then the new last position is looked up).
 * Nothing is appended if the call is refused (invalid arguments or parameters, or a scan
 * path this pool does not offer).  For the single-request scan
 * (nq <= 2; 16-bit and 8-bit pools) and the warp-level tensor scan in its 8-query form
 * (OILBIRD_PATH_MMA, nq <= 8), and up to 64 rows, the append has no kernel of its own: the
 * first CTAs of the scan normalise the rows before they start scanning (a row per CTA, or a
 * row per warp that has no query to prepare), and the warps that reach the
 * appended rows (the last rows of the pool) first wait, bounded, for a counter that says
 * all n have been written (a time-out raises the `stalled` status, see oilbird_pool_status).
 */
int oilbird_pool_step(oilbird_pool_t* pool, const void* states_bf16, const int32_t* tokens,
                      int64_t n, uint64_t trace_tag, uint32_t flags, const void* q_bf16,
                      int32_t nq, const oilbird_query_params* params,
                      const oilbird_query_out* out, void* cuda_stream);

/*
 * The same two operations with HOST buffers.  append_host copies its inputs into pinned
 * staging and enqueues upload + append; the caller's buffers are free again when it
 * returns, the rows are visible to later calls on the same stream.  query_host uploads
 * the queries (one copy), runs the query and returns after the results have landed in the
 * host arrays of `out` (it synchronises cuda_stream; the kernels write the results into
 * device-mapped pinned memory, so there is no copy back to wait for).
 * params->exclude_tag and every array of `out` are host pointers here.
 * n <= cfg.max_append.  All *_host calls of a pool must use one stream: the staging
 * buffers are reused in stream order.
 */
int oilbird_pool_append_host(oilbird_pool_t* pool, const void* states_bf16_host,
                             const int32_t* tokens_host, int64_t n, uint64_t trace_tag,
                             uint32_t flags, void* cuda_stream);
int oilbird_pool_query_host(oilbird_pool_t* pool, const void* q_bf16_host, int32_t nq,
                            const oilbird_query_params* params, const oilbird_query_out* out_host,
                            void* cuda_stream);

/* One serving step with host buffers: append_host (the rows committed since the last
 * step; n may be 0) followed by query_host, in one call. */
int oilbird_pool_step_host(oilbird_pool_t* pool, const void* states_bf16_host,
                           const int32_t* tokens_host, int64_t n, uint64_t trace_tag,
                           uint32_t flags, const void* q_bf16_host, int32_t nq,
                           const oilbird_query_params* params, const oilbird_query_out* out_host,
                           void* cuda_stream);

/*
 * The same step in two halves, so that the host work of one step (packing its inputs,
 * reading its results) overlaps the device work of another: several requests share a
 * pool and their lookups do not depend on one another.  `begin` copies the inputs into
 * the pinned block of `slot` (0 <= slot < OILBIRD_HOST_SLOTS; the caller's buffers are
 * free again when it returns), uploads them on a copy stream of the pool's own into the
 * slot's device staging block (so the upload runs under the kernels of the step before),
 * enqueues the step on cuda_stream behind that upload and returns without waiting; the
 * merge kernel writes the results into the slot's mapped block.  `end` waits
 * for that step alone (an event behind its kernels) and copies the results into the host
 * arrays of `out`, whose shape is the one `begin` was given (nq, params->k,
 * params->cont_len).  A slot holds one step: `begin` on a slot whose `end` has not been
 * called, and `end` on an idle slot, return OILBIRD_EINVAL and do nothing.  Steps take
 * effect in the order of their `begin` calls (one stream); `end` may be called in any
 * order.  params->exclude_tag is a host pointer, read during `begin`.  The synchronous
 * *_host calls have a slot and a staging block of their own and may be mixed in.
 */
#define OILBIRD_HOST_SLOTS 2
int oilbird_pool_step_host_begin(oilbird_pool_t* pool, const void* states_bf16_host,
                                 const int32_t* tokens_host, int64_t n, uint64_t trace_tag,
                                 uint32_t flags, const void* q_bf16_host, int32_t nq,
                                 const oilbird_query_params* params, int32_t slot,
                                 void* cuda_stream);
int oilbird_pool_step_host_end(oilbird_pool_t* pool, int32_t slot,
                               const oilbird_query_out* out_host);

/* Introspection (host side; none of these enqueue work unless stated). */
int64_t oilbird_pool_size(const oilbird_pool_t* pool);          /* rows appended so far  */
int32_t oilbird_pool_num_traces(const oilbird_pool_t* pool);
/* Synchronises cuda_stream, then reports the device counters. Returns OILBIRD_ESTALL
 * if a device-side wait ever gave up, else OILBIRD_OK. */
int oilbird_pool_status(oilbird_pool_t* pool, oilbird_pool_stats* stats, void* cuda_stream);
/*
 * Bounded waits.  The library's kernels wait on the device in three places only: a scan that
 * also appends the step's rows waits for a row counter, the tensor-core scan's warps wait
 * on shared-memory barriers for each other, and the candidate CTAs of a one-launch index
 * lookup wait for the flag word that hands them the probes (the recycled pool's fused step
 * waits like the first).  Every such wait gives up after limit_ns
 * nanoseconds (0 = the default, two seconds): the kernel raises the `stalled` status, lets
 * the copies it has in flight land, frees what it holds and returns, so the context stays
 * usable; oilbird_pool_status then returns OILBIRD_ESTALL until reset().  set_wait_limit
 * takes effect in stream order.  stall_selftest runs one small kernel that performs the
 * three kinds of wait on things that never happen (a counter nobody advances, a barrier
 * nobody arrives at, a flag nobody raises), so the give-up path can be exercised: after it,
 * status reports the stall.
 */
int oilbird_pool_set_wait_limit(oilbird_pool_t* pool, uint64_t limit_ns, void* cuda_stream);
int oilbird_pool_stall_selftest(oilbird_pool_t* pool, void* cuda_stream);
/*
 * Guard zones (pools created with OILBIRD_DEBUG_GUARDS).  Synchronises cuda_stream and
 * compares every sentinel byte behind the pool's arrays (keys, tokens, trace tables,
 * normalised queries, candidate lists, counters, exchange buffers, host staging) with the
 * value written at creation.  Returns OILBIRD_OK, or OILBIRD_EGUARD with the array and the
 * offset in oilbird_last_cuda_error().  EINVAL for a pool without guard zones.
 */
int oilbird_pool_check_guards(oilbird_pool_t* pool, void* cuda_stream);
/* Copy stored data to host memory (synchronous; for tests and debugging).
 * keys: [n,d] bf16; tokens, trace_ids: [n] int32; rows [row0, row0+n). */
int oilbird_pool_read_rows(oilbird_pool_t* pool, int64_t row0, int64_t n, void* keys_host,
                           int32_t* tokens_host, int32_t* trace_ids_host);
/*
 * 8-bit keys (OILBIRD_KEYS_E4M3).  The paper's Limitations section names quantisation as one
 * way to keep the store bounded and defines none; this is the library's format.  A stored
 * row is d FP8 E4M3 codes c_j and one fp32 scale:
 *     v_j = x_j / ||x||,   scale = fp32(max_j |v_j| / 448),   c_j = e4m3(v_j / scale)
 * (round to nearest, ties to the even code, saturating at +-448; a zero or non-finite row is
 * stored as zero codes with scale 0).  A score is fp32(scale * sum_j qn_j * value(c_j)), the
 * query normalised and rounded to bf16 as for 16-bit pools; everything after the scores is
 * unchanged.  A row takes d + 4 bytes instead of 2d.  d must be a multiple of 16.  Such
 * pools use the CUDA-core scan for one or two queries, the warp-level tensor scan for up to
 * eight (OILBIRD_PATH_MMA: codes as f16, eight queries per pass over the codes, d a multiple
 * of 256, else the CUDA-core scan two queries per pass) and the tcgen05 scan for larger
 * batches from 32 MB of codes on (OILBIRD_PATH_TENSOR: the codes are turned into f16 inside
 * the kernel and read once for the whole batch);
 * oilbird_query_static does not apply, and keys are read back with the call below
 * (oilbird_pool_read_rows then takes keys_host == NULL).
 * codes: [n,d] uint8; scales: [n] fp32; either may be NULL.
 */
int oilbird_pool_read_codes(oilbird_pool_t* pool, int64_t row0, int64_t n, uint8_t* codes_host,
                            float* scales_host);
/* Trace table as the host tracks it: up to max_traces entries each; returns the count. */
int32_t oilbird_pool_read_traces(const oilbird_pool_t* pool, int64_t* start, int64_t* end,
                                 uint64_t* tag, int32_t max_traces);

/*
 * Kernel timing for benchmarks: when enabled, every query brackets its scan kernel
 * with CUDA events on the caller's stream.  profile_read() synchronises those events
 * and returns up to max_n scan durations (milliseconds, oldest first) recorded since
 * the last read, and clears them.  At most 4096 are kept.
 */
int     oilbird_pool_profile(oilbird_pool_t* pool, int32_t enable);
int32_t oilbird_pool_profile_read(oilbird_pool_t* pool, float* scan_ms, int32_t max_n);
/* Number of kernels this library has launched for this pool since create(). */
int64_t oilbird_pool_launch_count(const oilbird_pool_t* pool);

/*
 * Recycled pool (paper Section 4 "(i b) Recycling"; Algorithm 1, recycled-pool line): a
 * ring buffer of records made from the draft-tree nodes that verification rejected.  A
 * record is keyed by the hidden state in front of the rejected token and by that token
 * (the anchor); its value is the short continuation the model endorsed from there (up to
 * six tokens in the paper).  When the ring is full the oldest record is overwritten.
 * A lookup with the current state and the current anchor token returns, best first, at
 * most m records whose anchor is equal and whose cosine with the query reaches `floor`
 * (paper: m = 4, floor = 0.8; here the floor filters every record, it is not a firing
 * condition); equal scores list the lower slot first.
 */
#define OILBIRD_RING_MAX_M        32   /* results per query                               */
#define OILBIRD_RING_MAX_ROLLOUT  16   /* tokens per stored continuation                  */
#define OILBIRD_RING_MAX_NQ       64   /* queries per call                                */

typedef struct oilbird_ring oilbird_ring_t;   /* opaque */

typedef struct {
  int32_t d;             /* key width, multiple of 8, 8..16384                           */
  int64_t capacity;      /* records (slots) the ring holds                               */
  int32_t max_rollout;   /* tokens per continuation, 1..OILBIRD_RING_MAX_ROLLOUT; 0 = 6  */
  int32_t device;        /* CUDA ordinal                                                 */
} oilbird_ring_config;

typedef struct {         /* all dev, caller-owned, written on every call                 */
  int32_t* slot;         /* [nq,m]  ring slot of each result, -1 padded                  */
  float*   score;        /* [nq,m]  cosine, -INF padded                                  */
  int32_t* count;        /* [nq]    number of results (<= m)                             */
  int32_t* rollout;      /* [nq,m,max_rollout] stored continuation, -1 padded            */
  int32_t* rollout_len;  /* [nq,m]  tokens before the first negative entry               */
} oilbird_ring_out;

int oilbird_ring_create (oilbird_ring_t** out, const oilbird_ring_config* cfg);
int oilbird_ring_destroy(oilbird_ring_t* ring);
int oilbird_ring_reset  (oilbird_ring_t* ring, void* cuda_stream);
int64_t oilbird_ring_size (const oilbird_ring_t* ring);   /* records held (<= capacity)   */
int64_t oilbird_ring_total(const oilbird_ring_t* ring);   /* records ever appended        */
/*
 * Append n records in order; record i goes to slot (total + i) mod capacity.  states: dev
 * [n,d] bf16 (normalised as for the trace pool), anchors: dev [n] int32, rollouts: dev
 * [n,max_rollout] int32 padded with -1.  If n exceeds the capacity only the last
 * `capacity` records are stored.  Enqueues on cuda_stream; never synchronises.
 */
int oilbird_ring_append(oilbird_ring_t* ring, const void* states_bf16, const int32_t* anchors,
                        const int32_t* rollouts, int64_t n, void* cuda_stream);
/*
 * Lookup for nq (state, anchor) pairs: q dev [nq,d] bf16, q_anchor dev [nq] int32,
 * 1 <= m <= OILBIRD_RING_MAX_M.  Only records whose anchor matches are scored, so the
 * cost is one pass over the anchors plus the keys of the matching records.
 * A query holding NaN/Inf returns nothing.  Errors: EINVAL.
 */
int oilbird_ring_query(oilbird_ring_t* ring, const void* q_bf16, const int32_t* q_anchor,
                       int32_t nq, int32_t m, float floor, const oilbird_ring_out* out,
                       void* cuda_stream);
/*
 * One verification pass in one call: oilbird_ring_append of n records (n may be 0) followed by
 * oilbird_ring_query, with the same results as the two calls.  The lookup's own kernel stores
 * the records before it scans (its first blocks take one record each; warps that reach a slot
 * written by the call wait, bounded, until all records are in), and the last block of a query
 * to finish merges the blocks' candidates and writes the answer, so the pass is one launch
 * (a plain oilbird_ring_query likewise); where the lookup needs more blocks than the GPU seats
 * at once the append gets a launch of its own.
 */
int oilbird_ring_step(oilbird_ring_t* ring, const void* states_bf16, const int32_t* anchors,
                      const int32_t* rollouts, int64_t n, const void* q_bf16,
                      const int32_t* q_anchor, int32_t nq, int32_t m, float floor,
                      const oilbird_ring_out* out, void* cuda_stream);
/* Copy stored records to the host (synchronous; tests and debugging). */
int oilbird_ring_read(oilbird_ring_t* ring, void* keys_host, int32_t* anchors_host,
                      int32_t* rollouts_host);
const char* oilbird_ring_last_error(void);      /* text of the last failing CUDA call     */

/*
 * Row sharding: one logical pool split by whole traces over several pools (one per GPU).
 * The merged answer is what a single pool holding every row at its global position would
 * return (Eq. 2 with the lowest-position tie rule; the theta test of Algorithm 1 on the
 * global best).  Positions are assigned by the caller: append_global() is append() plus
 * the global position of the first appended row, recorded when the call opens a trace (a
 * trace's rows are consecutive globally as they are locally).  A query on a sharded pool
 * is four steps: (1) oilbird_pool_query on every shard with theta = -INFINITY, so that
 * every neighbour gets its depth and continuation; (2) oilbird_pool_to_global on the
 * returned rows; (3) an all-gather of the shards' records (idx, score, cont_len,
 * cont_tok), by the caller's communication library, into one buffer of n_shards equal
 * slices; (4) oilbird_merge_shards, which selects the global top-k by (score descending,
 * global position ascending), applies theta to the merged best and copies the winners'
 * continuations (zero lengths and -1 tokens when not fired).  Depths are those the shards
 * assigned: fixed spans and D(s) are the same on a shard as in the whole pool, depth by rank
 * (OILBIRD_DEPTH_RANKED) is not, so it cannot be used in step (1).
 * gathered: dev, shard s starts at gathered + s*shard_stride; inside a slice, off_gidx
 * (int64 [nq,k], 8-byte aligned), off_score (float [nq,k]), off_len (int32 [nq,k]),
 * off_tok (int32 [nq,k,L]) are byte offsets.  n_shards * k <= 1024.
 */
int oilbird_pool_append_global(oilbird_pool_t* pool, const void* states_bf16,
                               const int32_t* tokens, int64_t n, uint64_t trace_tag,
                               uint32_t flags, int64_t global_row, void* cuda_stream);
int oilbird_pool_to_global(oilbird_pool_t* pool, const int32_t* idx /* dev [n] */,
                           int64_t* global_idx /* dev [n] */, int64_t n, void* cuda_stream);
int oilbird_merge_shards(int32_t n_shards, int32_t nq, int32_t k, int32_t L, float theta,
                         const void* gathered, size_t shard_stride, size_t off_gidx,
                         size_t off_score, size_t off_len, size_t off_tok, int64_t* out_gidx,
                         float* out_score, int32_t* out_fired, int32_t* out_len,
                         int32_t* out_tok, int32_t device, void* cuda_stream);

/*
 * Chain post-filter and tree merge (Algorithm 1, chain collection and merge lines;
 * Section 4 "(iii) Merge"; Eq. 4), for nq requests at once.  For each request the chains
 * are taken in order: the k semantic chains as oilbird_pool_query returns them
 * (cont_tok / cont_len: already by decreasing similarity, depth applied), then `ne` further
 * chains of the caller (lexical branches, recycled-pool continuations).  A semantic chain
 * with fewer than min_len tokens and any chain equal to one collected before it is
 * dropped.  The others are merged into the request's draft tree from the root: a token
 * already carried by a child of the current node is walked for free, any other token buys
 * a node, until `budget` nodes are bought or max_nodes is reached (the chain is cut there
 * and later chains are not reached).  cost = length - longest prefix already in the tree.
 * With root_attached != 0 nothing is shared: every chain hangs from the root as its own
 * branch (the paper's ablation arm).
 * Tree layout per request: node 0 is the root (the anchor token), tree_parent[0] = -1 (a
 * parent entry that does not name another node of the tree is read as -1: that node is
 * detached, nothing is followed out of range);
 * tree_tok / tree_parent [nq,max_nodes] and n_nodes [nq] are read and updated in place
 * (new nodes are numbered in the order they are bought); depth [nq,max_nodes] and mask
 * [nq,max_nodes] are written: bit j of mask[i] is set iff node j is node i or one of its
 * ancestors (the attention mask of tree verification).  status / bought / walked
 * [nq,k+ne]: OILBIRD_CHAIN_* code, nodes paid for (Eq. 4) and prefix walked, per chain.
 * All pointers are dev; extra_* may be NULL when ne = 0, sem_* when k = 0.
 */
#define OILBIRD_TREE_MAX_NODES   64
#define OILBIRD_CHAIN_SHORT        0   /* dropped: empty, or semantic and below min_len   */
#define OILBIRD_CHAIN_DUPLICATE    1   /* dropped: equal to a chain collected before it   */
#define OILBIRD_CHAIN_MERGED       2   /* merged completely                               */
#define OILBIRD_CHAIN_CUT          3   /* merged until the budget or max_nodes ran out    */
#define OILBIRD_CHAIN_NOT_REACHED  4   /* collected, but nothing was left to spend        */
typedef struct {
  int32_t budget;         /* B_ret, paper: 16                                            */
  int32_t max_nodes;      /* tree capacity and row stride, paper: 60; <= 64              */
  int32_t min_len;        /* shortest semantic chain kept, paper: 2                      */
  int32_t root_attached;  /* 0 = merge from the root (deployed), 1 = ablation            */
} oilbird_merge_params;
void oilbird_merge_params_default(oilbird_merge_params* p);
int oilbird_merge_chains(int32_t nq, const int32_t* sem_tok, const int32_t* sem_len, int32_t k,
                         int32_t L, const int32_t* extra_tok, const int32_t* extra_len,
                         int32_t ne, int32_t Le, int32_t* tree_tok, int32_t* tree_parent,
                         int32_t* n_nodes, int32_t* depth, uint64_t* mask, int32_t* status,
                         int32_t* bought, int32_t* walked, const oilbird_merge_params* params,
                         int32_t device, void* cuda_stream);

/*
 * Coarse index (the paper's Limitations section names "an index" next to eviction and
 * quantisation as a way to keep the lookup's cost from growing with the store, and defines
 * none; this is the library's reading): an inverted file over n_lists centroids the caller
 * supplies (raw states, dev [n_lists,d] bf16, normalised like keys; e.g. a sample of stored
 * states).  The pool is left as it is; the index adds, per row, the number of a list.
 *   - A row belongs to the list of the centroid that is the best neighbour of its STORED key
 *     taken as a query state (this library's lookup with k = 1 against the centroids; ties to
 *     the lowest centroid).
 *   - refresh() assigns every row appended since the last refresh and rebuilds the lists.
 *     Rows appended since then (the tail) have no list yet and are always scanned.
 *   - query() takes each query's n_probe best centroids (the same lookup, k = n_probe, at most
 *     OILBIRD_MAX_K), scores the rows of those lists and the tail exactly as
 *     oilbird_pool_query scores them, and returns the k best of them by (score descending,
 *     row ascending) with the firing rule, depths and continuations of Eq. 2 and Eq. 3.
 * The answer is oilbird_pool_query's answer restricted to the candidate rows: identical when
 * every list is probed, otherwise approximate (rows of lists that were not probed cannot be
 * found).  Pools of either key format.  In an 8-bit pool element j of stored row i is
 * fp32(value(code_ij) * scale_i), one rounding (the library's reading); a row is assigned
 * through those elements rounded to bf16, taken as a query state; candidates are scored as
 * oilbird_pool_query scores the rows of an 8-bit pool; training takes the means of the fp32
 * elements.  create() copies the centroids (enqueued on cuda_stream); the
 * caller's array is free again once that work has completed.  After oilbird_pool_reset or
 * oilbird_pool_evict_oldest the row numbers the index holds are stale: call
 * oilbird_index_reset (all rows become tail) and refresh again; until then refresh and query
 * refuse with EINVAL (the pool counts such calls and the index remembers the count its lists
 * were built under).  Index calls enqueue on
 * cuda_stream and use the pool's scratch, so they follow the pool's one-stream, one-thread
 * rule.  Destroy the index before its pool.
 * Launches: a lookup of one query with up to 32 probes and params->path ==
 * OILBIRD_PATH_AUTO is a single kernel (centroid scan, choice of the probes, candidate scan, merge, firing
 * rule and gather; its CTAs meet at four words of device memory per query, with the
 * library's bounded wait: a wait that runs out raises the pool's `stalled` status, and
 * oilbird_index_reset clears the words).  Batches, more probes and any explicit
 * params->path take four launches: oilbird_pool_query on the centroids (scan + merge), the
 * candidate scan, the merge.  The answers are the same.
 */
typedef struct oilbird_index oilbird_index_t;   /* opaque */
int oilbird_index_create (oilbird_index_t** out, oilbird_pool_t* pool, const void* centroids_bf16,
                          int32_t n_lists /* 1..65536 */, void* cuda_stream);
int oilbird_index_refresh(oilbird_index_t* index, void* cuda_stream);
int oilbird_index_reset  (oilbird_index_t* index, void* cuda_stream);
int oilbird_index_query  (oilbird_index_t* index, const void* q_bf16 /* dev [nq,d] */, int32_t nq,
                          int32_t n_probe, const oilbird_query_params* params,
                          const oilbird_query_out* out, void* cuda_stream);
int oilbird_index_destroy(oilbird_index_t* index);
int64_t oilbird_index_rows(const oilbird_index_t* index);        /* rows that have a list   */
/* Copy the index to host memory (synchronous; tests): assign [rows] (list of each row),
 * list_off [n_lists+1], list_rows [rows] (the rows of list l are list_rows[list_off[l] ..
 * list_off[l+1]), in no particular order).  Any pointer may be NULL. */
int oilbird_index_read(oilbird_index_t* index, int32_t* assign_host, int32_t* list_off_host,
                       int32_t* list_rows_host);
/*
 * Training (optional): `iterations` of Lloyd's algorithm on the rows the pool holds now, from
 * the centroids the index has.  One iteration assigns every row as refresh() does and then
 * replaces each centroid that has rows by the mean of its rows' stored keys (a centroid
 * without rows stays).  The mean is taken in fixed point so that it does not depend on the
 * order of the rows: element x contributes trunc(x * 2^30), the integers are summed exactly,
 * and the new raw centroid element is bf16(float(double(sum) / (count * 2^30))), rounded to
 * nearest even twice; the raw centroids are then normalised like any stored row.  Afterwards
 * the lists are rebuilt over all rows (as reset() + refresh()).  Deterministic.  d <= 8192.
 * read_centroids copies the raw centroids ([n_lists, d] bf16) to the host (synchronises).
 */
int oilbird_index_train(oilbird_index_t* index, int32_t iterations, void* cuda_stream);
int oilbird_index_read_centroids(oilbird_index_t* index, void* centroids_bf16_host);
const char* oilbird_index_last_error(void);

/*
 * Query without any allocation (the paper has no counterpart; this serves hosts of the
 * library that own all device memory themselves and must not let a library allocate:
 * for instance a serving engine that reserved the whole of HBM at start-up, where a
 * later driver allocation can fail or stall).  The caller keeps the pool's arrays in
 * its own memory, in the layout oilbird_pool_append produces (keys L2-normalised bf16),
 * and passes them in; results go to caller memory as in oilbird_pool_query.  The
 * candidate lists exchanged between the scan and the merge kernel live in a fixed
 * 1 MiB array inside the library image (reserved on every GPU that loads the library,
 * until the process exits), which bounds the call: nq <= OILBIRD_STATIC_MAX_NQ,
 * k <= OILBIRD_MAX_K, no exclusion tags, CUDA-core scan only (params->path AUTO or
 * GEMV).  Anything larger is rejected with OILBIRD_EINVAL and a message in
 * oilbird_query_static_error().
 * The call enqueues work on cuda_stream and returns; it calls no cudaMalloc / cudaFree.
 * The first call on a device also looks up the array's device address; make that first
 * call before any stream capture begins.  All calls on a device share the array, which
 * keeps the previous call's contents; each call rewrites what it reads and clears its
 * counters first, but two calls that overlap on the GPU (other streams, other threads)
 * race.  One host thread at a time.
 */
#define OILBIRD_STATIC_MAX_NQ 2
typedef struct {
  const void*    keys;       /* dev [n_rows,d] bf16, L2-normalised, row-major             */
  const int32_t* tokens;     /* dev [n_rows]                                              */
  const int32_t* trace_id;   /* dev [n_rows]  trace holding each row                      */
  const int32_t* trace_end;  /* dev [n_traces] one past the last row of each trace        */
  int64_t        n_rows;
  int32_t        d;          /* multiple of 8, 8..16384                                   */
  int32_t        device;     /* CUDA ordinal the arrays live on                           */
} oilbird_static_pool;
int oilbird_query_static(const oilbird_static_pool* pool, const void* q_bf16 /* dev [nq,d] */,
                         int32_t nq, const oilbird_query_params* params,
                         const oilbird_query_out* out, void* cuda_stream);
const char* oilbird_query_static_error(void);   /* why the last call was rejected        */

const char* oilbird_strerror(int code);
const char* oilbird_last_cuda_error(void);    /* text of the last failing CUDA call      */

#ifdef __cplusplus
}
#endif
#endif /* OILBIRD_H_ */
