/*
 * zipline.h - C ABI of the ZipLine barrier-selection library (CUDA, sm_100a).
 *
 * The operation (paper, Section III "The Problem" and Section IV "ZipLine",
 * Algorithm 2): n workers, worker p has R predicted iteration end timestamps
 * e^p_1 <= ... <= e^p_R.  One element is picked per worker to form Z; the
 * waiting time is d_Z = max(Z) - min(Z); the selection returned is
 * Z* = argmin d_Z and the next synchronisation barrier is max(Z*).  When
 * several Z reach the minimum the earliest barrier is taken (Fig. 3's caption
 * says that of equal minima the first one found wins).
 *
 * Every entry point is extern "C", takes plain pointers and sizes, and says
 * for each pointer whether it is host or device memory.  All device work is
 * done by the library's own kernels; there is no CPU fallback.
 */
#ifndef ZIPLINE_H
#define ZIPLINE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct zl_handle zl_handle;      /* opaque; owns device scratch only */

typedef enum {
    ZL_OK = 0,
    ZL_ERR_INVALID_ARG = 1,   /* null/misaligned pointer, size out of range, value outside [0, 2^62) */
    ZL_ERR_UNSUPPORTED = 2,   /* shape or magnitude the kernels cannot take (see zl_create)        */
    ZL_ERR_NOMEM = 3,
    ZL_ERR_CUDA = 4,          /* a CUDA runtime call failed; zl_last_cuda_error() has its code      */
    ZL_ERR_UNSORTED = 5,      /* per instance: a row is not non-decreasing                          */
    ZL_ERR_TIMEOUT = 6        /* per instance: an internal iteration limit was hit                  */
} zl_status;

typedef enum {
    ZL_OBJ_RANGE = 0,  /* d_Z = max(Z) - min(Z): the paper's objective function (Section III)   */
    ZL_OBJ_SUM = 1     /* d_Z = sum_p (max(Z) - z_p): total waiting time of all workers         */
} zl_objective;

enum {
    ZL_FLAG_CHECK_SORTED = 1,  /* verify every row is non-decreasing (one extra pass over the input) */
    ZL_FLAG_FULL_SWEEP = 2,    /* examine every timestamp even where the search could stop early    */
    ZL_FLAG_PREDICTOR = 4,     /* the handle also holds a [max_batch][n][R] buffer for zl_predict_select_batched */
    ZL_FLAG_DEBUG_CHECKS = 8,  /* kernels test every computed index against its buffer before using it and record the
                                  first violation instead of making the access (see zl_debug_report in zipline_debug.h) */
    ZL_FLAG_FORCE_FILTER = 16  /* RANGE: take the filter route even for instances small enough to be sorted whole
                                  (for tests: the route's kernels on shapes a brute-force search can check)        */
};

typedef struct {
    int32_t n_workers;     /* n >= 1                                      */
    int32_t lookahead_R;   /* R >= 1                                      */
    int32_t max_batch;     /* largest B passed to zl_select_batched       */
    int32_t objective;     /* zl_objective                                */
    int32_t device;        /* CUDA device ordinal                         */
    int32_t flags;         /* ZL_FLAG_*                                   */
} zl_config;

/*
 * Create a handle and allocate its device scratch for max_batch instances of
 * n x R timestamps (Section IV: the n x R matrix M, one row per worker).
 * cfg and out are host pointers.  ZL_ERR_UNSUPPORTED if n exceeds
 * zl_max_workers().  The handle is not thread safe; distinct handles are
 * independent.  The caller's current device is the same after the call as before it.
 *
 * Ordering: a handle has ONE set of scratch buffers, and every call on it reads and
 * writes them on the device.  Two calls on the same handle must therefore run one
 * after the other on the device: issue them on one stream, or order them with events.
 * Calls on one handle from two streams (or two host threads) without such ordering race
 * on the scratch and give wrong results; nothing detects it.  Use a handle per stream.
 */
zl_status zl_create(const zl_config *cfg, zl_handle **out);

/*
 * The ZipLine search (Section IV "ZipLine", Algorithm 2) on B independent
 * instances: merge the n sorted rows of an instance into time order (Omega),
 * sweep it keeping the latest element of every worker (Z), evaluate d_Z
 * wherever Z holds all n workers, keep the first minimum, then recover the
 * chosen iteration of every worker.
 *
 *   d_ts      device, read only, [B][n][R] int64 microseconds, 8-byte aligned;
 *             row p of instance b = worker p's end timestamps, non-decreasing,
 *             every value in [0, 2^62).
 *   B         1 .. max_batch.
 *   d_idx     device out, [B][n] int32: 0-based index of the last iteration worker p
 *             finishes at or before the barrier (the element of Z*).
 *   d_barrier device out, [B] int64: max(Z*).
 *   d_wait    device out, [B] int64: the minimum of the configured objective.
 *   d_status  device out, [B] int32 or NULL: ZL_OK, or the per-instance error; an
 *             instance in error gets idx = -1 and barrier = wait = INT64_MIN.
 *   cuda_stream  a cudaStream_t (0 = default stream).  The call only enqueues work
 *             and returns; outputs are valid once the stream has run.  It never
 *             allocates or synchronises.  The caller owns every buffer.  The current
 *             device must be the handle's (cfg.device): ZL_ERR_INVALID_ARG otherwise.
 *
 * Result definition: wait is the minimum of d_Z over all R^n selections;
 * barrier is the smallest max(Z) among the minimisers; idx[p] is the largest i
 * with e^p_i <= barrier.  Returns host-detectable errors only.
 */
zl_status zl_select_batched(zl_handle *h, const int64_t *d_ts, int32_t B,
                            int32_t *d_idx, int64_t *d_barrier, int64_t *d_wait,
                            int32_t *d_status, void *cuda_stream);

/*
 * Phase 1 of ZipLine (Introduction; Section II, first property; Section III): the R future end
 * timestamps of every worker are predicted from its most recent iteration interval under the
 * stable-environment assumption.  The paper gives no formula; this is constant-interval
 * extrapolation, e^p_i = last[p] + i * interval[p] for i = 1..R.
 *
 *   d_last      device, [B][n] int64: latest observed end timestamp of each worker, >= 0.
 *   d_interval  device, [B][n] int64: its most recent iteration interval in microseconds, >= 0.
 *   d_ts        device out, [B][n][R] int64, 16-byte aligned: the matrix zl_select_batched takes.
 *
 * A worker with a negative input gets a row of -1, one whose last prediction would reach 2^62 gets a
 * row of 2^62; zl_select_batched reports ZL_ERR_INVALID_ARG for such an instance.  Asynchronous on
 * cuda_stream; no handle, no scratch.
 */
zl_status zl_predict_batched(const int64_t *d_last, const int64_t *d_interval, int32_t B, int32_t n, int32_t R,
                             int64_t *d_ts, void *cuda_stream);

/*
 * Both phases of ZipLine in one call (the handle must have been created with ZL_FLAG_PREDICTOR, else
 * ZL_ERR_INVALID_ARG).  For the RANGE objective on shapes of more than 4096 timestamps the predicted matrix
 * is never written: the kernels generate e^p_i = last[p] + i * interval[p] where they would read a row, and
 * the filter pass settles a whole worker at once from its interval.  Otherwise (SUM, small shapes) the
 * prediction goes into the handle's own buffer and zl_select_batched runs on it.  Same results either way;
 * outputs, stream and error behaviour as for zl_select_batched (a worker with a negative input, or whose
 * last prediction would reach 2^62, makes its instance ZL_ERR_INVALID_ARG).
 */
zl_status zl_predict_select_batched(zl_handle *h, const int64_t *d_last, const int64_t *d_interval, int32_t B,
                                    int32_t *d_idx, int64_t *d_barrier, int64_t *d_wait, int32_t *d_status,
                                    void *cuda_stream);

/*
 * The paper's baselines (Section IV, Algorithm 1): GridScan designates the row with the earliest first
 * timestamp and, for each of its R points, takes from every other row the point at the shortest distance;
 * FullGridScan (full != 0) designates every row in turn (n*R candidate sets).  The candidate with the
 * smallest max(Z) - min(Z) wins, the first one on ties.  Heuristics: the result is never below
 * zl_select_batched's.  Readings: of two points of a row at equal distance the earlier one is taken, of
 * equal points the one with the lowest index.
 *
 *   d_ts       device, [B][n][R] int64, rows non-decreasing (as for zl_select_batched; not checked here).
 *   d_scratch  device, int64, B*R elements (B*n*R when full): the candidates' d_Z; contents undefined after.
 *   d_idx      device out, [B][n] int32: index of the element of Z* in each row.
 *   d_barrier, d_wait  device out, [B] int64: max(Z*) and max(Z*) - min(Z*).
 * Asynchronous on cuda_stream; no handle.
 */
zl_status zl_gridscan_batched(const int64_t *d_ts, int32_t B, int32_t n, int32_t R, int32_t full,
                              int64_t *d_scratch, int32_t *d_idx, int64_t *d_barrier, int64_t *d_wait,
                              void *cuda_stream);

/*
 * The same search with HOST buffers (same shapes and meaning as above):
 * copies the input to the device, runs the kernels, copies the results back
 * and waits for them.  Staging buffers are allocated by the first such call
 * on a handle (so that call allocates; later ones do not).  h_status may be
 * NULL.  Pinned host memory makes the copies asynchronous to the host until
 * the final wait; pageable memory works too.
 */
zl_status zl_select_batched_host(zl_handle *h, const int64_t *h_ts, int32_t B,
                                 int32_t *h_idx, int64_t *h_barrier, int64_t *h_wait,
                                 int32_t *h_status);

/*
 * Per-position intermediates of the sweep (Section IV "ZipLine": Omega sorted
 * by value, Z updated one element per step) for B small instances, each with
 * N = n*R <= zl_trace_max_elements().  Position k runs over Omega in
 * (timestamp, worker, iteration) order.  All pointers are device memory,
 * [B][N], and any of them may be NULL:
 *   om_t/om_p/om_i  the merged order (step 1: merge)
 *   delta, first    e^p_i - e^p_{i-1} (e^p_1 for i = 1) and first-appearance flag (step 2)
 *   S, cnt          inclusive prefix sums of delta and first (step 3)
 *   next, PM        e^p_{i+1} (INT64_MAX for i = R) and its exclusive prefix maximum (step 3)
 *   d_range         max(om_t, t0, PM) - om_t, t0 = max_p e^p_1; INT64_MAX when undefined (step 4)
 *   w_sum           n*om_t - S where cnt == n, else INT64_MAX (step 4)
 * Asynchronous on cuda_stream; no handle, no scratch.
 */
zl_status zl_trace_batched(const int64_t *d_ts, int32_t B, int32_t n, int32_t R,
                           int64_t *om_t, int32_t *om_p, int32_t *om_i,
                           int64_t *delta, int32_t *first, int64_t *S, int32_t *cnt,
                           int64_t *next, int64_t *PM, int64_t *d_range, int64_t *w_sum,
                           void *cuda_stream);

/*
 * The same search without a handle and without any allocation (the paper has no
 * counterpart; this exists for callers that cannot allocate device memory).
 *
 * Some programs may not call cudaMalloc where they need a barrier decision: a
 * parameter-server thread that runs inside a process whose framework has already
 * claimed all device memory for its own pool, a service with a fixed memory budget
 * that forbids allocation after start-up, or a latency-critical loop that must not
 * take the driver's allocation lock (cudaMalloc and cudaFree can stall every stream
 * of the device).  zl_create allocates the search's scratch with cudaMalloc; this entry
 * point keeps the scratch it needs (per-instance summaries and per-segment partial
 * results) in a fixed array compiled into the library instead, zl_noalloc_scratch_bytes()
 * bytes (about 400 KB) that every GPU using the library holds until the process exits.
 * It calls no cudaMalloc, cudaFree or other allocating routine.  Instances of at most
 * 4096 timestamps in batches of up to four per SM run the one-launch kernel, which needs
 * no scratch at all; everything else runs the segment sweep.  The faster filter route of
 * the RANGE objective needs buffers of about the size of the input and is only available
 * through a handle.
 *
 * Arguments are those of zl_create's configuration (n_workers, lookahead_R, objective,
 * flags) followed by those of zl_select_batched, with the same meaning, layout and
 * ownership; the device is the calling thread's current CUDA device, which must own
 * every buffer.  Asynchronous on cuda_stream.
 *
 * Limits: B <= zl_noalloc_max_batch() (256); a larger batch returns ZL_ERR_UNSUPPORTED
 * with a message on stderr and launches nothing.  (B times the number of time segments
 * must also fit the array; the built-in launch planner never picks that many, the test
 * is a guard.)
 *
 * First call on a device: looks up the array's device address and raises the sweep
 * kernel's shared-memory limit.  Make that first call outside any stream capture.
 *
 * Sharing: every call on a device uses the one array, which keeps whatever the last
 * call left there.  Nothing in it has to be cleared (each call rewrites all the
 * records it reads), but two calls whose kernels overlap on the GPU - different
 * streams, or different host threads - race on it and give wrong results.  Issue
 * them on one stream, or order them with events.
 */
zl_status zl_select_batched_noalloc(int32_t n_workers, int32_t lookahead_R, int32_t objective, int32_t flags,
                                    const int64_t *d_ts, int32_t B,
                                    int32_t *d_idx, int64_t *d_barrier, int64_t *d_wait,
                                    int32_t *d_status, void *cuda_stream);
int32_t  zl_noalloc_max_batch(void);       /* largest B of zl_select_batched_noalloc           */
size_t   zl_noalloc_scratch_bytes(void);   /* size of the fixed device array it works in       */

/* Free the scratch and the handle.  NULL is a no-op. */
zl_status zl_destroy(zl_handle *h);

/* Queries (host side). */
const char *zl_status_string(zl_status s);
size_t   zl_workspace_bytes(const zl_handle *h);      /* device scratch held by the handle      */
int32_t  zl_launches_per_call(const zl_handle *h);    /* kernels the next zl_select_batched enqueues */
int32_t  zl_segments_per_instance(const zl_handle *h, int32_t B);
int32_t  zl_route(const zl_handle *h);                /* route of the handle's calls: 0 segment sweep only, 1 RANGE filter route, 2 bucket route, 3 one launch (small instances) */
int32_t  zl_max_workers(void);                        /* largest supported n                     */
int32_t  zl_trace_max_elements(void);                 /* largest n*R for zl_trace_batched        */
int32_t  zl_last_cuda_error(const zl_handle *h);      /* cudaError_t of the last failed call     */

#ifdef __cplusplus
}
#endif
#endif /* ZIPLINE_H */
