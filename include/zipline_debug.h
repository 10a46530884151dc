/*
 * zipline_debug.h - measurement and tuning aids of the ZipLine library (none has a counterpart in the
 * paper).  They are exported by the same shared library as the calls of zipline.h but are not part of the
 * search's interface: per-stage timing, a load-only probe kernel, survivor counts of the last call and the
 * tuning knobs of a handle.
 */
#ifndef ZIPLINE_DEBUG_H
#define ZIPLINE_DEBUG_H

#include "zipline.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Optional per-stage timing (no counterpart in the paper; a measurement aid).
 * After zl_profile_begin(h, max_calls) every zl_select_batched on h records CUDA
 * events on the caller's stream between its stages, for up to max_calls calls.
 * zl_profile_read waits for the recorded calls, returns their number and, in
 * ms_stage[0..3], the summed milliseconds of: prologue (column scans, filter table),
 * filter pass, sort + sweep (the filtered-list kernel and the segment sweep kernel),
 * finalize; it then clears the record.  zl_profile_end releases the events.
 * All pointers are host pointers.
 */
zl_status zl_profile_begin(zl_handle *h, int32_t max_calls);
zl_status zl_profile_read(zl_handle *h, int32_t *calls, float *ms_stage);
zl_status zl_profile_end(zl_handle *h);

/*
 * Measurement aid (no counterpart in the paper): a kernel that only loads, a warp per row, the first
 * d_count[row] timestamps of each of `rows` rows of length R (16-byte loads where the layout allows)
 * and does nothing else.  Timed on the bytes the filter pass of the search reads, to show what
 * the memory system delivers for that access pattern.
 *
 *   d_ts     device, [rows][R] int64, 8-byte aligned.
 *   d_count  device, [rows] int32: how many leading timestamps of the row to read (clamped to 0..R).
 *   d_sink   device, one uint64 the caller owns (receives a checksum practically never; keeps the loads alive).
 *
 * Asynchronous on cuda_stream; no handle, no scratch, no allocation.
 */
zl_status zl_probe_read_batched(const int64_t *d_ts, const int32_t *d_count, int64_t rows, int32_t R,
                                uint64_t *d_sink, void *cuda_stream);

/*
 * Diagnostic (no counterpart in the paper): for the last zl_select_batched on h and each of
 * its first B instances, how many elements passed the RANGE filter pass (h_filtered), how many of
 * those passed the refinement (h_refined), and whether a survivor list overflowed, in which case
 * the segment sweep handled the instance instead (h_overflow).  On the bucket route (zl_route() == 2)
 * the three arrays hold the instance's time buckets, its tiles of buckets, and whether a bucket
 * outgrew its shared-memory batch (the segment sweep then handled the instance).  Host arrays of B
 * uint32, any of which may be NULL.  Synchronises the device.
 */
zl_status zl_filter_counts(zl_handle *h, int32_t B, uint32_t *h_filtered, uint32_t *h_refined, uint32_t *h_overflow);

/* Tuning knobs of a handle (host side; take effect at the next call).
 * key: "threads" (128..1024, power of two), "lanes_per_row" (1..32, power of two),
 * "segments" (time segments per instance, >= 1), "round_factor" (percent of the
 * nominal elements per round), "no_filter" (1: neither the RANGE filter route nor the bucket
 * route is used; every instance is swept by time segments), "filter_threads" / "filter_rows" (CTA size and rows per CTA of the
 * filter pass), "filter_round" (a row is requested up to its estimate rounded up to this many timestamps; power of two, 2..256), "prologue_threads" / "tail_threads" (CTA sizes of those kernels), "pdl_off" (bit k: launch the k-th kernel of the chain only after its predecessor has
 * finished instead of scheduling it early).  0 restores the built-in choice. */
zl_status zl_set_option(zl_handle *h, const char *key, int32_t value);

#ifdef __cplusplus
}
#endif
#endif /* ZIPLINE_DEBUG_H */
