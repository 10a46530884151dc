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

/*
 * A handle created with ZL_FLAG_DEBUG_CHECKS puts 64 bytes of a fixed pattern behind every scratch buffer it
 * allocates.  No kernel may write there: a changed byte means that some store ran past the end of its buffer
 * without an index check seeing it.  Waits for the device, reads the patterns back and reports how many buffers
 * carry one (*buffers; 0 for a handle without the flag) and how many of them are damaged (*damaged).  Host
 * pointers.  The patterns are not repaired.
 */
zl_status zl_check_canaries(zl_handle *h, int32_t *buffers, int32_t *damaged);

/*
 * Self-checks (no counterpart in the paper; the stand-in for a memory checker).  A handle created with
 * ZL_FLAG_DEBUG_CHECKS runs kernels in which every computed index into global or shared memory, and every bulk
 * copy, is compared with the extent of its buffer first; an index out of range is not used (the access is
 * skipped, nothing traps) and the first such event is recorded.  zl_debug_report waits for the device, copies the
 * record to h_record[0..3] (host) and clears it: [0] a code naming the access (0: no violation since the last
 * report), [1] the CTA, [2], [3] the low and high word of the offending index.  Covers the kernels of the
 * RANGE filter route that every call runs (k_range_head, k_filter / k_filter_arith, k_tail) and their ring variants.
 */
zl_status zl_debug_report(zl_handle *h, uint32_t *h_record);

/*
 * With the same flag the kernels of the RANGE filter route also note the GPU's nanosecond clock at their phase boundaries.
 * Records of 16 values: first k_range_head's, one per CTA, for each of the first `ctas` CTAs of the handle's last call (0 where a boundary was not passed): [0] start, [1] columns
 * done, [2] summary, [11] requests written, [12] slow rows walked, [13] partial table done, [3] before and [4] after
 * the cluster barrier, [5] merged table written, [6]..[9] the last kernel's CTA of the same index (start, dependency wait over, flags read, end);
 * behind max(max_batch, 8 x SMs) such records follow the ring variants' filter CTAs ([0] start, [1] table loaded, [2] pass done).
 * h_stamps: host, ctas * 16 uint64.  Synchronises.
 */
zl_status zl_debug_stamps(zl_handle *h, int32_t ctas, uint64_t *h_stamps);

/* Tuning knobs of a handle (host side; take effect at the next call).
 * key: "threads" (128..1024, power of two), "lanes_per_row" (1..32, power of two),
 * "segments" (time segments per instance, >= 1), "round_factor" (percent of the
 * nominal elements per round), "no_filter" (1: neither the RANGE filter route nor the bucket
 * route nor the one-launch route of small instances is used; every instance is swept by time segments), "rest_split" (RANGE filter route, what the tail kernel leaves undone: 1 a kernel per phase, 2 the single last kernel, 0 by the shape), "no_small" (1: small instances do not take the one-launch route but the one larger instances of the objective would), "max_rounds" (rounds a time segment of the segment sweep may take before its instance ends with ZL_ERR_TIMEOUT; 0: the bound that follows from the input's size), "tail_cap" (a power of two, 64..2048: survivors the checked tail kernel has room for), "filter_threads" / "filter_rows" (CTA size and rows per CTA of the
 * filter pass), "cluster" (CTAs per instance of the first kernel of the RANGE filter route, a power of two up to 8), "filter_stages" (ring slots per warp, 2..7), "filter_bulk" (the ring variants of the filter and tail kernels - 1: chunks of a row arrive by one bulk-copy request each, counted on an mbarrier; 2: in 16-byte pieces copied by every lane; 0, the default: the kernels of filter.cu, which are the faster ones on every workload measured), "checks_off" (1: a handle created with ZL_FLAG_DEBUG_CHECKS runs the unchecked kernels but still records the clock stamps), "filter_round" (a row is requested up to its estimate rounded up to this many timestamps; power of two, 2..1024; from 128 on it is also the ring slot size of the bulk-copy variant), "prologue_threads" / "tail_threads" (CTA sizes of those kernels), "pdl_off" (bit k: launch the k-th kernel of the chain only after its predecessor has
 * finished instead of scheduling it early).  0 restores the built-in choice. */
zl_status zl_set_option(zl_handle *h, const char *key, int32_t value);

#ifdef __cplusplus
}
#endif
#endif /* ZIPLINE_DEBUG_H */
