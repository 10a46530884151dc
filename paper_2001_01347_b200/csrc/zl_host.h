// Host side shared by the translation units: what one call enqueues (Pipeline), the launch plan of the
// segment sweep, the launch helper, and the stage launchers each kernel file exports.  Every kernel is
// launched from the file that defines it.
#pragma once
#include <cuda_runtime.h>
#include <string.h>

#include <algorithm>

#include "zl_types.cuh"

namespace zl {

inline int pow2_floor(int x) { int p = 1; while (p * 2 <= x) p *= 2; return p; }
inline int pow2_ceil(int x) { int p = 1; while (p < x) p *= 2; return p; }

// Shape of the segment sweep for one call.
struct LaunchPlan {
    int threads, G, nseg, cap, target; size_t smem;
    int G_rest, target_rest;                                      // lanes per row and round size when a CTA of 512 threads runs the sweep
    int threads_small, G_small, target_small;                     // the same for the one-launch route of small instances
};

// Everything one call enqueues, for both the handle-based and the fixed-scratch entry points.
struct Pipeline {
    const int64_t *ts; int B, n, R, objective, flags, num_sms;
    InstMeta *meta; SegResult *seg; int nres;
    FilterBufs fb;                                                // fb.table == nullptr: no filter route
    int filter_threads, filter_rows, filter_round;                // 0: automatic
    int pdl_off;                                                  // bit mask of kernels launched without early scheduling
    int prologue_threads, tail_threads;                           // 0: automatic
    int cluster, filter_stages, filter_bulk;                      // 0: automatic (cluster: CTAs per instance of k_range_head; filter_bulk: 1 copy engine, 2 per-lane copies)
    int tail_cap;                                                 // 0: default; else survivors the finishing CTA of the filter kernel has room for
    int rest_split;                                               // RANGE filter route's last stage: 0 by shape, 1 a kernel per phase, 2 the single kernel
    int small;                                                    // 1: the one-launch route (instances of a few thousand timestamps)
    int max_rounds;                                               // 0: automatic; else the segment sweep's round limit
    int rest_per_sm;                                              // CTAs of k_range_rest resident per SM (0: ask the runtime)
    int checks_off;                                               // debug handle: unchecked kernels, clock stamps still taken
    int32_t *idx; int64_t *barrier; int64_t *wait; int32_t *status;
};

// Launch with programmatic stream serialization: the kernel may be scheduled while its predecessor in
// the stream is still running; every kernel here waits for that predecessor (grid_dep_wait) before it
// touches memory.
template <typename... KArgs, typename... Args>
void launch_dep(bool early, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = early ? 1 : 0;
    cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---- stage launchers.  `fb` is the call's copy of the route buffers (all zero when no fast route is on);
// the filter and bucket stages fill in its per-call fields.  Each *_limits() raises the dynamic shared-memory
// limit of its file's kernels (once per device).

// prologue.cu: column scans for the bucket route and the plain segment sweep; the optional sortedness check
void enqueue_prologue(const Pipeline &q, const FilterBufs &fb, cudaStream_t st, const MatBatch &src);
void enqueue_prologue(const Pipeline &q, const FilterBufs &fb, cudaStream_t st, const AriBatch &src);
void enqueue_check_sorted(const Pipeline &q, cudaStream_t st);
cudaError_t prologue_limits();

// range_filter.cu: the RANGE filter route - k_range_head (summary, requests, filter table: a cluster per instance) and
// k_range_filter (the filter pass in many small CTAs; the CTA that finishes an instance's last block also finishes an
// instance with few survivors)
cudaError_t enqueue_range_head(const Pipeline &q, const FilterBufs &fb, cudaStream_t st, const MatBatch &src);
cudaError_t enqueue_range_head(const Pipeline &q, const FilterBufs &fb, cudaStream_t st, const AriBatch &src);
cudaError_t enqueue_range_filter(const Pipeline &q, FilterBufs &fb, cudaStream_t st, const MatBatch &src);
cudaError_t enqueue_range_filter(const Pipeline &q, FilterBufs &fb, cudaStream_t st, const AriBatch &src);
cudaError_t enqueue_range_tail(const Pipeline &q, FilterBufs &fb, cudaStream_t st, const MatBatch &src);
cudaError_t enqueue_range_tail(const Pipeline &q, FilterBufs &fb, cudaStream_t st, const AriBatch &src);
int range_head_cluster_size(int B, int n, int num_sms, int gmax);
cudaError_t range_limits();

// filter.cu: the filter pass and the kernel that finishes instances with few survivors; `mid` is recorded between them
void enqueue_filter(const Pipeline &q, FilterBufs &fb, cudaStream_t st, cudaEvent_t mid, const MatBatch &src);
void enqueue_filter(const Pipeline &q, FilterBufs &fb, cudaStream_t st, cudaEvent_t mid, const AriBatch &src);
cudaError_t filter_limits();

// heavy.cu: the phases for RANGE instances with many survivors as kernels of their own (large shapes)
void enqueue_heavy(const Pipeline &q, const FilterBufs &fb, cudaStream_t st);
cudaError_t heavy_limits();

// range_rest.cu: the route's last kernel - instances with many survivors (cell scan, refinement, bucket sweep), the segment
// sweep of instances whose lists overflowed, and every instance's outputs
cudaError_t enqueue_range_rest(const Pipeline &q, const FilterBufs &fb, const LaunchPlan &p, cudaStream_t st, const MatBatch &src);
cudaError_t enqueue_range_rest(const Pipeline &q, const FilterBufs &fb, const LaunchPlan &p, cudaStream_t st, const AriBatch &src);
cudaError_t range_rest_limits();

// sum_route.cu: the bucket route (plan, index pass, bucket kernel); `mid` is recorded before the bucket kernel
void enqueue_bucket_route(const Pipeline &q, FilterBufs &fb, cudaStream_t st, cudaEvent_t mid);
cudaError_t bucket_route_limits();

// small.cu: the whole search for small instances in one launch
void enqueue_small(const Pipeline &q, const LaunchPlan &p, cudaStream_t st, const MatBatch &src);
cudaError_t small_limits();

// sweep.cu: the segment sweep (fallback of the fast routes, or the whole search) and K5
void enqueue_sweep(const Pipeline &q, const FilterBufs &fb, const LaunchPlan &p, bool fast, cudaStream_t st, const MatBatch &src);
void enqueue_sweep(const Pipeline &q, const FilterBufs &fb, const LaunchPlan &p, bool fast, cudaStream_t st, const AriBatch &src);
// route: 0 only the segment sweep ran, 1 the RANGE filter route, 2 the bucket route
void enqueue_finalize(const Pipeline &q, const FilterBufs &fb, const LaunchPlan &p, int route, cudaStream_t st, const MatBatch &src);
void enqueue_finalize(const Pipeline &q, const FilterBufs &fb, const LaunchPlan &p, int route, cudaStream_t st, const AriBatch &src);
cudaError_t sweep_limits();

}  // namespace zl
