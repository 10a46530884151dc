// Host side of the ZipLine library: the handle, the launch plan, the order in which a call enqueues its stages,
// and the C ABI (include/zipline.h, include/zipline_debug.h).
//
// Per instance: n sorted rows of R int64 timestamps.  Every kernel of a call is enqueued on the caller's
// stream with programmatic stream serialization and starts with grid_dep_wait().
//
//   prologue.cu   k_prologue: column scans (tmin, t0 = max_p e^p_1, lmin = min_p e^p_R, span); for the RANGE filter
//                 route also the per-row estimates, the filter table and the per-call counters.
//   filter.cu     RANGE filter route: an element matters only if its `next` exceeds G, the running maximum of `next`
//                 over everything earlier (floored by t0).  k_filter streams the rows and keeps the survivors;
//                 k_tail finishes the instances with few survivors.
//   heavy.cu      instances with many survivors: G at every fine time cell, refinement, bucket sweep.
//   sum_route.cu  the bucket route (SUM, and RANGE instances that are one shared-memory batch): the whole instance
//                 is put into time order bucket by bucket.
//   sweep.cu      the segment sweep (fallback of both fast routes) and k_finalize (K5).
//   baselines.cu  GridScan / FullGridScan, the predictor, the per-position trace.
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>
#include <algorithm>
#include <mutex>
#include <new>
#include <type_traits>

#include "../../include/zipline.h"
#include "../../include/zipline_debug.h"
#include "zl_host.h"

// ================================================================================== host side
struct zl_handle {
    zl_config cfg;
    int num_sms;
    zl::InstMeta *d_meta;
    zl::SegResult *d_seg;
    int64_t *d_pred;         // ZL_FLAG_PREDICTOR: predicted timestamps, [max_batch][n][R]
    zl::FilterBufs fb;       // RANGE: buffers of the filter route (device), sized for max_batch
    int nres;                // SegResult slots per instance
    size_t ws_bytes;
    // host-buffer path
    int64_t *s_ts; int32_t *s_idx; int64_t *s_barrier; int64_t *s_wait; int32_t *s_status;
    cudaStream_t s_stream;
    size_t staging_bytes;
    // options (0 = automatic)
    int opt_threads, opt_lanes, opt_segments, opt_round_factor, opt_no_filter, opt_filter_threads, opt_filter_rows, opt_pdl_off, opt_prologue_threads, opt_tail_threads, opt_filter_round, opt_cluster, opt_filter_stages, opt_checks_off, opt_filter_bulk, opt_tail_cap, opt_max_rounds, opt_no_small, opt_rest_split;
    int epoch;               // calls so far: the two sets of per-call flags alternate
    int last_cuda_error;
    int launches;
    // optional per-kernel timing: PROF_EVENTS events per recorded call
    cudaEvent_t *prof_ev;
    int prof_cap, prof_calls;
    // ZL_FLAG_DEBUG_CHECKS: every scratch buffer ends in CANARY_BYTES bytes of a fixed pattern that no kernel may touch
    unsigned char *canary[24];
    int ncanary;
    // RANGE filter route: one word of pinned host memory that the last kernel of a call writes (did some instance have
    // more survivors than one CTA finishes?); the next call reads it, without waiting, to choose the form of its last stage
    uint32_t *h_hint, *d_hint;
};

namespace {

using zl::LaunchPlan;
using zl::Pipeline;
using zl::pow2_ceil;
using zl::pow2_floor;
constexpr int PROF_EVENTS = 5;
constexpr size_t CANARY_BYTES = 64;
constexpr int CANARY_BYTE = 0xC5;

// SRC: zl::MatBatch (the rows are read from q.ts) or zl::AriBatch (predicted rows, generated on the fly; RANGE, filter
// route or plain segment sweep only).
// RANGE filter route: from this many timestamps an instance on, what the filter and tail kernels leave undone goes
// through kernels of its own per phase instead of the single last kernel.
static bool range_rest_split(int n, int R, int forced) { return forced ? forced == 1 : (long long)n * R >= (1LL << 21); }

template <class SRC>
void enqueue(const Pipeline &q, const LaunchPlan &p, cudaStream_t st, cudaEvent_t *ev, const SRC src) {
    constexpr bool arith = std::is_same<SRC, zl::AriBatch>::value;
    const bool filter = q.fb.table != nullptr && q.objective == ZL_OBJ_RANGE;
    // the bucket route: every SUM shape it supports, and RANGE instances small enough to be a single bucket
    const bool sumfast = !arith && q.fb.flags != nullptr && q.fb.scap != 0 && (q.objective == ZL_OBJ_SUM || q.fb.table == nullptr);
    zl::FilterBufs fb = q.fb;
    if (!filter && !sumfast) memset(&fb, 0, sizeof(fb));
    if (ev) cudaEventRecord(ev[0], st);
    if constexpr (!arith) {
        if (q.small) {
            // a few thousand timestamps an instance: everything in one kernel
            zl::enqueue_small(q, p, st, src);
            if (ev) for (int k = 1; k < PROF_EVENTS; ++k) cudaEventRecord(ev[k], st);
            return;
        }
    }
    if (filter) zl::enqueue_range_head(q, fb, st, src);
    else zl::enqueue_prologue(q, fb, st, src);
    if constexpr (!arith) if (q.flags & ZL_FLAG_CHECK_SORTED) zl::enqueue_check_sorted(q, st);
    if (ev) cudaEventRecord(ev[1], st);
    if (filter) {
        // the filter kernel, then everything it left undone and the outputs in one more launch
        if (q.filter_bulk) {
            // on request: the variant of the two kernels whose rows arrive through a ring filled by the copy engine
            zl::enqueue_range_filter(q, fb, st, src);
            if (ev) cudaEventRecord(ev[2], st);
            zl::enqueue_range_tail(q, fb, st, src);
        } else {
            zl::enqueue_filter(q, fb, st, ev ? ev[2] : nullptr, src);
        }
        if (ev) cudaEventRecord(ev[3], st);
        if (!range_rest_split(q.n, q.R, q.rest_split)) {
            // everything the two kernels left undone, and the outputs, in one more launch
            zl::enqueue_range_rest(q, fb, p, st, src);
            if (ev) cudaEventRecord(ev[4], st);
            return;
        }
        // large instances: survivors by the million are the rule, every phase gets a grid of its own
        zl::enqueue_heavy(q, fb, st);
    } else if (sumfast) {
        if constexpr (!arith) zl::enqueue_bucket_route(q, fb, st, ev ? ev[2] : nullptr);
    } else if (ev) {
        cudaEventRecord(ev[2], st);
    }
    zl::enqueue_sweep(q, fb, p, filter || sumfast, st, src);
    if (ev) cudaEventRecord(ev[3], st);
    zl::enqueue_finalize(q, fb, p, filter ? 1 : sumfast ? 2 : 0, st, src);
    if (ev) cudaEventRecord(ev[4], st);
}

cudaError_t raise_shared_memory_limits() {
    cudaError_t e = zl::prologue_limits();
    if (e == cudaSuccess) e = zl::range_limits();
    if (e == cudaSuccess) e = zl::small_limits();
    if (e == cudaSuccess) e = zl::filter_limits();
    if (e == cudaSuccess) e = zl::heavy_limits();
    if (e == cudaSuccess) e = zl::range_rest_limits();
    if (e == cudaSuccess) e = zl::bucket_route_limits();
    if (e == cudaSuccess) e = zl::sweep_limits();
    return e;
}

LaunchPlan make_plan(const zl_handle *h, int B) {
    const int n = h->cfg.n_workers, R = h->cfg.lookahead_R;
    const long long N = (long long)n * R;
    LaunchPlan p;
    p.threads = h->opt_threads ? h->opt_threads : pow2_ceil((int)std::min<long long>(1024, std::max<long long>(128, (long long)n * 32)));
    p.G = h->opt_lanes ? h->opt_lanes : std::max(1, std::min(32, pow2_floor(std::max(1, p.threads / n))));
    if (p.G > p.threads) p.G = p.threads;
    // batch capacity in 8-byte nodes; wide (16-byte) instances get half, which must still hold one
    // node per worker
    int cap = std::max(h->cfg.objective == ZL_OBJ_SUM ? 8192 : 4096, pow2_ceil(2 * n));
    const int small = std::max(pow2_ceil((int)std::min<long long>(N, 1 << 20)), std::max(pow2_ceil(2 * n), 128));
    p.cap = std::min(cap, small);
    // time segments per instance: enough CTAs to fill the GPU a few times over, each long enough to
    // amortise its binary searches
    int nseg = 1;
    if (N > p.cap) {
        const int want = (4 * h->num_sms + B - 1) / B;
        const int most = (int)std::max<long long>(1, N / (16LL * n) / 4);
        nseg = std::max(1, std::min(std::min(want, most), zl::MAX_SEGMENTS));
    }
    if (h->opt_segments) nseg = std::min(h->opt_segments, zl::MAX_SEGMENTS);
    p.nseg = nseg;
    const int rf = h->opt_round_factor ? h->opt_round_factor : 75;
    long long target = (long long)n * std::max(p.G, 4) * rf / 100;
    if (h->cfg.objective == ZL_OBJ_SUM) target = std::min<long long>(target, (long long)p.cap * 45 / 100);
    target = std::min<long long>(target, (long long)p.cap * 4);
    p.target = (int)std::max<long long>(target, 32);
    p.smem = (((size_t)2 * n * sizeof(uint32_t) + 15) & ~(size_t)15) + (size_t)p.cap * 20;   // nodes, sorted nodes, slot counters
    p.G_rest = h->opt_lanes ? std::min(h->opt_lanes, 512) : std::max(1, std::min(32, pow2_floor(std::max(1, 512 / n))));
    long long target_rest = (long long)n * std::max(p.G_rest, 4) * rf / 100;
    target_rest = std::min<long long>(target_rest, (long long)p.cap * 4);
    p.target_rest = (int)std::max<long long>(target_rest, 32);
    // the one-launch route: about eight timestamps a thread
    p.threads_small = std::max(64, std::min(512, pow2_ceil((int)std::min<long long>(N / 8, 512))));
    p.G_small = h->opt_lanes ? std::min(h->opt_lanes, p.threads_small) : std::max(1, std::min(32, pow2_floor(std::max(1, p.threads_small / n))));
    long long target_small = (long long)n * std::max(p.G_small, 4) * rf / 100;
    if (h->cfg.objective == ZL_OBJ_SUM) target_small = std::min<long long>(target_small, (long long)p.cap * 45 / 100);
    target_small = std::min<long long>(target_small, (long long)p.cap * 4);
    p.target_small = (int)std::max<long long>(target_small, 32);
    return p;
}

zl_status cuda_fail(zl_handle *h, cudaError_t e) {
    if (h) h->last_cuda_error = (int)e;
    return e == cudaErrorMemoryAllocation ? ZL_ERR_NOMEM : ZL_ERR_CUDA;
}

// Makes `device` current for the life of the object and puts the caller's device back afterwards.
struct DeviceScope {
    int prev = -1;
    cudaError_t err = cudaSuccess;
    explicit DeviceScope(int device) {
        err = cudaGetDevice(&prev);
        if (err == cudaSuccess && prev != device) err = cudaSetDevice(device); else if (err == cudaSuccess) prev = -1;
    }
    ~DeviceScope() { if (prev >= 0) cudaSetDevice(prev); }
};

// The stream-ordered entry points only enqueue work: the caller's current device must be the handle's.
bool on_device(int device) {
    int cur = -1;
    return cudaGetDevice(&cur) == cudaSuccess && cur == device;
}

#define ZL_CUDA(h, call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return cuda_fail((h), e_); } while (0)

}  // namespace

extern "C" {

const char *zl_status_string(zl_status s) {
    switch (s) {
        case ZL_OK: return "ok";
        case ZL_ERR_INVALID_ARG: return "invalid argument";
        case ZL_ERR_UNSUPPORTED: return "unsupported shape or magnitude";
        case ZL_ERR_NOMEM: return "out of memory";
        case ZL_ERR_CUDA: return "CUDA runtime error";
        case ZL_ERR_UNSORTED: return "a row is not non-decreasing";
        case ZL_ERR_TIMEOUT: return "internal iteration limit reached";
    }
    return "unknown status";
}

int32_t zl_max_workers(void) { return zl::MAX_WORKERS; }

zl_status zl_create(const zl_config *cfg, zl_handle **out) {
    if (!cfg || !out) return ZL_ERR_INVALID_ARG;
    *out = nullptr;
    if (cfg->n_workers < 1 || cfg->lookahead_R < 1 || cfg->max_batch < 1) return ZL_ERR_INVALID_ARG;
    if (cfg->objective != ZL_OBJ_RANGE && cfg->objective != ZL_OBJ_SUM) return ZL_ERR_INVALID_ARG;
    if (cfg->flags & ~(ZL_FLAG_CHECK_SORTED | ZL_FLAG_FULL_SWEEP | ZL_FLAG_PREDICTOR | ZL_FLAG_DEBUG_CHECKS | ZL_FLAG_FORCE_FILTER)) return ZL_ERR_INVALID_ARG;
    if (cfg->n_workers > zl::MAX_WORKERS) return ZL_ERR_UNSUPPORTED;
    if ((long long)cfg->n_workers * cfg->lookahead_R > (1LL << 31) - 1) return ZL_ERR_UNSUPPORTED;
    if (cfg->max_batch > 65535) return ZL_ERR_UNSUPPORTED;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || cfg->device < 0 || cfg->device >= ndev) return ZL_ERR_CUDA;
    zl_handle *h = new (std::nothrow) zl_handle();
    if (!h) return ZL_ERR_NOMEM;
    memset(h, 0, sizeof(*h));
    h->cfg = *cfg;
    DeviceScope scope(cfg->device);                               // the caller's device is current again on return
    cudaError_t e = scope.err;
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->num_sms, cudaDevAttrMultiProcessorCount, cfg->device);
    // scratch buffers; a debug handle's end in canary bytes (zl_check_canaries)
    const bool canaries = (cfg->flags & ZL_FLAG_DEBUG_CHECKS) != 0;
    auto alloc = [&](void **ptr, size_t bytes) -> cudaError_t {
        if (!canaries) return cudaMalloc(ptr, bytes);
        const size_t body = (bytes + 15) & ~(size_t)15;
        cudaError_t a = cudaMalloc(ptr, body + CANARY_BYTES);
        if (a == cudaSuccess) a = cudaMemset((unsigned char *)*ptr + body, CANARY_BYTE, CANARY_BYTES);
        if (a == cudaSuccess && h->ncanary < 24) h->canary[h->ncanary++] = (unsigned char *)*ptr + body;
        return a;
    };
    const size_t meta_b = (size_t)cfg->max_batch * sizeof(zl::InstMeta);
    size_t filter_b = 0;
    h->nres = zl::MAX_SEGMENTS;
    // RANGE instances that fit one shared-memory batch are sorted whole by the bucket route; larger ones take the filter route
    const bool range_small = cfg->objective == ZL_OBJ_RANGE && (long long)cfg->n_workers * cfg->lookahead_R <= 4096 &&
                             !(cfg->flags & ZL_FLAG_FORCE_FILTER);
    if (cfg->objective == ZL_OBJ_RANGE && !range_small) {
        const long long N = (long long)cfg->n_workers * cfg->lookahead_R;
        const size_t mb = (size_t)cfg->max_batch;
        zl::FilterBufs &f = h->fb;
        f.cells = std::max(64, std::min(zl::FILTER_MAX_CELLS, pow2_ceil((int)std::min<long long>(cfg->lookahead_R, 1 << 20))));
        f.capb = (int)std::max<long long>(64, std::min<long long>(4096, pow2_ceil((int)std::min<long long>(N, 1 << 20))));
        f.nbk = (int)std::max<long long>(1, std::min<long long>(1024, pow2_ceil((int)std::min<long long>(N / 8 / f.capb, 1 << 20))));
        // small shapes: room for half of the instance's elements (at most four buckets), so that instances in which
        // many elements raise the running maximum stay on this route
        f.nbk = std::max(f.nbk, (int)std::min<long long>(4, pow2_ceil((int)std::max<long long>(1, N / 2 / f.capb))));
        f.fcells = (int)std::max<long long>(std::max(64, f.nbk), std::min<long long>(1 << 18, pow2_ceil((int)std::min<long long>(N / 64, 1 << 20))));
        f.grp = std::max(1, std::min(f.nbk, pow2_floor((int)std::max<long long>(1, (long long)f.nbk * cfg->max_batch / (8LL * std::max(1, h->num_sms))))));
        f.list1cap = (int)(N <= (1 << 17) ? N : N / 2);            // small shapes: room for every element
        h->nres = std::max(zl::MAX_SEGMENTS, (f.nbk + f.grp - 1) / f.grp);
        const size_t tiles = ((size_t)f.fcells + zl::SCAN_TILE - 1) / zl::SCAN_TILE;
        // the fused kernel runs up to max(max_batch, 8 x SMs) CTAs, each with a record of partial results and a partial table
        const size_t ctas = std::max<size_t>(mb, (size_t)h->num_sms * 8);
        const size_t sizes[12] = {mb * f.cells * 4, mb * cfg->n_workers * 4, mb * f.fcells * 4, std::max<size_t>(mb * cfg->n_workers, ctas) * 4,
                                  mb * (size_t)f.list1cap * 8, mb * f.nbk * 4, mb * f.nbk * f.capb * 8, mb * tiles * 4, 128,
                                  ctas * 4 * 8, ctas * f.cells * 4, mb * 4};
        void **ptrs[12] = {(void **)&f.table, (void **)&f.rowhint, (void **)&f.cellmax, (void **)&f.rcnt,
                           (void **)&f.list1, (void **)&f.bcnt, (void **)&f.list2, (void **)&f.tilemax, (void **)&f.flags,
                           (void **)&f.part, (void **)&f.ptab, (void **)&f.done};
        f.maxctas = (int)std::min<size_t>(ctas, 0x7fffffff);
        for (int i = 0; i < 12; ++i) {
            if (e == cudaSuccess) e = alloc(ptrs[i], sizes[i]);
            filter_b += sizes[i];
        }
        if (e == cudaSuccess) e = cudaMemset(f.flags, 0, 128);      // two sets of eight per-call words, then words that outlive a call
        if (e == cudaSuccess) e = cudaHostAlloc((void **)&h->h_hint, 64, cudaHostAllocMapped);
        if (e == cudaSuccess) { memset(h->h_hint, 0, 64); e = cudaHostGetDevicePointer((void **)&h->d_hint, h->h_hint, 0); }
        f.hint = h->d_hint;
        f.hint_last = e == cudaSuccess ? f.flags + 16 : nullptr;
        if (cfg->flags & ZL_FLAG_DEBUG_CHECKS) {
            // the violation record, then 16 clock stamps per CTA of the head kernel and of the filter kernel
            const size_t dbg_b = 64 + (ctas + mb * ((size_t)cfg->n_workers + 1) / 2 + 1) * 16 * 8;
            if (e == cudaSuccess) e = alloc((void **)&f.dbg, dbg_b);
            if (e == cudaSuccess) e = cudaMemset(f.dbg, 0, dbg_b);
            filter_b += dbg_b;
        }
    }
    if (cfg->objective == ZL_OBJ_SUM || range_small) {
        // bucket route: shared-memory batches of scap elements, buckets of about 11/16 of that
        const long long N = (long long)cfg->n_workers * cfg->lookahead_R;
        const size_t mb = (size_t)cfg->max_batch;
        zl::FilterBufs &f = h->fb;
        f.scap = N <= 4096 ? std::max(64, pow2_ceil((int)N)) : cfg->n_workers > 2048 ? 8192 : 4096;
        f.stiles = 1;
        bool on = true;
        if (N > f.scap) {
            f.sM = f.scap / 16 * 11;
            const long long nbk = N / f.sM + 1;
            f.stiles = (int)((nbk + zl::TILE_BK - 1) / zl::TILE_BK);
            f.scells = (int)std::max<long long>(1024, std::min<long long>(1 << 14, pow2_ceil((int)std::min<long long>(N / 64, 1 << 20))));
            on = nbk <= 12000 && cfg->lookahead_R <= 65535;       // boundaries fit shared memory, row indices are 16-bit
        }
        if (on) {
            const size_t nb1 = (size_t)f.stiles * zl::TILE_BK + 1;
            const size_t sizes[4] = {mb * nb1 * 4, 64, f.scells ? mb * f.stiles * cfg->n_workers * 32 : 64, 64};
            void **ptrs[4] = {(void **)&f.bnd, (void **)&f.cellacc, (void **)&f.itab, (void **)&f.flags};
            for (int i = 0; i < 4; ++i) {
                if (e == cudaSuccess) e = alloc(ptrs[i], sizes[i]);
                filter_b += sizes[i];
            }
            if (e == cudaSuccess) e = cudaMemset(f.flags, 0, 64);
            h->nres = std::max(zl::MAX_SEGMENTS, f.stiles * zl::TILE_BK);   // up to one result per bucket
        } else {
            memset(&f, 0, sizeof(f));
        }
    }
    const size_t seg_b = (size_t)cfg->max_batch * h->nres * sizeof(zl::SegResult);
    if (e == cudaSuccess) e = alloc((void **)&h->d_meta, meta_b);
    if (e == cudaSuccess) e = alloc((void **)&h->d_seg, seg_b);
    const size_t pred_b = (cfg->flags & ZL_FLAG_PREDICTOR) ? (size_t)cfg->max_batch * cfg->n_workers * cfg->lookahead_R * 8 : 0;
    if (e == cudaSuccess && pred_b) e = alloc((void **)&h->d_pred, pred_b);
    if (e == cudaSuccess) e = raise_shared_memory_limits();   // more than the default 48 KB of dynamic shared memory
    if (e != cudaSuccess) {
        zl_status st = cuda_fail(nullptr, e);
        cudaFree(h->d_meta); cudaFree(h->d_seg); cudaFree(h->d_pred);
        if (h->h_hint) cudaFreeHost(h->h_hint);
        cudaFree(h->fb.table); cudaFree(h->fb.rowhint); cudaFree(h->fb.cellmax); cudaFree(h->fb.rcnt);
        cudaFree(h->fb.list1); cudaFree(h->fb.bcnt); cudaFree(h->fb.list2); cudaFree(h->fb.tilemax); cudaFree(h->fb.flags);
        cudaFree(h->fb.bnd); cudaFree(h->fb.cellacc); cudaFree(h->fb.itab); cudaFree(h->fb.part); cudaFree(h->fb.ptab); cudaFree(h->fb.dbg); cudaFree(h->fb.done);
        delete h;
        return st;
    }
    h->ws_bytes = meta_b + seg_b + filter_b + pred_b;
    *out = h;
    return ZL_OK;
}

zl_status zl_profile_end(zl_handle *h) {
    if (!h) return ZL_ERR_INVALID_ARG;
    if (h->prof_ev) {
        for (int i = 0; i < PROF_EVENTS * h->prof_cap; ++i) cudaEventDestroy(h->prof_ev[i]);
        delete[] h->prof_ev;
    }
    h->prof_ev = nullptr;
    h->prof_cap = h->prof_calls = 0;
    return ZL_OK;
}

zl_status zl_profile_begin(zl_handle *h, int32_t max_calls) {
    if (!h || max_calls < 1 || max_calls > 65536) return ZL_ERR_INVALID_ARG;
    zl_profile_end(h);
    DeviceScope scope(h->cfg.device);
    ZL_CUDA(h, scope.err);
    h->prof_ev = new (std::nothrow) cudaEvent_t[PROF_EVENTS * (size_t)max_calls];
    if (!h->prof_ev) return ZL_ERR_NOMEM;
    for (int i = 0; i < PROF_EVENTS * max_calls; ++i) {
        cudaError_t e = cudaEventCreate(&h->prof_ev[i]);
        if (e != cudaSuccess) {
            for (int j = 0; j < i; ++j) cudaEventDestroy(h->prof_ev[j]);
            delete[] h->prof_ev;
            h->prof_ev = nullptr;
            return cuda_fail(h, e);
        }
    }
    h->prof_cap = max_calls;
    h->prof_calls = 0;
    return ZL_OK;
}

zl_status zl_profile_read(zl_handle *h, int32_t *calls, float *ms_stage) {
    if (!h || !calls || !ms_stage) return ZL_ERR_INVALID_ARG;
    DeviceScope scope(h->cfg.device);
    ZL_CUDA(h, scope.err);
    *calls = h->prof_calls;
    for (int k = 0; k < PROF_EVENTS - 1; ++k) ms_stage[k] = 0.f;
    for (int c = 0; c < h->prof_calls; ++c) {
        cudaEvent_t *ev = h->prof_ev + PROF_EVENTS * (size_t)c;
        ZL_CUDA(h, cudaEventSynchronize(ev[PROF_EVENTS - 1]));
        for (int k = 0; k < PROF_EVENTS - 1; ++k) {
            float ms = 0.f;
            ZL_CUDA(h, cudaEventElapsedTime(&ms, ev[k], ev[k + 1]));
            ms_stage[k] += ms;
        }
    }
    h->prof_calls = 0;
    return ZL_OK;
}

zl_status zl_destroy(zl_handle *h) {
    if (!h) return ZL_OK;
    DeviceScope scope(h->cfg.device);
    cudaFree(h->d_meta); cudaFree(h->d_seg); cudaFree(h->d_pred);
    cudaFree(h->fb.table); cudaFree(h->fb.rowhint); cudaFree(h->fb.cellmax); cudaFree(h->fb.rcnt);
    cudaFree(h->fb.list1); cudaFree(h->fb.bcnt); cudaFree(h->fb.list2); cudaFree(h->fb.tilemax); cudaFree(h->fb.flags);
    cudaFree(h->fb.bnd); cudaFree(h->fb.cellacc); cudaFree(h->fb.itab); cudaFree(h->fb.part); cudaFree(h->fb.ptab); cudaFree(h->fb.dbg); cudaFree(h->fb.done);
    cudaFree(h->s_ts); cudaFree(h->s_idx); cudaFree(h->s_barrier); cudaFree(h->s_wait); cudaFree(h->s_status);
    if (h->s_stream) cudaStreamDestroy(h->s_stream);
    if (h->h_hint) cudaFreeHost(h->h_hint);
    zl_profile_end(h);
    delete h;
    return ZL_OK;
}

zl_status zl_set_option(zl_handle *h, const char *key, int32_t value) {
    if (!h || !key || value < 0) return ZL_ERR_INVALID_ARG;
    auto is_pow2 = [](int v) { return v > 0 && (v & (v - 1)) == 0; };
    if (!strcmp(key, "threads")) {
        if (value && (!is_pow2(value) || value < 128 || value > 1024)) return ZL_ERR_INVALID_ARG;
        h->opt_threads = value;
    } else if (!strcmp(key, "lanes_per_row")) {
        if (value && (!is_pow2(value) || value > 32)) return ZL_ERR_INVALID_ARG;
        h->opt_lanes = value;
    } else if (!strcmp(key, "segments")) {
        if (value > zl::MAX_SEGMENTS) return ZL_ERR_INVALID_ARG;
        h->opt_segments = value;
    } else if (!strcmp(key, "no_filter")) {
        h->opt_no_filter = value != 0;
    } else if (!strcmp(key, "cluster")) {
        if (value > 8) return ZL_ERR_INVALID_ARG;
        h->opt_cluster = value;
    } else if (!strcmp(key, "filter_stages")) {
        if (value && (value < 2 || value > 7)) return ZL_ERR_INVALID_ARG;
        h->opt_filter_stages = value;
    } else if (!strcmp(key, "filter_bulk")) {
        if (value > 2) return ZL_ERR_INVALID_ARG;
        h->opt_filter_bulk = value;
    } else if (!strcmp(key, "rest_split")) {
        if (value > 2) return ZL_ERR_INVALID_ARG;
        h->opt_rest_split = value;                  // RANGE filter route, what the tail kernel leaves: 1 a kernel per phase, 2 the single last kernel
    } else if (!strcmp(key, "no_small")) {
        h->opt_no_small = value != 0;               // small instances take the route larger ones would (bucket route)
    } else if (!strcmp(key, "max_rounds")) {
        h->opt_max_rounds = value;                  // the segment sweep gives up (ZL_ERR_TIMEOUT) after this many rounds of a segment
    } else if (!strcmp(key, "tail_cap")) {
        if (value != 0 && (value < 64 || value > 2048 || (value & (value - 1)))) return ZL_ERR_INVALID_ARG;
        h->opt_tail_cap = (int)value;
    } else if (!strcmp(key, "checks_off")) {
        h->opt_checks_off = value != 0;             // a ZL_FLAG_DEBUG_CHECKS handle keeps its clock stamps but runs the unchecked kernels
    } else if (!strcmp(key, "filter_threads")) {
        if (value && (!is_pow2(value) || value < 64 || value > 1024)) return ZL_ERR_INVALID_ARG;
        h->opt_filter_threads = value;
    } else if (!strcmp(key, "prologue_threads") || !strcmp(key, "tail_threads")) {
        if (value && (!is_pow2(value) || value < 64 || value > 1024)) return ZL_ERR_INVALID_ARG;
        (key[0] == 'p' ? h->opt_prologue_threads : h->opt_tail_threads) = value;
    } else if (!strcmp(key, "pdl_off")) {
        h->opt_pdl_off = value;                 // bit k set: kernel k of the chain is launched without early scheduling
    } else if (!strcmp(key, "filter_round")) {
        if (value && (!is_pow2(value) || value < 2 || value > 1024)) return ZL_ERR_INVALID_ARG;
        h->opt_filter_round = value;
    } else if (!strcmp(key, "filter_rows")) {
        if (value > 65536) return ZL_ERR_INVALID_ARG;
        h->opt_filter_rows = value;
    } else if (!strcmp(key, "round_factor")) {
        if (value > 100000) return ZL_ERR_INVALID_ARG;
        h->opt_round_factor = value;
    } else {
        return ZL_ERR_INVALID_ARG;
    }
    return ZL_OK;
}

size_t zl_workspace_bytes(const zl_handle *h) { return h ? h->ws_bytes + h->staging_bytes : 0; }
// The one-launch route: instances of at most SMALL_MAX timestamps in batches of a few per SM (a CTA an instance, all
// resident at once: the call takes as long as one instance does), unless the handle asks for another route.  Larger
// batches of small instances get more out of the bucket route's kernels.
static bool small_route(const zl_handle *h) {
    return (long long)h->cfg.n_workers * h->cfg.lookahead_R <= zl::SMALL_MAX && h->cfg.max_batch <= 4 * std::max(1, h->num_sms) &&
           !h->opt_no_filter && !h->opt_no_small && !(h->cfg.flags & ZL_FLAG_FORCE_FILTER);
}

// The form of the RANGE filter route's last stage for the handle's next call: a kernel per phase when the shape is large,
// or when the previous call (as far as its word has arrived: the read does not wait) had instances with many survivors.
static int rest_split_now(const zl_handle *h) {
    if (h->opt_rest_split) return h->opt_rest_split == 1;
    if (range_rest_split(h->cfg.n_workers, h->cfg.lookahead_R, 0)) return 1;
    return h->h_hint && *(volatile const uint32_t *)h->h_hint != 0;
}

int32_t zl_launches_per_call(const zl_handle *h) {
    if (!h) return 0;
    if (small_route(h)) return 1;
    const bool filter = h->cfg.objective == ZL_OBJ_RANGE && !h->opt_no_filter && h->fb.table != nullptr;
    const bool sumfast = !filter && !h->opt_no_filter && h->fb.scap != 0;
    return (filter ? (rest_split_now(h) ? 9 : 4) : 3) + (sumfast ? (h->fb.scells ? 3 : 2) : 0) + ((h->cfg.flags & ZL_FLAG_CHECK_SORTED) ? 1 : 0);
}
int32_t zl_route(const zl_handle *h) {
    if (!h || h->opt_no_filter) return 0;
    if (small_route(h)) return 3;
    if (h->cfg.objective == ZL_OBJ_RANGE && h->fb.table != nullptr) return 1;
    return h->fb.scap != 0 ? 2 : 0;
}
int32_t zl_segments_per_instance(const zl_handle *h, int32_t B) { return h && B >= 1 ? make_plan(h, B).nseg : 0; }
int32_t zl_last_cuda_error(const zl_handle *h) { return h ? h->last_cuda_error : 0; }

zl_status zl_select_batched(zl_handle *h, const int64_t *d_ts, int32_t B, int32_t *d_idx, int64_t *d_barrier,
                            int64_t *d_wait, int32_t *d_status, void *cuda_stream) {
    if (!h || !d_ts || !d_idx || !d_barrier || !d_wait) return ZL_ERR_INVALID_ARG;
    if (B < 1 || B > h->cfg.max_batch) return ZL_ERR_INVALID_ARG;
    if (((uintptr_t)d_ts & 7) || ((uintptr_t)d_barrier & 7) || ((uintptr_t)d_wait & 7) || ((uintptr_t)d_idx & 3) ||
        ((uintptr_t)d_status & 3))
        return ZL_ERR_INVALID_ARG;
    if (!on_device(h->cfg.device)) return ZL_ERR_INVALID_ARG;     // the launches would go to another GPU than the handle's buffers
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int n = h->cfg.n_workers, R = h->cfg.lookahead_R, obj = h->cfg.objective;
    const LaunchPlan p = make_plan(h, B);
    if (p.smem > 200 * 1024) return ZL_ERR_UNSUPPORTED;

    cudaEvent_t *ev = (h->prof_ev && h->prof_calls < h->prof_cap) ? h->prof_ev + PROF_EVENTS * (size_t)h->prof_calls : nullptr;
    Pipeline q;
    q.ts = d_ts; q.B = B; q.n = n; q.R = R; q.objective = obj; q.flags = h->cfg.flags; q.num_sms = h->num_sms;
    q.meta = h->d_meta; q.seg = h->d_seg; q.nres = h->nres;
    q.fb = h->fb;
    q.filter_threads = h->opt_filter_threads; q.filter_rows = h->opt_filter_rows; q.filter_round = h->opt_filter_round; q.pdl_off = h->opt_pdl_off;
    q.prologue_threads = h->opt_prologue_threads; q.tail_threads = h->opt_tail_threads;
    if (h->opt_no_filter) { q.fb.table = nullptr; q.fb.scap = 0; }
    q.cluster = h->opt_cluster; q.filter_stages = h->opt_filter_stages;
    q.checks_off = h->opt_checks_off; q.filter_bulk = h->opt_filter_bulk; q.tail_cap = h->opt_tail_cap; q.rest_per_sm = 0; q.max_rounds = h->opt_max_rounds; q.small = small_route(h) ? 1 : 0; q.rest_split = rest_split_now(h) ? 1 : 2;
    if (q.fb.flags) {                           // the two sets of per-call flags alternate; a call zeroes the next call's set
        uint32_t *base = h->fb.flags;
        q.fb.flags = base + 8 * (h->epoch & 1);
        q.fb.flags_next = base + 8 * ((h->epoch + 1) & 1);
        ++h->epoch;
    }
    q.idx = d_idx; q.barrier = d_barrier; q.wait = d_wait; q.status = d_status;
    enqueue(q, p, st, ev, zl::MatBatch{d_ts});
    if (ev) ++h->prof_calls;
    ZL_CUDA(h, cudaGetLastError());
    h->launches += zl_launches_per_call(h);
    return ZL_OK;
}

zl_status zl_debug_stamps(zl_handle *h, int32_t ctas, uint64_t *h_stamps) {
    if (!h || !h_stamps || ctas < 1) return ZL_ERR_INVALID_ARG;
    if (!h->fb.dbg || ctas > (long long)h->fb.maxctas + ((long long)h->cfg.max_batch * (h->cfg.n_workers + 1)) / 2) return ZL_ERR_INVALID_ARG;
    DeviceScope scope(h->cfg.device);
    ZL_CUDA(h, scope.err);
    ZL_CUDA(h, cudaDeviceSynchronize());
    ZL_CUDA(h, cudaMemcpy(h_stamps, h->fb.dbg + 16, (size_t)ctas * 16 * 8, cudaMemcpyDeviceToHost));
    return ZL_OK;
}

zl_status zl_check_canaries(zl_handle *h, int32_t *buffers, int32_t *damaged) {
    if (!h || !buffers || !damaged) return ZL_ERR_INVALID_ARG;
    *buffers = h->ncanary;
    *damaged = 0;
    if (!h->ncanary) return ZL_OK;
    DeviceScope scope(h->cfg.device);
    ZL_CUDA(h, scope.err);
    ZL_CUDA(h, cudaDeviceSynchronize());
    for (int i = 0; i < h->ncanary; ++i) {
        unsigned char tail[CANARY_BYTES];
        ZL_CUDA(h, cudaMemcpy(tail, h->canary[i], CANARY_BYTES, cudaMemcpyDeviceToHost));
        bool ok = true;
        for (size_t k = 0; k < CANARY_BYTES; ++k) ok = ok && tail[k] == (unsigned char)CANARY_BYTE;
        if (!ok) ++*damaged;
    }
    return ZL_OK;
}

zl_status zl_debug_report(zl_handle *h, uint32_t *h_record) {
    if (!h || !h_record) return ZL_ERR_INVALID_ARG;
    memset(h_record, 0, 4 * sizeof(uint32_t));
    if (!h->fb.dbg) return ZL_OK;
    DeviceScope scope(h->cfg.device);
    ZL_CUDA(h, scope.err);
    ZL_CUDA(h, cudaDeviceSynchronize());
    ZL_CUDA(h, cudaMemcpy(h_record, h->fb.dbg, 4 * sizeof(uint32_t), cudaMemcpyDeviceToHost));
    ZL_CUDA(h, cudaMemset(h->fb.dbg, 0, 4 * sizeof(uint32_t)));
    return ZL_OK;
}

zl_status zl_filter_counts(zl_handle *h, int32_t B, uint32_t *h_filtered, uint32_t *h_refined, uint32_t *h_overflow) {
    if (!h || B < 1 || B > h->cfg.max_batch) return ZL_ERR_INVALID_ARG;
    DeviceScope scope(h->cfg.device);
    ZL_CUDA(h, scope.err);
    ZL_CUDA(h, cudaDeviceSynchronize());
    uint32_t *dst[3] = {h_filtered, h_refined, h_overflow};
    const size_t off[3] = {offsetof(zl::InstMeta, count), offsetof(zl::InstMeta, count2), offsetof(zl::InstMeta, overflow)};
    for (int i = 0; i < 3; ++i)
        if (dst[i])
            ZL_CUDA(h, cudaMemcpy2D(dst[i], sizeof(uint32_t), (const char *)h->d_meta + off[i], sizeof(zl::InstMeta),
                                    sizeof(uint32_t), (size_t)B, cudaMemcpyDeviceToHost));
    return ZL_OK;
}

zl_status zl_predict_select_batched(zl_handle *h, const int64_t *d_last, const int64_t *d_interval, int32_t B,
                                    int32_t *d_idx, int64_t *d_barrier, int64_t *d_wait, int32_t *d_status,
                                    void *cuda_stream) {
    if (!h || !h->d_pred) return ZL_ERR_INVALID_ARG;
    if (B < 1 || B > h->cfg.max_batch) return ZL_ERR_INVALID_ARG;
    if (!on_device(h->cfg.device)) return ZL_ERR_INVALID_ARG;
    if (h->cfg.objective == ZL_OBJ_RANGE && h->fb.table != nullptr) {
        // the filter route (and its fallback) on generated rows: the predicted matrix is never written
        if (!d_last || !d_interval || !d_idx || !d_barrier || !d_wait) return ZL_ERR_INVALID_ARG;
        if (((uintptr_t)d_last & 7) || ((uintptr_t)d_interval & 7) || ((uintptr_t)d_barrier & 7) || ((uintptr_t)d_wait & 7) ||
            ((uintptr_t)d_idx & 3) || ((uintptr_t)d_status & 3))
            return ZL_ERR_INVALID_ARG;
        const LaunchPlan p = make_plan(h, B);
        if (p.smem > 200 * 1024) return ZL_ERR_UNSUPPORTED;
        cudaEvent_t *ev = (h->prof_ev && h->prof_calls < h->prof_cap) ? h->prof_ev + PROF_EVENTS * (size_t)h->prof_calls : nullptr;
        Pipeline q;
        q.ts = nullptr; q.B = B; q.n = h->cfg.n_workers; q.R = h->cfg.lookahead_R; q.objective = ZL_OBJ_RANGE;
        q.flags = h->cfg.flags & ~ZL_FLAG_CHECK_SORTED; q.num_sms = h->num_sms;
        q.meta = h->d_meta; q.seg = h->d_seg; q.nres = h->nres;
        q.fb = h->fb;
        q.filter_threads = h->opt_filter_threads; q.filter_rows = h->opt_filter_rows; q.filter_round = h->opt_filter_round; q.pdl_off = h->opt_pdl_off;
        q.prologue_threads = h->opt_prologue_threads; q.tail_threads = h->opt_tail_threads;
        if (h->opt_no_filter) { q.fb.table = nullptr; q.fb.scap = 0; }
        q.cluster = h->opt_cluster; q.filter_stages = h->opt_filter_stages;
        q.checks_off = h->opt_checks_off; q.filter_bulk = h->opt_filter_bulk; q.tail_cap = h->opt_tail_cap; q.rest_per_sm = 0; q.max_rounds = h->opt_max_rounds; q.small = small_route(h) ? 1 : 0; q.rest_split = rest_split_now(h) ? 1 : 2;
        if (q.fb.flags) {                           // the two sets of per-call flags alternate; a call zeroes the next call's set
            uint32_t *base = h->fb.flags;
            q.fb.flags = base + 8 * (h->epoch & 1);
            q.fb.flags_next = base + 8 * ((h->epoch + 1) & 1);
            ++h->epoch;
        }
        q.idx = d_idx; q.barrier = d_barrier; q.wait = d_wait; q.status = d_status;
        enqueue(q, p, (cudaStream_t)cuda_stream, ev, zl::AriBatch{d_last, d_interval});
        if (ev) ++h->prof_calls;
        ZL_CUDA(h, cudaGetLastError());
        h->launches += zl_launches_per_call(h);
        return ZL_OK;
    }
    zl_status rc = zl_predict_batched(d_last, d_interval, B, h->cfg.n_workers, h->cfg.lookahead_R, h->d_pred, cuda_stream);
    if (rc != ZL_OK) return rc;
    ++h->launches;
    return zl_select_batched(h, h->d_pred, B, d_idx, d_barrier, d_wait, d_status, cuda_stream);
}

zl_status zl_select_batched_host(zl_handle *h, const int64_t *h_ts, int32_t B, int32_t *h_idx, int64_t *h_barrier,
                                 int64_t *h_wait, int32_t *h_status) {
    if (!h || !h_ts || !h_idx || !h_barrier || !h_wait) return ZL_ERR_INVALID_ARG;
    if (B < 1 || B > h->cfg.max_batch) return ZL_ERR_INVALID_ARG;
    const size_t n = h->cfg.n_workers, R = h->cfg.lookahead_R, mb = h->cfg.max_batch;
    DeviceScope scope(h->cfg.device);
    ZL_CUDA(h, scope.err);
    if (!h->s_ts) {
        ZL_CUDA(h, cudaStreamCreateWithFlags(&h->s_stream, cudaStreamNonBlocking));
        ZL_CUDA(h, cudaMalloc((void **)&h->s_ts, mb * n * R * 8));
        ZL_CUDA(h, cudaMalloc((void **)&h->s_idx, mb * n * 4));
        ZL_CUDA(h, cudaMalloc((void **)&h->s_barrier, mb * 8));
        ZL_CUDA(h, cudaMalloc((void **)&h->s_wait, mb * 8));
        ZL_CUDA(h, cudaMalloc((void **)&h->s_status, mb * 4));
        h->staging_bytes = mb * n * R * 8 + mb * n * 4 + mb * 20;
    }
    cudaStream_t st = h->s_stream;
    ZL_CUDA(h, cudaMemcpyAsync(h->s_ts, h_ts, (size_t)B * n * R * 8, cudaMemcpyHostToDevice, st));
    zl_status rc = zl_select_batched(h, h->s_ts, B, h->s_idx, h->s_barrier, h->s_wait, h->s_status, st);
    if (rc != ZL_OK) return rc;
    ZL_CUDA(h, cudaMemcpyAsync(h_idx, h->s_idx, (size_t)B * n * 4, cudaMemcpyDeviceToHost, st));
    ZL_CUDA(h, cudaMemcpyAsync(h_barrier, h->s_barrier, (size_t)B * 8, cudaMemcpyDeviceToHost, st));
    ZL_CUDA(h, cudaMemcpyAsync(h_wait, h->s_wait, (size_t)B * 8, cudaMemcpyDeviceToHost, st));
    if (h_status) ZL_CUDA(h, cudaMemcpyAsync(h_status, h->s_status, (size_t)B * 4, cudaMemcpyDeviceToHost, st));
    ZL_CUDA(h, cudaStreamSynchronize(st));
    return ZL_OK;
}

// ------------------------------------------------------------------------------ no-allocation entry point
// Scratch for zl_select_batched_noalloc lives in this fixed device array instead of a handle's
// cudaMalloc'ed buffers.  Layout: NOALLOC_MAX_BATCH InstMeta records, then NOALLOC_MAX_SEGS SegResult
// records.  Every GPU that loads the library holds these bytes until the process exits.
namespace {
constexpr int NOALLOC_MAX_BATCH = 256;
constexpr int NOALLOC_MAX_SEGS = 16384;                       // B * (time segments per instance) of one call
constexpr size_t NOALLOC_META_BYTES = (size_t)NOALLOC_MAX_BATCH * sizeof(zl::InstMeta);
constexpr size_t NOALLOC_BYTES = NOALLOC_META_BYTES + (size_t)NOALLOC_MAX_SEGS * sizeof(zl::SegResult);
static_assert(NOALLOC_META_BYTES % 256 == 0, "segment records must start on a 256-byte boundary");
constexpr int NOALLOC_MAX_DEVICES = 64;
}  // namespace

static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_BYTES];

namespace {
std::mutex g_noalloc_mutex;
void *g_noalloc_ptr[NOALLOC_MAX_DEVICES];                     // device address of the array, per device
int g_noalloc_sms[NOALLOC_MAX_DEVICES];
}  // namespace

int32_t zl_noalloc_max_batch(void) { return NOALLOC_MAX_BATCH; }
size_t zl_noalloc_scratch_bytes(void) { return NOALLOC_BYTES; }

zl_status zl_select_batched_noalloc(int32_t n_workers, int32_t lookahead_R, int32_t objective, int32_t flags,
                                    const int64_t *d_ts, int32_t B, int32_t *d_idx, int64_t *d_barrier,
                                    int64_t *d_wait, int32_t *d_status, void *cuda_stream) {
    if (!d_ts || !d_idx || !d_barrier || !d_wait) return ZL_ERR_INVALID_ARG;
    if (n_workers < 1 || lookahead_R < 1 || B < 1) return ZL_ERR_INVALID_ARG;
    if (objective != ZL_OBJ_RANGE && objective != ZL_OBJ_SUM) return ZL_ERR_INVALID_ARG;
    if (flags & ~(ZL_FLAG_CHECK_SORTED | ZL_FLAG_FULL_SWEEP)) return ZL_ERR_INVALID_ARG;
    if (((uintptr_t)d_ts & 7) || ((uintptr_t)d_barrier & 7) || ((uintptr_t)d_wait & 7) || ((uintptr_t)d_idx & 3) ||
        ((uintptr_t)d_status & 3))
        return ZL_ERR_INVALID_ARG;
    if (n_workers > zl::MAX_WORKERS || (long long)n_workers * lookahead_R > (1LL << 31) - 1) return ZL_ERR_UNSUPPORTED;
    if (B > NOALLOC_MAX_BATCH) {
        fprintf(stderr, "zl_select_batched_noalloc: B = %d exceeds the fixed scratch (at most %d instances per call)\n",
                B, NOALLOC_MAX_BATCH);
        return ZL_ERR_UNSUPPORTED;
    }
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NOALLOC_MAX_DEVICES) return ZL_ERR_CUDA;

    // a handle on the stack carries the shape to the launch planner; nothing is allocated for it
    zl_handle tmp;
    memset(&tmp, 0, sizeof(tmp));
    tmp.cfg.n_workers = n_workers; tmp.cfg.lookahead_R = lookahead_R; tmp.cfg.max_batch = B;
    tmp.cfg.objective = objective; tmp.cfg.device = dev; tmp.cfg.flags = flags;
    {
        // once per device, with that device current: the array's name is only a host-side stand-in, the
        // kernels need the address the runtime reports for it
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (!g_noalloc_ptr[dev]) {
            void *ptr = nullptr;
            cudaError_t e = cudaGetSymbolAddress((void **)&ptr, g_noalloc_scratch);
            if (e == cudaSuccess) e = cudaDeviceGetAttribute(&g_noalloc_sms[dev], cudaDevAttrMultiProcessorCount, dev);
            if (e == cudaSuccess) e = raise_shared_memory_limits();
            if (e != cudaSuccess || !ptr) return ZL_ERR_CUDA;
            g_noalloc_ptr[dev] = ptr;
        }
        tmp.num_sms = g_noalloc_sms[dev];
    }
    const LaunchPlan p = make_plan(&tmp, B);
    if (p.smem > 200 * 1024) return ZL_ERR_UNSUPPORTED;
    if ((long long)B * p.nseg > NOALLOC_MAX_SEGS) {
        fprintf(stderr, "zl_select_batched_noalloc: %d instances x %d time segments exceed the fixed scratch (%d records)\n",
                B, p.nseg, NOALLOC_MAX_SEGS);
        return ZL_ERR_UNSUPPORTED;
    }
    zl::InstMeta *meta = (zl::InstMeta *)g_noalloc_ptr[dev];
    zl::SegResult *seg = (zl::SegResult *)((unsigned char *)g_noalloc_ptr[dev] + NOALLOC_META_BYTES);
    // Nothing in the scratch has to start at zero: the prologue rewrites every InstMeta of this call and
    // every sweep CTA rewrites its SegResult before finalize reads them, so the last call's contents are
    // never read.  (The filter path of the handle-based entry point needs two more buffers and is not used here.)
    Pipeline q;
    q.ts = d_ts; q.B = B; q.n = n_workers; q.R = lookahead_R; q.objective = objective; q.flags = flags; q.num_sms = tmp.num_sms;
    q.meta = meta; q.seg = seg; q.nres = p.nseg;
    memset(&q.fb, 0, sizeof(q.fb));
    q.filter_threads = q.filter_rows = q.filter_round = 0; q.pdl_off = 0; q.prologue_threads = q.tail_threads = 0; q.cluster = q.filter_stages = 0; q.checks_off = 0; q.filter_bulk = 0; q.tail_cap = 0; q.rest_per_sm = 0; q.max_rounds = 0; q.rest_split = 0; q.small = (long long)n_workers * lookahead_R <= zl::SMALL_MAX && B <= 4 * std::max(1, tmp.num_sms) ? 1 : 0;
    q.idx = d_idx; q.barrier = d_barrier; q.wait = d_wait; q.status = d_status;
    enqueue(q, p, (cudaStream_t)cuda_stream, nullptr, zl::MatBatch{d_ts});
    return cudaGetLastError() == cudaSuccess ? ZL_OK : ZL_ERR_CUDA;
}

}  // extern "C"
