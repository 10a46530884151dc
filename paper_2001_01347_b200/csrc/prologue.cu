// k_prologue: column scans per instance (tmin, t0 = max_p e^p_1, lmin = min_p e^p_R, span) for the bucket route and the
// plain segment sweep.  k_check_sorted: the optional full check that every row is non-decreasing.
#include "zl_batch.cuh"
#include "zl_host.h"

namespace zl {

// ------------------------------------------------------------------------------ prologue
// Column scans per instance: tmin = min_p e^p_1, t0 = max_p e^p_1, lmin = min_p e^p_R, the span; validity of the
// instance.  (The RANGE filter route has its own first kernel, k_range_head.)
template <class SRC>
__global__ void __launch_bounds__(1024, 1) k_prologue(const SRC src, int n, int R, int objective, int flags,
                                                    InstMeta *meta, FilterBufs F) {
    grid_dep_wait();
    const int b = blockIdx.x, tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
    const typename SRC::Rows rows = src.inst(b, n, R);
    __shared__ uint64_t s[4][32];
    uint64_t mn1 = ~0ull, mx1 = 0, mnR = ~0ull, mxR = 0;      // order-preserving unsigned images of int64
    for (int p = tid; p < n; p += nt) {
        const auto rw = rows.row(p);
        const uint64_t e1 = (uint64_t)rw.at(0) ^ (1ull << 63);
        const uint64_t eR = (uint64_t)rw.at(R - 1) ^ (1ull << 63);
        mn1 = min(mn1, e1); mx1 = max(mx1, e1);
        mnR = min(mnR, eR); mxR = max(mxR, eR);
    }
    mn1 = warp_reduce(mn1, OpMin()); mx1 = warp_reduce(mx1, OpMax());
    mnR = warp_reduce(mnR, OpMin()); mxR = warp_reduce(mxR, OpMax());
    if (lane == 0) { s[0][warp] = mn1; s[1][warp] = mx1; s[2][warp] = mnR; s[3][warp] = mxR; }
    __syncthreads();
    if (b == 0 && tid < 3 && F.flags) { F.flags[tid] = 0; if (F.flags_next) F.flags_next[tid] = 0; }
    if (tid == 0) {
        uint64_t a = s[0][0], c = s[1][0], d = s[2][0], e = s[3][0];
        for (int w = 1; w < nw; ++w) { a = min(a, s[0][w]); c = max(c, s[1][w]); d = min(d, s[2][w]); e = max(e, s[3][w]); }
        const int64_t tmin = (int64_t)(a ^ (1ull << 63)), t0 = (int64_t)(c ^ (1ull << 63));
        const int64_t lmin = (int64_t)(d ^ (1ull << 63)), tmax = (int64_t)(e ^ (1ull << 63));
        InstMeta m;
        m.tmin = tmin;
        m.status = ZL_OK;
        m.cscale = 0; m.fscale = 0; m.count = 0; m.count2 = 0; m.overflow = 0; m.dmin = 0;
        if (tmin < 0 || tmax >= VALUE_LIMIT || tmax < tmin || lmin < tmin) {
            m.status = ZL_ERR_INVALID_ARG;     // outside [0, 2^62), or first/last columns out of order
            m.t0 = m.lmin = m.tend = 1; m.use32 = 1;
        } else {
            m.t0 = (uint64_t)(t0 - tmin) + 1;
            m.lmin = (uint64_t)(lmin - tmin) + 1;
            m.tend = (uint64_t)(tmax - tmin) + 1;
            m.use32 = m.tend < 0xfffffffeull;
            if (objective == ZL_OBJ_SUM && m.tend > (uint64_t)INT64_MAX / (uint64_t)n) m.status = ZL_ERR_UNSUPPORTED;
        }
        meta[b] = m;
    }
    (void)flags;
}

// Optional full check that every row is non-decreasing.
__global__ void k_check_sorted(const int64_t *ts, int n, int R, size_t total, InstMeta *meta) {
    grid_dep_wait();
    const size_t per = (size_t)n * R;
    for (size_t f = (size_t)blockIdx.x * blockDim.x + threadIdx.x; f < total; f += (size_t)gridDim.x * blockDim.x) {
        if ((f % R) == 0) continue;
        if (ldg64(ts + f) < ldg64(ts + f - 1)) atomicCAS(&meta[f / per].status, (int)ZL_OK, (int)ZL_ERR_UNSORTED);
    }
}

template <class SRC>
static void enqueue_prologue_t(const Pipeline &q, const FilterBufs &fb, cudaStream_t st, const SRC &src) {
    // many small instances: small CTAs so that several share an SM; few large ones: one large CTA each
    const bool many = q.B > 2 * q.num_sms;
    const int pthreads = q.prologue_threads ? q.prologue_threads
                         : many ? std::max(128, std::min(256, pow2_ceil(2 * q.n))) : std::max(512, std::min(1024, pow2_ceil(q.n)));
    // the first kernel of a call is scheduled early too: it waits (grid_dep_wait) for whatever precedes it in the stream
    launch_dep(!((q.pdl_off >> 9) & 1), k_prologue<SRC>, dim3(q.B), dim3(pthreads), 0, st, src, q.n, q.R, q.objective, q.flags, q.meta, fb);
}

void enqueue_check_sorted(const Pipeline &q, cudaStream_t st) {
    const size_t total = (size_t)q.B * q.n * q.R;
    const int blocks = (int)std::min<size_t>((total + 255) / 256, (size_t)q.num_sms * 16);
    launch_dep(!((q.pdl_off >> 0) & 1), k_check_sorted, dim3(blocks), dim3(256), 0, st, q.ts, q.n, q.R, total, q.meta);
}

void enqueue_prologue(const Pipeline &q, const FilterBufs &fb, cudaStream_t st, const MatBatch &src) { enqueue_prologue_t(q, fb, st, src); }
void enqueue_prologue(const Pipeline &q, const FilterBufs &fb, cudaStream_t st, const AriBatch &src) { enqueue_prologue_t(q, fb, st, src); }

cudaError_t prologue_limits() { return cudaSuccess; }

}  // namespace zl
