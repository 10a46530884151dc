// k_prologue: column scans per instance (tmin, t0 = max_p e^p_1, lmin = min_p e^p_R, span) and, on the RANGE
// filter route, the per-row estimates, the filter table and the per-call counters.  k_check_sorted: the optional
// full check that every row is non-decreasing.
#include "zl_batch.cuh"
#include "zl_host.h"

namespace zl {

// ------------------------------------------------------------------------------ prologue
// Column scans per instance, and (RANGE, 32-bit instances) the filter table.
//
// Filter table.  For the RANGE objective an element e matters only if next(e) > G(T(e)), where
// G(t) = max(t, t0, max{next(e') : T(e') < t}) is max(Z) of the best Z whose minimum is at time t:
//   - if next(e) <= G(T(e)) the element cannot raise the running maximum, so PM of every later
//     element is unchanged without it;
//   - and it is not needed as a candidate: moving min(Z) from e to the next element in time keeps
//     max(Z) and shrinks d_Z (or, among equal times, another element of the group qualifies).
// Any lower bound L(t) <= G(t) therefore gives an exact filter "keep e iff next(e) > max(T, L(T))".
// The table holds, per time cell c, L = max(t0, max over a few slow rows p of the first element of p
// at or after the cell's start) - every such element is next(e') of an element before the cell, or a
// first element (<= t0).  Slow rows (long iterations) are the ones that set G most of the time.

template <class SRC>
__global__ void __launch_bounds__(1024, 1) k_prologue(const SRC src, int n, int R, int objective, int flags,
                                                    InstMeta *meta, FilterBufs F) {
    grid_dep_wait();
    const int b = blockIdx.x, tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
    const typename SRC::Rows rows = src.inst(b, n, R);
    __shared__ uint64_t s[4][32];
    __shared__ InstMeta sm;
    __shared__ uint32_t tab[FILTER_MAX_CELLS];
    extern __shared__ __align__(16) unsigned char smem[];
    int64_t *col1 = (int64_t *)smem, *colR = col1 + n;        // first and last column: read once, used three times
    uint64_t mn1 = ~0ull, mx1 = 0, mnR = ~0ull, mxR = 0;      // order-preserving unsigned images of int64
    for (int p = tid; p < n; p += nt) {
        const auto rw = rows.row(p);
        const int64_t r1 = rw.at(0), rR = rw.at(R - 1);
        col1[p] = r1; colR[p] = rR;
        const uint64_t e1 = (uint64_t)r1 ^ (1ull << 63);
        const uint64_t eR = (uint64_t)rR ^ (1ull << 63);
        mn1 = min(mn1, e1); mx1 = max(mx1, e1);
        mnR = min(mnR, eR); mxR = max(mxR, eR);
    }
    mn1 = warp_reduce(mn1, OpMin()); mx1 = warp_reduce(mx1, OpMax());
    mnR = warp_reduce(mnR, OpMin()); mxR = warp_reduce(mxR, OpMax());
    if (lane == 0) { s[0][warp] = mn1; s[1][warp] = mx1; s[2][warp] = mnR; s[3][warp] = mxR; }
    __syncthreads();
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
            if (objective == ZL_OBJ_RANGE && F.table && m.use32 && m.status == ZL_OK) {
                // (T - 1) < lmin for every T <= lmin, so ((T - 1) * cscale) >> 32 < cells
                m.cscale = (uint32_t)max((uint64_t)1, min((uint64_t)0xffffffffu, ((uint64_t)F.cells << 32) / m.lmin));
                m.fscale = (uint32_t)max((uint64_t)1, min((uint64_t)0xffffffffu, ((uint64_t)F.fcells << 32) / m.lmin));
            }
        }
        sm = m;
    }
    __syncthreads();
    const InstMeta M = sm;
    if (b == 0 && tid < 3 && F.flags) { F.flags[tid] = 0; if (F.flags_next) F.flags_next[tid] = 0; }
    if (M.cscale != 0) {
        const uint32_t cells = (uint32_t)F.cells, cscale = M.cscale, lmin = (uint32_t)M.lmin;
        const uint32_t wcell = 0xffffffffu / cscale + 2;          // > 2^32 / cscale
        const int64_t tmin = M.tmin;
        uint32_t *cmx = F.cellmax + (size_t)b * F.fcells;
        for (uint32_t c = tid; c < cells; c += nt) tab[c] = (uint32_t)M.t0;
        for (uint32_t c = tid; c < (uint32_t)F.fcells; c += nt) cmx[c] = 0;
        for (int k = tid; k < F.nbk; k += nt) F.bcnt[(size_t)b * F.nbk + k] = 0;
        // per row: how many of its elements are expected to be <= lmin (rows are close to arithmetic);
        // the filter pass uses it only to decide how much of the row to request up front
        for (int p = tid; p < n; p += nt) {
            const uint64_t e1 = (uint64_t)(col1[p] - tmin) + 1;
            const uint64_t eR = (uint64_t)(colR[p] - tmin) + 1;
            uint64_t est = R;
            if (eR > e1 && (uint64_t)lmin < eR)
                est = (uint64_t)lmin <= e1 ? 1 : ((uint64_t)lmin - e1) * (uint64_t)(R - 1) / (eR - e1) + 8;
            F.rowhint[(size_t)b * n + p] = (uint32_t)min(est, (uint64_t)R);
        }
        __syncthreads();
        // one slow row per warp: the row with the longest span in the warp's group of rows
        const int groups = min(n, FILTER_ROWS);
        const int gsz = (n + groups - 1) / groups;
        for (int gidx = warp; gidx < groups; gidx += nw) {
            const int p0 = gidx * gsz, p1 = min(p0 + gsz, n);
            int bestp = -1;
            uint64_t bspan = 0;
            for (int p = p0 + lane; p < p1; p += 32) {
                const uint64_t span = (uint64_t)(colR[p] - col1[p]);
                if (bestp < 0 || span > bspan) { bspan = span; bestp = p; }
            }
            const uint64_t best = warp_reduce(bspan, OpMax());
            const unsigned who = __ballot_sync(FULL, bestp >= 0 && bspan == best);
            if (!who) continue;
            const int row = __shfl_sync(FULL, bestp, __ffs(who) - 1);
            const auto rp = rows.row(row);
            // element i is the first element of the row at or after every cell start in (e_{i-1}, e_i]:
            // the cells after the one holding e_{i-1}, up to the one holding e_i
            // (four 32-element steps are loaded before any is used: the loop is latency bound otherwise)
            for (int i0 = 1; i0 < R; i0 += 128) {
                uint32_t pv[4], cv[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int i = i0 + 32 * k + lane;
                    pv[k] = 0xffffffffu; cv[k] = 0;
                    if (i < R) {
                        pv[k] = (uint32_t)(rp.at(i - 1) - tmin + 1);
                        cv[k] = (uint32_t)(rp.at(i) - tmin + 1);
                    }
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (pv[k] <= lmin) {              // also false past the end of the row
                        const uint32_t c_from = cell_of(pv[k], cscale) + 1;
                        const uint32_t c_to = cv[k] <= lmin ? cell_of(cv[k], cscale) : cells - 1;
                        for (uint32_t c = c_from; c <= c_to && c < cells; ++c) atomicMax(&tab[c], cv[k]);
                    }
                }
                if (__shfl_sync(FULL, pv[3], 0) > lmin) break;    // the rest of the row lies after lmin
            }
        }
        __syncthreads();
        uint32_t *tg = F.table + (size_t)b * cells;
        // dmin: every T of cell c is <= tmax_c, so an element with next - T <= tab[c] - tmax_c for all c never passes
        uint32_t dloc = 0xffffffffu;
        for (uint32_t c = tid; c < cells; c += nt) {
            const uint32_t v = tab[c];
            tg[c] = v;
            // upper bound of the times of cell c: a cell spans fewer than wcell time units
            const uint64_t tmax_c = min((uint64_t)lmin, (uint64_t)(c + 1) * wcell + 1);
            dloc = min(dloc, (uint64_t)v > tmax_c ? (uint32_t)(v - tmax_c) : 0u);
        }
        dloc = warp_reduce(dloc, OpMin());
        __syncthreads();
        uint32_t *red = (uint32_t *)&s[0][0];
        if (lane == 0) red[warp] = dloc;
        __syncthreads();
        if (tid == 0) {
            uint32_t d = 0xffffffffu;
            for (int w = 0; w < nw; ++w) d = min(d, red[w]);
            sm.dmin = d;
        }
        __syncthreads();
    }
    if (tid == 0) meta[b] = sm;
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
    launch_dep(!((q.pdl_off >> 9) & 1), k_prologue<SRC>, dim3(q.B), dim3(pthreads), (size_t)q.n * 16, st, src, q.n, q.R, q.objective, q.flags, q.meta, fb);
    if (std::is_same<SRC, MatBatch>::value && (q.flags & ZL_FLAG_CHECK_SORTED)) {
        const size_t total = (size_t)q.B * q.n * q.R;
        const int blocks = (int)std::min<size_t>((total + 255) / 256, (size_t)q.num_sms * 16);
        launch_dep(!((q.pdl_off >> 0) & 1), k_check_sorted, dim3(blocks), dim3(256), 0, st, q.ts, q.n, q.R, total, q.meta);
    }
}

void enqueue_prologue(const Pipeline &q, const FilterBufs &fb, cudaStream_t st, const MatBatch &src) { enqueue_prologue_t(q, fb, st, src); }
void enqueue_prologue(const Pipeline &q, const FilterBufs &fb, cudaStream_t st, const AriBatch &src) { enqueue_prologue_t(q, fb, st, src); }

cudaError_t prologue_limits() {
    cudaError_t e = cudaFuncSetAttribute(k_prologue<MatBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_WORKERS * 16);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_prologue<AriBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_WORKERS * 16);
    return e;
}

}  // namespace zl
