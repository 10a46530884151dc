// ZipLine barrier-selection search for sm_100a: kernels and the C ABI (see include/zipline.h).
//
// Per instance: n sorted rows of R int64 timestamps.  Every kernel of a call is enqueued on the caller's
// stream with programmatic stream serialization and starts with grid_dep_wait().
//
//   k_prologue  column scans (tmin, t0 = max_p e^p_1, lmin = min_p e^p_R, span); for the RANGE filter
//               route also the per-row estimates, the filter table and the per-call counters.
//
// RANGE (max(Z) - min(Z)), filter route: an element matters only if its `next` exceeds G, the running
// maximum of `next` over everything earlier (floored by t0); see the comment above k_prologue.
//   k_filter    one warp per row streams the row in storage order (cp.async ring), forms (T, next),
//               tests it against the table and appends the survivors to per-CTA lists.
//   k_tail      instances with few survivors: refine, sort into time order, prefix max of next,
//               evaluate d = max(T, t0, PM) - T, keep the first minimum, recover the indices.
//   k_tilemax, k_cellscan, k_refine, k_buckets
//               instances with many survivors: G at every fine time cell, drop what cannot matter,
//               bucket by time, sort + scan + evaluate per group of buckets.
//
// SUM (sum_p (max(Z) - z_p)): every element matters, so the whole instance is put into time order, bucket by
// bucket (the bucket route; also taken by RANGE instances small enough to be one shared-memory batch).
//   k_sum_plan     bucket start times from the expected element density over the timeline.
//   k_sum_index    one streaming pass: per row and bucket, the index of the row's first element in the bucket.
//   k_sum_buckets  per bucket: gather the rows' runs (delta + first flag, or next), sort in shared memory,
//                  scan with the carry-in the runs' predecessors give, evaluate, keep the first minimum.
//
// Instances neither fast route can take (time span of 2^32 us or more, an overflowing list or bucket): the
// segment sweep.
//   k_sweep     the timeline is cut into time segments.  A CTA walks its segment in rounds: every row
//               advances a cursor over the elements inside the round's time window (the rows are
//               sorted, so the n-way merge is a set of cursors), attaches the payload the scan needs
//               (next / delta + first flag) and appends it to a shared-memory batch.  A full batch is
//               sorted into time order, scanned (prefix max of next / prefix sums of delta and flag)
//               and evaluated.  Carry-ins at a segment start come from per-row binary searches, so
//               segments are independent.
//
//   k_finalize  minimum over an instance's partial results, barrier, per-worker index recovery.
//
// Predicted rows (e_i = last + (i + 1) * interval) need not exist in memory: k_prologue, k_sweep, k_tail and
// k_finalize are templates over a row source (MatBatch reads the matrix, AriBatch computes the rule), and
// k_filter_arith is the filter pass on such rows.
//   k_trace     per-position intermediates of the steps for small instances (tests).
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
#include "zl_device.cuh"

namespace zl {

constexpr int MAX_WORKERS = 4096;
constexpr int MAX_SEGMENTS = 256;
constexpr int TRACE_MAX = 4096;
constexpr int64_t VALUE_LIMIT = (int64_t)1 << 62;

struct InstMeta {
    int64_t tmin;        // min_p e^p_1
    uint64_t t0;         // max_p e^p_1, relative (tmin -> 1)
    uint64_t lmin;       // min_p e^p_R, relative
    uint64_t tend;       // max_p e^p_R, relative  (= span + 1)
    int32_t status;      // zl_status of the instance
    int32_t use32;       // relative times fit 32 bits
    uint32_t cscale;     // filter route: time cell of relative time T = ((T - 1) * cscale) >> 32 (monotone in T);
                         // 0: the instance does not take the filter route
    uint32_t fscale;     // same map onto the fine cells of the refinement
    uint32_t count;      // survivors of the filter pass
    uint32_t count2;     // survivors of the refinement
    uint32_t overflow;   // a survivor list overflowed: the instance takes the segment sweep instead
    uint32_t dmin;       // no element whose own iteration (next - T) is this short can pass the filter table
};

struct SegResult {
    uint64_t d;          // objective value of the segment's best candidate
    uint64_t t;          // its relative time (min(Z) for RANGE, the barrier for SUM)
    int32_t valid;
    int32_t status;
};

// Where the rows of an instance come from: the stored [B][n][R] matrix, or - for predicted rows - the
// rule e_i = last + (i + 1) * interval itself, so that the matrix never has to exist in memory.  A worker with
// a negative input reads as a row of -1, one whose last prediction would reach 2^62 as a row of 2^62: both
// make the column scans report the instance invalid.
struct MatRow {
    const int64_t *p;
    __device__ __forceinline__ int64_t at(int i) const { return (int64_t)__ldg((const long long *)(p + i)); }
};
struct AriRow {
    int64_t l, v;
    __device__ __forceinline__ int64_t at(int i) const { return l + (int64_t)(i + 1) * v; }
};
struct MatRows {
    const int64_t *inst; int R;
    __device__ __forceinline__ MatRow row(int p) const { return MatRow{inst + (size_t)p * R}; }
};
struct AriRows {
    const int64_t *last, *iv; int R;
    __device__ __forceinline__ AriRow row(int p) const {
        const int64_t l = (int64_t)__ldg((const long long *)(last + p)), v = (int64_t)__ldg((const long long *)(iv + p));
        if (l < 0 || v < 0) return AriRow{-1, 0};
        if (__umul64hi((uint64_t)R, (uint64_t)v) != 0 || (uint64_t)R * (uint64_t)v >= (uint64_t)VALUE_LIMIT ||
            (uint64_t)l + (uint64_t)R * (uint64_t)v >= (uint64_t)VALUE_LIMIT) return AriRow{VALUE_LIMIT, 0};
        return AriRow{l, v};
    }
};
struct MatBatch {
    const int64_t *ts;
    typedef MatRows Rows;
    __device__ __forceinline__ MatRows inst(int b, int n, int R) const { return MatRows{ts + (size_t)b * n * R, R}; }
};
struct AriBatch {
    const int64_t *last, *iv;
    typedef AriRows Rows;
    __device__ __forceinline__ AriRows inst(int b, int n, int R) const { return AriRows{last + (size_t)b * n, iv + (size_t)b * n, R}; }
};

// Buffers of the RANGE filter route (all nullptr / 0 when the route is off).  The time up to lmin is
// cut into `cells` coarse cells (filter table, shared memory) and `fcells` fine cells (refinement);
// `nbk` buckets are runs of fcells / nbk consecutive fine cells.
struct FilterBufs {
    uint32_t *table;     // [B][cells]        lower bound of G at the start of each cell (from a few slow rows)
    uint32_t *rowhint;   // [B][n]            estimated number of elements of a row that are <= lmin
    uint32_t *cellmax;   // [B][fcells]       max `next` over the filter pass's survivors of each fine cell; after
                         //                   k_cellscan: G at the start of each fine cell
    uint32_t *tilemax;   // [B][fcells/4096]  max of cellmax per tile of 4096 fine cells (scratch of the cell scan)
    uint32_t *rcnt;      // [B][nreg]         survivors per region (one region per CTA of the filter pass)
    uint64_t *list1;     // [B][list1cap]     survivors of the filter pass as (T << 32 | next), by region
    uint32_t *flags;     // [3]               per call: some instance needs [0] scan/refine/buckets, [1] the segment sweep, [2] k_finalize
    uint32_t *bcnt;      // [B][nbk]          survivors of the refinement per bucket
    uint64_t *list2;     // [B][nbk][capb]    survivors of the refinement
    int32_t cells, fcells, nbk, capb, grp;   // grp: fewest buckets per CTA of the bucket sweep
    int32_t nreg, regcap, list1cap;          // set per call: regions per instance and their capacity
    // SUM bucket route (all nullptr / 0 when the route is off): the timeline is cut into `scells` uniform
    // cells; runs of cells form buckets of about `sM` elements; `stiles` tiles of TILE_BK buckets each.
    uint32_t *bnd;                           // [B][stiles*15 + 1]   time at which each bucket starts (non-decreasing)
    unsigned long long *cellacc;             // [B][scells + 1 + stiles*15 + 1]  scratch of the bucket plan
    uint16_t *itab;                          // [B][stiles][n][16]   per row: index of its first element in each bucket of the tile
    int32_t scells, sM, scap, stiles;        // scells == 0: every instance is a single bucket (n * R <= scap)
    int32_t ssub;                            // set per call: CTAs that share the buckets of one tile (small batches)
};

struct SweepParams {
    const int64_t *ts;
    InstMeta *meta;
    SegResult *seg;
    int32_t n, R, B, nseg, nres, G, cap, flags, target;   // nres: SegResult slots per instance
    int32_t filter;      // instances handled by the filter route are skipped
    const uint32_t *need; // filter on: [1] != 0 when some instance needs this sweep; nullptr: always run
};

// Buckets per CTA of the bucket sweep for an instance with `count` refined survivors: the static
// minimum `grp`, widened (by powers of two) so that a CTA expects about a quarter batch of survivors.
__device__ __forceinline__ int bucket_group(const FilterBufs &F, uint32_t count) {
    int g = F.grp;
    while (g < F.nbk && (uint64_t)count * (uint64_t)g * 2 < (uint64_t)F.nbk * (uint64_t)(F.capb / 2)) g <<= 1;
    return g;
}

// An instance goes through the filter route when it has a table and no survivor list overflowed.
__device__ __forceinline__ bool handled_by_filter(const InstMeta &M, int filter) {
    return filter && M.cscale != 0 && M.overflow == 0;
}

__device__ __forceinline__ uint32_t cell_of(uint32_t T, uint32_t cscale) { return __umulhi(T - 1, cscale); }

// Instances with at most this many survivors of the filter pass are finished by one CTA (k_tail);
// larger ones go through cell scan, refinement and the bucket sweep.
constexpr uint32_t TAIL_CAP = 2048;
__device__ __forceinline__ bool tail_instance(const InstMeta &M) { return M.count <= TAIL_CAP; }

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
constexpr int FILTER_ROWS = 32;      // rows that build the table
constexpr int FILTER_MAX_CELLS = 8192;

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
    if (b == 0 && tid < 3 && F.flags) F.flags[tid] = 0;
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

// ------------------------------------------------------------------------------ filter pass (RANGE)
// A CTA owns a block of rows of one instance (a "region").  Each warp streams its rows in storage
// order through a private shared-memory ring filled by 16-byte cp.async copies (FILTER_STAGES chunks of
// 64 timestamps in flight per warp), tests every element against the table and appends the survivors,
// as (T << 32 | next), to the region's list; the per-cell maximum of `next` over the survivors goes to
// cellmax for the refinement.  Rows whose length is odd, or a misaligned base, take 8-byte copies.
constexpr int FILTER_STAGES = 3;      // ring slots per warp
constexpr int FILTER_CHUNK = 256;     // timestamps per slot (FILTER_CHUNK / 64 16-byte copies per lane)
constexpr int FILTER_SLOT = FILTER_CHUNK + 2;   // + the successor of the slot's last element, + padding

__device__ __forceinline__ void cp_async16(void *smem, const void *gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"((uint32_t)__cvta_generic_to_shared(smem)), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async8(void *smem, const void *gmem) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;\n" ::"r"((uint32_t)__cvta_generic_to_shared(smem)), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
// wait until at most `pending` of this thread's most recent groups are still in flight
__device__ __forceinline__ void cp_async_wait_pending(int pending) {
    switch (pending) {
        case 0: asm volatile("cp.async.wait_group 0;\n" ::: "memory"); break;
        case 1: asm volatile("cp.async.wait_group 1;\n" ::: "memory"); break;
        case 2: asm volatile("cp.async.wait_group 2;\n" ::: "memory"); break;
        case 3: asm volatile("cp.async.wait_group 3;\n" ::: "memory"); break;
        case 4: asm volatile("cp.async.wait_group 4;\n" ::: "memory"); break;
        case 5: asm volatile("cp.async.wait_group 5;\n" ::: "memory"); break;
        case 6: asm volatile("cp.async.wait_group 6;\n" ::: "memory"); break;
        default: asm volatile("cp.async.wait_group 7;\n" ::: "memory"); break;
    }
}

struct FilterCtx {
    const uint32_t *tab; uint64_t *list; uint32_t *cellmax; unsigned int *scount;
    uint32_t cscale, fscale, lmin, regcap, dmin;
};

// Table test of the (up to) two elements of a lane, warp-aggregated append of the survivors.
__device__ __forceinline__ void filter_pair(const FilterCtx &c, int lane, bool va, uint32_t Ta, uint32_t na,
                                            bool vb, uint32_t Tb, uint32_t nb) {
    // cheap necessary condition first: most elements belong to fast workers and stop here
    bool ka = va && Ta <= c.lmin && na - Ta > c.dmin;
    bool kb = vb && Tb <= c.lmin && nb - Tb > c.dmin;
    if (!__any_sync(FULL, ka || kb)) return;
    if (ka) ka = na > max(Ta, c.tab[cell_of(Ta, c.cscale)]);
    if (kb) kb = nb > max(Tb, c.tab[cell_of(Tb, c.cscale)]);
    const unsigned ma = __ballot_sync(FULL, ka), mb = __ballot_sync(FULL, kb);
    if ((ma | mb) == 0) return;
    const int na_cnt = __popc(ma), tot = na_cnt + __popc(mb);
    unsigned base = 0;
    if (lane == 0) base = atomicAdd(c.scount, (unsigned)tot);
    base = __shfl_sync(FULL, base, 0);
    const unsigned below = (1u << lane) - 1u;
    if (ka) {
        const unsigned pos = base + __popc(ma & below);
        if (pos < c.regcap) c.list[pos] = ((uint64_t)Ta << 32) | na;
        atomicMax(&c.cellmax[cell_of(Ta, c.fscale)], na);
    }
    if (kb) {
        const unsigned pos = base + na_cnt + __popc(mb & below);
        if (pos < c.regcap) c.list[pos] = ((uint64_t)Tb << 32) | nb;
        atomicMax(&c.cellmax[cell_of(Tb, c.fscale)], nb);
    }
}

// The 64 elements of a slot starting at `off`: element pairs per lane, successor of the pair from the
// slot itself (the element after the slot's last one sits right behind it).  Returns the time of the
// last valid element handled by lane 31 (0xffffffff past the row's end).
__device__ __forceinline__ uint32_t filter_half(const FilterCtx &C, const int64_t *slot, int off, int i0, int lim, int R,
                                                uint32_t tminlo, int lane) {
    const int i = i0 + off + 2 * lane;
    const bool va = i < lim, vb = i + 1 < lim;                    // lim: end of what was requested of the row (<= R)
    const longlong2 ab = *reinterpret_cast<const longlong2 *>(slot + off + 2 * lane);
    const uint32_t Ta = va ? (uint32_t)(uint64_t)ab.x - tminlo : 0xffffffffu;
    const uint32_t Tb = vb ? (uint32_t)(uint64_t)ab.y - tminlo : 0xffffffffu;
    const uint32_t nb = i + 2 < R ? (uint32_t)(uint64_t)slot[off + 2 * lane + 2] - tminlo : 0xffffffffu;
    filter_pair(C, lane, va, Ta, Tb, vb, Tb, nb);
    return __shfl_sync(FULL, Tb, 31);
}

// 128 timestamps of a slot, with the one after them, that lie inside the row: no bounds checks, one vote
// for all four elements of a lane.  Returns the time of the last of the 128.
__device__ __forceinline__ uint32_t filter_slot_inside(const FilterCtx &C, const int64_t *slot, uint32_t tminlo, int lane) {
    const longlong2 p0 = *reinterpret_cast<const longlong2 *>(slot + 2 * lane);
    const longlong2 p1 = *reinterpret_cast<const longlong2 *>(slot + 64 + 2 * lane);
    const uint32_t a0 = (uint32_t)(uint64_t)p0.x - tminlo, b0 = (uint32_t)(uint64_t)p0.y - tminlo;
    const uint32_t a1 = (uint32_t)(uint64_t)p1.x - tminlo, b1 = (uint32_t)(uint64_t)p1.y - tminlo;
    const uint32_t n0 = (uint32_t)(uint64_t)slot[2 * lane + 2] - tminlo, n1 = (uint32_t)(uint64_t)slot[64 + 2 * lane + 2] - tminlo;
    const bool k = (a0 <= C.lmin && b0 - a0 > C.dmin) || (b0 <= C.lmin && n0 - b0 > C.dmin) ||
                   (a1 <= C.lmin && b1 - a1 > C.dmin) || (b1 <= C.lmin && n1 - b1 > C.dmin);
    if (__any_sync(FULL, k)) {                                   // rare: some element may pass the table
        filter_pair(C, lane, true, a0, b0, true, b0, n0);
        filter_pair(C, lane, true, a1, b1, true, b1, n1);
    }
    return __shfl_sync(FULL, b1, 31);
}

__global__ void __launch_bounds__(1024) k_filter(const int64_t *ts, int n, int R, int flags, int rows_per_cta, int req_round,
                                                  InstMeta *meta, FilterBufs F) {
    grid_dep_wait();
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ unsigned int scount;
    const int b = blockIdx.y, tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
    const InstMeta M = meta[b];
    uint32_t *rc = F.rcnt + (size_t)b * F.nreg + blockIdx.x;
    if (M.status != ZL_OK || M.cscale == 0) { if (tid == 0) *rc = 0; return; }
    const uint32_t cells = (uint32_t)F.cells, lmin = (uint32_t)M.lmin;
    const uint32_t tminlo = (uint32_t)(uint64_t)M.tmin - 1u;     // relative time = low word of t - tminlo
    uint32_t *tab = (uint32_t *)smem;
    int64_t *ring = (int64_t *)(smem + (size_t)cells * 4) + (size_t)warp * FILTER_STAGES * FILTER_SLOT;
    const uint32_t *tg = F.table + (size_t)b * cells;
    for (uint32_t c = tid; c < cells; c += nt) tab[c] = tg[c];
    if (tid == 0) scount = 0;
    __syncthreads();
    const bool full = (flags & ZL_FLAG_FULL_SWEEP) != 0;
    FilterCtx C;
    C.tab = tab; C.list = F.list1 + (size_t)b * F.list1cap + (size_t)blockIdx.x * F.regcap;
    C.cellmax = F.cellmax + (size_t)b * F.fcells; C.scount = &scount;
    C.cscale = M.cscale; C.fscale = M.fscale; C.lmin = lmin; C.regcap = (uint32_t)F.regcap; C.dmin = M.dmin;
    const int r0 = blockIdx.x * rows_per_cta, r1 = min(r0 + rows_per_cta, n);
    const bool vec2 = (R % 2 == 0) && (((uintptr_t)ts & 15) == 0);
    const size_t rstride = (size_t)nw * R;                        // between consecutive rows of this warp

    // this warp's rows, in rounds of up to 32: lane j holds the request of the round's j-th row, i.e. how many of
    // its leading timestamps are copied through the ring (a multiple of 64, or R)
    for (int rbase = r0 + warp; rbase < r1; rbase += 32 * nw) {
        const int nrows = min(32, (r1 - rbase + nw - 1) / nw);
        int req = 0;
        if (lane < nrows) req = full ? R : min(R, (int)((F.rowhint[(size_t)b * n + rbase + lane * nw] + (uint32_t)(req_round - 1)) & ~(uint32_t)(req_round - 1)));
        const int64_t *row_i = ts + ((size_t)b * n + rbase) * R, *row_p = row_i;
        int ji = 0, ci = 0, jp = 0, cp = 0, inflight = 0, slot_i = 0, slot_p = 0;
        int req_i = __shfl_sync(FULL, req, 0), req_p = req_i;
        bool finished = false;                                     // the row being processed needs nothing more
        while (jp < nrows) {
            while (inflight < FILTER_STAGES && ji < nrows) {
                int64_t *slot = ring + (size_t)slot_i * FILTER_SLOT;
                const int base = ci * FILTER_CHUNK;
                const int i = base + 2 * lane;
                if (vec2) {
#pragma unroll
                    for (int k = 0; k < FILTER_CHUNK / 64; ++k)
                        if (i + 64 * k < req_i) cp_async16(slot + 64 * k + 2 * lane, row_i + i + 64 * k);
                } else {
#pragma unroll
                    for (int k = 0; k < FILTER_CHUNK / 32; ++k) {
                        const int e = i + (k >> 1) * 64 + (k & 1);
                        if (e < req_i) cp_async8(slot + (k >> 1) * 64 + 2 * lane + (k & 1), row_i + e);
                    }
                }
                // the element after the last one copied into this slot (its successor)
                const int endi = min(base + FILTER_CHUNK, req_i);
                if (lane == 31 && endi < R) cp_async8(slot + (endi - base), row_i + endi);
                cp_async_commit();
                ++inflight;
                slot_i = slot_i + 1 == FILTER_STAGES ? 0 : slot_i + 1;
                if (endi == req_i) {
                    ci = 0; ++ji; row_i += rstride;
                    req_i = __shfl_sync(FULL, req, min(ji, 31));
                } else {
                    ++ci;
                }
            }
            cp_async_wait_pending(inflight - 1);
            __syncwarp();
            const int i0 = cp * FILTER_CHUNK;
            const int L = min(FILTER_CHUNK, req_p - i0);           // timestamps of the row in this slot
            if (!finished) {
                const int64_t *slot = ring + (size_t)slot_p * FILTER_SLOT;
                uint32_t lastT = 0;
#pragma unroll
                for (int sub = 0; sub < FILTER_CHUNK; sub += 128) {
                    if (sub >= L || (sub && !full && lastT > lmin)) break;   // rows are sorted: the rest is past lmin
                    if (sub + 128 <= L && i0 + sub + 128 < R) {
                        lastT = filter_slot_inside(C, slot + sub, tminlo, lane);
                    } else {
                        lastT = filter_half(C, slot, sub, i0, req_p, R, tminlo, lane);
                        if (sub + 64 < L && (full || lastT <= lmin)) lastT = filter_half(C, slot, sub + 64, i0, req_p, R, tminlo, lane);
                    }
                }
                finished = !full && lastT > lmin;                  // rows are sorted: nothing later is <= lmin
            }
            __syncwarp();
            --inflight;
            slot_p = slot_p + 1 == FILTER_STAGES ? 0 : slot_p + 1;
            if (i0 + L == req_p) {
                if (!finished && !full && req_p < R) {
                    // the request ended before the row did: continue with plain loads
                    for (int j0 = req_p; j0 < R; j0 += 64) {
                        const int i = j0 + 2 * lane;
                        const bool va = i < R, vb = i + 1 < R;
                        const uint32_t Ta = va ? (uint32_t)(uint64_t)ldg64(row_p + i) - tminlo : 0xffffffffu;
                        const uint32_t Tb = vb ? (uint32_t)(uint64_t)ldg64(row_p + i + 1) - tminlo : 0xffffffffu;
                        uint32_t nb = __shfl_down_sync(FULL, Ta, 1);
                        if (lane == 31) nb = i + 2 < R ? (uint32_t)(uint64_t)ldg64(row_p + i + 2) - tminlo : 0xffffffffu;
                        filter_pair(C, lane, va, Ta, Tb, vb, Tb, nb);
                        if (__shfl_sync(FULL, Tb, 31) > lmin) break;
                    }
                }
                cp = 0; ++jp; row_p += rstride; finished = false;
                req_p = __shfl_sync(FULL, req, min(jp, 31));
            } else {
                ++cp;
            }
        }
    }
    __syncthreads();
    if (tid == 0) {
        const unsigned c = scount;
        *rc = min(c, (unsigned)F.regcap);
        if (c > (unsigned)F.regcap) meta[b].overflow = 1;
        if (c) atomicAdd(&meta[b].count, c);
    }
}

// The filter pass on predicted rows e_i = last + (i + 1) * interval, which are generated instead of read.  An
// element's own iteration is the row's interval, so a whole row whose interval does not exceed dmin is settled
// at once (only its last element, whose next is infinite, can pass); the other rows are walked up to lmin, an
// element per lane.  Same regions, lists and counters as k_filter.
__global__ void __launch_bounds__(256) k_filter_arith(const AriBatch src, int n, int R, int rows_per_cta, InstMeta *meta, FilterBufs F) {
    grid_dep_wait();
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ unsigned int scount;
    const int b = blockIdx.y, tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
    const InstMeta M = meta[b];
    uint32_t *rc = F.rcnt + (size_t)b * F.nreg + blockIdx.x;
    if (M.status != ZL_OK || M.cscale == 0) { if (tid == 0) *rc = 0; return; }
    const uint32_t cells = (uint32_t)F.cells;
    uint32_t *tab = (uint32_t *)smem;
    const uint32_t *tg = F.table + (size_t)b * cells;
    for (uint32_t c = tid; c < cells; c += nt) tab[c] = tg[c];
    if (tid == 0) scount = 0;
    __syncthreads();
    FilterCtx C;
    C.tab = tab; C.list = F.list1 + (size_t)b * F.list1cap + (size_t)blockIdx.x * F.regcap;
    C.cellmax = F.cellmax + (size_t)b * F.fcells; C.scount = &scount;
    C.cscale = M.cscale; C.fscale = M.fscale; C.lmin = (uint32_t)M.lmin; C.regcap = (uint32_t)F.regcap; C.dmin = M.dmin;
    const AriRows rows = src.inst(b, n, R);
    const int r0 = blockIdx.x * rows_per_cta, r1 = min(r0 + rows_per_cta, n);
    for (int r = r0 + warp; r < r1; r += nw) {
        const AriRow rw = rows.row(r);
        const int64_t rel0 = rw.l - M.tmin + 1;                   // relative time of element i: rel0 + (i + 1) * v, >= 1
        const int64_t v = rw.v, room = (int64_t)M.lmin - rel0;
        // elements not after lmin: (i + 1) * v <= room
        const int cnt = v == 0 ? (room >= 0 ? R : 0) : room < v ? 0 : (int)min((int64_t)R, room / v);
        if (cnt == 0) continue;
        if ((uint64_t)v <= (uint64_t)M.dmin) {
            if (cnt == R) filter_pair(C, lane, lane == 0, (uint32_t)(rel0 + (int64_t)R * v), 0xffffffffu, false, 0u, 0u);
            continue;
        }
        for (int i0 = 0; i0 < cnt; i0 += 32) {
            const int i = i0 + lane;
            const uint32_t T = (uint32_t)(rel0 + (int64_t)(i + 1) * v);
            filter_pair(C, lane, i < cnt, T, i + 1 < R ? T + (uint32_t)v : 0xffffffffu, false, 0u, 0u);
        }
    }
    __syncthreads();
    if (tid == 0) {
        const unsigned c = scount;
        *rc = min(c, (unsigned)F.regcap);
        if (c > (unsigned)F.regcap) meta[b].overflow = 1;
        if (c) atomicAdd(&meta[b].count, c);
    }
}

// ------------------------------------------------------------------------------ refinement (RANGE)
// The per-cell maxima of the filter pass give G exactly at every fine cell start (the survivors contain
// every element that ever raises the running maximum): k_cellscan turns cellmax, in place, into its
// exclusive prefix maximum floored by t0.  A survivor whose `next` does not exceed G at the start of its
// own cell cannot matter either, so k_refine drops it; the rest go to their time bucket.
constexpr int SCAN_TILE = 4096;

// pass 1: maximum of every tile of SCAN_TILE fine cells.  A fixed grid walks the (tile, instance) pairs.
__global__ void __launch_bounds__(256) k_tilemax(const InstMeta *meta, FilterBufs F, int B) {
    grid_dep_wait();
    __shared__ uint64_t tmp[34];
    if (F.flags[0] == 0) return;                                  // no instance takes this route in this call
    const int tid = threadIdx.x, nt = blockDim.x;
    const int tiles = (F.fcells + SCAN_TILE - 1) / SCAN_TILE;
    for (int item = blockIdx.x; item < tiles * B; item += gridDim.x) {
        const int b = item / tiles, t = item % tiles;
        const InstMeta M = meta[b];
        if (M.status != ZL_OK || !handled_by_filter(M, 1) || tail_instance(M)) continue;
        const uint32_t *cmx = F.cellmax + (size_t)b * F.fcells + (size_t)t * SCAN_TILE;
        const int len = min(SCAN_TILE, F.fcells - t * SCAN_TILE);
        uint32_t loc = 0;
        for (int i = tid; i < len; i += nt) loc = max(loc, cmx[i]);
        uint32_t tot;
        block_scan_excl<uint32_t>(loc, OpMax(), 0u, (uint32_t *)tmp, &tot);
        if (tid == 0) F.tilemax[(size_t)b * tiles + t] = tot;
    }
}

// pass 2: each tile becomes, in place, the exclusive prefix maximum over all cells before each of its
// cells, floored by t0: coalesced in, every thread scans a run of consecutive cells in shared memory,
// coalesced out.
__global__ void __launch_bounds__(256) k_cellscan(const InstMeta *meta, FilterBufs F, int B) {
    grid_dep_wait();
    __shared__ uint64_t tmp[34];
    __shared__ uint32_t tile[SCAN_TILE];
    if (F.flags[0] == 0) return;
    const int tid = threadIdx.x, nt = blockDim.x;
    const int tiles = (F.fcells + SCAN_TILE - 1) / SCAN_TILE;
    for (int item = blockIdx.x; item < tiles * B; item += gridDim.x) {
        const int b = item / tiles, t = item % tiles;
        const InstMeta M = meta[b];
        if (M.status != ZL_OK || !handled_by_filter(M, 1) || tail_instance(M)) continue;
        uint32_t *cmx = F.cellmax + (size_t)b * F.fcells + (size_t)t * SCAN_TILE;
        const int len = min(SCAN_TILE, F.fcells - t * SCAN_TILE);
        uint32_t before = 0;
        for (int i = tid; i < t; i += nt) before = max(before, F.tilemax[(size_t)b * tiles + i]);
        uint32_t carry;
        block_scan_excl<uint32_t>(before, OpMax(), 0u, (uint32_t *)tmp, &carry);
        carry = max(carry, (uint32_t)M.t0);
        for (int i = tid; i < len; i += nt) tile[i] = cmx[i];
        __syncthreads();
        const int per = (len + nt - 1) / nt;
        const int c0 = min(tid * per, len), c1 = min(c0 + per, len);
        uint32_t loc = 0;
        for (int c = c0; c < c1; ++c) loc = max(loc, tile[c]);
        uint32_t tot;
        uint32_t run = max(block_scan_excl<uint32_t>(loc, OpMax(), 0u, (uint32_t *)tmp, &tot), carry);
        for (int c = c0; c < c1; ++c) { const uint32_t v = tile[c]; tile[c] = run; run = max(run, v); }
        __syncthreads();
        for (int i = tid; i < len; i += nt) cmx[i] = tile[i];
        __syncthreads();
    }
}

__global__ void __launch_bounds__(256) k_refine(InstMeta *meta, FilterBufs F, int B) {
    grid_dep_wait();
    if (F.flags[0] == 0) return;
    const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31;
    const int cpb_shift = __ffs(F.fcells / F.nbk) - 1;            // fine cells per bucket is a power of two
    for (int item = blockIdx.x; item < F.nreg * B; item += gridDim.x) {
        const int b = item / F.nreg, reg = item % F.nreg;
        const InstMeta M = meta[b];
        if (M.status != ZL_OK || !handled_by_filter(M, 1) || tail_instance(M)) continue;
        const uint32_t m = F.rcnt[(size_t)b * F.nreg + reg];
        if (m == 0) continue;
        const uint32_t *g = F.cellmax + (size_t)b * F.fcells;     // G at fine cell starts
        const uint64_t *src = F.list1 + (size_t)b * F.list1cap + (size_t)reg * F.regcap;
        uint32_t *bcnt = F.bcnt + (size_t)b * F.nbk;
        uint64_t *dst = F.list2 + (size_t)b * F.nbk * F.capb;
        unsigned kept = 0;
        bool over = false;
        // four elements a step, so that four list loads and then four table look-ups are in flight together
        for (uint32_t i0 = tid; i0 < m; i0 += 4 * nt) {
            uint64_t w[4];
            uint32_t c[4], gv[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) { const uint32_t i = i0 + k * nt; w[k] = i < m ? src[i] : 0ull; }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                c[k] = w[k] ? cell_of((uint32_t)(w[k] >> 32), M.fscale) : 0u;
                gv[k] = __ldg(g + c[k]);
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint32_t T = (uint32_t)(w[k] >> 32), nx = (uint32_t)w[k];
                if (w[k] && nx > max(T, gv[k])) {
                    const uint32_t bk = c[k] >> cpb_shift;
                    const uint32_t pos = atomicAdd(&bcnt[bk], 1u);
                    if (pos < (uint32_t)F.capb) dst[(size_t)bk * F.capb + pos] = w[k]; else over = true;
                    ++kept;
                }
            }
        }
        kept = warp_reduce(kept, OpAdd());
        if (lane == 0 && kept) atomicAdd(&meta[b].count2, kept);
        if (over) { meta[b].overflow = 1; F.flags[1] = 1; }
    }
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

// ------------------------------------------------------------------------------ batch engine
// Sort the batch into time order, scan it and evaluate every candidate; per-thread best is kept
// in (bd, bt).  RANGE: carry = max of `next` over everything before the batch.  SUM: carryS/carryC =
// sum of the latest element / number of started workers before the batch.
// Shared-memory workspace of a batch: `in` receives the nodes, `out` their sorted order.
template <typename K> struct BatchWS { Key<K> *in, *out; uint32_t *cnt; int cap; };

template <typename K, int OBJ>
__device__ void run_batch(const BatchWS<K> &ws, int m, K t0, int n, uint64_t *tmp64, K carryMax, uint64_t &carryS,
                          uint32_t &carryC, uint64_t &bd, uint64_t &bt) {
    if (m == 0) return;
    const Key<K> *keys;
    if (m <= 128) {
        // very small batches: every node counts the nodes that come before it (one barrier)
        for (int q = threadIdx.x; q < m; q += blockDim.x) {
            const Key<K> k = ws.in[q];
            int rank = 0;
            for (int i = 0; i < m; ++i) { const Key<K> o = ws.in[i]; rank += (k > o) || (!(o > k) && i < q); }
            ws.out[rank] = k;
        }
        __syncthreads();
        keys = ws.out;
    } else if (m <= 256) {
        // small batches: the comparison network (mostly warp-local steps) beats the bookkeeping of the slot sort
        int P2 = 64;
        while (P2 < m) P2 <<= 1;
        for (int i = m + threadIdx.x; i < P2; i += blockDim.x) ws.in[i] = Key<K>::inf();
        __syncthreads();
        bitonic_sort(ws.in, P2);
        keys = ws.in;
    } else {
        slot_sort<K>(ws.in, ws.out, ws.cnt, ws.cap, m, ws.cap, tmp64);
        keys = ws.out;
    }
    const int P = m;
    const int ipt = (P + blockDim.x - 1) / blockDim.x;
    const int k0 = threadIdx.x * ipt, k1 = min(k0 + ipt, m);
    if (OBJ == ZL_OBJ_RANGE) {
        K lmax = 0;
        for (int k = k0; k < k1; ++k) lmax = max(lmax, keys[k].v());
        K tot;
        K pm = block_scan_excl<K>(lmax, OpMax(), (K)0, (K *)tmp64, &tot);
        pm = max(pm, carryMax);
        for (int k = k0; k < k1; ++k) {
            const K T = keys[k].t();
            const K g = max(max(T, t0), pm);          // max(Z) of the best Z whose minimum is this element
            if (g != kinf<K>()) {
                const uint64_t d = (uint64_t)(g - T);
                if (d < bd || (d == bd && (uint64_t)T < bt)) { bd = d; bt = T; }
            }
            pm = max(pm, keys[k].v());
        }
    } else {
        uint64_t ls = 0;
        uint32_t lc = 0;
        for (int k = k0; k < k1; ++k) { ls += keys[k].v(); lc += keys[k].v() == keys[k].t(); }
        uint64_t tots;
        uint32_t totc;
        uint64_t s = block_scan_excl<uint64_t>(ls, OpAdd(), 0ull, tmp64, &tots) + carryS;
        uint32_t c = block_scan_excl<uint32_t>(lc, OpAdd(), 0u, (uint32_t *)tmp64, &totc) + carryC;
        for (int k = k0; k < k1; ++k) {
            const K T = keys[k].t(), dl = keys[k].v();
            s += dl;                                   // sum over started workers of their latest element
            c += dl == T;                              // a first element carries delta == T (previous = 0)
            if (c == (uint32_t)n) {
                const uint64_t w = (uint64_t)n * (uint64_t)T - s;
                if (w < bd || (w == bd && (uint64_t)T < bt)) { bd = w; bt = T; }
            }
        }
        carryS += tots;
        carryC += totc;
    }
    __syncthreads();
}

// Block minimum of (objective, time), compared as a pair, over the per-thread bests -> out.  red: 32 shared
// 64-bit words that nobody reads any more; every thread calls; two barriers.
__device__ void block_best_to_result(uint64_t bd, uint64_t bt, uint32_t status, uint64_t *red, unsigned int *sstatus,
                                     SegResult &out) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = (blockDim.x + 31) >> 5;
    __shared__ uint64_t red_t[32];
    for (int d = 16; d > 0; d >>= 1) {
        const uint64_t od = shfl_xor(bd, d), ot = shfl_xor(bt, d);
        if (od < bd || (od == bd && ot < bt)) { bd = od; bt = ot; }
    }
    if (lane == 0) { red[warp] = bd; red_t[warp] = bt; }
    if (status != ZL_OK) atomicMax(sstatus, status);
    __syncthreads();
    if (warp == 0) {
        uint64_t gd = lane < nw ? red[lane] : ~0ull, gt = lane < nw ? red_t[lane] : ~0ull;
        for (int d = 16; d > 0; d >>= 1) {
            const uint64_t od = shfl_xor(gd, d), ot = shfl_xor(gt, d);
            if (od < gd || (od == gd && ot < gt)) { gd = od; gt = ot; }
        }
        if (lane == 0) {
            out.d = gd; out.t = gt;
            out.valid = gd != ~0ull || gt != ~0ull;
            out.status = (int32_t)*sstatus;
        }
    }
    __syncthreads();
}

// ------------------------------------------------------------------------------ sweep
struct SweepShared {
    unsigned int count;       // nodes in the batch
    unsigned int overflow;
    unsigned int consumed;
    unsigned int pad;
    unsigned long long vmax;  // max `next` seen this round
    unsigned long long minhead;
    unsigned long long carryS;
    unsigned int carryC;
    unsigned int status;
    uint64_t tmp[34];
};

template <typename K, int OBJ, class ROWS>
__device__ void sweep_segment(const SweepParams &P, const InstMeta &M, const ROWS &rows, SweepShared &sh,
                              uint32_t *curA, uint32_t *curB, const BatchWS<K> &ws, int seg_index, SegResult &out) {
    Key<K> *keys = ws.in;
    const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31;
    const int n = P.n, R = P.R, G = P.G, NG = nt / G;
    const int gi = tid / G, g = tid % G;
    const unsigned gshift = lane & ~(G - 1);
    const unsigned gmask = G == 32 ? FULL : ((1u << G) - 1u);
    const K INF = kinf<K>();
    const int64_t tmin = M.tmin;
    const K t0 = (K)M.t0;

    // time range of this segment, relative times in [1, tend]
    const bool cut = OBJ == ZL_OBJ_RANGE && !(P.flags & ZL_FLAG_FULL_SWEEP);
    const uint64_t tend = cut ? M.lmin : M.tend;
    const uint64_t width = (tend + P.nseg - 1) / P.nseg;
    const uint64_t seg_lo = 1 + (uint64_t)seg_index * width;
    const uint64_t seg_hi = min(seg_lo + width, tend + 1);
    uint64_t bd = ~0ull, bt = ~0ull;          // per-thread best (objective, time)
    uint32_t status = ZL_OK;

    K floorv = 0;                              // max of next over every element before the current round
    if (tid == 0) { sh.count = 0; sh.carryS = 0; sh.carryC = 0; sh.vmax = 0; sh.status = 0; }
    __syncthreads();
    if (seg_lo <= tend) {
        // ---- carry-in: per-row lower bound of the segment start
        if (seg_index == 0) {
            for (int r = tid; r < n; r += nt) curA[r] = 0;
        } else {
            const int64_t a_raw = tmin + (int64_t)(seg_lo - 1);
            unsigned long long vloc = 0, sloc = 0;
            unsigned int cloc = 0;
            for (int r = tid; r < n; r += nt) {
                const auto row = rows.row(r);
                int lo = 0, hi = R;               // first index with row[i] >= a_raw
                while (lo < hi) {
                    const int mid = (lo + hi) >> 1;
                    if (row.at(mid) < a_raw) lo = mid + 1; else hi = mid;
                }
                curA[r] = (uint32_t)lo;
                if (lo > 0) {
                    if (OBJ == ZL_OBJ_RANGE) {
                        const unsigned long long v = lo < R ? (unsigned long long)(K)(row.at(lo) - tmin + 1) : (unsigned long long)INF;
                        vloc = max(vloc, v);
                    } else {
                        sloc += (unsigned long long)(K)(row.at(lo - 1) - tmin + 1);
                        cloc += 1;
                    }
                }
            }
            if (OBJ == ZL_OBJ_RANGE) {
                vloc = warp_reduce((uint64_t)vloc, OpMax());
                if (lane == 0) atomicMax(&sh.vmax, vloc);
            } else {
                sloc = warp_reduce((uint64_t)sloc, OpAdd());
                cloc = warp_reduce((uint32_t)cloc, OpAdd());
                if (lane == 0) { atomicAdd(&sh.carryS, sloc); atomicAdd(&sh.carryC, cloc); }
            }
        }
        __syncthreads();
        floorv = (K)sh.vmax;
        uint64_t carryS = sh.carryS;
        uint32_t carryC = sh.carryC;
        K carryMax = floorv;                   // prefix max of next before the current batch
        __syncthreads();

        uint32_t *cur = curA, *nxt = curB;
        uint64_t rlo = seg_lo;
        // nominal round: `target` elements out of the segment's share of the instance
        uint64_t delta = max((uint64_t)1, (seg_hi - seg_lo) / max((uint64_t)1, ((uint64_t)n * R / P.nseg) / max(1, P.target)));
        uint32_t count_before = 0;
        uint64_t rounds = 0;
        const uint64_t max_rounds = 4 * (uint64_t)n * R + 4096;

        while (rlo < seg_hi) {
            if (OBJ == ZL_OBJ_RANGE && cut && floorv == INF) break;     // a row ran out: no later Z is complete
            if (++rounds > max_rounds) { status = ZL_ERR_TIMEOUT; break; }
            const uint64_t rhi64 = min(rlo + delta, seg_hi);
            const K rhi = (K)rhi64;
            if (tid == 0) { sh.overflow = 0; sh.consumed = 0; sh.minhead = ~0ull; }
            __syncthreads();

            unsigned long long vloc = 0, hloc = ~0ull;
            unsigned int cons_n = 0;
            for (int rb = 0; rb < n; rb += NG) {
                const int r = rb + gi;
                const bool act = r < n;
                const auto row = rows.row(act ? r : 0);
                uint32_t c = act ? cur[r] : (uint32_t)R;
                bool more = act;
                for (;;) {
                    const uint32_t idx = c + g;
                    const bool have = more && idx < (uint32_t)R;
                    const K T = have ? (K)(row.at((int)idx) - tmin + 1) : INF;
                    const bool cons = have && T < rhi;
                    bool app = false;
                    Key<K> key = Key<K>::inf();
                    if (cons) {
                        ++cons_n;
                        if (OBJ == ZL_OBJ_RANGE) {
                            const K nx = idx + 1 < (uint32_t)R ? (K)(row.at((int)idx + 1) - tmin + 1) : INF;
                            vloc = max(vloc, (unsigned long long)nx);
                            app = nx > max(T, floorv);            // only elements that raise the running max matter
                            key = Key<K>::make(T, nx);
                        } else {
                            const K pv = idx > 0 ? (K)(row.at((int)idx - 1) - tmin + 1) : (K)0;
                            app = idx == 0 || T != pv;             // repeated timestamps of a row add nothing
                            key = Key<K>::make(T, T - pv);
                        }
                    }
                    const unsigned bal = __ballot_sync(FULL, cons);
                    const unsigned am = __ballot_sync(FULL, app);
                    if (am) {
                        const int leader = __ffs(am) - 1;
                        unsigned base = 0;
                        if (lane == leader) base = atomicAdd(&sh.count, __popc(am));
                        base = __shfl_sync(FULL, base, leader);
                        if (app) {
                            const unsigned slot = base + __popc(am & ((1u << lane) - 1u));
                            if (slot < (unsigned)P.cap) keys[slot] = key; else sh.overflow = 1;
                        }
                    }
                    const int m = __popc((bal >> gshift) & gmask);
                    const K headT = shfl_idx(T, (int)(gshift + min(m, G - 1)));
                    if (more) {
                        c += m;
                        if (m < G) { more = false; if (g == 0) hloc = min(hloc, (unsigned long long)headT); }
                    }
                    if (!__any_sync(FULL, more)) break;
                }
                if (act && g == 0) nxt[r] = c;
            }
            cons_n = warp_reduce((uint32_t)cons_n, OpAdd());
            hloc = warp_reduce((uint64_t)hloc, OpMin());
            if (OBJ == ZL_OBJ_RANGE) vloc = warp_reduce((uint64_t)vloc, OpMax());
            if (lane == 0) {
                atomicAdd(&sh.consumed, cons_n);
                atomicMin(&sh.minhead, hloc);
                if (OBJ == ZL_OBJ_RANGE) atomicMax(&sh.vmax, vloc);
            }
            __syncthreads();
            const bool overflow = sh.overflow != 0;
            const uint32_t consumed = sh.consumed;
            const uint32_t count = min(sh.count, (unsigned)P.cap);
            const uint64_t minhead = sh.minhead;
            const K vmax = (K)sh.vmax;
            __syncthreads();
            if (overflow) {
                // the round does not fit: flush what was there, or shorten the window; cursors are not committed
                if (count_before > 0) {
                    run_batch<K, OBJ>(ws, (int)count_before, t0, n, sh.tmp, carryMax, carryS, carryC, bd, bt);
                    carryMax = floorv;
                    count_before = 0;
                } else {
                    delta = max((uint64_t)1, delta >> 1);
                }
                if (tid == 0) { sh.count = 0; sh.vmax = (unsigned long long)floorv; }
                __syncthreads();
                continue;
            }
            // commit the round
            { uint32_t *t = cur; cur = nxt; nxt = t; }
            count_before = count;
            if (OBJ == ZL_OBJ_RANGE) floorv = max(floorv, vmax);
            rlo = max(rhi64, minhead == ~0ull ? seg_hi : (uint64_t)(K)minhead);
            {   // steer the window toward `target` elements per round
                const float f = (float)P.target / (float)max(consumed, (uint32_t)max(1, P.target / 4));
                delta = (uint64_t)fmaxf(1.f, fminf((float)delta * f, 4.0e18f));
            }
            if (count_before > (uint32_t)(P.cap / 2)) {
                run_batch<K, OBJ>(ws, (int)count_before, t0, n, sh.tmp, carryMax, carryS, carryC, bd, bt);
                carryMax = floorv;
                count_before = 0;
                if (tid == 0) sh.count = 0;
                __syncthreads();
            }
        }
        if (count_before > 0)
            run_batch<K, OBJ>(ws, (int)count_before, t0, n, sh.tmp, carryMax, carryS, carryC, bd, bt);
    }

    block_best_to_result(bd, bt, status, sh.tmp, &sh.status, out);
}

template <int OBJ, class SRC>
__global__ void __launch_bounds__(1024) k_sweep(const SweepParams P, const SRC src) {
    grid_dep_wait();
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ SweepShared sh;
    uint32_t *curA = (uint32_t *)smem;
    uint32_t *curB = curA + P.n;
    // shared memory: row cursors | batch nodes | sorted batch | slot counters
    unsigned char *kb = smem + (((size_t)2 * P.n * sizeof(uint32_t) + 15) & ~(size_t)15);
    unsigned char *kb2 = kb + (size_t)P.cap * 8;
    uint32_t *kcnt = (uint32_t *)(kb2 + (size_t)P.cap * 8);
    if (P.need && P.need[1] == 0) return;                        // the filter route finished every instance
    // a fixed number of CTAs walks the (instance, segment) pairs
    const int items = P.B * P.nseg;
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const int b = item / P.nseg, sidx = item % P.nseg;
        const InstMeta M = P.meta[b];
        if (handled_by_filter(M, P.filter)) continue;            // the bucket sweep wrote this instance's results
        SegResult &out = P.seg[(size_t)b * P.nres + sidx];
        if (M.status != ZL_OK) {
            if (threadIdx.x == 0) { out.d = ~0ull; out.t = ~0ull; out.valid = 0; out.status = ZL_OK; }
            continue;
        }
        const typename SRC::Rows inst = src.inst(b, P.n, P.R);
        if (M.use32) {
            const BatchWS<uint32_t> ws{(Key<uint32_t> *)kb, (Key<uint32_t> *)kb2, kcnt, P.cap};
            sweep_segment<uint32_t, OBJ>(P, M, inst, sh, curA, curB, ws, sidx, out);
        } else {
            SweepParams Q = P;
            Q.cap = P.cap / 2;                      // 16-byte nodes: half as many fit
            const BatchWS<uint64_t> ws{(Key<uint64_t> *)kb, (Key<uint64_t> *)kb2, kcnt, Q.cap};
            sweep_segment<uint64_t, OBJ>(Q, M, inst, sh, curA, curB, ws, sidx, out);
        }
        __syncthreads();
    }
}

// Sort and sweep the refined survivors.  CTA (g, b) takes buckets [g*grp, (g+1)*grp) of instance b in
// time order, packs whole buckets into shared-memory batches and runs each batch with the running
// maximum of `next` over everything before it (the prefix maximum of cellmax up to the batch's first cell).
__global__ void __launch_bounds__(256) k_buckets(const InstMeta *meta, FilterBufs F, int n, int nres, SegResult *seg, int B) {
    grid_dep_wait();
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ uint64_t tmp[34];
    __shared__ unsigned int sstatus, fill;
    if (F.flags[0] == 0) return;                                  // no instance takes this route in this call
    const int tid = threadIdx.x, nt = blockDim.x;
    const int ngroups = (F.nbk + F.grp - 1) / F.grp;
    Key<uint32_t> *keys = (Key<uint32_t> *)smem;
    const BatchWS<uint32_t> ws{keys, keys + F.capb, (uint32_t *)(keys + 2 * (size_t)F.capb), F.capb};
    for (int item = blockIdx.x; item < ngroups * B; item += gridDim.x) {
    const int b = item / ngroups, g = item % ngroups;
    __syncthreads();                                              // shared state of the previous item is done with
    const InstMeta M = meta[b];
    if (M.status != ZL_OK || !handled_by_filter(M, 1) || tail_instance(M)) continue;
    const uint32_t *bcnt = F.bcnt + (size_t)b * F.nbk;
    const uint32_t *g0 = F.cellmax + (size_t)b * F.fcells;        // G at fine cell starts (after k_cellscan)
    const uint64_t *list = F.list2 + (size_t)b * F.nbk * F.capb;
    const int grp = bucket_group(F, M.count2);
    if (g * grp >= F.nbk) continue;                              // fewer, wider groups than items for this instance
    const int first = g * grp, last = min(first + grp, F.nbk);
    const int cpb = F.fcells / F.nbk;
    if (tid == 0) { sstatus = 0; fill = 0; }
    __syncthreads();
    // running max of next over everything before the group's first cell
    const uint32_t carry0 = g0[(size_t)first * cpb];
    uint64_t bd = ~0ull, bt = ~0ull, cs = 0;
    uint32_t cc = 0;
    uint32_t mine = 0;
    for (int k = first + tid; k < last; k += nt) mine += min(bcnt[k], (uint32_t)F.capb);
    uint32_t group_total;
    block_scan_excl<uint32_t>(mine, OpAdd(), 0u, (uint32_t *)tmp, &group_total);
    if (group_total <= (uint32_t)F.capb) {
        // one batch: warps copy whole buckets side by side; offsets come from a running count
        const int lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
        for (int k = first + warp; k < last; k += nw) {
            const uint32_t c = min(bcnt[k], (uint32_t)F.capb);
            if (c == 0) continue;
            uint32_t off = 0;
            if (lane == 0) off = atomicAdd(&fill, c);
            off = __shfl_sync(FULL, off, 0);
            const uint64_t *src = list + (size_t)k * F.capb;
            for (uint32_t i = lane; i < c; i += 32) keys[off + i].w = src[i];
        }
        __syncthreads();
        run_batch<uint32_t, ZL_OBJ_RANGE>(ws, (int)group_total, (uint32_t)M.t0, n, tmp, carry0, cs, cc, bd, bt);
    } else {
        int m = 0;
        uint32_t carry_batch = carry0;
        for (int k = first; k < last; ++k) {
            const int c = (int)min(bcnt[k], (uint32_t)F.capb);
            if (c == 0) continue;
            if (m + c > F.capb) {
                run_batch<uint32_t, ZL_OBJ_RANGE>(ws, m, (uint32_t)M.t0, n, tmp, carry_batch, cs, cc, bd, bt);
                carry_batch = g0[(size_t)k * cpb];        // G at the start of the next batch's first bucket
                m = 0;
            }
            const uint64_t *src = list + (size_t)k * F.capb;
            for (int i = tid; i < c; i += nt) keys[m + i].w = src[i];
            m += c;
            __syncthreads();
        }
        if (m > 0) run_batch<uint32_t, ZL_OBJ_RANGE>(ws, m, (uint32_t)M.t0, n, tmp, carry_batch, cs, cc, bd, bt);
    }
    block_best_to_result(bd, bt, ZL_OK, tmp, &sstatus, seg[(size_t)b * nres + g]);
    }
}

// ------------------------------------------------------------------------------ SUM bucket route
// Every element matters for the prefix sums of the SUM objective, so the whole instance is put into
// time order - but never as one list in HBM.  The timeline is cut into buckets of about sM elements:
//   k_sum_plan     per instance: expected element density over uniform time cells from the rows' end points
//                  (rows are close to arithmetic), cumulated; bucket k starts at the time where the cumulated
//                  expectation reaches k * sM.
//   k_sum_index    one streaming pass: a warp per row reads the row in storage order and notes, for every
//                  bucket, the index of the row's first element in it (the index table; 2 bytes per row
//                  and bucket, tiles of TILE_BK buckets with 16 boundaries each).
//   k_sum_buckets  a CTA takes the buckets of a tile one after the other: it gathers each row's run
//                  [start, end) with independent loads (K2: delta from the row neighbour, first flag =
//                  delta == T), sorts the bucket in shared memory (K1 restricted to the bucket), scans delta
//                  and flag (K3) with the carry-in that the predecessors of the runs give directly
//                  (S = sum over rows of the last element before the bucket, cnt = rows that have one),
//                  evaluates n*T - S where cnt == n (K4) and keeps the first minimum (K5, per tile).
// A bucket that holds more than scap elements (rows far from arithmetic) sends its instance to the
// segment sweep instead.  An instance with n * R <= scap is a single bucket (no plan, no index table);
// RANGE instances of that size take this route too: the payload of a node is then the same row's next
// element and the scan is the exclusive prefix maximum, d = max(T, t0, PM) - T.
constexpr int TILE_BK = 15;           // buckets per tile: 16 boundaries = 32 bytes per row and tile
constexpr int SUM_FP = 12;            // fixed-point bits of the expected counts

// In-place prefix scan of a shared-memory array by the whole block: every warp takes a contiguous piece
// and walks it 32 elements a step.  tmp: 32 shared words of T.  Every thread calls.
template <typename T, typename Op, bool EXCLUSIVE>
__device__ void smem_scan_inplace(T *a, int len, Op op, T identity, T *tmp) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    const int seg = (((len + nw - 1) / nw) + 31) & ~31;
    const int w0 = min(warp * seg, len), w1 = min(w0 + seg, len);
    T tot = identity;
    for (int i = w0 + lane; i < w1; i += 32) tot = op(tot, a[i]);
    tot = warp_reduce(tot, op);
    if (lane == 0) tmp[warp] = tot;
    __syncthreads();
    T carry = identity;
    for (int w = 0; w < warp; ++w) carry = op(carry, tmp[w]);
    for (int base = w0; base < w1; base += 32) {
        const int i = base + lane;
        const T v = i < w1 ? a[i] : identity;
        T inc = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const T y = shfl_up(inc, d);
            if (lane >= d) inc = op(y, inc);
        }
        T exc = shfl_up(inc, 1);
        if (lane == 0) exc = identity;
        if (i < w1) a[i] = op(carry, EXCLUSIVE ? exc : inc);
        carry = op(carry, shfl_idx(inc, 31));
    }
    __syncthreads();
}

// Dynamic shared memory: (scells + 1) 64-bit cell accumulators, then stiles * TILE_BK + 1 32-bit boundaries.
__global__ void __launch_bounds__(1024) k_sum_plan(const int64_t *ts, int n, int R, InstMeta *meta, FilterBufs F) {
    grid_dep_wait();
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ uint64_t tmp[34];
    const int b = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
    const InstMeta M = meta[b];
    if (b == 0 && tid == 0) F.flags[2] = 1;                       // k_finalize writes every instance's outputs
    if (M.status != ZL_OK) return;
    if (!M.use32) { if (tid == 0) F.flags[1] = 1; return; }      // wide times: the segment sweep
    if (F.scells == 0) {                                          // the instance is one bucket
        if (tid == 0) { meta[b].cscale = 1; meta[b].count = 1; meta[b].count2 = 1; }
        return;
    }
    const uint32_t cells = (uint32_t)F.scells;
    unsigned long long *acc = (unsigned long long *)smem;
    uint32_t *bsm = (uint32_t *)(acc + cells + 1);
    // (T - 1) < tend for every T, so ((T - 1) * cscale) >> 32 < cells
    const uint32_t cscale = (uint32_t)max((uint64_t)1, min((uint64_t)0xffffffffu, ((uint64_t)cells << 32) / M.tend));
    for (uint32_t c = tid; c <= cells; c += nt) acc[c] = 0;
    __syncthreads();
    const int64_t *inst = ts + (size_t)b * n * R;
    const uint32_t tminlo = (uint32_t)(uint64_t)M.tmin - 1u;
    // a row spreads its R elements evenly over the cells between its first and its last element
    for (int p = tid; p < n; p += nt) {
        const uint32_t e1 = (uint32_t)(uint64_t)ldg64(inst + (size_t)p * R) - tminlo;
        const uint32_t eR = (uint32_t)(uint64_t)ldg64(inst + (size_t)p * R + R - 1) - tminlo;
        const uint32_t c1 = cell_of(e1, cscale), cR = cell_of(eR, cscale);
        const unsigned long long x = ((unsigned long long)R << SUM_FP) / (unsigned long long)(cR - c1 + 1);
        atomicAdd(&acc[c1], x);
        atomicAdd(&acc[cR + 1], 0ull - x);
    }
    __syncthreads();
    smem_scan_inplace<unsigned long long, OpAdd, false>(acc, (int)cells, OpAdd(), 0ull, (unsigned long long *)tmp);   // expected elements per cell
    if (tid == 0) acc[cells] = 0;
    __syncthreads();
    smem_scan_inplace<unsigned long long, OpAdd, true>(acc, (int)cells + 1, OpAdd(), 0ull, (unsigned long long *)tmp);  // ... before each cell; [cells]: all
    // bucket k starts where the cumulated expectation reaches k * sM (linear inside a cell)
    const unsigned long long per_bucket = (unsigned long long)F.sM << SUM_FP;
    const uint32_t nbmax = (uint32_t)(F.stiles * TILE_BK);
    const uint32_t nbk = (uint32_t)max(1ull, min((unsigned long long)nbmax, (acc[cells] + per_bucket - 1) / per_bucket));
    // one thread per boundary (few): the cell in which the cumulated expectation passes k * sM, by bisection
    for (uint32_t k = 1 + tid; k < nbk; k += nt) {
        const unsigned long long target = (unsigned long long)k * per_bucket;      // < acc[cells]
        uint32_t c0 = 0, c1 = cells - 1;                          // last cell with acc[c] <= target
        while (c0 < c1) {
            const uint32_t mid = (c0 + c1 + 1) >> 1;
            if (acc[mid] <= target) c0 = mid; else c1 = mid - 1;
        }
        const unsigned long long lo = acc[c0], hi = acc[c0 + 1];  // lo <= target < hi
        const unsigned long long start = ((unsigned long long)c0 << 32) / cscale + 1, next = ((unsigned long long)(c0 + 1) << 32) / cscale + 1;
        bsm[k] = (uint32_t)min(0xfffffffeull, start + (target - lo) * (next - start) / max(1ull, hi - lo));
    }
    if (tid == 0) { bsm[0] = 0; bsm[nbk] = 0xffffffffu; }
    __syncthreads();
    smem_scan_inplace<uint32_t, OpMax, false>(bsm, (int)nbk + 1, OpMax(), 0u, (uint32_t *)tmp);   // boundaries must not decrease
    uint32_t *bnd = F.bnd + (size_t)b * (nbmax + 1);
    for (uint32_t k = tid; k <= nbk; k += nt) bnd[k] = bsm[k];
    if (tid == 0) {
        meta[b].cscale = cscale;
        meta[b].count = nbk;                                      // buckets of this instance
        meta[b].count2 = (nbk + TILE_BK - 1) / TILE_BK;           // tiles
    }
}

// Boundary k of a row (k = 0..buckets) is the index of its first element at or after the start time of
// bucket k.  Tile t keeps boundaries 15t .. 15t + 15, so a multiple of 15 is stored twice (last slot of one
// tile, first of the next).
__device__ __forceinline__ void index_entry(uint16_t *tab, int n, int stiles, int row, int k, int i) {
    const int t = k / TILE_BK, s = k - t * TILE_BK;
    if (t < stiles) tab[((size_t)t * n + row) * 16 + s] = (uint16_t)i;
    if (s == 0 && t > 0) tab[((size_t)(t - 1) * n + row) * 16 + TILE_BK] = (uint16_t)i;
}

constexpr int INDEX_UNROLL = 4;       // 32-element steps loaded before any is used

// Dynamic shared memory: the bucket start times of the instance.
__global__ void __launch_bounds__(256) k_sum_index(const int64_t *ts, int n, int R, const InstMeta *meta, FilterBufs F) {
    grid_dep_wait();
    extern __shared__ __align__(16) unsigned char smem[];
    uint32_t *a = (uint32_t *)smem;                               // [nbk + 1], a[nbk] = 0xffffffff
    const int b = blockIdx.y, lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    const InstMeta M = meta[b];
    if (M.status != ZL_OK || M.cscale == 0) return;
    const uint32_t tminlo = (uint32_t)(uint64_t)M.tmin - 1u;
    const int nbk = (int)M.count;
    const uint32_t *bg = F.bnd + (size_t)b * (F.stiles * TILE_BK + 1);
    for (int k = threadIdx.x; k <= nbk; k += blockDim.x) a[k] = bg[k];
    __syncthreads();
    uint16_t *tab = F.itab + (size_t)b * F.stiles * n * 16;
    for (int row = blockIdx.x * nw + warp; row < n; row += gridDim.x * nw) {
        const int64_t *rp = ts + ((size_t)b * n + row) * R;
        int kc = -1;                                              // boundaries 0..kc of this row are written
        for (int i0 = 0; i0 < R; i0 += 32 * INDEX_UNROLL) {
            int64_t v[INDEX_UNROLL];
#pragma unroll
            for (int u = 0; u < INDEX_UNROLL; ++u) {
                const int i = i0 + 32 * u + lane;
                v[u] = i < R ? ldg64(rp + i) : 0;
            }
#pragma unroll
            for (int u = 0; u < INDEX_UNROLL; ++u) {
                const int ibase = i0 + 32 * u;
                if (ibase >= R) break;                            // warp-uniform
                // the step's 32 elements, ascending over the lanes; lanes past the row's end hold +inf
                const uint32_t T = ibase + lane < R ? (uint32_t)(uint64_t)v[u] - tminlo : 0xffffffffu;
                const uint32_t Tlast = __shfl_sync(FULL, T, min(31, R - 1 - ibase));
                // every boundary whose bucket starts at or before the step's last element is settled here:
                // lane l owns boundary kc + 1 + l and counts the elements before its start time
                for (;;) {
                    const int kk = kc + 1 + lane;
                    const uint32_t av = kk <= nbk ? a[kk] : 0xffffffffu;
                    const bool mine = av <= Tlast;                // a prefix of the lanes: start times do not decrease
                    int pos = 0;
#pragma unroll
                    for (int step = 16; step > 0; step >>= 1) {
                        const uint32_t tm = __shfl_sync(FULL, T, pos + step - 1);
                        if (tm < av) pos += step;
                    }
                    if (mine) index_entry(tab, n, F.stiles, row, kk, ibase + pos);
                    const int done = __popc(__ballot_sync(FULL, mine));
                    kc += done;
                    if (done < 32) break;
                }
            }
        }
        // buckets that start after the row's last element
        for (int kk = kc + 1 + lane; kk <= nbk; kk += 32) index_entry(tab, n, F.stiles, row, kk, R);
    }
}

// Exclusive prefix sums of two values per thread over the block, in thread order, and both totals.
// tmp: 68 shared 64-bit words that no call since the block's last two barriers used (callers alternate two
// buffers, so the call ends without a barrier).  Every thread calls.
__device__ __forceinline__ void block_scan_add2(uint64_t x1, uint64_t x2, uint64_t &e1, uint64_t &e2, uint64_t &t1,
                                                uint64_t &t2, uint64_t *tmp) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    uint64_t i1 = x1, i2 = x2;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint64_t y1 = shfl_up(i1, d), y2 = shfl_up(i2, d);
        if (lane >= d) { i1 += y1; i2 += y2; }
    }
    if (lane == 31) { tmp[warp] = i1; tmp[34 + warp] = i2; }
    __syncthreads();
    if (warp == 0) {
        const uint64_t w1 = lane < nw ? tmp[lane] : 0ull, w2 = lane < nw ? tmp[34 + lane] : 0ull;
        uint64_t a1 = w1, a2 = w2;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint64_t y1 = shfl_up(a1, d), y2 = shfl_up(a2, d);
            if (lane >= d) { a1 += y1; a2 += y2; }
        }
        if (lane < nw) { tmp[lane] = a1 - w1; tmp[34 + lane] = a2 - w2; }
        if (lane == nw - 1) { tmp[32] = a1; tmp[34 + 32] = a2; }
    }
    __syncthreads();
    e1 = tmp[warp] + (i1 - x1);
    e2 = tmp[34 + warp] + (i2 - x2);
    t1 = tmp[32];
    t2 = tmp[34 + 32];
}

// Slot counters are read in per-thread runs of consecutive slots: one padding word per 32 keeps those
// reads free of bank conflicts.
__device__ __forceinline__ int slot_pad(int s) { return s + (s >> 5); }

struct SumShared {
    unsigned int fill;        // nodes gathered so far
    unsigned int nlong;       // long runs noted for the cooperative pass
    unsigned int carryC;      // rows that have an element before the bucket
    unsigned int pad;
    unsigned long long carryS;   // sum of those elements
};

constexpr int SUM_SHORT = 4;          // runs of up to this many elements are gathered by the row's own thread

// Dynamic shared memory: gathered nodes [scap] | nodes in time order [scap] (before the sort: the list of
// long runs) | slot counters [scap + scap / 32 + 1] | rank of each gathered node inside its slot [scap].
template <int OBJ>
__global__ void __launch_bounds__(1024) k_sum_buckets(const int64_t *ts, int n, int R, int B, int early_stop, InstMeta *meta, FilterBufs F,
                                                     int nres, SegResult *seg) {
    grid_dep_wait();
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ uint64_t tmpA[68], tmpB[68];
    __shared__ unsigned int sstatus;
    __shared__ InstMeta sM;
    __shared__ SumShared sh;
    const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
    const int cap = F.scap, nslots = max(32, cap / 2);
    Key<uint32_t> *in = (Key<uint32_t> *)smem, *out = in + cap;
    uint32_t *cnt = (uint32_t *)(out + cap);               // [slot_pad(nslots) + 1]: the last one closes the last slot
    uint16_t *rk = (uint16_t *)(cnt + slot_pad(cap) + 2);
    uint2 *longs = (uint2 *)out;                                  // (row | start << 16, end | position << 16)
    const BatchWS<uint32_t> ws{in, out, cnt, cap};
    const bool single = F.scells == 0;
    const int per = max(1, nslots / nt);
    const int s0 = min(tid * per, nslots), s1 = min(s0 + per, nslots);
    // work item: (instance, tile, part of the tile); with few tiles in the batch a tile's buckets are shared out over
    // ssub CTAs, each of which leaves a result of its own
    const int per_inst = F.stiles * F.ssub;
    for (int item = blockIdx.x; item < per_inst * B; item += gridDim.x) {
        const int b = item / per_inst, ts_ = item - b * per_inst, t = ts_ / F.ssub, sub = ts_ - t * F.ssub;
        __syncthreads();                                          // shared state of the previous item is done with
        if (tid == 0) { sM = meta[b]; sstatus = 0; }              // one read: another CTA may set `overflow` meanwhile
        __syncthreads();
        const InstMeta M = sM;
        if (M.status != ZL_OK || M.cscale == 0 || M.overflow || t >= (int)M.count2) continue;
        const int64_t *inst = ts + (size_t)b * n * R;
        const uint32_t tminlo = (uint32_t)(uint64_t)M.tmin - 1u;
        const uint16_t *tab = single ? nullptr : F.itab + ((size_t)b * F.stiles + t) * n * 16;
        const uint32_t *bnd = single ? nullptr : F.bnd + (size_t)b * ((size_t)F.stiles * TILE_BK + 1) + (size_t)t * TILE_BK;
        const int jt = min(TILE_BK, (int)M.count - t * TILE_BK);  // buckets of this tile
        const int jper = (TILE_BK + F.ssub - 1) / F.ssub;
        const int j0 = sub * jper, j1 = min(jt, j0 + jper);         // ... and of this part of it (may be none)
        uint64_t bd = ~0ull, bt = ~0ull;
        bool over = false;
        for (int j = j0; j < j1; ++j) {
            for (int s = tid; s <= slot_pad(nslots); s += nt) cnt[s] = 0;
            if (tid == 0) { sh.fill = 0; sh.nlong = 0; sh.carryC = 0; sh.carryS = 0; }
            // times of the bucket lie in [lo, hi): slot = ((T - lo) * scale) >> 32 < nslots, monotone in T
            // RANGE: once some row's last element has passed no later Z is complete, so nodes after lmin are left out
            const uint32_t tcut = OBJ == ZL_OBJ_RANGE && early_stop ? (uint32_t)M.lmin : 0xffffffffu;
            const uint32_t lo = single ? 1u : __ldg(bnd + j);
            const uint64_t hi = single ? min(M.tend, (uint64_t)tcut) + 1 : min((uint64_t)__ldg(bnd + j + 1), M.tend + 1);
            const uint32_t scale = (uint32_t)min((uint64_t)0xffffffffu, ((uint64_t)nslots << 32) / max((uint64_t)1, hi - (uint64_t)lo));
            __syncthreads();
            // K2 and the counting half of the sort.  A row's run [s, e) of the bucket: short runs are gathered
            // by the row's thread (one round of independent loads), long ones are noted for whole warps.
            uint64_t myS = 0;
            uint32_t myC = 0;
            for (int r = tid; r < n; r += nt) {
                const int s = single ? 0 : (int)__ldg(tab + (size_t)r * 16 + j);
                const int e = single ? R : (int)__ldg(tab + (size_t)r * 16 + j + 1);
                const int c = e - s;
                const int64_t *rp = inst + (size_t)r * R;
                uint32_t v[SUM_SHORT + 2];                        // predecessor, the run, and (RANGE) the element after it
                v[0] = s > 0 ? (uint32_t)(uint64_t)ldg64(rp + s - 1) - tminlo : 0u;
#pragma unroll
                for (int k = 0; k < SUM_SHORT; ++k) v[k + 1] = k < c && c <= SUM_SHORT ? (uint32_t)(uint64_t)ldg64(rp + s + k) - tminlo : 0u;
                v[SUM_SHORT + 1] = 0xffffffffu;
                if (OBJ == ZL_OBJ_RANGE && c > 0 && c <= SUM_SHORT && e < R) v[SUM_SHORT + 1] = (uint32_t)(uint64_t)ldg64(rp + e) - tminlo;
                if (s > 0) { myS += v[0]; ++myC; }
                if (c <= 0) continue;
                // SUM reserves the run's places in one step; RANGE appends node by node (it leaves nodes out)
                const uint32_t o_run = OBJ == ZL_OBJ_SUM ? atomicAdd(&sh.fill, (uint32_t)c) : 0u;
                if (o_run + (uint32_t)c > (uint32_t)cap) continue;   // the bucket does not fit: noticed below
                if (c <= SUM_SHORT) {
#pragma unroll
                    for (int k = 0; k < SUM_SHORT; ++k) {
                        if (k < c && v[k + 1] <= tcut) {
                            const uint32_t T = v[k + 1];
                            const uint32_t o = OBJ == ZL_OBJ_SUM ? o_run + (uint32_t)k : atomicAdd(&sh.fill, 1u);
                            // payload: SUM T minus the row's previous element, RANGE the row's next element
                            in[o] = Key<uint32_t>::make(T, OBJ == ZL_OBJ_SUM ? T - v[k] : k + 1 < c ? v[k + 2] : v[SUM_SHORT + 1]);
                            rk[o] = (uint16_t)atomicAdd(&cnt[slot_pad((int)min(__umulhi(T - lo, scale), (uint32_t)nslots - 1u))], 1u);
                        }
                    }
                } else {
                    longs[atomicAdd(&sh.nlong, 1u)] = make_uint2((uint32_t)r | ((uint32_t)s << 16), (uint32_t)e | (o_run << 16));
                }
            }
            myS = warp_reduce(myS, OpAdd());
            myC = warp_reduce(myC, OpAdd());
            if (lane == 0 && myC) { atomicAdd(&sh.carryS, (unsigned long long)myS); atomicAdd(&sh.carryC, myC); }
            __syncthreads();
            if (OBJ == ZL_OBJ_SUM && sh.fill > (uint32_t)cap) { over = true; break; }   // uniform over the block
            const int nlong = (int)sh.nlong;
            uint64_t cS = sh.carryS;
            uint32_t cC = sh.carryC;
            if (OBJ == ZL_OBJ_SUM && sh.fill == 0) continue;
            for (int w = warp; w < nlong; w += nw) {
                const uint2 d = longs[w];
                const int r = (int)(d.x & 0xffffu), s = (int)(d.x >> 16), e = (int)(d.y & 0xffffu);
                const uint32_t o = d.y >> 16;
                const int64_t *rp = inst + (size_t)r * R;
                if (OBJ == ZL_OBJ_SUM) {
                    for (int i = s + lane; i < e; i += 32) {
                        const uint32_t T = (uint32_t)(uint64_t)ldg64(rp + i) - tminlo;
                        const uint32_t pv = i > 0 ? (uint32_t)(uint64_t)ldg64(rp + i - 1) - tminlo : 0u;
                        const uint32_t pos = o + (uint32_t)(i - s);
                        in[pos] = Key<uint32_t>::make(T, T - pv);
                        rk[pos] = (uint16_t)atomicAdd(&cnt[slot_pad((int)min(__umulhi(T - lo, scale), (uint32_t)nslots - 1u))], 1u);
                    }
                } else {
                    for (int i0 = s; i0 < e; i0 += 32) {
                        const int i = i0 + lane;
                        const uint32_t T = i < e ? (uint32_t)(uint64_t)ldg64(rp + i) - tminlo : 0xffffffffu;
                        const uint32_t pay = i + 1 < R ? (uint32_t)(uint64_t)ldg64(rp + i + 1) - tminlo : 0xffffffffu;
                        // the row is sorted: the lanes that stay are a prefix of the warp
                        const unsigned keep = __ballot_sync(FULL, i < e && T <= tcut);
                        unsigned base = 0;
                        if (lane == 0 && keep) base = atomicAdd(&sh.fill, (unsigned)__popc(keep));
                        const uint32_t pos = __shfl_sync(FULL, base, 0) + (uint32_t)lane;
                        if (((keep >> lane) & 1u) && pos < (uint32_t)cap) {
                            in[pos] = Key<uint32_t>::make(T, pay);
                            rk[pos] = (uint16_t)atomicAdd(&cnt[slot_pad((int)min(__umulhi(T - lo, scale), (uint32_t)nslots - 1u))], 1u);
                        }
                        if (keep != FULL) break;                  // the rest of the row lies after the cut (or the run ends)
                    }
                }
            }
            __syncthreads();
            const uint32_t m = sh.fill;
            if (m > (uint32_t)cap) { over = true; break; }         // uniform over the block (cannot happen for a single bucket)
            if (m == 0) continue;
            // slot counts -> slot starts
            uint32_t loc = 0, big = 0;
            for (int s = s0; s < s1; ++s) { const uint32_t c = cnt[slot_pad(s)]; loc += c; big |= c > (uint32_t)SLOT_MAX; }
            uint32_t tot;
            uint32_t run = block_scan_excl<uint32_t>(loc, OpAdd(), 0u, (uint32_t *)tmpB, &tot);
            if (__syncthreads_or((int)big)) {
                // many equal or nearly equal times: the general batch routine (comparison network) takes the gathered nodes
                run_batch<uint32_t, OBJ>(ws, (int)m, (uint32_t)M.t0, n, tmpA, (uint32_t)0, cS, cC, bd, bt);
                continue;
            }
            for (int s = s0; s < s1; ++s) { const uint32_t c = cnt[slot_pad(s)]; cnt[slot_pad(s)] = run; run += c; }
            if (tid == 0) cnt[slot_pad(nslots)] = m;
            __syncthreads();
            // nodes grouped by slot ...
            for (uint32_t q = tid; q < m; q += nt) {
                const Key<uint32_t> k = in[q];
                out[cnt[slot_pad((int)min(__umulhi(k.t() - lo, scale), (uint32_t)nslots - 1u))] + rk[q]] = k;
            }
            __syncthreads();
            // ... then every node to its rank among the few nodes of its slot: `in` becomes the bucket in time order (K1)
            for (uint32_t q = tid; q < m; q += nt) {
                const Key<uint32_t> k = out[q];
                const int sl = (int)min(__umulhi(k.t() - lo, scale), (uint32_t)nslots - 1u);
                const uint32_t sb = cnt[slot_pad(sl)], se = cnt[slot_pad(sl + 1)];
                uint32_t rank = sb;
                for (uint32_t i = sb; i < se; ++i) { const uint64_t w = out[i].w; rank += w < k.w || (w == k.w && i < q); }
                in[rank] = k;
            }
            __syncthreads();
            // K3 (sums of delta and of the first flags, carry-in from the runs' predecessors) and K4
            const int ipt = (int)((m + nt - 1) / nt);
            const int k0 = min((uint32_t)(tid * ipt), m), k1 = min((uint32_t)(k0 + ipt), m);
            if (OBJ == ZL_OBJ_SUM) {
                uint64_t ls = 0, lc = 0;
                for (int k = k0; k < k1; ++k) { const Key<uint32_t> x = in[k]; ls += x.v(); lc += x.v() == x.t(); }
                uint64_t sS, sC, tS, tC;
                block_scan_add2(ls, lc, sS, sC, tS, tC, tmpA);
                sS += cS;
                uint32_t c = (uint32_t)sC + cC;
                for (int k = k0; k < k1; ++k) {
                    const uint32_t T = in[k].t(), dl = in[k].v();
                    sS += dl;                              // sum over started workers of their latest element
                    c += dl == T;                          // a first element carries delta == T (previous = 0)
                    if (c == (uint32_t)n) {
                        const uint64_t w = (uint64_t)n * (uint64_t)T - sS;
                        if (w < bd || (w == bd && (uint64_t)T < bt)) { bd = w; bt = T; }
                    }
                }
            } else {
                // RANGE (single-bucket instances only: nothing is carried in): prefix max of next, d = max(T, t0, PM) - T
                uint32_t lmax = 0;
                for (int k = k0; k < k1; ++k) lmax = max(lmax, in[k].v());
                uint32_t totm;
                uint32_t pm = block_scan_excl<uint32_t>(lmax, OpMax(), 0u, (uint32_t *)tmpA, &totm);
                const uint32_t t0 = (uint32_t)M.t0;
                for (int k = k0; k < k1; ++k) {
                    const uint32_t T = in[k].t();
                    const uint32_t g = max(max(T, t0), pm);   // max(Z) of the best Z whose minimum is this element
                    if (g != 0xffffffffu) {
                        const uint64_t d = (uint64_t)(g - T);
                        if (d < bd || (d == bd && (uint64_t)T < bt)) { bd = d; bt = T; }
                    }
                    pm = max(pm, in[k].v());
                }
            }
        }
        __syncthreads();
        if (over) {
            if (tid == 0) { meta[b].overflow = 1; F.flags[1] = 1; }
            continue;
        }
        block_best_to_result(bd, bt, ZL_OK, tmpA, &sstatus, seg[(size_t)b * nres + ts_]);
    }
}

// Index of the last element of a sorted row that is <= bar (-1 if none).  Rows are close to arithmetic, so the
// position is first guessed from the row's end points.  Eight probes around the guess, eight elements apart and
// loaded together, then the seven elements between the two probes that bracket bar, loaded together: three
// rounds of loads in the usual case.  A guess that is further off is bracketed by doubling steps and bisected.
template <class ROW>
__device__ int last_index_not_after(const ROW &row, int R, int64_t bar) {
    const int64_t e0 = row.at(0), eR = row.at(R - 1);
    if (bar < e0) return -1;
    if (bar >= eR) return R - 1;
    // e0 <= bar < eR, R >= 2.  Invariant: row[lo - 1] <= bar, row[hi] > bar
    int lo, hi;
    int g = (int)((double)(bar - e0) * (double)(R - 1) / (double)(eR - e0));
    g = max(0, min(g, R - 2));
    {
        constexpr int S = 8, P = 8;                       // probes at g + S * (k - P/2), clamped to the row
        int64_t pv[P];
        int pi[P];
#pragma unroll
        for (int k = 0; k < P; ++k) { pi[k] = max(0, min(R - 1, g + S * (k - P / 2))); pv[k] = row.at(pi[k]); }
        lo = 1; hi = R - 1;
#pragma unroll
        for (int k = 0; k < P; ++k) {
            if (pv[k] <= bar) lo = max(lo, pi[k] + 1); else hi = min(hi, pi[k]);
        }
        if (hi - lo <= S - 1) {                            // bracketed between two neighbouring probes
            int64_t wv[S - 1];
#pragma unroll
            for (int k = 0; k < S - 1; ++k) wv[k] = row.at(min(lo + k, R - 1));
            int c = 0;
#pragma unroll
            for (int k = 0; k < S - 1; ++k) c += (lo + k < hi && wv[k] <= bar) ? 1 : 0;   // sorted: a prefix of the window
            return lo + c - 1;
        }
    }
    // the probes did not enclose bar closely: doubling steps from the nearer end of the bracket, then bisection
    if (lo > 1) {                                          // everything probed was <= bar: search upwards from lo
        const int top = hi;
        for (int step = 16; lo < hi; step <<= 1) {
            const int q = min(lo + step - 1, top - 1);
            if (q < lo) break;
            if (row.at(q) <= bar) lo = q + 1; else { hi = q; break; }
        }
    } else {                                               // everything probed was > bar: search downwards from hi
        for (int step = 16; lo < hi; step <<= 1) {
            const int q = max(hi - step, lo);
            if (row.at(q) > bar) hi = q; else { lo = q + 1; break; }
        }
    }
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (row.at(mid) <= bar) lo = mid + 1; else hi = mid;
    }
    return lo - 1;
}

// Instances with few survivors of the filter pass are finished by one CTA.  It first applies the
// refinement at the resolution of the coarse cells, in shared memory (maximum of next per cell,
// exclusive prefix maximum, drop every survivor whose next does not exceed the value at its cell's
// start), then sorts what is left and sweeps it.  Dropped survivors never hold the running maximum
// alone, so nothing has to be carried in.
template <class SRC>
__global__ void __launch_bounds__(1024, 1) k_tail(const InstMeta *meta, FilterBufs F, int n, int nres, SegResult *seg, int tcap,
                                                  const SRC src, int R, int32_t *idx, int64_t *barrier, int64_t *wait, int32_t *status) {
    grid_dep_wait();
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ uint64_t tmp[34];
    __shared__ unsigned int sstatus, fill;
    const int b = blockIdx.x, tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
    const InstMeta M = meta[b];
    if (tid == 0) {
        // tell the later kernels of this call whether they have anything to do
        const bool mine = M.status == ZL_OK && handled_by_filter(M, 1) && tail_instance(M);
        if (M.status == ZL_OK && !handled_by_filter(M, 1)) F.flags[1] = 1;
        else if (M.status == ZL_OK && !tail_instance(M)) F.flags[0] = 1;
        if (!mine) F.flags[2] = 1;                                 // k_finalize has to write this instance's outputs
    }
    if (M.status != ZL_OK || !handled_by_filter(M, 1) || !tail_instance(M)) return;
    uint32_t *g = (uint32_t *)smem;                               // [cells]
    Key<uint32_t> *keys = (Key<uint32_t> *)(smem + (size_t)F.cells * 4);
    const BatchWS<uint32_t> ws{keys, keys + tcap, (uint32_t *)(keys + 2 * (size_t)tcap), tcap};
    const int cells = F.cells;
    for (int c = tid; c < cells; c += nt) g[c] = 0;
    if (tid == 0) { sstatus = 0; fill = 0; }
    __syncthreads();
    for (int r = warp; r < F.nreg; r += nw) {
        const uint32_t c = F.rcnt[(size_t)b * F.nreg + r];
        const uint64_t *src = F.list1 + (size_t)b * F.list1cap + (size_t)r * F.regcap;
        for (uint32_t i = lane; i < c; i += 32) {
            const uint64_t w = src[i];
            atomicMax(&g[cell_of((uint32_t)(w >> 32), M.cscale)], (uint32_t)w);
        }
    }
    __syncthreads();
    {   // exclusive prefix maximum over the cells, floored by t0
        const int per = (cells + nt - 1) / nt;
        const int c0 = min(tid * per, cells), c1 = min(c0 + per, cells);
        uint32_t loc = 0;
        for (int c = c0; c < c1; ++c) loc = max(loc, g[c]);
        uint32_t tot;
        uint32_t run = max(block_scan_excl<uint32_t>(loc, OpMax(), 0u, (uint32_t *)tmp, &tot), (uint32_t)M.t0);
        for (int c = c0; c < c1; ++c) { const uint32_t v = g[c]; g[c] = run; run = max(run, v); }
    }
    __syncthreads();
    for (int r = warp; r < F.nreg; r += nw) {
        const uint32_t c = F.rcnt[(size_t)b * F.nreg + r];
        const uint64_t *src = F.list1 + (size_t)b * F.list1cap + (size_t)r * F.regcap;
        for (uint32_t i0 = 0; i0 < c; i0 += 32) {
            const uint32_t i = i0 + lane;
            const uint64_t w = i < c ? src[i] : 0ull;
            const uint32_t T = (uint32_t)(w >> 32), nx = (uint32_t)w;
            const bool keep = i < c && nx > max(T, g[cell_of(T, M.cscale)]);
            const unsigned km = __ballot_sync(FULL, keep);
            if (km == 0) continue;
            unsigned base = 0;
            if (lane == 0) base = atomicAdd(&fill, (unsigned)__popc(km));
            base = __shfl_sync(FULL, base, 0);
            if (keep) keys[base + __popc(km & ((1u << lane) - 1u))].w = w;
        }
    }
    __syncthreads();
    uint64_t bd = ~0ull, bt = ~0ull, cs = 0;
    uint32_t cc = 0;
    run_batch<uint32_t, ZL_OBJ_RANGE>(ws, (int)fill, (uint32_t)M.t0, n, tmp, (uint32_t)0, cs, cc, bd, bt);
    __shared__ SegResult best;
    block_best_to_result(bd, bt, ZL_OK, tmp, &sstatus, best);
    __syncthreads();
    // K5 for this instance right here: barrier, wait and the per-worker indices (k_finalize skips it)
    const int fst = best.valid ? ZL_OK : ZL_ERR_TIMEOUT;          // a valid instance always has a candidate
    const int64_t bar = fst == ZL_OK ? M.tmin + (int64_t)(best.t - 1) + (int64_t)best.d : INT64_MIN;
    if (tid == 0) {
        seg[(size_t)b * nres] = best;
        wait[b] = fst == ZL_OK ? (int64_t)best.d : INT64_MIN;
        barrier[b] = bar;
        if (status) status[b] = fst;
    }
    for (int p = tid; p < n; p += nt)
        idx[(size_t)b * n + p] = fst == ZL_OK ? last_index_not_after(src.inst(b, n, R).row(p), R, bar) : -1;
}

// ------------------------------------------------------------------------------ finalize
// grid (row blocks, B): every CTA reduces the instance's partial results, then recovers the indices of
// its block of rows; the CTA of row block 0 also writes wait, barrier and status.
template <class SRC>
__global__ void __launch_bounds__(256) k_finalize(const SRC src, int n, int R, int nseg, FilterBufs F, int nres,
                                                  int objective, int filter, const InstMeta *meta, const SegResult *seg,
                                                  int32_t *idx, int64_t *barrier, int64_t *wait, int32_t *status) {
    grid_dep_wait();
    const int b = blockIdx.y, tid = threadIdx.x;
    // filter: 0 only the segment sweep ran, 1 the RANGE filter route, 2 the bucket route
    if (filter && F.flags[2] == 0) return;                        // k_tail finished every instance of this call
    const InstMeta M = meta[b];
    if (filter == 1 && M.status == ZL_OK && handled_by_filter(M, filter) && tail_instance(M)) return;   // finished by k_tail
    __shared__ uint64_t red[34];
    __shared__ unsigned int sstatus;
    __shared__ SegResult best;
    if (tid == 0) sstatus = 0;
    __syncthreads();
    uint64_t bd = ~0ull, bt = ~0ull;
    uint32_t st = M.status;
    if (st == ZL_OK) {
        const int used = !handled_by_filter(M, filter) ? nseg
                         : filter == 2 ? (int)M.count2 * F.ssub                         // bucket route: one result per part of a tile
                         : tail_instance(M) ? 1 : (F.nbk + bucket_group(F, M.count2) - 1) / bucket_group(F, M.count2);
        for (int s = tid; s < used; s += blockDim.x) {
            const SegResult r = seg[(size_t)b * nres + s];
            if (r.status != ZL_OK) st = max(st, (uint32_t)r.status);
            if (r.valid && (r.d < bd || (r.d == bd && r.t < bt))) { bd = r.d; bt = r.t; }
        }
    }
    block_best_to_result(bd, bt, st, red, &sstatus, best);
    __syncthreads();
    int fst = (int)best.status;
    if (fst == ZL_OK && !best.valid) fst = ZL_ERR_TIMEOUT;         // cannot happen for valid input
    int64_t bar = INT64_MIN, wt = INT64_MIN;
    if (fst == ZL_OK) {
        const int64_t tm = M.tmin + (int64_t)(best.t - 1);
        bar = objective == ZL_OBJ_RANGE ? tm + (int64_t)best.d : tm;
        wt = (int64_t)best.d;
    }
    if (blockIdx.x == 0 && tid == 0) {
        wait[b] = wt;
        barrier[b] = bar;
        if (status) status[b] = fst;
    }
    // one thread per row: the number of elements <= barrier.  Rows are close to arithmetic, so the position is
    // first guessed from the row's end points, bracketed by doubling steps around the guess, then bisected.
    const int p = blockIdx.x * blockDim.x + tid;
    if (p < n) {
        int res = -1;
        if (fst == ZL_OK) {
            res = last_index_not_after(src.inst(b, n, R).row(p), R, bar);
        }
        idx[(size_t)b * n + p] = res;
    }
}

// ------------------------------------------------------------------------------ GridScan / FullGridScan
// Value of the point of a sorted row at the shortest distance from e (the earlier one on ties).
__device__ __forceinline__ int64_t nearest_value(const int64_t *row, int R, int64_t e) {
    int lo = 0, hi = R;                           // first index with row[i] >= e
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (ldg64(row + mid) < e) lo = mid + 1; else hi = mid;
    }
    if (lo == 0) return ldg64(row);
    const int64_t left = ldg64(row + lo - 1);
    if (lo == R) return left;
    const int64_t right = ldg64(row + lo);
    return e - left <= right - e ? left : right;
}

// Lowest index of a sorted row that holds value v (v occurs in the row).
__device__ __forceinline__ int first_index_of(const int64_t *row, int R, int64_t v) {
    int lo = 0, hi = R;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (ldg64(row + mid) < v) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// Row with the earliest first timestamp (lowest-numbered on ties); every thread of the block gets it.
__device__ int designated_row(const int64_t *inst, int n, int R, uint64_t *tmp) {
    uint64_t best = ~0ull;                         // (first timestamp, row) packed: timestamps are below 2^62
    uint64_t bestp = 0;
    for (int p = threadIdx.x; p < n; p += blockDim.x) {
        const uint64_t v = (uint64_t)ldg64(inst + (size_t)p * R);
        if (v < best) { best = v; bestp = (uint64_t)p; }
    }
    uint64_t tot;
    block_scan_excl<uint64_t>(best, OpMin(), ~0ull, tmp, &tot);
    uint64_t cand = best == tot ? bestp : ~0ull, totp;
    block_scan_excl<uint64_t>(cand, OpMin(), ~0ull, tmp, &totp);
    return (int)totp;
}

// d_Z of one candidate per CTA.  grid (candidates, B); candidate c = designated point (row c / R, index c % R)
// when full, else point c of the designated row.
__global__ void __launch_bounds__(256) k_gridscan_eval(const int64_t *ts, int n, int R, int full, int64_t *cand) {
    __shared__ uint64_t tmp[34];
    const int b = blockIdx.y, c = blockIdx.x;
    const int64_t *inst = ts + (size_t)b * n * R;
    const int q = full ? c / R : designated_row(inst, n, R, tmp);
    const int j = full ? c % R : c;
    const int64_t e = ldg64(inst + (size_t)q * R + j);
    uint64_t mx = (uint64_t)e, mn = (uint64_t)e;
    for (int p = threadIdx.x; p < n; p += blockDim.x) {
        if (p == q) continue;
        const uint64_t v = (uint64_t)nearest_value(inst + (size_t)p * R, R, e);
        mx = max(mx, v); mn = min(mn, v);
    }
    uint64_t gmx, gmn;
    block_scan_excl<uint64_t>(mx, OpMax(), 0ull, tmp, &gmx);
    block_scan_excl<uint64_t>(mn, OpMin(), ~0ull, tmp, &gmn);
    if (threadIdx.x == 0) cand[(size_t)b * gridDim.x + c] = (int64_t)(gmx - gmn);
}

// First minimal candidate of an instance, then its Z*.  grid B
__global__ void __launch_bounds__(256) k_gridscan_pick(const int64_t *ts, int n, int R, int full, int ncand, const int64_t *cand,
                                                       int32_t *idx, int64_t *barrier, int64_t *wait) {
    __shared__ uint64_t tmp[34];
    const int b = blockIdx.x;
    const int64_t *inst = ts + (size_t)b * n * R;
    uint64_t bd = ~0ull, bc = ~0ull;
    for (int c = threadIdx.x; c < ncand; c += blockDim.x) {
        const uint64_t d = (uint64_t)cand[(size_t)b * ncand + c];
        if (d < bd) { bd = d; bc = (uint64_t)c; }                 // a thread sees its candidates in ascending order
    }
    uint64_t gd, gc;
    block_scan_excl<uint64_t>(bd, OpMin(), ~0ull, tmp, &gd);
    block_scan_excl<uint64_t>(bd == gd ? bc : ~0ull, OpMin(), ~0ull, tmp, &gc);
    const int c = (int)gc;
    const int q = full ? c / R : designated_row(inst, n, R, tmp);
    const int j = full ? c % R : c;
    const int64_t e = ldg64(inst + (size_t)q * R + j);
    uint64_t mx = (uint64_t)e;
    for (int p = threadIdx.x; p < n; p += blockDim.x) {
        int res = j;
        if (p != q) {
            const int64_t v = nearest_value(inst + (size_t)p * R, R, e);
            res = first_index_of(inst + (size_t)p * R, R, v);
            mx = max(mx, (uint64_t)v);
        }
        idx[(size_t)b * n + p] = res;
    }
    uint64_t gmx;
    block_scan_excl<uint64_t>(mx, OpMax(), 0ull, tmp, &gmx);
    if (threadIdx.x == 0) { barrier[b] = (int64_t)gmx; wait[b] = (int64_t)gd; }
}

// ------------------------------------------------------------------------------ predictor
// One CTA per row: e_i = last + i * interval, i = 1..R, written with 16-byte stores where the row allows.
__global__ void __launch_bounds__(256) k_predict(const int64_t *last, const int64_t *interval, int R, int64_t *ts) {
    const size_t row = blockIdx.x;
    const int64_t l = ldg64(last + row), iv = ldg64(interval + row);
    int64_t *out = ts + row * (size_t)R;
    int64_t base = l, step = iv;
    if (l < 0 || iv < 0) { base = -1; step = 0; }                 // marks the instance invalid for the search
    else if (__umul64hi((uint64_t)R, (uint64_t)iv) != 0 || (uint64_t)R * (uint64_t)iv >= (uint64_t)VALUE_LIMIT ||
             (uint64_t)l + (uint64_t)R * (uint64_t)iv >= (uint64_t)VALUE_LIMIT) { base = VALUE_LIMIT; step = 0; }
    if ((R & 1) == 0 && (((uintptr_t)out) & 15) == 0) {
        for (int i = 2 * threadIdx.x; i < R; i += 2 * blockDim.x) {
            longlong2 v;
            v.x = base + (int64_t)(i + 1) * step;
            v.y = base + (int64_t)(i + 2) * step;
            *reinterpret_cast<longlong2 *>(out + i) = v;
        }
    } else {
        for (int i = threadIdx.x; i < R; i += blockDim.x) out[i] = base + (int64_t)(i + 1) * step;
    }
}

// ------------------------------------------------------------------------------ read probe
// Measurement aid: nothing but the loads of a row-prefix pass.  A warp per row reads the first count[row]
// timestamps of the row with 16-byte loads (8-byte loads for odd lengths or a misaligned base), 256 a round,
// and folds them into a checksum so that the loads cannot be dropped.  Timed beside k_filter it shows what the
// memory system delivers for the same bytes in the same access pattern.
__global__ void __launch_bounds__(128) k_probe_read(const int64_t *ts, const int32_t *count, long long rows, int R,
                                                  unsigned long long *sink) {
    const int lane = threadIdx.x & 31;
    const long long row = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (row >= rows) return;
    const int64_t *rp = ts + (size_t)row * R;
    const int L = max(0, min(R, __ldg(count + row)));
    const bool vec2 = (R % 2 == 0) && (((uintptr_t)ts & 15) == 0);
    unsigned long long acc = 0;
    for (int base = 0; base < L; base += 256) {
        if (vec2) {
            longlong2 v[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int i = base + 64 * k + 2 * lane;
                v[k] = i < L ? *reinterpret_cast<const longlong2 *>(rp + i) : make_longlong2(0, 0);
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) acc += (unsigned long long)(v[k].x ^ v[k].y);
        } else {
            int64_t v[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) { const int i = base + 32 * k + lane; v[k] = i < L ? ldg64(rp + i) : 0; }
#pragma unroll
            for (int k = 0; k < 8; ++k) acc += (unsigned long long)v[k];
        }
    }
    if (acc == 0x5eedf00dull) atomicAdd(sink, acc);               // practically never: keeps the loads alive
}

// ------------------------------------------------------------------------------ trace
struct TKey {
    uint64_t t; uint32_t f, pad;
    __device__ __forceinline__ bool operator>(const TKey &o) const { return t > o.t || (t == o.t && f > o.f); }
};

__global__ void __launch_bounds__(256) k_trace(const int64_t *ts, int n, int R,
                                               int64_t *om_t, int32_t *om_p, int32_t *om_i, int64_t *delta,
                                               int32_t *first, int64_t *S, int32_t *cnt, int64_t *next,
                                               int64_t *PM, int64_t *d_range, int64_t *w_sum) {
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ uint64_t tmp[34];
    TKey *keys = (TKey *)smem;
    const int N = n * R, b = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
    const int64_t *inst = ts + (size_t)b * N;
    int P = 64;
    while (P < N) P <<= 1;
    // step 1: merge = all (time, worker, iteration) in ascending order
    int64_t t0loc = INT64_MIN;
    for (int f = tid; f < P; f += nt) {
        TKey k;
        if (f < N) { k.t = (uint64_t)ldg64(inst + f); k.f = (uint32_t)f; if (f % R == 0) t0loc = max(t0loc, (int64_t)k.t); }
        else { k.t = ~0ull; k.f = 0xffffffffu; }
        k.pad = 0;
        keys[f] = k;
    }
    uint64_t t0u = warp_reduce((uint64_t)t0loc ^ (1ull << 63), OpMax());
    __shared__ unsigned long long s_t0;
    if (tid == 0) s_t0 = 0;
    __syncthreads();
    if ((tid & 31) == 0) atomicMax(&s_t0, (unsigned long long)t0u);
    __syncthreads();
    const int64_t t0 = (int64_t)(s_t0 ^ (1ull << 63));
    bitonic_sort(keys, P);
    const int ipt = (P + nt - 1) / nt;
    const int k0 = tid * ipt, k1 = min(k0 + ipt, N);
    // steps 2+3: per-element delta / flag / next, then the scans in Omega order
    uint64_t ls = 0, lm = 0;            // lm: max of next, order-preserving unsigned image of int64
    uint32_t lc = 0;
    for (int k = k0; k < k1; ++k) {
        const int f = (int)keys[k].f, i = f % R;
        const int64_t t = (int64_t)keys[k].t;
        ls += (uint64_t)(i == 0 ? t : t - ldg64(inst + f - 1));
        lc += i == 0;
        const int64_t nx = i == R - 1 ? INT64_MAX : ldg64(inst + f + 1);
        lm = max(lm, (uint64_t)((uint64_t)nx ^ (1ull << 63)));
    }
    uint64_t tots, totm;
    uint32_t totc;
    uint64_t s = block_scan_excl<uint64_t>(ls, OpAdd(), 0ull, tmp, &tots);
    uint32_t c = block_scan_excl<uint32_t>(lc, OpAdd(), 0u, (uint32_t *)tmp, &totc);
    uint64_t pmu = block_scan_excl<uint64_t>(lm, OpMax(), 0ull, tmp, &totm);   // 0 is the image of INT64_MIN
    for (int k = k0; k < k1; ++k) {
        const int f = (int)keys[k].f, p = f / R, i = f % R;
        const int64_t t = (int64_t)keys[k].t;
        const int64_t dl = i == 0 ? t : t - ldg64(inst + f - 1);
        const int64_t nx = i == R - 1 ? INT64_MAX : ldg64(inst + f + 1);
        s += (uint64_t)dl;
        c += i == 0;
        const int64_t pm = (int64_t)(pmu ^ (1ull << 63));
        const size_t o = (size_t)b * N + k;
        if (om_t) om_t[o] = t;
        if (om_p) om_p[o] = p;
        if (om_i) om_i[o] = i;
        if (delta) delta[o] = dl;
        if (first) first[o] = i == 0;
        if (S) S[o] = (int64_t)s;
        if (cnt) cnt[o] = (int32_t)c;
        if (next) next[o] = nx;
        if (PM) PM[o] = pm;
        // step 4: objective of the candidate at this position
        if (d_range) { const int64_t g = max(max(t, t0), pm); d_range[o] = g == INT64_MAX ? INT64_MAX : g - t; }
        if (w_sum) w_sum[o] = c == (uint32_t)n ? (int64_t)((uint64_t)n * (uint64_t)t - s) : INT64_MAX;
        pmu = max(pmu, (uint64_t)((uint64_t)nx ^ (1ull << 63)));
    }
}

}  // namespace zl

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
    int opt_threads, opt_lanes, opt_segments, opt_round_factor, opt_no_filter, opt_filter_threads, opt_filter_rows, opt_pdl_off, opt_prologue_threads, opt_tail_threads, opt_filter_round;
    int last_cuda_error;
    int launches;
    // optional per-kernel timing: PROF_EVENTS events per recorded call
    cudaEvent_t *prof_ev;
    int prof_cap, prof_calls;
};

namespace {

int pow2_floor(int x) { int p = 1; while (p * 2 <= x) p *= 2; return p; }
int pow2_ceil(int x) { int p = 1; while (p < x) p *= 2; return p; }

struct LaunchPlan { int threads, G, nseg, cap, target; size_t smem; };
constexpr int PROF_EVENTS = 5;

// Everything one call enqueues, for both the handle-based and the fixed-scratch entry points.
struct Pipeline {
    const int64_t *ts; int B, n, R, objective, flags, num_sms;
    zl::InstMeta *meta; zl::SegResult *seg; int nres;
    zl::FilterBufs fb;                                            // fb.table == nullptr: no filter route
    int filter_threads, filter_rows, filter_round;                // 0: automatic
    int pdl_off;                                                  // bit mask of kernels launched without early scheduling
    int prologue_threads, tail_threads;                           // 0: automatic
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

// SRC: zl::MatBatch (the rows are read from q.ts) or zl::AriBatch (predicted rows, generated on the fly; RANGE, filter
// route or plain segment sweep only).
template <class SRC>
void enqueue(const Pipeline &q, const LaunchPlan &p, cudaStream_t st, cudaEvent_t *ev, const SRC src) {
    constexpr bool arith = std::is_same<SRC, zl::AriBatch>::value;
    const bool filter = q.fb.table != nullptr && q.objective == ZL_OBJ_RANGE;
    // the bucket route: every SUM shape it supports, and RANGE instances small enough to be a single bucket
    const bool sumfast = !arith && q.fb.flags != nullptr && q.fb.scap != 0 && (q.objective == ZL_OBJ_SUM || q.fb.table == nullptr);
    zl::FilterBufs fb = q.fb;
    if (!filter && !sumfast) memset(&fb, 0, sizeof(fb));
    if (ev) cudaEventRecord(ev[0], st);
    // many small instances: small CTAs so that several share an SM; few large ones: one large CTA each
    const bool many = q.B > 2 * q.num_sms;
    const int pthreads = q.prologue_threads ? q.prologue_threads
                         : many ? std::max(128, std::min(256, pow2_ceil(2 * q.n))) : std::max(512, std::min(1024, pow2_ceil(q.n)));
    // the first kernel of a call is scheduled early too: it waits (grid_dep_wait) for whatever precedes it in the stream
    launch_dep(!((q.pdl_off >> 9) & 1), zl::k_prologue<SRC>, dim3(q.B), dim3(pthreads), (size_t)q.n * 16, st, src, q.n, q.R, q.objective, q.flags, q.meta, fb);
    if (!arith && (q.flags & ZL_FLAG_CHECK_SORTED)) {
        const size_t total = (size_t)q.B * q.n * q.R;
        const int blocks = (int)std::min<size_t>((total + 255) / 256, (size_t)q.num_sms * 16);
        launch_dep(!((q.pdl_off >> 0) & 1), zl::k_check_sorted, dim3(blocks), dim3(256), 0, st, q.ts, q.n, q.R, total, q.meta);
    }
    if (ev) cudaEventRecord(ev[1], st);
    if (filter) {
        int threads = std::max(64, std::min(256, 32 * pow2_ceil(std::min(q.n, 32))));
        if (q.filter_threads) threads = std::max(64, std::min(q.filter_threads, 32 * pow2_ceil(std::min(q.n, 32))));
        const int nw = threads / 32;
        long long rpc = ((long long)q.n * q.B / (16LL * q.num_sms) + nw - 1) / nw * nw;
        if (q.filter_rows) rpc = ((long long)q.filter_rows + nw - 1) / nw * nw;
        rpc = std::max<long long>(nw, std::min<long long>(rpc, (q.n + nw - 1) / nw * nw));
        fb.nreg = (int)((q.n + rpc - 1) / rpc);
        fb.regcap = fb.list1cap / fb.nreg;
        const size_t fsmem = (size_t)fb.cells * 4 + (size_t)nw * zl::FILTER_STAGES * zl::FILTER_SLOT * 8;
        if constexpr (arith)
            launch_dep(!((q.pdl_off >> 1) & 1), zl::k_filter_arith, dim3(fb.nreg, q.B), dim3(threads), (size_t)fb.cells * 4, st, src, q.n, q.R, (int)rpc, q.meta, fb);
        else
            launch_dep(!((q.pdl_off >> 1) & 1), zl::k_filter, dim3(fb.nreg, q.B), dim3(threads), fsmem, st, q.ts, q.n, q.R, q.flags, (int)rpc, q.filter_round ? q.filter_round : 8, q.meta, fb);
        if (ev) cudaEventRecord(ev[2], st);
        const int tcap = (int)std::min<long long>((long long)zl::TAIL_CAP, pow2_ceil(std::max(64, fb.list1cap)));
        launch_dep(!((q.pdl_off >> 2) & 1), zl::k_tail<SRC>, dim3(q.B), dim3(q.tail_threads ? q.tail_threads : many ? (tcap <= 1024 ? 128 : 256) : std::max(64, std::min(1024, tcap / 2))), (size_t)tcap * 20 + (size_t)fb.cells * 4, st,
                   (const zl::InstMeta *)q.meta, fb, q.n, q.nres, q.seg, tcap, src, q.R, q.idx, q.barrier, q.wait, q.status);
        // the route for instances with many survivors: fixed-size grids that return at once when no instance needs them
        const int tiles = (fb.fcells + zl::SCAN_TILE - 1) / zl::SCAN_TILE;
        const int wide = 4 * q.num_sms;
        launch_dep(!((q.pdl_off >> 3) & 1), zl::k_tilemax, dim3(std::min(tiles * q.B, wide)), dim3(256), 0, st, (const zl::InstMeta *)q.meta, fb, q.B);
        launch_dep(!((q.pdl_off >> 4) & 1), zl::k_cellscan, dim3(std::min(tiles * q.B, wide)), dim3(256), 0, st, (const zl::InstMeta *)q.meta, fb, q.B);
        launch_dep(!((q.pdl_off >> 5) & 1), zl::k_refine, dim3(std::min(fb.nreg * q.B, 8 * wide)), dim3(256), 0, st, q.meta, fb, q.B);
        const int ngroups = (fb.nbk + fb.grp - 1) / fb.grp;
        const int bthreads = std::max(64, std::min(256, fb.capb / 4));
        launch_dep(!((q.pdl_off >> 6) & 1), zl::k_buckets, dim3(std::min(ngroups * q.B, wide)), dim3(bthreads), (size_t)fb.capb * 20, st,
                   (const zl::InstMeta *)q.meta, fb, q.n, q.nres, q.seg, q.B);
    } else if (sumfast) {
        const bool single = fb.scells == 0;
        const size_t nb1 = (size_t)fb.stiles * zl::TILE_BK + 1;
        launch_dep(!((q.pdl_off >> 1) & 1), zl::k_sum_plan, dim3(q.B), dim3(single ? 32 : 1024), single ? 0 : ((size_t)fb.scells + 1) * 8 + nb1 * 4, st,
                   q.ts, q.n, q.R, q.meta, fb);
        if (!single) {
            const int nw = 8;
            const int row_blocks = std::max(1, std::min((q.n + nw - 1) / nw, (32 * q.num_sms + q.B - 1) / q.B));
            launch_dep(!((q.pdl_off >> 2) & 1), zl::k_sum_index, dim3(row_blocks, q.B), dim3(32 * nw), nb1 * 4, st, q.ts, q.n, q.R,
                       (const zl::InstMeta *)q.meta, fb);
        }
        if (ev) cudaEventRecord(ev[2], st);
        const long long N = (long long)q.n * q.R;
        int bthreads = single ? (int)std::max<long long>(64, std::min<long long>(1024, pow2_ceil((int)((N + 7) / 8))))
                              : (fb.scap > 4096 ? 1024 : 512);
        if (q.tail_threads) bthreads = q.tail_threads;
        // few tiles in the batch: share each tile's buckets out over several CTAs
        fb.ssub = single ? 1 : std::max(1, std::min(zl::TILE_BK, (2 * q.num_sms) / std::max(1, fb.stiles * q.B)));
        const int items = fb.stiles * fb.ssub * q.B;
        const size_t bsmem = (size_t)fb.scap * 18 + ((size_t)fb.scap + fb.scap / 32 + 2) * 4;
        if (q.objective == ZL_OBJ_SUM)
            launch_dep(!((q.pdl_off >> 3) & 1), zl::k_sum_buckets<ZL_OBJ_SUM>, dim3(std::min(items, 32 * q.num_sms)), dim3(bthreads), bsmem, st,
                       q.ts, q.n, q.R, q.B, 0, q.meta, fb, q.nres, q.seg);
        else
            launch_dep(!((q.pdl_off >> 3) & 1), zl::k_sum_buckets<ZL_OBJ_RANGE>, dim3(std::min(items, 32 * q.num_sms)), dim3(bthreads), bsmem, st,
                       q.ts, q.n, q.R, q.B, (q.flags & ZL_FLAG_FULL_SWEEP) ? 0 : 1, q.meta, fb, q.nres, q.seg);
    } else if (ev) {
        cudaEventRecord(ev[2], st);
    }
    zl::SweepParams sp;
    sp.ts = q.ts; sp.meta = q.meta; sp.seg = q.seg;
    sp.n = q.n; sp.R = q.R; sp.B = q.B; sp.nseg = p.nseg; sp.nres = q.nres; sp.G = p.G; sp.cap = p.cap;
    const bool fast = filter || sumfast;
    sp.flags = q.flags; sp.target = p.target; sp.filter = fast ? 1 : 0;
    sp.need = fast ? fb.flags : nullptr;
    // with a fast route on, the segment sweep is only the fallback: a small persistent grid
    const int items = p.nseg * q.B;
    const int sweep_ctas = fast ? std::min(items, 2 * q.num_sms) : items;
    if (q.objective == ZL_OBJ_RANGE) launch_dep(!((q.pdl_off >> 7) & 1), zl::k_sweep<ZL_OBJ_RANGE, SRC>, dim3(sweep_ctas), dim3(p.threads), p.smem, st, sp, src);
    else launch_dep(!((q.pdl_off >> 7) & 1), zl::k_sweep<ZL_OBJ_SUM, SRC>, dim3(sweep_ctas), dim3(p.threads), p.smem, st, sp, src);
    if (ev) cudaEventRecord(ev[3], st);
    const int fthreads = std::max(32, std::min(256, pow2_ceil(q.n)));
    launch_dep(!((q.pdl_off >> 8) & 1), zl::k_finalize<SRC>, dim3((q.n + fthreads - 1) / fthreads, q.B), dim3(fthreads), 0, st, src, q.n, q.R, p.nseg, fb, q.nres, q.objective,
                                                                  filter ? 1 : sumfast ? 2 : 0, q.meta, q.seg, q.idx, q.barrier, q.wait, q.status);
    if (ev) cudaEventRecord(ev[4], st);
}

cudaError_t raise_shared_memory_limits() {
    cudaError_t e = cudaFuncSetAttribute(zl::k_sweep<ZL_OBJ_RANGE, zl::MatBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(zl::k_sweep<ZL_OBJ_SUM, zl::MatBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(zl::k_sweep<ZL_OBJ_RANGE, zl::AriBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(zl::k_sweep<ZL_OBJ_SUM, zl::AriBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(zl::k_buckets, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(zl::k_filter, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(zl::k_tail<zl::MatBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(zl::k_tail<zl::AriBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(zl::k_prologue<zl::MatBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, zl::MAX_WORKERS * 16);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(zl::k_prologue<zl::AriBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, zl::MAX_WORKERS * 16);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(zl::k_sum_buckets<ZL_OBJ_SUM>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(zl::k_sum_buckets<ZL_OBJ_RANGE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(zl::k_sum_plan, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
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
    return p;
}

zl_status cuda_fail(zl_handle *h, cudaError_t e) {
    if (h) h->last_cuda_error = (int)e;
    return e == cudaErrorMemoryAllocation ? ZL_ERR_NOMEM : ZL_ERR_CUDA;
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
int32_t zl_trace_max_elements(void) { return zl::TRACE_MAX; }

zl_status zl_create(const zl_config *cfg, zl_handle **out) {
    if (!cfg || !out) return ZL_ERR_INVALID_ARG;
    *out = nullptr;
    if (cfg->n_workers < 1 || cfg->lookahead_R < 1 || cfg->max_batch < 1) return ZL_ERR_INVALID_ARG;
    if (cfg->objective != ZL_OBJ_RANGE && cfg->objective != ZL_OBJ_SUM) return ZL_ERR_INVALID_ARG;
    if (cfg->flags & ~(ZL_FLAG_CHECK_SORTED | ZL_FLAG_FULL_SWEEP | ZL_FLAG_PREDICTOR)) return ZL_ERR_INVALID_ARG;
    if (cfg->n_workers > zl::MAX_WORKERS) return ZL_ERR_UNSUPPORTED;
    if ((long long)cfg->n_workers * cfg->lookahead_R > (1LL << 31) - 1) return ZL_ERR_UNSUPPORTED;
    if (cfg->max_batch > 65535) return ZL_ERR_UNSUPPORTED;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || cfg->device < 0 || cfg->device >= ndev) return ZL_ERR_CUDA;
    zl_handle *h = new (std::nothrow) zl_handle();
    if (!h) return ZL_ERR_NOMEM;
    memset(h, 0, sizeof(*h));
    h->cfg = *cfg;
    cudaError_t e = cudaSetDevice(cfg->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->num_sms, cudaDevAttrMultiProcessorCount, cfg->device);
    const size_t meta_b = (size_t)cfg->max_batch * sizeof(zl::InstMeta);
    size_t filter_b = 0;
    h->nres = zl::MAX_SEGMENTS;
    // RANGE instances that fit one shared-memory batch are sorted whole by the bucket route; larger ones take the filter route
    const bool range_small = cfg->objective == ZL_OBJ_RANGE && (long long)cfg->n_workers * cfg->lookahead_R <= 4096;
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
        const size_t sizes[9] = {mb * f.cells * 4, mb * cfg->n_workers * 4, mb * f.fcells * 4, mb * cfg->n_workers * 4,
                                 mb * (size_t)f.list1cap * 8, mb * f.nbk * 4, mb * f.nbk * f.capb * 8, mb * tiles * 4, 64};
        void **ptrs[9] = {(void **)&f.table, (void **)&f.rowhint, (void **)&f.cellmax, (void **)&f.rcnt,
                          (void **)&f.list1, (void **)&f.bcnt, (void **)&f.list2, (void **)&f.tilemax, (void **)&f.flags};
        for (int i = 0; i < 9; ++i) {
            if (e == cudaSuccess) e = cudaMalloc(ptrs[i], sizes[i]);
            filter_b += sizes[i];
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
                if (e == cudaSuccess) e = cudaMalloc(ptrs[i], sizes[i]);
                filter_b += sizes[i];
            }
            h->nres = std::max(zl::MAX_SEGMENTS, f.stiles * zl::TILE_BK);   // up to one result per bucket
        } else {
            memset(&f, 0, sizeof(f));
        }
    }
    const size_t seg_b = (size_t)cfg->max_batch * h->nres * sizeof(zl::SegResult);
    if (e == cudaSuccess) e = cudaMalloc((void **)&h->d_meta, meta_b);
    if (e == cudaSuccess) e = cudaMalloc((void **)&h->d_seg, seg_b);
    const size_t pred_b = (cfg->flags & ZL_FLAG_PREDICTOR) ? (size_t)cfg->max_batch * cfg->n_workers * cfg->lookahead_R * 8 : 0;
    if (e == cudaSuccess && pred_b) e = cudaMalloc((void **)&h->d_pred, pred_b);
    if (e == cudaSuccess) e = raise_shared_memory_limits();   // more than the default 48 KB of dynamic shared memory
    if (e != cudaSuccess) {
        zl_status st = cuda_fail(nullptr, e);
        cudaFree(h->d_meta); cudaFree(h->d_seg); cudaFree(h->d_pred);
        cudaFree(h->fb.table); cudaFree(h->fb.rowhint); cudaFree(h->fb.cellmax); cudaFree(h->fb.rcnt);
        cudaFree(h->fb.list1); cudaFree(h->fb.bcnt); cudaFree(h->fb.list2); cudaFree(h->fb.tilemax); cudaFree(h->fb.flags);
        cudaFree(h->fb.bnd); cudaFree(h->fb.cellacc); cudaFree(h->fb.itab);
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
    ZL_CUDA(h, cudaSetDevice(h->cfg.device));
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
    cudaSetDevice(h->cfg.device);
    cudaFree(h->d_meta); cudaFree(h->d_seg); cudaFree(h->d_pred);
    cudaFree(h->fb.table); cudaFree(h->fb.rowhint); cudaFree(h->fb.cellmax); cudaFree(h->fb.rcnt);
    cudaFree(h->fb.list1); cudaFree(h->fb.bcnt); cudaFree(h->fb.list2); cudaFree(h->fb.tilemax); cudaFree(h->fb.flags);
    cudaFree(h->fb.bnd); cudaFree(h->fb.cellacc); cudaFree(h->fb.itab);
    cudaFree(h->s_ts); cudaFree(h->s_idx); cudaFree(h->s_barrier); cudaFree(h->s_wait); cudaFree(h->s_status);
    if (h->s_stream) cudaStreamDestroy(h->s_stream);
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
    } else if (!strcmp(key, "filter_threads")) {
        if (value && (!is_pow2(value) || value < 64 || value > 1024)) return ZL_ERR_INVALID_ARG;
        h->opt_filter_threads = value;
    } else if (!strcmp(key, "prologue_threads") || !strcmp(key, "tail_threads")) {
        if (value && (!is_pow2(value) || value < 64 || value > 1024)) return ZL_ERR_INVALID_ARG;
        (key[0] == 'p' ? h->opt_prologue_threads : h->opt_tail_threads) = value;
    } else if (!strcmp(key, "pdl_off")) {
        h->opt_pdl_off = value;                 // bit k set: kernel k of the chain is launched without early scheduling
    } else if (!strcmp(key, "filter_round")) {
        if (value && (!is_pow2(value) || value < 2 || value > 256)) return ZL_ERR_INVALID_ARG;
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
int32_t zl_launches_per_call(const zl_handle *h) {
    if (!h) return 0;
    const bool filter = h->cfg.objective == ZL_OBJ_RANGE && !h->opt_no_filter && h->fb.table != nullptr;
    const bool sumfast = !filter && !h->opt_no_filter && h->fb.scap != 0;
    return 3 + (filter ? 6 : 0) + (sumfast ? (h->fb.scells ? 3 : 2) : 0) + ((h->cfg.flags & ZL_FLAG_CHECK_SORTED) ? 1 : 0);
}
int32_t zl_route(const zl_handle *h) {
    if (!h || h->opt_no_filter) return 0;
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
    q.idx = d_idx; q.barrier = d_barrier; q.wait = d_wait; q.status = d_status;
    enqueue(q, p, st, ev, zl::MatBatch{d_ts});
    if (ev) ++h->prof_calls;
    ZL_CUDA(h, cudaGetLastError());
    h->launches += zl_launches_per_call(h);
    return ZL_OK;
}

zl_status zl_filter_counts(zl_handle *h, int32_t B, uint32_t *h_filtered, uint32_t *h_refined, uint32_t *h_overflow) {
    if (!h || B < 1 || B > h->cfg.max_batch) return ZL_ERR_INVALID_ARG;
    ZL_CUDA(h, cudaSetDevice(h->cfg.device));
    ZL_CUDA(h, cudaDeviceSynchronize());
    uint32_t *dst[3] = {h_filtered, h_refined, h_overflow};
    const size_t off[3] = {offsetof(zl::InstMeta, count), offsetof(zl::InstMeta, count2), offsetof(zl::InstMeta, overflow)};
    for (int i = 0; i < 3; ++i)
        if (dst[i])
            ZL_CUDA(h, cudaMemcpy2D(dst[i], sizeof(uint32_t), (const char *)h->d_meta + off[i], sizeof(zl::InstMeta),
                                    sizeof(uint32_t), (size_t)B, cudaMemcpyDeviceToHost));
    return ZL_OK;
}

zl_status zl_gridscan_batched(const int64_t *d_ts, int32_t B, int32_t n, int32_t R, int32_t full, int64_t *d_scratch,
                              int32_t *d_idx, int64_t *d_barrier, int64_t *d_wait, void *cuda_stream) {
    if (!d_ts || !d_scratch || !d_idx || !d_barrier || !d_wait || B < 1 || n < 1 || R < 1) return ZL_ERR_INVALID_ARG;
    if (B > 65535) return ZL_ERR_UNSUPPORTED;
    const long long ncand = full ? (long long)n * R : R;
    if (ncand > 0x7fffffffLL) return ZL_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int threads = std::max(32, std::min(256, pow2_ceil(n)));
    zl::k_gridscan_eval<<<dim3((unsigned)ncand, B), threads, 0, st>>>(d_ts, n, R, full ? 1 : 0, d_scratch);
    zl::k_gridscan_pick<<<B, 256, 0, st>>>(d_ts, n, R, full ? 1 : 0, (int)ncand, d_scratch, d_idx, d_barrier, d_wait);
    return cudaGetLastError() == cudaSuccess ? ZL_OK : ZL_ERR_CUDA;
}

zl_status zl_predict_batched(const int64_t *d_last, const int64_t *d_interval, int32_t B, int32_t n, int32_t R,
                             int64_t *d_ts, void *cuda_stream) {
    if (!d_last || !d_interval || !d_ts || B < 1 || n < 1 || R < 1) return ZL_ERR_INVALID_ARG;
    if (((uintptr_t)d_last & 7) || ((uintptr_t)d_interval & 7) || ((uintptr_t)d_ts & 15)) return ZL_ERR_INVALID_ARG;
    if ((long long)B * n > 0x7fffffffLL) return ZL_ERR_UNSUPPORTED;
    const int threads = std::max(32, std::min(256, pow2_ceil((R + 1) / 2)));
    zl::k_predict<<<(unsigned)((long long)B * n), threads, 0, (cudaStream_t)cuda_stream>>>(d_last, d_interval, R, d_ts);
    return cudaGetLastError() == cudaSuccess ? ZL_OK : ZL_ERR_CUDA;
}

zl_status zl_predict_select_batched(zl_handle *h, const int64_t *d_last, const int64_t *d_interval, int32_t B,
                                    int32_t *d_idx, int64_t *d_barrier, int64_t *d_wait, int32_t *d_status,
                                    void *cuda_stream) {
    if (!h || !h->d_pred) return ZL_ERR_INVALID_ARG;
    if (B < 1 || B > h->cfg.max_batch) return ZL_ERR_INVALID_ARG;
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
    ZL_CUDA(h, cudaSetDevice(h->cfg.device));
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

zl_status zl_trace_batched(const int64_t *d_ts, int32_t B, int32_t n, int32_t R, int64_t *om_t, int32_t *om_p,
                           int32_t *om_i, int64_t *delta, int32_t *first, int64_t *S, int32_t *cnt, int64_t *next,
                           int64_t *PM, int64_t *d_range, int64_t *w_sum, void *cuda_stream) {
    if (!d_ts || B < 1 || n < 1 || R < 1) return ZL_ERR_INVALID_ARG;
    if ((long long)n * R > zl::TRACE_MAX) return ZL_ERR_UNSUPPORTED;
    const int P = std::max(64, pow2_ceil(n * R));
    const size_t smem = (size_t)P * sizeof(zl::TKey);
    cudaError_t e = cudaFuncSetAttribute(zl::k_trace, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(zl::TRACE_MAX * sizeof(zl::TKey)));
    if (e != cudaSuccess) return ZL_ERR_CUDA;
    zl::k_trace<<<B, 256, smem, (cudaStream_t)cuda_stream>>>(d_ts, n, R, om_t, om_p, om_i, delta, first, S, cnt, next, PM, d_range, w_sum);
    return cudaGetLastError() == cudaSuccess ? ZL_OK : ZL_ERR_CUDA;
}

zl_status zl_probe_read_batched(const int64_t *d_ts, const int32_t *d_count, int64_t rows, int32_t R,
                                uint64_t *d_sink, void *cuda_stream) {
    if (!d_ts || !d_count || !d_sink || rows < 1 || R < 1) return ZL_ERR_INVALID_ARG;
    if (((uintptr_t)d_ts & 7) || ((uintptr_t)d_count & 3) || ((uintptr_t)d_sink & 7)) return ZL_ERR_INVALID_ARG;
    const long long blocks = (rows + 3) / 4;                      // four warps, one row each, per CTA
    if (blocks > 0x7fffffffLL) return ZL_ERR_UNSUPPORTED;
    zl::k_probe_read<<<(unsigned)blocks, 128, 0, (cudaStream_t)cuda_stream>>>(d_ts, d_count, (long long)rows, R,
                                                                            (unsigned long long *)d_sink);
    return cudaGetLastError() == cudaSuccess ? ZL_OK : ZL_ERR_CUDA;
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
    q.filter_threads = q.filter_rows = q.filter_round = 0; q.pdl_off = 0; q.prologue_threads = q.tail_threads = 0;
    q.idx = d_idx; q.barrier = d_barrier; q.wait = d_wait; q.status = d_status;
    enqueue(q, p, (cudaStream_t)cuda_stream, nullptr, zl::MatBatch{d_ts});
    return cudaGetLastError() == cudaSuccess ? ZL_OK : ZL_ERR_CUDA;
}

}  // extern "C"
