// Records shared by the ZipLine kernels and their host-side launchers: per-instance summary, partial results,
// row sources, the buffers of the fast routes, launch parameters.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/zipline.h"

namespace zl {

constexpr int MAX_WORKERS = 4096;
constexpr int MAX_SEGMENTS = 256;
constexpr int FILTER_ROWS = 32;       // rows that build the filter table
constexpr int FILTER_MAX_CELLS = 8192;
constexpr int SCAN_TILE = 4096;       // fine cells per tile of the cell scan
constexpr int TILE_BK = 15;           // bucket route: buckets per tile (16 boundaries = 32 bytes per row and tile)
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

// An instance's record read past the L1 cache: for kernels in which other CTAs update it between two of their phases.
__device__ __forceinline__ InstMeta load_meta_cg(const InstMeta *p) {
    static_assert(sizeof(InstMeta) == 64, "InstMeta is read as four 16-byte words");
    union { InstMeta m; uint4 q[4]; } u;
#pragma unroll
    for (int k = 0; k < 4; ++k) u.q[k] = __ldcg(reinterpret_cast<const uint4 *>(p) + k);
    return u.m;
}

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
    uint32_t *flags;     // [8]               per call: some instance needs [0] scan/refine/buckets, [1] the segment sweep; [4] arrivals at the
                         //                   grid-wide barriers of the route's last kernel, [5] one of its barriers gave up
    uint32_t *flags_next; // [8]              the flags of the handle's next call (the two sets alternate); zeroed by this call
    uint64_t *part;      // [ctas][4]         k_range_head: per-CTA minima / maxima of the first and last column
    uint32_t *hint;      // [1]               pinned host memory (device address), or nullptr: the call's last kernel notes here whether some
                         //                   instance had more survivors than one CTA finishes
    uint32_t *hint_last; // [1]               device: what was last written to `hint` (the word is written only when it changes)
    uint32_t *done;      // [B]               blocks of the filter pass that have finished, per instance (in the end: how many it had)
    uint32_t *ptab;      // [ctas][cells]     k_range_head: per-CTA partial filter tables
    int32_t maxctas;     //                   CTAs k_range_head's per-CTA records have room for
    uint32_t *dbg;       // [4]               ZL_FLAG_DEBUG_CHECKS: record of the first index violation (0: none)
    uint32_t *bcnt;      // [B][nbk]          survivors of the refinement per bucket
    uint64_t *list2;     // [B][nbk][capb]    survivors of the refinement
    int32_t cells, fcells, nbk, capb, grp;   // grp: fewest buckets per CTA of the bucket sweep
    int32_t nreg, regcap, list1cap;          // set per call: regions per instance and their capacity
    int32_t tailcap;                         // set per call: most survivors of the filter pass the tail kernel finishes an instance with
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
    int32_t max_rounds;   // 0: the bound that follows from the input's size; else rounds a segment may take before ZL_ERR_TIMEOUT
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
constexpr long long SMALL_MAX = 4096;    // instances of at most this many timestamps take the one-launch route
__device__ __forceinline__ bool tail_instance(const InstMeta &M, const FilterBufs &F) { return M.count <= (uint32_t)F.tailcap; }

}  // namespace zl
