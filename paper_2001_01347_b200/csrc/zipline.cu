// ZipLine barrier-selection search for sm_100a: kernels and the C ABI (see include/zipline.h).
//
// One call runs, per instance of n sorted rows of R int64 timestamps:
//   prologue   column scans: tmin, t0 = max_p e^p_1, lmin = min_p e^p_R, span
//   sweep      the timeline is cut into time segments, one CTA each.  A CTA walks its segment in
//              rounds: every row advances a cursor over the elements that fall in the round's time
//              window (the rows are already sorted, so the n-way merge is a set of cursors), attaches
//              to each element the payload the scan needs (next / delta+first flag), and appends it to
//              a shared-memory batch.  A full batch is sorted into time order (Omega), scanned
//              (prefix max of next / prefix sums of delta and flag) and evaluated, keeping the first
//              minimum.  Carry-ins at a segment start come from per-row binary searches, so segments
//              are independent.
//   finalize   minimum over the segments of an instance, barrier, per-worker index recovery.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>
#include <algorithm>
#include <mutex>
#include <new>

#include "../../include/zipline.h"
#include "zl_device.cuh"

namespace zl {

constexpr int MAX_WORKERS = 8192;
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
    uint32_t sh;         // filter table: cell c covers relative times [1 + (c << sh), 1 + ((c + 1) << sh))
    uint32_t ncell;      // cells in use (0: the instance does not take the filter path)
    uint32_t count;      // survivors appended by the filter pass (may run past the list capacity)
    uint32_t pad;
};

struct SegResult {
    uint64_t d;          // objective value of the segment's best candidate
    uint64_t t;          // its relative time (min(Z) for RANGE, the barrier for SUM)
    int32_t valid;
    int32_t status;
};

struct SweepParams {
    const int64_t *ts;
    InstMeta *meta;
    SegResult *seg;
    int32_t n, R, nseg, G, cap, flags, target;
    uint32_t listcap;    // > 0: instances whose filtered list fits are handled by k_small, not here
};

// An instance goes through the filter + small-sort path when it has a table and its survivors fit the list.
__device__ __forceinline__ bool handled_by_filter(const InstMeta &M, uint32_t listcap) {
    return listcap > 0 && M.ncell > 0 && M.count <= listcap;
}

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

__global__ void __launch_bounds__(1024) k_prologue(const int64_t *ts, int n, int R, int objective, int flags,
                                                    InstMeta *meta, uint32_t *table_all, int max_cells) {
    const int b = blockIdx.x, tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
    const int64_t *inst = ts + (size_t)b * n * R;
    __shared__ uint64_t s[4][32];
    __shared__ InstMeta sm;
    __shared__ uint32_t tab[FILTER_MAX_CELLS];
    uint64_t mn1 = ~0ull, mx1 = 0, mnR = ~0ull, mxR = 0;      // order-preserving unsigned images of int64
    for (int p = tid; p < n; p += nt) {
        const uint64_t e1 = (uint64_t)ldg64(inst + (size_t)p * R) ^ (1ull << 63);
        const uint64_t eR = (uint64_t)ldg64(inst + (size_t)p * R + R - 1) ^ (1ull << 63);
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
        m.sh = 0; m.ncell = 0; m.count = 0; m.pad = 0;
        if (tmin < 0 || tmax >= VALUE_LIMIT || tmax < tmin || lmin < tmin) {
            m.status = ZL_ERR_INVALID_ARG;     // outside [0, 2^62), or first/last columns out of order
            m.t0 = m.lmin = m.tend = 1; m.use32 = 1;
        } else {
            m.t0 = (uint64_t)(t0 - tmin) + 1;
            m.lmin = (uint64_t)(lmin - tmin) + 1;
            m.tend = (uint64_t)(tmax - tmin) + 1;
            m.use32 = m.tend < 0xfffffffeull;
            if (objective == ZL_OBJ_SUM && m.tend > (uint64_t)INT64_MAX / (uint64_t)n) m.status = ZL_ERR_UNSUPPORTED;
            if (objective == ZL_OBJ_RANGE && table_all && m.use32 && m.status == ZL_OK) {
                uint32_t sh = 0;
                while (((m.lmin - 1) >> sh) >= (uint64_t)max_cells) ++sh;
                m.sh = sh;
                m.ncell = (uint32_t)((m.lmin - 1) >> sh) + 1;
            }
        }
        sm = m;
    }
    __syncthreads();
    const InstMeta M = sm;
    if (M.ncell > 0) {
        const uint32_t ncell = M.ncell, sh = M.sh, lmin = (uint32_t)M.lmin;
        const int64_t tmin = M.tmin;
        for (uint32_t c = tid; c < ncell; c += nt) tab[c] = (uint32_t)M.t0;
        __syncthreads();
        // one slow row per warp: the row with the longest span in the warp's group of rows
        const int groups = min(n, FILTER_ROWS);
        const int gsz = (n + groups - 1) / groups;
        for (int gidx = warp; gidx < groups; gidx += nw) {
            const int p0 = gidx * gsz, p1 = min(p0 + gsz, n);
            uint64_t best = 0;                                   // (span << 20) | (row - p0) needs span < 2^44: use two steps
            int bestp = -1;
            uint64_t bspan = 0;
            for (int p = p0 + lane; p < p1; p += 32) {
                const uint64_t span = (uint64_t)(ldg64(inst + (size_t)p * R + R - 1) - ldg64(inst + (size_t)p * R));
                if (bestp < 0 || span > bspan) { bspan = span; bestp = p; }
            }
            best = warp_reduce(bspan, OpMax());
            const unsigned who = __ballot_sync(FULL, bestp >= 0 && bspan == best);
            if (!who) continue;
            const int row = __shfl_sync(FULL, bestp, __ffs(who) - 1);
            const int64_t *rp = inst + (size_t)row * R;
            // element i is the first element at or after every cell start in (e_{i-1}, e_i]
            for (int i0 = 1; i0 < R; i0 += 32) {
                const int i = i0 + lane;
                uint32_t prev = 0xffffffffu, curv = 0;
                if (i < R) {
                    prev = (uint32_t)(ldg64(rp + i - 1) - tmin + 1);
                    curv = (uint32_t)(ldg64(rp + i) - tmin + 1);
                }
                if (i < R && prev <= lmin) {
                    // cell starts are 1 + (c << sh); cells with prev < start <= curv
                    uint32_t c_from = ((prev - 1) >> sh) + 1;
                    uint32_t c_to = min((curv - 1) >> sh, ncell - 1);
                    for (uint32_t c = c_from; c <= c_to && c < ncell; ++c) atomicMax(&tab[c], curv);
                }
                const uint32_t first_prev = __shfl_sync(FULL, prev, 0);
                if (first_prev > lmin) break;                     // the rest of the row lies after lmin
            }
        }
        __syncthreads();
        uint32_t *tg = table_all + (size_t)b * max_cells;
        for (uint32_t c = tid; c < ncell; c += nt) tg[c] = tab[c];
    }
    if (tid == 0) meta[b] = M;
    (void)flags;
}

// ------------------------------------------------------------------------------ filter pass (RANGE)
// One warp per row streams the row in storage order (coalesced 256-byte chunks), keeps the elements
// that pass the table test and appends them, as (T << 32 | next), to the instance's list.
__global__ void __launch_bounds__(1024) k_filter(const int64_t *ts, int n, int R, int flags, int rows_per_cta,
                                                  InstMeta *meta, const uint32_t *table_all, int max_cells,
                                                  uint64_t *list_all, uint32_t listcap) {
    extern __shared__ __align__(16) unsigned char smem[];
    uint32_t *tab = (uint32_t *)smem;
    const int b = blockIdx.y, tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
    const InstMeta M = meta[b];
    if (M.status != ZL_OK || M.ncell == 0) return;
    const uint32_t ncell = M.ncell, sh = M.sh, lmin = (uint32_t)M.lmin;
    const int64_t tmin = M.tmin;
    const uint32_t *tg = table_all + (size_t)b * max_cells;
    for (uint32_t c = tid; c < ncell; c += nt) tab[c] = tg[c];
    __syncthreads();
    const bool full = (flags & ZL_FLAG_FULL_SWEEP) != 0;
    uint64_t *list = list_all + (size_t)b * listcap;
    unsigned int *counter = &meta[b].count;
    const int r0 = blockIdx.x * rows_per_cta, r1 = min(r0 + rows_per_cta, n);
    for (int r = r0 + warp; r < r1; r += nw) {
        if (*(volatile unsigned int *)counter > listcap) break;    // the list overflowed: this instance takes the general path
        const int64_t *row = ts + ((size_t)b * n + r) * R;
        uint32_t curT = lane < R ? (uint32_t)(ldg64(row + lane) - tmin + 1) : 0xffffffffu;
        for (int i0 = 0; i0 < R; i0 += 32) {
            const int inext = i0 + 32 + lane;
            const uint32_t nxtT = inext < R ? (uint32_t)(ldg64(row + inext) - tmin + 1) : 0xffffffffu;
            const uint32_t T = curT;
            uint32_t nx = __shfl_down_sync(FULL, T, 1);
            const uint32_t nfirst = __shfl_sync(FULL, nxtT, 0);
            if (lane == 31) nx = nfirst;                            // 0xffffffff past the end of the row
            const bool valid = i0 + lane < R && T <= lmin;
            bool keep = false;
            if (valid) {
                const uint32_t L = tab[(T - 1) >> sh];
                keep = nx > max(T, L);
            }
            const unsigned km = __ballot_sync(FULL, keep);
            if (km) {
                unsigned base = 0;
                const int leader = __ffs(km) - 1;
                if (lane == leader) base = atomicAdd(counter, __popc(km));
                base = __shfl_sync(FULL, base, leader);
                if (keep) {
                    const unsigned pos = base + __popc(km & ((1u << lane) - 1u));
                    if (pos < listcap) list[pos] = ((uint64_t)T << 32) | nx;
                }
            }
            if (!full && __shfl_sync(FULL, T, 31) > lmin) break;   // rows are sorted: nothing later is <= lmin
            curT = nxtT;
        }
    }
}

// Optional full check that every row is non-decreasing.
__global__ void k_check_sorted(const int64_t *ts, int n, int R, size_t total, InstMeta *meta) {
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
template <typename K, int OBJ>
__device__ void run_batch(Key<K> *keys, int m, K t0, int n, uint64_t *tmp64, K carryMax, uint64_t &carryS,
                          uint32_t &carryC, uint64_t &bd, uint64_t &bt) {
    if (m == 0) return;
    int P = 32;
    while (P < m) P <<= 1;
    for (int i = m + threadIdx.x; i < P; i += blockDim.x) keys[i] = Key<K>::inf();
    __syncthreads();
    bitonic_sort(keys, P);
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

// Block minimum of (objective, time) over the per-thread bests -> out.  red: 32 shared words.
__device__ void block_best_to_result(uint64_t bd, uint64_t bt, uint32_t status, uint64_t *red, unsigned int *sstatus,
                                     SegResult &out) {
    const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31;
    for (int d = 16; d > 0; d >>= 1) {
        const uint64_t od = shfl_xor(bd, d), ot = shfl_xor(bt, d);
        if (od < bd || (od == bd && ot < bt)) { bd = od; bt = ot; }
    }
    __syncthreads();
    if (lane == 0) red[tid >> 5] = bd;
    __syncthreads();
    // two steps: the minimum objective, then the minimum time among its holders
    uint64_t gd = ~0ull;
    for (int w = 0; w < (nt >> 5); ++w) gd = min(gd, red[w]);
    __syncthreads();
    if (lane == 0) red[tid >> 5] = bd == gd ? bt : ~0ull;
    __syncthreads();
    uint64_t gt = ~0ull;
    for (int w = 0; w < (nt >> 5); ++w) gt = min(gt, red[w]);
    if (status != ZL_OK) atomicMax(sstatus, status);
    __syncthreads();
    if (tid == 0) {
        out.d = gd; out.t = gt;
        out.valid = gd != ~0ull || gt != ~0ull;
        out.status = (int32_t)*sstatus;
    }
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

template <typename K, int OBJ>
__device__ void sweep_segment(const SweepParams &P, const InstMeta &M, const int64_t *inst, SweepShared &sh,
                              uint32_t *curA, uint32_t *curB, Key<K> *keys, SegResult &out) {
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
    const uint64_t seg_lo = 1 + (uint64_t)blockIdx.x * width;
    const uint64_t seg_hi = min(seg_lo + width, tend + 1);
    uint64_t bd = ~0ull, bt = ~0ull;          // per-thread best (objective, time)
    uint32_t status = ZL_OK;

    K floorv = 0;                              // max of next over every element before the current round
    if (tid == 0) { sh.count = 0; sh.carryS = 0; sh.carryC = 0; sh.vmax = 0; sh.status = 0; }
    __syncthreads();
    if (seg_lo <= tend) {
        // ---- carry-in: per-row lower bound of the segment start
        if (blockIdx.x == 0) {
            for (int r = tid; r < n; r += nt) curA[r] = 0;
        } else {
            const int64_t a_raw = tmin + (int64_t)(seg_lo - 1);
            unsigned long long vloc = 0, sloc = 0;
            unsigned int cloc = 0;
            for (int r = tid; r < n; r += nt) {
                const int64_t *row = inst + (size_t)r * R;
                int lo = 0, hi = R;               // first index with row[i] >= a_raw
                while (lo < hi) {
                    const int mid = (lo + hi) >> 1;
                    if (ldg64(row + mid) < a_raw) lo = mid + 1; else hi = mid;
                }
                curA[r] = (uint32_t)lo;
                if (lo > 0) {
                    if (OBJ == ZL_OBJ_RANGE) {
                        const unsigned long long v = lo < R ? (unsigned long long)(K)(ldg64(row + lo) - tmin + 1) : (unsigned long long)INF;
                        vloc = max(vloc, v);
                    } else {
                        sloc += (unsigned long long)(K)(ldg64(row + lo - 1) - tmin + 1);
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
                const int64_t *row = inst + (size_t)(act ? r : 0) * R;
                uint32_t c = act ? cur[r] : (uint32_t)R;
                bool more = act;
                for (;;) {
                    const uint32_t idx = c + g;
                    const bool have = more && idx < (uint32_t)R;
                    const K T = have ? (K)(ldg64(row + idx) - tmin + 1) : INF;
                    const bool cons = have && T < rhi;
                    bool app = false;
                    Key<K> key = Key<K>::inf();
                    if (cons) {
                        ++cons_n;
                        if (OBJ == ZL_OBJ_RANGE) {
                            const K nx = idx + 1 < (uint32_t)R ? (K)(ldg64(row + idx + 1) - tmin + 1) : INF;
                            vloc = max(vloc, (unsigned long long)nx);
                            app = nx > max(T, floorv);            // only elements that raise the running max matter
                            key = Key<K>::make(T, nx);
                        } else {
                            const K pv = idx > 0 ? (K)(ldg64(row + idx - 1) - tmin + 1) : (K)0;
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
                    run_batch<K, OBJ>(keys, (int)count_before, t0, n, sh.tmp, carryMax, carryS, carryC, bd, bt);
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
                run_batch<K, OBJ>(keys, (int)count_before, t0, n, sh.tmp, carryMax, carryS, carryC, bd, bt);
                carryMax = floorv;
                count_before = 0;
                if (tid == 0) sh.count = 0;
                __syncthreads();
            }
        }
        if (count_before > 0)
            run_batch<K, OBJ>(keys, (int)count_before, t0, n, sh.tmp, carryMax, carryS, carryC, bd, bt);
    }

    block_best_to_result(bd, bt, status, sh.tmp, &sh.status, out);
}

template <int OBJ>
__global__ void __launch_bounds__(1024) k_sweep(const SweepParams P) {
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ SweepShared sh;
    const int b = blockIdx.y;
    const InstMeta M = P.meta[b];
    SegResult &out = P.seg[(size_t)b * P.nseg + blockIdx.x];
    if (handled_by_filter(M, P.listcap)) return;             // k_small wrote this instance's result
    if (M.status != ZL_OK) {
        if (threadIdx.x == 0) { out.d = ~0ull; out.t = ~0ull; out.valid = 0; out.status = ZL_OK; }
        return;
    }
    uint32_t *curA = (uint32_t *)smem;
    uint32_t *curB = curA + P.n;
    unsigned char *kb = smem + (((size_t)2 * P.n * sizeof(uint32_t) + 15) & ~(size_t)15);
    const int64_t *inst = P.ts + (size_t)b * P.n * P.R;
    if (M.use32) {
        sweep_segment<uint32_t, OBJ>(P, M, inst, sh, curA, curB, (Key<uint32_t> *)kb, out);
    } else {
        SweepParams Q = P;
        Q.cap = P.cap / 2;                      // 16-byte nodes: half as many fit
        sweep_segment<uint64_t, OBJ>(Q, M, inst, sh, curA, curB, (Key<uint64_t> *)kb, out);
    }
}

// Sort and sweep the filtered list of an instance in one CTA.
__global__ void __launch_bounds__(1024) k_small(InstMeta *meta, const uint64_t *list_all, uint32_t listcap, int n,
                                                int nseg, SegResult *seg) {
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ uint64_t tmp[34];
    __shared__ unsigned int sstatus;
    const int b = blockIdx.x, tid = threadIdx.x;
    const InstMeta M = meta[b];
    if (M.status != ZL_OK || !handled_by_filter(M, listcap)) return;
    Key<uint32_t> *keys = (Key<uint32_t> *)smem;
    const uint64_t *list = list_all + (size_t)b * listcap;
    const int m = (int)M.count;
    for (int i = tid; i < m; i += blockDim.x) keys[i].w = list[i];
    if (tid == 0) sstatus = 0;
    __syncthreads();
    uint64_t bd = ~0ull, bt = ~0ull, cs = 0;
    uint32_t cc = 0;
    run_batch<uint32_t, ZL_OBJ_RANGE>(keys, m, (uint32_t)M.t0, n, tmp, (uint32_t)0, cs, cc, bd, bt);
    block_best_to_result(bd, bt, ZL_OK, tmp, &sstatus, seg[(size_t)b * nseg]);
}

// ------------------------------------------------------------------------------ finalize
__global__ void __launch_bounds__(256) k_finalize(const int64_t *ts, int n, int R, int nseg, int objective,
                                                  uint32_t listcap, const InstMeta *meta, const SegResult *seg,
                                                  int32_t *idx, int64_t *barrier, int64_t *wait, int32_t *status) {
    const int b = blockIdx.x;
    const InstMeta M = meta[b];
    __shared__ int64_t s_barrier;
    __shared__ int s_status;
    if (threadIdx.x == 0) {
        int st = M.status;
        uint64_t bd = ~0ull, bt = ~0ull;
        bool have = false;
        if (st == ZL_OK) {
            const int nseg_used = handled_by_filter(M, listcap) ? 1 : nseg;
            for (int s = 0; s < nseg_used; ++s) {
                const SegResult r = seg[(size_t)b * nseg + s];
                if (r.status != ZL_OK) st = max(st, r.status);
                if (!r.valid) continue;
                if (!have || r.d < bd || (r.d == bd && r.t < bt)) { bd = r.d; bt = r.t; have = true; }
            }
            if (st == ZL_OK && !have) st = ZL_ERR_TIMEOUT;     // cannot happen for valid input
        }
        if (st == ZL_OK) {
            const int64_t tm = M.tmin + (int64_t)(bt - 1);
            s_barrier = objective == ZL_OBJ_RANGE ? tm + (int64_t)bd : tm;
            wait[b] = (int64_t)bd;
            barrier[b] = s_barrier;
        } else {
            wait[b] = INT64_MIN;
            barrier[b] = INT64_MIN;
            s_barrier = INT64_MIN;
        }
        s_status = st;
        if (status) status[b] = st;
    }
    __syncthreads();
    const int64_t bar = s_barrier;
    const bool ok = s_status == ZL_OK;
    const int64_t *inst = ts + (size_t)b * n * R;
    for (int p = threadIdx.x; p < n; p += blockDim.x) {
        int res = -1;
        if (ok) {
            const int64_t *row = inst + (size_t)p * R;
            int lo = 0, hi = R;                   // number of elements <= barrier
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (ldg64(row + mid) <= bar) lo = mid + 1; else hi = mid;
            }
            res = lo - 1;
        }
        idx[(size_t)b * n + p] = res;
    }
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
    int P = 32;
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
    uint32_t *d_table;       // RANGE: filter tables, [max_batch][max_cells]
    uint64_t *d_list;        // RANGE: filtered (T, next) lists, [max_batch][listcap]
    int max_cells, listcap;
    size_t ws_bytes;
    // host-buffer path
    int64_t *s_ts; int32_t *s_idx; int64_t *s_barrier; int64_t *s_wait; int32_t *s_status;
    cudaStream_t s_stream;
    size_t staging_bytes;
    // options (0 = automatic)
    int opt_threads, opt_lanes, opt_segments, opt_round_factor, opt_no_filter;
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
    zl::InstMeta *meta; zl::SegResult *seg;
    uint32_t *table; uint64_t *list; int max_cells, listcap;      // table == nullptr: no filter path
    int32_t *idx; int64_t *barrier; int64_t *wait; int32_t *status;
};

void enqueue(const Pipeline &q, const LaunchPlan &p, cudaStream_t st, cudaEvent_t *ev) {
    const bool filter = q.table != nullptr && q.objective == ZL_OBJ_RANGE;
    const uint32_t listcap = filter ? (uint32_t)q.listcap : 0u;
    if (ev) cudaEventRecord(ev[0], st);
    zl::k_prologue<<<q.B, 1024, 0, st>>>(q.ts, q.n, q.R, q.objective, q.flags, q.meta, filter ? q.table : nullptr, q.max_cells);
    if (q.flags & ZL_FLAG_CHECK_SORTED) {
        const size_t total = (size_t)q.B * q.n * q.R;
        const int blocks = (int)std::min<size_t>((total + 255) / 256, (size_t)q.num_sms * 16);
        zl::k_check_sorted<<<blocks, 256, 0, st>>>(q.ts, q.n, q.R, total, q.meta);
    }
    if (ev) cudaEventRecord(ev[1], st);
    if (filter) {
        const int threads = std::max(64, std::min(1024, 32 * pow2_ceil(std::min(q.n, 32))));
        const int nw = threads / 32;
        long long rpc = ((long long)q.n * q.B / (4LL * q.num_sms) + nw - 1) / nw * nw;
        rpc = std::max<long long>(nw, std::min<long long>(rpc, (q.n + nw - 1) / nw * nw));
        const dim3 grid((unsigned)((q.n + rpc - 1) / rpc), q.B);
        zl::k_filter<<<grid, threads, (size_t)q.max_cells * 4, st>>>(q.ts, q.n, q.R, q.flags, (int)rpc, q.meta, q.table,
                                                                   q.max_cells, q.list, listcap);
    }
    if (ev) cudaEventRecord(ev[2], st);
    if (filter) {
        const int threads = std::max(128, std::min(1024, q.listcap / 4));
        zl::k_small<<<q.B, threads, (size_t)q.listcap * 8, st>>>(q.meta, q.list, listcap, q.n, p.nseg, q.seg);
    }
    zl::SweepParams sp;
    sp.ts = q.ts; sp.meta = q.meta; sp.seg = q.seg;
    sp.n = q.n; sp.R = q.R; sp.nseg = p.nseg; sp.G = p.G; sp.cap = p.cap; sp.flags = q.flags; sp.target = p.target;
    sp.listcap = listcap;
    const dim3 grid(p.nseg, q.B);
    if (q.objective == ZL_OBJ_RANGE) zl::k_sweep<ZL_OBJ_RANGE><<<grid, p.threads, p.smem, st>>>(sp);
    else zl::k_sweep<ZL_OBJ_SUM><<<grid, p.threads, p.smem, st>>>(sp);
    if (ev) cudaEventRecord(ev[3], st);
    zl::k_finalize<<<q.B, 256, 0, st>>>(q.ts, q.n, q.R, p.nseg, q.objective, listcap, q.meta, q.seg, q.idx, q.barrier, q.wait, q.status);
    if (ev) cudaEventRecord(ev[4], st);
}

cudaError_t raise_shared_memory_limits() {
    cudaError_t e = cudaFuncSetAttribute(zl::k_sweep<ZL_OBJ_RANGE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(zl::k_sweep<ZL_OBJ_SUM>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(zl::k_small, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
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
    int cap = std::max(8192, pow2_ceil(2 * n));
    const int small = std::max(pow2_ceil((int)std::min<long long>(N, 1 << 20)), std::max(pow2_ceil(2 * n), 64));
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
    if (h->cfg.objective == ZL_OBJ_SUM) target = std::min<long long>(target, (long long)p.cap * 45 / 100 / 2);
    target = std::min<long long>(target, (long long)p.cap * 4);
    p.target = (int)std::max<long long>(target, 32);
    p.smem = (((size_t)2 * n * sizeof(uint32_t) + 15) & ~(size_t)15) + (size_t)p.cap * 8;
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
    if (cfg->flags & ~(ZL_FLAG_CHECK_SORTED | ZL_FLAG_FULL_SWEEP)) return ZL_ERR_INVALID_ARG;
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
    const size_t seg_b = (size_t)cfg->max_batch * zl::MAX_SEGMENTS * sizeof(zl::SegResult);
    if (e == cudaSuccess) e = cudaMalloc((void **)&h->d_meta, meta_b);
    if (e == cudaSuccess) e = cudaMalloc((void **)&h->d_seg, seg_b);
    size_t table_b = 0, list_b = 0;
    if (cfg->objective == ZL_OBJ_RANGE) {
        const long long N = (long long)cfg->n_workers * cfg->lookahead_R;
        h->max_cells = std::max(64, std::min(zl::FILTER_MAX_CELLS, pow2_ceil((int)std::min<long long>(4LL * cfg->lookahead_R, 1 << 20))));
        h->listcap = std::max(64, std::min(16384, pow2_ceil((int)std::min<long long>(N, 1 << 20))));
        table_b = (size_t)cfg->max_batch * h->max_cells * sizeof(uint32_t);
        list_b = (size_t)cfg->max_batch * h->listcap * sizeof(uint64_t);
        if (e == cudaSuccess) e = cudaMalloc((void **)&h->d_table, table_b);
        if (e == cudaSuccess) e = cudaMalloc((void **)&h->d_list, list_b);
    }
    if (e == cudaSuccess) e = raise_shared_memory_limits();   // more than the default 48 KB of dynamic shared memory
    if (e != cudaSuccess) {
        zl_status st = cuda_fail(nullptr, e);
        cudaFree(h->d_meta); cudaFree(h->d_seg); cudaFree(h->d_table); cudaFree(h->d_list);
        delete h;
        return st;
    }
    h->ws_bytes = meta_b + seg_b + table_b + list_b;
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
    cudaFree(h->d_meta); cudaFree(h->d_seg); cudaFree(h->d_table); cudaFree(h->d_list);
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
    const bool filter = h->cfg.objective == ZL_OBJ_RANGE && !h->opt_no_filter;
    return 3 + (filter ? 2 : 0) + ((h->cfg.flags & ZL_FLAG_CHECK_SORTED) ? 1 : 0);
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
    q.meta = h->d_meta; q.seg = h->d_seg;
    q.table = h->opt_no_filter ? nullptr : h->d_table; q.list = h->d_list; q.max_cells = h->max_cells; q.listcap = h->listcap;
    q.idx = d_idx; q.barrier = d_barrier; q.wait = d_wait; q.status = d_status;
    enqueue(q, p, st, ev);
    if (ev) ++h->prof_calls;
    ZL_CUDA(h, cudaGetLastError());
    h->launches += zl_launches_per_call(h);
    return ZL_OK;
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
    const int P = std::max(32, pow2_ceil(n * R));
    const size_t smem = (size_t)P * sizeof(zl::TKey);
    cudaError_t e = cudaFuncSetAttribute(zl::k_trace, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(zl::TRACE_MAX * sizeof(zl::TKey)));
    if (e != cudaSuccess) return ZL_ERR_CUDA;
    zl::k_trace<<<B, 256, smem, (cudaStream_t)cuda_stream>>>(d_ts, n, R, om_t, om_p, om_i, delta, first, S, cnt, next, PM, d_range, w_sum);
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
    q.meta = meta; q.seg = seg;
    q.table = nullptr; q.list = nullptr; q.max_cells = 0; q.listcap = 0;
    q.idx = d_idx; q.barrier = d_barrier; q.wait = d_wait; q.status = d_status;
    enqueue(q, p, (cudaStream_t)cuda_stream, nullptr);
    return cudaGetLastError() == cudaSuccess ? ZL_OK : ZL_ERR_CUDA;
}

}  // extern "C"
