// k_range_fused: the RANGE search of an instance by one thread-block cluster in one launch.
//
// A cluster of G CTAs owns an instance; CTA `rank` owns a block of its rows.  The phases are those of the
// filter route (see prologue.cu and filter.cu for why the filter is exact), separated by cluster barriers;
// what the CTAs exchange goes through global scratch (the barrier orders it):
//   1  column scans of the own rows -> partial minima / maxima -> every CTA forms the instance summary;
//   2  partial filter table from the own slow rows -> merged table and dmin in every CTA;
//   3  the filter pass over the own rows: a warp per row, the row's leading timestamps arrive in a per-warp
//      ring of shared-memory slots through bulk copies (one request per chunk, issued by one lane, counted on
//      an mbarrier); 128 timestamps a step are tested against dmin, the few candidates against the table;
//      survivors go to the CTA's list;
//   4  CTA 0 finishes an instance with few survivors (refine, sort, prefix max, evaluate, first minimum);
//   5  every CTA recovers the indices of its own rows.
// Instances with many survivors, with a time span of 2^32 or more, or with a full list are left to the kernels
// of heavy.cu and sweep.cu, which the host enqueues behind this one (they return at once otherwise).
//
// With CHECK on (ZL_FLAG_DEBUG_CHECKS) every computed index into global or shared memory and every bulk copy
// is tested against the extent of its buffer first; a violation is recorded (which access, which CTA, the
// index; the first one wins) and the access is skipped, so a wrong index is reported instead of faulting.
#include <cooperative_groups.h>

#include "zl_batch.cuh"
#include "zl_host.h"

namespace cg = cooperative_groups;

namespace zl {

struct FusedParams {
    int n, R, B, flags, rpc, S, CH, tcap, slow, nres, vec2, prefetch;
    InstMeta *meta; SegResult *seg;
    int32_t *idx; int64_t *barrier; int64_t *wait; int32_t *status;
    uint32_t *dbg;                       // CHECK: [0] code of the first violation, [1] its CTA, [2..3] the index
    unsigned long long *stamps;          // debug handles: [ctas][16] nanosecond clock at the phase boundaries of every CTA
    uint32_t smem_bytes, ctas;
};

enum FusedAccess : int {
    ACC_PART = 1, ACC_PTAB, ACC_RCNT, ACC_LIST, ACC_CELLMAX, ACC_BCNT, ACC_META, ACC_SEG, ACC_IDX,
    ACC_COPY_SRC, ACC_COPY_DST, ACC_COPY_ALIGN, ACC_TAB, ACC_ARR, ACC_COLS, ACC_REQS, ACC_SLOT, ACC_KEYS
};

template <bool CHECK>
struct Guard {
    uint32_t *dbg; uint32_t cta;
    __device__ __forceinline__ bool ok(uint64_t i, uint64_t lim, int code) const {
        if (!CHECK) return true;
        if (i < lim) return true;
        if (atomicCAS(&dbg[0], 0u, (uint32_t)code) == 0u) { dbg[1] = cta; dbg[2] = (uint32_t)i; dbg[3] = (uint32_t)(i >> 32); }
        return false;
    }
};

__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

template <bool CHECK>
struct FCtx {
    uint32_t *tab; uint64_t *list; uint32_t *cellmax; unsigned int *scount;
    uint32_t cscale, fscale, lmin, regcap, dmin, tminlo;
    uint32_t cells, fcells;
    Guard<CHECK> g;
};

// A candidate (its own iteration is longer than dmin) against the table; survivors are rare, so each is
// appended on its own.
template <bool CHECK>
__device__ __forceinline__ void filter_candidate(const FCtx<CHECK> &c, uint32_t T, uint32_t nx) {
    const uint32_t cc = cell_of(T, c.cscale);
    if (!c.g.ok(cc, c.cells, ACC_TAB)) return;
    if (nx > max(T, c.tab[cc])) {
        const unsigned pos = atomicAdd(c.scount, 1u);
        if (pos < c.regcap) c.list[pos] = ((uint64_t)T << 32) | nx;
        const uint32_t fc = cell_of(T, c.fscale);
        if (c.g.ok(fc, c.fcells, ACC_CELLMAX)) atomicMax(&c.cellmax[fc], nx);
    }
}

// 128 timestamps of a slot that all lie inside the request, with the element after them: four per lane, no
// bounds checks.  Returns the time of the last of the 128.
template <bool CHECK>
__device__ __forceinline__ uint32_t filter_128(const FCtx<CHECK> &C, const int64_t *s, int lane) {
    const longlong2 p0 = *reinterpret_cast<const longlong2 *>(s + 2 * lane);
    const longlong2 p1 = *reinterpret_cast<const longlong2 *>(s + 64 + 2 * lane);
    const uint32_t a0 = (uint32_t)(uint64_t)p0.x - C.tminlo, b0 = (uint32_t)(uint64_t)p0.y - C.tminlo;
    const uint32_t a1 = (uint32_t)(uint64_t)p1.x - C.tminlo, b1 = (uint32_t)(uint64_t)p1.y - C.tminlo;
    const uint32_t n0 = (uint32_t)(uint64_t)s[2 * lane + 2] - C.tminlo, n1 = (uint32_t)(uint64_t)s[64 + 2 * lane + 2] - C.tminlo;
    const bool k0 = a0 <= C.lmin && b0 - a0 > C.dmin, k1 = b0 <= C.lmin && n0 - b0 > C.dmin;
    const bool k2 = a1 <= C.lmin && b1 - a1 > C.dmin, k3 = b1 <= C.lmin && n1 - b1 > C.dmin;
    if (k0 | k1 | k2 | k3) {                                      // few lanes, if any
        if (k0) filter_candidate(C, a0, b0);
        if (k1) filter_candidate(C, b0, n0);
        if (k2) filter_candidate(C, a1, b1);
        if (k3) filter_candidate(C, b1, n1);
    }
    return __shfl_sync(FULL, b1, 31);
}

// 64 timestamps starting at slot[off] = element i0 + off of the row, of which those below `lim` count; the
// successor of the row's last element is infinite.  Returns the time lane 31's second element has
// (0xffffffff past the end).
template <bool CHECK>
__device__ __forceinline__ uint32_t filter_64(const FCtx<CHECK> &C, const int64_t *slot, int off, int i0, int lim, int R, int lane) {
    const int i = i0 + off + 2 * lane;
    const bool va = i < lim, vb = i + 1 < lim;
    const longlong2 ab = *reinterpret_cast<const longlong2 *>(slot + off + 2 * lane);
    const uint32_t Ta = va ? (uint32_t)(uint64_t)ab.x - C.tminlo : 0xffffffffu;
    const uint32_t Tb = vb ? (uint32_t)(uint64_t)ab.y - C.tminlo : 0xffffffffu;
    const uint32_t na = i + 1 < R ? (uint32_t)(uint64_t)ab.y - C.tminlo : 0xffffffffu;
    const uint32_t nb = i + 2 < R ? (uint32_t)(uint64_t)slot[off + 2 * lane + 2] - C.tminlo : 0xffffffffu;
    if (va && Ta <= C.lmin && na - Ta > C.dmin) filter_candidate(C, Ta, na);
    if (vb && Tb <= C.lmin && nb - Tb > C.dmin) filter_candidate(C, Tb, nb);
    return __shfl_sync(FULL, Tb, 31);
}

// Elements j0, j0 + 1, ... of a row by plain loads (rows that cannot take bulk copies, and the rare row whose
// request ended before the row passed lmin).
template <bool CHECK>
__device__ __forceinline__ void filter_plain(const FCtx<CHECK> &C, const int64_t *row, int j0, int R, bool full, int lane) {
    for (; j0 < R; j0 += 64) {
        const int i = j0 + 2 * lane;
        const bool va = i < R, vb = i + 1 < R;
        const uint32_t Ta = va ? (uint32_t)(uint64_t)ldg64(row + i) - C.tminlo : 0xffffffffu;
        const uint32_t Tb = vb ? (uint32_t)(uint64_t)ldg64(row + i + 1) - C.tminlo : 0xffffffffu;
        uint32_t nb = __shfl_down_sync(FULL, Ta, 1);
        if (lane == 31) nb = i + 2 < R ? (uint32_t)(uint64_t)ldg64(row + i + 2) - C.tminlo : 0xffffffffu;
        if (va && Ta <= C.lmin && Tb - Ta > C.dmin) filter_candidate(C, Ta, Tb);
        if (vb && Tb <= C.lmin && nb - Tb > C.dmin) filter_candidate(C, Tb, nb);
        if (!full && __shfl_sync(FULL, Tb, 31) > C.lmin) break;
    }
}

// The filter pass of one warp over its rows r0 + warp, r0 + warp + nw, ... < r1 of the instance that starts
// `inst_off` timestamps into ts (stored rows; `total` timestamps in all).
// reqs[p]: how many leading timestamps of row r0 + p are requested through the ring (even; 0: none).
// Returns false when a copy did not arrive within the poll limit.
template <bool CHECK>
__device__ bool filter_rows_ring(const FCtx<CHECK> &C, const int64_t *ts, size_t inst_off, size_t total, int R, int r0, int r1,
                                 const uint32_t *reqs, int64_t *ring, uint64_t *bars, int S, int CH, bool full, int lane, int warp, int nw) {
    const int slot_elems = CH + 2;
    const int64_t *inst = ts + inst_off;
    uint32_t phase = 0;                                           // bit s: parity of slot s's next completion
    bool ok = true;
    for (int rbase = r0 + warp; rbase < r1; rbase += 32 * nw) {
        const int nrows = min(32, (r1 - rbase + nw - 1) / nw);
        const int req = lane < nrows ? (int)reqs[rbase - r0 + lane * nw] : 0;
        // producer cursor (ji, ci), consumer cursor (jp, cp): row of the round, chunk of the row
        int ji = 0, ci = 0, jp = 0, cp = 0, inflight = 0, si = 0, sp = 0;
        int req_i = __shfl_sync(FULL, req, 0), req_p = req_i;
        bool finished = false;
        while (jp < nrows) {
            while (inflight < S && ji < nrows) {
                if (req_i > 0) {
                    const int base = ci * CH;
                    const int endi = min(base + CH, req_i);
                    if (lane == 0) {
                        const uint32_t bytes = (uint32_t)(min(endi + 2, R) - base) * 8u;   // the chunk and the element after it
                        const size_t src = inst_off + (size_t)(rbase + ji * nw) * R + base;
                        bool go = true;
                        if (CHECK)
                            go = C.g.ok(src + bytes / 8 - 1, total, ACC_COPY_SRC) && C.g.ok(bytes / 8 - 1, (uint64_t)slot_elems, ACC_COPY_DST) &&
                                 C.g.ok((bytes & 15u) | (uint32_t)((uintptr_t)(ts + src) & 15u) | (uint32_t)(bytes == 0), 1, ACC_COPY_ALIGN);
                        fence_proxy_async();
                        mbar_expect_tx(&bars[si], go ? bytes : 0u);
                        if (go) bulk_copy_g2s(ring + (size_t)si * slot_elems, ts + src, bytes, &bars[si]);
                    }
                    ++inflight;
                    si = si + 1 == S ? 0 : si + 1;
                    if (endi < req_i) { ++ci; continue; }
                }
                ci = 0; ++ji;
                req_i = __shfl_sync(FULL, req, min(ji, 31));
            }
            const int64_t *row_p = inst + (size_t)(rbase + jp * nw) * R;
            if (req_p > 0) {
                if (ok && !mbar_wait_bounded(&bars[sp], (phase >> sp) & 1u)) ok = false;
                phase ^= 1u << sp;
                const int i0 = cp * CH;
                const int L = min(CH, req_p - i0);
                if (!finished && ok) {
                    const int64_t *slot = ring + (size_t)sp * slot_elems;
                    uint32_t lastT = 0;
                    for (int sub = 0; sub < L; sub += 128) {
                        if (sub && !full && lastT > C.lmin) break;          // rows are sorted: the rest is past lmin
                        if (sub + 128 <= L && i0 + sub + 128 < R) {
                            lastT = filter_128(C, slot + sub, lane);
                        } else {
                            lastT = filter_64(C, slot, sub, i0, req_p, R, lane);
                            if (sub + 64 < L && (full || lastT <= C.lmin)) lastT = filter_64(C, slot, sub + 64, i0, req_p, R, lane);
                        }
                    }
                    finished = !full && lastT > C.lmin;
                }
                __syncwarp();
                --inflight;
                sp = sp + 1 == S ? 0 : sp + 1;
                if (i0 + L < req_p) { ++cp; continue; }
            }
            // the row's request is used up: a row that has not passed lmin yet continues with plain loads
            if (!finished && ok && req_p < R) filter_plain(C, row_p, req_p, R, full, lane);
            cp = 0; ++jp; finished = false;
            req_p = __shfl_sync(FULL, req, min(jp, 31));
        }
    }
    return ok;
}

// The filter pass on predicted rows e_i = last + (i + 1) * interval: a row whose interval does not exceed dmin is
// settled at once (only its last element, whose next is infinite, can pass); the others are walked up to lmin.
template <bool CHECK>
__device__ void filter_rows_arith(const FCtx<CHECK> &C, const AriRows &rows, int R, int r0, int r1, int64_t tmin, int lane, int warp, int nw) {
    for (int r = r0 + warp; r < r1; r += nw) {
        const AriRow rw = rows.row(r);
        const int64_t rel0 = rw.l - tmin + 1;                     // relative time of element i: rel0 + (i + 1) * v, >= 1
        const int64_t v = rw.v, room = (int64_t)C.lmin - rel0;
        const int cnt = v == 0 ? (room >= 0 ? R : 0) : room < v ? 0 : (int)min((int64_t)R, room / v);
        if (cnt == 0) continue;
        if ((uint64_t)v <= (uint64_t)C.dmin) {
            if (cnt == R && lane == 0) filter_candidate(C, (uint32_t)(rel0 + (int64_t)R * v), 0xffffffffu);
            continue;
        }
        for (int i0 = 0; i0 < cnt; i0 += 32) {
            const int i = i0 + lane;
            const uint32_t T = (uint32_t)(rel0 + (int64_t)(i + 1) * v);
            if (i < cnt) filter_candidate(C, T, i + 1 < R ? T + (uint32_t)v : 0xffffffffu);
        }
    }
}

// Ask the memory system to bring a piece of global memory into the L2 (no destination, nothing to wait for).
__device__ __forceinline__ void prefetch_l2_bulk(const void *src, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}

// Barrier over the CTAs of an instance: the cluster's hardware barrier (it also orders their global writes), or,
// when one CTA has the instance to itself and the launch is an ordinary one, the CTA barrier.
template <bool CLUSTER>
__device__ __forceinline__ void group_sync() {
    if constexpr (CLUSTER) cg::this_cluster().sync();
    else __syncthreads();
}

// Shared-memory layout (dynamic): filter table [cells] u32 | requests [rpc] u32 | mbarriers [nw * S] | work area.
// The work area is, in turn: phases 1-2 the first and last element of the own rows [2 * rpc] int64 and one array
// of [cells] u32 per slow row in flight; phase 3 the ring [nw * S * (CH + 2)] int64; phase 4 the sort workspace,
// 20 bytes per node of capacity, with the table as per-cell maxima.  The barriers are invalidated when the filter
// pass is over and their bytes are not used for anything else.
template <class SRC, bool CHECK, bool CLUSTER>
__global__ void __launch_bounds__(512, 2) k_range_fused(const SRC src, const FusedParams P, FilterBufs F) {
    grid_dep_wait();
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ uint64_t red[4][16];
    __shared__ uint64_t tmp[34];
    __shared__ InstMeta sm;
    __shared__ SegResult best;
    __shared__ unsigned int scount, sstatus, fill, sflag;
    const int b = blockIdx.y, rank = blockIdx.x, G = gridDim.x;
    const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
    const int n = P.n, R = P.R, rpc = P.rpc, cells = F.cells;
    const int r0 = min(rank * rpc, n), r1 = min(r0 + rpc, n), nrows = r1 - r0;
    const size_t cta = (size_t)b * G + rank;
    const Guard<CHECK> gd{P.dbg, (uint32_t)cta};
#define ZL_STAMP(k) do { if (P.stamps && tid == 0) P.stamps[cta * 16 + (k)] = global_ns(); } while (0)
    ZL_STAMP(0);
    uint32_t *tab = (uint32_t *)smem;
    uint32_t *reqs = tab + cells;
    uint64_t *bars = (uint64_t *)(reqs + ((rpc + 1) & ~1));
    unsigned char *work = (unsigned char *)(((uintptr_t)(bars + (size_t)nw * P.S) + 15) & ~(uintptr_t)15);
    int64_t *ring = (int64_t *)work;
    int64_t *cols = (int64_t *)work;                              // phases 1-2
    uint32_t *arrs = (uint32_t *)(cols + 2 * (size_t)rpc);        // phase 2: [slow rows in flight][cells]
    const size_t work_bytes = P.smem_bytes - (size_t)(work - smem);
    const typename SRC::Rows rows = src.inst(b, n, R);
    constexpr bool arith = std::is_same<SRC, AriBatch>::value;
    const size_t total = (size_t)P.B * n * R;

    if (b == 0 && rank == 0 && tid < 3) F.flags_next[tid] = 0;
    if (!arith && lane == 0) {
        for (int s = 0; s < P.S; ++s) mbar_init(&bars[warp * P.S + s], 1);
        mbar_init_fence();
    }
    if constexpr (!arith) {
        // the first rows of every warp are wanted soon whatever the summary says: start them on their way to the L2
        if (P.vec2 && lane < P.prefetch) {
            const int r = r0 + warp + lane * nw;
            if (r < r1) prefetch_l2_bulk(src.ts + ((size_t)b * n + r) * R, (uint32_t)min(R, 256) * 8u);
        }
    }
    // ---- phase 1: first and last column of the own rows
    {
        uint64_t mn1 = ~0ull, mx1 = 0, mnR = ~0ull, mxR = 0;      // order-preserving unsigned images of int64
        for (int i = tid; i < 2 * nrows; i += nt) {
            const int64_t v = rows.row(r0 + (i >> 1)).at((i & 1) ? R - 1 : 0);
            if (gd.ok((uint64_t)i * 8 + 7, work_bytes, ACC_COLS)) cols[i] = v;
            const uint64_t u = (uint64_t)v ^ (1ull << 63);
            if (i & 1) { mnR = min(mnR, u); mxR = max(mxR, u); } else { mn1 = min(mn1, u); mx1 = max(mx1, u); }
        }
        mn1 = warp_reduce(mn1, OpMin()); mx1 = warp_reduce(mx1, OpMax());
        mnR = warp_reduce(mnR, OpMin()); mxR = warp_reduce(mxR, OpMax());
        if (lane == 0) { red[0][warp] = mn1; red[1][warp] = mx1; red[2][warp] = mnR; red[3][warp] = mxR; }
        __syncthreads();
        if (tid == 0 && gd.ok(cta * 4 + 3, (uint64_t)P.ctas * 4, ACC_PART)) {
            uint64_t a = red[0][0], c = red[1][0], d = red[2][0], e = red[3][0];
            for (int w = 1; w < nw; ++w) { a = min(a, red[0][w]); c = max(c, red[1][w]); d = min(d, red[2][w]); e = max(e, red[3][w]); }
            uint64_t *pp = F.part + cta * 4;
            pp[0] = a; pp[1] = c; pp[2] = d; pp[3] = e;
        }
    }
    ZL_STAMP(1);
    group_sync<CLUSTER>();
    ZL_STAMP(2);
    if (tid == 0) {
        uint64_t a = ~0ull, c = 0, d = ~0ull, e = 0;
        for (int r = 0; r < G; ++r) {
            if (!gd.ok(((size_t)b * G + r) * 4 + 3, (uint64_t)P.ctas * 4, ACC_PART)) continue;
            const uint64_t *pp = F.part + ((size_t)b * G + r) * 4;
            a = min(a, ldcg64(pp)); c = max(c, ldcg64(pp + 1)); d = min(d, ldcg64(pp + 2)); e = max(e, ldcg64(pp + 3));
        }
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
            if (m.use32) {
                // (T - 1) < lmin for every T <= lmin, so ((T - 1) * cscale) >> 32 < cells
                m.cscale = (uint32_t)max((uint64_t)1, min((uint64_t)0xffffffffu, ((uint64_t)cells << 32) / m.lmin));
                m.fscale = (uint32_t)max((uint64_t)1, min((uint64_t)0xffffffffu, ((uint64_t)F.fcells << 32) / m.lmin));
            }
        }
        sm = m;
        scount = 0; sstatus = 0; fill = 0; sflag = 0;
    }
    __syncthreads();
    InstMeta M = sm;
    const bool full = (P.flags & ZL_FLAG_FULL_SWEEP) != 0;
    if (M.status == ZL_OK && M.cscale != 0) {
        // ---- phase 2: partial table from the own slow rows, requests of the own rows, zeroed counters
        const uint32_t cscale = M.cscale, lmin = (uint32_t)M.lmin;
        const int64_t tmin = M.tmin;
        for (int c = tid; c < cells; c += nt) tab[c] = 0;
        {
            uint32_t *cmx = F.cellmax + (size_t)b * F.fcells;
            const int per = (F.fcells + G - 1) / G;
            const int c0 = min(rank * per, F.fcells), c1 = min(c0 + per, F.fcells);
            for (int c = c0 + tid; c < c1; c += nt)
                if (gd.ok((size_t)b * F.fcells + c, (size_t)P.B * F.fcells, ACC_CELLMAX)) cmx[c] = 0;
            if (rank == 0)
                for (int k = tid; k < F.nbk; k += nt)
                    if (gd.ok((size_t)b * F.nbk + k, (size_t)P.B * F.nbk, ACC_BCNT)) F.bcnt[(size_t)b * F.nbk + k] = 0;
        }
        for (int p = tid; p < nrows; p += nt) {
            // how many of the row's elements are expected to be <= lmin (rows are close to arithmetic), with some slack
            const uint64_t e1 = (uint64_t)(cols[2 * p] - tmin) + 1, eR = (uint64_t)(cols[2 * p + 1] - tmin) + 1;
            uint64_t est = R;
            if (eR > e1 && (uint64_t)lmin < eR)
                est = (uint64_t)lmin <= e1 ? 1 : ((uint64_t)lmin - e1) * (uint64_t)(R - 1) / (eR - e1) + 8;
            est = min(est, (uint64_t)R);
            if (gd.ok((uint64_t)p, (uint64_t)rpc, ACC_REQS))
                reqs[p] = !P.vec2 ? 0u : full ? (uint32_t)R : (uint32_t)min((uint64_t)R, (est + 7) & ~(uint64_t)7);
        }
        ZL_STAMP(11);
        // A slow row per group of own rows (the longest span).  Per row an array over the cells: every element of the
        // row up to the first one after lmin marks its cell with itself (the smallest wins); the suffix minimum over
        // the cells is then, per cell, the row's first element at or after the cell's start - which is the `next` of
        // an element before the cell, or the row's first element (<= t0).
        const int K = max(1, min(P.slow, nrows));
        const int gsz = (nrows + K - 1) / K;
        const int per = (cells + 31) / 32;                        // cells per lane of the suffix scan
        const int astride = cells + 32;                           // an array with one padding word per lane: cell c sits at c + c / per
        const size_t arr_room = work_bytes - (size_t)rpc * 16;
        const int kfit = (int)max((size_t)1, min((size_t)K, min((size_t)nw, arr_room / ((size_t)astride * 4))));   // rows in flight
        for (int k0 = 0; k0 < K; k0 += kfit) {
            const int kn = min(kfit, K - k0);
            const int wpg = max(1, nw / kn);                      // warps that share the walk of one row
            __syncthreads();
            for (int c = tid; c < kn * astride; c += nt)
                if (gd.ok((size_t)rpc * 16 + (size_t)c * 4 + 3, work_bytes, ACC_ARR)) arrs[c] = 0xffffffffu;
            __syncthreads();
            const int slot = warp / wpg, part = warp % wpg;
            if (slot < kn) {
                const int gidx = k0 + slot;
                const int p0 = gidx * gsz, p1 = min(p0 + gsz, nrows);
                int bestp = -1;
                uint64_t bspan = 0;
                for (int p = p0 + lane; p < p1; p += 32) {
                    const uint64_t span = (uint64_t)(cols[2 * p + 1] - cols[2 * p]);
                    if (bestp < 0 || span > bspan) { bspan = span; bestp = p; }
                }
                const uint64_t bst = warp_reduce(bspan, OpMax());
                const unsigned who = __ballot_sync(FULL, bestp >= 0 && bspan == bst);
                if (who) {
                    const int row = r0 + __shfl_sync(FULL, bestp, __ffs(who) - 1);
                    const auto rp = rows.row(row);
                    uint32_t *arr = arrs + (size_t)slot * astride;
                    for (int i0 = 128 * part; i0 < R; i0 += 128 * wpg) {
                        uint32_t pv[4], cv[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const int i = i0 + 32 * k + lane;
                            pv[k] = 0xffffffffu; cv[k] = 0;
                            if (i < R) {
                                pv[k] = i > 0 ? (uint32_t)(rp.at(i - 1) - tmin + 1) : 0u;
                                cv[k] = (uint32_t)(rp.at(i) - tmin + 1);
                            }
                        }
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            if (pv[k] <= lmin) {          // also false past the end of the row
                                const uint32_t c = cv[k] <= lmin ? cell_of(cv[k], cscale) : (uint32_t)cells - 1;
                                if (gd.ok(c, (uint64_t)cells, ACC_ARR)) atomicMin(&arr[c + c / per], cv[k]);
                            }
                        }
                        if (__shfl_sync(FULL, pv[3], 0) > lmin) break;    // the rest of the row lies after lmin
                    }
                }
            }
            __syncthreads();
            ZL_STAMP(12);
            // suffix minimum per array, by the row's first warp: lane l owns cells [l * per, (l + 1) * per); the result joins
            // the CTA's table cell by cell, consecutive lanes on consecutive cells
            if (slot < kn && part == 0) {
                uint32_t *arr = arrs + (size_t)slot * astride;
                const int c0 = min(lane * per, cells), c1 = min(c0 + per, cells);
                uint32_t loc = 0xffffffffu;
                for (int c = c1 - 1; c >= c0; --c) loc = min(loc, arr[c + lane]);
                uint32_t suf = loc;                               // minimum over this lane's cells and every later lane's
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const uint32_t y = __shfl_down_sync(FULL, suf, d);
                    if (lane + d < 32) suf = min(suf, y);
                }
                uint32_t run = __shfl_down_sync(FULL, suf, 1);    // ... over every later lane's only
                if (lane == 31) run = 0xffffffffu;
                for (int c = c1 - 1; c >= c0; --c) {
                    run = min(run, arr[c + lane]);
                    arr[c + lane] = run;
                }
                __syncwarp();
                for (int c = lane; c < cells; c += 32) {
                    const uint32_t v = arr[c + c / per];
                    if (v != 0xffffffffu) atomicMax(&tab[c], v);
                }
            }
        }
        __syncthreads();
        ZL_STAMP(13);
        {
            uint32_t *pt = F.ptab + cta * cells;
            for (int c = tid; c < cells; c += nt)
                if (gd.ok(cta * cells + c, (size_t)P.ctas * cells, ACC_PTAB)) pt[c] = tab[c];
        }
    }
    ZL_STAMP(3);
    group_sync<CLUSTER>();
    ZL_STAMP(4);
    bool copies_ok = true;
    if (M.status == ZL_OK && M.cscale != 0) {
        // merged table; dmin: every T of cell c is <= tmax_c, so an element with next - T <= tab[c] - tmax_c for all c never passes
        const uint32_t lmin = (uint32_t)M.lmin;
        const uint32_t wcell = 0xffffffffu / M.cscale + 2;        // a cell spans fewer than wcell time units
        uint32_t dloc = 0xffffffffu;
        for (int c = tid; c < cells; c += nt) {
            uint32_t v = (uint32_t)M.t0;
            uint32_t pvs[8];
#pragma unroll
            for (int r = 0; r < 8; ++r)
                pvs[r] = (r < G && gd.ok(((size_t)b * G + r) * cells + c, (size_t)P.ctas * cells, ACC_PTAB)) ? ldcg32(F.ptab + ((size_t)b * G + r) * cells + c) : 0u;
#pragma unroll
            for (int r = 0; r < 8; ++r) v = max(v, pvs[r]);
            tab[c] = v;
            const uint64_t tmax_c = min((uint64_t)lmin, (uint64_t)(c + 1) * wcell + 1);
            dloc = min(dloc, (uint64_t)v > tmax_c ? (uint32_t)(v - tmax_c) : 0u);
        }
        dloc = warp_reduce(dloc, OpMin());
        uint32_t *rd = (uint32_t *)&red[0][0];
        if (lane == 0) rd[warp] = dloc;
        __syncthreads();
        uint32_t d = 0xffffffffu;
        for (int w = 0; w < nw; ++w) d = min(d, rd[w]);
        M.dmin = d;
        ZL_STAMP(5);
        // ---- phase 3: the filter pass over the own rows
        FCtx<CHECK> C;
        C.tab = tab; C.regcap = (uint32_t)F.regcap;
        C.list = F.list1 + (size_t)b * F.list1cap + (size_t)rank * F.regcap;
        C.cellmax = F.cellmax + (size_t)b * F.fcells; C.scount = &scount;
        C.cscale = M.cscale; C.fscale = M.fscale; C.lmin = lmin; C.dmin = d;
        C.tminlo = (uint32_t)(uint64_t)M.tmin - 1u;               // relative time = low word of t - tminlo
        C.cells = (uint32_t)cells; C.fcells = (uint32_t)F.fcells; C.g = gd;
        if constexpr (arith) {
            filter_rows_arith(C, rows, R, r0, r1, M.tmin, lane, warp, nw);
        } else {
            if (CHECK && !gd.ok((size_t)(warp + 1) * P.S * (P.CH + 2) * 8 - 1, work_bytes, ACC_SLOT)) copies_ok = false;
            else copies_ok = filter_rows_ring(C, src.ts, (size_t)b * n * R, total, R, r0, r1, reqs, ring + (size_t)warp * P.S * (P.CH + 2),
                                              bars + warp * P.S, P.S, P.CH, full, lane, warp, nw);
        }
        if (!copies_ok) atomicMax(&sstatus, (unsigned)ZL_ERR_TIMEOUT);
        if (!arith && lane == 0 && copies_ok)                     // every copy of this warp has landed: its barriers are done with
            for (int s = 0; s < P.S; ++s) mbar_inval(&bars[warp * P.S + s]);
        __syncthreads();
        if (tid == 0) {
            // survivors of this region; beside it whether the list overflowed (bit 0) or a copy did not arrive (bit 1)
            const unsigned c = scount;
            if (gd.ok(cta, (uint64_t)P.ctas, ACC_RCNT)) F.rcnt[cta] = min(c, (unsigned)F.regcap);
            if (gd.ok(cta * 4 + 2, (uint64_t)P.ctas * 4, ACC_PART)) F.part[cta * 4 + 2] = (c > (unsigned)F.regcap ? 1u : 0u) | (sstatus ? 2u : 0u);
        }
    }
    ZL_STAMP(6);
    group_sync<CLUSTER>();
    ZL_STAMP(7);
    // ---- phase 4: CTA 0 finishes the instance when it can
    // sflag: 0 = finished here (best holds the result), 1 = left to the kernels behind this one, 2 = in error
    if (rank == 0) {
        unsigned total_s = 0, over = 0, bad = 0;
        if (M.status == ZL_OK && M.cscale != 0) {
            for (int r = tid; r < G; r += nt) {
                const unsigned fl = (unsigned)ldcg64(F.part + ((size_t)b * G + r) * 4 + 2);
                total_s += ldcg32(F.rcnt + (size_t)b * G + r); over |= fl & 1u; bad |= (fl >> 1) & 1u;
            }
            unsigned tt;
            block_scan_excl<uint32_t>(total_s, OpAdd(), 0u, (uint32_t *)tmp, &tt);
            total_s = tt;
            over = __syncthreads_or((int)over) != 0;
            bad = __syncthreads_or((int)bad) != 0;
        }
        M.count = total_s; M.overflow = over;
        const bool mine = M.status == ZL_OK && handled_by_filter(M, 1) && tail_instance(M) && !bad;
        if (tid == 0) {
            if (bad) M.status = ZL_ERR_TIMEOUT;
            if (gd.ok((uint64_t)b, (uint64_t)P.B, ACC_META)) P.meta[b] = M;
            if (M.status == ZL_OK && !handled_by_filter(M, 1)) F.flags[1] = 1;
            else if (M.status == ZL_OK && !tail_instance(M)) F.flags[0] = 1;
            if (M.status == ZL_OK && !mine) F.flags[2] = 1;
            sflag = mine ? 0u : M.status == ZL_OK ? 1u : 2u;
        }
        if (mine) {
            uint32_t *g = tab;                                    // the table is not needed any more
            Key<uint32_t> *keys = (Key<uint32_t> *)work;               // the ring's place; the barriers in front of it stay untouched
            const int tcap = P.tcap;
            const BatchWS<uint32_t> ws{keys, keys + tcap, (uint32_t *)(keys + 2 * (size_t)tcap), tcap};
            const bool room = gd.ok((size_t)tcap * 20 - 1, (uint64_t)work_bytes, ACC_KEYS);
            __syncthreads();
            for (int c = tid; c < cells; c += nt) g[c] = 0;
            __syncthreads();
            for (int r = warp; r < G; r += nw) {
                const uint32_t c = ldcg32(F.rcnt + (size_t)b * G + r);
                const uint64_t *lst = F.list1 + (size_t)b * F.list1cap + (size_t)r * F.regcap;
                for (uint32_t i = lane; i < c; i += 32) {
                    if (!gd.ok((size_t)b * F.list1cap + (size_t)r * F.regcap + i, (size_t)P.B * F.list1cap, ACC_LIST)) continue;
                    const uint64_t w = ldcg64(lst + i);
                    const uint32_t cc = cell_of((uint32_t)(w >> 32), M.cscale);
                    if (gd.ok(cc, (uint64_t)cells, ACC_TAB)) atomicMax(&g[cc], (uint32_t)w);
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
            for (int r = warp; r < G; r += nw) {
                const uint32_t c = ldcg32(F.rcnt + (size_t)b * G + r);
                const uint64_t *lst = F.list1 + (size_t)b * F.list1cap + (size_t)r * F.regcap;
                for (uint32_t i0 = 0; i0 < c; i0 += 32) {
                    const uint32_t i = i0 + lane;
                    const uint64_t w = i < c ? ldcg64(lst + i) : 0ull;
                    const uint32_t T = (uint32_t)(w >> 32), nx = (uint32_t)w;
                    const uint32_t cc = i < c ? cell_of(T, M.cscale) : 0u;
                    const bool keep = i < c && gd.ok(cc, (uint64_t)cells, ACC_TAB) && nx > max(T, g[cc]);
                    const unsigned km = __ballot_sync(FULL, keep);
                    if (km == 0) continue;
                    unsigned base = 0;
                    if (lane == 0) base = atomicAdd(&fill, (unsigned)__popc(km));
                    base = __shfl_sync(FULL, base, 0);
                    const unsigned pos = base + __popc(km & ((1u << lane) - 1u));
                    if (keep && room && gd.ok(pos, (uint64_t)tcap, ACC_KEYS)) keys[pos].w = w;
                }
            }
            __syncthreads();
            uint64_t bd = ~0ull, bt = ~0ull, cs = 0;
            uint32_t cc = 0;
            if (room) run_batch<uint32_t, ZL_OBJ_RANGE>(ws, (int)min(fill, (unsigned)tcap), (uint32_t)M.t0, n, tmp, (uint32_t)0, cs, cc, bd, bt);
            block_best_to_result(bd, bt, ZL_OK, tmp, &sstatus, best);
            __syncthreads();
            if (tid == 0) {
                const int fst = best.valid ? ZL_OK : ZL_ERR_TIMEOUT;          // a valid instance always has a candidate
                best.status = fst;
                if (gd.ok((size_t)b * P.nres, (size_t)P.B * P.nres, ACC_SEG)) P.seg[(size_t)b * P.nres] = best;
                P.wait[b] = fst == ZL_OK ? (int64_t)best.d : INT64_MIN;
                P.barrier[b] = fst == ZL_OK ? M.tmin + (int64_t)(best.t - 1) + (int64_t)best.d : INT64_MIN;
                if (P.status) P.status[b] = fst;
            }
        } else if (M.status != ZL_OK && tid == 0) {
            P.wait[b] = INT64_MIN; P.barrier[b] = INT64_MIN;
            if (P.status) P.status[b] = M.status;
        }
        if (tid == 0) {
            // what the other CTAs of the cluster need: the state of the instance and, when finished, its barrier
            uint64_t *pp = F.part + (size_t)b * G * 4;
            pp[0] = sflag;
            pp[1] = (sflag == 0 && best.status == ZL_OK) ? (uint64_t)(M.tmin + (int64_t)(best.t - 1) + (int64_t)best.d) : (uint64_t)INT64_MIN;
        }
    }
    ZL_STAMP(8);
    group_sync<CLUSTER>();
    ZL_STAMP(9);
    // ---- phase 5: indices of the own rows
    {
        const uint64_t *pp = F.part + (size_t)b * G * 4;
        const unsigned state = (unsigned)ldcg64(pp);
        const int64_t bar = (int64_t)ldcg64(pp + 1);
        if (state == 1) return;                                   // k_finalize writes this instance's outputs
        for (int p = tid; p < nrows; p += nt) {
            if (!gd.ok((size_t)b * n + r0 + p, (size_t)P.B * n, ACC_IDX)) continue;
            P.idx[(size_t)b * n + r0 + p] = (state == 0 && bar != INT64_MIN) ? last_index_not_after(rows.row(r0 + p), R, bar) : -1;
        }
        ZL_STAMP(10);
    }
#undef ZL_STAMP
}

// Cluster size for a batch of B instances: as many CTAs (of up to 512 threads) per instance as it takes to put about
// two on every SM, at most `gmax`, and never so many that a CTA is left with fewer than 16 rows.
int fused_cluster_size(int B, int n, int num_sms, int gmax) {
    const long long target = (long long)num_sms * 2;
    int G = 1;
    while (G < gmax && (long long)B * G * 2 <= target && n / (G * 2) >= 16) G *= 2;
    return G;
}

template <class SRC>
static cudaError_t enqueue_fused_t(const Pipeline &q, FilterBufs &fb, cudaStream_t st, const SRC &src) {
    int G = fused_cluster_size(q.B, q.n, q.num_sms, 8);
    if (q.cluster) G = std::max(1, std::min(pow2_floor(q.cluster), 8));
    while (G > 1 && ((long long)q.B * G > fb.maxctas || q.n / G < 1)) G /= 2;
    FusedParams P;
    memset(&P, 0, sizeof(P));
    P.n = q.n; P.R = q.R; P.B = q.B; P.flags = q.flags; P.nres = q.nres;
    P.meta = q.meta; P.seg = q.seg; P.idx = q.idx; P.barrier = q.barrier; P.wait = q.wait; P.status = q.status;
    P.rpc = (q.n + G - 1) / G;
    int threads = q.filter_threads ? q.filter_threads : 512;
    threads = std::max(32, std::min(threads, 32 * pow2_ceil(std::max(1, P.rpc))));
    threads = std::min(threads, 512);
    const int nw = threads / 32;
    P.S = q.filter_stages ? std::max(2, std::min(q.filter_stages, 8)) : 3;
    P.CH = q.filter_round >= 128 ? q.filter_round : 256;         // timestamps per ring slot
    P.slow = std::max(1, std::min(FILTER_ROWS / G, std::max(1, P.rpc / 16)));
    P.vec2 = (q.R % 2 == 0) && (((uintptr_t)q.ts & 15) == 0);
    P.prefetch = std::max(0, std::min(q.prefetch_rows, 32));
    fb.nreg = G;
    fb.regcap = fb.list1cap / G;
    P.tcap = (int)std::min<long long>((long long)TAIL_CAP, pow2_ceil(std::max(64, fb.list1cap)));
    const size_t head = (size_t)fb.cells * 4 + (size_t)((P.rpc + 1) & ~1) * 4 + (size_t)nw * P.S * 8 + 16;
    const size_t ring = (size_t)nw * P.S * (P.CH + 2) * 8;
    const size_t table = (size_t)P.rpc * 16 + (size_t)fb.cells * 4;              // columns and one slow row's array
    const size_t tail = (size_t)P.tcap * 20;
    const size_t smem = head + std::max(std::max(ring, table), tail);
    P.smem_bytes = (uint32_t)smem;
    P.ctas = (uint32_t)((size_t)q.B * G);
    P.dbg = fb.dbg;
    P.stamps = fb.dbg ? (unsigned long long *)(fb.dbg + 16) : nullptr;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(G, q.B); cfg.blockDim = dim3(threads); cfg.dynamicSmemBytes = smem; cfg.stream = st;
    // one CTA per instance: an ordinary launch; several: a cluster per instance
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (G > 1) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = G; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = 1;
        ++na;
    }
    if (!((q.pdl_off >> 1) & 1)) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr; cfg.numAttrs = na;
    const bool check = (q.flags & ZL_FLAG_DEBUG_CHECKS) && fb.dbg && !q.checks_off;
    if (G > 1) return check ? cudaLaunchKernelEx(&cfg, k_range_fused<SRC, true, true>, src, P, fb) : cudaLaunchKernelEx(&cfg, k_range_fused<SRC, false, true>, src, P, fb);
    return check ? cudaLaunchKernelEx(&cfg, k_range_fused<SRC, true, false>, src, P, fb) : cudaLaunchKernelEx(&cfg, k_range_fused<SRC, false, false>, src, P, fb);
}

cudaError_t enqueue_fused(const Pipeline &q, FilterBufs &fb, cudaStream_t st, const MatBatch &src) { return enqueue_fused_t(q, fb, st, src); }
cudaError_t enqueue_fused(const Pipeline &q, FilterBufs &fb, cudaStream_t st, const AriBatch &src) { return enqueue_fused_t(q, fb, st, src); }

template <class SRC>
static cudaError_t fused_limits_t() {
    cudaError_t e = cudaFuncSetAttribute(k_range_fused<SRC, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_range_fused<SRC, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_range_fused<SRC, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_range_fused<SRC, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    return e;
}

cudaError_t fused_limits() {
    cudaError_t e = fused_limits_t<MatBatch>();
    if (e == cudaSuccess) e = fused_limits_t<AriBatch>();
    return e;
}

}  // namespace zl
