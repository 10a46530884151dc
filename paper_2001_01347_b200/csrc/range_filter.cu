// The RANGE filter route (see the comment on the filter below for why it is exact), two kernels per call:
//
//   k_range_head    a cluster of G CTAs per instance: column scans of the own rows, the instance summary (tmin, t0,
//                   lmin, span), per row the number of leading timestamps the filter pass will ask for, a partial
//                   filter table from the own slow rows; CTA 0 merges the partial tables, derives dmin and leaves
//                   summary and table in global memory.  The CTAs exchange through global scratch; the cluster's
//                   hardware barrier orders it.
//   k_range_filter  many small CTAs, each with a block of an instance's rows: a warp per row, the row's leading
//                   timestamps arrive in a per-warp ring of shared-memory slots (16-byte asynchronous copies by every
//                   lane for the short prefixes of the early stop, one bulk-copy request per 4 KB chunk counted on an
//                   mbarrier for whole rows); 128 timestamps a step are tested against dmin, the few candidates
//                   against the table; survivors go to the CTA's list.  The CTA that finishes an instance's last block
//                   also finishes the instance when it has few survivors (refine, sort, prefix max, evaluate, first
//                   minimum); nobody waits for anybody.
// Instances with many survivors, with a time span of 2^32 or more, or with a full list are left to the kernels of
// heavy.cu and sweep.cu; k_finalize recovers the indices of every instance.
//
// The filter.  For the RANGE objective an element e matters only if next(e) > G(T(e)), where
// G(t) = max(t, t0, max{next(e') : T(e') < t}) is max(Z) of the best Z whose minimum is at time t:
//   - if next(e) <= G(T(e)) the element cannot raise the running maximum, so PM of every later element is unchanged
//     without it;
//   - and it is not needed as a candidate: moving min(Z) from e to the next element in time keeps max(Z) and shrinks
//     d_Z (or, among equal times, another element of the group qualifies).
// Any lower bound L(t) <= G(t) therefore gives an exact filter "keep e iff next(e) > max(T, L(T))".  The table holds,
// per time cell c, L = max(t0, max over a few slow rows p of the first element of p at or after the cell's start) -
// every such element is next(e') of an element before the cell, or a first element (<= t0).  Slow rows (long
// iterations) are the ones that set G most of the time.
//
// With CHECK on (ZL_FLAG_DEBUG_CHECKS) every computed index into global or shared memory and every copy request is
// tested against the extent of its buffer first; a violation is recorded (which access, which CTA, the index; the
// first one wins) and the access is skipped, so a wrong index is reported instead of faulting.
#include <cooperative_groups.h>

#include "zl_batch.cuh"
#include "zl_guard.cuh"
#include "zl_host.h"

namespace cg = cooperative_groups;

namespace zl {

struct RangeParams {
    int n, R, B, flags, rpc, S, CH, tcap, slow, nres, vec2, bulk, nreg;    // rpc: rows per CTA of the kernel at hand
    InstMeta *meta; SegResult *seg;
    int32_t *idx; int64_t *barrier; int64_t *wait; int32_t *status;
    uint32_t *dbg;                       // CHECK: [0] code of the first violation, [1] its CTA, [2..3] the index
    unsigned long long *stamps;          // debug handles: [ctas][16] nanosecond clock at the phase boundaries of every CTA
    uint32_t smem_bytes, ctas;           // of the kernel at hand
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
// successor of the row's last element is infinite.  Returns the time of the last of them that belongs to the request.
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
    const int last = min(63, lim - 1 - (i0 + off));               // the last of the 64 that belongs to the request
    return __shfl_sync(FULL, (last & 1) ? Tb : Ta, last >> 1);
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

// The four elements of a lane (time T[j], successor nx[j]; ok bit j: the element counts) against dmin and, those that
// pass, against the table; the survivors of the warp are appended together: one counter update a warp, whatever their
// number.  Every lane of the warp calls.
template <bool CHECK>
__device__ __forceinline__ void filter_quad(const FCtx<CHECK> &c, int lane, const uint32_t (&T)[4], const uint32_t (&nx)[4], unsigned okmask) {
    // cheap necessary condition first: most elements belong to fast workers and stop here
    bool k[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) k[j] = ((okmask >> j) & 1u) && T[j] <= c.lmin && nx[j] - T[j] > c.dmin;
    if (!__any_sync(FULL, k[0] | k[1] | k[2] | k[3])) return;
#pragma unroll
    for (int j = 0; j < 4; ++j)
        if (k[j]) { const uint32_t cc = cell_of(T[j], c.cscale); k[j] = c.g.ok(cc, c.cells, ACC_TAB) && nx[j] > max(T[j], c.tab[cc]); }
    if (!__any_sync(FULL, k[0] | k[1] | k[2] | k[3])) return;
    unsigned m[4];
    int tot = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) { m[j] = __ballot_sync(FULL, k[j]); tot += __popc(m[j]); }
    unsigned base = 0;
    if (lane == 0) base = atomicAdd(c.scount, (unsigned)tot);
    base = __shfl_sync(FULL, base, 0);
    const unsigned below = (1u << lane) - 1u;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        if (k[j]) {
            const unsigned pos = base + __popc(m[j] & below);
            if (pos < c.regcap) c.list[pos] = ((uint64_t)T[j] << 32) | nx[j];
            const uint32_t fc = cell_of(T[j], c.fscale);
            if (c.g.ok(fc, c.fcells, ACC_CELLMAX)) atomicMax(&c.cellmax[fc], nx[j]);
        }
        base += __popc(m[j]);
    }
}

// Table test of the (up to) two elements of a lane, for the plain-load paths.
template <bool CHECK>
__device__ __forceinline__ void filter_pair(const FCtx<CHECK> &c, int lane, bool va, uint32_t Ta, uint32_t na, bool vb, uint32_t Tb, uint32_t nb) {
    const uint32_t T[4] = {Ta, Tb, 0u, 0u}, nx[4] = {na, nb, 0u, 0u};
    filter_quad(c, lane, T, nx, (va ? 1u : 0u) | (vb ? 2u : 0u));
}

// Up to 128 timestamps of a slot starting at slot[off] = element i0 + off of the row, of which those below `lim` (the
// end of what was requested of the row, <= R) count: lane l holds elements 2l, 2l + 1, 64 + 2l and 65 + 2l of them,
// each one's successor from the slot itself (the element after the slot's last one sits right behind it; the row's
// last element has none).  Returns the time of the last of them that belongs to the request.
template <bool CHECK>
__device__ __forceinline__ uint32_t filter_partial(const FCtx<CHECK> &C, const int64_t *slot, int off, int i0, int lim, int R, int lane) {
    const int i = i0 + off + 2 * lane;
    const bool second = i0 + off + 64 < lim;                      // the same in every lane
    const longlong2 p0 = *reinterpret_cast<const longlong2 *>(slot + off + 2 * lane);
    uint32_t T[4], nx[4];
    T[0] = i < lim ? (uint32_t)(uint64_t)p0.x - C.tminlo : 0xffffffffu;
    T[1] = i + 1 < lim ? (uint32_t)(uint64_t)p0.y - C.tminlo : 0xffffffffu;
    nx[0] = i + 1 < R ? (uint32_t)(uint64_t)p0.y - C.tminlo : 0xffffffffu;
    nx[1] = i + 2 < R ? (uint32_t)(uint64_t)slot[off + 2 * lane + 2] - C.tminlo : 0xffffffffu;
    T[2] = T[3] = 0xffffffffu; nx[2] = nx[3] = 0xffffffffu;
    unsigned okmask = (i < lim ? 1u : 0u) | (i + 1 < lim ? 2u : 0u);
    if (second) {
        const longlong2 p1 = *reinterpret_cast<const longlong2 *>(slot + off + 64 + 2 * lane);
        T[2] = i + 64 < lim ? (uint32_t)(uint64_t)p1.x - C.tminlo : 0xffffffffu;
        T[3] = i + 65 < lim ? (uint32_t)(uint64_t)p1.y - C.tminlo : 0xffffffffu;
        nx[2] = i + 65 < R ? (uint32_t)(uint64_t)p1.y - C.tminlo : 0xffffffffu;
        nx[3] = i + 66 < R ? (uint32_t)(uint64_t)slot[off + 64 + 2 * lane + 2] - C.tminlo : 0xffffffffu;
        okmask |= (i + 64 < lim ? 4u : 0u) | (i + 65 < lim ? 8u : 0u);
    }
    filter_quad(C, lane, T, nx, okmask);
    // the last of the 128 that belongs to the request (the caller passes at least one): whether the row has passed lmin is
    // decided by a real element, never by the filler behind the request's end
    const int last = min(127, lim - 1 - (i0 + off));
    const int l64 = last & 63;
    const uint32_t v = last >= 64 ? ((l64 & 1) ? T[3] : T[2]) : ((l64 & 1) ? T[1] : T[0]);
    return __shfl_sync(FULL, v, l64 >> 1);
}

// 128 timestamps of a slot, with the one after them, that lie inside the row and the request: no bounds checks.
// Returns the time of the last of the 128.
template <bool CHECK>
__device__ __forceinline__ uint32_t filter_inside(const FCtx<CHECK> &C, const int64_t *slot, int lane) {
    const longlong2 p0 = *reinterpret_cast<const longlong2 *>(slot + 2 * lane);
    const longlong2 p1 = *reinterpret_cast<const longlong2 *>(slot + 64 + 2 * lane);
    uint32_t T[4], nx[4];
    T[0] = (uint32_t)(uint64_t)p0.x - C.tminlo; T[1] = (uint32_t)(uint64_t)p0.y - C.tminlo;
    T[2] = (uint32_t)(uint64_t)p1.x - C.tminlo; T[3] = (uint32_t)(uint64_t)p1.y - C.tminlo;
    nx[0] = T[1]; nx[1] = (uint32_t)(uint64_t)slot[2 * lane + 2] - C.tminlo;
    nx[2] = T[3]; nx[3] = (uint32_t)(uint64_t)slot[64 + 2 * lane + 2] - C.tminlo;
    filter_quad(C, lane, T, nx, 0xfu);
    return __shfl_sync(FULL, T[3], 31);
}

// The filter pass of one warp over stored rows of the CTA (rows first, first + step, ... of the instance `inst`, nown
// of them; reqs[j] belongs to the j-th): the warp's rows, every nw-th of the CTA's, through a private ring of RING_STAGES slots of RING_CHUNK
// timestamps, filled by 16-byte asynchronous copies of every lane (8-byte copies when the rows cannot take those).
// In rounds of up to 32 rows lane j holds the request of the round's j-th row, i.e. how many of its leading
// timestamps go through the ring; nothing the loop waits for is loaded inside it.
constexpr int RING_STAGES = 3;
constexpr int RING_CHUNK = 256;
constexpr int RING_SLOT = RING_CHUNK + 2;                         // + the successor of the slot's last element, + padding
template <bool CHECK>
__device__ void filter_rows_async(const FCtx<CHECK> &C, const int64_t *inst, int R, int first, int step, int nown, const uint32_t *reqs, int64_t *ring,
                                  bool vec2, bool full, int lane, int warp, int nw) {
    const size_t rstride = (size_t)nw * step * R;                 // between consecutive rows of this warp
    for (int jbase = warp; jbase < nown; jbase += 32 * nw) {
        const int nrows = min(32, (nown - jbase + nw - 1) / nw);
        int req = 0;
        if (lane < nrows) req = full ? R : min(R, (int)reqs[jbase + lane * nw]);
        const int64_t *row_i = inst + (size_t)(first + jbase * step) * R, *row_p = row_i;
        int ji = 0, ci = 0, jp = 0, cp = 0, inflight = 0, slot_i = 0, slot_p = 0;
        int req_i = __shfl_sync(FULL, req, 0), req_p = req_i;
        bool finished = false;                                     // the row being processed needs nothing more
        while (jp < nrows) {
            while (inflight < RING_STAGES && ji < nrows) {
                int64_t *slot = ring + (size_t)slot_i * RING_SLOT;
                const int base = ci * RING_CHUNK;
                const int i = base + 2 * lane;
                if (vec2) {
#pragma unroll
                    for (int k = 0; k < RING_CHUNK / 64; ++k)
                        if (i + 64 * k < req_i) cp_async16(slot + 64 * k + 2 * lane, row_i + i + 64 * k);
                } else {
#pragma unroll
                    for (int k = 0; k < RING_CHUNK / 32; ++k) {
                        const int e = i + (k >> 1) * 64 + (k & 1);
                        if (e < req_i) cp_async8(slot + (k >> 1) * 64 + 2 * lane + (k & 1), row_i + e);
                    }
                }
                // the element after the last one copied into this slot (its successor)
                const int endi = min(base + RING_CHUNK, req_i);
                if (lane == 31 && endi < R) cp_async8(slot + (endi - base), row_i + endi);
                cp_async_commit();
                ++inflight;
                slot_i = slot_i + 1 == RING_STAGES ? 0 : slot_i + 1;
                if (endi == req_i) {
                    ci = 0; ++ji; row_i += rstride;
                    req_i = __shfl_sync(FULL, req, min(ji, 31));
                } else {
                    ++ci;
                }
            }
            cp_async_wait_pending(inflight - 1);
            __syncwarp();
            const int i0 = cp * RING_CHUNK;
            const int L = min(RING_CHUNK, req_p - i0);             // timestamps of the row in this slot
            if (!finished) {
                const int64_t *slot = ring + (size_t)slot_p * RING_SLOT;
                uint32_t lastT = 0;
#pragma unroll
                for (int sub = 0; sub < RING_CHUNK; sub += 128) {
                    if (sub >= L || (sub && !full && lastT > C.lmin)) break;   // rows are sorted: the rest is past lmin
                    if (sub + 128 <= L && i0 + sub + 128 < R) {
                        lastT = filter_inside(C, slot + sub, lane);
                    } else {
                        lastT = filter_partial(C, slot, sub, i0, req_p, R, lane);
                    }
                }
                finished = !full && lastT > C.lmin;                // rows are sorted: nothing later is <= lmin
            }
            __syncwarp();
            --inflight;
            slot_p = slot_p + 1 == RING_STAGES ? 0 : slot_p + 1;
            if (i0 + L == req_p) {
                // the request ended before the row did (the requests are estimates): continue with plain loads
                if (!finished && !full && req_p < R) filter_plain(C, row_p, req_p, R, full, lane);
                cp = 0; ++jp; row_p += rstride; finished = false;
                req_p = __shfl_sync(FULL, req, min(jp, 31));
            } else {
                ++cp;
            }
        }
    }
}

// The same pass with bulk copies: a row's leading reqs[p] timestamps arrive in chunks of CH through the warp's ring of S
// shared-memory slots, one request to the copy engine per chunk, issued by lane 0 and counted on the slot's mbarrier;
// lane s remembers which row and chunk slot s holds.  (A request of 2 KB or less costs the copy engine about as much as
// one of 4 KB, and the prefix of a row that the early stop asks for is mostly that short: this variant is the slower one
// there and is kept as an option.)  Returns false when a copy did not arrive within the poll limit.
template <bool CHECK>
__device__ bool filter_rows_ring(const FCtx<CHECK> &C, const int64_t *ts, size_t inst_off, size_t total, int R, int first, int step, int nrows,
                                 const uint32_t *reqs, unsigned int *next_row, int64_t *ring, uint64_t *bars, int S, int CH, bool full,
                                 int lane) {
    const int slot_elems = CH + 2;
    const int64_t *inst = ts + inst_off;
    uint32_t phase = 0;                                           // bit s: parity of slot s's next completion
    bool ok = true, pdone = false;
    int prow = -1, preq = 0, pbase = 0;                           // producer: the row being requested, its request, the next chunk's start
    int inflight = 0, si = 0, sp = 0;
    int mrow = 0, mbase = 0;                                      // lane s < S: row and chunk start of slot s
    int fin_row = -1;                                             // a row that has passed lmin: its remaining chunks are only waited for
    for (;;) {
        while (inflight < S && !pdone) {
            if (prow < 0 || pbase >= preq) {
                int r = 0;
                if (lane == 0) r = (int)atomicAdd(next_row, 1u);
                r = __shfl_sync(FULL, r, 0);
                if (r >= nrows) { pdone = true; break; }
                prow = r; preq = (int)reqs[r]; pbase = 0;
                if (preq == 0) {                                  // plain loads, right away
                    filter_plain(C, inst + (size_t)(first + r * step) * R, 0, R, full, lane);
                    prow = -1;
                    continue;
                }
            }
            const int endi = min(pbase + CH, preq);
            if (lane == 0) {
                const uint32_t bytes = (uint32_t)(min(endi + 2, R) - pbase) * 8u;   // the chunk and the element after it
                const size_t src = inst_off + (size_t)(first + prow * step) * R + pbase;
                bool go = true;
                if (CHECK)
                    go = C.g.ok(src + bytes / 8 - 1, total, ACC_COPY_SRC) && C.g.ok(bytes / 8 - 1, (uint64_t)slot_elems, ACC_COPY_DST) &&
                         C.g.ok((bytes & 15u) | (uint32_t)((uintptr_t)(ts + src) & 15u) | (uint32_t)(bytes == 0), 1, ACC_COPY_ALIGN);
                fence_proxy_async();
                mbar_expect_tx(&bars[si], go ? bytes : 0u);
                if (go) bulk_copy_g2s(ring + (size_t)si * slot_elems, ts + src, bytes, &bars[si]);
            }
            if (lane == si) { mrow = prow; mbase = pbase; }
            ++inflight;
            si = si + 1 == S ? 0 : si + 1;
            pbase = endi;
        }
        if (inflight == 0) break;
        const int row = __shfl_sync(FULL, mrow, sp), i0 = __shfl_sync(FULL, mbase, sp);
        const int req = (int)reqs[row];
        if (ok && !mbar_wait_bounded(&bars[sp], (phase >> sp) & 1u)) ok = false;
        phase ^= 1u << sp;
        const int L = min(CH, req - i0);
        bool finished = row == fin_row;
        if (!finished && ok) {
            const int64_t *slot = ring + (size_t)sp * slot_elems;
            uint32_t lastT = 0;
            for (int sub = 0; sub < L; sub += 128) {
                if (sub && !full && lastT > C.lmin) break;        // rows are sorted: the rest is past lmin
                if (sub + 128 <= L && i0 + sub + 128 < R) {
                    lastT = filter_128(C, slot + sub, lane);
                } else {
                    lastT = filter_64(C, slot, sub, i0, req, R, lane);
                    if (sub + 64 < L && (full || lastT <= C.lmin)) lastT = filter_64(C, slot, sub + 64, i0, req, R, lane);
                }
            }
            if (!full && lastT > C.lmin) { finished = true; fin_row = row; }
        }
        __syncwarp();
        --inflight;
        sp = sp + 1 == S ? 0 : sp + 1;
        // the row's request is used up: a row that has not passed lmin yet continues with plain loads
        if (i0 + L >= req && !finished && ok && req < R) filter_plain(C, inst + (size_t)(first + row * step) * R, req, R, full, lane);
    }
    return ok;
}

// The filter pass on predicted rows e_i = last + (i + 1) * interval: a row whose interval does not exceed dmin is
// settled at once (only its last element, whose next is infinite, can pass); the others are walked up to lmin.
template <bool CHECK>
__device__ void filter_rows_arith(const FCtx<CHECK> &C, const AriRows &rows, int R, int first, int step, int nrows, int64_t tmin, int lane, int warp, int nw) {
    for (int j = warp; j < nrows; j += nw) {
        const AriRow rw = rows.row(first + j * step);
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

// Barrier over the CTAs of an instance: the cluster's hardware barrier (it also orders their global writes), or,
// when one CTA has the instance to itself and the launch is an ordinary one, the CTA barrier.
template <bool CLUSTER>
__device__ __forceinline__ void group_sync() {
    if constexpr (CLUSTER) cg::this_cluster().sync();
    else __syncthreads();
}

// k_range_head.  Dynamic shared memory: partial / merged table [cells] u32 | first and last element of the own rows
// [2 * rpc] int64 | one array of [cells + 32] u32 per slow row in flight.
template <class SRC, bool CHECK, bool CLUSTER>
__global__ void __launch_bounds__(512, 2) k_range_head(const SRC src, const RangeParams P, FilterBufs F) {
    grid_dep_wait();
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ uint64_t red[4][16];
    __shared__ InstMeta sm;
    const int b = blockIdx.y, rank = blockIdx.x, G = gridDim.x;
    const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
    const int n = P.n, R = P.R, rpc = P.rpc, cells = F.cells;
    const int r0 = min(rank * rpc, n), r1 = min(r0 + rpc, n), nrows = r1 - r0;
    const size_t cta = (size_t)b * G + rank;
    const Guard<CHECK> gd{P.dbg, (uint32_t)cta};
#define ZL_STAMP(k) do { if (P.stamps && tid == 0) P.stamps[cta * 16 + (k)] = global_ns(); } while (0)
    ZL_STAMP(0);
    uint32_t *tab = (uint32_t *)smem;
    int64_t *cols = (int64_t *)(tab + cells);
    uint32_t *arrs = (uint32_t *)(cols + 2 * (size_t)rpc);
    const size_t work_bytes = P.smem_bytes - (size_t)((unsigned char *)arrs - smem);
    const typename SRC::Rows rows = src.inst(b, n, R);

    if (b == 0 && rank == 0 && tid < 8) { F.flags[tid] = 0; F.flags_next[tid] = 0; }
    // ---- first and last column of the own rows; the CTAs of the cluster exchange their minima and maxima
    {
        uint64_t mn1 = ~0ull, mx1 = 0, mnR = ~0ull, mxR = 0;      // order-preserving unsigned images of int64
        for (int i = tid; i < 2 * nrows; i += nt) {
            const int64_t v = rows.row(r0 + (i >> 1)).at((i & 1) ? R - 1 : 0);
            if (gd.ok((uint64_t)i, (uint64_t)2 * rpc, ACC_COLS)) cols[i] = v;
            const uint64_t u = (uint64_t)v ^ (1ull << 63);
            if (i & 1) { mnR = min(mnR, u); mxR = max(mxR, u); } else { mn1 = min(mn1, u); mx1 = max(mx1, u); }
        }
        mn1 = warp_reduce(mn1, OpMin()); mx1 = warp_reduce(mx1, OpMax());
        mnR = warp_reduce(mnR, OpMin()); mxR = warp_reduce(mxR, OpMax());
        if (lane == 0) { red[0][warp] = mn1; red[1][warp] = mx1; red[2][warp] = mnR; red[3][warp] = mxR; }
        __syncthreads();
        if (tid < 4) {
            // thread k folds quantity k over the warps (minima for k = 0, 2; maxima for k = 1, 3)
            uint64_t a = red[tid][0];
            for (int w = 1; w < nw; ++w) a = (tid & 1) ? max(a, red[tid][w]) : min(a, red[tid][w]);
            red[tid][0] = a;
            if (CLUSTER && gd.ok(cta * 4 + tid, (uint64_t)P.ctas * 4, ACC_PART)) F.part[cta * 4 + tid] = a;
        }
    }
    ZL_STAMP(1);
    group_sync<CLUSTER>();
    if (CLUSTER) {
        // the partial values of every CTA of the cluster, one load per thread
        if (tid < 4 * G) {
            const int r = tid >> 2, k = tid & 3;
            red[k][r] = gd.ok(((size_t)b * G + r) * 4 + k, (uint64_t)P.ctas * 4, ACC_PART) ? ldcg64(F.part + ((size_t)b * G + r) * 4 + k) : ((k & 1) ? 0ull : ~0ull);
        }
        __syncthreads();
    }
    if (tid == 0) {
        uint64_t a = red[0][0], c = red[1][0], d = red[2][0], e = red[3][0];
        if (CLUSTER)
            for (int r = 1; r < G; ++r) { a = min(a, red[0][r]); c = max(c, red[1][r]); d = min(d, red[2][r]); e = max(e, red[3][r]); }
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
    }
    __syncthreads();
    ZL_STAMP(2);
    InstMeta M = sm;
    const bool full = (P.flags & ZL_FLAG_FULL_SWEEP) != 0;
    const bool routed = M.status == ZL_OK && M.cscale != 0;
    if (routed) {
        // ---- requests of the own rows, zeroed counters, partial table from the own slow rows
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
            if (gd.ok((size_t)b * n + r0 + p, (size_t)P.B * n, ACC_REQS))
                F.rowhint[(size_t)b * n + r0 + p] = full ? (uint32_t)R : (uint32_t)min((uint64_t)R, (est + 7) & ~(uint64_t)7);
        }
        ZL_STAMP(11);
        // A slow row per group of own rows (the longest span).  Per row an array over the cells: every element of the
        // row up to the first one after lmin marks its cell with itself (the smallest wins); the suffix minimum over
        // the cells is then, per cell, the row's first element at or after the cell's start.
        const int K = max(1, min(P.slow, nrows));
        const int gsz = (nrows + K - 1) / K;
        const int per = (cells + 31) / 32;                        // cells per lane of the suffix scan (a power of two)
        const int pshift = __ffs(per) - 1;
        const int astride = cells + 32;                           // an array with one padding word per lane: cell c sits at c + c / per
        const int kfit = (int)max((size_t)1, min((size_t)K, min((size_t)nw, work_bytes / ((size_t)astride * 4))));   // rows in flight
        for (int k0 = 0; k0 < K; k0 += kfit) {
            const int kn = min(kfit, K - k0);
            const int wpg = max(1, nw / kn);                      // warps that share the walk of one row
            __syncthreads();
            for (int c = tid; c < kn * astride; c += nt)
                if (gd.ok((size_t)c * 4 + 3, work_bytes, ACC_ARR)) arrs[c] = 0xffffffffu;
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
                                if (gd.ok(c, (uint64_t)cells, ACC_ARR)) atomicMin(&arr[c + (c >> pshift)], cv[k]);
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
#pragma unroll 4
                for (int c = c1 - 1; c >= c0; --c) loc = min(loc, arr[c + lane]);
                uint32_t suf = loc;                               // minimum over this lane's cells and every later lane's
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const uint32_t y = __shfl_down_sync(FULL, suf, d);
                    if (lane + d < 32) suf = min(suf, y);
                }
                uint32_t run = __shfl_down_sync(FULL, suf, 1);    // ... over every later lane's only
                if (lane == 31) run = 0xffffffffu;
#pragma unroll 4
                for (int c = c1 - 1; c >= c0; --c) {
                    run = min(run, arr[c + lane]);
                    arr[c + lane] = run;
                }
                __syncwarp();
                const int cstart = (slot * (cells / 8)) & (cells - 1);      // the rows' warps start at different cells
#pragma unroll 4
                for (int j = lane; j < cells; j += 32) {
                    const int c = (j + cstart) & (cells - 1);
                    const uint32_t v = arr[c + (c >> pshift)];
                    if (v != 0xffffffffu) atomicMax(&tab[c], v);
                }
            }
        }
        __syncthreads();
        ZL_STAMP(13);
        if (CLUSTER && rank != 0) {
            uint32_t *pt = F.ptab + cta * cells;
            for (int c = tid; c < cells; c += nt)
                if (gd.ok(cta * cells + c, (size_t)P.ctas * cells, ACC_PTAB)) pt[c] = tab[c];
        }
    }
    ZL_STAMP(3);
    group_sync<CLUSTER>();
    ZL_STAMP(4);
    if (rank != 0) return;
    // ---- CTA 0: merged table, dmin, the instance's record
    if (routed) {
        // dmin: every T of cell c is <= tmax_c, so an element with next - T <= tab[c] - tmax_c for all c never passes
        const uint32_t lmin = (uint32_t)M.lmin;
        const uint32_t wcell = 0xffffffffu / M.cscale + 2;        // a cell spans fewer than wcell time units
        uint32_t dloc = 0xffffffffu;
        uint32_t *tg = F.table + (size_t)b * cells;
        for (int c = tid; c < cells; c += nt) {
            uint32_t v = max((uint32_t)M.t0, tab[c]);
            if (CLUSTER) {
                uint32_t pvs[8];
#pragma unroll
                for (int r = 1; r < 8; ++r)
                    pvs[r] = (r < G && gd.ok(((size_t)b * G + r) * cells + c, (size_t)P.ctas * cells, ACC_PTAB)) ? ldcg32(F.ptab + ((size_t)b * G + r) * cells + c) : 0u;
#pragma unroll
                for (int r = 1; r < 8; ++r) v = max(v, pvs[r]);
            }
            tg[c] = v;
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
    }
    if (tid == 0) {
        if (gd.ok((uint64_t)b, (uint64_t)P.B, ACC_META)) P.meta[b] = M;
        F.done[b] = 0;
    }
    ZL_STAMP(5);
#undef ZL_STAMP
}

// k_range_filter.  grid (regions, B).  Dynamic shared memory: filter table [cells] u32 | requests of the own rows [rpc]
// u32 | mbarriers [nw * S] | the warps' rings.
template <class SRC, bool CHECK>
__global__ void __launch_bounds__(256, 4) k_range_filter(const SRC src, const RangeParams P, FilterBufs F) {
    grid_dep_wait();
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ uint64_t tmp[34];
    __shared__ unsigned int scount, sstatus, next_row;
    const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
    const int n = P.n, R = P.R, rpc = P.rpc, cells = F.cells;
    const int b = blockIdx.y, reg = blockIdx.x, nreg = gridDim.x;
    // the CTA's rows: reg, reg + nreg, ... - neighbouring rows often belong to workers of one kind, so every CTA of an
    // instance gets its share of each kind
    const int nrows = reg < n ? (n - reg + nreg - 1) / nreg : 0;
    const size_t cta = (size_t)b * nreg + reg;
    const Guard<CHECK> gd{P.dbg, (uint32_t)cta};
    uint32_t *tab = (uint32_t *)smem;
    uint32_t *reqs = tab + cells;
    uint64_t *bars = (uint64_t *)(reqs + ((rpc + 1) & ~1));
    unsigned char *work = (unsigned char *)(((uintptr_t)(bars + (size_t)nw * P.S) + 15) & ~(uintptr_t)15);
    int64_t *ring = (int64_t *)work;
    const size_t work_bytes = P.smem_bytes - (size_t)(work - smem);
    const typename SRC::Rows rows = src.inst(b, n, R);
    constexpr bool arith = std::is_same<SRC, AriBatch>::value;
    const size_t total = (size_t)P.B * n * R;
    const bool full = (P.flags & ZL_FLAG_FULL_SWEEP) != 0;
#define ZL_STAMP(k) do { if (P.stamps && tid == 0) P.stamps[((size_t)F.maxctas + cta) * 16 + (k)] = global_ns(); } while (0)
    ZL_STAMP(0);

    if (tid == 0) { scount = 0; sstatus = 0; next_row = 0; }
    if (!arith && P.bulk && lane == 0) {
        for (int s = 0; s < P.S; ++s) mbar_init(&bars[warp * P.S + s], 1);
        mbar_init_fence();
    }
    // the instance's record, its table and the own rows' requests in one round of loads (the table and the requests of
    // an instance that does not take the route are not used)
    InstMeta M = load_meta_cg(P.meta + b);
    {
        const uint32_t *tg = F.table + (size_t)b * cells;
        for (int c = tid; c < cells; c += nt) tab[c] = tg[c];
        for (int p = tid; p < nrows; p += nt)
            if (gd.ok((uint64_t)p, (uint64_t)rpc, ACC_REQS)) reqs[p] = F.rowhint[(size_t)b * n + reg + (size_t)p * nreg];
    }
    __syncthreads();
    const bool routed = M.status == ZL_OK && M.cscale != 0;
    if (routed) {
        ZL_STAMP(1);
        // ---- the filter pass over the own rows
        FCtx<CHECK> C;
        C.tab = tab; C.regcap = (uint32_t)F.regcap;
        C.list = F.list1 + (size_t)b * F.list1cap + (size_t)reg * F.regcap;
        C.cellmax = F.cellmax + (size_t)b * F.fcells; C.scount = &scount;
        C.cscale = M.cscale; C.fscale = M.fscale; C.lmin = (uint32_t)M.lmin; C.dmin = M.dmin;
        C.tminlo = (uint32_t)(uint64_t)M.tmin - 1u;               // relative time = low word of t - tminlo
        C.cells = (uint32_t)cells; C.fcells = (uint32_t)F.fcells; C.g = gd;
        bool copies_ok = true;
        if constexpr (arith) {
            filter_rows_arith(C, rows, R, reg, nreg, nrows, M.tmin, lane, warp, nw);
        } else {
            if (!P.bulk)
                filter_rows_async(C, src.ts + (size_t)b * n * R, R, reg, nreg, nrows, reqs, ring + (size_t)warp * RING_STAGES * RING_SLOT, P.vec2 != 0, full, lane, warp, nw);
            else if (CHECK && !gd.ok((size_t)(warp + 1) * P.S * (P.CH + 2) * 8 - 1, work_bytes, ACC_SLOT)) copies_ok = false;
            else
                copies_ok = filter_rows_ring(C, src.ts, (size_t)b * n * R, total, R, reg, nreg, nrows, reqs, &next_row,
                                             ring + (size_t)warp * P.S * (P.CH + 2), bars + warp * P.S, P.S, P.CH, full, lane);
        }
        if (!copies_ok) atomicMax(&sstatus, (unsigned)ZL_ERR_TIMEOUT);
        if (!arith && P.bulk && lane == 0 && copies_ok)           // every copy of this warp has landed: its barriers are done with
            for (int s = 0; s < P.S; ++s) mbar_inval(&bars[warp * P.S + s]);
        __syncthreads();
    }
    // ---- the block is done: its count, and its share of the instance's
    ZL_STAMP(2);
    if (tid == 0) {
        const unsigned c = routed ? scount : 0u;
        if (gd.ok(cta, (uint64_t)P.ctas, ACC_RCNT)) F.rcnt[cta] = min(c, (unsigned)F.regcap);
        if (gd.ok((uint64_t)b, (uint64_t)P.B, ACC_META)) {
            if (c > (unsigned)F.regcap) P.meta[b].overflow = 1;  // the list is cut short: the segment sweep takes the instance
            if (c) atomicAdd(&P.meta[b].count, c);
            if (sstatus) P.meta[b].status = (int32_t)sstatus;     // a copy did not arrive
        }
    }
#undef ZL_STAMP
}

// k_range_tail.  grid (B), up to 1024 threads.  Finishes the instances that the filter pass left with few survivors
// (at most TAIL_CAP): the maximum of `next` per coarse cell gives G at the cell starts, which removes most of what
// is left; the rest is sorted and swept in one batch, and the instance's outputs - barrier, wait, status and the
// per-worker indices - are written right here.  It also raises the call's flags for the instances it leaves to the
// kernels behind it.  Dynamic shared memory: per-cell maxima [cells] u32 | sort workspace (20 bytes per node).
template <class SRC, bool CHECK>
__global__ void __launch_bounds__(1024, 1) k_range_tail(const SRC src, const RangeParams P, FilterBufs F) {
    grid_dep_wait();
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ uint64_t tmp[34];
    __shared__ unsigned int sstatus, fill;
    __shared__ SegResult best;
    const int b = blockIdx.x, tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
    const int n = P.n, R = P.R, cells = F.cells, tcap = P.tcap;
    const Guard<CHECK> gd{P.dbg, (uint32_t)b};
    const InstMeta M = P.meta[b];
    const bool mine = M.status == ZL_OK && handled_by_filter(M, 1) && tail_instance(M, F);
    if (tid == 0) {
        // tell the last kernel of this call whether it has anything to do
        if (M.status == ZL_OK && !handled_by_filter(M, 1)) F.flags[1] = 1;
        else if (M.status == ZL_OK && !tail_instance(M, F)) F.flags[0] = 1;
        if (!mine) F.flags[2] = 1;                                 // the last kernel has to write this instance's outputs
    }
    if (!mine) return;
    uint32_t *g = (uint32_t *)smem;                               // [cells]
    Key<uint32_t> *keys = (Key<uint32_t> *)(smem + (size_t)cells * 4);
    const BatchWS<uint32_t> ws{keys, keys + tcap, (uint32_t *)(keys + 2 * (size_t)tcap), tcap};
    for (int c = tid; c < cells; c += nt) g[c] = 0;
    if (tid == 0) { sstatus = 0; fill = 0; }
    __syncthreads();
    for (int r = warp; r < F.nreg; r += nw) {
        const uint32_t c = F.rcnt[(size_t)b * F.nreg + r];
        const uint64_t *lst = F.list1 + (size_t)b * F.list1cap + (size_t)r * F.regcap;
        for (uint32_t i = lane; i < c; i += 32) {
            if (!gd.ok((size_t)r * F.regcap + i, (uint64_t)F.list1cap, ACC_LIST)) continue;
            const uint64_t w = lst[i];
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
    // a survivor whose next does not exceed the running maximum at its cell's start cannot matter either
    for (int r = warp; r < F.nreg; r += nw) {
        const uint32_t c = F.rcnt[(size_t)b * F.nreg + r];
        const uint64_t *lst = F.list1 + (size_t)b * F.list1cap + (size_t)r * F.regcap;
        for (uint32_t i0 = 0; i0 < c; i0 += 32) {
            const uint32_t i = i0 + lane;
            const uint64_t w = (i < c && gd.ok((size_t)r * F.regcap + i, (uint64_t)F.list1cap, ACC_LIST)) ? lst[i] : 0ull;
            const uint32_t T = (uint32_t)(w >> 32), nx = (uint32_t)w;
            const uint32_t cc = w ? cell_of(T, M.cscale) : 0u;
            const bool keep = w && gd.ok(cc, (uint64_t)cells, ACC_TAB) && nx > max(T, g[cc]);
            const unsigned km = __ballot_sync(FULL, keep);
            if (km == 0) continue;
            unsigned base = 0;
            if (lane == 0) base = atomicAdd(&fill, (unsigned)__popc(km));
            base = __shfl_sync(FULL, base, 0);
            const unsigned pos = base + __popc(km & ((1u << lane) - 1u));
            if (keep && gd.ok(pos, (uint64_t)tcap, ACC_KEYS)) keys[pos].w = w;
        }
    }
    __syncthreads();
    uint64_t bd = ~0ull, bt = ~0ull, cs = 0;
    uint32_t cc = 0;
    run_batch<uint32_t, ZL_OBJ_RANGE>(ws, (int)min(fill, (unsigned)tcap), (uint32_t)M.t0, n, tmp, (uint32_t)0, cs, cc, bd, bt);
    block_best_to_result(bd, bt, ZL_OK, tmp, &sstatus, best);
    __syncthreads();
    // the instance's outputs right here (the last kernel skips it)
    const int fst = best.valid ? ZL_OK : ZL_ERR_TIMEOUT;          // a valid instance always has a candidate
    const int64_t bar = fst == ZL_OK ? M.tmin + (int64_t)(best.t - 1) + (int64_t)best.d : INT64_MIN;
    if (tid == 0) {
        if (gd.ok((size_t)b * P.nres, (size_t)P.B * P.nres, ACC_SEG)) P.seg[(size_t)b * P.nres] = best;
        P.wait[b] = fst == ZL_OK ? (int64_t)best.d : INT64_MIN;
        P.barrier[b] = bar;
        if (P.status) P.status[b] = fst;
    }
    // the indices, 32 rows a warp
    for (int p0 = warp * 32; p0 < n; p0 += nt) {
        const int p = p0 + lane;
        int res = -1;
        if constexpr (std::is_same<SRC, MatBatch>::value) {
            const int64_t *rp = p < n ? src.ts + ((size_t)b * n + p) * R : nullptr;
            const int64_t e0 = rp ? (int64_t)ldg64(rp) : 0, eR = rp ? (int64_t)ldg64(rp + R - 1) : 0;
            if (fst == ZL_OK) res = last_index_not_after_warp(rp, R, bar, e0, eR);
        } else {
            if (p < n && fst == ZL_OK) res = last_index_not_after(src.inst(b, n, R).row(p), R, bar);
        }
        if (p < n && gd.ok((size_t)b * n + p, (size_t)P.B * n, ACC_IDX)) P.idx[(size_t)b * n + p] = res;
    }
}

// CTAs per instance of k_range_head for a batch of B instances: as many (of up to 512 threads) as it takes to put about
// two on every SM, at most `gmax`, and never so many that a CTA is left with fewer than 16 rows.
int range_head_cluster_size(int B, int n, int num_sms, int gmax) {
    const long long target = (long long)num_sms * 2;
    int G = 1;
    while (G < gmax && (long long)B * G * 2 <= target && n / (G * 2) >= 16) G *= 2;
    return G;
}

static void fill_params(RangeParams &P, const Pipeline &q, const FilterBufs &fb) {
    memset(&P, 0, sizeof(P));
    P.n = q.n; P.R = q.R; P.B = q.B; P.flags = q.flags; P.nres = q.nres;
    P.meta = q.meta; P.seg = q.seg; P.idx = q.idx; P.barrier = q.barrier; P.wait = q.wait; P.status = q.status;
    P.vec2 = (q.R % 2 == 0) && (((uintptr_t)q.ts & 15) == 0);
    P.dbg = fb.dbg;
}

template <class SRC>
static cudaError_t enqueue_range_head_t(const Pipeline &q, const FilterBufs &fb, cudaStream_t st, const SRC &src) {
    int G = range_head_cluster_size(q.B, q.n, q.num_sms, 8);
    if (q.cluster) G = std::max(1, std::min(pow2_floor(q.cluster), 8));
    while (G > 1 && ((long long)q.B * G > fb.maxctas || q.n / G < 1)) G /= 2;
    RangeParams P;
    fill_params(P, q, fb);
    P.rpc = (q.n + G - 1) / G;
    int threads = q.prologue_threads ? q.prologue_threads : 512;
    threads = std::max(32, std::min(std::min(threads, 512), 32 * pow2_ceil(std::max(1, (2 * P.rpc + 31) / 32))));
    const int nw = threads / 32;
    P.slow = std::max(1, std::min(FILTER_ROWS / G, std::max(1, P.rpc / 16)));
    const size_t arr = ((size_t)fb.cells + 32) * 4;
    const size_t smem = (size_t)fb.cells * 4 + (size_t)P.rpc * 16 + arr * (size_t)std::min(P.slow, nw);
    P.smem_bytes = (uint32_t)smem;
    P.ctas = (uint32_t)((size_t)q.B * G);
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
    if (!((q.pdl_off >> 9) & 1)) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr; cfg.numAttrs = na;
    const bool check = (q.flags & ZL_FLAG_DEBUG_CHECKS) && fb.dbg && !q.checks_off;
    if (G > 1) return check ? cudaLaunchKernelEx(&cfg, k_range_head<SRC, true, true>, src, P, fb) : cudaLaunchKernelEx(&cfg, k_range_head<SRC, false, true>, src, P, fb);
    return check ? cudaLaunchKernelEx(&cfg, k_range_head<SRC, true, false>, src, P, fb) : cudaLaunchKernelEx(&cfg, k_range_head<SRC, false, false>, src, P, fb);
}

template <class SRC>
static cudaError_t enqueue_range_filter_t(const Pipeline &q, FilterBufs &fb, cudaStream_t st, const SRC &src) {
    RangeParams P;
    fill_params(P, q, fb);
    // Many small CTAs (about sixteen per SM over the call, in several waves): the SMs pick them up as they finish, which
    // evens out the instances' different amounts of work.  An instance's rows are dealt out to its CTAs in turn.
    P.bulk = q.filter_bulk == 1 && P.vec2;
    P.S = !P.bulk ? 0 : q.filter_stages ? std::max(2, std::min(q.filter_stages, 7)) : 3;
    P.CH = !P.bulk ? 0 : q.filter_round >= 128 ? q.filter_round : (q.flags & ZL_FLAG_FULL_SWEEP) && q.R >= 512 ? 512 : 256;   // timestamps per ring slot
    int threads = std::max(64, std::min(256, 32 * pow2_ceil(std::min(q.n, 32))));
    if (q.filter_threads) threads = std::max(64, std::min(std::min(q.filter_threads, 256), 32 * pow2_ceil(std::min(q.n, 32))));
    const int nw = threads / 32;
    long long rpc = ((long long)q.n * q.B / (16LL * q.num_sms) + nw - 1) / nw * nw;
    if (q.filter_rows) rpc = q.filter_rows;
    rpc = std::max<long long>(nw, std::min<long long>(rpc, (q.n + nw - 1) / nw * nw));
    fb.nreg = (int)((q.n + rpc - 1) / rpc);
    P.rpc = (q.n + fb.nreg - 1) / fb.nreg;                        // rows of the CTAs that get the most
    dim3 grid(fb.nreg, q.B);
    fb.regcap = fb.list1cap / fb.nreg;
    P.nreg = fb.nreg;
    const size_t smem = (size_t)fb.cells * 4 + (size_t)((P.rpc + 1) & ~1) * 4 + (size_t)nw * P.S * 8 + 16 +
                        (P.bulk ? (size_t)nw * P.S * (P.CH + 2) * 8 : (size_t)nw * RING_STAGES * RING_SLOT * 8);
    P.smem_bytes = (uint32_t)smem;
    P.ctas = (uint32_t)((size_t)q.B * fb.nreg);
    P.stamps = fb.dbg ? (unsigned long long *)(fb.dbg + 16) : nullptr;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = grid; cfg.blockDim = dim3(threads); cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = ((q.pdl_off >> 1) & 1) ? 0 : 1;
    const bool check = (q.flags & ZL_FLAG_DEBUG_CHECKS) && fb.dbg && !q.checks_off;
    return check ? cudaLaunchKernelEx(&cfg, k_range_filter<SRC, true>, src, P, fb) : cudaLaunchKernelEx(&cfg, k_range_filter<SRC, false>, src, P, fb);
}

template <class SRC>
static cudaError_t enqueue_range_tail_t(const Pipeline &q, FilterBufs &fb, cudaStream_t st, const SRC &src) {
    RangeParams P;
    fill_params(P, q, fb);
    const bool many = q.B > 2 * q.num_sms;
    P.tcap = (int)std::min<long long>(many ? (long long)TAIL_CAP / 2 : (long long)TAIL_CAP, pow2_ceil(std::max(64, fb.list1cap)));
    fb.tailcap = P.tcap;
    const int threads = q.tail_threads ? q.tail_threads : many ? (P.tcap <= 1024 ? 128 : 256) : std::max(64, std::min(1024, P.tcap / 2));
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(q.B); cfg.blockDim = dim3(threads); cfg.dynamicSmemBytes = (size_t)P.tcap * 20 + (size_t)fb.cells * 4; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = ((q.pdl_off >> 2) & 1) ? 0 : 1;
    const bool check = (q.flags & ZL_FLAG_DEBUG_CHECKS) && fb.dbg && !q.checks_off;
    return check ? cudaLaunchKernelEx(&cfg, k_range_tail<SRC, true>, src, P, fb) : cudaLaunchKernelEx(&cfg, k_range_tail<SRC, false>, src, P, fb);
}

cudaError_t enqueue_range_head(const Pipeline &q, const FilterBufs &fb, cudaStream_t st, const MatBatch &src) { return enqueue_range_head_t(q, fb, st, src); }
cudaError_t enqueue_range_head(const Pipeline &q, const FilterBufs &fb, cudaStream_t st, const AriBatch &src) { return enqueue_range_head_t(q, fb, st, src); }
cudaError_t enqueue_range_filter(const Pipeline &q, FilterBufs &fb, cudaStream_t st, const MatBatch &src) { return enqueue_range_filter_t(q, fb, st, src); }
cudaError_t enqueue_range_filter(const Pipeline &q, FilterBufs &fb, cudaStream_t st, const AriBatch &src) { return enqueue_range_filter_t(q, fb, st, src); }
cudaError_t enqueue_range_tail(const Pipeline &q, FilterBufs &fb, cudaStream_t st, const MatBatch &src) { return enqueue_range_tail_t(q, fb, st, src); }
cudaError_t enqueue_range_tail(const Pipeline &q, FilterBufs &fb, cudaStream_t st, const AriBatch &src) { return enqueue_range_tail_t(q, fb, st, src); }

template <class SRC>
static cudaError_t range_limits_t() {
    const int big = 200 * 1024;
    cudaError_t e = cudaFuncSetAttribute(k_range_head<SRC, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_range_head<SRC, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_range_head<SRC, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_range_head<SRC, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_range_filter<SRC, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_range_filter<SRC, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_range_tail<SRC, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_range_tail<SRC, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
    return e;
}

cudaError_t range_limits() {
    cudaError_t e = range_limits_t<MatBatch>();
    if (e == cudaSuccess) e = range_limits_t<AriBatch>();
    return e;
}

}  // namespace zl
