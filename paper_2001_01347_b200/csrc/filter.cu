// The RANGE filter pass (k_filter on stored rows, k_filter_arith on predicted rows) and k_tail, which finishes
// the instances that are left with few survivors.  Each has an instantiation that tests its indices (CHECK), which a
// handle created with ZL_FLAG_DEBUG_CHECKS runs.
#include "zl_batch.cuh"
#include "zl_guard.cuh"
#include "zl_host.h"

namespace zl {

// ------------------------------------------------------------------------------ filter pass (RANGE)
// A CTA owns a block of rows of one instance (a "region").  Each warp streams its rows in storage
// order through a private shared-memory ring filled by 16-byte cp.async copies (FILTER_STAGES chunks of
// 64 timestamps in flight per warp), tests every element against the table and appends the survivors,
// as (T << 32 | next), to the region's list; the per-cell maximum of `next` over the survivors goes to
// cellmax for the refinement.  Rows whose length is odd, or a misaligned base, take 8-byte copies.
constexpr int FILTER_STAGES = 3;      // ring slots per warp
constexpr int FILTER_CHUNK = 256;     // timestamps per slot (FILTER_CHUNK / 64 16-byte copies per lane)
constexpr int FILTER_SLOT = FILTER_CHUNK + 2;   // + the successor of the slot's last element, + padding

template <bool CHECK>
struct FilterCtx {
    const uint32_t *tab; uint64_t *list; uint32_t *cellmax; unsigned int *scount;
    uint32_t cscale, fscale, lmin, regcap, dmin;
    uint32_t cells, fcells;
    Guard<CHECK> g;               // CHECK: table, list and cell indices are tested before they are used
};

// Table test of the (up to) two elements of a lane, warp-aggregated append of the survivors.
template <bool CHECK>
__device__ __forceinline__ void filter_pair(const FilterCtx<CHECK> &c, int lane, bool va, uint32_t Ta, uint32_t na,
                                            bool vb, uint32_t Tb, uint32_t nb) {
    // cheap necessary condition first: most elements belong to fast workers and stop here
    bool ka = va && Ta <= c.lmin && na - Ta > c.dmin;
    bool kb = vb && Tb <= c.lmin && nb - Tb > c.dmin;
    if (!__any_sync(FULL, ka || kb)) return;
    if (ka) { const uint32_t cc = cell_of(Ta, c.cscale); ka = c.g.ok(cc, c.cells, ACC_TAB) && na > max(Ta, c.tab[cc]); }
    if (kb) { const uint32_t cc = cell_of(Tb, c.cscale); kb = c.g.ok(cc, c.cells, ACC_TAB) && nb > max(Tb, c.tab[cc]); }
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
        const uint32_t fc = cell_of(Ta, c.fscale);
        if (c.g.ok(fc, c.fcells, ACC_CELLMAX)) atomicMax(&c.cellmax[fc], na);
    }
    if (kb) {
        const unsigned pos = base + na_cnt + __popc(mb & below);
        if (pos < c.regcap) c.list[pos] = ((uint64_t)Tb << 32) | nb;
        const uint32_t fc = cell_of(Tb, c.fscale);
        if (c.g.ok(fc, c.fcells, ACC_CELLMAX)) atomicMax(&c.cellmax[fc], nb);
    }
}

// The 64 elements of a slot starting at `off`: element pairs per lane, successor of the pair from the
// slot itself (the element after the slot's last one sits right behind it).  Returns the time of the
// last of them that belongs to the request.
template <bool CHECK>
__device__ __forceinline__ uint32_t filter_half(const FilterCtx<CHECK> &C, const int64_t *slot, int off, int i0, int lim, int R,
                                                uint32_t tminlo, int lane) {
    const int i = i0 + off + 2 * lane;
    const bool va = i < lim, vb = i + 1 < lim;                    // lim: end of what was requested of the row (<= R)
    const longlong2 ab = *reinterpret_cast<const longlong2 *>(slot + off + 2 * lane);
    const uint32_t Ta = va ? (uint32_t)(uint64_t)ab.x - tminlo : 0xffffffffu;
    const uint32_t Tb = vb ? (uint32_t)(uint64_t)ab.y - tminlo : 0xffffffffu;
    const uint32_t nb = i + 2 < R ? (uint32_t)(uint64_t)slot[off + 2 * lane + 2] - tminlo : 0xffffffffu;
    filter_pair(C, lane, va, Ta, Tb, vb, Tb, nb);
    // the last of the 64 that belongs to the request (the caller passes at least one): whether the row has passed lmin is
    // decided by a real element, never by the filler behind the request's end
    const int last = min(63, lim - 1 - (i0 + off));
    return __shfl_sync(FULL, (last & 1) ? Tb : Ta, last >> 1);
}

// 128 timestamps of a slot, with the one after them, that lie inside the row: no bounds checks, one vote
// for all four elements of a lane.  Returns the time of the last of the 128.
template <bool CHECK>
__device__ __forceinline__ uint32_t filter_slot_inside(const FilterCtx<CHECK> &C, const int64_t *slot, uint32_t tminlo, int lane) {
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

template <bool CHECK>
__global__ void __launch_bounds__(1024) k_filter(const int64_t *ts, int n, int R, int B, int flags, int rows_per_cta, int req_round,
                                                  InstMeta *meta, FilterBufs F) {
    grid_dep_wait();
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ unsigned int scount;
    const int b = blockIdx.y, tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
    const InstMeta M = meta[b];
    const Guard<CHECK> gd{F.dbg, (uint32_t)(b * gridDim.x + blockIdx.x)};
    uint32_t *rc = F.rcnt + (size_t)b * F.nreg + blockIdx.x;
    if (!gd.ok((size_t)b * F.nreg + blockIdx.x, (size_t)B * F.nreg, ACC_RCNT) ||
        !gd.ok((size_t)b * F.list1cap + ((size_t)blockIdx.x + 1) * F.regcap - 1, (size_t)B * F.list1cap, ACC_LIST)) return;
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
    FilterCtx<CHECK> C;
    C.tab = tab; C.list = F.list1 + (size_t)b * F.list1cap + (size_t)blockIdx.x * F.regcap;
    C.cellmax = F.cellmax + (size_t)b * F.fcells; C.scount = &scount;
    C.cscale = M.cscale; C.fscale = M.fscale; C.lmin = lmin; C.regcap = (uint32_t)F.regcap; C.dmin = M.dmin;
    C.cells = cells; C.fcells = (uint32_t)F.fcells; C.g = gd;
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
template <bool CHECK>
__global__ void __launch_bounds__(256) k_filter_arith(const AriBatch src, int n, int R, int B, int rows_per_cta, InstMeta *meta, FilterBufs F) {
    grid_dep_wait();
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ unsigned int scount;
    const int b = blockIdx.y, tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
    const InstMeta M = meta[b];
    const Guard<CHECK> gd{F.dbg, (uint32_t)(b * gridDim.x + blockIdx.x)};
    uint32_t *rc = F.rcnt + (size_t)b * F.nreg + blockIdx.x;
    if (!gd.ok((size_t)b * F.nreg + blockIdx.x, (size_t)B * F.nreg, ACC_RCNT) ||
        !gd.ok((size_t)b * F.list1cap + ((size_t)blockIdx.x + 1) * F.regcap - 1, (size_t)B * F.list1cap, ACC_LIST)) return;
    if (M.status != ZL_OK || M.cscale == 0) { if (tid == 0) *rc = 0; return; }
    const uint32_t cells = (uint32_t)F.cells;
    uint32_t *tab = (uint32_t *)smem;
    const uint32_t *tg = F.table + (size_t)b * cells;
    for (uint32_t c = tid; c < cells; c += nt) tab[c] = tg[c];
    if (tid == 0) scount = 0;
    __syncthreads();
    FilterCtx<CHECK> C;
    C.tab = tab; C.list = F.list1 + (size_t)b * F.list1cap + (size_t)blockIdx.x * F.regcap;
    C.cellmax = F.cellmax + (size_t)b * F.fcells; C.scount = &scount;
    C.cscale = M.cscale; C.fscale = M.fscale; C.lmin = (uint32_t)M.lmin; C.regcap = (uint32_t)F.regcap; C.dmin = M.dmin;
    C.cells = cells; C.fcells = (uint32_t)F.fcells; C.g = gd;
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

// Instances with few survivors of the filter pass are finished by one CTA.  It first applies the
// refinement at the resolution of the coarse cells, in shared memory (maximum of next per cell,
// exclusive prefix maximum, drop every survivor whose next does not exceed the value at its cell's
// start), then sorts what is left and sweeps it.  Dropped survivors never hold the running maximum
// alone, so nothing has to be carried in.
template <class SRC, bool CHECK>
__global__ void __launch_bounds__(1024, 1) k_tail(const InstMeta *meta, FilterBufs F, int n, int nres, SegResult *seg, int tcap,
                                                  const SRC src, int R, int B, int32_t *idx, int64_t *barrier, int64_t *wait, int32_t *status) {
    grid_dep_wait();
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ uint64_t tmp[34];
    __shared__ unsigned int sstatus, fill;
    const int b = blockIdx.x, tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
    const Guard<CHECK> gd{F.dbg, (uint32_t)b};
    const int cells = F.cells;
    const InstMeta M = meta[b];
    if (tid == 0) {
        // tell the later kernels of this call whether they have anything to do
        const bool mine = M.status == ZL_OK && handled_by_filter(M, 1) && tail_instance(M, F);
        if (M.status == ZL_OK && !handled_by_filter(M, 1)) F.flags[1] = 1;
        else if (M.status == ZL_OK && !tail_instance(M, F)) F.flags[0] = 1;
        if (!mine) F.flags[2] = 1;                                 // k_finalize has to write this instance's outputs
    }
    if (M.status != ZL_OK || !handled_by_filter(M, 1) || !tail_instance(M, F)) return;
    uint32_t *g = (uint32_t *)smem;                               // [cells]
    Key<uint32_t> *keys = (Key<uint32_t> *)(smem + (size_t)F.cells * 4);
    const BatchWS<uint32_t> ws{keys, keys + tcap, (uint32_t *)(keys + 2 * (size_t)tcap), tcap};
    for (int c = tid; c < cells; c += nt) g[c] = 0;
    if (tid == 0) { sstatus = 0; fill = 0; }
    __syncthreads();
    for (int r = warp; r < F.nreg; r += nw) {
        const uint32_t c = F.rcnt[(size_t)b * F.nreg + r];
        const uint64_t *src = F.list1 + (size_t)b * F.list1cap + (size_t)r * F.regcap;
        for (uint32_t i = lane; i < c; i += 32) {
            if (!gd.ok((size_t)b * F.list1cap + (size_t)r * F.regcap + i, (size_t)B * F.list1cap, ACC_LIST)) continue;
            const uint64_t w = src[i];
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
    for (int r = warp; r < F.nreg; r += nw) {
        const uint32_t c = F.rcnt[(size_t)b * F.nreg + r];
        const uint64_t *src = F.list1 + (size_t)b * F.list1cap + (size_t)r * F.regcap;
        for (uint32_t i0 = 0; i0 < c; i0 += 32) {
            const uint32_t i = i0 + lane;
            const uint64_t w = (i < c && gd.ok((size_t)b * F.list1cap + (size_t)r * F.regcap + i, (size_t)B * F.list1cap, ACC_LIST)) ? src[i] : 0ull;
            const uint32_t T = (uint32_t)(w >> 32), nx = (uint32_t)w;
            const uint32_t cc = i < c ? cell_of(T, M.cscale) : 0u;
            const bool keep = i < c && gd.ok(cc, (uint64_t)cells, ACC_TAB) && nx > max(T, g[cc]);
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
    run_batch<uint32_t, ZL_OBJ_RANGE>(ws, (int)fill, (uint32_t)M.t0, n, tmp, (uint32_t)0, cs, cc, bd, bt);
    __shared__ SegResult best;
    block_best_to_result(bd, bt, ZL_OK, tmp, &sstatus, best);
    __syncthreads();
    // K5 for this instance right here: barrier, wait and the per-worker indices (k_finalize skips it)
    const int fst = best.valid ? ZL_OK : ZL_ERR_TIMEOUT;          // a valid instance always has a candidate
    const int64_t bar = fst == ZL_OK ? M.tmin + (int64_t)(best.t - 1) + (int64_t)best.d : INT64_MIN;
    if (tid == 0) {
        if (gd.ok((size_t)b * nres, (size_t)B * nres, ACC_SEG)) seg[(size_t)b * nres] = best;
        wait[b] = fst == ZL_OK ? (int64_t)best.d : INT64_MIN;
        barrier[b] = bar;
        if (status) status[b] = fst;
    }
    for (int p = tid; p < n; p += nt)
        if (gd.ok((size_t)b * n + p, (size_t)B * n, ACC_IDX))
            idx[(size_t)b * n + p] = fst == ZL_OK ? last_index_not_after(src.inst(b, n, R).row(p), R, bar) : -1;
}

template <class SRC>
static void enqueue_filter_t(const Pipeline &q, FilterBufs &fb, cudaStream_t st, cudaEvent_t mid, const SRC &src) {
    constexpr bool arith = std::is_same<SRC, AriBatch>::value;
    const bool many = q.B > 2 * q.num_sms;
    int threads = std::max(64, std::min(256, 32 * pow2_ceil(std::min(q.n, 32))));
    if (q.filter_threads) threads = std::max(64, std::min(q.filter_threads, 32 * pow2_ceil(std::min(q.n, 32))));
    const int nw = threads / 32;
    long long rpc = ((long long)q.n * q.B / (16LL * q.num_sms) + nw - 1) / nw * nw;
    if (q.filter_rows) rpc = ((long long)q.filter_rows + nw - 1) / nw * nw;
    rpc = std::max<long long>(nw, std::min<long long>(rpc, (q.n + nw - 1) / nw * nw));
    fb.nreg = (int)((q.n + rpc - 1) / rpc);
    fb.regcap = fb.list1cap / fb.nreg;
    const size_t fsmem = (size_t)fb.cells * 4 + (size_t)nw * FILTER_STAGES * FILTER_SLOT * 8;
    // a debug handle runs the instantiations that test their indices
    const bool check = (q.flags & ZL_FLAG_DEBUG_CHECKS) && fb.dbg && !q.checks_off;
    if constexpr (arith) {
        if (check) launch_dep(!((q.pdl_off >> 1) & 1), k_filter_arith<true>, dim3(fb.nreg, q.B), dim3(threads), (size_t)fb.cells * 4, st, src, q.n, q.R, q.B, (int)rpc, q.meta, fb);
        else launch_dep(!((q.pdl_off >> 1) & 1), k_filter_arith<false>, dim3(fb.nreg, q.B), dim3(threads), (size_t)fb.cells * 4, st, src, q.n, q.R, q.B, (int)rpc, q.meta, fb);
    } else {
        if (check) launch_dep(!((q.pdl_off >> 1) & 1), k_filter<true>, dim3(fb.nreg, q.B), dim3(threads), fsmem, st, q.ts, q.n, q.R, q.B, q.flags, (int)rpc, q.filter_round ? q.filter_round : 8, q.meta, fb);
        else launch_dep(!((q.pdl_off >> 1) & 1), k_filter<false>, dim3(fb.nreg, q.B), dim3(threads), fsmem, st, q.ts, q.n, q.R, q.B, q.flags, (int)rpc, q.filter_round ? q.filter_round : 8, q.meta, fb);
    }
    if (mid) cudaEventRecord(mid, st);
    // instances with at most tcap survivors are finished by one CTA each; with many instances a smaller limit lets more
    // of those CTAs share an SM
    const int tcap = (int)std::min<long long>(many ? (long long)TAIL_CAP / 2 : (long long)TAIL_CAP, pow2_ceil(std::max(64, fb.list1cap)));
    fb.tailcap = tcap;
    const int tthreads = q.tail_threads ? q.tail_threads : many ? (tcap <= 1024 ? 128 : 256) : std::max(64, std::min(1024, tcap / 2));
    const size_t tsmem = (size_t)tcap * 20 + (size_t)fb.cells * 4;
    if (check) launch_dep(!((q.pdl_off >> 2) & 1), k_tail<SRC, true>, dim3(q.B), dim3(tthreads), tsmem, st,
                          (const InstMeta *)q.meta, fb, q.n, q.nres, q.seg, tcap, src, q.R, q.B, q.idx, q.barrier, q.wait, q.status);
    else launch_dep(!((q.pdl_off >> 2) & 1), k_tail<SRC, false>, dim3(q.B), dim3(tthreads), tsmem, st,
                    (const InstMeta *)q.meta, fb, q.n, q.nres, q.seg, tcap, src, q.R, q.B, q.idx, q.barrier, q.wait, q.status);
}

void enqueue_filter(const Pipeline &q, FilterBufs &fb, cudaStream_t st, cudaEvent_t mid, const MatBatch &src) { enqueue_filter_t(q, fb, st, mid, src); }
void enqueue_filter(const Pipeline &q, FilterBufs &fb, cudaStream_t st, cudaEvent_t mid, const AriBatch &src) { enqueue_filter_t(q, fb, st, mid, src); }

cudaError_t filter_limits() {
    cudaError_t e = cudaFuncSetAttribute(k_filter<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_filter<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tail<MatBatch, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tail<AriBatch, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tail<MatBatch, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tail<AriBatch, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    return e;
}

}  // namespace zl
