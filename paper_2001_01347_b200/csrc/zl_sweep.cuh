// The segment sweep of one (instance, time segment) pair and the final reduction of an instance: device code shared by
// the kernels that run them (k_sweep, k_finalize and the RANGE filter route's last kernel).
#pragma once
#include <cstddef>
#include <type_traits>

#include "zl_batch.cuh"

namespace zl {

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
        // Every round either commits (and then consumes an element, or moves the window to the next one: at most
        // n * R + 1 of those a segment) or does not fit: then it flushes the batch, or halves the window, which is at
        // least 1 and fits once it holds one element a row (the batch has room for that), so fewer than 70 rounds in
        // a row can fail to commit.  A segment that goes past either bound reports ZL_ERR_TIMEOUT instead of looping.
        uint64_t rounds = 0;
        uint32_t stalled = 0;
        const uint64_t max_rounds = P.max_rounds > 0 ? (uint64_t)P.max_rounds : 72 * ((uint64_t)n * R + 2);

        while (rlo < seg_hi) {
            if (OBJ == ZL_OBJ_RANGE && cut && floorv == INF) break;     // a row ran out: no later Z is complete
            if (++rounds > max_rounds || stalled > 72) { status = ZL_ERR_TIMEOUT; break; }
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
                ++stalled;
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
            stalled = 0;
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

// The (instance, segment) pairs of a call, walked by the CTAs of the grid.  Dynamic shared memory `smem`: row cursors
// [2n] u32 | batch nodes | sorted batch | slot counters (20 bytes per node of capacity).
template <int OBJ, class SRC>
__device__ void sweep_items(const SweepParams &P, const SRC &src, SweepShared &sh, unsigned char *smem) {
    static_assert(sizeof(SegResult) == 24 && offsetof(SegResult, valid) == 16 && offsetof(SegResult, status) == 20, "SegResult is read as three 8-byte words");
    uint32_t *curA = (uint32_t *)smem;
    uint32_t *curB = curA + P.n;
    unsigned char *kb = smem + (((size_t)2 * P.n * sizeof(uint32_t) + 15) & ~(size_t)15);
    unsigned char *kb2 = kb + (size_t)P.cap * 8;
    uint32_t *kcnt = (uint32_t *)(kb2 + (size_t)P.cap * 8);
    const int items = P.B * P.nseg;
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const int b = item / P.nseg, sidx = item % P.nseg;
        const InstMeta M = load_meta_cg(P.meta + b);
        if (handled_by_filter(M, P.filter)) continue;            // a fast route wrote this instance's results
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

// The word the host reads before its next call (pinned host memory): written across the bus only when it changes.
__device__ __forceinline__ void note_hint(const FilterBufs &F, bool many) {
    const uint32_t v = many ? 1u : 0u;
    if (*F.hint_last != v) { *F.hint_last = v; *F.hint = v; }
}

// ------------------------------------------------------------------------------ finalize
// The final step for 32 consecutive rows of an instance, by one warp: the minimum over the instance's partial results
// (every warp of the instance takes it for itself: there are few of them), then the indices of the warp's rows, a row
// per lane; the warp of the instance's first rows also writes wait, barrier and status.
// filter: 0 only the segment sweep ran, 1 the RANGE filter route (an instance with few survivors has one result, left
// by the filter kernel), 2 the bucket route.  `forced`: a status that overrides the instance's own when not ZL_OK.
// `pre`: the first and last element of the lane's row when the caller loaded them already (they are input: a kernel that
// is not the first of its call may read them before it waits for its predecessor), else nullptr.
struct RowEnds { int64_t e0, eR; };
// An instance's record and its first partial result, for a caller that loads them ahead of the call.
struct FirstResult { InstMeta M; uint64_t d, t; unsigned long long vs; };

__device__ __forceinline__ FirstResult load_first_result(const InstMeta *meta, const SegResult *seg, int b, int nres) {
    FirstResult f;
    f.M = load_meta_cg(meta + b);
    const unsigned long long *w0 = reinterpret_cast<const unsigned long long *>(seg + (size_t)b * nres);
    f.d = __ldcg(w0); f.t = __ldcg(w0 + 1); f.vs = __ldcg(w0 + 2);
    return f;
}

template <class SRC>
__device__ __forceinline__ RowEnds row_ends(const SRC &src, int b, int rowchunk, int n, int R) {
    RowEnds e{0, 0};
    const int p = rowchunk * 32 + (int)(threadIdx.x & 31);
    if (p < n) { const auto row = src.inst(b, n, R).row(p); e.e0 = row.at(0); e.eR = row.at(R - 1); }
    return e;
}

template <class SRC>
__device__ void finalize_rows(const SRC &src, int b, int rowchunk, int n, int R, int nseg, const FilterBufs &F, int nres, int objective,
                              int filter, const InstMeta *meta, const SegResult *seg, int32_t *idx, int64_t *barrier, int64_t *wait,
                              int32_t *status, uint32_t forced, const RowEnds *pre, const FirstResult *fr = nullptr, unsigned long long *stamps = nullptr) {
    static_assert(sizeof(SegResult) == 24 && offsetof(SegResult, valid) == 16 && offsetof(SegResult, status) == 20, "SegResult is read as three 8-byte words");
    const int lane = threadIdx.x & 31;
    // the instance's record, its first partial result (often the only one) and the row's end points: one round of loads
    const unsigned long long *w0 = reinterpret_cast<const unsigned long long *>(seg + (size_t)b * nres);
    const FirstResult f0 = fr ? *fr : load_first_result(meta, seg, b, nres);
    const InstMeta M = f0.M;
    const uint64_t d0 = f0.d, t0 = f0.t;
    const unsigned long long vs0 = f0.vs;
    if (filter == 1 && M.status == ZL_OK && handled_by_filter(M, 1) && tail_instance(M, F)) return;   // finished by the tail kernel
    const RowEnds ends = pre ? *pre : row_ends(src, b, rowchunk, n, R);
    uint64_t bd = ~0ull, bt = ~0ull;
    uint32_t st = max((uint32_t)M.status, forced);
    if (st == ZL_OK) {
        const int used = !handled_by_filter(M, filter) ? nseg
                         : filter == 2 ? (int)M.count2 * F.ssub                         // bucket route: one result per part of a tile
                         : tail_instance(M, F) ? 1 : (F.nbk + bucket_group(F, M.count2) - 1) / bucket_group(F, M.count2);
        for (int s = lane; s < used; s += 32) {
            // past the L1 cache: another CTA of this kernel may have written it
            const unsigned long long *w = w0 + 3 * (size_t)s;
            const uint64_t rd = s ? __ldcg(w) : d0, rt = s ? __ldcg(w + 1) : t0;
            const unsigned long long vs = s ? __ldcg(w + 2) : vs0;
            const int32_t rvalid = (int32_t)(uint32_t)vs, rstatus = (int32_t)(uint32_t)(vs >> 32);
            if (rstatus != ZL_OK) st = max(st, (uint32_t)rstatus);
            if (rvalid && (rd < bd || (rd == bd && rt < bt))) { bd = rd; bt = rt; }
        }
    }
    st = warp_reduce(st, OpMax());
    if (stamps && lane == 0) { unsigned long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); stamps[10] = t_; }
    const uint64_t dbest = warp_reduce(bd, OpMin());
    const uint64_t tbest = warp_reduce(bd == dbest ? bt : ~0ull, OpMin());
    int fst = (int)st;
    if (fst == ZL_OK && tbest == ~0ull) fst = ZL_ERR_TIMEOUT;      // no valid result: cannot happen for valid input
    int64_t bar = INT64_MIN, wt = INT64_MIN;
    if (fst == ZL_OK) {
        const int64_t tm = M.tmin + (int64_t)(tbest - 1);
        bar = objective == ZL_OBJ_RANGE ? tm + (int64_t)dbest : tm;
        wt = (int64_t)dbest;
    }
    if (rowchunk == 0 && lane == 0) {
        wait[b] = wt;
        barrier[b] = bar;
        if (status) status[b] = fst;
    }
    // a row per lane: the number of elements <= barrier.  Rows are close to arithmetic, so the position is first
    // guessed from the row's end points, bracketed by doubling steps around the guess, then bisected.
    const int p = rowchunk * 32 + lane;
    int res = -1;
    if constexpr (std::is_same<SRC, MatBatch>::value) {
        // stored rows: the warp looks at its rows' windows together
        if (fst == ZL_OK) res = last_index_not_after_warp(p < n ? src.ts + ((size_t)b * n + p) * R : nullptr, R, bar, ends.e0, ends.eR);
    } else {
        if (p < n && fst == ZL_OK) res = last_index_not_after(src.inst(b, n, R).row(p), R, bar, ends.e0, ends.eR);
    }
    if (stamps && lane == 0) { unsigned long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); stamps[14] = t_ + (res == -7); }
    if (p < n) idx[(size_t)b * n + p] = res;
}

// Every (instance, 32 rows) pair of a call, a warp each, by the warps of the grid.
template <class SRC>
__device__ void finalize_all(const SRC &src, int B, int n, int R, int nseg, const FilterBufs &F, int nres, int objective, int filter,
                             const InstMeta *meta, const SegResult *seg, int32_t *idx, int64_t *barrier, int64_t *wait, int32_t *status,
                             uint32_t forced, const RowEnds *first, const FirstResult *fr = nullptr, unsigned long long *stamps = nullptr) {
    const int wpb = blockDim.x >> 5, rc = (n + 31) / 32;
    const long long items = (long long)B * rc;
    // warp w of CTA c takes pairs c + gridDim.x * w, ...: when there are fewer pairs than warps, every CTA still gets some
    for (long long item = (long long)blockIdx.x + (long long)gridDim.x * (threadIdx.x >> 5); item < items; item += (long long)gridDim.x * wpb) {
        finalize_rows(src, (int)(item / rc), (int)(item % rc), n, R, nseg, F, nres, objective, filter, meta, seg, idx, barrier, wait, status, forced, first, fr, (threadIdx.x >> 5) == 0 ? stamps : nullptr);
        first = nullptr; fr = nullptr;
    }
}

// The record and first result of the warp's first pair's instance (any valid instance when the warp has no pair).
__device__ __forceinline__ FirstResult finalize_first_result(const InstMeta *meta, const SegResult *seg, int B, int n, int nres) {
    const int rc = (n + 31) / 32;
    const long long item = (long long)blockIdx.x + (long long)gridDim.x * (threadIdx.x >> 5);
    return load_first_result(meta, seg, item < (long long)B * rc ? (int)(item / rc) : 0, nres);
}

// The end points of the rows of the warp's first pair, for a caller that loads them before it waits for its predecessors.
template <class SRC>
__device__ __forceinline__ RowEnds finalize_first_ends(const SRC &src, int B, int n, int R) {
    const int rc = (n + 31) / 32;
    const long long item = (long long)blockIdx.x + (long long)gridDim.x * (threadIdx.x >> 5);
    if (item >= (long long)B * rc) return RowEnds{0, 0};
    return row_ends(src, (int)(item / rc), (int)(item % rc), n, R);
}

}  // namespace zl
