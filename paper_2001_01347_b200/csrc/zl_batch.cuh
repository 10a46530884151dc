// Device code shared by the routes: the batch engine (sort a shared-memory batch into time order, scan it,
// evaluate every candidate), the block reduction to a partial result, and the index search of K5.
#pragma once
#include "zl_device.cuh"
#include "zl_types.cuh"

namespace zl {

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
__device__ inline void block_best_to_result(uint64_t bd, uint64_t bt, uint32_t status, uint64_t *red, unsigned int *sstatus,
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

// Index of the last element of a sorted row that is <= bar (-1 if none).  Rows are close to arithmetic, so the
// position is first guessed from the row's end points, and the sixteen consecutive elements around the guess are
// loaded together (they share a cache line or two: the fewer distinct lines the call touches the better, since
// every one of them is a memory access of its own).  A guess that is further off looks at the sixteen elements on
// the side the answer lies on, twice at most, before it falls back to doubling steps and bisection.
template <class ROW>
__device__ int last_index_not_after(const ROW &row, int R, int64_t bar, int64_t e0, int64_t eR);

template <class ROW>
__device__ int last_index_not_after(const ROW &row, int R, int64_t bar) {
    return last_index_not_after(row, R, bar, row.at(0), row.at(R - 1));
}

// The same with the row's first and last element already at hand.
template <class ROW>
__device__ int last_index_not_after(const ROW &row, int R, int64_t bar, int64_t e0, int64_t eR) {
    if (bar < e0) return -1;
    if (bar >= eR) return R - 1;
    // e0 <= bar < eR, R >= 2.  Invariant: row[lo - 1] <= bar, row[hi] > bar
    int lo = 1, hi = R - 1;
    int g = (int)((double)(bar - e0) * (double)(R - 1) / (double)(eR - e0));
    g = max(0, min(g, R - 2));
    constexpr int W = 16;
    int a = max(0, min(g - W / 2 + 1, R - W)) & ~3;                // the window [a, a + W), on a 32-byte boundary of the row
    for (int it = 0; it < 3; ++it) {
        int64_t v[W];
#pragma unroll
        for (int k = 0; k < W; ++k) v[k] = row.at(min(a + k, R - 1));
        int c = 0, valid = 0;
#pragma unroll
        for (int k = 0; k < W; ++k) { valid += a + k < R ? 1 : 0; c += (a + k < R && v[k] <= bar) ? 1 : 0; }   // sorted: a prefix of the window
        if (c > 0 && c < valid) return a + c - 1;                  // the window holds the last element <= bar and its successor
        if (c == 0) hi = min(hi, a); else lo = max(lo, a + valid);
        if (lo >= hi) return lo - 1;
        a = c == 0 ? max(0, hi - W) : min(lo, max(0, R - W));
    }
    // the guess was far off: doubling steps from the nearer end of the bracket, then bisection
    if (lo > 1) {                                          // everything looked at was <= bar: search upwards from lo
        const int top = hi;
        for (int step = 16; lo < hi; step <<= 1) {
            const int q = min(lo + step - 1, top - 1);
            if (q < lo) break;
            if (row.at(q) <= bar) lo = q + 1; else { hi = q; break; }
        }
    } else {                                               // everything looked at was > bar: search downwards from hi
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

// The same for 32 stored rows at once, a row per lane (rowp == nullptr: the lane has none), by the whole warp: the
// windows - 32 consecutive elements around each row's guess - are loaded a row an instruction (two or three lines
// of memory, instead of one line per lane and element) and counted with a vote.  Rows whose answer three windows
// do not find fall back to bisection.  Every lane of the warp must call.
__device__ inline int last_index_not_after_warp(const int64_t *rowp, int R, int64_t bar, int64_t e0, int64_t eR) {
    const int lane = threadIdx.x & 31;
    constexpr int W = 32;
    int ans = -2;                                                 // -2: not known yet
    int lo = 1, hi = R - 1, a = 0;
    if (!rowp) ans = -1;
    else if (bar < e0) ans = -1;
    else if (bar >= eR) ans = R - 1;
    else {
        int g = (int)((double)(bar - e0) * (double)(R - 1) / (double)(eR - e0));
        g = max(0, min(g, R - 2));
        a = max(0, min(g - W / 2 + 1, R - W)) & ~3;               // on a 32-byte boundary of the row
    }
    for (int it = 0; it < 3; ++it) {
        const unsigned open = __ballot_sync(FULL, ans == -2);
        if (!open) break;
        // all the loads first, then the votes: the windows arrive together
        int64_t v[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const unsigned long long pw = __shfl_sync(FULL, (unsigned long long)(uintptr_t)rowp, i);
            const int ao = __shfl_sync(FULL, a, i);
            const bool in = ((open >> i) & 1u) && ao + lane < R;
            v[i] = in ? (int64_t)__ldg((const long long *)(uintptr_t)pw + ao + lane) : INT64_MAX;   // INT64_MAX: never <= bar (< 2^62)
        }
        int c = 0;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const unsigned le = __ballot_sync(FULL, v[i] <= bar);
            if (lane == i) c = __popc(le);
        }
        if (ans == -2) {
            const int valid = min(W, R - a);
            if (c > 0 && c < valid) ans = a + c - 1;              // the window holds the last element <= bar and its successor
            else {
                if (c == 0) hi = min(hi, a); else lo = max(lo, a + valid);
                if (lo >= hi) ans = lo - 1;
                else a = c == 0 ? max(0, hi - W) : min(lo, max(0, R - W));
            }
        }
    }
    if (ans == -2) {
        // far off the guess: bisection between what the windows established (row[lo - 1] <= bar < row[hi])
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if ((int64_t)__ldg((const long long *)rowp + mid) <= bar) lo = mid + 1; else hi = mid;
        }
        ans = lo - 1;
    }
    return ans;
}

}  // namespace zl
