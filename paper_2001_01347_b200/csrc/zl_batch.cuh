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
// position is first guessed from the row's end points.  Eight probes around the guess, eight elements apart and
// loaded together, then the seven elements between the two probes that bracket bar, loaded together: three
// rounds of loads in the usual case.  A guess that is further off is bracketed by doubling steps and bisected.
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

}  // namespace zl
