// RANGE filter route, instances with many survivors: G at every fine time cell (heavy_tilemax, heavy_cellscan), the
// refinement (heavy_refine) and the bucket sweep (heavy_buckets).  Each is one phase of the route's last kernel: every
// CTA of the grid walks the phase's items; a grid-wide barrier separates the phases.
#pragma once
#include "zl_batch.cuh"

namespace zl {

constexpr int REFINE_ILP = 8;           // survivors a thread of the refinement has in flight

// ------------------------------------------------------------------------------ refinement (RANGE)
// The per-cell maxima of the filter pass give G exactly at every fine cell start (the survivors contain
// every element that ever raises the running maximum): heavy_cellscan turns cellmax, in place, into its
// exclusive prefix maximum floored by t0.  A survivor whose `next` does not exceed G at the start of its
// own cell cannot matter either, so heavy_refine drops it; the rest go to their time bucket.

// pass 1: maximum of every tile of SCAN_TILE fine cells.  A fixed grid walks the (tile, instance) pairs.
static __device__ void heavy_tilemax(const InstMeta *meta, const FilterBufs &F, int B, uint64_t *tmp) {
    const int tid = threadIdx.x, nt = blockDim.x;
    const int tiles = (F.fcells + SCAN_TILE - 1) / SCAN_TILE;
    for (int item = blockIdx.x; item < tiles * B; item += gridDim.x) {
        const int b = item / tiles, t = item % tiles;
        const InstMeta M = load_meta_cg(meta + b);
        if (M.status != ZL_OK || !handled_by_filter(M, 1) || tail_instance(M, F)) continue;
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
static __device__ void heavy_cellscan(const InstMeta *meta, const FilterBufs &F, int B, uint64_t *tmp, uint32_t *tile) {
    const int tid = threadIdx.x, nt = blockDim.x;
    const int tiles = (F.fcells + SCAN_TILE - 1) / SCAN_TILE;
    for (int item = blockIdx.x; item < tiles * B; item += gridDim.x) {
        const int b = item / tiles, t = item % tiles;
        const InstMeta M = load_meta_cg(meta + b);
        if (M.status != ZL_OK || !handled_by_filter(M, 1) || tail_instance(M, F)) continue;
        uint32_t *cmx = F.cellmax + (size_t)b * F.fcells + (size_t)t * SCAN_TILE;
        const int len = min(SCAN_TILE, F.fcells - t * SCAN_TILE);
        uint32_t before = 0;
        for (int i = tid; i < t; i += nt) before = max(before, __ldcg(F.tilemax + (size_t)b * tiles + i));
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

static __device__ void heavy_refine(InstMeta *meta, const FilterBufs &F, int B) {
    const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31;
    const int cpb_shift = __ffs(F.fcells / F.nbk) - 1;            // fine cells per bucket is a power of two
    for (int item = blockIdx.x; item < F.nreg * B; item += gridDim.x) {
        const int b = item / F.nreg, reg = item % F.nreg;
        const InstMeta M = load_meta_cg(meta + b);
        if (M.status != ZL_OK || !handled_by_filter(M, 1) || tail_instance(M, F)) continue;
        const uint32_t m = F.rcnt[(size_t)b * F.nreg + reg];
        if (m == 0) continue;
        const uint32_t *g = F.cellmax + (size_t)b * F.fcells;     // G at fine cell starts
        const uint64_t *src = F.list1 + (size_t)b * F.list1cap + (size_t)reg * F.regcap;
        uint32_t *bcnt = F.bcnt + (size_t)b * F.nbk;
        uint64_t *dst = F.list2 + (size_t)b * F.nbk * F.capb;
        unsigned kept = 0;
        bool over = false;
        // REFINE_ILP elements a step, so that as many list loads and then as many table look-ups are in flight together
        for (uint32_t i0 = tid; i0 < m; i0 += REFINE_ILP * nt) {
            uint64_t w[REFINE_ILP];
            uint32_t c[REFINE_ILP], gv[REFINE_ILP];
#pragma unroll
            for (int k = 0; k < REFINE_ILP; ++k) { const uint32_t i = i0 + k * nt; w[k] = i < m ? src[i] : 0ull; }
#pragma unroll
            for (int k = 0; k < REFINE_ILP; ++k) {
                c[k] = w[k] ? cell_of((uint32_t)(w[k] >> 32), M.fscale) : 0u;
                gv[k] = __ldcg(g + c[k]);
            }
#pragma unroll
            for (int k = 0; k < REFINE_ILP; ++k) {
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

// Sort and sweep the refined survivors.  CTA (g, b) takes buckets [g*grp, (g+1)*grp) of instance b in
// time order, packs whole buckets into shared-memory batches and runs each batch with the running
// maximum of `next` over everything before it (the prefix maximum of cellmax up to the batch's first cell).
static __device__ void heavy_buckets(const InstMeta *meta, const FilterBufs &F, int n, int nres, SegResult *seg, int B, unsigned char *smem, uint64_t *tmp) {
    __shared__ unsigned int sstatus, fill;
    const int tid = threadIdx.x, nt = blockDim.x;
    const int ngroups = (F.nbk + F.grp - 1) / F.grp;
    Key<uint32_t> *keys = (Key<uint32_t> *)smem;
    const BatchWS<uint32_t> ws{keys, keys + F.capb, (uint32_t *)(keys + 2 * (size_t)F.capb), F.capb};
    for (int item = blockIdx.x; item < ngroups * B; item += gridDim.x) {
    const int b = item / ngroups, g = item % ngroups;
    __syncthreads();                                              // shared state of the previous item is done with
    const InstMeta M = load_meta_cg(meta + b);
    if (M.status != ZL_OK || !handled_by_filter(M, 1) || tail_instance(M, F)) continue;
    const uint32_t *bcnt = F.bcnt + (size_t)b * F.nbk;
    const uint32_t *g0 = F.cellmax + (size_t)b * F.fcells;        // G at fine cell starts (after heavy_cellscan)
    const uint64_t *list = F.list2 + (size_t)b * F.nbk * F.capb;
    const int grp = bucket_group(F, M.count2);
    if (g * grp >= F.nbk) continue;                              // fewer, wider groups than items for this instance
    const int first = g * grp, last = min(first + grp, F.nbk);
    const int cpb = F.fcells / F.nbk;
    if (tid == 0) { sstatus = 0; fill = 0; }
    __syncthreads();
    // running max of next over everything before the group's first cell
    const uint32_t carry0 = __ldcg(g0 + (size_t)first * cpb);
    uint64_t bd = ~0ull, bt = ~0ull, cs = 0;
    uint32_t cc = 0;
    uint32_t mine = 0;
    for (int k = first + tid; k < last; k += nt) mine += min(__ldcg(bcnt + k), (uint32_t)F.capb);
    uint32_t group_total;
    block_scan_excl<uint32_t>(mine, OpAdd(), 0u, (uint32_t *)tmp, &group_total);
    if (group_total <= (uint32_t)F.capb) {
        // one batch: warps copy whole buckets side by side; offsets come from a running count
        const int lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
        for (int k = first + warp; k < last; k += nw) {
            const uint32_t c = min(__ldcg(bcnt + k), (uint32_t)F.capb);
            if (c == 0) continue;
            uint32_t off = 0;
            if (lane == 0) off = atomicAdd(&fill, c);
            off = __shfl_sync(FULL, off, 0);
            const uint64_t *src = list + (size_t)k * F.capb;
            for (uint32_t i = lane; i < c; i += 32) keys[off + i].w = __ldcg(src + i);
        }
        __syncthreads();
        run_batch<uint32_t, ZL_OBJ_RANGE>(ws, (int)group_total, (uint32_t)M.t0, n, tmp, carry0, cs, cc, bd, bt);
    } else {
        int m = 0;
        uint32_t carry_batch = carry0;
        for (int k = first; k < last; ++k) {
            const int c = (int)min(__ldcg(bcnt + k), (uint32_t)F.capb);
            if (c == 0) continue;
            if (m + c > F.capb) {
                run_batch<uint32_t, ZL_OBJ_RANGE>(ws, m, (uint32_t)M.t0, n, tmp, carry_batch, cs, cc, bd, bt);
                carry_batch = __ldcg(g0 + (size_t)k * cpb);        // G at the start of the next batch's first bucket
                m = 0;
            }
            const uint64_t *src = list + (size_t)k * F.capb;
            for (int i = tid; i < c; i += nt) keys[m + i].w = __ldcg(src + i);
            m += c;
            __syncthreads();
        }
        if (m > 0) run_batch<uint32_t, ZL_OBJ_RANGE>(ws, m, (uint32_t)M.t0, n, tmp, carry_batch, cs, cc, bd, bt);
    }
    block_best_to_result(bd, bt, ZL_OK, tmp, &sstatus, seg[(size_t)b * nres + g]);
    }
}

}  // namespace zl
