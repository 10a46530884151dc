// The bucket route: the whole instance is put into time order bucket by bucket (SUM, and RANGE instances small
// enough to be one shared-memory batch).  k_sum_plan, k_sum_index, k_sum_buckets.
#include "zl_batch.cuh"
#include "zl_host.h"

namespace zl {

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

void enqueue_bucket_route(const Pipeline &q, FilterBufs &fb, cudaStream_t st, cudaEvent_t mid) {
    const bool single = fb.scells == 0;
    const size_t nb1 = (size_t)fb.stiles * TILE_BK + 1;
    launch_dep(!((q.pdl_off >> 1) & 1), k_sum_plan, dim3(q.B), dim3(single ? 32 : 1024), single ? 0 : ((size_t)fb.scells + 1) * 8 + nb1 * 4, st,
               q.ts, q.n, q.R, q.meta, fb);
    if (!single) {
        const int nw = 8;
        const int row_blocks = std::max(1, std::min((q.n + nw - 1) / nw, (32 * q.num_sms + q.B - 1) / q.B));
        launch_dep(!((q.pdl_off >> 2) & 1), k_sum_index, dim3(row_blocks, q.B), dim3(32 * nw), nb1 * 4, st, q.ts, q.n, q.R,
                   (const InstMeta *)q.meta, fb);
    }
    if (mid) cudaEventRecord(mid, st);
    const long long N = (long long)q.n * q.R;
    int bthreads = single ? (int)std::max<long long>(64, std::min<long long>(1024, pow2_ceil((int)((N + 7) / 8))))
                          : (fb.scap > 4096 ? 1024 : 512);
    if (q.tail_threads) bthreads = q.tail_threads;
    // few tiles in the batch: share each tile's buckets out over several CTAs
    fb.ssub = single ? 1 : std::max(1, std::min(TILE_BK, (2 * q.num_sms) / std::max(1, fb.stiles * q.B)));
    const int items = fb.stiles * fb.ssub * q.B;
    const size_t bsmem = (size_t)fb.scap * 18 + ((size_t)fb.scap + fb.scap / 32 + 2) * 4;
    if (q.objective == ZL_OBJ_SUM)
        launch_dep(!((q.pdl_off >> 3) & 1), k_sum_buckets<ZL_OBJ_SUM>, dim3(std::min(items, 32 * q.num_sms)), dim3(bthreads), bsmem, st,
                   q.ts, q.n, q.R, q.B, 0, q.meta, fb, q.nres, q.seg);
    else
        launch_dep(!((q.pdl_off >> 3) & 1), k_sum_buckets<ZL_OBJ_RANGE>, dim3(std::min(items, 32 * q.num_sms)), dim3(bthreads), bsmem, st,
                   q.ts, q.n, q.R, q.B, (q.flags & ZL_FLAG_FULL_SWEEP) ? 0 : 1, q.meta, fb, q.nres, q.seg);
}

cudaError_t bucket_route_limits() {
    cudaError_t e = cudaFuncSetAttribute(k_sum_buckets<ZL_OBJ_SUM>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_sum_buckets<ZL_OBJ_RANGE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_sum_plan, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    return e;
}

}  // namespace zl
