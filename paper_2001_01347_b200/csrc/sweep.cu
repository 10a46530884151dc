// The segment sweep (k_sweep: the general route, and the fallback of the fast routes) and k_finalize (K5: minimum
// over an instance's partial results, barrier, per-worker index recovery).
#include "zl_batch.cuh"
#include "zl_host.h"

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

template <int OBJ, class SRC>
__global__ void __launch_bounds__(1024) k_sweep(const SweepParams P, const SRC src) {
    grid_dep_wait();
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ SweepShared sh;
    uint32_t *curA = (uint32_t *)smem;
    uint32_t *curB = curA + P.n;
    // shared memory: row cursors | batch nodes | sorted batch | slot counters
    unsigned char *kb = smem + (((size_t)2 * P.n * sizeof(uint32_t) + 15) & ~(size_t)15);
    unsigned char *kb2 = kb + (size_t)P.cap * 8;
    uint32_t *kcnt = (uint32_t *)(kb2 + (size_t)P.cap * 8);
    if (P.need && P.need[1] == 0) return;                        // the filter route finished every instance
    // a fixed number of CTAs walks the (instance, segment) pairs
    const int items = P.B * P.nseg;
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const int b = item / P.nseg, sidx = item % P.nseg;
        const InstMeta M = P.meta[b];
        if (handled_by_filter(M, P.filter)) continue;            // the bucket sweep wrote this instance's results
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

// ------------------------------------------------------------------------------ finalize
// grid (row blocks, B): every CTA reduces the instance's partial results, then recovers the indices of
// its block of rows; the CTA of row block 0 also writes wait, barrier and status.
template <class SRC>
__global__ void __launch_bounds__(256) k_finalize(const SRC src, int n, int R, int nseg, FilterBufs F, int nres,
                                                  int objective, int filter, const InstMeta *meta, const SegResult *seg,
                                                  int32_t *idx, int64_t *barrier, int64_t *wait, int32_t *status) {
    grid_dep_wait();
    const int b = blockIdx.y, tid = threadIdx.x;
    // filter: 0 only the segment sweep ran, 1 the RANGE filter route, 2 the bucket route
    if (filter && F.flags[2] == 0) return;                        // k_tail finished every instance of this call
    const InstMeta M = meta[b];
    if (filter == 1 && M.status == ZL_OK && handled_by_filter(M, filter) && tail_instance(M)) return;   // finished by k_tail
    __shared__ uint64_t red[34];
    __shared__ unsigned int sstatus;
    __shared__ SegResult best;
    if (tid == 0) sstatus = 0;
    __syncthreads();
    uint64_t bd = ~0ull, bt = ~0ull;
    uint32_t st = M.status;
    if (st == ZL_OK) {
        const int used = !handled_by_filter(M, filter) ? nseg
                         : filter == 2 ? (int)M.count2 * F.ssub                         // bucket route: one result per part of a tile
                         : tail_instance(M) ? 1 : (F.nbk + bucket_group(F, M.count2) - 1) / bucket_group(F, M.count2);
        for (int s = tid; s < used; s += blockDim.x) {
            const SegResult r = seg[(size_t)b * nres + s];
            if (r.status != ZL_OK) st = max(st, (uint32_t)r.status);
            if (r.valid && (r.d < bd || (r.d == bd && r.t < bt))) { bd = r.d; bt = r.t; }
        }
    }
    block_best_to_result(bd, bt, st, red, &sstatus, best);
    __syncthreads();
    int fst = (int)best.status;
    if (fst == ZL_OK && !best.valid) fst = ZL_ERR_TIMEOUT;         // cannot happen for valid input
    int64_t bar = INT64_MIN, wt = INT64_MIN;
    if (fst == ZL_OK) {
        const int64_t tm = M.tmin + (int64_t)(best.t - 1);
        bar = objective == ZL_OBJ_RANGE ? tm + (int64_t)best.d : tm;
        wt = (int64_t)best.d;
    }
    if (blockIdx.x == 0 && tid == 0) {
        wait[b] = wt;
        barrier[b] = bar;
        if (status) status[b] = fst;
    }
    // one thread per row: the number of elements <= barrier.  Rows are close to arithmetic, so the position is
    // first guessed from the row's end points, bracketed by doubling steps around the guess, then bisected.
    const int p = blockIdx.x * blockDim.x + tid;
    if (p < n) {
        int res = -1;
        if (fst == ZL_OK) {
            res = last_index_not_after(src.inst(b, n, R).row(p), R, bar);
        }
        idx[(size_t)b * n + p] = res;
    }
}

template <class SRC>
static void enqueue_sweep_t(const Pipeline &q, const FilterBufs &fb, const LaunchPlan &p, bool fast, cudaStream_t st, const SRC &src) {
    SweepParams sp;
    sp.ts = q.ts; sp.meta = q.meta; sp.seg = q.seg;
    sp.n = q.n; sp.R = q.R; sp.B = q.B; sp.nseg = p.nseg; sp.nres = q.nres; sp.G = p.G; sp.cap = p.cap;
    sp.flags = q.flags; sp.target = p.target; sp.filter = fast ? 1 : 0;
    sp.need = fast ? fb.flags : nullptr;
    // with a fast route on, the segment sweep is only the fallback: a small persistent grid
    const int items = p.nseg * q.B;
    const int sweep_ctas = fast ? std::min(items, 2 * q.num_sms) : items;
    if (q.objective == ZL_OBJ_RANGE) launch_dep(!((q.pdl_off >> 7) & 1), k_sweep<ZL_OBJ_RANGE, SRC>, dim3(sweep_ctas), dim3(p.threads), p.smem, st, sp, src);
    else launch_dep(!((q.pdl_off >> 7) & 1), k_sweep<ZL_OBJ_SUM, SRC>, dim3(sweep_ctas), dim3(p.threads), p.smem, st, sp, src);
}

template <class SRC>
static void enqueue_finalize_t(const Pipeline &q, const FilterBufs &fb, const LaunchPlan &p, int route, cudaStream_t st, const SRC &src) {
    const int fthreads = std::max(32, std::min(256, pow2_ceil(q.n)));
    launch_dep(!((q.pdl_off >> 8) & 1), k_finalize<SRC>, dim3((q.n + fthreads - 1) / fthreads, q.B), dim3(fthreads), 0, st, src, q.n, q.R, p.nseg, fb, q.nres, q.objective,
               route, (const InstMeta *)q.meta, (const SegResult *)q.seg, q.idx, q.barrier, q.wait, q.status);
}

void enqueue_sweep(const Pipeline &q, const FilterBufs &fb, const LaunchPlan &p, bool fast, cudaStream_t st, const MatBatch &src) { enqueue_sweep_t(q, fb, p, fast, st, src); }
void enqueue_sweep(const Pipeline &q, const FilterBufs &fb, const LaunchPlan &p, bool fast, cudaStream_t st, const AriBatch &src) { enqueue_sweep_t(q, fb, p, fast, st, src); }
void enqueue_finalize(const Pipeline &q, const FilterBufs &fb, const LaunchPlan &p, int route, cudaStream_t st, const MatBatch &src) { enqueue_finalize_t(q, fb, p, route, st, src); }
void enqueue_finalize(const Pipeline &q, const FilterBufs &fb, const LaunchPlan &p, int route, cudaStream_t st, const AriBatch &src) { enqueue_finalize_t(q, fb, p, route, st, src); }

cudaError_t sweep_limits() {
    cudaError_t e = cudaFuncSetAttribute(k_sweep<ZL_OBJ_RANGE, MatBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_sweep<ZL_OBJ_SUM, MatBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_sweep<ZL_OBJ_RANGE, AriBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_sweep<ZL_OBJ_SUM, AriBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    return e;
}

}  // namespace zl
