// k_small: the whole search for instances of a few thousand timestamps in one launch, a CTA per instance - column
// scans, the optional sortedness check, the sweep of the instance as a single time segment, barrier, wait, status and
// the per-worker indices.  Nothing goes through global scratch: the instance's record and its result stay in shared
// memory.  The steps are the plain route's (k_prologue, k_sweep, k_finalize), run back to back by one CTA.
#include "zl_sweep.cuh"
#include "zl_host.h"

namespace zl {

template <int OBJ>
__global__ void __launch_bounds__(1024) k_small(const SweepParams P, const MatBatch src, int check_sorted,
                                                int32_t *idx, int64_t *barrier, int64_t *wait, int32_t *status) {
    grid_dep_wait();
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ SweepShared sh;
    __shared__ uint64_t s[4][32];
    __shared__ InstMeta sM;
    __shared__ SegResult res;
    __shared__ int unsorted;
    const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
    const int n = P.n, R = P.R;
    uint32_t *curA = (uint32_t *)smem;
    uint32_t *curB = curA + n;
    unsigned char *kb = smem + (((size_t)2 * n * sizeof(uint32_t) + 15) & ~(size_t)15);
    unsigned char *kb2 = kb + (size_t)P.cap * 8;
    uint32_t *kcnt = (uint32_t *)(kb2 + (size_t)P.cap * 8);
    for (int b = blockIdx.x; b < P.B; b += gridDim.x) {
        const MatRows rows = src.inst(b, n, R);
        // ---- column scans: tmin = min_p e^p_1, t0 = max_p e^p_1, lmin = min_p e^p_R, the span; validity
        uint64_t mn1 = ~0ull, mx1 = 0, mnR = ~0ull, mxR = 0;      // order-preserving unsigned images of int64
        for (int p = tid; p < n; p += nt) {
            const MatRow rw = rows.row(p);
            const uint64_t e1 = (uint64_t)rw.at(0) ^ (1ull << 63);
            const uint64_t eR = (uint64_t)rw.at(R - 1) ^ (1ull << 63);
            mn1 = min(mn1, e1); mx1 = max(mx1, e1);
            mnR = min(mnR, eR); mxR = max(mxR, eR);
        }
        mn1 = warp_reduce(mn1, OpMin()); mx1 = warp_reduce(mx1, OpMax());
        mnR = warp_reduce(mnR, OpMin()); mxR = warp_reduce(mxR, OpMax());
        if (lane == 0) { s[0][warp] = mn1; s[1][warp] = mx1; s[2][warp] = mnR; s[3][warp] = mxR; }
        if (tid == 0) unsorted = 0;
        __syncthreads();
        if (check_sorted) {
            // every row non-decreasing?  The instance is small: all its adjacent pairs, a pair per thread and step
            bool bad = false;
            const int64_t *inst = src.ts + (size_t)b * n * R;
            for (int f = tid; f < n * R; f += nt)
                if ((f % R) != 0 && ldg64(inst + f) < ldg64(inst + f - 1)) bad = true;
            if (bad) unsorted = 1;
        }
        if (tid == 0) {
            uint64_t a = s[0][0], c = s[1][0], d = s[2][0], e = s[3][0];
            for (int w = 1; w < nw; ++w) { a = min(a, s[0][w]); c = max(c, s[1][w]); d = min(d, s[2][w]); e = max(e, s[3][w]); }
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
                if (OBJ == ZL_OBJ_SUM && m.tend > (uint64_t)INT64_MAX / (uint64_t)n) m.status = ZL_ERR_UNSUPPORTED;
            }
            sM = m;
        }
        __syncthreads();
        InstMeta M = sM;
        if (M.status == ZL_OK && unsorted) M.status = ZL_ERR_UNSORTED;
        // ---- the sweep, the whole instance as one segment
        if (M.status == ZL_OK) {
            if (M.use32) {
                const BatchWS<uint32_t> ws{(Key<uint32_t> *)kb, (Key<uint32_t> *)kb2, kcnt, P.cap};
                sweep_segment<uint32_t, OBJ>(P, M, rows, sh, curA, curB, ws, 0, res);
            } else {
                SweepParams Q = P;
                Q.cap = P.cap / 2;                  // 16-byte nodes: half as many fit
                const BatchWS<uint64_t> ws{(Key<uint64_t> *)kb, (Key<uint64_t> *)kb2, kcnt, Q.cap};
                sweep_segment<uint64_t, OBJ>(Q, M, rows, sh, curA, curB, ws, 0, res);
            }
        }
        __syncthreads();
        // ---- outputs
        int fst = M.status;
        if (fst == ZL_OK && res.status != ZL_OK) fst = res.status;
        if (fst == ZL_OK && !res.valid) fst = ZL_ERR_TIMEOUT;      // cannot happen for valid input
        int64_t bar = INT64_MIN, wt = INT64_MIN;
        if (fst == ZL_OK) {
            const int64_t tm = M.tmin + (int64_t)(res.t - 1);
            bar = OBJ == ZL_OBJ_RANGE ? tm + (int64_t)res.d : tm;
            wt = (int64_t)res.d;
        }
        if (tid == 0) {
            wait[b] = wt;
            barrier[b] = bar;
            if (status) status[b] = fst;
        }
        for (int p = tid; p < n; p += nt)
            idx[(size_t)b * n + p] = fst == ZL_OK ? last_index_not_after(rows.row(p), R, bar) : -1;
        __syncthreads();
    }
}

void enqueue_small(const Pipeline &q, const LaunchPlan &p, cudaStream_t st, const MatBatch &src) {
    SweepParams sp;
    sp.ts = q.ts; sp.meta = q.meta; sp.seg = q.seg;
    sp.n = q.n; sp.R = q.R; sp.B = q.B; sp.nseg = 1; sp.nres = q.nres; sp.G = p.G_small; sp.cap = p.cap;
    sp.flags = q.flags; sp.target = p.target_small; sp.filter = 0;
    sp.need = nullptr;
    sp.max_rounds = q.max_rounds;
    const int grid = std::min(q.B, 32 * q.num_sms);
    const int check = (q.flags & ZL_FLAG_CHECK_SORTED) ? 1 : 0;
    if (q.objective == ZL_OBJ_RANGE)
        launch_dep(!((q.pdl_off >> 9) & 1), k_small<ZL_OBJ_RANGE>, dim3(grid), dim3(p.threads_small), p.smem, st, sp, src, check, q.idx, q.barrier, q.wait, q.status);
    else
        launch_dep(!((q.pdl_off >> 9) & 1), k_small<ZL_OBJ_SUM>, dim3(grid), dim3(p.threads_small), p.smem, st, sp, src, check, q.idx, q.barrier, q.wait, q.status);
}

cudaError_t small_limits() {
    cudaError_t e = cudaFuncSetAttribute(k_small<ZL_OBJ_RANGE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_small<ZL_OBJ_SUM>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    return e;
}

}  // namespace zl
