// The segment sweep (k_sweep: the general route, and the fallback of the bucket route) and k_finalize (minimum over an
// instance's partial results, barrier, per-worker index recovery).
#include "zl_sweep.cuh"
#include "zl_host.h"

namespace zl {

template <int OBJ, class SRC>
__global__ void __launch_bounds__(1024) k_sweep(const SweepParams P, const SRC src) {
    grid_dep_wait();
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ SweepShared sh;
    if (P.need && P.need[1] == 0) return;                        // the fast route finished every instance
    sweep_items<OBJ>(P, src, sh, smem);
}

// ------------------------------------------------------------------------------ finalize
// Every instance's outputs: a warp per 32 rows of an instance.
template <class SRC>
__global__ void __launch_bounds__(256) k_finalize(const SRC src, int B, int n, int R, int nseg, FilterBufs F, int nres,
                                                  int objective, int filter, const InstMeta *meta, const SegResult *seg,
                                                  int32_t *idx, int64_t *barrier, int64_t *wait, int32_t *status) {
    const RowEnds first = finalize_first_ends(src, B, n, R);
    // (Input, read before the wait: this is not the call's first kernel, and it starts only when every CTA of its predecessor
    // has exited, i.e. has passed its own wait, so whatever produced the input before the call had completed by then.)
    grid_dep_wait();
    if (filter == 1 && F.hint && blockIdx.x == 0 && threadIdx.x == 0) note_hint(F, F.flags[0] != 0u);   // for the host's next call
    if (filter == 1 && F.flags[2] == 0) return;                   // the tail kernel finished every instance of the call
    finalize_all(src, B, n, R, nseg, F, nres, objective, filter, meta, seg, idx, barrier, wait, status, 0u, &first);
}

template <class SRC>
static void enqueue_sweep_t(const Pipeline &q, const FilterBufs &fb, const LaunchPlan &p, bool fast, cudaStream_t st, const SRC &src) {
    SweepParams sp;
    sp.ts = q.ts; sp.meta = q.meta; sp.seg = q.seg;
    sp.n = q.n; sp.R = q.R; sp.B = q.B; sp.nseg = p.nseg; sp.nres = q.nres; sp.G = p.G; sp.cap = p.cap;
    sp.flags = q.flags; sp.target = p.target; sp.filter = fast ? 1 : 0;
    sp.need = fast ? fb.flags : nullptr;
    sp.max_rounds = q.max_rounds;
    // with a fast route on, the segment sweep is only the fallback: a small persistent grid
    const int items = p.nseg * q.B;
    const int sweep_ctas = fast ? std::min(items, 2 * q.num_sms) : items;
    if (q.objective == ZL_OBJ_RANGE) launch_dep(!((q.pdl_off >> 7) & 1), k_sweep<ZL_OBJ_RANGE, SRC>, dim3(sweep_ctas), dim3(p.threads), p.smem, st, sp, src);
    else launch_dep(!((q.pdl_off >> 7) & 1), k_sweep<ZL_OBJ_SUM, SRC>, dim3(sweep_ctas), dim3(p.threads), p.smem, st, sp, src);
}

template <class SRC>
static void enqueue_finalize_t(const Pipeline &q, const FilterBufs &fb, const LaunchPlan &p, int route, cudaStream_t st, const SRC &src) {
    const long long warps = (long long)q.B * ((q.n + 31) / 32);
    const int fthreads = (int)std::min<long long>(256, 32 * warps);
    const int grid = (int)std::min<long long>((warps * 32 + fthreads - 1) / fthreads, 16LL * q.num_sms);
    launch_dep(!((q.pdl_off >> 8) & 1), k_finalize<SRC>, dim3(grid), dim3(fthreads), 0, st, src, q.B, q.n, q.R, p.nseg, fb, q.nres, q.objective,
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
