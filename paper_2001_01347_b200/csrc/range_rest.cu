// The last kernel of the RANGE filter route (k_range_rest): whatever the filter kernel left undone, in one launch.
//   - instances with many survivors: cell scan, refinement and bucket sweep (zl_heavy.cuh), four phases;
//   - instances whose survivor lists overflowed: the segment sweep (zl_sweep.cuh), one phase;
//   - every instance: minimum over its partial results, barrier, wait, status and the per-worker indices.
// The phases of the first two kinds run only when a flag of the call says that some instance needs them; a grid-wide
// barrier follows each of them, so the grid is no larger than what is resident together.  In a
// call whose instances were all finished by the filter kernel the kernel is the index recovery alone, with no barrier.
#include "zl_heavy.cuh"
#include "zl_sweep.cuh"
#include "zl_host.h"

namespace zl {

constexpr int REST_THREADS = 512;                                  // CTA size of the kernel
constexpr unsigned GRID_POLL_LIMIT = 1u << 22;                     // polls of a grid-wide barrier before it gives up

// Every CTA of the grid arrives at the counter; the k-th barrier of the kernel is passed when gridDim.x * k arrivals
// have been counted.  What the CTAs wrote before the barrier is visible, past the L1 cache, to loads after it.  A CTA
// that polls GRID_POLL_LIMIT times without seeing the count reports it through `gaveup` and goes on: the call then ends
// with ZL_ERR_TIMEOUT for every instance instead of never ending.
__device__ __forceinline__ bool grid_barrier(unsigned int *arrivals, unsigned int *gaveup, unsigned int k) {
    __shared__ unsigned int ok;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(arrivals, 1u);
        const unsigned int want = gridDim.x * k;
        unsigned int polls = 0;
        bool seen = false;
        while (!(seen = ldcg32(arrivals) >= want) && ++polls < GRID_POLL_LIMIT) __nanosleep(64);
        if (!seen) atomicExch(gaveup, 1u);
        __threadfence();
        ok = seen;
    }
    __syncthreads();
    return ok != 0;
}

struct RestParams {
    int n, R, B, nres, nseg;
    int32_t *idx; int64_t *barrier; int64_t *wait; int32_t *status;
};

template <class SRC>
__global__ void __launch_bounds__(REST_THREADS) k_range_rest(const SRC src, const SweepParams SP, const RestParams P, FilterBufs F) {
    // debug handles: clock stamps 6..9 of the CTA's record (the records of the route's first kernel have room for them)
    unsigned long long *stamps = F.dbg && (int)blockIdx.x < F.maxctas ? (unsigned long long *)(F.dbg + 16) + (size_t)blockIdx.x * 16 : nullptr;
#define ZL_STAMP(k) do { if (stamps && threadIdx.x == 0) { unsigned long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); stamps[k] = t_; } } while (0)
    ZL_STAMP(6);
    const RowEnds first = finalize_first_ends(src, P.B, P.n, P.R);
    // (Input, read before the wait: this is not the call's first kernel, and it starts only when every CTA of its predecessor
    // has exited, i.e. has passed its own wait, so whatever produced the input before the call had completed by then.)
    grid_dep_wait();
    ZL_STAMP(7);
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ uint64_t tmp[34];
    __shared__ uint32_t tile[SCAN_TILE];
    __shared__ SweepShared sh;
    unsigned int k = 0;
    bool ok = true;
    const uint4 fl4 = __ldcg(reinterpret_cast<const uint4 *>(F.flags));        // [0] .. [3] together
    if (F.hint && blockIdx.x == 0 && threadIdx.x == 0) note_hint(F, fl4.x != 0u);   // for the host's next call
    if ((fl4.x | fl4.y | fl4.z) == 0) return;                     // the tail kernel finished every instance of the call
    const uint64_t fl = ((uint64_t)fl4.y << 32) | fl4.x;
    // in the same round of loads: what the outputs of the warp's first rows need (read again below if a phase ran)
    const FirstResult fr = finalize_first_result(SP.meta, SP.seg, P.B, P.n, P.nres);
    if ((uint32_t)fl) {
        // some instance has more survivors than one CTA finishes
        heavy_tilemax(SP.meta, F, P.B, tmp);
        ok &= grid_barrier(F.flags + 4, F.flags + 5, ++k);
        heavy_cellscan(SP.meta, F, P.B, tmp, tile);
        ok &= grid_barrier(F.flags + 4, F.flags + 5, ++k);
        heavy_refine(SP.meta, F, P.B);
        ok &= grid_barrier(F.flags + 4, F.flags + 5, ++k);
        heavy_buckets(SP.meta, F, P.n, P.nres, SP.seg, P.B, smem, tmp);
        ok &= grid_barrier(F.flags + 4, F.flags + 5, ++k);
    }
    // the same value in every CTA: the flag is raised by the filter kernel, or by the refinement before a barrier
    if (k ? ldcg32(F.flags + 1) != 0u : (uint32_t)(fl >> 32) != 0u) {
        sweep_items<ZL_OBJ_RANGE>(SP, src, sh, smem);
        ok &= grid_barrier(F.flags + 4, F.flags + 5, ++k);
    }
    if (k && ldcg32(F.flags + 5)) ok = false;                     // some CTA gave up at a barrier
    ZL_STAMP(8);
    finalize_all(src, P.B, P.n, P.R, P.nseg, F, P.nres, ZL_OBJ_RANGE, 1, SP.meta, SP.seg, P.idx, P.barrier, P.wait, P.status,
                 ok ? (uint32_t)ZL_OK : (uint32_t)ZL_ERR_TIMEOUT, &first, k ? nullptr : &fr, stamps);
    ZL_STAMP(9);
#undef ZL_STAMP
}

// Dynamic shared memory of the kernel: the larger of the bucket sweep's batch and the segment sweep's workspace.
static size_t rest_smem(const FilterBufs &fb, const LaunchPlan &p) { return std::max((size_t)fb.capb * 20, p.smem); }

template <class SRC>
static cudaError_t enqueue_range_rest_t(const Pipeline &q, const FilterBufs &fb, const LaunchPlan &p, cudaStream_t st, const SRC &src) {
    SweepParams sp;
    sp.ts = q.ts; sp.meta = q.meta; sp.seg = q.seg;
    sp.n = q.n; sp.R = q.R; sp.B = q.B; sp.nseg = p.nseg; sp.nres = q.nres; sp.G = p.G_rest; sp.cap = p.cap;
    sp.flags = q.flags; sp.target = p.target_rest; sp.filter = 1;
    sp.need = nullptr;
    sp.max_rounds = q.max_rounds;
    RestParams P;
    P.n = q.n; P.R = q.R; P.B = q.B; P.nres = q.nres; P.nseg = p.nseg;
    P.idx = q.idx; P.barrier = q.barrier; P.wait = q.wait; P.status = q.status;
    const size_t smem = rest_smem(fb, p);
    // as many CTAs as are resident together, and no more than the largest phase has items
    int per_sm = q.rest_per_sm;
    if (per_sm < 1) {
        cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_range_rest<SRC>, REST_THREADS, smem);
        if (e != cudaSuccess) return e;
        if (per_sm < 1) return cudaErrorLaunchOutOfResources;
    }
    const long long rb = ((q.n + 31) / 32 + REST_THREADS / 32 - 1) / (REST_THREADS / 32);   // CTAs' worth of warps for an instance's outputs
    const long long tiles = (fb.fcells + SCAN_TILE - 1) / SCAN_TILE, ngroups = (fb.nbk + fb.grp - 1) / fb.grp;
    const long long most = std::max(std::max(rb, tiles), std::max<long long>(std::max<long long>(fb.nreg, ngroups), p.nseg)) * q.B;
    const int grid = (int)std::max<long long>(1, std::min<long long>((long long)per_sm * q.num_sms, most));
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(REST_THREADS); cfg.dynamicSmemBytes = smem; cfg.stream = st;
    // An ordinary launch of no more CTAs than are resident together (a cooperative launch would say the same, but is not
    // scheduled early); the barriers give up after their poll limit in any case.
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = ((q.pdl_off >> 3) & 1) ? 0 : 1;
    return cudaLaunchKernelEx(&cfg, k_range_rest<SRC>, src, sp, P, fb);
}

cudaError_t enqueue_range_rest(const Pipeline &q, const FilterBufs &fb, const LaunchPlan &p, cudaStream_t st, const MatBatch &src) { return enqueue_range_rest_t(q, fb, p, st, src); }
cudaError_t enqueue_range_rest(const Pipeline &q, const FilterBufs &fb, const LaunchPlan &p, cudaStream_t st, const AriBatch &src) { return enqueue_range_rest_t(q, fb, p, st, src); }

cudaError_t range_rest_limits() {
    cudaError_t e = cudaFuncSetAttribute(k_range_rest<MatBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_range_rest<AriBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    return e;
}

}  // namespace zl
