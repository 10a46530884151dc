// RANGE filter route, instances with many survivors, as four kernels of their own (k_tilemax, k_cellscan, k_refine,
// k_buckets): for shapes so large that such instances are the rule, each phase gets a grid of its own size instead of
// sharing the one of the route's single last kernel.  The phases themselves are in zl_heavy.cuh.
#include "zl_heavy.cuh"
#include "zl_host.h"

namespace zl {

__global__ void __launch_bounds__(256) k_tilemax(const InstMeta *meta, FilterBufs F, int B) {
    grid_dep_wait();
    __shared__ uint64_t tmp[34];
    if (F.flags[0] == 0) return;                                  // no instance takes this route in this call
    heavy_tilemax(meta, F, B, tmp);
}

__global__ void __launch_bounds__(256) k_cellscan(const InstMeta *meta, FilterBufs F, int B) {
    grid_dep_wait();
    __shared__ uint64_t tmp[34];
    __shared__ uint32_t tile[SCAN_TILE];
    if (F.flags[0] == 0) return;
    heavy_cellscan(meta, F, B, tmp, tile);
}

__global__ void __launch_bounds__(256) k_refine(InstMeta *meta, FilterBufs F, int B) {
    grid_dep_wait();
    if (F.flags[0] == 0) return;
    heavy_refine(meta, F, B);
}

__global__ void __launch_bounds__(256) k_buckets(const InstMeta *meta, FilterBufs F, int n, int nres, SegResult *seg, int B) {
    grid_dep_wait();
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ uint64_t tmp[34];
    if (F.flags[0] == 0) return;
    heavy_buckets(meta, F, n, nres, seg, B, smem, tmp);
}

void enqueue_heavy(const Pipeline &q, const FilterBufs &fb, cudaStream_t st) {
    // fixed-size grids that return at once when no instance needs them
    const int tiles = (fb.fcells + SCAN_TILE - 1) / SCAN_TILE;
    const int wide = 4 * q.num_sms;
    launch_dep(!((q.pdl_off >> 3) & 1), k_tilemax, dim3(std::min(tiles * q.B, wide)), dim3(256), 0, st, (const InstMeta *)q.meta, fb, q.B);
    launch_dep(!((q.pdl_off >> 4) & 1), k_cellscan, dim3(std::min(tiles * q.B, wide)), dim3(256), 0, st, (const InstMeta *)q.meta, fb, q.B);
    launch_dep(!((q.pdl_off >> 5) & 1), k_refine, dim3(std::min(fb.nreg * q.B, 8 * wide)), dim3(256), 0, st, q.meta, fb, q.B);
    const int ngroups = (fb.nbk + fb.grp - 1) / fb.grp;
    const int bthreads = std::max(64, std::min(256, fb.capb / 4));
    launch_dep(!((q.pdl_off >> 6) & 1), k_buckets, dim3(std::min(ngroups * q.B, wide)), dim3(bthreads), (size_t)fb.capb * 20, st,
               (const InstMeta *)q.meta, fb, q.n, q.nres, q.seg, q.B);
}

cudaError_t heavy_limits() {
    return cudaFuncSetAttribute(k_buckets, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
}

}  // namespace zl
