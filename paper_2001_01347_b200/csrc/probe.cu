// Measurement aid: a kernel that only loads what the filter pass loads.
#include "zl_device.cuh"
#include "zl_types.cuh"
#include "../../include/zipline_debug.h"

namespace zl {

// ------------------------------------------------------------------------------ read probe
// Measurement aid: nothing but the loads of a row-prefix pass.  A warp per row reads the first count[row]
// timestamps of the row with 16-byte loads (8-byte loads for odd lengths or a misaligned base), 256 a round,
// and folds them into a checksum so that the loads cannot be dropped.  Timed beside k_filter it shows what the
// memory system delivers for the same bytes in the same access pattern.
__global__ void __launch_bounds__(128) k_probe_read(const int64_t *ts, const int32_t *count, long long rows, int R,
                                                  unsigned long long *sink) {
    const int lane = threadIdx.x & 31;
    const long long row = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (row >= rows) return;
    const int64_t *rp = ts + (size_t)row * R;
    const int L = max(0, min(R, __ldg(count + row)));
    const bool vec2 = (R % 2 == 0) && (((uintptr_t)ts & 15) == 0);
    unsigned long long acc = 0;
    for (int base = 0; base < L; base += 256) {
        if (vec2) {
            longlong2 v[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int i = base + 64 * k + 2 * lane;
                v[k] = i < L ? *reinterpret_cast<const longlong2 *>(rp + i) : make_longlong2(0, 0);
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) acc += (unsigned long long)(v[k].x ^ v[k].y);
        } else {
            int64_t v[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) { const int i = base + 32 * k + lane; v[k] = i < L ? ldg64(rp + i) : 0; }
#pragma unroll
            for (int k = 0; k < 8; ++k) acc += (unsigned long long)v[k];
        }
    }
    if (acc == 0x5eedf00dull) atomicAdd(sink, acc);               // practically never: keeps the loads alive
}

}  // namespace zl

extern "C" {

zl_status zl_probe_read_batched(const int64_t *d_ts, const int32_t *d_count, int64_t rows, int32_t R,
                                uint64_t *d_sink, void *cuda_stream) {
    if (!d_ts || !d_count || !d_sink || rows < 1 || R < 1) return ZL_ERR_INVALID_ARG;
    if (((uintptr_t)d_ts & 7) || ((uintptr_t)d_count & 3) || ((uintptr_t)d_sink & 7)) return ZL_ERR_INVALID_ARG;
    const long long blocks = (rows + 3) / 4;                      // four warps, one row each, per CTA
    if (blocks > 0x7fffffffLL) return ZL_ERR_UNSUPPORTED;
    zl::k_probe_read<<<(unsigned)blocks, 128, 0, (cudaStream_t)cuda_stream>>>(d_ts, d_count, (long long)rows, R,
                                                                            (unsigned long long *)d_sink);
    return cudaGetLastError() == cudaSuccess ? ZL_OK : ZL_ERR_CUDA;
}

}  // extern "C"
