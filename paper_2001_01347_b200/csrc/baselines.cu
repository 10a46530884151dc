// Entry points that need no handle: the paper's heuristic baselines GridScan / FullGridScan (Algorithm 1), the
// constant-interval predictor (phase 1 of ZipLine) and the per-position trace of the sweep for small instances.
#include <algorithm>

#include "zl_batch.cuh"
#include "zl_host.h"

namespace zl {

constexpr int TRACE_MAX = 4096;

// ------------------------------------------------------------------------------ GridScan / FullGridScan
// Value of the point of a sorted row at the shortest distance from e (the earlier one on ties).
__device__ __forceinline__ int64_t nearest_value(const int64_t *row, int R, int64_t e) {
    int lo = 0, hi = R;                           // first index with row[i] >= e
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (ldg64(row + mid) < e) lo = mid + 1; else hi = mid;
    }
    if (lo == 0) return ldg64(row);
    const int64_t left = ldg64(row + lo - 1);
    if (lo == R) return left;
    const int64_t right = ldg64(row + lo);
    return e - left <= right - e ? left : right;
}

// Lowest index of a sorted row that holds value v (v occurs in the row).
__device__ __forceinline__ int first_index_of(const int64_t *row, int R, int64_t v) {
    int lo = 0, hi = R;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (ldg64(row + mid) < v) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// Row with the earliest first timestamp (lowest-numbered on ties); every thread of the block gets it.
__device__ int designated_row(const int64_t *inst, int n, int R, uint64_t *tmp) {
    uint64_t best = ~0ull;                         // (first timestamp, row) packed: timestamps are below 2^62
    uint64_t bestp = 0;
    for (int p = threadIdx.x; p < n; p += blockDim.x) {
        const uint64_t v = (uint64_t)ldg64(inst + (size_t)p * R);
        if (v < best) { best = v; bestp = (uint64_t)p; }
    }
    uint64_t tot;
    block_scan_excl<uint64_t>(best, OpMin(), ~0ull, tmp, &tot);
    uint64_t cand = best == tot ? bestp : ~0ull, totp;
    block_scan_excl<uint64_t>(cand, OpMin(), ~0ull, tmp, &totp);
    return (int)totp;
}

// d_Z of one candidate per CTA.  grid (candidates, B); candidate c = designated point (row c / R, index c % R)
// when full, else point c of the designated row.
__global__ void __launch_bounds__(256) k_gridscan_eval(const int64_t *ts, int n, int R, int full, int64_t *cand) {
    __shared__ uint64_t tmp[34];
    const int b = blockIdx.y, c = blockIdx.x;
    const int64_t *inst = ts + (size_t)b * n * R;
    const int q = full ? c / R : designated_row(inst, n, R, tmp);
    const int j = full ? c % R : c;
    const int64_t e = ldg64(inst + (size_t)q * R + j);
    uint64_t mx = (uint64_t)e, mn = (uint64_t)e;
    for (int p = threadIdx.x; p < n; p += blockDim.x) {
        if (p == q) continue;
        const uint64_t v = (uint64_t)nearest_value(inst + (size_t)p * R, R, e);
        mx = max(mx, v); mn = min(mn, v);
    }
    uint64_t gmx, gmn;
    block_scan_excl<uint64_t>(mx, OpMax(), 0ull, tmp, &gmx);
    block_scan_excl<uint64_t>(mn, OpMin(), ~0ull, tmp, &gmn);
    if (threadIdx.x == 0) cand[(size_t)b * gridDim.x + c] = (int64_t)(gmx - gmn);
}

// First minimal candidate of an instance, then its Z*.  grid B
__global__ void __launch_bounds__(256) k_gridscan_pick(const int64_t *ts, int n, int R, int full, int ncand, const int64_t *cand,
                                                       int32_t *idx, int64_t *barrier, int64_t *wait) {
    __shared__ uint64_t tmp[34];
    const int b = blockIdx.x;
    const int64_t *inst = ts + (size_t)b * n * R;
    uint64_t bd = ~0ull, bc = ~0ull;
    for (int c = threadIdx.x; c < ncand; c += blockDim.x) {
        const uint64_t d = (uint64_t)cand[(size_t)b * ncand + c];
        if (d < bd) { bd = d; bc = (uint64_t)c; }                 // a thread sees its candidates in ascending order
    }
    uint64_t gd, gc;
    block_scan_excl<uint64_t>(bd, OpMin(), ~0ull, tmp, &gd);
    block_scan_excl<uint64_t>(bd == gd ? bc : ~0ull, OpMin(), ~0ull, tmp, &gc);
    const int c = (int)gc;
    const int q = full ? c / R : designated_row(inst, n, R, tmp);
    const int j = full ? c % R : c;
    const int64_t e = ldg64(inst + (size_t)q * R + j);
    uint64_t mx = (uint64_t)e;
    for (int p = threadIdx.x; p < n; p += blockDim.x) {
        int res = j;
        if (p != q) {
            const int64_t v = nearest_value(inst + (size_t)p * R, R, e);
            res = first_index_of(inst + (size_t)p * R, R, v);
            mx = max(mx, (uint64_t)v);
        }
        idx[(size_t)b * n + p] = res;
    }
    uint64_t gmx;
    block_scan_excl<uint64_t>(mx, OpMax(), 0ull, tmp, &gmx);
    if (threadIdx.x == 0) { barrier[b] = (int64_t)gmx; wait[b] = (int64_t)gd; }
}

// ------------------------------------------------------------------------------ predictor
// One CTA per row: e_i = last + i * interval, i = 1..R, written with 16-byte stores where the row allows.
__global__ void __launch_bounds__(256) k_predict(const int64_t *last, const int64_t *interval, int R, int64_t *ts) {
    const size_t row = blockIdx.x;
    const int64_t l = ldg64(last + row), iv = ldg64(interval + row);
    int64_t *out = ts + row * (size_t)R;
    int64_t base = l, step = iv;
    if (l < 0 || iv < 0) { base = -1; step = 0; }                 // marks the instance invalid for the search
    else if (__umul64hi((uint64_t)R, (uint64_t)iv) != 0 || (uint64_t)R * (uint64_t)iv >= (uint64_t)VALUE_LIMIT ||
             (uint64_t)l + (uint64_t)R * (uint64_t)iv >= (uint64_t)VALUE_LIMIT) { base = VALUE_LIMIT; step = 0; }
    if ((R & 1) == 0 && (((uintptr_t)out) & 15) == 0) {
        for (int i = 2 * threadIdx.x; i < R; i += 2 * blockDim.x) {
            longlong2 v;
            v.x = base + (int64_t)(i + 1) * step;
            v.y = base + (int64_t)(i + 2) * step;
            *reinterpret_cast<longlong2 *>(out + i) = v;
        }
    } else {
        for (int i = threadIdx.x; i < R; i += blockDim.x) out[i] = base + (int64_t)(i + 1) * step;
    }
}

// ------------------------------------------------------------------------------ trace
struct TKey {
    uint64_t t; uint32_t f, pad;
    __device__ __forceinline__ bool operator>(const TKey &o) const { return t > o.t || (t == o.t && f > o.f); }
};

__global__ void __launch_bounds__(256) k_trace(const int64_t *ts, int n, int R,
                                               int64_t *om_t, int32_t *om_p, int32_t *om_i, int64_t *delta,
                                               int32_t *first, int64_t *S, int32_t *cnt, int64_t *next,
                                               int64_t *PM, int64_t *d_range, int64_t *w_sum) {
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ uint64_t tmp[34];
    TKey *keys = (TKey *)smem;
    const int N = n * R, b = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
    const int64_t *inst = ts + (size_t)b * N;
    int P = 64;
    while (P < N) P <<= 1;
    // step 1: merge = all (time, worker, iteration) in ascending order
    int64_t t0loc = INT64_MIN;
    for (int f = tid; f < P; f += nt) {
        TKey k;
        if (f < N) { k.t = (uint64_t)ldg64(inst + f); k.f = (uint32_t)f; if (f % R == 0) t0loc = max(t0loc, (int64_t)k.t); }
        else { k.t = ~0ull; k.f = 0xffffffffu; }
        k.pad = 0;
        keys[f] = k;
    }
    uint64_t t0u = warp_reduce((uint64_t)t0loc ^ (1ull << 63), OpMax());
    __shared__ unsigned long long s_t0;
    if (tid == 0) s_t0 = 0;
    __syncthreads();
    if ((tid & 31) == 0) atomicMax(&s_t0, (unsigned long long)t0u);
    __syncthreads();
    const int64_t t0 = (int64_t)(s_t0 ^ (1ull << 63));
    bitonic_sort(keys, P);
    const int ipt = (P + nt - 1) / nt;
    const int k0 = tid * ipt, k1 = min(k0 + ipt, N);
    // steps 2+3: per-element delta / flag / next, then the scans in Omega order
    uint64_t ls = 0, lm = 0;            // lm: max of next, order-preserving unsigned image of int64
    uint32_t lc = 0;
    for (int k = k0; k < k1; ++k) {
        const int f = (int)keys[k].f, i = f % R;
        const int64_t t = (int64_t)keys[k].t;
        ls += (uint64_t)(i == 0 ? t : t - ldg64(inst + f - 1));
        lc += i == 0;
        const int64_t nx = i == R - 1 ? INT64_MAX : ldg64(inst + f + 1);
        lm = max(lm, (uint64_t)((uint64_t)nx ^ (1ull << 63)));
    }
    uint64_t tots, totm;
    uint32_t totc;
    uint64_t s = block_scan_excl<uint64_t>(ls, OpAdd(), 0ull, tmp, &tots);
    uint32_t c = block_scan_excl<uint32_t>(lc, OpAdd(), 0u, (uint32_t *)tmp, &totc);
    uint64_t pmu = block_scan_excl<uint64_t>(lm, OpMax(), 0ull, tmp, &totm);   // 0 is the image of INT64_MIN
    for (int k = k0; k < k1; ++k) {
        const int f = (int)keys[k].f, p = f / R, i = f % R;
        const int64_t t = (int64_t)keys[k].t;
        const int64_t dl = i == 0 ? t : t - ldg64(inst + f - 1);
        const int64_t nx = i == R - 1 ? INT64_MAX : ldg64(inst + f + 1);
        s += (uint64_t)dl;
        c += i == 0;
        const int64_t pm = (int64_t)(pmu ^ (1ull << 63));
        const size_t o = (size_t)b * N + k;
        if (om_t) om_t[o] = t;
        if (om_p) om_p[o] = p;
        if (om_i) om_i[o] = i;
        if (delta) delta[o] = dl;
        if (first) first[o] = i == 0;
        if (S) S[o] = (int64_t)s;
        if (cnt) cnt[o] = (int32_t)c;
        if (next) next[o] = nx;
        if (PM) PM[o] = pm;
        // step 4: objective of the candidate at this position
        if (d_range) { const int64_t g = max(max(t, t0), pm); d_range[o] = g == INT64_MAX ? INT64_MAX : g - t; }
        if (w_sum) w_sum[o] = c == (uint32_t)n ? (int64_t)((uint64_t)n * (uint64_t)t - s) : INT64_MAX;
        pmu = max(pmu, (uint64_t)((uint64_t)nx ^ (1ull << 63)));
    }
}

}  // namespace zl

extern "C" {

int32_t zl_trace_max_elements(void) { return zl::TRACE_MAX; }

zl_status zl_gridscan_batched(const int64_t *d_ts, int32_t B, int32_t n, int32_t R, int32_t full, int64_t *d_scratch,
                              int32_t *d_idx, int64_t *d_barrier, int64_t *d_wait, void *cuda_stream) {
    if (!d_ts || !d_scratch || !d_idx || !d_barrier || !d_wait || B < 1 || n < 1 || R < 1) return ZL_ERR_INVALID_ARG;
    if (B > 65535) return ZL_ERR_UNSUPPORTED;
    const long long ncand = full ? (long long)n * R : R;
    if (ncand > 0x7fffffffLL) return ZL_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int threads = std::max(32, std::min(256, zl::pow2_ceil(n)));
    zl::k_gridscan_eval<<<dim3((unsigned)ncand, B), threads, 0, st>>>(d_ts, n, R, full ? 1 : 0, d_scratch);
    zl::k_gridscan_pick<<<B, 256, 0, st>>>(d_ts, n, R, full ? 1 : 0, (int)ncand, d_scratch, d_idx, d_barrier, d_wait);
    return cudaGetLastError() == cudaSuccess ? ZL_OK : ZL_ERR_CUDA;
}

zl_status zl_predict_batched(const int64_t *d_last, const int64_t *d_interval, int32_t B, int32_t n, int32_t R,
                             int64_t *d_ts, void *cuda_stream) {
    if (!d_last || !d_interval || !d_ts || B < 1 || n < 1 || R < 1) return ZL_ERR_INVALID_ARG;
    if (((uintptr_t)d_last & 7) || ((uintptr_t)d_interval & 7) || ((uintptr_t)d_ts & 15)) return ZL_ERR_INVALID_ARG;
    if ((long long)B * n > 0x7fffffffLL) return ZL_ERR_UNSUPPORTED;
    const int threads = std::max(32, std::min(256, zl::pow2_ceil((R + 1) / 2)));
    zl::k_predict<<<(unsigned)((long long)B * n), threads, 0, (cudaStream_t)cuda_stream>>>(d_last, d_interval, R, d_ts);
    return cudaGetLastError() == cudaSuccess ? ZL_OK : ZL_ERR_CUDA;
}

zl_status zl_trace_batched(const int64_t *d_ts, int32_t B, int32_t n, int32_t R, int64_t *om_t, int32_t *om_p,
                           int32_t *om_i, int64_t *delta, int32_t *first, int64_t *S, int32_t *cnt, int64_t *next,
                           int64_t *PM, int64_t *d_range, int64_t *w_sum, void *cuda_stream) {
    if (!d_ts || B < 1 || n < 1 || R < 1) return ZL_ERR_INVALID_ARG;
    if ((long long)n * R > zl::TRACE_MAX) return ZL_ERR_UNSUPPORTED;
    const int P = std::max(64, zl::pow2_ceil(n * R));
    const size_t smem = (size_t)P * sizeof(zl::TKey);
    cudaError_t e = cudaFuncSetAttribute(zl::k_trace, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(zl::TRACE_MAX * sizeof(zl::TKey)));
    if (e != cudaSuccess) return ZL_ERR_CUDA;
    zl::k_trace<<<B, 256, smem, (cudaStream_t)cuda_stream>>>(d_ts, n, R, om_t, om_p, om_i, delta, first, S, cnt, next, PM, d_range, w_sum);
    return cudaGetLastError() == cudaSuccess ? ZL_OK : ZL_ERR_CUDA;
}

}  // extern "C"
