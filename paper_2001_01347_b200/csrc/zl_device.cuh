// Device-side building blocks of the ZipLine kernels: key packing, block-wide
// bitonic sort in shared memory, block-wide scans and reductions.  No CUB/Thrust.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace zl {

constexpr unsigned FULL = 0xffffffffu;

// ---------------------------------------------------------------------------------- keys
// A node of the sweep is (T, V): T = time relative to the instance (tmin -> 1), V = the
// payload the scan needs (RANGE: the same worker's next timestamp; SUM: T minus the same
// worker's previous timestamp).  32-bit instances pack both into one 64-bit word so that the
// sort moves a single register pair; wide instances use a 16-byte pair.
template <typename K> struct Key;

template <> struct Key<uint32_t> {
    uint64_t w;
    __device__ __forceinline__ static Key make(uint32_t t, uint32_t v) { return Key{((uint64_t)t << 32) | v}; }
    __device__ __forceinline__ static Key inf() { return Key{~0ull}; }
    __device__ __forceinline__ uint32_t t() const { return (uint32_t)(w >> 32); }
    __device__ __forceinline__ uint32_t v() const { return (uint32_t)w; }
    __device__ __forceinline__ bool operator>(const Key &o) const { return w > o.w; }
};

template <> struct Key<uint64_t> {
    uint64_t a, b;
    __device__ __forceinline__ static Key make(uint64_t t, uint64_t v) { return Key{t, v}; }
    __device__ __forceinline__ static Key inf() { return Key{~0ull, ~0ull}; }
    __device__ __forceinline__ uint64_t t() const { return a; }
    __device__ __forceinline__ uint64_t v() const { return b; }
    __device__ __forceinline__ bool operator>(const Key &o) const { return a > o.a || (a == o.a && b > o.b); }
};

template <typename K> __device__ __forceinline__ K kinf();
template <> __device__ __forceinline__ uint32_t kinf<uint32_t>() { return 0xffffffffu; }
template <> __device__ __forceinline__ uint64_t kinf<uint64_t>() { return ~0ull; }

// ---------------------------------------------------------------------------------- sort
// Ascending bitonic sort of keys[0..P) in shared memory, P a power of two >= 64, by the whole block
// (blockDim a multiple of 32).  Compare-exchange steps with distance j <= 32 stay inside the 64-key
// block that a warp's 32 consecutive pair indices cover, so runs of such steps are separated by
// __syncwarp() only; steps with a larger distance need the block barrier.
template <typename KeyT>
__device__ __forceinline__ void bitonic_step(KeyT *keys, int i, int j, int k) {
    const int lo = ((i & ~(j - 1)) << 1) | (i & (j - 1));
    const int hi = lo | j;
    const bool up = (lo & k) == 0;
    KeyT x = keys[lo], y = keys[hi];
    if ((x > y) == up) { keys[lo] = y; keys[hi] = x; }
}

template <typename KeyT>
__device__ void bitonic_sort(KeyT *keys, int P) {
    const int tid = threadIdx.x, nt = blockDim.x, half = P >> 1;
    for (int k = 2; k <= P; k <<= 1) {
        int j = k >> 1;
        for (; j > 32; j >>= 1) {
            for (int i = tid; i < half; i += nt) bitonic_step(keys, i, j, k);
            __syncthreads();
        }
        // j <= 32: each warp finishes its own 64-key blocks
        for (int i0 = tid; i0 < half; i0 += nt) {
            for (int jj = j; jj > 0; jj >>= 1) {
                bitonic_step(keys, i0, jj, k);
                __syncwarp();
            }
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------- scans
struct OpMax { template <typename T> __device__ __forceinline__ T operator()(T a, T b) const { return a > b ? a : b; } };
struct OpMin { template <typename T> __device__ __forceinline__ T operator()(T a, T b) const { return a < b ? a : b; } };
struct OpAdd { template <typename T> __device__ __forceinline__ T operator()(T a, T b) const { return a + b; } };

template <typename T> __device__ __forceinline__ T shfl_up(T v, int d) {
    if constexpr (sizeof(T) == 8) return (T)__shfl_up_sync(FULL, (unsigned long long)v, d);
    else return (T)__shfl_up_sync(FULL, (unsigned)v, d);
}
template <typename T> __device__ __forceinline__ T shfl_xor(T v, int d) {
    if constexpr (sizeof(T) == 8) return (T)__shfl_xor_sync(FULL, (unsigned long long)v, d);
    else return (T)__shfl_xor_sync(FULL, (unsigned)v, d);
}
template <typename T> __device__ __forceinline__ T shfl_idx(T v, int s) {
    if constexpr (sizeof(T) == 8) return (T)__shfl_sync(FULL, (unsigned long long)v, s);
    else return (T)__shfl_sync(FULL, (unsigned)v, s);
}

// One value per thread -> exclusive scan over the block in thread order (identity for thread 0)
// and the block total.  tmp: shared, 33 elements of T.  Contains two barriers; every thread calls.
template <typename T, typename Op>
__device__ T block_scan_excl(T x, Op op, T identity, T *tmp, T *total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    T inc = x;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        T y = shfl_up(inc, d);
        if (lane >= d) inc = op(y, inc);
    }
    if (lane == 31) tmp[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        T w = lane < nw ? tmp[lane] : identity;
        T winc = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            T y = shfl_up(winc, d);
            if (lane >= d) winc = op(y, winc);
        }
        T wexc = shfl_up(winc, 1);
        if (lane == 0) wexc = identity;
        if (lane < nw) tmp[lane] = wexc;
        if (lane == nw - 1) tmp[32] = winc;
    }
    __syncthreads();
    T exc = shfl_up(inc, 1);
    if (lane == 0) exc = identity;
    exc = op(tmp[warp], exc);
    *total = tmp[32];
    __syncthreads();                       // tmp may be reused by the caller right away
    return exc;
}

// ---------------------------------------------------------------------------------- slot sort
// Sort in[0..m) by (time, payload) into out[0..m): a counting sort on the time (nslots time slots
// between the batch's earliest and latest time, about one key per slot), then an insertion sort of
// the few keys that share a slot.  A batch in which one slot holds more than SLOT_MAX keys falls back
// to the bitonic network.  cnt: nslots words of shared memory; in and out hold cap >= m keys
// (cap a power of two >= 64); tmp: 34 shared 64-bit words.  All threads of the block call it.
constexpr int SLOT_MAX = 24;

template <typename K>
__device__ void slot_sort(Key<K> *in, Key<K> *out, uint32_t *cnt, int nslots, int m, int cap, uint64_t *tmp) {
    const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
    // range of times in the batch
    K lo = ~(K)0, hi = 0;
    for (int i = tid; i < m; i += nt) { const K t = in[i].t(); lo = min(lo, t); hi = max(hi, t); }
    lo = warp_reduce(lo, OpMin()); hi = warp_reduce(hi, OpMax());
    K *red = (K *)tmp;                                            // 32 entries of at most 8 bytes
    if (lane == 0) red[warp] = lo;
    for (int s = tid; s < nslots; s += nt) cnt[s] = 0;
    __syncthreads();
    for (int w = 0; w < nw; ++w) lo = min(lo, red[w]);
    __syncthreads();
    if (lane == 0) red[warp] = hi;
    __syncthreads();
    for (int w = 0; w < nw; ++w) hi = max(hi, red[w]);
    __syncthreads();
    int sh = 0;
    while (((hi - lo) >> sh) >= (K)nslots) ++sh;                  // slot = (t - lo) >> sh < nslots, monotone in t
    for (int i = tid; i < m; i += nt) atomicAdd(&cnt[(uint32_t)((in[i].t() - lo) >> sh)], 1u);
    __syncthreads();
    {   // exclusive prefix sum of the slot counts, in place; a slot that is too full is noted on the way
        const int per = (nslots + nt - 1) / nt;
        const int s0 = min(tid * per, nslots), s1 = min(s0 + per, nslots);
        uint32_t loc = 0, big = 0;
        for (int s = s0; s < s1; ++s) { loc += cnt[s]; big |= cnt[s] > (uint32_t)SLOT_MAX; }
        uint32_t tot;
        uint32_t run = block_scan_excl<uint32_t>(loc, OpAdd(), 0u, (uint32_t *)tmp, &tot);
        for (int s = s0; s < s1; ++s) { const uint32_t c = cnt[s]; cnt[s] = run; run += c; }
        uint32_t anybig;
        block_scan_excl<uint32_t>(big, OpMax(), 0u, (uint32_t *)tmp, &anybig);
        if (anybig) {
            // many equal or nearly equal times: the comparison network handles any distribution
            int P = 64;
            while (P < m) P <<= 1;
            for (int i = m + tid; i < P; i += nt) in[i] = Key<K>::inf();
            __syncthreads();
            bitonic_sort(in, P);
            for (int i = tid; i < m; i += nt) out[i] = in[i];
            __syncthreads();
            return;
        }
    }
    __syncthreads();
    for (int i = tid; i < m; i += nt) {
        const Key<K> k = in[i];
        out[atomicAdd(&cnt[(uint32_t)((k.t() - lo) >> sh)], 1u)] = k;      // cnt[s] ends as the end of slot s
    }
    __syncthreads();
    for (int s = tid; s < nslots; s += nt) {
        const int e = (int)cnt[s], b = s ? (int)cnt[s - 1] : 0;
        for (int i = b + 1; i < e; ++i) {                        // insertion sort of the slot's keys
            const Key<K> k = out[i];
            int j = i - 1;
            while (j >= b && out[j] > k) { out[j + 1] = out[j]; --j; }
            out[j + 1] = k;
        }
    }
    __syncthreads();
    (void)cap;
}

template <typename T, typename Op>
__device__ __forceinline__ T warp_reduce(T x, Op op) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) x = op(x, shfl_xor(x, d));
    return x;
}

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute has its
// launch prepared while its predecessor in the stream is still running.  grid_dep_wait() blocks until
// the predecessor grid has completed and its writes are visible (a no-op for a normally launched
// kernel); every kernel of the chain calls it first.  No kernel signals early: dependents that became
// resident while a long kernel was still running slowed that kernel down.
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ int64_t ldg64(const int64_t *p) { return (int64_t)__ldg((const long long *)p); }

// ---------------------------------------------------------------------------------- per-lane asynchronous copies
__device__ __forceinline__ void cp_async16(void *smem, const void *gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"((uint32_t)__cvta_generic_to_shared(smem)), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async8(void *smem, const void *gmem) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;\n" ::"r"((uint32_t)__cvta_generic_to_shared(smem)), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
// wait until at most `pending` of this thread's most recent groups are still in flight
__device__ __forceinline__ void cp_async_wait_pending(int pending) {
    switch (pending) {
        case 0: asm volatile("cp.async.wait_group 0;\n" ::: "memory"); break;
        case 1: asm volatile("cp.async.wait_group 1;\n" ::: "memory"); break;
        case 2: asm volatile("cp.async.wait_group 2;\n" ::: "memory"); break;
        case 3: asm volatile("cp.async.wait_group 3;\n" ::: "memory"); break;
        case 4: asm volatile("cp.async.wait_group 4;\n" ::: "memory"); break;
        case 5: asm volatile("cp.async.wait_group 5;\n" ::: "memory"); break;
        case 6: asm volatile("cp.async.wait_group 6;\n" ::: "memory"); break;
        default: asm volatile("cp.async.wait_group 7;\n" ::: "memory"); break;
    }
}

// ---------------------------------------------------------------------------------- bulk copies
// One thread asks the copy engine for a contiguous piece of global memory; the bytes land in shared memory
// and are counted on an mbarrier, whose phase completes when the announced number has arrived.  Both
// addresses and the size are multiples of 16 bytes.  No multicast: the destination is the CTA's own memory.
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t *bar, int arrivals) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(arrivals) : "memory");
}
// An mbarrier has to be invalidated before its bytes serve any other purpose (or are initialised again).
__device__ __forceinline__ void mbar_inval(uint64_t *bar) {
    asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_init_fence() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_copy_g2s(void *dst, const void *src, uint32_t bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// shared-memory reads through ordinary loads come before later writes of the copy engine to the same bytes
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Wait for the phase with the given parity; gives up after a bounded number of polls (each poll may itself be
// suspended by the hardware for a while) and reports it, so that a copy that never lands cannot hang the GPU.
constexpr int MBAR_POLL_LIMIT = 1 << 22;
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t *bar, uint32_t parity) {
    for (int spins = 0; spins < MBAR_POLL_LIMIT; ++spins)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ uint32_t ldcg32(const uint32_t *p) { return __ldcg(p); }
__device__ __forceinline__ uint64_t ldcg64(const uint64_t *p) { return (uint64_t)__ldcg((const unsigned long long *)p); }

}  // namespace zl
