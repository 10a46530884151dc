// Index self-checks of the RANGE filter route (ZL_FLAG_DEBUG_CHECKS): a kernel instantiated with CHECK tests every index
// it computes against the extent of what it indexes; the first violation is recorded - code, CTA, index - in the
// handle's record and the access is skipped.  Nothing traps, and an unchecked instantiation compiles the tests away.
#pragma once
#include <stdint.h>

namespace zl {

enum RangeAccess : int {
    ACC_PART = 1, ACC_PTAB, ACC_RCNT, ACC_LIST, ACC_CELLMAX, ACC_BCNT, ACC_META, ACC_SEG, ACC_IDX,
    ACC_COPY_SRC, ACC_COPY_DST, ACC_COPY_ALIGN, ACC_TAB, ACC_ARR, ACC_COLS, ACC_REQS, ACC_SLOT, ACC_KEYS
};

template <bool CHECK>
struct Guard {
    uint32_t *dbg; uint32_t cta;
    __device__ __forceinline__ bool ok(uint64_t i, uint64_t lim, int code) const {
        if (!CHECK) return true;
        if (i < lim) return true;
        if (atomicCAS(&dbg[0], 0u, (uint32_t)code) == 0u) { dbg[1] = cta; dbg[2] = (uint32_t)i; dbg[3] = (uint32_t)(i >> 32); }
        return false;
    }
};

}  // namespace zl
