// Checked build (-DBAOC_CHECKED): the stand-in for a memory checker on machines where none may be run.
//
// Every CTA of the streaming kernels first validates what it is about to touch: that its tile exists, that the tile
// names a block of the table, that the tile starts inside that block, and that every range of library-managed memory
// it will read or write (moments, previous gradient, codes, absmax values, row/column statistics and partial sums)
// lies inside the buffer the caller bound.  The first violation is recorded in a status record (what, which kernel, the
// offending numbers) and the CTA returns without touching memory: nothing traps, nothing asserts, the context stays
// usable, and the host reads the record with baoc_check_status().  Caller-owned arrays (gradients, parameters), whose
// true extents the library cannot know, are covered from the outside: the test harness surrounds every buffer with
// guard words and verifies them after the launches.
//
// In a normal build the macros below expand to nothing, the kernels keep their signatures and no check is compiled.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

#include "baoc_internal.h"

namespace baoc {

enum CheckCode : unsigned int { kChkNone = 0, kChkTileIndex = 1, kChkBlockIndex = 2, kChkTileStart = 3, kChkRange = 4, kChkNull = 5 };
enum CheckKernel : unsigned int {
    kKerStatsStep = 1, kKerStatsCombine = 2, kKerSampleGather = 3, kKerFinalSums = 4, kKerFinalHist = 5, kKerMomentReduce = 6,
    kKerFactoredReduce = 7, kKerFactoredCombine = 8, kKerFusedStep = 9, kKerSelfTest = 10, kKerFactoredNorms = 11, kKerFinalLast = 12, kKerSelectFirst = 13
};
#ifdef BAOC_CHECKED
#define BAOC_CHECK_PARAM , const CheckCtx ck
#define BAOC_CHECK_ARG(ctx) , ctx

static __device__ CheckRecord g_check;    // one per translation unit; the host side of each unit fetches its own

__device__ __forceinline__ bool check_fail(unsigned code, unsigned kernel, long long a, long long b, long long c, long long d) {
    if (atomicCAS(&g_check.code, 0u, code) == 0u) {
        g_check.kernel = kernel; g_check.a = a; g_check.b = b; g_check.c = c; g_check.d = d;
    }
    return false;
}
// this CTA's tile exists, names a block, and starts inside it
__device__ __forceinline__ bool check_tile(const CheckCtx& ck, unsigned kernel, long long tile, unsigned block, long long base,
                                           long long numel) {
    if (tile >= ck.n_tiles) return check_fail(kChkTileIndex, kernel, tile, ck.n_tiles, 0, 0);
    if (block >= unsigned(ck.n_blocks)) return check_fail(kChkBlockIndex, kernel, block, ck.n_blocks, tile, 0);
    if (base < 0 || base >= numel) return check_fail(kChkTileStart, kernel, base, numel, block, tile);
    return true;
}
// [p, p + bytes) lies inside the bound buffer
__device__ __forceinline__ bool check_range(const CheckCtx& ck, unsigned kernel, const void* p, long long bytes, int what) {
    const char* q = static_cast<const char*>(p);
    if (q == nullptr) return check_fail(kChkNull, kernel, what, 0, 0, 0);
    if (bytes < 0 || q < ck.lo || q + bytes > ck.hi)
        return check_fail(kChkRange, kernel, what, q - ck.lo, bytes, ck.hi - ck.lo);
    return true;
}
__device__ __forceinline__ bool check_caller_ptr(unsigned kernel, const void* p, int what) {
    if (p == nullptr) return check_fail(kChkNull, kernel, what, 0, 0, 0);
    return true;
}

// Host side, once per translation unit: copy the unit's record out and clear it.
#define BAOC_DEFINE_CHECK_FETCH(name)                                                            \
    int name(CheckRecord* out) {                                                                 \
        CheckRecord zero{};                                                                      \
        cudaError_t e = cudaMemcpyFromSymbol(out, g_check, sizeof(CheckRecord));                 \
        if (e == cudaSuccess) e = cudaMemcpyToSymbol(g_check, &zero, sizeof(CheckRecord));       \
        return int(e);                                                                           \
    }
#else
#define BAOC_CHECK_PARAM
#define BAOC_CHECK_ARG(ctx)
#define BAOC_DEFINE_CHECK_FETCH(name) \
    int name(CheckRecord* out) { *out = CheckRecord{}; return 0; }
#endif

}  // namespace baoc
