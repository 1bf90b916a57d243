// Bounds-checked build (-DPPOW_CHECKED): every index that a kernel computes from the problem's sizes
// (N, K, V, valid lengths, work items, tiles, token ids, pipeline stages) goes through PPOW_CHECK before
// it is used.  A failed check never traps: it counts the failure, remembers the first failing site, sets
// PPOW_FLAG_BOUNDS in the call's error word when one is at hand, and the access is skipped.  The ordinary
// build compiles the checks away.  This is the library's stand-in for a memory checker: run the shape and
// path tests against the checked library and require ppow_checked_failures() == 0.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#ifdef PPOW_CHECKED
namespace ppow {
// one counter per translation unit (no relocatable device code); ppow_checked_failures() adds them up
static __device__ unsigned int g_check_failures;
static __device__ unsigned int g_check_first_site;

__device__ __forceinline__ bool check_failed(unsigned int site, unsigned int *error_word)
{
    atomicAdd(&g_check_failures, 1u);
    atomicCAS(&g_check_first_site, 0u, site);
    if (error_word) atomicOr(error_word, 4u /* PPOW_FLAG_BOUNDS */);
    return false;
}

static inline int read_check_counters(unsigned int *failures, unsigned int *first_site)
{
    unsigned int f = 0, s = 0;
    if (cudaMemcpyFromSymbol(&f, g_check_failures, sizeof f) != cudaSuccess) return 1;
    if (cudaMemcpyFromSymbol(&s, g_check_first_site, sizeof s) != cudaSuccess) return 1;
    *failures += f;
    if (*first_site == 0) *first_site = s;
    return 0;
}
}  // namespace ppow
// true if the index is fine; otherwise records the failure and yields false (skip the access)
#define PPOW_CHECK(cond, site, error_word) ((cond) ? true : ppow::check_failed((site), (error_word)))
#else
#define PPOW_CHECK(cond, site, error_word) (true)
#endif

// Check sites (reported by ppow_checked_failures): 1xx row reduction, 2xx window scan, 3xx selection, 4xx training side.
