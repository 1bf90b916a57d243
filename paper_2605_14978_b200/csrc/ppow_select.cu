// ADAW window selection: indices of the n_keep largest scores, ordered by (score descending,
// index ascending).  Keys are made unique by the window index, so the result is deterministic.
//
// Two paths:
//   N <= RANK_MAX_N : rank by counting.  Every window's rank is the number of windows that sort
//                     before it; the window writes itself to selected[rank] if rank < n_keep.
//                     O(N^2) compares but fully parallel, no sort passes, no scratch.
//   larger N        : bitonic sort of 64-bit (key, index) pairs in the workspace, one launch per
//                     global stage, shared-memory stages fused.
#include "../../include/ppow.h"

#include "ppow_checked.cuh"

#include <cuda_runtime.h>

#include <atomic>

namespace ppow {

constexpr int RANK_MAX_N = 16384;
constexpr int RANK_THREADS = 256;
constexpr int SORT_THREADS = 512;
constexpr int SORT_TILE = 2 * SORT_THREADS * 2;   // 2048 keys sorted per CTA in shared memory

// Monotone map float -> uint32 such that a larger score gives a SMALLER key (so ascending key
// order is descending score order).  -0.0 is folded onto +0.0 first.
__device__ __forceinline__ uint32_t descending_key(float score)
{
    const uint32_t b = __float_as_uint(score + 0.0f);
    const uint32_t asc = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
    return ~asc;
}

__global__ void __launch_bounds__(RANK_THREADS) select_rank_kernel(const float *__restrict__ score, int32_t N,
                                                                   int32_t n_keep, int32_t *__restrict__ selected,
                                                                   uint8_t *__restrict__ mask)
{
    extern __shared__ uint32_t s_key[];   // [N]
    for (int32_t j = threadIdx.x; j < N; j += RANK_THREADS) s_key[j] = descending_key(__ldg(score + j));
    __syncthreads();

    const int lane = threadIdx.x & 31;
    const int32_t warps_per_block = RANK_THREADS / 32;
    const int32_t total_warps = gridDim.x * warps_per_block;
    for (int32_t i = blockIdx.x * warps_per_block + (threadIdx.x >> 5); i < N; i += total_warps) {
        const uint32_t ki = s_key[i];
        int32_t cnt = 0;
        for (int32_t j = lane; j < N; j += 32) {
            const uint32_t kj = s_key[j];
            cnt += (kj < ki) || (kj == ki && j < i);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
        if (lane == 0) {
            const bool keep = cnt < n_keep;
            if (keep && PPOW_CHECK(cnt >= 0 && i < N, 301, nullptr)) selected[cnt] = i;
            if (mask && PPOW_CHECK(i >= 0 && i < N, 302, nullptr)) mask[i] = keep ? 1 : 0;
        }
    }
}

// ---- bitonic path -------------------------------------------------------------------------------

__global__ void sort_init_kernel(const float *__restrict__ score, int32_t N, uint32_t n_pad,
                                 unsigned long long *__restrict__ keys)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_pad) return;
    keys[i] = (i < (uint32_t)N) ? (((unsigned long long)descending_key(score[i]) << 32) | i)
                                : 0xffffffffffffffffull;
}

__device__ __forceinline__ void compare_exchange(unsigned long long &a, unsigned long long &b, bool ascending)
{
    if ((a > b) == ascending) {
        const unsigned long long t = a; a = b; b = t;
    }
}

// All stages with stride < SORT_TILE of merge size k, for the tile owned by this CTA.
// first_j is the largest stride to run here (min(k/2, SORT_TILE/2)).
__global__ void __launch_bounds__(SORT_THREADS) sort_local_kernel(unsigned long long *__restrict__ keys, uint32_t k_lo,
                                                                   uint32_t k_hi)
{
    __shared__ unsigned long long s[SORT_TILE];
    const uint32_t base = blockIdx.x * SORT_TILE;
    for (uint32_t t = threadIdx.x; t < SORT_TILE; t += SORT_THREADS) s[t] = keys[base + t];
    __syncthreads();
    for (uint32_t k = k_lo; k <= k_hi; k <<= 1) {
        uint32_t j = (k >> 1) < (SORT_TILE >> 1) ? (k >> 1) : (SORT_TILE >> 1);
        for (; j > 0; j >>= 1) {
            for (uint32_t t = threadIdx.x; t < SORT_TILE / 2; t += SORT_THREADS) {
                const uint32_t lo = ((t & ~(j - 1)) << 1) | (t & (j - 1));
                const bool asc = (((base + lo) & k) == 0);
                if (PPOW_CHECK(lo + j < (uint32_t)SORT_TILE, 303, nullptr)) compare_exchange(s[lo], s[lo + j], asc);
            }
            __syncthreads();
        }
    }
    for (uint32_t t = threadIdx.x; t < SORT_TILE; t += SORT_THREADS) keys[base + t] = s[t];
}

__global__ void sort_global_step_kernel(unsigned long long *__restrict__ keys, uint32_t n_pad, uint32_t j, uint32_t k)
{
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n_pad / 2) return;
    const uint32_t lo = ((t & ~(j - 1)) << 1) | (t & (j - 1));
    if (!PPOW_CHECK(lo + j < n_pad, 304, nullptr)) return;
    unsigned long long a = keys[lo], b = keys[lo + j];
    const bool asc = ((lo & k) == 0);
    if ((a > b) == asc) { keys[lo] = b; keys[lo + j] = a; }
}

__global__ void sort_emit_kernel(const unsigned long long *__restrict__ keys, int32_t N, int32_t n_keep,
                                 int32_t *__restrict__ selected, uint8_t *__restrict__ mask)
{
    const int32_t r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= N) return;
    const int32_t idx = (int32_t)(keys[r] & 0xffffffffull);
    if (!PPOW_CHECK(idx >= 0 && idx < N, 305, nullptr)) return;
    if (r < n_keep) selected[r] = idx;
    if (mask) mask[idx] = (r < n_keep) ? 1 : 0;
}

static uint32_t next_pow2(uint32_t x)
{
    uint32_t p = 1;
    while (p < x) p <<= 1;
    return p;
}

}  // namespace ppow

using namespace ppow;

extern "C" size_t ppow_select_workspace_bytes(int32_t N)
{
    if (N <= 0 || N > (1 << 24)) return 0;
    if (N <= RANK_MAX_N) return 256;   // unused by the ranking path; kept non-zero so callers can pass one buffer
    uint32_t n_pad = next_pow2((uint32_t)N);
    if (n_pad < (uint32_t)SORT_TILE) n_pad = SORT_TILE;
    return (size_t)n_pad * sizeof(unsigned long long);
}

extern "C" ppow_status ppow_select_windows(const float *score, int32_t N, int32_t n_keep,
                                           int32_t *selected, uint8_t *mask,
                                           void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (N < 0 || N > (1 << 24) || n_keep < 0 || n_keep > N) return PPOW_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (N == 0) return PPOW_OK;
    if (!score || (n_keep > 0 && !selected)) return PPOW_ERR_INVALID_ARG;
    if (n_keep == 0) {
        if (mask && cudaMemsetAsync(mask, 0, (size_t)N, stream) != cudaSuccess) return PPOW_ERR_CUDA;
        return PPOW_OK;
    }
    if (N <= RANK_MAX_N) {
        // launch limits of the device, looked up once (host calls of a few microseconds each)
        static std::atomic<int> sms_of[64];
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return PPOW_ERR_CUDA;
        int sms = (dev >= 0 && dev < 64) ? sms_of[dev].load(std::memory_order_relaxed) : 0;
        if (sms <= 0) {
            if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
                return PPOW_ERR_CUDA;
            if (cudaFuncSetAttribute(select_rank_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     RANK_MAX_N * (int)sizeof(uint32_t)) != cudaSuccess)
                return PPOW_ERR_CUDA;
            if (dev >= 0 && dev < 64) sms_of[dev].store(sms, std::memory_order_relaxed);
        }
        const size_t smem = (size_t)N * sizeof(uint32_t);
        int grid = (N + (RANK_THREADS / 32) - 1) / (RANK_THREADS / 32);
        if (grid > sms * 4) grid = sms * 4;
        select_rank_kernel<<<grid, RANK_THREADS, smem, stream>>>(score, N, n_keep, selected, mask);
        if (cudaGetLastError() != cudaSuccess) {
            if (dev >= 0 && dev < 64) sms_of[dev].store(0, std::memory_order_relaxed);   // look the limits up again next time
            return PPOW_ERR_CUDA;
        }
        return PPOW_OK;
    }

    const size_t need = ppow_select_workspace_bytes(N);
    if (!workspace || ((uintptr_t)workspace % 256) || workspace_bytes < need) return PPOW_ERR_WORKSPACE;
    unsigned long long *keys = (unsigned long long *)workspace;
    uint32_t n_pad = next_pow2((uint32_t)N);
    if (n_pad < (uint32_t)SORT_TILE) n_pad = SORT_TILE;
    sort_init_kernel<<<(n_pad + 255) / 256, 256, 0, stream>>>(score, N, n_pad, keys);
    const uint32_t tiles = n_pad / SORT_TILE;
    // merge sizes up to the tile: entirely in shared memory
    sort_local_kernel<<<tiles, SORT_THREADS, 0, stream>>>(keys, 2, SORT_TILE);
    for (uint32_t k = SORT_TILE * 2; k <= n_pad; k <<= 1) {
        for (uint32_t j = k >> 1; j >= (uint32_t)SORT_TILE; j >>= 1)
            sort_global_step_kernel<<<(n_pad / 2 + 255) / 256, 256, 0, stream>>>(keys, n_pad, j, k);
        sort_local_kernel<<<tiles, SORT_THREADS, 0, stream>>>(keys, k, k);
    }
    sort_emit_kernel<<<(N + 255) / 256, 256, 0, stream>>>(keys, N, n_keep, selected, mask);
    return cudaGetLastError() == cudaSuccess ? PPOW_OK : PPOW_ERR_CUDA;
}

#ifdef PPOW_CHECKED
namespace ppow {
int read_check_counters_score(unsigned int *f, unsigned int *s);
int read_check_counters_train(unsigned int *f, unsigned int *s);
}
#endif

extern "C" ppow_status ppow_checked_failures(uint32_t *failures_host, uint32_t *first_site_host)
{
    if (!failures_host) return PPOW_ERR_INVALID_ARG;
#ifdef PPOW_CHECKED
    unsigned int f = 0, s = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return PPOW_ERR_CUDA;
    if (read_check_counters(&f, &s) || read_check_counters_score(&f, &s) || read_check_counters_train(&f, &s))
        return PPOW_ERR_CUDA;
    *failures_host = f;
    if (first_site_host) *first_site_host = s;
    return PPOW_OK;
#else
    *failures_host = 0;
    if (first_site_host) *first_site_host = 0;
    return PPOW_ERR_UNSUPPORTED;   // not the bounds-checked build
#endif
}

extern "C" const char *ppow_status_string(ppow_status status)
{
    switch (status) {
    case PPOW_OK: return "ok";
    case PPOW_ERR_INVALID_ARG: return "invalid argument";
    case PPOW_ERR_UNSUPPORTED: return "unsupported request";
    case PPOW_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case PPOW_ERR_CUDA: return "CUDA runtime error";
    case PPOW_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

extern "C" int ppow_version(void) { return 100; }
