// ppow_score_windows_noalloc: the scoring pass for callers that cannot provide scratch memory.
//
// ppow_score_windows needs a device workspace, and somebody has to allocate it.  Some callers
// cannot: a plain-C plugin or scheduler thread that sits beside a training framework has no handle
// on the framework's caching allocator, and the framework has usually claimed the whole device, so
// a raw cudaMalloc from the side either fails or stalls the device in the middle of a step; other
// callers run under a "nothing is allocated after start-up" rule.  For them the workspace lives
// here, in a fixed array in device global memory that is part of the loaded library image.
//
// Consequences the caller has to know about:
//   - every GPU that loads the library holds PPOW_NOALLOC_SCRATCH_BYTES until the process exits;
//   - requests that need more than that are refused (PPOW_ERR_UNSUPPORTED), nothing is launched;
//   - all calls on one device share the one array: two calls that overlap on the GPU (different
//     streams, or different host threads) race on it and corrupt each other's results.  The array
//     keeps the previous call's contents; the parts that must start at zero (work counter and
//     error word) are cleared on the stream at the start of every call;
//   - the first call on each device resolves the array's device address (cudaGetSymbolAddress),
//     which may load the module; make that first call outside any stream capture.  The address is
//     remembered per device ordinal for the life of the process: a process that destroys a device's
//     context (cudaDeviceReset) must not use this entry point on that device afterwards;
//   - the call's error word lives at the head of the array: read it with
//     ppow_noalloc_read_error_flags before the next call on the device overwrites it.
#include "../../include/ppow.h"

#include <cuda_runtime.h>

#include <mutex>

#define PPOW_NOALLOC_SCRATCH_BYTES (4u * 1024u * 1024u)
#define PPOW_NOALLOC_MAX_DEVICES 64

// In host code this name is only a handle for the runtime's symbol lookup, not a device address.
static __device__ __align__(256) unsigned char ppow_noalloc_scratch[PPOW_NOALLOC_SCRATCH_BYTES];

namespace {

std::mutex g_setup_lock;
void *g_scratch_addr[PPOW_NOALLOC_MAX_DEVICES];   // device address of the array, per device ordinal

// Device address of the scratch array on the current device; resolved once per device.
ppow_status scratch_address(void **addr)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return PPOW_ERR_CUDA;
    if (dev < 0 || dev >= PPOW_NOALLOC_MAX_DEVICES) return PPOW_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> guard(g_setup_lock);
    if (g_scratch_addr[dev] == nullptr) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, ppow_noalloc_scratch) != cudaSuccess || p == nullptr) return PPOW_ERR_CUDA;
        g_scratch_addr[dev] = p;
    }
    *addr = g_scratch_addr[dev];
    return PPOW_OK;
}

}  // namespace

extern "C" size_t ppow_noalloc_scratch_bytes(void) { return PPOW_NOALLOC_SCRATCH_BYTES; }

extern "C" ppow_status ppow_score_windows_noalloc(const ppow_params *params,
                                                  const void *draft_logits, const void *target_logits,
                                                  const int32_t *draft_tokens, const float *uniforms,
                                                  const int32_t *valid_len, const float *ref_logp,
                                                  const ppow_outputs *out, void *cuda_stream)
{
    if (!params) return PPOW_ERR_INVALID_ARG;
    const size_t need = ppow_score_workspace_bytes(params);   // 0 for parameters the scoring call would refuse
    if (need == 0) return (params->K > 32) ? PPOW_ERR_UNSUPPORTED : PPOW_ERR_INVALID_ARG;
    if (params->N == 0) return out ? PPOW_OK : PPOW_ERR_INVALID_ARG;
    if (need > PPOW_NOALLOC_SCRATCH_BYTES) return PPOW_ERR_UNSUPPORTED;   // beyond the built-in scratch
    void *scratch = nullptr;
    const ppow_status st = scratch_address(&scratch);
    if (st != PPOW_OK) return st;
    // the scoring call clears the counter and the error word at the head of the workspace itself
    return ppow_score_windows(params, draft_logits, target_logits, draft_tokens, uniforms, valid_len, ref_logp, out,
                              scratch, PPOW_NOALLOC_SCRATCH_BYTES, cuda_stream);
}

// The error word of the last ppow_score_windows_noalloc call on the current device (it sits at the head of
// the shared array): same semantics as ppow_read_error_flags, nothing allocated.
extern "C" ppow_status ppow_noalloc_read_error_flags(uint32_t *flags_host, void *cuda_stream)
{
    if (!flags_host) return PPOW_ERR_INVALID_ARG;
    void *scratch = nullptr;
    const ppow_status st = scratch_address(&scratch);
    if (st != PPOW_OK) return st;
    return ppow_read_error_flags(scratch, flags_host, cuda_stream);
}
