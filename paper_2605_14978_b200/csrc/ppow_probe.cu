// Measurement aids: a read-only streaming pass over a device buffer (the bandwidth a kernel that only
// reads can reach on this GPU, which is what the scoring pass is measured against besides the copy figure),
// and a query of how many kernels a scoring call launches.
#include "../../include/ppow.h"

#include <cuda_runtime.h>
#include <stdint.h>

namespace ppow {

constexpr int PROBE_THREADS = 256;
constexpr int PROBE_UNROLL = 8;   // 16-byte loads in flight per thread

// XOR of all 32-bit words of data[0 .. units) (16-byte units), folded into *checksum.
__global__ void __launch_bounds__(PROBE_THREADS) stream_read_kernel(const uint4 *__restrict__ data, size_t units,
                                                                    uint32_t *__restrict__ checksum)
{
    const size_t stride = (size_t)gridDim.x * PROBE_THREADS;
    size_t i = (size_t)blockIdx.x * PROBE_THREADS + threadIdx.x;
    uint4 x = make_uint4(0u, 0u, 0u, 0u);
    for (; i + (PROBE_UNROLL - 1) * stride < units; i += PROBE_UNROLL * stride) {
        uint4 v[PROBE_UNROLL];
#pragma unroll
        for (int j = 0; j < PROBE_UNROLL; ++j) v[j] = __ldcs(data + i + j * stride);
#pragma unroll
        for (int j = 0; j < PROBE_UNROLL; ++j) {
            x.x ^= v[j].x; x.y ^= v[j].y; x.z ^= v[j].z; x.w ^= v[j].w;
        }
    }
    for (; i < units; i += stride) {
        const uint4 v = __ldcs(data + i);
        x.x ^= v.x; x.y ^= v.y; x.z ^= v.z; x.w ^= v.w;
    }
    uint32_t w = x.x ^ x.y ^ x.z ^ x.w;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) w ^= __shfl_xor_sync(0xffffffffu, w, o);
    if ((threadIdx.x & 31) == 0 && w != 0u) atomicXor(checksum, w);
}

}  // namespace ppow

extern "C" ppow_status ppow_stream_read_probe(const void *data, size_t bytes, uint32_t *checksum, void *cuda_stream)
{
    if (!data || !checksum || bytes == 0 || bytes % 16 != 0 || ((uintptr_t)data % 16) != 0) return PPOW_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return PPOW_ERR_CUDA;
    if (cudaMemsetAsync(checksum, 0, sizeof(uint32_t), stream) != cudaSuccess) return PPOW_ERR_CUDA;
    const size_t units = bytes / 16;
    size_t want = (units + ppow::PROBE_THREADS - 1) / ppow::PROBE_THREADS;
    const size_t resident = (size_t)sms * 8;   // 8 CTAs of 256 threads fill an SM
    const unsigned grid = (unsigned)(want < resident ? want : resident);
    ppow::stream_read_kernel<<<grid, ppow::PROBE_THREADS, 0, stream>>>((const uint4 *)data, units, checksum);
    return cudaGetLastError() == cudaSuccess ? PPOW_OK : PPOW_ERR_CUDA;
}
