// Read-only streaming probe: the practical HBM ceiling for a kernel that, like decode attention, only reads.
// The roofline denominator of the decode kernels is a measured COPY bandwidth (read + write); a read-once scan
// can run above it. This kernel reads a buffer once with 16-byte streaming loads and keeps nothing, so that
// benchmarks can quote the read-only figure of the same GPU next to the copy figure.
#include "../../include/pd_debug.h"

#include <cuda_runtime.h>

namespace {

__global__ void read_probe_kernel(const uint4 *__restrict__ src, size_t n, uint4 *sink) {
    size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x;
    const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
    uint4 acc = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll 8
    for (; i < n; i += stride) {
        const uint4 v = __ldcs(src + i);
        acc.x ^= v.x; acc.y ^= v.y; acc.z ^= v.z; acc.w ^= v.w;
    }
    // a store the compiler cannot rule out keeps the loads alive; it practically never happens
    if (acc.x == 0x12345678u && acc.y == 77u && acc.z == 1u && acc.w == 2u) sink[0] = acc;
}

}  // namespace

extern "C" int pd_read_probe(const void *src, size_t bytes, int32_t blocks, int32_t threads, void *sink16, void *stream) {
    if (src == nullptr || sink16 == nullptr || (reinterpret_cast<uintptr_t>(src) & 15u) != 0 ||
        (reinterpret_cast<uintptr_t>(sink16) & 15u) != 0 || bytes < 16 || blocks < 1 || threads < 32 || threads > 1024)
        return PD_ERR_INVALID_ARG;
    read_probe_kernel<<<blocks, threads, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const uint4 *>(src), bytes / 16,
                                                                              static_cast<uint4 *>(sink16));
    return cudaGetLastError() == cudaSuccess ? PD_OK : PD_ERR_CUDA;
}
