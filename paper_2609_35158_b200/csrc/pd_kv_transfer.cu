// KV page gather / scatter: packing the pages of a sequence's new tokens into one
// contiguous buffer and unpacking such a buffer into freshly assigned pages.
//
// This is the device-side data movement of the cross-pool KV transfer in the
// disaggregated prefill model (Eq. 3, the B * dL * K / BW term): the prefill
// worker gathers, the transport (out of scope here) ships one contiguous buffer,
// the decode worker scatters. A pool page holds all KV heads contiguously
// ([H_kv][16][d] bf16), so a packed page is the K block followed by the V block
// and every copy is a run of 16-byte vectors. Pure bandwidth, bit-exact.
#include "pd_kernels.cuh"
#include "pd_ptx.cuh"

namespace pd {

namespace {

template <bool SCATTER>
__global__ void __launch_bounds__(256) kv_transfer_kernel(const TransferParams p) {
    const int b = blockIdx.y;
    grid_dependency_wait();
    launch_dependents();
    const int pb = p.page_begin[b], pe = p.page_end[b];
    const long long base = p.packed_page_offset[b];
    const size_t vec_per_block = static_cast<size_t>(p.Hkv) * kPageSize * p.D / 8;  // 16-byte vectors in a K (or V) block
    for (int lp = pb + blockIdx.x; lp < pe; lp += gridDim.x) {
        int page = (lp >= 0 && lp < p.MP) ? p.page_table[static_cast<size_t>(b) * p.MP + lp] : -1;
        if (page < 0 || page >= p.num_pages) {
            if (threadIdx.x == 0 && atomicCAS(p.status, kDevOk, kDevBadPage) == kDevOk) {
                p.status[1] = b;
                p.status[2] = page;
            }
            continue;
        }
        uint4 *packed = reinterpret_cast<uint4 *>(p.packed) + (static_cast<size_t>(base) + (lp - pb)) * 2 * vec_per_block;
        uint4 *kpool = reinterpret_cast<uint4 *>(p.k_pages) + static_cast<size_t>(page) * vec_per_block;
        uint4 *vpool = reinterpret_cast<uint4 *>(p.v_pages) + static_cast<size_t>(page) * vec_per_block;
        // four independent 16-byte loads in flight per thread before the first store
        for (size_t i = threadIdx.x; i < 2 * vec_per_block; i += 4 * 256) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const size_t j = i + u * 256;
                if (j < 2 * vec_per_block) {
                    const uint4 *pool = j < vec_per_block ? kpool + j : vpool + (j - vec_per_block);
                    v[u] = SCATTER ? __ldcs(packed + j) : __ldcs(pool);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const size_t j = i + u * 256;
                if (j < 2 * vec_per_block) {
                    uint4 *pool = j < vec_per_block ? kpool + j : vpool + (j - vec_per_block);
                    if (SCATTER) *pool = v[u]; else __stcs(packed + j, v[u]);
                }
            }
        }
    }
}

}  // namespace

cudaError_t launch_kv_transfer(const TransferParams &p, bool scatter, int num_sms, cudaStream_t stream) {
    if (p.B == 0) return cudaSuccess;
    int per_seq = (16 * num_sms + p.B - 1) / p.B;  // CTAs per sequence: about 16 per SM over the batch
    if (per_seq < 1) per_seq = 1;
    if (per_seq > p.MP) per_seq = p.MP;
    const dim3 grid(per_seq, p.B);
    if (scatter) return launch_pdl(kv_transfer_kernel<true>, grid, dim3(256), 0, stream, p.pdl != 0, p);
    return launch_pdl(kv_transfer_kernel<false>, grid, dim3(256), 0, stream, p.pdl != 0, p);
}

}  // namespace pd
