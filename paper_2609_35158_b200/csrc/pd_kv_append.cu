// One-token KV append into the paged cache: a pure 16-byte-vector copy.
//
// Every decode step the new token's K and V rows join the context of their
// sequence (Sec. 2.1). One CTA per sequence; each thread moves one 16-byte
// chunk of one KV head's K or V row. The destination slot follows from the
// sequence's current length and its page-table row.
#include "pd_kernels.cuh"
#include "pd_ptx.cuh"

namespace pd {

namespace {

__global__ void __launch_bounds__(256) kv_append_kernel(const AppendParams p) {
    const int b = blockIdx.x;
    grid_dependency_wait();  // the previous step's kernels still read the pools and the lengths
    launch_dependents();
    const int pos = p.ctx_lens[b];
    __syncthreads();  // everyone has read the length before thread 0 advances it
    const int logical = pos / kPageSize, slot = pos % kPageSize;
    int page = -1;
    bool ok = pos >= 0 && logical < p.MP;
    if (ok) {
        page = p.page_table[static_cast<size_t>(b) * p.MP + logical];
        ok = page >= 0 && page < p.num_pages;
    }
    if (!ok) {
        if (threadIdx.x == 0 && atomicCAS(p.status, kDevOk, pos < 0 || logical >= p.MP ? kDevBadLength : kDevBadPage) == kDevOk) {
            p.status[1] = b;
            p.status[2] = (pos < 0 || logical >= p.MP) ? pos : page;
        }
        return;
    }
    const int chunks_per_row = p.D / 8;                 // 16-byte chunks in one head row
    const int chunks_per_tensor = p.Hkv * chunks_per_row;
    for (int c = threadIdx.x; c < 2 * chunks_per_tensor; c += blockDim.x) {
        const int which = c / chunks_per_tensor;        // 0 = K, 1 = V
        const int rem = c - which * chunks_per_tensor;
        const int kvh = rem / chunks_per_row, j = rem - kvh * chunks_per_row;
        const __nv_bfloat16 *src = (which ? p.v_new : p.k_new) + (static_cast<size_t>(b) * p.Hkv + kvh) * p.D + j * 8;
        __nv_bfloat16 *dst = (which ? p.v_pages : p.k_pages) +
                             ((static_cast<size_t>(page) * p.Hkv + kvh) * kPageSize + slot) * p.D + j * 8;
        *reinterpret_cast<uint4 *>(dst) = __ldg(reinterpret_cast<const uint4 *>(src));
    }
    if (p.advance && threadIdx.x == 0) p.ctx_lens[b] = pos + 1;
}

}  // namespace

cudaError_t launch_kv_append(const AppendParams &p, cudaStream_t stream) {
    if (p.B == 0) return cudaSuccess;
    return launch_pdl(kv_append_kernel, dim3(p.B), dim3(256), 0, stream, p.pdl != 0, p);
}

}  // namespace pd
