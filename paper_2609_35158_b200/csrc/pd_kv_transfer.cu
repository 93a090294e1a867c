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

// The copy is driven by the bulk-copy engine: one thread per CTA streams 16 KB chunks global -> shared
// memory -> global through a ring of stages, with no register traffic at all. Loads run kBulkAhead chunks
// ahead of stores; the stage of chunk i was last read by the store of chunk i - kBulkStages, after which
// kBulkStages - kBulkAhead - 1 further store groups were committed, so that many may still be pending when
// the stage is reloaded.
constexpr int kBulkChunk = 16384, kBulkStages = 6, kBulkAhead = 3;

template <bool SCATTER>
__global__ void __launch_bounds__(32) kv_transfer_bulk_kernel(const TransferParams p) {
    extern __shared__ __align__(128) uint8_t ring[];
    __shared__ uint64_t bars[kBulkStages];
    const int b = blockIdx.y;
    if (threadIdx.x != 0) return;
    grid_dependency_wait();
    launch_dependents();
    for (int s = 0; s < kBulkStages; ++s) mbar_init(smem_u32(bars + s), 1);
    mbar_init_fence();
    const int pb = p.page_begin[b], pe = p.page_end[b];
    const long long base = p.packed_page_offset[b];
    const uint32_t block_bytes = static_cast<uint32_t>(p.Hkv) * kPageSize * p.D * p.elem_bytes;  // K (or V) block of a page
    const uint32_t scale_bytes = p.scales != nullptr ? static_cast<uint32_t>(p.Hkv) * 16u : 0u;  // the page's scale records
    const uint32_t chunks_per_block = (block_bytes + kBulkChunk - 1) / kBulkChunk;
    const uint32_t chunks_per_page = 2 * chunks_per_block + (scale_bytes ? 1u : 0u);
    const size_t packed_page_bytes = 2 * static_cast<size_t>(block_bytes) + scale_bytes;
    // this CTA's pages: pb + blockIdx.x, + gridDim.x, ...
    const int first = pb + blockIdx.x;
    const long long n_pages = first < pe ? (pe - first + gridDim.x - 1) / gridDim.x : 0;
    const long long n = n_pages * chunks_per_page;
    const uint32_t ring0 = smem_u32(ring);
    bool ok = true;

    // chunk i -> (pool address, packed address, bytes); a page with a bad id is skipped (bytes = 0) and reported
    auto locate = [&](long long i, uint8_t *&pool, uint8_t *&packed, uint32_t &bytes) {
        const int lp = first + static_cast<int>(i / chunks_per_page) * gridDim.x;
        const uint32_t c = static_cast<uint32_t>(i % chunks_per_page);
        const int page = (lp >= 0 && lp < p.MP) ? p.page_table[static_cast<size_t>(b) * p.MP + lp] : -1;
        if (page < 0 || page >= p.num_pages) {
            if (c == 0 && atomicCAS(p.status, kDevOk, kDevBadPage) == kDevOk) {
                p.status[1] = b;
                p.status[2] = page;
            }
            bytes = 0;
            return;
        }
        uint8_t *packed_page = reinterpret_cast<uint8_t *>(p.packed) + (static_cast<size_t>(base) + (lp - pb)) * packed_page_bytes;
        if (c == 2 * chunks_per_block) {  // the scale records
            bytes = scale_bytes;
            pool = reinterpret_cast<uint8_t *>(p.scales) + static_cast<size_t>(page) * scale_bytes;
            packed = packed_page + 2 * static_cast<size_t>(block_bytes);
            return;
        }
        const uint32_t which = c / chunks_per_block, off = (c % chunks_per_block) * kBulkChunk;
        bytes = min(static_cast<uint32_t>(kBulkChunk), block_bytes - off);
        pool = reinterpret_cast<uint8_t *>(which ? p.v_pages : p.k_pages) + static_cast<size_t>(page) * block_bytes + off;
        packed = packed_page + static_cast<size_t>(which) * block_bytes + off;
    };

    for (long long i = 0; i < n + kBulkAhead && ok; ++i) {
        if (i < n) {  // load chunk i
            const int s = static_cast<int>(i % kBulkStages);
            if (i >= kBulkStages) bulk_wait_group_read<kBulkStages - kBulkAhead - 1>();  // the store of chunk i - kBulkStages has read its stage
            uint8_t *pool = nullptr, *packed = nullptr;
            uint32_t bytes;
            locate(i, pool, packed, bytes);
            if (bytes > 0) {
                mbar_arrive_expect_tx(smem_u32(bars + s), bytes);
                bulk_load(ring0 + s * kBulkChunk, SCATTER ? packed : pool, bytes, smem_u32(bars + s));
            } else {
                mbar_arrive(smem_u32(bars + s));  // keep the phase count in step
            }
        }
        const long long j = i - kBulkAhead;
        if (j >= 0) {  // store chunk j
            const int s = static_cast<int>(j % kBulkStages);
            ok = mbar_wait(smem_u32(bars + s), static_cast<uint32_t>((j / kBulkStages) & 1));
            if (!ok) break;
            uint8_t *pool = nullptr, *packed = nullptr;
            uint32_t bytes;
            locate(j, pool, packed, bytes);
            if (bytes > 0) bulk_store(SCATTER ? pool : packed, ring0 + s * kBulkChunk, bytes);
            bulk_commit_group();  // one group per chunk, empty ones included, so the group count follows j
        }
    }
    bulk_wait_all();
    if (!ok && atomicCAS(p.status, kDevOk, kDevTimeout) == kDevOk) {
        p.status[1] = b;
        p.status[2] = blockIdx.x;
    }
}

}  // namespace

cudaError_t launch_kv_transfer(const TransferParams &p, bool scatter, int num_sms, cudaStream_t stream) {
    if (p.B == 0) return cudaSuccess;
    // CTAs per sequence: about 128 per SM over the batch. Many short-lived CTAs of a page or two each measured
    // 6.7 TB/s against 6.0 TB/s for two long-lived CTAs per SM: SMs that get more bandwidth simply take more CTAs.
    int per_seq = (128 * num_sms + p.B - 1) / p.B;
    per_seq = per_seq < 1 ? 1 : (per_seq > p.MP ? p.MP : per_seq);
    const dim3 grid(per_seq, p.B);
    const size_t smem = static_cast<size_t>(kBulkStages) * kBulkChunk;
    // the opt-in is per device and costs a microsecond: set it on every launch rather than track devices
    const cudaError_t e = scatter ? cudaFuncSetAttribute(kv_transfer_bulk_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                         static_cast<int>(smem))
                                  : cudaFuncSetAttribute(kv_transfer_bulk_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                         static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    if (scatter) return launch_pdl(kv_transfer_bulk_kernel<true>, grid, dim3(32), smem, stream, p.pdl != 0, p);
    return launch_pdl(kv_transfer_bulk_kernel<false>, grid, dim3(32), smem, stream, p.pdl != 0, p);
}

}  // namespace pd
