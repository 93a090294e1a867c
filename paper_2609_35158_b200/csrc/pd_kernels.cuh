// Parameter blocks and host-side launchers shared by the kernels and the C ABI.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

namespace pd {

constexpr int kPageSize = 16;       // tokens per page
constexpr int kMaxBatch = 4096;     // prefix sums of page counts live in shared memory
constexpr int kMaxLevels = 12;      // levels of the range plan (geometrically shrinking ranges, then a tail level)
// plan[0..1] total units (lo, hi), [2] levels, [3] ranges, [4] workers, then from word 8 one record of four
// words per level (start lo, start hi, pages per range, index of its first range) plus a closing sentinel
constexpr int kPlanHeaderWords = 8;
constexpr int kPlanWords = kPlanHeaderWords + 4 * (kMaxLevels + 1);
// status[0] code, [1] sequence, [2] detail, [3] unused, [4] next range to claim, [5] workers finished,
// [6] merge CTAs finished (only counted when the merge kernel reports completion to the host itself)
constexpr int kStatusWords = 8;
constexpr int kSchedNext = 4, kSchedDone = 5, kMergeDone = 6;

// Device-side fault codes latched in status[0] (first one wins).
constexpr int kDevOk = 0;
constexpr int kDevBadPage = 1;      // page id outside [0, num_pages)
constexpr int kDevBadLength = 2;    // ctx_len negative or past the page table
constexpr int kDevTimeout = 3;      // bounded wait on an asynchronous copy ran out

struct AttnParams {
    const __nv_bfloat16 *q;     // [B][Hq][D]
    const int32_t *page_table;  // [B][MP]
    const int32_t *ctx_lens;    // [B]
    __nv_bfloat16 *out;         // [B][Hq][D]
    float *lse;                 // [B][Hq] or null
    float *part_o;              // [slots][G][D] unnormalised partial outputs
    float2 *part_ml;            // [slots][G]    (running max in log2 units, running sum)
    int32_t *cum_pages;         // [B+1] exclusive prefix sum of pages per sequence (written by CTA 0)
    int32_t *plan;              // [kPlanWords]
    int32_t *status;            // [kStatusWords]
    int32_t B, Hq, Hkv, G, MP;
    int32_t num_pages;
    float scale_log2;           // sm_scale * log2(e)
    int32_t split_pages;        // 0 = automatic plan, > 0 = one level of ranges of that many pages
    int32_t max_ranges;         // partial slots available beyond one per (sequence, KV head)
    int32_t min_pages_auto;     // lower bound on pages per range in automatic mode
    int32_t halving_levels;     // automatic plan: number of levels whose ranges halve the remaining fair share
    int32_t static_fair_max;    // automatic plan: with a fair share of at most this many pages per worker, one equal range each (0 = never)
    int32_t tail_pages;         // automatic plan: pages per range of the last level
    int32_t pdl;                // launch with programmatic stream serialization
    // fused one-token append (all null / 0 for plain attention): ctx_lens holds the lengths BEFORE the
    // append; the kernel attends over ctx_lens + 1 tokens, takes the new token's K/V rows from k_new / v_new,
    // writes them into the pools and finally adds 1 to every length
    const __nv_bfloat16 *k_new, *v_new;  // [B][Hkv][D]
    __nv_bfloat16 *k_pool_w, *v_pool_w;  // the pools, writable
    int32_t *ctx_lens_w;
    int32_t fused;
    // FP8 pages (null for bf16 pools): {k_scale, v_scale, 0, 0} fp32 per (page, KV head)
    const float *kv_scales;
    int32_t merge_rows;         // rows per CTA of the merge kernel, 0 = chosen from the row count
    // Host-visible result (null / 0 otherwise): the merge kernel delivers every final row to out_host, the
    // device alias of a pinned host buffer [B][Hq][D] (rows the split kernel wrote to `out` are forwarded), and
    // its last CTA stores done_value to done_flag (device alias of a pinned host word) once all rows are out
    __nv_bfloat16 *out_host;
    int32_t *done_flag;
    int32_t done_value;
    unsigned long long *trace;  // optional [workers][4] ns timestamps: kernel entry, first data, last data, exit
};

struct AppendParams {
    const __nv_bfloat16 *k_new, *v_new;  // [B][Hkv][D]
    __nv_bfloat16 *k_pages, *v_pages;    // [NP][Hkv][16][D]
    const int32_t *page_table;
    int32_t *ctx_lens;
    int32_t *status;
    int32_t B, Hkv, D, MP;
    int32_t num_pages;
    int32_t advance;
    int32_t pdl;  // launch with programmatic stream serialization
};

struct TransferParams {
    __nv_bfloat16 *k_pages, *v_pages;    // [NP][Hkv][16][D] (read by gather, written by scatter)
    void *packed;                        // [packed pages][2][Hkv][16][D] (written by gather, read by scatter)
    const int32_t *page_table;           // [B][MP]
    const int32_t *page_begin, *page_end;    // [B] logical page range of every sequence
    const long long *packed_page_offset;     // [B] index of the sequence's first page in the packed buffer
    int32_t *status;
    int32_t B, Hkv, D, MP;
    int32_t num_pages;
    int32_t pdl;
    // FP8 pools: elem_bytes = 1 and the scale records [NP][Hkv][4] fp32 travel with their page (a packed page is
    // then K block, V block, Hkv records); bf16 pools: elem_bytes = 2, scales = null
    int32_t elem_bytes;
    float *scales;
};

struct PrefillParams {
    const __nv_bfloat16 *q;     // [total_q][Hq][D] packed new-token queries
    const int32_t *q_indptr;    // [B+1]
    const int32_t *page_table;  // [B][MP]
    const int32_t *ctx_lens;    // [B] lengths including the new tokens
    __nv_bfloat16 *out;         // [total_q][Hq][D]
    float *lse;                 // [total_q][Hq] or null
    int32_t *status;
    int32_t B, Hq, Hkv, G, MP;
    int32_t num_pages;
    float scale_log2;
    int32_t pdl;
    unsigned long long *trace;  // optional [trace_ctas][8] SM-clock cycles per phase of row thread 0
    int32_t trace_ctas;
    int32_t reverse_tiles;      // schedule a sequence's last query tiles (the longest contexts) first
    int32_t *order;             // [B] sequences by decreasing work, written by a small kernel before the attention (null = index order)
};

struct AppendTokensParams {
    const __nv_bfloat16 *k_new, *v_new;  // [total][Hkv][D]
    const int32_t *q_indptr;             // [B+1]
    __nv_bfloat16 *k_pages, *v_pages;
    const int32_t *page_table;
    int32_t *ctx_lens;
    int32_t *status;
    int32_t B, Hkv, D, MP;
    int32_t num_pages;
    int32_t pdl;
};

// Shape of one compiled variant of the split kernel.
// Whole-page FP8 quantisation: bf16 pools -> e4m3 pools + scale records.
struct QuantizeParams {
    const __nv_bfloat16 *k_pages, *v_pages;  // [num_pages][Hkv][16][D]
    const int32_t *tokens_in_page;           // [num_pages] leading slots that hold tokens
    uint8_t *k8, *v8;                        // [num_pages][Hkv][16][D]
    float *scales;                           // [num_pages][Hkv][4]
    int64_t num_pages;
    int32_t Hkv, D, pdl;
};

// One-token append into FP8 pools.
struct AppendFp8Params {
    const __nv_bfloat16 *k_new, *v_new;  // [B][Hkv][D]
    uint8_t *k8, *v8;
    float *scales;
    const int32_t *page_table;
    int32_t *ctx_lens;
    int32_t *status;
    int32_t B, Hkv, D, MP, num_pages, advance, pdl;
};

struct AttnVariant {
    int head_dim, warps, stages, hilo;
};

// Launches `kernel` so that it may overlap the tail of the previous kernel in the stream (programmatic
// dependent launch); every kernel of this library waits on the grid dependency before its first read
// of global memory, so this is safe after any predecessor.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, bool pdl,
                       Args &&...args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// Launchers (defined next to their kernels). They return the CUDA error of the launch.
cudaError_t launch_kv_append(const AppendParams &p, cudaStream_t stream);
cudaError_t prepare_decode_attn(const AttnVariant &v, size_t *smem_bytes);  // opt-in shared memory, once
cudaError_t launch_decode_attn(const AttnVariant &v, const CUtensorMap &tm_k, const CUtensorMap &tm_v,
                               const AttnParams &p, int num_ctas, size_t smem_bytes, cudaStream_t stream);
cudaError_t launch_lse_merge(int head_dim, const AttnParams &p, cudaStream_t stream);
// FP8 pages (head_dim 128): the split kernel writes the same partials and plan, so launch_lse_merge follows it
cudaError_t prepare_decode_attn_fp8(int head_dim);
cudaError_t launch_decode_attn_fp8(int head_dim, const CUtensorMap &tm_k, const CUtensorMap &tm_v, const AttnParams &p, int num_ctas,
                                   cudaStream_t stream);
cudaError_t launch_kv_quantize_pages(const QuantizeParams &p, cudaStream_t stream);
cudaError_t launch_kv_append_fp8(const AppendFp8Params &p, cudaStream_t stream);
cudaError_t prepare_prefill_attn(int head_dim);  // opt-in shared memory, once
cudaError_t launch_prefill_attn(int head_dim, const CUtensorMap &tm_k, const CUtensorMap &tm_v, const PrefillParams &p,
                                int max_q_len, cudaStream_t stream);
cudaError_t launch_kv_append_tokens(const AppendTokensParams &p, int max_q_len, cudaStream_t stream);
cudaError_t launch_kv_transfer(const TransferParams &p, bool scatter, int num_sms, cudaStream_t stream);

}  // namespace pd
