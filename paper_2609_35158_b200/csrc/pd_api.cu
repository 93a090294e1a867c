// C ABI of the paged decode-attention library: context, argument checks,
// tensor-map encoding and kernel launches. See include/pd.h for the contract.
#include "../../include/pd.h"
#include "../../include/pd_debug.h"

#include <chrono>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "pd_decode_plan.cuh"
#include "pd_kernels.cuh"

namespace {

using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || (cudaSetDevice(dev) == cudaSuccess);
    }
    ~DeviceGuard() {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

}  // namespace

struct pd_ctx {
    pd_config cfg{};
    int group = 0;
    int num_sms = 0;
    int num_ctas = 0;
    pd::AttnVariant variant{};
    size_t smem_bytes = 0;
    int max_ranges = 0;
    int min_pages_auto = 1;
    int halving_levels = 0;
    int tail_pages = 16;
    int pdl = 1;
    int merge_rows = 0;
    int prefill_reverse = 1, prefill_order = 1;
    size_t slots = 0;
    // device workspace (one allocation)
    void *workspace = nullptr;
    size_t workspace_bytes = 0;
    float *part_o = nullptr;
    float2 *part_ml = nullptr;
    int32_t *cum_pages = nullptr;
    int32_t *plan = nullptr;
    int32_t *status = nullptr;
    unsigned long long *trace = nullptr;  // per-worker timestamps, only in a PD_ENABLE_TUNING build with PD_TRACE_WORKERS=1
    int trace_workers = 0;
    // staging for pd_decode_step_host
    __nv_bfloat16 *stage_q = nullptr, *stage_k = nullptr, *stage_v = nullptr, *stage_out = nullptr;
    // tensor maps, cached per pool pointer
    EncodeTiledFn encode = nullptr;
    const void *map_k_ptr = nullptr, *map_v_ptr = nullptr;
    alignas(64) CUtensorMap tm_k{};
    alignas(64) CUtensorMap tm_v{};
    // the same for FP8 pools
    const void *map_k8_ptr = nullptr, *map_v8_ptr = nullptr;
    alignas(64) CUtensorMap tm_k8{};
    alignas(64) CUtensorMap tm_v8{};
    // pd_decode_step_host with pinned host buffers: the merge kernel writes the result to the host itself and
    // reports completion through this pinned word, which the host polls instead of synchronising the stream
    int32_t *done_flag_host = nullptr, *done_flag_dev = nullptr;
    int32_t done_seq = 0;
    int64_t host_steps_direct = 0, host_steps_staged = 0;
    __nv_bfloat16 *host_out_alias = nullptr;  // set for the duration of one pd_decode_step_host call
    cudaEvent_t ev_before = nullptr, ev_after = nullptr;  // optional timing hook around the split kernel
    bool prefill_ready = false;
    bool fp8_ready = false;
    int64_t launches = 0;
    char last_error[256] = {0};
};

namespace {

int fail(pd_ctx *ctx, int code, const char *what, cudaError_t err = cudaSuccess) {
    if (ctx != nullptr) {
        if (err != cudaSuccess) std::snprintf(ctx->last_error, sizeof ctx->last_error, "%s: %s", what, cudaGetErrorString(err));
        else std::snprintf(ctx->last_error, sizeof ctx->last_error, "%s", what);
    }
    return code;
}

bool aligned16(const void *p) { return p != nullptr && (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Kernel shape and plan parameters are fixed in the shipped build. A build with -DPD_ENABLE_TUNING reads them
// from the environment once, at pd_create, for experiments; no call after pd_create looks at the environment.
#ifdef PD_ENABLE_TUNING
int tune_int(const char *name, int fallback) {
    const char *v = std::getenv(name);
    return (v != nullptr && *v != '\0') ? std::atoi(v) : fallback;
}
#else
constexpr int tune_int(const char *, int fallback) { return fallback; }
#endif

// 2-D view of a pool: rows = (page, KV head, slot), columns = head_dim bf16.
// Box = 16 rows x 64 columns (128 B) with the 128-byte swizzle.
int encode_pool_map(pd_ctx *ctx, const void *pool, CUtensorMap *out) {
    const pd_config &c = ctx->cfg;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(c.head_dim),
                                static_cast<cuuint64_t>(c.num_pages) * c.num_kv_heads * c.page_size};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(c.head_dim) * 2};
    const cuuint32_t box[2] = {64, static_cast<cuuint32_t>(c.page_size)};
    const cuuint32_t elem_strides[2] = {1, 1};
    const CUresult r = ctx->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(pool), dims, strides, box,
                                   elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                   CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        std::snprintf(ctx->last_error, sizeof ctx->last_error, "cuTensorMapEncodeTiled failed (%d)", static_cast<int>(r));
        return PD_ERR_CUDA;
    }
    return PD_OK;
}

// The same view of an FP8 pool: columns = head_dim bytes, one box = 16 rows x 128 B.
int encode_pool_map_fp8(pd_ctx *ctx, const void *pool, CUtensorMap *out) {
    const pd_config &c = ctx->cfg;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(c.head_dim),
                                static_cast<cuuint64_t>(c.num_pages) * c.num_kv_heads * c.page_size};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(c.head_dim)};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(c.head_dim), static_cast<cuuint32_t>(c.page_size)};  // one row = head_dim bytes
    const cuuint32_t elem_strides[2] = {1, 1};
    const CUresult r = ctx->encode(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(pool), dims, strides, box,
                                   elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                   c.head_dim == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                                   CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        std::snprintf(ctx->last_error, sizeof ctx->last_error, "cuTensorMapEncodeTiled failed (%d)", static_cast<int>(r));
        return PD_ERR_CUDA;
    }
    return PD_OK;
}

int check_batch(pd_ctx *ctx, int32_t batch) {
    if (ctx == nullptr) return PD_ERR_INVALID_ARG;
    if (batch < 0 || batch > ctx->cfg.max_batch) return fail(ctx, PD_ERR_INVALID_ARG, "batch outside [0, max_batch]");
    return PD_OK;
}

}  // namespace

extern "C" {

int pd_version(void) { return 100; }

const char *pd_status_string(int status) {
    switch (status) {
        case PD_OK: return "ok";
        case PD_ERR_INVALID_ARG: return "invalid argument";
        case PD_ERR_UNSUPPORTED: return "unsupported geometry";
        case PD_ERR_CUDA: return "CUDA call failed";
        case PD_ERR_WORKSPACE: return "workspace too small";
        case PD_ERR_DEVICE_FAULT: return "kernel met an out-of-range page id or length";
        case PD_ERR_TIMEOUT: return "kernel gave up a bounded wait";
        default: return "unknown status";
    }
}

const char *pd_last_error(const pd_ctx *ctx) { return ctx != nullptr ? ctx->last_error : "null context"; }

int pd_create(const pd_config *cfg, pd_ctx **out) {
    if (out == nullptr) return PD_ERR_INVALID_ARG;
    *out = nullptr;
    if (cfg == nullptr) return PD_ERR_INVALID_ARG;
    if (cfg->num_q_heads <= 0 || cfg->num_kv_heads <= 0 || cfg->num_q_heads % cfg->num_kv_heads != 0 ||
        cfg->max_batch < 1 || cfg->max_batch > pd::kMaxBatch || cfg->max_pages_per_seq < 1 || cfg->num_pages < 1 ||
        cfg->device < 0)
        return PD_ERR_INVALID_ARG;
    const int group = cfg->num_q_heads / cfg->num_kv_heads;
    if (cfg->page_size != pd::kPageSize || (cfg->head_dim != 64 && cfg->head_dim != 128) ||
        (group != 1 && group != 2 && group != 4 && group != 8))
        return PD_ERR_UNSUPPORTED;
    // TMA row coordinates and page ids are 32-bit
    if (cfg->num_pages * cfg->num_kv_heads * cfg->page_size >= (int64_t(1) << 31)) return PD_ERR_UNSUPPORTED;
    if (static_cast<int64_t>(cfg->max_pages_per_seq) * cfg->page_size >= (int64_t(1) << 31)) return PD_ERR_UNSUPPORTED;

    DeviceGuard guard(cfg->device);
    if (!guard.ok) return PD_ERR_CUDA;
    cudaDeviceProp prop{};
    if (cudaGetDeviceProperties(&prop, cfg->device) != cudaSuccess) return PD_ERR_CUDA;
    if (prop.major != 10) return PD_ERR_UNSUPPORTED;  // built for sm_100a only

    pd_ctx *ctx = new (std::nothrow) pd_ctx();
    if (ctx == nullptr) return PD_ERR_CUDA;
    ctx->cfg = *cfg;
    ctx->group = group;
    ctx->num_sms = prop.multiProcessorCount;

    // kernel shape: one CTA per SM, each warp an independent worker with its own stage ring
    pd::AttnVariant v{};
    v.head_dim = cfg->head_dim;
    v.warps = tune_int("PD_TUNE_WARPS", cfg->head_dim == 128 ? 8 : 16);
    v.stages = tune_int("PD_TUNE_STAGES", 3);
    v.hilo = tune_int("PD_TUNE_HILO", 1);
    ctx->variant = v;
    ctx->num_ctas = ctx->num_sms * tune_int("PD_TUNE_CTAS_PER_SM", 1);
    ctx->min_pages_auto = tune_int("PD_TUNE_MIN_PAGES", 4);
    ctx->halving_levels = tune_int("PD_TUNE_LEVELS", 6);
    ctx->tail_pages = tune_int("PD_TUNE_TAIL", 16);
    ctx->pdl = tune_int("PD_TUNE_PDL", 1);
    ctx->merge_rows = tune_int("PD_TUNE_MERGE_ROWS", 0);
    ctx->prefill_reverse = tune_int("PD_TUNE_PREFILL_REVERSE", 1);
    ctx->prefill_order = tune_int("PD_TUNE_PREFILL_ORDER", 1);
    if (ctx->halving_levels < 0 || ctx->halving_levels > pd::kMaxLevels - 2 || ctx->tail_pages < 1) {
        delete ctx;
        return PD_ERR_INVALID_ARG;
    }
    cudaError_t err = pd::prepare_decode_attn(v, &ctx->smem_bytes);
    if (err != cudaSuccess) {
        delete ctx;
        return err == cudaErrorInvalidValue ? PD_ERR_UNSUPPORTED : PD_ERR_CUDA;
    }

    void *fn = nullptr;
    cudaDriverEntryPointQueryResult q{};
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || fn == nullptr ||
        q != cudaDriverEntryPointSuccess) {
        delete ctx;
        return PD_ERR_CUDA;
    }
    ctx->encode = reinterpret_cast<EncodeTiledFn>(fn);

    // workspace: partial slots = ranges + one per (sequence, KV head)
    const int n_workers = ctx->num_ctas * v.warps;
    ctx->max_ranges = 16 * n_workers;
    ctx->slots = static_cast<size_t>(ctx->max_ranges) + static_cast<size_t>(cfg->max_batch) * cfg->num_kv_heads;
    auto round256 = [](size_t n) { return (n + 255) & ~size_t(255); };
    const size_t b_part_o = round256(ctx->slots * group * cfg->head_dim * sizeof(float));
    const size_t b_part_ml = round256(ctx->slots * group * sizeof(float2));
    const size_t b_cum = round256((static_cast<size_t>(cfg->max_batch) + 1) * sizeof(int32_t));
    const size_t b_plan = round256(pd::kPlanWords * sizeof(int32_t));
    const size_t b_status = round256(pd::kStatusWords * sizeof(int32_t));
    const size_t b_q = round256(static_cast<size_t>(cfg->max_batch) * cfg->num_q_heads * cfg->head_dim * 2);
    const size_t b_kv = round256(static_cast<size_t>(cfg->max_batch) * cfg->num_kv_heads * cfg->head_dim * 2);
    const size_t b_trace = tune_int("PD_TRACE_WORKERS", 0) ? round256(static_cast<size_t>(n_workers) * 4 * 8) : 0;
    ctx->workspace_bytes = b_part_o + b_part_ml + b_cum + b_plan + b_status + 2 * b_q + 2 * b_kv + b_trace;
    err = cudaMalloc(&ctx->workspace, ctx->workspace_bytes);
    if (err != cudaSuccess) {
        delete ctx;
        return PD_ERR_CUDA;
    }
    char *w = static_cast<char *>(ctx->workspace);
    ctx->part_o = reinterpret_cast<float *>(w); w += b_part_o;
    ctx->part_ml = reinterpret_cast<float2 *>(w); w += b_part_ml;
    ctx->cum_pages = reinterpret_cast<int32_t *>(w); w += b_cum;
    ctx->plan = reinterpret_cast<int32_t *>(w); w += b_plan;
    ctx->status = reinterpret_cast<int32_t *>(w); w += b_status;
    ctx->stage_q = reinterpret_cast<__nv_bfloat16 *>(w); w += b_q;  // q, k_new, v_new are adjacent: one copy can fill them
    ctx->stage_k = reinterpret_cast<__nv_bfloat16 *>(w); w += b_kv;
    ctx->stage_v = reinterpret_cast<__nv_bfloat16 *>(w); w += b_kv;
    ctx->stage_out = reinterpret_cast<__nv_bfloat16 *>(w); w += b_q;
    if (b_trace != 0) {
        ctx->trace = reinterpret_cast<unsigned long long *>(w);
        ctx->trace_workers = n_workers;
    }
    err = cudaMemset(ctx->workspace, 0, ctx->workspace_bytes);
    if (err != cudaSuccess) {
        cudaFree(ctx->workspace);
        delete ctx;
        return PD_ERR_CUDA;
    }
    // optional: without the pinned word pd_decode_step_host keeps to copies and a stream synchronisation
    void *flag = nullptr, *flag_dev = nullptr;
    if (cudaHostAlloc(&flag, 64, cudaHostAllocMapped) == cudaSuccess) {
        if (cudaHostGetDevicePointer(&flag_dev, flag, 0) == cudaSuccess) {
            ctx->done_flag_host = static_cast<int32_t *>(flag);
            ctx->done_flag_dev = static_cast<int32_t *>(flag_dev);
            *ctx->done_flag_host = 0;
        } else {
            cudaFreeHost(flag);
        }
    }
    (void)cudaGetLastError();
    *out = ctx;
    return PD_OK;
}

int pd_destroy(pd_ctx *ctx) {
    if (ctx == nullptr) return PD_OK;
    DeviceGuard guard(ctx->cfg.device);
    cudaDeviceSynchronize();
    cudaFree(ctx->workspace);
    if (ctx->done_flag_host != nullptr) cudaFreeHost(ctx->done_flag_host);
    delete ctx;
    return PD_OK;
}

int pd_kv_append(pd_ctx *ctx, const void *k_new, const void *v_new, void *k_pages, void *v_pages,
                 const int32_t *page_table, int32_t *ctx_lens, int32_t batch, uint32_t call_flags, void *stream) {
    if (int rc = check_batch(ctx, batch)) return rc;
    if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_pages) || !aligned16(v_pages) || page_table == nullptr ||
        ctx_lens == nullptr)
        return fail(ctx, PD_ERR_INVALID_ARG, "pd_kv_append: null or misaligned pointer");
    if (call_flags & ~PD_APPEND_NO_ADVANCE) return fail(ctx, PD_ERR_INVALID_ARG, "pd_kv_append: unknown call flag");
    if (batch == 0) return PD_OK;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return fail(ctx, PD_ERR_CUDA, "cudaSetDevice");
    pd::AppendParams p{};
    p.k_new = static_cast<const __nv_bfloat16 *>(k_new);
    p.v_new = static_cast<const __nv_bfloat16 *>(v_new);
    p.k_pages = static_cast<__nv_bfloat16 *>(k_pages);
    p.v_pages = static_cast<__nv_bfloat16 *>(v_pages);
    p.page_table = page_table;
    p.ctx_lens = ctx_lens;
    p.status = ctx->status;
    p.B = batch;
    p.Hkv = ctx->cfg.num_kv_heads;
    p.D = ctx->cfg.head_dim;
    p.MP = ctx->cfg.max_pages_per_seq;
    p.num_pages = static_cast<int32_t>(ctx->cfg.num_pages);
    p.advance = (call_flags & PD_APPEND_NO_ADVANCE) ? 0 : 1;
    p.pdl = ctx->pdl;
    const cudaError_t err = pd::launch_kv_append(p, static_cast<cudaStream_t>(stream));
    if (err != cudaSuccess) return fail(ctx, PD_ERR_CUDA, "kv_append launch", err);
    ctx->launches += 1;
    return PD_OK;
}

namespace {

int kv_transfer(pd_ctx *ctx, bool scatter, void *k_pages, void *v_pages, float *kv_scales, const int32_t *page_table,
                const int32_t *page_begin, const int32_t *page_end, const int64_t *packed_page_offset, void *packed,
                int32_t batch, void *stream) {
    if (int rc = check_batch(ctx, batch)) return rc;
    if (!aligned16(k_pages) || !aligned16(v_pages) || !aligned16(packed) || page_table == nullptr ||
        page_begin == nullptr || page_end == nullptr || packed_page_offset == nullptr ||
        (kv_scales != nullptr && !aligned16(kv_scales)))
        return fail(ctx, PD_ERR_INVALID_ARG, "KV transfer: null or misaligned pointer");
    if (batch == 0) return PD_OK;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return fail(ctx, PD_ERR_CUDA, "cudaSetDevice");
    pd::TransferParams p{};
    p.k_pages = static_cast<__nv_bfloat16 *>(k_pages);
    p.v_pages = static_cast<__nv_bfloat16 *>(v_pages);
    p.packed = packed;
    p.page_table = page_table;
    p.page_begin = page_begin;
    p.page_end = page_end;
    p.packed_page_offset = reinterpret_cast<const long long *>(packed_page_offset);
    p.status = ctx->status;
    p.B = batch;
    p.Hkv = ctx->cfg.num_kv_heads;
    p.D = ctx->cfg.head_dim;
    p.MP = ctx->cfg.max_pages_per_seq;
    p.num_pages = static_cast<int32_t>(ctx->cfg.num_pages);
    p.pdl = ctx->pdl;
    p.elem_bytes = kv_scales != nullptr ? 1 : 2;
    p.scales = kv_scales;
    const cudaError_t err = pd::launch_kv_transfer(p, scatter, ctx->num_sms, static_cast<cudaStream_t>(stream));
    if (err != cudaSuccess) return fail(ctx, PD_ERR_CUDA, scatter ? "kv_scatter launch" : "kv_gather launch", err);
    ctx->launches += 1;
    return PD_OK;
}

}  // namespace

int pd_kv_gather(pd_ctx *ctx, const void *k_pages, const void *v_pages, const int32_t *page_table,
                 const int32_t *page_begin, const int32_t *page_end, const int64_t *packed_page_offset, void *packed,
                 int32_t batch, void *stream) {
    return kv_transfer(ctx, false, const_cast<void *>(k_pages), const_cast<void *>(v_pages), nullptr, page_table, page_begin,
                       page_end, packed_page_offset, packed, batch, stream);
}

int pd_kv_gather_fp8(pd_ctx *ctx, const void *k8, const void *v8, const float *kv_scales, const int32_t *page_table,
                     const int32_t *page_begin, const int32_t *page_end, const int64_t *packed_page_offset, void *packed,
                     int32_t batch, void *stream) {
    if (ctx != nullptr && kv_scales == nullptr) return fail(ctx, PD_ERR_INVALID_ARG, "pd_kv_gather_fp8: null kv_scales");
    return kv_transfer(ctx, false, const_cast<void *>(k8), const_cast<void *>(v8), const_cast<float *>(kv_scales), page_table,
                       page_begin, page_end, packed_page_offset, packed, batch, stream);
}

int pd_kv_scatter_fp8(pd_ctx *ctx, const void *packed, const int64_t *packed_page_offset, void *k8, void *v8,
                      float *kv_scales, const int32_t *page_table, const int32_t *page_begin, const int32_t *page_end,
                      int32_t batch, void *stream) {
    if (ctx != nullptr && kv_scales == nullptr) return fail(ctx, PD_ERR_INVALID_ARG, "pd_kv_scatter_fp8: null kv_scales");
    return kv_transfer(ctx, true, k8, v8, kv_scales, page_table, page_begin, page_end, packed_page_offset,
                       const_cast<void *>(packed), batch, stream);
}

int pd_kv_scatter(pd_ctx *ctx, const void *packed, const int64_t *packed_page_offset, void *k_pages, void *v_pages,
                  const int32_t *page_table, const int32_t *page_begin, const int32_t *page_end, int32_t batch,
                  void *stream) {
    return kv_transfer(ctx, true, k_pages, v_pages, nullptr, page_table, page_begin, page_end, packed_page_offset,
                       const_cast<void *>(packed), batch, stream);
}

}  // extern "C"

namespace {

// Split kernel + merge kernel. With k_new / v_new the split kernel also appends one token per sequence
// (the pools and the lengths are then written) and attends over the grown contexts.
int decode_attn_impl(pd_ctx *ctx, const char *who, const void *q, const void *k_new, const void *v_new, const void *k_pages,
                     const void *v_pages, const int32_t *page_table, const int32_t *ctx_lens, void *out, float *lse,
                     int32_t batch, float sm_scale, int32_t split_pages, void *stream) {
    const bool fused = k_new != nullptr;
    if (int rc = check_batch(ctx, batch)) return rc;
    if (!aligned16(q) || !aligned16(k_pages) || !aligned16(v_pages) || !aligned16(out) || page_table == nullptr ||
        ctx_lens == nullptr || (fused && (!aligned16(k_new) || !aligned16(v_new)))) {
        char msg[96];
        std::snprintf(msg, sizeof msg, "%s: null or misaligned pointer", who);
        return fail(ctx, PD_ERR_INVALID_ARG, msg);
    }
    if (!(sm_scale > 0.f) || !(sm_scale < 3.0e38f)) return fail(ctx, PD_ERR_INVALID_ARG, "sm_scale must be finite and positive");
    if (split_pages < 0) return fail(ctx, PD_ERR_INVALID_ARG, "split_pages must be >= 0");
    if (batch == 0) return PD_OK;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return fail(ctx, PD_ERR_CUDA, "cudaSetDevice");
    if (ctx->map_k_ptr != k_pages) {
        if (int rc = encode_pool_map(ctx, k_pages, &ctx->tm_k)) return rc;
        ctx->map_k_ptr = k_pages;
    }
    if (ctx->map_v_ptr != v_pages) {
        if (int rc = encode_pool_map(ctx, v_pages, &ctx->tm_v)) return rc;
        ctx->map_v_ptr = v_pages;
    }
    pd::AttnParams p{};
    p.q = static_cast<const __nv_bfloat16 *>(q);
    p.page_table = page_table;
    p.ctx_lens = ctx_lens;
    p.out = static_cast<__nv_bfloat16 *>(out);
    p.lse = lse;
    p.part_o = ctx->part_o;
    p.part_ml = ctx->part_ml;
    p.cum_pages = ctx->cum_pages;
    p.plan = ctx->plan;
    p.status = ctx->status;
    p.B = batch;
    p.Hq = ctx->cfg.num_q_heads;
    p.Hkv = ctx->cfg.num_kv_heads;
    p.G = ctx->group;
    p.MP = ctx->cfg.max_pages_per_seq;
    p.num_pages = static_cast<int32_t>(ctx->cfg.num_pages);
    p.scale_log2 = sm_scale * 1.4426950408889634f;
    p.split_pages = split_pages;
    p.max_ranges = ctx->max_ranges;
    p.min_pages_auto = ctx->min_pages_auto;
    p.halving_levels = ctx->halving_levels;
    p.tail_pages = ctx->tail_pages;
    const bool hooked = ctx->ev_before != nullptr;
    p.pdl = hooked ? 0 : ctx->pdl;  // timing events must bracket the split kernel alone: no overlap with neighbours
    p.merge_rows = ctx->merge_rows;
    p.trace = ctx->trace;
    if (ctx->host_out_alias != nullptr) {
        p.out_host = ctx->host_out_alias;
        p.done_flag = ctx->done_flag_dev;
        p.done_value = ctx->done_seq;
    }
    if (fused) {
        p.k_new = static_cast<const __nv_bfloat16 *>(k_new);
        p.v_new = static_cast<const __nv_bfloat16 *>(v_new);
        p.k_pool_w = static_cast<__nv_bfloat16 *>(const_cast<void *>(k_pages));
        p.v_pool_w = static_cast<__nv_bfloat16 *>(const_cast<void *>(v_pages));
        p.ctx_lens_w = const_cast<int32_t *>(ctx_lens);
        p.fused = 1;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (hooked) cudaEventRecord(ctx->ev_before, s);
    cudaError_t err = pd::launch_decode_attn(ctx->variant, ctx->tm_k, ctx->tm_v, p, ctx->num_ctas, ctx->smem_bytes, s);
    if (err != cudaSuccess) return fail(ctx, PD_ERR_CUDA, "decode_attn_split launch", err);
    if (hooked) {
        cudaEventRecord(ctx->ev_after, s);
        ctx->ev_before = nullptr;  // one-shot
        ctx->ev_after = nullptr;
    }
    err = pd::launch_lse_merge(ctx->cfg.head_dim, p, s);
    if (err != cudaSuccess) return fail(ctx, PD_ERR_CUDA, "lse_merge launch", err);
    ctx->launches += 2;
    return PD_OK;
}

}  // namespace

extern "C" {

int pd_decode_attn(pd_ctx *ctx, const void *q, const void *k_pages, const void *v_pages, const int32_t *page_table,
                   const int32_t *ctx_lens, void *out, float *lse, int32_t batch, float sm_scale, int32_t split_pages,
                   void *stream) {
    return decode_attn_impl(ctx, "pd_decode_attn", q, nullptr, nullptr, k_pages, v_pages, page_table, ctx_lens, out, lse,
                            batch, sm_scale, split_pages, stream);
}

int pd_decode_step(pd_ctx *ctx, const void *q, const void *k_new, const void *v_new, void *k_pages, void *v_pages,
                   const int32_t *page_table, int32_t *ctx_lens, void *out, float *lse, int32_t batch, float sm_scale,
                   int32_t split_pages, void *stream) {
    if (ctx == nullptr) return PD_ERR_INVALID_ARG;
    if (k_new == nullptr || v_new == nullptr) return fail(ctx, PD_ERR_INVALID_ARG, "pd_decode_step: null k_new / v_new");
    return decode_attn_impl(ctx, "pd_decode_step", q, k_new, v_new, k_pages, v_pages, page_table, ctx_lens, out, lse, batch,
                            sm_scale, split_pages, stream);
}

int pd_kv_quantize_pages(pd_ctx *ctx, const void *k_pages, const void *v_pages, const int32_t *tokens_in_page, void *k8,
                         void *v8, float *kv_scales, void *stream) {
    if (ctx == nullptr) return PD_ERR_INVALID_ARG;
    if (!aligned16(k_pages) || !aligned16(v_pages) || !aligned16(k8) || !aligned16(v8) || !aligned16(kv_scales) ||
        tokens_in_page == nullptr)
        return fail(ctx, PD_ERR_INVALID_ARG, "pd_kv_quantize_pages: null or misaligned pointer");
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return fail(ctx, PD_ERR_CUDA, "cudaSetDevice");
    pd::QuantizeParams p{};
    p.k_pages = static_cast<const __nv_bfloat16 *>(k_pages);
    p.v_pages = static_cast<const __nv_bfloat16 *>(v_pages);
    p.tokens_in_page = tokens_in_page;
    p.k8 = static_cast<uint8_t *>(k8);
    p.v8 = static_cast<uint8_t *>(v8);
    p.scales = kv_scales;
    p.num_pages = ctx->cfg.num_pages;
    p.Hkv = ctx->cfg.num_kv_heads;
    p.D = ctx->cfg.head_dim;
    p.pdl = ctx->pdl;
    const cudaError_t err = pd::launch_kv_quantize_pages(p, static_cast<cudaStream_t>(stream));
    if (err != cudaSuccess) return fail(ctx, PD_ERR_CUDA, "kv_quantize_pages launch", err);
    ctx->launches += 1;
    return PD_OK;
}

int pd_kv_append_fp8(pd_ctx *ctx, const void *k_new, const void *v_new, void *k8, void *v8, float *kv_scales,
                     const int32_t *page_table, int32_t *ctx_lens, int32_t batch, uint32_t call_flags, void *stream) {
    if (int rc = check_batch(ctx, batch)) return rc;
    if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k8) || !aligned16(v8) || !aligned16(kv_scales) ||
        page_table == nullptr || ctx_lens == nullptr)
        return fail(ctx, PD_ERR_INVALID_ARG, "pd_kv_append_fp8: null or misaligned pointer");
    if (batch == 0) return PD_OK;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return fail(ctx, PD_ERR_CUDA, "cudaSetDevice");
    pd::AppendFp8Params p{};
    p.k_new = static_cast<const __nv_bfloat16 *>(k_new);
    p.v_new = static_cast<const __nv_bfloat16 *>(v_new);
    p.k8 = static_cast<uint8_t *>(k8);
    p.v8 = static_cast<uint8_t *>(v8);
    p.scales = kv_scales;
    p.page_table = page_table;
    p.ctx_lens = ctx_lens;
    p.status = ctx->status;
    p.B = batch;
    p.Hkv = ctx->cfg.num_kv_heads;
    p.D = ctx->cfg.head_dim;
    p.MP = ctx->cfg.max_pages_per_seq;
    p.num_pages = static_cast<int32_t>(ctx->cfg.num_pages);
    p.advance = (call_flags & PD_APPEND_NO_ADVANCE) ? 0 : 1;
    p.pdl = ctx->pdl;
    const cudaError_t err = pd::launch_kv_append_fp8(p, static_cast<cudaStream_t>(stream));
    if (err != cudaSuccess) return fail(ctx, PD_ERR_CUDA, "kv_append_fp8 launch", err);
    ctx->launches += 1;
    return PD_OK;
}

}  // extern "C"

namespace {

constexpr int32_t kFp8StaticFairMax = 1024;  // pages per worker up to which the FP8 split kernel takes one equal range per worker

int fp8_attn_check_args(pd_ctx *ctx, const void *q, const void *k8, const void *v8, const float *kv_scales,
                        const int32_t *page_table, const int32_t *ctx_lens, const void *out, int32_t batch, float sm_scale,
                        int32_t split_pages) {
    if (int rc = check_batch(ctx, batch)) return rc;
    if (!aligned16(q) || !aligned16(k8) || !aligned16(v8) || !aligned16(kv_scales) || !aligned16(out) ||
        page_table == nullptr || ctx_lens == nullptr)
        return fail(ctx, PD_ERR_INVALID_ARG, "FP8 attention: null or misaligned pointer");
    if (!(sm_scale > 0.f) || !(sm_scale < 3.0e38f)) return fail(ctx, PD_ERR_INVALID_ARG, "sm_scale must be finite and positive");
    if (split_pages < 0) return fail(ctx, PD_ERR_INVALID_ARG, "split_pages must be >= 0");
    return PD_OK;
}

int decode_attn_fp8_impl(pd_ctx *ctx, const void *q, const void *k8, const void *v8, const float *kv_scales,
                         const int32_t *page_table, const int32_t *ctx_lens, void *out, float *lse, int32_t batch,
                         float sm_scale, int32_t split_pages, void *stream) {
    if (int rc = fp8_attn_check_args(ctx, q, k8, v8, kv_scales, page_table, ctx_lens, out, batch, sm_scale, split_pages)) return rc;
    if (batch == 0) return PD_OK;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return fail(ctx, PD_ERR_CUDA, "cudaSetDevice");
    if (!ctx->fp8_ready) {
        const cudaError_t e = pd::prepare_decode_attn_fp8(ctx->cfg.head_dim);
        if (e != cudaSuccess) return fail(ctx, PD_ERR_CUDA, "fp8 decode kernel attribute", e);
        ctx->fp8_ready = true;
    }
    if (ctx->map_k8_ptr != k8) {
        if (int rc = encode_pool_map_fp8(ctx, k8, &ctx->tm_k8)) return rc;
        ctx->map_k8_ptr = k8;
    }
    if (ctx->map_v8_ptr != v8) {
        if (int rc = encode_pool_map_fp8(ctx, v8, &ctx->tm_v8)) return rc;
        ctx->map_v8_ptr = v8;
    }
    pd::AttnParams p{};
    p.q = static_cast<const __nv_bfloat16 *>(q);
    p.kv_scales = kv_scales;
    p.page_table = page_table;
    p.ctx_lens = ctx_lens;
    p.out = static_cast<__nv_bfloat16 *>(out);
    p.lse = lse;
    p.part_o = ctx->part_o;
    p.part_ml = ctx->part_ml;
    p.cum_pages = ctx->cum_pages;
    p.plan = ctx->plan;
    p.status = ctx->status;
    p.B = batch;
    p.Hq = ctx->cfg.num_q_heads;
    p.Hkv = ctx->cfg.num_kv_heads;
    p.G = ctx->group;
    p.MP = ctx->cfg.max_pages_per_seq;
    p.num_pages = static_cast<int32_t>(ctx->cfg.num_pages);
    p.scale_log2 = sm_scale * 1.4426950408889634f;
    p.split_pages = split_pages;
    p.max_ranges = ctx->max_ranges;
    p.min_pages_auto = ctx->min_pages_auto;
    p.halving_levels = ctx->halving_levels;
    p.tail_pages = ctx->tail_pages;
    // Measured on configs[1..4] (call of split + merge, us): equal ranges 129 / 181 / 416 / 2168 against 138 / 196 /
    // 443 / 2139 for the halving plan, the opposite of the bf16 kernel (263 / 390 / 858 / 4075 against 236 / 345 /
    // 766 / 3623), whose workers differ in speed with their SM's distance to the memory they read.
    p.static_fair_max = kFp8StaticFairMax;
    const bool hooked = ctx->ev_before != nullptr;
    p.pdl = hooked ? 0 : ctx->pdl;
    p.merge_rows = ctx->merge_rows;
    p.trace = ctx->trace;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (hooked) cudaEventRecord(ctx->ev_before, s);
    cudaError_t err = pd::launch_decode_attn_fp8(ctx->cfg.head_dim, ctx->tm_k8, ctx->tm_v8, p, ctx->num_ctas, s);
    if (err != cudaSuccess) return fail(ctx, PD_ERR_CUDA, "decode_attn_split_fp8 launch", err);
    if (hooked) {
        cudaEventRecord(ctx->ev_after, s);
        ctx->ev_before = nullptr;
        ctx->ev_after = nullptr;
    }
    err = pd::launch_lse_merge(ctx->cfg.head_dim, p, s);
    if (err != cudaSuccess) return fail(ctx, PD_ERR_CUDA, "lse_merge launch", err);
    ctx->launches += 2;
    return PD_OK;
}

}  // namespace

extern "C" {

int pd_decode_attn_fp8(pd_ctx *ctx, const void *q, const void *k8, const void *v8, const float *kv_scales,
                       const int32_t *page_table, const int32_t *ctx_lens, void *out, float *lse, int32_t batch,
                       float sm_scale, int32_t split_pages, void *stream) {
    return decode_attn_fp8_impl(ctx, q, k8, v8, kv_scales, page_table, ctx_lens, out, lse, batch, sm_scale, split_pages, stream);
}

int pd_decode_step_fp8(pd_ctx *ctx, const void *q, const void *k_new, const void *v_new, void *k8, void *v8,
                       float *kv_scales, const int32_t *page_table, int32_t *ctx_lens, void *out, float *lse,
                       int32_t batch, float sm_scale, int32_t split_pages, void *stream) {
    if (ctx == nullptr) return PD_ERR_INVALID_ARG;
    if (k_new == nullptr || v_new == nullptr) return fail(ctx, PD_ERR_INVALID_ARG, "pd_decode_step_fp8: null k_new / v_new");
    // Two launches (three with the merge). A split kernel that also quantised and patched the new token measured
    // slower than this on every configuration (137 against 127 us on configs[3]), so there is none.
    if (int rc = fp8_attn_check_args(ctx, q, k8, v8, kv_scales, page_table, ctx_lens, out, batch, sm_scale, split_pages)) return rc;
    if (int rc = pd_kv_append_fp8(ctx, k_new, v_new, k8, v8, kv_scales, page_table, ctx_lens, batch, 0u, stream)) return rc;
    return decode_attn_fp8_impl(ctx, q, k8, v8, kv_scales, page_table, ctx_lens, out, lse, batch, sm_scale, split_pages, stream);
}

int pd_kv_append_tokens(pd_ctx *ctx, const void *k_new, const void *v_new, const int32_t *q_indptr, void *k_pages,
                        void *v_pages, const int32_t *page_table, int32_t *ctx_lens, int32_t batch, int32_t max_q_len,
                        void *stream) {
    if (int rc = check_batch(ctx, batch)) return rc;
    if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(k_pages) || !aligned16(v_pages) || q_indptr == nullptr ||
        page_table == nullptr || ctx_lens == nullptr)
        return fail(ctx, PD_ERR_INVALID_ARG, "pd_kv_append_tokens: null or misaligned pointer");
    if (max_q_len < 0) return fail(ctx, PD_ERR_INVALID_ARG, "max_q_len must be >= 0");
    if (batch == 0 || max_q_len == 0) return PD_OK;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return fail(ctx, PD_ERR_CUDA, "cudaSetDevice");
    pd::AppendTokensParams p{};
    p.k_new = static_cast<const __nv_bfloat16 *>(k_new);
    p.v_new = static_cast<const __nv_bfloat16 *>(v_new);
    p.q_indptr = q_indptr;
    p.k_pages = static_cast<__nv_bfloat16 *>(k_pages);
    p.v_pages = static_cast<__nv_bfloat16 *>(v_pages);
    p.page_table = page_table;
    p.ctx_lens = ctx_lens;
    p.status = ctx->status;
    p.B = batch;
    p.Hkv = ctx->cfg.num_kv_heads;
    p.D = ctx->cfg.head_dim;
    p.MP = ctx->cfg.max_pages_per_seq;
    p.num_pages = static_cast<int32_t>(ctx->cfg.num_pages);
    p.pdl = ctx->pdl;
    const cudaError_t err = pd::launch_kv_append_tokens(p, max_q_len, static_cast<cudaStream_t>(stream));
    if (err != cudaSuccess) return fail(ctx, PD_ERR_CUDA, "kv_append_tokens launch", err);
    ctx->launches += 2;
    return PD_OK;
}

int pd_prefill_attn(pd_ctx *ctx, const void *q, const int32_t *q_indptr, const void *k_pages, const void *v_pages,
                    const int32_t *page_table, const int32_t *ctx_lens, void *out, float *lse, int32_t batch,
                    int32_t max_q_len, float sm_scale, void *stream) {
    if (int rc = check_batch(ctx, batch)) return rc;
    if (!aligned16(q) || !aligned16(k_pages) || !aligned16(v_pages) || !aligned16(out) || q_indptr == nullptr ||
        page_table == nullptr || ctx_lens == nullptr)
        return fail(ctx, PD_ERR_INVALID_ARG, "pd_prefill_attn: null or misaligned pointer");
    if (!(sm_scale > 0.f) || !(sm_scale < 3.0e38f)) return fail(ctx, PD_ERR_INVALID_ARG, "sm_scale must be finite and positive");
    if (max_q_len < 0) return fail(ctx, PD_ERR_INVALID_ARG, "max_q_len must be >= 0");
    if (batch == 0 || max_q_len == 0) return PD_OK;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return fail(ctx, PD_ERR_CUDA, "cudaSetDevice");
    if (!ctx->prefill_ready) {
        const cudaError_t e = pd::prepare_prefill_attn(ctx->cfg.head_dim);
        if (e != cudaSuccess) return fail(ctx, PD_ERR_CUDA, "prefill kernel attribute", e);
        ctx->prefill_ready = true;
    }
    if (ctx->map_k_ptr != k_pages) {
        if (int rc = encode_pool_map(ctx, k_pages, &ctx->tm_k)) return rc;
        ctx->map_k_ptr = k_pages;
    }
    if (ctx->map_v_ptr != v_pages) {
        if (int rc = encode_pool_map(ctx, v_pages, &ctx->tm_v)) return rc;
        ctx->map_v_ptr = v_pages;
    }
    pd::PrefillParams p{};
    p.q = static_cast<const __nv_bfloat16 *>(q);
    p.q_indptr = q_indptr;
    p.page_table = page_table;
    p.ctx_lens = ctx_lens;
    p.out = static_cast<__nv_bfloat16 *>(out);
    p.lse = lse;
    p.status = ctx->status;
    p.B = batch;
    p.Hq = ctx->cfg.num_q_heads;
    p.Hkv = ctx->cfg.num_kv_heads;
    p.G = ctx->group;
    p.MP = ctx->cfg.max_pages_per_seq;
    p.num_pages = static_cast<int32_t>(ctx->cfg.num_pages);
    p.scale_log2 = sm_scale * 1.4426950408889634f;
    p.pdl = ctx->pdl;
    p.trace = ctx->trace;                    // the worker-trace buffer doubles as [CTA][16] phase counters
    p.trace_ctas = ctx->trace_workers / 4;
    p.reverse_tiles = ctx->prefill_reverse;
    p.order = ctx->prefill_order ? ctx->cum_pages : nullptr;  // the decode kernels' prefix-sum buffer is free here
    if (ctx->trace != nullptr) cudaMemsetAsync(ctx->trace, 0, static_cast<size_t>(ctx->trace_workers) * 32, static_cast<cudaStream_t>(stream));
    const cudaError_t err = pd::launch_prefill_attn(ctx->cfg.head_dim, ctx->tm_k, ctx->tm_v, p, max_q_len,
                                                    static_cast<cudaStream_t>(stream));
    if (err != cudaSuccess) return fail(ctx, PD_ERR_CUDA, "prefill_attn launch", err);
    ctx->launches += p.order != nullptr ? 2 : 1;
    return PD_OK;
}

int pd_decode_step_host(pd_ctx *ctx, const void *q_host, const void *k_new_host, const void *v_new_host, void *k_pages,
                        void *v_pages, const int32_t *page_table, int32_t *ctx_lens, void *out_host, int32_t batch,
                        float sm_scale, int32_t split_pages, void *stream) {
    if (int rc = check_batch(ctx, batch)) return rc;
    if (q_host == nullptr || k_new_host == nullptr || v_new_host == nullptr || out_host == nullptr)
        return fail(ctx, PD_ERR_INVALID_ARG, "pd_decode_step_host: null host pointer");
    if (batch == 0) return PD_OK;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return fail(ctx, PD_ERR_CUDA, "cudaSetDevice");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t nq = static_cast<size_t>(batch) * ctx->cfg.num_q_heads * ctx->cfg.head_dim * 2;
    const size_t nkv = static_cast<size_t>(batch) * ctx->cfg.num_kv_heads * ctx->cfg.head_dim * 2;
    // Host buffers that follow one another in memory (q, then k_new, then v_new) travel in one copy. Adjacent
    // addresses can still belong to separately pinned allocations, which a single copy may not span: if the
    // runtime refuses it, nothing was enqueued and the three buffers are copied one by one.
    const char *qh = static_cast<const char *>(q_host);
    bool adjacent = static_cast<const char *>(k_new_host) == qh + nq && static_cast<const char *>(v_new_host) == qh + nq + nkv;
    __nv_bfloat16 *dq = ctx->stage_q, *dk = ctx->stage_k, *dv = ctx->stage_v;
    cudaError_t err = cudaSuccess;
    if (adjacent) {
        err = cudaMemcpyAsync(dq, q_host, nq + 2 * nkv, cudaMemcpyHostToDevice, s);
        if (err == cudaSuccess) {
            dk = reinterpret_cast<__nv_bfloat16 *>(reinterpret_cast<char *>(dq) + nq);
            dv = reinterpret_cast<__nv_bfloat16 *>(reinterpret_cast<char *>(dq) + nq + nkv);
        } else {
            (void)cudaGetLastError();
            adjacent = false;
        }
    }
    if (!adjacent) {
        err = cudaMemcpyAsync(dq, q_host, nq, cudaMemcpyHostToDevice, s);
        if (err == cudaSuccess) err = cudaMemcpyAsync(dk, k_new_host, nkv, cudaMemcpyHostToDevice, s);
        if (err == cudaSuccess) err = cudaMemcpyAsync(dv, v_new_host, nkv, cudaMemcpyHostToDevice, s);
    }
    if (err != cudaSuccess) return fail(ctx, PD_ERR_CUDA, "host-to-device copy", err);
    // Result: if out_host is pinned memory the device can address, the merge kernel stores the rows there itself
    // and raises a pinned flag that this thread polls: no device-to-host copy operation and no stream
    // synchronisation sit behind the kernels. Otherwise the result is staged and copied.
    void *out_alias = nullptr;
    // (Measured on B200: the direct path saves ~15 us of a 270 us step with a 64 KB result and loses ~10 us of a
    // 420 us step with a 512 KB one, where the copy engine moves the rows faster than the merge kernel's stores
    // cross PCIe; hence the size limit.)
    constexpr size_t kDirectResultLimit = 256 * 1024;
    const bool direct = ctx->done_flag_host != nullptr && nq <= kDirectResultLimit &&
                        (reinterpret_cast<uintptr_t>(out_host) & 15u) == 0 &&
                        cudaHostGetDevicePointer(&out_alias, out_host, 0) == cudaSuccess && out_alias != nullptr;
    if (!direct) (void)cudaGetLastError();
    if (direct) {
        ctx->done_seq = ctx->done_seq == 0x7fffffff ? 1 : ctx->done_seq + 1;
        ctx->host_out_alias = static_cast<__nv_bfloat16 *>(out_alias);
    }
    const int rc = pd_decode_step(ctx, dq, dk, dv, k_pages, v_pages, page_table, ctx_lens, ctx->stage_out, nullptr, batch,
                                  sm_scale, split_pages, stream);
    ctx->host_out_alias = nullptr;
    if (rc != PD_OK) return rc;
    if (direct) {
        const volatile int32_t *flag = ctx->done_flag_host;
        const auto t0 = std::chrono::steady_clock::now();
        for (unsigned spins = 0; *flag != ctx->done_seq; ++spins) {
            if ((spins & 0xfff) == 0xfff) {
                if (cudaStreamQuery(s) == cudaSuccess && *flag != ctx->done_seq)  // the stream drained without the flag: a kernel gave up
                    return fail(ctx, PD_ERR_TIMEOUT, "pd_decode_step_host: the kernels finished without reporting the result");
                if (std::chrono::steady_clock::now() - t0 > std::chrono::seconds(10)) {
                    cudaStreamSynchronize(s);
                    return fail(ctx, PD_ERR_TIMEOUT, "pd_decode_step_host: no completion report within 10 s");
                }
            }
        }
        ctx->host_steps_direct += 1;
        return PD_OK;
    }
    err = cudaMemcpyAsync(out_host, ctx->stage_out, nq, cudaMemcpyDeviceToHost, s);
    if (err == cudaSuccess) err = cudaStreamSynchronize(s);
    if (err != cudaSuccess) return fail(ctx, PD_ERR_CUDA, "device-to-host copy", err);
    ctx->host_steps_staged += 1;
    return PD_OK;
}

int pd_host_step_counts(const pd_ctx *ctx, int64_t *direct, int64_t *staged) {
    if (ctx == nullptr) return PD_ERR_INVALID_ARG;
    if (direct != nullptr) *direct = ctx->host_steps_direct;
    if (staged != nullptr) *staged = ctx->host_steps_staged;
    return PD_OK;
}

int pd_device_status(pd_ctx *ctx, void *stream, int32_t *code, int32_t *seq, int32_t *detail) {
    if (ctx == nullptr) return PD_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return fail(ctx, PD_ERR_CUDA, "cudaSetDevice");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // only the fault latch (words 0..3) is read and cleared: the words behind it are the range-claim counters
    // of the split kernel, which a launch in flight on another stream must find untouched
    int32_t host[4] = {0, 0, 0, 0};
    cudaError_t err = cudaMemcpyAsync(host, ctx->status, sizeof host, cudaMemcpyDeviceToHost, s);
    if (err == cudaSuccess) err = cudaMemsetAsync(ctx->status, 0, sizeof host, s);
    if (err == cudaSuccess) err = cudaStreamSynchronize(s);
    if (err != cudaSuccess) return fail(ctx, PD_ERR_CUDA, "status read", err);
    int rc = PD_OK;
    if (host[0] == pd::kDevBadPage || host[0] == pd::kDevBadLength) rc = PD_ERR_DEVICE_FAULT;
    else if (host[0] == pd::kDevTimeout) rc = PD_ERR_TIMEOUT;
    if (code != nullptr) *code = rc;
    if (seq != nullptr) *seq = rc == PD_OK ? -1 : host[1];
    if (detail != nullptr) *detail = rc == PD_OK ? 0 : host[2];
    return rc;
}

int pd_plan_ranges(int64_t total_units, int32_t n_workers, int32_t split_pages, int32_t max_ranges, int32_t min_pages,
                   int32_t halving_levels, int32_t tail_pages, int64_t *starts, int32_t *lens, int32_t capacity,
                   int32_t *n_ranges) {
    if (n_ranges == nullptr || total_units < 0 || n_workers < 1 || split_pages < 0 || max_ranges < 1 || min_pages < 1 ||
        halving_levels < 0 || halving_levels > pd::kMaxLevels - 2 || tail_pages < 1 || capacity < 0 ||
        (capacity > 0 && (starts == nullptr || lens == nullptr)))
        return PD_ERR_INVALID_ARG;
    pd::AttnParams p{};
    p.split_pages = split_pages;
    p.max_ranges = max_ranges;
    p.min_pages_auto = min_pages;
    p.halving_levels = halving_levels;
    p.tail_pages = tail_pages;
    pd::Plan pl;
    pd::make_plan(pl, total_units, n_workers, p);  // the function the kernels run
    *n_ranges = pl.n_ranges;
    if (pl.n_ranges > capacity) return capacity == 0 ? PD_OK : PD_ERR_WORKSPACE;
    for (int r = 0; r < pl.n_ranges; ++r) {
        long long start;
        int len;
        pd::range_bounds(pl, r, start, len);
        starts[r] = start;
        lens[r] = len;
    }
    return PD_OK;
}

int pd_plan_walk(const int32_t *cum_pages, int32_t batch, int32_t num_kv_heads, int64_t first_unit, int32_t count,
                 int32_t *seq, int32_t *kv_head, int32_t *page) {
    if (cum_pages == nullptr || batch < 1 || num_kv_heads < 1 || first_unit < 0 || count < 0 ||
        (count > 0 && (seq == nullptr || kv_head == nullptr || page == nullptr)))
        return PD_ERR_INVALID_ARG;
    if (first_unit + count > static_cast<int64_t>(num_kv_heads) * cum_pages[batch]) return PD_ERR_INVALID_ARG;
    if (count == 0) return PD_OK;
    pd::Cursor c = pd::locate(cum_pages, batch, num_kv_heads, first_unit);
    for (int i = 0; i < count; ++i) {
        seq[i] = c.b;
        kv_head[i] = c.kvh;
        page[i] = c.page;
        pd::advance(c, cum_pages, batch, num_kv_heads);
    }
    return PD_OK;
}

int pd_set_profile_events(pd_ctx *ctx, void *before, void *after) {
    if (ctx == nullptr || ((before == nullptr) != (after == nullptr))) return PD_ERR_INVALID_ARG;
    ctx->ev_before = static_cast<cudaEvent_t>(before);
    ctx->ev_after = static_cast<cudaEvent_t>(after);
    return PD_OK;
}

int pd_read_worker_trace(pd_ctx *ctx, void *stream, uint64_t *host_out, int32_t max_workers, int32_t *num_workers) {
    if (ctx == nullptr || host_out == nullptr || num_workers == nullptr || max_workers < 0) return PD_ERR_INVALID_ARG;
    *num_workers = 0;
    if (ctx->trace == nullptr) return fail(ctx, PD_ERR_UNSUPPORTED, "tracing is off (needs a PD_ENABLE_TUNING build and PD_TRACE_WORKERS=1 at pd_create)");
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return fail(ctx, PD_ERR_CUDA, "cudaSetDevice");
    const int n = ctx->trace_workers < max_workers ? ctx->trace_workers : max_workers;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t err = cudaMemcpyAsync(host_out, ctx->trace, static_cast<size_t>(n) * 4 * 8, cudaMemcpyDeviceToHost, s);
    if (err == cudaSuccess) err = cudaStreamSynchronize(s);
    if (err != cudaSuccess) return fail(ctx, PD_ERR_CUDA, "trace read", err);
    *num_workers = n;
    return PD_OK;
}

int pd_workspace_bytes(const pd_ctx *ctx, size_t *bytes) {
    if (ctx == nullptr || bytes == nullptr) return PD_ERR_INVALID_ARG;
    *bytes = ctx->workspace_bytes;
    return PD_OK;
}

int pd_launch_count(const pd_ctx *ctx, int64_t *launches) {
    if (ctx == nullptr || launches == nullptr) return PD_ERR_INVALID_ARG;
    *launches = ctx->launches;
    return PD_OK;
}

int pd_last_plan(pd_ctx *ctx, void *stream, int64_t *total_units, int32_t *pages_per_range, int32_t *num_ranges,
                 int32_t *num_workers) {
    if (ctx == nullptr) return PD_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return fail(ctx, PD_ERR_CUDA, "cudaSetDevice");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int32_t host[pd::kPlanWords] = {0};
    cudaError_t err = cudaMemcpyAsync(host, ctx->plan, sizeof host, cudaMemcpyDeviceToHost, s);
    if (err == cudaSuccess) err = cudaStreamSynchronize(s);
    if (err != cudaSuccess) return fail(ctx, PD_ERR_CUDA, "plan read", err);
    if (total_units != nullptr)
        *total_units = (static_cast<int64_t>(host[1]) << 32) | static_cast<uint32_t>(host[0]);
    if (pages_per_range != nullptr) *pages_per_range = host[pd::kPlanHeaderWords + 2];  // first (largest) level
    if (num_ranges != nullptr) *num_ranges = host[3];
    if (num_workers != nullptr) *num_workers = host[4];
    return PD_OK;
}

}  // extern "C"
