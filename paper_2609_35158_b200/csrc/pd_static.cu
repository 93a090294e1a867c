// pd_decode_attn_static: decode attention for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc when they need attention:
// a serving engine that has handed the whole device to its own KV-cache pool,
// a plugin running inside another framework's memory budget, a process whose
// allocator is frozen once warm-up is over. pd_create allocates a workspace, so
// it is closed to them. This entry point runs the same split-KV kernels with
// their scratch (fp32 partials, page prefix sums, plan and status words) placed
// in a fixed array that is part of the library image. It calls no cudaMalloc,
// cudaFree or allocating library routine.
//
// The array is a file-scope __device__ symbol. On the host its name is only a
// stand-in: the device address is obtained once per device, with that device
// current, through cudaGetSymbolAddress, and that pointer is what the kernels
// receive.
#include "../../include/pd.h"

#include <mutex>

#include "pd_kernels.cuh"

namespace {

constexpr size_t kStaticScratchBytes = size_t(16) << 20;  // 16 MiB, held by every device that loads the library
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct DeviceSetup {
    bool ready = false;
    unsigned char *scratch = nullptr;  // device address of g_static_scratch on this device
    int num_sms = 0;
    size_t smem_bytes[2] = {0, 0};     // per head_dim variant: [0] = 64, [1] = 128
    bool variant_ready[2] = {false, false};
};

std::mutex g_mutex;
DeviceSetup g_setup[kMaxDevices];
EncodeTiledFn g_encode = nullptr;

pd::AttnVariant variant_for(int head_dim) {
    pd::AttnVariant v{};
    v.head_dim = head_dim;
    v.warps = 8;
    v.stages = head_dim == 128 ? 3 : 6;
    v.hilo = 1;
    return v;
}

size_t round256(size_t n) { return (n + 255) & ~size_t(255); }

int encode_map(const pd_config &c, const void *pool, CUtensorMap *out) {
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(c.head_dim),
                                static_cast<cuuint64_t>(c.num_pages) * c.num_kv_heads * c.page_size};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(c.head_dim) * 2};
    const cuuint32_t box[2] = {64, static_cast<cuuint32_t>(c.page_size)};
    const cuuint32_t elem_strides[2] = {1, 1};
    const CUresult r = g_encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(pool), dims, strides, box,
                                elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? PD_OK : PD_ERR_CUDA;
}

}  // namespace

extern "C" int pd_decode_attn_static(const pd_config *cfg, const void *q, const void *k_pages, const void *v_pages,
                                     const int32_t *page_table, const int32_t *ctx_lens, void *out, float *lse,
                                     int32_t batch, float sm_scale, void *stream) {
    if (cfg == nullptr) return PD_ERR_INVALID_ARG;
    if (cfg->num_q_heads <= 0 || cfg->num_kv_heads <= 0 || cfg->num_q_heads % cfg->num_kv_heads != 0 ||
        cfg->max_pages_per_seq < 1 || cfg->num_pages < 1 || cfg->device < 0 || cfg->device >= kMaxDevices)
        return PD_ERR_INVALID_ARG;
    const int group = cfg->num_q_heads / cfg->num_kv_heads;
    if (cfg->page_size != pd::kPageSize || (cfg->head_dim != 64 && cfg->head_dim != 128) ||
        (group != 1 && group != 2 && group != 4 && group != 8))
        return PD_ERR_UNSUPPORTED;
    if (cfg->num_pages * cfg->num_kv_heads * cfg->page_size >= (int64_t(1) << 31)) return PD_ERR_UNSUPPORTED;
    if (static_cast<int64_t>(cfg->max_pages_per_seq) * cfg->page_size >= (int64_t(1) << 31)) return PD_ERR_UNSUPPORTED;
    auto misaligned = [](const void *p) { return p == nullptr || (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
    if (misaligned(q) || misaligned(k_pages) || misaligned(v_pages) || misaligned(out) || page_table == nullptr ||
        ctx_lens == nullptr)
        return PD_ERR_INVALID_ARG;
    if (batch < 0 || batch > pd::kMaxBatch) return PD_ERR_INVALID_ARG;
    if (!(sm_scale > 0.f) || !(sm_scale < 3.0e38f)) return PD_ERR_INVALID_ARG;
    if (batch == 0) return PD_OK;

    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return PD_ERR_CUDA;
    if (prev != cfg->device && cudaSetDevice(cfg->device) != cudaSuccess) return PD_ERR_CUDA;
    struct Restore {
        int prev, dev;
        ~Restore() { if (prev != dev) cudaSetDevice(prev); }
    } restore{prev, cfg->device};

    const int vi = cfg->head_dim == 128 ? 1 : 0;
    const pd::AttnVariant variant = variant_for(cfg->head_dim);
    DeviceSetup local;
    {
        // once per device, with that device current: resolve the scratch symbol's device address
        std::lock_guard<std::mutex> lock(g_mutex);
        DeviceSetup &s = g_setup[cfg->device];
        if (!s.ready) {
            cudaDeviceProp prop{};
            if (cudaGetDeviceProperties(&prop, cfg->device) != cudaSuccess) return PD_ERR_CUDA;
            if (prop.major != 10) return PD_ERR_UNSUPPORTED;
            void *ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) return PD_ERR_CUDA;
            s.scratch = static_cast<unsigned char *>(ptr);
            s.num_sms = prop.multiProcessorCount;
            s.ready = true;
        }
        if (!s.variant_ready[vi]) {
            if (pd::prepare_decode_attn(variant, &s.smem_bytes[vi]) != cudaSuccess) return PD_ERR_CUDA;
            s.variant_ready[vi] = true;
        }
        if (g_encode == nullptr) {
            void *fn = nullptr;
            cudaDriverEntryPointQueryResult qres{};
            if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
                fn == nullptr || qres != cudaDriverEntryPointSuccess)
                return PD_ERR_CUDA;
            g_encode = reinterpret_cast<EncodeTiledFn>(fn);
        }
        local = s;
    }

    // carve the fixed array: status, plan, prefix sums, (m, l) pairs, partial outputs
    const int num_ctas = local.num_sms;
    const size_t workers = static_cast<size_t>(num_ctas) * variant.warps;
    const size_t slots = workers + static_cast<size_t>(batch) * cfg->num_kv_heads;
    const size_t off_status = 0;
    const size_t off_plan = off_status + round256(pd::kStatusWords * sizeof(int32_t));
    const size_t off_cum = off_plan + round256(pd::kPlanWords * sizeof(int32_t));
    const size_t off_ml = off_cum + round256((static_cast<size_t>(batch) + 1) * sizeof(int32_t));
    const size_t off_o = off_ml + round256(slots * group * sizeof(float2));
    const size_t end = off_o + round256(slots * group * cfg->head_dim * sizeof(float));
    if (end > kStaticScratchBytes) return PD_ERR_WORKSPACE;  // batch x KV heads too large for the fixed scratch

    alignas(64) CUtensorMap tm_k, tm_v;
    if (encode_map(*cfg, k_pages, &tm_k) != PD_OK || encode_map(*cfg, v_pages, &tm_v) != PD_OK) return PD_ERR_CUDA;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the array keeps the previous call's contents; the status latch and the range-claim counters must start at zero
    if (cudaMemsetAsync(local.scratch + off_status, 0, pd::kStatusWords * sizeof(int32_t), s) != cudaSuccess)
        return PD_ERR_CUDA;

    pd::AttnParams p{};
    p.q = static_cast<const __nv_bfloat16 *>(q);
    p.page_table = page_table;
    p.ctx_lens = ctx_lens;
    p.out = static_cast<__nv_bfloat16 *>(out);
    p.lse = lse;
    p.part_o = reinterpret_cast<float *>(local.scratch + off_o);
    p.part_ml = reinterpret_cast<float2 *>(local.scratch + off_ml);
    p.cum_pages = reinterpret_cast<int32_t *>(local.scratch + off_cum);
    p.plan = reinterpret_cast<int32_t *>(local.scratch + off_plan);
    p.status = reinterpret_cast<int32_t *>(local.scratch + off_status);
    p.B = batch;
    p.Hq = cfg->num_q_heads;
    p.Hkv = cfg->num_kv_heads;
    p.G = group;
    p.MP = cfg->max_pages_per_seq;
    p.num_pages = static_cast<int32_t>(cfg->num_pages);
    p.scale_log2 = sm_scale * 1.4426950408889634f;
    p.split_pages = 0;
    p.max_ranges = static_cast<int32_t>(workers);
    p.min_pages_auto = 4;
    p.halving_levels = 0;  // one level of equal ranges, one per worker: the partial count stays within the fixed array
    p.tail_pages = 16;
    if (pd::launch_decode_attn(variant, tm_k, tm_v, p, num_ctas, local.smem_bytes[vi], s) != cudaSuccess)
        return PD_ERR_CUDA;
    if (pd::launch_lse_merge(cfg->head_dim, p, s) != cudaSuccess) return PD_ERR_CUDA;
    return PD_OK;
}
