// Elastic KV pool on CUDA virtual memory management: a fixed device address range whose physical
// backing can be given up and taken back without the process, the addresses or anything derived
// from them (page ids, tensor maps, pointers held by the caller) changing.
//
// The intra-scale toggle (Sec. 4.6; Sec. 5 on releasing and restoring the KV cache) keeps the rollout
// process alive across a handoff and swaps only device state: the KV cache is released when training
// needs the memory and restored when the GPU comes back. Here that is pd_pool_resize(pool, 0) and pd_pool_resize(pool, capacity); a partial size
// keeps a prefix of the range resident, which is how a decode worker shrinks its cache (the H_max of
// the capacity constraint under Eq. 3) instead of dropping it. The time the two calls take is the KV
// part of T_toggle in Eq. 7.
//
// The range is backed chunk by chunk (one physical allocation per chunk) so that a resize touches
// only the chunks that change. Contents of a chunk do not survive its release. Host code only: no
// kernel is launched here.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <new>
#include <vector>

#include "../../include/pd.h"

namespace {

struct DriverApi {
    CUresult (*reserve)(CUdeviceptr *, size_t, size_t, CUdeviceptr, unsigned long long) = nullptr;
    CUresult (*addr_free)(CUdeviceptr, size_t) = nullptr;
    CUresult (*create)(CUmemGenericAllocationHandle *, size_t, const CUmemAllocationProp *, unsigned long long) = nullptr;
    CUresult (*release)(CUmemGenericAllocationHandle) = nullptr;
    CUresult (*map)(CUdeviceptr, size_t, size_t, CUmemGenericAllocationHandle, unsigned long long) = nullptr;
    CUresult (*unmap)(CUdeviceptr, size_t) = nullptr;
    CUresult (*set_access)(CUdeviceptr, size_t, const CUmemAccessDesc *, size_t) = nullptr;
    CUresult (*granularity)(size_t *, const CUmemAllocationProp *, CUmemAllocationGranularity_flags) = nullptr;
    bool ok = false;
};

template <typename F>
bool resolve(const char *name, F &fn) {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q{};
    if (cudaGetDriverEntryPoint(name, &p, cudaEnableDefault, &q) != cudaSuccess || p == nullptr ||
        q != cudaDriverEntryPointSuccess)
        return false;
    fn = reinterpret_cast<F>(p);
    return true;
}

const DriverApi &driver() {
    static const DriverApi api = [] {
        DriverApi a;
        a.ok = resolve("cuMemAddressReserve", a.reserve) && resolve("cuMemAddressFree", a.addr_free) &&
               resolve("cuMemCreate", a.create) && resolve("cuMemRelease", a.release) && resolve("cuMemMap", a.map) &&
               resolve("cuMemUnmap", a.unmap) && resolve("cuMemSetAccess", a.set_access) &&
               resolve("cuMemGetAllocationGranularity", a.granularity);
        return a;
    }();
    return api;
}

}  // namespace

struct pd_pool {
    int device = 0;
    CUdeviceptr base = 0;
    size_t capacity = 0;  // bytes reserved, a multiple of chunk
    size_t chunk = 0;     // bytes per physical allocation, a multiple of the device granularity
    std::vector<CUmemGenericAllocationHandle> handles;  // one per resident chunk, in address order
    CUmemAllocationProp prop{};
    char last_error[160] = {0};
};

namespace {

int pool_fail(pd_pool *pool, int code, const char *what, CUresult r) {
    if (pool != nullptr) std::snprintf(pool->last_error, sizeof pool->last_error, "%s failed (CUresult %d)", what, static_cast<int>(r));
    return code;
}

// Drops the last resident chunk.
int drop_chunk(pd_pool *pool) {
    const DriverApi &d = driver();
    const size_t i = pool->handles.size() - 1;
    CUresult r = d.unmap(pool->base + i * pool->chunk, pool->chunk);
    if (r != CUDA_SUCCESS) return pool_fail(pool, PD_ERR_CUDA, "cuMemUnmap", r);
    r = d.release(pool->handles[i]);
    pool->handles.pop_back();
    if (r != CUDA_SUCCESS) return pool_fail(pool, PD_ERR_CUDA, "cuMemRelease", r);
    return PD_OK;
}

// Backs the first non-resident chunk.
int add_chunk(pd_pool *pool) {
    const DriverApi &d = driver();
    const size_t i = pool->handles.size();
    CUmemGenericAllocationHandle h{};
    CUresult r = d.create(&h, pool->chunk, &pool->prop, 0);
    if (r != CUDA_SUCCESS) return pool_fail(pool, r == CUDA_ERROR_OUT_OF_MEMORY ? PD_ERR_WORKSPACE : PD_ERR_CUDA, "cuMemCreate", r);
    const CUdeviceptr at = pool->base + i * pool->chunk;
    r = d.map(at, pool->chunk, 0, h, 0);
    if (r != CUDA_SUCCESS) {
        d.release(h);
        return pool_fail(pool, PD_ERR_CUDA, "cuMemMap", r);
    }
    CUmemAccessDesc acc{};
    acc.location = pool->prop.location;
    acc.flags = CU_MEM_ACCESS_FLAGS_PROT_READWRITE;
    r = d.set_access(at, pool->chunk, &acc, 1);
    if (r != CUDA_SUCCESS) {
        d.unmap(at, pool->chunk);
        d.release(h);
        return pool_fail(pool, PD_ERR_CUDA, "cuMemSetAccess", r);
    }
    pool->handles.push_back(h);
    return PD_OK;
}

struct DeviceScope {
    int prev = -1;
    bool ok = false;
    explicit DeviceScope(int dev) {
        ok = cudaGetDevice(&prev) == cudaSuccess && cudaSetDevice(dev) == cudaSuccess && cudaFree(nullptr) == cudaSuccess;
    }
    ~DeviceScope() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

}  // namespace

extern "C" {

int pd_pool_create(int32_t device, uint64_t capacity_bytes, uint64_t chunk_bytes, pd_pool **out) {
    if (out == nullptr) return PD_ERR_INVALID_ARG;
    *out = nullptr;
    if (capacity_bytes == 0 || device < 0) return PD_ERR_INVALID_ARG;
    DeviceScope scope(device);
    if (!scope.ok) return PD_ERR_CUDA;
    const DriverApi &d = driver();
    if (!d.ok) return PD_ERR_UNSUPPORTED;
    pd_pool *pool = new (std::nothrow) pd_pool;
    if (pool == nullptr) return PD_ERR_CUDA;
    pool->device = device;
    pool->prop.type = CU_MEM_ALLOCATION_TYPE_PINNED;
    pool->prop.location.type = CU_MEM_LOCATION_TYPE_DEVICE;
    pool->prop.location.id = device;
    size_t gran = 0;
    CUresult r = d.granularity(&gran, &pool->prop, CU_MEM_ALLOC_GRANULARITY_RECOMMENDED);
    if (r != CUDA_SUCCESS || gran == 0) {
        delete pool;
        return PD_ERR_CUDA;
    }
    if (chunk_bytes == 0) chunk_bytes = 256ull << 20;
    pool->chunk = (chunk_bytes + gran - 1) / gran * gran;
    pool->capacity = (capacity_bytes + pool->chunk - 1) / pool->chunk * pool->chunk;
    r = d.reserve(&pool->base, pool->capacity, 0, 0, 0);
    if (r != CUDA_SUCCESS) {
        delete pool;
        return PD_ERR_CUDA;
    }
    pool->handles.reserve(pool->capacity / pool->chunk);
    *out = pool;
    return PD_OK;
}

int pd_pool_resize(pd_pool *pool, uint64_t resident_bytes, void *stream_to_drain) {
    if (pool == nullptr) return PD_ERR_INVALID_ARG;
    if (resident_bytes > pool->capacity) return pool_fail(pool, PD_ERR_INVALID_ARG, "pd_pool_resize: size above capacity", CUDA_SUCCESS);
    DeviceScope scope(pool->device);
    if (!scope.ok) return PD_ERR_CUDA;
    const size_t want = (resident_bytes + pool->chunk - 1) / pool->chunk;
    if (want < pool->handles.size()) {
        // Work that still reads or writes the chunks must have finished before they are unmapped.
        const cudaError_t e = stream_to_drain != nullptr ? cudaStreamSynchronize(static_cast<cudaStream_t>(stream_to_drain))
                                                         : cudaDeviceSynchronize();
        if (e != cudaSuccess) return pool_fail(pool, PD_ERR_CUDA, "synchronise before release", CUDA_ERROR_UNKNOWN);
    }
    while (pool->handles.size() > want)
        if (int rc = drop_chunk(pool)) return rc;
    while (pool->handles.size() < want)
        if (int rc = add_chunk(pool)) return rc;  // on failure the chunks backed so far stay resident
    return PD_OK;
}

void *pd_pool_base(const pd_pool *pool) { return pool != nullptr ? reinterpret_cast<void *>(pool->base) : nullptr; }
uint64_t pd_pool_capacity(const pd_pool *pool) { return pool != nullptr ? pool->capacity : 0; }
uint64_t pd_pool_chunk_bytes(const pd_pool *pool) { return pool != nullptr ? pool->chunk : 0; }
uint64_t pd_pool_resident_bytes(const pd_pool *pool) { return pool != nullptr ? pool->handles.size() * pool->chunk : 0; }
const char *pd_pool_last_error(const pd_pool *pool) { return pool != nullptr ? pool->last_error : "null pool"; }

int pd_pool_destroy(pd_pool *pool) {
    if (pool == nullptr) return PD_OK;
    int rc = PD_OK;
    {
        DeviceScope scope(pool->device);
        if (scope.ok) cudaDeviceSynchronize();
        while (!pool->handles.empty()) {
            const size_t before = pool->handles.size();
            if (int e = drop_chunk(pool)) rc = e;
            if (pool->handles.size() == before) break;  // the unmap failed and the chunk stays: do not spin on it
        }
        if (pool->base != 0 && driver().ok && driver().addr_free(pool->base, pool->capacity) != CUDA_SUCCESS) rc = PD_ERR_CUDA;
    }
    delete pool;
    return rc;
}

}  // extern "C"
