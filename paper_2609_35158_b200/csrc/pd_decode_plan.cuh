// Work decomposition shared by the split-KV decode kernels (bf16 and FP8 pages): the page prefix sums,
// the plan of ranges every CTA derives from the lengths alone, the cursor over (sequence, KV head, page)
// units and the per-warp page-id cache. See pd_decode_attn.cu for how the kernels use them.
#pragma once
#include "pd_kernels.cuh"
#include "pd_ptx.cuh"

namespace pd {

namespace {

constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleSlack = 8.f;  // log2 units a logit may exceed the running max before a rescale
constexpr int kClaimAhead = 2;  // pages left to issue in a range when the next range is claimed

struct Cursor {
    int b, kvh, page, np;  // np = pages of sequence b
};

// Page ids of 32 consecutive logical pages of one sequence, one per lane, plus
// the following 32 prefetched.
struct PageIdCache {
    int b, blk, val, nval;
};

// One level of the plan: `count` ranges of `size` units starting at unit `start`;
// `first` is the index of its first range. lv[n_levels] is a sentinel
// (start = total, first = number of ranges).
struct PlanLevel {
    long long start;
    int size, first;
};
struct Plan {
    long long total;
    int n_levels, n_ranges;
    PlanLevel lv[kMaxLevels + 1];
};

__device__ __forceinline__ void latch_status(int32_t *status, int code, int seq, int detail) {
    if (atomicCAS(status, kDevOk, code) == kDevOk) {
        status[1] = seq;
        status[2] = detail;
    }
}

__device__ __forceinline__ int clamp_len(int L, int MP) {
    return min(max(L, 0), MP * kPageSize);
}

// Exclusive prefix sum of pages per sequence into shared memory; cum[B] = total.
template <int THREADS>
__device__ void scan_pages(const AttnParams &p, int32_t *cum, int32_t *warp_sums) {
    const int tid = threadIdx.x;
    const int items = (p.B + THREADS - 1) / THREADS;
    const int begin = min(p.B, tid * items), end = min(p.B, begin + items);
    int sum = 0;
    for (int i = begin; i < end; ++i) {
        const int L = __ldg(p.ctx_lens + i) + p.fused;
        if (L < p.fused || L > p.MP * kPageSize) latch_status(p.status, kDevBadLength, i, L - p.fused);
        sum += (clamp_len(L, p.MP) + kPageSize - 1) / kPageSize;
    }
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, incl, o);
        if ((tid & 31) >= o) incl += t;
    }
    if ((tid & 31) == 31) warp_sums[tid >> 5] = incl;
    __syncthreads();
    int base = 0;
    for (int w = 0; w < (tid >> 5); ++w) base += warp_sums[w];
    int run = base + incl - sum;
    for (int i = begin; i < end; ++i) {
        cum[i] = run;
        run += (clamp_len(__ldg(p.ctx_lens + i) + p.fused, p.MP) + kPageSize - 1) / kPageSize;
    }
    if (tid == THREADS - 1) cum[p.B] = run;
    __syncthreads();
}

// The plan is a pure function of (total, workers, parameters): every CTA and the
// merge kernel's reader derive the same one.
__host__ __device__ inline void make_plan(Plan &pl, long long total, int n_workers, const AttnParams &p) {
    pl.total = total;
    int nl = 0, first = 0;
    long long pos = 0;
    if (p.split_pages > 0) {
        long long size = p.split_pages;
        if ((total + size - 1) / size > p.max_ranges) size = (total + p.max_ranges - 1) / p.max_ranges;
        pl.lv[0].start = 0; pl.lv[0].size = static_cast<int>(size); pl.lv[0].first = 0;
        first = static_cast<int>((total + size - 1) / size);
        nl = 1;
    } else {
        long long fair = (total + n_workers - 1) / n_workers;
        // a kernel whose workers all run at the same speed (the FP8 one: bound by its own instruction stream, not by
        // the memory system) gains nothing from claiming small ranges late and pays for every extra range
        const int levels = fair <= p.static_fair_max ? 0 : p.halving_levels;
        const int tail = static_cast<int>(max(static_cast<long long>(p.min_pages_auto),
                                              min(static_cast<long long>(p.tail_pages), fair)));
        for (int l = 0; l < levels && nl < kMaxLevels - 1; ++l) {
            const long long rem = total - pos;
            const long long size = (rem + 2ll * n_workers - 1) / (2ll * n_workers);
            if (size < 2ll * tail || first + 2 * n_workers > p.max_ranges) break;
            pl.lv[nl].start = pos; pl.lv[nl].size = static_cast<int>(size); pl.lv[nl].first = first;
            pos += size * n_workers;
            first += n_workers;
            ++nl;
        }
        const long long rem = total - pos;
        if (rem > 0 || nl == 0) {
            long long size = levels > 0 ? tail : max(fair, static_cast<long long>(p.min_pages_auto));
            const long long room = max(1, p.max_ranges - first);
            if ((rem + size - 1) / size > room) size = (rem + room - 1) / room;
            if (size < 1) size = 1;
            pl.lv[nl].start = pos; pl.lv[nl].size = static_cast<int>(size); pl.lv[nl].first = first;
            first += static_cast<int>((rem + size - 1) / size);
            ++nl;
        }
    }
    pl.lv[nl].start = total; pl.lv[nl].size = 1; pl.lv[nl].first = first;
    pl.n_levels = nl;
    pl.n_ranges = first;
}

__host__ __device__ __forceinline__ void range_bounds(const Plan &pl, int rid, long long &start, int &len) {
    int l = 0;
    while (l + 1 < pl.n_levels && rid >= pl.lv[l + 1].first) ++l;
    start = pl.lv[l].start + static_cast<long long>(rid - pl.lv[l].first) * pl.lv[l].size;
    len = static_cast<int>(min(static_cast<long long>(pl.lv[l].size), pl.lv[l + 1].start - start));
}

__host__ __device__ __forceinline__ Cursor locate(const int32_t *cum, int B, int Hkv, long long x) {
    const int y = static_cast<int>(x / Hkv);  // largest b with cum[b] <= y owns unit x
    int lo = 0, hi = B - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (cum[mid] <= y) lo = mid; else hi = mid - 1;
    }
    Cursor c;
    c.b = lo;
    c.np = cum[lo + 1] - cum[lo];
    const int rem = static_cast<int>(x - static_cast<long long>(Hkv) * cum[lo]);
    c.kvh = rem / c.np;
    c.page = rem - c.kvh * c.np;
    return c;
}

__host__ __device__ __forceinline__ void advance(Cursor &c, const int32_t *cum, int B, int Hkv) {
    if (++c.page >= c.np) {
        c.page = 0;
        if (++c.kvh == Hkv) {
            c.kvh = 0;
            do {
                ++c.b;
                c.np = (c.b < B) ? cum[c.b + 1] - cum[c.b] : 1;
            } while (c.b < B && c.np == 0);
        }
    }
}

__device__ __forceinline__ int page_id(PageIdCache &c, const AttnParams &p, int b, int page, int lane) {
    const int blk = page >> 5;
    if (c.b != b || c.blk != blk) {  // warp-uniform
        const int32_t *row = p.page_table + static_cast<size_t>(b) * p.MP;
        if (c.b == b && c.blk + 1 == blk) {
            c.val = c.nval;
        } else {
            const int idx = blk * 32 + lane;
            c.val = (idx < p.MP) ? __ldg(row + idx) : -1;
        }
        c.b = b;
        c.blk = blk;
        const int nidx = (blk + 1) * 32 + lane;
        c.nval = (nidx < p.MP) ? __ldg(row + nidx) : -1;
    }
    return __shfl_sync(0xffffffffu, c.val, page & 31);
}

}  // namespace

}  // namespace pd
