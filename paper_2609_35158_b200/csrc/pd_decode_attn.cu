// Split-KV decode attention over a paged bf16 KV cache, and the log-sum-exp merge.
//
// The operation is the per-sequence KV-read term of the decode cost model
// (Eq. 1: b, "extra KV-cache HBM reads"): one query token per sequence attends
// over every cached token of its KV head. The kernel is a scan of the cache at
// HBM speed; everything below serves that.
//
// Work decomposition. Units are (sequence, KV head, page) triples in that
// nesting order; their flattened list is cut into ranges of `per` units. A
// worker is ONE WARP: it owns a range, its own ring of shared-memory stages and
// its own mbarriers, issues its own TMA loads (lane 0) and never synchronises
// with another warp after the prologue. A range may cross (sequence, KV head)
// boundaries; each maximal piece inside one (sequence, KV head) is a segment.
// A segment that covers the whole context writes the final bf16 row directly;
// any other segment writes an fp32 partial to slot (range index + pair index),
// which is unique and contiguous per pair, and the merge kernel combines them.
//
// Data movement. A (page, KV head) tile is 16 tokens x D bf16, contiguous in
// HBM. It is fetched by tiled TMA as D/64 boxes of 16 rows x 128 B with the
// 128-byte swizzle, so ldmatrix reads are bank-conflict free. K and V of a page
// complete on separate mbarriers.
//
// Math. The query group (g <= 8 heads sharing the KV head) is the M dimension
// of mma.sync.m16n8k16 (rows g..15 are zero): S = Q K^T per page, online
// softmax in fp32 in log2 units with a lazy rescale, then O += P V with P split
// into a bf16 high and low part (two MMAs) so that P carries ~16 mantissa bits.
#include "pd_kernels.cuh"
#include "pd_ptx.cuh"

namespace pd {

namespace {

constexpr float kLn2 = 0.6931471805599453f;

struct Cursor {
    int b, kvh, page, np;  // np = pages of sequence b
};

// Page ids of 32 consecutive logical pages of one sequence, one per lane, plus
// the following 32 prefetched.
struct PageIdCache {
    int b, blk, val, nval;
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
        const int L = __ldg(p.ctx_lens + i);
        if (L < 0 || L > p.MP * kPageSize) latch_status(p.status, kDevBadLength, i, L);
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
        run += (clamp_len(__ldg(p.ctx_lens + i), p.MP) + kPageSize - 1) / kPageSize;
    }
    if (tid == THREADS - 1) cum[p.B] = run;
    __syncthreads();
}

__device__ __forceinline__ Cursor locate(const int32_t *cum, int B, int Hkv, int64_t x) {
    const int y = static_cast<int>(x / Hkv);  // largest b with cum[b] <= y owns unit x
    int lo = 0, hi = B - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (cum[mid] <= y) lo = mid; else hi = mid - 1;
    }
    Cursor c;
    c.b = lo;
    c.np = cum[lo + 1] - cum[lo];
    const int rem = static_cast<int>(x - static_cast<int64_t>(Hkv) * cum[lo]);
    c.kvh = rem / c.np;
    c.page = rem - c.kvh * c.np;
    return c;
}

__device__ __forceinline__ void advance(Cursor &c, const int32_t *cum, int B, int Hkv, int pages) {
    c.page += pages;
    if (c.page >= c.np) {
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

template <int D, int WARPS, int STAGES, bool HILO>
__global__ void __launch_bounds__(WARPS * 32, 1)
decode_attn_split_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                         const AttnParams p) {
    constexpr int THREADS = WARPS * 32;
    constexpr int HALVES = D / 64;             // 128-byte column blocks per row
    constexpr int HALF_BYTES = kPageSize * 128;  // one TMA box: 16 rows x 128 B
    constexpr int TILE_BYTES = HALVES * HALF_BYTES;
    constexpr int STAGE_BYTES = 2 * TILE_BYTES;  // K tile then V tile
    constexpr int KSTEPS = D / 16;
    constexpr int NTILES = D / 8;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring0 = (raw + 1023u) & ~1023u;  // swizzled boxes need 1024-byte alignment
    uint8_t *aligned = smem_raw + (ring0 - raw);
    uint64_t *bars = reinterpret_cast<uint64_t *>(aligned + WARPS * STAGES * STAGE_BYTES);
    int32_t *warp_sums = reinterpret_cast<int32_t *>(bars + WARPS * STAGES * 2);
    int32_t *cum = warp_sums + 32;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // ---- prologue (whole CTA): barriers, page prefix sums, the plan
    if (lane == 0) {
        for (int s = 0; s < STAGES * 2; ++s) mbar_init(smem_u32(bars + (warp * STAGES * 2 + s)), 1);
        mbar_init_fence();
    }
    if (tid == 0) {
        prefetch_tensormap(&tm_k);
        prefetch_tensormap(&tm_v);
    }
    scan_pages<THREADS>(p, cum, warp_sums);

    const int64_t total = static_cast<int64_t>(p.Hkv) * cum[p.B];
    const int n_workers = gridDim.x * WARPS;
    int64_t per;
    if (p.split_pages > 0) {
        per = p.split_pages;
        if ((total + per - 1) / per > p.max_ranges) per = (total + p.max_ranges - 1) / p.max_ranges;
    } else {
        per = (total + n_workers - 1) / n_workers;
        if (per < p.min_pages_auto) per = p.min_pages_auto;
    }
    if (per < 1) per = 1;
    const int64_t n_ranges = (total + per - 1) / per;
    if (blockIdx.x == 0) {
        for (int i = tid; i <= p.B; i += THREADS) p.cum_pages[i] = cum[i];
        if (tid == 0) {
            p.plan[0] = static_cast<int32_t>(total & 0xffffffffll);
            p.plan[1] = static_cast<int32_t>(total >> 32);
            p.plan[2] = static_cast<int32_t>(per);
            p.plan[3] = static_cast<int32_t>(n_ranges);
            p.plan[4] = n_workers;
        }
    }

    // ---- per-warp state
    const uint32_t ring = ring0 + warp * STAGES * STAGE_BYTES;
    const uint32_t bar0 = smem_u32(bars + warp * STAGES * 2);
    const uint64_t policy = l2_policy_evict_first();
    const int quad_row = lane >> 2;  // query head inside the group handled by this lane
    const int quad_col = (lane & 3) * 2;
    const int G = p.G;
    // ldmatrix lane addressing inside a tile (row = token, 16-byte chunk index swizzled by row & 7)
    const int mat = lane >> 3, r8 = lane & 7;
    const uint32_t k_row_off = (((mat >> 1) * 8 + r8) * 128);
    const int k_sel = mat & 1;
    const uint32_t v_row_off = (((mat & 1) * 8 + r8) * 128);
    const int v_sel = mat >> 1;

    PageIdCache pt;
    pt.b = -1; pt.blk = -1; pt.val = -1; pt.nval = -1;
    uint32_t stage = 0, parity = 0;  // ring position of the next page to consume
    bool alive = true;

    for (int64_t range = blockIdx.x * WARPS + warp; range < n_ranges && alive; range += n_workers) {
        const int64_t x0 = range * per;
        const int n_total = static_cast<int>(min(total - x0, per));
        Cursor cons = locate(cum, p.B, p.Hkv, x0);
        Cursor prod = cons;
        int issued = 0;

        auto issue = [&](uint32_t st) {
            int pid = page_id(pt, p, prod.b, prod.page, lane);
            if (pid < 0 || pid >= p.num_pages) {
                if (lane == 0) latch_status(p.status, kDevBadPage, prod.b, pid);
                pid = 0;
            }
            if (lane == 0) {
                const int32_t y = (pid * p.Hkv + prod.kvh) * kPageSize;
                const uint32_t dst = ring + st * STAGE_BYTES;
                const uint32_t bk = bar0 + st * 16, bv = bk + 8;
                mbar_arrive_expect_tx(bk, TILE_BYTES);
#pragma unroll
                for (int h = 0; h < HALVES; ++h) tma_load_2d(dst + h * HALF_BYTES, &tm_k, h * 64, y, bk, policy);
                mbar_arrive_expect_tx(bv, TILE_BYTES);
#pragma unroll
                for (int h = 0; h < HALVES; ++h)
                    tma_load_2d(dst + TILE_BYTES + h * HALF_BYTES, &tm_v, h * 64, y, bv, policy);
            }
            advance(prod, cum, p.B, p.Hkv, 1);
            ++issued;
        };

        {
            uint32_t st = stage;
            const int fill = min(STAGES, n_total);
            while (issued < fill) {
                issue(st);
                st = (st + 1 == STAGES) ? 0 : st + 1;
            }
        }

        int consumed = 0;
        while (consumed < n_total && alive) {
            // ---- segment: pages [page0, page0 + seg) of (b, kvh)
            const int b = cons.b, kvh = cons.kvh, page0 = cons.page;
            const int seg = min(n_total - consumed, cons.np - page0);
            const int L = clamp_len(__ldg(p.ctx_lens + b), p.MP);

            // Q fragments: row quad_row of the group, zero rows beyond the group
            uint32_t qa[KSTEPS][2];
            {
                const __nv_bfloat16 *qrow = p.q + (static_cast<size_t>(b) * p.Hq + kvh * G + quad_row) * D;
#pragma unroll
                for (int kk = 0; kk < KSTEPS; ++kk) {
                    if (quad_row < G) {
                        qa[kk][0] = __ldg(reinterpret_cast<const uint32_t *>(qrow + kk * 16 + quad_col));
                        qa[kk][1] = __ldg(reinterpret_cast<const uint32_t *>(qrow + kk * 16 + 8 + quad_col));
                    } else {
                        qa[kk][0] = 0u;
                        qa[kk][1] = 0u;
                    }
                }
            }
            float O[NTILES][4];
#pragma unroll
            for (int j = 0; j < NTILES; ++j) { O[j][0] = 0.f; O[j][1] = 0.f; O[j][2] = 0.f; O[j][3] = 0.f; }
            float m_run = -INFINITY, l_run = 0.f;

            for (int i = 0; i < seg; ++i) {
                const uint32_t kbase = ring + stage * STAGE_BYTES;
                const uint32_t vbase = kbase + TILE_BYTES;
                const uint32_t bk = bar0 + stage * 16, bv = bk + 8;
                const int valid = L - (page0 + i) * kPageSize;  // tokens of this page inside the context

                if (!__all_sync(0xffffffffu, mbar_wait(bk, parity))) { alive = false; break; }

                // S = Q K^T for 16 tokens: two 8-token column tiles, two accumulators each
                float Sa[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
                float Sb[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
                for (int kk = 0; kk < KSTEPS; ++kk) {
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4(b0, b1, b2, b3,
                                kbase + (kk >> 2) * HALF_BYTES + k_row_off + ((((kk & 3) * 2 + k_sel) ^ r8) << 4));
                    if (kk & 1) {
                        mma_bf16_16816(Sb[0], qa[kk][0], 0u, qa[kk][1], 0u, b0, b1);
                        mma_bf16_16816(Sb[1], qa[kk][0], 0u, qa[kk][1], 0u, b2, b3);
                    } else {
                        mma_bf16_16816(Sa[0], qa[kk][0], 0u, qa[kk][1], 0u, b0, b1);
                        mma_bf16_16816(Sa[1], qa[kk][0], 0u, qa[kk][1], 0u, b2, b3);
                    }
                }
                // this lane: row quad_row, tokens quad_col, +1, +8, +9 (log2 units)
                float s0 = (Sa[0][0] + Sb[0][0]) * p.scale_log2, s1 = (Sa[0][1] + Sb[0][1]) * p.scale_log2;
                float s2 = (Sa[1][0] + Sb[1][0]) * p.scale_log2, s3 = (Sa[1][1] + Sb[1][1]) * p.scale_log2;
                if (valid < kPageSize) {  // last page of the context: mask, never multiply
                    if (quad_col >= valid) s0 = -INFINITY;
                    if (quad_col + 1 >= valid) s1 = -INFINITY;
                    if (quad_col + 8 >= valid) s2 = -INFINITY;
                    if (quad_col + 9 >= valid) s3 = -INFINITY;
                }
                float mx = fmaxf(fmaxf(s0, s1), fmaxf(s2, s3));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                const float m_new = fmaxf(m_run, mx);
                if (__any_sync(0xffffffffu, m_new > m_run)) {  // lazy rescale of the running state
                    const float alpha = fast_exp2(m_run - m_new);
                    l_run *= alpha;
#pragma unroll
                    for (int j = 0; j < NTILES; ++j) { O[j][0] *= alpha; O[j][1] *= alpha; }
                    m_run = m_new;
                }
                const float p0 = fast_exp2(s0 - m_run), p1 = fast_exp2(s1 - m_run);
                const float p2 = fast_exp2(s2 - m_run), p3 = fast_exp2(s3 - m_run);
                l_run += (p0 + p1) + (p2 + p3);
                const __nv_bfloat162 h01 = __floats2bfloat162_rn(p0, p1), h23 = __floats2bfloat162_rn(p2, p3);
                const uint32_t pa0 = *reinterpret_cast<const uint32_t *>(&h01);
                const uint32_t pa2 = *reinterpret_cast<const uint32_t *>(&h23);
                uint32_t pl0 = 0u, pl2 = 0u;
                if (HILO) {
                    pl0 = pack_bf16x2(p0 - __low2float(h01), p1 - __high2float(h01));
                    pl2 = pack_bf16x2(p2 - __low2float(h23), p3 - __high2float(h23));
                }

                if (!__all_sync(0xffffffffu, mbar_wait(bv, parity))) { alive = false; break; }
                if (valid < kPageSize) {
                    // V rows past the context may hold NaN; 0 * NaN is NaN, so clear them first
                    for (int row = valid; row < kPageSize; ++row)
                        if (lane < HALVES * 8)
                            st_shared_zero16(vbase + (lane >> 3) * HALF_BYTES + row * 128 + (lane & 7) * 16);
                    __syncwarp();
                }
                // O += P V : 16 tokens (k) x D columns
#pragma unroll
                for (int j = 0; j < NTILES / 2; ++j) {
                    uint32_t v0, v1, v2, v3;
                    ldmatrix_x4_trans(v0, v1, v2, v3,
                                      vbase + (j >> 2) * HALF_BYTES + v_row_off + ((((j & 3) * 2 + v_sel) ^ r8) << 4));
                    mma_bf16_16816(O[2 * j], pa0, 0u, pa2, 0u, v0, v1);
                    mma_bf16_16816(O[2 * j + 1], pa0, 0u, pa2, 0u, v2, v3);
                    if (HILO) {
                        mma_bf16_16816(O[2 * j], pl0, 0u, pl2, 0u, v0, v1);
                        mma_bf16_16816(O[2 * j + 1], pl0, 0u, pl2, 0u, v2, v3);
                    }
                }
                __syncwarp();  // every lane has read this stage
                if (valid < kPageSize) fence_proxy_async();  // generic-proxy stores before the next TMA write
                if (issued < n_total) issue(stage);
                if (++stage == STAGES) { stage = 0; parity ^= 1u; }
            }
            if (!alive) break;

            // ---- end of segment: final row or partial
            float l_tot = l_run + __shfl_xor_sync(0xffffffffu, l_run, 1);
            l_tot += __shfl_xor_sync(0xffffffffu, l_tot, 2);
            if (quad_row < G) {
                const int h = kvh * G + quad_row;
                if (page0 == 0 && seg == cons.np) {
                    const float inv = 1.f / l_tot;
                    __nv_bfloat16 *orow = p.out + (static_cast<size_t>(b) * p.Hq + h) * D + quad_col;
#pragma unroll
                    for (int j = 0; j < NTILES; ++j)
                        *reinterpret_cast<__nv_bfloat162 *>(orow + j * 8) =
                            __floats2bfloat162_rn(O[j][0] * inv, O[j][1] * inv);
                    if (p.lse != nullptr && (lane & 3) == 0)
                        p.lse[static_cast<size_t>(b) * p.Hq + h] = (m_run + log2f(l_tot)) * kLn2;
                } else {
                    const size_t slot = static_cast<size_t>(range) + static_cast<size_t>(b) * p.Hkv + kvh;
                    float *orow = p.part_o + (slot * G + quad_row) * D + quad_col;
#pragma unroll
                    for (int j = 0; j < NTILES; ++j)
                        *reinterpret_cast<float2 *>(orow + j * 8) = make_float2(O[j][0], O[j][1]);
                    if ((lane & 3) == 0) p.part_ml[slot * G + quad_row] = make_float2(m_run, l_tot);
                }
            }
            consumed += seg;
            advance(cons, cum, p.B, p.Hkv, seg);
        }
    }
    if (!alive && lane == 0) latch_status(p.status, kDevTimeout, -1, blockIdx.x * WARPS + warp);
}

// One warp per (sequence, query head): combine that row's partials in slot order.
template <int D>
__global__ void __launch_bounds__(128) lse_merge_kernel(const AttnParams p) {
    constexpr int VEC = D / 32;
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= p.B * p.Hq) return;
    const int b = row / p.Hq, h = row - b * p.Hq;
    const int kvh = h / p.G, r = h - kvh * p.G;
    const int c0 = p.cum_pages[b], np = p.cum_pages[b + 1] - c0;
    __nv_bfloat16 *orow = p.out + static_cast<size_t>(row) * D + lane * VEC;
    if (np == 0) {  // empty context
#pragma unroll
        for (int v = 0; v < VEC; ++v) orow[v] = __float2bfloat16(0.f);
        if (p.lse != nullptr && lane == 0) p.lse[row] = -INFINITY;
        return;
    }
    const int64_t per = p.plan[2];
    const int64_t u0 = static_cast<int64_t>(p.Hkv) * c0 + static_cast<int64_t>(kvh) * np;
    const int64_t first = u0 / per, last = (u0 + np - 1) / per;
    if (first == last) return;  // written directly by the split kernel
    const int n = static_cast<int>(last - first) + 1;
    const size_t slot0 = static_cast<size_t>(first) + static_cast<size_t>(b) * p.Hkv + kvh;
    float M = -INFINITY;
    for (int i = lane; i < n; i += 32) M = fmaxf(M, p.part_ml[(slot0 + i) * p.G + r].x);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    float acc[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) acc[v] = 0.f;
    float Lsum = 0.f;
    for (int i = 0; i < n; ++i) {
        const float2 ml = p.part_ml[(slot0 + i) * p.G + r];
        const float w = exp2f(ml.x - M);
        Lsum += w * ml.y;
        const float *src = p.part_o + ((slot0 + i) * p.G + r) * D + lane * VEC;
        if (VEC == 4) {
            const float4 o = *reinterpret_cast<const float4 *>(src);
            acc[0] += w * o.x; acc[1] += w * o.y; acc[VEC - 2] += w * o.z; acc[VEC - 1] += w * o.w;
        } else {
            const float2 o = *reinterpret_cast<const float2 *>(src);
            acc[0] += w * o.x; acc[1] += w * o.y;
        }
    }
    const float inv = 1.f / Lsum;
#pragma unroll
    for (int v = 0; v < VEC; v += 2)
        *reinterpret_cast<__nv_bfloat162 *>(orow + v) = __floats2bfloat162_rn(acc[v] * inv, acc[v + 1] * inv);
    if (p.lse != nullptr && lane == 0) p.lse[row] = (M + log2f(Lsum)) * kLn2;
}

template <int D, int WARPS, int STAGES, bool HILO>
size_t smem_bytes_for() {
    // ring + 1 KB alignment slack + barriers + warp sums + prefix sums
    return static_cast<size_t>(WARPS) * STAGES * (2 * kPageSize * D * 2) + 1024 + WARPS * STAGES * 2 * 8 + 32 * 4 +
           (kMaxBatch + 1) * 4;
}

template <typename F>
cudaError_t dispatch(const AttnVariant &v, F &&f) {
#define PD_CASE(D_, W_, S_)                                                                         \
    if (v.head_dim == D_ && v.warps == W_ && v.stages == S_) {                                      \
        return v.hilo ? f(decode_attn_split_kernel<D_, W_, S_, true>, smem_bytes_for<D_, W_, S_, true>()) \
                      : f(decode_attn_split_kernel<D_, W_, S_, false>, smem_bytes_for<D_, W_, S_, false>()); \
    }
    PD_CASE(128, 8, 3)
    PD_CASE(128, 4, 6)
    PD_CASE(128, 12, 2)
    PD_CASE(128, 6, 4)
    PD_CASE(64, 8, 6)
    PD_CASE(64, 8, 3)
#undef PD_CASE
    return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t prepare_decode_attn(const AttnVariant &v, size_t *smem_bytes) {
    return dispatch(v, [&](auto kernel, size_t bytes) {
        *smem_bytes = bytes;
        return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes));
    });
}

cudaError_t launch_decode_attn(const AttnVariant &v, const CUtensorMap &tm_k, const CUtensorMap &tm_v,
                               const AttnParams &p, int num_ctas, size_t smem_bytes, cudaStream_t stream) {
    return dispatch(v, [&](auto kernel, size_t) {
        kernel<<<num_ctas, v.warps * 32, smem_bytes, stream>>>(tm_k, tm_v, p);
        return cudaGetLastError();
    });
}

cudaError_t launch_lse_merge(int head_dim, const AttnParams &p, cudaStream_t stream) {
    const int rows = p.B * p.Hq;
    const int blocks = (rows + 3) / 4;
    if (head_dim == 128) lse_merge_kernel<128><<<blocks, 128, 0, stream>>>(p);
    else lse_merge_kernel<64><<<blocks, 128, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace pd
