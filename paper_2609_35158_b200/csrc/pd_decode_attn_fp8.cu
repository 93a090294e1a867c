// Split-KV decode attention over FP8 (e4m3) KV pages with one scale per (page, KV head), plus the
// whole-page quantiser and the one-token FP8 append.
//
// The decode cost this library exists for is "extra KV-cache HBM reads" per concurrent sequence (Eq. 1):
// storing the cache in one byte per value halves those bytes. The paper has no such variant; the format
// is this repository's: K8 / V8 pools [num_pages][num_kv_heads][16][head_dim] of OCP E4M3 bytes and a scale
// record {k_scale, v_scale, 0, 0} (fp32) per (page, KV head); K_t = k_scale * e4m3(byte), likewise V.
//
// The kernel is the bf16 split kernel's skeleton (same plan of ranges, same warp-private TMA rings, same
// partial format, same merge kernel) with a different inner product:
//   * a tile is one 16 x head_dim byte TMA box (128-byte swizzle at head_dim 128, 64-byte at 64); the page's
//     scale record rides along as a 16-byte bulk copy on the K barrier; sixteen worker warps with three
//     stages each (six at head_dim 64) keep as many bytes in flight per SM as the bf16 kernel does;
//   * ldmatrix on the byte tile (viewed as b16) hands every lane four consecutive d of a token; two
//     cvt.rn.f16x2.e4m3x2 make them fp16 pairs, exactly, and Q is converted to fp16 once per segment with
//     the matching d order, so S^T = K8 Q^T runs on mma.sync fp16 (tokens as M, as in the bf16 kernel);
//     k_scale times sm_scale log2(e) multiplies the fp32 logits;
//   * for O^T += V^T P^T, ldmatrix.trans delivers (token 2t, token 2t+1) x (d, d+1) in one register; one
//     byte permute regroups it into the two fp16 pairs the A operand wants. P is fp16 (11 significant
//     bits, no high/low split needed). v_scale is folded into P relative to the largest scale of the segment
//     so far (O is kept in that unit and rescaled when a larger scale arrives), so the page's product
//     accumulates straight into O: no temporary accumulator, no per-element multiply.
// head_dim 64 or 128; |q| below the fp16 range (65504) is required.
#include "pd_decode_plan.cuh"
#include "pd_kernels.cuh"
#include "pd_ptx.cuh"

#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include <cstdlib>

namespace pd {

namespace {


__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t w) {
    const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162 *>(&w);
    const __half2 h = __float22half2_rn(__bfloat1622float2(b));
    return *reinterpret_cast<const uint32_t *>(&h);
}

// The 16-byte chunk of a tile row as the TMA swizzle stores it: rows of 128 B under the 128-byte swizzle (chunk
// index xor the row's low three bits), rows of 64 B under the 64-byte swizzle (xor bits 1-2 of the row); r8 is
// the row modulo 8. Either way the eight rows of an ldmatrix phase land in eight different 16-byte bank groups.
template <int D>
__device__ __forceinline__ int swizzled_chunk(int chunk, int r8) {
    return D == 128 ? (chunk ^ r8) : (chunk ^ ((r8 >> 1) & 3));
}

template <int D, int WARPS, int STAGES>
__global__ void __launch_bounds__(WARPS * 32, 1)
decode_attn_split_fp8_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                             const AttnParams p) {
    static_assert(D == 64 || D == 128, "head_dim 64 or 128");
    constexpr int THREADS = WARPS * 32;
    constexpr int TILE_BYTES = kPageSize * D;    // one TMA box: 16 rows x D bytes
    constexpr int STAGE_BYTES = 2 * TILE_BYTES;  // K tile then V tile
    constexpr int CHUNKS = D / 16;               // 16-byte chunks per row = MMAs per product

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring0 = (raw + 1023u) & ~1023u;
    uint8_t *aligned = smem_raw + (ring0 - raw);
    float4 *scale_slots = reinterpret_cast<float4 *>(aligned + WARPS * STAGES * STAGE_BYTES);  // [WARPS][STAGES]
    uint64_t *bars = reinterpret_cast<uint64_t *>(scale_slots + WARPS * STAGES);
    Plan *plan_s = reinterpret_cast<Plan *>(bars + WARPS * STAGES * 2);
    int32_t *stage_range = reinterpret_cast<int32_t *>(plan_s + 1);
    int32_t *warp_sums = stage_range + WARPS * STAGES;
    int32_t *cum = warp_sums + 32;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
#ifdef PD_ENABLE_TUNING
    // profiling build only (the kernel has no register to spare): per worker two words, the low 32 bits of
    // {entry, first data} and {last data, exit} in ns
    const unsigned long long t_entry = p.trace != nullptr ? global_timer_ns() : 0ull;
    unsigned long long t_first = 0ull, t_last = 0ull;
#endif

    launch_dependents();
    if (lane == 0) {
        for (int s = 0; s < STAGES * 2; ++s) mbar_init(smem_u32(bars + (warp * STAGES * 2 + s)), 1);
        mbar_init_fence();
    }
    if (tid == 0) {
        prefetch_tensormap(&tm_k);
        prefetch_tensormap(&tm_v);
    }
    grid_dependency_wait();
    scan_pages<THREADS>(p, cum, warp_sums);

    const int n_workers = gridDim.x * WARPS;
    if (tid == 0) make_plan(*plan_s, static_cast<long long>(p.Hkv) * cum[p.B], n_workers, p);
    __syncthreads();
    const Plan &pl = *plan_s;
    if (blockIdx.x == 0) {
        for (int i = tid; i <= p.B; i += THREADS) p.cum_pages[i] = cum[i];
        if (tid == 0) {
            p.plan[0] = static_cast<int32_t>(pl.total & 0xffffffffll);
            p.plan[1] = static_cast<int32_t>(pl.total >> 32);
            p.plan[2] = pl.n_levels;
            p.plan[3] = pl.n_ranges;
            p.plan[4] = n_workers;
        }
        if (tid <= pl.n_levels) {
            int32_t *rec = p.plan + kPlanHeaderWords + 4 * tid;
            rec[0] = static_cast<int32_t>(pl.lv[tid].start & 0xffffffffll);
            rec[1] = static_cast<int32_t>(pl.lv[tid].start >> 32);
            rec[2] = pl.lv[tid].size;
            rec[3] = pl.lv[tid].first;
        }
    }

    const int worker = blockIdx.x * WARPS + warp;
    const uint32_t ring = ring0 + warp * STAGES * STAGE_BYTES;
    const uint32_t bar0 = smem_u32(bars + warp * STAGES * 2);
    const uint32_t scale0 = smem_u32(scale_slots + warp * STAGES);
    const float4 *my_scales = scale_slots + warp * STAGES;
    int32_t *my_stage_range = stage_range + warp * STAGES;
    const uint64_t policy = l2_policy_evict_first();
    const int quad_row = lane >> 2;       // g: token row of the accumulators; head whose Q this lane holds as B operand
    const int quad_t = lane & 3;          // t
    const int quad_col = quad_t * 2;      // accumulator columns: heads quad_col and quad_col + 1
    const int G = p.G;
    const int mat = lane >> 3, r8 = lane & 7;
    const uint32_t k_row_off = (((mat & 1) * 8 + r8) * D);   // K tile: matrices 0/1 = tokens 0-7 / 8-15, 2/3 = next chunk
    const int k_sel = mat >> 1;
    const uint32_t v_row_off = (((mat >> 1) * 8 + r8) * D);  // V tile read transposed: matrices 0/1 = chunk, chunk + 1 of tokens 0-7
    const int v_sel = mat & 1;

    PageIdCache pt;
    pt.b = -1; pt.blk = -1; pt.val = -1; pt.nval = -1;

    Cursor prod;
    prod.b = 0; prod.kvh = 0; prod.page = 0; prod.np = 1;
    int p_rid = -1, p_left = 0;
    bool p_first = true, p_done = false, have_next = false;
    int next_raw = 0;
    uint32_t p_stage = 0;
    int inflight = 0;

    auto issue_next = [&]() -> bool {
        if (p_left == 0) {
            if (p_done) return false;
            int rid;
            if (p_first) {
                rid = worker;
                p_first = false;
            } else {
                if (!have_next && lane == 0) next_raw = atomicAdd(p.status + kSchedNext, 1);
                rid = n_workers + __shfl_sync(0xffffffffu, next_raw, 0);
                have_next = false;
            }
            if (rid >= pl.n_ranges) {
                p_done = true;
                return false;
            }
            long long start;
            range_bounds(pl, rid, start, p_left);
            prod = locate(cum, p.B, p.Hkv, start);
            p_rid = rid;
        }
        int pid = page_id(pt, p, prod.b, prod.page, lane);
        bool pid_ok = true;
        if (pid < 0 || pid >= p.num_pages) {
            if (lane == 0) latch_status(p.status, kDevBadPage, prod.b, pid);
            pid = 0;
            pid_ok = false;
        }
        {
            // lane 0: K box, lane 1: V box, lane 2: the scale record (16 B) - one warp instruction each kind
            const int32_t tile = pid * p.Hkv + prod.kvh;
            const uint32_t dst = ring + p_stage * STAGE_BYTES;
            const uint32_t bk = bar0 + p_stage * 16, bv = bk + 8;
            if (lane == 0) {
                my_stage_range[p_stage] = p_rid;
                mbar_arrive_expect_tx(bk, TILE_BYTES + 16);
                mbar_arrive_expect_tx(bv, TILE_BYTES);
            }
            __syncwarp();
            if (lane < 2)
                tma_load_2d(dst + lane * TILE_BYTES, lane ? static_cast<const void *>(&tm_v) : &tm_k, 0, tile * kPageSize,
                            lane ? bv : bk, policy);
            else if (lane == 2)
                bulk_load(scale0 + p_stage * 16, p.kv_scales + static_cast<size_t>(tile) * 4, 16, bk);
        }
        advance(prod, cum, p.B, p.Hkv);
        --p_left;
        if (p_left <= kClaimAhead && !have_next && !p_first) {
            if (lane == 0) next_raw = atomicAdd(p.status + kSchedNext, 1);
            have_next = true;
        }
        if (++p_stage == STAGES) p_stage = 0;
        ++inflight;
        __syncwarp();
        return true;
    };

    while (inflight < STAGES && issue_next()) {}

    Cursor cons;
    cons.b = 0; cons.kvh = 0; cons.page = 0; cons.np = 1;
    int c_rid = -1, c_left = 0;
    uint32_t stage = 0, parity = 0;
    bool alive = true, seg_open = false;
    int seg_page0 = 0, L = 0;
    // Q^T as the fp16 B operand: for chunk c, head quad_row, d = 16 c + 4 t + {0, 1} and + {2, 3}
    uint32_t qb[CHUNKS][2];
    // O^T: for chunk c, rows d = 16 c + 2 g (regs 0, 1) and 16 c + 2 g + 1 (regs 2, 3), columns heads quad_col, quad_col + 1
    float O[CHUNKS][4];
    float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.f, l_b = 0.f;
    // O is kept in units of v_ref, the largest |v_scale| the segment has met: a page's probabilities go to the
    // tensor core as p * v_scale / v_ref (fp32 product, at most p, then fp16), so its product accumulates
    // straight into O. What fp16 drops of a page whose scale is far below v_ref is below 2^-25 of v_ref per
    // code unit, i.e. nothing against the pages that set v_ref.
    float v_ref = 0.f;

    while (inflight > 0) {
        if (c_left == 0) {
            c_rid = my_stage_range[stage];
            long long start;
            range_bounds(pl, c_rid, start, c_left);
            cons = locate(cum, p.B, p.Hkv, start);
        }
        if (!seg_open) {
            seg_open = true;
            seg_page0 = cons.page;
            L = clamp_len(__ldg(p.ctx_lens + cons.b), p.MP);
            const __nv_bfloat16 *qrow = p.q + (static_cast<size_t>(cons.b) * p.Hq + cons.kvh * G + quad_row) * D;
#pragma unroll
            for (int c = 0; c < CHUNKS; ++c) {
                if (quad_row < G) {
                    const uint2 w = __ldg(reinterpret_cast<const uint2 *>(qrow + c * 16 + quad_t * 4));
                    qb[c][0] = bf16x2_to_f16x2(w.x);
                    qb[c][1] = bf16x2_to_f16x2(w.y);
                } else {
                    qb[c][0] = 0u;
                    qb[c][1] = 0u;
                }
            }
#pragma unroll
            for (int c = 0; c < CHUNKS; ++c) { O[c][0] = 0.f; O[c][1] = 0.f; O[c][2] = 0.f; O[c][3] = 0.f; }
            m_a = -INFINITY; m_b = -INFINITY;
            l_a = 0.f; l_b = 0.f;
            v_ref = 0.f;
        }

        const uint32_t kbase = ring + stage * STAGE_BYTES;
        const uint32_t vbase = kbase + TILE_BYTES;
        const uint32_t bk = bar0 + stage * 16, bv = bk + 8;
        const int valid = L - cons.page * kPageSize;

        if (!__all_sync(0xffffffffu, mbar_wait(bk, parity))) { alive = false; break; }
#ifdef PD_ENABLE_TUNING
        if (p.trace != nullptr) {
            t_last = global_timer_ns();
            if (t_first == 0ull) t_first = t_last;
        }
#endif
        const float4 sc = my_scales[stage];  // {k_scale, v_scale, -, -} of this page

        // S^T = K8 Q^T: one ldmatrix.x4 feeds two MMAs (two 16-byte chunks of d)
        float Se[4] = {0.f, 0.f, 0.f, 0.f}, So[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int kk = 0; kk < CHUNKS / 2; ++kk) {
            uint32_t r0, r1, r2, r3;  // (tokens g | g + 8) x (chunk 2 kk | 2 kk + 1), four consecutive d each
            ldmatrix_x4(r0, r1, r2, r3, kbase + k_row_off + (swizzled_chunk<D>(kk * 2 + k_sel, r8) << 4));
            mma_f16_16816(Se, e4m3x2_lo_to_f16x2(r0), e4m3x2_lo_to_f16x2(r1), e4m3x2_hi_to_f16x2(r0), e4m3x2_hi_to_f16x2(r1),
                          qb[2 * kk][0], qb[2 * kk][1]);
            mma_f16_16816(So, e4m3x2_lo_to_f16x2(r2), e4m3x2_lo_to_f16x2(r3), e4m3x2_hi_to_f16x2(r2), e4m3x2_hi_to_f16x2(r3),
                          qb[2 * kk + 1][0], qb[2 * kk + 1][1]);
        }
        const float ks = p.scale_log2 * sc.x;
        float s0 = (Se[0] + So[0]) * ks, s1 = (Se[1] + So[1]) * ks;
        float s2 = (Se[2] + So[2]) * ks, s3 = (Se[3] + So[3]) * ks;
        if (valid < kPageSize) {
            if (quad_row >= valid) { s0 = -INFINITY; s1 = -INFINITY; }
            if (quad_row + 8 >= valid) { s2 = -INFINITY; s3 = -INFINITY; }
        }
        float mx_a = fmaxf(s0, s2), mx_b = fmaxf(s1, s3);
        if (__any_sync(0xffffffffu, mx_a > m_a + kRescaleSlack || mx_b > m_b + kRescaleSlack)) {
#pragma unroll
            for (int o = 4; o < 32; o <<= 1) {
                mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, o));
                mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, o));
            }
            const float new_a = fmaxf(m_a, mx_a), new_b = fmaxf(m_b, mx_b);
            const float alpha_a = fast_exp2(m_a - new_a), alpha_b = fast_exp2(m_b - new_b);
            l_a *= alpha_a;
            l_b *= alpha_b;
#pragma unroll
            for (int c = 0; c < CHUNKS; ++c) {
                O[c][0] *= alpha_a; O[c][2] *= alpha_a;
                O[c][1] *= alpha_b; O[c][3] *= alpha_b;
            }
            m_a = new_a;
            m_b = new_b;
        }
        const float p0 = fast_exp2(s0 - m_a), p1 = fast_exp2(s1 - m_b);
        const float p2 = fast_exp2(s2 - m_a), p3 = fast_exp2(s3 - m_b);
        l_a += p0 + p2;
        l_b += p1 + p3;
        if (fabsf(sc.y) > v_ref) {  // the page's scale, so the whole warp branches together; rare after the first pages
            const float r = v_ref / fabsf(sc.y);  // 0 at the first page, where O is 0 anyway
#pragma unroll
            for (int c = 0; c < CHUNKS; ++c) { O[c][0] *= r; O[c][1] *= r; O[c][2] *= r; O[c][3] *= r; }
            v_ref = fabsf(sc.y);
        }
        const float vr = v_ref > 0.f ? sc.y / v_ref : 0.f;
        // P^T as the fp16 B operand: (token x head) fragments transposed to (head x token)
        const __half2 h01 = __floats2half2_rn(p0 * vr, p1 * vr), h23 = __floats2half2_rn(p2 * vr, p3 * vr);
        const uint32_t pb0 = movmatrix_trans(*reinterpret_cast<const uint32_t *>(&h01));
        const uint32_t pb1 = movmatrix_trans(*reinterpret_cast<const uint32_t *>(&h23));

        if (!__all_sync(0xffffffffu, mbar_wait(bv, parity))) { alive = false; break; }
        if (valid < kPageSize) {
            // V rows past the context may hold NaN codes; 0 * NaN is NaN, so clear them first
            for (int row = valid; row < kPageSize; ++row)
                if (lane < D / 16) st_shared_zero16(vbase + row * D + lane * 16);
            __syncwarp();
        }
        // O^T += V8^T (P v_scale / v_ref)^T, two chunks of d per ldmatrix
#pragma unroll
        for (int j = 0; j < CHUNKS / 2; ++j) {
            uint32_t r0, r1, r2, r3;  // (chunk 2 j | 2 j + 1) x (tokens 2t, 2t+1 | 2t+8, 2t+9), d = 2 g, 2 g + 1 of the chunk
            ldmatrix_x4_trans(r0, r1, r2, r3, vbase + v_row_off + (swizzled_chunk<D>(j * 2 + v_sel, r8) << 4));
            // bytes (tok a: d, d+1 | tok a+1: d, d+1) -> (d: tok a, a+1 | d+1: tok a, a+1)
            r0 = __byte_perm(r0, 0u, 0x3120);
            r1 = __byte_perm(r1, 0u, 0x3120);
            r2 = __byte_perm(r2, 0u, 0x3120);
            r3 = __byte_perm(r3, 0u, 0x3120);
            mma_f16_16816(O[2 * j], e4m3x2_lo_to_f16x2(r0), e4m3x2_hi_to_f16x2(r0), e4m3x2_lo_to_f16x2(r2), e4m3x2_hi_to_f16x2(r2),
                          pb0, pb1);
            mma_f16_16816(O[2 * j + 1], e4m3x2_lo_to_f16x2(r1), e4m3x2_hi_to_f16x2(r1), e4m3x2_lo_to_f16x2(r3), e4m3x2_hi_to_f16x2(r3),
                          pb0, pb1);
        }
        __syncwarp();
        if (valid < kPageSize) fence_proxy_async();  // generic-proxy stores before the next TMA write
        --inflight;
        issue_next();
        if (++stage == STAGES) { stage = 0; parity ^= 1u; }

        --c_left;
        const bool pair_end = cons.page + 1 == cons.np;
        if (c_left == 0 || pair_end) {
#pragma unroll
            for (int o = 4; o < 32; o <<= 1) {
                l_a += __shfl_xor_sync(0xffffffffu, l_a, o);
                l_b += __shfl_xor_sync(0xffffffffu, l_b, o);
            }
            const size_t row0 = static_cast<size_t>(cons.b) * p.Hq + cons.kvh * G + quad_col;
            const bool has_a = quad_col < G, has_b = quad_col + 1 < G;
            if (seg_page0 == 0 && pair_end) {
                const float inv_a = v_ref / l_a, inv_b = v_ref / l_b;
                __nv_bfloat16 *oa = p.out + row0 * D + 2 * quad_row, *ob = oa + D;
#pragma unroll
                for (int c = 0; c < CHUNKS; ++c) {
                    if (has_a)
                        *reinterpret_cast<__nv_bfloat162 *>(oa + 16 * c) = __floats2bfloat162_rn(O[c][0] * inv_a, O[c][2] * inv_a);
                    if (has_b)
                        *reinterpret_cast<__nv_bfloat162 *>(ob + 16 * c) = __floats2bfloat162_rn(O[c][1] * inv_b, O[c][3] * inv_b);
                }
                if (p.lse != nullptr && quad_row == 0) {
                    if (has_a) p.lse[row0] = (m_a + log2f(l_a)) * kLn2;
                    if (has_b) p.lse[row0 + 1] = (m_b + log2f(l_b)) * kLn2;
                }
            } else {
                const size_t slot = static_cast<size_t>(c_rid) + static_cast<size_t>(cons.b) * p.Hkv + cons.kvh;
                float *oa = p.part_o + (slot * G + quad_col) * D + 2 * quad_row, *ob = oa + D;
#pragma unroll
                for (int c = 0; c < CHUNKS; ++c) {
                    if (has_a) *reinterpret_cast<float2 *>(oa + 16 * c) = make_float2(O[c][0] * v_ref, O[c][2] * v_ref);
                    if (has_b) *reinterpret_cast<float2 *>(ob + 16 * c) = make_float2(O[c][1] * v_ref, O[c][3] * v_ref);
                }
                if (quad_row == 0) {
                    if (has_a) p.part_ml[slot * G + quad_col] = make_float2(m_a, l_a);
                    if (has_b) p.part_ml[slot * G + quad_col + 1] = make_float2(m_b, l_b);
                }
            }
            seg_open = false;
        }
        advance(cons, cum, p.B, p.Hkv);
    }

    if (lane == 0) {
        if (!alive) latch_status(p.status, kDevTimeout, -1, worker);
#ifdef PD_ENABLE_TUNING
        if (p.trace != nullptr) {  // the buffer holds four words per worker of the 8-warp bf16 kernel: two per worker here
            const unsigned long long t_exit = global_timer_ns();
            p.trace[2 * worker] = (t_entry & 0xffffffffull) | (t_first << 32);
            p.trace[2 * worker + 1] = (t_last & 0xffffffffull) | (t_exit << 32);
        }
#endif
        if (atomicAdd(p.status + kSchedDone, 1) == n_workers - 1) {  // the last worker re-arms the claim counter
            p.status[kSchedNext] = 0;
            p.status[kSchedDone] = 0;
        }
    }
}

template <int D, int WARPS, int STAGES>
constexpr size_t fp8_smem_bytes() {
    return static_cast<size_t>(WARPS) * STAGES * (2 * kPageSize * D) + 1024 + WARPS * STAGES * 16 + WARPS * STAGES * 2 * 8 +
           sizeof(Plan) + WARPS * STAGES * 4 + 32 * 4 + (kMaxBatch + 1) * 4;
}


// ---- whole-page quantiser: one CTA per (page, KV head), K then V
__device__ __forceinline__ float block_amax(float v, float *red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = red[0];
    for (int w = 1; w < static_cast<int>(blockDim.x >> 5); ++w) r = fmaxf(r, red[w]);
    __syncthreads();
    return r;
}

__device__ __forceinline__ uint8_t to_e4m3(float x, float scale) {
    // IEEE division (the build uses fast-math, so spell it out), then round to nearest even with saturation
    return static_cast<uint8_t>(__nv_cvt_float_to_fp8(__fdiv_rn(x, scale), __NV_SATFINITE, __NV_E4M3));
}

__global__ void __launch_bounds__(256) kv_quantize_pages_kernel(const QuantizeParams p) {
    __shared__ float red[8];
    grid_dependency_wait();
    launch_dependents();
    const int64_t tile = blockIdx.x;  // page * Hkv + kvh
    const int page = static_cast<int>(tile / p.Hkv);
    const int n = min(max(p.tokens_in_page[page], 0), kPageSize);
    const size_t base = static_cast<size_t>(tile) * kPageSize * p.D;
    const int count = n * p.D, total = kPageSize * p.D;
    for (int which = 0; which < 2; ++which) {
        const __nv_bfloat16 *src = (which ? p.v_pages : p.k_pages) + base;
        uint8_t *dst = (which ? p.v8 : p.k8) + base;
        float a = 0.f;
        for (int i = threadIdx.x; i < count; i += blockDim.x) {
            const float v = fabsf(__bfloat162float(src[i]));
            if (v > a) a = v;  // NaN never wins
        }
        const float amax = block_amax(a, red);
        const float scale = amax > 0.f ? __fdiv_rn(amax, 448.f) : 1.f;
        if (threadIdx.x == 0) p.scales[tile * 4 + which] = scale;
        for (int i = threadIdx.x; i < total; i += blockDim.x)
            dst[i] = i < count ? to_e4m3(__bfloat162float(src[i]), scale) : static_cast<uint8_t>(0);
    }
    if (threadIdx.x == 0) {
        p.scales[tile * 4 + 2] = 0.f;
        p.scales[tile * 4 + 3] = 0.f;
    }
}

// ---- one-token append into FP8 pages: CTA = sequence, warp = (KV head, K or V) pairs in turn
__global__ void __launch_bounds__(256) kv_append_fp8_kernel(const AppendFp8Params p) {
    const int b = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    grid_dependency_wait();
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
        if (threadIdx.x == 0 &&
            atomicCAS(p.status, kDevOk, pos < 0 || logical >= p.MP ? kDevBadLength : kDevBadPage) == kDevOk) {
            p.status[1] = b;
            p.status[2] = (pos < 0 || logical >= p.MP) ? pos : page;
        }
        return;
    }
    for (int item = warp; item < 2 * p.Hkv; item += static_cast<int>(blockDim.x >> 5)) {
        const int kvh = item >> 1, which = item & 1;
        const __nv_bfloat16 *src = (which ? p.v_new : p.k_new) + (static_cast<size_t>(b) * p.Hkv + kvh) * p.D;
        float *sc = p.scales + (static_cast<size_t>(page) * p.Hkv + kvh) * 4 + which;
        float scale;
        if (slot == 0) {  // the token opens the page: it sets the scale, with a factor two of headroom
            float a = 0.f;
            for (int i = lane; i < p.D; i += 32) {
                const float v = fabsf(__bfloat162float(src[i]));
                if (v > a) a = v;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
            scale = a > 0.f ? __fdiv_rn(a * 2.f, 448.f) : 1.f;
            if (lane == 0) *sc = scale;
        } else {
            scale = *sc;
        }
        uint8_t *dst = (which ? p.v8 : p.k8) + ((static_cast<size_t>(page) * p.Hkv + kvh) * kPageSize + slot) * p.D;
        for (int i = lane; i < p.D; i += 32) dst[i] = to_e4m3(__bfloat162float(src[i]), scale);
    }
    if (p.advance && threadIdx.x == 0) p.ctx_lens[b] = pos + 1;
}

}  // namespace

namespace {
// Worker warps per CTA x stages per warp: the bytes in flight per SM stay at 192 KB. The conversions make a
// page cost ~380 instructions in half the time a bf16 page has, and with two warps per scheduler the
// dependent chains (convert, MMA, softmax) left the issue slots idle: measured 4.4 TB/s with 8 warps x 6
// stages, 5.5 with 12 x 4, 6.3 with 16 x 3 (128 registers, no spills), which is the shape that is built.
constexpr int kFp8Warps = 16, kFp8Stages = 3;
// head_dim 64: tiles of 1 KB and 96 registers per thread, so more warps (the kernel is bound by its instruction
// stream there) and more stages per warp
// (measured on a configs[1]-shaped batch at d = 64: 16 x 6 4066 GB/s, 20 x 5 4425, 24 x 4 4366 with spills, 12 x 8 3413)
constexpr int kFp8Warps64 = 20, kFp8Stages64 = 5;
template <typename F>
cudaError_t with_fp8_kernel(int head_dim, F &&f) {
    if (head_dim == 64)
        return f(decode_attn_split_fp8_kernel<64, kFp8Warps64, kFp8Stages64>, fp8_smem_bytes<64, kFp8Warps64, kFp8Stages64>(), kFp8Warps64);
    return f(decode_attn_split_fp8_kernel<128, kFp8Warps, kFp8Stages>, fp8_smem_bytes<128, kFp8Warps, kFp8Stages>(), kFp8Warps);
}
}  // namespace

cudaError_t prepare_decode_attn_fp8(int head_dim) {
    auto set = [](auto *k, size_t bytes, int) {
        return cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes));
    };
    return with_fp8_kernel(head_dim, set);
}

cudaError_t launch_decode_attn_fp8(int head_dim, const CUtensorMap &tm_k, const CUtensorMap &tm_v, const AttnParams &p,
                                   int num_ctas, cudaStream_t stream) {
    auto go = [&](auto *k, size_t bytes, int warps) {
        return launch_pdl(k, dim3(num_ctas), dim3(warps * 32), bytes, stream, p.pdl != 0, tm_k, tm_v, p);
    };
    return with_fp8_kernel(head_dim, go);
}

cudaError_t launch_kv_quantize_pages(const QuantizeParams &p, cudaStream_t stream) {
    if (p.num_pages == 0) return cudaSuccess;
    return launch_pdl(kv_quantize_pages_kernel, dim3(static_cast<unsigned>(p.num_pages * p.Hkv)), dim3(256), 0, stream,
                      p.pdl != 0, p);
}

cudaError_t launch_kv_append_fp8(const AppendFp8Params &p, cudaStream_t stream) {
    if (p.B == 0) return cudaSuccess;
    return launch_pdl(kv_append_fp8_kernel, dim3(p.B), dim3(256), 0, stream, p.pdl != 0, p);
}

}  // namespace pd
