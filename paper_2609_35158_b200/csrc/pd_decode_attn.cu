// Split-KV decode attention over a paged bf16 KV cache, and the log-sum-exp merge.
//
// The operation is the per-sequence KV-read term of the decode cost model
// (Eq. 1: b, "extra KV-cache HBM reads"): one query token per sequence attends
// over every cached token of its KV head. The kernel is a scan of the cache at
// HBM speed; everything below serves that.
//
// Work decomposition. Units are (sequence, KV head, page) triples in that
// nesting order. Their flattened list is cut into ranges by a plan every CTA
// derives from the lengths alone: a few levels whose ranges are half of the
// remaining fair share per worker, then a tail level of short ranges. A worker
// is ONE WARP with its own ring of shared-memory stages and its own mbarriers;
// it issues its own TMA loads (lane 0) and never synchronises with another warp
// after the prologue. Its first range is its own index; further ranges are
// claimed in index order from one atomic counter, so SMs that get more
// bandwidth take more of the later, shorter ranges and all workers finish
// together. The loads of the next range are issued while the current one is
// still being consumed. Range boundaries do not depend on who claims what, so
// results are bit-reproducible.
//
// A range may cross (sequence, KV head) boundaries; each maximal piece inside
// one pair is a segment. A segment that covers the whole context writes the
// final bf16 row directly; any other segment writes an fp32 partial to slot
// (range index + pair index), unique and contiguous per pair, and the merge
// kernel combines them.
//
// Data movement. A (page, KV head) tile is 16 tokens x D bf16, contiguous in
// HBM. It is fetched by tiled TMA as D/64 boxes of 16 rows x 128 B with the
// 128-byte swizzle, so ldmatrix reads are bank-conflict free. K and V of a page
// complete on separate mbarriers.
//
// Math. Tokens are the M dimension of mma.sync.m16n8k16 and the query group
// (g <= 8 heads sharing the KV head, zero-padded to 8) is N, so no MMA row is
// wasted: S^T = K Q^T (one page = 16 tokens x 8 heads, 8 MMAs at D = 128), then
// O^T += V^T P^T (8 more). Softmax runs in fp32 in log2 units; the running max
// of a head is refreshed only when a logit exceeds it by more than 8 (a factor
// 256 of headroom), so the steady state needs one warp vote per page and no
// shuffles. P is split into a bf16 high and low part (two MMAs) so that it
// carries ~16 mantissa bits; movmatrix turns the S^T fragments into the B
// operand of the second product.
#include "pd_decode_plan.cuh"
#include "pd_kernels.cuh"
#include "pd_ptx.cuh"

namespace pd {

namespace {

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
    constexpr int MTILES = D / 16;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring0 = (raw + 1023u) & ~1023u;  // swizzled boxes need 1024-byte alignment
    uint8_t *aligned = smem_raw + (ring0 - raw);
    uint64_t *bars = reinterpret_cast<uint64_t *>(aligned + WARPS * STAGES * STAGE_BYTES);
    Plan *plan_s = reinterpret_cast<Plan *>(bars + WARPS * STAGES * 2);
    int32_t *stage_range = reinterpret_cast<int32_t *>(plan_s + 1);  // [WARPS][STAGES] range id of the page in a stage
    int32_t *stage_pid = stage_range + WARPS * STAGES;  // [WARPS][STAGES] physical page in a stage, -1 if it was clamped
    int32_t *warp_sums = stage_pid + WARPS * STAGES;
    int32_t *cum = warp_sums + 32;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned long long t_entry = p.trace != nullptr ? global_timer_ns() : 0ull;
    unsigned long long t_first = 0ull, t_last = 0ull;

    // ---- prologue (whole CTA): barriers, page prefix sums, the plan
    launch_dependents();  // the merge kernel may take its place on the SMs; it waits for this grid to finish
    if (lane == 0) {
        for (int s = 0; s < STAGES * 2; ++s) mbar_init(smem_u32(bars + (warp * STAGES * 2 + s)), 1);
        mbar_init_fence();
    }
    if (tid == 0) {
        prefetch_tensormap(&tm_k);
        prefetch_tensormap(&tm_v);
    }
    grid_dependency_wait();  // everything above is independent of the previous kernel's writes
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

    // ---- per-warp state
    const int worker = blockIdx.x * WARPS + warp;
    const uint32_t ring = ring0 + warp * STAGES * STAGE_BYTES;
    const uint32_t bar0 = smem_u32(bars + warp * STAGES * 2);
    int32_t *my_stage_range = stage_range + warp * STAGES;
    int32_t *my_stage_pid = stage_pid + warp * STAGES;
    const uint64_t policy = l2_policy_evict_first();
    const int quad_row = lane >> 2;        // B-fragment column of this lane: the query head whose Q it holds
    const int quad_col = (lane & 3) * 2;   // accumulator columns of this lane: heads quad_col and quad_col + 1
    const int G = p.G;
    // ldmatrix lane addressing inside a tile (row = token, 16-byte chunk index swizzled by row & 7)
    const int mat = lane >> 3, r8 = lane & 7;
    const uint32_t k_row_off = (((mat & 1) * 8 + r8) * 128);   // A operand: K tile, tokens x d
    const int k_sel = mat >> 1;
    const uint32_t v_row_off = (((mat >> 1) * 8 + r8) * 128);  // A operand: V tile read transposed, d x tokens
    const int v_sel = mat & 1;

    PageIdCache pt;
    pt.b = -1; pt.blk = -1; pt.val = -1; pt.nval = -1;

    // producer side: the range being issued, the cursor inside it, the claim made ahead of need
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
            // one TMA box per lane in a single warp instruction (lanes 0 .. 2*HALVES-1: K halves, then V
            // halves); issued one after another by one lane the boxes cost that lane ~170 cycles each
            const int32_t y = (pid * p.Hkv + prod.kvh) * kPageSize;
            const uint32_t dst = ring + p_stage * STAGE_BYTES;
            const uint32_t bk = bar0 + p_stage * 16, bv = bk + 8;
            if (lane == 0) {
                my_stage_range[p_stage] = p_rid;
                my_stage_pid[p_stage] = pid_ok ? pid : -1;
                mbar_arrive_expect_tx(bk, TILE_BYTES);
                mbar_arrive_expect_tx(bv, TILE_BYTES);
            }
            __syncwarp();
            if (lane < 2 * HALVES) {
                const bool is_v = lane >= HALVES;
                const int h = is_v ? lane - HALVES : lane;
                tma_load_2d(dst + (is_v ? TILE_BYTES : 0) + h * HALF_BYTES, is_v ? static_cast<const void *>(&tm_v) : &tm_k,
                            h * 64, y, is_v ? bv : bk, policy);
            }
        }
        advance(prod, cum, p.B, p.Hkv);
        --p_left;
        if (p_left <= kClaimAhead && !have_next && !p_first) {  // claim the next range before it is needed
            if (lane == 0) next_raw = atomicAdd(p.status + kSchedNext, 1);
            have_next = true;
        }
        if (++p_stage == STAGES) p_stage = 0;
        ++inflight;
        __syncwarp();
        return true;
    };

    while (inflight < STAGES && issue_next()) {}

    // consumer side
    Cursor cons;
    cons.b = 0; cons.kvh = 0; cons.page = 0; cons.np = 1;
    int c_rid = -1, c_left = 0;
    uint32_t stage = 0, parity = 0;  // ring position of the next page to consume
    bool alive = true, seg_open = false, seg_append = false;
    int seg_page0 = 0, L = 0;
    uint32_t qb[KSTEPS][2];     // Q^T as the B operand: head quad_row, d = 16 kk + quad_col (+1), and +8
    float O[MTILES][4];          // O^T: rows d = 16 j + quad_row (+8), columns heads quad_col, quad_col + 1
    float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.f, l_b = 0.f;  // per head (a = quad_col, b = quad_col + 1)

    while (inflight > 0) {
        if (c_left == 0) {  // first page of a range
            c_rid = my_stage_range[stage];
            long long start;
            range_bounds(pl, c_rid, start, c_left);
            cons = locate(cum, p.B, p.Hkv, start);
        }
        if (!seg_open) {  // first page of a segment: its queries, a fresh running state
            seg_open = true;
            seg_page0 = cons.page;
            const int L_raw = __ldg(p.ctx_lens + cons.b) + p.fused;
            L = clamp_len(L_raw, p.MP);
            seg_append = p.fused != 0 && L == L_raw && L > 0;  // never patch a row of a length that was clamped
            const __nv_bfloat16 *qrow = p.q + (static_cast<size_t>(cons.b) * p.Hq + cons.kvh * G + quad_row) * D;
#pragma unroll
            for (int kk = 0; kk < KSTEPS; ++kk) {
                if (quad_row < G) {
                    qb[kk][0] = __ldg(reinterpret_cast<const uint32_t *>(qrow + kk * 16 + quad_col));
                    qb[kk][1] = __ldg(reinterpret_cast<const uint32_t *>(qrow + kk * 16 + 8 + quad_col));
                } else {
                    qb[kk][0] = 0u;
                    qb[kk][1] = 0u;
                }
            }
#pragma unroll
            for (int j = 0; j < MTILES; ++j) { O[j][0] = 0.f; O[j][1] = 0.f; O[j][2] = 0.f; O[j][3] = 0.f; }
            m_a = -INFINITY; m_b = -INFINITY;
            l_a = 0.f; l_b = 0.f;
        }

        const uint32_t kbase = ring + stage * STAGE_BYTES;
        const uint32_t vbase = kbase + TILE_BYTES;
        const uint32_t bk = bar0 + stage * 16, bv = bk + 8;
        const int valid = L - cons.page * kPageSize;  // tokens of this page inside the context

        // fused append: the page that receives the new token is the last one of the pair. Its K and V rows
        // come from k_new / v_new: they are patched into the tile in shared memory (the pool still holds
        // whatever was in that slot) and written to the pool, which is the append itself.
        const bool appending = seg_append && cons.page == cons.np - 1;
        const int new_slot = (L - 1) & (kPageSize - 1);
        uint4 new_row = make_uint4(0u, 0u, 0u, 0u);
        constexpr int ROW_CHUNKS = D / 8;  // 16-byte chunks of one K (or V) row: lanes [0, ROW_CHUNKS) K, the next ones V
        if (appending && lane < 2 * ROW_CHUNKS) {
            const bool is_v = lane >= ROW_CHUNKS;
            const int c = is_v ? lane - ROW_CHUNKS : lane;
            const __nv_bfloat16 *src = (is_v ? p.v_new : p.k_new) + (static_cast<size_t>(cons.b) * p.Hkv + cons.kvh) * D + c * 8;
            new_row = __ldg(reinterpret_cast<const uint4 *>(src));
            const int pid = my_stage_pid[stage];
            if (pid >= 0) {
                __nv_bfloat16 *dst = (is_v ? p.v_pool_w : p.k_pool_w) +
                                     ((static_cast<size_t>(pid) * p.Hkv + cons.kvh) * kPageSize + new_slot) * D + c * 8;
                *reinterpret_cast<uint4 *>(dst) = new_row;
            }
        }
        if (!__all_sync(0xffffffffu, mbar_wait(bk, parity))) { alive = false; break; }
        if (p.trace != nullptr) {
            t_last = global_timer_ns();
            if (t_first == 0ull) t_first = t_last;
        }
        if (appending) {
            if (lane < ROW_CHUNKS) {
                const uint32_t a = kbase + (lane >> 3) * HALF_BYTES + new_slot * 128 + (((lane & 7) ^ (new_slot & 7)) << 4);
                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(new_row.x), "r"(new_row.y),
                             "r"(new_row.z), "r"(new_row.w) : "memory");
            }
            __syncwarp();
        }

        // S^T = K Q^T for the 16 tokens of the page (two accumulators shorten the dependent chain)
        float Se[4] = {0.f, 0.f, 0.f, 0.f}, So[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int kk = 0; kk < KSTEPS; ++kk) {
            uint32_t a0, a1, a2, a3;
            ldmatrix_x4(a0, a1, a2, a3,
                        kbase + (kk >> 2) * HALF_BYTES + k_row_off + ((((kk & 3) * 2 + k_sel) ^ r8) << 4));
            if (kk & 1) mma_bf16_16816(So, a0, a1, a2, a3, qb[kk][0], qb[kk][1]);
            else mma_bf16_16816(Se, a0, a1, a2, a3, qb[kk][0], qb[kk][1]);
        }
        // this lane: tokens quad_row and quad_row + 8, heads quad_col (a) and quad_col + 1 (b); log2 units
        float s0 = (Se[0] + So[0]) * p.scale_log2, s1 = (Se[1] + So[1]) * p.scale_log2;
        float s2 = (Se[2] + So[2]) * p.scale_log2, s3 = (Se[3] + So[3]) * p.scale_log2;
        if (valid < kPageSize) {  // last page of the context: mask, never multiply
            if (quad_row >= valid) { s0 = -INFINITY; s1 = -INFINITY; }
            if (quad_row + 8 >= valid) { s2 = -INFINITY; s3 = -INFINITY; }
        }
        float mx_a = fmaxf(s0, s2), mx_b = fmaxf(s1, s3);
        if (__any_sync(0xffffffffu, mx_a > m_a + kRescaleSlack || mx_b > m_b + kRescaleSlack)) {
            // some logit left the headroom of a running max: refresh both maxima over the page, rescale
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
            for (int j = 0; j < MTILES; ++j) {
                O[j][0] *= alpha_a; O[j][2] *= alpha_a;
                O[j][1] *= alpha_b; O[j][3] *= alpha_b;
            }
            m_a = new_a;
            m_b = new_b;
        }
        const float p0 = fast_exp2(s0 - m_a), p1 = fast_exp2(s1 - m_b);
        const float p2 = fast_exp2(s2 - m_a), p3 = fast_exp2(s3 - m_b);
        l_a += p0 + p2;
        l_b += p1 + p3;
        // P^T as the B operand: transpose the (token x head) fragments to (head x token)
        const __nv_bfloat162 h01 = __floats2bfloat162_rn(p0, p1), h23 = __floats2bfloat162_rn(p2, p3);
        const uint32_t pb0 = movmatrix_trans(*reinterpret_cast<const uint32_t *>(&h01));
        const uint32_t pb1 = movmatrix_trans(*reinterpret_cast<const uint32_t *>(&h23));
        uint32_t pl0 = 0u, pl1 = 0u;
        if (HILO) {
            pl0 = movmatrix_trans(pack_bf16x2(p0 - __low2float(h01), p1 - __high2float(h01)));
            pl1 = movmatrix_trans(pack_bf16x2(p2 - __low2float(h23), p3 - __high2float(h23)));
        }

        if (!__all_sync(0xffffffffu, mbar_wait(bv, parity))) { alive = false; break; }
        if (appending) {
            if (lane >= ROW_CHUNKS && lane < 2 * ROW_CHUNKS) {
                const int c = lane - ROW_CHUNKS;
                const uint32_t a = vbase + (c >> 3) * HALF_BYTES + new_slot * 128 + (((c & 7) ^ (new_slot & 7)) << 4);
                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(new_row.x), "r"(new_row.y),
                             "r"(new_row.z), "r"(new_row.w) : "memory");
            }
            __syncwarp();
        }
        if (valid < kPageSize) {
            // V rows past the context may hold NaN; 0 * NaN is NaN, so clear them first
            for (int row = valid; row < kPageSize; ++row)
                if (lane < HALVES * 8)
                    st_shared_zero16(vbase + (lane >> 3) * HALF_BYTES + row * 128 + (lane & 7) * 16);
            __syncwarp();
        }
        // O^T += V^T P^T : D rows (16 per MMA) x 8 heads, contraction over the 16 tokens
#pragma unroll
        for (int j = 0; j < MTILES; ++j) {
            uint32_t a0, a1, a2, a3;
            ldmatrix_x4_trans(a0, a1, a2, a3,
                              vbase + (j >> 2) * HALF_BYTES + v_row_off + ((((j & 3) * 2 + v_sel) ^ r8) << 4));
            mma_bf16_16816(O[j], a0, a1, a2, a3, pb0, pb1);
            if (HILO) mma_bf16_16816(O[j], a0, a1, a2, a3, pl0, pl1);
        }
        __syncwarp();  // every lane has read this stage
        if (valid < kPageSize || appending) fence_proxy_async();  // generic-proxy stores before the next TMA write
        --inflight;
        issue_next();  // refills the stage just freed (p_stage == stage here)
        if (++stage == STAGES) { stage = 0; parity ^= 1u; }

        // ---- end of segment: final row or partial
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
                const float inv_a = 1.f / l_a, inv_b = 1.f / l_b;
                __nv_bfloat16 *oa = p.out + row0 * D + quad_row, *ob = oa + D;
#pragma unroll
                for (int j = 0; j < MTILES; ++j) {
                    if (has_a) {
                        oa[16 * j] = __float2bfloat16(O[j][0] * inv_a);
                        oa[16 * j + 8] = __float2bfloat16(O[j][2] * inv_a);
                    }
                    if (has_b) {
                        ob[16 * j] = __float2bfloat16(O[j][1] * inv_b);
                        ob[16 * j + 8] = __float2bfloat16(O[j][3] * inv_b);
                    }
                }
                if (p.lse != nullptr && quad_row == 0) {
                    if (has_a) p.lse[row0] = (m_a + log2f(l_a)) * kLn2;
                    if (has_b) p.lse[row0 + 1] = (m_b + log2f(l_b)) * kLn2;
                }
            } else {
                const size_t slot = static_cast<size_t>(c_rid) + static_cast<size_t>(cons.b) * p.Hkv + cons.kvh;
                float *oa = p.part_o + (slot * G + quad_col) * D + quad_row, *ob = oa + D;
#pragma unroll
                for (int j = 0; j < MTILES; ++j) {
                    if (has_a) { oa[16 * j] = O[j][0]; oa[16 * j + 8] = O[j][2]; }
                    if (has_b) { ob[16 * j] = O[j][1]; ob[16 * j + 8] = O[j][3]; }
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

    bool last_worker = false;
    if (lane == 0) {
        if (!alive) latch_status(p.status, kDevTimeout, -1, worker);
        if (p.trace != nullptr) {
            unsigned long long *t = p.trace + static_cast<size_t>(worker) * 4;
            t[0] = t_entry; t[1] = t_first; t[2] = t_last; t[3] = global_timer_ns();
        }
        // the last worker to finish re-arms the claim counter for the next launch
        if (atomicAdd(p.status + kSchedDone, 1) == n_workers - 1) {
            p.status[kSchedNext] = 0;
            p.status[kSchedDone] = 0;
            last_worker = true;
        }
    }
    // fused append: the last worker to finish (every CTA has long read the old lengths) advances them
    if (p.fused != 0 && __shfl_sync(0xffffffffu, static_cast<int>(last_worker), 0)) {
        for (int i = lane; i < p.B; i += 32) {
            const int Lold = p.ctx_lens_w[i];
            if (Lold < 0 || Lold + 1 > p.MP * kPageSize) continue;  // latched as a bad length by the scan
            const int pid = __ldg(p.page_table + static_cast<size_t>(i) * p.MP + Lold / kPageSize);
            if (pid >= 0 && pid < p.num_pages) p.ctx_lens_w[i] = Lold + 1;  // a bad page id was latched by its reader
        }
    }
}

// Index of the range that holds unit x, from the plan the split kernel left in global memory.
__device__ __forceinline__ long long range_of_unit(const int32_t *plan, long long x) {
    const int n_levels = plan[2];
    const int32_t *rec = plan + kPlanHeaderWords;
    int l = 0;
    auto start_of = [&](int i) {
        return (static_cast<long long>(rec[4 * i + 1]) << 32) | static_cast<unsigned int>(rec[4 * i]);
    };
    while (l + 1 < n_levels && x >= start_of(l + 1)) ++l;
    return rec[4 * l + 3] + (x - start_of(l)) / rec[4 * l + 2];
}

// Each CTA merges R consecutive rows (query heads of one KV head; R divides the group size). Warp w
// works on row w % R and takes every (WARPS / R)-th partial of it, eight loads in flight, keeping a
// running (max, sum, output); the warps of a row are then combined through shared memory in warp
// order. The order of operations is fixed, so reruns are bit-identical.
template <int D, int WARPS, int R>
__device__ __forceinline__ void lse_merge_rows(const AttnParams &p) {
    constexpr int VEC = D / 32;
    constexpr int UNROLL = 8;
    constexpr int S = WARPS / R;  // warps sharing one row
    static_assert(WARPS % R == 0, "rows per CTA must divide the warp count");
    __shared__ float sm_o[WARPS][D];
    __shared__ float2 sm_ml[WARPS];
    __shared__ int32_t sm_plan[kPlanWords + 2];  // the plan, then the two prefix sums of this sequence
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int row = blockIdx.x * R + warp % R;
    const int sub = warp / R;
    const int b = (blockIdx.x * R) / p.Hq;  // all rows of the CTA belong to one sequence and one KV head
    const int h = row - b * p.Hq;
    const int G = p.G;
    const int kvh = h / G, r = h - kvh * G;
    grid_dependency_wait();  // partials, prefix sums and the plan come from the split kernel
    launch_dependents();
    // one round trip for everything the bookkeeping needs
    for (int i = threadIdx.x; i < kPlanWords + 2; i += WARPS * 32)
        sm_plan[i] = i < kPlanWords ? p.plan[i] : p.cum_pages[b + (i - kPlanWords)];
    __syncthreads();
    const int c0 = sm_plan[kPlanWords], np = sm_plan[kPlanWords + 1] - c0;
    // final rows go to the caller's device buffer, or straight to its pinned host buffer when that is given
    __nv_bfloat16 *orow = (p.out_host != nullptr ? p.out_host : p.out) + static_cast<size_t>(row) * D + lane * VEC;
    if (np == 0) {  // empty context: zero row, lse = -inf
        if (sub == 0) {
#pragma unroll
            for (int v = 0; v < VEC; ++v) orow[v] = __float2bfloat16(0.f);
            if (p.lse != nullptr && lane == 0) p.lse[row] = -INFINITY;
        }
        return;
    }
    const long long u0 = static_cast<long long>(p.Hkv) * c0 + static_cast<long long>(kvh) * np;
    const long long first = range_of_unit(sm_plan, u0), last = range_of_unit(sm_plan, u0 + np - 1);
    if (first == last) {  // written directly by the split kernel (the same for every row of the CTA)
        if (p.out_host != nullptr && sub == 0) {  // forward the row to the host buffer
            const __nv_bfloat16 *src = p.out + static_cast<size_t>(row) * D + lane * VEC;
#pragma unroll
            for (int v = 0; v < VEC; v += 2)
                *reinterpret_cast<__nv_bfloat162 *>(orow + v) = *reinterpret_cast<const __nv_bfloat162 *>(src + v);
        }
        return;
    }
    const int n = static_cast<int>(last - first) + 1;
    const size_t slot0 = static_cast<size_t>(first) + static_cast<size_t>(b) * p.Hkv + kvh;

    float m = -INFINITY, l = 0.f, acc[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) acc[v] = 0.f;
    for (int i0 = sub; i0 < n; i0 += S * UNROLL) {
        float2 ml[UNROLL];
        float o[UNROLL][VEC];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int i = i0 + u * S;
            if (i < n) {
                const size_t rec = (slot0 + i) * G + r;
                ml[u] = p.part_ml[rec];
                const float *src = p.part_o + rec * D + lane * VEC;
                if (VEC == 4) {
                    const float4 t = *reinterpret_cast<const float4 *>(src);
                    o[u][0] = t.x; o[u][1] = t.y; o[u][VEC - 2] = t.z; o[u][VEC - 1] = t.w;
                } else {
                    const float2 t = *reinterpret_cast<const float2 *>(src);
                    o[u][0] = t.x; o[u][1] = t.y;
                }
            } else {
                ml[u] = make_float2(-INFINITY, 0.f);
#pragma unroll
                for (int v = 0; v < VEC; ++v) o[u][v] = 0.f;
            }
        }
        float m_new = m;
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) m_new = fmaxf(m_new, ml[u].x);
        const float a = exp2f(m - m_new);  // m_new is finite: the first record of every batch exists
        l *= a;
#pragma unroll
        for (int v = 0; v < VEC; ++v) acc[v] *= a;
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const float w = exp2f(ml[u].x - m_new);
            l += w * ml[u].y;
#pragma unroll
            for (int v = 0; v < VEC; ++v) acc[v] += w * o[u][v];
        }
        m = m_new;
    }
#pragma unroll
    for (int v = 0; v < VEC; ++v) sm_o[warp][lane * VEC + v] = acc[v];
    if (lane == 0) sm_ml[warp] = make_float2(m, l);
    __syncthreads();
    if (sub == 0) {  // warp w < R finishes row w: its partners are warps w, w + R, w + 2R, ...
        float M = -INFINITY;
#pragma unroll
        for (int k = 0; k < S; ++k) M = fmaxf(M, sm_ml[warp + k * R].x);
        float Lsum = 0.f, out[VEC];
#pragma unroll
        for (int v = 0; v < VEC; ++v) out[v] = 0.f;
#pragma unroll
        for (int k = 0; k < S; ++k) {
            const float wt = exp2f(sm_ml[warp + k * R].x - M);  // warps without records carry m = -inf, weight 0
            Lsum += wt * sm_ml[warp + k * R].y;
#pragma unroll
            for (int v = 0; v < VEC; ++v) out[v] += wt * sm_o[warp + k * R][lane * VEC + v];
        }
        const float inv = 1.f / Lsum;
#pragma unroll
        for (int v = 0; v < VEC; v += 2)
            *reinterpret_cast<__nv_bfloat162 *>(orow + v) = __floats2bfloat162_rn(out[v] * inv, out[v + 1] * inv);
        if (p.lse != nullptr && lane == 0) p.lse[row] = (M + log2f(Lsum)) * kLn2;
    }
}

template <int D, int WARPS, int R>
__global__ void __launch_bounds__(WARPS * 32) lse_merge_kernel(const AttnParams p) {
    lse_merge_rows<D, WARPS, R>(p);
    if (p.done_flag != nullptr) {
        // completion report for a host that polls pinned memory instead of synchronising the stream: every CTA
        // makes its rows visible system-wide and takes a ticket; the last one stores the flag
        __syncthreads();
        if (threadIdx.x == 0) {
            __threadfence_system();
            if (atomicAdd(p.status + kMergeDone, 1) == static_cast<int>(gridDim.x) - 1) {
                p.status[kMergeDone] = 0;
                __threadfence_system();
                *reinterpret_cast<volatile int32_t *>(p.done_flag) = p.done_value;
            }
        }
    }
}

template <int D, int WARPS, int STAGES, bool HILO>
size_t smem_bytes_for() {
    // ring + 1 KB alignment slack + barriers + plan + stage tags + warp sums + prefix sums
    return static_cast<size_t>(WARPS) * STAGES * (2 * kPageSize * D * 2) + 1024 + WARPS * STAGES * 2 * 8 +
           sizeof(Plan) + 2 * WARPS * STAGES * 4 + 32 * 4 + (kMaxBatch + 1) * 4;
}

template <typename F>
cudaError_t dispatch(const AttnVariant &v, F &&f) {
#define PD_CASE(D_, W_, S_)                                                                         \
    if (v.head_dim == D_ && v.warps == W_ && v.stages == S_) {                                      \
        return v.hilo ? f(decode_attn_split_kernel<D_, W_, S_, true>, smem_bytes_for<D_, W_, S_, true>()) \
                      : f(decode_attn_split_kernel<D_, W_, S_, false>, smem_bytes_for<D_, W_, S_, false>()); \
    }
    PD_CASE(128, 8, 3)
    PD_CASE(64, 16, 3)  // pages of 4 KB: twice the warps keep the instruction stream from being the limit (6446 against 4966 GB/s)
    PD_CASE(64, 8, 6)   // the allocation-free entry point's shape (its fixed scratch is sized for 8 warps per CTA)
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
        return launch_pdl(kernel, dim3(num_ctas), dim3(v.warps * 32), smem_bytes, stream, p.pdl != 0, tm_k, tm_v, p);
    });
}

cudaError_t launch_lse_merge(int head_dim, const AttnParams &p, cudaStream_t stream) {
    // Few rows (low decode concurrency) mean many partials per row: all 8 warps of a CTA share one
    // row. With many rows the partial lists are short and CTA count dominates: a CTA takes several rows.
    const int rows = p.B * p.Hq;
    const bool pdl = p.pdl != 0;
    int r = p.merge_rows > 0 ? p.merge_rows : (rows <= 512 ? 1 : (rows <= 1024 ? 2 : 8));
    while (r > 1 && p.G % r != 0) r >>= 1;
#define PD_MERGE(D_, R_)                                                                                  \
    if (head_dim == D_ && r == R_)                                                                        \
        return launch_pdl(lse_merge_kernel<D_, 8, R_>, dim3(rows / R_), dim3(256), 0, stream, pdl, p);
    PD_MERGE(128, 1) PD_MERGE(128, 2) PD_MERGE(128, 4) PD_MERGE(128, 8)
    PD_MERGE(64, 1) PD_MERGE(64, 2) PD_MERGE(64, 4) PD_MERGE(64, 8)
#undef PD_MERGE
    return cudaErrorInvalidValue;
}

}  // namespace pd
