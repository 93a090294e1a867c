// Append-prefill attention over the paged KV cache for head_dim 64, the multi-token KV append, and the launch
// dispatch of both prefill kernels (head_dim 128 has its own kernel, pd_prefill_attn_d128.cu).
//
// Every turn of a multi-turn rollout starts by prefilling the new tokens of the
// turn (observation plus template, dL per trajectory in the prefill terms of
// Eq. 1 and Eq. 3) on top of the cached context (Sec. 2.1). With prefix caching
// only those dL tokens are computed, but each attends causally over the whole
// cached prefix and the new tokens up to itself. Unlike decode this is a dense
// contraction: 128 query rows share every K/V tile, so it runs on the
// fifth-generation tensor cores.
//
// One CTA (128 softmax threads + four service warps) owns 128 rows = 128/g consecutive new tokens x the g
// query heads of one KV head, row = head * (128/g) + token. It walks the context
// in blocks of 64 tokens (4 pages):
//   TMA      pages -> shared memory, [token][128 B] with the 128-byte
//            swizzle: K is a K-major operand, V an MN-major one, no transposes;
//            two stages of K+V; pages past the context are zero-filled
//   tcgen05  S = Q K^T into tensor memory (4 MMAs of 128x64x16, one thread)
//   threads  one thread per row: load its 64 logits from tensor memory, mask,
//            running max with a slack of 8 log2 units, exp2, row sum, P as a high and a low bf16
//            part back into tensor memory (a 64-element output row does not average the 2^-9
//            rounding of a single bf16 P away when a handful of tokens carry the row);
//            a rare correction pass rescales O
//   tcgen05  O += P V (P from tensor memory, 4 + 4 MMAs of 128x64x16 for the two parts of P)
// Four service warps issue the S MMAs, the O MMAs, the TMA loads of K and those
// of V (one box per lane), so the row threads never run issue code or meet at a
// CTA barrier: they hand over through mbarriers (logits read, probabilities written). The S MMA of block j+1 is
// issued as soon as every row holds block j's logits in registers, and two CTAs share each SM (tensor-memory
// columns 256 each), so one CTA's softmax overlaps the other's MMAs. All waits are
// bounded; a wait that runs out latches PD_ERR_TIMEOUT and the CTA unwinds and
// frees its tensor memory. (The kernel is a template over head_dim; only 64 is instantiated.)
#include "pd_kernels.cuh"
#include "pd_ptx.cuh"
#include "pd_tcgen05.cuh"

namespace pd {

namespace {

constexpr float kLn2f = 0.6931471805599453f;
constexpr float kSlack = 8.f;                 // log2 units a logit may exceed the running max before a rescale
constexpr int kRows = 128;                    // query rows per CTA (MMA M), one softmax thread each
constexpr int kThreads = kRows + 128;         // plus four service warps: S MMAs, O MMAs, K loads, V loads
constexpr int kBlock = 64;                    // context tokens per step (MMA N of S, K of O)
constexpr int kPagesPerBlock = kBlock / kPageSize;
constexpr int kQHalfBytes = kRows * 128;      // one 64-column half of the 128-row Q tile: 16 KB
constexpr int kHalfBytes = kBlock * 128;      // one 64-column half of a K or V tile of kBlock tokens
constexpr int kStages = 2;                    // K ring and V ring have two tiles each
static_assert(kStages == 2, "ring slots and logit buffers share the index j % 2 and its barriers");
// Two CTAs share an SM (96 KB of shared memory and 256 tensor-memory columns each): while one runs its
// softmax on the CUDA cores the other's MMAs keep the tensor cores busy.
constexpr int kTmemCols = 256;
// Tensor-memory columns: two logit buffers of kBlock columns (block j uses buffer j % 2; its probabilities
// overwrite the first kBlock / 2 columns of the same buffer once the logits are in registers), then the output.
constexpr int kColS = 0, kColO = 128;
// head_dim 64 only: the output takes 64 columns, which leaves room for the low halves of the probabilities
// (two buffers of kBlock / 2 columns). There P = P_hi + P_lo (two bf16, ~16 significant bits) and the O product
// is issued twice, as in the decode kernel: a 64-element output row does not average the 2^-9 rounding of a
// single bf16 P away when a handful of tokens carry the row.
constexpr int kColPlo = 192;

__device__ __forceinline__ void latch(int32_t *status, int code, int seq, int detail) {
    if (atomicCAS(status, kDevOk, code) == kDevOk) {
        status[1] = seq;
        status[2] = detail;
    }
}

template <int kD>
__global__ void __launch_bounds__(kThreads, 2)
prefill_attn_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                    const PrefillParams p) {
    constexpr int kHalves = kD / 64;               // 64-column (128-byte) halves of a head row
    constexpr int kQBytes = kHalves * kQHalfBytes;
    constexpr int kTileBytes = kHalves * kHalfBytes;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t tmem_slot;
    const int tid = threadIdx.x, warp = tid >> 5;
    const int kvh = blockIdx.y;
    const int G = p.G, TOK = kRows / G;

    grid_dependency_wait();
    launch_dependents();
    const int b = p.order != nullptr ? p.order[blockIdx.z] : static_cast<int>(blockIdx.z);  // heaviest sequences first
    const int q0 = p.q_indptr[b], q_len = p.q_indptr[b + 1] - q0;
    // tiles are scheduled in index order: start a sequence's last tiles (the longest contexts) first
    const int tile_start = static_cast<int>(p.reverse_tiles ? gridDim.x - 1 - blockIdx.x : blockIdx.x) * TOK;
    if (tile_start >= q_len) return;  // before any allocation
    const int L = min(max(p.ctx_lens[b], 0), p.MP * kPageSize);
    if (L < q_len) {  // the cache must already hold the new tokens
        if (tid == 0) latch(p.status, kDevBadLength, b, L);
        return;
    }
    const int n_tok = min(TOK, q_len - tile_start);
    const int pos0 = L - q_len + tile_start;        // absolute position of the tile's first token
    const int nb = (pos0 + n_tok - 1) / kBlock + 1;  // context blocks this tile can see
    const int n_pages = (L + kPageSize - 1) / kPageSize;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *aligned = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t q_s = base;
    const uint32_t k_ring = base + kQBytes, v_ring = k_ring + kStages * kTileBytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(aligned + kQBytes + 2 * kStages * kTileBytes);
    const uint32_t bar_k = smem_u32(bars), bar_v = smem_u32(bars + kStages);
    // [2] each: S_j is in logit buffer j % 2 and K tile j % 2 is free again (commit after the S MMA);
    // O += P_j V_j has completed and V tile j % 2 and logit buffer j % 2 are free again (commit after the O MMA)
    const uint32_t bar_s = smem_u32(bars + 2 * kStages);
    const uint32_t bar_pv = smem_u32(bars + 2 * kStages + 2);
    // [2]: every softmax warp wrote its rows of P_j (barrier j % 2). One barrier per parity: a softmax warp may
    // run a whole block ahead of another, and its arrival for block j + 1 must not count towards block j.
    const uint32_t bar_p_full = smem_u32(bars + 2 * kStages + 4);

    // ---- set-up: barriers, tensor memory, the Q tile
    if (tid == 0) {
        for (int i = 0; i < 2 * kStages + 4; ++i) mbar_init(smem_u32(bars + i), 1);
        mbar_init(bar_p_full, kRows / 32);  // one arrival per softmax warp
        mbar_init(bar_p_full + 8, kRows / 32);
        mbar_init_fence();
        prefetch_tensormap(&tm_k);
        prefetch_tensormap(&tm_v);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_slot), kTmemCols);
        tmem_relinquish_alloc_permit();
    }
    const int head = (tid & (kRows - 1)) / TOK, tok = (tid & (kRows - 1)) - head * TOK;
    const bool row_valid = tok < n_tok;
    const int my_pos = pos0 + (row_valid ? tok : n_tok - 1);  // padding rows mirror the last token
    if (tid < kRows) {
        const uint4 *src = reinterpret_cast<const uint4 *>(
            p.q + (static_cast<size_t>(q0 + tile_start + tok) * p.Hq + kvh * G + head) * kD);
#pragma unroll
        for (int c = 0; c < kD / 8; ++c) {
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (row_valid) v = __ldg(src + c);
            const uint32_t a = q_s + (c >> 3) * kQHalfBytes + sw128_offset(tid, c & 7);
            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
        }
    }
    fence_proxy_async();  // the Q tile was written with ordinary stores; the tensor core reads it through the async proxy
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tm = tmem_slot;
    bool ok = true;

    if (warp == kRows / 32) {
        // ================= S-MMA warp: lane 0 issues S_j = Q K_j^T into logit buffer j % 2 =================
        // Issuing a tcgen05.mma costs the issuing thread ~70 cycles; with the S and the O products issued by
        // one thread that thread was the bottleneck of the whole CTA, so each product has its own warp. The
        // only ordering the hardware would not give across two issuing threads is "O MMA of block j-2 before
        // the S MMA of block j" (same logit buffer), hence the wait on bar_pv.
        if ((tid & 31) == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(kRows, kBlock, false);
            for (int j = 0; j < nb && ok; ++j) {
                if (j >= 2) ok = mbar_wait(bar_pv + (j & 1) * 8, ((j - 2) >> 1) & 1);
                ok = ok && mbar_wait(bar_k + (j % kStages) * 8, (j / kStages) & 1);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t kst = k_ring + (j % kStages) * kTileBytes;
#pragma unroll
                for (int h = 0; h < kHalves; ++h)
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        umma_ss(tm + kColS + (j & 1) * kBlock, umma_smem_desc(q_s + h * kQHalfBytes + ks * 32, 16, 1024),
                                umma_smem_desc(kst + h * kHalfBytes + ks * 32, 16, 1024), idesc, (h | ks) != 0);
                umma_commit(bar_s + (j & 1) * 8);
            }
            if (!ok) latch(p.status, kDevTimeout, b, blockIdx.x);
        }
    } else if (warp == kRows / 32 + 1) {
        // ================= O-MMA warp: lane 0 issues O += P_j V_j =================
        if ((tid & 31) == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(kRows, kD, true);
            for (int j = 0; j < nb && ok; ++j) {
                ok = mbar_wait(bar_p_full + (j & 1) * 8, (j >> 1) & 1) && mbar_wait(bar_v + (j % kStages) * 8, (j / kStages) & 1);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t vst = v_ring + (j % kStages) * kTileBytes;
#pragma unroll
                for (int ks = 0; ks < kBlock / 16; ++ks)  // P from the first columns of logit buffer j % 2
                    umma_ts(tm + kColO, tm + kColS + (j & 1) * kBlock + ks * 8,
                            umma_smem_desc(vst + ks * 2048, kHalfBytes, 1024), idesc, (j | ks) != 0);
                if constexpr (kD == 64) {  // the low halves of P
#pragma unroll
                    for (int ks = 0; ks < kBlock / 16; ++ks)
                        umma_ts(tm + kColO, tm + kColPlo + (j & 1) * (kBlock / 2) + ks * 8,
                                umma_smem_desc(vst + ks * 2048, kHalfBytes, 1024), idesc, true);
                }
                umma_commit(bar_pv + (j & 1) * 8);
            }
            if (!ok) latch(p.status, kDevTimeout, b, blockIdx.x);
        }
    } else if (warp >= kRows / 32 + 2) {
        // ================= two TMA warps (one streams K, the other V): one box per lane =================
        // A tile of 64 tokens is 4 pages x (D / 64) halves = 8 (or 4) boxes of 2 KB. Issued one after another by a single
        // thread they cost ~170 cycles each; here lane l issues box l of the tile in one warp instruction.
        // Page ids are fetched 32 at a time (one per lane), a group ahead of need.
        const int lane = tid & 31;
        const uint64_t policy = l2_policy_evict_first();
        const int32_t oob_row = p.num_pages * p.Hkv * kPageSize;  // a TMA box that starts here is all zero fill
        const int32_t *pt_row = p.page_table + static_cast<size_t>(b) * p.MP;
        struct IdCache { int grp, val, nval; };
        auto load_group = [&](int grp) {
            const int idx = grp * 32 + lane;
            return (idx < n_pages) ? __ldg(pt_row + idx) : -1;
        };
        auto issue_tile_loads = [&](int j, const CUtensorMap *map, uint32_t ring, uint32_t bar0, IdCache &c) {
            const uint32_t st = ring + (j % kStages) * kTileBytes;
            const uint32_t bar = bar0 + (j % kStages) * 8;
            const int grp = (j * kPagesPerBlock) >> 5;  // the 4 pages of a block never straddle a group of 32
            if (grp != c.grp) {
                c.val = (grp == c.grp + 1) ? c.nval : load_group(grp);
                c.grp = grp;
                c.nval = load_group(grp + 1);
            }
            const int pg = (lane / kHalves) & (kPagesPerBlock - 1), h = lane % kHalves;
            const int lp = j * kPagesPerBlock + pg;
            int pid = __shfl_sync(0xffffffffu, c.val, lp & 31);
            int32_t y = oob_row;
            if (lp < n_pages) {
                if (pid < 0 || pid >= p.num_pages) {
                    if (lane < kHalves * kPagesPerBlock && h == 0) latch(p.status, kDevBadPage, b, pid);
                    pid = 0;
                }
                y = (pid * p.Hkv + kvh) * kPageSize;
            }
            if (lane == 0) mbar_arrive_expect_tx(bar, kTileBytes);
            __syncwarp();
            if (lane < kHalves * kPagesPerBlock)
                tma_load_2d(st + h * kHalfBytes + pg * (kPageSize * 128), map, h * 64, y, bar, policy);
        };
        // K and V have separate warps so that neither stream waits for the other's ring slot: a K tile is
        // reloaded as soon as the S MMA that read it has completed, a V tile as soon as its O MMA has. The
        // next phase of a slot's barrier cannot complete before the slot has been reloaded.
        const bool is_k = warp == kRows / 32 + 2;
        const CUtensorMap *map = is_k ? &tm_k : &tm_v;
        const uint32_t ring = is_k ? k_ring : v_ring, bar_full = is_k ? bar_k : bar_v, bar_free = is_k ? bar_s : bar_pv;
        IdCache cache{-2, -1, -1};
        for (int j = 0; j < min(nb, kStages); ++j) issue_tile_loads(j, map, ring, bar_full, cache);
        for (int j = 0; j + kStages < nb && ok; ++j) {
            ok = __all_sync(0xffffffffu, mbar_wait(bar_free + (j % kStages) * 8, (j / kStages) & 1));
            if (!ok) break;
            issue_tile_loads(j + kStages, map, ring, bar_full, cache);
        }
        if (!ok && lane == 0) latch(p.status, kDevTimeout, b, blockIdx.x);
    } else {
        // ================= softmax warps: one thread per query row =================
        const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
        float m_run = -INFINITY, l_run = 0.f;
        const bool tracing = p.trace != nullptr;
        long long ph[6] = {0, 0, 0, 0, 0, 0};  // cycles: wait S, load S, math, wait O, store P, total
        const long long t_begin = tracing ? clock64() : 0;
        for (int j = 0; j < nb && ok; ++j) {
            long long tc = tracing ? clock64() : 0;
            auto lap = [&](int i) {
                if (tracing) {
                    const long long now = clock64();
                    ph[i] += now - tc;
                    tc = now;
                }
            };
            // ---- logits of block j: tensor memory -> registers
            const uint32_t buf = tm + lane_base + kColS + (j & 1) * kBlock;
            ok = mbar_wait(bar_s + (j & 1) * 8, (j >> 1) & 1);
            lap(0);
            tc_fence_after_sync();
            uint32_t s[kBlock];
#pragma unroll
            for (int c = 0; c < kBlock / 32; ++c) tmem_ld32(buf + c * 32, *reinterpret_cast<uint32_t(*)[32]>(s + c * 32));
            tmem_wait_ld();
            lap(1);
            if (!ok) break;

            // ---- softmax of this thread's row. Logits stay raw; sm_scale * log2(e) > 0 is folded into the
            // exponent's FMA, so the row maximum can be taken on the raw values.
            const int t0 = j * kBlock;
            float mx = -INFINITY;
            if (t0 + kBlock - 1 > my_pos) {  // the block reaches past this row's position: mask by select
#pragma unroll
                for (int c = 0; c < kBlock; ++c) {
                    if (t0 + c > my_pos) s[c] = 0xff800000u;  // -inf
                    mx = fmaxf(mx, __uint_as_float(s[c]));
                }
            } else {  // four independent chains instead of one 64-long dependency
                float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
                for (int c = 0; c < kBlock; c += 4) {
                    m0 = fmaxf(m0, __uint_as_float(s[c]));
                    m1 = fmaxf(m1, __uint_as_float(s[c + 1]));
                    m2 = fmaxf(m2, __uint_as_float(s[c + 2]));
                    m3 = fmaxf(m3, __uint_as_float(s[c + 3]));
                }
                mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
            }
            mx *= p.scale_log2;
            float alpha = 1.f;
            if (mx > m_run + kSlack) {
                const float m_new = fmaxf(m_run, mx);
                alpha = fast_exp2(m_run - m_new);
                m_run = m_new;
            }
            // packed fp32x2 arithmetic: one FMA and one add per pair of logits
            const float2 sc2 = make_float2(p.scale_log2, p.scale_log2), nm2 = make_float2(-m_run, -m_run);
            float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
            uint32_t pk[kBlock / 2];
            if constexpr (kD == 64) {
                // P_hi over the first columns of the logit buffer (all logits are in registers), P_lo to its own
                // buffer, sixteen logits at a time
                const uint32_t plo = tm + lane_base + kColPlo + (j & 1) * (kBlock / 2);
#pragma unroll
                for (int c0 = 0; c0 < kBlock; c0 += 16) {
                    uint32_t hi[8], lo[8];
#pragma unroll
                    for (int c = c0; c < c0 + 16; c += 4) {
                        const float2 x0 = __ffma2_rn(make_float2(__uint_as_float(s[c]), __uint_as_float(s[c + 1])), sc2, nm2);
                        const float2 x1 = __ffma2_rn(make_float2(__uint_as_float(s[c + 2]), __uint_as_float(s[c + 3])), sc2, nm2);
                        const float2 e0 = make_float2(fast_exp2(x0.x), fast_exp2(x0.y));
                        const float2 e1 = make_float2(fast_exp2(x1.x), fast_exp2(x1.y));
                        acc0 = __fadd2_rn(acc0, e0);
                        acc1 = __fadd2_rn(acc1, e1);
                        const __nv_bfloat162 h0 = __floats2bfloat162_rn(e0.x, e0.y), h1 = __floats2bfloat162_rn(e1.x, e1.y);
                        const int i = (c - c0) >> 1;
                        hi[i] = *reinterpret_cast<const uint32_t *>(&h0);
                        hi[i + 1] = *reinterpret_cast<const uint32_t *>(&h1);
                        lo[i] = pack_bf16x2(e0.x - __low2float(h0), e0.y - __high2float(h0));
                        lo[i + 1] = pack_bf16x2(e1.x - __low2float(h1), e1.y - __high2float(h1));
                    }
                    tmem_st8(buf + (c0 >> 1), hi);
                    tmem_st8(plo + (c0 >> 1), lo);
                }
            } else {
#pragma unroll
                for (int c = 0; c < kBlock; c += 4) {
                    const float2 x0 = __ffma2_rn(make_float2(__uint_as_float(s[c]), __uint_as_float(s[c + 1])), sc2, nm2);
                    const float2 x1 = __ffma2_rn(make_float2(__uint_as_float(s[c + 2]), __uint_as_float(s[c + 3])), sc2, nm2);
                    const float2 e0 = make_float2(fast_exp2(x0.x), fast_exp2(x0.y));
                    const float2 e1 = make_float2(fast_exp2(x1.x), fast_exp2(x1.y));
                    acc0 = __fadd2_rn(acc0, e0);
                    acc1 = __fadd2_rn(acc1, e1);
                    pk[c >> 1] = pack_bf16x2(e0.x, e0.y);
                    pk[(c >> 1) + 1] = pack_bf16x2(e1.x, e1.y);
                }
            }
            const float sum0 = acc0.x + acc0.y, sum1 = acc1.x + acc1.y;
            l_run = l_run * alpha + (sum0 + sum1);
            lap(2);
            // rare: a running max moved by more than the slack. O must be rescaled, which needs the previous
            // block's O += P V to have finished. (P_j itself goes to its own buffer and needs no wait.)
            if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
                ok = mbar_wait(bar_pv + ((j - 1) & 1) * 8, ((j - 1) >> 1) & 1);
                tc_fence_after_sync();
                lap(3);
                {
#pragma unroll
                    for (int c = 0; c < kD / 32; ++c) {
                        uint32_t o[32];
                        tmem_ld32(tm + lane_base + kColO + c * 32, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                        tmem_st32(tm + lane_base + kColO + c * 32, o);
                    }
                }
            }
            if constexpr (kD != 64)
#pragma unroll
                for (int c = 0; c < kBlock / 64; ++c) tmem_st32(buf + c * 32, *reinterpret_cast<uint32_t(*)[32]>(pk + c * 32));
            tmem_wait_st();
            // V rows past the context inside the last page may hold NaN; 0 * NaN is NaN, so clear them
            const int valid_rows = L - t0;
            if (valid_rows < kBlock) {
                const uint32_t vst = v_ring + (j % kStages) * kTileBytes;
                ok = ok && mbar_wait(bar_v + (j % kStages) * 8, (j / kStages) & 1);  // the tile must have landed
                const int last = min(kBlock, (valid_rows + kPageSize - 1) / kPageSize * kPageSize);
                for (int i = tid; i < (last - valid_rows) * (kD / 8); i += kRows) {
                    const int r = valid_rows + i / (kD / 8), c = i % (kD / 8);
                    st_shared_zero16(vst + (c >> 3) * kHalfBytes + r * 128 + (c & 7) * 16);
                }
                fence_proxy_async();
            }
            tc_fence_before_sync();
            __syncwarp();
            if ((tid & 31) == 0) mbar_arrive(bar_p_full + (j & 1) * 8);
            lap(4);
        }
        if (tracing && tid == 0) {
            const int cta = (blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;
            if (cta < p.trace_ctas) {
                unsigned long long *t = p.trace + static_cast<size_t>(cta) * 16;
                for (int i = 0; i < 5; ++i) t[i] = static_cast<unsigned long long>(ph[i]);
                t[5] = static_cast<unsigned long long>(clock64() - t_begin);
                t[6] = static_cast<unsigned long long>(nb);
            }
        }

        // ---- epilogue: O / l -> bf16 rows
        if (ok) ok = mbar_wait(bar_pv + ((nb - 1) & 1) * 8, ((nb - 1) >> 1) & 1);
        tc_fence_after_sync();
        const float inv = 1.f / l_run;
        __nv_bfloat16 *orow = p.out + (static_cast<size_t>(q0 + tile_start + tok) * p.Hq + kvh * G + head) * kD;
#pragma unroll
        for (int c = 0; c < kD / 32; ++c) {
            uint32_t o[32];
            tmem_ld32(tm + lane_base + kColO + c * 32, o);
            tmem_wait_ld();
            if (row_valid && ok) {
#pragma unroll
                for (int i = 0; i < 32; i += 8) {
                    uint4 v;
                    v.x = pack_bf16x2(__uint_as_float(o[i]) * inv, __uint_as_float(o[i + 1]) * inv);
                    v.y = pack_bf16x2(__uint_as_float(o[i + 2]) * inv, __uint_as_float(o[i + 3]) * inv);
                    v.z = pack_bf16x2(__uint_as_float(o[i + 4]) * inv, __uint_as_float(o[i + 5]) * inv);
                    v.w = pack_bf16x2(__uint_as_float(o[i + 6]) * inv, __uint_as_float(o[i + 7]) * inv);
                    *reinterpret_cast<uint4 *>(orow + c * 32 + i) = v;
                }
            }
        }
        if (p.lse != nullptr && row_valid && ok)
            p.lse[static_cast<size_t>(q0 + tile_start + tok) * p.Hq + kvh * G + head] = (m_run + log2f(l_run)) * kLn2f;
        if (!ok && (tid & 31) == 0) latch(p.status, kDevTimeout, b, blockIdx.x);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, kTmemCols);
}

// Sequences ranked by the attention work of their turn, q_len * (context seen on average), heaviest first:
// CTAs start in block-index order, so the long sequences no longer end up as the tail of the grid.
// One thread per sequence counts the sequences that precede it (B <= 4096: at most 16 M comparisons).
__global__ void __launch_bounds__(256) prefill_order_kernel(const PrefillParams p) {
    grid_dependency_wait();
    launch_dependents();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= p.B) return;
    auto work = [&](int i) {
        const long long n = p.q_indptr[i + 1] - p.q_indptr[i];
        const long long L = p.ctx_lens[i];
        return n * (2 * L - n);  // twice the number of (query, key) pairs under the causal mask, up to O(n)
    };
    const long long mine = work(b);
    int rank = 0;
    for (int i = 0; i < p.B; ++i) {
        const long long w = work(i);
        rank += (w > mine || (w == mine && i < b)) ? 1 : 0;
    }
    p.order[rank] = b;
}

// Multi-token append: CTA (x, b) copies tokens x, x + gridDim.x, ... of sequence b. Lengths are read
// here and advanced by a separate tiny kernel, so no CTA sees a half-updated length.
__global__ void __launch_bounds__(256) kv_append_tokens_kernel(const AppendTokensParams p) {
    const int b = blockIdx.y;
    grid_dependency_wait();
    launch_dependents();
    const int r0 = p.q_indptr[b], n = p.q_indptr[b + 1] - r0;
    const int L = p.ctx_lens[b];
    if (n <= 0) return;
    if (L < 0 || (L + n + kPageSize - 1) / kPageSize > p.MP) {
        if (threadIdx.x == 0 && blockIdx.x == 0) latch(p.status, kDevBadLength, b, L);
        return;
    }
    const int chunks_per_row = p.D / 8, chunks_per_tensor = p.Hkv * chunks_per_row;
    for (int i = blockIdx.x; i < n; i += gridDim.x) {
        const int pos = L + i;
        const int page = p.page_table[static_cast<size_t>(b) * p.MP + pos / kPageSize];
        if (page < 0 || page >= p.num_pages) {
            if (threadIdx.x == 0) latch(p.status, kDevBadPage, b, page);
            continue;
        }
        for (int c = threadIdx.x; c < 2 * chunks_per_tensor; c += blockDim.x) {
            const int which = c / chunks_per_tensor, rem = c - which * chunks_per_tensor;
            const int kvh = rem / chunks_per_row, jj = rem - kvh * chunks_per_row;
            const __nv_bfloat16 *src = (which ? p.v_new : p.k_new) + (static_cast<size_t>(r0 + i) * p.Hkv + kvh) * p.D + jj * 8;
            __nv_bfloat16 *dst = (which ? p.v_pages : p.k_pages) +
                                 ((static_cast<size_t>(page) * p.Hkv + kvh) * kPageSize + pos % kPageSize) * p.D + jj * 8;
            *reinterpret_cast<uint4 *>(dst) = __ldg(reinterpret_cast<const uint4 *>(src));
        }
    }
}

__global__ void advance_lens_kernel(const AppendTokensParams p) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    grid_dependency_wait();
    launch_dependents();
    if (b >= p.B) return;
    const int n = p.q_indptr[b + 1] - p.q_indptr[b];
    const int L = p.ctx_lens[b];
    if (n > 0 && L >= 0 && (L + n + kPageSize - 1) / kPageSize <= p.MP) p.ctx_lens[b] = L + n;
}

}  // namespace

size_t prefill_smem_bytes(int head_dim) {
    const int halves = head_dim / 64;
    return static_cast<size_t>(halves) * (kQHalfBytes + 2 * kStages * kHalfBytes) + 1024 + (2 * kStages + 6) * 8 + 64;
}

// head_dim 128 has its own kernel (pd_prefill_attn_d128.cu: two query tiles per CTA, 128-token blocks)
cudaError_t prepare_prefill_attn_d128();
cudaError_t launch_prefill_attn_d128(const CUtensorMap &tm_k, const CUtensorMap &tm_v, const PrefillParams &p, int max_q_len,
                                     cudaStream_t stream);

cudaError_t prepare_prefill_attn(int head_dim) {
    if (head_dim == 128) return prepare_prefill_attn_d128();
    const int bytes = static_cast<int>(prefill_smem_bytes(head_dim));
    return cudaFuncSetAttribute(prefill_attn_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

cudaError_t launch_prefill_attn(int head_dim, const CUtensorMap &tm_k, const CUtensorMap &tm_v, const PrefillParams &p,
                                int max_q_len, cudaStream_t stream) {
    if (p.B == 0 || max_q_len <= 0) return cudaSuccess;
    if (p.order != nullptr) {
        const cudaError_t e = launch_pdl(prefill_order_kernel, dim3((p.B + 255) / 256), dim3(256), 0, stream, p.pdl != 0, p);
        if (e != cudaSuccess) return e;
    }
    if (head_dim == 128) return launch_prefill_attn_d128(tm_k, tm_v, p, max_q_len, stream);
    const int tok = kRows / p.G;
    const dim3 grid((max_q_len + tok - 1) / tok, p.Hkv, p.B);
    return launch_pdl(prefill_attn_kernel<64>, grid, dim3(kThreads), prefill_smem_bytes(head_dim), stream, p.pdl != 0, tm_k, tm_v, p);
}

cudaError_t launch_kv_append_tokens(const AppendTokensParams &p, int max_q_len, cudaStream_t stream) {
    if (p.B == 0 || max_q_len <= 0) return cudaSuccess;
    const dim3 grid(max_q_len < 64 ? max_q_len : 64, p.B);
    cudaError_t err = launch_pdl(kv_append_tokens_kernel, grid, dim3(256), 0, stream, p.pdl != 0, p);
    if (err != cudaSuccess) return err;
    return launch_pdl(advance_lens_kernel, dim3((p.B + 127) / 128), dim3(128), 0, stream, p.pdl != 0, p);
}

}  // namespace pd
