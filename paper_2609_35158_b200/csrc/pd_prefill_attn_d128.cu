// Append-prefill attention for head_dim 128: two query tiles per CTA on the fifth-generation tensor cores.
//
// Same operation as pd_prefill_attn.cu (the prefill terms B * dL * t_prefill of Eq. 1 and Eq. 3: the new
// tokens of a turn attend causally over the cached prefix and themselves, Sec. 2.1); this file is the
// head_dim 128 kernel, built around two measured facts: a tcgen05.mma with M = 128 occupies the tensor pipe
// for at least ~64 cycles whatever its N, so logit products must be N = 128 to run at full rate; and the
// special-function unit delivers 16 exponentials per clock per SM, which for 128 x 128 logits is exactly the
// time of the two products of that block, so nothing in the softmax may sit on the critical path.
//
// One CTA per SM owns TWO tiles of 128 query rows (2 x 128/g consecutive new tokens x the g query heads of
// one KV head; row = head * (128/g) + token) that share every K and V tile. It walks the context in blocks
// of 128 tokens (8 pages):
//   TMA      pages -> shared memory as [half of d][token][128 B] with the 128-byte swizzle (K is a K-major
//            operand, V an MN-major one, no transposes); two K tiles and two V tiles in flight
//   tcgen05  one issuing thread, order  O0(j) S0(j+1) O1(j) S1(j+1):  S_t = Q_t K^T (8 x 128x128x16) into the
//            tile's 128 logit columns of tensor memory, O_t += P_t V in two parts of 64 tokens (4 x 128x128x16
//            each, P_t from tensor memory), the first part issued while the row threads work on the second
//   softmax  one warpgroup per tile, one thread per row, 64 logits (one part) at a time: x = s * scale - m in
//            registers against the row's running reference m as it stands, the reference raised (and the x
//            shifted in place) only when a logit exceeds it by more than 8 log2 units, exp2 on the
//            special-function unit (a polynomial share on the FMA pipe measured slower: the packed FMA
//            instructions issue at half rate), P as bf16 over the first 64 columns of the tile's own logit
//            buffer. While tile 0's warpgroup works, the tensor pipe runs tile 1's products, and vice versa.
// Tensor memory: S0 | S1 | O0 | O1, 128 columns each (all 512). The MMAs of one thread execute in issue order,
// so "O_t(j) before S_t(j+1)" (P_t lives in S_t's columns) needs no barrier, and a commit that follows S_t(j)
// also covers O_t(j-1): a row thread that holds S_t(j) may rescale O_t at once. Every wait is bounded; a
// wait that runs out latches PD_ERR_TIMEOUT, the CTA unwinds and frees its tensor memory.
#include "pd_kernels.cuh"
#include "pd_ptx.cuh"
#include "pd_tcgen05.cuh"

#include <type_traits>

namespace pd {

namespace {

constexpr float kLn2f = 0.6931471805599453f;
constexpr float kSlack = 8.f;                  // log2 units a logit may exceed the running max before a rescale
constexpr int kD = 128;
constexpr int kRows = 128;                     // query rows per tile (MMA M), one softmax thread each
constexpr int kTiles = 2;                      // query tiles per CTA
constexpr int kBlock = 128;                    // context tokens per step (MMA N of S, K of O)
constexpr int kPagesPerBlock = kBlock / kPageSize;
constexpr int kThreads = kTiles * kRows + 128;  // two softmax warpgroups + MMA warp, K loader, V loader, one spare
constexpr int kQHalfBytes = kRows * 128;       // one 64-column half of one Q tile: 16 KB
constexpr int kQTileBytes = 2 * kQHalfBytes;
constexpr int kHalfBytes = kBlock * 128;       // one 64-column half of a K or V tile: 16 KB
constexpr int kTileBytes = 2 * kHalfBytes;     // 32 KB
constexpr int kStages = 2;
constexpr int kTmemCols = 512;
constexpr int kColS = 0, kColO = 256;          // S_t at kColS + 128 t, O_t at kColO + 128 t
constexpr int kPParts = 2;                     // P and the O product of a block go in two parts of 64 tokens
constexpr int kPartKeys = kBlock / kPParts;

// Cycle stamps of CTA (0,0,0) for a timeline of the hand-overs; compiled in only by a profiling build.
#if defined(PD_ENABLE_TUNING) && defined(PD_PF_LIFE)
// -DPD_PF_LIFE instead records the life of the first CTAs of the grid, one record of 8 words per CTA:
// [entry, setup done, first logits, loop end, exit] in ns of the global timer, then block count << 32 | SM id
__device__ __forceinline__ unsigned long long smid() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(r));
    return r;
}
#define PD_STAMP(region, per_block, j, k)
#define PD_LIFE(k, v)                                                                                            \
    if (p.trace != nullptr && life_id * 8 + 8 <= p.trace_ctas * 16) p.trace[life_id * 8 + (k)] = (v);
#elif defined(PD_ENABLE_TUNING)
#define PD_LIFE(k, v)
constexpr int kLogFirst = 8, kLogBlocks = 16;
#define PD_STAMP(region, per_block, j, k)                                                                       \
    if (p.trace != nullptr && (blockIdx.x | blockIdx.y | blockIdx.z) == 0 && (j) >= kLogFirst &&                  \
        (j) < kLogFirst + kLogBlocks)                                                                            \
        p.trace[1024 * (region) + ((region) >= 3 ? ((threadIdx.x >> 5) & 3) * 64 : 0) + ((j) - kLogFirst) * (per_block) + (k)] = static_cast<unsigned long long>(clock64());
#else
#define PD_STAMP(region, per_block, j, k)
#define PD_LIFE(k, v)
#endif

__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

__device__ __forceinline__ void latch(int32_t *status, int code, int seq, int detail) {
    if (atomicCAS(status, kDevOk, code) == kDevOk) {
        status[1] = seq;
        status[2] = detail;
    }
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
prefill_attn_d128_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                         const PrefillParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t tmem_slot;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int kvh = blockIdx.y;
    const int G = p.G, TOK = kRows / G;            // tokens per tile
    const int CTA_TOK = kTiles * TOK;              // tokens per CTA

    grid_dependency_wait();
    launch_dependents();
#if defined(PD_ENABLE_TUNING) && defined(PD_PF_LIFE)
    const int life_id = tid == 0 ? static_cast<int>(blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z)) : 1 << 30;
    PD_LIFE(0, global_timer_ns())
    PD_LIFE(5, 0)
#endif
    const int b = p.order != nullptr ? p.order[blockIdx.z] : static_cast<int>(blockIdx.z);  // heaviest sequences first
    const int q0 = p.q_indptr[b], q_len = p.q_indptr[b + 1] - q0;
    // CTAs are scheduled in index order: start a sequence's last tokens (the longest contexts) first
    const int cta_start = static_cast<int>(p.reverse_tiles ? gridDim.x - 1 - blockIdx.x : blockIdx.x) * CTA_TOK;
    if (cta_start >= q_len) return;  // before any allocation
    const int L = min(max(p.ctx_lens[b], 0), p.MP * kPageSize);
    if (L < q_len) {  // the cache must already hold the new tokens
        if (tid == 0) latch(p.status, kDevBadLength, b, L);
        return;
    }
    const int n_tok = min(CTA_TOK, q_len - cta_start);           // valid tokens of this CTA, over both tiles
    const int pos0 = L - q_len + cta_start;                      // absolute position of the CTA's first token
    const int nb = (pos0 + n_tok - 1) / kBlock + 1;              // context blocks the CTA's last token can see
    const int n_pages = (L + kPageSize - 1) / kPageSize;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *aligned = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t q_s = base;
    const uint32_t k_ring = base + kTiles * kQTileBytes, v_ring = k_ring + kStages * kTileBytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(aligned + kTiles * kQTileBytes + 2 * kStages * kTileBytes);
    // [2] K tile landed, [2] V tile landed (transaction barriers)
    const uint32_t bar_k = smem_u32(bars), bar_v = smem_u32(bars + 2);
    // [2] K slot free again (commit after S1 of the block it held), [2] V slot free (commit after O1)
    const uint32_t bar_kfree = smem_u32(bars + 4), bar_vfree = smem_u32(bars + 6);
    // [2] S_t of the current block is in tensor memory (and every earlier product has completed)
    const uint32_t bar_s = smem_u32(bars + 8);
    // [2 tiles][2 parts] every warp of tile t's warpgroup wrote its rows of that part of P_t. One barrier per part:
    // the warps of a warpgroup are not in step, and a fast warp's second arrival must not count towards the first
    // part (with one barrier and two phases per block a waiter that looks late finds the parity it waits for two
    // phases on and never wakes)
    const uint32_t bar_p = smem_u32(bars + 10);
    // [2] the last O_t product has completed; [2] the first part's O_t product of the current block has completed
    const uint32_t bar_o = smem_u32(bars + 14);

    if (tid == 0) {
        for (int i = 0; i < 10; ++i) mbar_init(smem_u32(bars + i), 1);
        for (int i = 0; i < 4; ++i) mbar_init(bar_p + i * 8, kRows / 32);
        for (int i = 0; i < 4; ++i) mbar_init(bar_o + i * 8, 1);
        mbar_init_fence();
        prefetch_tensormap(&tm_k);
        prefetch_tensormap(&tm_v);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_slot), kTmemCols);
        tmem_relinquish_alloc_permit();
    }
    // ---- the Q tiles: thread r of warpgroup t stages row r of tile t
    const int tile = tid >> 7, row = tid & (kRows - 1);
    const int head = row / TOK, tok = tile * TOK + (row - head * TOK);  // token index inside the CTA
    const bool row_valid = tid < kTiles * kRows && tok < n_tok;
    const int my_pos = pos0 + min(tok, n_tok - 1);  // padding rows mirror the last token
    if (tid < kTiles * kRows) {
        const uint4 *src = reinterpret_cast<const uint4 *>(
            p.q + (static_cast<size_t>(q0 + cta_start + min(tok, n_tok - 1)) * p.Hq + kvh * G + head) * kD);
#pragma unroll
        for (int c = 0; c < kD / 8; ++c) {
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (row_valid) v = __ldg(src + c);
            const uint32_t a = q_s + tile * kQTileBytes + (c >> 3) * kQHalfBytes + sw128_offset(row, c & 7);
            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
        }
    }
    fence_proxy_async();  // the Q tiles were written with ordinary stores; the tensor core reads them through the async proxy
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tm = tmem_slot;
    PD_LIFE(1, global_timer_ns())
    PD_LIFE(5, (static_cast<unsigned long long>(nb) << 32) | smid())
    bool ok = true;

    if (warp == kTiles * 4) {
        // ================= MMA warp: one thread issues every product =================
        if (lane == 0) {
            constexpr uint32_t idesc_s = umma_idesc_bf16(kRows, kBlock, false);
            constexpr uint32_t idesc_o = umma_idesc_bf16(kRows, kD, true);
            auto issue_s = [&](int t, int j) {  // S_t(j) = Q_t K_j^T
                const uint32_t kst = k_ring + (j % kStages) * kTileBytes;
                const uint32_t qt = q_s + t * kQTileBytes;
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        umma_ss(tm + kColS + t * kBlock, umma_smem_desc(qt + h * kQHalfBytes + ks * 32, 16, 1024),
                                umma_smem_desc(kst + h * kHalfBytes + ks * 32, 16, 1024), idesc_s, (h | ks) != 0);
                umma_commit(bar_s + t * 8);
                if (t == kTiles - 1) umma_commit(bar_kfree + (j % kStages) * 8);
            };
            auto issue_o = [&](int t, int j, int part) {  // O_t += P_t(j)[:, part] V_j[part], P_t in the first 64 columns of S_t
                const uint32_t vst = v_ring + (j % kStages) * kTileBytes + part * (kPartKeys / 16) * 2048;
#pragma unroll
                for (int ks = 0; ks < kPartKeys / 16; ++ks)
                    umma_ts(tm + kColO + t * kD, tm + kColS + t * kBlock + (part * (kPartKeys / 16) + ks) * 8,
                            umma_smem_desc(vst + ks * 2048, kHalfBytes, 1024), idesc_o, (j | part | ks) != 0);
                if (part == kPParts - 1) {
                    if (t == kTiles - 1) umma_commit(bar_vfree + (j % kStages) * 8);
                    if (j == nb - 1) umma_commit(bar_o + t * 8);
                } else {
                    umma_commit(bar_o + (2 + t) * 8);  // lets a row thread rescale O_t between the two parts (rare)
                }
            };
            ok = mbar_wait(bar_k, 0);
            if (ok) {
                tc_fence_after_sync();
                issue_s(0, 0);
                issue_s(1, 0);
            }
            // Nothing queues behind the tensor pipe: a cycle this thread spends between two products is a cycle the
            // pipe idles (a satisfied mbarrier wait costs it ~90). So the waits that are satisfied long before they
            // are needed (the V tile of this block, the K tile of the next) are taken just ahead of a wait on P,
            // where the thread would be standing anyway.
            for (int j = 0; j < nb && ok; ++j) {
                PD_STAMP(0, 12, j, 0)
                ok = mbar_wait(bar_v + (j % kStages) * 8, (j >> 1) & 1) && mbar_wait(bar_p, j & 1);
                if (!ok) break;
                tc_fence_after_sync();
                PD_STAMP(0, 12, j, 1)
                issue_o(0, j, 0);
                PD_STAMP(0, 12, j, 2)
                if (j + 1 < nb) ok = mbar_wait(bar_k + ((j + 1) % kStages) * 8, ((j + 1) >> 1) & 1);
                ok = ok && mbar_wait(bar_p + 8, j & 1);
                if (!ok) break;
                tc_fence_after_sync();
                PD_STAMP(0, 12, j, 3)
                issue_o(0, j, 1);
                PD_STAMP(0, 12, j, 4)
                PD_STAMP(0, 12, j, 5)
                if (j + 1 < nb) issue_s(0, j + 1);
                PD_STAMP(0, 12, j, 6)
                ok = mbar_wait(bar_p + 16, j & 1);
                if (!ok) break;
                tc_fence_after_sync();
                PD_STAMP(0, 12, j, 7)
                issue_o(1, j, 0);
                PD_STAMP(0, 12, j, 8)
                ok = mbar_wait(bar_p + 24, j & 1);
                if (!ok) break;
                tc_fence_after_sync();
                PD_STAMP(0, 12, j, 9)
                issue_o(1, j, 1);
                PD_STAMP(0, 12, j, 10)
                if (j + 1 < nb) issue_s(1, j + 1);
                PD_STAMP(0, 12, j, 11)
            }
            if (!ok) latch(p.status, kDevTimeout, b, blockIdx.x);
        }
    } else if (warp == kTiles * 4 + 1 || warp == kTiles * 4 + 2) {
        // ================= two TMA warps (one streams K, the other V): one box per lane =================
        // A tile of 128 tokens is 8 pages x 2 halves = 16 boxes of 2 KB; lane l issues box l in one warp
        // instruction. Page ids are fetched 32 at a time (one per lane), a group ahead of need.
        const uint64_t policy = l2_policy_evict_first();
        const int32_t oob_row = p.num_pages * p.Hkv * kPageSize;  // a TMA box that starts here is all zero fill
        const int32_t *pt_row = p.page_table + static_cast<size_t>(b) * p.MP;
        const bool is_k = warp == kTiles * 4 + 1;
        const CUtensorMap *map = is_k ? &tm_k : &tm_v;
        const uint32_t ring = is_k ? k_ring : v_ring, bar_full = is_k ? bar_k : bar_v, bar_free = is_k ? bar_kfree : bar_vfree;
        int c_grp = -2, c_val = -1, c_nval = -1;
        auto load_group = [&](int grp) {
            const int idx = grp * 32 + lane;
            return (idx < n_pages) ? __ldg(pt_row + idx) : -1;
        };
        auto issue_tile_loads = [&](int j) {
            const uint32_t st = ring + (j % kStages) * kTileBytes;
            const uint32_t bar = bar_full + (j % kStages) * 8;
            const int grp = (j * kPagesPerBlock) >> 5;  // the 8 pages of a block never straddle a group of 32
            if (grp != c_grp) {
                c_val = (grp == c_grp + 1) ? c_nval : load_group(grp);
                c_grp = grp;
                c_nval = load_group(grp + 1);
            }
            const int pg = (lane >> 1) & (kPagesPerBlock - 1), h = lane & 1;
            const int lp = j * kPagesPerBlock + pg;
            int pid = __shfl_sync(0xffffffffu, c_val, lp & 31);
            int32_t y = oob_row;
            if (lp < n_pages) {
                if (pid < 0 || pid >= p.num_pages) {
                    if (lane < 2 * kPagesPerBlock && h == 0) latch(p.status, kDevBadPage, b, pid);
                    pid = 0;
                }
                y = (pid * p.Hkv + kvh) * kPageSize;
            }
            if (lane == 0) mbar_arrive_expect_tx(bar, kTileBytes);
            __syncwarp();
            if (lane < 2 * kPagesPerBlock)
                tma_load_2d(st + h * kHalfBytes + pg * (kPageSize * 128), map, h * 64, y, bar, policy);
        };
        for (int j = 0; j < min(nb, kStages); ++j) issue_tile_loads(j);
        for (int j = 0; j + kStages < nb && ok; ++j) {
            ok = __all_sync(0xffffffffu, mbar_wait(bar_free + (j % kStages) * 8, (j >> 1) & 1));
            if (!ok) break;
            issue_tile_loads(j + kStages);
        }
        if (!ok && lane == 0) latch(p.status, kDevTimeout, b, blockIdx.x);
    } else if (warp < kTiles * 4) {
        // ================= softmax warpgroups: warpgroup t owns tile t, one thread per query row =================
        const int t = tile;
        const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t s_buf = tm + lane_base + kColS + t * kBlock;
        const uint32_t o_buf = tm + lane_base + kColO + t * kD;
        float m_run = -INFINITY, l_run = 0.f;
        const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
        for (int j = 0; j < nb && ok; ++j) {
            if (row == 0) { PD_STAMP(1 + t, 6, j, 0) }
            ok = mbar_wait(bar_s + t * 8, j & 1);
            tc_fence_after_sync();
            if (!ok) break;
            if (row == 0) { PD_STAMP(1 + t, 6, j, 1) }
            if (j == 0) { PD_LIFE(2, global_timer_ns()) }
            const int t0 = j * kBlock;
            const bool masked = t0 + kBlock - 1 > my_pos;  // the block reaches past this row's position
            // V rows past the context inside the last page may hold NaN; 0 * NaN is NaN, so tile 0's warpgroup
            // clears them (both tiles' products of this block are issued after its first arrival below)
            const int valid_rows = L - t0;
            if (t == 0 && valid_rows < kBlock) {
                const uint32_t vst = v_ring + (j % kStages) * kTileBytes;
                ok = ok && mbar_wait(bar_v + (j % kStages) * 8, (j >> 1) & 1);  // the tile must have landed
                const int last = min(kBlock, (valid_rows + kPageSize - 1) / kPageSize * kPageSize);
                for (int i = row; i < (last - valid_rows) * (kD / 8); i += kRows) {
                    const int r = valid_rows + i / (kD / 8), c = i % (kD / 8);
                    st_shared_zero16(vst + (c >> 3) * kHalfBytes + r * 128 + (c & 7) * 16);
                }
                fence_proxy_async();
            }
            // ---- one part of 64 tokens at a time, in two passes over registers. Pass 1: x = s * scale - m against
            // the running reference m of the row AS IT STANDS, in place, and the largest x. Only if that exceeds the
            // slack (rare; the first part of the first block always, its reference is a placeholder) is the
            // reference raised by it: what the row has accumulated is rescaled and the x are shifted in their
            // registers, nothing is recomputed. Pass 2: exponentials, row sum, P stored 32 tokens at a time so the
            // stores overlap the arithmetic. Blocks no row of the warp sees masked (all but the last one or two)
            // run a copy without the mask selects.
            float blk_sum = 0.f;
            auto load_part = [&](int part, uint32_t (&sreg)[kPartKeys]) {
#pragma unroll
                for (int c = 0; c < kPartKeys / 32; ++c)
                    tmem_ld32(s_buf + part * kPartKeys + c * 32, *reinterpret_cast<uint32_t(*)[32]>(sreg + c * 32));
            };
            auto pass1 = [&](auto masked_c, int part, uint32_t (&sreg)[kPartKeys], float (&x)[kPartKeys]) {
                constexpr bool kMasked = decltype(masked_c)::value;
                const bool first = j == 0 && part == 0;
                if (kMasked) {  // mask by select: masked logits become -inf, their exponentials exact zeros
                    const int visible = my_pos - (t0 + part * kPartKeys) + 1;  // logits of this part the row may see
#pragma unroll
                    for (int c = 0; c < kPartKeys; ++c)
                        if (c >= visible) sreg[c] = 0xff800000u;
                }
                if (first) m_run = 0.f;  // placeholder; the branch below replaces it by the part's maximum
                {
                    const float2 nm2 = make_float2(-m_run, -m_run);
                    float xm[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int c = 0; c < kPartKeys; c += 4) {
                        const float2 u = __ffma2_rn(make_float2(__uint_as_float(sreg[c]), __uint_as_float(sreg[c + 1])), sc2, nm2);
                        const float2 v = __ffma2_rn(make_float2(__uint_as_float(sreg[c + 2]), __uint_as_float(sreg[c + 3])), sc2, nm2);
                        x[c] = u.x, x[c + 1] = u.y, x[c + 2] = v.x, x[c + 3] = v.y;
                        xm[(c >> 2) & 1] = max3(xm[(c >> 2) & 1], u.x, u.y);
                        xm[2 + ((c >> 2) & 1)] = max3(xm[2 + ((c >> 2) & 1)], v.x, v.y);
                    }
                    const float xmax = fmaxf(fmaxf(xm[0], xm[1]), fmaxf(xm[2], xm[3]));
                    if (first || __any_sync(0xffffffffu, xmax > kSlack)) {
                        float shift = 0.f, alpha = 1.f;
                        if (first || xmax > kSlack) {  // position 0 is visible to every row, so the first maximum is finite
                            shift = xmax;
                            alpha = fast_exp2(-xmax);
                            m_run += xmax;
                        }
                        if (!first) {
                            if (part > 0) {  // the first part's product of this block must be over before O_t is touched
                                ok = ok && mbar_wait(bar_o + (2 + t) * 8, j & 1);
                                tc_fence_after_sync();
                            }
                            // the commit that announced S_t(j) also covers O_t(j-1)
#pragma unroll 1
                            for (int c = 0; c < kD / 16; ++c) {
                                uint32_t o[16];
                                tmem_ld16(o_buf + c * 16, o);
                                tmem_wait_ld();
#pragma unroll
                                for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                                tmem_st16(o_buf + c * 16, o);
                            }
                            tmem_wait_st();
                            l_run *= alpha;
                            blk_sum *= alpha;
                        }
                        const float2 ns2 = make_float2(-shift, -shift);
#pragma unroll
                        for (int c = 0; c < kPartKeys; c += 2) {
                            const float2 u = __fadd2_rn(make_float2(x[c], x[c + 1]), ns2);
                            x[c] = u.x, x[c + 1] = u.y;
                        }
                    }
                }
            };
            auto pass2 = [&](int part, float (&x)[kPartKeys]) {
                float2 a0 = make_float2(0.f, 0.f), a1 = make_float2(0.f, 0.f);
#pragma unroll
                for (int c0 = 0; c0 < kPartKeys; c0 += 32) {
                    uint32_t pk[16];
#pragma unroll
                    for (int c = c0; c < c0 + 32; c += 8) {
                        float2 e[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) e[u] = make_float2(fast_exp2(x[c + 2 * u]), fast_exp2(x[c + 2 * u + 1]));
                        a0 = __fadd2_rn(a0, __fadd2_rn(e[0], e[1]));
                        a1 = __fadd2_rn(a1, __fadd2_rn(e[2], e[3]));
#pragma unroll
                        for (int u = 0; u < 4; ++u) pk[((c - c0) >> 1) + u] = pack_bf16x2(e[u].x, e[u].y);
                    }
                    // P over the first 64 columns of the tile's logit buffer (columns this thread has already consumed)
                    tmem_st16(s_buf + ((part * kPartKeys + c0) >> 1), pk);
                }
                blk_sum += (a0.x + a0.y) + (a1.x + a1.y);
                tmem_wait_st();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_p + (t * 2 + part) * 8);
                if (row == 0) { PD_STAMP(1 + t, 6, j, 3 + part) }
            };
            // the second part's logits are fetched while the first part's exponentials run
            auto do_block = [&](auto masked_c) {
                uint32_t sa[kPartKeys], sb[kPartKeys];
                float x[kPartKeys];
                load_part(0, sa);
                tmem_wait_ld();
                if (row == 0) { PD_STAMP(1 + t, 6, j, 2) }
                pass1(masked_c, 0, sa, x);
                load_part(1, sb);
                pass2(0, x);
                tmem_wait_ld();
                pass1(masked_c, 1, sb, x);
                pass2(1, x);
            };
            if (__any_sync(0xffffffffu, masked)) do_block(std::true_type{});
            else do_block(std::false_type{});
            l_run += blk_sum;
        }

        // ---- epilogue: O_t / l -> bf16 rows
        PD_LIFE(3, global_timer_ns())
        if (ok) ok = mbar_wait(bar_o + t * 8, 0);
        tc_fence_after_sync();
        const float inv = 1.f / l_run;
        __nv_bfloat16 *orow = p.out + (static_cast<size_t>(q0 + cta_start + min(tok, n_tok - 1)) * p.Hq + kvh * G + head) * kD;
#pragma unroll
        for (int c = 0; c < kD / 32; ++c) {
            uint32_t o[32];
            tmem_ld32(o_buf + c * 32, o);
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
            p.lse[static_cast<size_t>(q0 + cta_start + tok) * p.Hq + kvh * G + head] = (m_run + log2f(l_run)) * kLn2f;
        if (!ok && lane == 0) latch(p.status, kDevTimeout, b, blockIdx.x);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, kTmemCols);
    PD_LIFE(4, global_timer_ns())
}

}  // namespace

size_t prefill_d128_smem_bytes() { return static_cast<size_t>(kTiles) * kQTileBytes + 2 * kStages * kTileBytes + 1024 + 18 * 8 + 64; }

cudaError_t prepare_prefill_attn_d128() {
    return cudaFuncSetAttribute(prefill_attn_d128_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                static_cast<int>(prefill_d128_smem_bytes()));
}

cudaError_t launch_prefill_attn_d128(const CUtensorMap &tm_k, const CUtensorMap &tm_v, const PrefillParams &p, int max_q_len,
                                     cudaStream_t stream) {
    const int cta_tok = kTiles * (kRows / p.G);
    const dim3 grid((max_q_len + cta_tok - 1) / cta_tok, p.Hkv, p.B);
    return launch_pdl(prefill_attn_d128_kernel, grid, dim3(kThreads), prefill_d128_smem_bytes(), stream, p.pdl != 0, tm_k, tm_v, p);
}

}  // namespace pd
