/*
 * pd.h - C ABI of the paged decode-attention library (CUDA, sm_100a).
 *
 * The library covers the per-sequence term of the paper's decode cost model:
 * in Eq. 1 a decode iteration costs A + b*B/N, where b is the marginal cost of
 * one more concurrent sequence and comes mainly from that sequence's KV-cache
 * HBM reads; Eq. 2 lowers the concurrency to B/(1+theta) while sequences wait
 * on the environment. The two operations behind that term are exported here:
 * the attention of one new query token per sequence over its cached context,
 * and the append of that token's K/V to the cache (Sec. 2.1: every generated
 * token joins its trajectory's context).
 *
 * Data layout (a choice of this library; the paper describes none):
 *   q, out         [batch][num_q_heads][head_dim]                      bf16
 *   k_new, v_new   [batch][num_kv_heads][head_dim]                     bf16
 *   k_pages,
 *   v_pages        [num_pages][num_kv_heads][page_size][head_dim]      bf16
 *   page_table     [batch][max_pages_per_seq] int32; entry i is the physical
 *                  page of tokens [i*page_size, (i+1)*page_size); entries at or
 *                  past ceil(ctx_lens[b]/page_size) are never read
 *   ctx_lens       [batch] int32, tokens visible to the query
 *   lse            [batch][num_q_heads] fp32, natural log of sum exp(scaled logits)
 * Query head h reads KV head h / (num_q_heads / num_kv_heads).
 *
 * Unless a function says otherwise every pointer is a DEVICE pointer to memory
 * the caller owns, 16-byte aligned, on the device given at pd_create; `stream`
 * is a cudaStream_t passed as void* (NULL = the default stream). Calls enqueue
 * work and return without synchronising. Return value: PD_OK or a negative
 * PD_ERR_* code; nothing throws, aborts or prints. The library owns only the
 * workspace pd_create allocates.
 */
#ifndef PD_H
#define PD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PD_OK 0
#define PD_ERR_INVALID_ARG (-1)  /* null/misaligned pointer, size out of the configured range */
#define PD_ERR_UNSUPPORTED (-2)  /* geometry this build has no kernel for                     */
#define PD_ERR_CUDA (-3)         /* a CUDA runtime/driver call failed (allocation, launch)    */
#define PD_ERR_WORKSPACE (-4)    /* request exceeds the workspace sized at pd_create          */
#define PD_ERR_DEVICE_FAULT (-5) /* a kernel met an out-of-range page id or position          */
#define PD_ERR_TIMEOUT (-6)      /* a kernel gave up a bounded wait on an asynchronous copy   */

/* pd_config.flags */
#define PD_FLAG_NONE 0u
/* pd_kv_append call_flags */
#define PD_APPEND_NO_ADVANCE 1u /* leave ctx_lens unchanged */

typedef struct pd_ctx pd_ctx; /* opaque */

typedef struct pd_config {
    int32_t num_q_heads;       /* multiple of num_kv_heads; group size in {1,2,4,8}           */
    int32_t num_kv_heads;
    int32_t head_dim;          /* 64 or 128                                                   */
    int32_t page_size;         /* 16                                                          */
    int32_t max_batch;         /* 1 .. 4096; sizes the workspace and the host-step staging    */
    int32_t max_pages_per_seq; /* row length of page_table                                    */
    int64_t num_pages;         /* pages in each pool                                          */
    int32_t device;            /* CUDA ordinal                                                */
    uint32_t flags;
} pd_config;

/*
 * Creates a context on cfg->device: checks the geometry, allocates the workspace
 * for split partials (device) and the staging buffers pd_decode_step_host uses.
 * *out is NULL on failure. Not thread-safe per context; use one context per
 * host thread or serialise calls.
 */
int pd_create(const pd_config *cfg, pd_ctx **out);

/* Synchronises the device, frees the workspace. NULL is accepted. */
int pd_destroy(pd_ctx *ctx);

/*
 * KV append (Sec. 2.1, growth of the context by one token per decode step).
 * For every b < batch: pos = ctx_lens[b]; the head_dim bf16 values of each KV
 * head of k_new[b] and v_new[b] are copied, bit for bit, to slot pos % page_size
 * of page page_table[b][pos / page_size] in k_pages / v_pages; then ctx_lens[b]
 * becomes pos + 1 (unless PD_APPEND_NO_ADVANCE). A sequence whose position is
 * past the table or whose page id is outside [0, num_pages) is skipped, its
 * length is not advanced, and the fault is latched for pd_device_status.
 * The page for pos must already be in the table (page allocation is the
 * caller's job).
 */
int pd_kv_append(pd_ctx *ctx, const void *k_new, const void *v_new, void *k_pages, void *v_pages,
                 const int32_t *page_table, int32_t *ctx_lens, int32_t batch, uint32_t call_flags,
                 void *stream);

/*
 * Decode attention (the KV-read term b of Eq. 1): for every b < batch and query
 * head h, out[b][h] = softmax(sm_scale * q[b][h] . K^T) V over the ctx_lens[b]
 * cached tokens of KV head h / group, and, if lse is not NULL,
 * lse[b][h] = log sum_t exp(sm_scale * q[b][h] . K_t). ctx_lens[b] == 0 gives
 * out = 0 and lse = -inf. Slots past ctx_lens[b] and unused pages may hold
 * anything (NaN included) and do not influence the result.
 *
 * The flattened list of (sequence, KV head, page) units is cut into ranges that
 * worker warps claim in order, long ranges first and short ones last, so that
 * few long sequences (low decode concurrency, Eq. 2) still occupy every SM and
 * all SMs finish together; a range that holds only part of a (sequence, KV
 * head) context produces an fp32 partial (unnormalised output, running max,
 * running sum) in the workspace and a second kernel merges the partials of each
 * row by log-sum-exp. split_pages = 0 derives the ranges from the total page
 * count and the SM count of the device; split_pages > 0 forces ranges of that
 * many pages (raised silently if the workspace could not hold the resulting
 * partials). Range boundaries never depend on timing, so results are
 * bit-reproducible run to run for a fixed split_pages and device.
 *
 * sm_scale must be finite and positive. q/out rows are head_dim bf16.
 */
int pd_decode_attn(pd_ctx *ctx, const void *q, const void *k_pages, const void *v_pages,
                   const int32_t *page_table, const int32_t *ctx_lens, void *out, float *lse,
                   int32_t batch, float sm_scale, int32_t split_pages, void *stream);

/*
 * One decode step in two launches (Sec. 2.1: the new token joins the context,
 * then attends over it): the result is that of pd_kv_append (advancing)
 * followed by pd_decode_attn, but the append runs inside the split kernel.
 * ctx_lens holds the lengths BEFORE the append on entry and the grown lengths
 * after the kernels ran. The worker that reads a sequence's last page takes
 * the new token's K/V rows from k_new / v_new instead of the pool (whatever
 * the pool held in that slot is ignored) and stores them to the pool, bit for
 * bit. Error behaviour as pd_kv_append: a sequence with no room in its table
 * row or a bad page id at the new position is latched for pd_device_status,
 * its pools and length stay as they were (its output is then unspecified).
 * Shapes as pd_kv_append and pd_decode_attn; out rows of the step are
 * attention over ctx_lens[b] + 1 tokens.
 * The call only enqueues kernels on `stream` (no allocation, no synchronisation;
 * the tensor maps of a pool pointer are encoded on the host the first time it is
 * seen), so a run of steps can be captured in a CUDA graph after one eager call
 * and replayed: the lengths advance on the device with every replay.
 */
int pd_decode_step(pd_ctx *ctx, const void *q, const void *k_new, const void *v_new, void *k_pages,
                   void *v_pages, const int32_t *page_table, int32_t *ctx_lens, void *out, float *lse,
                   int32_t batch, float sm_scale, int32_t split_pages, void *stream);

/*
 * One whole decode step for callers that hold the step's activations on the
 * HOST: copies q_host, k_new_host, v_new_host (host pointers, pinned or
 * pageable, same shapes as q/k_new/v_new) to device staging, runs pd_decode_step
 * (appending, advancing ctx_lens, attending over the grown contexts), copies the
 * result to out_host (host, [batch][num_q_heads][head_dim] bf16) and waits for
 * the stream, so out_host is valid on return. The cache itself (k_pages,
 * v_pages, page_table, ctx_lens) stays on the device. If k_new_host starts where
 * q_host ends and v_new_host where k_new_host ends, the three travel in one copy.
 * A result of at most 256 KB whose buffer is pinned host memory the device can
 * address is stored there by the merge kernel itself, which then raises a pinned
 * flag the call polls (no copy-back operation, no stream synchronisation);
 * larger or pageable results are staged on the device and copied back.
 */
int pd_decode_step_host(pd_ctx *ctx, const void *q_host, const void *k_new_host, const void *v_new_host,
                        void *k_pages, void *v_pages, const int32_t *page_table, int32_t *ctx_lens,
                        void *out_host, int32_t batch, float sm_scale, int32_t split_pages, void *stream);

/*
 * Append-prefill: the step that opens every turn of a multi-turn rollout
 * (Sec. 2.1; the prefill terms B * dL * t_prefill of Eq. 1 and Eq. 3). The new
 * turn's tokens are appended to the cached context and each of them attends
 * causally over the cached prefix and the new tokens up to and including
 * itself; with prefix caching only these tokens are computed.
 *
 * New tokens are packed: sequence b owns rows [q_indptr[b], q_indptr[b+1]) of
 * q / out ([total][num_q_heads][head_dim] bf16), of k_new / v_new
 * ([total][num_kv_heads][head_dim] bf16) and of lse ([total][num_q_heads] fp32,
 * may be NULL). q_indptr is a DEVICE int32 array of batch + 1 entries;
 * max_q_len is a host-side upper bound on q_indptr[b+1] - q_indptr[b] (it sizes
 * the grid; a larger value only launches idle blocks).
 *
 * pd_kv_append_tokens copies the rows of sequence b to positions ctx_lens[b],
 * ctx_lens[b] + 1, ... (their pages must already be in the table) and then adds
 * the token count to ctx_lens[b]; a sequence that would run past its table row
 * or meets a page id outside [0, num_pages) is skipped or partly written and
 * latched for pd_device_status. Bit-exact.
 *
 * pd_prefill_attn expects the cache to hold the new tokens already and
 * ctx_lens[b] = L_b to count them: query i of sequence b sits at position
 * L_b - q_len_b + i and out = softmax(sm_scale * q . K_{0..pos}^T) V_{0..pos}.
 * The kernel runs on the
 * tcgen05 tensor cores with fp32 accumulation; P is rounded to bf16 before the
 * second product.
 */
int pd_kv_append_tokens(pd_ctx *ctx, const void *k_new, const void *v_new, const int32_t *q_indptr,
                        void *k_pages, void *v_pages, const int32_t *page_table, int32_t *ctx_lens,
                        int32_t batch, int32_t max_q_len, void *stream);
int pd_prefill_attn(pd_ctx *ctx, const void *q, const int32_t *q_indptr, const void *k_pages,
                    const void *v_pages, const int32_t *page_table, const int32_t *ctx_lens, void *out,
                    float *lse, int32_t batch, int32_t max_q_len, float sm_scale, void *stream);

/*
 * KV page gather / scatter: the device-side data movement of the cross-pool KV
 * transfer in the disaggregated prefill model (Eq. 3, the B * dL * K / BW term).
 * The prefill side packs the pages that hold a sequence's new tokens into one
 * contiguous buffer; the decode side unpacks such a buffer into pages it has
 * assigned itself. The transport between the two is not part of this library.
 *
 * For every b < batch the logical pages [page_begin[b], page_end[b]) are moved.
 * The packed buffer is [packed pages][2][num_kv_heads][page_size][head_dim]
 * bf16: packed page packed_page_offset[b] + i holds the K block, then the V
 * block, of logical page page_begin[b] + i (whole pages; slots past the
 * sequence's length travel as they are). page_begin, page_end (int32) and
 * packed_page_offset (int64, normally the exclusive prefix sum of the page
 * counts) are DEVICE arrays supplied by the caller, who also sizes `packed`.
 * Ranges of different sequences must not overlap in the packed buffer. A page
 * id outside [0, num_pages) is skipped and latched for pd_device_status.
 * K = 2 * num_kv_heads * head_dim * 2 bytes per token per layer.
 */
int pd_kv_gather(pd_ctx *ctx, const void *k_pages, const void *v_pages, const int32_t *page_table,
                 const int32_t *page_begin, const int32_t *page_end, const int64_t *packed_page_offset,
                 void *packed, int32_t batch, void *stream);
int pd_kv_scatter(pd_ctx *ctx, const void *packed, const int64_t *packed_page_offset, void *k_pages,
                  void *v_pages, const int32_t *page_table, const int32_t *page_begin,
                  const int32_t *page_end, int32_t batch, void *stream);

/*
 * Decode attention without any allocation (the paper has no counterpart; this
 * is a packaging variant of pd_decode_attn for restricted hosts).
 *
 * For callers that cannot allocate device memory at the time they need
 * attention: an engine that has already given the whole device to its own
 * KV-cache pool, a plugin that lives inside another framework's memory budget,
 * a process whose allocator is frozen after warm-up. pd_create calls cudaMalloc
 * and is therefore closed to them; this function needs no context. It computes
 * what pd_decode_attn computes, within the same tolerances (the ranges are one
 * level of equal size, one per worker warp, so that the number of partials is
 * known in advance; the summation order and hence the last bits differ), with
 * the kernels' scratch (fp32 partials, page prefix sums, plan and status words)
 * held in a fixed 16 MiB array inside the library image. Every device that loads the
 * library carries that array until the process exits. The function calls no
 * cudaMalloc, cudaFree or allocating library routine.
 *
 * Geometry comes from *cfg (num_q_heads, num_kv_heads, head_dim, page_size,
 * max_pages_per_seq, num_pages, device; max_batch and flags are ignored); the
 * tensors are the caller's, as for pd_decode_attn. Limit: the partials must fit
 * the fixed array, i.e. (SM count * 8 + batch * num_kv_heads) * group *
 * (head_dim * 4 + 8) bytes plus 4 * (batch + 1) bytes of prefix sums and about
 * 1.5 KB of rounding and control words <= 16 MiB - on a 148-SM device batch <=
 * 860 at 32/8 heads and head_dim 128, batch <= 712 at 32/4 heads. Larger
 * batches return PD_ERR_WORKSPACE and launch nothing.
 *
 * The first call on each device resolves the array's device address and sets
 * the kernel's shared-memory attribute; make that first call outside any CUDA
 * stream capture. All calls on a device share the one array, which keeps the
 * previous call's contents (the function itself clears the few words that must
 * start at zero: the status latch and the range-claim counters): two calls whose kernels may overlap on
 * the GPU - different streams, or concurrent host threads - race on it. Issue
 * them on one stream or order them with events. There is no context to query,
 * so nothing a kernel latches is reported: an out-of-range page id is clamped
 * to page 0, a length outside [0, max_pages_per_seq * page_size] is clamped to
 * that interval, and rows whose worker gave up a bounded wait stay unwritten,
 * all silently. Callers that need those reports use pd_decode_attn.
 */
int pd_decode_attn_static(const pd_config *cfg, const void *q, const void *k_pages, const void *v_pages,
                          const int32_t *page_table, const int32_t *ctx_lens, void *out, float *lse,
                          int32_t batch, float sm_scale, void *stream);

/*
 * Waits for `stream` (pass the stream the context's kernels were issued on, so
 * that the report covers them), then reports and clears the first fault a kernel
 * of this context latched since the last call: *code is PD_OK, PD_ERR_DEVICE_FAULT or
 * PD_ERR_TIMEOUT; *seq the sequence index (or -1); *detail the offending page
 * id / position. Any of the three output pointers may be NULL. Returns *code.
 */
int pd_device_status(pd_ctx *ctx, void *stream, int32_t *code, int32_t *seq, int32_t *detail);

/* Bytes of device workspace the context holds. */
int pd_workspace_bytes(const pd_ctx *ctx, size_t *bytes);

/* Number of kernels this context has launched since pd_create. */
int pd_launch_count(const pd_ctx *ctx, int64_t *launches);

/*
 * Plan of the most recent pd_decode_attn call, read back from the device after
 * waiting for `stream`: total (sequence, KV head, page) units, pages per range
 * of the first (longest) level of ranges, number of ranges over all levels,
 * number of worker warps launched. For tests and reporting.
 */
int pd_last_plan(pd_ctx *ctx, void *stream, int64_t *total_units, int32_t *pages_per_range,
                 int32_t *num_ranges, int32_t *num_workers);

/*
 * The decode kernels' work decomposition, run on the host (no device needed; the same functions the
 * kernels execute). Units are (sequence, KV head, page) triples in that nesting order.
 * pd_plan_ranges: the plan for `total_units` units and `n_workers` worker warps under the given
 * parameters (split_pages as in pd_decode_attn; max_ranges, min_pages, halving_levels, tail_pages as a
 * context holds them: 16 * workers, 4, 6, 16 by default). *n_ranges receives the number of ranges;
 * range r covers units [starts[r], starts[r] + lens[r]). capacity = 0 only counts. The FP8 entry points
 * plan with halving_levels = 0 (one equal range per worker, 16 worker warps per SM) while the fair share
 * ceil(total_units / n_workers) is at most 1024 pages, and as above beyond that.
 * pd_plan_walk: the triples of `count` consecutive units from `first_unit`, given the exclusive prefix
 * sums of pages per sequence (cum_pages, batch + 1 entries): how a worker finds the start of a range and
 * steps through it.
 */
int pd_plan_ranges(int64_t total_units, int32_t n_workers, int32_t split_pages, int32_t max_ranges,
                   int32_t min_pages, int32_t halving_levels, int32_t tail_pages, int64_t *starts, int32_t *lens,
                   int32_t capacity, int32_t *n_ranges);
int pd_plan_walk(const int32_t *cum_pages, int32_t batch, int32_t num_kv_heads, int64_t first_unit,
                 int32_t count, int32_t *seq, int32_t *kv_head, int32_t *page);

/*
 * ---- PD decision engine (host-only, no CUDA): the paper's makespan models and plan arithmetic.
 * The decode-side inputs b and K are quantities this library measures: b is the slope of the decode
 * step time over the number of concurrent sequences (pd_fit_decode_cost on timings of pd_decode_attn),
 * K the KV bytes per token that pd_kv_gather / pd_kv_scatter move. Times in seconds, sizes in bytes.
 */
typedef struct pd_cost_model {
    double B;          /* trajectories in the rollout batch                                          */
    double S;          /* interaction turns on the slowest trajectory                                 */
    double r;          /* tokens generated per turn                                                   */
    double dL;         /* prompt tokens added per turn                                                */
    double theta;      /* bubble ratio (1 - f) / f, f = fraction of trajectories actively decoding    */
    double A;          /* fixed cost of a decode iteration (weight reads, kernel dispatch)            */
    double b;          /* marginal cost of one more concurrent sequence (KV-cache HBM reads)          */
    double t_prefill;  /* prefill time per token                                                      */
    double T_over;     /* per-turn overhead of colocation (prefill/decode switching)                  */
    double T_env;      /* environment interaction time                                                */
    double K_bytes;    /* KV transfer volume per token                                                */
    double BW;         /* bandwidth between the prefill and decode pools, bytes per second            */
    double K_seq_bytes;/* KV-cache size per trajectory                                                */
    double H_max_bytes;/* HBM capacity per worker available to the KV cache                           */
    double prefill_tokens_per_worker; /* tokens a prefill worker absorbs per step; 0 = do not check   */
} pd_cost_model;

typedef struct pd_target {
    int32_t N_P, N_D, N_C; /* prefill, decode, colocated workers: fully colocated or fully disaggregated */
    double makespan;       /* predicted batch makespan of this configuration                             */
} pd_target;

/* Eq. 1: colocated makespan on N workers. NaN on invalid input. */
double pd_makespan_coloc(const pd_cost_model *m, int32_t N);
/* Eq. 2-3: T_dis = max(T_prefill, T_decode) + T_env; the two paths are returned if the pointers are set. */
double pd_makespan_disagg(const pd_cost_model *m, int32_t N_P, int32_t N_D, double *T_prefill, double *T_decode);
/* Capacity constraints of Sec. 4.2: B K_seq <= N_D H_max, and B S dL <= N_P prefill_tokens_per_worker. */
int32_t pd_feasible_disagg(const pd_cost_model *m, int32_t N_P, int32_t N_D);
/*
 * Online decision (Sec. 4.3.2): enumerates N_P in [1, N_k - 1] over the feasible splits, compares the
 * best with colocation and returns the configuration of minimal predicted makespan. With `current` set,
 * mode-dependent hysteresis applies: an alternative is admitted only if its predicted makespan is lower
 * than the current one by more than threshold x current makespan (strictly), the threshold being
 * ratio_threshold for another ratio of the current mode and mode_threshold for a colocation <->
 * disaggregation switch; the best admitted alternative is returned (a refused mode switch does not block a
 * ratio adjustment that clears ratio_threshold), else `current` with its makespan. A current
 * configuration that is infeasible or sized for another N_k forces the switch to the overall minimum.
 * The paper publishes no threshold values and does not say whether the gain is absolute or relative;
 * they are parameters and the gain is relative here.
 */
int pd_decide(const pd_cost_model *m, int32_t N_k, const pd_target *current, double ratio_threshold,
              double mode_threshold, pd_target *out);
/*
 * Minimal-change plan (Eq. 5-6). Slots are stable worker ids 0 .. n_slots-1; cur_active / dst_active
 * flag membership in the current and target active sets, cur_role[w] in [0, n_roles) is the role of a
 * currently active worker, dst_role_count[r] the number of workers role r needs (their sum must equal
 * the target set's size). new_role[w] receives the role of every target worker (-1 elsewhere):
 * survivors keep their role up to its target count, the rest of the deficits go to survivors that must
 * switch and then to joining workers. *d_worker = joins + departures, *d_role = survivors that switch.
 */
int pd_min_change_plan(const int32_t *cur_active, const int32_t *cur_role, const int32_t *dst_active,
                       int32_t n_slots, const int32_t *dst_role_count, int32_t n_roles, int32_t *new_role,
                       int32_t *d_worker, int32_t *d_role);
/* Eq. 7: borrow training GPUs iff (R / B) (T_ded - T_full) > T_toggle. */
int32_t pd_toggle_gate(double R, double B, double T_ded, double T_full, double T_toggle);
/* Least-squares line step_seconds = A + b * concurrency over n >= 2 measurements. */
int pd_fit_decode_cost(const double *concurrency, const double *step_seconds, int32_t n, double *A, double *b);

/* ---- FP8 KV pages. The paper has no counterpart (its decode cost b is the KV-cache HBM read per
 * concurrent sequence, Eq. 1; one byte per cached value halves it); the format is this library's:
 *   k8, v8     [num_pages][num_kv_heads][16][head_dim] bytes, OCP FP8 E4M3 (bias 7, no infinities,
 *              0x7f / 0xff = NaN, largest finite value 448), device, 16-byte aligned
 *   kv_scales  [num_pages][num_kv_heads][4] fp32 = {k_scale, v_scale, 0, 0}, device, 16-byte aligned
 * and K_t = k_scale * e4m3(byte), V_t = v_scale * e4m3(byte). head_dim 64 or 128.
 */

/*
 * Quantises every (page, KV head) tile of the bf16 pools: amax over the first tokens_in_page[page]
 * slots (device int32 [num_pages], 0..16; NaN ignored), scale = amax / 448 in fp32 (1 if amax = 0),
 * code = e4m3(x / scale) with IEEE fp32 division, round to nearest even, saturating; slots past
 * tokens_in_page are written as 0. Covers all cfg.num_pages pages.
 */
int pd_kv_quantize_pages(pd_ctx *ctx, const void *k_pages, const void *v_pages, const int32_t *tokens_in_page,
                         void *k8, void *v8, float *kv_scales, void *stream);

/*
 * One-token append into FP8 pools; positions, skipping and error reporting as pd_kv_append. A token
 * that opens a page (slot 0) sets that page's k_scale and v_scale from its own rows,
 * scale = (amax * 2) / 448 (1 if amax = 0): a factor two of headroom for the 15 tokens that follow.
 * Any other token is quantised with the page's stored scales and saturates at +-448.
 */
int pd_kv_append_fp8(pd_ctx *ctx, const void *k_new, const void *v_new, void *k8, void *v8, float *kv_scales,
                     const int32_t *page_table, int32_t *ctx_lens, int32_t batch, uint32_t call_flags,
                     void *stream);

/*
 * pd_decode_attn over FP8 pools: same outputs, plan, split_pages meaning, error behaviour and
 * bit-reproducibility. q is bf16 with |q| below the fp16 range (65504): the products run in fp16 with
 * fp32 accumulation, scales are applied in fp32.
 */
int pd_decode_attn_fp8(pd_ctx *ctx, const void *q, const void *k8, const void *v8, const float *kv_scales,
                       const int32_t *page_table, const int32_t *ctx_lens, void *out, float *lse,
                       int32_t batch, float sm_scale, int32_t split_pages, void *stream);

/*
 * pd_decode_step for FP8 pools: pd_kv_append_fp8 (advancing) followed by pd_decode_attn_fp8, enqueued by one
 * call (append, split and merge kernels; a split kernel that also quantised the new token measured slower and
 * is not built). Arguments are validated before anything is enqueued; results are those of the two calls.
 * ctx_lens holds the lengths BEFORE the append on entry. Errors as pd_kv_append_fp8 and pd_decode_attn_fp8.
 */
int pd_decode_step_fp8(pd_ctx *ctx, const void *q, const void *k_new, const void *v_new, void *k8, void *v8,
                       float *kv_scales, const int32_t *page_table, int32_t *ctx_lens, void *out, float *lse,
                       int32_t batch, float sm_scale, int32_t split_pages, void *stream);

/*
 * pd_kv_gather / pd_kv_scatter for FP8 pools: a packed page is the K block, the V block (num_kv_heads *
 * 16 * head_dim bytes each) and the page's num_kv_heads scale records (16 bytes each), so the scales
 * travel with their page. K = 2 * num_kv_heads * head_dim + num_kv_heads bytes per token per layer.
 * Everything else as the bf16 calls.
 */
int pd_kv_gather_fp8(pd_ctx *ctx, const void *k8, const void *v8, const float *kv_scales, const int32_t *page_table,
                     const int32_t *page_begin, const int32_t *page_end, const int64_t *packed_page_offset,
                     void *packed, int32_t batch, void *stream);
int pd_kv_scatter_fp8(pd_ctx *ctx, const void *packed, const int64_t *packed_page_offset, void *k8, void *v8,
                      float *kv_scales, const int32_t *page_table, const int32_t *page_begin,
                      const int32_t *page_end, int32_t batch, void *stream);

/* ---- Elastic KV pool on CUDA virtual memory management (Sec. 4.6: the intra-scale toggle keeps the
 * rollout process and swaps device state; Sec. 5: the KV cache is released when training begins and
 * restored when the GPU is available again). A pool is a device address range of `capacity` bytes whose
 * first `resident` bytes are backed by physical memory, in chunks. Resizing changes the backing only:
 * the base address, and with it page ids, pointers and tensor maps derived from it, stay valid across
 * release and restore. Contents of a chunk are lost when it is released; a restored chunk holds
 * unspecified bytes. The non-resident part of the range must not be accessed (the caller's page
 * allocator must hand out only pages below resident_bytes). The wall time of pd_pool_resize(pool, 0)
 * plus pd_pool_resize(pool, capacity) is the KV-cache share of T_toggle in Eq. 7.
 * Host calls, synchronous; not thread-safe per pool. */
typedef struct pd_pool pd_pool; /* opaque */

/* Reserves the address range on `device`; nothing is resident yet. chunk_bytes = 0 picks 256 MiB; it is
 * rounded up to the device's allocation granularity and capacity up to a whole number of chunks.
 * PD_ERR_UNSUPPORTED if the driver lacks the virtual-memory calls. */
int pd_pool_create(int32_t device, uint64_t capacity_bytes, uint64_t chunk_bytes, pd_pool **out);
/* Makes ceil(resident_bytes / chunk) chunks resident, releasing or backing chunks at the end of the
 * resident prefix. Before chunks are released the call waits for `stream_to_drain` (a cudaStream_t as
 * void*; NULL = the whole device), so no kernel still touches them. PD_ERR_WORKSPACE when the device has
 * no memory for a chunk (the chunks backed so far stay resident), PD_ERR_INVALID_ARG above capacity. */
int pd_pool_resize(pd_pool *pool, uint64_t resident_bytes, void *stream_to_drain);
/* Device pointer to the start of the range (256-byte aligned at least), fixed for the pool's lifetime. */
void *pd_pool_base(const pd_pool *pool);
uint64_t pd_pool_capacity(const pd_pool *pool);
uint64_t pd_pool_chunk_bytes(const pd_pool *pool);
uint64_t pd_pool_resident_bytes(const pd_pool *pool);
const char *pd_pool_last_error(const pd_pool *pool);
/* Synchronises the device, releases every chunk and the address range. NULL is accepted. */
int pd_pool_destroy(pd_pool *pool);

const char *pd_status_string(int status);

/* Text of the most recent failure recorded by this context (CUDA error string
 * included where one exists); owned by the context, valid until the next call. */
const char *pd_last_error(const pd_ctx *ctx);
int pd_version(void);

#ifdef __cplusplus
}
#endif
#endif /* PD_H */
