/*
 * pd_debug.h - measurement hooks of the paged decode-attention library.
 *
 * Not part of the operations of pd.h (the paper has no counterpart for them):
 * a one-shot CUDA-event bracket around the split kernel, which benchmarks use
 * to time the kernel that the KV-read term b of Eq. 1 is spent in, and a
 * per-worker timestamp trace for profiling builds. Conventions as in pd.h.
 */
#ifndef PD_DEBUG_H
#define PD_DEBUG_H

#include "pd.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Timing hook for benchmarks: the NEXT pd_decode_attn of this context records
 * `before` on its stream just ahead of the split kernel and `after` right behind
 * it (both cudaEvent_t passed as void*, owned by the caller, who must keep them
 * alive until the work has run), then the hook clears itself. That call launches
 * its kernels without programmatic overlap, so the events bracket the split
 * kernel alone, not the merge. Two event records cost several microseconds of
 * stream time: hook a sample of the steps, not all of them. Passing two NULLs
 * cancels a pending hook.
 */
int pd_set_profile_events(pd_ctx *ctx, void *before, void *after);

/*
 * Per-worker timestamps of the most recent pd_decode_attn, for profiling the
 * start-up and tail of the split kernel. Available only in a library built
 * with -DPD_ENABLE_TUNING when the environment variable PD_TRACE_WORKERS=1 was
 * set at pd_create (otherwise PD_ERR_UNSUPPORTED; the shipped build reads no
 * environment variable). Waits for `stream`, then copies up to max_workers
 * records of four uint64 nanosecond values (%globaltimer: kernel entry, first
 * tile landed, last tile landed, exit) to host_out (HOST pointer) and stores
 * the number of records in *num_workers. After a pd_prefill_attn the same
 * buffer holds, per CTA (in launch order) and as four consecutive records, the
 * SM-clock cycles row thread 0 spent waiting for S, loading S, in the softmax
 * arithmetic, waiting for O, storing P, in total, and its block count.
 */
int pd_read_worker_trace(pd_ctx *ctx, void *stream, uint64_t *host_out, int32_t max_workers, int32_t *num_workers);

/*
 * How many pd_decode_step_host calls of this context delivered their result straight into the caller's pinned
 * host buffer (the merge kernel stores the rows and raises a pinned flag the call polls) and how many staged it
 * on the device and copied it back. Either pointer may be NULL.
 */
int pd_host_step_counts(const pd_ctx *ctx, int64_t *direct, int64_t *staged);

/*
 * Read-only streaming probe: launches a kernel of `blocks` x `threads` that reads `bytes` (a multiple of 16
 * is read) from src once with 16-byte streaming loads and stores nothing (sink16 is a 16-byte device
 * buffer the kernel is formally allowed to write). Timed with events by the caller, it gives the read-only
 * HBM ceiling of the GPU, to set beside the copy bandwidth that serves as the roofline denominator of the
 * decode kernels (Eq. 1's b is a read). No context is needed; src and sink16 are device pointers, 16-byte aligned.
 */
int pd_read_probe(const void *src, size_t bytes, int32_t blocks, int32_t threads, void *sink16, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* PD_DEBUG_H */
