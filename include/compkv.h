/*
 * compkv.h -- C ABI of the CompKV decode-step library for NVIDIA B200 (sm_100a).
 *
 * The library implements the decode hot path of compensation-aware block-sparse
 * attention over a paged KV cache:
 *   per-block summaries {|b|, mean key, grouped key variance, mean value}  (Sec. 4.1-4.2, Eq. 8)
 *   -> per-query block score S_b = sum_g phat_{g,b} * sigma_hat^2_{g,b}    (Eq. 8-10)
 *   -> mandatory blocks + stable top-k under a token budget                (Eq. 11)
 *   -> exact attention on the selected blocks, block-mean compensation for
 *      every other block, one shared softmax normaliser                    (Eq. 12)
 * plus a dense decode attention over the same cache (Eq. 12 with every block selected).
 *
 * Conventions
 *   - Every pointer documented "device" is device memory owned by the caller; "host" is
 *     host memory.  The library allocates NO device memory: summaries and scratch live in
 *     two caller-provided device buffers sized by ckv_query_sizes().  A ckv_ctx is a small
 *     host object.
 *   - All calls that take a stream enqueue work on it and return without synchronising
 *     (ckv_step_host and ckv_read_status synchronise the stream before returning).
 *   - One context is used from one stream at a time: every call works in the context's workspace (block terms,
 *     partials, split counters, staging) and some keep per-call state in the host object, so two calls on the
 *     same context must not overlap on the GPU, nor be issued from two host threads at once.  Use one context
 *     per concurrent stream; contexts are independent.
 *   - Return value: 0 (CKV_OK) or a negative ckv_status.  Nothing throws or aborts.
 *     Problems only the device can see (a page id outside the pool, a sequence that outgrew
 *     its page table, a non-finite score) set a bit in a device status word and the
 *     offending access is skipped; read it with ckv_read_status().
 *   - One "unit" = one sequence x one KV head, with the G = num_q_heads / num_kv_heads query
 *     heads that share it; a selected block set is shared by those G heads (Sec. 3.1).
 *   - Blocks are cut from token 0 in fixed size block_size; the last block of a sequence may
 *     be partial.  X_s = ceil(N_s / block_size) blocks in sequence s.
 *
 * Tensor layouts (row-major, innermost last)
 *   K / V pools  [num_pages][num_kv_heads][page_size][head_dim]   kv_dtype (bf16, or fp32 in the debug layout)
 *   page_table   [batch][max_pages_per_seq] int32, max_pages_per_seq = max_blocks_per_seq * block_size / page_size
 *   seq_lens     [batch] int32
 *   q, out       [batch][num_q_heads][head_dim]                   kv_dtype
 *   k_new, v_new [batch][num_kv_heads][head_dim]                  kv_dtype
 *   sel_ids      [batch][num_kv_heads][K_cap] int32, K_cap = budget_tokens / block_size, ascending, padded with -1
 *   sel_cnt      [batch][num_kv_heads] int32
 *   lse          [batch][num_q_heads] fp32 (natural log of the shared normaliser), may be NULL
 */
#ifndef COMPKV_H_
#define COMPKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st *ckv_stream;   /* a cudaStream_t */
typedef struct ckv_ctx ckv_ctx;

enum ckv_dtype { CKV_BF16 = 0, CKV_F32 = 1 };

enum ckv_status {
  CKV_OK = 0,
  CKV_ERR_INVALID_ARG = -1,       /* NULL pointer, batch out of range, ... */
  CKV_ERR_BAD_LAYOUT = -2,        /* a ckv_layout field outside what the kernels support */
  CKV_ERR_BUDGET_TOO_SMALL = -3,  /* budget cannot hold the mandatory blocks (Eq. 11 needs K >= |F|) */
  CKV_ERR_CAPACITY = -4,          /* a caller buffer is smaller than ckv_query_sizes() asks for */
  CKV_ERR_CUDA = -5,              /* a CUDA runtime call failed; ckv_last_cuda_error() has the code */
  CKV_ERR_TIMEOUT = -6            /* reserved: a bounded device-side wait ran out */
};

/* bits of the device status word */
enum ckv_device_status {
  CKV_DEV_BAD_PAGE = 1,     /* page table entry outside [0, num_pages): the page was skipped */
  CKV_DEV_SEQ_FULL = 2,     /* append past max_blocks_per_seq * block_size: the token was dropped */
  CKV_DEV_NONFINITE = 4,    /* a block score was NaN/Inf: it was ranked as 0 */
  CKV_DEV_TIMEOUT = 8,      /* a bounded wait inside a kernel ran out: the step's results are invalid */
  CKV_DEV_BAD_COPY = 16     /* a kernel refused to issue a bulk copy whose arguments failed its checks */
};

/* Bits of ckv_layout.variant: the scorer / merge ablations of Sec. 5.3 and App. A.6.  0 is the method as printed. */
enum ckv_variant {
  CKV_VARIANT_FIRST_ORDER_MASS = 1,  /* estimated mass without the sigma^2/2 term of Eq. 9 */
  CKV_VARIANT_RANK_BY_MASS = 2,      /* S_b = sum_g p_hat (no outer variance factor in Eq. 10) */
  CKV_VARIANT_DROP = 4               /* unselected blocks are dropped: no mean compensation in Eq. 12 */
};

typedef struct ckv_layout {
  int32_t num_q_heads;        /* multiple of num_kv_heads; G = ratio in {1, 2, 4, 8} */
  int32_t num_kv_heads;
  int32_t head_dim;           /* 128 */
  int32_t block_size;         /* 16, 32 or 64 tokens; multiple of page_size (Sec. 5.1 uses 16) */
  int32_t page_size;          /* 16 */
  int32_t var_groups;         /* r of Eq. 8: a power of two dividing head_dim/2, or head_dim */
  int32_t group_layout;       /* coordinate groups of App. A.4: 0 = RoPE pair p is (2p, 2p+1), i.e. groups are
                                 contiguous coordinate ranges; 1 = pair p is (p, p + head_dim/2) */
  int32_t kv_dtype;           /* CKV_BF16, or CKV_F32 (debug layout: fp32 pools, q and out) */
  int32_t max_batch;
  int32_t max_blocks_per_seq; /* page-table row stride is max_blocks_per_seq * block_size / page_size */
  int32_t num_pages;          /* pages in each pool; page ids are range-checked against it */
  int32_t sink_blocks;        /* mandatory leading blocks (Sec. 4.2: 1) */
  int32_t recent_blocks;      /* mandatory trailing blocks (Sec. 4.2: 2) */
  float   sm_scale;           /* logit scale; 0 means 1/sqrt(head_dim) (Sec. 3.1) */
  int32_t variant;            /* OR of ckv_variant bits; 0 = the method as printed */
  int32_t stat_bf16;          /* 0: mean keys / mean values kept at fp32 precision (the paper's choice, Sec. 4.3).  A
                                 decode step reads the mean keys and variances in full; with kv_dtype CKV_BF16 and
                                 var_groups 4 it reads the mean values at bf16 precision (the compensation term of
                                 Eq. 12 ends in a bf16 output row; the stored summaries keep their precision);
                                 1: kept as bf16 (half the summary bytes; block scores then differ from the fp32
                                 layout's by up to ~1e-2 relative).  Needs kv_dtype CKV_BF16 and
                                 var_groups < head_dim.  Variances stay fp32. */
} ckv_layout;

/* Library version (major * 100 + minor). */
int ckv_version(void);

/* Human-readable name of a ckv_status (static storage). */
const char *ckv_strerror(int status);

/* cudaError_t of the last failed CUDA call made by this library on the calling thread (0 if none). */
int ckv_last_cuda_error(void);

/* Sizes in bytes of the two device buffers a context needs (Sec. 4.2: 2d + r + 1 scalars per
 * block; the count |b| is implied by seq_lens, so 2d + r 32-bit scalars are stored).
 * stats_bytes: block summaries for max_batch sequences.  workspace_bytes: scratch for one
 * decode step at max_batch (block log-weights, scores, split partials, host staging).
 * Host-only; validates the layout (CKV_ERR_BAD_LAYOUT).  Besides the per-field ranges a layout must keep
 * max_batch * num_kv_heads <= 65535, max_blocks_per_seq * block_size <= 2^30, and
 * max_batch * num_kv_heads * ceil(max_blocks_per_seq / 32) < 2^24 (the kernels' index arithmetic is exact below that;
 * summaries of that many blocks would need half a terabyte). */
int ckv_query_sizes(const ckv_layout *layout, size_t *stats_bytes, size_t *workspace_bytes);

/* Byte offsets, inside the stats buffer, of its three regions (the "selection region" holds
 * mean keys and grouped variances, the "mean-values region" the mean values; Sec. 4.3):
 *   kmean [max_batch][num_kv_heads][max_blocks_per_seq] rows of 512 bytes
 *   dbar  [max_batch][num_kv_heads][max_blocks_per_seq][var_groups] fp32
 *   vmean [max_batch][num_kv_heads][max_blocks_per_seq] rows of 512 bytes
 * A mean-key / mean-value row holds its 128 entries as split bf16 pairs (hi = bf16(x),
 * lo = bf16(x - hi): 32 bits per entry, relative error <= 2^-18) in a bank-swizzled chunk
 * order private to the kernels; use ckv_stats_export() to read summaries.  Host-only. */
int ckv_stats_offsets(const ckv_layout *layout, size_t *kmean_off, size_t *dbar_off, size_t *vmean_off);

/* Create a context over caller-owned device buffers (256-byte aligned, at least the sizes
 * ckv_query_sizes() returned; the buffers must outlive the context).  Clears the device
 * status word on `stream`.  *out receives a host object to be freed with ckv_destroy(). */
int ckv_create(const ckv_layout *layout, void *stats_dev, size_t stats_bytes, void *work_dev,
               size_t work_bytes, ckv_stream stream, ckv_ctx **out);
void ckv_destroy(ckv_ctx *ctx);

/* Build the summaries of every block of `batch` prefilled sequences from the paged cache
 * (Eq. 8 right half; Sec. 4.2): |b|, mean key, mean value and, per coordinate group, the
 * population variance of the keys around the block mean (fp32: two passes over each 16-token page, mean first and
 * deviations from it second; the pages of a longer block are joined with the pairwise update of Chan et al.).
 * Sequence s of this call uses summary rows of batch slot s.
 * max_seq_len_host: an upper bound (host) on seq_lens[s], used only to size the grid. */
int ckv_stats_build(ckv_ctx *ctx, const void *k_pool, const void *v_pool, const int32_t *page_table,
                    const int32_t *seq_lens, int batch, int max_seq_len_host, ckv_stream stream);

/* Write the summaries of `batch` sequences as plain fp32 arrays (device):
 *   kmean, vmean [batch][num_kv_heads][max_blocks_per_seq][head_dim], dbar [...][var_groups].
 * Rows at or past X_s are unspecified.  For inspection and tests. */
int ckv_stats_export(ckv_ctx *ctx, int batch, float *kmean, float *dbar, float *vmean, ckv_stream stream);

/* Append one token per sequence (Sec. 4.2 "updated incrementally", App. D.1): writes
 * k_new / v_new at position seq_lens[s] of the paged cache, recomputes the summary of the
 * active (last) block from its resident tokens with the same arithmetic as ckv_stats_build
 * (so build(N) + appends == build(N + m) bit for bit), leaves completed blocks untouched, and
 * increments seq_lens[s].  The page table must already map the page of the new position. */
int ckv_append(ckv_ctx *ctx, void *k_pool, void *v_pool, const int32_t *page_table, int32_t *seq_lens,
               const void *k_new, const void *v_new, int batch, ckv_stream stream);

/* One compensated sparse decode step (Eq. 8-12) for `batch` sequences, one query token each.
 *   budget_tokens: exact-read budget in tokens, mandatory blocks included (Sec. 5.1);
 *                  K = budget_tokens / block_size blocks; K >= X_s selects every block of s,
 *                  which makes the result dense attention.
 *   out:     attention output, kv_dtype (fp32 accumulation, rounded once; App. D.1).
 *   sel_ids: selected block ids per unit in position order; sel_cnt their number.
 * The cache is read through page_table; summaries must be current (build / append).
 * Returns CKV_ERR_BUDGET_TOO_SMALL when K < sink_blocks + recent_blocks and K * block_size <
 * max_seq_len_host (some sequence could not hold its mandatory blocks). */
int ckv_decode(ckv_ctx *ctx, const void *q, const void *k_pool, const void *v_pool,
               const int32_t *page_table, const int32_t *seq_lens, int batch, int max_seq_len_host,
               int budget_tokens, void *out, float *lse, int32_t *sel_ids, int32_t *sel_cnt,
               ckv_stream stream);

/* Chunked prefill: append new_lens[s] tokens to sequence s from contiguous rows and bring the summaries of every
 * block they touch up to date, in one pass (Sec. 4.2: summaries are built as the cache is filled; the new keys and
 * values are read once, not written first and read back by ckv_stats_build).
 *   k_src, v_src: [batch][src_stride_tokens][num_kv_heads][head_dim], device, kv_dtype; row t of sequence s is the
 *                 token at position seq_lens[s] + t.
 *   new_lens:     int32 [batch] (device), 0 .. src_stride_tokens; max_new_host >= every new_lens[s] (host, sizes the grid).
 *   seq_lens:     holds N on entry and N + new_lens once the call has run.  Tokens past the capacity
 *                 max_blocks_per_seq * block_size are dropped and CKV_DEV_SEQ_FULL is set.
 * The page table must already map the pages of the new positions.  A chunk may start and end anywhere inside a
 * block; the result equals ckv_append called once per token, and ckv_stats_build over the filled cache, bit for bit.
 * Uses the context's split counters: not to be overlapped with a decode call on another stream. */
int ckv_prefill(ckv_ctx *ctx, void *k_pool, void *v_pool, const int32_t *page_table, int32_t *seq_lens,
                const void *k_src, const void *v_src, const int32_t *new_lens, int src_stride_tokens, int batch,
                int max_new_host, ckv_stream stream);

/* One decode step in one call: the results, the cache, the summaries, the lengths and the errors are those of
 * ckv_append(k_new, v_new) followed by ckv_decode(q, ...), bit for bit (Sec. 4.3: the new token enters the cache
 * and the summaries before blocks are selected; seq_lens holds N on entry and N + 1 once the step has run;
 * max_seq_len_host bounds the lengths after the append).  It is three launches, not four: a step can only change
 * the last block of a sequence, so a few CTAs of the scan launch write the new rows and redo that block's summary
 * while the other CTAs stream the summaries of all the other blocks; seq_lens is updated inside that launch, after
 * every CTA has read it.  (Batches above 1024 sequences take the two-call route.)  The decode arguments are
 * validated before anything is appended. */
int ckv_step(ckv_ctx *ctx, const void *q, const void *k_new, const void *v_new, void *k_pool, void *v_pool,
             const int32_t *page_table, int32_t *seq_lens, int batch, int max_seq_len_host, int budget_tokens,
             void *out, float *lse, int32_t *sel_ids, int32_t *sel_cnt, ckv_stream stream);

/* Dense decode attention over the whole paged cache (Sec. 3.1; Eq. 12 with S = all blocks),
 * split along the sequence with a log-sum-exp merge.  Same tile code as the sparse path. */
int ckv_dense_decode(ckv_ctx *ctx, const void *q, const void *k_pool, const void *v_pool,
                     const int32_t *page_table, const int32_t *seq_lens, int batch, int max_seq_len_host,
                     void *out, float *lse, ckv_stream stream);

/* Dense decode attention without a context and without any caller-provided scratch.  (The paper has no
 * counterpart: this entry point exists for hosts that cannot give the library device memory to work in -- a
 * plugin handed only the operation's own tensors, code under a memory pool or a capture that forbids
 * cudaMalloc, a process whose device memory is already committed to the KV cache.)
 * Same inputs, outputs and result as ckv_dense_decode(), with `layout` passed directly.  The split partials
 * live in a fixed device array inside the library image (4 MiB + 1 KiB, held by every GPU that loads the
 * library until the process exits); the call allocates nothing.  Two limits, checked before anything is
 * launched (CKV_ERR_CAPACITY): batch * num_q_heads * 528 B * 64 must fit in 4 MiB, and batch * num_kv_heads must
 * not exceed 192 (one split counter per unit in the last KiB).  All calls share that array: calls that overlap
 * on the GPU (other streams, other host threads) race on it, so serialise them.  The first call on a device
 * looks up the array's device address, and the first call with a given (device, group size, kv_dtype) sets the
 * attributes of that layout's kernels: make those calls outside any stream capture.  Unlike the context calls,
 * this one has no way of returning what only the device can see: a page id outside the pool is skipped (the
 * page contributes nothing) and the status word that records it, which lives in the array, is cleared by the
 * next call unread.  A failed CUDA call returns CKV_ERR_CUDA and leaves its code for ckv_last_cuda_error(). */
int ckv_dense_decode_static(const ckv_layout *layout, const void *q, const void *k_pool, const void *v_pool,
                            const int32_t *page_table, const int32_t *seq_lens, int batch, int max_seq_len_host,
                            void *out, float *lse, ckv_stream stream);

/* Diagnostic, not part of the decode step: exact per-block logit statistics of every query head over the whole
 * cache (Eq. 3; App. B.1).  For sequence s, query head g and block b < ceil(N_s / block_size) the kernel writes, at
 * [s][g][b] of three device fp32 arrays shaped [batch][num_q_heads][max_blocks_per_seq],
 *   logZ  = log sum_{j in b} exp(z_j),  zmean = mean_{j in b} z_j,  zvar = population variance of z_j,
 * with z_j = sm_scale * q_g . k_j.  Entries of blocks past a sequence's end are left untouched.  Exact block masses,
 * compensation residuals and the KL divergences of a selection follow from these by block-level arithmetic
 * (paper_2609_26300_b200/diagnostics.py).  Reads every key once: as expensive as a dense decode. */
int ckv_exact_blocks(ckv_ctx *ctx, const void *q, const void *k_pool, const int32_t *page_table,
                     const int32_t *seq_lens, int batch, int max_seq_len_host, float *logZ, float *zmean,
                     float *zvar, ckv_stream stream);

/* Copy the block scores S_b of the last ckv_decode (Eq. 10) into dst (device),
 * fp32 [batch][num_kv_heads][max_blocks_per_seq]; entries at or past X_s are unspecified.
 * Mandatory blocks carry their score too (they are excluded from the ranking, not from Eq. 9). */
int ckv_copy_scores(ckv_ctx *ctx, float *dst, int batch, ckv_stream stream);

/* One whole decode step from HOST buffers: brings q, k_new, v_new to the device, runs ckv_step,
 * brings out / sel_ids / sel_cnt back and returns when they are complete in the caller's buffers
 * (all work the call put on the stream has then finished).  Host buffers should be pinned: buffers the
 * device can address (pinned, registered or managed memory, 16-byte aligned) are moved by two small
 * kernels of the library and the call waits on a pinned word its last kernel stores; pageable buffers
 * take six copies and a stream synchronisation (about 20 us more per call).  A caller that comes back with the
 * same buffers, arrays and sizes on a stream of its own (not the default stream, not a capturing one) has its
 * second such call captured as a CUDA graph and the later ones replayed (the length bound is rounded up to a
 * multiple of 1024 inside, so the graph lasts that many steps); the graph is the context's and goes with it.
 * Device staging comes out of the workspace.  seq_lens (device) is incremented.  max_seq_len_host bounds the lengths AFTER the append.  The id staging area holds
 * max_blocks_per_seq ids per unit: budget_tokens / block_size beyond that is CKV_ERR_INVALID_ARG. */
int ckv_step_host(ckv_ctx *ctx, const void *q_host, const void *k_new_host, const void *v_new_host,
                  void *k_pool, void *v_pool, const int32_t *page_table, int32_t *seq_lens, int batch,
                  int max_seq_len_host, int budget_tokens, void *out_host, int32_t *sel_ids_host,
                  int32_t *sel_cnt_host, ckv_stream stream);

/* Read and clear the device status word (bits of ckv_device_status); synchronises `stream`. */
int ckv_read_status(ckv_ctx *ctx, int32_t *host_status, ckv_stream stream);

/* How the decode step treats the last block of every sequence (the only block a step can change).  In "tail
 * mode" a few CTAs of the scan launch own that block -- and, in ckv_step, append the new token to it inside the
 * same launch -- while the other CTAs stream the remaining summaries; otherwise the scan covers every block and
 * ckv_step appends in a launch of its own.  The results agree to rounding (the last block's two per-head terms are
 * computed by different code); tail mode is the faster one once the scan runs for tens of microseconds.
 * mode: CKV_TAIL_AUTO (default: chosen per call from the batch and max_seq_len_host), CKV_TAIL_OFF, CKV_TAIL_ON
 * (honoured up to 1024 sequences).  Returns CKV_ERR_INVALID_ARG for a null context or an unknown mode. */
enum ckv_tail_mode { CKV_TAIL_AUTO = 0, CKV_TAIL_OFF = 1, CKV_TAIL_ON = 2 };
int ckv_set_tail_mode(ckv_ctx *ctx, int mode);

/* ---- measurement ---------------------------------------------------------------------------------------------
 * Not part of the decode path: these calls exist so that a benchmark can time the library's own launches with
 * CUDA events on the launching stream, and count them. */

/* ckv_decode with CUDA events recorded on `stream` between its four kernels (summary scan, score +
 * top-k selection, exact attention on the selected blocks, merge; the bf16 layout merges inside the attention
 * kernel, its fourth duration is then an empty interval).  Waits for the step to finish and writes the four
 * durations in milliseconds to stage_ms_host[0..3] (host).  For measurement only. */
int ckv_decode_profile(ckv_ctx *ctx, const void *q, const void *k_pool, const void *v_pool,
                       const int32_t *page_table, const int32_t *seq_lens, int batch, int max_seq_len_host,
                       int budget_tokens, void *out, float *lse, int32_t *sel_ids, int32_t *sel_cnt,
                       ckv_stream stream, float *stage_ms_host);

/* The summary scan of ckv_decode (Eq. 8-10 logits and the all-block compensation sums of Eq. 12) launched
 * `reps` times back to back between two CUDA events on `stream`; waits, and writes the average duration of
 * one launch in milliseconds to *avg_ms_host (host).  The scan only rewrites its own workspace rows, so the
 * repetitions are idempotent; the summaries of the bench workloads exceed L2, so every launch streams them
 * from HBM.  For measurement only (the roofline figure of the dominant kernel). */
int ckv_scan_profile(ckv_ctx *ctx, const void *q, const int32_t *seq_lens, int batch, int max_seq_len_host,
                     int reps, ckv_stream stream, float *avg_ms_host);

/* Number of kernel launches the library has enqueued through this context so far. */
int64_t ckv_launch_count(const ckv_ctx *ctx);

/* ---- test hook ------------------------------------------------------------------------------------------------
 * Every wait inside a kernel is bounded: after a number of polls it gives up, sets CKV_DEV_TIMEOUT, drains the
 * copies it has in flight and the launch returns -- nothing traps and nothing waits for ever.  ckv_debug_set() lets
 * a test make that happen without a fault: spin_limit replaces the number of polls (0 restores the default, 2^22),
 * and CKV_DEBUG_SKIP_FILL makes the producer thread of the summary scan's first CTA announce its first
 * shared-memory fill and never issue it, so that the waits on it run out.  The decode step that follows reports
 * CKV_DEV_TIMEOUT through ckv_read_status() and its results are invalid; with the flag cleared the next step is
 * correct again.  The paper has no counterpart.  Not for production use. */
enum ckv_debug_flags { CKV_DEBUG_SKIP_FILL = 1 };
int ckv_debug_set(ckv_ctx *ctx, uint32_t spin_limit, int flags);

#ifdef __cplusplus
}
#endif
#endif /* COMPKV_H_ */
