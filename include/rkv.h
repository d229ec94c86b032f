/*
 * rkv.h -- C ABI of the B200 (sm_100a) implementation of R-KV's periodic decode-time
 * KV-cache compression step.
 *
 * What one call computes, per (sequence b, KV head h), with L = seq_lens[b],
 * n = L - alpha candidate tokens (the last alpha cached tokens are the observation
 * tokens and are always kept; Section 3.1) and k = budget - alpha:
 *
 *   importance   I_i    Eq. 2-4: scaled logits of the alpha observation queries of each of
 *                       the G query heads of the group against the n candidate keys, max
 *                       over the group, ONE softmax over the keys, sliding max over the
 *                       window {i-W .. i+W-1}, mean over the alpha queries.
 *   redundancy   R_i    Eq. 5-6 and the retention rule of Section 3.3: cosine similarity
 *                       of all candidate keys, zero diagonal; per token the entries of the
 *                       (up to) beta largest positions j with S[j][i] > T are zeroed;
 *                       column mean (divided by n); softmax over the n tokens.
 *   joint score  Z_i    Eq. 7: lambda * I_i - (1 - lambda) * R_i.
 *   selection           the k candidates with the largest Z, per KV head (Section 3.4);
 *                       equal scores: the later position is kept.
 *   compaction          Algorithm 1's gather + concatenate, in place: rows [0, budget) of
 *                       K and V become the kept rows in ascending original position (the
 *                       k selected candidates, then the alpha observation tokens).
 *
 * All pointers in the signatures are DEVICE pointers unless the name starts with
 * "host_".  The library never allocates or frees device memory; scratch comes from
 * the caller through rkv_desc_t.workspace (rkv_compress_static alone uses an array
 * built into the library instead).  Calls enqueue
 * work on the given stream and do not synchronise.  Errors are return codes; nothing
 * throws or aborts.
 */
#ifndef RKV_H_
#define RKV_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define RKV_API __attribute__((visibility("default")))
#else
#define RKV_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    RKV_OK = 0,
    RKV_ERR_INVALID_ARG = 1, /* null / misaligned pointer, size out of range */
    RKV_ERR_UNSUPPORTED = 2, /* head_dim not 64 / 128 / 256, unknown dtype, cap or query group too large */
    RKV_ERR_WORKSPACE = 3,   /* workspace missing or too small */
    RKV_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed */
    RKV_ERR_TIMEOUT = 5      /* device status only: a bounded wait inside a kernel ran out */
} rkv_status_t;

/* Element type of the caches.
 *   RKV_BF16, RKV_F32: k_cache, v_cache and q_window all hold that type.
 *   RKV_FP8_E4M3: k_cache and v_cache hold 8-bit E4M3 codes (1 sign bit, 4 exponent bits with bias 7, 3 mantissa bits,
 *     no infinities; one byte per element, rows of head_dim bytes); q_window (and q_new of rkv_push_query) is bf16.
 *     Eq. 1-7 are evaluated on the values the codes stand for: the keys are widened to bf16 (exactly; every E4M3 value
 *     is a bf16 value) into the workspace, which grows by (batch * n_kv_heads * (budget + buffer) + 128) * head_dim * 2
 *     bytes (nothing more for head_dim 64, whose padded copy exists anyway), and every scoring stage runs on that copy as for a bf16 cache.  The compaction moves the stored bytes; no
 *     scale factor is applied or needed (cosine similarity does not see a per-tensor scale; fold a key scale into
 *     the queries for Eq. 2).  rkv_decode_attention takes this type too (q_new bf16): the codes are widened on their
 *     way to the tensor cores, no copy is kept. */
typedef enum { RKV_BF16 = 0, RKV_F32 = 1, RKV_FP8_E4M3 = 2 } rkv_dtype_t;

/* rkv_desc_t.flags */
#define RKV_FLAG_SIMT_SCORES 1u /* score with the plain fp32 CUDA-core kernel instead of the tcgen05
                                   kernels (always used for RKV_F32; a debugging aid for RKV_BF16) */
#define RKV_FLAG_ROWBLOCK_SCORES 2u /* bf16: score with the row-block tcgen05 kernel (forms the full similarity
                                   matrix) instead of the default two-pass kernels (every token against the last
                                   key tile first, then only the tokens still short of partners against the
                                   earlier tiles, last to first); a cross-check */

#define RKV_FLAG_MEAN_THEN_POOL 4u /* importance in Algorithm 1's order: mean over the alpha query rows first, then the
                                   pooling (read as Eq. 4's max over the same window); default is Eq. 4's order */

#define RKV_FLAG_HEAD_MEAN 8u /* Algorithm 1's aggregated selection: the joint scores of a sequence's KV heads are
                                   averaged and ONE set of positions is kept for all of them (every head's index
                                   list is the same); default is one set per KV head.  One more launch. */

#define RKV_FLAG_GQA_MEAN_POOL 16u /* Eq. 3 with the mean instead of the max over the query heads of a group (the
                                   pooling the paper's appendix ascribes to earlier work); still taken on the scaled
                                   logits, before the one softmax.  Default is the max (Eq. 3). */

#define RKV_FLAG_NO_SYMMETRIC 32u /* never take the symmetric route of the second scoring pass (by default a head in
                                   which, after the first pass, more than 4/5 of the tokens still lack their partner is
                                   scored by forming each pair of key tiles once; beta = 1 only).  A cross-check. */

/* stage bits for rkv_compress_stages */
#define RKV_STAGE_PREP 1u    /* key inverse norms and per-tile sums of normalised keys */
#define RKV_STAGE_SCORES 2u  /* Eq. 2-3 pooled logits; Eq. 5 matrix + retention rule + Eq. 6 column means */
#define RKV_STAGE_SELECT 4u  /* Eq. 3 softmax, Eq. 4, Eq. 6 softmax, Eq. 7, top-k, index list */
#define RKV_STAGE_GATHER 8u  /* in-place compaction of K and V, seq_lens update */
#define RKV_STAGE_ALL 15u

#define RKV_MAX_CAP 8192     /* largest supported budget + buffer */
#define RKV_MAX_GROUP_ROWS 112 /* largest supported (n_q_heads / n_kv_heads) * alpha */

/*
 * Problem descriptor.  Plain data, owned by the caller, copied on use.
 * Fill it with rkv_desc_default() first, then set the shape fields.
 */
typedef struct rkv_desc {
    int32_t batch;       /* sequences; layers that fire together are folded into this dimension */
    int32_t n_kv_heads;  /* KV heads per sequence */
    int32_t n_q_heads;   /* query heads; G = n_q_heads / n_kv_heads must be integral (G = 1: Eq. 1) */
    int32_t head_dim;    /* d: 64, 128 or 256.  The tensor-core scoring kernels are built for bf16 keys with d = 128;
                            bf16 and 8-bit caches with d = 64 are scored by them on a copy of the keys (and of the
                            observation queries) padded with zeros to 128 in the workspace -- dot products and norms do
                            not see the padding --; d = 256 and fp32 caches are scored by the CUDA-core kernel
                            (correct, but far slower) */
    int32_t dtype;       /* rkv_dtype_t of k_cache and v_cache (and of q_window, except for 8-bit caches: bf16) */
    int32_t pool_w;      /* W of Eq. 4; 0 = no pooling.  Range [0, 64].  Default 4 (the paper prints no value) */
    int32_t beta;        /* beta of Section 3.3; 0 = rule off.  Default 1 (the paper prints no value) */
    float sim_threshold; /* T of Section 3.3, in [0, 1].  Default 0.5 (the paper prints no value) */
    float eps;           /* epsilon of Eq. 5, >= 0.  Default 1e-8 */
    uint32_t flags;      /* RKV_FLAG_* */
    void *workspace;     /* device scratch, 256-byte aligned, >= rkv_workspace_bytes(); contents are
                            undefined between calls; two calls that overlap on the GPU need two workspaces */
    size_t workspace_bytes;
    int32_t *device_status; /* optional device int32; kernels store the first error they meet into it if it holds 0
                               (RKV_ERR_INVALID_ARG for seq_lens[b] > cap or < 0, RKV_ERR_TIMEOUT).  The caller
                               zeroes it and reads it after synchronising the stream.  The library only ever
                               writes it: a value left over from an earlier call changes nothing in a later one.
                               What a call does after an error is stated with rkv_compress below. */
    /* optional device dumps of the scores, each [batch][n_kv_heads][cap] float, first n entries written */
    float *dbg_I, *dbg_Sbar, *dbg_R, *dbg_Z;
    /* optional: 5 cudaEvent_t handles; event s is recorded before stage s (prep, scores, select, gather)
       and event 4 after the last stage, on the call's stream */
    void *const *stage_events;
    /* optional: 4 more cudaEvent_t handles that split the multi-kernel stages: recorded after the first scoring
       pass, after the listing kernel between the passes, after the row statistics and after the importance
       kernel (with a scoring kernel that is a single launch the first two coincide with the stage's start) */
    void *const *kernel_events;
    /* optional device uint64[8], written at the end of the scoring stage: [0] = 128 x 128 x 128 tile products the
       tensor-core kernels executed in this call, [2] = work items of the second scoring pass, [5] = (listed token,
       key tile) pairs the second pass had to form (its useful work: items pad the tokens to whole 128-row tiles);
       the other words are internal */
    unsigned long long *dbg_counters;
    /* limit of every bounded wait inside the kernels, in GPU clock ticks; 0 = the default (about two seconds).
       A wait that runs out is an error (RKV_ERR_TIMEOUT), never a hang.  Values below about a million ticks can
       expire during ordinary memory latency: leave it at 0 outside of tests. */
    int64_t wait_limit_cycles;
    /* optional device int32[batch]: a budget of its own for every sequence (the budget-ratio experiments of Section
       4.2: the budget as a share of each sequence's length), alpha < budgets[b] <= budget.  NULL: every sequence
       uses the call's `budget`.  The call's `budget` stays the maximum: it fixes the cache capacity (budget +
       buffer) and the row length of out_idx.  Sequence b is compressed when seq_lens[b] > budgets[b]; it keeps
       budgets[b] tokens, out_idx[b][h][budgets[b] ..] = -1, and seq_lens[b] becomes budgets[b].  A value out of
       range is treated like an invalid length: the sequence is skipped and RKV_ERR_INVALID_ARG recorded. */
    const int32_t *budgets;
    /* optional: PAGED caches (the paper's last section names the reallocation cost of paged serving frameworks as the
       method's limitation; here the compaction stays in place, page by page).  block_table is a device int32
       [batch][n_kv_heads][(budget + buffer) / 128]: the page that holds rows [128 t, 128 t + 128) of head (b, h).
       k_cache and v_cache are then page POOLS [pool_pages][128][head_dim] (same dtype, 16-byte aligned), a page
       holding 128 consecutive rows of one (sequence, KV head); budget + buffer must be a multiple of 128; the pages of
       one call must be distinct.  Every entry point that takes k_cache / v_cache follows the table (rkv_compress*,
       rkv_append, rkv_decode_attention; not rkv_compress_host).  The compaction moves rows between a head's own pages
       only and never changes the table: after a compression the head's first budget rows, in table order, are the kept
       ones.  NULL: contiguous caches as described with rkv_compress. */
    const int32_t *block_table;
    int64_t pool_pages;
} rkv_desc_t;

/* Fill *desc with the defaults above (pool_w 4, beta 1, T 0.5, eps 1e-8, head_dim 128, bf16), zero elsewhere. */
RKV_API void rkv_desc_default(rkv_desc_t *desc);

/* Bytes of device scratch a call with this descriptor and these sizes needs (0 if the arguments are invalid). */
RKV_API size_t rkv_workspace_bytes(const rkv_desc_t *desc, int32_t budget, int32_t buffer, int32_t alpha);

/* Install *desc (copied) as the calling thread's current descriptor, used by rkv_compress(). */
RKV_API int rkv_set_desc(const rkv_desc_t *desc);

/*
 * One firing of the compression step (Section 3.1; Algorithm 1) for every sequence in the batch.
 *
 *   k_cache, v_cache  [batch][n_kv_heads][cap][head_dim], cap = budget + buffer, contiguous, 16-byte aligned;
 *                     modified in place
 *   q_window          [batch][n_q_heads][alpha][head_dim]: the query states of the last alpha tokens (the
 *                     paper's query cache); query head q belongs to KV head q / G
 *   seq_lens          [batch] int32, in/out: cached length L of each sequence
 *   out_idx           [batch][n_kv_heads][budget] int32, out
 *   stream            cudaStream_t (NULL = the legacy default stream)
 *
 * For each b with budget < seq_lens[b] <= cap: rows [0, budget) of every head hold the kept rows in ascending
 * original position, rows [budget, cap) are unspecified, out_idx[b][h] lists the kept original positions
 * (ascending; the last alpha are L-alpha .. L-1) and seq_lens[b] becomes budget.
 * For seq_lens[b] <= budget (Algorithm 1's guard) nothing changes; out_idx[b][h][j] = j for j < L, -1 after.
 * seq_lens[b] > cap or < 0 cannot be seen without a sync: that sequence alone is skipped (its caches and length
 * stay as they are, out_idx[b] = -1), RKV_ERR_INVALID_ARG is stored to device_status, and every other sequence
 * of the batch is compressed as usual.
 * If a bounded wait inside a kernel runs out (RKV_ERR_TIMEOUT in device_status), the scores of the call are
 * incomplete: the remaining kernels then leave ALL caches and lengths of the batch unmodified and set every
 * entry of out_idx to -1.  The state that carries this between the kernels lives in the workspace and is reset by
 * each call, so nothing has to be cleared before the next one.
 * Requires 1 <= alpha < budget, buffer >= 1, cap <= RKV_MAX_CAP, G * alpha <= RKV_MAX_GROUP_ROWS,
 * lambda in [0, 1].  Host-detectable errors return before anything is launched.
 * Uses the thread's current descriptor (rkv_set_desc).
 */
RKV_API int rkv_compress(void *k_cache, void *v_cache, const void *q_window, int32_t *seq_lens, int32_t budget,
                 int32_t buffer, int32_t alpha, float lambda, int32_t *out_idx, void *stream);

/* The same with an explicit descriptor. */
RKV_API int rkv_compress_ex(const rkv_desc_t *desc, void *k_cache, void *v_cache, const void *q_window,
                    int32_t *seq_lens, int32_t budget, int32_t buffer, int32_t alpha, float lambda,
                    int32_t *out_idx, void *stream);

/* The same, running only the stages in stage_mask (RKV_STAGE_*); stages hand their results on through the
 * workspace, so running them one by one in order equals one full call.  For per-stage timing and tests. */
RKV_API int rkv_compress_stages(const rkv_desc_t *desc, void *k_cache, void *v_cache, const void *q_window,
                        int32_t *seq_lens, int32_t budget, int32_t buffer, int32_t alpha, float lambda,
                        int32_t *out_idx, void *stream, uint32_t stage_mask);

/*
 * End-to-end form with HOST buffers (pinned memory recommended): copies host_k_cache, host_v_cache,
 * host_q_window and host_seq_lens to device staging inside desc->workspace, runs the step, and copies back
 * rows [0, budget) of K and V of every head, seq_lens and out_idx -- all asynchronously on `stream`; the
 * results are valid once the stream is synchronised.  desc->workspace must hold rkv_host_workspace_bytes().
 * Shapes and semantics as rkv_compress.
 */
RKV_API size_t rkv_host_workspace_bytes(const rkv_desc_t *desc, int32_t budget, int32_t buffer, int32_t alpha);
RKV_API int rkv_compress_host(const rkv_desc_t *desc, void *host_k_cache, void *host_v_cache, const void *host_q_window,
                      int32_t *host_seq_lens, int32_t budget, int32_t buffer, int32_t alpha, float lambda,
                      int32_t *host_out_idx, void *stream);

/*
 * rkv_compress_ex for callers that cannot provide a workspace.  (The paper has no counterpart: this is a
 * deployment convenience, not a step of the method.)
 *
 * Who needs it: code that may not call cudaMalloc, or any allocator built on it, at the point where the
 * buffer fills -- an inference server whose memory pool already owns all of the GPU's memory and hands out
 * nothing beyond KV blocks, a plug-in running inside another framework's callback where allocation is
 * forbidden, a real-time loop that must not take the driver's allocation lock.  For them the scratch lives in
 * a fixed array inside the library's device image, RKV_STATIC_SCRATCH_BYTES (32 MiB) large.  Every GPU that
 * loads the library carries that array until the process ends, used or not.
 *
 * Arguments, layouts, results and error codes are those of rkv_compress_ex; desc->workspace and
 * desc->workspace_bytes are ignored.  In addition:
 *   - a shape whose rkv_workspace_bytes() exceeds RKV_STATIC_SCRATCH_BYTES is refused with RKV_ERR_WORKSPACE
 *     before anything is launched (rkv_workspace_bytes() tells what a shape needs).  32 MiB covers, for example,
 *     256 head-problems at budget 1024 + buffer 128 (all 32 layers of an 8-KV-head model, batch 1);
 *     larger batches are split into several calls over sub-ranges of the batch dimension, one after the other.
 *   - the call makes no cudaMalloc / cudaFree and calls no allocating library routine.
 *   - the FIRST call on each device looks up the array's device address (with that device current) and caches
 *     it; make that first call outside any stream capture (a first call that arrives while `stream` is being
 *     captured is refused with RKV_ERR_INVALID_ARG before the lookup).
 *   - all calls on a device share the one array, which still holds the previous call's contents.  The few
 *     words that have to start at zero (work counters, per-head tickets) are cleared by the call itself, on the
 *     stream, before its first kernel; everything else is written by one stage before the next reads it.  But
 *     two calls that overlap on the GPU (different streams, no dependency between them) race on
 *     it and corrupt each other's scores.  Serialise them, or give one of them a workspace of its own through
 *     rkv_compress_ex.
 */
#define RKV_STATIC_SCRATCH_BYTES (32u << 20)
RKV_API int rkv_compress_static(const rkv_desc_t *desc, void *k_cache, void *v_cache, const void *q_window,
                        int32_t *seq_lens, int32_t budget, int32_t buffer, int32_t alpha, float lambda,
                        int32_t *out_idx, void *stream);

/* The two cache updates of a decode step that surround the compression, so that a whole decode segment (buffer
 * appends, then rkv_compress when seq_lens reaches budget + buffer: Section 3.1) can be enqueued, or captured in a
 * CUDA graph, through this library alone.  Both only enqueue work on `stream` (two launches / one launch) and use no
 * workspace.
 *
 * rkv_append: the newly generated token of every sequence enters the buffer part of its cache.
 *   k_new, v_new [batch, n_kv_heads, head_dim] (device, dtype of the cache, 16-byte aligned) are copied to row
 *   seq_lens[b] of every KV head of sequence b in k_cache / v_cache [batch, n_kv_heads, budget + buffer, head_dim];
 *   then seq_lens[b] += 1.  A sequence whose cache is full (seq_lens[b] == budget + buffer: the caller has to compress
 *   first) or whose length is invalid is left unchanged and RKV_ERR_INVALID_ARG is written to desc->device_status.
 * rkv_push_query: Algorithm 1's observation buffer M_alpha as a ring.
 *   q_new [batch, n_q_heads, head_dim] becomes row `slot` (0 <= slot < alpha; the caller passes its step counter modulo
 *   alpha) of every query head's window in q_window [batch, n_q_heads, alpha, head_dim].  The order of the alpha rows
 *   plays no part in the scores (Eq. 4 averages over them), so no row is ever moved.
 * Return codes as for rkv_compress_ex. */
RKV_API int rkv_append(const rkv_desc_t *desc, void *k_cache, void *v_cache, const void *k_new, const void *v_new,
                       int32_t *seq_lens, int32_t budget, int32_t buffer, void *stream);
RKV_API int rkv_push_query(const rkv_desc_t *desc, void *q_window, const void *q_new, int32_t alpha, int32_t slot,
                           void *stream);

/*
 * The attention of a decode step over the cache as it stands (Section 3.1: between two firings the model decodes
 * against the retained tokens plus the buffer; Eq. 1 with one query row per head), so that a whole decode segment --
 * rkv_push_query, rkv_decode_attention, rkv_append, and rkv_compress when the buffer is full -- runs through this
 * library:
 *   out[b][q] = sum_j softmax_j( q_new[b][q] . K[b][q / G][j] / sqrt(head_dim) ) V[b][q / G][j],  j < seq_lens[b]
 *   k_cache, v_cache  [batch][n_kv_heads][budget + buffer][head_dim] (device, desc->dtype), read only
 *   q_new             [batch][n_q_heads][head_dim] (device, desc->dtype -- bf16 for 8-bit caches --, 16-byte aligned)
 *   seq_lens          [batch] int32 (device), read only; 0 gives a zero output row; a value outside
 *                     [0, budget + buffer] gives a zero row and RKV_ERR_INVALID_ARG in desc->device_status
 *   out               [batch][n_q_heads][head_dim] float32 (device, 16-byte aligned)
 * bf16 and 8-bit caches: both contractions on the tensor cores (bf16 products, fp32 accumulation, the softmax weights carried as
 * two bf16 parts, i.e. to fp32 accuracy), softmax in fp32; fp32 caches: fp32 arithmetic throughout.  head_dim 128 (any
 * cache type) or 64 (bf16 caches: tiles padded to 128 on their way to the tensor cores), and G = n_q_heads /
 * n_kv_heads up to 8 (RKV_ERR_UNSUPPORTED otherwise).  The rows of a head are cut into splits (with
 * few head-problems, to fill the GPU; for bf16 and 8-bit caches also whenever budget + buffer exceeds 1920 rows, what one block
 * holds scores for) whose partial results go through desc->workspace: rkv_decode_workspace_bytes() says how much that
 * needs (0 when there is a single split; never more than a compression of the same shape needs, so one workspace
 * serves both).  Enqueues one or two kernels on `stream`; return codes as for rkv_compress_ex.
 */
RKV_API size_t rkv_decode_workspace_bytes(const rkv_desc_t *desc, int32_t budget, int32_t buffer);
RKV_API int rkv_decode_attention(const rkv_desc_t *desc, const void *k_cache, const void *v_cache, const void *q_new,
                                 const int32_t *seq_lens, float *out, int32_t budget, int32_t buffer, void *stream);

/*
 * Self-test of the kernels' failure detection (no counterpart in the paper).  Every wait inside the tensor-core
 * kernels is bounded; this call makes such a wait run out on purpose, in a tiny kernel of its own (one block that
 * allocates tensor memory, waits with the given limit on a barrier nothing arrives at, calls off a second waiting
 * thread through the block's abort flag and leaves through the scoring kernels' kind of exit).  Nothing hangs,
 * faults or traps; the context stays usable and later calls on the stream run normally.
 *   device_status  device int32, must hold 0: receives RKV_ERR_TIMEOUT
 *   report_words   device uint64[8], 8-byte aligned, zeroed by the call: [0] != 0: abort recorded, [1] ticks the
 *                  first wait lasted, [2] = 0: it returned "failed", [3] ticks the second wait lasted, [4] = 1: the
 *                  second wait was called off before its own limit, [5] = 1: the block reached its end
 *   limit_cycles   limit of the first wait in GPU clock ticks, 1000 .. the default limit (about two seconds)
 * Enqueues one memset and one launch on `stream`; returns RKV_ERR_INVALID_ARG for bad arguments.
 */
RKV_API int rkv_selftest_wait_expiry(int32_t *device_status, unsigned long long *report_words, int64_t limit_cycles,
                                     void *stream);

/* Number of kernels a call launches (for launch accounting; the memset that precedes the prep kernel is not
 * counted).  rkv_launch_count_for() is exact for the given sizes; rkv_launch_count(), which does not know them, gives
 * the count for large caches (small ones run the select stage as one kernel instead of three). */
RKV_API int rkv_launch_count(const rkv_desc_t *desc, uint32_t stage_mask);
RKV_API int rkv_launch_count_for(const rkv_desc_t *desc, int32_t budget, int32_t buffer, int32_t alpha,
                         uint32_t stage_mask);

/* Human-readable name of a status code. */
RKV_API const char *rkv_status_string(int status);

/* Text of the last CUDA error seen by the calling thread inside the library ("" if none). */
RKV_API const char *rkv_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* RKV_H_ */
