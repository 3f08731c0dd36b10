/*
 * spf.h -- C ABI of the speculative-prefill scoring / selection library for NVIDIA B200 (sm_100a).
 *
 * The library covers the data-parallel part of "Cross-Family Speculative Prefill" that runs between
 * the draft model's forward pass and the assembly of the compressed prompt text:
 *
 *   spf_score          Appendix A.1.1 / Algorithm 1 "AggregateMaxMean": attention of the lookahead
 *                      queries over the prompt keys, max over (layer, head), mean over lookahead.
 *   spf_chunk_pool     Appendix A.1.2 / Algorithm 1 "AvgPool1D" + "PartitionIntoChunks": smoothing
 *                      and per-chunk mean.
 *   spf_select_topk    Appendix A.1.2 / Algorithm 1 "TopKChunks".
 *   spf_compact_spans  Section 3.2 / Algorithm 1 "MergeAdjacentChunks" + "MapDraftChunksToTextSpans".
 *
 * Around them: spf_keep_count / spf_keep_rate / spf_snap_budget (Section 3.1, keep rate) and spf_concat_with_delim
 * (Algorithm 1 "ConcatWithDelim") on the host; spf_score_paged (paged key cache), spf_score_fp8 (8-bit key cache),
 * spf_score_shard_lse /
 * spf_score_shard_apply (one prompt's keys over several GPUs); spf_score_extra, spf_chunk_pool_edge,
 * spf_select_topk_forced (switches for points the paper leaves open); spf_compress_host (the four calls for host
 * buffers); spf_score_static (no allocation).
 *
 * Symbols: N prompt tokens (the paper's S), m lookahead queries (the paper's N), L layers, Hq query
 * heads (the paper's H), Hkv key heads, G = Hq / Hkv, d head dimension, c chunk size, C = ceil(N / c),
 * k chunks kept, w pooling kernel.
 *
 * General conventions
 *   - Every pointer is DEVICE memory owned by the caller unless its comment says HOST.  The library
 *     never frees or keeps caller memory and allocates nothing per call.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  All work is
 *     enqueued on it; no call synchronises the stream or the device.
 *   - Return value: SPF_OK (0) or a negative spf_status.  Argument checks happen on the host before
 *     anything is launched; a call that fails them launches nothing.  spf_last_error() gives the text of
 *     the calling thread's last failure.
 *   - Conditions only the device can see are written to `dev_status` (see spf_score).
 *   - Nothing here falls back to the CPU: unsupported shapes return SPF_ERR_UNSUPPORTED.
 */
#ifndef SPF_H_
#define SPF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(_WIN32)
#define SPF_API
#else
#define SPF_API __attribute__((visibility("default")))
#endif

typedef enum {
  SPF_OK = 0,
  SPF_ERR_INVALID_ARG = -1, /* null pointer, non-positive size, misaligned K rows, k > C, ...      */
  SPF_ERR_UNSUPPORTED = -2, /* shape outside what the kernels cover (see spf_score)                 */
  SPF_ERR_WORKSPACE = -3,   /* workspace missing, misaligned or smaller than the size query says    */
  SPF_ERR_CUDA = -4,        /* a CUDA runtime call failed (no device, launch error)                 */
  SPF_ERR_TIMEOUT = -5,     /* device status only: a bounded wait inside a kernel ran out           */
  SPF_ERR_RANGE = -6        /* device status only: a softmax row sum overflowed fp32 in the fused path */
} spf_status;

/* Draft-model attention geometry shared by all prompts of a call. */
typedef struct {
  int32_t n_layers;     /* L >= 1                                                                  */
  int32_t n_q_heads;    /* Hq, multiple of n_kv_heads                                              */
  int32_t n_kv_heads;   /* Hkv                                                                     */
  int32_t head_dim;     /* d: 64 or 128                                                            */
  int32_t n_lookahead;  /* m: 1..32, with G * roundup(m, 8) <= 64                                   */
  float softmax_scale;  /* multiplies q.k before the softmax; <= 0 selects 1/sqrt(d)                */
} spf_shape;

/* One prompt.  An array of these expresses a ragged batch; prompts are independent. */
typedef struct {
  int64_t n_tokens;            /* N >= 1                                                            */
  const void* const* k_layers; /* HOST array of L device pointers; layer l is bf16 [Hkv][N][d],
                                  post-RoPE, element (h, s, j) at h*k_stride_head + s*k_stride_tok + j */
  int64_t k_stride_head;       /* in elements                                                       */
  int64_t k_stride_tok;        /* in elements, >= d, multiple of 8 (rows start 16-byte aligned)     */
  const void* q;               /* bf16 [L][Hq][m][d], contiguous, post-RoPE lookahead queries       */
  float* importance;           /* out: fp32 [N], the token importance I                             */
  float* lse;                  /* out, may be NULL: fp32 [L][Hq][m], natural-log sum-exp of each
                                  softmax row, so that p = exp(scale * q.k - lse)                   */
} spf_prompt;

/*
 * Bytes of scratch spf_score needs for these prompts (0 on invalid arguments; the reason is left in
 * spf_last_error()).  The scratch holds packed queries, per-split softmax partials and row
 * log-sum-exps; one buffer serves all prompts of the call in turn.
 */
SPF_API size_t spf_score_workspace_bytes(const spf_shape* shape, const spf_prompt* prompts, int32_t n_prompts);

/*
 * Token importance (Appendix A.1.1; Algorithm 1, AggregateMaxMean).  For every prompt:
 *     z[l,h,i,s] = scale * sum_j Q[l,h,i,j] * K[l, h / G, s, j]         (GQA: head h reads key head h / G)
 *     p[l,h,i,s] = exp(z[l,h,i,s]) / sum_{s'} exp(z[l,h,i,s'])           softmax over the N prompt keys
 *     A[i,s]     = max over all (l,h) of p[l,h,i,s]                      max over layer and head first,
 *     I[s]       = (1/m) * sum_i A[i,s]                                  then the mean over lookahead
 * written to prompts[p].importance (and the row log-sum-exps to prompts[p].lse when not NULL).
 * bf16 inputs, fp32 accumulation and softmax.  The attention tensor itself is never stored.
 *
 * `shape`, `prompts` and the k_layers arrays are HOST memory, read during the call only.
 * `workspace`: device, 256-byte aligned, at least spf_score_workspace_bytes(...) bytes; contents on
 * entry are irrelevant, contents on exit unspecified.  Calls that share a workspace must be ordered
 * on one stream.
 * `dev_status`: device int32, may be NULL (device-side conditions then go unreported).  Kernels store a
 * negative spf_status there when a device-side condition occurs; they never trap.  The caller zeroes it
 * before the call and reads it after synchronising.  Conditions:
 *   SPF_ERR_TIMEOUT  a bounded wait of the fused path ran out (2 s): the kernel returned without results.
 *                    The fused kernel needs all its CTAs resident at once and asks the runtime for that at
 *                    launch; the wait can still run out if the GPU is shared so heavily that a hand-over
 *                    between CTAs takes seconds.
 *   SPF_ERR_RANGE    fused path only.  Its first sweep sums exp2(logit - r) per softmax row in fp32, with one
 *                    reference r per (layer, kv-head): 60 base-2 units above the smallest logit that the rows of
 *                    that kv-head have against the key at position N / 2.  No row can underflow (its largest
 *                    term is at least 2^-60, and what is flushed is 2^66 times smaller), whatever the spread
 *                    between the heads of a group.  A row sum overflows when some logit lies about 188 -
 *                    log2(number of such keys) base-2 units -- 157 at the very least, about 109 nats -- above that
 *                    smallest sample logit.  The importance is then invalid and the call should be repeated on
 *                    the general path (spf_set_score_path(1)), which has no such limit.
 * Errors: SPF_ERR_INVALID_ARG, SPF_ERR_UNSUPPORTED (d not 64/128, Hq % Hkv != 0, m > 32,
 * G * roundup(m,8) > 64, L > 128; with the fused path forced, also shapes outside it or a grid that cannot be
 * co-resident on the device), SPF_ERR_WORKSPACE, SPF_ERR_CUDA.  All prompts are validated before the first
 * launch; a shape that only the forced fused path refuses is found when its prompt's turn comes, after earlier
 * prompts of the batch have been enqueued.
 */
SPF_API int32_t spf_score(const spf_shape* shape, const spf_prompt* prompts, int32_t n_prompts, void* workspace,
                          size_t workspace_bytes, int32_t* dev_status, void* cuda_stream);

/*
 * spf_score with a larger softmax denominator -- a switch for a point the paper leaves open (Section 3 describes the
 * attention of each lookahead step "over the prompt", Appendix A.1.1 slices it to the prompt length): in the draft
 * model, lookahead step i also attends to the i - 1 tokens generated before it and to itself, so its probabilities
 * over the prompt sum to less than 1.  `extra_lse` is a HOST array of n_prompts DEVICE pointers (an entry may be
 * NULL), each fp32 [L][Hq][m]: the natural log of sum exp(scale * q.k) over those non-prompt keys of row (l, h, i),
 * as the draft model's attention kernel reports it.  Then
 *     p[l,h,i,s] = exp(z[l,h,i,s]) / (sum_{s'} exp(z[l,h,i,s']) + exp(extra_lse[l,h,i]))
 * and everything downstream is unchanged; prompts[p].lse receives the log of the whole denominator.  With
 * extra_lse == NULL, or all entries NULL, this is spf_score.  Arguments, workspace and errors as for spf_score.
 */
SPF_API int32_t spf_score_extra(const spf_shape* shape, const spf_prompt* prompts, int32_t n_prompts,
                                const float* const* extra_lse, void* workspace, size_t workspace_bytes, int32_t* dev_status,
                                void* cuda_stream);

/*
 * spf_score on a PAGED key cache (Section 3.1: the paper's serving system keeps KV caches in 4k-token blocks; a draft
 * model served the same way has its prompt keys scattered over a block pool).  Same computation as spf_score.
 *
 *   k_pools        HOST array of L device pointers; layer l's pool is bf16 [n_pool_blocks][Hkv][block_tokens][d],
 *                  contiguous, 16-byte aligned, post-RoPE
 *   block_tokens   tokens per block, a positive multiple of 128
 *   block_table    DEVICE int32 [ceil(N / block_tokens)]: logical block b of the prompt is pool block block_table[b].
 *                  Entries must lie in [0, n_pool_blocks); the kernels cannot report a bad entry, but its keys then
 *                  read as zeros (or, for the one sampled reference key, from a clamped block) instead of faulting.
 *                  Rows of the last block beyond n_tokens are never used.
 *   q, importance, lse   as in spf_prompt
 *
 * Both kernel paths read paged caches (spf_set_score_path applies); shapes, errors and dev_status as for spf_score.
 * Workspace: spf_score_paged_workspace_bytes(...), rules as for spf_score.
 */
typedef struct {
  int64_t n_tokens;
  const void* const* k_pools;
  int64_t n_pool_blocks;
  int32_t block_tokens;
  const int32_t* block_table;
  const void* q;
  float* importance;
  float* lse;
} spf_paged_prompt;

SPF_API size_t spf_score_paged_workspace_bytes(const spf_shape* shape, const spf_paged_prompt* prompts, int32_t n_prompts);
SPF_API int32_t spf_score_paged(const spf_shape* shape, const spf_paged_prompt* prompts, int32_t n_prompts, void* workspace,
                                size_t workspace_bytes, int32_t* dev_status, void* cuda_stream);

/*
 * spf_score on an 8-BIT key cache (Section 3.1: the paper's serving system keeps KV caches in block-quantised form; a
 * draft model served the same way holds its prompt keys in 8 bits).  The cache format is an input format: key
 * (l, hk, s, j) has the value
 *     k_scale[l * Hkv + hk] * E4M3(byte at k_layers[l] + hk * k_stride_head + s * k_stride_tok + j)
 * with E4M3 the 8-bit floating-point format of 1 sign, 4 exponent (bias 7) and 3 mantissa bits, subnormals, no
 * infinities (the byte patterns 0x7F / 0xFF, NaN, must not occur).  The key scale is folded into the softmax scale of
 * its (layer, kv-head).  Queries are given in bf16.
 *
 *   k_layers       HOST array of L device pointers (8-byte aligned), layer l uint8 [Hkv][N][d]; strides in bytes,
 *                  k_stride_tok >= d, both strides multiples of 8
 *   k_scale        DEVICE fp32 [L][Hkv], positive and finite
 *   others         as in spf_prompt
 *
 * Kernel paths, chosen as in spf_score (spf_set_score_path):
 *   fused     needs 16-byte aligned layer pointers and strides (and a shape spf_score's fused path takes).  The tensor
 *             cores multiply the E4M3 keys by E4M3 operands only, so each bf16 query is handed to them as the sum of two
 *             E4M3 terms after a power-of-two scaling per (layer, kv-head): exact for every element within 2^9 of the
 *             largest |q| of its (layer, kv-head), off by at most 2^-17 of that largest value below.  Accumulation is
 *             fp32.  Range limits and `dev_status` as for spf_score's fused path (SPF_ERR_RANGE, SPF_ERR_TIMEOUT).
 *   general   any cache the layout rules above admit.  Bytes are widened to bf16 exactly; arithmetic and error are
 *             those of spf_score's general path; `dev_status` is not written.
 * With the path left automatic, caches the fused path cannot read go to the general kernels; with the fused path
 * forced they are refused with SPF_ERR_UNSUPPORTED.  Workspace: spf_score_fp8_workspace_bytes(...), rules as for
 * spf_score.
 */
typedef struct {
  int64_t n_tokens;
  const void* const* k_layers;
  int64_t k_stride_head;
  int64_t k_stride_tok;
  const float* k_scale;
  const void* q;
  float* importance;
  float* lse;
} spf_fp8_prompt;

SPF_API size_t spf_score_fp8_workspace_bytes(const spf_shape* shape, const spf_fp8_prompt* prompts, int32_t n_prompts);
SPF_API int32_t spf_score_fp8(const spf_shape* shape, const spf_fp8_prompt* prompts, int32_t n_prompts, void* workspace,
                              size_t workspace_bytes, int32_t* dev_status, void* cuda_stream);

/*
 * One long prompt over several GPUs (Appendix A.1.1 is per prompt; this shards its keys).  Each rank holds a contiguous
 * range of the prompt's keys for all layers and describes it as an spf_prompt of its own (n_tokens = the range's
 * length).  A softmax row spans all ranks, so scoring takes two calls with one exchange between them:
 *
 *   spf_score_shard_lse     writes to prompt->lse (required) the natural-log sum-exp of every row over THIS rank's keys;
 *                           prompt->importance is ignored.
 *   (caller)                combines the ranks' values: lse_all = log sum_r exp(lse_r) -- e.g. a max all-reduce and a
 *                           sum all-reduce of exp(lse_r - max), L * Hq * m floats.
 *   spf_score_shard_apply   given lse_all (device fp32 [L][Hq][m]) writes the importance of this rank's keys, exactly
 *                           what spf_score would give them in the whole prompt; prompt->lse is ignored.
 *
 * Pooling needs a halo of pool_kernel / 2 importance values from each neighbour, the top-k needs all ranks' chunk
 * scores; both are the caller's exchanges.  These two calls use the general two-sweep kernels (one sweep each);
 * workspace as spf_score_workspace_bytes for the shard, errors as spf_score.
 */
SPF_API int32_t spf_score_shard_lse(const spf_shape* shape, const spf_prompt* prompt, void* workspace, size_t workspace_bytes,
                                    void* cuda_stream);
SPF_API int32_t spf_score_shard_apply(const spf_shape* shape, const spf_prompt* prompt, const float* lse, void* workspace,
                                      size_t workspace_bytes, void* cuda_stream);

/*
 * The same two calls on the kernels spf_score would pick (spf_set_score_path applies): where the shard's shape allows it,
 * the fused kernel runs with one of its two visits only -- spf_score_shard_lse_ex streams the shard's keys once and
 * leaves the row log-sum-exps, spf_score_shard_apply_ex streams them once and leaves the importance -- so a rank reads
 * its keys at the fused kernel's rate instead of the general kernels'.  `dev_status` as for spf_score: a row sum of the
 * first call can overflow fp32 (SPF_ERR_RANGE: repeat that call with spf_score_shard_lse), a bounded wait can run out
 * (SPF_ERR_TIMEOUT).  Workspace: spf_score_workspace_bytes for the shard.
 */
SPF_API int32_t spf_score_shard_lse_ex(const spf_shape* shape, const spf_prompt* prompt, void* workspace, size_t workspace_bytes,
                                       int32_t* dev_status, void* cuda_stream);
SPF_API int32_t spf_score_shard_apply_ex(const spf_shape* shape, const spf_prompt* prompt, const float* lse, void* workspace,
                                         size_t workspace_bytes, int32_t* dev_status, void* cuda_stream);

/*
 * Chooses the kernels behind spf_score, process-wide: 0 = automatic (the fused single-kernel path when
 * the shape allows it, else the general two-sweep path), 1 = always the general path, 2 = always the
 * fused path (spf_score then returns SPF_ERR_UNSUPPORTED for shapes outside it: G not in {1,2,4,8},
 * more than 64 layers, or a prompt too long for the per-CTA state).  Both compute the same function
 * (Appendix A.1.1).  Meant for tests and measurements.  Returns the previous setting; an invalid value
 * changes nothing.
 */
SPF_API int32_t spf_set_score_path(int32_t path);

/*
 * Diagnostic (no counterpart in the paper): checks that a device-side wait of the fused kernel gives up
 * instead of hanging.  Enqueues a one-CTA kernel that waits, with the kernels' own bounded wait and a
 * 20 ms limit, on a barrier nothing ever signals.  After synchronising, *dev_status (device int32, zeroed
 * by the caller) must read SPF_ERR_TIMEOUT and the context must still be usable.
 */
SPF_API int32_t spf_selftest_bounded_wait(int32_t* dev_status, void* cuda_stream);

/*
 * spf_score without a caller-provided workspace (the paper has no counterpart; this exists for
 * deployment reasons only).
 *
 * Some callers cannot hand over scratch memory because they cannot allocate any at the point where
 * they score a prompt: a serving engine that has already given all free HBM to its KV-cache pool, a
 * plugin that runs inside someone else's process under a no-allocation rule, or code on a path where
 * the implicit device-wide synchronisation of cudaMalloc / cudaFree is not acceptable.  For them the
 * library keeps SPF_STATIC_SCRATCH_BYTES of scratch in a static device array of its own (part of the
 * loaded module: every GPU that loads the library holds it until the process exits) and this call
 * uses it in place of `workspace`.  It computes exactly what spf_score computes with the general
 * two-sweep kernels and calls no allocating routine.
 *
 *   - Arguments and results are those of spf_score; inputs and outputs are still the caller's.
 *   - Prompts whose scratch need (spf_score_workspace_bytes gives an upper bound) exceeds
 *     SPF_STATIC_SCRATCH_BYTES are rejected with SPF_ERR_WORKSPACE before anything is launched.
 *   - The first call on each device looks up the array's device address (with that device current)
 *     and caches it.  CUDA loads a library's device code lazily, so that first lookup is also the
 *     moment the array itself (8 MiB) comes to exist on the device: make the first call at start-up,
 *     BEFORE the application hands the remaining HBM to its own pools (afterwards the lookup can fail
 *     with SPF_ERR_CUDA for lack of memory), outside any stream capture, with the device that owns
 *     `cuda_stream` current.  Any small prompt will do for that call.
 *   - Every call on a device shares the one array, and the array keeps whatever the previous call
 *     left in it.  The kernels write each scratch word before they read it, so nothing needs
 *     clearing between calls; but two calls whose kernels overlap on the GPU (different streams,
 *     no ordering) race on it and give wrong results.  Order them on one stream or with events.
 */
#define SPF_STATIC_SCRATCH_BYTES (8u << 20)
SPF_API int32_t spf_score_static(const spf_shape* shape, const spf_prompt* prompts, int32_t n_prompts,
                                 void* cuda_stream);

/*
 * Smoothing and chunk means (Appendix A.1.2; Algorithm 1, AvgPool1D and PartitionIntoChunks;
 * kernel size 13 and chunk size 32 / 128 in Appendix A.3):
 *     S[s]  = (1/w) * sum_{t = s - w/2}^{s + w/2} I[t]      terms outside [0, N) count as zero
 *     cs[j] = mean of S over tokens [j*c, min((j+1)*c, N))
 * importance: fp32 [N] in; chunk_scores: fp32 [ceil(N/c)] out.  pool_kernel w is odd, 1 <= w <= 255
 * (1 = no smoothing); chunk c >= 1.
 */
SPF_API int32_t spf_chunk_pool(const float* importance, int64_t n_tokens, int32_t pool_kernel, int32_t chunk,
                               float* chunk_scores, void* cuda_stream);

/*
 * Top-k chunks (Appendix A.1.2; Algorithm 1, TopKChunks): the indices of the k largest chunk scores,
 * equal scores resolved toward the lower index, written in ascending order.
 * chunk_scores: fp32 [n_chunks] in (finite); kept_chunks: int32 [k] out; 1 <= k <= n_chunks < 2^31.
 */
SPF_API int32_t spf_select_topk(const float* chunk_scores, int64_t n_chunks, int64_t k, int32_t* kept_chunks,
                                void* cuda_stream);

/*
 * Merge and compaction (Section 3.2; Algorithm 1, MergeAdjacentChunks and MapDraftChunksToTextSpans).
 * kept_chunks: int32 [k], ascending, distinct, each in [0, ceil(N/c)) -- as spf_select_topk writes them.
 * Runs of consecutive kept chunks become one token span [a, b) (b clipped to N); its character span
 * is [char_start[a], char_end[b-1]).  Kept tokens keep their original order.
 *   token_ids, char_start, char_end : int32 [N] in (character offsets of each draft token in the text)
 *   out_ids        int32 [>= min(k*c, N)]  kept token ids, n_kept of them
 *   out_pos        int32 [>= min(k*c, N)]  their original positions; may be NULL
 *   out_tok_spans  int32 [k][2]            n_spans rows (a, b)
 *   out_char_spans int32 [k][2]            n_spans rows (char_start[a], char_end[b-1])
 *   out_counts     int64 [2]               {n_kept, n_spans}
 * Rows beyond n_kept / n_spans are left untouched.
 */
SPF_API int32_t spf_compact_spans(const int32_t* kept_chunks, int64_t k, int32_t chunk, int64_t n_tokens,
                                  const int32_t* token_ids, const int32_t* char_start, const int32_t* char_end,
                                  int32_t* out_ids, int32_t* out_pos, int32_t* out_tok_spans,
                                  int32_t* out_char_spans, int64_t* out_counts, void* cuda_stream);

/*
 * spf_select_topk followed by spf_compact_spans in ONE launch (Algorithm 1, TopKChunks ... MapDraftChunksToTextSpans):
 * both steps are latency-bound, and chaining them inside one CTA saves a launch per prompt.  Arguments, layouts and
 * results are those of the two calls (kept_chunks receives the k indices as spf_select_topk writes them); n_chunks must
 * equal ceil(n_tokens / chunk).  Results are identical to the two separate calls.
 */
SPF_API int32_t spf_select_compact(const float* chunk_scores, int64_t n_chunks, int64_t k, int32_t chunk, int64_t n_tokens,
                                   const int32_t* token_ids, const int32_t* char_start, const int32_t* char_end,
                                   int32_t* kept_chunks, int32_t* out_ids, int32_t* out_pos, int32_t* out_tok_spans,
                                   int32_t* out_char_spans, int64_t* out_counts, void* cuda_stream);

/*
 * Batched forms of the three selection calls (Algorithm 1 runs AvgPool1D ... MapDraftChunksToTextSpans per prompt; a
 * serving step has many prompts).  `items` is a HOST array of n_items descriptors, read during the call only; every
 * pointer inside a descriptor is DEVICE memory with the layout and size the single-prompt call states.  One launch
 * serves up to 32 prompts (more are split into several launches); results are identical to n_items single calls.
 * pool_kernel and chunk are shared by the batch.  Errors as the single-prompt calls, reported with the item index
 * before anything is launched.
 */
typedef struct {
  const float* importance; /* fp32 [n_tokens]                  */
  int64_t n_tokens;
  float* chunk_scores;     /* out: fp32 [ceil(n_tokens / chunk)] */
} spf_pool_item;

typedef struct {
  const float* chunk_scores; /* fp32 [n_chunks] */
  int64_t n_chunks;
  int64_t k;
  int32_t* kept_chunks;      /* out: int32 [k], ascending */
} spf_topk_item;

typedef struct {
  const int32_t* kept_chunks;
  int64_t k;
  int64_t n_tokens;
  const int32_t* token_ids;
  const int32_t* char_start;
  const int32_t* char_end;
  int32_t* out_ids;
  int32_t* out_pos;          /* may be NULL */
  int32_t* out_tok_spans;
  int32_t* out_char_spans;
  int64_t* out_counts;
} spf_compact_item;

SPF_API int32_t spf_chunk_pool_batch(const spf_pool_item* items, int32_t n_items, int32_t pool_kernel, int32_t chunk,
                                     void* cuda_stream);
SPF_API int32_t spf_select_topk_batch(const spf_topk_item* items, int32_t n_items, void* cuda_stream);
SPF_API int32_t spf_compact_spans_batch(const spf_compact_item* items, int32_t n_items, int32_t chunk, void* cuda_stream);

/*
 * Variants for two points the paper leaves open (Algorithm 1 names the operations, Appendix A.3 gives kernel 13 and
 * the chunk sizes, nothing else).  Same arguments, layouts and errors as the calls they extend.
 *
 * spf_chunk_pool_edge: edge_rule 0 is spf_chunk_pool (every window is divided by pool_kernel, tokens beyond the
 *   prompt's ends count as zeros); edge_rule 1 divides each window by the number of tokens it really covers, so
 *   the first and last pool_kernel/2 tokens are not damped.  Other values: SPF_ERR_INVALID_ARG.
 * spf_select_topk_forced: the first and / or the last chunk (system prompt / attention sink, and the question at
 *   the end of the prompt) are kept whatever their scores; they count towards k, the remaining k - forced are
 *   the best of the other chunks, ties to the lower index.  k smaller than the number of forced chunks:
 *   SPF_ERR_INVALID_ARG.  With both flags 0 it is spf_select_topk.
 */
SPF_API int32_t spf_chunk_pool_edge(const float* importance, int64_t n_tokens, int32_t pool_kernel, int32_t chunk,
                                    int32_t edge_rule, float* chunk_scores, void* cuda_stream);
SPF_API int32_t spf_select_topk_forced(const float* chunk_scores, int64_t n_chunks, int64_t k, int32_t force_first,
                                       int32_t force_last, int32_t* kept_chunks, void* cuda_stream);

/*
 * The whole path for ONE prompt whose inputs and results live in HOST memory (Algorithm 1 from AggregateMaxMean to
 * MapDraftChunksToTextSpans): copies the inputs to the device, runs spf_score -> spf_chunk_pool -> spf_select_topk
 * -> spf_compact_spans, copies the selection back.  This is the entry for a caller that holds the draft model's
 * tensors on the host or on another device; a caller whose tensors are already on this GPU chains the four calls
 * itself.  Unlike every other call it SYNCHRONISES `cuda_stream` (twice: once to learn the counts, once at the end).
 *
 *   k_layers_host   HOST array of L HOST pointers, layer l bf16 [Hkv][N][d] contiguous (pinned memory copies at full
 *                   PCIe / NVLink-C2C speed, pageable memory works)
 *   q_host          HOST bf16 [L][Hq][m][d]
 *   token_ids_host, char_start_host, char_end_host   HOST int32 [N]
 *   params          chunk size c, pooling kernel w (odd), keep rate rho: k = spf_keep_count(ceil(N / c), rho)
 *   arena           DEVICE scratch owned by the caller, 256-byte aligned, at least spf_compress_host_arena_bytes(...)
 *                   bytes; holds the device copies of the inputs, every intermediate and the scoring workspace
 *   out_ids_host, out_pos_host (may be NULL)   HOST int32 [min(k * c, N)]
 *   out_tok_spans_host, out_char_spans_host     HOST int32 [k][2]
 *   out_counts_host                             HOST int64 [2]: {n_kept, n_spans}; only that many rows are written
 *
 * If the fused scoring kernel reports SPF_ERR_RANGE or SPF_ERR_TIMEOUT the prompt is scored again with the general
 * kernels before anything is returned.  Errors: as the four calls; SPF_ERR_WORKSPACE for a small or misaligned arena;
 * a device-side status that survives the retry is returned as the call's status.
 */
typedef struct {
  int32_t chunk;        /* c >= 1                       */
  int32_t pool_kernel;  /* w, odd, 1..255               */
  double keep_ratio;    /* rho in (0, 1]                */
} spf_select_params;

SPF_API size_t spf_compress_host_arena_bytes(const spf_shape* shape, int64_t n_tokens, const spf_select_params* params);
SPF_API int32_t spf_compress_host(const spf_shape* shape, int64_t n_tokens, const void* const* k_layers_host, const void* q_host,
                                  const int32_t* token_ids_host, const int32_t* char_start_host, const int32_t* char_end_host,
                                  const spf_select_params* params, void* arena, size_t arena_bytes, int32_t* out_ids_host,
                                  int32_t* out_pos_host, int32_t* out_tok_spans_host, int32_t* out_char_spans_host,
                                  int64_t* out_counts_host, void* cuda_stream);

/*
 * Host helper for the keep rate of Section 3.1: the number of chunks a keep rate rho retains,
 * clamp(ceil(rho * n_chunks), 1, n_chunks).  Pure host arithmetic; returns 0 if n_chunks < 1.
 */
SPF_API int64_t spf_keep_count(int64_t n_chunks, double keep_ratio);

/*
 * Host helpers for the keep rate of Section 3.1.  The keep rate is defined on the TARGET model's tokenisation:
 * rho = compressed target length / original target length, per sample.  The paper picks compressed lengths that
 * are whole KV-cache blocks of the serving system (8k, 16k, 24k, 32k tokens with 4k-token blocks).
 *
 * spf_keep_rate:        min(1, budget_tokens / target_tokens); 0 if target_tokens < 1 or budget_tokens < 1.
 * spf_snap_budget:      the largest multiple of block_tokens that is <= desired_tokens, at least one block;
 *                       0 if block_tokens < 1 or desired_tokens < 1.
 * Pure host arithmetic.
 */
SPF_API double spf_keep_rate(int64_t target_tokens, int64_t budget_tokens);
SPF_API int64_t spf_snap_budget(int64_t desired_tokens, int64_t block_tokens);

/*
 * ConcatWithDelim of Algorithm 1 (Section 3.2, Appendix A.3): builds the compressed prompt text from the character
 * spans that spf_compact_spans produced.  Host routine, host pointers throughout.
 *
 *   text, text_bytes     the prompt as UTF-8 (need not be NUL-terminated)
 *   char_spans           int32 [n_spans][2], half-open [start, end) in CHARACTERS (Unicode code points, as a
 *                        tokenizer's offset mapping counts them), ascending and non-overlapping
 *   delim, delim_bytes   UTF-8 delimiter (e.g. "[...]" or "// omitted"); written between consecutive spans only,
 *                        never before the first or after the last; may be empty
 *   out, out_capacity    receives the compressed text (not NUL-terminated); may be NULL with capacity 0 to query
 *
 * Returns the number of bytes of the compressed text.  Nothing is written unless out_capacity is at least that.
 * A negative return is a status code: SPF_ERR_INVALID_ARG for null / negative arguments, spans that are not
 * ascending, overlap or reach beyond the text's last character.  Bytes of the form 10xxxxxx are counted as
 * continuations of the preceding character; the text is not otherwise validated.
 */
SPF_API int64_t spf_concat_with_delim(const char* text, int64_t text_bytes, const int32_t* char_spans, int64_t n_spans,
                                      const char* delim, int64_t delim_bytes, char* out, int64_t out_capacity);

/* Text of a status code (static storage). */
SPF_API const char* spf_status_string(int32_t status);
/* Text of the calling thread's most recent failure ("" if none).  Thread-local storage. */
SPF_API const char* spf_last_error(void);
/* Library version, e.g. "0.1.0". */
SPF_API const char* spf_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SPF_H_ */
