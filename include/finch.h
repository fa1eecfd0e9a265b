/*
 * finch.h -- C ABI of the B200 (sm_100a) library for Finch's prompt-guided KV-cache
 * compression step (arXiv 2408.00167, Section "Method").
 *
 * Problem statement (Section "Problem Formulation"): given a prompt and a long text
 * processed chunk by chunk, keep in a fixed-size KV cache only the key/value pairs
 * that are most relevant to the prompt.  One *step* takes the compressed cache so
 * far plus the new chunk (together: the N = c + m candidates), scores every
 * candidate by the attention the prompt's query rows give it, keeps the top-r
 * candidates per layer and selection group, and writes their K/V rows, in original
 * order, into the next cache.
 *
 * Conventions common to every call
 * --------------------------------
 *  - All tensor pointers are DEVICE pointers unless a parameter says "host".
 *    The caller owns every buffer, including the workspace; the library allocates
 *    only the context and one 4-byte device status word and frees only those.
 *  - Work is enqueued asynchronously on `cuda_stream` (a cudaStream_t passed as
 *    void*; NULL = the legacy default stream).  No call synchronises except
 *    finch_device_status and finch_step_host.
 *  - Arguments are validated on the host; a call that returns anything but FINCH_OK
 *    has enqueued nothing.  Nothing throws or aborts across this boundary.  Kernels
 *    never trap: device-side anomalies (inconsistent batch metadata, a bounded wait
 *    that ran out) set bits in the status word, read with finch_device_status.
 *  - A context is bound to one device and is not thread-safe; use it from one host
 *    thread and one stream at a time.
 *  - There is no CPU fallback.  finch_ctx_create fails with FINCH_ERR_UNSUPPORTED on a
 *    device that is not compute capability 10.x.  A context created with device < 0 is
 *    validation-only: every call checks its arguments exactly as usual, then returns
 *    FINCH_ERR_UNSUPPORTED instead of enqueuing work (finch_workspace_bytes still works).
 *
 * Layouts
 * -------
 *  A finch_tensor views [n_layers][heads][tokens][head_dim] with head_dim contiguous
 *  and the three outer strides given in ELEMENTS.  Base pointer and every stride
 *  times the element size must be multiples of 16 bytes.
 *
 *  Batches are packed along the token axis ("cu_seqlens" style), with three offset
 *  arrays of batch+1 int32 each (device memory):
 *     prompt_q        heads = n_q_heads,  request b owns token rows [q_off[b], q_off[b+1])
 *     chunk_k/chunk_v heads = n_kv_heads, request b owns rows [chunk_off[b], chunk_off[b+1])
 *     cache_*, out_*  heads = n_kv_heads, request b owns a region of CAPACITY
 *                     cache_off[b+1]-cache_off[b] rows starting at cache_off[b], of which the first
 *                     cache_len[b] (input) or out_len[b] (output) rows are valid
 *  Candidate j of request b is cache row j for j < cache_len[b], else chunk row j - cache_len[b]
 *  (Method, bullet "Extract prompt-guided submatrix": columns 1..m+c).  N_b = cache_len[b] + chunk_len[b].
 *
 *  Selection groups: G = n_kv_heads groups per layer in FINCH_GROUP_PER_KV_HEAD mode (a group sums the
 *  n_q_heads/n_kv_heads query heads that share one KV head) or G = 1 in FINCH_GROUP_PER_LAYER mode (the paper's
 *  sum over all H heads; the one index list then applies to every KV head of the layer).
 *     scores    float32 [n_layers][G][total_cache + total_chunk], request b at cache_off[b] + chunk_off[b], N_b valid
 *     kept_idx  int32   [n_layers][G][total_cache],               request b at cache_off[b], out_len[b] valid
 *     cache_pos / out_pos int32 [n_layers][G][total_cache]  original token position of each cached row
 *     chunk_pos int32   [total_chunk]                       original token position of each chunk row
 *     row_lse   float32 [n_layers][n_q_heads][total_q]      natural-log sum-exp of each prompt row's logits
 */
#ifndef FINCH_H_
#define FINCH_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct finch_ctx finch_ctx; /* opaque */

typedef enum {
    FINCH_OK = 0,
    FINCH_ERR_INVALID_ARG = 1,         /* null pointer, negative size, overlap of outputs with inputs ...        */
    FINCH_ERR_UNSUPPORTED = 2,         /* no sm_100 device, head_dim / dtype the kernels do not cover            */
    FINCH_ERR_BAD_LAYOUT = 3,          /* pointer or stride not 16-byte aligned                                  */
    FINCH_ERR_WORKSPACE_TOO_SMALL = 4, /* ws_bytes below finch_workspace_bytes                                   */
    FINCH_ERR_OOM = 5,                 /* host or device allocation of the context failed                        */
    FINCH_ERR_CUDA = 6,                /* a CUDA runtime/driver call failed (launch error, bad stream ...)        */
    FINCH_ERR_DEVICE_STATUS = 7        /* finch_device_status found a non-zero status word                       */
} finch_status;

typedef enum { FINCH_F32 = 0, FINCH_BF16 = 1 } finch_dtype;

typedef enum { FINCH_GROUP_PER_KV_HEAD = 0, FINCH_GROUP_PER_LAYER = 1 } finch_group_mode;

/* Bits of the device status word. */
enum {
    FINCH_DEV_BAD_BATCH = 1,   /* device-side batch metadata exceeds the host bounds given in finch_batch      */
    FINCH_DEV_TIMEOUT = 2,     /* a bounded wait inside a kernel ran out                                       */
    FINCH_DEV_BAD_INDEX = 4    /* finch_compact met a kept index outside [0, N_b)                              */
};

typedef struct {
    int32_t n_layers, n_q_heads, n_kv_heads, head_dim; /* head_dim: a multiple of 32, at most 256             */
    int32_t dtype;       /* finch_dtype of Q, K and V                                                         */
    int32_t group_mode;  /* finch_group_mode                                                                  */
    float scale;         /* logit scale; 0 selects 1/sqrt(head_dim) (Background, the attention equation)      */
    int32_t max_batch, max_prompt, max_candidates; /* upper bounds used for validation                        */
    int32_t device;      /* CUDA device ordinal; negative = validation-only context                           */
    /* Rotary re-positioning of the kept keys (Method, paragraph "Managing the Cache").  rope_theta = 0: K rows are
     * copied bit for bit.  rope_theta > 0 (the rotary base, 10000 for Llama 2): K rows are taken to carry rotary
     * embeddings at their candidate index -- the cache's rows at their slots, the chunk's rows after them -- and
     * the compaction rotates each kept row by (output slot - candidate index) positions, so that it arrives embedded
     * at its new slot.  rope_pairing 0 rotates coordinate pairs (t, t + head_dim/2), the layout of the Llama
     * implementation; 1 rotates pairs (2t, 2t + 1), RoFormer's own.  V rows are never rotated.                     */
    float rope_theta;
    int32_t rope_pairing;
} finch_config;

typedef struct {
    void *ptr;
    int64_t stride_layer, stride_head, stride_tok; /* in elements */
} finch_tensor;

typedef struct {
    int32_t batch;
    const int32_t *q_off, *chunk_off, *cache_off; /* device, [batch+1]                                        */
    const int32_t *cache_len, *budget;            /* device, [batch]; budget[b] = r, at most the capacity     */
    int32_t total_q, total_chunk, total_cache;    /* host copies of q_off[batch], chunk_off[batch], cache_off[batch] */
    int32_t max_q, max_cache, max_chunk, max_budget; /* host upper bounds over the requests (grid sizing)      */
    /* Optional (NULL = absent), device, [n_layers][n_q_heads][total_q] fp32, natural log: for every prompt row the
     * log-sum-exp of its scaled logits against the keys it attends to besides the candidates -- in the paper's
     * full forward pass the prompt's own (causally visible) keys, "N = m + n^que + c" (Method, bullet "Extract
     * prompt-guided submatrix").  When given, exp(value) is added to the row's softmax denominator, so the weights
     * are those of the full attention row and a row's candidate weights sum to less than 1; -inf adds nothing.
     * Without it the softmax runs over the candidates only.  row_lse then reports the full denominator's log.  */
    const float *prompt_self_lse;
    /* Optional (NULL = absent), device, [total_q] int32: query row i of a request attends to that request's first
     * row_limit[i] candidates only (values are clamped to [0, N_b]; a row with 0 contributes nothing).  This is the
     * causal mask of query rows that are themselves document tokens -- the paper's ablation that conditions on the
     * whole input or on the document only instead of the prompt: pass the chunk's queries (and the prompt's) as
     * prompt_q, with row_limit = cache_len + position in the chunk + 1 for a chunk row and N_b for a prompt row.
     * With row_norm != 0 every row's weights are multiplied by the fraction of the candidates it sees, the per-row
     * reading of the Normalization bullet, count(row != 0) / (m + c): a token that sees only itself then scores
     * 1/(m + c) instead of the "score of 1" of the positional-bias paragraph.  Both scoring paths take it (the
     * tensor-core kernels have a masked instantiation that only such batches use).                              */
    const int32_t *row_limit;
    int32_t row_norm;
} finch_batch;

/* Create a context for one model shape on one device.  Fails with FINCH_ERR_UNSUPPORTED when the device is not
 * compute capability 10.x or the shape is not covered, FINCH_ERR_INVALID_ARG on inconsistent fields
 * (n_q_heads not a multiple of n_kv_heads, non-positive sizes, a rotary base below 1).  *out is set only on success.
 * Device memory the context owns, freed by finch_ctx_destroy: a 4-byte status word, a side stream with three events
 * (used by finch_step_host), and, with rope_theta > 0, the cosine/sine table of the re-positioning,
 * (max_candidates + 1) x head_dim/2 pairs of fp32 (2 MiB for 4096 candidates and head_dim 128), computed in double
 * precision on the host during this call. */
finch_status finch_ctx_create(const finch_config *cfg, finch_ctx **out);

/* Free the context and its status word.  NULL is ignored.  Work still in flight must be synchronised first. */
void finch_ctx_destroy(finch_ctx *ctx);

/* Bytes of device workspace that finch_score / finch_select / finch_step need for this batch (the maximum over
 * the three; finch_step includes room for the scores when the caller passes scores == NULL).  Pure host
 * arithmetic: callable without touching the device. */
finch_status finch_workspace_bytes(const finch_ctx *ctx, const finch_batch *batch, size_t *out);

/* Prompt-guided scoring (Method, bullets "Sum over heads", "Extract prompt-guided submatrix", "Selection of top r
 * position" up to A^agg; Background, the attention equation):
 *     s[h,p,j]  = scale * <q[h,p], k[kv(h),j]>          for the candidates j < N_b
 *     w[h,p,j]  = exp(s[h,p,j] - lse[h,p])               softmax over the candidates only, or, with
 *                                                        batch->prompt_self_lse, over candidates and prompt keys
 *     scores[j] = sum over the group's heads h and the prompt rows p of w[h,p,j]
 * The normalisation bullet's factor count(A != 0)/(m+c) is a constant on this path (prompt rows see every
 * candidate) and is not applied.  row_lse may be NULL; the workspace is always required.  Entries of `scores`
 * beyond N_b are left untouched.  bf16 inputs with head_dim 64 or 128 take the tensor-core path (either group mode),
 * everything else warp-level dot products; accumulation, softmax and the column sums are fp32 in a fixed order, so results
 * are run-to-run identical. */
finch_status finch_score(finch_ctx *ctx, const finch_tensor *prompt_q, const finch_tensor *cache_k,
                         const finch_tensor *chunk_k, const finch_batch *batch, float *scores, float *row_lse,
                         void *ws, size_t ws_bytes, void *cuda_stream);

/* Which kernels finch_score and finch_step run for a batch (given a workspace of finch_workspace_bytes).  Host
 * arithmetic, nothing is enqueued, works on a validation-only context.  (The paper prescribes no kernel; this is how
 * its prompt x candidate block, Section "Method", is tiled here.)
 *  - FINCH_SCORE_ONE_KERNEL: bf16, head_dim 64 or 128, a single request without row_limit, at most four 128-row
 *    query tiles per KV head (queries per KV head x ceil(prompt rows / 64) <= 8), and a window length for its key
 *    tiles exists: a divisor W of the tiles per (layer, KV head) unit with W >= 4 (or the whole unit),
 *    tiles / W <= 8, the persistent grid's CTA x window slots >= 85 % full, and W x SMs x tile bytes <= 40 MiB
 *    unless no shorter window qualifies; of several the fullest, longer ones preferred.
 *    *window receives W (key tiles of 128 candidates).  Both sweeps of the softmax run in one persistent kernel.
 *  - FINCH_SCORE_TWO_LAUNCH: bf16, head_dim 64 or 128 otherwise (several requests, causal rows, longer prompts, no
 *    usable window): row statistics and column sums in two tensor-core launches.  *window = 0.
 *  - FINCH_SCORE_WARP_LEVEL: fp32 inputs or another head_dim.  *window = 0.
 * A batch whose tensors the TMA unit cannot describe (an outer stride of 2^40 bytes or more) takes the warp-level
 * kernels regardless; that depends on the tensors, not on the batch, and is not reported here.
 * `window` may be NULL.  Errors: as finch_workspace_bytes. */
enum { FINCH_SCORE_WARP_LEVEL = 0, FINCH_SCORE_TWO_LAUNCH = 1, FINCH_SCORE_ONE_KERNEL = 2 };
finch_status finch_score_plan(const finch_ctx *ctx, const finch_batch *batch, int32_t *path, int32_t *window);

/* The same scores and row_lse as finch_score, for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is an integration aid.)  Some hosts of this library may not call cudaMalloc at all -- a plugin
 * inside a serving process whose memory pool owns the whole device, or a step that must stay clear of the driver's
 * allocator for latency reasons -- and so cannot supply finch_score's workspace.  Here everything finch_score
 * keeps in that workspace lives in a fixed array inside the library image instead (8 MiB of device memory on every
 * GPU that loads the library, held until the process exits).  The call itself allocates and frees nothing.
 *  - Limit: n_layers * n_q_heads * total_q must not exceed finch_score_static_max_rows() (2^20 rows); a larger
 *    batch is rejected with FINCH_ERR_WORKSPACE_TOO_SMALL and nothing is enqueued -- use finch_score then.
 *  - Which kernels run: the tensor-core kernels need more of the array than one entry per prompt row (in 8-byte
 *    entries, for a single request: 32 per prompt row plus 2 per layer, KV head and candidate; for a batch of
 *    requests: 5 per prompt row plus the same 2 per candidate).  A batch within the row limit whose need
 *    exceeds the array's 2^20 entries -- a whole 32-layer step of 4096 candidates does -- runs on the warp-level
 *    kernels instead: the same result within the score tolerance, many times slower.  finch_score_static_path
 *    tells which it will be.  Because the kernels (or their key ranges) can differ from finch_score's, the two
 *    calls agree within the score tolerance, max(1e-3 relative, 1e-5 absolute), not bit for bit.
 *  - The first call on each device looks up the array's device address.  Make that first call before starting any
 *    stream capture.  On EVERY call the context's device must be the current device (FINCH_ERR_INVALID_ARG
 *    otherwise): the address belongs to that GPU.
 *  - Every call on a device shares the one array, which keeps the previous call's contents.  Nothing in it has
 *    to start at zero: each call overwrites every entry it later reads.  Two calls whose kernels overlap on the
 *    GPU (different streams, or different contexts on one device) race on it: serialise them. */
finch_status finch_score_static(finch_ctx *ctx, const finch_tensor *prompt_q, const finch_tensor *cache_k,
                                const finch_tensor *chunk_k, const finch_batch *batch, float *scores, float *row_lse,
                                void *cuda_stream);

/* The row limit of finch_score_static. */
size_t finch_score_static_max_rows(void);

/* Host arithmetic, nothing is enqueued: *tensor_cores = 1 when finch_score_static would run this batch on the
 * tensor-core kernels (bf16, head_dim 64 or 128, and the batch's scratch fits the built-in array), 0 when it would
 * take the warp-level kernels.  (The paper has no counterpart.)  A batch whose tensors the TMA unit cannot describe
 * (an outer stride of 2^40 bytes or more) takes the warp-level kernels regardless. */
finch_status finch_score_static_path(const finch_ctx *ctx, const finch_batch *batch, int32_t *tensor_cores);

/* Top-r selection (Method, bullet "Selection of top r position": t = top-r(A^agg, r)).  For every layer, group and
 * request keeps r' = min(budget[b], N_b) candidates with the largest scores; among equal scores the lower
 * candidate index wins; -0 equals +0; a NaN ranks below every number.  Writes the kept candidate indices in
 * strictly increasing order to kept_idx and r' to out_len[b].  No full sort is performed.  ws may be NULL. */
finch_status finch_select(finch_ctx *ctx, const float *scores, const finch_batch *batch, int32_t *kept_idx,
                          int32_t *out_len, void *ws, size_t ws_bytes, void *cuda_stream);

/* Cache management (Method, paragraph "Managing the Cache"; "Compression Output"): copies the K and V rows and the
 * positions of the kept candidates, bit for bit, into rows [0, out_len[b]) of each request's region of
 * out_k / out_v / out_pos, for every KV head of the group.  out_* must not overlap cache_* or chunk_* (the gather
 * runs in parallel; coinciding base pointers are rejected with FINCH_ERR_INVALID_ARG).  cache_pos may be NULL only
 * if max_cache is 0. */
finch_status finch_compact(finch_ctx *ctx, const int32_t *kept_idx, const int32_t *out_len,
                           const finch_tensor *cache_k, const finch_tensor *cache_v, const int32_t *cache_pos,
                           const finch_tensor *chunk_k, const finch_tensor *chunk_v, const int32_t *chunk_pos,
                           const finch_batch *batch, const finch_tensor *out_k, const finch_tensor *out_v,
                           int32_t *out_pos, void *cuda_stream);

/* The fused step  finch_step(prompt_q, cache_kv, chunk_kv, budget) -> cache_kv, kept_positions:
 * score -> select -> compact enqueued back to back with no host synchronisation in between.  `scores` may be NULL
 * (they then live in the workspace).  kept_idx receives the kept candidate indices, out_pos their original token
 * positions.  Same argument rules as the three calls above. */
finch_status finch_step(finch_ctx *ctx, const finch_tensor *prompt_q, const finch_tensor *cache_k,
                        const finch_tensor *cache_v, const int32_t *cache_pos, const finch_tensor *chunk_k,
                        const finch_tensor *chunk_v, const int32_t *chunk_pos, const finch_batch *batch,
                        const finch_tensor *out_k, const finch_tensor *out_v, int32_t *out_pos, int32_t *kept_idx,
                        int32_t *out_len, float *scores, void *ws, size_t ws_bytes, void *cuda_stream);

/* The same step for a caller whose new inputs live in HOST memory (the end-to-end path: the paper's chunk loop,
 * Section "Method", "Document Segmentation", feeds one chunk per step).  host_prompt_q, host_chunk_k, host_chunk_v
 * are dense [n_layers][heads][tokens][head_dim] arrays and host_chunk_pos a dense [total_chunk] array, preferably in
 * pinned memory; they are copied into the caller's DEVICE staging tensors stage_* (which must be dense and of the
 * same shapes), the step runs on them and on the device-resident cache, and kept_idx / out_len are copied back to
 * host_kept_idx [n_layers][G][total_cache] / host_out_len [batch].  The compressed cache (out_k, out_v, out_pos)
 * stays on the device for the next step.  The chunk's V rows, which only the compaction reads, and the kept
 * indices on their way back travel on a second stream that the context owns, ordered against `cuda_stream` by
 * events, so the scoring kernels run while V is still being copied.  Unlike the other calls this one WAITS, for
 * both streams, before it returns.
 * The workspace must hold finch_workspace_bytes (scores live there).  Errors as for finch_step, plus
 * FINCH_ERR_BAD_LAYOUT when a staging tensor is not dense. */
finch_status finch_step_host(finch_ctx *ctx, const void *host_prompt_q, const void *host_chunk_k,
                             const void *host_chunk_v, const int32_t *host_chunk_pos, const finch_tensor *stage_q,
                             const finch_tensor *stage_chunk_k, const finch_tensor *stage_chunk_v,
                             int32_t *stage_chunk_pos, const finch_tensor *cache_k, const finch_tensor *cache_v,
                             const int32_t *cache_pos, const finch_batch *batch, const finch_tensor *out_k,
                             const finch_tensor *out_v, int32_t *out_pos, int32_t *kept_idx, int32_t *out_len,
                             int32_t *host_kept_idx, int32_t *host_out_len, void *ws, size_t ws_bytes,
                             void *cuda_stream);

/* Synchronises `cuda_stream`, copies the status word to *out (host) and clears it.  Returns FINCH_ERR_DEVICE_STATUS
 * when the word was non-zero, FINCH_ERR_CUDA when the stream reports an error. */
finch_status finch_device_status(finch_ctx *ctx, void *cuda_stream, int32_t *out);

/* Number of CUDA kernels this context has enqueued since it was created (host counter, for instrumentation).
 * The paper has no counterpart. */
finch_status finch_launch_count(const finch_ctx *ctx, uint64_t *out);

/* Static, NUL-terminated description of a status code. */
const char *finch_status_string(finch_status s);

#ifdef __cplusplus
}
#endif
#endif /* FINCH_H_ */
