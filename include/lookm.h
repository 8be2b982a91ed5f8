/*
 * lookm.h -- C ABI of the B200 (sm_100a) implementation of LOOK-M's one-shot, prefill-time
 * KV-cache compression (arXiv 2406.18139, Section 3).
 *
 * Per layer, per request and per KV head the library
 *   1. scores every prompt key by the column sum of the prompt's causal softmax attention (Eq. 4),
 *   2. keeps the recent window and the Top-N of the other tokens with text ranked before image
 *      tokens (Eq. 5-8),
 *   3. matches every evicted key to its most cosine-similar kept key (Eq. 9),
 *   4. folds the evicted K/V rows into their kept rows by averaged, pivotal or weighted merging
 *      (Eq. 10-12) and writes the kept rows as a dense cache ordered by position (Eq. 6-7).
 *
 * Conventions common to every entry point
 *   - All tensors are DEVICE memory unless the parameter name ends in `_host`.  Q/K/V and the
 *     output caches are bf16; head_dim must be 128; the feature index is contiguous.
 *   - Batches are packed along the token axis: request r owns tokens
 *     [cu_seqlens_host[r], cu_seqlens_host[r+1]).  A single prompt is n_requests = 1.
 *   - "kept"/"evicted" lists hold positions relative to the request start, ascending.  With
 *     B_r = min(budget_r, L_r) and E_r = L_r - B_r, the list of (request r, KV head h) starts at
 *     element  n_kv_heads * sum_{r'<r} B_r' + h * B_r   (kept lists) or
 *              n_kv_heads * sum_{r'<r} E_r' + h * E_r   (evicted, assign and sim arrays).
 *   - Every buffer is owned by the caller.  The library allocates nothing and never modifies
 *     inputs; outputs and workspace must not overlap inputs.  No result depends on an earlier
 *     call: the only state kept between calls is per host thread and diagnostic (the event handles
 *     given to lookm_set_stage_events and the launch count lookm_last_launch_count returns), plus
 *     per-device facts cached on first use (SM count, kernel attributes, the address of the
 *     lookm_merge_noalloc scratch).  `workspace`
 *     must be 256-byte aligned and at least lookm_workspace_size() bytes; its first bytes hold
 *     the device status word.  Calls that share a workspace must not overlap on the GPU.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t; NULL = default stream) and the call
 *     returns without synchronising.  Host outputs (`*_host`) are computed from the arguments and
 *     are valid on return.
 *   - Return value: a lookm_status.  Argument errors are found before anything is enqueued.
 *     Device-side waits are bounded; if one expires the kernel finishes without its results and
 *     lookm_device_status() reports LOOKM_ERR_DEVICE_TIMEOUT.  Nothing traps.
 *   - Edge rules: seq_len <= budget copies the prompt unchanged (out_len = seq_len);
 *     recent_window >= budget keeps only the last `budget` tokens; budget <= 0, seq_len <= 0 or
 *     recent_window < 0 is LOOKM_ERR_INVALID_ARG.
 */
#ifndef LOOKM_H_
#define LOOKM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LOOKM_OK = 0,
    LOOKM_ERR_INVALID_ARG = 1,
    LOOKM_ERR_UNSUPPORTED = 2,        /* e.g. head_dim != 128, or a device that is not sm_100 */
    LOOKM_ERR_WORKSPACE_TOO_SMALL = 3,
    LOOKM_ERR_CUDA = 4,               /* a CUDA runtime/driver call failed */
    LOOKM_ERR_DEVICE_TIMEOUT = 5,     /* a bounded device-side wait expired */
    LOOKM_ERR_DEVICE_BAD_INDEX = 6    /* a caller-supplied index list held an out-of-range entry */
} lookm_status;

typedef enum {
    LOOKM_MERGE_AVERAGE = 0,          /* Eq. 10 */
    LOOKM_MERGE_PIVOTAL = 1,          /* Eq. 11 */
    LOOKM_MERGE_WEIGHTED = 2,         /* Eq. 12 */
    LOOKM_MERGE_NONE = 3              /* eviction alone (Eq. 6-7): kept rows are copied, evicted rows
                                         dropped; no matching is done for such a request */
} lookm_merge_mode;

/* Shapes and strides (in elements) of Q [tokens, n_q_heads, head_dim] and of K and V
 * [tokens, n_kv_heads, head_dim] (K and V share strides).  Strides must be multiples of 8
 * elements and the base pointers 16-byte aligned (TMA requirements).  n_q_heads must be a
 * multiple of n_kv_heads; query heads [h*g, (h+1)*g) share KV head h and their scores are
 * summed.  softmax_scale = 0 selects 1/sqrt(head_dim); it must not be negative. */
typedef struct {
    int n_q_heads, n_kv_heads, head_dim;
    long long q_stride_tok, q_stride_head;
    long long kv_stride_tok, kv_stride_head;
    float softmax_scale;
} lookm_layout;

/* Bytes of workspace that any entry point below needs for this batch (seq_lens_host: n_requests
 * entries).  The size covers every budget, so budgets_host is only validated and may be NULL.
 * Returns 0 on invalid arguments. */
size_t lookm_workspace_size(const lookm_layout* layout, int n_requests, const int* seq_lens_host,
                            const int* budgets_host);

/* The whole path for one prompt (Section 3.2-3.3, Eq. 4-12).
 *   q, k, v        [seq_len, heads, 128] bf16 with the strides of `layout`
 *   modality_mask  [seq_len] bytes, 1 = image token, 0 = text token
 *   out_k, out_v   [n_kv_heads, out_len, 128] bf16, contiguous; row order = ascending position,
 *                  the Top-N tokens first, then the recent window (Eq. 6-7)
 *   out_len_host   receives min(seq_len, budget) */
int lookm_compress_layer(const void* q, const void* k, const void* v, const uint8_t* modality_mask,
                         int seq_len, int budget, int recent_window, int merge_mode,
                         const lookm_layout* layout, void* out_k, void* out_v, int* out_len_host,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The whole path for a packed ragged batch; each request has its own budget, window and merge
 * mode (host arrays of n_requests entries).
 *   out_k, out_v          [sum_r out_len_r, n_kv_heads, 128] bf16, requests in order
 *   out_cu_seqlens_host   [n_requests + 1] prefix sums of out_len_r */
int lookm_compress_varlen(const void* q, const void* k, const void* v, const uint8_t* modality_mask,
                          const int* cu_seqlens_host, int n_requests, const int* budgets_host,
                          const int* windows_host, const int* merge_modes_host,
                          const lookm_layout* layout, void* out_k, void* out_v,
                          int* out_cu_seqlens_host, void* workspace, size_t workspace_bytes,
                          void* cuda_stream);

/* Options of the whole-path calls below; a NULL pointer or an all-zero struct selects the
 * behaviour of lookm_compress_layer / lookm_compress_varlen.
 *   flags            LOOKM_OPT_NO_TEXT_PRIOR: leave the boost of Eq. 5 out and rank the candidates
 *                    by A_s alone (Eq. 8 on the raw scores: the paper's merging rows without the
 *                    text prior).  modality_mask is then not read and may be NULL.
 *   lse              device [n_q_heads, total_tokens] fp32, natural-log row log-sum-exp of the
 *                    prompt's causal attention, e.g. as the caller's prefill attention kernel
 *                    left it (Eq. 4 takes its scores from that very attention).  When not NULL the
 *                    first score sweep is skipped.  It must belong to the same q, k and scale.
 *   out_stride_head  lookm_compress_layer_opt only: elements between two heads of out_k / out_v,
 *                    so that the compressed rows can be written into a cache with room for
 *                    generated tokens ([n_kv_heads, capacity, 128]: capacity * 128).  0 selects
 *                    the dense out_len * 128; otherwise a multiple of 8, at least out_len * 128. */
#define LOOKM_OPT_NO_TEXT_PRIOR 1u
typedef struct {
    unsigned flags;
    const float* lse;
    long long out_stride_head;
} lookm_options;

/* lookm_compress_layer / lookm_compress_varlen with options (Section 3.2-3.3, Eq. 4-12). */
int lookm_compress_layer_opt(const void* q, const void* k, const void* v, const uint8_t* modality_mask,
                             int seq_len, int budget, int recent_window, int merge_mode,
                             const lookm_layout* layout, const lookm_options* options, void* out_k,
                             void* out_v, int* out_len_host, void* workspace, size_t workspace_bytes,
                             void* cuda_stream);
int lookm_compress_varlen_opt(const void* q, const void* k, const void* v, const uint8_t* modality_mask,
                              const int* cu_seqlens_host, int n_requests, const int* budgets_host,
                              const int* windows_host, const int* merge_modes_host,
                              const lookm_layout* layout, const lookm_options* options, void* out_k,
                              void* out_v, int* out_cu_seqlens_host, void* workspace,
                              size_t workspace_bytes, void* cuda_stream);

/* Step 1 alone (Eq. 4): scores[h, t] = sum over the query heads of KV head h and over the rows
 * i >= t of the same request of softmax_row_i(q_i . k * scale)[t].
 *   scores  [n_kv_heads, total_tokens] fp32
 *   lse     [n_q_heads, total_tokens] fp32, natural-log row log-sum-exp.  If lse_is_input != 0
 *           it is read (e.g. produced by the caller's prefill attention) and the first sweep is
 *           skipped; otherwise it is written.  May be NULL when lse_is_input == 0 (the workspace
 *           then holds it). */
int lookm_score(const void* q, const void* k, const int* cu_seqlens_host, int n_requests,
                const lookm_layout* layout, float* scores, float* lse, int lse_is_input,
                void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The selection alone (Eq. 5-8), fed with given scores [n_kv_heads, total_tokens] (fp32; the
 * method's scores are positive, other finite values are ordered numerically).
 *   modality_mask  NULL switches the text prior off: every candidate is ranked by its score alone
 *               (Eq. 8 without Eq. 5)
 *   kept_idx    kept positions, ascending (layout above)
 *   evict_idx   evicted positions, ascending
 *   rank        [n_kv_heads, total_tokens]: evicted token -> its index in the evicted list,
 *               kept token -> -1 - slot.  May be NULL. */
int lookm_select(const float* scores, const uint8_t* modality_mask, const int* cu_seqlens_host,
                 int n_requests, const int* budgets_host, const int* windows_host, int n_kv_heads,
                 int* kept_idx, int* evict_idx, int* rank, void* workspace, size_t workspace_bytes,
                 void* cuda_stream);

/* The matching alone (Eq. 9): for every evicted key the kept slot of largest cosine similarity
 * on the original keys (lowest slot on ties) and that similarity. */
int lookm_match(const void* k, const int* kept_idx, const int* evict_idx, const int* cu_seqlens_host,
                int n_requests, const int* budgets_host, const lookm_layout* layout, int* assign,
                float* sim, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The decision part of the matching alone: row argmax (lowest slot on ties) of given similarity
 * matrices.  sim_matrix holds, per (request, head) in the order of the evicted lists, a dense
 * row-major [E_r, B_r] fp32 block (block of (r, h) starts at element
 * n_kv_heads * sum_{r'<r} E_r' B_r' + h * E_r * B_r). */
int lookm_match_from_sim(const float* sim_matrix, const int* cu_seqlens_host, int n_requests,
                         const int* budgets_host, int n_kv_heads, int* assign, float* sim,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The merging alone (Eq. 10-12 and the compaction of Eq. 6-7), fed with given lists.
 * Requests whose mode is LOOKM_MERGE_NONE only have their kept rows copied; assign and sim may be
 * NULL when every request of the call has that mode.
 * varlen_output = 0: out [n_kv_heads, out_len, 128] (requires n_requests == 1);
 * varlen_output = 1: out [sum_r out_len_r, n_kv_heads, 128]. */
int lookm_merge(const void* k, const void* v, const int* kept_idx, const int* evict_idx,
                const int* assign, const float* sim, const int* cu_seqlens_host, int n_requests,
                const int* budgets_host, const int* merge_modes_host, const lookm_layout* layout,
                int varlen_output, void* out_k, void* out_v, void* workspace,
                size_t workspace_bytes, void* cuda_stream);

/* ---- the step after the path: token generation over the compressed cache ----------------------
 *
 * One generation step of one layer (Section 3.1 "Token Generation", Eq. 2-3): the new token's key
 * and value rows are appended to the cache (Eq. 2), then every query head attends over all rows of
 * its KV head, the new one included:  out = softmax(q K^T * scale) V  (Eq. 3; no mask, every cached
 * row precedes the new token; nothing is evicted any more).  The cache is the output of the calls
 * above (rows after compression) or an uncompressed cache; bf16, head_dim 128.
 *
 * Row t of KV head h of request r lives at element
 *     (cache_begin[r] + t) * cache_stride_row + h * cache_stride_head
 * of cache_k / cache_v, which covers [n_kv_heads, capacity, 128] caches (stride_row = 128,
 * stride_head = capacity * 128; see lookm_options.out_stride_head) and packed
 * [rows, n_kv_heads, 128] caches (stride_row = n_kv_heads * 128, stride_head = 128).  Strides are
 * multiples of 8 elements, base pointers 16-byte aligned.  The caller guarantees room for row
 * cache_len (the appended one).  softmax_scale = 0 selects 1/sqrt(head_dim). */
typedef struct {
    int n_q_heads, n_kv_heads, head_dim;
    long long cache_stride_row, cache_stride_head;
    float softmax_scale;
} lookm_cache_layout;

/* Bytes of workspace (256-byte aligned) a generation step over caches of these lengths needs
 * (partial results of the cache splits); it grows with n_requests and
 * n_q_heads, not with the cache lengths.  Returns 0 on invalid arguments. */
size_t lookm_decode_workspace_size(const lookm_cache_layout* layout, int n_requests,
                                   const int* cache_lens_host);

/* One step for one request.
 *   q             [n_q_heads, 128] bf16: the new token's query rows
 *   k_new, v_new  [n_kv_heads, 128] bf16: its key and value rows; written to cache row cache_len
 *                 (they must not lie inside the cache)
 *   cache_k/_v    read (rows 0 .. cache_len - 1) and extended by one row; cache_len >= 0
 *   out           [n_q_heads, 128] fp32
 * Asynchronous on cuda_stream like every other call; calls that share a workspace must not overlap
 * on the GPU.  Results do not depend on timing (fixed order of additions). */
int lookm_decode_step(const void* q, const void* k_new, const void* v_new, void* cache_k,
                      void* cache_v, int cache_len, const lookm_cache_layout* layout, float* out,
                      void* workspace, size_t workspace_bytes, void* cuda_stream);

/* One step for a batch of requests with their own caches and lengths.
 *   q [n_requests, n_q_heads, 128], k_new / v_new [n_requests, n_kv_heads, 128] bf16,
 *   out [n_requests, n_q_heads, 128] fp32; cache_begin_host / cache_lens_host: n_requests entries. */
int lookm_decode_step_varlen(const void* q, const void* k_new, const void* v_new, void* cache_k,
                             void* cache_v, const long long* cache_begin_host,
                             const int* cache_lens_host, int n_requests,
                             const lookm_cache_layout* layout, float* out, void* workspace,
                             size_t workspace_bytes, void* cuda_stream);

/* Byte offsets, inside the workspace, of the intermediate results a whole-path call leaves behind
 * (layouts as described at the top: scores [n_kv_heads, T] fp32, lse [n_q_heads, T] fp32,
 * rank [n_kv_heads, T] i32, kept/evicted/assign lists i32, sim fp32).  They stay valid until
 * the next call that uses the workspace and let a harness inspect every step of Eq. 4-9. */
typedef struct {
    size_t status, lse, scores, rank, kept_idx, evict_idx, assign, sim;
} lookm_workspace_offsets;
int lookm_workspace_layout(const lookm_layout* layout, int n_requests, const int* seq_lens_host,
                           lookm_workspace_offsets* offsets_host);

/* The merging step for callers that must not allocate device memory.  (The paper has no
 * counterpart to this entry point; it exists for deployment reasons only.)
 *
 * Some hosts of this library cannot call cudaMalloc at the point where they compress a cache: an
 * inference server that has handed all device memory to its own pool and forbids driver
 * allocations on the serving path (they serialise with other streams), or a plug-in that runs
 * inside someone else's memory budget and has nowhere to put a workspace.  For them this variant
 * of lookm_merge keeps its scratch (request table, entry lists, sort buffers, partial-sum records,
 * status word) in a fixed array inside the library's device image, LOOKM_NOALLOC_SCRATCH_BYTES
 * large, which every GPU that loads the library holds until the process exits.  Inputs and outputs are still the
 * caller's, with the meaning and layouts of lookm_merge.
 *
 * Limits: the scratch needs 28 bytes per (KV head, token), 4 per kept row and about 2.5 KB for
 * each of the merge kernel's work units (one per warp of the GPU, about 6 MB on a 148-SM part), so
 * n_kv_heads * total_tokens may be at most about 330,000 (32 heads x 8192 tokens uses 13.7 MB);
 * larger batches return LOOKM_ERR_WORKSPACE_TOO_SMALL before anything is enqueued.
 * The call performs no cudaMalloc/cudaFree and calls no allocating routine.
 *
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 * that device current) and caches it.  With lazy module loading that look-up can make the driver
 * load this library's device image, the 16 MiB array included, at that moment: make the first
 * call (a tiny warm-up batch will do) at start-up, outside any stream capture and off the serving
 * path.  The cached address belongs to the device's primary context and is stale once that context
 * has been reset.
 *
 * All calls on a device share the one array, and it keeps what the previous call left in it.
 * Each call clears the status word and rewrites everything it later reads, so back-to-back calls
 * on one stream are safe; calls that can overlap on the GPU (different streams without an
 * ordering between them) race on the array and must be serialised by the caller.
 * lookm_noalloc_status() is lookm_device_status() for this scratch. */
#define LOOKM_NOALLOC_SCRATCH_BYTES (16u << 20)
int lookm_merge_noalloc(const void* k, const void* v, const int* kept_idx, const int* evict_idx,
                        const int* assign, const float* sim, const int* cu_seqlens_host,
                        int n_requests, const int* budgets_host, const int* merge_modes_host,
                        const lookm_layout* layout, int varlen_output, void* out_k, void* out_v,
                        void* cuda_stream);
int lookm_noalloc_status(void* cuda_stream);

/* Optional per-stage timing.  While set (per host thread), every whole-path call records the
 * caller's events (cudaEvent_t handles in a host array that must stay alive) on its stream at the
 * step boundaries: [0] start, [1] after the first score sweep, [2] after the second (Eq. 4),
 * [3] after the selection (Eq. 5-8; the same launch computes the key norms of Eq. 9), [4] after
 * the kept-key compaction, [5] after the matching (Eq. 9), [6] after the assignment inversion, [7] after merge + compaction (Eq. 10-12).
 * n_events must be LOOKM_N_STAGE_EVENTS; a NULL entry skips that boundary; pass NULL, 0 to stop.
 * Nothing is recorded otherwise. */
#define LOOKM_N_STAGE_EVENTS 8
int lookm_set_stage_events(void* const* events_host, int n_events);

/* Synchronises `cuda_stream`, then returns and clears the device status word kept at the start
 * of `workspace` (LOOKM_OK if no kernel reported a problem since the last call that used this
 * workspace began). */
int lookm_device_status(void* workspace, void* cuda_stream);

/* Self-test of what happens when a device-side wait runs out (deployment aid; Eq. 4-12 contain no
 * waits, so the paper has nothing to cite here).  Enqueues one CTA that waits, with the very wait
 * routine and abort protocol of the tensor-core kernels and a limit of `limit_us` microseconds
 * (1 .. 100000), on a barrier at which nobody ever arrives.  The wait expires, the CTA returns, and
 * lookm_device_status(workspace, stream) then reports LOOKM_ERR_DEVICE_TIMEOUT; the CUDA context
 * stays usable.  workspace: at least 256 bytes, 256-byte aligned (only its status word is used). */
int lookm_selftest_wait_expiry(int limit_us, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Number of kernels the last call on this host thread enqueued (for launch accounting). */
int lookm_last_launch_count(void);

const char* lookm_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* LOOKM_H_ */
