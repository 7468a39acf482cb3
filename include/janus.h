/*
 * janus.h - C boundary of the B200 append-prefill library for top-k sparse-attention layers.
 *
 * One sparse layer of an append prefill runs, for the M newly appended tokens of a session with L cached
 * history tokens (S = L + M keys; the paper's P and L, Table 1):
 *
 *     janus_indexer_scores -> janus_topk -> janus_page_demand -> janus_sparse_attn_prefill
 *
 * Conventions (all entry points)
 *   - plain C ABI, no exceptions; every function returns an int status (JANUS_OK or JANUS_ERR_*).
 *   - every data pointer is a DEVICE pointer owned by the caller, unless a comment says "host".
 *     The library never allocates or frees device memory; scratch, where a call needs it, is the
 *     caller's `ws` buffer of at least janus_<fn>_workspace_size(...) bytes (may be NULL when 0).
 *     (janus_indexer_topk_static alone brings its own scratch: a fixed array in the library's device image.)
 *   - calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = default stream).
 *   - host-detectable problems (NULL pointer, bad size, misalignment, unsupported shape) return an
 *     error code and launch nothing.
 *   - conditions only visible on the device (index out of range, output capacity exceeded, a bounded
 *     wait that gave up) are written to *dev_status (first error wins; 0 = none) and the offending
 *     element is skipped; nothing traps.  dev_status may be NULL.  The caller zeroes it.
 *   - positions, token indices and page ids are 0-based.  Padding in index arrays is -1.
 */
#ifndef JANUS_H_
#define JANUS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* host return codes */
#define JANUS_OK 0
#define JANUS_ERR_INVALID_ARG 1         /* NULL/negative/misaligned argument                      */
#define JANUS_ERR_UNSUPPORTED 2         /* shape or dtype combination has no kernel               */
#define JANUS_ERR_WORKSPACE_TOO_SMALL 3
#define JANUS_ERR_CUDA 4                /* a CUDA call failed; see janus_last_cuda_error()        */

/* values written to *dev_status by kernels */
#define JANUS_DEV_OK 0
#define JANUS_DEV_INDEX_OUT_OF_RANGE 101   /* a token index or page id outside its table (skipped)   */
#define JANUS_DEV_CAPACITY_EXCEEDED 102    /* more pages/runs than `capacity`; counts are still true */
#define JANUS_DEV_WAIT_TIMEOUT 103         /* a bounded in-kernel wait gave up; output is incomplete */

/* dtype of the indexer operands */
#define JANUS_DTYPE_BF16 0
#define JANUS_DTYPE_FP8_E4M3 1
#define JANUS_DTYPE_FP8_Q_FP4_K 2   /* FP8 E4M3 queries, FP4 E2M1 keys (Sec. 5.1), two per byte, element 2i in the low nibble of
                                       byte i; k_stride_tok counts elements (a multiple of 64), k_idx is 32-byte aligned,
                                       D_I = 128, scales as for FP8.  Taken by janus_indexer_scores, janus_indexer_topk(_static)
                                       and janus_indexer_scores_batch, on tensor-core shapes only (else JANUS_ERR_UNSUPPORTED);
                                       janus_indexer_topk then works through a score matrix in its workspace */

/* Library version (major*10000 + minor*100 + patch). */
int janus_version(void);

/* cudaError_t of the most recent failed CUDA call made by this library on the calling thread (0 if none). */
int janus_last_cuda_error(void);

/*
 * Indexer scores - the scoring half of Eq. 1 (Sec. 2.2): relevance of every visible token for each new token.
 * The paper leaves the scoring function to the model reports; this library computes, in fp32 accumulation,
 *
 *     scores[t, s] = sum_{h < H_I} w[t, h] * max(0, < q_idx[t, h, :], k_idx[s, :] >)  (+ row_bias[t] * col_bias[s])
 *
 * for s <= q_pos0 + t when `causal` (the token itself included), for every s < n_keys otherwise; masked entries
 * are written as -inf.  One indexer key per token is shared by all indexer heads.
 *
 *   q_idx        [M, H_I, D_I]   bf16 or E4M3 bytes; token stride q_stride_tok elements (>= H_I*D_I), heads contiguous
 *   k_idx        [n_keys, D_I]   same dtype; token stride k_stride_tok elements
 *   w            [M, H_I]        fp32, any sign
 *   q_scale      FP8 only: per-head scales [H_I] (q_scale_stride_tok = 0) or per (token, head) [M, H_I]
 *                (q_scale_stride_tok = H_I); every scale > 0.  NULL for bf16.  True query = e4m3 * q_scale.
 *   k_scale      FP8 only: per-key scales [n_keys], every scale > 0.  NULL for bf16.
 *   row_bias, col_bias  optional rank-1 additive term, both NULL or both given ([M] and [n_keys] fp32).
 *   q_pos0       position of new token 0 among the keys (= L for an append prefill over history + new tokens)
 *   scores       [M, scores_ld] fp32 out, scores_ld >= n_keys and a multiple of 4; columns >= n_keys untouched
 *
 * D_I must be a multiple of 16.  Pointers must be 16-byte aligned; strides multiples of 16 bytes.
 * The tensor-core kernel serves H_I in {4, 8, 16, 32, 64} with D_I in {64, 128} and dense q_idx
 * (q_stride_tok == H_I*D_I); other shapes run a slower general kernel.
 */
size_t janus_indexer_scores_workspace_size(int M, int H_I, int D_I, int64_t n_keys, int dtype);
int janus_indexer_scores(const void* q_idx, int64_t q_stride_tok,
                         const void* k_idx, int64_t k_stride_tok,
                         const float* w,
                         const float* q_scale, int64_t q_scale_stride_tok,
                         const float* k_scale,
                         const float* row_bias, const float* col_bias,
                         int M, int H_I, int D_I, int64_t n_keys,
                         int64_t q_pos0, int causal, int dtype,
                         float* scores, int64_t scores_ld,
                         void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);

/*
 * Per-row top-k - the selection half of Eq. 1 (Sec. 2.2): for each new token, the indices of its
 * min(k, prefix) highest-scoring visible keys, prefix = min(n_keys, q_pos0 + t + 1) when causal, else n_keys.
 * Only scores[t, 0:prefix] is read.  Ties at the threshold are broken arbitrarily; output order is
 * unspecified; unused slots are -1.  NaN scores are not supported.
 *
 *   scores  [M, scores_ld] fp32 (scores_ld a multiple of 4, base 16-byte aligned)
 *   idx     [M, k] int32 out
 *   count   [M] int32 out (number of valid indices per row) or NULL
 *   kth     [M] fp32 out (the smallest selected score per row; -inf for an empty row) or NULL
 */
size_t janus_topk_workspace_size(int M, int64_t n_keys, int k);
int janus_topk(const float* scores, int64_t scores_ld, int M, int64_t n_keys,
               int64_t q_pos0, int causal, int k,
               int32_t* idx, int32_t* count, float* kth,
               void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);

/*
 * Indexer scores and per-row top-k in one call - Eq. 1 (Sec. 2.2) without the [M, n_keys] score matrix in memory.
 * Same operands and semantics as janus_indexer_scores followed by janus_topk (same masking, same tie freedom, same
 * outputs idx / count / kth); scores only ever exist as short per-row candidate lists in the workspace.
 * A sampled estimate of each row's k-th score decides which scores the indexer keeps; rows the estimate misjudges are
 * recomputed exactly, so the result never depends on the sample.  Shapes the tensor-core indexer does not take (and
 * head counts other than 64, or 32 with 256-byte rows), fewer than 16384 keys visible to every row, k > 4096 or more
 * than 8192 keys beyond the first row's prefix run the two calls internally with the scores in the workspace.
 *
 *   ws   device scratch of at least janus_indexer_topk_workspace_size(...) bytes, 16-byte aligned; contents undefined on
 *        return; two calls sharing a workspace must not overlap on the device.
 */
size_t janus_indexer_topk_workspace_size(int M, int H_I, int D_I, int64_t n_keys, int64_t q_pos0, int causal, int dtype, int k);
int janus_indexer_topk(const void* q_idx, int64_t q_stride_tok,
                       const void* k_idx, int64_t k_stride_tok,
                       const float* w,
                       const float* q_scale, int64_t q_scale_stride_tok,
                       const float* k_scale,
                       const float* row_bias, const float* col_bias,
                       int M, int H_I, int D_I, int64_t n_keys,
                       int64_t q_pos0, int causal, int dtype, int k,
                       int32_t* idx, int32_t* count, float* kth,
                       void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);
/* Diagnostic: byte offset inside `ws` of an int32 that holds, after janus_indexer_topk has run, how many rows the sampled
 * threshold misjudged (they were recomputed exactly, so the result does not depend on it); -1 when this problem takes
 * the score-matrix route and has no such counter.  Same arguments as janus_indexer_topk_workspace_size. */
int64_t janus_indexer_topk_fallback_counter_offset(int M, int H_I, int D_I, int64_t n_keys, int64_t q_pos0, int causal, int dtype, int k);

/*
 * janus_indexer_topk on scratch built into the library - no counterpart in the paper; a convenience of this library.
 *
 * Every other entry point takes its scratch from the caller.  This one is for callers that have none to give and cannot
 * get any: code running inside a host program that has already handed all free device memory to its own KV-cache pool
 * and lends none of it out, or a loop so latency-critical that it may not call the CUDA allocator (releasing device
 * memory waits for the device to go idle).  The call allocates and frees nothing, on the host side of CUDA or through
 * any library; its scratch is a fixed array of JANUS_STATIC_SCRATCH_BYTES in the library's device image, present once
 * on every device that loads the library.
 *
 * Arguments, outputs and semantics are those of janus_indexer_topk without `ws` / `ws_bytes`.
 *
 *   Limit     janus_indexer_topk_workspace_size(...) for the same arguments must not exceed
 *             JANUS_STATIC_SCRATCH_BYTES; otherwise the call returns JANUS_ERR_WORKSPACE_TOO_SMALL and touches
 *             nothing.  64 MiB covers, for example, 128 new tokens over 131072 cached keys, or 64 over 262144
 *             (64 x 128 FP8 indexer, k = 2048); a 4096-token chunk at that history needs the caller's workspace.
 *   Set-up    the first call on a device looks up the array's address on that device (no allocation) and keeps it;
 *             the device whose stream is passed must be the current device.  Make that first call before any
 *             stream capture begins.
 *   Sharing   all calls on one device use the same array.  Each call clears the counters it needs itself, so
 *             nothing has to be zeroed beforehand and leftovers of earlier calls do not matter; but two calls that
 *             may run at the same time (different streams, or different host threads without ordering between
 *             their streams) race on it and give wrong results.  Order them on one stream or with events.
 */
#define JANUS_STATIC_SCRATCH_BYTES (64 << 20)
int janus_indexer_topk_static(const void* q_idx, int64_t q_stride_tok,
                              const void* k_idx, int64_t k_stride_tok,
                              const float* w,
                              const float* q_scale, int64_t q_scale_stride_tok,
                              const float* k_scale,
                              const float* row_bias, const float* col_bias,
                              int M, int H_I, int D_I, int64_t n_keys,
                              int64_t q_pos0, int causal, int dtype, int k,
                              int32_t* idx, int32_t* count, float* kth,
                              int32_t* dev_status, void* stream);

/*
 * Page demand - union of the selections (Sec. 2.2), best-effort read packing into maximal runs of physically
 * adjacent pages (Sec. 4.3) and the corrective-read set "exact minus predicted" (Sec. 4.2).
 *
 *   A      = { page_table[s / page_size] : s in idx, 0 <= s < demand_limit }      (history tokens only: demand_limit = L)
 *   bitmap = A as n_phys_pages bits (bit p of word p/32), fully overwritten
 *   pages  = A ascending;  runs = maximal (start, len) with start..start+len-1 in A, ascending
 *   miss   = A minus the set in predicted_bitmap, ascending;  miss_runs = its maximal runs
 *
 *   idx               [n_rows, k] int32, any block of selections (-1 ignored)
 *   page_table        [n_logical_pages] int32 logical -> physical page id
 *   predicted_bitmap  NULL (then miss = A), or the `bitmap` output of an earlier call on the predicted selection
 *   pages, runs       out, room for `capacity` pages / `capacity` (start,len) pairs; counts in *n_pages, *n_runs (device)
 *   miss_pages, n_miss, miss_runs, n_miss_runs   out, all four given or all four NULL
 *
 * If a list would exceed `capacity`, only its first `capacity` entries are written, the count still holds the
 * true total and *dev_status becomes JANUS_DEV_CAPACITY_EXCEEDED.  Out-of-range tokens or page ids are skipped
 * with JANUS_DEV_INDEX_OUT_OF_RANGE.  Results are bit-exact and independent of launch geometry.
 */
size_t janus_page_demand_workspace_size(int64_t n_rows, int k, int64_t n_phys_pages);
int janus_page_demand(const int32_t* idx, int64_t n_rows, int k,
                      int64_t demand_limit, int page_size,
                      const int32_t* page_table, int64_t n_logical_pages, int64_t n_phys_pages,
                      const uint32_t* predicted_bitmap,
                      uint32_t* bitmap,
                      int32_t* pages, int32_t* n_pages,
                      int32_t* runs, int32_t* n_runs,
                      int32_t* miss_pages, int32_t* n_miss,
                      int32_t* miss_runs, int32_t* n_miss_runs,
                      int64_t capacity,
                      void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);

/*
 * Union of page sets - synchronisation-free parallel prediction (Sec. 4.2, Eq. 3): the history is cut into disjoint
 * shards, every shard selects its own top-(k/N) and builds its own page set with janus_page_demand; the predicted set
 * the exact pass is compared against is the union of the per-shard sets.
 *
 *     dst |= src        (both bitmaps of n_phys_pages bits, as written by janus_page_demand)
 */
int janus_page_union(uint32_t* dst, const uint32_t* src, int64_t n_phys_pages, void* stream);

/*
 * Sparse attention over the selected rows only (Sec. 2.2, "core attention"):
 *
 *     out[t, h, :] = sum_{s in idx[t]} softmax_s( softmax_scale * < q[t, h, :d_qk], K_s[:d_qk] > ) * V_s[:d_v]
 *
 * with an fp32 online softmax.  Token s lives at element offset
 *     page_table[s / page_size] * page_stride + (s % page_size) * tok_stride + h_kv * head_stride
 * of k_pool (keys, d_qk values) and v_pool (values, d_v values); query head h reads kv head h * n_kv_heads / H_q.
 * v_pool may alias k_pool (latent layout: the value is the first d_v dims of the key row; then d_v <= d_qk, else
 * JANUS_ERR_INVALID_ARG).
 * A selected token beyond the page table, or whose page table entry is negative, is skipped with
 * JANUS_DEV_INDEX_OUT_OF_RANGE.  The upper end of the pool is not known to this call: a physical page id past the pool
 * is NOT caught here.  janus_page_demand on the same idx and page table checks every id against n_phys_pages.
 *
 *   q     [M, H_q, d_qk] bf16, dense
 *   idx   [M, k] int32, -1 padded (any position); duplicates are attended twice
 *   out   [M, H_q, d_v] bf16 out (round-to-nearest-even); an empty selection gives zeros
 *   lse   [M, H_q] fp32 out, log-sum-exp of the scaled logits (-inf for an empty selection), or NULL
 *
 * d_qk and d_v multiples of 8, d_qk <= 576, d_v <= 512, H_q a multiple of n_kv_heads; strides (in elements)
 * multiples of 8.  The tensor-core kernel serves the latent shape (n_kv_heads = 1, H_q = 128, d_qk = 576, d_v = 512).
 */
size_t janus_sparse_attn_prefill_workspace_size(int M, int H_q, int d_qk, int d_v, int k);
int janus_sparse_attn_prefill(const void* q, int M, int H_q, int d_qk,
                              const void* k_pool, const void* v_pool,
                              int64_t page_stride, int64_t tok_stride, int64_t head_stride,
                              int n_kv_heads, int d_v,
                              const int32_t* idx, int k,
                              int page_size, const int32_t* page_table, int64_t n_logical_pages,
                              float softmax_scale,
                              void* out, float* lse,
                              void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);

/*
 * Entry granularity - selection and attention per entry, a region of `entry_size` consecutive tokens (footnote of
 * Sec. 2.2; the paper does not define the entry-level scoring or masking, this library's reading is stated here).
 * The indexer has one key per entry: entry scores are janus_indexer_scores over the entry keys with causal = 0.
 *
 *   janus_topk_entries   janus_topk over entries: row t (position q_pos0 + t) may select the entries that hold a token at
 *                        or before its position, i.e. entries 0 .. (q_pos0 + t) / entry_size.  scores [M, scores_ld] fp32.
 *   janus_entry_expand   idx_tokens[t, e * entry_size + j] = idx_entries[t, e] * entry_size + j if that token is at or
 *                        before position q_pos0 + t, else -1 ([M, k_e * entry_size] int32).  The result feeds
 *                        janus_page_demand and janus_sparse_attn_prefill like any token selection.
 *
 *   janus_entry_pool_scores   the other reading of the same footnote: the indexer scores tokens as usual and an entry's
 *                        score is the maximum over its tokens that the row may see,
 *                            entry_scores[t, e] = max { scores[t, s] : e*E <= s < (e+1)*E, s <= q_pos0 + t }   (causal;
 *                            every token of the entry otherwise), -inf for an entry without a visible token.
 *                        scores [M, scores_ld] fp32 from janus_indexer_scores; entry_scores [M, entry_ld] fp32 out,
 *                        entry_ld >= ceil(n_keys / entry_size) (a multiple of 4 if janus_topk_entries follows).
 *
 * A selection shared by a group of layers (index reuse) needs no call of its own: pass the same idx to the attention of
 * every layer of the group.
 */
int janus_topk_entries(const float* scores, int64_t scores_ld, int M, int64_t n_entries,
                       int64_t q_pos0, int entry_size, int k,
                       int32_t* idx, int32_t* count, float* kth, int32_t* dev_status, void* stream);
int janus_entry_pool_scores(const float* scores, int64_t scores_ld, int M, int64_t n_keys, int64_t q_pos0, int causal,
                            int entry_size, float* entry_scores, int64_t entry_ld, void* stream);
int janus_entry_expand(const int32_t* idx_entries, int M, int k_e, int entry_size, int64_t q_pos0,
                       int32_t* idx_tokens, void* stream);

/*
 * Decode step over a batch of sessions (Sec. 2.2, "Decode phase"): one new token per session, processed like an append
 * prefill with a single appended token.  Session b has its own history, so the per-session arrays are concatenated and
 * addressed through offsets held in device memory:
 *
 *   key_offsets    [B + 1] int64: session b's indexer keys (cached history plus the new token's own key) are rows
 *                  key_offsets[b] .. key_offsets[b+1] of k_idx; every offset is a multiple of 4 (pad between sessions),
 *                  so that score rows stay 16-byte aligned.  k_scale / col_bias / scores use the same row numbering.
 *   table_offsets  [B + 1] int64: session b's page table is page_tables[table_offsets[b] .. table_offsets[b+1]);
 *                  physical page ids are global (one KV pool for all sessions).
 *
 * janus_indexer_scores_batch   scores[key_offsets[b] + s] = indexer score of session b's query against its key s
 *                              (no causal mask: the new token sees all of its session's keys).  q_idx [B, H_I, D_I]
 *                              contiguous, w [B, H_I], q_scale [B, H_I] or [H_I]; max_keys = an upper bound of the
 *                              longest session (host value, sizes the launch; at most total_keys, else
 *                              JANUS_ERR_INVALID_ARG); total_keys = rows of k_idx.  A session whose offsets leave
 *                              [0, total_keys] is cut back to the part inside with JANUS_DEV_INDEX_OUT_OF_RANGE.
 *                              Tensor-core path only: H_I = 64 and 128- or 256-byte rows, else JANUS_ERR_UNSUPPORTED.
 *                              dtype JANUS_DTYPE_FP8_Q_FP4_K: keys packed two per byte (D_I = 128, k_idx 32-byte aligned,
 *                              k_stride_tok a multiple of 64 elements), scales as for FP8.
 * janus_topk_batch             idx[b, 0:k) = top-k of the row_lengths[b] scores starting at scores[row_offsets[b]] (positions inside
 *                              the session, -1 padded), count / kth as in janus_topk.  row_offsets [B + 1] and row_lengths
 *                              [B] are int64 device arrays; row_lengths may be NULL (rows then run up to the next offset);
 *                              offsets are multiples of 4.  A row whose offset is negative or not a multiple of 4, or whose
 *                              length is negative, is left empty (idx -1, count 0) with JANUS_DEV_INDEX_OUT_OF_RANGE.
 * janus_page_demand_batch      janus_page_demand over all rows at once: row r marks page_tables[table_offsets[r] + s / page_size]
 *                              for its selected tokens s < demand_limits[r] (the session's cached history length) into one
 *                              bitmap over the global pool; lists, runs and the miss set against `predicted_bitmap` (for
 *                              decode: the pages already resident) as in janus_page_demand.  A negative table offset
 *                              makes that row's table empty (its tokens are reported and skipped).
 * janus_sparse_attn_decode     janus_sparse_attn_prefill with one query row per session and per-row page tables.
 */
int janus_indexer_scores_batch(const void* q_idx, const void* k_idx, int64_t k_stride_tok,
                               const float* w,
                               const float* q_scale, int64_t q_scale_stride_tok,
                               const float* k_scale,
                               const float* row_bias, const float* col_bias,
                               int B, int H_I, int D_I,
                               const int64_t* key_offsets, int64_t total_keys, int64_t max_keys,
                               int dtype, float* scores, int32_t* dev_status, void* stream);
int janus_topk_batch(const float* scores, const int64_t* row_offsets, const int64_t* row_lengths, int B, int k,
                     int32_t* idx, int32_t* count, float* kth, int32_t* dev_status, void* stream);
int janus_page_demand_batch(const int32_t* idx, int64_t n_rows, int k,
                            const int64_t* demand_limits, int page_size,
                            const int32_t* page_tables, const int64_t* table_offsets, int64_t n_phys_pages,
                            const uint32_t* predicted_bitmap,
                            uint32_t* bitmap,
                            int32_t* pages, int32_t* n_pages,
                            int32_t* runs, int32_t* n_runs,
                            int32_t* miss_pages, int32_t* n_miss,
                            int32_t* miss_runs, int32_t* n_miss_runs,
                            int64_t capacity, int32_t* dev_status, void* stream);
int janus_sparse_attn_decode(const void* q, int B, int H_q, int d_qk,
                             const void* k_pool, const void* v_pool,
                             int64_t page_stride, int64_t tok_stride, int64_t head_stride,
                             int n_kv_heads, int d_v,
                             const int32_t* idx, int k, int page_size,
                             const int32_t* page_tables, const int64_t* table_offsets,
                             float softmax_scale, void* out, float* lse,
                             int32_t* dev_status, void* stream);

/*
 * Diagnostics.  The paper has no counterpart for either call.
 *
 * janus_selftest_bounded_wait   Every wait inside the tensor-core kernels (on an mbarrier: a copy that has not landed, a
 *                               tensor-memory slot that is not free) gives up after a fixed number of polls, writes
 *                               JANUS_DEV_WAIT_TIMEOUT to *dev_status and lets the kernel return normally.  This call runs
 *                               that wait on a barrier nobody arrives on, with `max_polls` polls (1 .. 65536), so that the
 *                               time-out path can be exercised without a broken pipeline: afterwards *dev_status is
 *                               JANUS_DEV_WAIT_TIMEOUT, *elapsed_ns (device int64, may be NULL) holds how long the wait
 *                               took, and the context is as usable as before.
 * janus_fp8_mma_probe           Launches `n_ctas` CTAs (one per SM is the intended use) that each issue `fills_per_cta`
 *                               dense FP8 E4M3 tensor-core accumulator fills (M = 128, N = 256, K = 128; operands in shared
 *                               memory, nothing else in the kernel) and writes the launch's flop count to *flop_per_launch
 *                               (host double, may be NULL).  Timed by the caller with events on `stream`, it gives the FP8
 *                               tensor rate this GPU sustains under its power limit: the denominator of the indexer's
 *                               roofline fraction.  Asynchronous; uses no device memory besides *dev_status.
 */
int janus_selftest_bounded_wait(int max_polls, int64_t* elapsed_ns, int32_t* dev_status, void* stream);
int janus_fp8_mma_probe(int n_ctas, int fills_per_cta, double* flop_per_launch /* host */, int32_t* dev_status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* JANUS_H_ */
