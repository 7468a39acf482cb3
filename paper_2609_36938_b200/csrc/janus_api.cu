// Entry points that validate arguments and pick a kernel: janus_indexer_scores, janus_sparse_attn_prefill,
// plus the version / error queries.  janus_topk and janus_page_demand live beside their kernels.
#include "janus_common.cuh"

namespace janus {

static thread_local int g_last_cuda_error = 0;
void set_last_cuda_error(cudaError_t e) { g_last_cuda_error = static_cast<int>(e); }

int launch_indexer_generic(const void* q_idx, int64_t q_stride_tok, const void* k_idx, int64_t k_stride_tok, const float* w,
                           const float* q_scale, int64_t q_scale_stride_tok, const float* k_scale, const float* row_bias,
                           const float* col_bias, int M, int H, int D, int64_t n_keys, int64_t q_pos0, int causal, int dtype,
                           float* scores, int64_t ld, cudaStream_t stream);
bool indexer_tc_supported(int M, int H, int D, int64_t n_keys, int64_t q_stride_tok, int64_t k_stride_tok, int dtype);
int launch_indexer_tc(const void* q_idx, const void* k_idx, int64_t k_stride_tok, const float* w, const float* q_scale,
                      int64_t q_scale_stride_tok, const float* k_scale, const float* row_bias, const float* col_bias, int M, int H,
                      int D, int64_t n_keys, int64_t q_pos0, int causal, int dtype, float* scores, int64_t ld, int32_t* dev_status,
                      cudaStream_t stream, const float* thr = nullptr, int32_t* cand_cnt = nullptr, void* cand = nullptr, int cand_cap = 0);

bool indexer_tc_batch_supported(int B, int H, int D, int64_t total_keys, int dtype);
int launch_indexer_tc_batch(const void* q_idx, const void* k_idx, int64_t k_stride_tok, const float* w, const float* q_scale,
                            int64_t q_scale_stride_tok, const float* k_scale, const float* row_bias, const float* col_bias, int B, int H, int D,
                            int64_t total_keys, int64_t max_keys, const int64_t* key_offsets, int dtype, float* scores, int32_t* dev_status,
                            cudaStream_t stream);

int launch_sparse_attn_generic(const void* q, int M, int H_q, int d_qk, const void* k_pool, const void* v_pool, int64_t page_stride,
                               int64_t tok_stride, int64_t head_stride, int n_kv_heads, int d_v, const int32_t* idx, int k,
                               int page_size, const int32_t* page_table, int64_t n_logical_pages, const int64_t* table_offsets,
                               float softmax_scale, void* out, float* lse, int32_t* dev_status, cudaStream_t stream);

bool sparse_attn_latent_tc_supported(int M, int H_q, int d_qk, const void* k_pool, const void* v_pool, int64_t page_stride,
                                     int64_t tok_stride, int n_kv_heads, int d_v, int k);
int launch_sparse_attn_latent_tc(const void* q, int M, const void* pool, int64_t page_stride, int64_t tok_stride, const int32_t* idx, int k,
                                 int page_size, const int32_t* page_table, int64_t n_logical_pages, const int64_t* table_offsets,
                                 float softmax_scale, void* out, float* lse, int32_t* dev_status, cudaStream_t stream);

// Host-side checks shared by the entry points that take indexer operands.  JANUS_OK also for empty problems.
int validate_indexer_args(const void* q_idx, int64_t q_stride_tok, const void* k_idx, int64_t k_stride_tok, const float* w,
                          const float* q_scale, int64_t q_scale_stride_tok, const float* k_scale, const float* row_bias,
                          const float* col_bias, int M, int H_I, int D_I, int64_t n_keys, int64_t q_pos0, int dtype) {
    if (M < 0 || H_I <= 0 || D_I <= 0 || n_keys < 0 || q_pos0 < 0) return JANUS_ERR_INVALID_ARG;
    const bool k_fp4 = dtype == JANUS_DTYPE_FP8_Q_FP4_K;
    if (dtype != JANUS_DTYPE_BF16 && dtype != JANUS_DTYPE_FP8_E4M3 && !k_fp4) return JANUS_ERR_UNSUPPORTED;
    if ((D_I % 16) != 0) return JANUS_ERR_UNSUPPORTED;
    if (M == 0 || n_keys == 0) return JANUS_OK;
    const int esz = dtype == JANUS_DTYPE_BF16 ? 2 : 1;
    if (!q_idx || !k_idx || !w) return JANUS_ERR_INVALID_ARG;
    if (!aligned16(q_idx) || !aligned16(k_idx)) return JANUS_ERR_INVALID_ARG;
    if (q_stride_tok < static_cast<int64_t>(H_I) * D_I || k_stride_tok < D_I) return JANUS_ERR_INVALID_ARG;
    if ((q_stride_tok * esz) % 16 != 0) return JANUS_ERR_INVALID_ARG;
    if (k_fp4) {   // two key elements per byte: rows start on 32-byte boundaries (what the 4-bit tensor-map type asks for)
        if ((k_stride_tok % 64) != 0 || (reinterpret_cast<uintptr_t>(k_idx) & 31u) != 0) return JANUS_ERR_INVALID_ARG;
    } else if ((k_stride_tok * esz) % 16 != 0) {
        return JANUS_ERR_INVALID_ARG;
    }
    if ((row_bias == nullptr) != (col_bias == nullptr)) return JANUS_ERR_INVALID_ARG;
    if (dtype != JANUS_DTYPE_BF16) {
        if (!q_scale || !k_scale) return JANUS_ERR_INVALID_ARG;
        if (q_scale_stride_tok != 0 && q_scale_stride_tok != H_I) return JANUS_ERR_INVALID_ARG;
    } else if (q_scale || k_scale) {
        return JANUS_ERR_INVALID_ARG;
    }
    return JANUS_OK;
}

}  // namespace janus

extern "C" int janus_version(void) { return 100; }

extern "C" int janus_last_cuda_error(void) { return janus::g_last_cuda_error; }

extern "C" size_t janus_indexer_scores_workspace_size(int, int, int, int64_t, int) { return 0; }

extern "C" int janus_indexer_scores(const void* q_idx, int64_t q_stride_tok, const void* k_idx, int64_t k_stride_tok, const float* w,
                                    const float* q_scale, int64_t q_scale_stride_tok, const float* k_scale, const float* row_bias,
                                    const float* col_bias, int M, int H_I, int D_I, int64_t n_keys, int64_t q_pos0, int causal,
                                    int dtype, float* scores, int64_t scores_ld, void* /*ws*/, size_t /*ws_bytes*/,
                                    int32_t* dev_status, void* stream_) {
    using namespace janus;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int vrc = validate_indexer_args(q_idx, q_stride_tok, k_idx, k_stride_tok, w, q_scale, q_scale_stride_tok, k_scale, row_bias, col_bias,
                                          M, H_I, D_I, n_keys, q_pos0, dtype);
    if (vrc != JANUS_OK) return vrc;
    if (M == 0 || n_keys == 0) return JANUS_OK;
    if (!scores || !aligned16(scores)) return JANUS_ERR_INVALID_ARG;
    if (scores_ld < n_keys || (scores_ld & 3) != 0) return JANUS_ERR_INVALID_ARG;
    if (indexer_tc_supported(M, H_I, D_I, n_keys, q_stride_tok, k_stride_tok, dtype))
        return launch_indexer_tc(q_idx, k_idx, k_stride_tok, w, q_scale, q_scale_stride_tok, k_scale, row_bias, col_bias, M, H_I, D_I,
                                 n_keys, q_pos0, causal, dtype, scores, scores_ld, dev_status, stream);
    if (dtype == JANUS_DTYPE_FP8_Q_FP4_K) return JANUS_ERR_UNSUPPORTED;   // 4-bit keys: tensor-core shapes only
    return launch_indexer_generic(q_idx, q_stride_tok, k_idx, k_stride_tok, w, q_scale, q_scale_stride_tok, k_scale, row_bias, col_bias,
                                  M, H_I, D_I, n_keys, q_pos0, causal, dtype, scores, scores_ld, stream);
}

extern "C" int janus_indexer_scores_batch(const void* q_idx, const void* k_idx, int64_t k_stride_tok, const float* w, const float* q_scale,
                                          int64_t q_scale_stride_tok, const float* k_scale, const float* row_bias, const float* col_bias,
                                          int B, int H_I, int D_I, const int64_t* key_offsets, int64_t total_keys, int64_t max_keys,
                                          int dtype, float* scores, int32_t* dev_status, void* stream_) {
    using namespace janus;
    // FP4 keys: the shared checks see an FP8 problem (queries are FP8, the scales are the same); the key array has its own rules
    const bool k_fp4 = dtype == JANUS_DTYPE_FP8_Q_FP4_K;
    if (k_fp4 && B > 0 && total_keys > 0 &&
        (D_I != 128 || (k_stride_tok % 64) != 0 || (reinterpret_cast<uintptr_t>(k_idx) & 31u) != 0)) return k_idx ? JANUS_ERR_UNSUPPORTED : JANUS_ERR_INVALID_ARG;
    const int vrc = validate_indexer_args(q_idx, static_cast<int64_t>(H_I) * D_I, k_idx, k_stride_tok, w, q_scale, q_scale_stride_tok, k_scale,
                                          row_bias, col_bias, B, H_I, D_I, total_keys, 0, k_fp4 ? JANUS_DTYPE_FP8_E4M3 : dtype);
    if (vrc != JANUS_OK) return vrc;
    if (max_keys < 0 || max_keys > total_keys) return JANUS_ERR_INVALID_ARG;
    if (B == 0 || total_keys == 0) return JANUS_OK;
    if (!key_offsets || !scores || !aligned16(scores)) return JANUS_ERR_INVALID_ARG;
    if (!indexer_tc_batch_supported(B, H_I, D_I, total_keys, dtype)) return JANUS_ERR_UNSUPPORTED;
    return launch_indexer_tc_batch(q_idx, k_idx, k_stride_tok, w, q_scale, q_scale_stride_tok, k_scale, row_bias, col_bias, B, H_I, D_I,
                                   total_keys, max_keys, key_offsets, dtype, scores, dev_status, static_cast<cudaStream_t>(stream_));
}

extern "C" size_t janus_sparse_attn_prefill_workspace_size(int, int, int, int, int) { return 0; }

namespace janus {
// Shared by the prefill and the decode entry points: `table_offsets` is NULL (one page table for all rows) or [M + 1].
static int sparse_attn_dispatch(const void* q, int M, int H_q, int d_qk, const void* k_pool, const void* v_pool, int64_t page_stride,
                                int64_t tok_stride, int64_t head_stride, int n_kv_heads, int d_v, const int32_t* idx, int k, int page_size,
                                const int32_t* page_table, int64_t n_logical_pages, const int64_t* table_offsets, float softmax_scale,
                                void* out, float* lse, int32_t* dev_status, cudaStream_t stream) {
    if (M < 0 || H_q <= 0 || d_qk <= 0 || d_v <= 0 || n_kv_heads <= 0 || k < 0 || page_size <= 0 || n_logical_pages < 0)
        return JANUS_ERR_INVALID_ARG;
    if (H_q % n_kv_heads != 0) return JANUS_ERR_INVALID_ARG;
    if ((d_qk % 8) != 0 || (d_v % 8) != 0 || d_qk > 576 || d_v > 512) return JANUS_ERR_UNSUPPORTED;
    if (M == 0) return JANUS_OK;
    if (!q || !k_pool || !v_pool || !out || !page_table || (k > 0 && !idx)) return JANUS_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_pool) || !aligned16(v_pool) || !aligned16(out)) return JANUS_ERR_INVALID_ARG;
    if ((page_stride % 8) != 0 || (tok_stride % 8) != 0 || (head_stride % 8) != 0) return JANUS_ERR_INVALID_ARG;
    if (v_pool == k_pool && d_v > d_qk) return JANUS_ERR_INVALID_ARG;   // an aliased value row is a prefix of the key row
    if (M > 2147483647 / 2) return JANUS_ERR_UNSUPPORTED;
    if (softmax_scale > 0.f &&
        sparse_attn_latent_tc_supported(M, H_q, d_qk, k_pool, v_pool, page_stride, tok_stride, n_kv_heads, d_v, k))
        return launch_sparse_attn_latent_tc(q, M, k_pool, page_stride, tok_stride, idx, k, page_size, page_table, n_logical_pages,
                                            table_offsets, softmax_scale, out, lse, dev_status, stream);
    return launch_sparse_attn_generic(q, M, H_q, d_qk, k_pool, v_pool, page_stride, tok_stride, head_stride, n_kv_heads, d_v, idx, k,
                                      page_size, page_table, n_logical_pages, table_offsets, softmax_scale, out, lse, dev_status, stream);
}
}  // namespace janus

extern "C" int janus_sparse_attn_prefill(const void* q, int M, int H_q, int d_qk, const void* k_pool, const void* v_pool,
                                         int64_t page_stride, int64_t tok_stride, int64_t head_stride, int n_kv_heads, int d_v,
                                         const int32_t* idx, int k, int page_size, const int32_t* page_table,
                                         int64_t n_logical_pages, float softmax_scale, void* out, float* lse, void* /*ws*/,
                                         size_t /*ws_bytes*/, int32_t* dev_status, void* stream_) {
    return janus::sparse_attn_dispatch(q, M, H_q, d_qk, k_pool, v_pool, page_stride, tok_stride, head_stride, n_kv_heads, d_v, idx, k, page_size,
                                       page_table, n_logical_pages, nullptr, softmax_scale, out, lse, dev_status,
                                       static_cast<cudaStream_t>(stream_));
}

extern "C" int janus_sparse_attn_decode(const void* q, int B, int H_q, int d_qk, const void* k_pool, const void* v_pool,
                                        int64_t page_stride, int64_t tok_stride, int64_t head_stride, int n_kv_heads, int d_v,
                                        const int32_t* idx, int k, int page_size, const int32_t* page_tables,
                                        const int64_t* table_offsets, float softmax_scale, void* out, float* lse,
                                        int32_t* dev_status, void* stream_) {
    if (B > 0 && !table_offsets) return JANUS_ERR_INVALID_ARG;
    return janus::sparse_attn_dispatch(q, B, H_q, d_qk, k_pool, v_pool, page_stride, tok_stride, head_stride, n_kv_heads, d_v, idx, k, page_size,
                                       page_tables, 0, table_offsets, softmax_scale, out, lse, dev_status, static_cast<cudaStream_t>(stream_));
}
