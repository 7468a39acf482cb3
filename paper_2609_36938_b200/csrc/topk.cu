// janus_topk: per-row selection of the k largest scores over the causal prefix (Eq. 1, Sec. 2.2).
//
// A CTA works on one query row at a time; the CTAs resident on the device walk the rows with stride gridDim.x.  The row
// (0.5-1 MB of fp32 at 128K-256K keys) is read from HBM once:
//   1. a strided sample of the row (512 x 32-byte sectors) gives a conservative threshold whose
//      expected rank is a little above k;
//   2. one streaming pass with 16-byte loads keeps only the elements at or above that threshold
//      in a shared-memory candidate buffer (~1.5-3 % of the row pass the one-compare filter);
//   3. an exact selection runs on the candidates in shared memory: 2048-bucket histograms over a
//      shrinking key range (buckets are linear in the order-preserving integer key, so they spread
//      over whatever range the scores occupy) until the bucket of the k-th key holds at most 256
//      keys, which are then ranked directly.
// If the sample misjudges the row (fewer than k candidates, or more than the buffer holds) the
// same exact selection runs over the row in global memory instead; that path is slower, never
// wrong.  Rows that fit the buffer skip the sampling step.
#include <algorithm>

#include "topk_select.cuh"

namespace janus {

constexpr int TK_CAP = 8192;        // 73 KB of shared memory per CTA keeps three CTAs on an SM
constexpr int TK_CAP_SMALL = 5632;  // 54 KB: four CTAs on an SM (all 2048 threads), for rows whose candidate list is sure to fit

template <int CAP>
__global__ void __launch_bounds__(TK_THREADS)
topk_rows_kernel(const float* __restrict__ scores, int64_t ld, int M, int64_t n_keys, int64_t q_pos0, int causal, int k,
                 int32_t* __restrict__ idx, int32_t* __restrict__ count, float* __restrict__ kth) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    using TopkShared = TopkSharedT<CAP>;
    TopkShared& sh = *reinterpret_cast<TopkShared*>(smem_raw);
    // resident CTAs walk the rows with stride gridDim.x, each asking for the head of its next row ahead of time
    for (int t = blockIdx.x; t < M; t += gridDim.x) {
        const int64_t prefix64 = causal ? min(n_keys, q_pos0 + t + 1) : n_keys;
        const int t_next = t + gridDim.x;
        const int64_t prefix_next = t_next < M ? (causal ? min(n_keys, q_pos0 + t_next + 1) : n_keys) : 0;
        topk_row(scores + static_cast<int64_t>(t) * ld, static_cast<int>(prefix64), k, t, idx + static_cast<int64_t>(t) * k, count, kth, sh,
                 t_next < M ? scores + static_cast<int64_t>(t_next) * ld : nullptr, static_cast<int>(prefix_next));
        __syncthreads();   // the selection state in shared memory is reused by the next row
    }
}

// Entry granularity (footnote of Sec. 2.2): columns are entries of `entry_size` consecutive tokens; row t (position
// q_pos0 + t) may select the entries that hold a token at or before its position: entries 0 .. (q_pos0 + t) / entry_size.
template <int CAP>
__global__ void __launch_bounds__(TK_THREADS)
topk_entries_kernel(const float* __restrict__ scores, int64_t ld, int M, int64_t n_entries, int64_t q_pos0, int entry_size, int k,
                    int32_t* __restrict__ idx, int32_t* __restrict__ count, float* __restrict__ kth) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    using TopkShared = TopkSharedT<CAP>;
    TopkShared& sh = *reinterpret_cast<TopkShared*>(smem_raw);
    const int t = blockIdx.x;
    int64_t prefix = (q_pos0 + t) / entry_size + 1;
    if (prefix > n_entries) prefix = n_entries;
    topk_row(scores + static_cast<int64_t>(t) * ld, static_cast<int>(prefix), k, t, idx + static_cast<int64_t>(t) * k, count, kth, sh);
}

// Token selection of an entry selection: slot e * E + j of row t = entry * E + j if that token is at or before q_pos0 + t.
__global__ void entry_expand_kernel(const int32_t* __restrict__ idx_e, int M, int k_e, int entry_size, int64_t q_pos0,
                                    int32_t* __restrict__ idx_tok) {
    const int64_t n = static_cast<int64_t>(M) * k_e * entry_size;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t slot = i / entry_size;            // (t, e)
        const int j = static_cast<int>(i - slot * entry_size);
        const int64_t t = slot / k_e;
        const int32_t ent = __ldg(idx_e + slot);
        const int64_t tok = static_cast<int64_t>(ent) * entry_size + j;
        idx_tok[i] = (ent >= 0 && tok <= q_pos0 + t) ? static_cast<int32_t>(tok) : -1;
    }
}

// Pooled entry scores (the second reading of the entry footnote of Sec. 2.2): an entry scores as the best of its tokens the
// row may see.  One warp per (row, entry) strip: lanes read consecutive floats (coalesced), a warp shuffle takes the maximum.
__global__ void __launch_bounds__(256)
entry_pool_kernel(const float* __restrict__ scores, int64_t ld, int M, int64_t n_keys, int64_t q_pos0, int causal, int entry_size,
                  int64_t n_entries, float* __restrict__ out, int64_t out_ld) {
    const int lane = threadIdx.x & 31;
    const int64_t warp_id = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    const int64_t n_warps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
    const float neg_inf = __int_as_float(0xff800000);
    for (int64_t item = warp_id; item < static_cast<int64_t>(M) * n_entries; item += n_warps) {
        const int64_t t = item / n_entries, e = item - t * n_entries;
        const int64_t prefix = causal ? (n_keys < q_pos0 + t + 1 ? n_keys : q_pos0 + t + 1) : n_keys;
        const int64_t a = e * entry_size;
        const int64_t b = a + entry_size < prefix ? a + entry_size : prefix;
        const float* row = scores + t * ld;
        float m = neg_inf;
        for (int64_t s = a + lane; s < b; s += 32) m = fmaxf(m, __ldg(row + s));
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
        if (lane == 0) out[t * out_ld + e] = m;
    }
}

// Batch form (decode over many sessions): row b starts at scores[row_offsets[b]] and has row_lengths[b] elements (or runs
// up to the next row's start when row_lengths is NULL), every element visible.
template <int CAP>
__global__ void __launch_bounds__(TK_THREADS)
topk_ragged_kernel(const float* __restrict__ scores, const int64_t* __restrict__ row_offsets, const int64_t* __restrict__ row_lengths, int k,
                   int32_t* __restrict__ idx, int32_t* __restrict__ count, float* __restrict__ kth, int32_t* dev_status) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    using TopkShared = TopkSharedT<CAP>;
    TopkShared& sh = *reinterpret_cast<TopkShared*>(smem_raw);
    const int b = blockIdx.x;
    const int64_t off = row_offsets[b];
    const int64_t n = row_lengths != nullptr ? row_lengths[b] : row_offsets[b + 1] - off;
    // the offsets come from device memory: a row that starts before the array, off a 16-byte boundary (the row is read with
    // 16-byte loads) or has a negative or unrepresentable length is reported and left empty, never read
    if (off < 0 || (off & 3) != 0 || n < 0 || n > 2147483639) {
        for (int i = threadIdx.x; i < k; i += blockDim.x) idx[static_cast<int64_t>(b) * k + i] = -1;
        if (threadIdx.x == 0) {
            if (count != nullptr) count[b] = 0;
            if (kth != nullptr) kth[b] = __int_as_float(0xff800000);
            report(dev_status, JANUS_DEV_INDEX_OUT_OF_RANGE);
        }
        return;
    }
    topk_row(scores + off, static_cast<int>(n), k, b, idx + static_cast<int64_t>(b) * k, count, kth, sh);
}

}  // namespace janus

extern "C" int janus_topk_entries(const float* scores, int64_t scores_ld, int M, int64_t n_entries, int64_t q_pos0, int entry_size, int k,
                                  int32_t* idx, int32_t* count, float* kth, int32_t* /*dev_status*/, void* stream_) {
    using namespace janus;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (M < 0 || n_entries < 0 || k <= 0 || q_pos0 < 0 || entry_size <= 0 || scores_ld < n_entries) return JANUS_ERR_INVALID_ARG;
    if (n_entries >= (int64_t(1) << 31) - 8) return JANUS_ERR_UNSUPPORTED;
    if (M == 0) return JANUS_OK;
    if (!idx) return JANUS_ERR_INVALID_ARG;
    if (n_entries > 0 && (!scores || !aligned16(scores) || (scores_ld & 3) != 0)) return JANUS_ERR_INVALID_ARG;
    const size_t smem = sizeof(TopkSharedT<TK_CAP>);
    JANUS_CUDA_CHECK(cudaFuncSetAttribute(topk_entries_kernel<TK_CAP>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    topk_entries_kernel<TK_CAP><<<M, TK_THREADS, smem, stream>>>(scores, scores_ld, M, n_entries, q_pos0, entry_size, k, idx, count, kth);
    JANUS_CUDA_CHECK(cudaGetLastError());
    return JANUS_OK;
}

extern "C" int janus_entry_pool_scores(const float* scores, int64_t scores_ld, int M, int64_t n_keys, int64_t q_pos0, int causal, int entry_size,
                                       float* entry_scores, int64_t entry_ld, void* stream_) {
    using namespace janus;
    if (M < 0 || n_keys < 0 || q_pos0 < 0 || entry_size <= 0 || scores_ld < n_keys) return JANUS_ERR_INVALID_ARG;
    const int64_t n_entries = (n_keys + entry_size - 1) / entry_size;
    if (entry_ld < n_entries) return JANUS_ERR_INVALID_ARG;
    if (M == 0 || n_entries == 0) return JANUS_OK;
    if (!scores || !entry_scores) return JANUS_ERR_INVALID_ARG;
    const int64_t items = static_cast<int64_t>(M) * n_entries;
    int64_t blocks = (items + 7) / 8;                        // eight warps per block, one strip each
    if (blocks > 148 * 16) blocks = 148 * 16;
    entry_pool_kernel<<<static_cast<unsigned>(blocks), 256, 0, static_cast<cudaStream_t>(stream_)>>>(scores, scores_ld, M, n_keys, q_pos0, causal,
                                                                                                    entry_size, n_entries, entry_scores, entry_ld);
    JANUS_CUDA_CHECK(cudaGetLastError());
    return JANUS_OK;
}

extern "C" int janus_entry_expand(const int32_t* idx_entries, int M, int k_e, int entry_size, int64_t q_pos0, int32_t* idx_tokens,
                                  void* stream_) {
    using namespace janus;
    if (M < 0 || k_e < 0 || entry_size <= 0 || q_pos0 < 0) return JANUS_ERR_INVALID_ARG;
    const int64_t n = static_cast<int64_t>(M) * k_e * entry_size;
    if (n == 0) return JANUS_OK;
    if (!idx_entries || !idx_tokens) return JANUS_ERR_INVALID_ARG;
    if (static_cast<int64_t>(k_e) * entry_size > 2147483647) return JANUS_ERR_UNSUPPORTED;
    int64_t blocks = (n + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    entry_expand_kernel<<<static_cast<unsigned>(blocks), 256, 0, static_cast<cudaStream_t>(stream_)>>>(idx_entries, M, k_e, entry_size, q_pos0,
                                                                                                       idx_tokens);
    JANUS_CUDA_CHECK(cudaGetLastError());
    return JANUS_OK;
}

extern "C" int janus_topk_batch(const float* scores, const int64_t* row_offsets, const int64_t* row_lengths, int B, int k, int32_t* idx,
                                int32_t* count, float* kth, int32_t* dev_status, void* stream_) {
    using namespace janus;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (B < 0 || k <= 0) return JANUS_ERR_INVALID_ARG;
    if (B == 0) return JANUS_OK;
    if (!idx || !row_offsets || !scores || !aligned16(scores)) return JANUS_ERR_INVALID_ARG;
    // row lengths live on the device: the large candidate buffer serves any length
    const size_t smem = sizeof(TopkSharedT<TK_CAP>);
    JANUS_CUDA_CHECK(cudaFuncSetAttribute(topk_ragged_kernel<TK_CAP>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    topk_ragged_kernel<TK_CAP><<<B, TK_THREADS, smem, stream>>>(scores, row_offsets, row_lengths, k, idx, count, kth, dev_status);
    JANUS_CUDA_CHECK(cudaGetLastError());
    return JANUS_OK;
}

extern "C" size_t janus_topk_workspace_size(int, int64_t, int) { return 0; }

extern "C" int janus_topk(const float* scores, int64_t scores_ld, int M, int64_t n_keys, int64_t q_pos0, int causal, int k,
                          int32_t* idx, int32_t* count, float* kth, void* /*ws*/, size_t /*ws_bytes*/,
                          int32_t* /*dev_status*/, void* stream_) {
    using namespace janus;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (M < 0 || n_keys < 0 || k <= 0 || q_pos0 < 0 || scores_ld < n_keys) return JANUS_ERR_INVALID_ARG;
    if (n_keys >= (int64_t(1) << 31) - 8) return JANUS_ERR_UNSUPPORTED;
    if (M == 0) return JANUS_OK;
    if (!idx) return JANUS_ERR_INVALID_ARG;
    if (n_keys > 0 && (!scores || !aligned16(scores) || (scores_ld & 3) != 0)) return JANUS_ERR_INVALID_ARG;
    // The candidate list of a row holds what passes the sampled threshold: about n * r / 4096 elements for the sample rank
    // r = e + 4 sqrt(e) + 8, e = 4096 k / n, give or take n sqrt(r) / 4096.  When that plus five deviations fits the small
    // buffer for the longest row, four CTAs share an SM instead of three.
    const double n_max = static_cast<double>(causal ? (n_keys < q_pos0 + M ? n_keys : q_pos0 + M) : n_keys);
    bool small = false;
    if (n_max > TK_CAP) {
        const double e = 4096.0 * k / n_max, r = e + 4.0 * sqrt(e) + 8.0;
        small = n_max * (r + 5.0 * sqrt(r)) / 4096.0 <= TK_CAP_SMALL && k <= TK_CAP_SMALL / 2;
    }
    int n_sm = 0, dev = 0, per_sm = 0;
    JANUS_CUDA_CHECK(cudaGetDevice(&dev));
    JANUS_CUDA_CHECK(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
    if (small) {
        const size_t smem = sizeof(TopkSharedT<TK_CAP_SMALL>);
        JANUS_CUDA_CHECK(cudaFuncSetAttribute(topk_rows_kernel<TK_CAP_SMALL>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
        JANUS_CUDA_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, topk_rows_kernel<TK_CAP_SMALL>, TK_THREADS, smem));
        const int grid = std::min(M, std::max(1, per_sm) * n_sm);
        topk_rows_kernel<TK_CAP_SMALL><<<grid, TK_THREADS, smem, stream>>>(scores, scores_ld, M, n_keys, q_pos0, causal, k, idx, count, kth);
    } else {
        const size_t smem = sizeof(TopkSharedT<TK_CAP>);
        JANUS_CUDA_CHECK(cudaFuncSetAttribute(topk_rows_kernel<TK_CAP>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
        JANUS_CUDA_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, topk_rows_kernel<TK_CAP>, TK_THREADS, smem));
        const int grid = std::min(M, std::max(1, per_sm) * n_sm);
        topk_rows_kernel<TK_CAP><<<grid, TK_THREADS, smem, stream>>>(scores, scores_ld, M, n_keys, q_pos0, causal, k, idx, count, kth);
    }
    JANUS_CUDA_CHECK(cudaGetLastError());
    return JANUS_OK;
}
