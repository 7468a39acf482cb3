// General-shape indexer kernel on the fp32 ALUs (Eq. 1, Sec. 2.2, scoring part):
//     scores[t,s] = sum_h w[t,h] * relu(<q[t,h,:], k[s,:]>) + row_bias[t]*col_bias[s],  -inf where masked.
// Serves the shapes the tensor-core kernel does not (odd head counts, strided queries).  One thread per
// key; a tile of 128 keys is kept transposed in shared memory and reused by a chunk of query tokens.
#include "janus_common.cuh"

namespace janus {

constexpr int IG_KEYS = 128;     // keys per CTA (one per thread)
constexpr int IG_TOKENS = 16;    // query tokens per CTA

template <int DTYPE>
__device__ __forceinline__ float load_elem(const void* base, int64_t i) {
    if (DTYPE == JANUS_DTYPE_BF16) return bf16_bits_to_float(reinterpret_cast<const uint16_t*>(base)[i]);
    return e4m3_to_float(reinterpret_cast<const uint8_t*>(base)[i]);
}

template <int DTYPE>
__global__ void __launch_bounds__(IG_KEYS)
indexer_generic_kernel(const void* __restrict__ q_idx, int64_t q_stride_tok, const void* __restrict__ k_idx, int64_t k_stride_tok,
                       const float* __restrict__ w, const float* __restrict__ q_scale, int64_t q_scale_stride_tok,
                       const float* __restrict__ k_scale, const float* __restrict__ row_bias, const float* __restrict__ col_bias,
                       int M, int H, int D, int64_t n_keys, int64_t q_pos0, int causal, float* __restrict__ scores, int64_t ld) {
    extern __shared__ float smem[];
    float* ks = smem;                       // [D][IG_KEYS] transposed key tile
    float* qs = smem + D * IG_KEYS;         // [H][D] one query token
    const int tid = threadIdx.x;
    const int64_t s0 = static_cast<int64_t>(blockIdx.x) * IG_KEYS;
    const int t0 = blockIdx.y * IG_TOKENS;
    const int64_t s = s0 + tid;
    const bool key_ok = s < n_keys;
    const float neg_inf = __int_as_float(0xff800000);

    // a CTA whose keys are all masked for all of its tokens only writes -inf
    const int t_last = min(M, t0 + IG_TOKENS) - 1;
    const bool any_visible = !causal || s0 <= q_pos0 + t_last;
    if (any_visible) {
        for (int e = tid; e < D * IG_KEYS; e += IG_KEYS) {
            const int key = e / D, d = e % D;
            float v = 0.f;
            if (s0 + key < n_keys) v = load_elem<DTYPE>(k_idx, (s0 + key) * k_stride_tok + d);
            ks[d * IG_KEYS + key] = v;
        }
    }
    const float kscale = (k_scale != nullptr && key_ok) ? k_scale[s] : 1.f;
    const float cb = (col_bias != nullptr && key_ok) ? col_bias[s] : 0.f;
    for (int t = t0; t <= t_last; ++t) {
        const bool visible = key_ok && (!causal || s <= q_pos0 + t);
        const bool tile_visible = !causal || s0 <= q_pos0 + t;
        float acc = 0.f;
        if (tile_visible) {
            __syncthreads();
            for (int e = tid; e < H * D; e += IG_KEYS) {
                float v = load_elem<DTYPE>(q_idx, static_cast<int64_t>(t) * q_stride_tok + e);
                if (q_scale != nullptr) v *= q_scale[static_cast<int64_t>(t) * q_scale_stride_tok + e / D];
                qs[e] = v;
            }
            __syncthreads();
            for (int h = 0; h < H; ++h) {
                const float* qh = qs + h * D;
                float dot = 0.f;
#pragma unroll 8
                for (int d = 0; d < D; ++d) dot = fmaf(qh[d], ks[d * IG_KEYS + tid], dot);
                acc = fmaf(w[static_cast<int64_t>(t) * H + h], fmaxf(dot, 0.f), acc);
            }
            acc *= kscale;
            if (row_bias != nullptr) acc = fmaf(row_bias[t], cb, acc);
        }
        if (key_ok) scores[static_cast<int64_t>(t) * ld + s] = visible ? acc : neg_inf;
    }
}

int launch_indexer_generic(const void* q_idx, int64_t q_stride_tok, const void* k_idx, int64_t k_stride_tok, const float* w,
                           const float* q_scale, int64_t q_scale_stride_tok, const float* k_scale, const float* row_bias,
                           const float* col_bias, int M, int H, int D, int64_t n_keys, int64_t q_pos0, int causal, int dtype,
                           float* scores, int64_t ld, cudaStream_t stream) {
    const size_t smem = sizeof(float) * (static_cast<size_t>(D) * IG_KEYS + static_cast<size_t>(H) * D);
    if (smem > 200 * 1024) return JANUS_ERR_UNSUPPORTED;
    dim3 grid(static_cast<unsigned>((n_keys + IG_KEYS - 1) / IG_KEYS), static_cast<unsigned>((M + IG_TOKENS - 1) / IG_TOKENS));
    if (grid.y > 65535) return JANUS_ERR_UNSUPPORTED;
    if (dtype == JANUS_DTYPE_BF16) {
        JANUS_CUDA_CHECK(cudaFuncSetAttribute(indexer_generic_kernel<JANUS_DTYPE_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
        indexer_generic_kernel<JANUS_DTYPE_BF16><<<grid, IG_KEYS, smem, stream>>>(q_idx, q_stride_tok, k_idx, k_stride_tok, w, q_scale, q_scale_stride_tok,
                                                                                k_scale, row_bias, col_bias, M, H, D, n_keys, q_pos0, causal, scores, ld);
    } else {
        JANUS_CUDA_CHECK(cudaFuncSetAttribute(indexer_generic_kernel<JANUS_DTYPE_FP8_E4M3>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
        indexer_generic_kernel<JANUS_DTYPE_FP8_E4M3><<<grid, IG_KEYS, smem, stream>>>(q_idx, q_stride_tok, k_idx, k_stride_tok, w, q_scale, q_scale_stride_tok,
                                                                                    k_scale, row_bias, col_bias, M, H, D, n_keys, q_pos0, causal, scores, ld);
    }
    JANUS_CUDA_CHECK(cudaGetLastError());
    return JANUS_OK;
}

}  // namespace janus
