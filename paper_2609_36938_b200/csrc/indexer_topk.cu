// janus_indexer_topk: indexer scores and per-row top-k (Eq. 1, Sec. 2.2) without materialising the score matrix.
//
//   1. 4096 keys sampled evenly from the part of the history every row can see are gathered and scored for all rows
//      with the tensor-core indexer (3 % of its work at 128K keys);
//   2. per row, the sample gives a threshold whose expected rank in the row is safely above k;
//   3. the tensor-core indexer runs over all keys in candidate mode: its epilogue appends every visible score at or above
//      the row's threshold to the row's candidate list (a few per cent of the row) instead of storing 4 bytes per pair;
//   4. per row, the exact top-k is selected among the candidates in shared memory.
// A row whose candidate list came out shorter than k or longer than its buffer (the sample misjudged it) is recomputed
// from the operands on the fp32 ALUs into a scratch row and selected from there: slower, never wrong.
// Scratch (sample, thresholds, candidate lists, fallback rows) lives in the caller's workspace.
// Shapes the tensor-core indexer does not take, and problems too small to sample, run the two-call path
// (scores in the workspace, then the row-wise top-k).
#include <mutex>

#include "sm100_ptx.cuh"
#include "topk_select.cuh"

namespace janus {

constexpr int FT_NS = 4096;          // sampled keys (512 chunks of 8 consecutive keys)
constexpr int FT_CAP = 16384;        // candidate slots per row; FT_CAP / 2 when the expected lists are short enough
constexpr int FT_FB_CTAS = 32;       // CTAs (and scratch rows) of the fallback kernel
constexpr int FT_FB_CAP = 8192;      // candidate slots of the fallback's row-wise top-k

using SampleShared = TopkSharedT<FT_NS>;
using FallbackShared = TopkSharedT<FT_FB_CAP>;

bool indexer_tc_supported(int M, int H, int D, int64_t n_keys, int64_t q_stride_tok, int64_t k_stride_tok, int dtype);
bool indexer_tc_candidates_supported(int H, int D, int dtype);
int launch_indexer_tc(const void* q_idx, const void* k_idx, int64_t k_stride_tok, const float* w, const float* q_scale,
                      int64_t q_scale_stride_tok, const float* k_scale, const float* row_bias, const float* col_bias, int M, int H,
                      int D, int64_t n_keys, int64_t q_pos0, int causal, int dtype, float* scores, int64_t ld, int32_t* dev_status,
                      cudaStream_t stream, const float* thr, int32_t* cand_cnt, void* cand, int cand_cap);
int validate_indexer_args(const void* q_idx, int64_t q_stride_tok, const void* k_idx, int64_t k_stride_tok, const float* w,
                          const float* q_scale, int64_t q_scale_stride_tok, const float* k_scale, const float* row_bias,
                          const float* col_bias, int M, int H_I, int D_I, int64_t n_keys, int64_t q_pos0, int dtype);

// ---- workspace layout --------------------------------------------------------------------------------------------------
struct FusedLayout {
    bool fused;            // false: two-call path, `scores` is the only region
    int cap;               // candidate slots per row
    int64_t p0;            // keys every row can see (sampling range)
    int64_t ld;            // row pitch of score rows (floats)
    size_t k_sample, ks_sample, cb_sample, sc_sample, thr, cand_cnt, fb_count, fb_rows, cand, fb_buf, scores, total;
};

static size_t align_up(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

FusedLayout fused_layout(int M, int H, int D, int64_t n_keys, int64_t q_pos0, int causal, int dtype, int k) {
    FusedLayout L{};
    const int esz = dtype == JANUS_DTYPE_BF16 ? 2 : 1;
    L.p0 = causal ? (n_keys < q_pos0 + 1 ? n_keys : q_pos0 + 1) : n_keys;
    L.ld = (n_keys + 3) / 4 * 4;
    L.fused = indexer_tc_supported(M, H, D, n_keys, static_cast<int64_t>(H) * D, D, dtype) && indexer_tc_candidates_supported(H, D, dtype) &&
              L.p0 >= 4 * FT_NS && n_keys > FT_CAP &&
              k <= FT_CAP / 4 && n_keys - L.p0 <= FT_CAP / 2;
    L.cap = FT_CAP;
    if (L.fused) {
        // half-size lists (three selection CTAs per SM instead of one) when the list expected at the sampled threshold, plus
        // every key beyond the sampled range, still fits them
        const double expect = static_cast<double>(FT_NS) * k / static_cast<double>(L.p0);
        const double frac = (expect + 6.0 * sqrt(expect) + 8.0) / FT_NS;
        if (k <= FT_CAP / 8 && frac * static_cast<double>(n_keys) + static_cast<double>(n_keys - L.p0) <= FT_CAP / 2) L.cap = FT_CAP / 2;
    }
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t o = off; off += align_up(bytes); return o; };
    if (L.fused) {
        L.k_sample = take(static_cast<size_t>(FT_NS) * D * esz);
        L.ks_sample = take(sizeof(float) * FT_NS);
        L.cb_sample = take(sizeof(float) * FT_NS);
        L.sc_sample = take(sizeof(float) * FT_NS * static_cast<size_t>(M));
        L.thr = take(sizeof(float) * M);
        L.cand_cnt = take(sizeof(int32_t) * M);
        L.fb_count = take(sizeof(int32_t) * 4);
        L.fb_rows = take(sizeof(int32_t) * M);
        L.cand = take(sizeof(int2) * static_cast<size_t>(L.cap) * M);
        L.fb_buf = take(sizeof(float) * static_cast<size_t>(L.ld) * FT_FB_CTAS);
    } else {
        L.scores = take(sizeof(float) * static_cast<size_t>(L.ld) * M);
    }
    L.total = off;
    return L;
}

// ---- 1. sample gather ----------------------------------------------------------------------------------------------------
// Sample j = chunk j/8, element j%8; chunk i starts at key 8 * floor(i * (p0/8 - 1) / 511).
__device__ __forceinline__ int64_t sample_position(int j, int64_t p0) {
    const int64_t n8 = p0 >> 3;
    return 8 * ((static_cast<int64_t>(j >> 3) * (n8 - 1)) / 511) + (j & 7);
}

__global__ void ft_gather_sample_kernel(const unsigned char* __restrict__ k_idx, int64_t k_row_bytes, int row_vecs, const float* __restrict__ k_scale,
                                        const float* __restrict__ col_bias, int64_t p0, uint4* __restrict__ k_sample, float* __restrict__ ks_sample,
                                        float* __restrict__ cb_sample) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;      // one 16-byte vector of one sampled key row
    if (i >= FT_NS * row_vecs) return;
    const int j = i / row_vecs, v = i - j * row_vecs;
    const int64_t pos = sample_position(j, p0);
    k_sample[i] = __ldg(reinterpret_cast<const uint4*>(k_idx + pos * k_row_bytes) + v);
    if (v == 0) {
        if (k_scale != nullptr) ks_sample[j] = k_scale[pos];
        if (col_bias != nullptr) cb_sample[j] = col_bias[pos];
    }
}

// ---- 2. per-row threshold from the sample ----------------------------------------------------------------------------------
__global__ void __launch_bounds__(TK_THREADS)
ft_threshold_kernel(const float* __restrict__ sc_sample, int M, int64_t n_keys, int64_t q_pos0, int causal, int k, int cap, float* __restrict__ thr,
                    int32_t* __restrict__ cand_cnt, int32_t* __restrict__ fb_count) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SampleShared& sh = *reinterpret_cast<SampleShared*>(smem_raw);
    const int t = blockIdx.x, tid = threadIdx.x;
    const int64_t n = causal ? (n_keys < q_pos0 + t + 1 ? n_keys : q_pos0 + t + 1) : n_keys;
    if (tid == 0) {
        cand_cnt[t] = 0;
        if (t == 0) fb_count[0] = 0;
    }
    const float neg_inf = __int_as_float(0xff800000);
    if (n <= cap) {                          // the whole prefix fits the candidate list
        if (tid == 0) thr[t] = neg_inf;
        return;
    }
    // rank in the sample whose value sits six standard deviations below the expected position of the row's k-th score
    const float expect = static_cast<float>(FT_NS) * static_cast<float>(k) / static_cast<float>(n);
    const int r = static_cast<int>(expect + 6.0f * sqrtf(expect) + 8.0f);
    if (r >= FT_NS) {
        if (tid == 0) thr[t] = neg_inf;
        return;
    }
    const float* row = sc_sample + static_cast<int64_t>(t) * FT_NS;
    for (int i = tid; i < FT_NS; i += TK_THREADS) sh.cand_key[i] = float_to_key(row[i]);
    __syncthreads();
    int dummy;
    SmemSource s{sh.cand_key, nullptr, FT_NS};
    const uint32_t T = select_kth(s, r, sh, &dummy);
    if (tid == 0) thr[t] = key_to_float(T);
}

// ---- 4. exact selection among a row's candidates ------------------------------------------------------------------------------
template <int CAP>
__global__ void __launch_bounds__(TK_THREADS)
ft_select_kernel(const int2* __restrict__ cand, const int32_t* __restrict__ cand_cnt, int M, int64_t n_keys, int64_t q_pos0, int causal, int k,
                 int32_t* __restrict__ idx, int32_t* __restrict__ count, float* __restrict__ kth, int32_t* __restrict__ fb_count,
                 int32_t* __restrict__ fb_rows) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    using Shared = TopkSharedT<CAP>;
    Shared& sh = *reinterpret_cast<Shared*>(smem_raw);
    const int t = blockIdx.x, tid = threadIdx.x;
    const int64_t n64 = causal ? (n_keys < q_pos0 + t + 1 ? n_keys : q_pos0 + t + 1) : n_keys;
    const int n = static_cast<int>(n64 < 0 ? 0 : n64);
    const int n_sel = n < k ? n : k;
    const int n_c = cand_cnt[t];
    int32_t* out = idx + static_cast<int64_t>(t) * k;
    if (n_c < n_sel || n_c > CAP) {       // the sample misjudged this row: hand it to the fallback kernel
        if (tid == 0) fb_rows[atomicAdd(fb_count, 1)] = t;
        return;
    }
    if (tid == 0) { sh.out_pos = 0; sh.eq_taken = 0; }
    const int2* row = cand + static_cast<int64_t>(t) * CAP;
    for (int i = tid; i < n_c; i += TK_THREADS) {
        const int2 c = row[i];
        sh.cand_key[i] = float_to_key(__int_as_float(c.x));
        sh.cand_idx[i] = c.y;
    }
    __syncthreads();
    SmemSource s{sh.cand_key, sh.cand_idx, n_c};
    uint32_t T = 0u;
    if (n_sel > 0) {
        int n_eq;
        T = select_kth(s, n_sel, sh, &n_eq);
        emit_selection(s, T, n_eq, out, sh);
    }
    for (int i = n_sel + tid; i < k; i += TK_THREADS) out[i] = -1;
    if (tid == 0) {
        if (count) count[t] = n_sel;
        if (kth) kth[t] = n_sel > 0 ? key_to_float(T) : __int_as_float(0xff800000);
    }
}

// ---- 5. fallback: rows the sample misjudged are recomputed on the fp32 ALUs and selected row-wise ---------------------------
template <int DTYPE>
__device__ __forceinline__ void decode16(const uint4& u, float (&v)[16], int& n) {
    const uint32_t wds[4] = {u.x, u.y, u.z, u.w};
    if (DTYPE == JANUS_DTYPE_BF16) {
        n = 8;
#pragma unroll
        for (int j = 0; j < 4; ++j) { v[2 * j] = __uint_as_float(wds[j] << 16); v[2 * j + 1] = __uint_as_float(wds[j] & 0xffff0000u); }
    } else {
        n = 16;
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int b = 0; b < 4; ++b) v[4 * j + b] = e4m3_to_float(static_cast<uint8_t>(wds[j] >> (8 * b)));
    }
}

template <int DTYPE>
__global__ void __launch_bounds__(TK_THREADS)
ft_fallback_kernel(const unsigned char* __restrict__ q_idx, const unsigned char* __restrict__ k_idx, int64_t k_row_bytes, const float* __restrict__ w,
                   const float* __restrict__ q_scale, int64_t q_scale_stride_tok, const float* __restrict__ k_scale,
                   const float* __restrict__ row_bias, const float* __restrict__ col_bias, int M, int H, int D, int64_t n_keys, int64_t q_pos0,
                   int causal, int k, int32_t* __restrict__ idx, int32_t* __restrict__ count, float* __restrict__ kth,
                   const int32_t* __restrict__ fb_count, const int32_t* __restrict__ fb_rows, float* __restrict__ fb_buf, int64_t ld) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    FallbackShared& sh = *reinterpret_cast<FallbackShared*>(smem_raw);
    float* qs = reinterpret_cast<float*>(smem_raw + sizeof(FallbackShared));   // [H][D] query of the row, pre-multiplied by q_scale
    float* wq = qs + H * D;                                                     // [H] head weights of the row
    const int tid = threadIdx.x;
    const int esz = DTYPE == JANUS_DTYPE_BF16 ? 2 : 1;
    float* buf = fb_buf + static_cast<int64_t>(blockIdx.x) * ld;
    const int n_fb = fb_count[0];
    for (int f = blockIdx.x; f < n_fb; f += gridDim.x) {
        const int t = fb_rows[f];
        const int64_t n64 = causal ? (n_keys < q_pos0 + t + 1 ? n_keys : q_pos0 + t + 1) : n_keys;
        const int n = static_cast<int>(n64);
        __syncthreads();
        for (int e = tid; e < H * D; e += TK_THREADS) {
            const unsigned char* qp = q_idx + (static_cast<int64_t>(t) * H * D + e) * esz;
            float v = DTYPE == JANUS_DTYPE_BF16 ? bf16_bits_to_float(*reinterpret_cast<const uint16_t*>(qp)) : e4m3_to_float(*qp);
            if (q_scale != nullptr) v *= q_scale[static_cast<int64_t>(t) * q_scale_stride_tok + e / D];
            qs[e] = v;
        }
        for (int h = tid; h < H; h += TK_THREADS) wq[h] = w[static_cast<int64_t>(t) * H + h];
        __syncthreads();
        const float rb = row_bias != nullptr ? row_bias[t] : 0.f;
        for (int s = tid; s < n; s += TK_THREADS) {
            const uint4* krow = reinterpret_cast<const uint4*>(k_idx + static_cast<int64_t>(s) * k_row_bytes);
            float acc = 0.f;
            for (int hb = 0; hb < H; hb += 4) {       // four heads at a time; the key row is re-read from L1 for each group
                float part[4] = {0.f, 0.f, 0.f, 0.f};
                int d = 0;
                for (int v = 0; d < D; ++v) {
                    float kv[16];
                    int nv;
                    decode16<DTYPE>(__ldg(krow + v), kv, nv);
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        if (e < nv) {
#pragma unroll
                            for (int hh = 0; hh < 4; ++hh) part[hh] = fmaf(qs[(hb + hh) * D + d + e], kv[e], part[hh]);
                        }
                    }
                    d += nv;
                }
#pragma unroll
                for (int hh = 0; hh < 4; ++hh) acc = fmaf(wq[hb + hh], fmaxf(part[hh], 0.f), acc);
            }
            if (k_scale != nullptr) acc *= k_scale[s];
            if (col_bias != nullptr) acc = fmaf(rb, col_bias[s], acc);
            buf[s] = acc;
        }
        __syncthreads();
        topk_row(buf, n, k, t, idx + static_cast<int64_t>(t) * k, count, kth, sh);
    }
}

}  // namespace janus

extern "C" size_t janus_indexer_topk_workspace_size(int M, int H_I, int D_I, int64_t n_keys, int64_t q_pos0, int causal, int dtype, int k) {
    if (M <= 0 || H_I <= 0 || D_I <= 0 || n_keys <= 0 || k <= 0) return 0;
    return janus::fused_layout(M, H_I, D_I, n_keys, q_pos0, causal, dtype, k).total;
}

extern "C" int64_t janus_indexer_topk_fallback_counter_offset(int M, int H_I, int D_I, int64_t n_keys, int64_t q_pos0, int causal, int dtype, int k) {
    if (M <= 0 || H_I <= 0 || D_I <= 0 || n_keys <= 0 || k <= 0) return -1;
    const janus::FusedLayout L = janus::fused_layout(M, H_I, D_I, n_keys, q_pos0, causal, dtype, k);
    return L.fused ? static_cast<int64_t>(L.fb_count) : -1;
}

extern "C" int janus_indexer_topk(const void* q_idx, int64_t q_stride_tok, const void* k_idx, int64_t k_stride_tok, const float* w,
                                  const float* q_scale, int64_t q_scale_stride_tok, const float* k_scale, const float* row_bias,
                                  const float* col_bias, int M, int H_I, int D_I, int64_t n_keys, int64_t q_pos0, int causal, int dtype,
                                  int k, int32_t* idx, int32_t* count, float* kth, void* ws, size_t ws_bytes, int32_t* dev_status,
                                  void* stream_) {
    using namespace janus;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int vrc = validate_indexer_args(q_idx, q_stride_tok, k_idx, k_stride_tok, w, q_scale, q_scale_stride_tok, k_scale, row_bias, col_bias,
                                          M, H_I, D_I, n_keys, q_pos0, dtype);
    if (vrc != JANUS_OK) return vrc;
    if (k <= 0) return JANUS_ERR_INVALID_ARG;
    if (M == 0) return JANUS_OK;
    if (!idx) return JANUS_ERR_INVALID_ARG;
    if (n_keys >= (int64_t(1) << 31) - 8) return JANUS_ERR_UNSUPPORTED;
    FusedLayout L = fused_layout(M, H_I, D_I, n_keys, q_pos0, causal, dtype, k);
    if (q_stride_tok != static_cast<int64_t>(H_I) * D_I && L.fused) {   // strided queries: the two-call path
        L = FusedLayout{};
        L.ld = (n_keys + 3) / 4 * 4;
        L.total = align_up(sizeof(float) * static_cast<size_t>(L.ld) * M);
    }
    if (n_keys > 0 && (ws == nullptr || ws_bytes < L.total || !aligned16(ws))) return JANUS_ERR_WORKSPACE_TOO_SMALL;
    unsigned char* base = static_cast<unsigned char*>(ws);

    if (!L.fused) {
        float* scores = reinterpret_cast<float*>(base + L.scores);
        int rc = janus_indexer_scores(q_idx, q_stride_tok, k_idx, k_stride_tok, w, q_scale, q_scale_stride_tok, k_scale, row_bias, col_bias, M,
                                      H_I, D_I, n_keys, q_pos0, causal, dtype, scores, L.ld, nullptr, 0, dev_status, stream_);
        if (rc != JANUS_OK) return rc;
        return janus_topk(scores, L.ld, M, n_keys, q_pos0, causal, k, idx, count, kth, nullptr, 0, dev_status, stream_);
    }

    const bool fp8 = dtype == JANUS_DTYPE_FP8_E4M3;
    const int esz = fp8 ? 1 : 2;
    const int row_vecs = D_I * esz / 16;
    float* ks_sample = fp8 ? reinterpret_cast<float*>(base + L.ks_sample) : nullptr;
    float* cb_sample = col_bias != nullptr ? reinterpret_cast<float*>(base + L.cb_sample) : nullptr;
    float* sc_sample = reinterpret_cast<float*>(base + L.sc_sample);
    float* thr = reinterpret_cast<float*>(base + L.thr);
    int32_t* cand_cnt = reinterpret_cast<int32_t*>(base + L.cand_cnt);
    int32_t* fb_count = reinterpret_cast<int32_t*>(base + L.fb_count);
    int32_t* fb_rows = reinterpret_cast<int32_t*>(base + L.fb_rows);
    int2* cand = reinterpret_cast<int2*>(base + L.cand);
    float* fb_buf = reinterpret_cast<float*>(base + L.fb_buf);

    // 1. sample
    ft_gather_sample_kernel<<<(FT_NS * row_vecs + 255) / 256, 256, 0, stream>>>(static_cast<const unsigned char*>(k_idx), k_stride_tok * esz, row_vecs,
                                                                                k_scale, col_bias, L.p0,
                                                                                reinterpret_cast<uint4*>(base + L.k_sample), ks_sample, cb_sample);
    JANUS_CUDA_CHECK(cudaGetLastError());
    int rc = launch_indexer_tc(q_idx, base + L.k_sample, D_I, w, q_scale, q_scale_stride_tok, ks_sample, cb_sample ? row_bias : nullptr, cb_sample, M,
                               H_I, D_I, FT_NS, q_pos0, 0, dtype, sc_sample, FT_NS, dev_status, stream, nullptr, nullptr, nullptr, 0);
    if (rc != JANUS_OK) return rc;
    // 2. thresholds (also clears the candidate counters)
    JANUS_CUDA_CHECK(cudaFuncSetAttribute(ft_threshold_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(sizeof(SampleShared))));
    ft_threshold_kernel<<<M, TK_THREADS, sizeof(SampleShared), stream>>>(sc_sample, M, n_keys, q_pos0, causal, k, L.cap, thr, cand_cnt, fb_count);
    JANUS_CUDA_CHECK(cudaGetLastError());
    // 3. the indexer over all keys, appending candidates
    rc = launch_indexer_tc(q_idx, k_idx, k_stride_tok, w, q_scale, q_scale_stride_tok, k_scale, row_bias, col_bias, M, H_I, D_I, n_keys, q_pos0, causal,
                           dtype, nullptr, 0, dev_status, stream, thr, cand_cnt, cand, L.cap);
    if (rc != JANUS_OK) return rc;
    // 4. exact selection per row
    if (L.cap == FT_CAP) {
        using Sh = TopkSharedT<FT_CAP>;
        JANUS_CUDA_CHECK(cudaFuncSetAttribute(ft_select_kernel<FT_CAP>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(sizeof(Sh))));
        ft_select_kernel<FT_CAP><<<M, TK_THREADS, sizeof(Sh), stream>>>(cand, cand_cnt, M, n_keys, q_pos0, causal, k, idx, count, kth, fb_count, fb_rows);
    } else {
        using Sh = TopkSharedT<FT_CAP / 2>;
        JANUS_CUDA_CHECK(cudaFuncSetAttribute(ft_select_kernel<FT_CAP / 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(sizeof(Sh))));
        ft_select_kernel<FT_CAP / 2><<<M, TK_THREADS, sizeof(Sh), stream>>>(cand, cand_cnt, M, n_keys, q_pos0, causal, k, idx, count, kth, fb_count,
                                                                           fb_rows);
    }
    JANUS_CUDA_CHECK(cudaGetLastError());
    // 5. rows the sample misjudged (normally none: the kernel then returns at once)
    const size_t fb_smem = sizeof(FallbackShared) + sizeof(float) * (static_cast<size_t>(H_I) * D_I + H_I);
    const unsigned char* qb = static_cast<const unsigned char*>(q_idx);
    const unsigned char* kb = static_cast<const unsigned char*>(k_idx);
    if (fp8) {
        JANUS_CUDA_CHECK(cudaFuncSetAttribute(ft_fallback_kernel<JANUS_DTYPE_FP8_E4M3>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(fb_smem)));
        ft_fallback_kernel<JANUS_DTYPE_FP8_E4M3><<<FT_FB_CTAS, TK_THREADS, fb_smem, stream>>>(
            qb, kb, k_stride_tok * esz, w, q_scale, q_scale_stride_tok, k_scale, row_bias, col_bias, M, H_I, D_I, n_keys, q_pos0, causal, k, idx, count,
            kth, fb_count, fb_rows, fb_buf, L.ld);
    } else {
        JANUS_CUDA_CHECK(cudaFuncSetAttribute(ft_fallback_kernel<JANUS_DTYPE_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(fb_smem)));
        ft_fallback_kernel<JANUS_DTYPE_BF16><<<FT_FB_CTAS, TK_THREADS, fb_smem, stream>>>(
            qb, kb, k_stride_tok * esz, w, q_scale, q_scale_stride_tok, k_scale, row_bias, col_bias, M, H_I, D_I, n_keys, q_pos0, causal, k, idx, count,
            kth, fb_count, fb_rows, fb_buf, L.ld);
    }
    JANUS_CUDA_CHECK(cudaGetLastError());
    return JANUS_OK;
}

// ---- the same call on scratch that ships with the library ---------------------------------------------------------------------
// Some callers have no device memory to hand over as a workspace and no way to get any: a plug-in running inside a serving
// engine that has already given every free byte of HBM to its KV-cache pool and lends plug-ins none of it, or a
// latency-critical loop that may not call the CUDA allocator because freeing device memory waits for the whole device.
// For them the scratch is a fixed array in the library's own device image.  It exists once per device and is shared by every
// call on that device.
namespace janus {

static __device__ __align__(256) unsigned char ft_static_scratch[JANUS_STATIC_SCRATCH_BYTES];

// Device address of the array on the device that is current now, looked up the first time that device is seen.
static int static_scratch_address(void** out) {
    constexpr int MAX_DEVICES = 64;
    static std::mutex mu;
    static void* address[MAX_DEVICES] = {};
    int dev = -1;
    JANUS_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return JANUS_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(mu);
    if (address[dev] == nullptr) {
        void* ptr = nullptr;
        JANUS_CUDA_CHECK(cudaGetSymbolAddress((void**)&ptr, ft_static_scratch));
        if (ptr == nullptr || !aligned16(ptr)) return JANUS_ERR_CUDA;
        address[dev] = ptr;
    }
    *out = address[dev];
    return JANUS_OK;
}

}  // namespace janus

extern "C" int janus_indexer_topk_static(const void* q_idx, int64_t q_stride_tok, const void* k_idx, int64_t k_stride_tok, const float* w,
                                         const float* q_scale, int64_t q_scale_stride_tok, const float* k_scale, const float* row_bias,
                                         const float* col_bias, int M, int H_I, int D_I, int64_t n_keys, int64_t q_pos0, int causal, int dtype,
                                         int k, int32_t* idx, int32_t* count, float* kth, int32_t* dev_status, void* stream_) {
    using namespace janus;
    // the size check comes first: a problem that does not fit is refused before anything touches the device
    if (M < 0 || H_I <= 0 || D_I <= 0 || n_keys < 0 || k <= 0) return JANUS_ERR_INVALID_ARG;
    if (M > 0 && n_keys > 0) {
        const FusedLayout L = fused_layout(M, H_I, D_I, n_keys, q_pos0, causal, dtype, k);
        size_t need = L.total;
        if (L.fused && q_stride_tok != static_cast<int64_t>(H_I) * D_I)   // strided queries take the two-call route
            need = align_up(sizeof(float) * static_cast<size_t>(L.ld) * M);
        if (need > static_cast<size_t>(JANUS_STATIC_SCRATCH_BYTES)) return JANUS_ERR_WORKSPACE_TOO_SMALL;
    }
    void* scratch = nullptr;
    const int rc = static_scratch_address(&scratch);
    if (rc != JANUS_OK) return rc;
    return janus_indexer_topk(q_idx, q_stride_tok, k_idx, k_stride_tok, w, q_scale, q_scale_stride_tok, k_scale, row_bias, col_bias, M, H_I, D_I,
                              n_keys, q_pos0, causal, dtype, k, idx, count, kth, scratch, static_cast<size_t>(JANUS_STATIC_SCRATCH_BYTES), dev_status,
                              stream_);
}
