// General-shape sparse attention over the selected rows (Sec. 2.2, "core attention") on the fp32 ALUs.
// One CTA handles one query token and a group of G query heads that share a kv head.  Selected rows are
// gathered through the page table with 16-byte loads into padded shared-memory tiles of 32 keys; the
// softmax is the usual online form (running max and sum in fp32, accumulators rescaled when the max moves).
// Serves multi-head layouts (a single query head per kv head is a matrix-vector problem with nothing for
// tensor cores to do) and any shape the latent tensor-core kernel does not take.
#include "janus_common.cuh"

namespace janus {

constexpr int AG_THREADS = 128;
constexpr int AG_KT = 32;  // keys per tile

template <int G>
__global__ void __launch_bounds__(AG_THREADS)
sparse_attn_generic_kernel(const uint16_t* __restrict__ q, int M, int H_q, int d_qk, const uint16_t* __restrict__ k_pool,
                           const uint16_t* __restrict__ v_pool, int64_t page_stride, int64_t tok_stride, int64_t head_stride,
                           int n_kv_heads, int d_v, const int32_t* __restrict__ idx, int k, int page_size,
                           const int32_t* __restrict__ page_table, int64_t n_logical_pages, const int64_t* __restrict__ table_offsets,
                           float softmax_scale, uint16_t* __restrict__ out, float* __restrict__ lse, int32_t* dev_status) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int kpad = d_qk + 8, vpad = d_v + 8;             // row pitch in bf16: odd multiple of 16 bytes -> conflict-free 16 B reads
    const bool v_alias = (v_pool == k_pool);
    uint16_t* ks = reinterpret_cast<uint16_t*>(smem_raw);                    // [AG_KT][kpad]
    uint16_t* vs = v_alias ? ks : ks + AG_KT * kpad;                         // [AG_KT][vpad or kpad]
    const int v_pitch = v_alias ? kpad : vpad;
    float* qs = reinterpret_cast<float*>(ks + AG_KT * kpad + (v_alias ? 0 : AG_KT * vpad));   // [G][d_qk]
    float* ps = qs + G * d_qk;                                               // [G][AG_KT] logits -> probabilities
    float* corr = ps + G * AG_KT;                                            // [G] maximum logit of this tile
    int* srow = reinterpret_cast<int*>(corr + G);                           // [AG_KT] selected token or -1

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int t = blockIdx.x;
    if (table_offsets != nullptr) {     // every row has a page table of its own (a batch of sessions)
        const int64_t tbl = table_offsets[t];
        n_logical_pages = table_offsets[t + 1] - tbl;
        if (tbl < 0) n_logical_pages = 0;          // a table that starts before the array: every selected token is reported and skipped
        else page_table += tbl;
    }
    const int heads_per_kv = H_q / n_kv_heads;
    const int groups_per_kv = (heads_per_kv + G - 1) / G;
    const int hk = blockIdx.y / groups_per_kv;
    const int h0 = hk * heads_per_kv + (blockIdx.y % groups_per_kv) * G;
    const int g_count = min(G, hk * heads_per_kv + heads_per_kv - h0);

    for (int e = tid; e < G * d_qk; e += AG_THREADS) {
        const int g = e / d_qk, d = e % d_qk;
        qs[e] = g < g_count ? bf16_bits_to_float(q[(static_cast<int64_t>(t) * H_q + h0 + g) * d_qk + d]) * softmax_scale : 0.f;
    }
    float m_run[G], l_run[G];   // replicated in every thread (all threads see the same logits)
    float acc[G][4];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        m_run[g] = __int_as_float(0xff800000);
        l_run[g] = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[g][j] = 0.f;
    }
    const int c0 = tid * 4;                 // this thread owns value columns c0..c0+3
    const int32_t* my_idx = idx + static_cast<int64_t>(t) * k;

    for (int base = 0; base < k; base += AG_KT) {
        __syncthreads();
        if (tid < AG_KT) {
            int s = base + tid < k ? my_idx[base + tid] : -1;
            // a token beyond the page table, or a negative physical page id in it, is reported and skipped
            if (s >= 0 && (s / page_size >= n_logical_pages || __ldg(page_table + s / page_size) < 0)) { report(dev_status, JANUS_DEV_INDEX_OUT_OF_RANGE); s = -1; }
            srow[tid] = s;
        }
        __syncthreads();
        // gather: one warp per row at a time, 16 bytes per lane
        for (int r = warp; r < AG_KT; r += AG_THREADS / 32) {
            const int s = srow[r];
            if (s < 0) continue;
            const int64_t off = static_cast<int64_t>(__ldg(page_table + s / page_size)) * page_stride +
                                static_cast<int64_t>(s % page_size) * tok_stride + static_cast<int64_t>(hk) * head_stride;
            const uint4* src = reinterpret_cast<const uint4*>(k_pool + off);
            uint4* dst = reinterpret_cast<uint4*>(ks + r * kpad);
            for (int c = lane; c < d_qk / 8; c += 32) dst[c] = __ldg(src + c);
            if (!v_alias) {
                const uint4* vsrc = reinterpret_cast<const uint4*>(v_pool + off);
                uint4* vdst = reinterpret_cast<uint4*>(vs + r * vpad);
                for (int c = lane; c < d_v / 8; c += 32) vdst[c] = __ldg(vsrc + c);
            }
        }
        __syncthreads();
        // logits: (g, key) pairs spread over the threads
        for (int p = tid; p < G * AG_KT; p += AG_THREADS) {
            const int g = p / AG_KT, r = p % AG_KT;
            float dot = __int_as_float(0xff800000);
            if (srow[r] >= 0 && g < g_count) {
                dot = 0.f;
                const uint4* kr = reinterpret_cast<const uint4*>(ks + r * kpad);
                const float* qg = qs + g * d_qk;
                for (int c = 0; c < d_qk / 8; ++c) {
                    const uint4 u = kr[c];
                    const uint32_t wds[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        dot = fmaf(qg[c * 8 + 2 * j], __uint_as_float(wds[j] << 16), dot);
                        dot = fmaf(qg[c * 8 + 2 * j + 1], __uint_as_float(wds[j] & 0xffff0000u), dot);
                    }
                }
            }
            ps[p] = dot;
        }
        __syncthreads();
        // tile maximum per head, one warp per head
        for (int g = warp; g < G; g += AG_THREADS / 32) {
            float mx = ps[g * AG_KT + lane];
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
            if (lane == 0) corr[g] = mx;
        }
        __syncthreads();
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float tile_max = corr[g];
            const float m_new = fmaxf(m_run[g], tile_max);
            if (m_new == __int_as_float(0xff800000)) continue;   // nothing selected so far
            const float scale_old = __expf(m_run[g] - m_new);     // exp(-inf) = 0 on the first tile
            float tile_sum = 0.f;
            for (int r = 0; r < AG_KT; ++r) tile_sum += __expf(ps[g * AG_KT + r] - m_new);
            l_run[g] = l_run[g] * scale_old + tile_sum;
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[g][j] *= scale_old;
            m_run[g] = m_new;
        }
        // P.V for this thread's four value columns
        if (c0 < d_v) {
            for (int r = 0; r < AG_KT; ++r) {
                if (srow[r] < 0) continue;
                const uint2 u = *reinterpret_cast<const uint2*>(vs + r * v_pitch + c0);
                const float v0 = __uint_as_float(u.x << 16), v1 = __uint_as_float(u.x & 0xffff0000u);
                const float v2 = __uint_as_float(u.y << 16), v3 = __uint_as_float(u.y & 0xffff0000u);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float p = __expf(ps[g * AG_KT + r] - m_run[g]);
                    acc[g][0] = fmaf(p, v0, acc[g][0]);
                    acc[g][1] = fmaf(p, v1, acc[g][1]);
                    acc[g][2] = fmaf(p, v2, acc[g][2]);
                    acc[g][3] = fmaf(p, v3, acc[g][3]);
                }
            }
        }
    }
#pragma unroll
    for (int g = 0; g < G; ++g) {
        if (g >= g_count) continue;
        const float inv = l_run[g] > 0.f ? 1.f / l_run[g] : 0.f;
        const int64_t o = (static_cast<int64_t>(t) * H_q + h0 + g) * d_v;
        if (c0 < d_v) {
            __nv_bfloat162 a = __floats2bfloat162_rn(acc[g][0] * inv, acc[g][1] * inv);
            __nv_bfloat162 b = __floats2bfloat162_rn(acc[g][2] * inv, acc[g][3] * inv);
            uint2 pk;
            pk.x = *reinterpret_cast<uint32_t*>(&a);
            pk.y = *reinterpret_cast<uint32_t*>(&b);
            *reinterpret_cast<uint2*>(out + o + c0) = pk;
        }
        if (lse != nullptr && tid == 0)
            lse[static_cast<int64_t>(t) * H_q + h0 + g] = l_run[g] > 0.f ? m_run[g] + logf(l_run[g]) : __int_as_float(0xff800000);
    }
}

template <int G>
static int launch_g(const void* q, int M, int H_q, int d_qk, const void* k_pool, const void* v_pool, int64_t page_stride,
                    int64_t tok_stride, int64_t head_stride, int n_kv_heads, int d_v, const int32_t* idx, int k, int page_size,
                    const int32_t* page_table, int64_t n_logical_pages, const int64_t* table_offsets, float softmax_scale, void* out,
                    float* lse, int32_t* dev_status, cudaStream_t stream) {
    const bool v_alias = (v_pool == k_pool);
    size_t smem = sizeof(uint16_t) * AG_KT * (d_qk + 8) + (v_alias ? 0 : sizeof(uint16_t) * AG_KT * (d_v + 8)) +
                  sizeof(float) * (G * d_qk + G * AG_KT + G) + sizeof(int) * AG_KT;
    JANUS_CUDA_CHECK(cudaFuncSetAttribute(sparse_attn_generic_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    const int heads_per_kv = H_q / n_kv_heads;
    dim3 grid(M, n_kv_heads * ((heads_per_kv + G - 1) / G));
    sparse_attn_generic_kernel<G><<<grid, AG_THREADS, smem, stream>>>(
        static_cast<const uint16_t*>(q), M, H_q, d_qk, static_cast<const uint16_t*>(k_pool), static_cast<const uint16_t*>(v_pool),
        page_stride, tok_stride, head_stride, n_kv_heads, d_v, idx, k, page_size, page_table, n_logical_pages, table_offsets,
        softmax_scale, static_cast<uint16_t*>(out), lse, dev_status);
    JANUS_CUDA_CHECK(cudaGetLastError());
    return JANUS_OK;
}

int launch_sparse_attn_generic(const void* q, int M, int H_q, int d_qk, const void* k_pool, const void* v_pool, int64_t page_stride,
                               int64_t tok_stride, int64_t head_stride, int n_kv_heads, int d_v, const int32_t* idx, int k,
                               int page_size, const int32_t* page_table, int64_t n_logical_pages, const int64_t* table_offsets,
                               float softmax_scale, void* out, float* lse, int32_t* dev_status, cudaStream_t stream) {
    const int heads_per_kv = H_q / n_kv_heads;
#define JANUS_AG_ARGS q, M, H_q, d_qk, k_pool, v_pool, page_stride, tok_stride, head_stride, n_kv_heads, d_v, idx, k, page_size, \
                      page_table, n_logical_pages, table_offsets, softmax_scale, out, lse, dev_status, stream
    if (heads_per_kv >= 8) return launch_g<8>(JANUS_AG_ARGS);
    if (heads_per_kv >= 4) return launch_g<4>(JANUS_AG_ARGS);
    if (heads_per_kv >= 2) return launch_g<2>(JANUS_AG_ARGS);
    return launch_g<1>(JANUS_AG_ARGS);
#undef JANUS_AG_ARGS
}

}  // namespace janus
