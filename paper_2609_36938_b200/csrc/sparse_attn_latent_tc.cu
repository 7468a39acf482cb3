// Tensor-core sparse attention for the latent layout (Sec. 2.2, "core attention"): one shared KV row of 576 bf16
// per token (keys = all 576 dims, values = the first 512), 128 query heads, selection idx[t, 0:k).
//
//     out[t,h,:] = sum_{s in idx[t]} softmax_s(scale * <q[t,h,:576], row_s[:576]>) * row_s[:512]
//
// Shape of the problem on one SM.  The heads of one token form the MMA M axis (128 heads = 128 TMEM lanes), so the
// fp32 output accumulator is 128 lanes x 512 columns = all of tensor memory.  The value dimension is therefore
// split in two: CTA (t, c) owns value columns [256c, 256c+256) and recomputes the logits, which only need
// tensor memory for 32 keys at a time.  Shared memory cannot hold the 144 KB query tile next to a useful key ring,
// so query dims [0,320) stay in shared memory (5 swizzle atoms) and dims [320,576) live in tensor memory as a
// TMEM-resident A operand; that leaves room for a 4-deep ring of 32-key tiles (36 KB each).
//
// Per 32-key tile:  gather warps copy the selected rows through the page table with 16-byte cp.async into the
// swizzled K-major layout (9 atoms of 64 dims);  the MMA thread issues S = Q.K^T (36 MMAs 128x32x16) and, one tile
// behind, O += P.V (2 MMAs 128x256x16 with V read MN-major out of the same rows);  softmax warps (thread = head)
// read S from TMEM, keep a running max / sum in fp32 registers, write P as bf16 back to TMEM.  The running max is
// only moved when a tile exceeds it by more than 2^8, so O is rescaled (in TMEM) a handful of times per row.
// Every wait is bounded; on a timeout the CTA reports JANUS_DEV_WAIT_TIMEOUT and winds down.
#include "janus_common.cuh"
#include "sm100_ptx.cuh"

namespace janus {

using namespace ptx;

constexpr int LA_HEADS = 128;
constexpr int LA_DQK = 576;
constexpr int LA_DV = 512;
constexpr int LA_DV_HALF = 256;
constexpr int LA_BK = 32;                 // keys per tile
constexpr int LA_STAGES = 4;
constexpr int LA_ATOMS = 9;               // 576 / 64
constexpr int LA_Q_SMEM_ATOMS = 5;        // query dims [0,320) in shared memory
constexpr int LA_Q_TMEM_ATOMS = 4;        // query dims [320,576) in tensor memory
constexpr int LA_Q_ATOM_BYTES = LA_HEADS * 128;        // 16 KB
constexpr int LA_K_ATOM_BYTES = LA_BK * 128;           // 4 KB
constexpr int LA_STAGE_BYTES = LA_ATOMS * LA_K_ATOM_BYTES;   // 36 KB
constexpr int LA_THREADS = 32 * 9;        // warp 0: MMA + TMA; warps 1-4: gather; warps 5-8: softmax
constexpr int LA_GATHER_WARPS = 4;
constexpr int LA_LAG = 2;                 // gather tiles in flight per warp beyond the one being issued
// tensor-memory columns
constexpr uint32_t LA_COL_O = 0, LA_COL_S = 256, LA_COL_P = 320, LA_COL_Q = 352;   // S: 2x32, P: 2x16, Q: 128

struct LaShared {
    uint64_t q_full, qt_full;
    uint64_t k_full[LA_STAGES], k_empty[LA_STAGES];
    uint64_t s_full[2], p_full[2];
    uint64_t pv_done;
    uint32_t vmask[LA_STAGES];
    uint32_t tmem_base;
    int aborted;
};

struct LaParams {
    const uint16_t* q;
    const uint16_t* pool;
    int64_t page_stride, tok_stride;
    const int32_t* idx;
    int k;
    int page_size, page_shift;
    const int32_t* page_table;
    int64_t n_logical_pages;
    float scale_log2e;        // softmax_scale * log2(e)
    uint16_t* out;
    float* lse;
    int M;
    int32_t* dev_status;
};

__device__ __forceinline__ float fast_exp2(float x) {   // ex2.approx: 2 ulp, exp2(-inf) = 0
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

__global__ void __launch_bounds__(LA_THREADS, 1)
sparse_attn_latent_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const LaParams p) {
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char* q_smem = smem;                                              // 5 atoms x [128 heads x 128 B]
    unsigned char* k_smem = smem + LA_Q_SMEM_ATOMS * LA_Q_ATOM_BYTES;          // 4 stages x 9 atoms x [32 keys x 128 B]
    LaShared* sh = reinterpret_cast<LaShared*>(k_smem + LA_STAGES * LA_STAGE_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t = blockIdx.x >> 1;
    const int half = blockIdx.x & 1;
    const int n_tiles = (p.k + LA_BK - 1) / LA_BK;

    if ((smem_u32(smem) & 1023u) != 0u) {
        if (threadIdx.x == 0) report(p.dev_status, JANUS_DEV_WAIT_TIMEOUT);
        return;
    }
    // an earlier CTA of this launch gave up on a wait: do not start new work on a broken pipeline
    if (p.dev_status != nullptr && *reinterpret_cast<volatile int32_t*>(p.dev_status) == JANUS_DEV_WAIT_TIMEOUT) return;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&sh->q_full), 1);
        mbar_init(smem_u32(&sh->qt_full), 4);
        for (int s = 0; s < LA_STAGES; ++s) { mbar_init(smem_u32(&sh->k_full[s]), LA_GATHER_WARPS); mbar_init(smem_u32(&sh->k_empty[s]), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&sh->s_full[b]), 1); mbar_init(smem_u32(&sh->p_full[b]), 4); }
        mbar_init(smem_u32(&sh->pv_done), 1);
        sh->aborted = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmap_q);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&sh->tmem_base), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;
    volatile int* aborted = &sh->aborted;

    if (warp == 0) {
        // ================================================================== TMA (query) + MMA issue, one thread
        if (lane == 0) {
            const uint32_t qf = smem_u32(&sh->q_full);
            mbar_expect_tx(qf, LA_Q_SMEM_ATOMS * LA_Q_ATOM_BYTES);
            for (int a = 0; a < LA_Q_SMEM_ATOMS; ++a)
                tma_load_2d(smem_u32(q_smem + a * LA_Q_ATOM_BYTES), &tmap_q, a * 64, t * LA_HEADS, qf);
            constexpr uint32_t idesc_qk = umma_idesc_major(1u, LA_HEADS, LA_BK, 0u, 0u);
            constexpr uint32_t idesc_pv = umma_idesc_major(1u, LA_HEADS, LA_DV_HALF, 0u, 1u);
            bool ok = mbar_wait(qf, 0) && mbar_wait(smem_u32(&sh->qt_full), 0);
            tc_fence_after();
            auto issue_pv = [&](int j) {   // O += P_j . V_j   (V = atoms 4*half .. 4*half+3 of the tile, MN-major)
                const int st = j % LA_STAGES, b = j & 1;
                const uint32_t v_base = smem_u32(k_smem + st * LA_STAGE_BYTES + (4 * half) * LA_K_ATOM_BYTES);
#pragma unroll
                for (int ks = 0; ks < LA_BK / 16; ++ks)
                    umma_bf16_ts(tmem_base + LA_COL_O, tmem_base + LA_COL_P + b * 16 + ks * 8,
                                 umma_desc_mn_sw128(v_base + ks * 2048, LA_K_ATOM_BYTES), idesc_pv, (j > 0 || ks > 0) ? 1u : 0u);
                umma_commit(smem_u32(&sh->k_empty[st]));
                umma_commit(smem_u32(&sh->pv_done));
            };
            for (int i = 0; i < n_tiles && ok; ++i) {
                const int st = i % LA_STAGES, b = i & 1;
                ok = mbar_wait(smem_u32(&sh->k_full[st]), static_cast<uint32_t>(i / LA_STAGES) & 1u) && !*aborted;
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_s = tmem_base + LA_COL_S + b * 32;
                const uint32_t kb = smem_u32(k_smem + st * LA_STAGE_BYTES);
                uint32_t acc = 0;
#pragma unroll
                for (int a = 0; a < LA_Q_SMEM_ATOMS; ++a) {
                    const uint32_t qa = smem_u32(q_smem + a * LA_Q_ATOM_BYTES);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {
                        umma<false>(d_s, umma_desc_sw128(qa + ks * 32), umma_desc_sw128(kb + a * LA_K_ATOM_BYTES + ks * 32), idesc_qk, acc);
                        acc = 1;
                    }
                }
#pragma unroll
                for (int a = 0; a < LA_Q_TMEM_ATOMS; ++a) {
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        umma_bf16_ts(d_s, tmem_base + LA_COL_Q + a * 32 + ks * 8,
                                     umma_desc_sw128(kb + (LA_Q_SMEM_ATOMS + a) * LA_K_ATOM_BYTES + ks * 32), idesc_qk, 1u);
                }
                umma_commit(smem_u32(&sh->s_full[b]));
                if (i >= 1) {
                    ok = mbar_wait(smem_u32(&sh->p_full[(i - 1) & 1]), static_cast<uint32_t>((i - 1) >> 1) & 1u) && !*aborted;
                    if (!ok) break;
                    tc_fence_after();
                    issue_pv(i - 1);
                }
            }
            if (ok && n_tiles > 0) {
                ok = mbar_wait(smem_u32(&sh->p_full[(n_tiles - 1) & 1]), static_cast<uint32_t>((n_tiles - 1) >> 1) & 1u) && !*aborted;
                if (ok) {
                    tc_fence_after();
                    issue_pv(n_tiles - 1);
                }
            }
            if (!ok) { *aborted = 1; report(p.dev_status, JANUS_DEV_WAIT_TIMEOUT); }
        }
    } else if (warp <= LA_GATHER_WARPS) {
        // ================================================================== gather: 4 warps x 8 rows of each tile
        const int g = warp - 1;
        const int32_t* my_idx = p.idx + static_cast<int64_t>(t) * p.k;
        bool ok = true;
        auto arrive_tile = [&](int j) {   // this warp's copies of tile j have landed: publish them to the MMA proxy
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->k_full[j % LA_STAGES]));
        };
        // Address resolution runs ahead of the copies so that neither the index load (HBM) nor the page-table load sits
        // on the per-tile critical path: indices are fetched two tiles ahead, page ids one tile ahead.
        auto load_raw = [&](int tile) -> int {
            const int slot = tile * LA_BK + lane;
            return (tile < n_tiles && slot < p.k) ? __ldg(my_idx + slot) : -1;
        };
        auto page_of = [&](int s_tok, int& within) -> int {   // returns the physical page id (or -1), issues the table load
            within = 0;
            if (s_tok < 0) return -1;
            const int64_t lp = p.page_shift >= 0 ? (s_tok >> p.page_shift) : (s_tok / p.page_size);
            within = p.page_shift >= 0 ? (s_tok & (p.page_size - 1)) : (s_tok % p.page_size);
            if (lp >= p.n_logical_pages) { report(p.dev_status, JANUS_DEV_INDEX_OUT_OF_RANGE); return -1; }
            return __ldg(p.page_table + lp);
        };
        int within_cur, within_nxt = 0;
        int page_cur = page_of(load_raw(0), within_cur);     // tile 0
        int raw_nxt = load_raw(1);                            // tile 1 (translated in iteration 0)
        int page_nxt = -1;
        for (int i = 0; i < n_tiles; ++i) {
            const int st = i % LA_STAGES;
            const int raw_nxt2 = load_raw(i + 2);             // consumed next iteration
            page_nxt = page_of(raw_nxt, within_nxt);          // table load issued now, consumed next iteration
            if (ok) ok = mbar_wait(smem_u32(&sh->k_empty[st]), (static_cast<uint32_t>(i / LA_STAGES) & 1u) ^ 1u) && !*aborted;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            // lane r holds the address of row r of the tile
            const int s = page_cur;                           // >= 0 iff the row is valid
            const unsigned char* row_ptr = reinterpret_cast<const unsigned char*>(p.pool);
            if (s >= 0) row_ptr += (static_cast<int64_t>(page_cur) * p.page_stride + static_cast<int64_t>(within_cur) * p.tok_stride) * 2;
            const uint32_t valid_mask = __ballot_sync(0xffffffffu, s >= 0);
            if (g == 0 && lane == 0) sh->vmask[st] = valid_mask;
            const uint32_t stage_base = smem_u32(k_smem + st * LA_STAGE_BYTES);
#pragma unroll
            for (int rr = 0; rr < LA_BK / LA_GATHER_WARPS; ++rr) {
                const int r = g * (LA_BK / LA_GATHER_WARPS) + rr;
                const unsigned char* src = reinterpret_cast<const unsigned char*>(__shfl_sync(0xffffffffu, reinterpret_cast<uint64_t>(row_ptr), r));
                const uint32_t bytes = ((valid_mask >> r) & 1u) ? 16u : 0u;
                // 72 chunks of 16 bytes per row: chunk c -> atom c/8, position (c%8) ^ (r%8) inside the 128-byte row
#pragma unroll
                for (int cc = 0; cc < 3; ++cc) {
                    const int c = lane + 32 * cc;
                    if (c < 72) {
                        const uint32_t dst = stage_base + (c >> 3) * LA_K_ATOM_BYTES + r * 128 + (((c & 7) ^ (r & 7)) << 4);
                        cp_async16(dst, src + c * 16, bytes);
                    }
                }
            }
            cp_async_commit();
            page_cur = page_nxt; within_cur = within_nxt; raw_nxt = raw_nxt2;
            if (i >= LA_LAG) {
                cp_async_wait<LA_LAG>();
                arrive_tile(i - LA_LAG);
            }
        }
        cp_async_wait<0>();
        if (ok) {
            for (int j = max(0, n_tiles - LA_LAG); j < n_tiles; ++j) arrive_tile(j);
        } else if (lane == 0) {
            *aborted = 1;
            report(p.dev_status, JANUS_DEV_WAIT_TIMEOUT);
        }
    } else {
        // ================================================================== softmax + output: 4 warps, thread = head
        const int quad = warp & 3;                         // warps 5,6,7,8 -> TMEM lane quadrants 1,2,3,0
        const int h = quad * 32 + lane;
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
        // query dims [320,576) of this head -> tensor memory, two bf16 per 32-bit column
        {
            const uint4* src = reinterpret_cast<const uint4*>(p.q + (static_cast<int64_t>(t) * LA_HEADS + h) * LA_DQK + LA_Q_SMEM_ATOMS * 64);
#pragma unroll
            for (int a = 0; a < LA_Q_TMEM_ATOMS; ++a) {
                uint32_t r[32];
#pragma unroll
                for (int v = 0; v < 8; ++v) {
                    const uint4 u = __ldg(src + a * 8 + v);
                    r[4 * v + 0] = u.x; r[4 * v + 1] = u.y; r[4 * v + 2] = u.z; r[4 * v + 3] = u.w;
                }
                tmem_st32_wait(lane_addr + LA_COL_Q + a * 32, r);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->qt_full));
        }
        const float neg_inf = __int_as_float(0xff800000);
        float m_ref = neg_inf;      // reference maximum (log2 domain) the exponentials are taken against
        float l_sum = 0.f;
        bool ok = true;
        for (int i = 0; i < n_tiles; ++i) {
            const int st = i % LA_STAGES, b = i & 1;
            if (ok) ok = mbar_wait(smem_u32(&sh->k_full[st]), static_cast<uint32_t>(i / LA_STAGES) & 1u) &&
                         mbar_wait(smem_u32(&sh->s_full[b]), static_cast<uint32_t>(i >> 1) & 1u) && !*aborted;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t vmask = sh->vmask[st];
            uint32_t r[32];
            tmem_ld32_wait(lane_addr + LA_COL_S + b * 32, r);
            float x[32];
            float tile_max = neg_inf;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                x[j] = ((vmask >> j) & 1u) ? __uint_as_float(r[j]) * p.scale_log2e : neg_inf;
                tile_max = fmaxf(tile_max, x[j]);
            }
            // move the reference maximum only when this tile exceeds it by more than 2^8 (or on first use)
            float corr = 1.f;
            bool moved = false;
            if (tile_max > m_ref + 8.f) {
                moved = (l_sum > 0.f);
                corr = moved ? fast_exp2(m_ref - tile_max) : 1.f;
                l_sum *= corr;
                m_ref = tile_max;
            }
            if (__any_sync(0xffffffffu, moved) && i > 0) {
                // rescale O in tensor memory: the previous tile's P.V must have completed first
                ok = mbar_wait(smem_u32(&sh->pv_done), static_cast<uint32_t>(i - 1) & 1u);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
#pragma unroll 1
                for (int c = 0; c < LA_DV_HALF / 32; ++c) {
                    uint32_t o[32];
                    tmem_ld32_wait(lane_addr + LA_COL_O + c * 32, o);
#pragma unroll
                    for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * corr);
                    tmem_st32_wait(lane_addr + LA_COL_O + c * 32, o);
                }
            }
            const float m_use = (m_ref == neg_inf) ? 0.f : m_ref;
            uint32_t pk[16];
            float tile_sum = 0.f;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const float p0 = fast_exp2(x[2 * j] - m_use), p1 = fast_exp2(x[2 * j + 1] - m_use);
                tile_sum += p0 + p1;
                pk[j] = pack_bf16x2(p0, p1);
            }
            l_sum += tile_sum;
            tmem_st16_wait(lane_addr + LA_COL_P + b * 16, pk);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->p_full[b]));
        }
        // ---- output: wait for the last P.V, normalise, round to bf16
        if (ok && n_tiles > 0) {
            ok = mbar_wait(smem_u32(&sh->pv_done), static_cast<uint32_t>(n_tiles - 1) & 1u) && !*aborted;
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            tc_fence_after();
            const float inv = l_sum > 0.f ? 1.f / l_sum : 0.f;
            const bool have_o = n_tiles > 0 && __any_sync(0xffffffffu, l_sum > 0.f);   // some P.V has written O
            uint16_t* orow = p.out + (static_cast<int64_t>(t) * LA_HEADS + h) * LA_DV + half * LA_DV_HALF;
#pragma unroll 1
            for (int c = 0; c < LA_DV_HALF / 32; ++c) {
                uint32_t o[32];
                if (have_o) {
                    tmem_ld32_wait(lane_addr + LA_COL_O + c * 32, o);
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) o[j] = 0u;
                }
                uint4* dst = reinterpret_cast<uint4*>(orow + c * 32);
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    uint4 u;
                    u.x = pack_bf16x2(__uint_as_float(o[8 * v + 0]) * inv, __uint_as_float(o[8 * v + 1]) * inv);
                    u.y = pack_bf16x2(__uint_as_float(o[8 * v + 2]) * inv, __uint_as_float(o[8 * v + 3]) * inv);
                    u.z = pack_bf16x2(__uint_as_float(o[8 * v + 4]) * inv, __uint_as_float(o[8 * v + 5]) * inv);
                    u.w = pack_bf16x2(__uint_as_float(o[8 * v + 6]) * inv, __uint_as_float(o[8 * v + 7]) * inv);
                    dst[v] = u;
                }
            }
            if (p.lse != nullptr && half == 0)
                p.lse[static_cast<int64_t>(t) * LA_HEADS + h] = l_sum > 0.f ? (m_ref + log2f(l_sum)) * 0.6931471805599453f : neg_inf;
        } else if (lane == 0) {
            *aborted = 1;
            report(p.dev_status, JANUS_DEV_WAIT_TIMEOUT);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

bool sparse_attn_latent_tc_supported(int M, int H_q, int d_qk, const void* k_pool, const void* v_pool, int64_t page_stride,
                                     int64_t tok_stride, int n_kv_heads, int d_v, int k) {
    if (H_q != LA_HEADS || d_qk != LA_DQK || d_v != LA_DV || n_kv_heads != 1 || k_pool != v_pool) return false;
    if ((page_stride % 8) != 0 || (tok_stride % 8) != 0 || tok_stride < LA_DQK) return false;
    if (M > (1 << 30) / LA_HEADS || k <= 0) return false;
    return true;
}

int launch_sparse_attn_latent_tc(const void* q, int M, const void* pool, int64_t page_stride, int64_t tok_stride, const int32_t* idx, int k,
                                 int page_size, const int32_t* page_table, int64_t n_logical_pages, float softmax_scale, void* out,
                                 float* lse, int32_t* dev_status, cudaStream_t stream) {
    LaParams p;
    p.q = static_cast<const uint16_t*>(q);
    p.pool = static_cast<const uint16_t*>(pool);
    p.page_stride = page_stride;
    p.tok_stride = tok_stride;
    p.idx = idx;
    p.k = k;
    p.page_size = page_size;
    p.page_shift = -1;
    if ((page_size & (page_size - 1)) == 0) {
        p.page_shift = 0;
        while ((1 << p.page_shift) < page_size) ++p.page_shift;
    }
    p.page_table = page_table;
    p.n_logical_pages = n_logical_pages;
    p.scale_log2e = softmax_scale * 1.4426950408889634f;
    p.out = static_cast<uint16_t*>(out);
    p.lse = lse;
    p.M = M;
    p.dev_status = dev_status;
    CUtensorMap tq;
    if (!make_tmap_2d_sw128(&tq, q, 2, static_cast<uint64_t>(M) * LA_HEADS, LA_DQK, static_cast<uint64_t>(LA_DQK) * 2, LA_HEADS, 64))
        return JANUS_ERR_CUDA;
    const size_t smem = LA_Q_SMEM_ATOMS * LA_Q_ATOM_BYTES + LA_STAGES * LA_STAGE_BYTES + sizeof(LaShared) + 16;
    JANUS_CUDA_CHECK(cudaFuncSetAttribute(sparse_attn_latent_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    sparse_attn_latent_tc_kernel<<<2 * M, LA_THREADS, smem, stream>>>(tq, p);
    JANUS_CUDA_CHECK(cudaGetLastError());
    return JANUS_OK;
}

}  // namespace janus
