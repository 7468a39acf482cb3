// Tensor-core sparse attention for the latent layout (Sec. 2.2, "core attention"): one shared KV row of 576 bf16
// per token (keys = all 576 dims, values = the first 512), 128 query heads, selection idx[t, 0:k).
//
//     out[t,h,:] = sum_{s in idx[t]} softmax_s(scale * <q[t,h,:576], row_s[:576]>) * row_s[:512]
//
// Shape of the problem on one SM.  The heads of one token form the MMA M axis (128 heads = 128 TMEM lanes), so the
// fp32 output accumulator is 128 lanes x 512 columns = all of tensor memory.  The value dimension is therefore
// split in two: CTA (t, c) owns value columns [256c, 256c+256) and recomputes the logits.  Shared memory cannot hold
// the 144 KB query tile next to a useful key ring, so query dims [0,256) stay in shared memory (4 swizzle atoms) and
// dims [256,576) live in tensor memory as a TMEM-resident A operand.  Tensor memory: O 256 columns, two logit
// buffers of 48 columns (the bf16 probabilities overwrite the first 24 columns of their logits), query tail 160.
//
// Keys move in half-tiles of 24 rows (27 KB; a ring of six), two of which form one 48-key tile with the rows of
// each 64-dim atom contiguous, so that S = Q.K^T is issued as 36 MMAs of 128x48x16 per tile and three tiles are
// resident: one being multiplied, one landing, one being issued.  Each of six gather warps owns one ring slot: it resolves the 24 rows through the page table and copies them with 16-byte cp.async into the
// swizzled layout (the index load for its next half-tile is issued before the copies);  the MMA thread issues S for tile i+1 before O += P.V
// of tile i (3 MMAs 128x256x16, V read MN-major out of the same rows) and frees each half-tile as soon as the
// P.V MMAs that read it are done;  softmax warps (thread = head) read S from TMEM, keep a running max / sum in fp32 registers
// and write P as bf16 back to TMEM.  The running max is only moved when a tile exceeds it by more than 2^8, so O
// is rescaled (in TMEM) a handful of times per row.
// Every wait is bounded; on a timeout the CTA reports JANUS_DEV_WAIT_TIMEOUT and winds down.
#include "janus_common.cuh"
#include "sm100_ptx.cuh"

namespace janus {

using namespace ptx;

constexpr int LA_HEADS = 128;
constexpr int LA_DQK = 576;
constexpr int LA_DV = 512;
constexpr int LA_DV_HALF = 256;
constexpr int LA_BK = 24;                 // keys per half-tile (gather / release granularity)
constexpr int LA_BUFS = 3;                // 48-key tile buffers in the ring
constexpr int LA_STAGES = 2 * LA_BUFS;    // half-tiles in the ring; half-tiles 2j, 2j+1 form tile j
constexpr int LA_TILE = 2 * LA_BK;        // keys per MMA tile
constexpr int LA_ATOMS = 9;               // 576 / 64
constexpr int LA_Q_SMEM_ATOMS = 4;        // query dims [0,256) in shared memory
constexpr int LA_Q_TMEM_ATOMS = 5;        // query dims [256,576) in tensor memory
constexpr int LA_Q_ATOM_BYTES = LA_HEADS * 128;        // 16 KB
constexpr int LA_K_ATOM_BYTES = LA_TILE * 128;         // 6 KB: one 64-dim atom of a 48-key tile
constexpr int LA_TILE_BYTES = LA_ATOMS * LA_K_ATOM_BYTES;    // 54 KB per 48-key tile
constexpr int LA_GATHER_WARPS = LA_STAGES;   // one gather warp per ring slot
constexpr int LA_THREADS = 32 * (1 + LA_GATHER_WARPS + 4);   // warp 0: MMA + TMA; warps 1-6: gather; warps 7-10: softmax
// tensor-memory columns
constexpr uint32_t LA_COL_O = 0, LA_COL_S = 256, LA_COL_Q = 352;   // O 256 | S (and P) 2 x 48 | query tail 160

struct LaShared {
    uint64_t q_full, qt_full;
    uint64_t k_full[LA_BUFS], k_empty[LA_BUFS];   // per 48-key tile buffer: rows landed / P.V of the tile done
    uint64_t s_full[2], p_full[2];
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

// Optional per-role cycle accounting for tuning (off in the product build): with -DJANUS_ATTN_PROFILE the lse output of
// token t receives, instead of the log-sum-exp, the cycles each role spent in total and inside its waits.
#ifdef JANUS_ATTN_PROFILE
#define LA_PROF_DECL(name) long long name = 0
#define LA_PROF_WAIT(acc, expr) ([&] { const long long _t0 = clock64(); const bool _r = (expr); acc += clock64() - _t0; return _r; }())
#define LA_PROF_NOW() clock64()
#define LA_PROF_PUT(slot, v) do { if (p.lse != nullptr && half == 0) p.lse[static_cast<int64_t>(t) * LA_HEADS + (slot)] = static_cast<float>(v); } while (0)
#else
#define LA_PROF_DECL(name)
#define LA_PROF_WAIT(acc, expr) (expr)
#define LA_PROF_NOW() 0
#define LA_PROF_PUT(slot, v) do { } while (0)
#endif

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
    unsigned char* k_smem = smem + LA_Q_SMEM_ATOMS * LA_Q_ATOM_BYTES;          // 3 tiles x 9 atoms x [48 keys x 128 B]
    LaShared* sh = reinterpret_cast<LaShared*>(k_smem + LA_BUFS * LA_TILE_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t = blockIdx.x >> 1;
    const int half = blockIdx.x & 1;
    const int n_tiles = (p.k + LA_TILE - 1) / LA_TILE;     // 64-key tiles
    const int n_half = 2 * n_tiles;                         // 32-key half-tiles (the last may be all padding)

    if ((smem_u32(smem) & 1023u) != 0u) {
        if (threadIdx.x == 0) report(p.dev_status, JANUS_DEV_WAIT_TIMEOUT);
        return;
    }
    // an earlier CTA of this launch gave up on a wait: do not start new work on a broken pipeline
    if (p.dev_status != nullptr && *reinterpret_cast<volatile int32_t*>(p.dev_status) == JANUS_DEV_WAIT_TIMEOUT) return;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&sh->q_full), 1);
        mbar_init(smem_u32(&sh->qt_full), 4);
        for (int s = 0; s < LA_BUFS; ++s) { mbar_init(smem_u32(&sh->k_full[s]), 2); mbar_init(smem_u32(&sh->k_empty[s]), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&sh->s_full[b]), 1); mbar_init(smem_u32(&sh->p_full[b]), 4); }
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
        // ================================================================== TMA (query) + MMA issue
        // The whole warp runs the loop (uniform control flow and address arithmetic); only lane 0 issues.
        const bool leader = lane == 0;
        const uint32_t qf = smem_u32(&sh->q_full);
        if (leader) {
            mbar_expect_tx(qf, LA_Q_SMEM_ATOMS * LA_Q_ATOM_BYTES);
            for (int a = 0; a < LA_Q_SMEM_ATOMS; ++a)
                tma_load_2d(smem_u32(q_smem + a * LA_Q_ATOM_BYTES), &tmap_q, a * 64, t * LA_HEADS, qf);
        }
        constexpr uint32_t idesc_qk = umma_idesc_major(1u, LA_HEADS, LA_TILE, 0u, 0u);
        constexpr uint32_t idesc_pv = umma_idesc_major(1u, LA_HEADS, LA_DV_HALF, 0u, 1u);
        LA_PROF_DECL(w_kfull); LA_PROF_DECL(w_pfull); LA_PROF_DECL(w_q);
        const long long prof_t0 = LA_PROF_NOW();
        bool ok = LA_PROF_WAIT(w_q, mbar_wait(qf, 0) && mbar_wait(smem_u32(&sh->qt_full), 0));
        tc_fence_after();
        const uint32_t q_lo = umma_desc_lo(smem_u32(q_smem), 16);
        const uint32_t k_lo = umma_desc_lo(smem_u32(k_smem), 16);
        const uint32_t v_lo = umma_desc_lo(smem_u32(k_smem + (4 * half) * LA_K_ATOM_BYTES), LA_K_ATOM_BYTES);
        auto issue_pv = [&](int j) {   // O += P_j . V_j   (V = atoms 4*half .. 4*half+3 of tile j, MN-major)
            const int b = j & 1, buf = j % LA_BUFS;
            const uint32_t vb = v_lo + static_cast<uint32_t>(buf * (LA_TILE_BYTES >> 4));
            const uint32_t pa = tmem_base + LA_COL_S + b * LA_TILE;
            if (leader) {
#pragma unroll
                for (int ks = 0; ks < LA_TILE / 16; ++ks)
                    umma_bf16_ts_lohi(tmem_base + LA_COL_O, pa + ks * 8, vb + ks * (2048 >> 4), idesc_pv, (j > 0 || ks > 0) ? 1u : 0u);
                umma_commit(smem_u32(&sh->k_empty[buf]));   // tile buffer free again, and "P.V of tile j done" for the softmax warps
            }
        };
        for (int i = 0; i < n_tiles && ok; ++i) {
            const int b = i & 1, buf = i % LA_BUFS;
            const uint32_t ph = static_cast<uint32_t>(i / LA_BUFS) & 1u;   // tile i is the (i/3)-th use of its buffer
            ok = LA_PROF_WAIT(w_kfull, mbar_wait(smem_u32(&sh->k_full[buf]), ph));
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_s = tmem_base + LA_COL_S + b * LA_TILE;
            const uint32_t kb = k_lo + static_cast<uint32_t>(buf * (LA_TILE_BYTES >> 4));
            if (leader) {
#pragma unroll
                for (int a = 0; a < LA_Q_SMEM_ATOMS; ++a) {
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        umma_bf16_ss_lohi(d_s, q_lo + a * (LA_Q_ATOM_BYTES >> 4) + ks * 2, kb + a * (LA_K_ATOM_BYTES >> 4) + ks * 2, idesc_qk,
                                          (a > 0 || ks > 0) ? 1u : 0u);
                }
#pragma unroll
                for (int a = 0; a < LA_Q_TMEM_ATOMS; ++a) {
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        umma_bf16_ts_lohi(d_s, tmem_base + LA_COL_Q + a * 32 + ks * 8, kb + (LA_Q_SMEM_ATOMS + a) * (LA_K_ATOM_BYTES >> 4) + ks * 2,
                                          idesc_qk, 1u);
                }
                umma_commit(smem_u32(&sh->s_full[b]));
            }
            if (i >= 1) {
                ok = LA_PROF_WAIT(w_pfull, mbar_wait(smem_u32(&sh->p_full[(i - 1) & 1]), static_cast<uint32_t>((i - 1) >> 1) & 1u));
                if (!ok) break;
                tc_fence_after();
                issue_pv(i - 1);
            }
        }
        if (ok && n_tiles > 0) {
            ok = mbar_wait(smem_u32(&sh->p_full[(n_tiles - 1) & 1]), static_cast<uint32_t>((n_tiles - 1) >> 1) & 1u);
            if (ok) {
                tc_fence_after();
                issue_pv(n_tiles - 1);
            }
        }
        if (!ok && leader) { *aborted = 1; report(p.dev_status, JANUS_DEV_WAIT_TIMEOUT); }
        if (leader) { LA_PROF_PUT(0, LA_PROF_NOW() - prof_t0); LA_PROF_PUT(1, w_kfull); LA_PROF_PUT(2, w_pfull); LA_PROF_PUT(9, w_q); }
    } else if (warp <= LA_GATHER_WARPS) {
        // ================================================================== gather: warp g owns ring slot g (half-tiles g, g+6, ...)
        // A warp copies whole half-tiles (24 rows x 1152 bytes), so address resolution is done once per half-tile and no
        // two warps ever synchronise; the whole ring can be in flight.  Because a warp always returns to the same slot,
        // the slot's barrier is exactly one phase ahead of it at most, which the parity wait relies on.
        const int g = warp - 1;
        const int32_t* my_idx = p.idx + static_cast<int64_t>(t) * p.k;
        bool ok = true;
        LA_PROF_DECL(w_kempty); LA_PROF_DECL(w_group);
        const long long prof_t0 = LA_PROF_NOW();
        auto load_raw = [&](int hi) -> int {                 // lane r < 24 owns row r of half-tile hi
            const int slot = hi * LA_BK + lane;
            return (lane < LA_BK && hi < n_half && slot < p.k) ? __ldg(my_idx + slot) : -1;
        };
        int raw = load_raw(g);
        for (int hi = g; hi < n_half; hi += LA_GATHER_WARPS) {
            const int st = hi % LA_STAGES;
            // resolve this half-tile's rows; fetch the indices of this warp's next half-tile while the copies run
            int s_tok = raw;
            const unsigned char* row_ptr = reinterpret_cast<const unsigned char*>(p.pool);
            if (s_tok >= 0) {
                const int64_t lp = p.page_shift >= 0 ? (s_tok >> p.page_shift) : (s_tok / p.page_size);
                const int within = p.page_shift >= 0 ? (s_tok & (p.page_size - 1)) : (s_tok % p.page_size);
                if (lp >= p.n_logical_pages) {
                    report(p.dev_status, JANUS_DEV_INDEX_OUT_OF_RANGE);
                    s_tok = -1;
                } else {
                    row_ptr += (static_cast<int64_t>(__ldg(p.page_table + lp)) * p.page_stride + static_cast<int64_t>(within) * p.tok_stride) * 2;
                }
            }
            raw = load_raw(hi + LA_GATHER_WARPS);
            const uint32_t valid_mask = __ballot_sync(0xffffffffu, s_tok >= 0);
            // the buffer must have been released by the P.V three tiles back
            ok = LA_PROF_WAIT(w_kempty, mbar_wait(smem_u32(&sh->k_empty[st >> 1]), (static_cast<uint32_t>(hi / LA_STAGES) & 1u) ^ 1u));
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (lane == 0) sh->vmask[st] = valid_mask;
            // half-tile st = rows [24*(st&1), +24) of tile buffer st>>1
            const uint32_t stage_base = smem_u32(k_smem + (st >> 1) * LA_TILE_BYTES + (st & 1) * LA_BK * 128);
#pragma unroll 4
            for (int r = 0; r < LA_BK; ++r) {
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
            LA_PROF_WAIT(w_group, (cp_async_wait<0>(), true));
            fence_proxy_async();              // publish the landed rows to the MMA (async) proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->k_full[st >> 1]));
        }
        if (!ok && lane == 0) {
            *aborted = 1;
            report(p.dev_status, JANUS_DEV_WAIT_TIMEOUT);
        }
        if (g == 0 && lane == 0) { LA_PROF_PUT(3, LA_PROF_NOW() - prof_t0); LA_PROF_PUT(4, w_kempty); LA_PROF_PUT(5, w_group); }
    } else {
        // ================================================================== softmax + output: 4 warps, thread = head
        const int quad = warp & 3;                         // warps 7..10 -> TMEM lane quadrants 3,0,1,2
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
        LA_PROF_DECL(w_sfull); LA_PROF_DECL(w_pv);
        const long long prof_t0 = LA_PROF_NOW();
        for (int i = 0; i < n_tiles; ++i) {
            const int b = i & 1, buf = i % LA_BUFS;
            const uint32_t ph_k = static_cast<uint32_t>(i / LA_BUFS) & 1u, ph_s = static_cast<uint32_t>(i >> 1) & 1u;
            // k_full is complete long before s_full; waiting on it as well makes the validity masks written by the gather
            // warps visible to this thread directly rather than through the MMA warp
            if (ok) ok = LA_PROF_WAIT(w_sfull, mbar_wait(smem_u32(&sh->k_full[buf]), ph_k) && mbar_wait(smem_u32(&sh->s_full[b]), ph_s));
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            // key j of the tile is valid iff bit j of the 48-bit mask is set
            const uint64_t vm = static_cast<uint64_t>(sh->vmask[2 * buf]) | (static_cast<uint64_t>(sh->vmask[2 * buf + 1]) << LA_BK);
            const uint32_t s_addr = lane_addr + LA_COL_S + b * LA_TILE;
            float x[LA_TILE];
            float tile_max = neg_inf;
            {
                uint32_t r[32];
                tmem_ld32_wait(s_addr, r);
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    x[j] = ((vm >> j) & 1ull) ? __uint_as_float(r[j]) * p.scale_log2e : neg_inf;
                    tile_max = fmaxf(tile_max, x[j]);
                }
                uint32_t r2[16];
                tmem_ld16_wait(s_addr + 32, r2);
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    x[32 + j] = ((vm >> (32 + j)) & 1ull) ? __uint_as_float(r2[j]) * p.scale_log2e : neg_inf;
                    tile_max = fmaxf(tile_max, x[32 + j]);
                }
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
                ok = mbar_wait(smem_u32(&sh->k_empty[(i - 1) % LA_BUFS]), static_cast<uint32_t>((i - 1) / LA_BUFS) & 1u);
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
            uint32_t pk[16], pk2[8];
            float tile_sum = 0.f;
#pragma unroll
            for (int j = 0; j < LA_TILE / 2; ++j) {
                const float p0 = fast_exp2(x[2 * j] - m_use), p1 = fast_exp2(x[2 * j + 1] - m_use);
                tile_sum += p0 + p1;
                if (j < 16) pk[j] = pack_bf16x2(p0, p1); else pk2[j - 16] = pack_bf16x2(p0, p1);
            }
            l_sum += tile_sum;
            tmem_st16_wait(s_addr, pk);          // P overwrites the first 24 columns of its own logits
            tmem_st8_wait(s_addr + 16, pk2);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->p_full[b]));
        }
        // ---- output: wait for the last P.V, normalise, round to bf16
        if (ok && n_tiles > 0) {
            ok = LA_PROF_WAIT(w_pv, mbar_wait(smem_u32(&sh->k_empty[(n_tiles - 1) % LA_BUFS]), static_cast<uint32_t>((n_tiles - 1) / LA_BUFS) & 1u));
            ok = __all_sync(0xffffffffu, ok);
        }
        const long long prof_loop = LA_PROF_NOW() - prof_t0;
        (void)prof_loop;
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
#ifndef JANUS_ATTN_PROFILE
            if (p.lse != nullptr && half == 0)
                p.lse[static_cast<int64_t>(t) * LA_HEADS + h] = l_sum > 0.f ? (m_ref + log2f(l_sum)) * 0.6931471805599453f : neg_inf;
#else
            if (warp == 1 + LA_GATHER_WARPS && lane == 0) { LA_PROF_PUT(6, prof_loop); LA_PROF_PUT(7, w_sfull); LA_PROF_PUT(8, w_pv); LA_PROF_PUT(10, LA_PROF_NOW() - prof_t0); }
#endif
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
    const size_t smem = LA_Q_SMEM_ATOMS * LA_Q_ATOM_BYTES + LA_BUFS * LA_TILE_BYTES + sizeof(LaShared) + 16;
    JANUS_CUDA_CHECK(cudaFuncSetAttribute(sparse_attn_latent_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    sparse_attn_latent_tc_kernel<<<2 * M, LA_THREADS, smem, stream>>>(tq, p);
    JANUS_CUDA_CHECK(cudaGetLastError());
    return JANUS_OK;
}

}  // namespace janus
