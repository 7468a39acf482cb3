// Tensor-core sparse attention for the latent layout (Sec. 2.2, "core attention"): one shared KV row of 576 bf16
// per token (keys = all 576 dims, values = the first 512), 128 query heads, selection idx[t, 0:k).
//
//     out[t,h,:] = sum_{s in idx[t]} softmax_s(scale * <q[t,h,:576], row_s[:576]>) * row_s[:512]
//
// Shape of the problem.  The heads of one token form the MMA M axis (128 heads = 128 TMEM lanes), so the fp32 output
// accumulator, 128 lanes x 512 columns, is all of one SM's tensor memory.  One token is therefore handled by a
// cluster of two CTAs that split the work along the *feature* axis, so that nothing is computed or fetched twice:
//
//   CTA 0 owns row bytes [0,512)    = dims [0,256):    value half 0, and the first 256 dims of the logit contraction;
//   CTA 1 owns row bytes [512,1152) = dims [256,576):  value half 1, and the last 320 dims of the contraction.
//
// Each CTA gathers only its own bytes of every selected row, computes a partial logit tile S_c = Q_c . K_c^T
// (128 heads x 64 keys, fp32 in tensor memory), and the two partial tiles are exchanged through distributed shared
// memory: the exchange warps send the 64 partial logits of every head into the peer's exchange buffer with asynchronous
// remote stores that are counted on the peer's mbarrier as they land.  The partial logits travel as fp16 (11 significant
// bits; P itself is bf16): the link between the two SMs is the slowest step of the tile loop, and half the bytes also
// make room for a fourth ring buffer.  Each CTA adds the peer's values to its own fp32 partial logits, runs the fp32
// online softmax, writes P (bf16) to its own place in tensor memory and accumulates O_c += P . V_c with V_c read
// MN-major from the gathered rows (the value half of CTA c is the first 256 dims of the bytes it owns).
//
// Per CTA: tensor memory = O 256 | two logit buffers of 64 | P 32 | queries 96 columns (three atoms of 64 dims as the A
// operand; the fourth atom, and the 64 rope dims on CTA 1, sit in shared memory).  Keys move in half-tiles of 32 rows
// through a ring of four 64-key tiles.  Warp roles (12 warps, 168 registers per thread available):
//   warp 0       issues the MMAs in the order their inputs become ready: a logit tile (12 MMAs 128x64x16 from tensor
//                memory + 4 or 8 from shared memory) needs its rows and a logit buffer that every reader has in registers,
//                so it runs about two tiles ahead of the softmax; O += P.V (4 MMAs 128x256x16) needs P;
//   warps 1-3    gather: warp g owns the ring slots s with s % 3 == g, resolves its 32 rows through the page table (one
//                half-tile ahead) and copies this CTA's bytes with 16-byte cp.async into the 128-byte-swizzled K-major
//                layout, 4 rows x 128 bytes per instruction;
//   warps 4-7    exchange: as soon as a partial logit tile is complete they take it into registers, free the logit
//                buffer and send it to the peer; after a token's last tile they load the next token's queries (prefetched
//                into L2 one token earlier);
//   warps 8-11   softmax (thread = head): add the peer's partial logits, fp32 online softmax, write P.
// The kernel is persistent: one cluster per SM pair loops over tokens, and the ring, the logit buffers and all barrier
// phases run on across tokens, so a token's prologue (queries into tensor memory, first gathers) hides behind the previous
// token's last tiles and output.
// The running max only moves when a tile exceeds it by more than 2^8, so O is rescaled (in tensor memory) a handful of
// times per row.  Every wait is bounded; on a timeout the CTA reports JANUS_DEV_WAIT_TIMEOUT, and both CTAs of the
// cluster still meet at the final cluster barrier.
#include <cuda_fp16.h>

#include "janus_common.cuh"
#include "sm100_ptx.cuh"

namespace janus {

using namespace ptx;

constexpr int LP_HEADS = 128;
constexpr int LP_DQK = 576;
constexpr int LP_DV = 512;
constexpr int LP_DVH = 256;
constexpr int LP_HALF = 32;                 // rows per half-tile (gather / ring-slot granularity)
constexpr int LP_TILE = 2 * LP_HALF;        // keys per MMA tile
constexpr int LP_BUFS = 4;                  // 64-key tile buffers
constexpr int LP_SLOTS = 2 * LP_BUFS;       // ring slots (half-tiles)
constexpr int LP_GATHER_WARPS = 3;          // warp g owns the ring slots s with s % 3 == g; 12 warps in all leave
                                            // 168 registers per thread, which the softmax needs to stay out of local memory
constexpr int LP_ATOMS_MAX = 5;             // 64-dim atoms owned by a CTA: 4 (CTA 0) or 5 (CTA 1)
constexpr int LP_K_ATOM_BYTES = LP_TILE * 128;                   // 8 KB
constexpr int LP_TILE_BYTES = LP_ATOMS_MAX * LP_K_ATOM_BYTES;    // 40 KB
constexpr int LP_XBUF_BYTES = LP_TILE * LP_HEADS * 2;            // 16 KB: partial logits from the peer, [key/8][head][8] fp16
constexpr int LP_Q_ATOM_BYTES = LP_HEADS * 128;                  // 16 KB
constexpr int LP_XCHG_WARP0 = 1 + LP_GATHER_WARPS;               // first exchange warp
constexpr int LP_SMAX_WARP0 = LP_XCHG_WARP0 + 4;                 // first softmax warp
constexpr int LP_THREADS = 32 * (LP_SMAX_WARP0 + 4);             // 12 warps
constexpr int LP_Q_TMEM_ATOMS = 3;                               // query atoms kept in tensor memory; the others sit in shared memory
constexpr int LP_QS_BYTES = 2 * LP_Q_ATOM_BYTES;                 // 32 KB: owned query atom 3 (and 4 on CTA 1)
constexpr uint32_t LP_COL_O = 0, LP_COL_S = 256, LP_COL_P = 384, LP_COL_Q = 416;   // O 256 | 2 x 64 logits | P 32 | 3 x 32 query

struct LpShared {
    uint64_t q_full, qt_full;
    uint64_t k_full[LP_BUFS], k_empty[LP_BUFS];   // per tile buffer: rows landed (2 half-tiles) / P.V of the tile done
    uint64_t s_full[2];                           // logits of the tile using logit buffer b are complete
    uint64_t s_free[2];                           // every reader (4 softmax + 4 exchange warps) has logit buffer b in registers
    uint64_t p_full;                              // P of the tile is in tensor memory
    uint64_t x_full[2];                           // the peer's partial logits of the tile using logit buffer b have arrived
    uint64_t x_empty[2];                          // the PEER has read this CTA's previous partial logits out of its exchange buffer b
    uint32_t vmask[LP_SLOTS];
    uint32_t tmem_base;
    uint32_t start_abort[2];
};

struct LpParams {
    const uint16_t* q;
    const uint16_t* pool;
    int64_t page_stride, tok_stride;
    const int32_t* idx;
    int k;
    int page_size, page_shift;
    const int32_t* page_table;
    int64_t n_logical_pages;
    const int64_t* table_offsets;   // NULL, or [M + 1]: row t uses page_table[table_offsets[t] .. table_offsets[t + 1])
    float scale_log2e;        // softmax_scale * log2(e)
    uint16_t* out;
    float* lse;
    int M;
    int32_t* dev_status;
};

__device__ __forceinline__ float lp_exp2(float x) {   // ex2.approx: 2 ulp, exp2(-inf) = 0
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t lp_pack_f16x2(float lo, float hi) {   // saturating: a logit beyond the fp16 range stays finite
    const __half2 v = __floats2half2_rn(fminf(fmaxf(lo, -65504.f), 65504.f), fminf(fmaxf(hi, -65504.f), 65504.f));
    return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t lp_pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(LP_THREADS, 1)
sparse_attn_latent_pair_kernel(const __grid_constant__ CUtensorMap tmap_q, const LpParams p) {
    extern __shared__ __align__(1024) unsigned char smem[];
    unsigned char* k_smem = smem;                                              // 3 tiles x 5 atoms x [64 keys x 128 B]
    unsigned char* xbuf = smem + LP_BUFS * LP_TILE_BYTES;                      // 2 x [64 keys / 8][128 heads][8 keys] fp16
    unsigned char* q_smem = smem + LP_BUFS * LP_TILE_BYTES + 2 * LP_XBUF_BYTES;    // owned query atom 3 (and 4 on CTA 1), each [128 heads x 128 B]
    LpShared* sh = reinterpret_cast<LpShared*>(q_smem + LP_QS_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t c = cluster_ctarank();          // 0 or 1: which bytes of the rows this CTA owns
    const uint32_t peer = c ^ 1u;
    // persistent: cluster `cid` handles tokens cid, cid + n_clusters, ...; the key ring, the logit buffers and every barrier
    // phase run on across tokens (tiles are counted globally), so the next token's rows are gathered, and its queries
    // loaded, while the current token's last tiles and output are still in flight
    const int cid = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
    const int n_my = cid < p.M ? (p.M - cid + n_clusters - 1) / n_clusters : 0;
    const int n_atoms = 4 + static_cast<int>(c);
    const int n_tiles = (p.k + LP_TILE - 1) / LP_TILE;
    const int n_half = 2 * n_tiles;

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&sh->q_full), 1);
        mbar_init(smem_u32(&sh->qt_full), 4);
        for (int s = 0; s < LP_BUFS; ++s) { mbar_init(smem_u32(&sh->k_full[s]), 2); mbar_init(smem_u32(&sh->k_empty[s]), 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&sh->s_full[b]), 1);
            mbar_init(smem_u32(&sh->s_free[b]), 8);
            mbar_init(smem_u32(&sh->x_full[b]), 1);
            mbar_init(smem_u32(&sh->x_empty[b]), 4);
        }
        mbar_init(smem_u32(&sh->p_full), 4);
        fence_mbar_init();
        prefetch_tensormap(&tmap_q);
        // start-up agreement: if this CTA should not start (misaligned shared memory, or an earlier CTA of the launch gave
        // up on a wait), both CTAs of the cluster must skip the work, so the flag is written to both of them
        uint32_t flag = ((smem_u32(smem) & 1023u) != 0u) ? 1u : 0u;
        if (p.dev_status != nullptr && *reinterpret_cast<volatile int32_t*>(p.dev_status) == JANUS_DEV_WAIT_TIMEOUT) flag = 1u;
        sh->start_abort[c] = flag;
        st_cluster_u32(mapa_shared(smem_u32(&sh->start_abort[c]), peer), flag);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&sh->tmem_base), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                            // barriers of both CTAs are initialised, start flags exchanged
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;
    const bool start_abort = (sh->start_abort[0] | sh->start_abort[1]) != 0u;
    if (start_abort && threadIdx.x == 0 && (smem_u32(smem) & 1023u) != 0u) report(p.dev_status, JANUS_DEV_WAIT_TIMEOUT);

    if (start_abort) {
        // nothing to do
    } else if (warp == 0) {
        // ================================================================== MMA issue
        // Lane 0 runs the whole role.  Logit tiles and P.V products are issued in whatever order their inputs become
        // ready (P.V first when both are).  P has a place of its own in tensor memory, so a logit tile only needs its rows
        // and a logit buffer whose previous contents every reader holds in registers: it is issued while the softmax of
        // two tiles earlier is still running, and the softmax does not wait for the tensor pipe to turn around.
        const uint32_t qf = smem_u32(&sh->q_full);
        auto fetch_q = [&](int it) {       // owned query atom 3 (and 4 on CTA 1) of all heads of this cluster's token `it`
            const int y = (cid + it * n_clusters) * LP_HEADS;
            mbar_expect_tx(qf, static_cast<uint32_t>((n_atoms - LP_Q_TMEM_ATOMS) * LP_Q_ATOM_BYTES));
            tma_load_2d(smem_u32(q_smem), &tmap_q, 256 * static_cast<int>(c) + 64 * LP_Q_TMEM_ATOMS, y, qf);
            if (c == 1u) tma_load_2d(smem_u32(q_smem + LP_Q_ATOM_BYTES), &tmap_q, 512, y, qf);
        };
        if (lane == 0) {
            if (n_my > 0) fetch_q(0);
            constexpr uint32_t idesc_qk = umma_idesc_major(1u, LP_HEADS, LP_TILE, 0u, 0u);
            constexpr uint32_t idesc_pv = umma_idesc_major(1u, LP_HEADS, LP_DVH, 0u, 1u);

            const uint32_t q_lo = umma_desc_lo(smem_u32(q_smem), 16);
            const uint32_t k_lo = umma_desc_lo(smem_u32(k_smem), 16);
            const uint32_t v_lo = umma_desc_lo(smem_u32(k_smem), LP_K_ATOM_BYTES);     // value half = first four owned atoms
            bool ok = true;
            int s_next = 0, pv_next = 0;                 // next logit tile / next P.V to issue, counted over all tokens
            for (int it = 0; it < n_my && ok; ++it) {
                ok = (mbar_wait(qf, static_cast<uint32_t>(it) & 1u) && mbar_wait(smem_u32(&sh->qt_full), static_cast<uint32_t>(it) & 1u));
                if (!ok) break;
                tc_fence_after();
                const int tok_begin = it * n_tiles, tok_end = tok_begin + n_tiles;
                uint32_t idle = 0;
                while (pv_next < tok_end) {
                    if (pv_next < s_next && mbar_test_wait(smem_u32(&sh->p_full), static_cast<uint32_t>(pv_next) & 1u)) {
                        // O += P_j . V_j
                        tc_fence_after();
                        const int j = pv_next, buf = j % LP_BUFS;
                        const uint32_t vb = v_lo + static_cast<uint32_t>(buf * (LP_TILE_BYTES >> 4));
#pragma unroll
                        for (int ks = 0; ks < LP_TILE / 16; ++ks)
                            umma_bf16_ts_lohi(tmem_base + LP_COL_O, tmem_base + LP_COL_P + ks * 8, vb + ks * (2048 >> 4), idesc_pv,
                                              (j > tok_begin || ks > 0) ? 1u : 0u);
                        umma_commit(smem_u32(&sh->k_empty[buf]));   // tile buffer and P free again; "P.V of tile j done" for the softmax warps
                        ++pv_next;
                        idle = 0;
                    } else if (s_next < tok_end && mbar_test_wait(smem_u32(&sh->k_full[s_next % LP_BUFS]), static_cast<uint32_t>(s_next / LP_BUFS) & 1u) &&
                               (s_next < 2 || mbar_test_wait(smem_u32(&sh->s_free[s_next & 1]), static_cast<uint32_t>((s_next - 2) >> 1) & 1u))) {
                        // S_j = Q . K_j^T into logit buffer j & 1
                        tc_fence_after();
                        const int b = s_next & 1, buf = s_next % LP_BUFS;
                        const uint32_t d_s = tmem_base + LP_COL_S + b * LP_TILE;
                        const uint32_t kb = k_lo + static_cast<uint32_t>(buf * (LP_TILE_BYTES >> 4));
#pragma unroll
                        for (int a = 0; a < LP_Q_TMEM_ATOMS; ++a) {
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks)
                                umma_bf16_ts_lohi(d_s, tmem_base + LP_COL_Q + a * 32 + ks * 8, kb + a * (LP_K_ATOM_BYTES >> 4) + ks * 2, idesc_qk,
                                                  (a > 0 || ks > 0) ? 1u : 0u);
                        }
#pragma unroll
                        for (int a = LP_Q_TMEM_ATOMS; a < LP_ATOMS_MAX; ++a) {
                            if (a < n_atoms) {
#pragma unroll
                                for (int ks = 0; ks < 4; ++ks)
                                    umma_bf16_ss_lohi(d_s, q_lo + (a - LP_Q_TMEM_ATOMS) * (LP_Q_ATOM_BYTES >> 4) + ks * 2,
                                                      kb + a * (LP_K_ATOM_BYTES >> 4) + ks * 2, idesc_qk, 1u);
                            }
                        }
                        umma_commit(smem_u32(&sh->s_full[b]));
                        ++s_next;
                        idle = 0;
                    } else if (++idle > (1u << 21)) {     // nothing became ready for some two million probes (a few tenths of a second): give up
                        ok = false;
                        break;
                    }
                }
                if (!ok) break;
                // every P of the token exists, so every logit MMA of the token has completed: its queries may be replaced;
                // the output of the token is read out of O before the softmax warps produce the next token's first P
                if (it + 1 < n_my) fetch_q(it + 1);
            }
            if (!ok) report(p.dev_status, JANUS_DEV_WAIT_TIMEOUT);
        }
        __syncwarp();
    } else if (warp <= LP_GATHER_WARPS) {
        // ================================================================== gather: warp g owns the ring slots s with s % 3 == g
        // A warp copies whole half-tiles (32 rows, this CTA's bytes of each), so address resolution is done once per
        // half-tile and no two warps ever synchronise.  Because every use of a slot is made by the same warp, the slot's
        // barrier is at most one phase ahead of it, which the parity wait relies on.
        const int g = warp - 1;
        const int total_half = n_my * n_half;                  // half-tiles of all tokens of this cluster, counted globally
        const int g_sub = lane & 7, g_rr = lane >> 3;          // this lane copies piece g_sub of the 128-byte groups of rows 4q + g_rr
        const uint32_t g_sw0 = static_cast<uint32_t>((g_sub ^ g_rr) << 4), g_sw1 = static_cast<uint32_t>((g_sub ^ (4 + g_rr)) << 4);   // even / odd q
        const int64_t seg_off = 512 * static_cast<int64_t>(c); // first owned byte of a row
        bool ok = true;

        int64_t tbl_nxt = 0, tbl_n_nxt = p.n_logical_pages;     // page table (start, length) of the query row the last load_raw was for
        auto load_raw = [&](int gh) -> int {                   // lane r owns row r of global half-tile gh
            if (gh >= total_half) return -1;
            const int it = gh / n_half;
            const int slot = (gh - it * n_half) * LP_HALF + lane;
            const int64_t t_row = cid + it * n_clusters;
            if (p.table_offsets != nullptr) {                  // every query row has a page table of its own (a batch of sessions)
                tbl_nxt = __ldg(p.table_offsets + t_row);
                tbl_n_nxt = __ldg(p.table_offsets + t_row + 1) - tbl_nxt;
                if (tbl_nxt < 0) tbl_n_nxt = 0;                // a table that starts before the array: its tokens are reported and skipped
            }
            return slot < p.k ? __ldg(p.idx + t_row * p.k + slot) : -1;
        };
        auto resolve = [&](int s_tok, int64_t tbl, int64_t tbl_n, bool& valid) -> const unsigned char* {   // first owned byte of the row of token s_tok
            const unsigned char* ptr = reinterpret_cast<const unsigned char*>(p.pool) + seg_off;
            valid = false;
            if (s_tok >= 0) {
                const int64_t lp = p.page_shift >= 0 ? (s_tok >> p.page_shift) : (s_tok / p.page_size);
                const int within = p.page_shift >= 0 ? (s_tok & (p.page_size - 1)) : (s_tok % p.page_size);
                const int32_t phys = lp < tbl_n ? __ldg(p.page_table + tbl + lp) : -1;
                if (phys < 0) {     // beyond the page table, or a negative physical page id in it
                    report(p.dev_status, JANUS_DEV_INDEX_OUT_OF_RANGE);
                } else {
                    ptr += (static_cast<int64_t>(phys) * p.page_stride + static_cast<int64_t>(within) * p.tok_stride) * 2;
                    valid = true;
                }
            }
            return ptr;
        };
        // rows are resolved one half-tile ahead and indices fetched two ahead, so neither load is waited for in the loop
        auto next_owned = [&](int gh) -> int {                 // the next half-tile after gh whose ring slot this warp owns
            do { ++gh; } while ((gh & (LP_SLOTS - 1)) % LP_GATHER_WARPS != g);
            return gh;
        };
        bool valid_cur, valid_nxt = false;
        const int raw0 = load_raw(g);
        const unsigned char* row_ptr = resolve(raw0, tbl_nxt, tbl_n_nxt, valid_cur);
        const unsigned char* row_nxt = row_ptr;
        int hi_nxt = next_owned(g);
        int raw_nxt = load_raw(hi_nxt);
        for (int hi = g; hi < total_half; hi = hi_nxt, hi_nxt = next_owned(hi_nxt)) {
            const int buf = (hi >> 1) % LP_BUFS, hf = hi & 1;
            const bool s_ok = valid_cur;
            const uint32_t valid_mask = __ballot_sync(0xffffffffu, s_ok);
            // the tile buffer must have been released by the P.V three tiles back
            ok = (mbar_wait(smem_u32(&sh->k_empty[buf]), (static_cast<uint32_t>((hi >> 1) / LP_BUFS) & 1u) ^ 1u));
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (lane == 0) sh->vmask[2 * buf + hf] = valid_mask;
            const uint32_t stage_base = smem_u32(k_smem + buf * LP_TILE_BYTES + hf * LP_HALF * 128);
            // One instruction copies 128 contiguous bytes (8 lanes x 16, one whole line) of each of 4 rows, so a row pointer is
            // fetched from its owner lane once per 4 rows and every copy is a single instruction with immediate offsets: the
            // 128-byte group a of the owned bytes is row r of atom a, its 16-byte pieces at positions piece ^ (r % 8).
            // (Half lines of 8 rows per instruction, the same number of instructions, were 2.4 % slower: the copies are
            // bound by the rate at which the load/store unit takes these instructions, about 28 cycles each.)
            const uint32_t lo = static_cast<uint32_t>(reinterpret_cast<uint64_t>(row_ptr)), hi32 = static_cast<uint32_t>(reinterpret_cast<uint64_t>(row_ptr) >> 32);
#pragma unroll
            for (int q = 0; q < LP_HALF / 4; ++q) {
                const int r = 4 * q + g_rr;
                const uint64_t pr = (static_cast<uint64_t>(__shfl_sync(0xffffffffu, hi32, r)) << 32) | __shfl_sync(0xffffffffu, lo, r);
                const unsigned char* src = reinterpret_cast<const unsigned char*>(pr) + g_sub * 16;
                const uint32_t bytes = ((valid_mask >> r) & 1u) ? 16u : 0u;
                const uint32_t d = stage_base + static_cast<uint32_t>(r * 128) + ((q & 1) ? g_sw1 : g_sw0);
#pragma unroll
                for (int a = 0; a < 4; ++a) cp_async16(d + a * LP_K_ATOM_BYTES, src + a * 128, bytes);
                if (c == 1u) cp_async16(d + 4 * LP_K_ATOM_BYTES, src + 512, bytes);
            }
            cp_async_commit();
            row_nxt = resolve(raw_nxt, tbl_nxt, tbl_n_nxt, valid_nxt);   // page-table load overlaps the copies in flight
            raw_nxt = load_raw(next_owned(hi_nxt));
            cp_async_wait<0>();
            fence_proxy_async();              // publish the landed rows to the MMA (async) proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->k_full[buf]));
            row_ptr = row_nxt;
            valid_cur = valid_nxt;
        }
        if (!ok && lane == 0) report(p.dev_status, JANUS_DEV_WAIT_TIMEOUT);
    } else if (warp < LP_SMAX_WARP0) {
        // ================================================================== exchange: partial logits -> the peer's buffer
        const int quad = warp & 3;                         // warps 4..7 -> TMEM lane quadrants 0..3
        const int h = quad * 32 + lane;
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
        const uint32_t peer_xbuf = mapa_shared(smem_u32(xbuf), peer);
        const uint32_t peer_xfull = mapa_shared(smem_u32(&sh->x_full[0]), peer);
        // this CTA's first 256 query dims of head h of the cluster's token `it` -> tensor memory, two bf16 per 32-bit column
        auto load_q = [&](int it) {
            const uint4* src = reinterpret_cast<const uint4*>(p.q + (static_cast<int64_t>(cid + it * n_clusters) * LP_HEADS + h) * LP_DQK + 256 * c);
#pragma unroll
            for (int a = 0; a < LP_Q_TMEM_ATOMS; ++a) {
                uint32_t r[32];
#pragma unroll
                for (int v = 0; v < 8; ++v) {
                    const uint4 u = __ldg(src + a * 8 + v);
                    r[4 * v + 0] = u.x; r[4 * v + 1] = u.y; r[4 * v + 2] = u.z; r[4 * v + 3] = u.w;
                }
                tmem_st32_wait(lane_addr + LP_COL_Q + a * 32, r);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->qt_full));
        };
        if (n_my > 0) load_q(0);
        bool ok = true;
        int gi = 0;
        for (int it = 0; it < n_my && ok; ++it) {
        if (it + 1 < n_my) {
            // the next token's queries are wanted the moment this token's last logit tile is done: have them in L2 by then
            const unsigned char* nq = reinterpret_cast<const unsigned char*>(p.q + (static_cast<int64_t>(cid + (it + 1) * n_clusters) * LP_HEADS + h) * LP_DQK + 256 * c);
#pragma unroll
            for (int a = 0; a < 4; ++a) prefetch_l2(nq + a * 128);
            prefetch_l2(nq + 496);
        }
        for (int i = 0; i < n_tiles; ++i, ++gi) {
            const int b = gi & 1;
            const uint32_t ph = static_cast<uint32_t>(gi >> 1) & 1u;
            ok = mbar_wait(smem_u32(&sh->s_full[b]), ph);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t s_addr = lane_addr + LP_COL_S + b * LP_TILE;
            uint32_t r0[32], r1[32];
            tmem_ld32_issue(s_addr, r0);
            tmem_ld32_issue(s_addr + 32, r1);
            tmem_ld_wait(r0);
            tmem_ld_wait(r1);
            // the partial logits are in registers: the logit buffer may take the tile after next
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->s_free[b]));
            // the peer must have read what this CTA sent two tiles ago into the same exchange buffer
            ok = mbar_wait(smem_u32(&sh->x_empty[b]), ph ^ 1u);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            // The partial logits travel as fp16 (11 significant bits: the same order of rounding as P, which is bf16), which
            // halves the traffic between the two SMs, the slowest link of the tile loop.  [key/8][head][8 keys]: a warp
            // stores 512 contiguous bytes per instruction; every 16 bytes are counted on the peer's barrier when they land.
            const uint32_t dst = peer_xbuf + static_cast<uint32_t>(b * LP_XBUF_BYTES + h * 16);
            const uint32_t bar = peer_xfull + static_cast<uint32_t>(b * 8);
#pragma unroll
            for (int j8 = 0; j8 < 4; ++j8)
                st_async_cluster_f32x4(dst + static_cast<uint32_t>(j8 * LP_HEADS * 16),
                                       __uint_as_float(lp_pack_f16x2(__uint_as_float(r0[8 * j8]), __uint_as_float(r0[8 * j8 + 1]))),
                                       __uint_as_float(lp_pack_f16x2(__uint_as_float(r0[8 * j8 + 2]), __uint_as_float(r0[8 * j8 + 3]))),
                                       __uint_as_float(lp_pack_f16x2(__uint_as_float(r0[8 * j8 + 4]), __uint_as_float(r0[8 * j8 + 5]))),
                                       __uint_as_float(lp_pack_f16x2(__uint_as_float(r0[8 * j8 + 6]), __uint_as_float(r0[8 * j8 + 7]))), bar);
#pragma unroll
            for (int j8 = 0; j8 < 4; ++j8)
                st_async_cluster_f32x4(dst + static_cast<uint32_t>((4 + j8) * LP_HEADS * 16),
                                       __uint_as_float(lp_pack_f16x2(__uint_as_float(r1[8 * j8]), __uint_as_float(r1[8 * j8 + 1]))),
                                       __uint_as_float(lp_pack_f16x2(__uint_as_float(r1[8 * j8 + 2]), __uint_as_float(r1[8 * j8 + 3]))),
                                       __uint_as_float(lp_pack_f16x2(__uint_as_float(r1[8 * j8 + 4]), __uint_as_float(r1[8 * j8 + 5]))),
                                       __uint_as_float(lp_pack_f16x2(__uint_as_float(r1[8 * j8 + 6]), __uint_as_float(r1[8 * j8 + 7]))), bar);
        }
            // the token's last logit tile is complete, so nothing reads its queries any more: bring in the next token's
            if (ok && it + 1 < n_my) load_q(it + 1);
        }
        if (!ok && lane == 0) report(p.dev_status, JANUS_DEV_WAIT_TIMEOUT);
    } else {
        // ================================================================== softmax + output: 4 warps, thread = head
        const int quad = warp & 3;
        const int h = quad * 32 + lane;
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
        const float neg_inf = __int_as_float(0xff800000);
        const bool out_al32 = (reinterpret_cast<uint64_t>(p.out) & 31u) == 0u;
        bool ok = true;
        const uint32_t peer_xempty = mapa_shared(smem_u32(&sh->x_empty[0]), peer);
        int gi = 0;                 // tiles done so far, over all tokens
        for (int it = 0; it < n_my && ok; ++it) {
        const int t = cid + it * n_clusters;
        float m_ref = neg_inf;      // reference maximum (scaled, log2 domain) the exponentials are taken against
        float l_sum = 0.f;
        for (int i = 0; i < n_tiles; ++i, ++gi) {
            const int b = gi & 1, buf = gi % LP_BUFS;
            const uint32_t ph_k = static_cast<uint32_t>(gi / LP_BUFS) & 1u, ph_s = static_cast<uint32_t>(gi >> 1) & 1u;
            // this CTA's exchange barrier for the tile: expect the peer's 32 KB of partial logits
            if (warp == LP_SMAX_WARP0 && lane == 0) mbar_expect_tx(smem_u32(&sh->x_full[b]), LP_XBUF_BYTES);
            // k_full is complete long before s_full; waiting on it as well makes the validity masks written by the gather
            // warps visible to this thread directly rather than through the MMA warp
            ok = mbar_wait(smem_u32(&sh->k_full[buf]), ph_k) && mbar_wait(smem_u32(&sh->s_full[b]), ph_s);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t s_addr = lane_addr + LP_COL_S + b * LP_TILE;
            float2 x[LP_TILE / 2];          // logits of keys 2j, 2j+1
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                uint32_t r[32];
                tmem_ld32_wait(s_addr + hf * 32, r);
#pragma unroll
                for (int j = 0; j < 16; ++j) x[hf * 16 + j] = make_float2(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
            }
            // the logits are in registers: the logit buffer may take the tile after next
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->s_free[b]));
            // the peer's partial logits of the same tile (bytes counted as they land: visible once the phase completes)
            ok = mbar_wait(smem_u32(&sh->x_full[b]), ph_s);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            float tile_max = neg_inf;
            {
                const uint4* xin = reinterpret_cast<const uint4*>(xbuf + b * LP_XBUF_BYTES) + h;
#pragma unroll
                for (int j8 = 0; j8 < LP_TILE / 8; ++j8) {
                    const uint4 pv = xin[j8 * LP_HEADS];
                    x[4 * j8 + 0] = fadd2(x[4 * j8 + 0], __half22float2(*reinterpret_cast<const __half2*>(&pv.x)));
                    x[4 * j8 + 1] = fadd2(x[4 * j8 + 1], __half22float2(*reinterpret_cast<const __half2*>(&pv.y)));
                    x[4 * j8 + 2] = fadd2(x[4 * j8 + 2], __half22float2(*reinterpret_cast<const __half2*>(&pv.z)));
                    x[4 * j8 + 3] = fadd2(x[4 * j8 + 3], __half22float2(*reinterpret_cast<const __half2*>(&pv.w)));
                }
                const uint32_t vm0 = sh->vmask[2 * buf], vm1 = sh->vmask[2 * buf + 1];
                if ((vm0 & vm1) != 0xffffffffu) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        x[j].x = ((vm0 >> (2 * j)) & 1u) ? x[j].x : neg_inf;
                        x[j].y = ((vm0 >> (2 * j + 1)) & 1u) ? x[j].y : neg_inf;
                        x[16 + j].x = ((vm1 >> (2 * j)) & 1u) ? x[16 + j].x : neg_inf;
                        x[16 + j].y = ((vm1 >> (2 * j + 1)) & 1u) ? x[16 + j].y : neg_inf;
                    }
                }
                float mx[4] = {neg_inf, neg_inf, neg_inf, neg_inf};
#pragma unroll
                for (int j = 0; j < LP_TILE / 2; j += 4) {
                    mx[0] = fmax3(mx[0], x[j].x, x[j].y); mx[1] = fmax3(mx[1], x[j + 1].x, x[j + 1].y);
                    mx[2] = fmax3(mx[2], x[j + 2].x, x[j + 2].y); mx[3] = fmax3(mx[3], x[j + 3].x, x[j + 3].y);
                }
                tile_max = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
            }
            // the exchange buffer has been read: the peer may send the tile after next into it
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster_relaxed(peer_xempty + static_cast<uint32_t>(b * 8));
            tile_max *= p.scale_log2e;                       // softmax_scale > 0
            // move the reference maximum only when this tile exceeds it by more than 2^8 (or on first use)
            float corr = 1.f;
            bool moved = false;
            if (tile_max > m_ref + 8.f) {
                moved = (l_sum > 0.f);
                corr = moved ? lp_exp2(m_ref - tile_max) : 1.f;
                l_sum *= corr;
                m_ref = tile_max;
            }
            if (__any_sync(0xffffffffu, moved) && i > 0) {
                // rescale O in tensor memory: the previous tile's P.V must have completed first
                ok = mbar_wait(smem_u32(&sh->k_empty[(gi - 1) % LP_BUFS]), static_cast<uint32_t>((gi - 1) / LP_BUFS) & 1u);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
#pragma unroll 1
                for (int cc = 0; cc < LP_DVH / 32; ++cc) {
                    uint32_t o[32];
                    tmem_ld32_wait(lane_addr + LP_COL_O + cc * 32, o);
#pragma unroll
                    for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * corr);
                    tmem_st32_wait(lane_addr + LP_COL_O + cc * 32, o);
                }
            }
            const float neg_m = (m_ref == neg_inf) ? 0.f : -m_ref;
            // P is rounded to bf16 (one pack instruction per pair); the row sum adds the very same rounded values, so the
            // normalisation stays consistent and the log-sum-exp is not biased
            uint32_t pk[32];
            float2 ts[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
            const float2 sc2 = make_float2(p.scale_log2e, p.scale_log2e), nm2 = make_float2(neg_m, neg_m);
#pragma unroll
            for (int j = 0; j < LP_TILE / 2; ++j) {
                const float2 e = ffma2(x[j], sc2, nm2);
                pk[j] = lp_pack_bf16x2(lp_exp2(e.x), lp_exp2(e.y));       // low half = bf16(p of key 2j), high half = bf16(p of key 2j+1)
                ts[j & 3] = fadd2(ts[j & 3], make_float2(__uint_as_float(pk[j] << 16), __uint_as_float(pk[j] & 0xffff0000u)));
            }
            const float2 t01 = fadd2(ts[0], ts[1]), t23 = fadd2(ts[2], ts[3]);
            const float2 t4 = fadd2(t01, t23);
            const float tile_sum = t4.x + t4.y;
            l_sum += tile_sum;
            // P has one buffer: the previous tile's P.V must have completed
            if (gi > 0) {
                ok = mbar_wait(smem_u32(&sh->k_empty[(gi - 1) % LP_BUFS]), static_cast<uint32_t>((gi - 1) / LP_BUFS) & 1u);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
            }
            tmem_st32_wait(lane_addr + LP_COL_P, pk);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->p_full));
        }
        if (!ok) break;
        // ---- output: wait for the token's last P.V, normalise, round to bf16.  The next token's first P is produced by
        // these same warps afterwards, so its P.V cannot overwrite O before O has been read here.
        ok = mbar_wait(smem_u32(&sh->k_empty[(gi - 1) % LP_BUFS]), static_cast<uint32_t>((gi - 1) / LP_BUFS) & 1u);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        const float inv = l_sum > 0.f ? 1.f / l_sum : 0.f;
        const bool have_o = __any_sync(0xffffffffu, l_sum > 0.f);   // some P.V of this token has written O
        uint16_t* orow = p.out + (static_cast<int64_t>(t) * LP_HEADS + h) * LP_DV + c * LP_DVH;
#pragma unroll 1
        for (int cc = 0; cc < LP_DVH / 32; ++cc) {
            uint32_t o[32];
            if (have_o) {
                tmem_ld32_wait(lane_addr + LP_COL_O + cc * 32, o);
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) o[j] = 0u;
            }
            uint32_t w[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) w[j] = lp_pack_bf16x2(__uint_as_float(o[2 * j]) * inv, __uint_as_float(o[2 * j + 1]) * inv);
            if (out_al32) {      // whole 32-byte sectors per thread: half the store instructions and transactions
                st_global_v8(orow + cc * 32, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
                st_global_v8(orow + cc * 32 + 16, w[8], w[9], w[10], w[11], w[12], w[13], w[14], w[15]);
            } else {
                uint4* dst = reinterpret_cast<uint4*>(orow + cc * 32);
#pragma unroll
                for (int v = 0; v < 4; ++v) dst[v] = make_uint4(w[4 * v], w[4 * v + 1], w[4 * v + 2], w[4 * v + 3]);
            }
        }
        if (p.lse != nullptr && c == 0u)
            p.lse[static_cast<int64_t>(t) * LP_HEADS + h] = l_sum > 0.f ? (m_ref + log2f(l_sum)) * 0.6931471805599453f : neg_inf;
        }
        if (!ok && lane == 0) report(p.dev_status, JANUS_DEV_WAIT_TIMEOUT);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
    cluster_sync_all();   // neither CTA leaves while the other may still write into its shared memory or arrive on its barriers
}

bool sparse_attn_latent_tc_supported(int M, int H_q, int d_qk, const void* k_pool, const void* v_pool, int64_t page_stride,
                                     int64_t tok_stride, int n_kv_heads, int d_v, int k) {
    if (H_q != LP_HEADS || d_qk != LP_DQK || d_v != LP_DV || n_kv_heads != 1 || k_pool != v_pool) return false;
    if ((page_stride % 8) != 0 || (tok_stride % 8) != 0 || tok_stride < LP_DQK) return false;
    if (M > (1 << 30) / LP_HEADS || k <= 0) return false;
    return true;
}

int launch_sparse_attn_latent_tc(const void* q, int M, const void* pool, int64_t page_stride, int64_t tok_stride, const int32_t* idx, int k,
                                 int page_size, const int32_t* page_table, int64_t n_logical_pages, const int64_t* table_offsets,
                                 float softmax_scale, void* out, float* lse, int32_t* dev_status, cudaStream_t stream) {
    LpParams p;
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
    p.table_offsets = table_offsets;
    p.scale_log2e = softmax_scale * 1.4426950408889634f;
    p.out = static_cast<uint16_t*>(out);
    p.lse = lse;
    p.M = M;
    p.dev_status = dev_status;
    CUtensorMap tq;
    if (!make_tmap_2d_sw128(&tq, q, 2, static_cast<uint64_t>(M) * LP_HEADS, LP_DQK, static_cast<uint64_t>(LP_DQK) * 2, LP_HEADS, 64))
        return JANUS_ERR_CUDA;
    const size_t smem = LP_BUFS * LP_TILE_BYTES + 2 * LP_XBUF_BYTES + LP_QS_BYTES + sizeof(LpShared) + 16;
    static_assert(LP_BUFS * LP_TILE_BYTES + 2 * LP_XBUF_BYTES + LP_QS_BYTES + sizeof(LpShared) + 16 <= 227 * 1024, "shared memory");
    JANUS_CUDA_CHECK(cudaFuncSetAttribute(sparse_attn_latent_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    // persistent launch: as many 2-CTA clusters as the device keeps resident at once (one CTA per SM), each looping over tokens
    static int resident_clusters[64] = {};
    int dev = 0;
    JANUS_CUDA_CHECK(cudaGetDevice(&dev));
    int n_clusters = (dev >= 0 && dev < 64) ? resident_clusters[dev] : 0;
    if (n_clusters <= 0) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * 148);
        cfg.blockDim = dim3(LP_THREADS);
        cfg.dynamicSmemBytes = smem;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2;
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        if (cudaOccupancyMaxActiveClusters(&n_clusters, sparse_attn_latent_pair_kernel, &cfg) != cudaSuccess || n_clusters <= 0) {
            (void)cudaGetLastError();
            int sms = 0;
            JANUS_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
            n_clusters = sms / 2;
        }
        if (n_clusters <= 0) n_clusters = 1;
        if (dev >= 0 && dev < 64) resident_clusters[dev] = n_clusters;
    }
    if (n_clusters > M) n_clusters = M;
    sparse_attn_latent_pair_kernel<<<2 * n_clusters, LP_THREADS, smem, stream>>>(tq, p);   // clusters of 2 CTAs (compile-time cluster dims)
    JANUS_CUDA_CHECK(cudaGetLastError());
    return JANUS_OK;
}

}  // namespace janus
