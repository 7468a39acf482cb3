// Tensor-core indexer (Eq. 1, Sec. 2.2, scoring part) for sm_100a:
//     scores[t,s] = k_scale[s] * sum_h (w[t,h]*q_scale[h]) * relu(<q[t,h,:], k[s,:]>) + row_bias[t]*col_bias[s]
//
// Mapping.  The dense contraction is K . Q^T with a reduction depth of only D_I, followed by a ReLU and a
// weighted sum over heads for every accumulator.  Keys go on the MMA M axis (128 keys -> the 128 TMEM lanes)
// and (token, head) pairs on the N axis (256 TMEM columns = 256/H_I tokens x H_I heads), so that after a
// tcgen05.ld every epilogue thread owns one key, holds all heads of a token in its own registers, and reduces
// over heads with no cross-lane traffic; a warp's 32 keys are 32 consecutive floats of one score row.
//
// One CTA keeps NQ query sub-tiles (NQ*256 (token,head) rows, 128 KB) stationary in shared memory and streams
// 128-key tiles past them through a TMA ring; each key tile feeds NQ MMAs (128 x 256 x D_I), whose fp32
// accumulators alternate between the two 256-column halves of tensor memory, so the epilogue of one
// overlaps the MMA of the next.  Warp roles: warp 0 issues TMA, warp 1 issues MMA (one thread each) and owns
// the TMEM allocation, the other warps are two epilogue groups (one per TMEM half).  In score-matrix mode a group is
// eight warps (two per TMEM lane quadrant, each reducing half of the slot's columns): with four epilogue warps per
// scheduler one warp's wait for its tensor-memory load or its weights is covered by the others.  Candidate mode and
// the ragged decode mode keep four warps per group.
// Every wait is bounded; on a timeout the CTA reports JANUS_DEV_WAIT_TIMEOUT and winds down normally.
#include "janus_common.cuh"
#include "sm100_ptx.cuh"

namespace janus {

using namespace ptx;

constexpr int TC_KEYS = 128;        // keys per tile = MMA M
constexpr int TC_N = 256;           // (token, head) rows per MMA = MMA N
constexpr int TC_THREADS = 320;     // candidate mode: 1 TMA warp + 1 MMA warp + 8 epilogue warps
constexpr int TC_THREADS16 = 576;   // score-matrix mode: 16 epilogue warps, two per TMEM lane quadrant and slot, each takes half the columns
constexpr int TC_THREADS_RAGGED = 192;   // ragged mode: one epilogue group (4 warps), so that four CTAs fit an SM
constexpr int TC_SMEM_BUDGET = 227 * 1024;
constexpr int TC_MAX_STAGES = 6;

struct TcParams {
    const float* w;
    const float* q_scale;
    int64_t q_scale_stride_tok;
    const float* k_scale;
    const float* row_bias;
    const float* col_bias;
    float* scores;
    int64_t ld;
    int64_t n_keys;
    int64_t q_pos0;
    int M, H, causal;
    int n_tiles;          // ceil(n_keys / 128)
    int tiles_per_cta;    // key tiles per CTA (grid.x chunks)
    int nq;               // query sub-tiles per CTA
    int atoms;            // 128-byte swizzle atoms per row (row bytes / 128)
    int stages;           // key ring depth
    int32_t* dev_status;
};

// Candidate mode (fused indexer + top-k): instead of storing scores, every visible score >= thr[t] is appended to row t's
// candidate list; `scores` is unused.  A kernel parameter of its own: the score-matrix kernel's code does not depend on it.
struct TcCandParams {
    const float* thr;     // [M] per-row thresholds
    int32_t* cand_cnt;    // [M] candidates appended so far (may exceed cand_cap: only the first cand_cap are stored)
    int2* cand;           // [M, cand_cap] (score bits, key index)
    int cand_cap;
    // ragged batch mode (decode over many sessions): query row b scores the keys key_offsets[b] .. key_offsets[b+1] of one
    // concatenated key array, no causal mask, and its scores go to scores[key_offsets[b] + s]
    const int64_t* key_offsets;
    // ragged batch mode only: keys are FP4 E2M1, two per byte; the TMA expands 16 of them into the first 8 bytes of every
    // 16-byte shared-memory chunk, which is the layout the f8f6f4 MMA expects for 4-bit operands
    int k_fp4;
};

// Candidate mode stages appends in shared memory: each epilogue warp owns, for each of its (at most TC_CAND_TPW) tokens,
// TC_CAND_SLOTS (score, key) slots, and moves a full set to the row's global list with one counter update.
constexpr int TC_CAND_TPW = 8;
constexpr int TC_CAND_SLOTS = 32;
constexpr int TC_CAND_STAGE_BYTES = 8 * TC_CAND_TPW * TC_CAND_SLOTS * static_cast<int>(sizeof(int2));

struct TcBarriers {
    uint64_t q_full;
    uint64_t k_full[TC_MAX_STAGES];
    uint64_t k_empty[TC_MAX_STAGES];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t mma_drain;       // abort path only: every MMA issued so far has completed
    uint32_t tmem_base;
    int aborted;
};

// One 32-column chunk of accumulators: 2 * ReLU, half weight, reduce over heads; a token's sum is complete every H columns.
// Pairs of columns go through packed fp32 FMAs into up to four independent accumulator pairs, so the reduction is
// neither one long dependent chain nor one instruction per element.
template <int H, class Store>
__device__ __forceinline__ void reduce_chunk(const uint32_t (&r)[32], const float* __restrict__ wchunk, int col0, float2 (&acc)[4], Store&& store) {
    constexpr int NACC = (H / 2 < 4) ? H / 2 : 4;
#pragma unroll
    for (int i4 = 0; i4 < 8; ++i4) {
        const float4 wv = *reinterpret_cast<const float4*>(wchunk + 4 * i4);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int i = 4 * i4 + 2 * j;                      // first column of the pair inside the chunk
            const int col = col0 + i;
            const float2 w2 = j == 0 ? make_float2(wv.x, wv.y) : make_float2(wv.z, wv.w);
            // 2 * max(x, 0) = x + |x|, exactly: an add (full-rate FMA pipe, |x| is an operand modifier) instead of a max (the
            // half-rate pipe, which 256 of them per thread and tile would saturate before the tensor pipe); the weights
            // carry the factor 1/2
            const float xa = __uint_as_float(r[i]), xb = __uint_as_float(r[i + 1]);
            const float2 x2 = make_float2(xa + fabsf(xa), xb + fabsf(xb));
            float2& a = acc[(col / 2) % NACC];
            a = ffma2(w2, x2, a);
            if (((col + 2) % H) == 0) {
                float v = 0.f;
#pragma unroll
                for (int q = 0; q < NACC; ++q) {
                    v += acc[q].x + acc[q].y;
                    acc[q] = make_float2(0.f, 0.f);
                }
                store(col / H, v);
            }
        }
    }
}

template <int H, bool FP8, bool CAND, bool RAGGED>
__global__ void __launch_bounds__(RAGGED ? TC_THREADS_RAGGED : ((CAND) ? TC_THREADS : TC_THREADS16), RAGGED ? 4 : 1)
indexer_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k, const TcParams p, const TcCandParams cp) {
    extern __shared__ __align__(1024) unsigned char smem[];
    constexpr int TPS = TC_N / H;                      // tokens per query sub-tile
    const int atoms = p.atoms, nq = p.nq, stages = p.stages;
    // ragged mode keeps only what one query row needs (H rows of Q, H accumulator columns per slot), so that two CTAs fit an SM
    constexpr int QROWS = RAGGED ? H : TC_N;           // rows of a query sub-tile in shared memory
    constexpr int SLOT_COLS = RAGGED ? H : TC_N;       // TMEM columns of one accumulator slot
    constexpr int TMEM_COLS = RAGGED ? 2 * H : 512;
    static_assert(TMEM_COLS >= 32 && (TMEM_COLS & (TMEM_COLS - 1)) == 0, "TMEM allocations are powers of two of at least 32 columns");
    const int q_sub_bytes = atoms * QROWS * 128;       // one query sub-tile
    const int k_stage_bytes = atoms * TC_KEYS * 128;   // one key tile
    unsigned char* q_smem = smem;
    unsigned char* k_smem = smem + nq * q_sub_bytes;
    float* ws = reinterpret_cast<float*>(k_smem + stages * k_stage_bytes);   // [nq*256] w * q_scale, column order
    float* rbs = ws + nq * TC_N;                                             // [nq*TPS] row_bias of this CTA's tokens
    float* thrs = rbs + nq * TPS;                                            // [nq*TPS] candidate thresholds of this CTA's tokens
    int2* cstage = reinterpret_cast<int2*>(thrs + nq * TPS);                 // candidate staging (candidate mode only)
    TcBarriers* bars = reinterpret_cast<TcBarriers*>(reinterpret_cast<unsigned char*>(cstage) + (CAND ? TC_CAND_STAGE_BYTES : 0));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tpc = nq * TPS;                                   // tokens per CTA
    int t0 = blockIdx.y * tpc;
    int64_t key_base = 0, key_count = p.n_keys;                 // this CTA's keys: rows key_base .. key_base + key_count of k_idx
    int n_tiles = p.n_tiles;
    if constexpr (RAGGED) {
        t0 = blockIdx.y;                                        // one query row per grid row; the sub-tile's other rows are not stored
        key_base = cp.key_offsets[blockIdx.y];
        key_count = cp.key_offsets[blockIdx.y + 1] - key_base;
        // the offsets come from device memory: a session that lies outside the key array (p.n_keys rows) is reported and cut
        // back to the part inside it, so that neither the per-key scale / bias reads nor the score writes leave their arrays
        if (key_base < 0 || key_count < 0 || key_base > p.n_keys || key_count > p.n_keys - key_base) {
            if (threadIdx.x == 0) report(p.dev_status, JANUS_DEV_INDEX_OUT_OF_RANGE);
            if (key_base < 0 || key_base > p.n_keys) { key_base = 0; key_count = 0; }
            if (key_count < 0) key_count = 0;
            if (key_count > p.n_keys - key_base) key_count = p.n_keys - key_base;
        }
        n_tiles = static_cast<int>((key_count + TC_KEYS - 1) / TC_KEYS);
    }
    const int t_hi = min(p.M, t0 + tpc) - 1;                    // last real token of this CTA
    const int tile_begin = blockIdx.x * p.tiles_per_cta;
    const int tile_end = min(n_tiles, tile_begin + p.tiles_per_cta);
    // key tiles with at least one visible (token, key) pair come first
    int vis_end = tile_end;
    if (p.causal) {
        const int64_t last_visible_tile = (p.q_pos0 + t_hi) / TC_KEYS;
        vis_end = last_visible_tile + 1 < tile_end ? static_cast<int>(last_visible_tile + 1) : tile_end;
        if (vis_end < tile_begin) vis_end = tile_begin;
    }
    const int n_vis = vis_end - tile_begin;

    if ((smem_u32(smem) & 1023u) != 0u) {   // swizzled tiles need 1024-byte alignment
        if (threadIdx.x == 0) report(p.dev_status, JANUS_DEV_WAIT_TIMEOUT);
        return;
    }
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars->q_full), 1);
        for (int s = 0; s < stages; ++s) { mbar_init(smem_u32(&bars->k_full[s]), 1); mbar_init(smem_u32(&bars->k_empty[s]), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&bars->tmem_full[s]), 1); mbar_init(smem_u32(&bars->tmem_empty[s]), (!CAND && !RAGGED) ? 8 : 4); }
        mbar_init(smem_u32(&bars->mma_drain), 1);
        // an earlier CTA of this launch gave up on a wait: this one starts no work on a broken pipeline.  One thread reads the
        // status word and the whole CTA follows that one reading (a second reading could differ and split the roles).
        bars->aborted = (p.dev_status != nullptr && *reinterpret_cast<volatile int32_t*>(p.dev_status) == JANUS_DEV_WAIT_TIMEOUT) ? 1 : 0;
        fence_mbar_init();
        prefetch_tensormap(&tmap_q);
        prefetch_tensormap(&tmap_k);
    }
    if (warp == 1 && n_vis > 0) {
        tmem_alloc(smem_u32(&bars->tmem_base), TMEM_COLS);
        tmem_relinquish();
    }
    // per-column weights (w * q_scale) and per-token bias factors of this CTA
    constexpr int NTHREADS = RAGGED ? TC_THREADS_RAGGED : (CAND ? TC_THREADS : TC_THREADS16);
    for (int n = threadIdx.x; n < nq * TC_N; n += NTHREADS) {
        const int t = t0 + n / H, h = n % H;
        float v = 0.f;
        if (t < p.M) {
            v = p.w[static_cast<int64_t>(t) * H + h];
            if (FP8) v *= p.q_scale[static_cast<int64_t>(t) * p.q_scale_stride_tok + h];
        }
        ws[n] = 0.5f * v;      // the epilogue forms 2 * relu
    }
    for (int n = threadIdx.x; n < tpc; n += NTHREADS) {
        rbs[n] = (p.row_bias != nullptr && t0 + n < p.M) ? p.row_bias[t0 + n] : 0.f;
        if constexpr (CAND) thrs[n] = t0 + n < p.M ? cp.thr[t0 + n] : 0.f;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;
    volatile int* aborted = &bars->aborted;
    const bool run = *aborted == 0;       // read once, after the barrier: the same value in every thread

    if (!run) {
        // nothing to do: tensor memory goes back below
    } else if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0 && n_vis > 0) {
            const int atom_elems = FP8 ? 128 : 64;
            const uint32_t qf = smem_u32(&bars->q_full);
            mbar_expect_tx(qf, static_cast<uint32_t>(nq * q_sub_bytes));
            for (int j = 0; j < nq; ++j)
                for (int a = 0; a < atoms; ++a)
                    tma_load_2d(smem_u32(q_smem + j * q_sub_bytes + a * QROWS * 128), &tmap_q, a * atom_elems, (t0 + j * TPS) * H, qf);
            int issued = 0;
            int s = 0;                 // ring stage and its phase bit, advanced per tile (a division per tile costs a thread
            uint32_t ph = 0;           // that issues everything on its own more than the copy it starts)
            for (int it = 0; it < n_vis; ++it, s = (s + 1 == stages ? 0 : s + 1), ph ^= (s == 0 ? 1u : 0u)) {
                if (!mbar_wait(smem_u32(&bars->k_empty[s]), ph ^ 1u) || *aborted) { *aborted = 1; report(p.dev_status, JANUS_DEV_WAIT_TIMEOUT); break; }
                const uint32_t kf = smem_u32(&bars->k_full[s]);
                // packed 4-bit keys: the copy is counted in the bytes it reads (half of what it occupies in shared memory)
                mbar_expect_tx(kf, static_cast<uint32_t>((FP8 && cp.k_fp4) ? k_stage_bytes / 2 : k_stage_bytes));
                for (int a = 0; a < atoms; ++a)
                    tma_load_2d(smem_u32(k_smem + s * k_stage_bytes + a * TC_KEYS * 128), &tmap_k, a * atom_elems,
                                static_cast<int>(key_base) + (tile_begin + it) * TC_KEYS, kf);
                issued = it + 1;
            }
            if (*aborted) {   // let the copies already in flight land before the CTA leaves
                mbar_wait(qf, 0);
                for (int it = max(0, issued - stages); it < issued; ++it)
                    mbar_wait(smem_u32(&bars->k_full[it % stages]), static_cast<uint32_t>(it / stages) & 1u);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0 && n_vis > 0) {
            // ragged: only the first query row's heads (N = H); the keys (the A operand) may be E2M1 (format 5) against E4M3 queries
            const uint32_t idesc = umma_idesc(FP8 ? 0u : 1u, TC_KEYS, RAGGED ? H : TC_N) | ((FP8 && cp.k_fp4) ? (5u << 7) : 0u);
            bool ok = mbar_wait(smem_u32(&bars->q_full), 0);
            uint32_t cnt = 0;
            // descriptors of the first key stage / first query sub-tile; every other operand is a constant number of 16-byte
            // units further on, so stepping through the tiles is one 64-bit add
            const uint64_t kdesc0 = umma_desc_sw128(smem_u32(k_smem)), qdesc0 = umma_desc_sw128(smem_u32(q_smem));
            int s = 0;
            uint32_t ph = 0;
            for (int it = 0; it < n_vis && ok; ++it, s = (s + 1 == stages ? 0 : s + 1), ph ^= (s == 0 ? 1u : 0u)) {
                ok = mbar_wait(smem_u32(&bars->k_full[s]), ph) && !*aborted;
                if (!ok) break;
                tc_fence_after();
                const uint64_t kdesc_s = kdesc0 + static_cast<uint64_t>((s * k_stage_bytes) >> 4);
                // ragged mode has one query sub-tile, so consecutive key tiles alternate between the two TMEM halves
                for (int j = 0; j < nq; ++j, ++cnt) {
                    const uint32_t slot = cnt & 1u, use = cnt >> 1;
                    ok = mbar_wait(smem_u32(&bars->tmem_empty[slot]), (use & 1u) ^ 1u) && !*aborted;
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + slot * SLOT_COLS;
                    uint32_t acc = 0;
                    for (int a = 0; a < atoms; ++a) {
                        const uint64_t ka = kdesc_s + static_cast<uint64_t>((a * TC_KEYS * 128) >> 4);
                        const uint64_t qa = qdesc0 + static_cast<uint64_t>((j * q_sub_bytes + a * QROWS * 128) >> 4);
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {   // 32 bytes of K per instruction (16 bf16 or 32 e4m3)
                            umma<FP8>(d_tmem, ka + 2 * ks, qa + 2 * ks, idesc, acc);
                            acc = 1;
                        }
                    }
                    umma_commit(smem_u32(&bars->tmem_full[slot]));
                }
                if (!ok) break;
                umma_commit(smem_u32(&bars->k_empty[s]));
            }
            if (!ok) {
                *aborted = 1;
                report(p.dev_status, JANUS_DEV_WAIT_TIMEOUT);
                // tensor memory is freed after the barrier below: the instructions already issued finish first
                umma_commit(smem_u32(&bars->mma_drain));
                mbar_wait(smem_u32(&bars->mma_drain), 0);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue: warps 2 and up
        constexpr int NCHUNK = RAGGED ? H / 32 : TC_N / 32;   // 32-column chunks to reduce (ragged: the first query row only)
        static_assert(NCHUNK % 2 == 0, "chunks are processed in pairs");
        constexpr bool W16 = !CAND && !RAGGED;
        const int e = ((warp - 2) >> 2) & 1;    // epilogue group = TMEM half it drains
        const int chalf = W16 ? (warp - 2) >> 3 : 0;   // 16 warps: which half of the slot's columns
        const int quad = warp & 3;              // TMEM lanes 32*quad .. 32*quad+31
        const float neg_inf = __int_as_float(0xff800000);
        bool ok = true;
        // candidate staging of this warp: lane i keeps the fill count of the warp's token slot i
        int2* my_stage = cstage + (warp - 2) * TC_CAND_TPW * TC_CAND_SLOTS;
        int cand_fill = 0;
        auto cand_flush = [&](int slot, int t, int c) {
            __syncwarp();                                        // the staged entries were written by other lanes
            int base = 0;
            if (lane == 0) base = atomicAdd(cp.cand_cnt + t, c);
            base = __shfl_sync(0xffffffffu, base, 0);
            if (lane < c && base + lane < cp.cand_cap) cp.cand[static_cast<int64_t>(t) * cp.cand_cap + base + lane] = my_stage[slot * TC_CAND_SLOTS + lane];
            __syncwarp();                                        // slots are free again
        };
        for (int it = 0; it < n_vis && ok; ++it) {
            const int64_t s_local = static_cast<int64_t>(tile_begin + it) * TC_KEYS + quad * 32 + lane;
            const bool key_ok = s_local < key_count;
            const int64_t s = key_base + s_local;               // row of k_idx (and of k_scale / col_bias; ragged: of scores)
            const float kscale = (FP8 && key_ok) ? p.k_scale[s] : 1.f;
            const float cb = (p.col_bias != nullptr && key_ok) ? p.col_bias[s] : 0.f;
            // score-matrix and candidate modes: group e drains the sub-tiles j = e, e+2, .. of every key tile (nq is even);
            // ragged mode (nq = 1, one group): key tile `it` sits in slot it % 2
            for (int j = RAGGED ? 0 : e; j < nq; j += 2) {
                const int slot = RAGGED ? (it & 1) : e;     // ragged: the one group takes both slots in turn
                const uint32_t use = static_cast<uint32_t>(it * nq + j) >> 1;
                ok = mbar_wait(smem_u32(&bars->tmem_full[slot]), use & 1u) && !*aborted;
                if (!ok) break;
                tc_fence_after();
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + slot * SLOT_COLS;
                const int tsub0 = t0 + j * TPS;
                float2 acc[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
                auto store = [&](int tt, float v) {
                    const int t = tsub0 + tt;
                    if constexpr (RAGGED) {
                        if (tt == 0 && j == 0 && key_ok) {
                            float out = v * kscale;
                            out = fmaf(rbs[0], cb, out);
                            p.scores[s] = out;
                        }
                    } else if constexpr (!CAND) {
                        if (t < p.M && key_ok) {
                            float out = v * kscale;
                            out = fmaf(rbs[j * TPS + tt], cb, out);
                            if (p.causal && s > p.q_pos0 + t) out = neg_inf;
                            p.scores[static_cast<int64_t>(t) * p.ld + s] = out;
                        }
                    } else {
                        // all 32 lanes (32 consecutive keys of one token) get here together
                        float out = v * kscale;
                        out = fmaf(rbs[j * TPS + tt], cb, out);
                        const bool masked = p.causal && s > p.q_pos0 + t;
                        const bool pass = t < p.M && key_ok && !masked && out >= thrs[j * TPS + tt];
                        const uint32_t m = __ballot_sync(0xffffffffu, pass);
                        if (m != 0u) {
                            const int slot = (j >> 1) * TPS + tt;
                            int c = __shfl_sync(0xffffffffu, cand_fill, slot);
                            const int n = __popc(m);
                            if (c + n > TC_CAND_SLOTS) { cand_flush(slot, t, c); c = 0; }
                            if (pass) my_stage[slot * TC_CAND_SLOTS + c + __popc(m & ((1u << lane) - 1u))] = make_int2(__float_as_int(out), static_cast<int>(s));
                            if (lane == slot) cand_fill = c + n;
                        }
                    }
                };
                // two register buffers: the load of the next 32 columns is in flight while this one is reduced
                uint32_t ra[32], rb[32];
                constexpr int CPW = W16 ? NCHUNK / 2 : NCHUNK;       // chunks per warp
                const int cbase = chalf * CPW;
                tmem_ld32_issue(taddr + cbase * 32, ra);
                if constexpr (W16) {
#pragma unroll
                for (int cc = 0; cc < CPW; cc += 2) {
                    const int c = cbase + cc;
                    tmem_ld_wait(ra);
                    tmem_ld32_issue(taddr + (c + 1) * 32, rb);
                    auto st = [&](int tt, float v) { store(tt + (cbase * 32) / H, v); };
                    reduce_chunk<H>(ra, ws + j * TC_N + c * 32, cc * 32, acc, st);
                    tmem_ld_wait(rb);
                    if (cc + 2 < CPW) {
                        tmem_ld32_issue(taddr + (c + 2) * 32, ra);
                    } else {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&bars->tmem_empty[slot]));
                    }
                    reduce_chunk<H>(rb, ws + j * TC_N + (c + 1) * 32, (cc + 1) * 32, acc, st);
                }
                } else
#pragma unroll
                for (int c = 0; c < NCHUNK; c += 2) {
                    tmem_ld_wait(ra);
                    tmem_ld32_issue(taddr + (c + 1) * 32, rb);
                    reduce_chunk<H>(ra, ws + j * TC_N + c * 32, c * 32, acc, store);
                    tmem_ld_wait(rb);
                    if (c + 2 < NCHUNK) {
                        tmem_ld32_issue(taddr + (c + 2) * 32, ra);
                    } else {
                        // every column of this TMEM half is in registers: hand it back before the last reduction
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&bars->tmem_empty[slot]));
                    }
                    reduce_chunk<H>(rb, ws + j * TC_N + (c + 1) * 32, (c + 1) * 32, acc, store);
                }
            }
        }
        if (!ok && lane == 0) { *aborted = 1; report(p.dev_status, JANUS_DEV_WAIT_TIMEOUT); }
        if (CAND) {
            for (int slot = 0; slot < TC_CAND_TPW; ++slot) {
                const int c = __shfl_sync(0xffffffffu, cand_fill, slot);
                if (c > 0) cand_flush(slot, t0 + (2 * (slot / TPS) + e) * TPS + slot % TPS, c);
            }
        }
        // key tiles no token of this CTA may see: -inf (score-matrix mode only)
        for (int tile = vis_end + e; !CAND && !RAGGED && chalf == 0 && tile < tile_end; tile += 2) {
            const int64_t s = static_cast<int64_t>(tile) * TC_KEYS + quad * 32 + lane;
            if (s < p.n_keys)
                for (int t = t0; t <= t_hi; ++t) p.scores[static_cast<int64_t>(t) * p.ld + s] = neg_inf;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1 && n_vis > 0) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ---- host side ---------------------------------------------------------------------------------------------
PFN_encodeTiled get_encode_tiled() {
    static PFN_encodeTiled fn = nullptr;
    if (fn == nullptr) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess && qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<PFN_encodeTiled>(p);
    }
    return fn;
}

bool make_tmap_2d_sw128(CUtensorMap* map, const void* base, int elem_bytes, uint64_t rows, uint64_t cols, uint64_t row_pitch_bytes,
                        uint32_t box_rows, uint32_t box_cols) {
    PFN_encodeTiled enc = get_encode_tiled();
    if (enc == nullptr) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {row_pitch_bytes};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    // elem_bytes 0: 4-bit elements, 16 of them expanded to a 16-byte aligned shared-memory chunk (box_cols must be 128)
    const CUtensorMapDataType dt = elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                                   : elem_bytes == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B;
    return enc(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool indexer_tc_supported(int M, int H, int D, int64_t n_keys, int64_t q_stride_tok, int64_t /*k_stride_tok*/, int dtype) {
    if (!(H == 4 || H == 8 || H == 16 || H == 32 || H == 64)) return false;
    const int row_bytes = D * (dtype == JANUS_DTYPE_BF16 ? 2 : 1);
    if (row_bytes != 128 && row_bytes != 256) return false;
    if (dtype == JANUS_DTYPE_FP8_Q_FP4_K && D != 128) return false;     // the packed 4-bit TMA box is 128 elements
    if (q_stride_tok != static_cast<int64_t>(H) * D) return false;
    if (static_cast<int64_t>(M) * H >= (int64_t(1) << 31) || n_keys >= (int64_t(1) << 31) - 256) return false;
    return true;
}

// Candidate mode needs every epilogue warp's tokens to fit its staging slots, whatever sub-tile count the launch picks.
bool indexer_tc_candidates_supported(int H, int D, int dtype) {
    const int row_bytes = D * (dtype == JANUS_DTYPE_BF16 ? 2 : 1);
    const int nq_max = row_bytes == 128 ? 4 : 2;
    if (dtype == JANUS_DTYPE_FP8_Q_FP4_K) return false;                 // the sample gather and the exact fallback read 8- and 16-bit keys
    return (H == 32 || H == 64) && (nq_max / 2) * (TC_N / H) <= TC_CAND_TPW;
}

template <int H, bool FP8, bool CAND, bool RAGGED = false>
static int launch_tc(const CUtensorMap& tq, const CUtensorMap& tk, const TcParams& p, const TcCandParams& cp, dim3 grid, size_t smem,
                     cudaStream_t stream) {
    JANUS_CUDA_CHECK(cudaFuncSetAttribute(indexer_tc_kernel<H, FP8, CAND, RAGGED>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    indexer_tc_kernel<H, FP8, CAND, RAGGED><<<grid, RAGGED ? TC_THREADS_RAGGED : (CAND ? TC_THREADS : TC_THREADS16), smem, stream>>>(tq, tk, p, cp);
    JANUS_CUDA_CHECK(cudaGetLastError());
    return JANUS_OK;
}

int launch_indexer_tc(const void* q_idx, const void* k_idx, int64_t k_stride_tok, const float* w, const float* q_scale,
                      int64_t q_scale_stride_tok, const float* k_scale, const float* row_bias, const float* col_bias, int M, int H,
                      int D, int64_t n_keys, int64_t q_pos0, int causal, int dtype, float* scores, int64_t ld, int32_t* dev_status,
                      cudaStream_t stream, const float* thr, int32_t* cand_cnt, void* cand, int cand_cap) {
    const bool k_fp4 = dtype == JANUS_DTYPE_FP8_Q_FP4_K;
    const bool fp8 = dtype == JANUS_DTYPE_FP8_E4M3 || k_fp4;
    const int esz = fp8 ? 1 : 2;
    TcParams p;
    p.w = w; p.q_scale = q_scale; p.q_scale_stride_tok = q_scale_stride_tok; p.k_scale = k_scale;
    p.row_bias = row_bias; p.col_bias = col_bias; p.scores = scores; p.ld = ld; p.n_keys = n_keys; p.q_pos0 = q_pos0;
    p.M = M; p.H = H; p.causal = causal; p.dev_status = dev_status;
    const TcCandParams cp{thr, cand_cnt, static_cast<int2*>(cand), cand_cap, nullptr, k_fp4 ? 1 : 0};
    p.atoms = D * esz / 128;
    p.nq = p.atoms == 1 ? 4 : 2;
    const int tps = TC_N / H;
    while (p.nq > 2 && static_cast<int64_t>(p.nq / 2) * tps >= M) p.nq /= 2;   // small M: do not load empty sub-tiles
    const int q_bytes = p.nq * p.atoms * TC_N * 128;
    const int k_stage = p.atoms * TC_KEYS * 128;
    const bool cand_mode = thr != nullptr;
    if (cand_mode && (p.nq + 1) / 2 * tps > TC_CAND_TPW) return JANUS_ERR_UNSUPPORTED;
    const int tail = static_cast<int>(sizeof(float)) * (p.nq * TC_N + 2 * p.nq * tps) + (cand_mode ? TC_CAND_STAGE_BYTES : 0) +
                     static_cast<int>(sizeof(TcBarriers)) + 16;
    p.stages = (TC_SMEM_BUDGET - q_bytes - tail) / k_stage;
    if (p.stages > TC_MAX_STAGES) p.stages = TC_MAX_STAGES;
    if (p.stages < 2) return JANUS_ERR_UNSUPPORTED;
    const size_t smem = static_cast<size_t>(q_bytes) + static_cast<size_t>(p.stages) * k_stage + tail;
    p.n_tiles = static_cast<int>((n_keys + TC_KEYS - 1) / TC_KEYS);
    const int tpc = p.nq * tps;
    const int n_groups = (M + tpc - 1) / tpc;
    int64_t per = (static_cast<int64_t>(p.n_tiles) * n_groups + 148 * 4 - 1) / (148 * 4);
    if (per < 2) per = 2;
    if (per > (cand_mode ? 64 : 256)) per = cand_mode ? 64 : 256;     // a CTA's start-up (query tile load, tensor-memory allocation) is paid once per `per` key tiles:
                                  // 256 against 64 was 1-2 % at 131072 keys x 4096 rows, with still about seven waves of CTAs
    p.tiles_per_cta = static_cast<int>(per);
    dim3 grid((p.n_tiles + p.tiles_per_cta - 1) / p.tiles_per_cta, n_groups);
    if (grid.y > 65535) return JANUS_ERR_UNSUPPORTED;

    CUtensorMap tq, tk;
    const uint32_t box_cols = fp8 ? 128 : 64;
    if (!make_tmap_2d_sw128(&tq, q_idx, esz, static_cast<uint64_t>(M) * H, D, static_cast<uint64_t>(D) * esz, TC_N, box_cols)) return JANUS_ERR_CUDA;
    if (k_fp4) {   // packed 4-bit keys: the copy expands 16 of them into the low halves of a 16-byte chunk
        if (!make_tmap_2d_sw128(&tk, k_idx, 0, static_cast<uint64_t>(n_keys), D, static_cast<uint64_t>(k_stride_tok) / 2, TC_KEYS, 128))
            return JANUS_ERR_CUDA;
    } else if (!make_tmap_2d_sw128(&tk, k_idx, esz, static_cast<uint64_t>(n_keys), D, static_cast<uint64_t>(k_stride_tok) * esz, TC_KEYS, box_cols)) {
        return JANUS_ERR_CUDA;
    }

#define JANUS_TC_CASE(HH, CC)                                                         \
    case HH:                                                                          \
        return fp8 ? launch_tc<HH, true, CC>(tq, tk, p, cp, grid, smem, stream) : launch_tc<HH, false, CC>(tq, tk, p, cp, grid, smem, stream);
    if (cand_mode) {
        switch (H) {   // head counts whose tokens per epilogue warp fit the staging slots
            JANUS_TC_CASE(32, true)
            JANUS_TC_CASE(64, true)
        }
        return JANUS_ERR_UNSUPPORTED;
    }
    switch (H) {
        JANUS_TC_CASE(4, false)
        JANUS_TC_CASE(8, false)
        JANUS_TC_CASE(16, false)
        JANUS_TC_CASE(32, false)
        JANUS_TC_CASE(64, false)
    }
#undef JANUS_TC_CASE
    return JANUS_ERR_UNSUPPORTED;
}

// Ragged batch (decode): B query rows, row b against keys key_offsets[b] .. key_offsets[b+1] of one concatenated array.
bool indexer_tc_batch_supported(int B, int H, int D, int64_t total_keys, int dtype) {
    const int row_bytes = D * (dtype == JANUS_DTYPE_BF16 ? 2 : 1);
    if (dtype == JANUS_DTYPE_FP8_Q_FP4_K && D != 128) return false;      // the packed 4-bit TMA box is 128 elements
    return H == 64 && (row_bytes == 128 || row_bytes == 256) && static_cast<int64_t>(B) * H < (int64_t(1) << 31) &&
           total_keys < (int64_t(1) << 31) - 256 && B <= 65535;
}

int launch_indexer_tc_batch(const void* q_idx, const void* k_idx, int64_t k_stride_tok, const float* w, const float* q_scale,
                            int64_t q_scale_stride_tok, const float* k_scale, const float* row_bias, const float* col_bias, int B, int H, int D,
                            int64_t total_keys, int64_t max_keys, const int64_t* key_offsets, int dtype, float* scores, int32_t* dev_status,
                            cudaStream_t stream) {
    const bool k_fp4 = dtype == JANUS_DTYPE_FP8_Q_FP4_K;
    const bool fp8 = dtype == JANUS_DTYPE_FP8_E4M3 || k_fp4;
    const int esz = fp8 ? 1 : 2;
    TcParams p;
    p.w = w; p.q_scale = q_scale; p.q_scale_stride_tok = q_scale_stride_tok; p.k_scale = k_scale;
    p.row_bias = row_bias; p.col_bias = col_bias; p.scores = scores; p.ld = 0; p.n_keys = total_keys; p.q_pos0 = 0;
    p.M = B; p.H = H; p.causal = 0; p.dev_status = dev_status;
    const TcCandParams cp{nullptr, nullptr, nullptr, 0, key_offsets, k_fp4 ? 1 : 0};
    p.atoms = D * esz / 128;
    p.nq = 1;
    const int tps = TC_N / H;
    const int q_bytes = p.nq * p.atoms * H * 128;           // one query row: H (head) rows of the B operand
    const int k_stage = p.atoms * TC_KEYS * 128;
    const int tail = static_cast<int>(sizeof(float)) * (p.nq * TC_N + 2 * p.nq * tps) + static_cast<int>(sizeof(TcBarriers)) + 16;
    // One query row per CTA leaves the single MMA-issuing thread as the limit of a CTA, so several CTAs share an SM: four with
    // one-byte operands (each a quarter of the SM's shared memory less the 1 KB the system keeps per CTA, 2 x H of the 512
    // TMEM columns, 6 warps of at most 80 registers), two with bf16 (a key stage is 32 KB).
    const int budget = (227 * 1024) / (fp8 ? 4 : 2) - 1024;
    p.stages = (budget - q_bytes - tail) / k_stage;
    if (p.stages > TC_MAX_STAGES) p.stages = TC_MAX_STAGES;
    if (p.stages < 2) return JANUS_ERR_UNSUPPORTED;
    const size_t smem = static_cast<size_t>(q_bytes) + static_cast<size_t>(p.stages) * k_stage + tail;
    const int max_tiles = static_cast<int>((max_keys + TC_KEYS - 1) / TC_KEYS);
    p.n_tiles = max_tiles;
    int64_t per = (static_cast<int64_t>(max_tiles) * B + 148 * 4 - 1) / (148 * 4);
    if (per < 2) per = 2;
    if (per > 64) per = 64;
    p.tiles_per_cta = static_cast<int>(per);
    dim3 grid((max_tiles + p.tiles_per_cta - 1) / p.tiles_per_cta, B);
    CUtensorMap tq, tk;
    const uint32_t box_cols = fp8 ? 128 : 64;
    if (!make_tmap_2d_sw128(&tq, q_idx, esz, static_cast<uint64_t>(B) * H, D, static_cast<uint64_t>(D) * esz, H, box_cols)) return JANUS_ERR_CUDA;
    if (k_fp4) {
        if (!make_tmap_2d_sw128(&tk, k_idx, 0, static_cast<uint64_t>(total_keys), D, static_cast<uint64_t>(k_stride_tok) / 2, TC_KEYS, 128))
            return JANUS_ERR_CUDA;
    } else if (!make_tmap_2d_sw128(&tk, k_idx, esz, static_cast<uint64_t>(total_keys), D, static_cast<uint64_t>(k_stride_tok) * esz, TC_KEYS, box_cols)) {
        return JANUS_ERR_CUDA;
    }
    return fp8 ? launch_tc<64, true, false, true>(tq, tk, p, cp, grid, smem, stream) : launch_tc<64, false, false, true>(tq, tk, p, cp, grid, smem, stream);
}

}  // namespace janus
