// Shared device code of the top-k selection (Eq. 1, Sec. 2.2, selection part): exact k-th selection over a candidate set
// with 2048-bucket histograms over a shrinking key range, and the sampled single-pass top-k of one fp32 row.
// Used by janus_topk (materialised scores) and by janus_indexer_topk (candidates appended by the indexer epilogue).
#pragma once

#include "janus_common.cuh"

namespace janus {

constexpr int TK_THREADS = 512;
constexpr int TK_BUCKETS = 2048;
constexpr int TK_SAMPLE = 4096;     // 512 threads x 8 floats (one 32-byte sector each)
constexpr int TK_DIRECT = 256;      // a bucket of at most this many keys is ranked directly instead of split further

template <int CAP>
struct TopkSharedT {
    static constexpr int kCap = CAP;      // candidate slots (key + index = 8 bytes each)
    uint32_t cand_key[CAP];
    int32_t cand_idx[CAP];
    int hist[TK_BUCKETS];
    int scan[40];
    int n_cand;
    int out_pos;
    int eq_taken;
    uint32_t red_lo, red_hi;
    int sel_bucket, sel_above, sel_count;
    int n_small;
};

struct SmemSource {
    const uint32_t* key;
    const int32_t* idx;
    int n;
    __device__ __forceinline__ int size() const { return n; }
    __device__ __forceinline__ uint32_t key_at(int i) const { return key[i]; }
    __device__ __forceinline__ int32_t idx_at(int i) const { return idx ? idx[i] : i; }
};
struct GlobalSource {
    const float* row;
    int n;
    __device__ __forceinline__ int size() const { return n; }
    __device__ __forceinline__ uint32_t key_at(int i) const { return float_to_key(__ldcg(row + i)); }
    __device__ __forceinline__ int32_t idx_at(int i) const { return i; }
};

// Exact `need`-th largest key of a source (1 <= need <= number of elements).
// Returns the threshold key T and, in *n_eq_take, how many elements equal to T belong to the selection.
// Every thread of the CTA must call it; results are uniform.
template <class Src, class Sh>
__device__ uint32_t select_kth(const Src& src, int need, Sh& sh, int* n_eq_take) {
    const int tid = threadIdx.x;
    const int n = src.size();
    // range of the active keys
    uint32_t lo = 0xffffffffu, hi = 0u;
    for (int i = tid; i < n; i += TK_THREADS) {
        const uint32_t key = src.key_at(i);
        lo = min(lo, key);
        hi = max(hi, key);
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        lo = min(lo, __shfl_xor_sync(0xffffffffu, lo, d));
        hi = max(hi, __shfl_xor_sync(0xffffffffu, hi, d));
    }
    if (tid == 0) { sh.red_lo = 0xffffffffu; sh.red_hi = 0u; }
    __syncthreads();
    if ((tid & 31) == 0) { atomicMin(&sh.red_lo, lo); atomicMax(&sh.red_hi, hi); }
    __syncthreads();
    lo = sh.red_lo;
    hi = sh.red_hi;
    __syncthreads();

    for (int iter = 0; iter < 8 && lo < hi; ++iter) {
        const uint32_t range = hi - lo;
        const int bits = 32 - __clz(range);                   // range < 2^bits
        const int shift = bits > 11 ? bits - 11 : 0;          // (range >> shift) < 2048
        for (int i = tid; i < TK_BUCKETS; i += TK_THREADS) sh.hist[i] = 0;
        __syncthreads();
        for (int i = tid; i < n; i += TK_THREADS) {
            const uint32_t key = src.key_at(i);
            if (key >= lo && key <= hi) atomicAdd(&sh.hist[(key - lo) >> shift], 1);
        }
        __syncthreads();
        // walk the buckets from the top: thread t owns the 4 buckets 2047-4t .. 2044-4t
        int c[4];
        int mine = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) { c[j] = sh.hist[TK_BUCKETS - 1 - (4 * tid + j)]; mine += c[j]; }
        int total;
        int above = block_exclusive_scan<TK_THREADS>(mine, sh.scan, &total);
        if (above < need && need <= above + mine) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (above < need && need <= above + c[j]) { sh.sel_bucket = TK_BUCKETS - 1 - (4 * tid + j); sh.sel_above = above; sh.sel_count = c[j]; }
                above += c[j];
            }
        }
        __syncthreads();
        const uint32_t b = static_cast<uint32_t>(sh.sel_bucket);
        need -= sh.sel_above;
        const uint32_t new_lo = lo + (b << shift);
        if (b < (range >> shift)) hi = new_lo + ((1u << shift) - 1u);   // the top bucket keeps hi (and cannot overflow)
        lo = new_lo;
        const int m = sh.sel_count;                                    // keys inside [lo, hi]
        __syncthreads();
        if (lo < hi && m <= TK_DIRECT) {
            // Few keys are left: instead of two more histogram passes (each a sweep over the source plus a block scan), copy
            // them out (the histogram array is free) and count, for every key, the keys above and equal to it.
            uint32_t* small = reinterpret_cast<uint32_t*>(sh.hist);
            if (tid == 0) sh.n_small = 0;
            __syncthreads();
            for (int i = tid; i < n; i += TK_THREADS) {
                const uint32_t key = src.key_at(i);
                if (key >= lo && key <= hi) small[atomicAdd(&sh.n_small, 1)] = key;
            }
            __syncthreads();
            for (int i = tid >> 5; i < m; i += TK_THREADS / 32) {      // a warp per key, its lanes striding over the others
                const uint32_t mine = small[i];
                int g = 0, e = 0;
                for (int j = tid & 31; j < m; j += 32) {
                    const uint32_t other = small[j];
                    g += other > mine ? 1 : 0;
                    e += other == mine ? 1 : 0;
                }
                g = __reduce_add_sync(0xffffffffu, g);
                e = __reduce_add_sync(0xffffffffu, e);
                if ((tid & 31) == 0 && g < need && need <= g + e) { sh.red_lo = mine; sh.sel_above = need - g; }   // equal keys write equal values
            }
            __syncthreads();
            const uint32_t T = sh.red_lo;
            *n_eq_take = sh.sel_above;
            __syncthreads();
            return T;
        }
    }
    *n_eq_take = need;   // lo == hi: `need` of the elements equal to lo complete the selection
    return lo;
}

// Writes the selection (all keys > T, plus n_eq of the keys == T) to out[0..k).
template <class Src, class Sh>
__device__ void emit_selection(const Src& src, uint32_t T, int n_eq, int32_t* out, Sh& sh) {
    const int n = src.size();
    for (int i = threadIdx.x; i < n; i += TK_THREADS) {
        const uint32_t key = src.key_at(i);
        if (key > T) {
            out[atomicAdd(&sh.out_pos, 1)] = src.idx_at(i);
        } else if (key == T) {
            if (atomicAdd(&sh.eq_taken, 1) < n_eq) out[atomicAdd(&sh.out_pos, 1)] = src.idx_at(i);
        }
    }
}

// Keeps x (at row position i) if it is at or above the streaming threshold.  The float comparison admits a superset of
// the exact key comparison (it treats -0 and +0 alike); the exact selection afterwards works on keys.
template <class Sh>
__device__ __forceinline__ void keep_if_candidate(float x, int i, float thr_f, Sh& sh) {
    if (x >= thr_f) {
        const int pos = atomicAdd(&sh.n_cand, 1);
        if (pos < Sh::kCap) { sh.cand_key[pos] = float_to_key(x); sh.cand_idx[pos] = i; }
    }
}

// The same for the sixteen elements a thread holds after four 16-byte loads (x[u] = elements e0 + u * e_step .. + 3): the
// thread counts its candidates, reserves that many slots with one atomic and writes them.  One element in thirty passes, so
// an atomic per element (even aggregated over the warp) costs several times the instructions of the comparison itself and
// made the streaming pass issue-bound rather than memory-bound.
template <class Sh>
__device__ __forceinline__ void keep_candidates16(const float4 (&x)[4], int e0, int e_step, float thr_f, Sh& sh) {
    int c = 0;
#pragma unroll
    for (int u = 0; u < 4; ++u)
        c += (x[u].x >= thr_f ? 1 : 0) + (x[u].y >= thr_f ? 1 : 0) + (x[u].z >= thr_f ? 1 : 0) + (x[u].w >= thr_f ? 1 : 0);
    if (c == 0) return;
    int o = atomicAdd(&sh.n_cand, c);
    auto put = [&](float v, int e) {
        if (v >= thr_f) {
            if (o < Sh::kCap) { sh.cand_key[o] = float_to_key(v); sh.cand_idx[o] = e; }
            ++o;
        }
    };
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int e = e0 + u * e_step;
        put(x[u].x, e); put(x[u].y, e + 1); put(x[u].z, e + 2); put(x[u].w, e + 3);
    }
}

__device__ __forceinline__ void topk_prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

// ---- the three phases of a row (n > k), callable separately so that several CTAs can share the streaming pass of one row

// Streaming threshold of a row as an order-preserving key (0: keep everything): the sample value of a rank a few standard
// deviations below where the row's k-th value is expected.  Thread i reads 8 consecutive floats at an evenly spread,
// 32-byte aligned offset; the candidate buffer of `sh` is the scratch.  Every thread of the CTA calls it; the result is
// uniform and depends on the row only.
template <class Sh>
__device__ uint32_t topk_sample_threshold(const float* __restrict__ row, int n, int k, Sh& sh) {
    const int tid = threadIdx.x;
    uint32_t thr = 0u;
    if (n > Sh::kCap) {
        const float4* row4 = reinterpret_cast<const float4*>(row);
        const int n8 = n >> 3;                       // complete 8-float groups
        const int g = static_cast<int>((static_cast<int64_t>(tid) * (n8 - 1)) / (TK_THREADS - 1));
        const float4 a = __ldcg(row4 + 2 * g), b = __ldcg(row4 + 2 * g + 1);
        uint32_t* skey = sh.cand_key;                // the candidate buffer is free at this point
        skey[tid * 8 + 0] = float_to_key(a.x); skey[tid * 8 + 1] = float_to_key(a.y);
        skey[tid * 8 + 2] = float_to_key(a.z); skey[tid * 8 + 3] = float_to_key(a.w);
        skey[tid * 8 + 4] = float_to_key(b.x); skey[tid * 8 + 5] = float_to_key(b.y);
        skey[tid * 8 + 6] = float_to_key(b.z); skey[tid * 8 + 7] = float_to_key(b.w);
        __syncthreads();
        const float expect = static_cast<float>(TK_SAMPLE) * static_cast<float>(k) / static_cast<float>(n);
        const int r = static_cast<int>(expect + 4.0f * sqrtf(expect) + 8.0f);
        if (r < TK_SAMPLE) {
            int dummy;
            SmemSource s{skey, nullptr, TK_SAMPLE};
            thr = select_kth(s, r, sh, &dummy);
        }
        __syncthreads();
    }
    return thr;
}

// One streaming pass over the 16-byte groups [f4_begin, f4_end) of the row (and, with `tail`, the n % 4 elements after the
// last whole group): elements at or above the threshold go to the candidate buffer of `dst`, which may be another CTA's
// shared memory (a cluster-mapped reference).
template <class Sh>
__device__ void topk_stream(const float* __restrict__ row, int n, int f4_begin, int f4_end, bool tail, uint32_t thr, Sh& dst) {
    const int tid = threadIdx.x;
    const float4* row4 = reinterpret_cast<const float4*>(row);
    const float thr_f = thr == 0u ? __int_as_float(0xff800000) : key_to_float(thr);
    constexpr int UNROLL = 4;                     // 16-byte loads in flight per thread
    int i = f4_begin + tid;
    for (; i + (UNROLL - 1) * TK_THREADS < f4_end; i += UNROLL * TK_THREADS) {
        float4 x[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) x[u] = __ldcs(row4 + i + u * TK_THREADS);
        keep_candidates16(x, 4 * i, 4 * TK_THREADS, thr_f, dst);
    }
    for (; i < f4_end; i += TK_THREADS) {
        const float4 x = __ldcs(row4 + i);
        keep_if_candidate(x.x, 4 * i, thr_f, dst);
        keep_if_candidate(x.y, 4 * i + 1, thr_f, dst);
        keep_if_candidate(x.z, 4 * i + 2, thr_f, dst);
        keep_if_candidate(x.w, 4 * i + 3, thr_f, dst);
    }
    const int n4 = n >> 2;
    if (tail && tid < n - 4 * n4) keep_if_candidate(__ldcg(row + 4 * n4 + tid), 4 * n4 + tid, thr_f, dst);
}

// Exact selection over the candidates in `sh` (over the whole row in global memory when the sample misjudged it: fewer than
// k candidates, or more than the buffer holds) and emission of the k indices, count and k-th value.
template <class Sh>
__device__ void topk_finish(const float* __restrict__ row, int n, int k, int t, int32_t* __restrict__ out, int32_t* __restrict__ count,
                            float* __restrict__ kth, Sh& sh) {
    const int n_cand = sh.n_cand;
    uint32_t T;
    int n_eq;
    if (n_cand >= k && n_cand <= Sh::kCap) {
        SmemSource s{sh.cand_key, sh.cand_idx, n_cand};
        T = select_kth(s, k, sh, &n_eq);
        emit_selection(s, T, n_eq, out, sh);
    } else {
        GlobalSource s{row, n};
        T = select_kth(s, k, sh, &n_eq);
        emit_selection(s, T, n_eq, out, sh);
    }
    if (threadIdx.x == 0) {
        if (count) count[t] = n < k ? n : k;
        if (kth) kth[t] = key_to_float(T);
    }
}

// Top-k of one fp32 row of n elements (16-byte aligned) by the whole CTA (TK_THREADS threads): out[0..k) receives the
// indices (-1 padded), count[t] / kth[t] the number selected and the smallest selected value (either may be NULL).
// `next_row` (may be NULL): the row this CTA takes next.  The sample sectors of that row are requested into L2 once this
// row's streaming pass is over, so the next sample does not start with a DRAM round trip.  (Requesting the head of the next
// row as well, 96 to 512 KB, made the kernel slower: 0.49 -> 0.50 .. 0.58 ms at 4096 rows of 135168.)
template <class Sh>
__device__ void topk_row(const float* __restrict__ row, int n, int k, int t, int32_t* __restrict__ out, int32_t* __restrict__ count,
                         float* __restrict__ kth, Sh& sh, const float* __restrict__ next_row = nullptr, int next_n = 0) {
    const int tid = threadIdx.x;

    if (tid == 0) { sh.n_cand = 0; sh.out_pos = 0; sh.eq_taken = 0; }
    __syncthreads();

    if (n <= k) {  // the whole prefix is selected
        for (int i = tid; i < k; i += TK_THREADS) out[i] = i < n ? i : -1;
        if (kth != nullptr || count != nullptr) {
            float mn = __int_as_float(0x7f800000);
            for (int i = tid; i < n; i += TK_THREADS) mn = fminf(mn, __ldcg(row + i));
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, d));
            if (tid == 0) sh.red_lo = 0xffffffffu;
            __syncthreads();
            if ((tid & 31) == 0) atomicMin(&sh.red_lo, float_to_key(mn));
            __syncthreads();
            if (tid == 0) {
                if (count) count[t] = n;
                if (kth) kth[t] = n > 0 ? key_to_float(sh.red_lo) : __int_as_float(0xff800000);
            }
        }
        return;
    }

    const uint32_t thr = topk_sample_threshold(row, n, k, sh);
    topk_stream(row, n, 0, n >> 2, true, thr, sh);
    if (next_row != nullptr && next_n > Sh::kCap) {
        const int n8 = next_n >> 3;
        const int g = static_cast<int>((static_cast<int64_t>(tid) * (n8 - 1)) / (TK_THREADS - 1));
        topk_prefetch_l2(next_row + 8 * g);                                   // the sample sector this thread will read
    }
    __syncthreads();
    topk_finish(row, n, k, t, out, count, kth, sh);
}

}  // namespace janus
