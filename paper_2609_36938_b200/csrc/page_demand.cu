// janus_page_demand: union of selected tokens -> physical page bitmap, ascending page list,
// maximal runs of adjacent physical pages, and the miss set "exact minus predicted"
// (union of selections: Sec. 2.2; corrective reads: Sec. 4.2; read packing: Sec. 4.3).
//
// Kernel 1 (mark) streams the index block with 16-byte loads and sets page bits.  When the bitmap
// fits in shared memory each CTA ORs into a private copy first and only touches a global word once
// per CTA; bits are tested before the atomic so a saturated union costs no atomics at all.
// Kernel 2 (lists) is one CTA that turns a bitmap into ordered lists with block-wide scans.
#include "janus_common.cuh"

namespace janus {

constexpr int MARK_THREADS = 256;
constexpr int MARK_SMEM_WORDS = 8192;  // 32 KB: bitmaps up to 262144 pages stay in shared memory
constexpr int LIST_THREADS = 1024;

__device__ __forceinline__ void mark_one(int s, int64_t demand_limit, int page_size, int page_shift,
                                         const int32_t* __restrict__ page_table, int64_t n_logical_pages,
                                         int64_t n_phys_pages, uint32_t* bm, int32_t* dev_status) {
    if (s < 0 || static_cast<int64_t>(s) >= demand_limit) return;
    const int64_t lp = page_shift >= 0 ? (s >> page_shift) : (s / page_size);
    if (lp >= n_logical_pages) { report(dev_status, JANUS_DEV_INDEX_OUT_OF_RANGE); return; }
    const int32_t p = __ldg(page_table + lp);
    if (p < 0 || static_cast<int64_t>(p) >= n_phys_pages) { report(dev_status, JANUS_DEV_INDEX_OUT_OF_RANGE); return; }
    const uint32_t bit = 1u << (p & 31);
    uint32_t* wp = bm + (p >> 5);
    if ((*reinterpret_cast<volatile uint32_t*>(wp) & bit) == 0u) atomicOr(wp, bit);
}

template <bool USE_SMEM>
__global__ void __launch_bounds__(MARK_THREADS)
page_mark_kernel(const int32_t* __restrict__ idx, int64_t n_idx, int64_t demand_limit, int page_size, int page_shift,
                 const int32_t* __restrict__ page_table, int64_t n_logical_pages, int64_t n_phys_pages,
                 uint32_t* __restrict__ bitmap, int n_words, int32_t* dev_status) {
    __shared__ uint32_t sbm[USE_SMEM ? MARK_SMEM_WORDS : 1];
    uint32_t* bm = bitmap;
    if (USE_SMEM) {
        for (int i = threadIdx.x; i < n_words; i += MARK_THREADS) sbm[i] = 0u;
        __syncthreads();
        bm = sbm;
    }
    const int64_t n_vec = n_idx >> 2;  // idx is 16-byte aligned
    const int4* idx4 = reinterpret_cast<const int4*>(idx);
    const int64_t stride = static_cast<int64_t>(gridDim.x) * MARK_THREADS;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * MARK_THREADS + threadIdx.x; i < n_vec; i += stride) {
        const int4 v = __ldg(idx4 + i);
        mark_one(v.x, demand_limit, page_size, page_shift, page_table, n_logical_pages, n_phys_pages, bm, dev_status);
        mark_one(v.y, demand_limit, page_size, page_shift, page_table, n_logical_pages, n_phys_pages, bm, dev_status);
        mark_one(v.z, demand_limit, page_size, page_shift, page_table, n_logical_pages, n_phys_pages, bm, dev_status);
        mark_one(v.w, demand_limit, page_size, page_shift, page_table, n_logical_pages, n_phys_pages, bm, dev_status);
    }
    if (blockIdx.x == 0) {
        for (int64_t i = (n_vec << 2) + threadIdx.x; i < n_idx; i += MARK_THREADS)
            mark_one(idx[i], demand_limit, page_size, page_shift, page_table, n_logical_pages, n_phys_pages, bm, dev_status);
    }
    if (USE_SMEM) {
        __syncthreads();
        for (int i = threadIdx.x; i < n_words; i += MARK_THREADS) {
            const uint32_t v = sbm[i];
            if (v != 0u && (__ldcg(bitmap + i) & v) != v) atomicOr(bitmap + i, v);
        }
    }
}

// Turns one bitmap (optionally "a AND NOT b") into: ascending ids, maximal runs, counts.
// Single CTA; words are consumed LIST_THREADS at a time, one word per thread.
__device__ void bitmap_to_lists(const uint32_t* __restrict__ a, const uint32_t* __restrict__ not_b, int n_words,
                                int64_t n_bits, int32_t* __restrict__ ids, int32_t* __restrict__ n_ids,
                                int32_t* __restrict__ runs, int32_t* __restrict__ n_runs, int64_t capacity,
                                int32_t* dev_status, int* scan_scratch) {
    int id_base = 0, run_base = 0, end_base = 0;
    auto word_at = [&](int i) -> uint32_t {
        if (i < 0 || i >= n_words) return 0u;
        uint32_t v = a[i];
        if (not_b != nullptr) v &= ~not_b[i];
        if (i == n_words - 1 && (n_bits & 31)) v &= (1u << (n_bits & 31)) - 1u;  // ignore bits past the last page
        return v;
    };
    for (int base = 0; base < n_words; base += LIST_THREADS) {
        const int i = base + threadIdx.x;
        const uint32_t v = word_at(i);
        const uint32_t prev_top = word_at(i - 1) >> 31;
        const uint32_t next_bot = word_at(i + 1) & 1u;
        const uint32_t starts = v & ~((v << 1) | prev_top);          // set, and the page below is not
        const uint32_t ends = v & ~((v >> 1) | (next_bot << 31));    // set, and the page above is not
        int tot_ids, tot_starts, tot_ends;
        int o_id = block_exclusive_scan<LIST_THREADS>(__popc(v), scan_scratch, &tot_ids) + id_base;
        int o_st = block_exclusive_scan<LIST_THREADS>(__popc(starts), scan_scratch, &tot_starts) + run_base;
        int o_en = block_exclusive_scan<LIST_THREADS>(__popc(ends), scan_scratch, &tot_ends) + end_base;
        uint32_t m = v;
        while (m) {
            const int b = __ffs(m) - 1;
            m &= m - 1;
            if (o_id < capacity) ids[o_id] = i * 32 + b;
            ++o_id;
        }
        m = starts;
        while (m) {
            const int b = __ffs(m) - 1;
            m &= m - 1;
            if (o_st < capacity) runs[2 * o_st] = i * 32 + b;
            ++o_st;
        }
        m = ends;
        while (m) {  // the j-th end closes the j-th start; store end+1, converted to a length below
            const int b = __ffs(m) - 1;
            m &= m - 1;
            if (o_en < capacity) runs[2 * o_en + 1] = i * 32 + b + 1;
            ++o_en;
        }
        id_base += tot_ids;
        run_base += tot_starts;
        end_base += tot_ends;
    }
    __syncthreads();
    const int n_r = run_base < capacity ? run_base : static_cast<int>(capacity);
    for (int j = threadIdx.x; j < n_r; j += LIST_THREADS) runs[2 * j + 1] -= runs[2 * j];
    if (threadIdx.x == 0) {
        *n_ids = id_base;
        *n_runs = run_base;
        if (id_base > capacity || run_base > capacity) report(dev_status, JANUS_DEV_CAPACITY_EXCEEDED);
    }
    __syncthreads();
}

__global__ void __launch_bounds__(LIST_THREADS)
page_lists_kernel(const uint32_t* __restrict__ bitmap, const uint32_t* __restrict__ predicted, int n_words, int64_t n_phys_pages,
                  int32_t* pages, int32_t* n_pages, int32_t* runs, int32_t* n_runs,
                  int32_t* miss_pages, int32_t* n_miss, int32_t* miss_runs, int32_t* n_miss_runs,
                  int64_t capacity, int32_t* dev_status) {
    __shared__ int scan_scratch[40];
    bitmap_to_lists(bitmap, nullptr, n_words, n_phys_pages, pages, n_pages, runs, n_runs, capacity, dev_status, scan_scratch);
    if (miss_pages != nullptr)
        bitmap_to_lists(bitmap, predicted, n_words, n_phys_pages, miss_pages, n_miss, miss_runs, n_miss_runs, capacity,
                        dev_status, scan_scratch);
}

// Large pools (a decode batch addresses the whole KV pool: 10^5 pages and more): the same lists built by one CTA per
// 1024-word chunk.  A CTA first counts the ids / run starts / run ends of all words before its chunk (a few KB of bitmap
// for the sizes this path is used for), then writes its part exactly like the single-CTA kernel; run lengths need every
// start and end, so a small second kernel turns (start, end+1) into (start, length).  blockIdx.y = 0: the set itself,
// 1: the miss set (bitmap AND NOT predicted).
constexpr int LIST_MAX_CHUNKS = 64;

__global__ void __launch_bounds__(LIST_THREADS)
page_lists_chunk_kernel(const uint32_t* __restrict__ bitmap, const uint32_t* __restrict__ predicted, int n_words, int64_t n_phys_pages,
                        int32_t* pages, int32_t* n_pages, int32_t* runs, int32_t* n_runs, int32_t* miss_pages, int32_t* n_miss,
                        int32_t* miss_runs, int32_t* n_miss_runs, int64_t capacity, int32_t* dev_status) {
    __shared__ int scan_scratch[3 * 33];
    const bool miss = blockIdx.y == 1;
    const uint32_t* a = bitmap;
    const uint32_t* not_b = miss ? predicted : nullptr;
    int32_t* ids = miss ? miss_pages : pages;
    int32_t* n_ids = miss ? n_miss : n_pages;
    int32_t* out_runs = miss ? miss_runs : runs;
    int32_t* out_n_runs = miss ? n_miss_runs : n_runs;
    auto word_at = [&](int i) -> uint32_t {
        if (i < 0 || i >= n_words) return 0u;
        uint32_t v = a[i];
        if (not_b != nullptr) v &= ~not_b[i];
        if (i == n_words - 1 && (n_phys_pages & 31)) v &= (1u << (n_phys_pages & 31)) - 1u;
        return v;
    };
    auto starts_of = [&](int i, uint32_t v) { return v & ~((v << 1) | (word_at(i - 1) >> 31)); };
    auto ends_of = [&](int i, uint32_t v) { return v & ~((v >> 1) | ((word_at(i + 1) & 1u) << 31)); };
    const int base = blockIdx.x * LIST_THREADS;
    // ---- everything before this chunk
    int c_id = 0, c_st = 0, c_en = 0;
    for (int i = threadIdx.x; i < base; i += LIST_THREADS) {
        const uint32_t v = word_at(i);
        c_id += __popc(v);
        c_st += __popc(starts_of(i, v));
        c_en += __popc(ends_of(i, v));
    }
    // ids, run starts and run ends are scanned together: one set of block barriers per scan instead of three
    int before[3] = {c_id, c_st, c_en}, skip[3], bases[3];
    block_exclusive_scan3<LIST_THREADS>(before, scan_scratch, skip, bases);
    const int id_base = bases[0], run_base = bases[1], end_base = bases[2];
    // ---- this chunk
    const int i = base + threadIdx.x;
    const uint32_t v = word_at(i);
    const uint32_t starts = starts_of(i, v), ends = ends_of(i, v);
    int mine[3] = {__popc(v), __popc(starts), __popc(ends)}, offs[3], tots[3];
    block_exclusive_scan3<LIST_THREADS>(mine, scan_scratch, offs, tots);
    const int tot_ids = tots[0], tot_starts = tots[1];
    int o_id = offs[0] + id_base, o_st = offs[1] + run_base, o_en = offs[2] + end_base;
    uint32_t m = v;
    while (m) {
        const int b = __ffs(m) - 1;
        m &= m - 1;
        if (o_id < capacity) ids[o_id] = i * 32 + b;
        ++o_id;
    }
    m = starts;
    while (m) {
        const int b = __ffs(m) - 1;
        m &= m - 1;
        if (o_st < capacity) out_runs[2 * o_st] = i * 32 + b;
        ++o_st;
    }
    m = ends;
    while (m) {  // the j-th end closes the j-th start; end+1 is stored and turned into a length by the second kernel
        const int b = __ffs(m) - 1;
        m &= m - 1;
        if (o_en < capacity) out_runs[2 * o_en + 1] = i * 32 + b + 1;
        ++o_en;
    }
    if (blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) {
        const int total_ids = id_base + tot_ids, total_runs = run_base + tot_starts;
        *n_ids = total_ids;
        *out_n_runs = total_runs;
        if (total_ids > capacity || total_runs > capacity) report(dev_status, JANUS_DEV_CAPACITY_EXCEEDED);
    }
}

__global__ void page_run_lengths_kernel(int32_t* runs, const int32_t* n_runs, int32_t* miss_runs, const int32_t* n_miss_runs, int64_t capacity) {
    int32_t* r = blockIdx.y == 1 ? miss_runs : runs;
    int64_t n = blockIdx.y == 1 ? *n_miss_runs : *n_runs;
    if (n > capacity) n = capacity;
    for (int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; j < n; j += static_cast<int64_t>(gridDim.x) * blockDim.x)
        r[2 * j + 1] -= r[2 * j];
}

// Chooses between the one-CTA list kernel (small bitmaps: one launch, no second pass) and the chunked pair.
static int launch_page_lists(const uint32_t* bitmap, const uint32_t* predicted, int n_words, int64_t n_phys_pages, int32_t* pages,
                             int32_t* n_pages, int32_t* runs, int32_t* n_runs, int32_t* miss_pages, int32_t* n_miss, int32_t* miss_runs,
                             int32_t* n_miss_runs, int64_t capacity, int32_t* dev_status, cudaStream_t stream);

// Batch form (decode over many sessions): row r of idx belongs to a session with its own page table
// page_tables[table_offsets[r] .. table_offsets[r+1]) and its own history length demand_limits[r]; physical page ids are
// global, so all rows mark one bitmap.  Sizes are small (rows x k indices), so this is the plain one-index-per-thread form.
__global__ void __launch_bounds__(MARK_THREADS)
page_mark_rows_kernel(const int32_t* __restrict__ idx, int64_t n_rows, int k, const int64_t* __restrict__ demand_limits, int page_size,
                      int page_shift, const int32_t* __restrict__ page_tables, const int64_t* __restrict__ table_offsets,
                      int64_t n_phys_pages, uint32_t* __restrict__ bitmap, int32_t* dev_status) {
    const int64_t n_idx = n_rows * k;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * MARK_THREADS;
    for (int64_t e = static_cast<int64_t>(blockIdx.x) * MARK_THREADS + threadIdx.x; e < n_idx; e += stride) {
        const int64_t r = e / k;
        const int64_t off = __ldg(table_offsets + r);
        // a table that starts before the array has no pages: its selected tokens are reported and skipped
        mark_one(__ldg(idx + e), __ldg(demand_limits + r), page_size, page_shift, page_tables + (off < 0 ? 0 : off),
                 off < 0 ? 0 : __ldg(table_offsets + r + 1) - off, n_phys_pages, bitmap, dev_status);
    }
}

static int launch_page_lists(const uint32_t* bitmap, const uint32_t* predicted, int n_words, int64_t n_phys_pages, int32_t* pages,
                             int32_t* n_pages, int32_t* runs, int32_t* n_runs, int32_t* miss_pages, int32_t* n_miss, int32_t* miss_runs,
                             int32_t* n_miss_runs, int64_t capacity, int32_t* dev_status, cudaStream_t stream) {
    const int n_chunks = (n_words + LIST_THREADS - 1) / LIST_THREADS;
    if (n_chunks >= 2 && n_chunks <= LIST_MAX_CHUNKS) {
        const dim3 grid(n_chunks, miss_pages != nullptr ? 2 : 1);
        page_lists_chunk_kernel<<<grid, LIST_THREADS, 0, stream>>>(bitmap, predicted, n_words, n_phys_pages, pages, n_pages, runs, n_runs, miss_pages,
                                                                   n_miss, miss_runs, n_miss_runs, capacity, dev_status);
        JANUS_CUDA_CHECK(cudaGetLastError());
        page_run_lengths_kernel<<<dim3(64, grid.y), 256, 0, stream>>>(runs, n_runs, miss_runs, n_miss_runs, capacity);
        JANUS_CUDA_CHECK(cudaGetLastError());
        return JANUS_OK;
    }
    page_lists_kernel<<<1, LIST_THREADS, 0, stream>>>(bitmap, predicted, n_words, n_phys_pages, pages, n_pages, runs, n_runs, miss_pages, n_miss,
                                                     miss_runs, n_miss_runs, capacity, dev_status);
    JANUS_CUDA_CHECK(cudaGetLastError());
    return JANUS_OK;
}

__global__ void page_union_kernel(uint32_t* __restrict__ dst, const uint32_t* __restrict__ src, int n_words) {
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n_words; i += gridDim.x * blockDim.x) dst[i] |= src[i];
}

}  // namespace janus

extern "C" int janus_page_union(uint32_t* dst, const uint32_t* src, int64_t n_phys_pages, void* stream_) {
    using namespace janus;
    if (!dst || !src || n_phys_pages <= 0) return JANUS_ERR_INVALID_ARG;
    if (n_phys_pages > (int64_t(1) << 31) - 64) return JANUS_ERR_UNSUPPORTED;
    const int n_words = static_cast<int>((n_phys_pages + 31) / 32);
    const int blocks = n_words < 256 * 148 ? (n_words + 255) / 256 : 148;
    page_union_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream_)>>>(dst, src, n_words);
    JANUS_CUDA_CHECK(cudaGetLastError());
    return JANUS_OK;
}

extern "C" size_t janus_page_demand_workspace_size(int64_t, int, int64_t) { return 0; }

extern "C" int janus_page_demand(const int32_t* idx, int64_t n_rows, int k, int64_t demand_limit, int page_size,
                                 const int32_t* page_table, int64_t n_logical_pages, int64_t n_phys_pages,
                                 const uint32_t* predicted_bitmap, uint32_t* bitmap, int32_t* pages, int32_t* n_pages,
                                 int32_t* runs, int32_t* n_runs, int32_t* miss_pages, int32_t* n_miss, int32_t* miss_runs,
                                 int32_t* n_miss_runs, int64_t capacity, void* /*ws*/, size_t /*ws_bytes*/,
                                 int32_t* dev_status, void* stream_) {
    using namespace janus;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (n_rows < 0 || k < 0 || page_size <= 0 || n_logical_pages < 0 || n_phys_pages <= 0 || capacity < 0 || demand_limit < 0)
        return JANUS_ERR_INVALID_ARG;
    if (n_phys_pages > (int64_t(1) << 31) - 64) return JANUS_ERR_UNSUPPORTED;
    if (!bitmap || !pages || !n_pages || !runs || !n_runs || !page_table) return JANUS_ERR_INVALID_ARG;
    const int n_miss_ptrs = (miss_pages != nullptr) + (n_miss != nullptr) + (miss_runs != nullptr) + (n_miss_runs != nullptr);
    if (n_miss_ptrs != 0 && n_miss_ptrs != 4) return JANUS_ERR_INVALID_ARG;
    const int64_t n_idx = n_rows * static_cast<int64_t>(k);
    if (n_idx > 0 && (!idx || !aligned16(idx))) return JANUS_ERR_INVALID_ARG;

    const int n_words = static_cast<int>((n_phys_pages + 31) / 32);
    JANUS_CUDA_CHECK(cudaMemsetAsync(bitmap, 0, sizeof(uint32_t) * n_words, stream));
    if (n_idx > 0) {
        int page_shift = -1;
        if ((page_size & (page_size - 1)) == 0) {
            page_shift = 0;
            while ((1 << page_shift) < page_size) ++page_shift;
        }
        const int64_t n_vec = (n_idx + 3) / 4;
        int64_t blocks = (n_vec + MARK_THREADS * 8 - 1) / (MARK_THREADS * 8);
        if (blocks < 1) blocks = 1;
        if (blocks > 148 * 8) blocks = 148 * 8;
        if (n_words <= MARK_SMEM_WORDS)
            page_mark_kernel<true><<<static_cast<unsigned>(blocks), MARK_THREADS, 0, stream>>>(
                idx, n_idx, demand_limit, page_size, page_shift, page_table, n_logical_pages, n_phys_pages, bitmap, n_words, dev_status);
        else
            page_mark_kernel<false><<<static_cast<unsigned>(blocks), MARK_THREADS, 0, stream>>>(
                idx, n_idx, demand_limit, page_size, page_shift, page_table, n_logical_pages, n_phys_pages, bitmap, n_words, dev_status);
        JANUS_CUDA_CHECK(cudaGetLastError());
    }
    return launch_page_lists(bitmap, predicted_bitmap, n_words, n_phys_pages, pages, n_pages, runs, n_runs, miss_pages, n_miss, miss_runs,
                             n_miss_runs, capacity, dev_status, stream);
}

extern "C" int janus_page_demand_batch(const int32_t* idx, int64_t n_rows, int k, const int64_t* demand_limits, int page_size,
                                       const int32_t* page_tables, const int64_t* table_offsets, int64_t n_phys_pages,
                                       const uint32_t* predicted_bitmap, uint32_t* bitmap, int32_t* pages, int32_t* n_pages,
                                       int32_t* runs, int32_t* n_runs, int32_t* miss_pages, int32_t* n_miss, int32_t* miss_runs,
                                       int32_t* n_miss_runs, int64_t capacity, int32_t* dev_status, void* stream_) {
    using namespace janus;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (n_rows < 0 || k < 0 || page_size <= 0 || n_phys_pages <= 0 || capacity < 0) return JANUS_ERR_INVALID_ARG;
    if (n_phys_pages > (int64_t(1) << 31) - 64) return JANUS_ERR_UNSUPPORTED;
    if (!bitmap || !pages || !n_pages || !runs || !n_runs) return JANUS_ERR_INVALID_ARG;
    const int n_miss_ptrs = (miss_pages != nullptr) + (n_miss != nullptr) + (miss_runs != nullptr) + (n_miss_runs != nullptr);
    if (n_miss_ptrs != 0 && n_miss_ptrs != 4) return JANUS_ERR_INVALID_ARG;
    const int64_t n_idx = n_rows * static_cast<int64_t>(k);
    if (n_idx > 0 && (!idx || !demand_limits || !page_tables || !table_offsets)) return JANUS_ERR_INVALID_ARG;

    const int n_words = static_cast<int>((n_phys_pages + 31) / 32);
    JANUS_CUDA_CHECK(cudaMemsetAsync(bitmap, 0, sizeof(uint32_t) * n_words, stream));
    if (n_idx > 0) {
        int page_shift = -1;
        if ((page_size & (page_size - 1)) == 0) {
            page_shift = 0;
            while ((1 << page_shift) < page_size) ++page_shift;
        }
        int64_t blocks = (n_idx + MARK_THREADS * 4 - 1) / (MARK_THREADS * 4);
        if (blocks > 148 * 8) blocks = 148 * 8;
        page_mark_rows_kernel<<<static_cast<unsigned>(blocks), MARK_THREADS, 0, stream>>>(idx, n_rows, k, demand_limits, page_size, page_shift,
                                                                                          page_tables, table_offsets, n_phys_pages, bitmap,
                                                                                          dev_status);
        JANUS_CUDA_CHECK(cudaGetLastError());
    }
    return launch_page_lists(bitmap, predicted_bitmap, n_words, n_phys_pages, pages, n_pages, runs, n_runs, miss_pages, n_miss, miss_runs,
                             n_miss_runs, capacity, dev_status, stream);
}
