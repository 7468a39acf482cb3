// Diagnostics with no counterpart in the paper: a self-test of the bounded in-kernel wait every tensor-core kernel of
// this library relies on, and a probe of the dense FP8 tensor rate (the denominator of the indexer's roofline).
#include "janus_common.cuh"
#include "sm100_ptx.cuh"

namespace janus {

using namespace ptx;

// One thread waits on an mbarrier nobody ever arrives on, with the limit the caller gives, and reports the time-out the
// way the product kernels do: status word, then a normal return.
__global__ void bounded_wait_selftest_kernel(uint32_t max_polls, unsigned long long* elapsed_ns, int32_t* dev_status) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        fence_mbar_init();
        unsigned long long t0, t1;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
        const bool ok = mbar_wait(smem_u32(&bar), 0, max_polls);
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
        if (elapsed_ns != nullptr) *elapsed_ns = t1 - t0;
        if (!ok) report(dev_status, JANUS_DEV_WAIT_TIMEOUT);
    }
}

// Dense FP8 (E4M3 x E4M3, fp32 accumulate) tcgen05 loop: each CTA keeps four 128 x 128-byte A tiles and four 256 x 128-byte B
// tiles in shared memory (128-byte swizzle, the indexer's operand shapes) and issues M = 128, N = 256, K = 32 instructions
// back to back into the two halves of tensor memory; nothing reads the accumulators.  2 * 128 * 256 * 128 flop per fill.
// Consecutive fills take different operand tiles (16 combinations in turn), so that the figure does not rest on one fixed
// bit pattern going through the datapath (it made no difference when measured: 3260-3280 TFLOP/s sustained either way).
constexpr int PROBE_THREADS = 64;
constexpr int PROBE_SETS = 4;
constexpr int PROBE_A_BYTES = 128 * 128, PROBE_B_BYTES = 256 * 128;

__global__ void __launch_bounds__(PROBE_THREADS, 1) fp8_mma_probe_kernel(int fills, int32_t* dev_status) {
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ uint64_t done[2];
    __shared__ uint32_t tmem_base_s;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if ((smem_u32(smem) & 1023u) != 0u) {
        if (threadIdx.x == 0) report(dev_status, JANUS_DEV_WAIT_TIMEOUT);
        return;
    }
    // operand bytes: a fixed pseudo-random pattern of finite E4M3 codes (bit 3 cleared: never the NaN code S.1111.111)
    for (int i = threadIdx.x; i < PROBE_SETS * (PROBE_A_BYTES + PROBE_B_BYTES) / 4; i += PROBE_THREADS) {
        uint32_t v = (static_cast<uint32_t>(i) * 2654435761u) ^ (blockIdx.x * 40503u);
        v ^= v >> 13;
        reinterpret_cast<uint32_t*>(smem)[i] = v & 0xf7f7f7f7u;
    }
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&done[0]), 1);
        mbar_init(smem_u32(&done[1]), 1);
        fence_mbar_init();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_s), 512);
        tmem_relinquish();
    }
    fence_proxy_async();     // the tensor core reads the bytes written above through the async proxy
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    if (warp == 1 && lane == 0) {
        const uint32_t idesc = umma_idesc(0u, 128, 256);
        const uint64_t adesc0 = umma_desc_sw128(smem_u32(smem)), bdesc0 = umma_desc_sw128(smem_u32(smem + PROBE_SETS * PROBE_A_BYTES));
        bool ok = true;
        for (int f = 0; f < fills && ok; ++f) {
            const uint32_t slot = f & 1u, use = static_cast<uint32_t>(f) >> 1;
            // at most two fills are in flight: wait for the fill that used this half before
            if (f >= 2) ok = mbar_wait(smem_u32(&done[slot]), (use & 1u) ^ 1u);
            if (!ok) break;
            tc_fence_after();
            const uint64_t adesc = adesc0 + static_cast<uint64_t>(((f & 3) * PROBE_A_BYTES) >> 4);
            const uint64_t bdesc = bdesc0 + static_cast<uint64_t>((((f >> 2) & 3) * PROBE_B_BYTES) >> 4);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) umma<true>(tmem_base + slot * 256, adesc + 2 * ks, bdesc + 2 * ks, idesc, ks > 0 ? 1u : 0u);
            umma_commit(smem_u32(&done[slot]));
        }
        // every issued instruction has completed before tensor memory goes back
        for (int f = max(0, fills - 2); f < fills && ok; ++f) ok = mbar_wait(smem_u32(&done[f & 1]), (static_cast<uint32_t>(f) >> 1) & 1u);
        if (!ok) report(dev_status, JANUS_DEV_WAIT_TIMEOUT);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace janus

extern "C" int janus_selftest_bounded_wait(int max_polls, int64_t* elapsed_ns, int32_t* dev_status, void* stream_) {
    using namespace janus;
    if (max_polls < 1 || max_polls > (1 << 16)) return JANUS_ERR_INVALID_ARG;     // the self-test itself stays short
    bounded_wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream_)>>>(static_cast<uint32_t>(max_polls),
                                                                                  reinterpret_cast<unsigned long long*>(elapsed_ns), dev_status);
    JANUS_CUDA_CHECK(cudaGetLastError());
    return JANUS_OK;
}

extern "C" int janus_fp8_mma_probe(int n_ctas, int fills_per_cta, double* flop_per_launch, int32_t* dev_status, void* stream_) {
    using namespace janus;
    if (n_ctas < 1 || n_ctas > 65535 || fills_per_cta < 1 || fills_per_cta > (1 << 24)) return JANUS_ERR_INVALID_ARG;
    const size_t smem = static_cast<size_t>(PROBE_SETS) * (PROBE_A_BYTES + PROBE_B_BYTES);
    JANUS_CUDA_CHECK(cudaFuncSetAttribute(fp8_mma_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    fp8_mma_probe_kernel<<<n_ctas, PROBE_THREADS, smem, static_cast<cudaStream_t>(stream_)>>>(fills_per_cta, dev_status);
    JANUS_CUDA_CHECK(cudaGetLastError());
    if (flop_per_launch != nullptr) *flop_per_launch = 2.0 * 128 * 256 * 128 * static_cast<double>(fills_per_cta) * n_ctas;
    return JANUS_OK;
}
