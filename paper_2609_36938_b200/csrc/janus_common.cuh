// Shared host/device helpers of the janus kernels (status words, format decode, small scans).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp8.h>
#include <stdint.h>

#include "../../include/janus.h"

namespace janus {

// ---- host-side error bookkeeping -------------------------------------------------------------
void set_last_cuda_error(cudaError_t e);

#define JANUS_CUDA_CHECK(expr)                         \
    do {                                               \
        cudaError_t _e = (expr);                       \
        if (_e != cudaSuccess) {                       \
            janus::set_last_cuda_error(_e);            \
            return JANUS_ERR_CUDA;                     \
        }                                              \
    } while (0)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ---- device-side status word: first error wins ------------------------------------------------
__device__ __forceinline__ void report(int32_t* dev_status, int code) {
    if (dev_status != nullptr) atomicCAS(dev_status, 0, code);
}

// ---- storage formats ----------------------------------------------------------------------------
__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }

__device__ __forceinline__ float e4m3_to_float(uint8_t c) {
    __half_raw h = __nv_cvt_fp8_to_halfraw(static_cast<__nv_fp8_storage_t>(c), __NV_E4M3);
    return __half2float(__half(h));
}

// fp32 -> key whose unsigned order is the float order (larger float, larger key)
__device__ __forceinline__ uint32_t float_to_key(float x) {
    uint32_t u = __float_as_uint(x);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_to_float(uint32_t k) {
    uint32_t u = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
    return __uint_as_float(u);
}

// ---- block-wide exclusive scan of one int per thread (THREADS a multiple of 32, <= 1024) ---------
// `warp_sums` is shared scratch of at least 33 ints.  Returns the exclusive prefix; *total = block sum.
template <int THREADS>
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_sums, int* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        int y = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += y;
    }
    __syncthreads();  // protect warp_sums from a previous use
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int s = (lane < THREADS / 32) ? warp_sums[lane] : 0;
        int si = s;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            int y = __shfl_up_sync(0xffffffffu, si, d);
            if (lane >= d) si += y;
        }
        if (lane < THREADS / 32) warp_sums[lane] = si - s;  // exclusive offset of each warp
        if (lane == 31) warp_sums[32] = si;                  // block total
    }
    __syncthreads();
    *total = warp_sums[32];
    return warp_sums[warp] + incl - v;
}

// The same for three ints per thread at once (one set of barriers instead of three).  `warp_sums` holds 3 x 33 ints.
template <int THREADS>
__device__ __forceinline__ void block_exclusive_scan3(int (&v)[3], int* warp_sums, int (&excl)[3], int (&total)[3]) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl[3] = {v[0], v[1], v[2]};
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
#pragma unroll
        for (int q = 0; q < 3; ++q) {
            const int y = __shfl_up_sync(0xffffffffu, incl[q], d);
            if (lane >= d) incl[q] += y;
        }
    }
    __syncthreads();  // protect warp_sums from a previous use
    if (lane == 31) {
#pragma unroll
        for (int q = 0; q < 3; ++q) warp_sums[33 * q + warp] = incl[q];
    }
    __syncthreads();
    if (warp < 3) {   // warp q scans the warp totals of value q
        const int q = warp;
        const int sv = (lane < THREADS / 32) ? warp_sums[33 * q + lane] : 0;
        int si = sv;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, si, d);
            if (lane >= d) si += y;
        }
        if (lane < THREADS / 32) warp_sums[33 * q + lane] = si - sv;
        if (lane == 31) warp_sums[33 * q + 32] = si;
    }
    __syncthreads();
#pragma unroll
    for (int q = 0; q < 3; ++q) {
        total[q] = warp_sums[33 * q + 32];
        excl[q] = warp_sums[33 * q + warp] + incl[q] - v[q];
    }
}

}  // namespace janus
