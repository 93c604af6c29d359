// Helpers shared by the per-token quantiser kernels: a token row is owned by a group of TPR threads (32..256) of a
// 256-thread block; these are the group-wide barrier, reductions and scan.
#pragma once

#include "internal.h"

namespace a48q {

constexpr int kBlock = 256;

template <int TPR>
__device__ __forceinline__ void group_sync(int group) {
    if (TPR == 32) {
        __syncwarp();
    } else if (TPR == kBlock) {
        __syncthreads();
    } else {
        asm volatile("bar.sync %0, %1;" ::"r"(group + 1), "r"(TPR) : "memory");
    }
}

template <int TPR>
__device__ __forceinline__ double group_sum(double v, double* red, int group) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (TPR == 32) return v;
    constexpr int WPG = TPR / 32;
    int warp = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0) red[warp] = v;
    group_sync<TPR>(group);
    double r = 0.0;
#pragma unroll
    for (int i = 0; i < WPG; ++i) r += red[group * WPG + i];
    group_sync<TPR>(group);
    return r;
}

template <int TPR>
__device__ __forceinline__ unsigned group_max(unsigned v, unsigned* red, int group) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
    if (TPR == 32) return v;
    constexpr int WPG = TPR / 32;
    int warp = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0) red[warp] = v;
    group_sync<TPR>(group);
    unsigned r = 0;
#pragma unroll
    for (int i = 0; i < WPG; ++i) r = max(r, red[group * WPG + i]);
    group_sync<TPR>(group);
    return r;
}

__device__ __forceinline__ int clampi(int v, int lo, int hi) { return v < lo ? lo : (v > hi ? hi : v); }

__device__ __forceinline__ uint32_t pack4(int a, int b, int c, int d) {
    return (uint32_t)(a & 0xff) | ((uint32_t)(b & 0xff) << 8) | ((uint32_t)(c & 0xff) << 16) |
           ((uint32_t)(d & 0xff) << 24);
}

// Exclusive scan of cnt over the TPR threads of a group in thread order; returns
// the exclusive prefix and the group total.
template <int TPR>
__device__ __forceinline__ unsigned group_excl_scan(unsigned cnt, unsigned* red, int group, unsigned& total) {
    const int lane = threadIdx.x & 31;
    unsigned incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        unsigned n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
    }
    if (TPR == 32) {
        total = __shfl_sync(0xffffffffu, incl, 31);
        return incl - cnt;
    }
    constexpr int WPG = TPR / 32;
    const int warp = threadIdx.x >> 5;
    if (lane == 31) red[warp] = incl;
    group_sync<TPR>(group);
    unsigned base = 0, tot = 0;
#pragma unroll
    for (int i = 0; i < WPG; ++i) {
        unsigned w = red[group * WPG + i];
        if (group * WPG + i < warp) base += w;
        tot += w;
    }
    group_sync<TPR>(group);
    total = tot;
    return base + incl - cnt;
}

// Four consecutive entries of a row that is fp32 or (BF16) bf16 in memory; `row` is the row's first byte.  A bf16
// value widens to fp32 exactly: its 16 bits are the upper half of the fp32 pattern.
template <bool BF16>
__device__ __forceinline__ float4 load_row4(const void* row, int idx) {
    if (BF16) {
        const uint2 u = __ldg(reinterpret_cast<const uint2*>(row) + idx);
        return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u), __uint_as_float(u.y << 16),
                           __uint_as_float(u.y & 0xffff0000u));
    }
    return __ldg(reinterpret_cast<const float4*>(row) + idx);
}
template <bool BF16>
__device__ __forceinline__ const void* row_ptr(const void* X, size_t row, int K) {
    return reinterpret_cast<const char*>(X) + row * (size_t)K * (BF16 ? 2 : 4);
}

}  // namespace a48q
