// Per-token activation quantisers: Eq. 7 (INT4 absmean) and Eq. 8-9 (FP4 E2M1 MinMax); the top-K + INT8
// quantiser of Eq. 1+3 is in quant_topk.cu.
//
// One token row is owned by a group of TPR threads (32..256) of a 256-thread
// block and lives in registers between the reduction and the rounding pass, so
// the row is read from HBM exactly once with 128-bit coalesced loads.  Scales
// are evaluated in float64 so that a code can differ from a float64 CPU
// evaluation only when x*scale sits within rounding noise (~1e-15) of a tie.
#include "internal.h"
#include "quant_common.cuh"

namespace {

using namespace a48q;

// RMSNorm applied in registers: a = fp32(x * r * g), r = 1/sqrt(mean(x^2)+eps) in float64.
template <int TPR, int V>
__device__ __forceinline__ void rmsnorm_inplace(float4 (&v)[V], int t, int nv, int K, const float* gain,
                                                double norm_eps, double* red, int group) {
    double ss = 0.0;
#pragma unroll
    for (int i = 0; i < V; ++i)
        ss += (double)v[i].x * v[i].x + (double)v[i].y * v[i].y + (double)v[i].z * v[i].z + (double)v[i].w * v[i].w;
    ss = group_sum<TPR>(ss, red, group);
    double r = 1.0 / sqrt(ss / (double)K + norm_eps);
    const float4* g4 = reinterpret_cast<const float4*>(gain);
#pragma unroll
    for (int i = 0; i < V; ++i) {
        int idx = i * TPR + t;
        if (idx < nv) {
            float4 g = g4[idx];
            v[i].x = (float)((double)v[i].x * r * (double)g.x);
            v[i].y = (float)((double)v[i].y * r * (double)g.y);
            v[i].z = (float)((double)v[i].z * r * (double)g.z);
            v[i].w = (float)((double)v[i].w * r * (double)g.w);
        }
    }
}

// ---------------------------------------------------------------------------- Eq. 7
// ADD: the row is X + R (a residual connection), formed while loading and written to SUM for the later residual.
// E2M1 grid code of x*2^b (Eq. 8-9 with E = 2, M = 1): the exponent of the binade, floored at 1, sets the step
// 2^(e-1): 1 below 4, 2 in [4, 8), 4 from 8 on; the code is step * round(x*2^b / step), an integer in
// {0, +-1, +-2, +-3, +-4, +-6, +-8, +-12}.  Evaluated in float64 like the rest of the scale arithmetic.
__device__ __forceinline__ int fp4_grid_code(double xp) {
    const double ax = fabs(xp);
    const double inv_step = ax < 4.0 ? 1.0 : (ax < 8.0 ? 0.5 : 0.25), step = ax < 4.0 ? 1.0 : (ax < 8.0 ? 2.0 : 4.0);
    return __double2int_rn(step * rint(xp * inv_step));
}

// FP4 false: Eq. 7 (absmean, codes in [-8, 7]).  FP4 true: Eq. 8-9 (MinMax E2M1, grid codes) with the same
// fused front ends.
template <int TPR, int V, bool NORM, bool ADD, bool FP4 = false, bool BF16IN = false>
__global__ void __launch_bounds__(kBlock) quant_int4_kernel(const float* __restrict__ X, int M, int K, double eps,
                                                            int8_t* __restrict__ codes, float* __restrict__ scale,
                                                            const float* __restrict__ gain, double norm_eps,
                                                            const float* __restrict__ R, float* __restrict__ SUM) {
    constexpr int G = kBlock / TPR;
    __shared__ double red[kBlock / 32];
    a48_pdl_prologue();
    const int group = threadIdx.x / TPR, t = threadIdx.x % TPR;
    const int row = blockIdx.x * G + group;
    if (row >= M) return;
    const int nv = K >> 2;
    const void* xr = row_ptr<BF16IN>(X, (size_t)row, K);
    float4 v[V];
#pragma unroll
    for (int i = 0; i < V; ++i) {
        int idx = i * TPR + t;
        v[i] = idx < nv ? load_row4<BF16IN>(xr, idx) : make_float4(0.f, 0.f, 0.f, 0.f);
        if (ADD && idx < nv) {
            const float4 r = __ldg(reinterpret_cast<const float4*>(R + (size_t)row * K) + idx);
            v[i] = make_float4(v[i].x + r.x, v[i].y + r.y, v[i].z + r.z, v[i].w + r.w);
            reinterpret_cast<float4*>(SUM + (size_t)row * K)[idx] = v[i];
        }
    }
    if (NORM) rmsnorm_inplace<TPR, V>(v, t, nv, K, gain, norm_eps, red, group);
    uint32_t* out = reinterpret_cast<uint32_t*>(codes + (size_t)row * K);
    if constexpr (FP4) {
        float gm = 0.f;
#pragma unroll
        for (int i = 0; i < V; ++i)
            gm = fmaxf(fmaxf(fmaxf(gm, fabsf(v[i].x)), fmaxf(fabsf(v[i].y), fabsf(v[i].z))), fabsf(v[i].w));
        const unsigned gmax = group_max<TPR>(__float_as_uint(gm), reinterpret_cast<unsigned*>(red), group);
        const double amax = (double)__uint_as_float(gmax);
        const double two_b = amax > 0.0 ? 12.0 / amax : 0.0;  // 2^b of Eq. 9
#pragma unroll
        for (int i = 0; i < V; ++i) {
            int idx = i * TPR + t;
            if (idx < nv)
                out[idx] = pack4(fp4_grid_code((double)v[i].x * two_b), fp4_grid_code((double)v[i].y * two_b),
                                 fp4_grid_code((double)v[i].z * two_b), fp4_grid_code((double)v[i].w * two_b));
        }
        if (t == 0) scale[row] = (float)(amax / 12.0);
        return;
    }
    double s = 0.0;
#pragma unroll
    for (int i = 0; i < V; ++i)
        s += (double)fabsf(v[i].x) + (double)fabsf(v[i].y) + (double)fabsf(v[i].z) + (double)fabsf(v[i].w);
    s = group_sum<TPR>(s, red, group);
    const double beta = s / (double)K;
    const double mult = sqrt(7.0) / (beta + eps);
#pragma unroll
    for (int i = 0; i < V; ++i) {
        int idx = i * TPR + t;
        if (idx < nv) {
            int a = clampi(__double2int_rn(mult * (double)v[i].x), -8, 7);
            int b = clampi(__double2int_rn(mult * (double)v[i].y), -8, 7);
            int c = clampi(__double2int_rn(mult * (double)v[i].z), -8, 7);
            int d = clampi(__double2int_rn(mult * (double)v[i].w), -8, 7);
            out[idx] = pack4(a, b, c, d);
        }
    }
    if (t == 0) scale[row] = (float)(beta / sqrt(7.0));
}

// Any K (unaligned or very long rows): one block per row, the row re-read from L2.
template <bool NORM>
__global__ void __launch_bounds__(kBlock) quant_int4_generic_kernel(const float* __restrict__ X, int M, int K,
                                                                    double eps, int8_t* __restrict__ codes,
                                                                    float* __restrict__ scale,
                                                                    const float* __restrict__ gain, double norm_eps) {
    __shared__ double red[kBlock / 32];
    const int row = blockIdx.x;
    const float* xr = X + (size_t)row * K;
    double r = 1.0;
    if (NORM) {
        double ss = 0.0;
        for (int j = threadIdx.x; j < K; j += kBlock) ss += (double)xr[j] * xr[j];
        ss = group_sum<kBlock>(ss, red, 0);
        r = 1.0 / sqrt(ss / (double)K + norm_eps);
    }
    auto val = [&](int j) -> float { return NORM ? (float)((double)xr[j] * r * (double)gain[j]) : xr[j]; };
    double s = 0.0;
    for (int j = threadIdx.x; j < K; j += kBlock) s += (double)fabsf(val(j));
    s = group_sum<kBlock>(s, red, 0);
    const double beta = s / (double)K;
    const double mult = sqrt(7.0) / (beta + eps);
    for (int j = threadIdx.x; j < K; j += kBlock)
        codes[(size_t)row * K + j] = (int8_t)clampi(__double2int_rn(mult * (double)val(j)), -8, 7);
    if (threadIdx.x == 0) scale[row] = (float)(beta / sqrt(7.0));
}

// ---------------------------------------------------------------------------- Eq. 8-9 (E2M1)
template <bool NORM>
__global__ void __launch_bounds__(kBlock) quant_fp4_generic_kernel(const float* __restrict__ X, int M, int K,
                                                                   int8_t* __restrict__ codes, float* __restrict__ scale,
                                                                   const float* __restrict__ gain, double norm_eps) {
    __shared__ double red[kBlock / 32];
    const int row = blockIdx.x, t = threadIdx.x;
    const float* xr = X + (size_t)row * K;
    double r = 1.0;
    if (NORM) {
        double ss = 0.0;
        for (int j = t; j < K; j += kBlock) ss += (double)xr[j] * xr[j];
        ss = group_sum<kBlock>(ss, red, 0);
        r = 1.0 / sqrt(ss / (double)K + norm_eps);
    }
    auto val = [&](int j) -> float { return NORM ? (float)((double)xr[j] * r * (double)gain[j]) : xr[j]; };
    unsigned gmax = 0;
    for (int j = t; j < K; j += kBlock) gmax = max(gmax, __float_as_uint(val(j)) & 0x7fffffffu);
    gmax = group_max<kBlock>(gmax, reinterpret_cast<unsigned*>(red), 0);
    const double amax = (double)__uint_as_float(gmax);
    const double two_b = amax > 0.0 ? 12.0 / amax : 0.0;  // 2^b of Eq. 9 with E=2, M=1
    for (int j = t; j < K; j += kBlock) codes[(size_t)row * K + j] = (int8_t)fp4_grid_code((double)val(j) * two_b);
    if (t == 0) scale[row] = (float)(amax / 12.0);
}

// ---------------------------------------------------------------------------- compacted form of a code row
// The channels with a non-zero code, in ascending channel order, as (index, code) pairs: what a consumer of
// Eq. 1 needs when it skips the masked channels.  One block per row; a thread owns four consecutive channels
// per step, so thread order is channel order and an exclusive scan of the per-thread counts gives the places.
__global__ void __launch_bounds__(kBlock) compact_codes_kernel(const int8_t* __restrict__ codes, int M, int K, int cap,
                                                               uint16_t* __restrict__ idx, int8_t* __restrict__ val,
                                                               int32_t* __restrict__ count) {
    __shared__ unsigned red[kBlock / 32];
    const int row = blockIdx.x, t = threadIdx.x;
    const int8_t* cr = codes + (size_t)row * K;
    const bool words = (K & 3) == 0;  // rows then start on a 4-byte boundary
    unsigned running = 0;
    for (int j0 = 0; j0 < K; j0 += kBlock * 4) {
        const int j = j0 + 4 * t;
        int c[4];
        if (words && j + 3 < K) {
            const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(cr + j));
#pragma unroll
            for (int q = 0; q < 4; ++q) c[q] = (int)(int8_t)(w >> (8 * q));
        } else {
#pragma unroll
            for (int q = 0; q < 4; ++q) c[q] = j + q < K ? (int)cr[j + q] : 0;
        }
        const unsigned cnt = (unsigned)(c[0] != 0) + (c[1] != 0) + (c[2] != 0) + (c[3] != 0);
        unsigned total;
        unsigned at = running + group_excl_scan<kBlock>(cnt, red, 0, total);
        running += total;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            if (c[q] != 0) {
                if (at < (unsigned)cap) {
                    idx[(size_t)row * cap + at] = (uint16_t)(j + q);
                    val[(size_t)row * cap + at] = (int8_t)c[q];
                }
                ++at;
            }
        }
    }
    if (t == 0) count[row] = (int32_t)running;
}

template <bool NORM, bool ADD = false, bool FP4 = false, bool BF16IN = false>
void launch_int4(const float* X, int M, int K, double eps, int8_t* codes, float* scale, const float* gain,
                 double norm_eps, cudaStream_t st, const float* R = nullptr, float* SUM = nullptr) {
    const int nv = K / 4;
    const bool fast = (K % 4 == 0) && nv <= 256 * 12;
#define A48_Q4(TPR, V)                                                                                             \
    a48_launch_pdl(quant_int4_kernel<TPR, V, NORM, ADD, FP4, BF16IN>, dim3((M + (kBlock / TPR) - 1) / (kBlock / TPR)),    \
                   dim3(kBlock), 0, st, X, M, K, eps, codes, scale, gain, norm_eps, R, SUM)
    if (!fast && FP4) quant_fp4_generic_kernel<NORM><<<M, kBlock, 0, st>>>(X, M, K, codes, scale, gain, norm_eps);
    else if (!fast) quant_int4_generic_kernel<NORM><<<M, kBlock, 0, st>>>(X, M, K, eps, codes, scale, gain, norm_eps);
    else if (nv <= 32 * 4) A48_Q4(32, 4);
    else if (nv <= 64 * 4) A48_Q4(64, 4);
    else if (nv <= 128 * 4) A48_Q4(128, 4);
    else if (nv <= 256 * 4) A48_Q4(256, 4);
    else if (nv <= 256 * 8) A48_Q4(256, 8);
    else A48_Q4(256, 12);
#undef A48_Q4
}

}  // namespace

bitnet_a48_status a48_launch_quant_int4(const float* X, int M, int K, float eps, int8_t* codes, float* scale,
                                        const float* gain, float norm_eps, cudaStream_t st) {
    if (gain) launch_int4<true>(X, M, K, (double)eps, codes, scale, gain, (double)norm_eps, st);
    else launch_int4<false>(X, M, K, (double)eps, codes, scale, nullptr, 0.0, st);
    A48_CUDA_TRY(cudaGetLastError());
    return BITNET_A48_OK;
}

bitnet_a48_status a48_launch_quant_int4_bf16(const uint16_t* X, int M, int K, float eps, int8_t* codes, float* scale,
                                             cudaStream_t st) {
    if (!((K % 4 == 0) && K / 4 <= 256 * 12)) return BITNET_A48_ERR_UNSUPPORTED;  // the register kernels only
    launch_int4<false, false, false, true>(reinterpret_cast<const float*>(X), M, K, (double)eps, codes, scale, nullptr, 0.0, st);
    A48_CUDA_TRY(cudaGetLastError());
    return BITNET_A48_OK;
}

// RMSNorm + INT4 of X + R with the sum written to SUM (the residual add fused into the quantiser's load); shapes of
// the register kernels only.
bitnet_a48_status a48_launch_quant_int4_add(const float* X, const float* R, float* SUM, int M, int K, float eps,
                                            int8_t* codes, float* scale, const float* gain, float norm_eps,
                                            cudaStream_t st) {
    if (!((K % 4 == 0) && K / 4 <= 256 * 12) || !gain) return BITNET_A48_ERR_UNSUPPORTED;
    launch_int4<true, true>(X, M, K, (double)eps, codes, scale, gain, (double)norm_eps, st, R, SUM);
    A48_CUDA_TRY(cudaGetLastError());
    return BITNET_A48_OK;
}

// gain != nullptr: RMSNorm in front, as for the INT4 quantiser.
bitnet_a48_status a48_launch_quant_fp4(const float* X, int M, int K, int8_t* codes, float* scale, const float* gain,
                                       float norm_eps, cudaStream_t st) {
    if (gain) launch_int4<true, false, true>(X, M, K, 0.0, codes, scale, gain, (double)norm_eps, st);
    else launch_int4<false, false, true>(X, M, K, 0.0, codes, scale, nullptr, 0.0, st);
    A48_CUDA_TRY(cudaGetLastError());
    return BITNET_A48_OK;
}

// RMSNorm + FP4 of X + R with the sum written to SUM; shapes of the register kernels only.
bitnet_a48_status a48_launch_quant_fp4_add(const float* X, const float* R, float* SUM, int M, int K, int8_t* codes,
                                           float* scale, const float* gain, float norm_eps, cudaStream_t st) {
    if (!((K % 4 == 0) && K / 4 <= 256 * 12) || !gain) return BITNET_A48_ERR_UNSUPPORTED;
    launch_int4<true, true, true>(X, M, K, 0.0, codes, scale, gain, (double)norm_eps, st, R, SUM);
    A48_CUDA_TRY(cudaGetLastError());
    return BITNET_A48_OK;
}

bitnet_a48_status a48_launch_compact_codes(const int8_t* codes, int M, int K, int cap, uint16_t* idx, int8_t* val,
                                           int32_t* count, cudaStream_t st) {
    compact_codes_kernel<<<M, kBlock, 0, st>>>(codes, M, K, cap, idx, val, count);
    A48_CUDA_TRY(cudaGetLastError());
    return BITNET_A48_OK;
}
