// Per-token activation quantisers: Eq. 7 (INT4 absmean), Eq. 1+3 (top-K + INT8
// absmax) and Eq. 8-9 (FP4 E2M1 MinMax).
//
// One token row is owned by a group of TPR threads (32..256) of a 256-thread
// block and lives in registers between the reduction and the rounding pass, so
// the row is read from HBM exactly once with 128-bit coalesced loads.  Scales
// are evaluated in float64 so that a code can differ from a float64 CPU
// evaluation only when x*scale sits within rounding noise (~1e-15) of a tie.
#include "internal.h"

namespace {

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
template <int TPR, int V, bool NORM, bool ADD>
__global__ void __launch_bounds__(kBlock) quant_int4_kernel(const float* __restrict__ X, int M, int K, double eps,
                                                            int8_t* __restrict__ codes, float* __restrict__ scale,
                                                            const float* __restrict__ gain, double norm_eps,
                                                            const float* __restrict__ R, float* __restrict__ SUM) {
    constexpr int G = kBlock / TPR;
    __shared__ double red[kBlock / 32];
    const int group = threadIdx.x / TPR, t = threadIdx.x % TPR;
    const int row = blockIdx.x * G + group;
    if (row >= M) return;
    const int nv = K >> 2;
    const float4* xr = reinterpret_cast<const float4*>(X + (size_t)row * K);
    float4 v[V];
#pragma unroll
    for (int i = 0; i < V; ++i) {
        int idx = i * TPR + t;
        v[i] = idx < nv ? __ldg(xr + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
        if (ADD && idx < nv) {
            const float4 r = __ldg(reinterpret_cast<const float4*>(R + (size_t)row * K) + idx);
            v[i] = make_float4(v[i].x + r.x, v[i].y + r.y, v[i].z + r.z, v[i].w + r.w);
            reinterpret_cast<float4*>(SUM + (size_t)row * K)[idx] = v[i];
        }
    }
    if (NORM) rmsnorm_inplace<TPR, V>(v, t, nv, K, gain, norm_eps, red, group);
    double s = 0.0;
#pragma unroll
    for (int i = 0; i < V; ++i)
        s += (double)fabsf(v[i].x) + (double)fabsf(v[i].y) + (double)fabsf(v[i].z) + (double)fabsf(v[i].w);
    s = group_sum<TPR>(s, red, group);
    const double beta = s / (double)K;
    const double mult = sqrt(7.0) / (beta + eps);
    uint32_t* out = reinterpret_cast<uint32_t*>(codes + (size_t)row * K);
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

// ---------------------------------------------------------------------------- Eq. 1 + 3
// Finds, for one row, the 31-bit key tau of the k-th largest |x| by an 8-bit
// radix select (4 passes over the keys held in registers or re-read from
// memory), and how many entries equal to tau are kept (keep_eq) out of eq_total.
struct Select {
    unsigned tau, keep_eq, eq_total;
};

// hist: 256 bins of this group; sel: 2 words of this group.
// for_each_key(f) calls f(key) for every valid element owned by the thread.
template <int TPR, class ForEachKey>
__device__ __forceinline__ Select radix_select(int k, unsigned* hist, unsigned* sel, int group, int t,
                                               ForEachKey for_each_key) {
    unsigned prefix = 0, kr = (unsigned)k, eq_total = 0;
#pragma unroll 1
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        for (int b = t; b < 256; b += TPR) hist[b] = 0;
        group_sync<TPR>(group);
        for_each_key([&](unsigned u) {
            if (pass == 0 || (u >> (shift + 8)) == prefix) atomicAdd(&hist[(u >> shift) & 255u], 1u);
        });
        group_sync<TPR>(group);
        if (t < 32) {
            // lane l owns bins 255-8l-7 .. 255-8l; lanes ascend as digits descend
            unsigned h[8], c = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                h[i] = hist[255 - 8 * t - i];
                c += h[i];
            }
            unsigned incl = c;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                unsigned n = __shfl_up_sync(0xffffffffu, incl, o);
                if (t >= o) incl += n;
            }
            unsigned excl = incl - c;
            if (incl >= kr && excl < kr) {
                unsigned cum = excl;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (cum < kr && cum + h[i] >= kr) {
                        sel[0] = 255 - 8 * t - i;
                        sel[1] = kr - cum;
                        sel[2] = h[i];
                    }
                    cum += h[i];
                }
            }
        }
        group_sync<TPR>(group);
        prefix = (prefix << 8) | sel[0];
        kr = sel[1];
        eq_total = sel[2];
        // the next pass clears hist only after this sync, and sel is rewritten
        // only after the next two syncs, so no extra barrier is needed here
    }
    return Select{prefix, kr, eq_total};
}

// The same selection for a whole block working on one row, with far fewer instructions per element: the first
// pass (the 8 exponent bits) runs over the registers as above; the elements of the chosen binade - about a third
// of a row of real data - are then copied into shared memory, and the three remaining passes (8, 8 and 7 mantissa
// bits) walk that list instead of testing every element of the row again.
// The first pass and the copy take the raw float bits: sign and exponent together index 512 bins (one shift per
// element; the two halves are added when the bins are scanned), and the binade test is a mask and a compare.
// hist: 512 bins; sel: 4 words; cand: room for every key of the row.
template <class ForEachRaw>
__device__ __forceinline__ Select radix_select_compact(int k, unsigned* hist, unsigned* sel, unsigned* cand, int t,
                                                       ForEachRaw for_each_raw) {
    unsigned prefix = 0, kr = (unsigned)k, eq_total = 0, n_cand = 0;
#pragma unroll 1
    for (int pass = 0; pass < 4; ++pass) {
        const int bits = pass == 3 ? 7 : 8;
        const int shift = pass == 0 ? 23 : (pass == 1 ? 15 : (pass == 2 ? 7 : 0));
        hist[t] = 0;
        if (pass == 0) hist[t + 256] = 0;
        if (pass == 0 && t == 0) sel[3] = 0;
        __syncthreads();
        if (pass == 0) {
            for_each_raw([&](unsigned r) { atomicAdd(&hist[r >> 23], 1u); });
        } else {
            for (unsigned j = t; j < n_cand; j += kBlock) {
                const unsigned u = cand[j];
                if ((u >> (shift + bits)) == prefix) atomicAdd(&hist[(u >> shift) & ((1u << bits) - 1u)], 1u);
            }
        }
        __syncthreads();
        if (t < 32) {
            // lane l owns bins 255-8l-7 .. 255-8l; lanes ascend as digits descend
            unsigned h[8], c = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                h[i] = hist[255 - 8 * t - i];
                if (pass == 0) h[i] += hist[511 - 8 * t - i];  // the same binade with the sign bit set
                c += h[i];
            }
            unsigned incl = c;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                unsigned n = __shfl_up_sync(0xffffffffu, incl, o);
                if (t >= o) incl += n;
            }
            unsigned excl = incl - c;
            if (incl >= kr && excl < kr) {
                unsigned cum = excl;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (cum < kr && cum + h[i] >= kr) {
                        sel[0] = 255 - 8 * t - i;
                        sel[1] = kr - cum;
                        sel[2] = h[i];
                    }
                    cum += h[i];
                }
            }
        }
        __syncthreads();
        prefix = (prefix << bits) | sel[0];
        kr = sel[1];
        eq_total = sel[2];
        if (pass == 0) {
            // this thread's elements of the chosen binade go to a range of the list reserved with one atomic
            const unsigned binade = prefix << 23;
            unsigned mine = 0;
            for_each_raw([&](unsigned r) { mine += (r & 0x7f800000u) == binade; });
            unsigned pos = mine ? atomicAdd(&sel[3], mine) : 0u;
            for_each_raw([&](unsigned r) {
                if ((r & 0x7f800000u) == binade) cand[pos++] = r & 0x7fffffffu;
            });
            __syncthreads();
            n_cand = sel[3];
        }
    }
    return Select{prefix, kr, eq_total};
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

// GLU: the row to quantise is up * ReLU(gate)^2 (Eq. 5), formed while loading: X is the gate projection and U the up
// projection, and the product never goes to memory.
template <int TPR, int V, bool GLU>
__global__ void __launch_bounds__(kBlock, V >= 8 ? 4 : 6)
    topk_quant_int8_kernel(const float* __restrict__ X, const float* __restrict__ U, int M, int K, int k, double eps,
                           int8_t* __restrict__ codes, float* __restrict__ scale, uint32_t* __restrict__ mask_bits) {
    constexpr int G = kBlock / TPR;
    constexpr bool ONE_ROW = TPR == kBlock;  // the block owns one row: candidate list in dynamic shared memory
    __shared__ unsigned hist[ONE_ROW ? 512 : G * 256];
    __shared__ unsigned sel[G][4];
    __shared__ unsigned red[kBlock / 32];
    extern __shared__ unsigned cand[];  // K words when ONE_ROW
    const int group = threadIdx.x / TPR, t = threadIdx.x % TPR;
    const int row = blockIdx.x * G + group;
    if (row >= M) return;
    const int nv = K >> 2;
    const float4* xr = reinterpret_cast<const float4*>(X + (size_t)row * K);
    float4 v[V];
#pragma unroll
    for (int i = 0; i < V; ++i) {
        int idx = i * TPR + t;
        v[i] = idx < nv ? __ldg(xr + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
        if (GLU && idx < nv) {
            const float4 u = __ldg(reinterpret_cast<const float4*>(U + (size_t)row * K) + idx);
            auto f = [](float gg, float uu) { float r = gg > 0.f ? gg : 0.f; return uu * (r * r); };
            v[i] = make_float4(f(v[i].x, u.x), f(v[i].y, u.y), f(v[i].z, u.z), f(v[i].w, u.w));
        }
    }
    auto key = [](float f) { return __float_as_uint(f) & 0x7fffffffu; };

    float gm = 0.f;  // max |x| as a float maximum (one instruction per element); its bits are the largest key
#pragma unroll
    for (int i = 0; i < V; ++i)
        gm = fmaxf(fmaxf(fmaxf(gm, fabsf(v[i].x)), fmaxf(fabsf(v[i].y), fabsf(v[i].z))), fabsf(v[i].w));
    unsigned gmax = group_max<TPR>(__float_as_uint(gm), red, group);
    const double gamma = (double)__uint_as_float(gmax);
    const double mult = 127.0 / (gamma + eps);

    auto for_each_key = [&](auto f) {
#pragma unroll
        for (int i = 0; i < V; ++i) {
            if (i * TPR + t < nv) {
                f(key(v[i].x));
                f(key(v[i].y));
                f(key(v[i].z));
                f(key(v[i].w));
            }
        }
    };
    auto for_each_raw = [&](auto f) {
#pragma unroll
        for (int i = 0; i < V; ++i) {
            if (i * TPR + t < nv) {
                f(__float_as_uint(v[i].x));
                f(__float_as_uint(v[i].y));
                f(__float_as_uint(v[i].z));
                f(__float_as_uint(v[i].w));
            }
        }
    };
    Select s;
    if constexpr (ONE_ROW) s = radix_select_compact(k, hist, sel[0], cand, t, for_each_raw);
    else s = radix_select<TPR>(k, hist + group * 256, sel[group], group, t, for_each_key);
    const bool ordered = s.eq_total != s.keep_eq;  // a tie straddles the k-th place: lowest indices win
    unsigned running = 0;
    uint32_t* out = reinterpret_cast<uint32_t*>(codes + (size_t)row * K);
    const int mask_words = (K + 31) >> 5;
    if (!ordered && !mask_bits) {
        // The usual case (uniform over the row's threads): every entry equal to tau is kept, so the mask is one
        // comparison, and no bitmap is wanted.  The clip of Eq. 3 is left out here: |127 x / (gamma + eps)| <= 127
        // for every finite x of the row, so it cannot fire.
#pragma unroll
        for (int i = 0; i < V; ++i) {
            const int idx = i * TPR + t;
            if (idx < nv) {
                const int a = key(v[i].x) >= s.tau ? __double2int_rn(mult * (double)v[i].x) : 0;
                const int b = key(v[i].y) >= s.tau ? __double2int_rn(mult * (double)v[i].y) : 0;
                const int c = key(v[i].z) >= s.tau ? __double2int_rn(mult * (double)v[i].z) : 0;
                const int d = key(v[i].w) >= s.tau ? __double2int_rn(mult * (double)v[i].w) : 0;
                out[idx] = pack4(a, b, c, d);
            }
        }
        if (t == 0) scale[row] = (float)(gamma / 127.0);
        return;
    }
#pragma unroll
    for (int i = 0; i < V; ++i) {
        const int idx = i * TPR + t;
        const bool valid = idx < nv;
        const unsigned u0 = key(v[i].x), u1 = key(v[i].y), u2 = key(v[i].z), u3 = key(v[i].w);
        const bool e0 = valid && u0 == s.tau, e1 = valid && u1 == s.tau, e2 = valid && u2 == s.tau,
                   e3 = valid && u3 == s.tau;
        bool k0 = valid && u0 > s.tau, k1 = valid && u1 > s.tau, k2 = valid && u2 > s.tau, k3 = valid && u3 > s.tau;
        if (!ordered) {
            k0 |= e0; k1 |= e1; k2 |= e2; k3 |= e3;
        } else {
            unsigned cnt = (unsigned)e0 + e1 + e2 + e3, total;
            unsigned base = running + group_excl_scan<TPR>(cnt, red, group, total);
            running += total;
            k0 |= e0 && base < s.keep_eq; base += e0;
            k1 |= e1 && base < s.keep_eq; base += e1;
            k2 |= e2 && base < s.keep_eq; base += e2;
            k3 |= e3 && base < s.keep_eq;
        }
        if (valid) {
            int a = k0 ? clampi(__double2int_rn(mult * (double)v[i].x), -128, 127) : 0;
            int b = k1 ? clampi(__double2int_rn(mult * (double)v[i].y), -128, 127) : 0;
            int c = k2 ? clampi(__double2int_rn(mult * (double)v[i].z), -128, 127) : 0;
            int d = k3 ? clampi(__double2int_rn(mult * (double)v[i].w), -128, 127) : 0;
            out[idx] = pack4(a, b, c, d);
        }
        if (mask_bits) {  // uniform across the group
            unsigned nib = ((unsigned)k0 | (unsigned)k1 << 1 | (unsigned)k2 << 2 | (unsigned)k3 << 3) << (4 * (t & 7));
            nib |= __shfl_xor_sync(0xffffffffu, nib, 1);
            nib |= __shfl_xor_sync(0xffffffffu, nib, 2);
            nib |= __shfl_xor_sync(0xffffffffu, nib, 4);
            int word = idx >> 3;
            if ((t & 7) == 0 && word < mask_words) mask_bits[(size_t)row * mask_words + word] = nib;
        }
    }
    if (t == 0) scale[row] = (float)(gamma / 127.0);
}

__global__ void __launch_bounds__(kBlock)
    topk_quant_int8_generic_kernel(const float* __restrict__ X, int M, int K, int k, double eps,
                                   int8_t* __restrict__ codes, float* __restrict__ scale,
                                   uint32_t* __restrict__ mask_bits) {
    __shared__ unsigned hist[256];
    __shared__ unsigned sel[4];
    __shared__ unsigned red[kBlock / 32];
    const int row = blockIdx.x, t = threadIdx.x;
    const float* xr = X + (size_t)row * K;
    auto key = [](float f) { return __float_as_uint(f) & 0x7fffffffu; };
    unsigned gmax = 0;
    for (int j = t; j < K; j += kBlock) gmax = max(gmax, key(xr[j]));
    gmax = group_max<kBlock>(gmax, red, 0);
    const double gamma = (double)__uint_as_float(gmax);
    const double mult = 127.0 / (gamma + eps);
    Select s = radix_select<kBlock>(k, hist, sel, 0, t, [&](auto f) {
        for (int j = t; j < K; j += kBlock) f(key(xr[j]));
    });
    const int mask_words = (K + 31) >> 5;
    unsigned running = 0;
    for (int j0 = 0; j0 < K; j0 += kBlock) {  // index order: chunk-major, then thread
        const int j = j0 + t;
        const bool valid = j < K;
        const unsigned u = valid ? key(xr[j]) : 0u;
        const bool eq = valid && u == s.tau;
        bool keep = valid && u > s.tau;
        unsigned total;
        unsigned base = running + group_excl_scan<kBlock>((unsigned)eq, red, 0, total);
        running += total;
        keep |= eq && base < s.keep_eq;
        if (valid) codes[(size_t)row * K + j] = (int8_t)(keep ? clampi(__double2int_rn(mult * (double)xr[j]), -128, 127) : 0);
        if (mask_bits) {
            unsigned bits = __ballot_sync(0xffffffffu, keep);
            if ((t & 31) == 0 && (j >> 5) < mask_words) mask_bits[(size_t)row * mask_words + (j >> 5)] = bits;
        }
    }
    if (t == 0) scale[row] = (float)(gamma / 127.0);
}

// ---------------------------------------------------------------------------- Eq. 8-9 (E2M1)
__global__ void __launch_bounds__(kBlock) quant_fp4_generic_kernel(const float* __restrict__ X, int M, int K,
                                                                   int8_t* __restrict__ codes,
                                                                   float* __restrict__ scale) {
    __shared__ unsigned red[kBlock / 32];
    const int row = blockIdx.x, t = threadIdx.x;
    const float* xr = X + (size_t)row * K;
    unsigned gmax = 0;
    for (int j = t; j < K; j += kBlock) gmax = max(gmax, __float_as_uint(xr[j]) & 0x7fffffffu);
    gmax = group_max<kBlock>(gmax, red, 0);
    const double amax = (double)__uint_as_float(gmax);
    const double two_b = amax > 0.0 ? 12.0 / amax : 0.0;  // 2^b of Eq. 9 with E=2, M=1
    for (int j = t; j < K; j += kBlock) {
        double xp = (double)xr[j] * two_b;
        double ax = fabs(xp);
        int e = ax > 0.0 ? max(ilogb(ax), 1) : 1;  // exponent of the binade, floored at 1
        double step = ldexp(1.0, e - 1);
        codes[(size_t)row * K + j] = (int8_t)__double2int_rn(step * rint(xp / step));
    }
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

template <bool NORM, bool ADD = false>
void launch_int4(const float* X, int M, int K, double eps, int8_t* codes, float* scale, const float* gain,
                 double norm_eps, cudaStream_t st, const float* R = nullptr, float* SUM = nullptr) {
    const int nv = K / 4;
    const bool fast = (K % 4 == 0) && nv <= 256 * 12;
#define A48_Q4(TPR, V)                                                                                           \
    quant_int4_kernel<TPR, V, NORM, ADD><<<(M + (kBlock / TPR) - 1) / (kBlock / TPR), kBlock, 0, st>>>(         \
        X, M, K, eps, codes, scale, gain, norm_eps, R, SUM)
    if (!fast) quant_int4_generic_kernel<NORM><<<M, kBlock, 0, st>>>(X, M, K, eps, codes, scale, gain, norm_eps);
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

template <bool GLU>
bitnet_a48_status launch_topk(const float* X, const float* U, int M, int K, int k, double e, int8_t* codes, float* scale,
                              uint32_t* mask_bits, cudaStream_t st) {
    const int nv = K / 4;
#define A48_TK(TPR, V)                                                                                              \
    do {                                                                                                            \
        const size_t dyn = TPR == kBlock ? (size_t)K * sizeof(unsigned) : 0; /* candidate list of the one-row kernels */ \
        if (dyn > 40 * 1024)                                                                                        \
            cudaFuncSetAttribute(topk_quant_int8_kernel<TPR, V, GLU>, cudaFuncAttributeMaxDynamicSharedMemorySize,  \
                                 64 * 1024);                                                                        \
        topk_quant_int8_kernel<TPR, V, GLU><<<(M + (kBlock / TPR) - 1) / (kBlock / TPR), kBlock, dyn, st>>>(         \
            X, U, M, K, k, e, codes, scale, mask_bits);                                                             \
    } while (0)
    if (nv <= 32 * 4) A48_TK(32, 4);
    else if (nv <= 64 * 4) A48_TK(64, 4);
    else if (nv <= 128 * 4) A48_TK(128, 4);
    else if (nv <= 256 * 4) A48_TK(256, 4);
    else if (nv <= 256 * 8) A48_TK(256, 8);
    else A48_TK(256, 12);
#undef A48_TK
    A48_CUDA_TRY(cudaGetLastError());
    return BITNET_A48_OK;
}

bool a48_topk_quant_fast_shape(int K) { return (K % 4 == 0) && K / 4 <= 256 * 12; }

bitnet_a48_status a48_launch_topk_quant_int8(const float* X, int M, int K, int k, float eps, int8_t* codes,
                                             float* scale, uint32_t* mask_bits, cudaStream_t st) {
    if (a48_topk_quant_fast_shape(K)) return launch_topk<false>(X, nullptr, M, K, k, (double)eps, codes, scale, mask_bits, st);
    topk_quant_int8_generic_kernel<<<M, kBlock, 0, st>>>(X, M, K, k, (double)eps, codes, scale, mask_bits);
    A48_CUDA_TRY(cudaGetLastError());
    return BITNET_A48_OK;
}

// Top-K + INT8 of up * ReLU(gate)^2 (Eq. 5 fused into the quantiser's load); shapes of the register kernels only.
bitnet_a48_status a48_launch_topk_quant_int8_glu(const float* gate, const float* up, int M, int K, int k, float eps,
                                                 int8_t* codes, float* scale, cudaStream_t st) {
    if (!a48_topk_quant_fast_shape(K)) return BITNET_A48_ERR_UNSUPPORTED;
    return launch_topk<true>(gate, up, M, K, k, (double)eps, codes, scale, nullptr, st);
}

bitnet_a48_status a48_launch_quant_fp4(const float* X, int M, int K, int8_t* codes, float* scale, cudaStream_t st) {
    quant_fp4_generic_kernel<<<M, kBlock, 0, st>>>(X, M, K, codes, scale);
    A48_CUDA_TRY(cudaGetLastError());
    return BITNET_A48_OK;
}

bitnet_a48_status a48_launch_compact_codes(const int8_t* codes, int M, int K, int cap, uint16_t* idx, int8_t* val,
                                           int32_t* count, cudaStream_t st) {
    compact_codes_kernel<<<M, kBlock, 0, st>>>(codes, M, K, cap, idx, val, count);
    A48_CUDA_TRY(cudaGetLastError());
    return BITNET_A48_OK;
}
