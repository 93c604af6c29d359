// Sparsify-then-quantise for the intermediate states, Eq. 1 and 3: per token gamma = max|x|, the mask of the k
// largest |x| (ties: lowest index first), codes = RoundClip(127 x / (gamma + eps), -128, 127) where kept, else 0.
//
// One token row is owned by a group of TPR threads (32..256) of a 256-thread block and lives in registers from
// its single 128-bit coalesced load to the store of the codes.  What bounds such a kernel on this machine is not
// HBM but (a) shared-memory atomics, which cost about a clock per distinct address of a warp's request, and (b)
// the integer/compare pipe, which runs at half the rate of the float pipe.  The selection is therefore arranged so
// that few entries touch a bin of their own and most arithmetic is float multiply-add:
//   pass 0  histogram of the exponent bits (raw bits index 512 bins, the sign halves are folded in the scan);
//           real rows hit a handful of bins, and a warp's increments of one bin are merged by the hardware.
//           This locates the binade of the k-th largest |x| and its rank inside the binade.
//   pass 1  a window of 254 equal-width bins is laid around the value that linear interpolation inside the binade
//           predicts for that rank (+-16 % of the binade); every entry goes to bin rne(255*sat((|x|-lo)/(hi-lo))) -
//           three float instructions and an integer multiply-add for the address - so entries outside the window
//           (about 90 % of the row) land in the two end bins and are merged.  Because the top bin counts everything
//           above the window, a scan from the top with the row's own k gives the exact bin of the k-th entry and its
//           rank in that bin.  Every step of the bin function rounds monotonically, so a bin is an interval of |x|;
//           its two end points are found as floats by evaluating the same function around the analytic estimate.
//   codes   every entry at or above the bin's lower end gets its code; the few entries inside the bin are listed
//           on the way, one warp then ranks them by (|x| descending, index ascending) and clears the codes of those
//           that lose, which settles ties exactly.
// If the k-th entry's code is zero anyway (everything at or below its binade quantises to 0, as in rows that are
// mostly zeros after ReLU^2) no selection is needed at all.  If the window misses, the bin holds more entries than
// the list, or the search for the end points fails, the row takes the cold path: a 4-pass radix select over the
// row re-read from L2.  All of these decisions are verified by exact counts, so they cost time, never correctness.
// The codes are rounded in float32 with a proof of exactness per entry: x*s is evaluated with the float
// neighbours s_lo < s < s_hi of the float64 scale s = 127/(gamma+eps), each as one fused multiply-add onto
// 1.5*2^23 + 128, which rounds the exact product to the nearest integer (ties to even) and leaves code + 128 in the
// low byte.  Rounding is monotone, so when both give the same integer the float64 evaluation rounds to it as
// well; the few entries where they differ (the product sits within ~1e-5 of a tie) are redone in float64.  Either
// way a code can differ from a float64 CPU evaluation only when x*s sits within float64 rounding noise of a tie.
#include "internal.h"
#include "quant_common.cuh"

namespace {

using namespace a48q;

constexpr int kCand = 64;  // entries of the chosen sub-bin that the ranking warp can take

struct Select {
    unsigned tau, keep_eq, eq_total;  // key of the k-th largest |x|; how many entries equal to tau are kept; how many exist
};

// Warp 0 of the group scans 256 (or, FOLD, 2 x 256) bins from the top digit down and finds the bin that holds the
// kr-th entry: sel[0] = digit, sel[1] = rank inside that bin (1-based from its top), sel[2] = its count.
template <bool FOLD>
__device__ __forceinline__ void scan_bins(const unsigned* hist, unsigned kr, unsigned* sel, int lane) {
    // lane l owns bins 255-8l-7 .. 255-8l; lanes ascend as digits descend
    unsigned h[8], c = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        h[i] = hist[255 - 8 * lane - i];
        if (FOLD) h[i] += hist[511 - 8 * lane - i];  // the same binade with the sign bit set
        c += h[i];
    }
    unsigned incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        unsigned n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
    }
    const unsigned excl = incl - c;
    if (incl >= kr && excl < kr) {
        unsigned cum = excl;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (cum < kr && cum + h[i] >= kr) {
                sel[0] = 255 - 8 * lane - i;
                sel[1] = kr - cum;
                sel[2] = h[i];
            }
            cum += h[i];
        }
    }
}

// The cold form of the last pass for one row (a bitmap is wanted, or more equal values straddle the k-th place than
// the ranking list holds): the row is read again (it is in L2), a group-wide scan per 4*TPR entries numbers the
// entries equal to tau so that the lowest indices win, float64 rounding throughout.  Not unrolled: it is rarely run
// and must not crowd the instruction cache of the common path.
template <int TPR, bool GLU, bool BF16IN = false>
__device__ __noinline__ void cold_final(const float* __restrict__ xrow, const float* __restrict__ urow, int K, unsigned tau,
                                        unsigned keep_eq, bool ordered, double mult, int8_t* __restrict__ crow,
                                        uint32_t* __restrict__ mrow, unsigned* red, int group, int t) {
    const int nv = K >> 2, mask_words = (K + 31) >> 5;
    auto key = [](float f) { return __float_as_uint(f) & 0x7fffffffu; };
    unsigned running = 0;
#pragma unroll 1
    for (int i0 = 0; i0 < nv; i0 += TPR) {
        const int idx = i0 + t;
        const bool valid = idx < nv;
        float4 x = valid ? load_row4<BF16IN>(xrow, idx) : make_float4(0.f, 0.f, 0.f, 0.f);
        if (GLU && valid) {
            const float4 u = __ldg(reinterpret_cast<const float4*>(urow) + idx);
            auto f = [](float gg, float uu) { float r = gg > 0.f ? gg : 0.f; return uu * (r * r); };
            x = make_float4(f(x.x, u.x), f(x.y, u.y), f(x.z, u.z), f(x.w, u.w));
        }
        const unsigned u0 = key(x.x), u1 = key(x.y), u2 = key(x.z), u3 = key(x.w);
        const bool e0 = valid && u0 == tau, e1 = valid && u1 == tau, e2 = valid && u2 == tau, e3 = valid && u3 == tau;
        bool k0 = valid && u0 > tau, k1 = valid && u1 > tau, k2 = valid && u2 > tau, k3 = valid && u3 > tau;
        if (!ordered) {
            k0 |= e0; k1 |= e1; k2 |= e2; k3 |= e3;
        } else {
            unsigned cnt = (unsigned)e0 + e1 + e2 + e3, total;
            unsigned base = running + group_excl_scan<TPR>(cnt, red, group, total);
            running += total;
            k0 |= e0 && base < keep_eq; base += e0;
            k1 |= e1 && base < keep_eq; base += e1;
            k2 |= e2 && base < keep_eq; base += e2;
            k3 |= e3 && base < keep_eq;
        }
        if (valid) {
            int a = k0 ? clampi(__double2int_rn(mult * (double)x.x), -128, 127) : 0;
            int b = k1 ? clampi(__double2int_rn(mult * (double)x.y), -128, 127) : 0;
            int c = k2 ? clampi(__double2int_rn(mult * (double)x.z), -128, 127) : 0;
            int d = k3 ? clampi(__double2int_rn(mult * (double)x.w), -128, 127) : 0;
            reinterpret_cast<uint32_t*>(crow)[idx] = pack4(a, b, c, d);
        }
        if (mrow) {  // uniform across the group
            unsigned nib = ((unsigned)k0 | (unsigned)k1 << 1 | (unsigned)k2 << 2 | (unsigned)k3 << 3) << (4 * (t & 7));
            nib |= __shfl_xor_sync(0xffffffffu, nib, 1);
            nib |= __shfl_xor_sync(0xffffffffu, nib, 2);
            nib |= __shfl_xor_sync(0xffffffffu, nib, 4);
            int word = idx >> 3;
            if ((t & 7) == 0 && word < mask_words) mrow[word] = nib;
        }
    }
}

__device__ __forceinline__ void red_shared_inc(unsigned addr) {
    asm volatile("red.shared.add.u32 [%0], 1;" ::"r"(addr) : "memory");
}

constexpr float kMagic = 12582912.f;           // 1.5 * 2^23: the floats around it are the integers
constexpr unsigned kMagicBits = 0x4B400000u;   // its bit pattern; the pattern of kMagic + n is kMagicBits + n
constexpr float kWindowBins = 255.f;           // bins 0 and 255 also take what lies outside the window

// Bin of |x| in the window [lo, lo + 1/inv_w): every step rounds monotonically, so bins are intervals of |x|.
// Both the histogram pass and the search for a bin's end points go through this one function.
__device__ __forceinline__ unsigned window_bin_bits(float ax, float lo, float inv_w) {
    const float g = __saturatef(__fmul_rn(__fadd_rn(ax, -lo), inv_w));
    return __float_as_uint(__fmaf_rn(g, kWindowBins, kMagic));  // kMagicBits + bin
}

// Smallest float f >= 0 with window_bin(f) >= b, searched by the 32 lanes of a warp around the analytic estimate;
// returns false when it is not within 16 ulps of it (the caller then takes the cold path).
__device__ __forceinline__ bool bin_lower_end(unsigned b, float lo, float inv_w, int lane, float& out) {
    const float est = lo + ((float)b - 0.5f) / (kWindowBins * inv_w);
    const unsigned cand = __float_as_uint(est) + (unsigned)lane - 16u;
    const bool ge = window_bin_bits(__uint_as_float(cand), lo, inv_w) >= kMagicBits + b;
    const unsigned m = __ballot_sync(0xffffffffu, ge);
    // monotone: the lanes at or above the end point are a suffix; it must start strictly inside the 32 candidates
    if (m == 0u || (m & 1u)) return false;
    out = __uint_as_float(__float_as_uint(est) + (unsigned)(__ffs(m) - 1) - 16u);
    return true;
}

// Cold path of one row: exact 4-pass radix select over the row re-read from memory, then cold_final.
template <int TPR, bool GLU, bool BF16IN>
__device__ __noinline__ void cold_row(const float* __restrict__ xrow, const float* __restrict__ urow, int K, int k, double mult,
                                      int8_t* __restrict__ crow, unsigned* hist, unsigned* sel, unsigned* red, int group,
                                      int t) {
    const int nv = K >> 2;
    unsigned prefix = 0, kr = (unsigned)k, eq_total = 0;
#pragma unroll 1
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        for (int b = t; b < 256; b += TPR) hist[b] = 0;
        group_sync<TPR>(group);
#pragma unroll 1
        for (int idx = t; idx < nv; idx += TPR) {
            float4 x = load_row4<BF16IN>(xrow, idx);
            if (GLU) {
                const float4 u = __ldg(reinterpret_cast<const float4*>(urow) + idx);
                auto f = [](float gg, float uu) { float r = gg > 0.f ? gg : 0.f; return uu * (r * r); };
                x = make_float4(f(x.x, u.x), f(x.y, u.y), f(x.z, u.z), f(x.w, u.w));
            }
            const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const unsigned u = __float_as_uint(xs[q]) & 0x7fffffffu;
                if (pass == 0 || (u >> (shift + 8)) == prefix) atomicAdd(&hist[(u >> shift) & 255u], 1u);
            }
        }
        group_sync<TPR>(group);
        if (t < 32) scan_bins<false>(hist, kr, sel, t);
        group_sync<TPR>(group);
        prefix = (prefix << 8) | sel[0];
        kr = sel[1];
        eq_total = sel[2];
        group_sync<TPR>(group);  // sel is rewritten by the next scan only after every thread has read it
    }
    cold_final<TPR, GLU, BF16IN>(xrow, urow, K, prefix, kr, eq_total != kr, mult, crow, nullptr, red, group, t);
}

// GLU: the row to quantise is up * ReLU(gate)^2 (Eq. 5), formed while loading: X is the gate projection and U the up
// projection, and the product never goes to memory.
// EXACT: V == ceil(K/4 / TPR), so only the last of a thread's V vectors can lie beyond the row.
template <int TPR, int V, bool GLU, bool EXACT, bool BF16IN = false>
__global__ void __launch_bounds__(kBlock, V <= 4 ? 5 : 4)
    topk_quant_int8_kernel(const float* __restrict__ X, const float* __restrict__ U, int M, int K, int k, double eps,
                           int8_t* __restrict__ codes, float* __restrict__ scale) {
    constexpr int G = kBlock / TPR;
    __shared__ __align__(2048) unsigned hist0[G][512];  // aligned so that a bin's address is base | offset
    __shared__ __align__(16) unsigned hist1[G][256];
    __shared__ unsigned cand_key[G][kCand];
    __shared__ unsigned cand_idx[G][kCand];
    __shared__ unsigned sel[G][8];
    __shared__ unsigned red[kBlock / 32];
    a48_pdl_prologue();
    const int group = threadIdx.x / TPR, t = threadIdx.x % TPR;
    const int row = blockIdx.x * G + group;
    if (row >= M) return;
    const int nv = K >> 2;
    const void* xr = row_ptr<BF16IN>(X, (size_t)row, K);
    // whether this thread's vector i lies inside the row: known at compile time for all but the last when EXACT
    const bool last_ok = (V - 1) * TPR + t < nv;
    auto inside = [&](int i) { return (EXACT && i < V - 1) ? true : (EXACT ? last_ok : i * TPR + t < nv); };
    float4 v[V];
#pragma unroll
    for (int i = 0; i < V; ++i) {
        const int idx = i * TPR + t;
        v[i] = inside(i) ? load_row4<BF16IN>(xr, idx) : make_float4(0.f, 0.f, 0.f, 0.f);
        if (GLU && inside(i)) {
            const float4 u = __ldg(reinterpret_cast<const float4*>(U + (size_t)row * K) + idx);
            auto f = [](float gg, float uu) { float r = gg > 0.f ? gg : 0.f; return uu * (r * r); };
            v[i] = make_float4(f(v[i].x, u.x), f(v[i].y, u.y), f(v[i].z, u.z), f(v[i].w, u.w));
        }
    }
    unsigned* h0 = hist0[group];
    unsigned* h1 = hist1[group];
    unsigned* sl = sel[group];
    const unsigned h0_addr = (unsigned)__cvta_generic_to_shared(h0), h1_addr = (unsigned)__cvta_generic_to_shared(h1);
    for (int b = t; b < 512; b += TPR) h0[b] = 0;
    for (int b = t; b < 256; b += TPR) h1[b] = 0;
    if (t == 0) sl[7] = 0;  // entries listed so far

    float gm = 0.f;  // max |x| as a float maximum (one instruction per element); its bits are the largest key
#pragma unroll
    for (int i = 0; i < V; ++i)
        gm = fmaxf(fmaxf(fmaxf(gm, fabsf(v[i].x)), fmaxf(fabsf(v[i].y), fabsf(v[i].z))), fabsf(v[i].w));
    unsigned gmax = group_max<TPR>(__float_as_uint(gm), red, group);
    if (TPR == 32) __syncwarp();  // (wider groups passed a barrier inside group_max: the bins are clear)
    const double gamma = (double)__uint_as_float(gmax);
    const double mult = 127.0 / (gamma + eps);
    const float s_mid = (float)mult;
    if (t == 0) scale[row] = (float)(gamma / 127.0);

    auto for_each = [&](auto f) {
#pragma unroll
        for (int i = 0; i < V; ++i) {
            if (inside(i)) {
                f(v[i].x);
                f(v[i].y);
                f(v[i].z);
                f(v[i].w);
            }
        }
    };

    // ---- pass 0: exponent (sign and exponent index 512 bins; the scan folds the two halves)
    for_each([&](float x) { red_shared_inc(h0_addr | ((__float_as_uint(x) >> 21) & 0x7fcu)); });
    group_sync<TPR>(group);
    // sl[0..2]: exponent bits of the k-th entry's binade, its rank in the binade from the top, the binade's count
    // sl[3]: 0 = window laid (sl[4] = lo, sl[5] = 1/width), 1 = every entry keeps its code, 2 = cold path
    if (t < 32) {
        scan_bins<true>(h0, (unsigned)k, sl, t);
        __syncwarp();
        if (t == 0) {
            const unsigned e = sl[0];
            const float base = __uint_as_float(e << 23);  // lower end of the binade
            unsigned mode = 0;
            if (e >= 254u) mode = 2;
            else if (__uint_as_float((e + 1u) << 23) * s_mid < 0.49f) mode = 1;  // codes at or below this binade are 0
            else if (e == 0u) mode = 2;
            else {
                const float from_top = ((float)sl[1] - 0.5f) / (float)sl[2];
                const float centre = base * (2.f - from_top), half = 0.16f * base;
                sl[4] = __float_as_uint(centre - half);
                sl[5] = __float_as_uint(1.f / (2.f * half));
            }
            sl[3] = mode;
        }
    }
    group_sync<TPR>(group);
    unsigned mode = sl[3];
    float lo_f = 0.f, hi_f = 0.f;  // entries at or above lo_f keep their code; those below hi_f are listed and ranked
    unsigned kr = 0;
    if (mode == 0u) {
        // ---- pass 1: window bins
        const float lo_w = __uint_as_float(sl[4]), inv_w = __uint_as_float(sl[5]);
        const unsigned bias = h1_addr - 4u * kMagicBits;
        for_each([&](float x) { red_shared_inc(bias + 4u * window_bin_bits(fabsf(x), lo_w, inv_w)); });
        group_sync<TPR>(group);
        if (t < 32) {
            scan_bins<false>(h1, (unsigned)k, sl, t);
            __syncwarp();
            const unsigned b = sl[0];
            bool ok = b >= 1u && b <= 254u && sl[2] <= (unsigned)kCand;
            float lo_end = 0.f, hi_end = 0.f;
            ok = ok && bin_lower_end(b, lo_w, inv_w, t, lo_end);
            ok = ok && bin_lower_end(b + 1u, lo_w, inv_w, t, hi_end);
            if (t == 0) {
                sl[3] = ok ? 0u : 2u;
                sl[4] = __float_as_uint(lo_end);
                sl[5] = __float_as_uint(hi_end);
            }
        }
        group_sync<TPR>(group);
        mode = sl[3];
        lo_f = __uint_as_float(sl[4]);
        hi_f = __uint_as_float(sl[5]);
        kr = sl[1];
    }
    if (mode == 2u) {
        cold_row<TPR, GLU, BF16IN>(reinterpret_cast<const float*>(xr), GLU ? U + (size_t)row * K : nullptr, K, k, mult,
                                   codes + (size_t)row * K, h1, sl, red, group, t);
        return;
    }

    // ---- codes.  The clip of Eq. 3 is left out: |127 x / (gamma + eps)| <= 127 for every finite x of the row.
    uint32_t* out = reinterpret_cast<uint32_t*>(codes + (size_t)row * K);
    const float s_hi = __uint_as_float(__float_as_uint(s_mid) + 1u), s_lo = __uint_as_float(__float_as_uint(s_mid) - 1u);
    // |x| - lo_f is exact for |x| in [lo_f, 2 lo_f] and the bin is far narrower than that, so an entry is listed
    // exactly when 0 <= |x| - lo_f < hi_f - lo_f; as bit patterns (negative floats are large unsigned numbers) that is
    // one unsigned comparison, and the smallest pattern of a vector tells whether any of its four entries is listed
    const unsigned width_bits = __float_as_uint(hi_f - lo_f);
    constexpr float kMagic128 = kMagic + 128.f;  // low byte of the sum's pattern = code + 128
#pragma unroll
    for (int i = 0; i < V; ++i) {
        if (!inside(i)) continue;
        const float x[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
        unsigned b[4], smallest = 0xffffffffu;
        float differ = 0.f;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const unsigned above = __float_as_uint(__fadd_rn(fabsf(x[q]), -lo_f));
            smallest = min(smallest, above);
            const float xk = (int)above >= 0 ? x[q] : 0.f;  // dropped entries round to code 0
            const float hi = __fmaf_rn(xk, s_hi, kMagic128);
            const float d = __fadd_rn(hi, -__fmaf_rn(xk, s_lo, kMagic128));  // 0 or +-1, exactly
            differ = __fmaf_rn(d, d, differ);
            b[q] = __float_as_uint(hi);
        }
        if ((smallest < width_bits) | (differ != 0.f)) {  // rare
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const unsigned above = __float_as_uint(__fadd_rn(fabsf(x[q]), -lo_f));
                // a product within ~1e-5 of a rounding tie: float64 decides, as the definition does
                if (differ != 0.f)
                    b[q] = kMagicBits + 128u + ((int)above >= 0 ? (unsigned)__double2int_rn(mult * (double)x[q]) : 0u);
                if (above < width_bits) {
                    const unsigned at = atomicAdd(&sl[7], 1u);
                    cand_key[group][at] = __float_as_uint(x[q]) & 0x7fffffffu;
                    cand_idx[group][at] = (unsigned)((i * TPR + t) * 4 + q);
                }
            }
        }
        // the four patterns are kMagicBits + (code + 128): a multiply-add chain puts the low bytes side by side, the
        // constant takes the upper bits out again, and flipping each byte's top bit turns code + 128 into the code
        const unsigned packed = ((b[3] * 256u + b[2]) * 256u + b[1]) * 256u + b[0];
        out[i * TPR + t] = (packed - kMagicBits * 0x01010101u) ^ 0x80808080u;
    }
    if (mode != 0u) return;  // nothing is listed (uniform over the group)
    // ---- the listed entries rank each other by (|x| descending, index ascending); those ranked kr or later lose
    group_sync<TPR>(group);
    if (t < 32) {
        const unsigned n = sl[7];
#pragma unroll
        for (int half = 0; half < kCand / 32; ++half) {
            const unsigned mine = t + 32 * half;
            if (mine < n) {
                const unsigned ck = cand_key[group][mine], ci = cand_idx[group][mine];
                unsigned ahead = 0;
                for (unsigned j = 0; j < n; ++j) {
                    const unsigned ok = cand_key[group][j], oi = cand_idx[group][j];
                    ahead += (ok > ck) || (ok == ck && oi < ci);
                }
                if (ahead >= kr) codes[(size_t)row * K + ci] = 0;
            }
        }
    }
}

// Any K (unaligned or very long rows): one block per row, the row re-read from L2; 4-pass 8-bit radix select.
__device__ __forceinline__ Select radix_select_generic(int k, unsigned* hist, unsigned* sel, int t, const float* xr, int K) {
    unsigned prefix = 0, kr = (unsigned)k, eq_total = 0;
#pragma unroll 1
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        hist[t] = 0;
        __syncthreads();
        for (int j = t; j < K; j += kBlock) {
            const unsigned u = __float_as_uint(xr[j]) & 0x7fffffffu;
            if (pass == 0 || (u >> (shift + 8)) == prefix) atomicAdd(&hist[(u >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (t < 32) scan_bins<false>(hist, kr, sel, t);
        __syncthreads();
        prefix = (prefix << 8) | sel[0];
        kr = sel[1];
        eq_total = sel[2];
        __syncthreads();
    }
    return Select{prefix, kr, eq_total};
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
    Select s = radix_select_generic(k, hist, sel, t, xr, K);
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

template <int TPR, int V, bool GLU, bool EXACT, bool BF16IN>
void launch_one(const float* X, const float* U, int M, int K, int k, double e, int8_t* codes, float* scale, cudaStream_t st) {
    constexpr int G = kBlock / TPR;
    a48_launch_pdl(topk_quant_int8_kernel<TPR, V, GLU, EXACT, BF16IN>, dim3((M + G - 1) / G), dim3(kBlock), 0, st, X, U, M, K, k, e, codes,
                   scale);
}

template <bool GLU, bool BF16IN = false>
bitnet_a48_status launch_topk(const float* X, const float* U, int M, int K, int k, double e, int8_t* codes, float* scale,
                              cudaStream_t st) {
    const int nv = K / 4;
#define A48_TK(TPR, V, EXACT) launch_one<TPR, V, GLU, EXACT, BF16IN>(X, U, M, K, k, e, codes, scale, st)
    if (nv <= 32 * 4) A48_TK(32, 4, false);
    else if (nv <= 64 * 4) A48_TK(64, 4, false);
    else if (nv <= 128 * 4) A48_TK(128, 4, false);
    else if (nv <= 128 * 8) {  // up to 4096 features: two rows per block, V = ceil(nv / 128)
        switch ((nv + 127) / 128) {
            case 5: A48_TK(128, 5, true); break;
            case 6: A48_TK(128, 6, true); break;
            case 7: A48_TK(128, 7, true); break;
            default: A48_TK(128, 8, true); break;
        }
    } else {  // up to 12288 features: one row per block, V = ceil(nv / 256)
        switch ((nv + 255) / 256) {
            case 5: A48_TK(256, 5, true); break;
            case 6: A48_TK(256, 6, true); break;
            case 7: A48_TK(256, 7, true); break;
            case 8: A48_TK(256, 8, true); break;
            case 9: A48_TK(256, 9, true); break;
            case 10: A48_TK(256, 10, true); break;
            case 11: A48_TK(256, 11, true); break;
            default: A48_TK(256, 12, true); break;
        }
    }
#undef A48_TK
    A48_CUDA_TRY(cudaGetLastError());
    return BITNET_A48_OK;
}

}  // namespace

bool a48_topk_quant_fast_shape(int K) { return (K % 4 == 0) && K / 4 <= 256 * 12; }

bitnet_a48_status a48_launch_topk_quant_int8(const float* X, int M, int K, int k, float eps, int8_t* codes,
                                             float* scale, uint32_t* mask_bits, cudaStream_t st) {
    // (the bitmap is an optional extra of the API: a call that wants it takes the kernel that re-reads the row)
    if (a48_topk_quant_fast_shape(K) && !mask_bits) return launch_topk<false>(X, nullptr, M, K, k, (double)eps, codes, scale, st);
    topk_quant_int8_generic_kernel<<<M, kBlock, 0, st>>>(X, M, K, k, (double)eps, codes, scale, mask_bits);
    A48_CUDA_TRY(cudaGetLastError());
    return BITNET_A48_OK;
}

bitnet_a48_status a48_launch_topk_quant_int8_bf16(const uint16_t* X, int M, int K, int k, float eps, int8_t* codes,
                                                  float* scale, cudaStream_t st) {
    if (!a48_topk_quant_fast_shape(K)) return BITNET_A48_ERR_UNSUPPORTED;  // the register kernels only
    return launch_topk<false, true>(reinterpret_cast<const float*>(X), nullptr, M, K, k, (double)eps, codes, scale, st);
}

// Top-K + INT8 of up * ReLU(gate)^2 (Eq. 5 fused into the quantiser's load); shapes of the register kernels only.
bitnet_a48_status a48_launch_topk_quant_int8_glu(const float* gate, const float* up, int M, int K, int k, float eps,
                                                 int8_t* codes, float* scale, cudaStream_t st) {
    if (!a48_topk_quant_fast_shape(K)) return BITNET_A48_ERR_UNSUPPORTED;
    return launch_topk<true>(gate, up, M, K, k, (double)eps, codes, scale, st);
}
