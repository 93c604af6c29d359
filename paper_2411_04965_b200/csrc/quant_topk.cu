// Sparsify-then-quantise for the intermediate states, Eq. 1 and 3: per token gamma = max|x|, the mask of the k
// largest |x| (ties: lowest index first), codes = RoundClip(127 x / (gamma + eps), -128, 127) where kept, else 0.
//
// One token row is owned by a group of TPR threads (32..256) of a 256-thread block and lives in registers from
// its single 128-bit coalesced load to the store of the codes.  The k-th largest magnitude is found exactly by a
// radix select on the bit pattern of |x| (order-preserving as an unsigned integer):
//   pass 0  histogram of the 8 exponent bits (raw bits index 512 bins, the sign halves are folded in the scan);
//           real rows hit a handful of bins, and increments of one bin from one warp are merged by the hardware;
//   pass 1  histogram of the next 8 mantissa bits of the entries in the chosen binade;
//   codes   every entry at or above the chosen sub-bin's lower bound gets its code; the few entries inside the
//           sub-bin (a few dozen at most on real data) are listed on the way, one warp then ranks them against
//           each other by (|x| descending, index ascending) and clears the codes of those that lose.  A sub-bin
//           with more entries than the list holds (many equal values, e.g. zeros after ReLU^2) takes two more
//           histogram passes instead, which give the exact key of the k-th entry.
// The codes are then rounded in float32 with a proof of exactness per entry: x*s is evaluated with the float
// neighbours s_lo < s < s_hi of the float64 scale s = 127/(gamma+eps), each as one fused multiply-add onto
// 1.5*2^23, which rounds the exact product to the nearest integer (ties to even).  Rounding is monotone, so when
// both give the same integer the float64 evaluation rounds to it as well; the few entries where they differ (the
// product sits within ~1e-5 of a tie) are redone in float64.  Either way a code can differ from a float64 CPU
// evaluation only when x*s sits within float64 rounding noise of a tie.
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
template <int TPR, bool GLU>
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
        float4 x = valid ? __ldg(reinterpret_cast<const float4*>(xrow) + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
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
// increments the word at addr when z == 0 (one predicated instruction instead of a branch around it)
__device__ __forceinline__ void red_shared_inc_if_zero(unsigned addr, unsigned z) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.u32 p, %1, 0;\n\t@p red.shared.add.u32 [%0], 1;\n\t}" ::"r"(addr), "r"(z) : "memory");
}

// GLU: the row to quantise is up * ReLU(gate)^2 (Eq. 5), formed while loading: X is the gate projection and U the up
// projection, and the product never goes to memory.
// EXACT: V == ceil(K/4 / TPR), so only the last of a thread's V vectors can lie beyond the row.
template <int TPR, int V, bool GLU, bool EXACT>
__global__ void __launch_bounds__(kBlock, V <= 4 ? 5 : 4)
    topk_quant_int8_kernel(const float* __restrict__ X, const float* __restrict__ U, int M, int K, int k, double eps,
                           int8_t* __restrict__ codes, float* __restrict__ scale, uint32_t* __restrict__ mask_bits) {
    constexpr int G = kBlock / TPR;
    __shared__ __align__(2048) unsigned hist0[G][512];  // aligned so that a bin's address is base | offset
    __shared__ __align__(16) unsigned hist1[G][260];  // 256 bins and one (index 256) for entries outside the binade
    __shared__ unsigned cand_key[G][kCand];
    __shared__ unsigned cand_idx[G][kCand];
    __shared__ unsigned sel[G][4];
    __shared__ unsigned red[kBlock / 32];
    const int group = threadIdx.x / TPR, t = threadIdx.x % TPR;
    const int row = blockIdx.x * G + group;
    if (row >= M) return;
    const int nv = K >> 2;
    const float4* xr = reinterpret_cast<const float4*>(X + (size_t)row * K);
    // whether this thread's vector i lies inside the row: known at compile time for all but the last when EXACT
    const bool last_ok = (V - 1) * TPR + t < nv;
    auto inside = [&](int i) { return (EXACT && i < V - 1) ? true : (EXACT ? last_ok : i * TPR + t < nv); };
    float4 v[V];
#pragma unroll
    for (int i = 0; i < V; ++i) {
        const int idx = i * TPR + t;
        v[i] = inside(i) ? __ldg(xr + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
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
    for (int b = t; b < 257; b += TPR) h1[b] = 0;
    if (t == 0) sl[3] = 0;

    float gm = 0.f;  // max |x| as a float maximum (one instruction per element); its bits are the largest key
#pragma unroll
    for (int i = 0; i < V; ++i)
        gm = fmaxf(fmaxf(fmaxf(gm, fabsf(v[i].x)), fmaxf(fabsf(v[i].y), fabsf(v[i].z))), fabsf(v[i].w));
    unsigned gmax = group_max<TPR>(__float_as_uint(gm), red, group);
    if (TPR == 32) __syncwarp();  // (wider groups passed a barrier inside group_max: the bins are clear)
    const double gamma = (double)__uint_as_float(gmax);
    const double mult = 127.0 / (gamma + eps);

    auto for_each_raw = [&](auto f) {
#pragma unroll
        for (int i = 0; i < V; ++i) {
            if (inside(i)) {
                f(__float_as_uint(v[i].x));
                f(__float_as_uint(v[i].y));
                f(__float_as_uint(v[i].z));
                f(__float_as_uint(v[i].w));
            }
        }
    };

    // ---- pass 0: exponent (sign and exponent index 512 bins; the scan folds the two halves)
    for_each_raw([&](unsigned r) { red_shared_inc(h0_addr | ((r >> 21) & 0x7fcu)); });
    group_sync<TPR>(group);
    if (t < 32) scan_bins<true>(h0, (unsigned)k, sl, t);
    group_sync<TPR>(group);
    const unsigned binade = sl[0] << 23;
    // ---- pass 1: the next 8 mantissa bits of the entries in that binade
    // (no test per entry: with the sign shifted out, the distance to the binade's lower end is below 2^24 inside
    // the binade, and wraps to a large number below it; everything else lands in the spare bin)
    const unsigned binade2 = binade << 1;
    for_each_raw([&](unsigned r) { red_shared_inc(h1_addr + 4u * min(((r << 1) - binade2) >> 16, 256u)); });
    const unsigned kr1 = sl[1];
    group_sync<TPR>(group);
    if (t < 32) scan_bins<false>(h1, kr1, sl, t);
    group_sync<TPR>(group);
    unsigned prefix = (binade >> 15) | sl[0];  // the 16 leading bits of the key
    unsigned kr = sl[1], eq_total = sl[2];
    // Entries at or above lo are kept for now; the few below hi (the chosen sub-bin) are listed while the codes are
    // written, ranked afterwards, and the losers' codes are cleared.
    float lo_f = __uint_as_float(prefix << 15), hi_f = __uint_as_float((prefix << 15) + 0x8000u);
    bool listed = true;
    if (eq_total > (unsigned)kCand || mask_bits) {
        // ---- many entries share the 16 leading bits (equal values, e.g. zeros): two more histogram passes (8 and 7
        // bits) give the exact key of the k-th entry
        listed = false;
#pragma unroll 1
        for (int pass = 2; pass < 4; ++pass) {
            const int bits = pass == 3 ? 7 : 8, shift = pass == 2 ? 7 : 0;
            for (int b = t; b < 256; b += TPR) h1[b] = 0;
            group_sync<TPR>(group);
            for_each_raw([&](unsigned r) {
                const unsigned u = r & 0x7fffffffu;
                red_shared_inc_if_zero(h1_addr + 4u * ((u >> shift) & ((1u << bits) - 1u)), (u >> (shift + bits)) ^ prefix);
            });
            group_sync<TPR>(group);
            if (t < 32) scan_bins<false>(h1, kr, sl, t);
            group_sync<TPR>(group);
            prefix = (prefix << bits) | sl[0];
            kr = sl[1];
            eq_total = sl[2];
            group_sync<TPR>(group);  // sel is rewritten by the next scan only after every thread has read it
        }
        // prefix is now the key tau; kr of the eq_total entries equal to it are kept.  Which ones matters only when
        // not all are, a bitmap is wanted or tau != 0 (a kept zero and a dropped zero both have code 0).
        const bool ordered = eq_total != kr;
        if (mask_bits || (ordered && prefix != 0u)) {
            if (t == 0) scale[row] = (float)(gamma / 127.0);
            const int mask_words = (K + 31) >> 5;
            cold_final<TPR, GLU>(X + (size_t)row * K, GLU ? U + (size_t)row * K : nullptr, K, prefix, kr, ordered, mult,
                                 codes + (size_t)row * K, mask_bits ? mask_bits + (size_t)row * mask_words : nullptr, red,
                                 group, t);
            return;
        }
        lo_f = __uint_as_float(prefix);
        hi_f = 0.f;  // nothing is listed
    }

    // ---- codes.  The clip of Eq. 3 is left out: |127 x / (gamma + eps)| <= 127 for every finite x of the row.
    uint32_t* out = reinterpret_cast<uint32_t*>(codes + (size_t)row * K);
    if (t == 0) scale[row] = (float)(gamma / 127.0);
    const float s_mid = (float)mult;
    const float s_hi = __uint_as_float(__float_as_uint(s_mid) + 1u), s_lo = __uint_as_float(__float_as_uint(s_mid) - 1u);
    constexpr float kMagic = 12582912.f;  // 1.5 * 2^23: floats there are the integers, the low byte is the code
#pragma unroll
    for (int i = 0; i < V; ++i) {
        if (!inside(i)) continue;
        const float x[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
        unsigned code[4], differ = 0;
        float lowest_kept = INFINITY;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const unsigned hi = __float_as_uint(__fmaf_rn(x[q], s_hi, kMagic));
            differ |= hi ^ __float_as_uint(__fmaf_rn(x[q], s_lo, kMagic));
            const bool keep = fabsf(x[q]) >= lo_f;
            code[q] = keep ? hi : 0u;
            lowest_kept = fminf(lowest_kept, keep ? fabsf(x[q]) : INFINITY);
        }
        if ((differ != 0u) | (lowest_kept < hi_f)) {  // rare
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const bool keep = fabsf(x[q]) >= lo_f;
                // a product within ~1e-5 of a rounding tie: float64 decides, as the definition does
                if (differ) code[q] = keep ? (unsigned)__double2int_rn(mult * (double)x[q]) : 0u;
                if (keep && fabsf(x[q]) < hi_f) {
                    const unsigned at = atomicAdd(&sl[3], 1u);
                    cand_key[group][at] = __float_as_uint(x[q]) & 0x7fffffffu;
                    cand_idx[group][at] = (unsigned)((i * TPR + t) * 4 + q);
                }
            }
        }
        out[i * TPR + t] = __byte_perm(__byte_perm(code[0], code[1], 0x0040), __byte_perm(code[2], code[3], 0x0040), 0x5410);
    }
    if (!listed) return;  // (uniform over the group)
    // ---- the listed entries rank each other by (|x| descending, index ascending); those ranked kr or later lose
    group_sync<TPR>(group);
    if (t < 32) {
        const unsigned n = sl[3];
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

template <int TPR, int V, bool GLU, bool EXACT>
void launch_one(const float* X, const float* U, int M, int K, int k, double e, int8_t* codes, float* scale,
                uint32_t* mask_bits, cudaStream_t st) {
    constexpr int G = kBlock / TPR;
    topk_quant_int8_kernel<TPR, V, GLU, EXACT><<<(M + G - 1) / G, kBlock, 0, st>>>(X, U, M, K, k, e, codes, scale, mask_bits);
}

template <bool GLU>
bitnet_a48_status launch_topk(const float* X, const float* U, int M, int K, int k, double e, int8_t* codes, float* scale,
                              uint32_t* mask_bits, cudaStream_t st) {
    const int nv = K / 4;
#define A48_TK(TPR, V, EXACT) launch_one<TPR, V, GLU, EXACT>(X, U, M, K, k, e, codes, scale, mask_bits, st)
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
