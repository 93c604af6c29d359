// Low-bit attention (Section 3, low-bit attention paragraph): post-RoPE absmax quantisation of the query, key and
// value heads, a packed key/value cache of 4 or 3 bits per entry (the heads of position 0, the bos token, keep
// 4 bits in a 3-bit cache), and the decode attention that reads it.
//
// Quantiser of one head vector x (one token, one head), Eq. 3 with b bits in place of 8: gamma = max|x|,
// L = 2^(b-1) - 1, q = RoundClip(L/(gamma+eps) * x, -(L+1), L), value gamma/L * q; the unsigned integer
// u = q + L + 1 is what the cache stores.  The scale arithmetic is float64 as in the other quantisers.
//
// Cache layout (one buffer for keys, one for values; bitnet_a48_kv_cache_bytes gives its size):
//   codes  [B][n_heads][ctx_cap][row_bytes]   row = the head's entries as a little-endian bit stream, entry i at
//                                             bits [i*b, (i+1)*b); row_bytes = b * head_dim_padded / 8 with the
//                                             head dimension padded to a multiple of 32 entries (12- or 16-byte
//                                             granules of 32 entries)
//   scales [B][n_heads][ctx_cap] fp32         gamma / L
//   bos    [B][n_heads][row_bytes at 4 bits]  only in a 3-bit cache: the 4-bit codes of position 0
// A 3-bit cache holds 52 bytes per head vector of 128 entries where fp32 holds 512.
#include "internal.h"

namespace {

__host__ __device__ inline int padded_dim(int hd) { return (hd + 31) / 32 * 32; }
__host__ __device__ inline int row_bytes(int hd, int bits) { return padded_dim(hd) * bits / 8; }

struct KvView {
    uint8_t* codes;
    float* scales;
    uint8_t* bos;  // nullptr unless bits == 3
    int bits, row, row4;
};

__host__ __device__ inline KvView kv_view(void* base, int B, int nh, int cap, int hd, int bits) {
    KvView v;
    v.bits = bits;
    v.row = row_bytes(hd, bits);
    v.row4 = row_bytes(hd, 4);
    v.codes = static_cast<uint8_t*>(base);
    const size_t codes_bytes = ((size_t)B * nh * cap * v.row + 15) / 16 * 16;
    v.scales = reinterpret_cast<float*>(v.codes + codes_bytes);
    const size_t scale_bytes = ((size_t)B * nh * cap * 4 + 15) / 16 * 16;
    v.bos = bits == 3 ? v.codes + codes_bytes + scale_bytes : nullptr;
    return v;
}

// One warp quantises one head vector held as hd <= 128 floats, lane l owning entries 4l..4l+3 (zero past hd).
// Returns the codes of the lane (as unsigned u = q + L + 1, 0 for padding... padding stores u of q = 0) and the scale.
__device__ __forceinline__ void quant_head_warp(const float (&x)[4], int bits, double eps, unsigned (&u)[4], float& scale_out) {
    float gm = fmaxf(fmaxf(fabsf(x[0]), fabsf(x[1])), fmaxf(fabsf(x[2]), fabsf(x[3])));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) gm = fmaxf(gm, __shfl_xor_sync(0xffffffffu, gm, o));
    const int L = (1 << (bits - 1)) - 1;
    const double gamma = (double)gm;
    const double s = (double)L / (gamma + eps);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int q = __double2int_rn(s * (double)x[i]);
        q = q < -(L + 1) ? -(L + 1) : (q > L ? L : q);
        u[i] = (unsigned)(q + L + 1);
    }
    scale_out = (float)(gamma / (double)L);
}

// Writes the warp's 128 (padded) entries of `bits` bits each as a bit stream: lane l's four entries are bits
// [4l*bits, (4l+4)*bits).  With 4 bits that is two bytes per lane; with 3 bits twelve bits per lane, so lanes pair
// up to three bytes.  Only the first row_bytes(hd) bytes exist.
__device__ __forceinline__ void store_codes_warp(uint8_t* row, int nbytes, const unsigned (&u)[4], int bits, int lane) {
    if (bits == 4) {
        const unsigned v = u[0] | (u[1] << 4) | (u[2] << 8) | (u[3] << 12);
        if (2 * lane + 1 < nbytes) *reinterpret_cast<uint16_t*>(row + 2 * lane) = (uint16_t)v;
    } else {
        const unsigned v = u[0] | (u[1] << 3) | (u[2] << 6) | (u[3] << 9);  // 12 bits
        const unsigned other = __shfl_xor_sync(0xffffffffu, v, 1);
        if ((lane & 1) == 0) {
            const unsigned w = v | (other << 12);  // 24 bits of lanes l, l+1
            const int at = 3 * (lane >> 1);
            if (at + 2 < nbytes) {
                row[at] = (uint8_t)w;
                row[at + 1] = (uint8_t)(w >> 8);
                row[at + 2] = (uint8_t)(w >> 16);
            }
        }
    }
}

// RoPE on (i, i + hd/2) pairs for q and k, then the head quantisers.  One warp per (token, head); hd <= 128,
// lane l owns entries 4l..4l+3 (the rotation partner of entry i sits in lane (l + hd/8) mod (hd/4)... fetched from
// memory instead: every lane reads its four entries and their four partners).
// table: nullptr (a few tokens: the angles are evaluated here) or cos/sin pairs [T][hd/2].
// q is overwritten with the rotated (and, q_bits != 0, quantise-dequantised) query.  The rotated key and the value
// go to the packed caches at position pos0 + t; dq_k / dq_v (may be nullptr) receive their dequantised fp32 values
// at position pos0 + t of copies laid out [B][nh][pos0 + T][hd] for the prefill attention kernel (the positions before
// pos0 come from dequant_prefix_kernel).
__global__ void __launch_bounds__(256) rope_quant_cache_kernel(float* __restrict__ q, const float* __restrict__ k,
                                                               const float* __restrict__ v, const float2* __restrict__ table,
                                                               double base, int B, int T, int nh,
                                                               int hd, int pos0, int cap, int q_bits, int kv_bits, double eps,
                                                               void* kcache, void* vcache, float* __restrict__ dq_k,
                                                               float* __restrict__ dq_v) {
    a48_pdl_prologue();
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= B * T * nh) return;
    const int h = warp % nh, m = warp / nh, t = m % T, b = m / T;
    const int half = hd / 2, pos = pos0 + t;
    const size_t src = (size_t)m * nh * hd + (size_t)h * hd;
    float qr[4], kr[4], vr[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int e = 4 * lane + i;
        qr[i] = kr[i] = vr[i] = 0.f;
        if (e < hd) {
            const int j = e < half ? e : e - half;  // index of the rotation pair
            float c, s;
            if (table) {  // cos/sin of (pos0 + t) * base^(-j/half), evaluated in float64 by the caller's table kernel
                const float2 cs = table[t * half + j];
                c = cs.x;
                s = cs.y;
            } else {
                const double ang = (double)pos * pow(base, -(double)j / (double)half);
                double sn, cn;
                sincos(ang, &sn, &cn);
                c = (float)cn;
                s = (float)sn;
            }
            const float ql = q[src + j], qh = q[src + j + half], kl = k[src + j], kh = k[src + j + half];
            qr[i] = e < half ? ql * c - qh * s : qh * c + ql * s;
            kr[i] = e < half ? kl * c - kh * s : kh * c + kl * s;
            vr[i] = v[src + e];
        }
    }
    __syncwarp();  // every lane has read the q entries it needs before any lane overwrites them
    unsigned u[4];
    float sc;
    if (q_bits) {
        quant_head_warp(qr, q_bits, eps, u, sc);
        const int L = (1 << (q_bits - 1)) - 1;
#pragma unroll
        for (int i = 0; i < 4; ++i) qr[i] = sc * (float)((int)u[i] - (L + 1));
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
        if (4 * lane + i < hd) q[src + 4 * lane + i] = qr[i];
    const int use_bits = (kv_bits == 3 && pos == 0) ? 4 : kv_bits;  // the bos heads keep 4 bits
    const int L = (1 << (use_bits - 1)) - 1;
    const size_t slot = ((size_t)b * nh + h) * cap + pos;
    const size_t dq = (((size_t)b * nh + h) * (pos0 + T) + pos) * hd;  // copies hold positions 0 .. pos0 + T - 1
    for (int which = 0; which < 2; ++which) {
        const float(&x)[4] = which == 0 ? kr : vr;
        KvView view = kv_view(which == 0 ? kcache : vcache, B, nh, cap, hd, kv_bits);
        quant_head_warp(x, use_bits, eps, u, sc);
        uint8_t* row = (kv_bits == 3 && pos == 0) ? view.bos + ((size_t)b * nh + h) * view.row4 : view.codes + slot * view.row;
        store_codes_warp(row, use_bits == 4 ? view.row4 : view.row, u, use_bits, lane);
        if (lane == 0) view.scales[slot] = sc;
        float* out = which == 0 ? dq_k : dq_v;
        if (out) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (4 * lane + i < hd) out[dq + 4 * lane + i] = sc * (float)((int)u[i] - (L + 1));
        }
    }
}

// Eight entries of a row as floats (u - offset, not yet scaled).  Lane `sub` of the 16 lanes that share a row owns
// entries 8*sub..8*sub+7: one 32-bit word at 4 bits, 24 bits out of a 12-byte granule at 3 bits (the granule's three
// words are loaded by all four lanes that share it).
__device__ __forceinline__ void load8(const uint8_t* row, int bits, int sub, bool inside, float (&f)[8]) {
    unsigned w;
    if (!inside) {  // this lane's entries lie beyond the (padded) head: nothing is read
        w = 0;
    } else if (bits == 4) {
        w = __ldg(reinterpret_cast<const unsigned*>(row) + sub);
    } else {
        const unsigned* g = reinterpret_cast<const unsigned*>(row) + 3 * (sub >> 2);
        const unsigned w0 = __ldg(g), w1 = __ldg(g + 1), w2 = __ldg(g + 2);
        const int i = sub & 3;  // bits [24 i, 24 i + 24) of the 96-bit granule
        w = i == 0 ? w0 : (i == 1 ? __funnelshift_r(w0, w1, 24) : (i == 2 ? __funnelshift_r(w1, w2, 16) : (w2 >> 8)));
    }
    const unsigned mask = (1u << bits) - 1u;
    const float offset = 8388608.f + (float)(1 << (bits - 1));  // 2^23 + L + 1
#pragma unroll
    for (int i = 0; i < 8; ++i)
        f[i] = __uint_as_float(0x4B000000u | ((w >> (bits * i)) & mask)) - offset;  // exact: u - (L + 1)
}

// Positions 0 .. pos0-1 of the packed caches as fp32, into copies laid out [B][nh][rows][hd]: what a prefill that
// starts behind cached positions hands to the attention kernel.  One warp per (sequence, head, position): lanes 0-15
// take the key row, lanes 16-31 the value row, eight entries each.
__global__ void __launch_bounds__(256) dequant_prefix_kernel(const void* kcache, const void* vcache, int B, int nh, int hd, int pos0,
                                                             int cap, int rows, int kv_bits, float* __restrict__ dq_k,
                                                             float* __restrict__ dq_v) {
    a48_pdl_prologue();
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31, sub = lane & 15, which = lane >> 4;
    if (warp >= (long long)B * nh * pos0) return;
    const int pos = (int)(warp % pos0);
    const size_t head = (size_t)(warp / pos0);  // b * nh + h
    const KvView view = kv_view(const_cast<void*>(which == 0 ? kcache : vcache), B, nh, cap, hd, kv_bits);
    const bool bos = kv_bits == 3 && pos == 0;  // position 0 keeps 4 bits in a 3-bit cache
    const int bits = bos ? 4 : kv_bits;
    const size_t slot = head * cap + pos;
    const uint8_t* row = bos ? view.bos + head * view.row4 : view.codes + slot * view.row;
    float f[8];
    load8(row, bits, sub, 8 * sub < padded_dim(hd), f);
    const float sc = view.scales[slot];
    float* out = (which == 0 ? dq_k : dq_v) + (head * rows + pos) * hd;
#pragma unroll
    for (int i = 0; i < 8; ++i)
        if (8 * sub + i < hd) out[8 * sub + i] = sc * f[i];
}

constexpr int ATTN_SPLITS = 8;

__device__ __forceinline__ float ld_cluster_f32(const float* p, unsigned rank) {
    float v;
    asm volatile(
        "{\n\t.reg .b32 ra;\n\tmapa.shared::cluster.u32 ra, %1, %2;\n\tld.shared::cluster.f32 %0, [ra];\n\t}"
        : "=f"(v)
        : "r"((unsigned)__cvta_generic_to_shared(p)), "r"(rank));
    return v;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

constexpr int kChunkKeys = 256;  // keys staged in shared memory at a time

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((unsigned)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src)
                 : "memory");
}

// Eight entries of a staged row (shared memory), as load8 does from global memory.
__device__ __forceinline__ void unpack8(const uint8_t* row, int bits, int sub, bool inside, float (&f)[8]) {
    unsigned w = 0;
    if (inside) {
        if (bits == 4) {
            w = reinterpret_cast<const unsigned*>(row)[sub];
        } else {
            const unsigned* g = reinterpret_cast<const unsigned*>(row) + 3 * (sub >> 2);
            const unsigned w0 = g[0], w1 = g[1], w2 = g[2];
            const int i = sub & 3;
            w = i == 0 ? w0 : (i == 1 ? __funnelshift_r(w0, w1, 24) : (i == 2 ? __funnelshift_r(w1, w2, 16) : (w2 >> 8)));
        }
    }
    const unsigned mask = (1u << bits) - 1u;
    const float offset = 8388608.f + (float)(1 << (bits - 1));
#pragma unroll
    for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(0x4B000000u | ((w >> (bits * i)) & mask)) - offset;
}

// Decode attention over the packed cache for a few queries per sequence: the keys of one (query, head, batch) are
// split over the ATTN_SPLITS CTAs of a cluster.  A CTA copies its keys' codes and scales (contiguous in the cache:
// 52 bytes per key at 3 bits) into shared memory with cp.async, up to kChunkKeys keys at a time, so that the whole
// stretch is in flight at once; then every half-warp takes one key at a time (lane `sub` of the half-warp owns
// entries 8 sub .. 8 sub + 7 of the head, head_dim <= 128) with online softmax per half-warp, and the partial
// results are combined through shared memory and distributed shared memory as in the fp32 kernel.  In a 3-bit cache
// position 0 (4-bit codes in the side table) is read straight from global memory by one half-warp.
// Dynamic shared memory: K rows | V rows | K scales | V scales of one chunk (+ 3 keys of alignment slack each).
__global__ void __launch_bounds__(256) attn_row_lowbit_kernel(const float* __restrict__ q, const void* kcache, const void* vcache,
                                                              int B, int T, int nh, int hd, int pos0, int cap, int kv_bits,
                                                              float scale, float* __restrict__ out) {
    constexpr int HALVES = 16;  // half-warps per CTA
    extern __shared__ __align__(16) uint8_t stage[];
    __shared__ float sm_m[HALVES], sm_l[HALVES];
    __shared__ float sm_o[HALVES][128];
    __shared__ float cta_ml[2];
    __shared__ float cta_o[128];
    a48_pdl_prologue();
    const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z / T, t = blockIdx.z % T;
    const int lane = threadIdx.x & 31, sub = lane & 15, halfw = threadIdx.x >> 4;
    const size_t H = (size_t)nh * hd;
    const float* qr = q + ((size_t)b * T + t) * H + (size_t)h * hd;
    const KvView kview = kv_view(const_cast<void*>(kcache), B, nh, cap, hd, kv_bits);
    const KvView vview = kv_view(const_cast<void*>(vcache), B, nh, cap, hd, kv_bits);
    const int row = kview.row;
    const size_t rows_bytes = ((size_t)(kChunkKeys + 3) * row + 15) / 16 * 16;
    uint8_t* sk = stage;
    uint8_t* sv = stage + rows_bytes;
    float* sks = reinterpret_cast<float*>(stage + 2 * rows_bytes);
    float* svs = sks + kChunkKeys + 4;
    float qreg[8], o[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int col = 8 * sub + i;
        qreg[i] = col < hd ? qr[col] * scale : 0.f;
        o[i] = 0.f;
    }
    float m = -INFINITY, l = 0.f;
    const int n_keys = pos0 + t + 1;
    const int per = (n_keys + ATTN_SPLITS - 1) / ATTN_SPLITS;
    const int j_begin = split * per, j_end = min(n_keys, (split + 1) * per);
    const size_t head = (size_t)b * nh + h;
    const unsigned half_mask = 0xffffu << (lane & 16);
    const bool mine = 8 * sub < padded_dim(hd);
    // The kernel is bound by the instructions it issues per key (ncu: 118 per key with one softmax step and two expf per
    // key), so the exponentials are ex2.approx of a difference times log2 e (two units in the last place; 2^-inf = 0)
    // and four keys share one step of the online softmax.
    constexpr float kLog2e = 1.4426950408889634f;
    auto exp2a = [](float x) {
        float y;
        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
        return y;
    };
    auto half_sum = [&](float v) {
#pragma unroll
        for (int off = 8; off > 0; off >>= 1) v += __shfl_xor_sync(half_mask, v, off);
        return v;
    };
    auto take = [&](const float (&kf)[8], const float (&vf)[8], float ks, float vs) {  // one key into the running softmax
        float dot = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) dot += qreg[i] * kf[i];
        dot = half_sum(dot) * ks;
        const float m_new = fmaxf(m, dot);
        const float corr = exp2a((m - m_new) * kLog2e);
        const float pr = exp2a((dot - m_new) * kLog2e);
        l = l * corr + pr;
        const float pv = pr * vs;
#pragma unroll
        for (int i = 0; i < 8; ++i) o[i] = o[i] * corr + pv * vf[i];
        m = m_new;
    };
    const bool bos_table = kv_bits == 3;  // position 0 is not in the 3-bit rows
    if (bos_table && j_begin == 0 && j_end > 0 && halfw == 0) {
        float kf[8], vf[8];
        load8(kview.bos + head * kview.row4, 4, sub, mine, kf);
        load8(vview.bos + head * vview.row4, 4, sub, mine, vf);
        take(kf, vf, __ldg(kview.scales + head * cap), __ldg(vview.scales + head * cap));
    }
    for (int c0 = j_begin; c0 < j_end; c0 += kChunkKeys) {
        const int c1 = min(c0 + kChunkKeys, j_end);
        const int ca = c0 & ~3;  // copies start on a 16-byte boundary of the cache: four keys are a multiple of 16 bytes
        const size_t first = head * cap + ca;
        const int code_pieces = ((c1 - ca) * row + 15) / 16, scale_pieces = (c1 - ca + 3) / 4;
        __syncthreads();  // the previous chunk has been consumed
        for (int i = threadIdx.x; i < code_pieces; i += 256) {
            cp_async16(sk + 16 * i, kview.codes + first * row + 16 * (size_t)i);
            cp_async16(sv + 16 * i, vview.codes + first * row + 16 * (size_t)i);
        }
        for (int i = threadIdx.x; i < scale_pieces; i += 256) {
            cp_async16(sks + 4 * i, kview.scales + first + 4 * (size_t)i);
            cp_async16(svs + 4 * i, vview.scales + first + 4 * (size_t)i);
        }
        asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
        __syncthreads();
        for (int j = c0 + halfw; j < c1; j += 4 * HALVES) {  // keys j, j + 16, j + 32, j + 48 of this half-warp
            float dot[4];
            int at[4];
            bool any = false;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int ju = j + HALVES * u;
                const bool valid = ju < c1 && !(bos_table && ju == 0);
                at[u] = (valid ? ju : j) - ca;  // (a key that does not count is read where key j is and given no weight)
                float kf[8];
                unpack8(sk + (size_t)at[u] * row, kv_bits, sub, mine, kf);
                float d = 0.f;
#pragma unroll
                for (int i = 0; i < 8; ++i) d += qreg[i] * kf[i];
                dot[u] = valid ? half_sum(d) * sks[at[u]] : -INFINITY;
                any |= valid;
            }
            if (!any) continue;  // (position 0 alone, which the side table holds)
            const float m_new = fmaxf(fmaxf(m, dot[0]), fmaxf(fmaxf(dot[1], dot[2]), dot[3]));
            const float corr = exp2a((m - m_new) * kLog2e);
            float pr[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) pr[u] = exp2a((dot[u] - m_new) * kLog2e);
            l = l * corr + ((pr[0] + pr[1]) + (pr[2] + pr[3]));
#pragma unroll
            for (int i = 0; i < 8; ++i) o[i] *= corr;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                float vf[8];
                unpack8(sv + (size_t)at[u] * row, kv_bits, sub, mine, vf);
                const float pv = pr[u] * svs[at[u]];
#pragma unroll
                for (int i = 0; i < 8; ++i) o[i] += pv * vf[i];
            }
            m = m_new;
        }
    }
    if (sub == 0) {
        sm_m[halfw] = m;
        sm_l[halfw] = l;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) sm_o[halfw][8 * sub + i] = o[i];
    __syncthreads();
    if (threadIdx.x < 128) {
        const int col = threadIdx.x;
        float mm = -INFINITY;
        for (int w = 0; w < HALVES; ++w) mm = fmaxf(mm, sm_m[w]);
        float ll = 0.f, acc = 0.f;
        for (int w = 0; w < HALVES; ++w) {
            if (sm_m[w] == -INFINITY) continue;
            const float f = expf(sm_m[w] - mm);
            ll += sm_l[w] * f;
            acc += sm_o[w][col] * f;
        }
        if (col == 0) {
            cta_ml[0] = mm;
            cta_ml[1] = ll;
        }
        cta_o[col] = acc;
    }
    cluster_sync_all();  // every CTA's partial is in its shared memory
    constexpr int CPR = 128 / ATTN_SPLITS;  // columns finished by each rank
    if (threadIdx.x < CPR) {
        const int col = split * CPR + (int)threadIdx.x;
        float pm[ATTN_SPLITS], pl[ATTN_SPLITS], po[ATTN_SPLITS];
#pragma unroll
        for (int r = 0; r < ATTN_SPLITS; ++r) {
            pm[r] = ld_cluster_f32(&cta_ml[0], (unsigned)r);
            pl[r] = ld_cluster_f32(&cta_ml[1], (unsigned)r);
            po[r] = ld_cluster_f32(&cta_o[col], (unsigned)r);
        }
        float mm = -INFINITY;
#pragma unroll
        for (int r = 0; r < ATTN_SPLITS; ++r) mm = fmaxf(mm, pm[r]);
        float ll = 0.f, acc = 0.f;
#pragma unroll
        for (int r = 0; r < ATTN_SPLITS; ++r) {
            const float f = pm[r] == -INFINITY ? 0.f : expf(pm[r] - mm);
            ll += pl[r] * f;
            acc += po[r] * f;
        }
        if (col < hd) out[((size_t)b * T + t) * H + (size_t)h * hd + col] = acc / ll;
    }
    cluster_sync_all();  // nobody leaves while a peer may still read its shared memory
}

}  // namespace

size_t a48_kv_cache_bytes(int B, int nh, int cap, int hd, int bits) {
    if (bits == 0) return (size_t)B * nh * cap * hd * 4;
    const size_t codes = ((size_t)B * nh * cap * row_bytes(hd, bits) + 15) / 16 * 16;
    const size_t scales = ((size_t)B * nh * cap * 4 + 15) / 16 * 16;
    const size_t bos = bits == 3 ? ((size_t)B * nh * row_bytes(hd, 4) + 15) / 16 * 16 : 0;
    return codes + scales + bos + 16;  // (the attention kernel copies whole 16-byte pieces: slack for the last one)
}

bitnet_a48_status a48_launch_rope_quant_cache(float* q, const float* k, const float* v, const float2* table, double base,
                                              int B, int T, int nh,
                                              int hd, int pos0, int cap, int q_bits, int kv_bits, float eps, void* kcache,
                                              void* vcache, float* dq_k, float* dq_v, cudaStream_t st) {
    if (hd > 128 || hd % 4 != 0) return BITNET_A48_ERR_UNSUPPORTED;
    const long long warps = (long long)B * T * nh;
    const unsigned blocks = (unsigned)((warps * 32 + 255) / 256);
    A48_CUDA_TRY(a48_launch_pdl(rope_quant_cache_kernel, dim3(blocks), dim3(256), 0, st, q, k, v, table, base, B, T, nh, hd, pos0,
                                cap, q_bits, kv_bits, (double)eps, kcache, vcache, dq_k, dq_v));
    return BITNET_A48_OK;
}

bitnet_a48_status a48_launch_dequant_prefix(const void* kcache, const void* vcache, int B, int nh, int hd, int pos0, int cap, int rows,
                                            int kv_bits, float* dq_k, float* dq_v, cudaStream_t st) {
    if (hd > 128 || hd % 4 != 0 || pos0 <= 0) return BITNET_A48_ERR_UNSUPPORTED;
    const long long warps = (long long)B * nh * pos0;
    const unsigned blocks = (unsigned)((warps * 32 + 255) / 256);
    A48_CUDA_TRY(a48_launch_pdl(dequant_prefix_kernel, dim3(blocks), dim3(256), 0, st, kcache, vcache, B, nh, hd, pos0, cap, rows,
                                kv_bits, dq_k, dq_v));
    return BITNET_A48_OK;
}

bitnet_a48_status a48_launch_attn_row_lowbit(const float* q, const void* kcache, const void* vcache, int B, int T, int nh,
                                             int hd, int pos0, int cap, int kv_bits, float* out, cudaStream_t st) {
    if (hd > 128) return BITNET_A48_ERR_UNSUPPORTED;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ATTN_SPLITS, (unsigned)nh, (unsigned)(B * T));
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = ATTN_SPLITS;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    const size_t rows_bytes = ((size_t)(kChunkKeys + 3) * row_bytes(hd, kv_bits) + 15) / 16 * 16;
    cfg.dynamicSmemBytes = 2 * rows_bytes + 2 * (size_t)(kChunkKeys + 4) * sizeof(float);  // at most 36 KB
    A48_CUDA_TRY(cudaLaunchKernelEx(&cfg, attn_row_lowbit_kernel, q, kcache, vcache, B, T, nh, hd, pos0, cap, kv_bits,
                                    1.f / sqrtf((float)hd), out));
    return BITNET_A48_OK;
}
