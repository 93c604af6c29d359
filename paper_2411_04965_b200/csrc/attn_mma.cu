// Causal softmax attention for prefill on the tensor cores (the block glue around the BitLinears, Section 2.1).
//
// Attention is two contractions per head, S = Q K^T and O = P V, which the fp32 SIMT kernel of block.cu runs at a
// few per cent of what the tensor cores do.  The block's tolerance against the float64 oracle does not allow plain
// bf16 or tf32 operands: a score that is 1e-3 off moves its probability by as much, and the quantisers that follow
// the attention turn a 1e-5 difference into flipped codes.  So every operand is split into three bf16 numbers,
// x = x0 + x1 + x2 with x0 = bf16(x), x1 = bf16(x - x0), x2 = bf16(x - x0 - x1) (the subtractions are exact, the
// three carry the 24 significant bits of x), and every product is the six MMAs x_i * y_j with i + j <= 2, accumulated
// in fp32.  What is dropped is below 2^-24 of a product: fp32 accuracy at a sixth of the bf16 tensor rate, still
// twice the SIMT kernel.  Measured against a float64 attention on random heads, the result is two to ten times closer
// than a sequential fp32 evaluation; with two parts (three MMAs) it is ten times further away, which the quantisers
// after the attention turn into flipped codes.
//
// Two kernels.  split_heads_kernel writes the three parts of the queries of the call and of the keys and values of
// positions [0, pos0 + T) (read from the fp32 cache) as bf16 arrays [B][heads][rows padded to a tile][head dim
// padded to 16], zero-filled padding.  attn_mma_kernel: one CTA per (128 queries, head, sequence), 8 warps of 16
// query rows each; the query parts stay in shared memory, key/value tiles of BK positions are double-buffered with
// cp.async; mma.sync.m16n8k16 with ldmatrix-fed fragments (transposed loads for V), online softmax on the
// accumulator fragments in registers, the probabilities re-used as the A operand of the second contraction without
// leaving registers.
#include <cuda_bf16.h>

#include "internal.h"

namespace {

constexpr int BQ = 128, WARPS = 8, THREADS = 32 * WARPS, PAD = 8, NS = 3;
// key/value positions per tile: what two stages of 2 * NS arrays leave room for beside the query parts
__host__ __device__ constexpr int tile_keys(int hdp) { return hdp <= 64 ? 64 : 32; }
constexpr int kKeyPad = 64;  // key rows of the split arrays are padded to this (covers both tile sizes)

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src)
                 : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* smem_row) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"((uint32_t)__cvta_generic_to_shared(smem_row)));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* smem_row) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"((uint32_t)__cvta_generic_to_shared(smem_row)));
}
// D[16x8] += A[16x16] (bf16, row) * B[16x8] (bf16, col), fp32 accumulators
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// The tensor core adds its products to the accumulator with truncation, so every MMA costs up to one unit in the last
// place of whatever the accumulator holds, always toward zero.  The leading products (part 0 times part 0) and the
// correction products (orders 1 .. NS - 1, 2^-8 and less of the leading ones) therefore go to different accumulators:
// the corrections are truncated at their own small magnitude, and the leading sum sees one MMA per step of 16.
// One step of 16 along the contraction for up to four 8-wide column blocks: a = the parts of the A fragment, b[p] =
// the parts of the B fragments of column blocks 2p and 2p + 1.  Consecutive MMAs go to different accumulators, so that
// none waits for the one before it.
__device__ __forceinline__ void mma_group(float (&lead)[4][4], float (&corr)[4][4], const uint32_t (&a)[NS][4],
                                          const uint32_t (&b)[2][NS][4], int blocks) {
#pragma unroll
    for (int order = NS - 1; order >= 1; --order)
#pragma unroll
        for (int ia = 0; ia <= order; ++ia)
#pragma unroll
            for (int n = 0; n < 4; ++n)
                if (n < blocks) mma_bf16(corr[n], a[ia], b[n >> 1][order - ia][2 * (n & 1)], b[n >> 1][order - ia][2 * (n & 1) + 1]);
#pragma unroll
    for (int n = 0; n < 4; ++n)
        if (n < blocks) mma_bf16(lead[n], a[0], b[n >> 1][0][2 * (n & 1)], b[n >> 1][0][2 * (n & 1) + 1]);
}
// a pair of floats as the NS bf16x2 words of their parts (first value in the low half)
__device__ __forceinline__ void split2(float x, float y, uint32_t (&w)[NS]) {
#pragma unroll
    for (int i = 0; i < NS; ++i) {
        const __nv_bfloat16 xb = __float2bfloat16_rn(x), yb = __float2bfloat16_rn(y);
        w[i] = (uint32_t)__bfloat16_as_ushort(xb) | ((uint32_t)__bfloat16_as_ushort(yb) << 16);
        x -= __bfloat162float(xb);
        y -= __bfloat162float(yb);
    }
}

// src rows of hd floats -> NS arrays (part_stride elements apart) of rows of hdp bf16, zero past hd and for rows >=
// rows_valid.  mode 0: queries, src = q [B*T][nh*hd], row (b, h, r) = token r of sequence b; mode 1: cache
// [B][nh][cap][hd].
__global__ void __launch_bounds__(256) split_heads_kernel(const float* __restrict__ src, int mode, int B, int nh, int hd, int hdp,
                                                          int rows_valid, int rows_pad, int T, int cap,
                                                          __nv_bfloat16* __restrict__ parts, size_t part_stride) {
    a48_pdl_prologue();
    const int pairs = hdp / 2;
    const size_t total = (size_t)B * nh * rows_pad * pairs;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % pairs) * 2;
        const size_t row = i / pairs;
        const int r = (int)(row % rows_pad);
        const size_t bh = row / rows_pad;
        const int h = (int)(bh % nh), b = (int)(bh / nh);
        float x = 0.f, y = 0.f;
        if (r < rows_valid && c < hd) {
            const float* p = mode == 0 ? src + ((size_t)b * T + r) * ((size_t)nh * hd) + (size_t)h * hd + c
                                       : src + (((size_t)b * nh + h) * cap + r) * hd + c;
            x = p[0];
            y = c + 1 < hd ? p[1] : 0.f;
        }
        uint32_t w[NS];
        split2(x, y, w);
#pragma unroll
        for (int a = 0; a < NS; ++a) reinterpret_cast<uint32_t*>(parts + a * part_stride)[i] = w[a];
    }
}

// Dynamic shared memory (bf16): the NS query parts [BQ][HDP+PAD], then two stages of NS key parts and NS value parts
// [BK][HDP+PAD].  qs / ks / vs: part 0 of the split arrays, the other parts q_stride / kv_stride elements apart.
template <int HDP>
__global__ void __launch_bounds__(THREADS, 1) attn_mma_kernel(const __nv_bfloat16* __restrict__ qs, size_t q_stride,
                                                              const __nv_bfloat16* __restrict__ ks, const __nv_bfloat16* __restrict__ vs,
                                                              size_t kv_stride, int T, int t_pad, int n_keys, int k_pad, int nh, int hd,
                                                              int pos0, float scale, float* __restrict__ out) {
    constexpr int BK = tile_keys(HDP), LD = HDP + PAD, KS = HDP / 16, NB = HDP / 8;
    extern __shared__ __align__(16) __nv_bfloat16 smem[];
    __nv_bfloat16* sq = smem;                 // part a: sq + a * BQ * LD
    __nv_bfloat16* skv = smem + NS * BQ * LD;  // stage s, array a (K parts, then V parts): skv + (s * 2 * NS + a) * BK * LD
    a48_pdl_prologue();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tq = lane & 3;
    const int q0 = blockIdx.x * BQ, h = blockIdx.y, b = blockIdx.z;
    const size_t bh = (size_t)b * nh + h;
    const __nv_bfloat16* gq = qs + (bh * t_pad + q0) * HDP;
    const __nv_bfloat16* gk = ks + bh * k_pad * HDP;
    const __nv_bfloat16* gv = vs + bh * k_pad * HDP;
    constexpr int CH = HDP / 8;  // 16-byte chunks per row
    for (int i = tid; i < NS * BQ * CH; i += THREADS) {
        const int a = i / (BQ * CH), r = (i / CH) % BQ, c = i % CH;
        cp_async16(sq + (a * BQ + r) * LD + c * 8, gq + a * q_stride + (size_t)r * HDP + c * 8);
    }
    auto load_tile = [&](int stage, int k0) {
        for (int i = tid; i < 2 * NS * BK * CH; i += THREADS) {
            const int a = i / (BK * CH), r = (i / CH) % BK, c = i % CH;
            const __nv_bfloat16* src = (a < NS ? gk + a * kv_stride : gv + (a - NS) * kv_stride) + (size_t)(k0 + r) * HDP + c * 8;
            cp_async16(skv + ((stage * 2 * NS + a) * BK + r) * LD + c * 8, src);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    const int q_last = min(q0 + BQ, T) - 1;
    const int keys_needed = min(n_keys, pos0 + q_last + 1);  // causal: nothing beyond the last query's own position
    const int n_tiles = (keys_needed + BK - 1) / BK;
    load_tile(0, 0);  // (its group also covers the query copies above)

    float o[NB][4];
#pragma unroll
    for (int n = 0; n < NB; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};  // rows g and g + 8 of this warp's 16
    const int row0 = q0 + warp * 16 + g;                              // query index of row g (row g + 8: + 8)
    // ldmatrix row addresses: A fragments (row = lane % 16, k half = lane / 16), B fragments of two key blocks
    // (key = lane % 8 + 8 * (lane / 16), k half = (lane / 8) % 2), transposed V fragments (key = lane % 16, dim half = lane / 16)
    const int a_row = warp * 16 + (lane & 15), a_col = (lane >> 4) * 8;
    const int b_row = (lane & 7) + ((lane >> 4) << 3), b_col = ((lane >> 3) & 1) * 8;
    const int v_row = lane & 15, v_col = (lane >> 4) * 8;

    for (int tile = 0; tile < n_tiles; ++tile) {
        const int stage = tile & 1, k0 = tile * BK;
        if (tile + 1 < n_tiles) {
            load_tile(stage ^ 1, k0 + BK);
            asm volatile("cp.async.wait_group 1;" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncthreads();
        const __nv_bfloat16* sk = skv + (stage * 2 * NS) * BK * LD;       // part a: sk + a * BK * LD
        const __nv_bfloat16* sv = skv + (stage * 2 * NS + NS) * BK * LD;  // part a: sv + a * BK * LD
        // ---- S = Q K^T for this warp's 16 rows and the tile's keys
        float s[BK / 32][4][4], sc[BK / 32][4][4];  // [group of 32 keys][block of 8 keys]: leading products | corrections
#pragma unroll
        for (int gk = 0; gk < BK / 32; ++gk)
#pragma unroll
            for (int n = 0; n < 4; ++n)
#pragma unroll
                for (int e = 0; e < 4; ++e) s[gk][n][e] = sc[gk][n][e] = 0.f;
#pragma unroll
        for (int kk = 0; kk < KS; ++kk) {
            uint32_t qa[NS][4];
#pragma unroll
            for (int a = 0; a < NS; ++a) ldmatrix_x4(qa[a], sq + (a * BQ + a_row) * LD + kk * 16 + a_col);
#pragma unroll
            for (int gk = 0; gk < BK / 32; ++gk) {
                uint32_t kb[2][NS][4];  // two key blocks per ldmatrix
#pragma unroll
                for (int p = 0; p < 2; ++p)
#pragma unroll
                    for (int a = 0; a < NS; ++a) ldmatrix_x4(kb[p][a], sk + (a * BK + gk * 32 + p * 16 + b_row) * LD + kk * 16 + b_col);
                mma_group(s[gk], sc[gk], qa, kb, 4);
            }
        }
        // ---- scale, causal mask, online softmax (rows g and g + 8; a row's scores sit in the 4 lanes of a quad)
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int n = 0; n < BK / 8; ++n) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int key = k0 + n * 8 + 2 * tq + (e & 1), qrow = row0 + (e >> 1) * 8;
                const bool ok = key <= pos0 + qrow && key < n_keys;
                float& v = s[n >> 2][n & 3][e];
                v = ok ? (v + sc[n >> 2][n & 3][e]) * scale : -INFINITY;
                mx[e >> 1] = fmaxf(mx[e >> 1], v);
            }
        }
        float corr[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
            const float m_new = fmaxf(m_run[r], mx[r]);
            corr[r] = (m_run[r] == -INFINITY) ? 0.f : expf(m_run[r] - m_new);
            m_run[r] = m_new;
        }
        float sum[2] = {0.f, 0.f};
        uint32_t pw[BK / 8][2][NS];  // the parts of the probabilities as bf16x2: [key block][row g | row g + 8][part]
#pragma unroll
        for (int n = 0; n < BK / 8; ++n) {
            float p[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float mr = m_run[e >> 1];
                const float v = s[n >> 2][n & 3][e];
                p[e] = (v == -INFINITY || mr == -INFINITY) ? 0.f : expf(v - mr);
                sum[e >> 1] += p[e];
            }
            split2(p[0], p[1], pw[n][0]);
            split2(p[2], p[3], pw[n][1]);
        }
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            sum[r] += __shfl_xor_sync(0xffffffffu, sum[r], 1);
            sum[r] += __shfl_xor_sync(0xffffffffu, sum[r], 2);
            l_run[r] = l_run[r] * corr[r] + sum[r];
        }
#pragma unroll
        for (int n = 0; n < NB; ++n) {
            o[n][0] *= corr[0];
            o[n][1] *= corr[0];
            o[n][2] *= corr[1];
            o[n][3] *= corr[1];
        }
        // ---- O += P V: the accumulator fragments of two key blocks are the A fragment of one 16-key step.  The tile's
        // contribution is summed in accumulators of its own (corrections first) and added to O in fp32 afterwards, so
        // that O itself is rounded to nearest once per tile instead of truncated by every MMA.
        uint32_t pa[BK / 16][NS][4];
#pragma unroll
        for (int kk = 0; kk < BK / 16; ++kk)
#pragma unroll
            for (int a = 0; a < NS; ++a) {
                pa[kk][a][0] = pw[2 * kk][0][a];
                pa[kk][a][1] = pw[2 * kk][1][a];
                pa[kk][a][2] = pw[2 * kk + 1][0][a];
                pa[kk][a][3] = pw[2 * kk + 1][1][a];
            }
#pragma unroll
        for (int gd = 0; gd < (NB + 3) / 4; ++gd) {  // groups of up to four blocks of 8 head dims
            const int blocks = NB - 4 * gd < 4 ? NB - 4 * gd : 4;
            float t[4][4], tc[4][4];
#pragma unroll
            for (int n = 0; n < 4; ++n)
#pragma unroll
                for (int e = 0; e < 4; ++e) t[n][e] = tc[n][e] = 0.f;
#pragma unroll
            for (int kk = 0; kk < BK / 16; ++kk) {
                uint32_t vb[2][NS][4];  // two blocks of 8 head dims per transposed ldmatrix
#pragma unroll
                for (int p = 0; p < 2; ++p)
                    if (2 * p < blocks)
#pragma unroll
                        for (int a = 0; a < NS; ++a)
                            ldmatrix_x4_trans(vb[p][a], sv + (a * BK + kk * 16 + v_row) * LD + (gd * 2 + p) * 16 + v_col);
                mma_group(t, tc, pa[kk], vb, blocks);
            }
#pragma unroll
            for (int n = 0; n < 4; ++n)
                if (n < blocks)
#pragma unroll
                    for (int e = 0; e < 4; ++e) o[4 * gd + n][e] += t[n][e] + tc[n][e];
        }
        __syncthreads();  // everybody is done with this stage before the copy of tile + 2 lands in it
    }
    // ---- out = O / l
    const size_t H = (size_t)nh * hd;
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int q = row0 + r * 8;
        if (q >= T) continue;
        const float inv = 1.f / l_run[r];
        float* dst = out + ((size_t)b * T + q) * H + (size_t)h * hd;
#pragma unroll
        for (int n = 0; n < NB; ++n) {
            const int col = n * 8 + 2 * tq;
            if (col < hd) dst[col] = o[n][2 * r] * inv;
            if (col + 1 < hd) dst[col + 1] = o[n][2 * r + 1] * inv;
        }
    }
}

size_t up256(size_t v) { return (v + 255) / 256 * 256; }
// the head dimension as the kernel is compiled for it (a multiple of 16 that covers hd)
int pick_hdp(int hd) { return hd <= 64 ? 64 : (hd <= 96 ? 96 : (hd <= 112 ? 112 : 128)); }

template <int HDP>
bitnet_a48_status launch_attn(const __nv_bfloat16* qs, size_t q_stride, const __nv_bfloat16* ks, const __nv_bfloat16* vs,
                              size_t kv_stride, int B, int T, int t_pad, int n_keys, int k_pad, int nh, int hd, int pos0, float* out,
                              cudaStream_t st) {
    constexpr int LD = HDP + PAD, BK = tile_keys(HDP);
    constexpr size_t smem = (size_t)(NS * BQ + 4 * NS * BK) * LD * sizeof(__nv_bfloat16);
    static_assert(smem <= 232448, "query parts and two key/value stages must fit the shared memory of one CTA");
    A48_CUDA_TRY(cudaFuncSetAttribute(attn_mma_kernel<HDP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    A48_CUDA_TRY(a48_launch_pdl(attn_mma_kernel<HDP>, dim3((T + BQ - 1) / BQ, nh, B), dim3(THREADS), smem, st, qs, q_stride, ks, vs,
                                kv_stride, T, t_pad, n_keys, k_pad, nh, hd, pos0, 1.f / sqrtf((float)hd), out));
    return BITNET_A48_OK;
}

}  // namespace

bool a48_attn_mma_supported(int hd) { return hd % 2 == 0 && hd <= 128; }

// Scratch for the split operands: the parts of the queries (rows padded to 128) and of the keys and values (rows
// padded to 64).
size_t a48_attn_mma_workspace_bytes(int B, int nh, int hd, int T, int n_keys) {
    const size_t hdp = (size_t)pick_hdp(hd), t_pad = (size_t)(T + BQ - 1) / BQ * BQ, k_pad = (size_t)(n_keys + kKeyPad - 1) / kKeyPad * kKeyPad;
    return NS * up256((size_t)B * nh * t_pad * hdp * 2) + 2 * NS * up256((size_t)B * nh * k_pad * hdp * 2);
}

// q [B*T][nh*hd] (already rotated); kcache / vcache fp32 [B][nh][cap][hd] holding positions [0, pos0 + T).
bitnet_a48_status a48_launch_attn_mma(const float* q, const float* kcache, const float* vcache, int B, int T, int nh, int hd, int pos0,
                                      int cap, float* out, void* ws, cudaStream_t st) {
    if (!a48_attn_mma_supported(hd)) return BITNET_A48_ERR_UNSUPPORTED;
    const int hdp = pick_hdp(hd), n_keys = pos0 + T;
    const int t_pad = (T + BQ - 1) / BQ * BQ, k_pad = (n_keys + kKeyPad - 1) / kKeyPad * kKeyPad;
    char* base = static_cast<char*>(ws);
    const size_t qb = up256((size_t)B * nh * t_pad * hdp * 2), kb = up256((size_t)B * nh * k_pad * hdp * 2);
    __nv_bfloat16* qs = reinterpret_cast<__nv_bfloat16*>(base);
    __nv_bfloat16* ks = reinterpret_cast<__nv_bfloat16*>(base + NS * qb);
    __nv_bfloat16* vs = reinterpret_cast<__nv_bfloat16*>(base + NS * qb + NS * kb);
    const size_t q_stride = qb / 2, kv_stride = kb / 2;
    int dev = 0, sms = 0;
    A48_CUDA_TRY(cudaGetDevice(&dev));
    A48_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const dim3 grid(sms * 8), block(256);
    A48_CUDA_TRY(a48_launch_pdl(split_heads_kernel, grid, block, 0, st, q, 0, B, nh, hd, hdp, T, t_pad, T, cap, qs, q_stride));
    A48_CUDA_TRY(a48_launch_pdl(split_heads_kernel, grid, block, 0, st, kcache, 1, B, nh, hd, hdp, n_keys, k_pad, T, cap, ks, kv_stride));
    A48_CUDA_TRY(a48_launch_pdl(split_heads_kernel, grid, block, 0, st, vcache, 1, B, nh, hd, hdp, n_keys, k_pad, T, cap, vs, kv_stride));
    switch (hdp) {
        case 64: return launch_attn<64>(qs, q_stride, ks, vs, kv_stride, B, T, t_pad, n_keys, k_pad, nh, hd, pos0, out, st);
        case 96: return launch_attn<96>(qs, q_stride, ks, vs, kv_stride, B, T, t_pad, n_keys, k_pad, nh, hd, pos0, out, st);
        case 112: return launch_attn<112>(qs, q_stride, ks, vs, kv_stride, B, T, t_pad, n_keys, k_pad, nh, hd, pos0, out, st);
        default: return launch_attn<128>(qs, q_stride, ks, vs, kv_stride, B, T, t_pad, n_keys, k_pad, nh, hd, pos0, out, st);
    }
}
