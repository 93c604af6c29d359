// Transformer block around the BitLinear calls (Section 2.1, Eq. 5): RMSNorm
// (fused into the INT4 quantiser), RoPE, causal softmax attention, ReLU²GLU and
// the residual adds.  Everything here is fp32 glue; the contractions go through
// the same quantiser and linear launchers the public entry points use.
#include "internal.h"

namespace {

size_t up256(size_t v) { return (v + 255) / 256 * 256; }

struct BlockWs {
    size_t codes, scale, q, k, v, att, hres, tmp, gate, up, rope, kc, vc, mma, lin, total;
};

BlockWs block_ws(const bitnet_a48_block* blk, int B, int T) {
    const size_t M = (size_t)B * T, H = blk->cfg.hidden, F = blk->cfg.ffn;
    const size_t hd = H / blk->cfg.n_heads;
    BlockWs w;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t r = o; o += up256(bytes); return r; };
    w.codes = take(M * (H > F ? H : F));
    w.scale = take(M * 4);
    w.q = take(M * H * 4);
    w.k = take(M * H * 4);
    w.v = take(M * H * 4);
    w.att = take(M * H * 4);
    w.hres = take(M * H * 4);
    w.tmp = take(M * H * 4);
    w.gate = take(M * F * 4);
    w.up = take(M * F * 4);
    w.rope = take((size_t)T * (hd / 2) * 8);
    // positions a call can reach: the cache's capacity, or the call's own tokens without a cache
    const int reach = blk->cfg.ctx_cap > T ? blk->cfg.ctx_cap : T;
    // keys/values of a call without a cache; with a packed cache, the fp32 copies of every reachable position that a
    // prefill hands to the attention kernel
    const size_t kv_rows = blk->cfg.kv_bits != 0 && T > 8 ? (size_t)B * reach : M;
    w.kc = take(kv_rows * H * 4);
    w.vc = take(kv_rows * H * 4);
    // operands of the tensor-core prefill attention split into bf16 parts: queries of the call, keys/values of every
    // reachable position
    w.mma = take(T > 8 && a48_attn_tc_supported((int)hd) ? a48_attn_tc_workspace_bytes(B, blk->cfg.n_heads, (int)hd, T, reach) : 0);
    size_t lin = 0;
    for (int i = 0; i < 7; ++i) {
        size_t b = bitnet_a48_linear_workspace_bytes(blk->w[i], (int)M);
        lin = b > lin ? b : lin;
    }
    {  // q,k,v and gate,up go out as one call each
        size_t b = bitnet_a48_linear_multi_workspace_bytes(3, blk->w, (int)M);
        lin = b > lin ? b : lin;
        b = bitnet_a48_linear_multi_workspace_bytes(2, blk->w + 4, (int)M);
        lin = b > lin ? b : lin;
    }
    w.lin = take(lin);
    w.total = o;
    return w;
}

// cos/sin of position * base^(-2i/head_dim), evaluated in float64, stored as fp32.
__global__ void rope_table_kernel(int pos0, int T, int half, double base, float2* __restrict__ table) {
    int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= T * half) return;
    int t = idx / half, i = idx % half;
    double ang = (double)(pos0 + t) * pow(base, -(double)i / (double)half);
    double s, c;
    sincos(ang, &s, &c);
    table[idx] = make_float2((float)c, (float)s);
}

// Rotates q in place on (i, i+hd/2) pairs, rotates k, and stores rotated k and v
// into the cache rows [b][h][pos0+t][:].  table == nullptr (a few tokens): the angle is evaluated here, with the
// expression of rope_table_kernel, instead of in a launch of its own.
__global__ void rope_cache_kernel(float* __restrict__ q, const float* __restrict__ k, const float* __restrict__ v,
                                  const float2* __restrict__ table, double base, int B, int T, int nh, int hd, int pos0,
                                  int cap, float* __restrict__ kcache, float* __restrict__ vcache) {
    a48_pdl_prologue();
    const int half = hd / 2;
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    size_t total = (size_t)B * T * nh * half;
    if (idx >= total) return;
    int i = (int)(idx % half);
    int h = (int)((idx / half) % nh);
    size_t m = idx / ((size_t)half * nh);
    int t = (int)(m % T), b = (int)(m / T);
    float2 cs;
    if (table) {
        cs = table[t * half + i];
    } else {
        double ang = (double)(pos0 + t) * pow(base, -(double)i / (double)half);
        double sn, cn;
        sincos(ang, &sn, &cn);
        cs = make_float2((float)cn, (float)sn);
    }
    size_t src = m * (size_t)nh * hd + (size_t)h * hd + i;
    float ql = q[src], qh = q[src + half];
    q[src] = ql * cs.x - qh * cs.y;
    q[src + half] = qh * cs.x + ql * cs.y;
    float kl = k[src], kh = k[src + half];
    size_t dst = (((size_t)b * nh + h) * cap + (pos0 + t)) * hd + i;
    kcache[dst] = kl * cs.x - kh * cs.y;
    kcache[dst + half] = kh * cs.x + kl * cs.y;
    vcache[dst] = v[src];
    vcache[dst + half] = v[src + half];
}

// Causal softmax(q k^T / sqrt(hd)) v for query tiles of 64, keys streamed in tiles
// of 64 through shared memory, fp32 throughout, online softmax.
// grid: (ceil(T/64), nh, B); block: 256 threads as 16 (query groups) x 16.
template <int HDP>
__global__ void __launch_bounds__(256) attn_tile_kernel(const float* __restrict__ q, const float* __restrict__ kcache,
                                                        const float* __restrict__ vcache, int T, int nh, int hd,
                                                        int pos0, int cap, float scale, float* __restrict__ out) {
    constexpr int BQ = 64, BK = 64, LD = HDP + 4, LDS_ = BK + 1, CPT = HDP / 16;
    extern __shared__ float smem[];
    float* Qs = smem;               // [BQ][LD]
    float* Ks = Qs + BQ * LD;       // [BK][LD]
    float* Vs = Ks + BK * LD;       // [BK][LD]
    float* Ss = Vs + BK * LD;       // [BQ][LDS_]
    float* row_m = Ss + BQ * LDS_;  // [BQ]
    float* row_l = row_m + BQ;
    float* row_c = row_l + BQ;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int q0 = blockIdx.x * BQ, h = blockIdx.y, b = blockIdx.z;
    const size_t H = (size_t)nh * hd;
    const float* kbase = kcache + ((size_t)b * nh + h) * cap * hd;
    const float* vbase = vcache + ((size_t)b * nh + h) * cap * hd;

    for (int i = tid; i < BQ * (HDP / 4); i += 256) {
        int r = i / (HDP / 4), c4 = i % (HDP / 4);
        float4 val = make_float4(0.f, 0.f, 0.f, 0.f);
        if (q0 + r < T && c4 * 4 < hd)
            val = *reinterpret_cast<const float4*>(q + ((size_t)b * T + q0 + r) * H + (size_t)h * hd + c4 * 4);
        *reinterpret_cast<float4*>(Qs + r * LD + c4 * 4) = val;
    }
    if (tid < BQ) {
        row_m[tid] = -INFINITY;
        row_l[tid] = 0.f;
    }
    float o[4][CPT];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int c = 0; c < CPT; ++c) o[i][c] = 0.f;

    const int q_last = min(q0 + BQ, T) - 1;
    const int n_keys = pos0 + q_last + 1;  // causal: keys up to the last query's own position
    for (int k0 = 0; k0 < n_keys; k0 += BK) {
        __syncthreads();
        for (int i = tid; i < BK * (HDP / 4); i += 256) {
            int r = i / (HDP / 4), c4 = i % (HDP / 4);
            float4 kv = make_float4(0.f, 0.f, 0.f, 0.f), vv = kv;
            if (k0 + r < n_keys && c4 * 4 < hd) {
                kv = *reinterpret_cast<const float4*>(kbase + (size_t)(k0 + r) * hd + c4 * 4);
                vv = *reinterpret_cast<const float4*>(vbase + (size_t)(k0 + r) * hd + c4 * 4);
            }
            *reinterpret_cast<float4*>(Ks + r * LD + c4 * 4) = kv;
            *reinterpret_cast<float4*>(Vs + r * LD + c4 * 4) = vv;
        }
        __syncthreads();
        // S sub-tile: queries 4ty..4ty+3, keys tx, tx+16, tx+32, tx+48
        float s[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) s[i][j] = 0.f;
#pragma unroll 4
        for (int d = 0; d < HDP; d += 4) {
            float4 qa[4], ka[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) qa[i] = *reinterpret_cast<const float4*>(Qs + (4 * ty + i) * LD + d);
#pragma unroll
            for (int j = 0; j < 4; ++j) ka[j] = *reinterpret_cast<const float4*>(Ks + (tx + 16 * j) * LD + d);
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    s[i][j] += qa[i].x * ka[j].x + qa[i].y * ka[j].y + qa[i].z * ka[j].z + qa[i].w * ka[j].w;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                int qpos = pos0 + q0 + 4 * ty + i, kpos = k0 + tx + 16 * j;
                Ss[(4 * ty + i) * LDS_ + tx + 16 * j] = (kpos <= qpos && kpos < n_keys) ? s[i][j] * scale : -INFINITY;
            }
        __syncthreads();
        {  // online softmax: 4 threads per query row, 16 keys each
            int r = tid >> 2, part = tid & 3;
            float mx = -INFINITY;
#pragma unroll
            for (int j = 0; j < 16; ++j) mx = fmaxf(mx, Ss[r * LDS_ + part * 16 + j]);
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            float m_old = row_m[r], m_new = fmaxf(m_old, mx);
            float sum = 0.f;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                float sv = Ss[r * LDS_ + part * 16 + j];
                float p = (sv == -INFINITY) ? 0.f : expf(sv - m_new);
                Ss[r * LDS_ + part * 16 + j] = p;
                sum += p;
            }
            sum += __shfl_xor_sync(0xffffffffu, sum, 1);
            sum += __shfl_xor_sync(0xffffffffu, sum, 2);
            float corr = (m_old == -INFINITY) ? 0.f : expf(m_old - m_new);
            __syncwarp();
            if (part == 0) {
                row_m[r] = m_new;
                row_l[r] = row_l[r] * corr + sum;
                row_c[r] = corr;
            }
        }
        __syncthreads();
        // O = O*corr + P V : queries 4ty..4ty+3, columns tx*CPT..tx*CPT+CPT-1
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float c = row_c[4 * ty + i];
#pragma unroll
            for (int cc = 0; cc < CPT; ++cc) o[i][cc] *= c;
        }
#pragma unroll 4
        for (int kk = 0; kk < BK; ++kk) {
            float p[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) p[i] = Ss[(4 * ty + i) * LDS_ + kk];
            float vreg[CPT];
#pragma unroll
            for (int c4 = 0; c4 < CPT / 4; ++c4) {
                float4 t4 = *reinterpret_cast<const float4*>(Vs + kk * LD + tx * CPT + c4 * 4);
                vreg[c4 * 4 + 0] = t4.x; vreg[c4 * 4 + 1] = t4.y; vreg[c4 * 4 + 2] = t4.z; vreg[c4 * 4 + 3] = t4.w;
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int cc = 0; cc < CPT; ++cc) o[i][cc] += p[i] * vreg[cc];
        }
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int r = 4 * ty + i;
        if (q0 + r >= T) continue;
        float inv = 1.f / row_l[r];
#pragma unroll
        for (int cc = 0; cc < CPT; ++cc) {
            int col = tx * CPT + cc;
            if (col < hd) out[((size_t)b * T + q0 + r) * H + (size_t)h * hd + col] = o[i][cc] * inv;
        }
    }
}

// Few queries per sequence (decode): the keys of one (query, head, batch) are split over the ATTN_SPLITS CTAs
// of a thread-block cluster, so that a batch-1 step at a 2048-token context runs on 256 CTAs instead of 32 and
// streams the fp32 cache at memory speed.  Inside a CTA the 8 warps stride over the keys, four keys per
// iteration (their loads are in flight together), each lane holding hd/32 (rounded up) columns; online softmax
// per warp, warps meet in shared memory.  The CTAs of a cluster then combine through distributed shared memory:
// rank r reads every rank's (max, sum) and its own 1/ATTN_SPLITS share of the output columns.
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

// AHEAD: the loads of the next four keys are issued before the current four are taken.  With few CTAs (one sequence)
// a warp's rounds of loads are what is left to wait for; with many CTAs their number hides them and the registers are
// better spent on residency.
template <int CPL, bool AHEAD>
__global__ void __launch_bounds__(256) attn_row_kernel(const float* __restrict__ q, const float* __restrict__ kcache,
                                                       const float* __restrict__ vcache, int T, int nh, int hd,
                                                       int pos0, int cap, float scale, float* __restrict__ out) {
    constexpr int COLS = 32 * CPL;
    static_assert(COLS % ATTN_SPLITS == 0, "every rank finishes the same number of columns");
    __shared__ float sm_m[8], sm_l[8];
    __shared__ float sm_o[8][COLS];
    __shared__ float cta_ml[2];  // this CTA's running max and sum, read by the peers
    __shared__ float cta_o[COLS];
    a48_pdl_prologue();
    const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z / T, t = blockIdx.z % T;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const size_t H = (size_t)nh * hd;
    const float* qr = q + ((size_t)b * T + t) * H + (size_t)h * hd;
    const float* kbase = kcache + ((size_t)b * nh + h) * cap * hd;
    const float* vbase = vcache + ((size_t)b * nh + h) * cap * hd;
    // Rows that are a whole number of 128-byte lines (head dim a multiple of 32): lane l owns the CPL consecutive head
    // dims CPL*l .. CPL*l + CPL-1 and reads them with one or two 128-bit loads (64-bit at CPL = 2).  Other head dims
    // (100): lane l owns l, l + 32, ..., one 32-bit load each - measured, the wide loads lose a fifth of the bandwidth
    // on rows that start in the middle of a line.
    const bool vec = (hd & 31) == 0;
    auto col_of = [&](int c) { return vec ? lane * CPL + c : lane + 32 * c; };
    const bool whole = vec && lane * CPL + CPL <= hd;
    float qreg[CPL], o[CPL];
#pragma unroll
    for (int c = 0; c < CPL; ++c) {
        qreg[c] = col_of(c) < hd ? qr[col_of(c)] * scale : 0.f;
        o[c] = 0.f;
    }
    float m = -INFINITY, l = 0.f;
    const int n_keys = pos0 + t + 1;
    const int per = (n_keys + ATTN_SPLITS - 1) / ATTN_SPLITS;
    const int j_end = min(n_keys, (split + 1) * per);
    auto load_row = [&](const float* __restrict__ row, float (&x)[CPL]) {
        if (whole) {
            if constexpr (CPL == 2) {
                const float2 f = __ldg(reinterpret_cast<const float2*>(row + lane * CPL));
                x[0] = f.x, x[1] = f.y;
            } else {
#pragma unroll
                for (int c = 0; c < CPL; c += 4) {
                    const float4 f = __ldg(reinterpret_cast<const float4*>(row + lane * CPL + c));
                    x[c] = f.x, x[c + 1] = f.y, x[c + 2] = f.z, x[c + 3] = f.w;
                }
            }
        } else if (vec) {  // lanes past the head have nothing to read
#pragma unroll
            for (int c = 0; c < CPL; ++c) x[c] = 0.f;
        } else {
#pragma unroll
            for (int c = 0; c < CPL; ++c) x[c] = lane + 32 * c < hd ? __ldg(row + lane + 32 * c) : 0.f;
        }
    };
    // The kernel is bound by the instructions it issues per key, so four keys share one step of the online softmax
    // (one rescale of the running output instead of four), and the exponentials are ex2.approx of a difference
    // times log2 e (two units in the last place, as in the prefill kernel; 2^-inf = 0 covers keys past the end).
    constexpr float kLog2e = 1.4426950408889634f;
    auto exp2a = [](float x) {
        float y;
        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
        return y;
    };
    auto load4 = [&](int j, float (&kk)[4][CPL], float (&vv)[4][CPL]) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int jj = max(min(j + 8 * u, j_end - 1), 0);  // (a row past the end is read again and given no weight)
            load_row(kbase + (size_t)jj * hd, kk[u]);
            load_row(vbase + (size_t)jj * hd, vv[u]);
        }
    };
    auto take4 = [&](int j, const float (&kk)[4][CPL], const float (&vv)[4][CPL]) {
        float dot[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            dot[u] = 0.f;
#pragma unroll
            for (int c = 0; c < CPL; ++c) dot[u] += qreg[c] * kk[u][c];
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
#pragma unroll
            for (int u = 0; u < 4; ++u) dot[u] += __shfl_xor_sync(0xffffffffu, dot[u], off);
        }
#pragma unroll
        for (int u = 1; u < 4; ++u)
            if (j + 8 * u >= j_end) dot[u] = -INFINITY;
        const float m_new = fmaxf(fmaxf(m, dot[0]), fmaxf(fmaxf(dot[1], dot[2]), dot[3]));  // finite: key j exists
        const float corr = exp2a((m - m_new) * kLog2e);
        float pr[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) pr[u] = exp2a((dot[u] - m_new) * kLog2e);
        l = l * corr + ((pr[0] + pr[1]) + (pr[2] + pr[3]));
#pragma unroll
        for (int c = 0; c < CPL; ++c)
            o[c] = o[c] * corr + ((pr[0] * vv[0][c] + pr[1] * vv[1][c]) + (pr[2] * vv[2][c] + pr[3] * vv[3][c]));
        m = m_new;
    };
    const int j0 = split * per + warp;
    if constexpr (AHEAD) {
        float ka[4][CPL], va[4][CPL], kb[4][CPL], vb[4][CPL];
        if (j0 < j_end) load4(j0, ka, va);
        for (int j = j0; j < j_end; j += 64) {
            if (j + 32 < j_end) load4(j + 32, kb, vb);
            take4(j, ka, va);
            if (j + 64 < j_end) load4(j + 64, ka, va);
            if (j + 32 < j_end) take4(j + 32, kb, vb);
        }
    } else {
        for (int j = j0; j < j_end; j += 32) {
            float kk[4][CPL], vv[4][CPL];
            load4(j, kk, vv);
            take4(j, kk, vv);
        }
    }
    if (lane == 0) {
        sm_m[warp] = m;
        sm_l[warp] = l;
    }
#pragma unroll
    for (int c = 0; c < CPL; ++c) sm_o[warp][col_of(c)] = o[c];
    __syncthreads();
    if (warp == 0) {
        float mm = -INFINITY;
        for (int w = 0; w < 8; ++w) mm = fmaxf(mm, sm_m[w]);
        float ll = 0.f;
        float acc[CPL];
#pragma unroll
        for (int c = 0; c < CPL; ++c) acc[c] = 0.f;
        for (int w = 0; w < 8; ++w) {
            if (sm_m[w] == -INFINITY) continue;
            float f = expf(sm_m[w] - mm);
            ll += sm_l[w] * f;
#pragma unroll
            for (int c = 0; c < CPL; ++c) acc[c] += sm_o[w][col_of(c)] * f;
        }
        if (lane == 0) {
            cta_ml[0] = mm;
            cta_ml[1] = ll;
        }
#pragma unroll
        for (int c = 0; c < CPL; ++c) cta_o[col_of(c)] = acc[c];
    }
    cluster_sync_all();  // every CTA's partial is in its shared memory
    constexpr int CPR = COLS / ATTN_SPLITS;  // columns finished by each rank
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

template <int CPL>
cudaError_t launch_attn_row(const float* q, const float* kcache, const float* vcache, int B, int T, int nh, int hd,
                            int pos0, int cap, float* out, cudaStream_t st) {
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
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const float scale = 1.f / sqrtf((float)hd);
    if ((long long)ATTN_SPLITS * nh * B * T <= 2ll * sms)
        return cudaLaunchKernelEx(&cfg, attn_row_kernel<CPL, true>, q, kcache, vcache, T, nh, hd, pos0, cap, scale, out);
    return cudaLaunchKernelEx(&cfg, attn_row_kernel<CPL, false>, q, kcache, vcache, T, nh, hd, pos0, cap, scale, out);
}

__global__ void add_kernel(const float* __restrict__ a, const float* __restrict__ b, float* __restrict__ y, size_t n4) {
    a48_pdl_prologue();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n4) return;
    float4 x = reinterpret_cast<const float4*>(a)[i], z = reinterpret_cast<const float4*>(b)[i];
    reinterpret_cast<float4*>(y)[i] = make_float4(x.x + z.x, x.y + z.y, x.z + z.z, x.w + z.w);
}

// Eq. 5: up ⊙ ReLU²(gate), written over gate.
__global__ void relu2glu_kernel(float* __restrict__ gate, const float* __restrict__ up, size_t n4) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n4) return;
    float4 g = reinterpret_cast<float4*>(gate)[i], u = reinterpret_cast<const float4*>(up)[i];
    auto f = [](float gg, float uu) { float r = gg > 0.f ? gg : 0.f; return uu * (r * r); };
    reinterpret_cast<float4*>(gate)[i] = make_float4(f(g.x, u.x), f(g.y, u.y), f(g.z, u.z), f(g.w, u.w));
}

template <int HDP>
bitnet_a48_status launch_attn_tile(const float* q, const float* kc, const float* vc, int B, int T, int nh, int hd,
                                   int pos0, int cap, float* out, cudaStream_t st) {
    constexpr int LD = HDP + 4;
    size_t smem = (size_t)(3 * 64 * LD + 64 * 65 + 3 * 64) * sizeof(float);
    A48_CUDA_TRY(cudaFuncSetAttribute(attn_tile_kernel<HDP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    dim3 grid((T + 63) / 64, nh, B);
    attn_tile_kernel<HDP><<<grid, 256, smem, st>>>(q, kc, vc, T, nh, hd, pos0, cap, 1.f / sqrtf((float)hd), out);
    return BITNET_A48_OK;
}

// Prefill attention: the tensor-core kernel where it takes the shape (head dim <= 128, tensor-copy coordinates within
// 32 bits), the fp32 tile kernel otherwise.
bitnet_a48_status prefill_attention(const float* q, const float* kc, const float* vc, int B, int T, int nh, int hd, int pos0,
                                    int cap, float* att, void* mma_ws, cudaStream_t st) {
    if (a48_attn_tc_supported(hd)) {
        const bitnet_a48_status s = a48_launch_attn_tc(q, kc, vc, B, T, nh, hd, pos0, cap, att, mma_ws, st);
        if (s != BITNET_A48_ERR_UNSUPPORTED) return s;
    }
    if (hd <= 64) return launch_attn_tile<64>(q, kc, vc, B, T, nh, hd, pos0, cap, att, st);
    if (hd <= 128) return launch_attn_tile<128>(q, kc, vc, B, T, nh, hd, pos0, cap, att, st);
    return launch_attn_tile<256>(q, kc, vc, B, T, nh, hd, pos0, cap, att, st);
}

}  // namespace

size_t a48_block_workspace_bytes(const bitnet_a48_block* blk, int B, int T) { return block_ws(blk, B, T).total; }

bitnet_a48_status a48_block_forward(const bitnet_a48_block* blk, const float* X, int B, int T, int pos0,
                                    float* kcache, float* vcache, float* Y, void* ws, size_t ws_bytes,
                                    cudaStream_t st) {
    const bitnet_a48_block_config& c = blk->cfg;
    const int H = c.hidden, F = c.ffn, nh = c.n_heads, hd = H / nh, M = B * T;
    if (hd % 4 != 0 || hd > 256 || H % 4 != 0 || F % 4 != 0) return BITNET_A48_ERR_SHAPE;
    if ((c.q_bits != 0 && c.q_bits != 4) || (c.kv_bits != 0 && c.kv_bits != 3 && c.kv_bits != 4)) return BITNET_A48_ERR_INVALID_ARG;
    if ((c.q_bits != 0 || c.kv_bits != 0) && hd > 128) return BITNET_A48_ERR_UNSUPPORTED;
    if (c.kv_bits != 0 && c.ctx_cap % 4 != 0) return BITNET_A48_ERR_SHAPE;  // packed rows are copied in 16-byte pieces
    if (B > 65535 || nh > 65535) return BITNET_A48_ERR_SHAPE;
    BlockWs o = block_ws(blk, B, T);
    char* base = static_cast<char*>(ws);
    int8_t* codes = reinterpret_cast<int8_t*>(base + o.codes);
    float* scale = reinterpret_cast<float*>(base + o.scale);
    float* q = reinterpret_cast<float*>(base + o.q);
    float* k = reinterpret_cast<float*>(base + o.k);
    float* v = reinterpret_cast<float*>(base + o.v);
    float* att = reinterpret_cast<float*>(base + o.att);
    float* hres = reinterpret_cast<float*>(base + o.hres);
    float* tmp = reinterpret_cast<float*>(base + o.tmp);
    float* gate = reinterpret_cast<float*>(base + o.gate);
    float* up = reinterpret_cast<float*>(base + o.up);
    float2* rope = reinterpret_cast<float2*>(base + o.rope);
    void* lin = base + o.lin;
    const size_t lin_bytes = ws_bytes - o.lin;
    int cap = c.ctx_cap;
    const bool caller_cache = kcache != nullptr;
    if (!kcache) {  // keys/values of this call only: keep them in the workspace
        kcache = reinterpret_cast<float*>(base + o.kc);
        vcache = reinterpret_cast<float*>(base + o.vc);
        cap = T;
    }
    bitnet_a48_status s;
#define A48_TRY(e) do { s = (e); if (s != BITNET_A48_OK) return s; } while (0)
    auto linear = [&](int wi, bitnet_a48_act kind, float* out) {
        return bitnet_a48_linear_ex(blk->w[wi], codes, scale, M, kind, BITNET_A48_ALGO_AUTO, out, nullptr, lin,
                                    lin_bytes, st);
    };
    // the decode kernel wants its scratch zero on entry and leaves it zero
    if (o.total > o.lin) A48_CUDA_TRY(cudaMemsetAsync(lin, 0, o.total - o.lin, st));
    // attention sub-layer (Eq. 6-7; FP4 variant: Eq. 8-9 in the same places)
    const bool fp4 = c.act_fp4 != 0;
    const bitnet_a48_act dense_kind = fp4 ? BITNET_A48_ACT_FP4 : BITNET_A48_ACT_INT4;
    if (fp4) A48_TRY(a48_launch_quant_fp4(X, M, H, codes, scale, blk->g_attn, c.norm_eps, st));
    else A48_TRY(a48_launch_quant_int4(X, M, H, c.quant_eps, codes, scale, blk->g_attn, c.norm_eps, st));
    {
        float* qkv[3] = {q, k, v};
        A48_TRY(bitnet_a48_linear_multi(3, blk->w, codes, scale, M, dense_kind, qkv, lin, lin_bytes, st));
    }
    const bool lowbit = c.q_bits != 0 || c.kv_bits != 0;
    if (lowbit) {
        // Section 3, low-bit attention: post-RoPE absmax quantisation of the heads; packed key/value cache
        if (c.kv_bits != 0 && !caller_cache) return BITNET_A48_ERR_UNSUPPORTED;
        const bool inline_angles = T <= 8;
        int n = T * (hd / 2);
        if (!inline_angles) rope_table_kernel<<<(n + 255) / 256, 256, 0, st>>>(pos0, T, hd / 2, (double)c.rope_base, rope);
        float* dq_k = reinterpret_cast<float*>(base + o.kc);
        float* dq_v = reinterpret_cast<float*>(base + o.vc);
        if (c.kv_bits == 0) return BITNET_A48_ERR_UNSUPPORTED;  // quantised queries go with a quantised cache
        const bool tile_path = T > 8;  // prefill: attention runs on dequantised fp32 copies
        A48_TRY(a48_launch_rope_quant_cache(q, k, v, inline_angles ? nullptr : rope, (double)c.rope_base, B, T, nh, hd, pos0,
                                            c.ctx_cap, c.q_bits, c.kv_bits, c.quant_eps, kcache, vcache,
                                            tile_path ? dq_k : nullptr, tile_path ? dq_v : nullptr, st));
        if (!tile_path) {
            A48_TRY(a48_launch_attn_row_lowbit(q, kcache, vcache, B, T, nh, hd, pos0, c.ctx_cap, c.kv_bits, att, st));
        } else {
            // a prefill behind cached positions: those come out of the packed cache into the fp32 copies first
            if (pos0 > 0)
                A48_TRY(a48_launch_dequant_prefix(kcache, vcache, B, nh, hd, pos0, c.ctx_cap, pos0 + T, c.kv_bits, dq_k, dq_v, st));
            A48_TRY(prefill_attention(q, dq_k, dq_v, B, T, nh, hd, pos0, pos0 + T, att, base + o.mma, st));
        }
    } else {
    {
        int n = T * (hd / 2);
        const bool inline_angles = T <= 8;  // decode: every thread evaluates its own angle, one launch fewer
        if (!inline_angles) rope_table_kernel<<<(n + 255) / 256, 256, 0, st>>>(pos0, T, hd / 2, (double)c.rope_base, rope);
        size_t total = (size_t)M * nh * (hd / 2);
        A48_CUDA_TRY(a48_launch_pdl(rope_cache_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, st, q, k, v,
                                    inline_angles ? nullptr : rope, (double)c.rope_base, B, T, nh, hd, pos0, cap, kcache,
                                    vcache));
    }
    if (T <= 8) {
        if (hd <= 64) A48_CUDA_TRY(launch_attn_row<2>(q, kcache, vcache, B, T, nh, hd, pos0, cap, att, st));
        else if (hd <= 128) A48_CUDA_TRY(launch_attn_row<4>(q, kcache, vcache, B, T, nh, hd, pos0, cap, att, st));
        else A48_CUDA_TRY(launch_attn_row<8>(q, kcache, vcache, B, T, nh, hd, pos0, cap, att, st));
    } else {
        A48_TRY(prefill_attention(q, kcache, vcache, B, T, nh, hd, pos0, cap, att, base + o.mma, st));
    }
    }
    if (fp4) {  // the floating-point variant quantises the attention output densely (no top-K)
        A48_TRY(a48_launch_quant_fp4(att, M, H, codes, scale, nullptr, 0.f, st));
        A48_TRY(linear(3, BITNET_A48_ACT_FP4, tmp));
    } else {
        A48_TRY(a48_launch_topk_quant_int8(att, M, H, c.k_o, c.quant_eps, codes, scale, nullptr, st));
        A48_TRY(linear(3, BITNET_A48_ACT_TOPK_INT8, tmp));
    }
    const size_t nH4 = (size_t)M * H / 4, nF4 = (size_t)M * F / 4;
    // feed-forward sub-layer: h = x + attention output, formed (and written for the last residual) in the quantiser's load
    if (a48_topk_quant_fast_shape(H)) {
        if (fp4) A48_TRY(a48_launch_quant_fp4_add(X, tmp, hres, M, H, codes, scale, blk->g_ffn, c.norm_eps, st));
        else A48_TRY(a48_launch_quant_int4_add(X, tmp, hres, M, H, c.quant_eps, codes, scale, blk->g_ffn, c.norm_eps, st));
    } else {
        A48_CUDA_TRY(a48_launch_pdl(add_kernel, dim3((unsigned)((nH4 + 255) / 256)), dim3(256), 0, st, X, tmp, hres, nH4));
        if (fp4) A48_TRY(a48_launch_quant_fp4(hres, M, H, codes, scale, blk->g_ffn, c.norm_eps, st));
        else A48_TRY(a48_launch_quant_int4(hres, M, H, c.quant_eps, codes, scale, blk->g_ffn, c.norm_eps, st));
    }
    {
        float* gu[2] = {gate, up};
        A48_TRY(bitnet_a48_linear_multi(2, blk->w + 4, codes, scale, M, dense_kind, gu, lin, lin_bytes, st));
    }
    if (a48_topk_quant_fast_shape(F)) {
        // Eq. 5 inside the quantiser's load: the product up * ReLU(gate)^2 is never written
        A48_TRY(a48_launch_topk_quant_int8_glu(gate, up, M, F, c.k_down, c.quant_eps, codes, scale, st));
    } else {
        relu2glu_kernel<<<(unsigned)((nF4 + 255) / 256), 256, 0, st>>>(gate, up, nF4);
        A48_TRY(a48_launch_topk_quant_int8(gate, M, F, c.k_down, c.quant_eps, codes, scale, nullptr, st));
    }
    if (a48_decode_supported(blk->w[6], M)) {
        // a few tokens: the last residual add rides in the decode kernel's epilogue (one launch fewer)
        a48_decode_residual = hres;
        s = linear(6, BITNET_A48_ACT_TOPK_INT8, Y);
        a48_decode_residual = nullptr;
        if (s != BITNET_A48_OK) return s;
    } else {
        A48_TRY(linear(6, BITNET_A48_ACT_TOPK_INT8, tmp));
        A48_CUDA_TRY(a48_launch_pdl(add_kernel, dim3((unsigned)((nH4 + 255) / 256)), dim3(256), 0, st, hres, tmp, Y, nH4));
    }
#undef A48_TRY
    A48_CUDA_TRY(cudaGetLastError());
    return BITNET_A48_OK;
}
