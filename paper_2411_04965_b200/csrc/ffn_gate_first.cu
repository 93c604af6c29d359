// Gate-first evaluation of the feed-forward sub-layer for a few tokens (Section 2.1, paragraph after Eq. 5;
// Section 3, "Sparsity"): the gate projection runs first, and the up projection is evaluated only for the output
// channels n whose ReLU²(gate[n]) is non-zero for at least one of the tokens - the other rows of W_up are never
// fetched.  Eq. 5's product goes straight into the top-K + INT8 quantiser and the down projection.
//
// The up rows come from the canonical packed layout (row-major, K/4 bytes per row, byte j = channels 4j..4j+3,
// field f at bits 2f), where one row is one contiguous run (1 KB at K = 4096).  A warp owns a row at a time: a
// ballot over the tokens' gates decides whether the row is needed; if so every lane loads 16-byte pieces of it and
// contracts them with dp4a.  Masking a packed word with 0x03030303 << 2f leaves, in byte b, the field of channel
// 16w + 4b + f scaled by 4^f, so the token codes are staged once per CTA in that order (a 4x4 byte transpose of
// every 16 codes) and the factor 4^f is shifted out of the four partial sums at the end.  The +1 of the encoding
// e = t + 1 is removed with sum_k x[m,k].
#include "internal.h"

namespace {

constexpr int kThreads = 256, kWarps = kThreads / 32;

// sum of four u8 x s8 products plus c
__device__ __forceinline__ int dp4a_u8s8(uint32_t a, int b, int c) {
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// inter[m, n] = up[m, n] * ReLU(gate[m, n])^2 for the rows that are needed, 0 for the others.
// Dynamic shared memory: xt [MT][K] bytes (transposed codes) | xsum [MT] int.
template <int MT>
__global__ void __launch_bounds__(kThreads) up_rows_kernel(const uint8_t* __restrict__ l0, int K4, const int8_t* __restrict__ codes,
                                                           const float* __restrict__ scale, const float* __restrict__ alpha,
                                                           const float* __restrict__ gate, int M, int F, int K,
                                                           float* __restrict__ inter, int32_t* __restrict__ rows_fetched) {
    extern __shared__ __align__(16) uint8_t smem[];
    uint32_t* xt = reinterpret_cast<uint32_t*>(smem);  // [MT][K/16][4]
    int* xsum = reinterpret_cast<int*>(smem + (size_t)MT * K);
    const int groups = K / 16, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x < MT) xsum[threadIdx.x] = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < MT * groups; i += kThreads) {
        const int m = i / groups, g = i % groups;
        uint4 c = make_uint4(0, 0, 0, 0);
        if (m < M) c = *reinterpret_cast<const uint4*>(codes + (size_t)m * K + 16 * g);
        // byte f of word b is code 16g + 4b + f; xt word f holds the codes 16g + 4b + f for b = 0..3
        uint4 t;
        const uint32_t lo01 = __byte_perm(c.x, c.y, 0x5140), hi01 = __byte_perm(c.x, c.y, 0x7362);
        const uint32_t lo23 = __byte_perm(c.z, c.w, 0x5140), hi23 = __byte_perm(c.z, c.w, 0x7362);
        t.x = __byte_perm(lo01, lo23, 0x5410);
        t.y = __byte_perm(lo01, lo23, 0x7632);
        t.z = __byte_perm(hi01, hi23, 0x5410);
        t.w = __byte_perm(hi01, hi23, 0x7632);
        *reinterpret_cast<uint4*>(xt + (size_t)i * 4) = t;
        int s = __dp4a((int)c.x, 0x01010101, __dp4a((int)c.y, 0x01010101, __dp4a((int)c.z, 0x01010101, __dp4a((int)c.w, 0x01010101, 0))));
        if (s) atomicAdd(&xsum[m], s);
    }
    __syncthreads();
    const float al = __ldg(alpha);
    const int pieces = K4 / 16;  // 16-byte pieces per row; piece p holds the 16-code groups 4p..4p+3
    int fetched = 0;
    for (int n = blockIdx.x * kWarps + warp; n < F; n += gridDim.x * kWarps) {
        const float g_lane = lane < M ? __ldg(gate + (size_t)lane * F + n) : 0.f;
        const unsigned need = __ballot_sync(0xffffffffu, g_lane > 0.f);
        if (need == 0u) {  // ReLU²(gate) is zero for every token: the row of W_up is not fetched
            if (lane < M) inter[(size_t)lane * F + n] = 0.f;
            continue;
        }
        ++fetched;
        int acc[MT][4];
#pragma unroll
        for (int m = 0; m < MT; ++m) acc[m][0] = acc[m][1] = acc[m][2] = acc[m][3] = 0;
        const uint4* row = reinterpret_cast<const uint4*>(l0 + (size_t)n * K4);
        for (int p = lane; p < pieces; p += 32) {
            const uint4 w4 = __ldg(row + p);
            const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    const uint4 x = *reinterpret_cast<const uint4*>(xt + ((size_t)m * groups + 4 * p + j) * 4);
                    acc[m][0] = dp4a_u8s8(w[j] & 0x03030303u, (int)x.x, acc[m][0]);
                    acc[m][1] = dp4a_u8s8(w[j] & 0x0c0c0c0cu, (int)x.y, acc[m][1]);
                    acc[m][2] = dp4a_u8s8(w[j] & 0x30303030u, (int)x.z, acc[m][2]);
                    acc[m][3] = dp4a_u8s8(w[j] & 0xc0c0c0c0u, (int)x.w, acc[m][3]);
                }
            }
        }
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            // (the masked bytes are unsigned fields times 4^f; the shifts take the factor out exactly)
            int v = acc[m][0] + (acc[m][1] >> 2) + (acc[m][2] >> 4) + (acc[m][3] >> 6);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (lane == m && m < M) {
                const float up = (float)(v - xsum[m]) * (__ldg(scale + m) * al);  // prefactors of Eq. 2 and 7
                const float r = g_lane > 0.f ? g_lane : 0.f;
                inter[(size_t)m * F + n] = up * (r * r);  // Eq. 5
            }
        }
    }
    if (rows_fetched) {
        if (lane == 0 && fetched) atomicAdd(rows_fetched, fetched);  // (the count is the same in every lane)
    }
}

size_t up256(size_t v) { return (v + 255) / 256 * 256; }

struct FfnWs {
    size_t codes4, scale4, gate, inter, codes8, scale8, lin, total;
};

FfnWs ffn_ws(const bitnet_a48_weight* gate, const bitnet_a48_weight* down, int M) {
    const size_t H = gate->K, F = gate->N;
    FfnWs w;
    size_t o = 0;
    auto take = [&](size_t b) { size_t r = o; o += up256(b); return r; };
    w.codes4 = take((size_t)M * H);
    w.scale4 = take((size_t)M * 4);
    w.gate = take((size_t)M * F * 4);
    w.inter = take((size_t)M * F * 4);
    w.codes8 = take((size_t)M * F);
    w.scale8 = take((size_t)M * 4);
    size_t a = bitnet_a48_linear_workspace_bytes(gate, M), b = bitnet_a48_linear_workspace_bytes(down, M);
    w.lin = take(a > b ? a : b);
    w.total = o;
    return w;
}

}  // namespace

extern "C" size_t bitnet_a48_ffn_gate_first_workspace_bytes(const bitnet_a48_weight* gate, const bitnet_a48_weight* up,
                                                            const bitnet_a48_weight* down, int M) {
    if (!gate || !up || !down || M <= 0) return 0;
    const FfnWs o = ffn_ws(gate, down, M);
    const bitnet_a48_weight* gu[2] = {gate, up};
    const size_t multi = bitnet_a48_linear_multi_workspace_bytes(2, gu, M);  // the dense form's fused gate+up launch
    return o.lin + (multi > o.total - o.lin ? multi : o.total - o.lin);
}

// The same sub-layer evaluated densely (gate and up as one fused launch over every row, Eq. 5 inside the top-K
// quantiser's load): the reference point for what gate-first saves.
extern "C" bitnet_a48_status bitnet_a48_ffn_dense(const bitnet_a48_weight* gate, const bitnet_a48_weight* up,
                                                  const bitnet_a48_weight* down, const float* X_dev, int M, int k_down,
                                                  float eps, float* Y_dev, void* workspace_dev, size_t workspace_bytes,
                                                  void* stream) {
    if (!gate || !up || !down || !X_dev || !Y_dev || !workspace_dev) return BITNET_A48_ERR_INVALID_ARG;
    const int H = gate->K, F = gate->N;
    if (up->N != F || up->K != H || down->N != H || down->K != F) return BITNET_A48_ERR_SHAPE;
    if (M <= 0 || M > 8 || !a48_topk_quant_fast_shape(F)) return BITNET_A48_ERR_UNSUPPORTED;
    if (k_down < 1 || k_down > F || !(eps >= 0.f)) return BITNET_A48_ERR_INVALID_ARG;
    if (!a48_aligned16(X_dev) || !a48_aligned16(Y_dev) || !a48_aligned16(workspace_dev)) return BITNET_A48_ERR_ALIGNMENT;
    const FfnWs o = ffn_ws(gate, down, M);
    // the fused gate+up launch may want more scratch than either matrix alone
    const bitnet_a48_weight* gu[2] = {gate, up};
    const size_t multi = bitnet_a48_linear_multi_workspace_bytes(2, gu, M);
    if (workspace_bytes < o.lin + (multi > o.total - o.lin ? multi : o.total - o.lin)) return BITNET_A48_ERR_NOMEM;
    cudaStream_t st = (cudaStream_t)stream;
    char* base = static_cast<char*>(workspace_dev);
    int8_t* codes4 = reinterpret_cast<int8_t*>(base + o.codes4);
    float* scale4 = reinterpret_cast<float*>(base + o.scale4);
    float* gate_y = reinterpret_cast<float*>(base + o.gate);
    float* up_y = reinterpret_cast<float*>(base + o.inter);
    int8_t* codes8 = reinterpret_cast<int8_t*>(base + o.codes8);
    float* scale8 = reinterpret_cast<float*>(base + o.scale8);
    void* lin = base + o.lin;
    const size_t lin_bytes = workspace_bytes - o.lin;
    A48_CUDA_TRY(cudaMemsetAsync(lin, 0, lin_bytes, st));
    bitnet_a48_status s = bitnet_a48_quant_int4(X_dev, M, H, eps, codes4, scale4, stream);
    if (s != BITNET_A48_OK) return s;
    float* ys[2] = {gate_y, up_y};
    s = bitnet_a48_linear_multi(2, gu, codes4, scale4, M, BITNET_A48_ACT_INT4, ys, lin, lin_bytes, stream);
    if (s != BITNET_A48_OK) return s;
    s = a48_launch_topk_quant_int8_glu(gate_y, up_y, M, F, k_down, eps, codes8, scale8, st);
    if (s != BITNET_A48_OK) return s;
    return bitnet_a48_linear(down, codes8, scale8, M, BITNET_A48_ACT_TOPK_INT8, Y_dev, nullptr, lin, lin_bytes, stream);
}

extern "C" bitnet_a48_status bitnet_a48_ffn_gate_first(const bitnet_a48_weight* gate, const bitnet_a48_weight* up,
                                                       const bitnet_a48_weight* down, const float* X_dev, int M, int k_down,
                                                       float eps, float* Y_dev, float* inter_dev, int32_t* rows_fetched_dev,
                                                       void* workspace_dev, size_t workspace_bytes, void* stream) {
    if (!gate || !up || !down || !X_dev || !Y_dev || !workspace_dev) return BITNET_A48_ERR_INVALID_ARG;
    const int H = gate->K, F = gate->N;
    if (up->N != F || up->K != H || down->N != H || down->K != F) return BITNET_A48_ERR_SHAPE;
    if (M <= 0 || M > 8) return BITNET_A48_ERR_UNSUPPORTED;
    if (k_down < 1 || k_down > F || !(eps >= 0.f)) return BITNET_A48_ERR_INVALID_ARG;
    // a row of the canonical layout must be a whole number of 16-byte pieces, and the codes of a token must fit
    // the CTA's shared memory next to nothing else
    if (H % 64 != 0 || (size_t)8 * H + 64 > 200 * 1024) return BITNET_A48_ERR_UNSUPPORTED;
    if (!a48_aligned16(X_dev) || !a48_aligned16(Y_dev) || !a48_aligned16(inter_dev) || !a48_aligned16(rows_fetched_dev) ||
        !a48_aligned16(workspace_dev))
        return BITNET_A48_ERR_ALIGNMENT;
    const FfnWs o = ffn_ws(gate, down, M);
    if (workspace_bytes < o.total) return BITNET_A48_ERR_NOMEM;
    cudaStream_t st = (cudaStream_t)stream;
    char* base = static_cast<char*>(workspace_dev);
    int8_t* codes4 = reinterpret_cast<int8_t*>(base + o.codes4);
    float* scale4 = reinterpret_cast<float*>(base + o.scale4);
    float* gate_y = reinterpret_cast<float*>(base + o.gate);
    float* inter = inter_dev ? inter_dev : reinterpret_cast<float*>(base + o.inter);
    int8_t* codes8 = reinterpret_cast<int8_t*>(base + o.codes8);
    float* scale8 = reinterpret_cast<float*>(base + o.scale8);
    void* lin = base + o.lin;
    const size_t lin_bytes = o.total - o.lin;
    if (lin_bytes) A48_CUDA_TRY(cudaMemsetAsync(lin, 0, lin_bytes, st));  // the decode kernel's scratch starts at zero
    if (rows_fetched_dev) A48_CUDA_TRY(cudaMemsetAsync(rows_fetched_dev, 0, sizeof(int32_t), st));
    bitnet_a48_status s = bitnet_a48_quant_int4(X_dev, M, H, eps, codes4, scale4, stream);  // Eq. 7
    if (s != BITNET_A48_OK) return s;
    s = bitnet_a48_linear(gate, codes4, scale4, M, BITNET_A48_ACT_INT4, gate_y, nullptr, lin, lin_bytes, stream);  // Eq. 6
    if (s != BITNET_A48_OK) return s;
    {
        const int mt = M == 1 ? 1 : (M == 2 ? 2 : (M <= 4 ? 4 : 8));
        const size_t smem = (size_t)mt * H + 64;
        int dev = 0, sms = 0;
        A48_CUDA_TRY(cudaGetDevice(&dev));
        A48_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        const int grid = sms * 2;
#define A48_UP(MT)                                                                                                       \
    do {                                                                                                                  \
        if (smem > 48 * 1024)                                                                                             \
            A48_CUDA_TRY(cudaFuncSetAttribute(up_rows_kernel<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
        up_rows_kernel<MT><<<grid, kThreads, smem, st>>>(up->l0, up->K4, codes4, scale4, up->alpha_dev, gate_y, M, F, H, inter, \
                                                         rows_fetched_dev);                                               \
    } while (0)
        if (mt == 1) A48_UP(1);
        else if (mt == 2) A48_UP(2);
        else if (mt == 4) A48_UP(4);
        else A48_UP(8);
#undef A48_UP
        A48_CUDA_TRY(cudaGetLastError());
    }
    s = bitnet_a48_topk_quant_int8(inter, M, F, k_down, eps, codes8, scale8, nullptr, stream);  // Eq. 1 and 3
    if (s != BITNET_A48_OK) return s;
    return bitnet_a48_linear(down, codes8, scale8, M, BITNET_A48_ACT_TOPK_INT8, Y_dev, nullptr, lin, lin_bytes, stream);
}
