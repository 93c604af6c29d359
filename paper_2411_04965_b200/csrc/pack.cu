// Weight quantiser (Eq. 2) and the packed layouts of the ternary codes.
#include "internal.h"
#include "layouts.cuh"

namespace {

constexpr int kSumThreads = 256;
constexpr int kSumBlocksMax = 1024;

__device__ __forceinline__ double block_sum(double v, double* smem) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) smem[warp] = v;
    __syncthreads();
    double r = 0.0;
    if (warp == 0) {
        r = lane < (blockDim.x >> 5) ? smem[lane] : 0.0;
        for (int o = 16; o > 0; o >>= 1) r += __shfl_xor_sync(0xffffffffu, r, o);
    }
    return r;  // valid in warp 0
}

// Pass 1 of alpha = mean|W| (Eq. 2): per-block partial sums in float64, fixed order.
__global__ void abs_sum_partial_kernel(const float* __restrict__ W, size_t n, double* __restrict__ partial) {
    __shared__ double smem[kSumThreads / 32];
    double s = 0.0;
    size_t n4 = n / 4;
    const float4* W4 = reinterpret_cast<const float4*>(W);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        float4 v = W4[i];
        s += (double)fabsf(v.x) + (double)fabsf(v.y) + (double)fabsf(v.z) + (double)fabsf(v.w);
    }
    if (blockIdx.x == 0 && threadIdx.x < (n & 3)) s += (double)fabsf(W[n4 * 4 + threadIdx.x]);
    double r = block_sum(s, smem);
    if (threadIdx.x == 0) partial[blockIdx.x] = r;
}

__global__ void abs_sum_final_kernel(const double* __restrict__ partial, int nblocks, size_t n,
                                     double* __restrict__ alpha64, float* __restrict__ alpha32) {
    __shared__ double smem[kSumThreads / 32];
    double s = 0.0;
    for (int i = threadIdx.x; i < nblocks; i += blockDim.x) s += partial[i];
    double r = block_sum(s, smem);
    if (threadIdx.x == 0) {
        double a = r / (double)n;
        *alpha64 = a;
        *alpha32 = (float)a;
    }
}

// Pass 2 of Eq. 2: t = RoundClip(W/(alpha+eps), -1, 1) in float64, four codes per byte.
__global__ void ternarise_pack_kernel(const float* __restrict__ W, int N, int K, int K4, double eps,
                                      const double* __restrict__ alpha64, uint8_t* __restrict__ l0) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)N * K4) return;
    int n = (int)(idx / K4), j = (int)(idx % K4);
    double den = *alpha64 + eps;
    unsigned byte = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int k = 4 * j + i;
        int t = 0;
        if (k < K) {
            double r = rint((double)W[(size_t)n * K + k] / den);
            t = r < -1.0 ? -1 : (r > 1.0 ? 1 : (int)r);
        }
        byte |= (unsigned)(t + 1) << (2 * i);
    }
    l0[idx] = (uint8_t)byte;
}

__global__ void unpack_l0_kernel(const uint8_t* __restrict__ l0, int N, int K, int K4, int8_t* __restrict__ codes) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)N * K) return;
    int n = (int)(idx / K), k = (int)(idx % K);
    codes[idx] = (int8_t)a48_l0_code(l0, K4, n, k);
}

// Builds one of the tiled layouts from the canonical one: one thread per 32-bit
// word of the destination, each field looked up through the layout's index map.
template <class Layout>
__global__ void relayout_kernel(const uint8_t* __restrict__ l0, int N, int K, int K4, Layout lay,
                                uint32_t* __restrict__ dst, size_t nwords) {
    size_t widx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (widx >= nwords) return;
    uint32_t word = 0;
#pragma unroll
    for (int f = 0; f < 16; ++f) {
        int n, k;
        lay.field_to_nk(widx, f, n, k);
        int t = (n < N && k < K) ? a48_l0_code(l0, K4, n, k) : 0;
        word |= (uint32_t)(t + 1) << (2 * f);
    }
    dst[widx] = word;
}

template <class Layout>
__global__ void unpack_layout_kernel(const uint32_t* __restrict__ src, int N, int K, Layout lay,
                                     int8_t* __restrict__ codes, size_t nwords) {
    size_t widx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (widx >= nwords) return;
    uint32_t word = src[widx];
#pragma unroll
    for (int f = 0; f < 16; ++f) {
        int n, k;
        lay.field_to_nk(widx, f, n, k);
        if (n < N && k < K) codes[(size_t)n * K + k] = (int8_t)((int)((word >> (2 * f)) & 3u) - 1);
    }
}

// int8 codes [Np][Kp], zero outside [N][K]
__global__ void expand_i8_kernel(const uint8_t* __restrict__ l0, int N, int K, int K4, int Np, int Kp,
                                 int8_t* __restrict__ dst) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)Np * Kp) return;
    int n = (int)(idx / Kp), k = (int)(idx % Kp);
    dst[idx] = (n < N && k < K) ? (int8_t)a48_l0_code(l0, K4, n, k) : (int8_t)0;
}

// Five codes per byte: b = sum_i (t_i + 1) * 3^i over channels 5j .. 5j+4 of a row (code 0 past K and in the row padding).
__global__ void pack_trit5_kernel(const uint8_t* __restrict__ l0, int N, int K, int K4, int row_bytes, uint8_t* __restrict__ dst) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)N * row_bytes) return;
    const int n = (int)(idx / row_bytes), j = (int)(idx % row_bytes);
    unsigned b = 0, pw = 1;
#pragma unroll
    for (int i = 0; i < 5; ++i) {
        const int k = 5 * j + i;
        b += (unsigned)((k < K ? a48_l0_code(l0, K4, n, k) : 0) + 1) * pw;
        pw *= 3;
    }
    dst[idx] = (uint8_t)b;
}

__global__ void unpack_trit5_kernel(const uint8_t* __restrict__ src, int N, int K, int row_bytes, int8_t* __restrict__ codes) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)N * K) return;
    const int n = (int)(idx / K), k = (int)(idx % K);
    unsigned b = src[(size_t)n * row_bytes + k / 5];
    for (int i = 0; i < k % 5; ++i) b /= 3;
    codes[idx] = (int8_t)((int)(b % 3) - 1);
}

template <class Layout>
void run_relayout(const bitnet_a48_weight* w, Layout lay, uint8_t* dst, size_t bytes, cudaStream_t st) {
    size_t nwords = bytes / 4;
    relayout_kernel<Layout><<<(unsigned)((nwords + 255) / 256), 256, 0, st>>>(
        w->l0, w->N, w->K, w->K4, lay, reinterpret_cast<uint32_t*>(dst), nwords);
}

template <class Layout>
void run_unpack_layout(const bitnet_a48_weight* w, Layout lay, const uint8_t* src, size_t bytes, int8_t* codes,
                       cudaStream_t st) {
    size_t nwords = bytes / 4;
    unpack_layout_kernel<Layout><<<(unsigned)((nwords + 255) / 256), 256, 0, st>>>(
        reinterpret_cast<const uint32_t*>(src), w->N, w->K, lay, codes, nwords);
}

}  // namespace

bitnet_a48_status a48_launch_pack(bitnet_a48_weight* w, const float* W_dev, float eps, cudaStream_t st) {
    size_t n = (size_t)w->N * w->K;
    int nblocks = (int)((n / 4 + kSumThreads - 1) / kSumThreads);
    nblocks = nblocks < 1 ? 1 : (nblocks > kSumBlocksMax ? kSumBlocksMax : nblocks);
    abs_sum_partial_kernel<<<nblocks, kSumThreads, 0, st>>>(W_dev, n, w->partial_dev);
    abs_sum_final_kernel<<<1, kSumThreads, 0, st>>>(w->partial_dev, nblocks, n, w->alpha64_dev, w->alpha_dev);
    size_t nbytes = (size_t)w->N * w->K4;
    ternarise_pack_kernel<<<(unsigned)((nbytes + 255) / 256), 256, 0, st>>>(W_dev, w->N, w->K, w->K4, (double)eps,
                                                                         w->alpha64_dev, w->l0);
    if (w->gemm) run_relayout(w, GemmLayout{w->Kp}, w->gemm, (size_t)w->Np * w->Kp / 4, st);
    if (w->decode) run_relayout(w, DecodeLayout{w->Kp}, w->decode, w->decode_bytes, st);
    if (w->sparse) run_relayout(w, SparseLayout{w->Np}, w->sparse, w->sparse_bytes, st);
    if (w->trit5) {
        size_t nb = (size_t)w->N * w->trit5_row;
        pack_trit5_kernel<<<(unsigned)((nb + 255) / 256), 256, 0, st>>>(w->l0, w->N, w->K, w->K4, w->trit5_row, w->trit5);
    }
    if (w->i8) {
        size_t n8 = (size_t)w->Np * w->Kp;
        expand_i8_kernel<<<(unsigned)((n8 + 255) / 256), 256, 0, st>>>(w->l0, w->N, w->K, w->K4, w->Np, w->Kp, w->i8);
    }
    A48_CUDA_TRY(cudaGetLastError());
    return BITNET_A48_OK;
}

bitnet_a48_status a48_launch_unpack_l0(const bitnet_a48_weight* w, int8_t* codes_dev, cudaStream_t st) {
    size_t n = (size_t)w->N * w->K;
    unpack_l0_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(w->l0, w->N, w->K, w->K4, codes_dev);
    A48_CUDA_TRY(cudaGetLastError());
    return BITNET_A48_OK;
}

bitnet_a48_status a48_launch_unpack_layout(const bitnet_a48_weight* w, unsigned layout, int8_t* codes_dev,
                                           cudaStream_t st) {
    if (layout == BITNET_A48_LAYOUT_GEMM && w->gemm)
        run_unpack_layout(w, GemmLayout{w->Kp}, w->gemm, (size_t)w->Np * w->Kp / 4, codes_dev, st);
    else if (layout == BITNET_A48_LAYOUT_DECODE && w->decode)
        run_unpack_layout(w, DecodeLayout{w->Kp}, w->decode, w->decode_bytes, codes_dev, st);
    else if (layout == BITNET_A48_LAYOUT_SPARSE && w->sparse)
        run_unpack_layout(w, SparseLayout{w->Np}, w->sparse, w->sparse_bytes, codes_dev, st);
    else if (layout == BITNET_A48_LAYOUT_TRIT5 && w->trit5) {
        size_t n = (size_t)w->N * w->K;
        unpack_trit5_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(w->trit5, w->N, w->K, w->trit5_row, codes_dev);
    } else
        return BITNET_A48_ERR_UNSUPPORTED;
    A48_CUDA_TRY(cudaGetLastError());
    return BITNET_A48_OK;
}
