// Plain tiled BitLinear contraction (Eq. 1 / Eq. 6) on dp4a: any M, N, K.
// It is the in-tree cross-check for the tensor-core and decode kernels and the
// path for shapes those kernels do not take.  acc is exact int32; the rescale
// y = fp32(acc)·(scale[m]·alpha) applies the prefactors of Eq. 2, 3 and 7.
#include "internal.h"

namespace {

constexpr int BM = 32, BN = 64, BK = 64;  // tile: 32 tokens x 64 outputs, 64 channels per step

// byte of four 2-bit fields (e = t+1) -> four int8 codes in one word
__device__ __forceinline__ uint32_t expand_byte(unsigned b) {
    uint32_t x = (b & 3u) | ((b & 12u) << 6) | ((b & 48u) << 12) | ((b & 192u) << 18);
    return (x + 0x7f7f7f7fu) ^ 0x80808080u;  // per byte: e - 1
}

__global__ void __launch_bounds__(256) linear_simple_kernel(const uint8_t* __restrict__ l0, int K4,
                                                            const int8_t* __restrict__ codes,
                                                            const float* __restrict__ scale,
                                                            const float* __restrict__ alpha, int M, int N, int K,
                                                            float* __restrict__ Y, int32_t* __restrict__ acc_out, int y_bf16) {
    __shared__ uint32_t sa[BM][BK / 4 + 1];
    __shared__ uint32_t sw[BN][BK / 4 + 1];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;  // tx: outputs tx, tx+32; ty: tokens 4ty..4ty+3
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    int acc[4][2] = {};
    for (int k0 = 0; k0 < K; k0 += BK) {
        // activations: 32 rows x 16 words
        for (int i = threadIdx.x; i < BM * (BK / 4); i += 256) {
            int r = i / (BK / 4), c = i % (BK / 4);
            int m = m0 + r, k = k0 + 4 * c;
            uint32_t word = 0;
            if (m < M) {
#pragma unroll
                for (int b = 0; b < 4; ++b)
                    if (k + b < K) word |= (uint32_t)(uint8_t)codes[(size_t)m * K + k + b] << (8 * b);
            }
            sa[r][c] = word;
        }
        // weights: 64 rows x 16 packed bytes -> 16 words of int8 each
        for (int i = threadIdx.x; i < BN * (BK / 4); i += 256) {
            int r = i / (BK / 4), c = i % (BK / 4);
            int n = n0 + r, j = (k0 >> 2) + c;
            sw[r][c] = (n < N && j < K4) ? expand_byte(l0[(size_t)n * K4 + j]) : 0u;
        }
        __syncthreads();
#pragma unroll
        for (int c = 0; c < BK / 4; ++c) {
            int w0 = (int)sw[tx][c], w1 = (int)sw[tx + 32][c];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                int a = (int)sa[4 * ty + i][c];
                acc[i][0] = __dp4a(a, w0, acc[i][0]);
                acc[i][1] = __dp4a(a, w1, acc[i][1]);
            }
        }
        __syncthreads();
    }
    const float al = *alpha;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int m = m0 + 4 * ty + i;
        if (m >= M) continue;
        float s = scale[m] * al;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            int n = n0 + tx + 32 * j;
            if (n >= N) continue;
            a48_store_y(Y, (size_t)m * N + n, (float)acc[i][j] * s, y_bf16);
            if (acc_out) acc_out[(size_t)m * N + n] = acc[i][j];
        }
    }
}

}  // namespace

bitnet_a48_status a48_launch_linear_simple(const bitnet_a48_weight* w, const int8_t* codes, const float* scale,
                                           int M, float* Y, int32_t* acc, cudaStream_t st) {
    dim3 grid((w->N + BN - 1) / BN, (M + BM - 1) / BM);
    if (grid.y > 65535) return BITNET_A48_ERR_SHAPE;
    linear_simple_kernel<<<grid, 256, 0, st>>>(w->l0, w->K4, codes, scale, w->alpha_dev, M, w->N, w->K, Y, acc, a48_y_bf16);
    A48_CUDA_TRY(cudaGetLastError());
    return BITNET_A48_OK;
}
