// Decode BitLinear (Eq. 1 / Eq. 6, up to 8 tokens) over the densest byte packing of ternary weights: five codes per
// byte, b = sum_i (t_i + 1) * 3^i <= 242, i.e. 1.6 bits per weight where the paper counts log2(3) = 1.58 (Section 1)
// and the other layouts of this library spend 2.  A row of W is ceil(K/5) bytes, padded to a multiple of 16.
//
// Base-3 digits do not come apart with shifts and masks, so a byte is decoded through a 243-entry table in shared
// memory (two words per entry: the int8 codes t_0..t_3, and t_4), and the token codes are staged once per CTA in
// the matching groups of five (two words per group: x_0..x_3, and x_4).  Each table lookup then feeds two dp4a.
// One warp owns a row at a time and streams it with 16-byte loads.  This trades arithmetic for bytes: a fifth
// fewer bytes from HBM, about twice the instructions per weight of the 2-bit kernels.
#include "internal.h"

namespace {

constexpr int kThreads = 256, kWarps = kThreads / 32;

// Dynamic shared memory: xg [MT][groups] uint2 | lut [243] uint2.
template <int MT>
__global__ void __launch_bounds__(kThreads) decode_trit5_kernel(const uint8_t* __restrict__ wt, int row_bytes, const int8_t* __restrict__ codes,
                                                                const float* __restrict__ scale, const float* __restrict__ alpha,
                                                                int M, int N, int K, float* __restrict__ Y, int32_t* __restrict__ acc_out) {
    extern __shared__ __align__(16) uint8_t smem[];
    a48_pdl_prologue();
    const int groups = row_bytes;  // one group of five channels per weight byte (zero codes past K)
    uint2* xg = reinterpret_cast<uint2*>(smem);
    uint2* lut = xg + (size_t)MT * groups;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int b = threadIdx.x; b < 243; b += kThreads) {
        int d[5], v = b;
#pragma unroll
        for (int i = 0; i < 5; ++i) {
            d[i] = v % 3 - 1;
            v /= 3;
        }
        lut[b] = make_uint2((uint32_t)(d[0] & 0xff) | ((uint32_t)(d[1] & 0xff) << 8) | ((uint32_t)(d[2] & 0xff) << 16) |
                                ((uint32_t)(d[3] & 0xff) << 24),
                            (uint32_t)(d[4] & 0xff));
    }
    for (int i = threadIdx.x; i < MT * groups; i += kThreads) {
        const int m = i / groups, g = i % groups;
        uint32_t lo = 0, hi = 0;
        if (m < M) {
#pragma unroll
            for (int j = 0; j < 5; ++j) {
                const int k = 5 * g + j;
                const uint32_t c = k < K ? (uint32_t)(uint8_t)codes[(size_t)m * K + k] : 0u;
                if (j < 4) lo |= c << (8 * j);
                else hi = c;
            }
        }
        // group g = 16 p + s is the s-th byte of the 16-byte piece p that lane p % 32 loads: stored [m][s][p], so that
        // the 32 lanes of a warp, which hold consecutive pieces, read consecutive words
        xg[((size_t)m * 16 + (g & 15)) * (groups / 16) + (g >> 4)] = make_uint2(lo, hi);
    }
    __syncthreads();
    const float al = __ldg(alpha);
    const int pieces = row_bytes / 16;
    for (int n = blockIdx.x * kWarps + warp; n < N; n += gridDim.x * kWarps) {
        int acc[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) acc[m] = 0;
        const uint4* row = reinterpret_cast<const uint4*>(wt + (size_t)n * row_bytes);
        for (int p = lane; p < pieces; p += 32) {
            const uint4 w4 = __ldg(row + p);
            const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const uint2 t = lut[(w[j] >> (8 * b)) & 0xffu];
#pragma unroll
                    for (int m = 0; m < MT; ++m) {
                        const uint2 x = xg[((size_t)m * 16 + 4 * j + b) * pieces + p];
                        acc[m] = __dp4a((int)t.y, (int)x.y, __dp4a((int)t.x, (int)x.x, acc[m]));
                    }
                }
            }
        }
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            int v = acc[m];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (lane == m && m < M) {
                Y[(size_t)m * N + n] = (float)v * (__ldg(scale + m) * al);  // prefactors of Eq. 2, 3 and 7
                if (acc_out) acc_out[(size_t)m * N + n] = v;
            }
        }
    }
}

}  // namespace

bool a48_decode_trit5_supported(const bitnet_a48_weight* w, int M) {
    return w->trit5 != nullptr && M >= 1 && M <= 8 && (size_t)8 * w->trit5_row * 8 + 243 * 8 <= 200 * 1024;
}

bitnet_a48_status a48_launch_decode_trit5(const bitnet_a48_weight* w, const int8_t* codes, const float* scale, int M, float* Y,
                                          int32_t* acc, cudaStream_t st) {
    if (!a48_decode_trit5_supported(w, M)) return BITNET_A48_ERR_UNSUPPORTED;
    const int mt = M == 1 ? 1 : (M == 2 ? 2 : (M <= 4 ? 4 : 8));
    const size_t smem = (size_t)mt * w->trit5_row * 8 + 243 * 8;
    int dev = 0, sms = 0;
    A48_CUDA_TRY(cudaGetDevice(&dev));
    A48_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    int grid = sms * 4;
    if (grid * kWarps > w->N) grid = (w->N + kWarps - 1) / kWarps;
#define A48_T5(MT)                                                                                                          \
    do {                                                                                                                     \
        if (smem > 48 * 1024)                                                                                                \
            A48_CUDA_TRY(cudaFuncSetAttribute(decode_trit5_kernel<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
        A48_CUDA_TRY(a48_launch_pdl(decode_trit5_kernel<MT>, dim3(grid), dim3(kThreads), smem, st, w->trit5, w->trit5_row, codes, \
                                    scale, w->alpha_dev, M, w->N, w->K, Y, acc));                                            \
    } while (0)
    if (mt == 1) A48_T5(1);
    else if (mt == 2) A48_T5(2);
    else if (mt == 4) A48_T5(4);
    else A48_T5(8);
#undef A48_T5
    return BITNET_A48_OK;
}
