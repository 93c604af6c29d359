// Decode BitLinear (Eq. 1 / Eq. 6, up to 8 tokens) over the densest byte packing of ternary weights: five codes per
// byte, b = sum_i (t_i + 1) * 3^i <= 242, i.e. 1.6 bits per weight where the paper counts log2(3) = 1.58 (Section 1)
// and the other layouts of this library spend 2.  A row of W is ceil(K/5) bytes, padded to a multiple of 16.
//
// Base-3 digits do not come apart with shifts and masks, so a byte is decoded through a 243-entry table in shared
// memory (two words per entry: the int8 codes t_0..t_3, and t_4), and the token codes are staged once per CTA in
// the matching groups of five (two words per group: x_0..x_3, and x_4).  Each table lookup then feeds two dp4a.
// The lanes of a warp look up unrelated bytes, so the table is kept in 16 copies, lane l reading copy l % 16: an
// entry's copies fill one 128-byte line, every lane pair has banks of its own, and no lookup waits for another.
// One warp owns a row at a time and streams it with 16-byte loads.  This trades arithmetic for bytes: a fifth
// fewer bytes from HBM, about twice the instructions per weight of the 2-bit kernels.
#include "internal.h"

namespace {

constexpr int kThreads = 512, kWarps = kThreads / 32;  // one CTA per SM: staging the codes and the table is paid once

constexpr int kLutCopies = 16;
constexpr int kMaxPieces = 5;  // 16-byte pieces of a row per lane: rows of up to 5 * 32 * 16 * 5 = 12800 channels

// Dynamic shared memory: xg [MT][groups] uint2 | lut [243][kLutCopies] uint2.
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
    for (int i = threadIdx.x; i < 243 * kLutCopies; i += kThreads) {
        const int b = i / kLutCopies;
        int d[5], v = b;
#pragma unroll
        for (int i = 0; i < 5; ++i) {
            d[i] = v % 3 - 1;
            v /= 3;
        }
        lut[i] = make_uint2((uint32_t)(d[0] & 0xff) | ((uint32_t)(d[1] & 0xff) << 8) | ((uint32_t)(d[2] & 0xff) << 16) |
                                ((uint32_t)(d[3] & 0xff) << 24),
                            (uint32_t)(d[4] & 0xff));
    }
    // the token codes, 16 at a time, scattered to their groups of five (byte j of a group's two words is code 5g + j;
    // group g = 16 p + s is the s-th byte of the 16-byte piece p that lane p % 32 loads: stored [m][s][p], so that the
    // 32 lanes of a warp, which hold consecutive pieces, read consecutive words)
    for (int i = threadIdx.x; i < MT * groups; i += kThreads) xg[i] = make_uint2(0u, 0u);
    __syncthreads();
    {
        uint8_t* xb = reinterpret_cast<uint8_t*>(xg);
        const int chunks = (K + 15) / 16;
        for (int i = threadIdx.x; i < M * chunks; i += kThreads) {
            const int m = i / chunks, k0 = 16 * (i % chunks);
            __align__(16) uint8_t c[16];
            if (k0 + 16 <= K && (K & 15) == 0) {
                *reinterpret_cast<uint4*>(c) = __ldg(reinterpret_cast<const uint4*>(codes + (size_t)m * K + k0));
            } else {
#pragma unroll
                for (int q = 0; q < 16; ++q) c[q] = k0 + q < K ? (uint8_t)codes[(size_t)m * K + k0 + q] : (uint8_t)0;
            }
#pragma unroll
            for (int q = 0; q < 16; ++q) {
                const int k = k0 + q, g = k / 5, j = k - 5 * g;
                if (k < K) xb[(((size_t)m * 16 + (g & 15)) * (groups / 16) + (g >> 4)) * 8 + j] = c[q];
            }
        }
    }
    __syncthreads();
    const float al = __ldg(alpha);
    const int pieces = row_bytes / 16;
    // A warp's rows are walked with the next row's pieces already requested (up to kMaxPieces 16-byte pieces per lane,
    // i.e. rows of up to 12800 channels), so that a lane always has a row's worth of loads in flight.
    const int stride = gridDim.x * kWarps;
    uint4 cur[kMaxPieces], nxt[kMaxPieces];
    auto fetch = [&](int n, uint4 (&dst)[kMaxPieces]) {
        const uint4* row = reinterpret_cast<const uint4*>(wt + (size_t)n * row_bytes);
#pragma unroll
        for (int i = 0; i < kMaxPieces; ++i) {
            const int p = lane + 32 * i;
            dst[i] = (n < N && p < pieces) ? __ldg(row + p) : make_uint4(0u, 0u, 0u, 0u);
        }
    };
    int n = blockIdx.x * kWarps + warp;
    fetch(n, cur);
    for (; n < N; n += stride) {
        fetch(n + stride, nxt);
        int acc[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) acc[m] = 0;
#pragma unroll
        for (int i = 0; i < kMaxPieces; ++i) {
            const int p = lane + 32 * i;
            if (p >= pieces) break;
            const uint32_t w[4] = {cur[i].x, cur[i].y, cur[i].z, cur[i].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const uint2 t = lut[((w[j] >> (8 * b)) & 0xffu) * kLutCopies + (lane & (kLutCopies - 1))];
#pragma unroll
                    for (int m = 0; m < MT; ++m) {
                        const uint2 x = xg[((size_t)m * 16 + 4 * j + b) * pieces + p];
                        acc[m] = __dp4a((int)t.y, (int)x.y, __dp4a((int)t.x, (int)x.x, acc[m]));
                    }
                }
            }
        }
#pragma unroll
        for (int i = 0; i < kMaxPieces; ++i) cur[i] = nxt[i];
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
    return w->trit5 != nullptr && M >= 1 && M <= 8 && w->trit5_row <= kMaxPieces * 32 * 16 && (size_t)8 * w->trit5_row * 8 + 243 * 8 * kLutCopies <= 200 * 1024;
}

bitnet_a48_status a48_launch_decode_trit5(const bitnet_a48_weight* w, const int8_t* codes, const float* scale, int M, float* Y,
                                          int32_t* acc, cudaStream_t st) {
    if (!a48_decode_trit5_supported(w, M)) return BITNET_A48_ERR_UNSUPPORTED;
    const int mt = M == 1 ? 1 : (M == 2 ? 2 : (M <= 4 ? 4 : 8));
    const size_t smem = (size_t)mt * w->trit5_row * 8 + 243 * 8 * kLutCopies;
    int dev = 0, sms = 0;
    A48_CUDA_TRY(cudaGetDevice(&dev));
    A48_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    int grid = sms;
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
