// Zero-skipping decode BitLinear for one token whose codes come from the top-K quantiser (Eq. 1): only the
// weight rows of input channels with a non-zero code are fetched: the saving in weight traffic that the paper
// attributes to activation sparsity (Section 1; Eq. 1).  It reads the channel-major layout (row k = the 2-bit codes of every output for
// channel k, see SparseLayout), so skipping a channel skips one contiguous row.
//
// Grid: (blocks of 1024 outputs) x (segments of the channel range).  A CTA first lists the non-zero channels of
// its segment, then four groups of 64 threads walk the list, each thread holding 16 outputs (one packed word per
// channel): acc[f] += x * e_f with e = t+1, the offset removed with the sum of the x it used.  The groups are
// added in shared memory; the segments meet in the same zero-restoring 64-bit scratch words the dense decode
// kernel uses (count in the high bits, biased sum in the low 40), and the last arriver rescales and stores.
#include "internal.h"

namespace {

constexpr int THREADS = 256;
constexpr int NB = 1024;         // outputs per CTA
constexpr int WORDS = NB / 16;   // packed words per channel row and CTA
constexpr int GROUPS = THREADS / WORDS;
constexpr int MAX_SEG = 512;     // channels per segment (bounds the list)

__global__ void __launch_bounds__(THREADS) decode_sparse_kernel(const uint32_t* __restrict__ wsp, int row_words,
                                                                const int8_t* __restrict__ codes,
                                                                const float* __restrict__ scale,
                                                                const float* __restrict__ alpha, float* __restrict__ Y,
                                                                int32_t* __restrict__ acc_out,
                                                                unsigned long long* __restrict__ ws, int N, int K,
                                                                int seg_len, int nseg) {
    __shared__ uint32_t list[MAX_SEG];  // channel << 8 | code byte
    __shared__ int n_list;
    __shared__ int part[GROUPS][NB];
    const int nb = blockIdx.x, seg = blockIdx.y;
    const int k0 = seg * seg_len, k1 = min(k0 + seg_len, K);
    if (threadIdx.x == 0) n_list = 0;
    __syncthreads();
    for (int k = k0 + threadIdx.x; k < k1; k += THREADS) {
        const int x = codes[k];
        if (x != 0) list[atomicAdd(&n_list, 1)] = ((uint32_t)k << 8) | (uint32_t)(uint8_t)x;
    }
    __syncthreads();
    const int n = n_list;
    const int grp = threadIdx.x / WORDS, wi = threadIdx.x % WORDS;
    const int word_idx = nb * WORDS + wi;
    const bool live = word_idx < row_words;
    int acc[16];
#pragma unroll
    for (int f = 0; f < 16; ++f) acc[f] = 0;
    int xs = 0;
    if (live) {
        for (int i = grp; i < n; i += 4 * GROUPS) {  // four channels in flight per thread
            uint32_t w[4];
            int x[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int j = i + u * GROUPS;
                const uint32_t e = j < n ? list[j] : 0u;
                x[u] = (int)(int8_t)(e & 0xffu);
                w[u] = j < n ? __ldg(wsp + (size_t)(e >> 8) * row_words + word_idx) : 0u;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                xs += x[u];
#pragma unroll
                for (int f = 0; f < 16; ++f) acc[f] += x[u] * (int)((w[u] >> (2 * f)) & 3u);
            }
        }
    }
#pragma unroll
    for (int f = 0; f < 16; ++f) part[grp][wi * 16 + f] = acc[f] - xs;  // e = t + 1
    __syncthreads();
    constexpr unsigned long long kLow = (1ull << 40) - 1;
    constexpr long long kBias = 1ll << 31;
    for (int o = threadIdx.x; o < NB; o += THREADS) {
        const int out = nb * NB + o;
        if (out >= N) continue;
        long long sum = 0;
#pragma unroll
        for (int g = 0; g < GROUPS; ++g) sum += part[g][o];
        if (nseg > 1) {
            unsigned long long* slot = ws + (size_t)out * 8;  // token 0 of the [row][8 tokens] scratch
            const unsigned long long mine = (1ull << 40) | (unsigned long long)(sum + kBias);
            const unsigned long long old = atomicAdd(slot, mine);
            if ((long long)(old >> 40) != nseg - 1) continue;
            sum = (long long)((old & kLow) + (mine & kLow)) - (long long)nseg * kBias;
            *slot = 0;
        }
        Y[out] = (float)(int)sum * (scale[0] * __ldg(alpha));  // prefactors of Eq. 2 and 3
        if (acc_out) acc_out[out] = (int)sum;
    }
}

int sm_count() {
    static int n[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    int& c = n[dev & 63];
    if (!c) cudaDeviceGetAttribute(&c, cudaDevAttrMultiProcessorCount, dev);
    return c;
}

}  // namespace

// The segments of one output meet in a 64-bit word whose low 40 bits add up one biased sum (about 2^31) per
// segment: at most 255 segments of at most MAX_SEG channels keep that sum below 2^40.
bool a48_decode_sparse_supported(const bitnet_a48_weight* w, int M) {
    return w->sparse != nullptr && M == 1 && (w->K + MAX_SEG - 1) / MAX_SEG <= 255;
}

size_t a48_decode_sparse_workspace_bytes(const bitnet_a48_weight* w, int M) {
    if (!a48_decode_sparse_supported(w, M)) return 0;
    return ((size_t)((w->N + 15) / 16) * 16 * 8 * sizeof(unsigned long long) + 255) / 256 * 256;  // same shape as the dense decode scratch
}

bitnet_a48_status a48_launch_decode_sparse(const bitnet_a48_weight* w, const int8_t* codes, const float* scale, int M,
                                           float* Y, int32_t* acc, void* ws, size_t ws_bytes, cudaStream_t st) {
    if (M != 1) return BITNET_A48_ERR_UNSUPPORTED;
    const size_t need = a48_decode_sparse_workspace_bytes(w, M);
    if (!ws || ws_bytes < need) return BITNET_A48_ERR_NOMEM;
    const int row_words = w->Np / 16;
    const int nblocks = (w->N + NB - 1) / NB;
    int nseg = (2 * sm_count() + nblocks - 1) / nblocks;  // about two CTAs per SM
    if (nseg < 1) nseg = 1;
    if (nseg > 255) nseg = 255;  // what the meeting word has room for
    int seg_len = (w->K + nseg - 1) / nseg;
    if (seg_len < 32) seg_len = 32;
    if (seg_len > MAX_SEG) seg_len = MAX_SEG;
    nseg = (w->K + seg_len - 1) / seg_len;
    if (nseg > 255) return BITNET_A48_ERR_UNSUPPORTED;  // (also what a48_decode_sparse_supported promises)
    dim3 grid((unsigned)nblocks, (unsigned)nseg);
    decode_sparse_kernel<<<grid, THREADS, 0, st>>>(reinterpret_cast<const uint32_t*>(w->sparse), row_words, codes, scale,
                                                  w->alpha_dev, Y, acc, static_cast<unsigned long long*>(ws), w->N,
                                                  w->K, seg_len, nseg);
    A48_CUDA_TRY(cudaGetLastError());
    return BITNET_A48_OK;
}
