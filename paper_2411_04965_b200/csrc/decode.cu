// Decode BitLinear (Eq. 1 / Eq. 6) for up to 8 tokens: streams every byte of the
// 2-bit packed weights once at HBM speed.
//
// The matrix is 11 MB at the 7B shape, about 1.7 us of HBM time, so the kernel is
// built to have all of its bytes in flight at once: the 16-row tiles are dealt to
// thread-block clusters, the cluster's CTAs split K between them, and a producer
// warp in every CTA requests the CTA's whole share with bulk copies into a ring
// of shared-memory slots right at the start.  Eight consumer warps turn each slot
// (one 16-row tile over this CTA's K range) into int32 partial sums with
// mma.sync m16n8k32 (u8 x s8): the fragment-major layout makes one 128-bit
// shared-memory load per lane the A fragments of four MMAs, the 2-bit fields
// e = t+1 being isolated with a shift and a mask; the offset is removed afterwards
// by subtracting sum_k x[m,k] of the CTA's K range.  The K-split partial sums are
// added across the cluster through distributed shared memory (no global scratch,
// no atomics), rescaled by scale[m]*alpha and stored.
#include <cuda.h>

#include "internal.h"

namespace {

constexpr int CONSUMER_WARPS = 8;
constexpr int THREADS = 32 * (CONSUMER_WARPS + 1);
constexpr int UNIT_BYTES = 512;       // 16 rows x 128 channels of 2-bit codes
constexpr int MAX_SLOTS = 32;
constexpr int MAX_TILES = 64;         // 16-row tiles per cluster (bounds the partial-sum buffer)
constexpr int RING_BYTES = 96 * 1024;
constexpr int TOK = 8;                // tokens per launch (one MMA column group)
constexpr unsigned long long kWaitClocks = 4000000000ull;

__device__ unsigned int g_decode_status[4];

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait; false when it ran out of time (the first such event is recorded).
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, uint32_t id, uint32_t iter) {
    const unsigned long long t0 = clock64();
    uint32_t spins = 0;
    while (true) {
        if (mbar_try(bar, parity)) return true;
        if ((++spins & 255u) == 0 && clock64() - t0 > kWaitClocks) {
            if (atomicCAS(&g_decode_status[0], 0u, (unsigned)BITNET_A48_ERR_TIMEOUT) == 0u) {
                g_decode_status[1] = id;
                g_decode_status[2] = blockIdx.x;
                g_decode_status[3] = iter;
            }
            return false;
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t id, uint32_t iter) {
    if (mbar_try(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, id, iter);
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ int ld_peer_s32(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    int v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(v) : "r"(remote) : "memory");
    return v;
}
// C[16x8] += A[16x32] (u8) * B[32x8] (s8)
__device__ __forceinline__ void mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct DecodeParams {
    const uint8_t* wdec;  // fragment-major packed weights
    const int8_t* codes;  // [M, K]
    const float* scale;   // [M]
    const float* alpha;
    float* Y;             // [M, N]
    int32_t* acc;         // [M, N] or nullptr
    int M, N, K;
    int kchunks;          // 128-channel chunks per row of units
    int ntiles;           // 16-row tiles that hold at least one real row
    int nclusters, csize; // clusters in the grid, CTAs per cluster
    int nslots, slot_bytes, act_row_bytes;
};

// Dynamic shared memory: ring [nslots][slot_bytes] | act [TOK][act_row_bytes] | partial [MAX_TILES][16][TOK] s32 |
// csum [TOK] s32 | full[MAX_SLOTS], empty[MAX_SLOTS] mbarriers.
__global__ void __launch_bounds__(THREADS) decode_kernel(const DecodeParams p) {
    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t* ring = smem;
    uint8_t* act = ring + (size_t)p.nslots * p.slot_bytes;
    int* partial = reinterpret_cast<int*>(act + TOK * p.act_row_bytes);
    int* csum = partial + MAX_TILES * 16 * TOK;
    uint64_t* bars = reinterpret_cast<uint64_t*>(csum + TOK);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * MAX_SLOTS;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();
    const int cid = blockIdx.x / p.csize;
    const int kc0 = (int)((long long)rank * p.kchunks / p.csize), kc1 = (int)((long long)(rank + 1) * p.kchunks / p.csize);
    const int nkc = kc1 - kc0;
    const int t0 = (int)((long long)cid * p.ntiles / p.nclusters), t1 = (int)((long long)(cid + 1) * p.ntiles / p.nclusters);
    const int nparts = t1 - t0;
    const uint32_t part_bytes = (uint32_t)nkc * UNIT_BYTES;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.nslots; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    bool ok = true;
    if (warp == CONSUMER_WARPS) {
        // ------------------------------------------------------------- producer: the CTA's whole share, at once
        if (lane == 0 && nkc > 0) {
            for (int j = 0; j < nparts && ok; ++j) {
                const int s = j % p.nslots;
                if (j >= p.nslots) ok = mbar_wait(bar_empty + 8 * s, ((j / p.nslots) - 1) & 1, 1, j);
                if (!ok) break;
                mbar_expect_tx(bar_full + 8 * s, part_bytes);
                bulk_load(smem_u32(ring + (size_t)s * p.slot_bytes),
                          p.wdec + ((size_t)(t0 + j) * p.kchunks + kc0) * UNIT_BYTES, part_bytes, bar_full + 8 * s);
            }
        }
    } else {
        // ------------------------------------------------------------- consumers
        // Stage this CTA's K range of the activation codes, permuted so that the eight
        // words a thread needs for one 128-channel chunk are contiguous:
        // word (chunk, r = 8i + 4h + tig)  ->  chunk*32 + tig*8 + 2i + h.
        const int tid = threadIdx.x;
        const int nwords = nkc * 32;
        for (int idx = tid; idx < TOK * nwords; idx += 32 * CONSUMER_WARPS) {
            const int m = idx / nwords, wsrc = idx % nwords;
            const int kcl = wsrc >> 5, r = wsrc & 31;
            const int k = (kc0 + kcl) * 128 + 4 * r;
            uint32_t v = 0;
            if (m < p.M && k < p.K) v = *reinterpret_cast<const uint32_t*>(p.codes + (size_t)m * p.K + k);
            const int dst = kcl * 32 + (r & 3) * 8 + (r >> 3) * 2 + ((r >> 2) & 1);
            *reinterpret_cast<uint32_t*>(act + (size_t)m * p.act_row_bytes + 4 * dst) = v;
        }
        asm volatile("bar.sync 1, %0;" ::"n"(32 * CONSUMER_WARPS) : "memory");
        {   // warp w: sum of the staged codes of token w (the offset of the e = t+1 encoding)
            const uint32_t* row = reinterpret_cast<const uint32_t*>(act + (size_t)warp * p.act_row_bytes);
            int s = 0;
            for (int i = lane; i < nwords; i += 32) s = __dp4a((int)row[i], 0x01010101, s);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (lane == 0) csum[warp] = s;
        }
        asm volatile("bar.sync 1, %0;" ::"n"(32 * CONSUMER_WARPS) : "memory");

        const int g = lane >> 2, tig = lane & 3;
        const int cs0 = csum[2 * tig], cs1 = csum[2 * tig + 1];
        const uint8_t* arow = act + (size_t)g * p.act_row_bytes + tig * 32;
        for (int j = warp; j < nparts; j += CONSUMER_WARPS) {
            const int s = j % p.nslots;
            int c[4] = {0, 0, 0, 0};
            if (nkc > 0) {
                ok = __all_sync(0xffffffffu, mbar_wait(bar_full + 8 * s, (j / p.nslots) & 1, 2, j)) && ok;
                if (ok) {
                    const uint8_t* slot = ring + (size_t)s * p.slot_bytes + lane * 16;
#pragma unroll 2
                    for (int u = 0; u < nkc; ++u) {
                        const uint4 a = *reinterpret_cast<const uint4*>(slot + u * UNIT_BYTES);
                        const uint4 b_lo = *reinterpret_cast<const uint4*>(arow + u * 128);
                        const uint4 b_hi = *reinterpret_cast<const uint4*>(arow + u * 128 + 16);
                        constexpr uint32_t kMask = 0x03030303u;
                        mma_u8s8(c, a.x & kMask, a.y & kMask, a.z & kMask, a.w & kMask, b_lo.x, b_lo.y);
                        mma_u8s8(c, (a.x >> 2) & kMask, (a.y >> 2) & kMask, (a.z >> 2) & kMask, (a.w >> 2) & kMask, b_lo.z,
                                 b_lo.w);
                        mma_u8s8(c, (a.x >> 4) & kMask, (a.y >> 4) & kMask, (a.z >> 4) & kMask, (a.w >> 4) & kMask, b_hi.x,
                                 b_hi.y);
                        mma_u8s8(c, (a.x >> 6) & kMask, (a.y >> 6) & kMask, (a.z >> 6) & kMask, (a.w >> 6) & kMask, b_hi.z,
                                 b_hi.w);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_empty + 8 * s);
            }
            // rows g and g+8 of the tile, tokens 2*tig and 2*tig+1
            int2* dst = reinterpret_cast<int2*>(partial + ((size_t)j * 16 + g) * TOK + 2 * tig);
            dst[0] = make_int2(c[0] - cs0, c[1] - cs1);
            dst[8 * TOK / 2] = make_int2(c[2] - cs0, c[3] - cs1);
        }
    }
    // ----------------------------------------------------------------- add the K-split partial sums across the cluster
    cluster_sync();
    {
        const float alpha = *p.alpha;
        const uint32_t partial_addr = smem_u32(partial);
        for (int j = (int)rank; j < nparts; j += p.csize) {
            for (int v = threadIdx.x; v < 16 * TOK; v += THREADS) {
                const int row = v / TOK, m = v % TOK;
                const int n = (t0 + j) * 16 + row;
                int sum = 0;
                for (int rr = 0; rr < p.csize; ++rr) sum += ld_peer_s32(partial_addr + 4 * (j * 16 * TOK + v), (uint32_t)rr);
                if (m < p.M && n < p.N) {
                    const size_t o = (size_t)m * p.N + n;
                    p.Y[o] = (float)sum * (p.scale[m] * alpha);  // prefactors of Eq. 2, 3 and 7
                    if (p.acc) p.acc[o] = sum;
                }
            }
        }
    }
    cluster_sync();  // a peer may still be reading this CTA's partial sums
}

int sm_count() {
    static int n = 0;
    if (!n) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    }
    return n;
}

size_t smem_bytes(int nslots, int slot_bytes, int act_row_bytes) {
    return (size_t)nslots * slot_bytes + (size_t)TOK * act_row_bytes + (size_t)MAX_TILES * 16 * TOK * 4 + TOK * 4 +
           2 * MAX_SLOTS * 8;
}

}  // namespace

bool a48_decode_supported(const bitnet_a48_weight* w, int M) {
    return w->decode != nullptr && M >= 1 && M <= TOK && w->K % 16 == 0;
}
bool a48_decode_sparse_supported(const bitnet_a48_weight*, int) { return false; }
size_t a48_decode_workspace_bytes(const bitnet_a48_weight*, int) { return 0; }

bitnet_a48_status a48_launch_decode(const bitnet_a48_weight* w, const int8_t* codes, const float* scale, int M,
                                    float* Y, int32_t* acc, void*, size_t, cudaStream_t st) {
    DecodeParams p;
    p.wdec = w->decode;
    p.codes = codes;
    p.scale = scale;
    p.alpha = w->alpha_dev;
    p.Y = Y;
    p.acc = acc;
    p.M = M;
    p.N = w->N;
    p.K = w->K;
    p.kchunks = w->Kp / 128;
    p.ntiles = (w->N + 15) / 16;
    p.csize = p.kchunks >= 16 ? 4 : (p.kchunks >= 4 ? 2 : 1);
    const int max_nkc = (p.kchunks + p.csize - 1) / p.csize;
    p.slot_bytes = max_nkc * UNIT_BYTES;
    p.act_row_bytes = max_nkc * 128 + 16;
    if (p.slot_bytes > RING_BYTES) return BITNET_A48_ERR_UNSUPPORTED;
    int nclusters = sm_count() / p.csize;
    if (nclusters > p.ntiles) nclusters = p.ntiles;
    if ((p.ntiles + nclusters - 1) / nclusters > MAX_TILES) nclusters = (p.ntiles + MAX_TILES - 1) / MAX_TILES;
    p.nclusters = nclusters;
    const int parts_max = (p.ntiles + nclusters - 1) / nclusters;
    int nslots = RING_BYTES / p.slot_bytes;
    if (nslots > MAX_SLOTS) nslots = MAX_SLOTS;
    if (nslots > parts_max) nslots = parts_max;
    p.nslots = nslots;
    const size_t smem = smem_bytes(nslots, p.slot_bytes, p.act_row_bytes);
    static size_t smem_set = 0;
    if (smem > smem_set) {
        A48_CUDA_TRY(cudaFuncSetAttribute(decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        smem_set = smem;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(nclusters * p.csize));
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)p.csize;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    A48_CUDA_TRY(cudaLaunchKernelEx(&cfg, decode_kernel, p));
    return BITNET_A48_OK;
}

bitnet_a48_status a48_launch_decode_sparse(const bitnet_a48_weight*, const int8_t*, const float*, int, float*, int32_t*,
                                           void*, size_t, cudaStream_t) {
    return BITNET_A48_ERR_UNSUPPORTED;
}

bitnet_a48_status a48_read_decode_status(unsigned int words_host[4]) {
    A48_CUDA_TRY(cudaMemcpyFromSymbol(words_host, g_decode_status, sizeof(unsigned int) * 4));
    const unsigned int zero[4] = {0, 0, 0, 0};
    A48_CUDA_TRY(cudaMemcpyToSymbol(g_decode_status, zero, sizeof(zero)));
    return BITNET_A48_OK;
}
