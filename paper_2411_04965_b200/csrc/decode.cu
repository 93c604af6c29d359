// Decode BitLinear (Eq. 1 / Eq. 6) for up to 8 tokens: streams every byte of the
// 2-bit packed weights once at HBM speed.
//
// One matrix is 11 MB at the 7B shape, about 1.7 us of HBM time, so the kernel is
// built to have all of its bytes in flight at once and to keep every SM equally
// busy.  The packed matrix is a sequence of 512-byte units (16 output rows x 128
// channels, ordered tile by tile, see DecodeLayout).  The sequence is cut into one
// contiguous, equally long piece per CTA whatever the tile boundaries ("stream-K"),
// and every thread requests its 16 bytes of every unit of its warp's share with
// cp.async right at the start, before anything else happens.  Inside a piece a warp
// takes every sixteenth 128-channel chunk, over all tiles of the piece, so that it
// loads the token codes of a chunk once and reuses them for each tile.
//
// A warp turns each unit into int32 partial sums with four mma.sync m16n8k32
// (u8 x s8): one 128-bit shared-memory load per lane is the A fragments of the four
// MMAs, the 2-bit fields e = t+1 being isolated with a shift and a mask; the token
// codes are the B fragments, copied once per CTA into shared memory (rows padded by
// 16 bytes, which keeps the fragment loads free of bank conflicts) by the first
// cp.async group, ahead of the weights.  Sums of a tile are added up in shared memory.
// A tile that lies wholly inside the CTA's piece is finished there.  The at most
// two tiles a piece shares with its neighbours go through a global scratch array
// of 64-bit words, one per (row, token): a contributor adds its partial sum
// (biased to be non-negative) to the low 40 bits and 1 to the bits above with a
// single atomic; whoever sees from the returned old value that everybody else has
// been there holds the complete sum, finishes the element and stores zero back, so
// that the scratch is clean for the next call.  One round trip, no fences, no
// waiting.  Finishing means removing the offset of the encoding (sum_k x[m,k], once
// per row) and applying scale[m]*alpha.
#include <cuda.h>

#include "internal.h"

namespace {

constexpr int WARPS = 16;
constexpr int THREADS = 32 * WARPS;
constexpr int UNIT_BYTES = 512;   // 16 rows x 128 channels of 2-bit codes
constexpr int TOK = 8;            // tokens per launch (one MMA column group)
constexpr int MAX_SHARE = 288;    // units per CTA (144 KB of packed weights)
constexpr int MAX_TILES = 64;     // tiles a CTA's piece may touch (bounds the shared partial-sum array)
constexpr int MAX_GROUPS = 8;     // cp.async commit groups of weights per thread
constexpr int NTL = 6;            // tiles whose accumulators a warp carries in registers at a time

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)),
                 "l"(gmem_src)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// Waits until at most `pending` of this thread's commit groups are still in flight.
__device__ __forceinline__ void cp_async_wait(int pending) {
    switch (pending) {
        case 0: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
        case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
        case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
        case 3: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
        case 4: asm volatile("cp.async.wait_group 4;" ::: "memory"); break;
        case 5: asm volatile("cp.async.wait_group 5;" ::: "memory"); break;
        case 6: asm volatile("cp.async.wait_group 6;" ::: "memory"); break;
        case 7: asm volatile("cp.async.wait_group 7;" ::: "memory"); break;
        default: asm volatile("cp.async.wait_group 8;" ::: "memory"); break;
    }
}
static_assert(MAX_GROUPS <= 8, "cp_async_wait covers up to 8 pending groups");

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
    unsigned long long* ws;  // [ntiles][16][TOK]: arrivals << 40 | biased partial sums of shared tiles; zero between calls
    int M, N, K;
    int kchunks;          // units per tile (128-channel chunks of the padded K)
    int units;            // ntiles * kchunks
    int grid;             // CTAs
    int act_row_bytes;    // padded K + 16
};

// CTA that owns unit u when `units` units are cut into `grid` pieces [c*units/grid, (c+1)*units/grid).
__device__ __forceinline__ int owner_of(int u, int units, int grid) {
    return (int)((((long long)u + 1) * grid + units - 1) / units) - 1;
}

// Dynamic shared memory: wbuf [share][512] | act [M][act_row_bytes] | sacc [MAX_TILES][16][TOK] s32 | csum [TOK] s32
__global__ void __launch_bounds__(THREADS) decode_kernel(const DecodeParams p, int share_max) {
    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t* wbuf = smem;
    uint8_t* act = wbuf + (size_t)share_max * UNIT_BYTES;
    int* sacc = reinterpret_cast<int*>(act + (size_t)p.M * p.act_row_bytes);
    int* csum = sacc + MAX_TILES * 16 * TOK;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int u0 = (int)((long long)blockIdx.x * p.units / p.grid), u1 = (int)((long long)(blockIdx.x + 1) * p.units / p.grid);
    const int share = u1 - u0;
    const int first_tile = u0 / p.kchunks;
    const int ntl = share > 0 ? (u1 - 1) / p.kchunks - first_tile + 1 : 0;  // tiles this piece touches

    // ---- first group: the token codes, rows of K bytes in 16-byte pieces (pieces past K are written as zeros)
    const int row_pieces = p.kchunks * 8, real_pieces = p.K / 16;
    for (int idx = threadIdx.x; idx < p.M * row_pieces; idx += THREADS) {
        const int m = idx / row_pieces, c = idx % row_pieces;
        uint8_t* dst = act + (size_t)m * p.act_row_bytes + c * 16;
        if (c < real_pieces) cp_async16(dst, p.codes + (size_t)m * p.K + c * 16);
        else *reinterpret_cast<uint4*>(dst) = make_uint4(0, 0, 0, 0);
    }
    cp_async_commit();
    // ---- then this warp's units: chunks warp, warp + WARPS, ... of every tile of the piece.  Nothing here
    // depends on anything but the weights.
    const int my_chunks = p.kchunks > warp ? (p.kchunks - warp + WARPS - 1) / WARPS : 0;
    const int per_group = (my_chunks + MAX_GROUPS - 1) / MAX_GROUPS;  // chunks per commit group
    const int ngroups = per_group ? (my_chunks + per_group - 1) / per_group : 0;
    for (int j = 0; j < my_chunks; ++j) {
        const int kc = warp + j * WARPS;
        for (int tl = 0; tl < ntl; ++tl) {
            const int u = (first_tile + tl) * p.kchunks + kc;
            if (u >= u0 && u < u1)
                cp_async16(wbuf + (size_t)(u - u0) * UNIT_BYTES + lane * 16, p.wdec + (size_t)u * UNIT_BYTES + lane * 16);
        }
        if (j % per_group == per_group - 1 || j == my_chunks - 1) cp_async_commit();
    }

    for (int i = threadIdx.x; i < MAX_TILES * 16 * TOK; i += THREADS) sacc[i] = 0;
    if (threadIdx.x < TOK) csum[threadIdx.x] = 0;
    __syncthreads();
    // sum of the codes of every token (the offset of the e = t+1 encoding): each thread adds up the pieces it copied
    cp_async_wait(ngroups);
    {
        int s = 0, cur = -1;
        for (int idx = threadIdx.x; idx < p.M * row_pieces; idx += THREADS) {
            const int m = idx / row_pieces, c = idx % row_pieces;
            if (m != cur) {
                if (cur >= 0) atomicAdd(csum + cur, s);
                cur = m;
                s = 0;
            }
            const uint4 v = *reinterpret_cast<const uint4*>(act + (size_t)m * p.act_row_bytes + c * 16);
            s = __dp4a((int)v.x, 0x01010101, s);
            s = __dp4a((int)v.y, 0x01010101, s);
            s = __dp4a((int)v.z, 0x01010101, s);
            s = __dp4a((int)v.w, 0x01010101, s);
        }
        if (cur >= 0) atomicAdd(csum + cur, s);
    }
    __syncthreads();

    // ---- this warp's units -> partial sums of their tiles.  Up to NTL tiles are carried in registers at a time
    // and walked side by side, so that consecutive MMAs are independent; one flush per tile at the end.
    const int g = lane >> 2, tig = lane & 3;
    const bool tok_ok = g < p.M;  // B-fragment column g is token g; columns of missing tokens stay zero
    const uint8_t* arow = act + (size_t)(tok_ok ? g : 0) * p.act_row_bytes + tig * 4;
    for (int tb = 0; tb < ntl; tb += NTL) {
        int c[NTL][4];
#pragma unroll
        for (int t = 0; t < NTL; ++t) c[t][0] = c[t][1] = c[t][2] = c[t][3] = 0;
        for (int j = 0; j < my_chunks; ++j) {
            const int kc = warp + j * WARPS;
            if (tb == 0 && j % per_group == 0) cp_async_wait(ngroups - 1 - j / per_group);  // a lane reads only its own copies
            // B fragments of MMA q: channels 32q + 4tig .. +3 and 32q + 16 + 4tig .. +3 of token g
            uint32_t b[4][2];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                b[q][0] = tok_ok ? *reinterpret_cast<const uint32_t*>(arow + kc * 128 + q * 32) : 0u;
                b[q][1] = tok_ok ? *reinterpret_cast<const uint32_t*>(arow + kc * 128 + q * 32 + 16) : 0u;
            }
            uint4 a[NTL];
            bool have[NTL];
#pragma unroll
            for (int t = 0; t < NTL; ++t) {
                const int u = (first_tile + tb + t) * p.kchunks + kc;
                have[t] = tb + t < ntl && u >= u0 && u < u1;
                a[t] = make_uint4(0, 0, 0, 0);
                if (have[t]) a[t] = *reinterpret_cast<const uint4*>(wbuf + (size_t)(u - u0) * UNIT_BYTES + lane * 16);
            }
            constexpr uint32_t kMask = 0x03030303u;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
#pragma unroll
                for (int t = 0; t < NTL; ++t)
                    if (have[t])
                        mma_u8s8(c[t], (a[t].x >> (2 * q)) & kMask, (a[t].y >> (2 * q)) & kMask, (a[t].z >> (2 * q)) & kMask,
                                 (a[t].w >> (2 * q)) & kMask, b[q][0], b[q][1]);
            }
        }
#pragma unroll
        for (int t = 0; t < NTL; ++t) {
            if (tb + t >= ntl) continue;
            // rows g and g+8 of the tile, tokens 2*tig and 2*tig+1
            int* dst = sacc + ((size_t)(tb + t) * 16 + g) * TOK + 2 * tig;
            if (2 * tig < p.M) {
                atomicAdd(dst, c[t][0]);
                atomicAdd(dst + 8 * TOK, c[t][2]);
            }
            if (2 * tig + 1 < p.M) {
                atomicAdd(dst + 1, c[t][1]);
                atomicAdd(dst + 8 * TOK + 1, c[t][3]);
            }
        }
    }
    __syncthreads();

    // ---- finish the tiles: one thread per (tile, row, token)
    const float alpha = *p.alpha;
    constexpr unsigned long long kLow = (1ull << 40) - 1;
    constexpr long long kBias = 1ll << 31;
    for (int idx = threadIdx.x; idx < ntl * 16 * p.M; idx += THREADS) {
        const int m = idx % p.M, row = (idx / p.M) % 16, tl = idx / (16 * p.M);
        const int tile = first_tile + tl;
        const int tb = tile * p.kchunks, te = tb + p.kchunks;
        long long sum = sacc[(tl * 16 + row) * TOK + m];
        if (tb < u0 || te > u1) {  // shared with neighbours
            const long long contributors = owner_of(te - 1, p.units, p.grid) - owner_of(tb, p.units, p.grid) + 1;
            unsigned long long* slot = p.ws + ((size_t)tile * 16 + row) * TOK + m;
            const unsigned long long mine = (1ull << 40) | (unsigned long long)(sum + kBias);
            const unsigned long long old = atomicAdd(slot, mine);
            if ((long long)(old >> 40) != contributors - 1) continue;  // somebody later will finish this element
            sum = (long long)((old & kLow) + (mine & kLow)) - contributors * kBias;
            *slot = 0;
        }
        const int n = tile * 16 + row;
        if (n < p.N) {
            const int v = (int)sum - csum[m];
            const size_t o = (size_t)m * p.N + (size_t)n;
            p.Y[o] = (float)v * (p.scale[m] * alpha);  // prefactors of Eq. 2, 3 and 7
            if (p.acc) p.acc[o] = v;
        }
    }
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

size_t align256(size_t v) { return (v + 255) / 256 * 256; }
size_t ws_bytes_for(const bitnet_a48_weight* w) {
    return align256((size_t)((w->N + 15) / 16) * 16 * TOK * sizeof(unsigned long long));
}

}  // namespace

bool a48_decode_supported(const bitnet_a48_weight* w, int M) {
    return w->decode != nullptr && M >= 1 && M <= TOK && w->K % 16 == 0 && (size_t)M * (w->Kp + 16) <= 96 * 1024 &&
           (long long)((w->N + 15) / 16) * (w->Kp / 128) < (1ll << 31);
}
bool a48_decode_sparse_supported(const bitnet_a48_weight*, int) { return false; }
size_t a48_decode_workspace_bytes(const bitnet_a48_weight* w, int M) {
    return a48_decode_supported(w, M) ? ws_bytes_for(w) : 0;
}

bitnet_a48_status a48_launch_decode(const bitnet_a48_weight* w, const int8_t* codes, const float* scale, int M,
                                    float* Y, int32_t* acc, void* ws, size_t ws_bytes, cudaStream_t st) {
    if (!ws || ws_bytes < a48_decode_workspace_bytes(w, M)) return BITNET_A48_ERR_NOMEM;
    DecodeParams p;
    p.wdec = w->decode;
    p.codes = codes;
    p.scale = scale;
    p.alpha = w->alpha_dev;
    p.Y = Y;
    p.acc = acc;
    p.ws = static_cast<unsigned long long*>(ws);
    p.M = M;
    p.N = w->N;
    p.K = w->K;
    p.kchunks = w->Kp / 128;
    const long long ntiles = (w->N + 15) / 16;
    p.units = (int)(ntiles * p.kchunks);
    p.act_row_bytes = w->Kp + 16;
    // one piece per SM unless a piece would then not fit: at most MAX_SHARE units and MAX_TILES tiles per piece
    long long grid = sm_count();
    if (grid > p.units) grid = p.units;
    long long cap = MAX_SHARE;
    const long long tile_cap = (long long)(MAX_TILES - 2) * p.kchunks;
    if (tile_cap < cap) cap = tile_cap;
    if ((p.units + grid - 1) / grid > cap) grid = (p.units + cap - 1) / cap;
    p.grid = (int)grid;
    const int share_max = (int)((p.units + grid - 1) / grid);
    const size_t smem = (size_t)share_max * UNIT_BYTES + (size_t)M * p.act_row_bytes + (size_t)MAX_TILES * 16 * TOK * 4 + TOK * 4;
    if (smem > 227 * 1024 - 64) return BITNET_A48_ERR_UNSUPPORTED;
    static size_t smem_set = 0;
    if (smem > smem_set) {
        A48_CUDA_TRY(cudaFuncSetAttribute(decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        smem_set = smem;
    }
    decode_kernel<<<(unsigned)grid, THREADS, smem, st>>>(p, share_max);
    A48_CUDA_TRY(cudaGetLastError());
    return BITNET_A48_OK;
}

bitnet_a48_status a48_launch_decode_sparse(const bitnet_a48_weight*, const int8_t*, const float*, int, float*, int32_t*,
                                           void*, size_t, cudaStream_t) {
    return BITNET_A48_ERR_UNSUPPORTED;
}
