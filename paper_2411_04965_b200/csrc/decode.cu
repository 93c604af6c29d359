// Decode BitLinear (Eq. 1 / Eq. 6) for up to 8 tokens: streams every byte of the
// 2-bit packed weights once at HBM speed.
//
// One matrix is 11 MB at the 7B shape, about 1.7 us of HBM time, so the kernel is
// built to have all of its bytes in flight at once and to keep every SM equally
// busy.  The packed matrix is a sequence of 512-byte units (16 output rows x 128
// channels, ordered tile by tile, see DecodeLayout).  The sequence is cut into one
// contiguous, equally long piece per CTA whatever the tile boundaries ("stream-K"),
// and the CTA requests its whole piece with cp.async right at the start, before
// anything else happens (and, under programmatic dependent launch, before the
// kernel ahead of it in the stream has finished).  Inside a piece a warp takes
// every eighth 128-channel chunk, over all tiles of the piece, so that it loads the
// token codes of a chunk once and reuses them for each tile.
//
// A warp turns each unit into int32 partial sums with four mma.sync m16n8k32
// (u8 x s8): one 128-bit shared-memory load per lane is the A fragments of the four
// MMAs, the 2-bit fields e = t+1 being isolated with a shift and a mask; the token
// codes are the B fragments, copied once per CTA into shared memory (rows padded by
// 16 bytes, which keeps the fragment loads free of bank conflicts) by bulk copies
// with a barrier of their own.  With a single token the same fields go through dp4a
// on the CUDA cores instead, which wastes no MMA columns.  Sums of a tile are added
// up in shared memory.
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

#include <type_traits>

#include "internal.h"

namespace {

constexpr int WARPS_MANY = 8;   // warps per CTA of the mma.sync form (2..8 tokens)
constexpr int WARPS_ONE = 12;   // ... of the one-token form
constexpr int UNIT_BYTES = 512;   // 16 rows x 128 channels of 2-bit codes
constexpr int TOK = 8;            // tokens per launch (one MMA column group)
constexpr int MAX_SHARE = 288;    // units per CTA (144 KB of packed weights)
constexpr int MAX_TILES = 24;     // tiles a CTA's piece may touch (bounds the shared partial-sum array)
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

__device__ unsigned int g_decode_status[4];
constexpr unsigned long long kWaitClocks = 4000000000ull;  // ~2 s at 2 GHz

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
// Bounded wait; when it runs out of time the first such event is recorded and the caller carries on.
__device__ __noinline__ void mbar_wait_bounded(uint32_t bar, uint32_t parity) {
    const unsigned long long t0 = clock64();
    uint32_t spins = 0;
    while (!mbar_try(bar, parity)) {
        if ((++spins & 255u) == 0 && clock64() - t0 > kWaitClocks) {
            if (atomicCAS(&g_decode_status[0], 0u, (unsigned)BITNET_A48_ERR_TIMEOUT) == 0u) {
                g_decode_status[1] = 100;
                g_decode_status[2] = blockIdx.x;
                g_decode_status[3] = 0;
            }
            return;
        }
    }
}

// sum of four u8 x s8 products plus c
__device__ __forceinline__ int dp4a_u8s8(uint32_t a, int b, int c) {
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

constexpr int MAX_MATS = 4;  // matrices of one K that one launch can run on the same token codes

struct DecodeParams {
    // The launch sees the 16-row tiles of its matrices as one sequence: matrix j owns tiles [tile_base[j], tile_base[j+1]).
    const uint8_t* wdec[MAX_MATS];  // fragment-major packed weights
    const float* alpha[MAX_MATS];
    float* Y[MAX_MATS];             // [M, N_j]
    int32_t* acc[MAX_MATS];         // [M, N_j] or nullptr
    int N[MAX_MATS];
    int tile_base[MAX_MATS + 1];
    int count;
    const int8_t* codes;  // [M, K]
    const float* scale;   // [M]
    unsigned long long* ws;  // [ntiles][16][TOK]: arrivals << 40 | biased partial sums of shared tiles; zero between calls
    int M, K;
    int kchunks;          // units per tile (128-channel chunks of the padded K)
    int units;            // ntiles * kchunks
    int grid;             // CTAs
    int tile_aligned;     // pieces end on tile boundaries: no tile is shared, the scratch stays untouched
    int piece_q, piece_r; // the first piece_r pieces hold piece_q + 1 items (tiles if tile_aligned, else units), the rest piece_q
    int act_row_bytes;    // padded K + 16
    int y_bf16;           // outputs are bf16 instead of fp32
    const float* residual;  // fp32 [M, N_0] added to the outputs of matrix 0, or nullptr
};

__device__ __forceinline__ int matrix_of(const DecodeParams& p, int tile) {
    int j = 0;
    while (j + 1 < p.count && tile >= p.tile_base[j + 1]) ++j;
    return j;
}

// First item of piece c when the items are dealt as piece_r pieces of piece_q + 1 followed by pieces of piece_q.
__device__ __forceinline__ int piece_begin(const DecodeParams& p, int c) { return c * p.piece_q + min(c, p.piece_r); }
// Piece that owns unit u (stream-K pieces, items = units).
__device__ __forceinline__ int owner_of(const DecodeParams& p, int u) {
    const int big = p.piece_r * (p.piece_q + 1);
    return u < big ? u / (p.piece_q + 1) : p.piece_r + (u - big) / p.piece_q;
}

// Dynamic shared memory: wbuf [share][512] | act [M][act_row_bytes] | sacc [MAX_TILES][16][TOK] s32 | csum [TOK] s32
// NW warps per CTA; ONE_TOKEN compiles the dp4a walk alone (M == 1: fewer registers, so twelve warps fit twice on
// an SM and shorten the walk that has to follow the dependency wait), otherwise the mma.sync walk alone.
template <int NW, bool ONE_TOKEN>
__global__ void __launch_bounds__(32 * NW, ONE_TOKEN ? 2 : 1) decode_kernel(const DecodeParams p, int share_max) {
    constexpr int WARPS = NW, THREADS = 32 * NW;
    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t* wbuf = smem;
    uint8_t* act = wbuf + (size_t)share_max * UNIT_BYTES;
    int* sacc = reinterpret_cast<int*>(act + (size_t)p.M * p.act_row_bytes);
    int* csum = sacc + MAX_TILES * 16 * TOK;
    __shared__ uint64_t act_bar;  // completes when the token codes have landed
    const uint32_t bar = (uint32_t)__cvta_generic_to_shared(&act_bar);
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int u0 = piece_begin(p, blockIdx.x), u1 = piece_begin(p, blockIdx.x + 1);  // no divisions on the way to the first copy
    if (p.tile_aligned) {
        u0 *= p.kchunks;
        u1 *= p.kchunks;
    }
    const int share = u1 - u0;
    const int first_tile = u0 / p.kchunks;
    const int ntl = share > 0 ? (u1 - 1) / p.kchunks - first_tile + 1 : 0;  // tiles this piece touches

    // ---- request the whole piece.  Copy group gq is chunks [gq*cg, (gq+1)*cg) of every tile of the piece (cg a
    // multiple of the warp count); the CTA's threads share each contiguous run 16 bytes at a time.  Nothing here
    // depends on anything but the weights, so it runs before the wait for the kernel ahead of this one in the
    // stream (programmatic dependent launch): the weight stream of this call overlaps the tail of the previous one.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // (twelve warps: at most five groups, so that a group still gives every warp two units at K = 11008)
    constexpr int GROUPS = ONE_TOKEN ? 5 : MAX_GROUPS;
    const int cg = WARPS * ((p.kchunks + WARPS * GROUPS - 1) / (WARPS * GROUPS));
    const int ngroups = (p.kchunks + cg - 1) / cg;
    // Pieces of one to six whole tiles (the usual case at model shapes) run code compiled for their tile count,
    // with the per-tile addresses in registers: a copy or a fragment load then costs one multiply-add.
    const bool whole = p.tile_aligned && ntl >= 1 && ntl <= NTL;
    auto for_tile_count = [&](auto f) {
        switch (ntl) {
            case 1: f(std::integral_constant<int, 1>{}); break;
            case 2: f(std::integral_constant<int, 2>{}); break;
            case 3: f(std::integral_constant<int, 3>{}); break;
            case 4: f(std::integral_constant<int, 4>{}); break;
            case 5: f(std::integral_constant<int, 5>{}); break;
            default: f(std::integral_constant<int, 6>{}); break;
        }
    };
    if (whole) {
        for_tile_count([&](auto nt_c) {
            constexpr int NT = decltype(nt_c)::value;
            const uint8_t* src[NT];
            uint32_t dst[NT];
#pragma unroll
            for (int t = 0; t < NT; ++t) {
                const int tile = first_tile + t, j = matrix_of(p, tile);
                src[t] = p.wdec[j] + lane * 16 + (size_t)(tile - p.tile_base[j]) * p.kchunks * UNIT_BYTES;
                dst[t] = (uint32_t)__cvta_generic_to_shared(wbuf) + lane * 16 + (uint32_t)(t * p.kchunks) * UNIT_BYTES;
            }
            for (int gq = 0; gq < ngroups; ++gq) {
                const int c_hi = min(gq * cg + cg, p.kchunks);
                for (int kc = gq * cg + warp; kc < c_hi; kc += WARPS) {
#pragma unroll
                    for (int t = 0; t < NT; ++t)
                        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst[t] + (uint32_t)kc * UNIT_BYTES),
                                     "l"(src[t] + (size_t)kc * UNIT_BYTES)
                                     : "memory");
                }
                cp_async_commit();
            }
        });
    } else {
        // a warp takes whole units (lane l the l-th 16 bytes of each), so that one cp.async instruction moves 512
        // contiguous bytes and the only arithmetic per copy is the unit index
        const uint32_t dst0 = (uint32_t)__cvta_generic_to_shared(wbuf) + lane * 16 - (uint32_t)u0 * UNIT_BYTES;
        for (int gq = 0; gq < ngroups; ++gq) {
            const int c_lo = gq * cg, c_hi = min(c_lo + cg, p.kchunks);
            for (int tl = 0; tl < ntl; ++tl) {
                const int base = (first_tile + tl) * p.kchunks;
                const int j = matrix_of(p, first_tile + tl);
                const uint8_t* src0 = p.wdec[j] + lane * 16 - (size_t)p.tile_base[j] * p.kchunks * UNIT_BYTES;
                for (int u = base + c_lo + warp; u < base + c_hi; u += WARPS)
                    if (u >= u0 && u < u1)
                        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst0 + (uint32_t)u * UNIT_BYTES),
                                     "l"(src0 + (size_t)u * UNIT_BYTES)
                                     : "memory");
            }
            cp_async_commit();
        }
    }
    // ---- the token codes: one bulk copy per row, tracked by a barrier of their own so that waiting for them does
    // not mean waiting for the weights (pieces past K are written as zeros).  They, the scratch and the outputs may
    // belong to the previous kernel until it has completed.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int row_pieces = p.kchunks * 8, real_pieces = p.K / 16;
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"((uint32_t)(p.M * p.K)) : "memory");
        for (int m = 0; m < p.M; ++m)
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"((uint32_t)__cvta_generic_to_shared(act + (size_t)m * p.act_row_bytes)),
                         "l"(p.codes + (size_t)m * p.K), "r"((uint32_t)p.K), "r"(bar)
                         : "memory");
    }
    for (int idx = threadIdx.x; idx < p.M * (row_pieces - real_pieces); idx += THREADS) {
        const int m = idx / (row_pieces - real_pieces), c = real_pieces + idx % (row_pieces - real_pieces);
        *reinterpret_cast<uint4*>(act + (size_t)m * p.act_row_bytes + c * 16) = make_uint4(0, 0, 0, 0);
    }

    for (int i = threadIdx.x; i < ntl * 16 * TOK; i += THREADS) sacc[i] = 0;
    if (threadIdx.x < TOK) csum[threadIdx.x] = 0;
    __syncthreads();
    mbar_wait_bounded(bar, 0);  // the token codes are in shared memory

    // ---- this warp's units -> partial sums of their tiles.  Up to NTL tiles are carried in registers at a time
    // and walked side by side, so that consecutive MMAs are independent; one flush per tile at the end.
    const int g = lane >> 2, tig = lane & 3;
    const bool tok_ok = g < p.M;  // B-fragment column g is token g; columns of missing tokens stay zero
    const uint8_t* arow = act + (size_t)(tok_ok ? g : 0) * p.act_row_bytes + tig * 4;
    if constexpr (ONE_TOKEN) {
        // One token: the MMA would spend seven of its eight columns on nothing, so the CUDA cores do it with dp4a.
        // A word masked with 0x03030303 << 2q is four u8 fields e * 4^q of one row and one 32-channel slice; the
        // sums of slice q carry the factor 4^q, which an exact shift removes at the end.  Rows g (words 0, 2) and
        // g+8 (words 1, 3); the four lanes of a quad hold different channels of the same rows.
        int xsum = 0;
        if (whole) {
            for_tile_count([&](auto nt_c) {
                constexpr int NT = decltype(nt_c)::value;
                int lo[NT][4], hi[NT][4];
#pragma unroll
                for (int t = 0; t < NT; ++t)
#pragma unroll
                    for (int q = 0; q < 4; ++q) lo[t][q] = hi[t][q] = 0;
                const uint8_t* a0 = wbuf + lane * 16;
                const uint32_t tile_bytes = (uint32_t)p.kchunks * UNIT_BYTES;
                for (int gq = 0; gq < ngroups; ++gq) {
                    cp_async_wait(ngroups - 1 - gq);  // group gq has landed for every thread
                    __syncthreads();
                    const int c_hi = min(gq * cg + cg, p.kchunks);
                    for (int kc = gq * cg + warp; kc < c_hi; kc += WARPS) {
                        int b[4][2];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            b[q][0] = *reinterpret_cast<const int*>(act + kc * 128 + q * 32 + tig * 4);
                            b[q][1] = *reinterpret_cast<const int*>(act + kc * 128 + q * 32 + 16 + tig * 4);
                            xsum = __dp4a(b[q][1], 0x01010101, __dp4a(b[q][0], 0x01010101, xsum));
                        }
                        uint4 a[NT];
#pragma unroll
                        for (int t = 0; t < NT; ++t)
                            a[t] = *reinterpret_cast<const uint4*>(a0 + t * tile_bytes + (uint32_t)kc * UNIT_BYTES);
#pragma unroll
                        for (int t = 0; t < NT; ++t) {
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const uint32_t mq = 0x03030303u << (2 * q);
                                lo[t][q] = dp4a_u8s8(a[t].x & mq, b[q][0], lo[t][q]);
                                lo[t][q] = dp4a_u8s8(a[t].z & mq, b[q][1], lo[t][q]);
                                hi[t][q] = dp4a_u8s8(a[t].y & mq, b[q][0], hi[t][q]);
                                hi[t][q] = dp4a_u8s8(a[t].w & mq, b[q][1], hi[t][q]);
                            }
                        }
                    }
                }
#pragma unroll
                for (int t = 0; t < NT; ++t) {
                    int r0 = lo[t][0] + (lo[t][1] >> 2) + (lo[t][2] >> 4) + (lo[t][3] >> 6);
                    int r1 = hi[t][0] + (hi[t][1] >> 2) + (hi[t][2] >> 4) + (hi[t][3] >> 6);
                    r0 += __shfl_xor_sync(0xffffffffu, r0, 1);
                    r1 += __shfl_xor_sync(0xffffffffu, r1, 1);
                    r0 += __shfl_xor_sync(0xffffffffu, r0, 2);
                    r1 += __shfl_xor_sync(0xffffffffu, r1, 2);
                    if (tig == 0) {
                        atomicAdd(sacc + ((size_t)t * 16 + g) * TOK, r0);
                        atomicAdd(sacc + ((size_t)t * 16 + g + 8) * TOK, r1);
                    }
                }
            });
        } else {
        // the walk is compiled for 3, 4, 5 and 6 tiles side by side: blank slots would cost as much as real ones
        auto walk = [&](auto nt_c) {
            constexpr int NT = decltype(nt_c)::value;
            for (int tb = 0; tb < ntl; tb += NT) {
                int lo[NT][4], hi[NT][4];
    #pragma unroll
                for (int t = 0; t < NT; ++t)
    #pragma unroll
                    for (int q = 0; q < 4; ++q) lo[t][q] = hi[t][q] = 0;
                for (int gq = 0; gq < ngroups; ++gq) {
                    if (tb == 0) {  // group gq has landed for every thread
                        cp_async_wait(ngroups - 1 - gq);
                        __syncthreads();
                    }
                    for (int kc = gq * cg + warp; kc < min((gq + 1) * cg, p.kchunks); kc += WARPS) {
                    int b[4][2];
    #pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        b[q][0] = *reinterpret_cast<const int*>(act + kc * 128 + q * 32 + tig * 4);
                        b[q][1] = *reinterpret_cast<const int*>(act + kc * 128 + q * 32 + 16 + tig * 4);
                    }
                    if (tb == 0) {  // this chunk's share of sum_k x[k]: every quad holds the same words, quad 0 reports
    #pragma unroll
                        for (int q = 0; q < 4; ++q) xsum = __dp4a(b[q][1], 0x01010101, __dp4a(b[q][0], 0x01010101, xsum));
                    }
                    // all tiles are loaded, units outside the piece from a valid address and then blanked: no branches
                    uint4 a[NT];
    #pragma unroll
                    for (int t = 0; t < NT; ++t) {
                        const int u = (first_tile + tb + t) * p.kchunks + kc;
                        const bool have = tb + t < ntl && u >= u0 && u < u1;
                        a[t] = *reinterpret_cast<const uint4*>(wbuf + (size_t)(have ? u - u0 : 0) * UNIT_BYTES + lane * 16);
                        if (!have) a[t] = make_uint4(0, 0, 0, 0);
                    }
    #pragma unroll
                    for (int t = 0; t < NT; ++t) {
    #pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const uint32_t mq = 0x03030303u << (2 * q);
                            lo[t][q] = dp4a_u8s8(a[t].x & mq, b[q][0], lo[t][q]);
                            lo[t][q] = dp4a_u8s8(a[t].z & mq, b[q][1], lo[t][q]);
                            hi[t][q] = dp4a_u8s8(a[t].y & mq, b[q][0], hi[t][q]);
                            hi[t][q] = dp4a_u8s8(a[t].w & mq, b[q][1], hi[t][q]);
                        }
                    }
                    }
                }
    #pragma unroll
                for (int t = 0; t < NT; ++t) {
                    if (tb + t >= ntl) continue;
                    int r0 = lo[t][0] + (lo[t][1] >> 2) + (lo[t][2] >> 4) + (lo[t][3] >> 6);
                    int r1 = hi[t][0] + (hi[t][1] >> 2) + (hi[t][2] >> 4) + (hi[t][3] >> 6);
                    r0 += __shfl_xor_sync(0xffffffffu, r0, 1);
                    r1 += __shfl_xor_sync(0xffffffffu, r1, 1);
                    r0 += __shfl_xor_sync(0xffffffffu, r0, 2);
                    r1 += __shfl_xor_sync(0xffffffffu, r1, 2);
                    if (tig == 0) {
                        atomicAdd(sacc + ((size_t)(tb + t) * 16 + g) * TOK, r0);
                        atomicAdd(sacc + ((size_t)(tb + t) * 16 + g + 8) * TOK, r1);
                    }
                }
            }
        };
        if (ntl <= 3) walk(std::integral_constant<int, 3>{});
        else if (ntl == 4) walk(std::integral_constant<int, 4>{});
        else if (ntl == 5) walk(std::integral_constant<int, 5>{});
        else walk(std::integral_constant<int, NTL>{});
        }
        xsum += __shfl_xor_sync(0xffffffffu, xsum, 1);
        xsum += __shfl_xor_sync(0xffffffffu, xsum, 2);
        if (lane == 0) atomicAdd(csum, xsum);
    }
    if constexpr (!ONE_TOKEN) {
    int xsum = 0;  // this lane's share of sum_k x[g][k]
    auto walk = [&](auto nt_c) {
    constexpr int NT = decltype(nt_c)::value;
    for (int tb = 0; tb < ntl; tb += NT) {
        int c[NT][4];
#pragma unroll
        for (int t = 0; t < NT; ++t) c[t][0] = c[t][1] = c[t][2] = c[t][3] = 0;
        for (int gq = 0; gq < ngroups; ++gq) {
            if (tb == 0) {  // group gq has landed for every thread
                cp_async_wait(ngroups - 1 - gq);
                __syncthreads();
            }
            for (int kc = gq * cg + warp; kc < min((gq + 1) * cg, p.kchunks); kc += WARPS) {
            // B fragments of MMA q: channels 32q + 4tig .. +3 and 32q + 16 + 4tig .. +3 of token g
            uint32_t b[4][2];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                b[q][0] = tok_ok ? *reinterpret_cast<const uint32_t*>(arow + kc * 128 + q * 32) : 0u;
                b[q][1] = tok_ok ? *reinterpret_cast<const uint32_t*>(arow + kc * 128 + q * 32 + 16) : 0u;
                if (tb == 0) xsum = __dp4a((int)b[q][1], 0x01010101, __dp4a((int)b[q][0], 0x01010101, xsum));
            }
            // all tiles are loaded, units outside the piece from a valid address and then blanked (a zero A fragment
            // adds nothing), so that no MMA sits behind a branch
            uint4 a[NT];
#pragma unroll
            for (int t = 0; t < NT; ++t) {
                const int u = (first_tile + tb + t) * p.kchunks + kc;
                const bool have = tb + t < ntl && u >= u0 && u < u1;
                a[t] = *reinterpret_cast<const uint4*>(wbuf + (size_t)(have ? u - u0 : 0) * UNIT_BYTES + lane * 16);
                if (!have) a[t] = make_uint4(0, 0, 0, 0);
            }
            constexpr uint32_t kMask = 0x03030303u;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
#pragma unroll
                for (int t = 0; t < NT; ++t)
                        mma_u8s8(c[t], (a[t].x >> (2 * q)) & kMask, (a[t].y >> (2 * q)) & kMask, (a[t].z >> (2 * q)) & kMask,
                                 (a[t].w >> (2 * q)) & kMask, b[q][0], b[q][1]);
            }
            }
        }
#pragma unroll
        for (int t = 0; t < NT; ++t) {
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
    };
    if (ntl <= 3) walk(std::integral_constant<int, 3>{});
    else if (ntl == 4) walk(std::integral_constant<int, 4>{});
    else if (ntl == 5) walk(std::integral_constant<int, 5>{});
    else walk(std::integral_constant<int, NTL>{});
    xsum += __shfl_xor_sync(0xffffffffu, xsum, 1);
    xsum += __shfl_xor_sync(0xffffffffu, xsum, 2);
    if (tig == 0 && tok_ok) atomicAdd(csum + g, xsum);
    }
    __syncthreads();

    // ---- finish the tiles: one thread per (tile, row, token)
    constexpr unsigned long long kLow = (1ull << 40) - 1;
    constexpr long long kBias = 1ll << 31;
    for (int idx = threadIdx.x; idx < ntl * 16 * p.M; idx += THREADS) {
        const int m = idx % p.M, row = (idx / p.M) % 16, tl = idx / (16 * p.M);
        const int tile = first_tile + tl;
        const int tb = tile * p.kchunks, te = tb + p.kchunks;
        long long sum = sacc[(tl * 16 + row) * TOK + m];
        if (tb < u0 || te > u1) {  // shared with neighbours
            const long long contributors = owner_of(p, te - 1) - owner_of(p, tb) + 1;
            unsigned long long* slot = p.ws + ((size_t)tile * 16 + row) * TOK + m;
            const unsigned long long mine = (1ull << 40) | (unsigned long long)(sum + kBias);
            const unsigned long long old = atomicAdd(slot, mine);
            if ((long long)(old >> 40) != contributors - 1) continue;  // somebody later will finish this element
            sum = (long long)((old & kLow) + (mine & kLow)) - contributors * kBias;
            *slot = 0;
        }
        const int j = matrix_of(p, tile);
        const int n = (tile - p.tile_base[j]) * 16 + row;
        if (n < p.N[j]) {
            const int v = (int)sum - csum[m];
            const size_t o = (size_t)m * p.N[j] + (size_t)n;
            float y = (float)v * (p.scale[m] * __ldg(p.alpha[j]));  // prefactors of Eq. 2, 3 and 7
            if (p.residual) y += p.residual[o];
            a48_store_y(p.Y[j], o, y, p.y_bf16);
            if (p.acc[j]) p.acc[j][o] = v;
        }
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

size_t align256(size_t v) { return (v + 255) / 256 * 256; }
size_t ws_bytes_for(const bitnet_a48_weight* w) {
    return align256((size_t)((w->N + 15) / 16) * 16 * TOK * sizeof(unsigned long long));
}

}  // namespace

bool a48_decode_supported(const bitnet_a48_weight* w, int M) {
    return w->decode != nullptr && M >= 1 && M <= TOK && w->K % 16 == 0 && (size_t)M * (w->Kp + 16) <= 96 * 1024 &&
           (long long)((w->N + 15) / 16) * (w->Kp / 128) < (1ll << 31);
}
size_t a48_decode_workspace_bytes(const bitnet_a48_weight* w, int M) {
    return a48_decode_supported(w, M) ? ws_bytes_for(w) : 0;
}

bitnet_a48_status a48_launch_decode(const bitnet_a48_weight* w, const int8_t* codes, const float* scale, int M,
                                    float* Y, int32_t* acc, void* ws, size_t ws_bytes, cudaStream_t st) {
    return a48_launch_decode_multi(1, &w, codes, scale, M, &Y, &acc, ws, ws_bytes, st);
}

size_t a48_decode_multi_workspace_bytes(int count, const bitnet_a48_weight* const* ws_, int M) {
    size_t total = 0;
    for (int j = 0; j < count; ++j) {
        if (!a48_decode_supported(ws_[j], M) || ws_[j]->K != ws_[0]->K) return 0;
        total += ws_bytes_for(ws_[j]);
    }
    return total;
}

bitnet_a48_status a48_launch_decode_multi(int count, const bitnet_a48_weight* const* wv, const int8_t* codes,
                                          const float* scale, int M, float* const* Y, int32_t* const* acc, void* ws,
                                          size_t ws_bytes, cudaStream_t st) {
    if (count < 1 || count > MAX_MATS) return BITNET_A48_ERR_LIMIT;
    const size_t need = a48_decode_multi_workspace_bytes(count, wv, M);
    if (need == 0) return BITNET_A48_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < need) return BITNET_A48_ERR_NOMEM;
    const bitnet_a48_weight* w = wv[0];
    DecodeParams p = {};
    long long ntiles = 0;
    bool prefetch_ok = true;
    for (int j = 0; j < count; ++j) {
        p.wdec[j] = wv[j]->decode;
        p.alpha[j] = wv[j]->alpha_dev;
        p.Y[j] = Y[j];
        p.acc[j] = acc ? acc[j] : nullptr;
        p.N[j] = wv[j]->N;
        p.tile_base[j] = (int)ntiles;
        ntiles += (wv[j]->N + 15) / 16;
        prefetch_ok = prefetch_ok && wv[j]->decode_prefetch_ok;
    }
    p.tile_base[count] = (int)ntiles;
    p.count = count;
    p.codes = codes;
    p.scale = scale;
    p.ws = static_cast<unsigned long long*>(ws);
    p.M = M;
    p.K = w->K;
    p.kchunks = w->Kp / 128;
    if (ntiles * p.kchunks >= (1ll << 31)) return BITNET_A48_ERR_UNSUPPORTED;
    p.units = (int)(ntiles * p.kchunks);
    p.act_row_bytes = w->Kp + 16;
    p.y_bf16 = a48_y_bf16;
    p.residual = count == 1 ? a48_decode_residual : nullptr;
    // one piece per SM unless a piece would then not fit: at most MAX_SHARE units and MAX_TILES tiles per piece
    long long grid = sm_count();
    if (grid > p.units) grid = p.units;
    long long cap = MAX_SHARE;
    const long long tile_cap = (long long)(MAX_TILES - 2) * p.kchunks;
    if (tile_cap < cap) cap = tile_cap;
    if ((p.units + grid - 1) / grid > cap) {
        // more pieces than SMs: a whole number of rounds (pieces of two rounds can share an SM when they are small)
        const long long rounds = (p.units + (long long)sm_count() * cap - 1) / ((long long)sm_count() * cap);
        grid = rounds * sm_count();
    }
    // Two CTAs must fit on an SM for a launch to request its weights while its predecessor still computes: with
    // many tokens the staged codes take room, so the pieces get shorter (more rounds of pieces) until they do.
    const size_t fixed_smem = (size_t)M * p.act_row_bytes + (size_t)MAX_TILES * 16 * TOK * 4 + TOK * 4;
    // (Only while the pieces stay whole tiles: pieces that share every tile pay more in fix-ups than the overlap
    // gives back - 13.4 us instead of 9 us for 4096 x 11008 at four tokens.)
    while (fixed_smem <= 64 * 1024 && grid % sm_count() == 0 && grid < 2ll * sm_count() && p.units / grid > 32 &&
           ntiles >= grid + sm_count() &&
           fixed_smem + (size_t)((p.units + grid - 1) / grid) * UNIT_BYTES > 112 * 1024)
        grid += sm_count();
    p.grid = (int)grid;
    int share_max = (int)((p.units + grid - 1) / grid);
    // With at least one tile per SM, whole tiles per piece cost a little balance (a piece is at most one tile longer
    // than the average) and save the round trip through the scratch, which is the longer of the two at these sizes.
    const long long aligned_share = ((ntiles + grid - 1) / grid) * p.kchunks;
    p.tile_aligned = grid % sm_count() == 0 && ntiles >= grid && aligned_share <= cap;
    if (p.tile_aligned) share_max = (int)aligned_share;
    const long long items = p.tile_aligned ? ntiles : (long long)p.units;
    p.piece_q = (int)(items / grid);
    p.piece_r = (int)(items % grid);
    const size_t smem = (size_t)share_max * UNIT_BYTES + (size_t)M * p.act_row_bytes + (size_t)MAX_TILES * 16 * TOK * 4 + TOK * 4;
    if (smem > 227 * 1024 - 64) return BITNET_A48_ERR_UNSUPPORTED;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = prefetch_ok ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int dev = 0;
    A48_CUDA_TRY(cudaGetDevice(&dev));
    // one token: the dp4a form with twelve warps; more: the mma.sync form with eight (the attribute is per device)
    if (M == 1) {
        static size_t smem_set_dev[64] = {};
        size_t& smem_set = smem_set_dev[dev & 63];
        if (smem > smem_set) {
            A48_CUDA_TRY(cudaFuncSetAttribute(decode_kernel<WARPS_ONE, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)smem));
            smem_set = smem;
        }
        cfg.blockDim = dim3(32 * WARPS_ONE);
        A48_CUDA_TRY(cudaLaunchKernelEx(&cfg, decode_kernel<WARPS_ONE, true>, p, share_max));
    } else {
        static size_t smem_set_dev[64] = {};
        size_t& smem_set = smem_set_dev[dev & 63];
        if (smem > smem_set) {
            A48_CUDA_TRY(cudaFuncSetAttribute(decode_kernel<WARPS_MANY, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)smem));
            smem_set = smem;
        }
        cfg.blockDim = dim3(32 * WARPS_MANY);
        A48_CUDA_TRY(cudaLaunchKernelEx(&cfg, decode_kernel<WARPS_MANY, false>, p, share_max));
    }
    for (int j = 0; j < count; ++j) wv[j]->decode_prefetch_ok = true;
    return BITNET_A48_OK;
}

bitnet_a48_status a48_read_decode_status(unsigned int words_host[4]) {
    A48_CUDA_TRY(cudaMemcpyFromSymbol(words_host, g_decode_status, sizeof(unsigned int) * 4));
    const unsigned int zero[4] = {0, 0, 0, 0};
    A48_CUDA_TRY(cudaMemcpyToSymbol(g_decode_status, zero, sizeof(zero)));
    return BITNET_A48_OK;
}


// ---------------------------------------------------------------------------------------------------------------
// Decode without any allocation: the scratch of the decode kernel lives in the library image.
namespace {

constexpr int kStaticMaxN = 16384;  // output features the built-in scratch covers
// 64-bit fix-up words, one per (row, token): 1 MiB that every device loading the library holds until exit.
static __device__ __align__(256) unsigned long long g_static_scratch[(size_t)kStaticMaxN * TOK];
constexpr int kMaxDevices = 64;
void* g_static_scratch_ptr[kMaxDevices];  // device address of the array, per device, filled on first use

}  // namespace

extern "C" bitnet_a48_status bitnet_a48_linear_decode_static(const bitnet_a48_weight* w, const int8_t* codes_dev,
                                                             const float* scale_dev, int M, float* Y_dev,
                                                             void* stream) {
    if (!w || !codes_dev || !scale_dev || !Y_dev) return BITNET_A48_ERR_INVALID_ARG;
    if (M <= 0) return BITNET_A48_ERR_SHAPE;
    if (!a48_aligned16(codes_dev) || !a48_aligned16(scale_dev) || !a48_aligned16(Y_dev)) return BITNET_A48_ERR_ALIGNMENT;
    if (w->N > kStaticMaxN) return BITNET_A48_ERR_LIMIT;
    if (!a48_decode_supported(w, M)) return BITNET_A48_ERR_UNSUPPORTED;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        return BITNET_A48_ERR_CUDA;
    }
    if (!g_static_scratch_ptr[dev]) {
        // In host code the array's name is only a handle; kernels need the address the runtime gives for it.
        void* ptr = nullptr;
        A48_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
        g_static_scratch_ptr[dev] = ptr;
    }
    const size_t bytes = a48_decode_workspace_bytes(w, M);  // <= sizeof(g_static_scratch) because N <= kStaticMaxN
    cudaStream_t st = (cudaStream_t)stream;
    // the array keeps whatever the last call left (zeros, unless a call was cut short): start from zeros
    A48_CUDA_TRY(cudaMemsetAsync(g_static_scratch_ptr[dev], 0, bytes, st));
    return a48_launch_decode(w, codes_dev, scale_dev, M, Y_dev, nullptr, g_static_scratch_ptr[dev], bytes, st);
}
