// Causal softmax attention for prefill on the fifth-generation tensor cores (the block glue around the BitLinears,
// Section 2.1).
//
// Attention is two contractions per head, S = Q K^T and O = P V.  The block's tolerance against the float64 oracle
// does not allow plain bf16 or tf32 operands: a score that is 1e-3 off moves its probability by as much, and the
// quantisers that follow the attention turn a 1e-5 difference into flipped codes.  So every operand is split into
// three bf16 numbers, x = x0 + x1 + x2 with x0 = bf16(x), x1 = bf16(x - x0), x2 = bf16(x - x0 - x1) (the subtractions
// are exact, the three carry the 24 significant bits of x), and every product is the six MMAs x_i * y_j with
// i + j <= 2.  What is dropped is below 2^-24 of a product.  The tensor core adds to its accumulator with less care
// than an fp32 add (measured with mma.sync: truncation), so of the six MMAs of a step the five corrections (2^-8 and
// less of the leading product) are issued first, for all steps of a tile, and the leading products last: the
// truncation acts on small sums until the few leading MMAs come.  Measured against a float64 attention this is as
// accurate as separate accumulators for leading and correction terms, and closer than a sequential fp32 evaluation.
// The running output lives in registers: every key tile is contracted into a fresh accumulator and added in fp32.
//
// Kernels.  attn_split_kernel writes the parts of the queries of the call and of the keys of positions
// [0, pos0 + T) as bf16 arrays [part][B * heads][rows padded to a tile][head dim padded to 64 or 128];
// attn_split_vt_kernel writes the parts of the values transposed, [part][B * heads][head dim][keys], so that the
// shared-memory operands of both contractions are K-major.  attn_tc_kernel: one CTA per (128 queries, head,
// sequence), 1 per SM, the tiles with the most keys first.
//   warp 9, two lanes: tensor copies (TMA, 128-byte swizzle) of key tiles (64 keys) and value tiles, two buffers
//     each: K(t+2) is requested when S(t) has completed, V(t+2) when O(t) has.
//   warp 8, one lane: all tcgen05.mma, both with the A operand in tensor memory: S(t) = Q K(t)^T (the query parts are
//     stored to tensor memory once per CTA) into one of two score buffers; O(t) = P(t) V(t) with the parts of P that
//     the softmax threads stored over the scores.  The pipe runs S(0), S(1), O(0), S(2), O(1), ...: the scores of
//     the next tile are ready while the softmax of this one is taken.  Tensor memory: 192 columns of query parts,
//     2 x 96 of scores / P, 128 of output = all 512.  Measured, the MMAs set the pace: a 128 x 64 x 16 MMA of S
//     takes about 49 clocks where its arithmetic is 32, a 128 x 128 x 16 MMA of O 71 (64).
//   warps 0-7: two threads per query row (tensor-memory lane), each with half of the tile's keys and half of the head
//     dimension: read S(t), exchange the row maximum through shared memory, exponentials, split P into parts, store
//     them to tensor memory, add O(t-1) (which ran meanwhile) to the running output and rescale it.
// Every wait is bounded; a wait that gives up records itself (bitnet_a48_kernel_status) and lets every later wait of
// the CTA fall through, so the kernel ends by itself; the copy lanes then wait for their copies in flight.
#include <cuda.h>
#include <cuda_bf16.h>

#include "internal.h"

namespace {

constexpr int TQ = 128;  // queries per CTA = MMA M = tensor-memory lanes
constexpr int TK = 64;   // keys per tile: one 128-byte swizzle row of bf16
constexpr int NS = 3;    // parts per operand
constexpr int SOFTMAX_WARPS = 8, MMA_WARP = SOFTMAX_WARPS, TMA_WARP = SOFTMAX_WARPS + 1, THREADS = 32 * (SOFTMAX_WARPS + 2);
constexpr int TMEM_COLS = 512;
// Tensor-memory columns: the three parts of the 128 queries (two elements per column), two score buffers (64 columns
// of scores; the three parts of P, two keys per column, are stored over them once every thread has read its scores),
// the accumulator of O(t).
constexpr int COL_Q = 0, COL_SP = 192, SP_BUF = 96, COL_O = COL_SP + 2 * SP_BUF;
constexpr unsigned long long kWaitClocks = 4000000000ull;  // ~2 s at 2 GHz
constexpr unsigned long long kDrainClocks = 400000000ull;  // what the issuer grants its copies in flight when it gives up

__device__ unsigned int g_attn_status[4];

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
// Bounded wait.  Once any wait of the CTA has given up (*abort_flag), every wait returns at once.
__device__ __noinline__ void mbar_wait_slow(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, uint32_t id, uint32_t iter,
                                            unsigned long long limit) {
    const unsigned long long t0 = clock64();
    uint32_t spins = 0;
    while (!mbar_try(bar, parity)) {
        if ((++spins & 255u) == 0) {
            if (*abort_flag && limit == kWaitClocks) return;
            if (clock64() - t0 > limit) {
                *abort_flag = 1;
                if (atomicCAS(&g_attn_status[0], 0u, (unsigned)BITNET_A48_ERR_TIMEOUT) == 0u) {
                    g_attn_status[1] = id;
                    g_attn_status[2] = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
                    g_attn_status[3] = iter;
                }
                return;
            }
        }
    }
}
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, uint32_t id, uint32_t iter) {
    if (mbar_try(bar, parity)) return;
    if (*abort_flag) return;
    mbar_wait_slow(bar, parity, abort_flag, id, iter, kWaitClocks);
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem desc], bf16 operands, fp32 accumulators
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Shared-memory matrix descriptor of a K-major operand tile whose rows are 128 bytes (64 bf16), laid down by TMA with
// the 128-byte swizzle: 8-row groups are 1024 bytes apart.  16 elements further along K = +32 bytes = +2 in the
// address field.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3ffffu) >> 4);
    d |= (uint64_t)(1024u >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// kind::f16 instruction descriptor: bf16 x bf16 -> f32, both operands K-major, M x N tile.
__host__ __device__ constexpr uint32_t idesc_bf16(int m, int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
          "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void softmax_warps_sync() { asm volatile("bar.sync 1, %0;" ::"n"(32 * SOFTMAX_WARPS) : "memory"); }

// a pair of floats: the bf16x2 word of their leading parts (first value in the low half); x and y keep the rest
__device__ __forceinline__ uint32_t take_part(float& x, float& y) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
    const uint32_t w = *reinterpret_cast<const uint32_t*>(&h);
    x -= __uint_as_float(w << 16);
    y -= __uint_as_float(w & 0xffff0000u);
    return w;
}
// 2^x, two units in the last place at most; 2^-inf = 0
__device__ __forceinline__ float exp2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// four floats -> the two bf16x2 words of each part
__device__ __forceinline__ void split4(float (&v)[4], uint2 (&w)[NS]) {
#pragma unroll
    for (int a = 0; a < NS; ++a) {
        w[a].x = take_part(v[0], v[1]);
        w[a].y = take_part(v[2], v[3]);
    }
}
// four consecutive floats of a row of hd, zero past the row's end
__device__ __forceinline__ void load4(const float* __restrict__ row, int c, int hd, bool vec, float (&v)[4]) {
    if (vec && c + 3 < hd) {
        const float4 f = *reinterpret_cast<const float4*>(row + c);
        v[0] = f.x, v[1] = f.y, v[2] = f.z, v[3] = f.w;
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = c + j < hd ? row[c + j] : 0.f;
    }
}

// src rows of hd floats -> NS parts (part_stride elements apart) of rows of HDP bf16, zero past hd and for rows >=
// rows_valid.  mode 0: queries, src = q [B*T][nh*hd], row (b, h, r) = token r of sequence b; mode 1: cache
// [B][nh][cap][hd].  grid (rows_pad / 64, nh, B): a block takes 64 rows of one head, a thread four head dims at a time.
template <int HDP>
__global__ void __launch_bounds__(256) attn_split_kernel(const float* __restrict__ src, int mode, int hd, int rows_valid, int rows_pad,
                                                         int T, int cap, __nv_bfloat16* __restrict__ parts, size_t part_stride) {
    a48_pdl_prologue();
    constexpr int QUADS = HDP / 4, ROWS = 256 / QUADS;  // threads per row, rows per pass
    const int nh = gridDim.y, h = blockIdx.y, b = blockIdx.z;
    const size_t bh = (size_t)b * nh + h;
    const int c = (threadIdx.x % QUADS) * 4;
    const float* base = mode == 0 ? src + (size_t)b * T * nh * hd + (size_t)h * hd : src + bh * cap * hd;
    const size_t pitch = mode == 0 ? (size_t)nh * hd : (size_t)hd;
    const bool vec = (hd & 3) == 0 && (reinterpret_cast<uintptr_t>(src) & 15) == 0;
    for (int r = blockIdx.x * 64 + threadIdx.x / QUADS; r < blockIdx.x * 64 + 64; r += ROWS) {
        float v[4] = {0.f, 0.f, 0.f, 0.f};
        if (r < rows_valid && c < hd) load4(base + r * pitch, c, hd, vec, v);
        uint2 w[NS];
        split4(v, w);
        const size_t o = (bh * rows_pad + r) * HDP + c;
#pragma unroll
        for (int a = 0; a < NS; ++a) *reinterpret_cast<uint2*>(parts + a * part_stride + o) = w[a];
    }
}

// The values of one head and 64 positions, transposed: vcache [B*nh][cap][hd] -> parts [part][B*nh][HDP][k_pad].
// grid (k_pad / 64, nh, B); a tile of 64 keys goes through shared memory.
template <int HDP>
__global__ void __launch_bounds__(256) attn_split_vt_kernel(const float* __restrict__ vcache, int hd, int n_keys, int k_pad, int cap,
                                                            __nv_bfloat16* __restrict__ parts, size_t part_stride) {
    constexpr int LD = HDP + 1;
    __shared__ float vt_tile[TK * LD];  // [64 keys][HDP + 1]
    a48_pdl_prologue();
    const int k0 = blockIdx.x * TK;
    const size_t bh = (size_t)blockIdx.z * gridDim.y + blockIdx.y;
    const bool vec = (hd & 3) == 0 && (reinterpret_cast<uintptr_t>(vcache) & 15) == 0;
    for (int i = threadIdx.x; i < TK * (HDP / 4); i += 256) {
        const int key = i / (HDP / 4), d = (i % (HDP / 4)) * 4;
        float v[4] = {0.f, 0.f, 0.f, 0.f};
        if (k0 + key < n_keys && d < hd) load4(vcache + (bh * cap + k0 + key) * hd, d, hd, vec, v);
#pragma unroll
        for (int j = 0; j < 4; ++j) vt_tile[key * LD + d + j] = v[j];
    }
    __syncthreads();
    for (int i = threadIdx.x; i < HDP * (TK / 4); i += 256) {  // a thread: one head dim, four keys
        const int d = i / (TK / 4), kq = (i % (TK / 4)) * 4;
        float v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = vt_tile[(kq + j) * LD + d];
        uint2 w[NS];
        split4(v, w);
        const size_t o = (bh * HDP + d) * (size_t)k_pad + k0 + kq;
#pragma unroll
        for (int a = 0; a < NS; ++a) *reinterpret_cast<uint2*>(parts + a * part_stride + o) = w[a];
    }
}

struct AttnParams {
    int T, t_pad, n_keys, k_pad, nh, hd, pos0, bh_total;
    float scale;
    const __nv_bfloat16* q_parts;  // [part][B * heads][t_pad][HDP]
    size_t q_part;                 // elements per part
    float* out;
};

template <int HDP>
struct AttnCfg {
    static constexpr int KB = HDP / 64;  // 128-byte blocks per key row
    static constexpr int K_BLOCK = TK * 128, V_PART = HDP * 128;
    static constexpr int K_BYTES = NS * KB * K_BLOCK, V_BYTES = NS * V_PART;  // one key tile, one value tile
    static constexpr int SMEM_BYTES = 2 * K_BYTES + 2 * V_BYTES + 1024 /*alignment slack*/ + 4096 /*barriers, row maxima*/;
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
    static_assert(NS * HDP / 2 <= COL_SP && TK <= SP_BUF && NS * TK / 2 <= SP_BUF && COL_O + HDP <= TMEM_COLS, "tensor memory budget");
};

// barrier ids reported through the status words
enum { WAIT_Q = 20, WAIT_K = 21, WAIT_V = 22, WAIT_S = 23, WAIT_O = 24, WAIT_P = 25, WAIT_DRAIN = 26 };

template <int HDP>
__global__ void __launch_bounds__(THREADS, 1)
    attn_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, const AttnParams p) {
    using C = AttnCfg<HDP>;
    constexpr int KB = C::KB, OD = HDP / 2;  // OD: head dims per softmax thread
    constexpr int QW = HDP / 4;              // tensor-memory columns of a thread's share of one query part
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* ctrl = smem + 2 * C::K_BYTES + 2 * C::V_BYTES;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ctrl + 96);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(ctrl + 100);
    float* row_max = reinterpret_cast<float*>(ctrl + 1024);  // [tile parity][half][row]
    const uint32_t sk = smem_u32(smem), sv = sk + 2 * C::K_BYTES;
    // barriers: q | k[2] | v[2] | s[2] | o | p
    const uint32_t bar_q = smem_u32(ctrl), bar_k = bar_q + 8, bar_v = bar_q + 24, bar_s = bar_q + 40, bar_o = bar_q + 56, bar_p = bar_q + 64;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        mbar_init(bar_q, 32 * SOFTMAX_WARPS);
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar_k + 8 * i, 1);
            mbar_init(bar_v + 8 * i, 1);
            mbar_init(bar_s + 8 * i, 1);
        }
        mbar_init(bar_o, 1);
        mbar_init(bar_p, 32 * SOFTMAX_WARPS);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == MMA_WARP) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    a48_pdl_prologue();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int q0 = ((int)gridDim.x - 1 - (int)blockIdx.x) * TQ;  // the tiles with the most keys first
    const int h = blockIdx.y, b = blockIdx.z, bh = b * p.nh + h;
    const int keys_needed = min(p.n_keys, p.pos0 + min(q0 + TQ, p.T));  // causal: nothing beyond the last query's position
    const int n_tiles = (keys_needed + TK - 1) / TK;

    if (warp == TMA_WARP) {
        // ------------------------------------------------------------- tensor copies
        // Two buffers for keys, two for values.  Lane 0 requests K(t+2) when S(t) has completed, lane 1 requests V(t+2)
        // when O(t) has: two lanes, so that a key tile never waits behind a value tile's turn.
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_k)) : "memory");
            auto load_k = [&](int t) {
                const uint32_t bar = bar_k + 8 * (t & 1), dst = sk + (t & 1) * C::K_BYTES;
                mbar_expect_tx(bar, C::K_BYTES);
#pragma unroll
                for (int a = 0; a < NS; ++a)
#pragma unroll
                    for (int kb = 0; kb < KB; ++kb)
                        tma_load_2d(dst + (a * KB + kb) * C::K_BLOCK, &tm_k, kb * 64, (a * p.bh_total + bh) * p.k_pad + t * TK, bar);
            };
            load_k(0);
            if (n_tiles > 1) load_k(1);
            int issued = min(n_tiles, 2);
            for (; issued < n_tiles; ++issued) {
                const int t = issued - 2;
                mbar_wait(bar_s + 8 * (t & 1), (t >> 1) & 1, abort_flag, WAIT_S, t);  // S(t) has read its key tile
                if (*abort_flag) break;
                load_k(issued);
            }
            if (*abort_flag)  // a wait gave up: the copies in flight must land before the shared memory goes back
                for (int t = max(issued - 2, 0); t < issued; ++t)
                    mbar_wait_slow(bar_k + 8 * (t & 1), (t >> 1) & 1, abort_flag, WAIT_DRAIN, t & 1, kDrainClocks);
        } else if (lane == 1) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_v)) : "memory");
            auto load_v = [&](int t) {
                const uint32_t bar = bar_v + 8 * (t & 1), dst = sv + (t & 1) * C::V_BYTES;
                mbar_expect_tx(bar, C::V_BYTES);
#pragma unroll
                for (int a = 0; a < NS; ++a) tma_load_2d(dst + a * C::V_PART, &tm_v, t * TK, (a * p.bh_total + bh) * HDP, bar);
            };
            load_v(0);
            if (n_tiles > 1) load_v(1);
            int issued = min(n_tiles, 2);
            for (; issued < n_tiles; ++issued) {
                const int t = issued - 2;
                mbar_wait(bar_o, t & 1, abort_flag, WAIT_O, t);  // O(t) has read its value tile
                if (*abort_flag) break;
                load_v(issued);
            }
            if (*abort_flag)
                for (int t = max(issued - 2, 0); t < issued; ++t)
                    mbar_wait_slow(bar_v + 8 * (t & 1), (t >> 1) & 1, abort_flag, WAIT_DRAIN, 2 + (t & 1), kDrainClocks);
        }
        __syncwarp();
    } else if (warp == MMA_WARP) {
        if (lane == 0) {
            // ------------------------------------------------------------- MMAs
            // Both contractions take their A operand from tensor memory (the query parts, stored there once by the
            // softmax threads; the parts of P) and their B operand from shared memory.  Per product the five
            // corrections are issued first and the leading product last, so that the truncating accumulate of the
            // tensor core acts on small sums until the few leading MMAs come: one accumulator then is as accurate
            // as separate ones for the leading and the correction terms (measured against float64).
            constexpr uint32_t idesc_s = idesc_bf16(TQ, TK), idesc_o = idesc_bf16(TQ, HDP);
            const uint32_t t_q = tmem_base + COL_Q, t_o = tmem_base + COL_O;
            // the correction products, smallest first: (part of A, part of B)
            constexpr int CA[5] = {0, 1, 2, 0, 1}, CB[5] = {2, 1, 0, 1, 0};
            // S(t) = Q K(t)^T into score buffer t % 2: HDP / 16 steps of six MMAs
            auto issue_s = [&](int t) {
                mbar_wait(bar_k + 8 * (t & 1), (t >> 1) & 1, abort_flag, WAIT_K, t);
                tc_fence_after();
                const uint32_t t_s = tmem_base + COL_SP + (t & 1) * SP_BUF, kbuf = sk + (t & 1) * C::K_BYTES;
#pragma unroll
                for (int pass = 0; pass < 2; ++pass)
#pragma unroll
                    for (int ks = 0; ks < HDP / 16; ++ks) {
                        uint64_t kd[NS];
#pragma unroll
                        for (int a = 0; a < NS; ++a) kd[a] = smem_desc_sw128(kbuf + (a * KB + ks / 4) * C::K_BLOCK) + 2 * (ks % 4);
                        if (pass == 0) {
#pragma unroll
                            for (int c = 0; c < 5; ++c) mma_ts(t_s, t_q + CA[c] * (HDP / 2) + 8 * ks, kd[CB[c]], idesc_s, (ks | c) != 0);
                        } else {
                            mma_ts(t_s, t_q + 8 * ks, kd[0], idesc_s, 1);
                        }
                    }
                tc_commit(bar_s + 8 * (t & 1));
            };
            mbar_wait(bar_q, 0, abort_flag, WAIT_Q, 0);
            issue_s(0);
            if (n_tiles > 1) issue_s(1);
            for (int t = 0; t < n_tiles; ++t) {
                const uint32_t par = t & 1;
                mbar_wait(bar_p, par, abort_flag, WAIT_P, t);  // P(t) is stored and O(t-1) has been read
                mbar_wait(bar_v + 8 * par, (t >> 1) & 1, abort_flag, WAIT_V, t);
                tc_fence_after();
                // ---- O(t) = P(t) V(t): four steps of 16 keys; P(t) sits where S(t) was
                const uint32_t t_p = tmem_base + COL_SP + par * SP_BUF, vbuf = sv + par * C::V_BYTES;
#pragma unroll
                for (int pass = 0; pass < 2; ++pass)
#pragma unroll
                    for (int j = 0; j < TK / 16; ++j) {
                        uint64_t vd[NS];
#pragma unroll
                        for (int a = 0; a < NS; ++a) vd[a] = smem_desc_sw128(vbuf + a * C::V_PART) + 2 * j;
                        if (pass == 0) {
#pragma unroll
                            for (int c = 0; c < 5; ++c) mma_ts(t_o, t_p + CA[c] * (TK / 2) + 8 * j, vd[CB[c]], idesc_o, (j | c) != 0);
                        } else {
                            mma_ts(t_o, t_p + 8 * j, vd[0], idesc_o, 1);
                        }
                    }
                tc_commit(bar_o);
                if (t + 2 < n_tiles) issue_s(t + 2);  // behind O(t) on the pipe, so P(t) is not overwritten early
            }
            mbar_wait(bar_o, (n_tiles - 1) & 1, abort_flag, WAIT_O, n_tiles);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------- softmax and running output
        const int quad = warp & 3, half = warp >> 2;
        const int row = quad * 32 + lane, q = q0 + row;
        const uint32_t lanes = tmem_base + ((uint32_t)(quad * 32) << 16);
        // ---- this thread's half of its query row, part by part, into tensor memory (two elements per column)
        {
            const __nv_bfloat16* src = p.q_parts + ((size_t)bh * p.t_pad + q) * HDP + half * OD;
#pragma unroll
            for (int a = 0; a < NS; ++a) {
                uint32_t w[QW];
                const uint4* s4 = reinterpret_cast<const uint4*>(src + a * p.q_part);
#pragma unroll
                for (int i = 0; i < QW / 4; ++i) {
                    const uint4 v = __ldg(s4 + i);
                    w[4 * i] = v.x, w[4 * i + 1] = v.y, w[4 * i + 2] = v.z, w[4 * i + 3] = v.w;
                }
                if constexpr (QW == 32) tmem_st32(lanes + COL_Q + a * (HDP / 2) + half * QW, w);
                else tmem_st16(lanes + COL_Q + a * (HDP / 2) + half * QW, w);
            }
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            tc_fence_before();
            mbar_arrive(bar_q);
        }
        const int lim = min(p.pos0 + q, p.n_keys - 1);  // the last key this query sees
        constexpr float kLog2e = 1.4426950408889634f;
        float o[OD];
#pragma unroll
        for (int d = 0; d < OD; ++d) o[d] = 0.f;
        float m_run = -INFINITY, l_run = 0.f;
        // o += O(t), this thread's head dims
        auto add_tile = [&](int t) {
            mbar_wait(bar_o, t & 1, abort_flag, WAIT_O, t);
            tc_fence_after();
#pragma unroll
            for (int c0 = 0; c0 < OD; c0 += 32) {
                uint32_t acc[32];
                tmem_ld32(lanes + COL_O + half * OD + c0, acc);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int i = 0; i < 32; ++i) o[c0 + i] += __uint_as_float(acc[i]);
            }
        };
        for (int t = 0; t < n_tiles; ++t) {
            const uint32_t par = t & 1;
            const uint32_t buf = lanes + COL_SP + par * SP_BUF;
            float s[32];
            float mx = -INFINITY;
            mbar_wait(bar_s + 8 * par, (t >> 1) & 1, abort_flag, WAIT_S, t);
            tc_fence_after();
            {
                uint32_t acc[32];
                tmem_ld32(buf + 32 * half, acc);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                const int key0 = t * TK + 32 * half;
                if (t * TK + TK - 1 <= min(p.pos0 + q0, p.n_keys - 1)) {  // every query of the CTA sees the whole tile
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        s[i] = __uint_as_float(acc[i]) * p.scale;
                        mx = fmaxf(mx, s[i]);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        s[i] = key0 + i <= lim ? __uint_as_float(acc[i]) * p.scale : -INFINITY;
                        mx = fmaxf(mx, s[i]);
                    }
                }
            }
            row_max[(par * 2 + half) * TQ + row] = mx;
            softmax_warps_sync();  // (also: every thread has read its scores, so P may go where they were)
            mx = fmaxf(mx, row_max[(par * 2 + (half ^ 1)) * TQ + row]);
            // exp(s - m) as 2^((s - m) log2 e): the difference is formed first, so the constant's rounding only
            // touches the probability relatively.  Key 0 is visible to every query, so m_new is finite.
            const float m_new = fmaxf(m_run, mx);
            const float corr = exp2_approx((m_run - m_new) * kLog2e);
            m_run = m_new;
            float sum = 0.f;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                s[i] = exp2_approx((s[i] - m_new) * kLog2e);
                sum += s[i];
            }
            l_run = l_run * corr + sum;
#pragma unroll
            for (int a = 0; a < NS; ++a) {
                uint32_t w[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) w[i] = take_part(s[2 * i], s[2 * i + 1]);
                tmem_st16(buf + a * (TK / 2) + 16 * half, w);
            }
            if (t > 0) add_tile(t - 1);  // O(t-1) ran while the exponentials above were taken
            if (__any_sync(0xffffffffu, corr != 1.f)) {  // (the maximum settles after a few tiles)
#pragma unroll
                for (int d = 0; d < OD; ++d) o[d] *= corr;
            }
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            tc_fence_before();
            mbar_arrive(bar_p);  // P(t) is in place and the output accumulator is free for O(t)
        }
        add_tile(n_tiles - 1);
        // ---- out = O / l (the two halves of a row add their sums)
        const int lb = n_tiles & 1;  // the buffer the last tile did not use
        row_max[(lb * 2 + half) * TQ + row] = l_run;
        softmax_warps_sync();
        const float inv = 1.f / (l_run + row_max[(lb * 2 + (half ^ 1)) * TQ + row]);
        if (q < p.T) {
            float* dst = p.out + ((size_t)b * p.T + q) * ((size_t)p.nh * p.hd) + (size_t)h * p.hd + half * OD;
            const int valid = p.hd - half * OD;  // head dims of this half that exist
            if ((p.hd & 3) == 0) {
#pragma unroll
                for (int d = 0; d < OD; d += 4)
                    if (d < valid) *reinterpret_cast<float4*>(dst + d) = make_float4(o[d] * inv, o[d + 1] * inv, o[d + 2] * inv, o[d + 3] * inv);
            } else {
#pragma unroll
                for (int d = 0; d < OD; ++d)
                    if (d < valid) dst[d] = o[d] * inv;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == MMA_WARP) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// bf16 matrix [rows, cols] row-major, box = 64 columns (128 bytes) x box_rows, 128-byte swizzle.
bool make_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int pick_hdp(int hd) { return hd <= 64 ? 64 : 128; }

struct Extents {
    int hdp, t_pad, k_pad;
    size_t q_part, kv_part;  // elements per part
};
Extents extents(int B, int nh, int hd, int T, int n_keys) {
    Extents e;
    e.hdp = pick_hdp(hd);
    e.t_pad = (T + TQ - 1) / TQ * TQ;
    e.k_pad = (n_keys + TK - 1) / TK * TK;
    e.q_part = (size_t)B * nh * e.t_pad * e.hdp;
    e.kv_part = (size_t)B * nh * e.k_pad * e.hdp;
    return e;
}

template <int HDP>
bitnet_a48_status launch_attn(const CUtensorMap& mk, const CUtensorMap& mv, const AttnParams& p, int B, cudaStream_t st) {
    using C = AttnCfg<HDP>;
    A48_CUDA_TRY(cudaFuncSetAttribute(attn_tc_kernel<HDP>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
    A48_CUDA_TRY(a48_launch_pdl(attn_tc_kernel<HDP>, dim3(p.t_pad / TQ, p.nh, B), dim3(THREADS), (size_t)C::SMEM_BYTES, st, mk, mv, p));
    return BITNET_A48_OK;
}

}  // namespace

bool a48_attn_tc_supported(int hd) { return hd >= 1 && hd <= 128; }

// Scratch for the split operands: the parts of the queries (rows padded to 128), of the keys and of the transposed
// values (positions padded to 64).
size_t a48_attn_tc_workspace_bytes(int B, int nh, int hd, int T, int n_keys) {
    const Extents e = extents(B, nh, hd, T, n_keys);
    return NS * 2 * (e.q_part + 2 * e.kv_part);
}

// q [B*T][nh*hd] (already rotated); kcache / vcache fp32 [B][nh][cap][hd] holding positions [0, pos0 + T).
bitnet_a48_status a48_launch_attn_tc(const float* q, const float* kcache, const float* vcache, int B, int T, int nh, int hd, int pos0,
                                     int cap, float* out, void* ws, cudaStream_t st) {
    if (!a48_attn_tc_supported(hd) || B > 65535 || nh > 65535) return BITNET_A48_ERR_UNSUPPORTED;
    const int n_keys = pos0 + T;
    const Extents e = extents(B, nh, hd, T, n_keys);
    const size_t bh = (size_t)B * nh;
    if (NS * bh * (size_t)(e.t_pad > e.k_pad ? e.t_pad : e.k_pad) >= (1ull << 31) || NS * bh * e.hdp >= (1ull << 31))
        return BITNET_A48_ERR_UNSUPPORTED;  // tensor-copy coordinates are 32-bit
    __nv_bfloat16* qs = static_cast<__nv_bfloat16*>(ws);
    __nv_bfloat16* ks = qs + NS * e.q_part;
    __nv_bfloat16* vs = ks + NS * e.kv_part;
    CUtensorMap mk, mv;
    if (!make_map(&mk, ks, NS * bh * e.k_pad, e.hdp, TK) || !make_map(&mv, vs, NS * bh * e.hdp, e.k_pad, e.hdp)) return BITNET_A48_ERR_CUDA;
    const dim3 block(256), grid_q(e.t_pad / 64, nh, B), grid_k(e.k_pad / 64, nh, B), grid_v(e.k_pad / TK, nh, B);
    if (e.hdp == 64) {
        A48_CUDA_TRY(a48_launch_pdl(attn_split_kernel<64>, grid_q, block, 0, st, q, 0, hd, T, e.t_pad, T, cap, qs, e.q_part));
        A48_CUDA_TRY(a48_launch_pdl(attn_split_kernel<64>, grid_k, block, 0, st, kcache, 1, hd, n_keys, e.k_pad, T, cap, ks, e.kv_part));
        A48_CUDA_TRY(a48_launch_pdl(attn_split_vt_kernel<64>, grid_v, block, 0, st, vcache, hd, n_keys, e.k_pad, cap, vs, e.kv_part));
    } else {
        A48_CUDA_TRY(a48_launch_pdl(attn_split_kernel<128>, grid_q, block, 0, st, q, 0, hd, T, e.t_pad, T, cap, qs, e.q_part));
        A48_CUDA_TRY(a48_launch_pdl(attn_split_kernel<128>, grid_k, block, 0, st, kcache, 1, hd, n_keys, e.k_pad, T, cap, ks, e.kv_part));
        A48_CUDA_TRY(a48_launch_pdl(attn_split_vt_kernel<128>, grid_v, block, 0, st, vcache, hd, n_keys, e.k_pad, cap, vs, e.kv_part));
    }
    AttnParams p;
    p.T = T;
    p.t_pad = e.t_pad;
    p.n_keys = n_keys;
    p.k_pad = e.k_pad;
    p.nh = nh;
    p.hd = hd;
    p.pos0 = pos0;
    p.bh_total = (int)bh;
    p.scale = 1.f / sqrtf((float)hd);
    p.q_parts = qs;
    p.q_part = e.q_part;
    p.out = out;
    return e.hdp == 64 ? launch_attn<64>(mk, mv, p, B, st) : launch_attn<128>(mk, mv, p, B, st);
}

bitnet_a48_status a48_read_attn_status(unsigned int words_host[4]) {
    A48_CUDA_TRY(cudaMemcpyFromSymbol(words_host, g_attn_status, sizeof(unsigned int) * 4));
    const unsigned int zero[4] = {0, 0, 0, 0};
    A48_CUDA_TRY(cudaMemcpyToSymbol(g_attn_status, zero, sizeof(zero)));
    return BITNET_A48_OK;
}
