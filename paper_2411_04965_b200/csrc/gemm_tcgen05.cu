// Prefill BitLinear contraction (Eq. 1 / Eq. 6) on the 5th-generation tensor cores:
// tcgen05.mma kind::i8 (s8 x s8 -> s32) with the accumulators in tensor memory.
//
// Orientation.  The MMA computes D[128 x 192] = A[128 x K] * B[K x 192] with
//   A = a tile of 128 weight rows (output features n), expanded to int8 codes,
//   B = a tile of 192 tokens of activation codes (row-major [M,K] is exactly the
//       K-major operand layout the MMA wants),
// so the accumulator holds Y^T: TMEM lane = output feature, TMEM column = token.
// The epilogue thread that owns lane n writes Y[m, n] for consecutive m, which
// makes every warp store a contiguous 128-byte run of one output row.
//
// Two variants share the pipeline:
//   TS (default): the 2-bit weights are staged into shared memory by a bulk
//       copy on the same pipeline stage as the activation tile (8 KB per 256
//       channels), widened to int8 in registers by eight expander warps with a
//       byte-permute lookup, and written into tensor memory with tcgen05.st; the
//       MMA takes A from tensor memory.  Only the packed form touches shared
//       memory, whose bandwidth is left to the activation operand.
//   SS: both operands come from shared memory via TMA; A is a pre-expanded int8
//       copy of the weights (BITNET_A48_LAYOUT_I8).  Comparison / bring-up variant.
//
// A pipeline stage ("unit") covers 256 channels for TS (two 128-byte swizzle
// rows of the activation tile and 8 KB of packed weights): one thread issues all
// MMAs, and what it pays per stage (one barrier wait, one commit, the loop) is
// spread over eight MMAs instead of four.  Tensor memory (512 columns) holds two
// 192-column accumulators, so the epilogue of one tile drains while the MMAs of
// the next tile run, and two 64-column slots of the expanded weight operand.
//
// Barriers per stage s: full[s] (TMA bytes landed), empty[s] (the MMAs that read
// the stage have completed - one tcgen05.commit - and the expanders have read
// its packed weights).  The same commit frees the tensor-memory slot the stage's
// expanded weights sat in, so the expanders wait on empty[] of the stage two
// units back instead of on a barrier of their own.  afull[g]: slot g written.
//
// Warp roles (one persistent CTA per SM): warp 0 TMA producer, warp 1 MMA issuer
// and TMEM owner, warps 2-9 weight expanders (TS only; two groups of four, group
// g takes every second unit, unit it goes to slot it % slots), warps 10-17
// epilogue (two per tensor-memory lane quadrant, each draining half of the
// accumulator columns).  Every mbarrier wait is bounded; a wait that gives up
// records a status word and the CTA drains and exits without touching tensor
// memory again.
//
// A fourth form, gemm_pair_kernel further down, puts one 256-row tile on a pair of CTAs (cta_group::2).
// Three forms of this kernel:
//   - 192-token tiles (prefill): as described above.
//   - 64-token tiles (at most 64 tokens in the call): MMA N = 64, eight pipeline
//     stages, six slots for the expanded weights, activation box as high as the
//     call has tokens.
//   - split-K: with fewer tiles than SMs the channels of a tile are cut into up to
//     eight ranges, one CTA each; the CTAs of a tile form a thread-block cluster
//     and exchange their int32 partial sums through distributed shared memory
//     (stores into the owner's shared memory between two cluster barriers).
// One launch can walk the tiles of up to four weight matrices that share K and
// the activation codes (q/k/v, gate/up).
#include <cuda.h>

#include <algorithm>

#include "internal.h"

namespace {

constexpr int TILE_N = 128;  // weight rows per tile  (MMA M)
constexpr int TILE_M_WIDE = 192;   // tokens per tile (MMA N) of the prefill kernel
constexpr int TILE_M_SKINNY = 64;  // ... and of the kernel for at most 64 tokens
constexpr int TILE_M_TINY = 32;    // ... and of the same kernel for at most 32 tokens (half the token bytes per unit)
constexpr int TILE_M_MID = 128;    // ... and where 128-token tiles cover the call with as few tiles as 192-token ones
constexpr int BK = 128;      // channels per 128-byte swizzle row of int8
constexpr int UMMA_K = 32;   // channels per kind::i8 MMA
constexpr int ACC_BUFS = 2;
constexpr int TMEM_COLS = 512;
constexpr int A_TILE_BYTES = TILE_N * BK;
constexpr int W_PACKED_BYTES = TILE_N * BK / 4;  // 128 rows x 128 channels of 2-bit codes
constexpr int kMaxSplit = 8;  // CTAs that may share a tile's channels: the portable cluster size
constexpr unsigned long long kWaitClocks = 4000000000ull;  // ~2 s at 2 GHz

template <bool TS, int TM>
struct Cfg {
    static constexpr int TILE_M = TM;
    static constexpr int ACC_COLS = TM;
    static constexpr int B_TILE_BYTES = TM * BK;
    // Expander groups of four warps (TS).  A group spends about 740 clocks on a unit; at 64 tokens the kernel is
    // bound by the fill rate of shared memory (24 KB per unit and CTA), so two groups are enough there too.
    static constexpr int EXPAND_GROUPS = 2;
    static constexpr int EPI_SPLIT = TM >= 64 ? 2 : 1;  // epilogue warps per lane quadrant
    static constexpr int NUM_THREADS = 32 * (2 + 4 * EXPAND_GROUPS + 4 * EPI_SPLIT);
    static constexpr int EPI_COLS = TM / EPI_SPLIT;
    static_assert(EPI_COLS % 32 == 0, "the epilogue drains 32 columns at a time");
    static constexpr int KBU = TS ? 2 : 1;  // 128-channel blocks per pipeline stage
    // the narrow activation tile leaves room for a deeper ring: more weight bytes in flight per SM
    static constexpr int STAGES = TM <= TILE_M_SKINNY ? 8 : (TS ? 4 : 5);
    // Tensor-memory slots of the expanded weight operand, 64 columns each.  A slot is busy from the expanders'
    // store until the MMAs that read it have completed, a round trip of well over a thousand clocks whatever
    // the MMA's size; two slots leave that round trip exposed, the narrow accumulators make room for more.
    static constexpr int A_SLOTS = TM <= TILE_M_SKINNY ? 6 : 2;
    static_assert(A_SLOTS % EXPAND_GROUPS == 0, "unit it goes to group it % groups and to slot it % slots");
    static constexpr int STAGE_BYTES = KBU * (B_TILE_BYTES + (TS ? W_PACKED_BYTES : A_TILE_BYTES));
    static constexpr int A_SLOT_COLS = KBU * BK / 4;
    // a stage is released by the MMA commit and, for TS, by one lane of each expander warp of one group
    static constexpr int EMPTY_ARRIVALS = TS ? 5 : 1;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 1024 /*barriers*/;
    static_assert(ACC_BUFS * ACC_COLS + (TS ? A_SLOTS * A_SLOT_COLS : 0) <= TMEM_COLS, "tensor memory budget");
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
    static_assert(STAGES * STAGE_BYTES >= (TM + kMaxSplit) * TILE_N * 4, "split-K: ksplit slots of ceil(TM / ksplit) token rows");
    static_assert(STAGES > A_SLOTS, "the stage A_SLOTS units back must still be distinct");
};

__device__ unsigned int g_status[4];

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

// Bounded wait.  Returns false when the CTA is aborting or the wait ran out of
// time; in the latter case the first such event is recorded in g_status.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, uint32_t id,
                                            uint32_t iter) {
    const unsigned long long t0 = clock64();
    uint32_t spins = 0;
    while (true) {
        if (mbar_try(bar, parity)) return true;
        if ((++spins & 255u) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > kWaitClocks) {
                *abort_flag = 1;
                if (atomicCAS(&g_status[0], 0u, (unsigned)BITNET_A48_ERR_TIMEOUT) == 0u) {
                    g_status[1] = id;
                    g_status[2] = blockIdx.x;
                    g_status[3] = iter;
                }
                return false;
            }
        }
    }
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, uint32_t id,
                                          uint32_t iter) {
    if (mbar_try(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag, id, iter);
}

// True in exactly one lane of a converged warp (the same lane on every call).
__device__ __forceinline__ bool elect_one() {
    uint32_t pred = 0;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}

// Untiled bulk copy global -> shared; both addresses 16-byte aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// D[tmem] (+)= A[smem desc] * B[smem desc]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// D[tmem] += A[tmem] * B[smem desc given as two words]
__device__ __forceinline__ void mma_ts_acc(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi,
                                           uint32_t idesc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 d;\n\tsetp.eq.b32 p, 0, 0;\n\tmov.b64 d, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], d, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc)
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem desc]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Shared-memory matrix descriptor of a K-major operand tile whose rows are 128
// bytes, laid down by TMA with the 128-byte swizzle: 8-row groups are 1024 bytes
// apart (stride byte offset), the leading byte offset is unused for this layout.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3ffffu) >> 4);        // start address, bits [0,14)
    d |= (uint64_t)(1024u >> 4) << 32;              // stride byte offset, bits [32,46)
    d |= (uint64_t)1 << 46;                         // descriptor version for sm_100
    d |= (uint64_t)2 << 61;                         // layout type: 128-byte swizzle
    return d;
}

// kind::i8 instruction descriptor: s8 x s8 -> s32, both operands K-major, M x N tile.
__host__ __device__ constexpr uint32_t idesc_i8(int m, int n) {
    return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
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

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(0u), "r"(sel));
    return d;
}

// One packed word (16 fields e = t+1) -> four words of int8 codes, in the field
// order of the tile-major layout: output q takes the fields at bits s_q + 4j,
// s_q = {0, 2, 16, 18}.  Two fields share a nibble, so after masking every
// nibble is a selector 0..2 into the byte table {-1, 0, +1}.
__device__ __forceinline__ void expand_word(uint32_t p, uint32_t* out) {
    constexpr uint32_t kTable = 0x000100ffu;
    const uint32_t q = p & 0x33333333u, r = (p >> 2) & 0x33333333u;
    out[0] = prmt(kTable, q);
    out[1] = prmt(kTable, r);
    out[2] = prmt(kTable, q >> 16);
    out[3] = prmt(kTable, r >> 16);
}

constexpr int MAX_MATS = 4;  // weight matrices (one K, one set of codes) that one launch can take

struct GemmParams {
    // Matrix j of the launch owns the weight-row tiles tile_base[j] .. tile_base[j+1]-1 of every token tile.
    const uint8_t* wt[MAX_MATS];   // tile-major packed weights (TS)
    const float* alpha[MAX_MATS];  // device scalars
    float* Y[MAX_MATS];            // [M, N_j]
    int y_bf16;                    // outputs are bf16 instead of fp32
    int N[MAX_MATS];
    int tile_base[MAX_MATS + 1];
    int count;
    const float* scale;   // [M]
    int32_t* acc;         // [M, N_0] or nullptr (single-matrix launches only)
    int M, K;
    int kblocks, n_tiles /* all matrices together */, m_tiles;
    // Rows of the activation tile that the tensor copy brings in (the box height of the tensor map): the tile
    // height, or less when the call has fewer tokens.  The MMAs still read the whole tile; what the rows beyond
    // hold ends up in accumulator columns of tokens that do not exist and is never stored.
    int act_rows;
    // Split-K (few tiles, many SMs): the channels of a tile are cut into ksplit ranges, one CTA each, and the
    // ksplit CTAs of a tile form one thread-block cluster (cluster rank = range).  Rank o owns a 1/ksplit share
    // of the tile's tokens: once every CTA of the cluster has its accumulator complete (first cluster barrier,
    // after which nobody's pipeline stages are in use), each CTA stores its int32 partial sums for o's tokens
    // into slot `own rank` of a buffer in o's shared memory (distributed shared memory, stores only); after the
    // second barrier o adds the ksplit slots and writes those rows of Y.
    int ksplit;
    // Divisions on the path to the first copy cost a single thread hundreds of clocks each, so the host hands
    // over what they would compute: the unit range of every part, and multipliers that turn the divisions by
    // ksplit and by n_tiles into a multiply-high (0 stands for a divisor of 1).
    int ubegin[kMaxSplit + 1];
    unsigned int ksplit_magic, n_tiles_magic;
};

// floor(n / d) for n * d < 2^32, with magic = floor(2^32 / d) + 1 (d > 1) or 0 (d == 1).
__device__ __forceinline__ int fast_div(int n, unsigned int magic) {
    return magic ? (int)__umulhi((unsigned int)n, magic) : n;
}

// Which matrix a weight-row tile (index over all matrices) belongs to.
__device__ __forceinline__ int matrix_of(const GemmParams& p, int nt) {
    int j = 0;
    while (j + 1 < p.count && nt >= p.tile_base[j + 1]) ++j;
    return j;
}

__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address, in the cluster's shared window, of this CTA's shared-memory address `addr` in the CTA of rank `rank`.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_s32(uint32_t cluster_addr, int v) {
    asm volatile("st.shared::cluster.s32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}

template <bool TS, int TM>
__global__ void __launch_bounds__((Cfg<TS, TM>::NUM_THREADS), 1)
    gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tm_act, const __grid_constant__ CUtensorMap tm_w,
                        const GemmParams p) {
    using C = Cfg<TS, TM>;
    constexpr int STAGES = C::STAGES, KBU = C::KBU, TILE_M = C::TILE_M, ACC_COLS = C::ACC_COLS, A_SLOTS = C::A_SLOTS;
    constexpr int EXPAND_GROUPS = C::EXPAND_GROUPS, EPI_SPLIT = C::EPI_SPLIT;
    constexpr int B_TILE_BYTES = C::B_TILE_BYTES, EPI_COLS = C::EPI_COLS;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* ctrl = smem + STAGES * C::STAGE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(ctrl);  // full[S] empty[S] afull[A] acc_full[2] acc_empty[2] epi
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ctrl + 512);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(ctrl + 516);

    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * STAGES;
    const uint32_t bar_afull = bar_empty + 8 * STAGES;
    const uint32_t bar_acc_full = bar_afull + 8 * A_SLOTS, bar_acc_empty = bar_acc_full + 8 * ACC_BUFS;
    const uint32_t smem_base = smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // Touch the launch parameters now: their first (cold) reads then overlap the prologue instead of sitting
    // in front of the producer's first copy.
    asm volatile("" ::"r"(p.ksplit), "r"(p.n_tiles), "r"(p.m_tiles), "r"(p.kblocks), "r"(p.tile_base[1]), "r"(p.M),
                 "r"(p.N[0]), "l"(p.wt[0]), "l"(p.scale), "l"(p.Y[0]));
    if (threadIdx.x == 0) {
        // start fetching the tensor-map descriptors now: the first tensor copy otherwise waits for them
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_act)) : "memory");
        if (!TS) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_w)) : "memory");
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, C::EMPTY_ARRIVALS);
        }
        for (int s = 0; s < A_SLOTS; ++s) mbar_init(bar_afull + 8 * s, 128);
        for (int b = 0; b < ACC_BUFS; ++b) {
            mbar_init(bar_acc_full + 8 * b, 1);
            mbar_init(bar_acc_empty + 8 * b, 128 * EPI_SPLIT);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_acc = tmem_base;
    const uint32_t tmem_a = tmem_base + ACC_BUFS * ACC_COLS;
    const int total_tiles = p.n_tiles * p.m_tiles;
    const int total_items = total_tiles * p.ksplit;  // item = tile * ksplit + part; split: one item per CTA
    int cluster_syncs = 0;               // cluster barriers this thread has passed (split-K)

    if (warp == 0) {
        // ------------------------------------------------------------- TMA producer
        // The warp walks the loop in lockstep; per unit lane 0 posts the byte count and the weights' bulk copy,
        // and lanes 1.. issue one tensor copy each (the same instruction, so they go out together).
        uint32_t it = 0, s = 0, ph = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
            const int tile = fast_div(item, p.ksplit_magic), part = item - tile * p.ksplit;
            const int u_begin = p.ubegin[part], u_end = p.ubegin[part + 1];
            const int mt = fast_div(tile, p.n_tiles_magic), nt = tile - mt * p.n_tiles;
            const int mj = matrix_of(p, nt), ntl = nt - p.tile_base[mj];
            const int m0 = mt * TILE_M, n0 = ntl * TILE_N;
            const uint8_t* wtile = p.wt[mj] + (size_t)ntl * p.kblocks * W_PACKED_BYTES;
            const int h = lane - 1;  // the 128-channel block this lane copies (activation tile; SS: then weights)
            for (int u = u_begin; u < u_end; ++u, ++it) {
                ok = __all_sync(0xffffffffu, mbar_wait(bar_empty + 8 * s, ph ^ 1, abort_flag, 1, it));
                if (!ok) break;
                const uint32_t dst = smem_base + s * C::STAGE_BYTES, bar = bar_full + 8 * s;
                if (lane == 0) {
                    mbar_expect_tx(bar, (uint32_t)(KBU * (p.act_rows * BK + (TS ? W_PACKED_BYTES : A_TILE_BYTES))));
                    if (TS)  // the weights come from HBM, the activation tile mostly from L2
                        bulk_load(dst + KBU * B_TILE_BYTES, wtile + (size_t)u * KBU * W_PACKED_BYTES, KBU * W_PACKED_BYTES,
                                  bar);
                }
                __syncwarp();
                if (h >= 0 && h < KBU) tma_load_2d(dst + h * B_TILE_BYTES, &tm_act, (u * KBU + h) * BK, m0, bar);
                if (!TS && h >= KBU && h < 2 * KBU)
                    tma_load_2d(dst + KBU * B_TILE_BYTES + (h - KBU) * A_TILE_BYTES, &tm_w, (u * KBU + h - KBU) * BK, n0, bar);
                __syncwarp();
                if (++s == (uint32_t)STAGES) { s = 0; ph ^= 1; }
            }
        }
        if (!ok && lane == 0) {
            // aborting: let the copies already issued land before the CTA exits
            for (uint32_t back = 1; back <= (uint32_t)STAGES && back <= it; ++back) {
                const uint32_t j = it - back, sj = j % STAGES, pj = (j / STAGES) & 1;
                const unsigned long long t0 = clock64();
                while (!mbar_try(bar_full + 8 * sj, pj) && clock64() - t0 < kWaitClocks) {
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------- MMA issuer
        // The whole warp walks the loop in lockstep so that indices and descriptors stay
        // warp-uniform; one elected lane issues the MMAs and the commits.  With TS the
        // issuer waits only for the expanded weights: the expanders arrive on that barrier
        // after they have themselves seen the stage's TMA barrier complete.
        constexpr uint32_t idesc = idesc_i8(TILE_N, TILE_M);
        const bool leader = elect_one();  // the same lane issues every MMA and commit
        uint32_t it = 0, tcount = 0;
        uint32_t s = 0, ph = 0;  // stage ring position and phase, advanced without divisions
        bool ok = true;
        for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x, ++tcount) {
            const int part = item - fast_div(item, p.ksplit_magic) * p.ksplit;
            const int u_begin = p.ubegin[part], u_end = p.ubegin[part + 1];
            const uint32_t ab = tcount % ACC_BUFS, pab = (tcount / ACC_BUFS) & 1;
            const uint32_t d_tmem = tmem_acc + ab * ACC_COLS;
            ok = __all_sync(0xffffffffu, mbar_wait(bar_acc_empty + 8 * ab, pab ^ 1, abort_flag, 2, tcount));
            if (!ok) break;
            tc_fence_after();
            for (int u = u_begin; u < u_end; ++u, ++it) {
                const uint32_t slot = it % A_SLOTS, pslot = (it / A_SLOTS) & 1;
                const uint32_t bar_in = TS ? bar_afull + 8 * slot : bar_full + 8 * s;
                ok = __all_sync(0xffffffffu, mbar_wait(bar_in, TS ? pslot : ph, abort_flag, TS ? 4 : 3, it));
                if (!ok) break;
                tc_fence_after();
                if (leader) {
                    const uint32_t b_addr = smem_base + s * C::STAGE_BYTES;
#pragma unroll
                    for (int h = 0; h < KBU; ++h) {
                        const uint64_t b_desc = smem_desc_sw128(b_addr + h * B_TILE_BYTES);
                        // advancing 32 channels = 32 bytes inside the swizzle row = +2 in the address field
                        if (TS) {
                            const uint32_t b_lo = (uint32_t)b_desc, b_hi = (uint32_t)(b_desc >> 32);
                            const uint32_t a_t = tmem_a + slot * C::A_SLOT_COLS + h * (BK / 4);
#pragma unroll
                            for (int j = 0; j < BK / UMMA_K; ++j) {
                                if (h == 0 && j == 0 && u == u_begin) mma_ts(d_tmem, a_t, b_desc, idesc, 0u);
                                else mma_ts_acc(d_tmem, a_t + j * (UMMA_K / 4), b_lo + 2 * j, b_hi, idesc);
                            }
                        } else {
                            const uint64_t a_desc = smem_desc_sw128(b_addr + KBU * B_TILE_BYTES + h * A_TILE_BYTES);
#pragma unroll
                            for (int j = 0; j < BK / UMMA_K; ++j)
                                mma_ss(d_tmem, a_desc + 2 * j, b_desc + 2 * j, idesc, (u > u_begin || h > 0 || j > 0) ? 1u : 0u);
                        }
                    }
                    tc_commit(bar_empty + 8 * s);
                }
                __syncwarp();
                if (++s == (uint32_t)STAGES) { s = 0; ph ^= 1; }
            }
            if (ok && leader) tc_commit(bar_acc_full + 8 * ab);
            __syncwarp();
        }
    } else if (warp < 2 + 4 * EXPAND_GROUPS) {
        // ------------------------------------------------------------- weight expanders (TS)
        if (TS) {
            const int quad = warp & 3;            // TMEM lanes 32*quad .. 32*quad+31 belong to this warp
            const int row = quad * 32 + lane;     // weight row inside the tile = TMEM lane
            const uint32_t group = (uint32_t)(warp - 2) >> 2;  // takes the units with it % groups == group
            const uint32_t a_lanes = tmem_a + ((uint32_t)(quad * 32) << 16);
            long long total_units = 0;  // units of all items of this CTA
            for (int item = blockIdx.x; item < total_items; item += gridDim.x) {
                const int part = item - fast_div(item, p.ksplit_magic) * p.ksplit;
                total_units += p.ubegin[part + 1] - p.ubegin[part];
            }
            bool ok = true;
            for (long long it64 = group; it64 < total_units && ok; it64 += EXPAND_GROUPS) {
                const uint32_t it = (uint32_t)it64;
                const uint32_t s = it % STAGES, ph = (it / STAGES) & 1, slot = it % A_SLOTS;
                const uint32_t a_dst = a_lanes + slot * C::A_SLOT_COLS;
                ok = __all_sync(0xffffffffu, mbar_wait(bar_full + 8 * s, ph, abort_flag, 7, it));
                if (!ok) break;
                const uint4* src = reinterpret_cast<const uint4*>(smem + s * C::STAGE_BYTES + KBU * B_TILE_BYTES);
                uint32_t v[KBU][32];
#pragma unroll
                for (int h = 0; h < KBU; ++h) {
                    const uint4 lo = src[h * 256 + row], hi = src[h * 256 + 128 + row];
                    expand_word(lo.x, v[h] + 0);
                    expand_word(lo.y, v[h] + 4);
                    expand_word(lo.z, v[h] + 8);
                    expand_word(lo.w, v[h] + 12);
                    expand_word(hi.x, v[h] + 16);
                    expand_word(hi.y, v[h] + 20);
                    expand_word(hi.z, v[h] + 24);
                    expand_word(hi.w, v[h] + 28);
                }
                __syncwarp();  // every lane has consumed its packed words: the stage's weight bytes are free
                if (lane == 0) mbar_arrive(bar_empty + 8 * s);
                if (it >= (uint32_t)A_SLOTS) {
                    // the slot was last read by the MMAs of unit it - A_SLOTS; their commit completes that stage's empty phase
                    const uint32_t j = it - A_SLOTS, sj = j % STAGES, pj = (j / STAGES) & 1;
                    ok = __all_sync(0xffffffffu, mbar_wait(bar_empty + 8 * sj, pj, abort_flag, 5, it));
                    if (!ok) break;
                }
                tc_fence_after();
#pragma unroll
                for (int h = 0; h < KBU; ++h) tmem_st32(a_dst + h * (BK / 4), v[h]);
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                tc_fence_before();
                mbar_arrive(bar_afull + 8 * slot);
            }
        }
    } else {
        // ------------------------------------------------------------- epilogue
        const int quad = warp & 3;
        const int cbase = ((warp - (2 + 4 * EXPAND_GROUPS)) >> 2) * EPI_COLS;  // this warp's share of the token columns
        uint32_t tcount = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x, ++tcount) {
            const int tile = fast_div(item, p.ksplit_magic);
            const int mt = fast_div(tile, p.n_tiles_magic), nt = tile - mt * p.n_tiles, mj = matrix_of(p, nt);
            const int m0 = mt * TILE_M, n0 = (nt - p.tile_base[mj]) * TILE_N;
            const int N = p.N[mj];
            const float alpha = __ldg(p.alpha[mj]);
            const uint32_t ab = tcount % ACC_BUFS, pab = (tcount / ACC_BUFS) & 1;
            ok = __all_sync(0xffffffffu, mbar_wait(bar_acc_full + 8 * ab, pab, abort_flag, 6, tcount));
            if (!ok) break;
            tc_fence_after();
            if (p.ksplit > 1) {
                cluster_sync_all();  // every CTA of the cluster is past its last MMA: stage memory is free everywhere
                ++cluster_syncs;
            }
            const int n = n0 + quad * 32 + lane;
            const bool n_ok = n < N;
#pragma unroll 1
            for (int c0 = cbase; c0 < cbase + EPI_COLS; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(tmem_acc + ((uint32_t)(quad * 32) << 16) + ab * ACC_COLS + c0, r);
                const int mrow = m0 + c0;
                const int valid = p.M - mrow;  // tokens of this chunk that exist
                const size_t o = (size_t)mrow * N + n;
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (!n_ok) continue;
                if (p.ksplit > 1) {
                    // token c of the tile belongs to rank c / per, row c % per; this CTA writes slot `part`
                    const int tokens = min(TILE_M, p.M - m0), per = (tokens + p.ksplit - 1) / p.ksplit;
                    const int part = item - tile * p.ksplit;
                    int owner = c0 / per, row = c0 - owner * per;
                    const uint32_t slot_addr = smem_base + (uint32_t)((part * per) * TILE_N + quad * 32 + lane) * 4u;
                    uint32_t dst = map_to_rank(slot_addr, (uint32_t)min(owner, p.ksplit - 1));
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        if (j < valid) st_cluster_s32(dst + (uint32_t)(row * TILE_N) * 4u, (int)r[j]);
                        if (++row == per) {
                            row = 0;
                            ++owner;
                            dst = map_to_rank(slot_addr, (uint32_t)min(owner, p.ksplit - 1));
                        }
                    }
                    continue;
                }
                float* yp = p.Y[mj] + o;
                const float* sp = p.scale + mrow;
                // y = fp32(acc) * (scale[m] * alpha): the prefactors of Eq. 2, 3 and 7
                if (p.y_bf16) {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (j < valid) a48_store_y(p.Y[mj], o + (size_t)j * N, (float)(int)r[j] * (__ldg(sp + j) * alpha), 1);
                } else if (valid >= 32) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        *yp = (float)(int)r[j] * (__ldg(sp + j) * alpha);
                        yp += N;
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (j < valid) yp[(size_t)j * N] = (float)(int)r[j] * (__ldg(sp + j) * alpha);
                }
                if (p.acc) {
                    int32_t* ap = p.acc + o;
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (j < valid) ap[(size_t)j * N] = (int)r[j];
                }
            }
            tc_fence_before();
            mbar_arrive(bar_acc_empty + 8 * ab);
        }
    }
    if (p.ksplit > 1) {
        // Every thread of every CTA of the cluster passes exactly two cluster barriers, also after an abort.  The
        // epilogue warps took the first one as soon as their accumulator was complete.
        __syncwarp();
        for (; cluster_syncs < 2; ++cluster_syncs) cluster_sync_all();
        const int te = (int)threadIdx.x - 32 * (2 + 4 * EXPAND_GROUPS);  // index among the epilogue threads
        if (te >= 0 && !*abort_flag) {
            const int tile = fast_div((int)blockIdx.x, p.ksplit_magic), rank = (int)blockIdx.x - tile * p.ksplit;
            const int mt = fast_div(tile, p.n_tiles_magic), nt = tile - mt * p.n_tiles, mj = matrix_of(p, nt), N = p.N[mj];
            const int m0 = mt * TILE_M, nl = te & (TILE_N - 1), n = (nt - p.tile_base[mj]) * TILE_N + nl;
            const int tokens = min(TILE_M, p.M - m0);
            const int per = (tokens + p.ksplit - 1) / p.ksplit;  // tokens owned by each rank
            const int rows = min(per, tokens - rank * per);      // ... and by this one (may be <= 0)
            const float alpha = __ldg(p.alpha[mj]);
            const int* slots = reinterpret_cast<const int*>(smem);
            if (n < N) {
                for (int row = te >> 7; row < rows; row += 128 * EPI_SPLIT / TILE_N) {
                    int sum = 0;
#pragma unroll
                    for (int q = 0; q < kMaxSplit; ++q)
                        if (q < p.ksplit) sum += slots[(q * per + row) * TILE_N + nl];
                    const int m = m0 + rank * per + row;
                    const size_t e = (size_t)m * N + n;
                    a48_store_y(p.Y[mj], e, (float)sum * (__ldg(p.scale + m) * alpha), p.y_bf16);
                    if (p.acc) p.acc[e] = sum;
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ---- CTA-pair form (cta_group::2) ------------------------------------------------------------------------------
// Two CTAs on neighbouring SMs (a cluster of two) work on one tile of 256 weight rows x 192 tokens.  Each CTA
// expands and holds the 128 weight rows of its half in its own tensor memory and accumulates their 192 outputs
// per token there; the token tile is split the other way: each CTA stages 96 of the 192 tokens in its shared
// memory and the MMA (issued by the CTA of rank 0 for both) reads the two halves.  An activation byte thus feeds
// 256 weight rows instead of 128: the traffic from L2 into an SM per MMA, which is what the single-CTA kernel's
// stalls trace back to, is halved, and the ring of stages reaches twice as far ahead in time.
// Protocol across the pair: the expanders of both CTAs arrive on the afull barriers of rank 0 (remote arrive for
// rank 1) after they have seen their own stage land, so rank 0's issuer knows weights and tokens of both CTAs
// are in place; one commit per stage is multicast to the empty barriers of both CTAs (stage and tensor-memory
// slot free in both), one per tile to both acc_full barriers; the epilogue threads of both CTAs arrive on rank
// 0's acc_empty.  No TMA multicast is used: every CTA copies its own half.
template <int TOK_, int A_SLOTS_, int STAGES_>
struct PairCfg {
    static constexpr int TOK = TOK_, HALF = TOK / 2, KBU = 2;
    static constexpr int B_HALF_BYTES = HALF * BK;
    static constexpr int STAGE_BYTES = KBU * (B_HALF_BYTES + W_PACKED_BYTES);
    static constexpr int STAGES = STAGES_;
    static constexpr int A_SLOTS = A_SLOTS_, A_SLOT_COLS = KBU * BK / 4, ACC_COLS = TOK;
    static constexpr int EXPAND_GROUPS = 2, EPI_SPLIT = 2;
    static constexpr int EPI_FIRST = (TOK / 32 + 1) / 2 * 32;  // columns drained by the first epilogue warp of a quadrant
    static constexpr int NUM_THREADS = 32 * (2 + 4 * EXPAND_GROUPS + 4 * EPI_SPLIT);
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 + 1024;
    static_assert(HALF % 8 == 0 && TOK % 32 == 0, "swizzle rows and 32-column epilogue chunks");
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
    static_assert(ACC_BUFS * ACC_COLS + A_SLOTS * A_SLOT_COLS <= TMEM_COLS, "tensor memory budget");
    static_assert(STAGES > A_SLOTS, "the stage A_SLOTS units back must still be distinct");
};

__device__ __forceinline__ void mbar_arrive_rank(uint32_t bar, uint32_t rank) {
    asm volatile(
        "{\n\t.reg .b32 ra;\n\tmapa.shared::cluster.u32 ra, %0, %1;\n\t"
        "mbarrier.arrive.shared::cluster.b64 _, [ra];\n\t}" ::"r"(bar), "r"(rank)
        : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {  // arrives on `bar` in both CTAs of the pair
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
                 "h"((unsigned short)3)
                 : "memory");
}
__device__ __forceinline__ void mma_ts_pair(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc),
        "r"(accumulate)
        : "memory");
}

struct PairParams {
    const uint8_t* wt;
    const float* alpha;
    const float* scale;
    float* Y;
    int y_bf16;  // outputs are bf16 instead of fp32
    int32_t* acc;
    int M, N, kblocks, n_pairs, m_tiles;
    int n_tiles128;  // 128-row weight tiles in the packed layout; an odd count leaves the last pair's second CTA
                     // without rows of its own: it re-reads the last tile and stores nothing
    unsigned int n_pairs_magic;
};

template <class PC>
__global__ void __launch_bounds__(PC::NUM_THREADS, 1)
    gemm_pair_kernel(const __grid_constant__ CUtensorMap tm_act, const PairParams p) {
    constexpr int TOK = PC::TOK, HALF = PC::HALF, KBU = PC::KBU, B_HALF_BYTES = PC::B_HALF_BYTES;
    constexpr int STAGE_BYTES = PC::STAGE_BYTES, STAGES = PC::STAGES, A_SLOTS = PC::A_SLOTS, A_SLOT_COLS = PC::A_SLOT_COLS;
    constexpr int ACC_COLS = PC::ACC_COLS, EXPAND_GROUPS = PC::EXPAND_GROUPS, EPI_SPLIT = PC::EPI_SPLIT;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* ctrl = smem + STAGES * STAGE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(ctrl);  // full[S] empty[S] afull[A] acc_full[2] acc_empty[2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ctrl + 512);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(ctrl + 516);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * STAGES;
    const uint32_t bar_afull = bar_empty + 8 * STAGES;
    const uint32_t bar_acc_full = bar_afull + 8 * A_SLOTS, bar_acc_empty = bar_acc_full + 8 * ACC_BUFS;
    const uint32_t smem_base = smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = (int)(blockIdx.x & 1u);       // rank in the pair; rank 0 issues the MMAs
    const int pair = (int)(blockIdx.x >> 1), pairs = (int)(gridDim.x >> 1);

    asm volatile("" ::"r"(p.n_pairs), "r"(p.m_tiles), "r"(p.kblocks), "r"(p.M), "r"(p.N), "l"(p.wt), "l"(p.scale), "l"(p.Y));
    if (threadIdx.x == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_act)) : "memory");
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 5);  // four expander warps of this CTA and the multicast commit
        }
        // afull and acc_empty are used in rank 0 only; one lane per warp arrives for its warp (a release at
        // cluster scope by every thread cost ~1400 clocks per unit)
        for (int s = 0; s < A_SLOTS; ++s) mbar_init(bar_afull + 8 * s, 2 * 4);  // one expander group of each CTA
        for (int b = 0; b < ACC_BUFS; ++b) {
            mbar_init(bar_acc_full + 8 * b, 1);
            mbar_init(bar_acc_empty + 8 * b, 2 * 4 * EPI_SPLIT);  // the epilogue warps of both CTAs
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // the peer's barriers are initialised and its tensor memory is allocated
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_acc = tmem_base;
    const uint32_t tmem_a = tmem_base + ACC_BUFS * ACC_COLS;
    const int total_tiles = p.n_pairs * p.m_tiles;
    const int kunits = p.kblocks / KBU;

    if (warp == 0) {
        // ------------------------------------------------------------- TMA producer (both CTAs, own halves)
        uint32_t it = 0, s = 0, ph = 0;
        bool ok = true;
        for (int tile = pair; tile < total_tiles && ok; tile += pairs) {
            const int mt = fast_div(tile, p.n_pairs_magic), pn = tile - mt * p.n_pairs;
            const int m0 = mt * TOK + rank * HALF;  // this CTA stages its half of the token tile
            const uint8_t* wtile = p.wt + (size_t)min(2 * pn + rank, p.n_tiles128 - 1) * p.kblocks * W_PACKED_BYTES;
            const int h = lane - 1;
            for (int u = 0; u < kunits; ++u, ++it) {
                ok = __all_sync(0xffffffffu, mbar_wait(bar_empty + 8 * s, ph ^ 1, abort_flag, 11, it));
                if (!ok) break;
                const uint32_t dst = smem_base + s * STAGE_BYTES, bar = bar_full + 8 * s;
                if (lane == 0) {
                    mbar_expect_tx(bar, STAGE_BYTES);
                    bulk_load(dst + KBU * B_HALF_BYTES, wtile + (size_t)u * KBU * W_PACKED_BYTES, KBU * W_PACKED_BYTES, bar);
                }
                __syncwarp();
                if (h >= 0 && h < KBU) tma_load_2d(dst + h * B_HALF_BYTES, &tm_act, (u * KBU + h) * BK, m0, bar);
                __syncwarp();
                if (++s == (uint32_t)STAGES) { s = 0; ph ^= 1; }
            }
        }
        if (!ok && lane == 0) {
            for (uint32_t back = 1; back <= (uint32_t)STAGES && back <= it; ++back) {
                const uint32_t j = it - back, sj = j % STAGES, pj = (j / STAGES) & 1;
                const unsigned long long t0 = clock64();
                while (!mbar_try(bar_full + 8 * sj, pj) && clock64() - t0 < kWaitClocks) {
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------- MMA issuer (rank 0 only)
        if (rank == 0) {
            constexpr uint32_t idesc = idesc_i8(2 * TILE_N, TOK);
            const bool leader = elect_one();
            uint32_t it = 0, tcount = 0, s = 0;
            bool ok = true;
            for (int tile = pair; tile < total_tiles && ok; tile += pairs, ++tcount) {
                const uint32_t ab = tcount % ACC_BUFS, pab = (tcount / ACC_BUFS) & 1;
                const uint32_t d_tmem = tmem_acc + ab * ACC_COLS;
                ok = __all_sync(0xffffffffu, mbar_wait(bar_acc_empty + 8 * ab, pab ^ 1, abort_flag, 12, tcount));
                if (!ok) break;
                tc_fence_after();
                for (int u = 0; u < kunits; ++u, ++it) {
                    const uint32_t slot = it % A_SLOTS, pslot = (it / A_SLOTS) & 1;
                    ok = __all_sync(0xffffffffu, mbar_wait(bar_afull + 8 * slot, pslot, abort_flag, 14, it));
                    if (!ok) break;
                    tc_fence_after();
                    if (leader) {
                        const uint32_t b_addr = smem_base + s * STAGE_BYTES;
#pragma unroll
                        for (int h = 0; h < KBU; ++h) {
                            const uint64_t b_desc = smem_desc_sw128(b_addr + h * B_HALF_BYTES);
                            const uint32_t a_t = tmem_a + slot * A_SLOT_COLS + h * (BK / 4);
#pragma unroll
                            for (int j = 0; j < BK / UMMA_K; ++j)
                                mma_ts_pair(d_tmem, a_t + j * (UMMA_K / 4), b_desc + 2 * j, idesc, (u > 0 || h > 0 || j > 0) ? 1u : 0u);
                        }
                        tc_commit_pair(bar_empty + 8 * s);
                    }
                    __syncwarp();
                    if (++s == (uint32_t)STAGES) s = 0;
                }
                if (ok && leader) tc_commit_pair(bar_acc_full + 8 * ab);
                __syncwarp();
            }
        }
    } else if (warp < 2 + 4 * EXPAND_GROUPS) {
        // ------------------------------------------------------------- weight expanders (both CTAs)
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        const uint32_t group = (uint32_t)(warp - 2) >> 2;
        const uint32_t a_lanes = tmem_a + ((uint32_t)(quad * 32) << 16);
        const int my_tiles = (total_tiles - pair + pairs - 1) / pairs;
        const long long total_units = (long long)kunits * (my_tiles > 0 ? my_tiles : 0);
        bool ok = true;
        for (long long it64 = group; it64 < total_units && ok; it64 += EXPAND_GROUPS) {
            const uint32_t it = (uint32_t)it64;
            const uint32_t s = it % STAGES, ph = (it / STAGES) & 1, slot = it % A_SLOTS;
            const uint32_t a_dst = a_lanes + slot * A_SLOT_COLS;
            ok = __all_sync(0xffffffffu, mbar_wait(bar_full + 8 * s, ph, abort_flag, 17, it));
            if (!ok) break;
            const uint4* src = reinterpret_cast<const uint4*>(smem + s * STAGE_BYTES + KBU * B_HALF_BYTES);
            uint32_t v[KBU][32];
#pragma unroll
            for (int h = 0; h < KBU; ++h) {
                const uint4 lo = src[h * 256 + row], hi = src[h * 256 + 128 + row];
                expand_word(lo.x, v[h] + 0);
                expand_word(lo.y, v[h] + 4);
                expand_word(lo.z, v[h] + 8);
                expand_word(lo.w, v[h] + 12);
                expand_word(hi.x, v[h] + 16);
                expand_word(hi.y, v[h] + 20);
                expand_word(hi.z, v[h] + 24);
                expand_word(hi.w, v[h] + 28);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty + 8 * s);
            if (it >= (uint32_t)A_SLOTS) {
                const uint32_t j = it - A_SLOTS, sj = j % STAGES, pj = (j / STAGES) & 1;
                ok = __all_sync(0xffffffffu, mbar_wait(bar_empty + 8 * sj, pj, abort_flag, 15, it));
                if (!ok) break;
            }
            tc_fence_after();
#pragma unroll
            for (int h = 0; h < KBU; ++h) tmem_st32(a_dst + h * (BK / 4), v[h]);
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_rank(bar_afull + 8 * slot, 0u);  // this warp's rows are in tensor memory, the tokens have landed
        }
    } else {
        // ------------------------------------------------------------- epilogue (both CTAs, own 128 rows)
        const int quad = warp & 3;
        const int half = (warp - (2 + 4 * EXPAND_GROUPS)) >> 2;
        const int c_begin = half ? PC::EPI_FIRST : 0, c_end = half ? TOK : PC::EPI_FIRST;
        const float alpha = __ldg(p.alpha);
        uint32_t tcount = 0;
        bool ok = true;
        for (int tile = pair; tile < total_tiles && ok; tile += pairs, ++tcount) {
            const int mt = fast_div(tile, p.n_pairs_magic), pn = tile - mt * p.n_pairs;
            const int m0 = mt * TOK, n = (2 * pn + rank) * TILE_N + quad * 32 + lane;
            const uint32_t ab = tcount % ACC_BUFS, pab = (tcount / ACC_BUFS) & 1;
            ok = __all_sync(0xffffffffu, mbar_wait(bar_acc_full + 8 * ab, pab, abort_flag, 16, tcount));
            if (!ok) break;
            tc_fence_after();
#pragma unroll 1
            for (int c0 = c_begin; c0 < c_end; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(tmem_acc + ((uint32_t)(quad * 32) << 16) + ab * ACC_COLS + c0, r);
                const int mrow = m0 + c0;
                const int valid = p.M - mrow;
                const size_t o = (size_t)mrow * p.N + n;
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (n >= p.N) continue;
                float* yp = p.Y + o;
                const float* sp = p.scale + mrow;
                if (p.y_bf16) {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (j < valid) a48_store_y(p.Y, o + (size_t)j * p.N, (float)(int)r[j] * (__ldg(sp + j) * alpha), 1);
                } else if (valid >= 32) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        *yp = (float)(int)r[j] * (__ldg(sp + j) * alpha);
                        yp += p.N;
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (j < valid) yp[(size_t)j * p.N] = (float)(int)r[j] * (__ldg(sp + j) * alpha);
                }
                if (p.acc) {
                    int32_t* ap = p.acc + o;
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (j < valid) ap[(size_t)j * p.N] = (int)r[j];
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_rank(bar_acc_empty + 8 * ab, 0u);
        }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // both CTAs are done with both tensor memories and with each other's barriers
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ---- host side -----------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// int8 matrix [rows, cols] row-major (row pitch = pitch bytes), box = 128 bytes x box_rows, 128-byte swizzle.
bool make_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint64_t pitch, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {pitch};
    cuuint32_t box[2] = {BK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int sm_count() {
    static int n[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    int& c = n[dev & 63];
    if (!c) cudaDeviceGetAttribute(&c, cudaDevAttrMultiProcessorCount, dev);
    return c;
}

// How a call is cut into work items.  With fewer tiles than SMs the channels of a tile are split over `ksplit`
// CTAs (one cluster); the cost of a split, in pipeline units per CTA, is rounds * (units per item + a fixed
// per-item charge for filling the pipeline and for the reduction through distributed shared memory).
struct Plan {
    int tile_m, n_tiles, m_tiles, ksplit;
};

// Time model of a launch above 64 tokens: rounds of tiles over the SMs times the time of a pipeline unit, which the
// token sweep gives as about 0.43 us on 128-token tiles, 0.54 us on 192-token tiles and 0.50 us on 192-token tiles of
// a CTA pair (4096 -> 11008 and 11008 -> 4096, 128 to 2048 tokens); the unit count and the fixed cost of a launch
// are the same for the forms compared.
long long single_cost(int n_tiles, int M, int tile_m) {
    const long long tiles = (long long)n_tiles * ((M + tile_m - 1) / tile_m), sms = sm_count();
    return (tiles + sms - 1) / sms * (tile_m == TILE_M_MID ? 43 : 54);
}
long long pair_cost(int n_tiles, int M) {
    const long long items = (long long)((n_tiles + 1) / 2) * ((M + 191) / 192), slots = sm_count() / 2;
    return (items + slots - 1) / slots * 50;
}

Plan make_plan(int count, const bitnet_a48_weight* const* ws, int M, bool ts) {
    Plan pl;
    pl.n_tiles = 0;
    for (int j = 0; j < count; ++j) pl.n_tiles += (ws[j]->N + TILE_N - 1) / TILE_N;
    // above 64 tokens: 128- or 192-token tiles, whichever leaves the CTAs less to do (fewer idle slots in the last
    // round of tiles against a longer unit)
    const bool mid = M > TILE_M_SKINNY && single_cost(pl.n_tiles, M, TILE_M_MID) < single_cost(pl.n_tiles, M, TILE_M_WIDE);
    pl.tile_m = M <= TILE_M_TINY ? TILE_M_TINY : (M <= TILE_M_SKINNY ? TILE_M_SKINNY : (mid ? TILE_M_MID : TILE_M_WIDE));
    pl.m_tiles = (M + pl.tile_m - 1) / pl.tile_m;
    const int tiles = pl.n_tiles * pl.m_tiles, sms = sm_count();
    const int kunits = ws[0]->Kp / BK / (ts ? 2 : 1);
    // fixed cost of a wave of CTAs in units: launch, prologue, first copy, epilogue come to about 5 us, a unit to
    // 0.33-0.47 us (measured); with 3 a split into two waves was chosen for 512 tokens x 4096 x 11008 and lost 2x
    constexpr int kItemCharge = 10;
    pl.ksplit = 1;
    long long best = (long long)((tiles + sms - 1) / sms) * (kunits + kItemCharge);
    for (int ks = 2; ks <= kMaxSplit && ks <= kunits && tiles < sms; ++ks) {
        const int slots = sms / ks * ks;  // whole clusters only
        const long long rounds = ((long long)tiles * ks + slots - 1) / slots;
        const long long cost = rounds * ((kunits + ks - 1) / ks + kItemCharge + 2);
        if (cost * 10 < best * 9) {  // a split has to pay for itself by a clear margin
            best = cost;
            pl.ksplit = ks;
        }
    }
    return pl;
}

template <bool TS, int TM>
bitnet_a48_status launch(int count, const bitnet_a48_weight* const* ws, const int8_t* codes, const float* scale, int M,
                         float* const* Y, int32_t* acc, Plan pl, cudaStream_t st) {
    using C = Cfg<TS, TM>;
    static bool attr_set[64] = {};        // the attribute is per device
    static signed char cluster_ok[64][kMaxSplit + 1] = {};  // 0 unknown, 1 the device can host such a cluster, -1 it cannot
    int dev = 0;
    A48_CUDA_TRY(cudaGetDevice(&dev));
    dev &= 63;
    if (!attr_set[dev]) {
        A48_CUDA_TRY(cudaFuncSetAttribute(gemm_tcgen05_kernel<TS, TM>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          C::SMEM_BYTES));
        attr_set[dev] = true;
    }
    const bitnet_a48_weight* w = ws[0];
    CUtensorMap tm_act, tm_w;
    const int act_rows = M >= TM ? TM : (M + 15) / 16 * 16;
    if (!make_map(&tm_act, codes, (uint64_t)M, (uint64_t)w->K, (uint64_t)w->K, (uint32_t)act_rows)) return BITNET_A48_ERR_CUDA;
    if (TS) {
        tm_w = tm_act;  // unused
    } else if (!make_map(&tm_w, w->i8, (uint64_t)w->Np, (uint64_t)w->Kp, (uint64_t)w->Kp, TILE_N)) {
        return BITNET_A48_ERR_CUDA;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(C::NUM_THREADS);
    cfg.dynamicSmemBytes = C::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    if (pl.ksplit > 1) {
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)pl.ksplit;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cfg.gridDim = dim3((unsigned)(pl.n_tiles * pl.m_tiles * pl.ksplit));
        signed char& okc = cluster_ok[dev][pl.ksplit];
        if (okc == 0) {
            int clusters = 0;
            okc = cudaOccupancyMaxActiveClusters(&clusters, gemm_tcgen05_kernel<TS, TM>, &cfg) == cudaSuccess &&
                          clusters >= 1
                      ? 1
                      : -1;
            if (okc < 0) (void)cudaGetLastError();
        }
        if (okc < 0) {  // whole tiles instead
            pl.ksplit = 1;
            cfg.attrs = nullptr;
            cfg.numAttrs = 0;
        }
    }
    GemmParams p = {};
    p.count = count;
    p.tile_base[0] = 0;
    for (int j = 0; j < count; ++j) {
        p.wt[j] = ws[j]->gemm;
        p.alpha[j] = ws[j]->alpha_dev;
        p.Y[j] = Y[j];
        p.N[j] = ws[j]->N;
        p.tile_base[j + 1] = p.tile_base[j] + (ws[j]->N + TILE_N - 1) / TILE_N;
    }
    p.scale = scale;
    p.acc = acc;
    p.y_bf16 = a48_y_bf16;
    p.M = M;
    p.K = w->K;
    p.kblocks = w->Kp / BK;
    p.n_tiles = pl.n_tiles;
    p.m_tiles = pl.m_tiles;
    p.ksplit = pl.ksplit;
    p.act_rows = act_rows;
    {
        const int kunits = p.kblocks / C::KBU;
        for (int i = 0; i <= kMaxSplit; ++i) p.ubegin[i] = i <= pl.ksplit ? (int)((long long)i * kunits / pl.ksplit) : kunits;
        auto magic = [](int d) { return d > 1 ? (unsigned int)((1ull << 32) / (unsigned)d) + 1u : 0u; };
        p.ksplit_magic = magic(pl.ksplit);
        p.n_tiles_magic = magic(pl.n_tiles);
        // the multiply-high is exact while dividend * divisor < 2^32
        if ((unsigned long long)pl.n_tiles * pl.m_tiles * pl.ksplit * (pl.n_tiles > pl.ksplit ? pl.n_tiles : pl.ksplit) >= (1ull << 32))
            return BITNET_A48_ERR_SHAPE;
    }
    if (pl.ksplit == 1) {
        const int total = p.n_tiles * p.m_tiles;
        cfg.gridDim = dim3((unsigned)(total < sm_count() ? total : sm_count()));
    }
    A48_CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_tcgen05_kernel<TS, TM>, tm_act, tm_w, p));
    return BITNET_A48_OK;
}

template <class PC>
bitnet_a48_status launch_pair(const bitnet_a48_weight* w, const int8_t* codes, const float* scale, int M, float* Y,
                              int32_t* acc, cudaStream_t st) {
    static signed char ready[64] = {};  // per device: 0 unknown, 1 attribute set and a pair can be hosted, -1 not
    int dev = 0;
    A48_CUDA_TRY(cudaGetDevice(&dev));
    dev &= 63;
    CUtensorMap tm_act;
    if (!make_map(&tm_act, codes, (uint64_t)M, (uint64_t)w->K, (uint64_t)w->K, PC::HALF)) return BITNET_A48_ERR_CUDA;
    PairParams p;
    p.wt = w->gemm;
    p.alpha = w->alpha_dev;
    p.scale = scale;
    p.Y = Y;
    p.y_bf16 = a48_y_bf16;
    p.acc = acc;
    p.M = M;
    p.N = w->N;
    p.kblocks = w->Kp / BK;
    p.n_tiles128 = (w->N + TILE_N - 1) / TILE_N;
    p.n_pairs = (p.n_tiles128 + 1) / 2;
    p.m_tiles = (M + PC::TOK - 1) / PC::TOK;
    p.n_pairs_magic = p.n_pairs > 1 ? (unsigned int)((1ull << 32) / (unsigned)p.n_pairs) + 1u : 0u;
    const long long total = (long long)p.n_pairs * p.m_tiles;
    if (total * p.n_pairs >= (1ll << 32)) return BITNET_A48_ERR_SHAPE;
    const int pairs_max = sm_count() / 2;
    const int pairs = total < pairs_max ? (int)total : pairs_max;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * pairs));
    cfg.blockDim = dim3(PC::NUM_THREADS);
    cfg.dynamicSmemBytes = PC::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (ready[dev] == 0) {
        A48_CUDA_TRY(cudaFuncSetAttribute(gemm_pair_kernel<PC>, cudaFuncAttributeMaxDynamicSharedMemorySize, PC::SMEM_BYTES));
        int clusters = 0;
        ready[dev] = cudaOccupancyMaxActiveClusters(&clusters, gemm_pair_kernel<PC>, &cfg) == cudaSuccess && clusters >= 1 ? 1 : -1;
        if (ready[dev] < 0) (void)cudaGetLastError();
    }
    if (ready[dev] < 0) return BITNET_A48_ERR_UNSUPPORTED;
    A48_CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_pair_kernel<PC>, tm_act, p));
    return BITNET_A48_OK;
}

}  // namespace

bool a48_gemm_pair_supported(const bitnet_a48_weight* w, int M) { return a48_gemm_tcgen05_supported(w, M, false); }

// Whether the library's own choice for these matrices on the same tokens is a CTA-pair launch per matrix rather than
// one single-CTA launch over all their tiles.
bool a48_gemm_pair_preferred(int count, const bitnet_a48_weight* const* ws, int M) {
    if (M < 384) return false;
    int n_all = 0;
    long long pairs = 0;
    for (int j = 0; j < count; ++j) {
        if (!a48_gemm_pair_supported(ws[j], M)) return false;
        const int n = (ws[j]->N + TILE_N - 1) / TILE_N;
        n_all += n;
        pairs += pair_cost(n, M);
    }
    const long long single = std::min(single_cost(n_all, M, TILE_M_MID), single_cost(n_all, M, TILE_M_WIDE));
    return pairs <= single;
}

bitnet_a48_status a48_launch_gemm_pair(const bitnet_a48_weight* w, const int8_t* codes, const float* scale, int M,
                                       float* Y, int32_t* acc, cudaStream_t st) {
    if (!a48_gemm_pair_supported(w, M)) return BITNET_A48_ERR_UNSUPPORTED;
    // 192 tokens, two weight slots, seven 32 KB stages: measured 4-8 % ahead of 160 tokens / three slots / eight
    // stages and 15 % ahead of 128 / four / nine
    return launch_pair<PairCfg<192, 2, 7>>(w, codes, scale, M, Y, acc, st);
}

bool a48_gemm_tcgen05_supported(const bitnet_a48_weight* w, int M, bool ss) {
    if (w->K % 16 != 0 || M < 1) return false;  // TMA needs a 16-byte row pitch
    return ss ? w->i8 != nullptr : w->gemm != nullptr;
}

bitnet_a48_status a48_launch_gemm_tcgen05(const bitnet_a48_weight* w, const int8_t* codes, const float* scale, int M,
                                          float* Y, int32_t* acc, bool ss, cudaStream_t st) {
    const Plan pl = make_plan(1, &w, M, !ss);
    if (pl.tile_m == TILE_M_SKINNY)
        return ss ? launch<false, TILE_M_SKINNY>(1, &w, codes, scale, M, &Y, acc, pl, st)
                  : launch<true, TILE_M_SKINNY>(1, &w, codes, scale, M, &Y, acc, pl, st);
    if (pl.tile_m == TILE_M_TINY)
        return ss ? launch<false, TILE_M_TINY>(1, &w, codes, scale, M, &Y, acc, pl, st)
                  : launch<true, TILE_M_TINY>(1, &w, codes, scale, M, &Y, acc, pl, st);
    if (pl.tile_m == TILE_M_MID)
        return ss ? launch<false, TILE_M_MID>(1, &w, codes, scale, M, &Y, acc, pl, st)
                  : launch<true, TILE_M_MID>(1, &w, codes, scale, M, &Y, acc, pl, st);
    return ss ? launch<false, TILE_M_WIDE>(1, &w, codes, scale, M, &Y, acc, pl, st)
              : launch<true, TILE_M_WIDE>(1, &w, codes, scale, M, &Y, acc, pl, st);
}

bool a48_gemm_tcgen05_multi_supported(int count, const bitnet_a48_weight* const* ws, int M) {
    if (count < 1 || count > MAX_MATS) return false;
    for (int j = 0; j < count; ++j)
        if (!a48_gemm_tcgen05_supported(ws[j], M, false) || ws[j]->K != ws[0]->K) return false;
    return true;
}

bitnet_a48_status a48_launch_gemm_tcgen05_multi(int count, const bitnet_a48_weight* const* ws, const int8_t* codes,
                                                const float* scale, int M, float* const* Y, cudaStream_t st) {
    if (!a48_gemm_tcgen05_multi_supported(count, ws, M)) return BITNET_A48_ERR_UNSUPPORTED;
    const Plan pl = make_plan(count, ws, M, true);
    if (pl.tile_m == TILE_M_TINY) return launch<true, TILE_M_TINY>(count, ws, codes, scale, M, Y, nullptr, pl, st);
    if (pl.tile_m == TILE_M_MID) return launch<true, TILE_M_MID>(count, ws, codes, scale, M, Y, nullptr, pl, st);
    return pl.tile_m == TILE_M_SKINNY ? launch<true, TILE_M_SKINNY>(count, ws, codes, scale, M, Y, nullptr, pl, st)
                                      : launch<true, TILE_M_WIDE>(count, ws, codes, scale, M, Y, nullptr, pl, st);
}

bitnet_a48_status a48_read_kernel_status(unsigned int words_host[4]) {
    A48_CUDA_TRY(cudaDeviceSynchronize());
    A48_CUDA_TRY(cudaMemcpyFromSymbol(words_host, g_status, sizeof(unsigned int) * 4));
    const unsigned int zero[4] = {0, 0, 0, 0};
    A48_CUDA_TRY(cudaMemcpyToSymbol(g_status, zero, sizeof(zero)));
    unsigned int dec[4];
    bitnet_a48_status ds = a48_read_decode_status(dec);
    if (ds != BITNET_A48_OK) return ds;
    if (words_host[0] == 0 && dec[0] != 0)
        for (int i = 0; i < 4; ++i) words_host[i] = dec[i];
    ds = a48_read_attn_status(dec);
    if (ds != BITNET_A48_OK) return ds;
    if (words_host[0] == 0 && dec[0] != 0)
        for (int i = 0; i < 4; ++i) words_host[i] = dec[i];
    return BITNET_A48_OK;
}
