// Internal declarations shared by the translation units of libbitnet_a48.so.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "bitnet_a48.h"

#define A48_CUDA_TRY(expr)                                  \
    do {                                                    \
        cudaError_t err__ = (expr);                         \
        if (err__ != cudaSuccess) return BITNET_A48_ERR_CUDA; \
    } while (0)

// Launch with programmatic dependent launch allowed: the kernel may be made resident while the kernel ahead of it in
// the stream still runs.  Kernels launched this way call a48_pdl_prologue() before they touch memory, which waits
// for that predecessor to complete, so the ordering a plain launch gives is kept and only the launch latency is
// hidden (it is several microseconds per launch in a decode step made of a dozen tiny kernels).
#ifdef __CUDACC__
__device__ __forceinline__ void a48_pdl_prologue() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
template <typename... KArgs, typename... Args>
static inline cudaError_t a48_launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                         Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// Output element type of the contraction kernels for the call in flight on this host thread: 0 = fp32, 1 = bf16
// (round to nearest even of the fp32 result).  Set by bitnet_a48_linear_bf16 around its dispatch, read by the
// launchers, which pass it to their kernels as a parameter.
extern thread_local int a48_y_bf16;
// A residual to add in the decode kernel's epilogue for the call in flight on this host thread (fp32 [M, N], or
// nullptr): Y = R + fp32(acc)*(scale*alpha), the sum a separate elementwise kernel would form.  Set by the block's
// decode step around its last BitLinear; honoured by the single-matrix decode launch only.
extern thread_local const float* a48_decode_residual;
#ifdef __CUDACC__
#include <cuda_bf16.h>
// Stores y as element `index` of an fp32 or a bf16 array.
__device__ __forceinline__ void a48_store_y(float* base, size_t index, float y, int bf16) {
    if (bf16) reinterpret_cast<__nv_bfloat16*>(base)[index] = __float2bfloat16_rn(y);
    else base[index] = y;
}
#endif

static inline bool a48_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline int a48_round_up(int x, int m) { return (x + m - 1) / m * m; }

// 2-bit encoding of a ternary code t in every layout: e = t + 1 (0 -> -1, 1 -> 0, 2 -> +1).
//
// Canonical layout ("l0"): row-major [N][K4] bytes with K4 = ceil(K/4); byte j of
// row n holds k = 4j..4j+3, the lowest two bits first; positions beyond K hold
// code 0.
struct bitnet_a48_weight {
    int N, K;
    int K4;          // bytes per canonical row
    int Np, Kp;      // N rounded up to 256, K rounded up to 256 (tiled layouts)
    unsigned flags;  // BITNET_A48_LAYOUT_* present
    float* alpha_dev;      // fp32 alpha
    double* alpha64_dev;   // float64 alpha (packing only)
    double* partial_dev;   // per-block partial sums of |W|
    uint8_t* l0;           // canonical layout, N*K4 bytes
    uint8_t* gemm;         // tile-major layout, Np*Kp/4 bytes (or NULL)
    uint8_t* decode;       // fragment-major layout (or NULL)
    uint8_t* sparse;       // channel-major layout (or NULL)
    int8_t* i8;            // int8 codes [Np][Kp], zero padded (or NULL)
    uint8_t* trit5;        // five codes per byte, row-major, trit5_row bytes per row (or NULL)
    int trit5_row;         // ceil(K/5) rounded up to 16
    size_t decode_bytes, sparse_bytes;
    // false until the first decode launch: that one is fully ordered after the packing kernels, later ones may
    // start fetching weights while the kernel ahead of them in the stream is still finishing
    mutable bool decode_prefetch_ok;
};

struct bitnet_a48_block {
    bitnet_a48_block_config cfg;
    const bitnet_a48_weight* w[7];  // q k v o gate up down
    const float* g_attn;
    const float* g_ffn;
};

// ---- pack.cu
bitnet_a48_status a48_launch_pack(bitnet_a48_weight* w, const float* W_dev, float eps, cudaStream_t st);
bitnet_a48_status a48_launch_unpack_l0(const bitnet_a48_weight* w, int8_t* codes_dev, cudaStream_t st);
bitnet_a48_status a48_launch_unpack_layout(const bitnet_a48_weight* w, unsigned layout, int8_t* codes_dev,
                                           cudaStream_t st);

// ---- quant.cu
// gain == nullptr: plain quantiser.  gain != nullptr: x is first RMS-normalised
// (eps norm_eps) and multiplied by gain, rounded to fp32, then quantised.
bitnet_a48_status a48_launch_quant_int4(const float* X, int M, int K, float eps, int8_t* codes, float* scale,
                                        const float* gain, float norm_eps, cudaStream_t st);
bitnet_a48_status a48_launch_topk_quant_int8(const float* X, int M, int K, int k, float eps, int8_t* codes,
                                             float* scale, uint32_t* mask_bits, cudaStream_t st);
bool a48_topk_quant_fast_shape(int K);
// bf16 rows in (widened exactly to fp32), otherwise as the fp32 forms
bitnet_a48_status a48_launch_quant_int4_bf16(const uint16_t* X, int M, int K, float eps, int8_t* codes, float* scale,
                                             cudaStream_t st);
bitnet_a48_status a48_launch_topk_quant_int8_bf16(const uint16_t* X, int M, int K, int k, float eps, int8_t* codes,
                                                  float* scale, cudaStream_t st);
bitnet_a48_status a48_launch_quant_int4_add(const float* X, const float* R, float* SUM, int M, int K, float eps,
                                            int8_t* codes, float* scale, const float* gain, float norm_eps,
                                            cudaStream_t st);
bitnet_a48_status a48_launch_topk_quant_int8_glu(const float* gate, const float* up, int M, int K, int k, float eps,
                                                 int8_t* codes, float* scale, cudaStream_t st);
bitnet_a48_status a48_launch_quant_fp4(const float* X, int M, int K, int8_t* codes, float* scale, const float* gain,
                                       float norm_eps, cudaStream_t st);
bitnet_a48_status a48_launch_quant_fp4_add(const float* X, const float* R, float* SUM, int M, int K, int8_t* codes,
                                           float* scale, const float* gain, float norm_eps, cudaStream_t st);
bitnet_a48_status a48_launch_compact_codes(const int8_t* codes, int M, int K, int cap, uint16_t* idx, int8_t* val,
                                           int32_t* count, cudaStream_t st);

// ---- linear_simple.cu
bitnet_a48_status a48_launch_linear_simple(const bitnet_a48_weight* w, const int8_t* codes, const float* scale,
                                           int M, float* Y, int32_t* acc, cudaStream_t st);

// ---- gemm_tcgen05.cu
// ss = true: both operands from shared memory (needs the int8 copy); false: weights expanded into tensor memory.
bool a48_gemm_tcgen05_supported(const bitnet_a48_weight* w, int M, bool ss);
bitnet_a48_status a48_launch_gemm_tcgen05(const bitnet_a48_weight* w, const int8_t* codes, const float* scale, int M,
                                          float* Y, int32_t* acc, bool ss, cudaStream_t st);
// CTA-pair form (one tile of 256 weight rows per two SMs).
bool a48_gemm_pair_supported(const bitnet_a48_weight* w, int M);
bool a48_gemm_pair_preferred(int count, const bitnet_a48_weight* const* ws, int M);
bitnet_a48_status a48_launch_gemm_pair(const bitnet_a48_weight* w, const int8_t* codes, const float* scale, int M,
                                       float* Y, int32_t* acc, cudaStream_t st);
// Up to four weight matrices with one K on the same codes in one launch (tile-major layout, tensor-memory operand).
bool a48_gemm_tcgen05_multi_supported(int count, const bitnet_a48_weight* const* ws, int M);
bitnet_a48_status a48_launch_gemm_tcgen05_multi(int count, const bitnet_a48_weight* const* ws, const int8_t* codes,
                                                const float* scale, int M, float* const* Y, cudaStream_t st);
bitnet_a48_status a48_read_kernel_status(unsigned int words_host[4]);

// ---- decode.cu
bool a48_decode_supported(const bitnet_a48_weight* w, int M);
bool a48_decode_sparse_supported(const bitnet_a48_weight* w, int M);
size_t a48_decode_workspace_bytes(const bitnet_a48_weight* w, int M);
size_t a48_decode_sparse_workspace_bytes(const bitnet_a48_weight* w, int M);
bitnet_a48_status a48_launch_decode(const bitnet_a48_weight* w, const int8_t* codes, const float* scale, int M,
                                    float* Y, int32_t* acc, void* ws, size_t ws_bytes, cudaStream_t st);
// Several matrices of one K (all with the decode layout) on the same token codes in one launch, e.g. q, k and v.
size_t a48_decode_multi_workspace_bytes(int count, const bitnet_a48_weight* const* w, int M);
bitnet_a48_status a48_launch_decode_multi(int count, const bitnet_a48_weight* const* w, const int8_t* codes,
                                          const float* scale, int M, float* const* Y, int32_t* const* acc, void* ws,
                                          size_t ws_bytes, cudaStream_t st);
bitnet_a48_status a48_read_decode_status(unsigned int words_host[4]);
bitnet_a48_status a48_launch_decode_sparse(const bitnet_a48_weight* w, const int8_t* codes, const float* scale,
                                           int M, float* Y, int32_t* acc, void* ws, size_t ws_bytes,
                                           cudaStream_t st);

// ---- attn_lowbit.cu (Section 3, low-bit attention)
size_t a48_kv_cache_bytes(int B, int nh, int cap, int hd, int bits);
bitnet_a48_status a48_launch_rope_quant_cache(float* q, const float* k, const float* v, const float2* table, double base,
                                              int B, int T, int nh, int hd, int pos0, int cap, int q_bits, int kv_bits,
                                              float eps, void* kcache, void* vcache, float* dq_k, float* dq_v,
                                              cudaStream_t st);
bitnet_a48_status a48_launch_dequant_prefix(const void* kcache, const void* vcache, int B, int nh, int hd, int pos0, int cap,
                                            int rows, int kv_bits, float* dq_k, float* dq_v, cudaStream_t st);
bitnet_a48_status a48_launch_attn_row_lowbit(const float* q, const void* kcache, const void* vcache, int B, int T, int nh,
                                             int hd, int pos0, int cap, int kv_bits, float* out, cudaStream_t st);

// ---- decode_trit5.cu
bool a48_decode_trit5_supported(const bitnet_a48_weight* w, int M);
bitnet_a48_status a48_launch_decode_trit5(const bitnet_a48_weight* w, const int8_t* codes, const float* scale, int M, float* Y,
                                          int32_t* acc, cudaStream_t st);

// ---- attn_tcgen05.cu (prefill attention on the tensor cores, operands split into bf16 parts)
bool a48_attn_tc_supported(int hd);
size_t a48_attn_tc_workspace_bytes(int B, int nh, int hd, int T, int n_keys);
bitnet_a48_status a48_launch_attn_tc(const float* q, const float* kcache, const float* vcache, int B, int T, int nh, int hd,
                                     int pos0, int cap, float* out, void* ws, cudaStream_t st);
bitnet_a48_status a48_read_attn_status(unsigned int words_host[4]);

// ---- block.cu
size_t a48_block_workspace_bytes(const bitnet_a48_block* blk, int B, int T);
bitnet_a48_status a48_block_forward(const bitnet_a48_block* blk, const float* X, int B, int T, int pos0,
                                    float* kcache, float* vcache, float* Y, void* ws, size_t ws_bytes,
                                    cudaStream_t st);
