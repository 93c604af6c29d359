/*
 * bitnet_a48.h — C ABI of the B200 (sm_100a) BitLinear forward of BitNet a4.8
 * (arXiv 2411.04965).
 *
 * Conventions shared by every call
 *   - Pointers named *_dev are DEVICE memory owned by the caller and must be
 *     16-byte aligned (BITNET_A48_ERR_ALIGNMENT otherwise).  Pointers named
 *     *_host are host memory.  The only library-owned memory sits behind the
 *     opaque weight / block handles and is released by the matching *_free.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls enqueue work on it and return without synchronising unless the
 *     comment of the call says otherwise.
 *   - Matrices are row-major.  Activations are X[M,K] (M tokens, K features);
 *     weights are W[N,K] (N output features), because the paper writes
 *     Y = Q_a(X) · Q_w(W)^T (Eq. 1, Eq. 6).
 *   - No call aborts or throws: every failure is a status code, and arguments
 *     are validated on the host before anything is launched.  Inputs must be
 *     finite; on NaN/Inf the codes are unspecified but no fault occurs.
 *   - There is no CPU fallback: without a CUDA device every compute call
 *     returns BITNET_A48_ERR_CUDA.
 */
#ifndef BITNET_A48_H
#define BITNET_A48_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    BITNET_A48_OK = 0,
    BITNET_A48_ERR_INVALID_ARG = 1, /* null pointer, k out of range, bad enum */
    BITNET_A48_ERR_SHAPE = 2,       /* non-positive or unsupported extent */
    BITNET_A48_ERR_ALIGNMENT = 3,   /* a device pointer is not 16-byte aligned */
    BITNET_A48_ERR_UNSUPPORTED = 4, /* requested kernel cannot run this shape / layout missing */
    BITNET_A48_ERR_CUDA = 5,        /* a CUDA runtime call failed */
    BITNET_A48_ERR_TIMEOUT = 6,     /* a bounded in-kernel wait gave up (see bitnet_a48_kernel_status) */
    BITNET_A48_ERR_NOMEM = 7,       /* workspace too small or allocation failed */
    BITNET_A48_ERR_LIMIT = 8        /* size beyond a documented fixed maximum */
} bitnet_a48_status;

/* Which activation quantiser produced the codes given to bitnet_a48_linear. */
typedef enum {
    BITNET_A48_ACT_INT4 = 0,      /* Eq. 7: codes in [-8,7], scale = beta/sqrt(7) */
    BITNET_A48_ACT_TOPK_INT8 = 1, /* Eq. 1+3: codes in [-127,127], zero where masked, scale = gamma/127 */
    BITNET_A48_ACT_FP4 = 2        /* Eq. 8-9: grid codes in {0,±1,±2,±3,±4,±6,±8,±12}, scale = |x|max/12 */
} bitnet_a48_act;

/* Packed layouts a weight handle can carry (bit mask for pack_ternary). */
#define BITNET_A48_LAYOUT_GEMM 1u   /* tile-major, for the tcgen05 prefill kernel */
#define BITNET_A48_LAYOUT_DECODE 2u /* fragment-major, for the weight-streaming decode kernel */
#define BITNET_A48_LAYOUT_SPARSE 4u /* channel-major, for the zero-skipping batch-1 decode kernel */
#define BITNET_A48_LAYOUT_ALL 7u
/* One int8 code per weight (4x the packed size); only the shared-memory-operand
 * variant of the tensor-core kernel reads it.  Not part of LAYOUT_ALL. */
#define BITNET_A48_LAYOUT_I8 8u
/* Five codes per byte (b = sum (t_i + 1) 3^i, 1.6 bits per weight: the "1.58-bit" of Section 1 rounded up to whole
 * bytes), row-major, rows padded to 16 bytes; read by the BITNET_A48_ALGO_DECODE_TRIT5 kernel.  Not part of LAYOUT_ALL. */
#define BITNET_A48_LAYOUT_TRIT5 16u

/* Kernel selection for bitnet_a48_linear_ex (tests and benchmarks force one). */
typedef enum {
    BITNET_A48_ALGO_AUTO = 0,
    BITNET_A48_ALGO_SIMPLE = 1,       /* tiled dp4a kernel, any shape; the in-tree cross-check */
    BITNET_A48_ALGO_GEMM_TCGEN05 = 2, /* prefill: tcgen05 kind::i8, int32 accumulators in TMEM */
    BITNET_A48_ALGO_DECODE = 3,       /* M <= 8: streams every weight byte once */
    BITNET_A48_ALGO_DECODE_SPARSE = 4, /* M == 1: fetches only channels whose code is non-zero */
    BITNET_A48_ALGO_GEMM_TCGEN05_I8 = 5, /* comparison variant: int8 weight copy staged through shared memory */
    BITNET_A48_ALGO_GEMM_TCGEN05_PAIR = 6, /* tcgen05 cta_group::2: two SMs per tile of 256 weight rows */
    BITNET_A48_ALGO_DECODE_TRIT5 = 7  /* M <= 8 over the five-codes-per-byte layout (a fifth fewer weight bytes) */
} bitnet_a48_algo;

typedef struct bitnet_a48_weight bitnet_a48_weight; /* packed ternary matrix + alpha + N, K */
typedef struct bitnet_a48_block bitnet_a48_block;   /* one transformer block: 7 weights, 2 gains, dims */

const char* bitnet_a48_status_string(bitnet_a48_status s);

/* ---------------------------------------------------------------------------
 * Weight quantiser, Eq. 2:  Q_w(W) = alpha·RoundClip(W/(alpha+eps), -1, 1),
 * alpha = mean|W| over the whole matrix; RoundClip is Eq. 4 with round-half-to-
 * even.  Reads W_dev (fp32 [N,K]), stores the codes at 2 bits per weight in the
 * layouts named by layout_flags (a canonical row-major layout is always kept)
 * and alpha (computed in float64, kept as fp32) in device memory.
 * Allocates the handle's device buffers (cudaMalloc; may synchronise), then
 * enqueues the packing kernels on `stream`.  *out is owned by the caller and
 * released with bitnet_a48_weight_free.  K < 2^24 and N*K < 2^40.
 */
bitnet_a48_status bitnet_a48_pack_ternary(const float* W_dev, int N, int K, float eps, unsigned layout_flags,
                                          bitnet_a48_weight** out, void* stream);

/* Expands the canonical packed layout back to one int8 code per weight
 * (codes_dev [N,K], values in {-1,0,1}) and copies alpha to *alpha_host.
 * Either output may be NULL.  Synchronises `stream`. */
bitnet_a48_status bitnet_a48_weight_unpack(const bitnet_a48_weight* w, int8_t* codes_dev, float* alpha_host,
                                           void* stream);
/* Expands one of the optional layouts (a single BITNET_A48_LAYOUT_* bit) to
 * int8 codes, for checking that every layout holds the same matrix. */
bitnet_a48_status bitnet_a48_weight_unpack_layout(const bitnet_a48_weight* w, unsigned layout, int8_t* codes_dev,
                                                  void* stream);
bitnet_a48_status bitnet_a48_weight_dims(const bitnet_a48_weight* w, int* N, int* K, unsigned* layout_flags);
/* Bytes of packed weight data a kernel reads for this matrix (N*K/4 rounded up per row). */
size_t bitnet_a48_weight_packed_bytes(const bitnet_a48_weight* w);
/* Bytes of one optional layout (a single BITNET_A48_LAYOUT_* bit) as stored, 0 if the handle does not carry it. */
size_t bitnet_a48_weight_layout_bytes(const bitnet_a48_weight* w, unsigned layout);
void bitnet_a48_weight_free(bitnet_a48_weight* w);

/* ---------------------------------------------------------------------------
 * Activation quantiser for the inputs of attention and FFN, Eq. 7:
 *   per token m: beta = mean_k|x|;  codes = RoundClip(sqrt7/(beta+eps)·x, -8, 7);
 *   scale[m] = beta/sqrt7.
 * X_dev fp32 [M,K] -> codes_dev int8 [M,K] (one code per byte), scale_dev fp32 [M].
 * The mean and the multiply are evaluated in float64.  K <= 2^20.
 */
bitnet_a48_status bitnet_a48_quant_int4(const float* X_dev, int M, int K, float eps, int8_t* codes_dev,
                                        float* scale_dev, void* stream);

/* ---------------------------------------------------------------------------
 * Sparsify-then-quantise for the intermediate states, Eq. 1 and 3:
 *   per token m: gamma = max_k|x|; q = RoundClip(127/(gamma+eps)·x, -128, 127);
 *   mask = the k largest |x| (ties: lowest index first; -0 ties +0);
 *   codes = q·mask; scale[m] = gamma/127.
 * mask_bits_dev is NULL or uint32 [M, ceil(K/32)], bit (j%32) of word j/32 = mask of feature j.
 * 1 <= k <= K <= 2^20.
 */
bitnet_a48_status bitnet_a48_topk_quant_int8(const float* X_dev, int M, int K, int k, float eps,
                                             int8_t* codes_dev, float* scale_dev, uint32_t* mask_bits_dev,
                                             void* stream);

/* Compacted form of code rows for consumers that skip masked channels (Section 2.1: the masked entries of
 * Eq. 1 contribute nothing to the contraction; a channel is skipped iff its code is 0, which also covers
 * kept entries that quantise to 0).  For every row m of codes_dev [M, K] (int8, row-major): the channels
 * with a non-zero code in ascending order, idx_dev [M, cap] (uint16 channel index) and val_dev [M, cap]
 * (the code), and count_dev[m] = the number of non-zero codes of the row.  Only the first min(count, cap)
 * entries of a row are written; count > cap tells the caller that the row did not fit (cap >= k always fits
 * the output of bitnet_a48_topk_quant_int8).  All buffers caller-owned device memory, 16-byte aligned;
 * K <= 65535; asynchronous on `stream`. */
bitnet_a48_status bitnet_a48_compact_codes(const int8_t* codes_dev, int M, int K, int cap, uint16_t* idx_dev,
                                           int8_t* val_dev, int32_t* count_dev, void* stream);

/* FP4 (E2M1) MinMax quantiser, Eq. 8-9: per token, 2^b = 12/|x|max, step =
 * 2^(max(floor(log2|x·2^b|),1)-1), code = step·round(x·2^b/step) (an integer in
 * {0,±1,±2,±3,±4,±6,±8,±12}), scale[m] = |x|max/12.  Same shapes as quant_int4. */
bitnet_a48_status bitnet_a48_quant_fp4(const float* X_dev, int M, int K, int8_t* codes_dev, float* scale_dev,
                                       void* stream);

/* ---------------------------------------------------------------------------
 * BitLinear contraction and rescale, Eq. 1 / Eq. 6:
 *   acc[m,n] = sum_k codes[m,k]·t[n,k]   (exact, int32)
 *   Y[m,n]   = fp32(acc[m,n]) · (scale[m] · alpha)
 * codes_dev int8 [M,K], scale_dev fp32 [M], Y_dev fp32 [M,N]; acc_dev is NULL or
 * int32 [M,N] (the raw accumulators, for parity checks).  `kind` tells which
 * quantiser made the codes (the result does not depend on it; for top-K inputs at
 * M == 1 it lets the call take the zero-skipping kernel when the handle carries the
 * SPARSE layout but not the DECODE one - with both present the dense streaming
 * kernel is the faster of the two at model shapes and is taken).
 * workspace_dev: at least bitnet_a48_linear_workspace_bytes(w, M) bytes, or NULL
 * when that is 0.  The decode kernel (M <= 8) adds the partial sums of tiles that
 * two CTAs share into this scratch: it must be zero-filled before its first use
 * (cudaMemset), every call leaves it zero-filled again, and two calls that may
 * overlap on the device must not share it.  Nothing is allocated and nothing
 * synchronises.
 */
bitnet_a48_status bitnet_a48_linear(const bitnet_a48_weight* w, const int8_t* codes_dev, const float* scale_dev,
                                    int M, bitnet_a48_act kind, float* Y_dev, int32_t* acc_dev,
                                    void* workspace_dev, size_t workspace_bytes, void* stream);
/* Same, with the kernel chosen by the caller.  BITNET_A48_ERR_UNSUPPORTED when
 * that kernel cannot run the shape or the handle lacks its layout. */
bitnet_a48_status bitnet_a48_linear_ex(const bitnet_a48_weight* w, const int8_t* codes_dev, const float* scale_dev,
                                       int M, bitnet_a48_act kind, bitnet_a48_algo algo, float* Y_dev,
                                       int32_t* acc_dev, void* workspace_dev, size_t workspace_bytes, void* stream);
size_t bitnet_a48_linear_workspace_bytes(const bitnet_a48_weight* w, int M);

/* ---------------------------------------------------------------------------
 * bf16 activations at the boundary (Section 1: the activations around the 4- and 8-bit codes are what is left to move
 * once the weights are 1.58-bit; bf16 halves those bytes).  The quantisers read bf16 rows, widened exactly to fp32
 * and then quantised as Eq. 7 / Eq. 1 + 3 say (same codes and scales as the fp32 entry points give on the widened
 * values); the contraction writes bf16(Y) = round-to-nearest-even of the fp32 result of Eq. 1 / Eq. 6.
 * X_bf16_dev uint16 [M, K] (bf16 bit patterns), K a multiple of 8 and at most 12288; Y_bf16_dev uint16 [M, N].
 * bitnet_a48_linear_bf16 picks its kernel like bitnet_a48_linear (decode for M <= 8, tensor-core forms above). */
bitnet_a48_status bitnet_a48_quant_int4_bf16(const uint16_t* X_bf16_dev, int M, int K, float eps, int8_t* codes_dev,
                                             float* scale_dev, void* stream);
bitnet_a48_status bitnet_a48_topk_quant_int8_bf16(const uint16_t* X_bf16_dev, int M, int K, int k, float eps,
                                                  int8_t* codes_dev, float* scale_dev, void* stream);
bitnet_a48_status bitnet_a48_linear_bf16(const bitnet_a48_weight* w, const int8_t* codes_dev, const float* scale_dev,
                                         int M, bitnet_a48_act kind, uint16_t* Y_bf16_dev, void* workspace_dev,
                                         size_t workspace_bytes, void* stream);

/* Several BitLinears on the SAME activation codes (Eq. 6: q, k and v share the attention input; gate and up
 * share the FFN input): Y_dev[j] = BitLinear(weights[j]) for j < count, all weights with the same K.
 * For M <= 8 and count <= 4 with the DECODE layout this is one launch that streams the matrices as one
 * sequence of tiles (a launch costs more than the HBM time of one 7B-shape matrix); for 9..383 tokens,
 * count <= 4 and the GEMM layout it is one launch of the tensor-core kernel over the tiles of all matrices;
 * otherwise it is `count` calls of bitnet_a48_linear one after the other.  Results are identical to separate
 * calls.
 * workspace_dev: bitnet_a48_linear_multi_workspace_bytes bytes, zero-filled before first use, left zero-filled
 * (same contract as bitnet_a48_linear). */
bitnet_a48_status bitnet_a48_linear_multi(int count, const bitnet_a48_weight* const weights[], const int8_t* codes_dev,
                                          const float* scale_dev, int M, bitnet_a48_act kind, float* const Y_dev[],
                                          void* workspace_dev, size_t workspace_bytes, void* stream);
size_t bitnet_a48_linear_multi_workspace_bytes(int count, const bitnet_a48_weight* const weights[], int M);

/* Decode BitLinear (M <= 8 tokens, weights packed with BITNET_A48_LAYOUT_DECODE) for callers that cannot
 * allocate device memory.  (The paper has no counterpart: this is a convenience of this library.)
 * Some hosts of this code may not call cudaMalloc or any allocator at all once they are running: a plugin
 * inside a serving process whose memory is handed out once at start-up and then frozen, a real-time loop
 * that must not take the allocator's locks, a call made while a stream is being captured.  Such callers
 * cannot give bitnet_a48_linear the scratch it asks for.  Here the scratch is an array inside the library
 * image (1 MiB on every GPU that loads the library, until the process exits); the caller passes only the
 * inputs and the output, and the call performs no cudaMalloc, cudaFree or other allocating call.
 *   - Result: identical, bit for bit, to bitnet_a48_linear_ex(..., BITNET_A48_ALGO_DECODE, ...).
 *   - Limits: N <= 16384 output features (BITNET_A48_ERR_LIMIT beyond), M <= 8 and the DECODE layout
 *     (BITNET_A48_ERR_UNSUPPORTED otherwise).
 *   - The first call on each device looks up the array's device address (with that device current);
 *     make that first call outside any stream capture.
 *   - All calls on a device share the one array.  Each call clears the part it uses on `stream` and then
 *     runs the kernel on `stream`; two calls that can overlap on the GPU (different streams) race on it
 *     and give wrong results - serialise them.
 * Enqueues on `stream` and returns without synchronising. */
bitnet_a48_status bitnet_a48_linear_decode_static(const bitnet_a48_weight* w, const int8_t* codes_dev,
                                                  const float* scale_dev, int M, float* Y_dev, void* stream);

/* One BitLinear end to end from HOST buffers (Eq. 6 with kind INT4, Eq. 1 with
 * kind TOPK_INT8 and top-k count k): copies X_host fp32 [M,K] to the device,
 * quantises, contracts, rescales and copies Y back to Y_host fp32 [M,N].
 * X_host / Y_host should be page-locked for full copy speed.  workspace_dev
 * must hold bitnet_a48_bitlinear_host_workspace_bytes(w, M) bytes.
 * Synchronises `stream` before returning. */
bitnet_a48_status bitnet_a48_bitlinear_host(const bitnet_a48_weight* w, const float* X_host, int M,
                                            bitnet_a48_act kind, int k, float eps, float* Y_host,
                                            void* workspace_dev, size_t workspace_bytes, void* stream);
/* The same without the final synchronisation: everything is enqueued on `stream`, Y_host is valid once the
 * stream has been synchronised.  Calls on different streams (each with its own workspace, page-locked host
 * buffers) overlap their host-to-device copy, compute and device-to-host copy. */
bitnet_a48_status bitnet_a48_bitlinear_host_async(const bitnet_a48_weight* w, const float* X_host, int M,
                                                  bitnet_a48_act kind, int k, float eps, float* Y_host,
                                                  void* workspace_dev, size_t workspace_bytes, void* stream);
size_t bitnet_a48_bitlinear_host_workspace_bytes(const bitnet_a48_weight* w, int M);

/* ---------------------------------------------------------------------------
 * Transformer block in the BitNet b1.58 layout with every projection a
 * BitLinear (Section 2.1): INT4 inputs for q,k,v and gate,up (Eq. 6-7), top-K +
 * INT8 inputs for the attention output and FFN down projections (Eq. 1, 3),
 * ReLU²GLU (Eq. 5).  Readings where the paper is silent: pre-RMSNorm with
 * gains, RoPE on (i, i+head_dim/2) pairs, causal softmax attention in fp32,
 * fp32 KV cache laid out [B][n_heads][ctx_cap][head_dim], no biases.
 */
typedef struct {
    int hidden, n_heads, ffn;
    int k_o, k_down;   /* top-k counts for the o_proj and down_proj inputs */
    int ctx_cap;       /* positions each KV-cache row can hold */
    float norm_eps, quant_eps, rope_base;
    /* Floating-point variant (Section 2.3, sentence before Eq. 8): non-zero = the inputs of q/k/v, of the attention
     * output projection (then without top-K) and of gate/up are quantised to FP4 (Eq. 8-9); the down projection's
     * input stays top-K + INT8.  0 = the integer model. */
    int act_fp4;
    /* Low-bit attention (Section 3, low-bit attention paragraph): post-RoPE absmax quantisation per head vector.
     * q_bits: 0 (fp32 queries) or 4.  kv_bits: 0 (fp32 cache), 4 or 3; with 3 the position-0 (bos) heads keep 4 bits.
     * With kv_bits != 0 the caches passed to bitnet_a48_block_forward are packed (bitnet_a48_kv_cache_bytes). */
    int q_bits, kv_bits;
} bitnet_a48_block_config;

/* weights: q, k, v, o [hidden,hidden], gate, up [ffn,hidden], down [hidden,ffn] in this order.
 * The block borrows the weight handles and the gain vectors (fp32 [hidden], device);
 * they must outlive it. */
bitnet_a48_status bitnet_a48_block_create(const bitnet_a48_block_config* cfg, const bitnet_a48_weight* const weights[7],
                                          const float* gain_attn_dev, const float* gain_ffn_dev, bitnet_a48_block** out);
void bitnet_a48_block_free(bitnet_a48_block* blk);
/* Bytes of ONE cache buffer (keys or values) for B sequences of ctx_cap positions: B*n_heads*ctx_cap*head_dim*4 with
 * kv_bits == 0; with kv_bits 4 or 3 the packed layout of Section 3's low-bit attention - per head vector a
 * little-endian bit stream of kv_bits-bit unsigned codes (head_dim padded to a multiple of 32 entries), then one
 * fp32 scale per head vector, then (3-bit only) the 4-bit codes of position 0.  The caller allocates it (16-byte
 * aligned); its contents are written by bitnet_a48_block_forward only. */
size_t bitnet_a48_kv_cache_bytes(const bitnet_a48_block* blk, int B);
size_t bitnet_a48_block_workspace_bytes(const bitnet_a48_block* blk, int B, int T);
/* X_dev fp32 [B*T, hidden] -> Y_dev fp32 [B*T, hidden].  Tokens of batch b sit at
 * positions pos0..pos0+T-1; their keys/values are written into the caches at
 * those positions and attention reads positions 0..own position.  The caches
 * may be NULL only when pos0 == 0 and T is the whole sequence (keys/values then
 * live in the workspace).  With kv_bits != 0 the caches are packed buffers of bitnet_a48_kv_cache_bytes bytes
 * (passed through the same pointers), head_dim <= 128 and ctx_cap a multiple of 4; a call of more than 8 tokens
 * per sequence reads the cached positions through fp32 copies in the workspace (whose size then grows with ctx_cap);
 * q_bits != 0 needs kv_bits != 0.
 * All kernels run on `stream`; nothing synchronises. */
bitnet_a48_status bitnet_a48_block_forward(const bitnet_a48_block* blk, const float* X_dev, int B, int T, int pos0,
                                           float* kcache_dev, float* vcache_dev, float* Y_dev, void* workspace_dev,
                                           size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------
 * The attention of the block on its own, for a prefill (Section 2.1: between the q/k/v BitLinears and the output
 * BitLinear the block keeps the ordinary causal softmax attention; bitnet_a48_block_forward runs this same kernel
 * for more than 8 tokens per sequence).  out[t] = sum_j softmax_j(q[t] . k[j] / sqrt(head_dim)) v[j] per head, where
 * token t of sequence b sits at position pos0 + t and sees positions 0 .. pos0 + t of that sequence's cache.
 *   q_dev       fp32 [B*T, n_heads*head_dim], already rotated (read only)
 *   kcache_dev, vcache_dev  fp32 [B, n_heads, ctx_cap, head_dim]; positions 0 .. pos0+T-1 are read, nothing is written
 *   out_dev     fp32 [B*T, n_heads*head_dim]
 *   workspace_dev  bitnet_a48_attention_prefill_workspace_bytes(B, n_heads, head_dim, T, pos0 + T) bytes, 16-byte
 *               aligned (it receives the operands split into bf16 parts; no need to clear it)
 * 1 <= head_dim <= 128 (BITNET_A48_ERR_UNSUPPORTED above), pos0 + T <= ctx_cap, B and n_heads at most 65535.  The
 * contractions run on the tensor cores with every fp32 operand split into three bf16 parts, which keeps the result
 * within fp32 rounding of the definition (about 4e-8 |score| relative to the largest output of a row).  All
 * kernels run on `stream`; nothing synchronises; a bounded wait that gives up reports through
 * bitnet_a48_kernel_status. */
size_t bitnet_a48_attention_prefill_workspace_bytes(int B, int n_heads, int head_dim, int T, int n_keys);
bitnet_a48_status bitnet_a48_attention_prefill(const float* q_dev, const float* kcache_dev, const float* vcache_dev, int B,
                                               int T, int n_heads, int head_dim, int pos0, int ctx_cap, float* out_dev,
                                               void* workspace_dev, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------
 * Feed-forward sub-layer for M <= 8 tokens with the gate projection first (Section 2.1, paragraph after Eq. 5;
 * Section 3 "Sparsity"): INT4 input (Eq. 7) -> gate BitLinear (Eq. 6) -> up BitLinear only for the output channels n
 * with ReLU²(gate[m, n]) != 0 for some token m (the other rows of W_up are not read) -> Eq. 5 -> top-k + INT8
 * (Eq. 1, 3) -> down BitLinear.  The result equals the dense evaluation of the same sub-layer.
 * gate, up: [ffn, hidden]; down: [hidden, ffn]; hidden a multiple of 64.  X_dev fp32 [M, hidden] is the normalised
 * input; Y_dev fp32 [M, hidden].  inter_dev: NULL or fp32 [M, ffn], receives Eq. 5's product (0 where skipped).
 * rows_fetched_dev: NULL or one int32 that receives the number of rows of W_up that were read.
 * workspace_dev: bitnet_a48_ffn_gate_first_workspace_bytes bytes.  Asynchronous on `stream`; allocates nothing. */
bitnet_a48_status bitnet_a48_ffn_gate_first(const bitnet_a48_weight* gate, const bitnet_a48_weight* up,
                                            const bitnet_a48_weight* down, const float* X_dev, int M, int k_down, float eps,
                                            float* Y_dev, float* inter_dev, int32_t* rows_fetched_dev, void* workspace_dev,
                                            size_t workspace_bytes, void* stream);
/* The same sub-layer evaluated densely (Eq. 5-7, Eq. 1, 3): gate and up as one fused launch over every row.  Same
 * shapes, limits and workspace as bitnet_a48_ffn_gate_first (ffn a multiple of 4 and at most 12288); it is the
 * reference point for what gate-first evaluation saves. */
bitnet_a48_status bitnet_a48_ffn_dense(const bitnet_a48_weight* gate, const bitnet_a48_weight* up,
                                       const bitnet_a48_weight* down, const float* X_dev, int M, int k_down, float eps,
                                       float* Y_dev, void* workspace_dev, size_t workspace_bytes, void* stream);
size_t bitnet_a48_ffn_gate_first_workspace_bytes(const bitnet_a48_weight* gate, const bitnet_a48_weight* up,
                                                 const bitnet_a48_weight* down, int M);

/* Reads the device-side status words that kernels with bounded waits set when
 * a wait gives up (0 = no kernel has reported anything) and clears them.
 * Synchronises the device.  words_host receives 4 values: [0] error code,
 * [1] barrier id, [2] block index, [3] iteration. */
bitnet_a48_status bitnet_a48_kernel_status(unsigned int words_host[4]);

#ifdef __cplusplus
}
#endif
#endif /* BITNET_A48_H */
