// extern "C" entry points: argument validation, handle management, dispatch.
#include <new>

#include "internal.h"

thread_local int a48_y_bf16 = 0;
thread_local const float* a48_decode_residual = nullptr;

namespace {

constexpr int kMaxFeatures = 1 << 20;

bool have_device() {
    static int cached = -1;  // the answer cannot change within a process
    if (cached < 0) {
        int n = 0;
        cached = (cudaGetDeviceCount(&n) == cudaSuccess && n > 0) ? 1 : 0;
        if (!cached) cudaGetLastError();
    }
    return cached == 1;
}

void free_weight_buffers(bitnet_a48_weight* w) {
    cudaFree(w->alpha_dev);
    cudaFree(w->alpha64_dev);
    cudaFree(w->partial_dev);
    cudaFree(w->l0);
    cudaFree(w->gemm);
    cudaFree(w->decode);
    cudaFree(w->sparse);
    cudaFree(w->i8);
    cudaFree(w->trit5);
}

bitnet_a48_status check_act_args(const void* X, int M, int K, const void* codes, const void* scale) {
    if (!X || !codes || !scale) return BITNET_A48_ERR_INVALID_ARG;
    if (M <= 0 || K <= 0 || K > kMaxFeatures) return BITNET_A48_ERR_SHAPE;
    if (!a48_aligned16(X) || !a48_aligned16(codes) || !a48_aligned16(scale)) return BITNET_A48_ERR_ALIGNMENT;
    if (!have_device()) return BITNET_A48_ERR_CUDA;
    return BITNET_A48_OK;
}

}  // namespace

extern "C" {

const char* bitnet_a48_status_string(bitnet_a48_status s) {
    switch (s) {
        case BITNET_A48_OK: return "ok";
        case BITNET_A48_ERR_INVALID_ARG: return "invalid argument";
        case BITNET_A48_ERR_SHAPE: return "unsupported shape";
        case BITNET_A48_ERR_ALIGNMENT: return "device pointer not 16-byte aligned";
        case BITNET_A48_ERR_UNSUPPORTED: return "kernel or layout not available for this call";
        case BITNET_A48_ERR_CUDA: return "CUDA runtime error";
        case BITNET_A48_ERR_TIMEOUT: return "bounded in-kernel wait gave up";
        case BITNET_A48_ERR_NOMEM: return "workspace too small or allocation failed";
        case BITNET_A48_ERR_LIMIT: return "size beyond a fixed maximum";
    }
    return "unknown status";
}

bitnet_a48_status bitnet_a48_pack_ternary(const float* W_dev, int N, int K, float eps, unsigned layout_flags,
                                          bitnet_a48_weight** out, void* stream) {
    if (!W_dev || !out || (layout_flags & ~(BITNET_A48_LAYOUT_ALL | BITNET_A48_LAYOUT_I8 | BITNET_A48_LAYOUT_TRIT5)) || !(eps >= 0.f)) return BITNET_A48_ERR_INVALID_ARG;
    if (N <= 0 || K <= 0 || K >= (1 << 24) || (size_t)N * (size_t)K >= ((size_t)1 << 40)) return BITNET_A48_ERR_SHAPE;
    if (!a48_aligned16(W_dev)) return BITNET_A48_ERR_ALIGNMENT;
    if (!have_device()) return BITNET_A48_ERR_CUDA;
    bitnet_a48_weight* w = new (std::nothrow) bitnet_a48_weight();
    if (!w) return BITNET_A48_ERR_NOMEM;
    w->N = N;
    w->K = K;
    w->K4 = (K + 3) / 4;
    w->Np = a48_round_up(N, 256);
    w->Kp = a48_round_up(K, 256);
    w->flags = layout_flags;
    w->decode_bytes = (size_t)w->Np * w->Kp / 4;
    w->sparse_bytes = (size_t)K * w->Np / 4;
    w->trit5_row = a48_round_up((K + 4) / 5, 16);
    bool ok = cudaMalloc(&w->alpha_dev, 16) == cudaSuccess && cudaMalloc(&w->alpha64_dev, 16) == cudaSuccess &&
              cudaMalloc(&w->partial_dev, 1024 * sizeof(double)) == cudaSuccess &&
              cudaMalloc(&w->l0, (size_t)N * w->K4) == cudaSuccess;
    if (ok && (layout_flags & BITNET_A48_LAYOUT_GEMM)) ok = cudaMalloc(&w->gemm, (size_t)w->Np * w->Kp / 4) == cudaSuccess;
    if (ok && (layout_flags & BITNET_A48_LAYOUT_DECODE)) ok = cudaMalloc(&w->decode, w->decode_bytes) == cudaSuccess;
    if (ok && (layout_flags & BITNET_A48_LAYOUT_SPARSE)) ok = cudaMalloc(&w->sparse, w->sparse_bytes) == cudaSuccess;
    if (ok && (layout_flags & BITNET_A48_LAYOUT_I8)) ok = cudaMalloc(&w->i8, (size_t)w->Np * w->Kp) == cudaSuccess;
    if (ok && (layout_flags & BITNET_A48_LAYOUT_TRIT5)) ok = cudaMalloc(&w->trit5, (size_t)N * w->trit5_row) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        free_weight_buffers(w);
        delete w;
        return BITNET_A48_ERR_NOMEM;
    }
    bitnet_a48_status s = a48_launch_pack(w, W_dev, eps, (cudaStream_t)stream);
    if (s != BITNET_A48_OK) {
        free_weight_buffers(w);
        delete w;
        return s;
    }
    *out = w;
    return BITNET_A48_OK;
}

bitnet_a48_status bitnet_a48_weight_unpack(const bitnet_a48_weight* w, int8_t* codes_dev, float* alpha_host,
                                           void* stream) {
    if (!w) return BITNET_A48_ERR_INVALID_ARG;
    if (codes_dev) {
        bitnet_a48_status s = a48_launch_unpack_l0(w, codes_dev, (cudaStream_t)stream);
        if (s != BITNET_A48_OK) return s;
    }
    if (alpha_host)
        A48_CUDA_TRY(cudaMemcpyAsync(alpha_host, w->alpha_dev, sizeof(float), cudaMemcpyDeviceToHost,
                                     (cudaStream_t)stream));
    A48_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    return BITNET_A48_OK;
}

bitnet_a48_status bitnet_a48_weight_unpack_layout(const bitnet_a48_weight* w, unsigned layout, int8_t* codes_dev,
                                                  void* stream) {
    if (!w || !codes_dev) return BITNET_A48_ERR_INVALID_ARG;
    return a48_launch_unpack_layout(w, layout, codes_dev, (cudaStream_t)stream);
}

bitnet_a48_status bitnet_a48_weight_dims(const bitnet_a48_weight* w, int* N, int* K, unsigned* layout_flags) {
    if (!w) return BITNET_A48_ERR_INVALID_ARG;
    if (N) *N = w->N;
    if (K) *K = w->K;
    if (layout_flags) *layout_flags = w->flags;
    return BITNET_A48_OK;
}

size_t bitnet_a48_weight_packed_bytes(const bitnet_a48_weight* w) { return w ? (size_t)w->N * w->K4 : 0; }

size_t bitnet_a48_weight_layout_bytes(const bitnet_a48_weight* w, unsigned layout) {
    if (!w) return 0;
    switch (layout) {
        case BITNET_A48_LAYOUT_GEMM: return w->gemm ? (size_t)w->Np * w->Kp / 4 : 0;
        case BITNET_A48_LAYOUT_DECODE: return w->decode ? w->decode_bytes : 0;
        case BITNET_A48_LAYOUT_SPARSE: return w->sparse ? w->sparse_bytes : 0;
        case BITNET_A48_LAYOUT_I8: return w->i8 ? (size_t)w->Np * w->Kp : 0;
        case BITNET_A48_LAYOUT_TRIT5: return w->trit5 ? (size_t)w->N * w->trit5_row : 0;
        default: return 0;
    }
}

void bitnet_a48_weight_free(bitnet_a48_weight* w) {
    if (!w) return;
    free_weight_buffers(w);
    delete w;
}

bitnet_a48_status bitnet_a48_quant_int4(const float* X_dev, int M, int K, float eps, int8_t* codes_dev,
                                        float* scale_dev, void* stream) {
    bitnet_a48_status s = check_act_args(X_dev, M, K, codes_dev, scale_dev);
    if (s != BITNET_A48_OK) return s;
    if (!(eps >= 0.f)) return BITNET_A48_ERR_INVALID_ARG;
    return a48_launch_quant_int4(X_dev, M, K, eps, codes_dev, scale_dev, nullptr, 0.f, (cudaStream_t)stream);
}

bitnet_a48_status bitnet_a48_topk_quant_int8(const float* X_dev, int M, int K, int k, float eps, int8_t* codes_dev,
                                             float* scale_dev, uint32_t* mask_bits_dev, void* stream) {
    if (!X_dev || !codes_dev || !scale_dev) return BITNET_A48_ERR_INVALID_ARG;
    if (M <= 0 || K <= 0 || K > kMaxFeatures) return BITNET_A48_ERR_SHAPE;
    if (k < 1 || k > K || !(eps >= 0.f)) return BITNET_A48_ERR_INVALID_ARG;
    if (!a48_aligned16(X_dev) || !a48_aligned16(codes_dev) || !a48_aligned16(scale_dev) ||
        !a48_aligned16(mask_bits_dev))
        return BITNET_A48_ERR_ALIGNMENT;
    if (!have_device()) return BITNET_A48_ERR_CUDA;
    return a48_launch_topk_quant_int8(X_dev, M, K, k, eps, codes_dev, scale_dev, mask_bits_dev,
                                      (cudaStream_t)stream);
}

bitnet_a48_status bitnet_a48_quant_fp4(const float* X_dev, int M, int K, int8_t* codes_dev, float* scale_dev,
                                       void* stream) {
    bitnet_a48_status s = check_act_args(X_dev, M, K, codes_dev, scale_dev);
    if (s != BITNET_A48_OK) return s;
    return a48_launch_quant_fp4(X_dev, M, K, codes_dev, scale_dev, nullptr, 0.f, (cudaStream_t)stream);
}

bitnet_a48_status bitnet_a48_compact_codes(const int8_t* codes_dev, int M, int K, int cap, uint16_t* idx_dev,
                                           int8_t* val_dev, int32_t* count_dev, void* stream) {
    if (!codes_dev || !idx_dev || !val_dev || !count_dev) return BITNET_A48_ERR_INVALID_ARG;
    if (M <= 0 || K <= 0 || K > 65535 || cap <= 0) return BITNET_A48_ERR_SHAPE;  // indices are 16-bit
    if (!a48_aligned16(codes_dev) || !a48_aligned16(idx_dev) || !a48_aligned16(val_dev) || !a48_aligned16(count_dev))
        return BITNET_A48_ERR_ALIGNMENT;
    if (!have_device()) return BITNET_A48_ERR_CUDA;
    return a48_launch_compact_codes(codes_dev, M, K, cap, idx_dev, val_dev, count_dev, (cudaStream_t)stream);
}

size_t bitnet_a48_linear_workspace_bytes(const bitnet_a48_weight* w, int M) {
    if (!w || M <= 0) return 0;
    const size_t dense = a48_decode_workspace_bytes(w, M), sparse = a48_decode_sparse_workspace_bytes(w, M);
    return dense > sparse ? dense : sparse;
}

bitnet_a48_status bitnet_a48_linear_ex(const bitnet_a48_weight* w, const int8_t* codes_dev, const float* scale_dev,
                                       int M, bitnet_a48_act kind, bitnet_a48_algo algo, float* Y_dev,
                                       int32_t* acc_dev, void* workspace_dev, size_t workspace_bytes, void* stream) {
    if (!w || !codes_dev || !scale_dev || !Y_dev) return BITNET_A48_ERR_INVALID_ARG;
    if ((int)kind < 0 || (int)kind > 2 || (int)algo < 0 || (int)algo > 7) return BITNET_A48_ERR_INVALID_ARG;
    if (M <= 0) return BITNET_A48_ERR_SHAPE;
    if (!a48_aligned16(codes_dev) || !a48_aligned16(scale_dev) || !a48_aligned16(Y_dev) || !a48_aligned16(acc_dev) ||
        !a48_aligned16(workspace_dev))
        return BITNET_A48_ERR_ALIGNMENT;
    if (!have_device()) return BITNET_A48_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    const bool automatic = algo == BITNET_A48_ALGO_AUTO;
    if (automatic) {
        // At the 3B/7B shapes one launch is latency-bound, and the dense kernel (dp4a on whole rows) beats the
        // zero-skipping one although it moves twice the bytes; the latter is taken when it is the only one possible.
        if (a48_decode_supported(w, M))
            algo = BITNET_A48_ALGO_DECODE;
        else if (M == 1 && kind == BITNET_A48_ACT_TOPK_INT8 && a48_decode_sparse_supported(w, M) && !a48_y_bf16)
            algo = BITNET_A48_ALGO_DECODE_SPARSE;
        else if (a48_decode_trit5_supported(w, M) && !w->gemm && !a48_y_bf16)
            algo = BITNET_A48_ALGO_DECODE_TRIT5;  // a handle packed for decode at 1.6 bits per weight only
        else if (a48_gemm_pair_preferred(1, &w, M))
            algo = BITNET_A48_ALGO_GEMM_TCGEN05_PAIR;  // from 384 tokens on, unless 128-token tiles fill the SMs better
        else if (a48_gemm_tcgen05_supported(w, M, false))
            algo = BITNET_A48_ALGO_GEMM_TCGEN05;
        else
            algo = BITNET_A48_ALGO_SIMPLE;
    }
    if (automatic && algo == BITNET_A48_ALGO_GEMM_TCGEN05_PAIR) {
        // the pair form can still decline (a device that cannot host a two-CTA cluster of this size, a shape beyond its
        // index arithmetic): the library's own choice then falls back to the single-CTA form, then to the simple kernel
        bitnet_a48_status s = a48_launch_gemm_pair(w, codes_dev, scale_dev, M, Y_dev, acc_dev, st);
        if (s != BITNET_A48_ERR_UNSUPPORTED && s != BITNET_A48_ERR_SHAPE) return s;
        algo = a48_gemm_tcgen05_supported(w, M, false) ? BITNET_A48_ALGO_GEMM_TCGEN05 : BITNET_A48_ALGO_SIMPLE;
    }
    if (automatic && algo == BITNET_A48_ALGO_GEMM_TCGEN05) {
        bitnet_a48_status s = a48_launch_gemm_tcgen05(w, codes_dev, scale_dev, M, Y_dev, acc_dev, false, st);
        if (s != BITNET_A48_ERR_UNSUPPORTED && s != BITNET_A48_ERR_SHAPE) return s;
        algo = BITNET_A48_ALGO_SIMPLE;
    }
    switch (algo) {
        case BITNET_A48_ALGO_SIMPLE:
            return a48_launch_linear_simple(w, codes_dev, scale_dev, M, Y_dev, acc_dev, st);
        case BITNET_A48_ALGO_GEMM_TCGEN05:
            if (!a48_gemm_tcgen05_supported(w, M, false)) return BITNET_A48_ERR_UNSUPPORTED;
            return a48_launch_gemm_tcgen05(w, codes_dev, scale_dev, M, Y_dev, acc_dev, false, st);
        case BITNET_A48_ALGO_GEMM_TCGEN05_I8:
            if (!a48_gemm_tcgen05_supported(w, M, true)) return BITNET_A48_ERR_UNSUPPORTED;
            return a48_launch_gemm_tcgen05(w, codes_dev, scale_dev, M, Y_dev, acc_dev, true, st);
        case BITNET_A48_ALGO_GEMM_TCGEN05_PAIR:
            return a48_launch_gemm_pair(w, codes_dev, scale_dev, M, Y_dev, acc_dev, st);
        case BITNET_A48_ALGO_DECODE:
            if (!a48_decode_supported(w, M)) return BITNET_A48_ERR_UNSUPPORTED;
            return a48_launch_decode(w, codes_dev, scale_dev, M, Y_dev, acc_dev, workspace_dev, workspace_bytes, st);
        case BITNET_A48_ALGO_DECODE_TRIT5:
            return a48_launch_decode_trit5(w, codes_dev, scale_dev, M, Y_dev, acc_dev, st);
        case BITNET_A48_ALGO_DECODE_SPARSE:
            if (!a48_decode_sparse_supported(w, M)) return BITNET_A48_ERR_UNSUPPORTED;
            return a48_launch_decode_sparse(w, codes_dev, scale_dev, M, Y_dev, acc_dev, workspace_dev,
                                            workspace_bytes, st);
        default:
            return BITNET_A48_ERR_INVALID_ARG;
    }
}

bitnet_a48_status bitnet_a48_linear(const bitnet_a48_weight* w, const int8_t* codes_dev, const float* scale_dev,
                                    int M, bitnet_a48_act kind, float* Y_dev, int32_t* acc_dev,
                                    void* workspace_dev, size_t workspace_bytes, void* stream) {
    return bitnet_a48_linear_ex(w, codes_dev, scale_dev, M, kind, BITNET_A48_ALGO_AUTO, Y_dev, acc_dev,
                                workspace_dev, workspace_bytes, stream);
}

bitnet_a48_status bitnet_a48_linear_bf16(const bitnet_a48_weight* w, const int8_t* codes_dev, const float* scale_dev,
                                         int M, bitnet_a48_act kind, uint16_t* Y_bf16_dev, void* workspace_dev,
                                         size_t workspace_bytes, void* stream) {
    a48_y_bf16 = 1;  // the kernels this call launches store bf16
    const bitnet_a48_status s = bitnet_a48_linear_ex(w, codes_dev, scale_dev, M, kind, BITNET_A48_ALGO_AUTO,
                                                     reinterpret_cast<float*>(Y_bf16_dev), nullptr, workspace_dev,
                                                     workspace_bytes, stream);
    a48_y_bf16 = 0;
    return s;
}

bitnet_a48_status bitnet_a48_quant_int4_bf16(const uint16_t* X_bf16_dev, int M, int K, float eps, int8_t* codes_dev,
                                             float* scale_dev, void* stream) {
    bitnet_a48_status s = check_act_args(X_bf16_dev, M, K, codes_dev, scale_dev);
    if (s != BITNET_A48_OK) return s;
    if (!(eps >= 0.f)) return BITNET_A48_ERR_INVALID_ARG;
    return a48_launch_quant_int4_bf16(X_bf16_dev, M, K, eps, codes_dev, scale_dev, (cudaStream_t)stream);
}

bitnet_a48_status bitnet_a48_topk_quant_int8_bf16(const uint16_t* X_bf16_dev, int M, int K, int k, float eps,
                                                  int8_t* codes_dev, float* scale_dev, void* stream) {
    bitnet_a48_status s = check_act_args(X_bf16_dev, M, K, codes_dev, scale_dev);
    if (s != BITNET_A48_OK) return s;
    if (k < 1 || k > K || !(eps >= 0.f)) return BITNET_A48_ERR_INVALID_ARG;
    return a48_launch_topk_quant_int8_bf16(X_bf16_dev, M, K, k, eps, codes_dev, scale_dev, (cudaStream_t)stream);
}

size_t bitnet_a48_linear_multi_workspace_bytes(int count, const bitnet_a48_weight* const weights[], int M) {
    if (count < 1 || !weights || M <= 0) return 0;
    for (int j = 0; j < count; ++j)
        if (!weights[j]) return 0;
    size_t fused = count <= 4 ? a48_decode_multi_workspace_bytes(count, weights, M) : 0;
    if (fused) return fused;
    size_t single = 0;  // one call after the other: the largest single requirement
    for (int j = 0; j < count; ++j) {
        size_t b = bitnet_a48_linear_workspace_bytes(weights[j], M);
        single = b > single ? b : single;
    }
    return single;
}

bitnet_a48_status bitnet_a48_linear_multi(int count, const bitnet_a48_weight* const weights[], const int8_t* codes_dev,
                                          const float* scale_dev, int M, bitnet_a48_act kind, float* const Y_dev[],
                                          void* workspace_dev, size_t workspace_bytes, void* stream) {
    if (count < 1 || !weights || !codes_dev || !scale_dev || !Y_dev) return BITNET_A48_ERR_INVALID_ARG;
    if ((int)kind < 0 || (int)kind > 2) return BITNET_A48_ERR_INVALID_ARG;
    if (M <= 0) return BITNET_A48_ERR_SHAPE;
    for (int j = 0; j < count; ++j) {
        if (!weights[j] || !Y_dev[j]) return BITNET_A48_ERR_INVALID_ARG;
        if (weights[j]->K != weights[0]->K) return BITNET_A48_ERR_SHAPE;
        if (!a48_aligned16(Y_dev[j])) return BITNET_A48_ERR_ALIGNMENT;
    }
    if (!a48_aligned16(codes_dev) || !a48_aligned16(scale_dev) || !a48_aligned16(workspace_dev))
        return BITNET_A48_ERR_ALIGNMENT;
    if (!have_device()) return BITNET_A48_ERR_CUDA;
    if (count <= 4 && a48_decode_multi_workspace_bytes(count, weights, M) > 0)
        return a48_launch_decode_multi(count, weights, codes_dev, scale_dev, M, Y_dev, nullptr, workspace_dev,
                                       workspace_bytes, (cudaStream_t)stream);
    {  // beyond the decode kernel's token count: one tensor-core launch over the tiles of all matrices
        bool any_decode = false;
        for (int j = 0; j < count; ++j) any_decode = any_decode || a48_decode_supported(weights[j], M);
        // (where CTA pairs win, a launch per matrix on pairs is faster than the grouped single-CTA launch)
        if (!any_decode && !a48_gemm_pair_preferred(count, weights, M) && a48_gemm_tcgen05_multi_supported(count, weights, M))
            return a48_launch_gemm_tcgen05_multi(count, weights, codes_dev, scale_dev, M, Y_dev, (cudaStream_t)stream);
    }
    for (int j = 0; j < count; ++j) {
        bitnet_a48_status s = bitnet_a48_linear(weights[j], codes_dev, scale_dev, M, kind, Y_dev[j], nullptr, workspace_dev,
                                                workspace_bytes, stream);
        if (s != BITNET_A48_OK) return s;
    }
    return BITNET_A48_OK;
}

// Workspace of the host-buffer entry point: X | codes | scale | Y | linear workspace, each 256-byte aligned.
static size_t host_ws_layout(const bitnet_a48_weight* w, int M, size_t off[5]) {
    auto up = [](size_t v) { return (v + 255) / 256 * 256; };
    size_t o = 0;
    off[0] = o; o += up((size_t)M * w->K * 4);
    off[1] = o; o += up((size_t)M * w->K);
    off[2] = o; o += up((size_t)M * 4);
    off[3] = o; o += up((size_t)M * w->N * 4);
    off[4] = o; o += up(bitnet_a48_linear_workspace_bytes(w, M));
    return o;
}

size_t bitnet_a48_bitlinear_host_workspace_bytes(const bitnet_a48_weight* w, int M) {
    if (!w || M <= 0) return 0;
    size_t off[5];
    return host_ws_layout(w, M, off);
}

bitnet_a48_status bitnet_a48_bitlinear_host(const bitnet_a48_weight* w, const float* X_host, int M,
                                            bitnet_a48_act kind, int k, float eps, float* Y_host,
                                            void* workspace_dev, size_t workspace_bytes, void* stream) {
    bitnet_a48_status s = bitnet_a48_bitlinear_host_async(w, X_host, M, kind, k, eps, Y_host, workspace_dev,
                                                          workspace_bytes, stream);
    if (s != BITNET_A48_OK) return s;
    A48_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    return BITNET_A48_OK;
}

bitnet_a48_status bitnet_a48_bitlinear_host_async(const bitnet_a48_weight* w, const float* X_host, int M,
                                                  bitnet_a48_act kind, int k, float eps, float* Y_host,
                                                  void* workspace_dev, size_t workspace_bytes, void* stream) {
    if (!w || !X_host || !Y_host || !workspace_dev) return BITNET_A48_ERR_INVALID_ARG;
    if (M <= 0) return BITNET_A48_ERR_SHAPE;
    if (!a48_aligned16(workspace_dev)) return BITNET_A48_ERR_ALIGNMENT;
    size_t off[5];
    if (workspace_bytes < host_ws_layout(w, M, off)) return BITNET_A48_ERR_NOMEM;
    cudaStream_t st = (cudaStream_t)stream;
    char* base = static_cast<char*>(workspace_dev);
    float* X = reinterpret_cast<float*>(base + off[0]);
    int8_t* codes = reinterpret_cast<int8_t*>(base + off[1]);
    float* scale = reinterpret_cast<float*>(base + off[2]);
    float* Y = reinterpret_cast<float*>(base + off[3]);
    A48_CUDA_TRY(cudaMemcpyAsync(X, X_host, (size_t)M * w->K * 4, cudaMemcpyHostToDevice, st));
    bitnet_a48_status s;
    if (kind == BITNET_A48_ACT_INT4) s = bitnet_a48_quant_int4(X, M, w->K, eps, codes, scale, stream);
    else if (kind == BITNET_A48_ACT_TOPK_INT8) s = bitnet_a48_topk_quant_int8(X, M, w->K, k, eps, codes, scale, nullptr, stream);
    else if (kind == BITNET_A48_ACT_FP4) s = bitnet_a48_quant_fp4(X, M, w->K, codes, scale, stream);
    else return BITNET_A48_ERR_INVALID_ARG;
    if (s != BITNET_A48_OK) return s;
    const size_t lin_bytes = bitnet_a48_linear_workspace_bytes(w, M);
    if (lin_bytes) A48_CUDA_TRY(cudaMemsetAsync(base + off[4], 0, lin_bytes, st));
    s = bitnet_a48_linear(w, codes, scale, M, kind, Y, nullptr, base + off[4], workspace_bytes - off[4], stream);
    if (s != BITNET_A48_OK) return s;
    A48_CUDA_TRY(cudaMemcpyAsync(Y_host, Y, (size_t)M * w->N * 4, cudaMemcpyDeviceToHost, st));
    return BITNET_A48_OK;
}

bitnet_a48_status bitnet_a48_block_create(const bitnet_a48_block_config* cfg, const bitnet_a48_weight* const weights[7],
                                          const float* gain_attn_dev, const float* gain_ffn_dev,
                                          bitnet_a48_block** out) {
    if (!cfg || !weights || !gain_attn_dev || !gain_ffn_dev || !out) return BITNET_A48_ERR_INVALID_ARG;
    const int H = cfg->hidden, F = cfg->ffn;
    if (H <= 0 || F <= 0 || cfg->n_heads <= 0 || H % cfg->n_heads != 0 || (H / cfg->n_heads) % 2 != 0 ||
        cfg->ctx_cap < 0)
        return BITNET_A48_ERR_SHAPE;
    if (cfg->k_o < 1 || cfg->k_o > H || cfg->k_down < 1 || cfg->k_down > F) return BITNET_A48_ERR_INVALID_ARG;
    if (!a48_aligned16(gain_attn_dev) || !a48_aligned16(gain_ffn_dev)) return BITNET_A48_ERR_ALIGNMENT;
    const int dims[7][2] = {{H, H}, {H, H}, {H, H}, {H, H}, {F, H}, {F, H}, {H, F}};
    for (int i = 0; i < 7; ++i) {
        if (!weights[i]) return BITNET_A48_ERR_INVALID_ARG;
        if (weights[i]->N != dims[i][0] || weights[i]->K != dims[i][1]) return BITNET_A48_ERR_SHAPE;
    }
    bitnet_a48_block* b = new (std::nothrow) bitnet_a48_block();
    if (!b) return BITNET_A48_ERR_NOMEM;
    b->cfg = *cfg;
    for (int i = 0; i < 7; ++i) b->w[i] = weights[i];
    b->g_attn = gain_attn_dev;
    b->g_ffn = gain_ffn_dev;
    *out = b;
    return BITNET_A48_OK;
}

void bitnet_a48_block_free(bitnet_a48_block* blk) { delete blk; }

size_t bitnet_a48_kv_cache_bytes(const bitnet_a48_block* blk, int B) {
    if (!blk || B <= 0 || blk->cfg.ctx_cap <= 0) return 0;
    const bitnet_a48_block_config& c = blk->cfg;
    return a48_kv_cache_bytes(B, c.n_heads, c.ctx_cap, c.hidden / c.n_heads, c.kv_bits);
}

size_t bitnet_a48_block_workspace_bytes(const bitnet_a48_block* blk, int B, int T) {
    if (!blk || B <= 0 || T <= 0) return 0;
    return a48_block_workspace_bytes(blk, B, T);
}

bitnet_a48_status bitnet_a48_block_forward(const bitnet_a48_block* blk, const float* X_dev, int B, int T, int pos0,
                                           float* kcache_dev, float* vcache_dev, float* Y_dev, void* workspace_dev,
                                           size_t workspace_bytes, void* stream) {
    if (!blk || !X_dev || !Y_dev || !workspace_dev) return BITNET_A48_ERR_INVALID_ARG;
    if (B <= 0 || T <= 0 || pos0 < 0 || (long long)B * T > (1 << 24)) return BITNET_A48_ERR_SHAPE;
    const bool no_cache = !kcache_dev || !vcache_dev;
    if (no_cache && (pos0 != 0 || kcache_dev || vcache_dev)) return BITNET_A48_ERR_INVALID_ARG;
    if (!no_cache && pos0 + T > blk->cfg.ctx_cap) return BITNET_A48_ERR_SHAPE;
    if (!a48_aligned16(X_dev) || !a48_aligned16(Y_dev) || !a48_aligned16(workspace_dev) ||
        !a48_aligned16(kcache_dev) || !a48_aligned16(vcache_dev))
        return BITNET_A48_ERR_ALIGNMENT;
    if (workspace_bytes < a48_block_workspace_bytes(blk, B, T)) return BITNET_A48_ERR_NOMEM;
    if (!have_device()) return BITNET_A48_ERR_CUDA;
    return a48_block_forward(blk, X_dev, B, T, pos0, kcache_dev, vcache_dev, Y_dev, workspace_dev, workspace_bytes,
                             (cudaStream_t)stream);
}

size_t bitnet_a48_attention_prefill_workspace_bytes(int B, int n_heads, int head_dim, int T, int n_keys) {
    if (B <= 0 || n_heads <= 0 || T <= 0 || n_keys < T || !a48_attn_tc_supported(head_dim)) return 0;
    return a48_attn_tc_workspace_bytes(B, n_heads, head_dim, T, n_keys);
}

bitnet_a48_status bitnet_a48_attention_prefill(const float* q_dev, const float* kcache_dev, const float* vcache_dev, int B,
                                               int T, int n_heads, int head_dim, int pos0, int ctx_cap, float* out_dev,
                                               void* workspace_dev, size_t workspace_bytes, void* stream) {
    if (!q_dev || !kcache_dev || !vcache_dev || !out_dev || !workspace_dev) return BITNET_A48_ERR_INVALID_ARG;
    if (B <= 0 || T <= 0 || n_heads <= 0 || head_dim <= 0 || pos0 < 0 || (long long)B * T > (1 << 24)) return BITNET_A48_ERR_SHAPE;
    if ((long long)pos0 + T > ctx_cap || B > 65535 || n_heads > 65535) return BITNET_A48_ERR_SHAPE;
    if (!a48_attn_tc_supported(head_dim)) return BITNET_A48_ERR_UNSUPPORTED;
    if (!a48_aligned16(q_dev) || !a48_aligned16(kcache_dev) || !a48_aligned16(vcache_dev) || !a48_aligned16(out_dev) ||
        !a48_aligned16(workspace_dev))
        return BITNET_A48_ERR_ALIGNMENT;
    if (workspace_bytes < a48_attn_tc_workspace_bytes(B, n_heads, head_dim, T, pos0 + T)) return BITNET_A48_ERR_NOMEM;
    if (!have_device()) return BITNET_A48_ERR_CUDA;
    return a48_launch_attn_tc(q_dev, kcache_dev, vcache_dev, B, T, n_heads, head_dim, pos0, ctx_cap, out_dev, workspace_dev,
                              (cudaStream_t)stream);
}

bitnet_a48_status bitnet_a48_kernel_status(unsigned int words_host[4]) {
    if (!words_host) return BITNET_A48_ERR_INVALID_ARG;
    if (!have_device()) return BITNET_A48_ERR_CUDA;
    return a48_read_kernel_status(words_host);
}

}  // extern "C"
