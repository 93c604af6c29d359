// placeholder until the decode kernels land
#include "internal.h"
bool a48_decode_supported(const bitnet_a48_weight*, int) { return false; }
bool a48_decode_sparse_supported(const bitnet_a48_weight*, int) { return false; }
size_t a48_decode_workspace_bytes(const bitnet_a48_weight*, int) { return 0; }
bitnet_a48_status a48_launch_decode(const bitnet_a48_weight*, const int8_t*, const float*, int, float*, int32_t*, void*,
                                    size_t, cudaStream_t) { return BITNET_A48_ERR_UNSUPPORTED; }
bitnet_a48_status a48_launch_decode_sparse(const bitnet_a48_weight*, const int8_t*, const float*, int, float*, int32_t*,
                                           void*, size_t, cudaStream_t) { return BITNET_A48_ERR_UNSUPPORTED; }
