// placeholder until the tcgen05 kernel lands
#include "internal.h"
bool a48_gemm_tcgen05_supported(const bitnet_a48_weight*, int) { return false; }
bitnet_a48_status a48_launch_gemm_tcgen05(const bitnet_a48_weight*, const int8_t*, const float*, int, float*, int32_t*,
                                          cudaStream_t) { return BITNET_A48_ERR_UNSUPPORTED; }
bitnet_a48_status a48_read_kernel_status(unsigned int words_host[4]) {
    for (int i = 0; i < 4; ++i) words_host[i] = 0;
    return BITNET_A48_OK;
}
