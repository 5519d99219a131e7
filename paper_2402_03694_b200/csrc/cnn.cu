// S4 (1-D CNN): placeholder translation unit until the fused tcgen05 kernel lands.
#include "tc_common.cuh"

int sf_cnn_prepare(sf_slow*, const float*, const float*, const float*, const float*, const float*, const float*) {
    return SF_ERR_UNSUPPORTED;
}
int sf_cnn_bf16_forward(sf_ctx*, const sf_slow*, const void*, const uint32_t*, uint32_t, float*, uint8_t*, void*, cudaStream_t) {
    return SF_ERR_UNSUPPORTED;
}
