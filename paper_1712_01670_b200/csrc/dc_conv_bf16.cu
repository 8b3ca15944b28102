// Tensor-core partial convolution (bf16): placeholder until the tcgen05 kernel lands.
#include "dc_common.cuh"

int dc_conv_bf16_supported(const dc_cache*, int) { return 0; }
int dc_launch_conv_bf16(dc_cache*, int, const void*, void*, const int32_t*, const int32_t*, const uint32_t*, int)
{
    return DC_ERR_CONFIG;
}
int dc_pack_weights_bf16(dc_cache*, int) { return DC_OK; }
