// Tensor-core engine (placeholder until the tcgen05 kernels land): reports that
// no layer is supported, so every contraction runs on the FFMA engine.
#include "fw_umma.h"

namespace fw {
bool umma_gram_supported(const fw_layer_desc&, const void*, int64_t) { return false; }
fw_status umma_gram_group(fw_layer* const*, const void* const*, const int64_t*, const int64_t*,
                          const std::vector<int>&, int32_t*, cudaStream_t) { return FW_ERR_UNSUPPORTED; }
bool umma_gq_supported(const fw_layer_desc&) { return false; }
fw_status umma_gq_group(fw_layer* const*, const float* const*, float* const*, const std::vector<int>&, int, float,
                        cudaStream_t) { return FW_ERR_UNSUPPORTED; }
}  // namespace fw
