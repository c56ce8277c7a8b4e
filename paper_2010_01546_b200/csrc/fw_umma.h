// Tensor-core (tcgen05 / TMEM / TMA) engine: entry points used by the host API.
#ifndef FW_UMMA_H_
#define FW_UMMA_H_
#include <vector>
#include "fw_internal.h"

struct fw_layer;

namespace fw {

// Whether the tensor-core Gram kernel can take this layer's X (shape, alignment).
bool umma_gram_supported(const fw_layer_desc& d, const void* X, int64_t ldx);
// Gram partials + column sums for the listed layers of a group; fills splits[i].
fw_status umma_gram_group(fw_layer* const* L, const void* const* X, const int64_t* rows, const int64_t* ldx,
                          const std::vector<int>& idx, int32_t* splits, cudaStream_t s);
// Whether the tensor-core G * Qs kernel can take this layer.
bool umma_gq_supported(const fw_layer_desc& d);
fw_status umma_gq_group(fw_layer* const* L, const float* const* G, float* const* out,
                        const std::vector<int>& idx, int epi, float lr, cudaStream_t s);

}  // namespace fw
#endif
