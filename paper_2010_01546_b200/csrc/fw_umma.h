// Tensor-core (tcgen05 / TMEM / TMA) engine: entry points used by the host API.
#ifndef FW_UMMA_H_
#define FW_UMMA_H_
#include <vector>
#include "fw_internal.h"

namespace fw {

// True when the driver exposes tensor-map encoding (needed by every kernel of this engine).
bool umma_available();
// Returns and clears the engine's device-side status (0 = ok, > 0 = a bounded wait ran out, < 0 = read failed).
int umma_take_status();

// ---- G~ = G Qs (+ fused SGD) ----
struct UmmaGqItem {
  const float* Qs;   // M x M
  const float* G;    // N x M
  float* out;        // N x M: G~ (EPI_STORE) or W (EPI_SGD)
  int32_t M, N;
};
bool umma_gq_supported(const fw_layer_desc& d);
fw_status umma_gq_launch(const UmmaGqItem* items, int n, int epi, float lr, cudaStream_t s);

// ---- Gram X^T X + column sums ----
struct UmmaGramItem {
  const void* X;       // rows x M, fp32 or bf16
  int64_t rows, ldx;
  int32_t M;
  int32_t x_bf16;
  const float* shift;  // per-column shift subtracted before the product (fp32 X), may be null
  float* gram_part;    // split_cap x M x M
  float* colsum_part;  // split_cap x M
  int32_t split_cap;
  int32_t splits_out;  // filled by the launcher
  int32_t tag;         // caller's index of this item (the launcher may reorder items)
};
bool umma_gram_supported(const fw_layer_desc& d, const void* X, int64_t ldx);
bool umma_gram_unshifted(const fw_layer_desc& d, int64_t rows);
fw_status umma_gram_launch(UmmaGramItem* items, int n, cudaStream_t s);

// ---- D = A^T B, square fp32 matrices (re-sync products) ----
struct UmmaAtbItem {
  const float* A;   // M x M row-major
  const float* B;   // M x M row-major
  float* C;         // M x M row-major
  int32_t M;
};
fw_status umma_atb_launch(const UmmaAtbItem* items, int n, cudaStream_t s);

}  // namespace fw
#endif
