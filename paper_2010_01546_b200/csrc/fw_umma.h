// Tensor-core (tcgen05 / TMEM / TMA) engine: entry points used by the host API.
#ifndef FW_UMMA_H_
#define FW_UMMA_H_
#include <vector>
#include <cuda.h>
#include "fw_internal.h"

namespace fw {

// True when the driver exposes tensor-map encoding (needed by every kernel of this engine).
bool umma_available();
// A bounded wait that ran out records where (a code > 0) in the status word its item points to: the owning layer's
// own status word in its workspace, so one layer's time-out is never reported to another.

// Test aid: one thread waits on a barrier nobody arrives on, for at most `polls` polls, then records code 901.
cudaError_t launch_wait_probe(int32_t* status, uint32_t polls, cudaStream_t s);

// ---- G~ = G Qs (+ fused SGD) ----
struct UmmaGqItem {
  const float* Qs;   // M x M, row-major: the right-hand matrix of out = G Qs (any fp32 matrix, not only Qs)
  const float* G;    // N x M
  float* out;        // N x M: G~ (EPI_STORE) or W (EPI_SGD)
  int32_t M;
  int64_t N;
  int32_t* status;   // the layer's time-out word
  int32_t* nonfinite;  // the layer's non-finite word: set when the product holds a NaN or Inf (may be null)
  float* part;       // scratch for the partial tiles of a K split (may be null: no split)
  int64_t part_floats;
  const float* colbias;  // optional, length M: subtracted from every row of the product
};
// out = G Qs on CTA pairs (256 x 512 tiles, K split with a fixed-order reduction); M a multiple of 4, >= 16
bool umma_gq_pair_supported(int M);
fw_status umma_gq_pair_launch(const UmmaGqItem* items, int n, int epi, float lr, int prof_class, cudaStream_t s);
// K-major fp32 operand: 2-D row-major [outer][inner] tensor, boxes of box_inner (32) floats x box_outer rows,
// 128-byte swizzle
bool tmap_encode_kmajor_f32(CUtensorMap* m, const void* base, uint64_t inner, uint64_t outer, uint64_t ld,
                            uint32_t box_inner, uint32_t box_outer);

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
  int32_t* status;     // the layer's time-out word
  const float* pmean;  // unshifted blocks: pilot mean whose outer product the CTA-pair kernel takes out of its
                       // accumulators as the rows go by (null: no correction)
  float corr_out;      // filled by the launcher: rows' worth of that outer product taken out, over all splits
  // implicit im2col (k = 3, stride 1, padding 1): X is the zero-padded fp32 activation [B][H + 2][W + 2][C] and the
  // rows of the patch matrix are never materialised; rows = B H W, M = 9 C
  int32_t im2col;
  int32_t i2c_B, i2c_H, i2c_W, i2c_C;
};
// stage geometry of an implicit-im2col layer: pixels per stage along x (bw) and y (bh); false if the shape has none
bool umma_gram_im2col_geometry(int H, int W, int C, int want_rows, int* bw, int* bh);
bool umma_gram_supported(const fw_layer_desc& d, const void* X, int64_t ldx);
bool umma_gram_unshifted(const fw_layer_desc& d, int64_t rows);
fw_status umma_gram_launch(UmmaGramItem* items, int n, cudaStream_t s);

// MN-major operand chunks of a row-major matrix: 2-D boxes of one chunk, and a chunked 3-D view (chunk_cols
// columns, rows, cols / chunk_cols) whose box delivers box_chunks chunks with one TMA instruction.
// fp32: 32-column chunks, 128-byte rows with 32-byte swizzle atoms; bf16: 32-column chunks with the 64-byte
// swizzle or 64-column chunks with the 128-byte swizzle.
bool tmap_encode_2d(CUtensorMap* m, bool bf16, const void* base, uint64_t inner, uint64_t outer, uint64_t ld,
                    uint32_t box_inner, uint32_t box_outer);
bool tmap_encode_chunked_3d(CUtensorMap* m, bool bf16, const void* base, uint64_t cols, uint64_t rows, uint64_t ld,
                            uint32_t box_rows, uint32_t box_chunks, uint32_t chunk_cols);

// ---- the same two products on CTA pairs (cta_group::2), for matrices too large for one CTA's TMEM ----
// 256 x 512 output tiles per pair of SMs: each CTA stages its own 128 rows of A and its half of B.
bool umma_pair_gram_eligible(const UmmaGramItem& it);
bool umma_pair_atb_eligible(int M);
int umma_pair_split_cap(int M);
fw_status umma_pair_gram_launch(UmmaGramItem* items, int n, cudaStream_t s);

// ---- D = A^T B, square fp32 matrices (re-sync products) ----
struct UmmaAtbItem {
  const float* A;   // M x M row-major
  const float* B;   // M x M row-major
  float* C;         // M x M row-major
  int32_t M;
  int32_t sym;      // the product is symmetric: only its upper triangle is taken from the accumulators and mirrored
  int32_t* status;  // the layer's time-out word
};
fw_status umma_atb_launch(const UmmaAtbItem* items, int n, cudaStream_t s);
fw_status umma_pair_atb_launch(const UmmaAtbItem* items, int n, cudaStream_t s);

}  // namespace fw
#endif
