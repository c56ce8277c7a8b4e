// Internal definitions shared by the library's translation units (host + device).
// Not part of the public interface.
#ifndef FW_INTERNAL_H_
#define FW_INTERNAL_H_

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "fw.h"

namespace fw {

// ---------------------------------------------------------------------------
// Device-resident description of one layer.  A copy sits at the start of the
// layer's workspace; kernels receive pointers to it.  All pointers point into
// the same workspace.
// ---------------------------------------------------------------------------
struct LayerDev {
  int32_t M, N;
  int32_t init;         // fw_init
  int32_t x_dtype;      // fw_dtype of X
  float alpha, beta, gamma, delta, eps, c_rel, c_abs;
  float pad1;
  // moments
  float* mu;            // M   running mean
  float* mu_prev;       // M   mean before the last update (for Eq. 31)
  float* phi;           // M   running uncentred feature power
  float* shift;         // M   pilot mean used to centre X inside the Gram pass
  float* Phix;          // MxM running covariance
  // transform state
  float* Phiy;          // MxM T Phix T^T
  float* Tt;            // MxM T^T (stored transposed so that t = T^T v is a row GEMV)
  float* Q;             // MxM T^T T
  float* Qs;            // MxM smoothed Q (aliases Q when beta == 0)
  float* tmp;           // MxM Pt = (T Phix)^T: re-sync intermediate, and state of the leaky (gamma < 1) update
  // recursion vectors
  float* xi2;           // M   squared column norms
  float* cvec;          // M   correlations with column m'
  float* wvec;          // M   alignment weights
  float* pv[2];         // M   ping-pong power-iteration vectors (unnormalised)
  float* v;             // M   unit vector v_e
  float* u;             // M   Phiy v
  float* t;             // M   T^T v
  float* part;          // 3 x part_stride per-block partial sums
  int32_t part_stride;
  int32_t pad2;
  float* scal;          // SC_* floats
  int32_t* iscal;       // IS_* ints
  // Gram scratch
  float* gram_part;     // split_cap x M x M partial Gram matrices
  float* colsum_part;   // split_cap x M partial column sums
  int32_t split_cap;
  int32_t pad3;
  // a block spread over several calls (FW_COV_ACCUMULATE): sums of the calls before the committing one
  float* gram_acc;      // M x M (upper-triangle tiles)
  float* colsum_acc;    // M
  // G Qs formed here when the caller asks for it in place
  float* gq_tmp;        // N x M
  // pilot mean of an unshifted tensor-core block: its outer product is taken out of the Gram accumulators as the
  // rows go by (and put back by the moment kernels), so that the accumulators hold centred sums
  float* pmean;         // M
};

// The pilot mean as the tensor core reads it: rounded to bf16 (nearest even) for bf16 X, truncated to TF32 for
// fp32 X.  The Gram kernel that subtracts n c c^T and the moment kernels that add it back both use this value.
__host__ __device__ inline float corr_round(float c, int bf16) {
  union { float f; uint32_t u; } v;
  v.f = c;
  if (bf16) v.u = (v.u + 0x7fffu + ((v.u >> 16) & 1u)) & 0xffff0000u;
  else v.u &= 0xffffe000u;
  return v.f;
}
constexpr int kCorrEveryStages = 8;   // CTA-pair Gram: one correction MMA per accumulator every eight stages


enum { SC_LAMBDA_BAR = 0, SC_LAMBDA_E = 1, SC_G_E = 2, SC_A_E = 3, SC_LAST_NORM2 = 4, SC_COUNT = 8 };
enum { IS_MPRIME = 0, IS_SETSIZE = 1, IS_STATUS_NOSUB = 2, IS_STATUS_NONFINITE = 3, IS_STATUS_TIMEOUT = 4,
       IS_GRID_BAR = 5 /* grid-barrier counter and, after it, the abort flag of the persistent recursion */, IS_COUNT = 8 };

constexpr int kGemvRowsPerBlock = 32;   // rows of a matrix handled by one CTA of a GEMV pass (default shape)
constexpr int kGemvMinRowsPerBlock = 8; // smallest pass shape: sizes the per-block partial sums
constexpr int kGemvThreads = 256;

// Argument block of a grouped launch: up to FW_MAX_GROUP layers.
struct GroupDev {
  int32_t n;
  int32_t pad;
  const LayerDev* layer[FW_MAX_GROUP];
};

struct PtrTable {
  const void* p[FW_MAX_GROUP];
};

struct Rows64 {
  int64_t v[FW_MAX_GROUP];
};

// First CTA of each layer in a flat grid over the upper-triangle 32x32 tiles of all layers of a group
// (a grid sized for the largest layer is mostly empty CTAs when the layers differ in size).
struct TileTable {
  int32_t tile0[FW_MAX_GROUP + 1];
};
inline int fill_tile_table(TileTable& t, const int32_t* layer_M, int n) {
  int total = 0;
  for (int i = 0; i < n; ++i) {
    const int k = (layer_M[i] + 31) / 32;
    t.tile0[i] = total;
    total += k * (k + 1) / 2;
  }
  t.tile0[n] = total;
  return total;
}
#ifdef __CUDACC__
// Flat index over the upper-triangle tiles (bj >= bi) of a T x T tile grid, row by row -> (bi, bj).
__device__ __forceinline__ void tri_decode(int t, int T, int& bi, int& bj) {
  // tiles before row b: b T - b (b - 1) / 2
  int b = (int)(((2.f * T + 1.f) - sqrtf((2.f * T + 1.f) * (2.f * T + 1.f) - 8.f * (float)t)) * 0.5f);
  if (b < 0) b = 0;
  if (b > T - 1) b = T - 1;
  while (b > 0 && b * T - b * (b - 1) / 2 > t) --b;
  while (b + 1 < T && (b + 1) * T - (b + 1) * b / 2 <= t) ++b;
  bi = b;
  bj = b + (t - (b * T - b * (b - 1) / 2));
}
#endif

// One problem of a grouped FFMA GEMM:  C (m x n) = op(A) (m x k) * B (k x n)
//   a_kmajor = 1: A is stored k x m (row-major, m contiguous)   [Gram, T^T-products]
//   a_kmajor = 0: A is stored m x k (row-major, k contiguous)
//   B is stored k x n row-major.
//   sym = 1: only tiles with tile_col >= tile_row are computed (C symmetric).
//   splits > 1: split s writes its partial to C + s * c_split_stride.
// Epilogues: EPI_STORE  C = acc
//            EPI_SGD    C = C - lr * acc      (C is then the weight matrix)
//            EPI_SYMM   C[i,j] = C[j,i] = acc for the upper tiles (sym = 1, splits = 1)
enum { EPI_STORE = 0, EPI_SGD = 1, EPI_SYMM = 2 };
struct GemmProblem {
  const void* A;
  const void* B;
  float* C;
  const float* shift;      // optional per-column shift subtracted from A and B elements (Gram)
  float* colsum;           // optional per-split column sums of (A - shift)  (Gram)
  int64_t lda, ldb, ldc;
  int64_t c_split_stride;
  int32_t m, n;
  int64_t k;
  int32_t a_kmajor, sym, splits, epi;
  int32_t tiles_m, tiles_n, ntiles, first_cta;   // filled by the launcher
  float lr;
  int32_t in_bf16;         // A and B elements are bf16 (Gram on bf16 X)
  int32_t* nonfinite;      // optional: set to 1 when the product holds a NaN or Inf
  const float* colbias;    // optional, EPI_STORE: subtracted from every row of the product (length n)
};
struct GemmGroup {
  int32_t n;
  int32_t total_ctas;
  GemmProblem p[FW_MAX_GROUP];
};

// ---------------------------------------------------------------------------
// launch accounting / optional per-class event timing (host only, fw_api.cu)
// ---------------------------------------------------------------------------
// Largest dynamic shared-memory size a kernel has been opted into, per device (the attribute is per device).
struct SmemAttrCache { size_t set[64] = {0}; };
template <class F>
inline cudaError_t ensure_dyn_smem(F* func, size_t bytes, SmemAttrCache& c) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); dev = -1; }
  if (dev >= 0 && dev < 64 && bytes <= c.set[dev]) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess && dev >= 0 && dev < 64) c.set[dev] = bytes;
  return e;
}

// Tuning aids (environment variables, read once by the host API; none changes results).
struct Tuning {
  int pair_min_m;      // FW_PAIR_MIN_M   smallest dimension the CTA-pair kernels take (default 289)
  int pair_splits;     // FW_PAIR_SPLITS  row slabs per problem of the CTA-pair kernels (0: chosen by the scheduler)
  int pair_debug;      // FW_PAIR_DEBUG   print the chosen slabs
  int pass_shape;      // FW_PASS_SHAPE   42 / 24 / 18 / 41: shape of the streaming recursion passes (0: automatic)
  int persist_max_mb;  // FW_PERSIST_MAX_MB  largest total state (MB of 4 M^2 over the large layers of a call) the
                       //                 persistent recursion launch takes (default 512; 0: never)
  int gram_waves_pct;  // FW_GRAM_WAVES_PCT  CTAs of a single-CTA Gram launch, in percent of the SM count (default 200)
};
const Tuning& tuning();

void prof_open(int cls, cudaStream_t s);    // call right before a kernel launch
void prof_close(int cls, cudaStream_t s);   // call right after it
struct ProfScope {
  int cls; cudaStream_t s;
  ProfScope(int c, cudaStream_t st) : cls(c), s(st) { prof_open(cls, s); }
  ~ProfScope() { prof_close(cls, s); }
};

// ---------------------------------------------------------------------------
// launchers (defined in the .cu files)
// ---------------------------------------------------------------------------
cudaError_t launch_gemm_ffma(GemmGroup& g, cudaStream_t s, int prof_class);
// to_pmean != 0: the means go to the layers' pmean vectors instead of their shift vectors
cudaError_t launch_pilot_mean(const GroupDev& g, const PtrTable& X, const Rows64& rows, const Rows64& ldx,
                              int in_bf16, int max_M, int to_pmean, cudaStream_t s);
// rows: the block's rows (all calls since the last commit); use_acc[i] != 0: the accumulated sums of the block's
// earlier calls are added to this call's partial sums
// corr[i] > 0: the Gram kernel took corr[i] c c^T (c = corr_round of the layer's pmean) out of this call's sums
cudaError_t launch_moments(const GroupDev& g, const Rows64& rows, const int32_t* splits, const int32_t* first,
                           const int32_t* use_acc, const float* corr, const int32_t* layer_M, const PtrTable& W,
                           const PtrTable& b, int max_M, int max_N, bool any_params, cudaStream_t s);
// acc (+)= sum over the splits of this call's partial sums (a call that does not close its block);
// fresh[i] != 0: the first call of the block, acc is overwritten
cudaError_t launch_accumulate(const GroupDev& g, const int32_t* splits, const int32_t* fresh, const float* corr,
                              const int32_t* layer_M, cudaStream_t s);
cudaError_t launch_recursion_step(const GroupDev& g, int P, int step, const PtrTable& traces, int max_M,
                                  bool any_leaky, int row_blocks, cudaStream_t s);
cudaError_t launch_smooth(const GroupDev& g, int max_M, cudaStream_t s);
// Whitening from the eigenvalue decomposition (fw_evd.cu): one-sided Jacobi in fp64 on src[i], then (with_v) T, Q, Phi_y
size_t evd_scratch_bytes(int M);
cudaError_t launch_evd(int n, const float* const* src, const int* layer_M, void* const* scratch,
                       int32_t* const* status, const float* eps, bool with_v, float g_max, float* const* T_out,
                       float* const* Q_out, float* const* Y_out, float* const* lam_out, float* const* kappa_out,
                       cudaStream_t s);
bool recursion_cluster_supported(int M);
// CTAs of a 16-CTA cluster the on-chip recursion gives a layer of size M (1, 2, 4, 8, 16; 0: not on chip)
int recursion_cluster_ctas(int M);
cudaError_t launch_recursion_cluster(const GroupDev& g, const PtrTable& traces, const int* layer_M, int K, int P,
                                     cudaStream_t s);
// All K steps of a group of large gamma = 1 layers as one persistent cooperative launch.  bar_words: two ints in the
// leading layer's workspace (barrier counter, abort flag); bar_base_host: the host's count of arrivals at that
// counter so far, advanced by the launch.
bool recursion_persist_supported(const int* layer_M, const float* layer_gamma, int n);
cudaError_t launch_recursion_persist(const GroupDev& g, const PtrTable& traces, const int* layer_M, int K, int P,
                                     int32_t* bar_words, int32_t* status, uint32_t* bar_base_host, cudaStream_t s);
// zero-padded copies [B][H + 2][W + 2][C] of n NHWC fp32 activations in one launch; dst_floats[i] (a multiple of 4)
// floats of dst[i] are written in all
cudaError_t launch_pad_nhwc(int n, const float* const* src, float* const* dst, const int* B, const int* H, const int* W,
                            const int* C, const int64_t* dst_floats, cudaStream_t s);
cudaError_t launch_init_identity(const LayerDev* dev, int M, cudaStream_t s);
cudaError_t launch_transpose(const float* src, float* dst, int M, cudaStream_t s);
// out[j] = sum_k A[k][j] x[k] for a row-major M x M matrix A (A^T x)
cudaError_t launch_matT_vec(const float* A, const float* x, float* out, int M, cudaStream_t s);
cudaError_t launch_trace_lambda(const LayerDev* dev, int M, cudaStream_t s);
cudaError_t launch_sgd_bias(float* b, const float* gb, float lr, int N, cudaStream_t s);
cudaError_t launch_sgd_bias_group(const GroupDev& g, const PtrTable& b, const PtrTable& gb, float lr, int max_N,
                                  cudaStream_t s);
cudaError_t launch_axpy_step(float* W, const float* G, float lr, int64_t n, cudaStream_t s);
// v <- momentum v + (G + wd W); W <- W - lr v
cudaError_t launch_momentum_step(float* W, const float* G, float* v, float lr, float momentum, float wd, int64_t n,
                                 cudaStream_t s);
// rho = M / sum_ij A_ij^2 / (A_ii A_jj) of a symmetric M x M matrix, one float
cudaError_t launch_whiteness(const float* A, int M, float* out, cudaStream_t s);

}  // namespace fw
#endif
