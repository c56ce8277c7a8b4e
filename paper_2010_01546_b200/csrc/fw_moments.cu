// Moment kernels around the Gram pass (Eqs. 2-5, 37-38, 31):
//   pilot_mean     column means of the first rows of X, used to centre X inside
//                  the Gram pass so that the one-pass covariance does not cancel
//   moments_vec    reduce the split column sums, update mu, phi, lam_bar
//   moments_mat    reduce the split Gram partials, centre on the updated mean,
//                  running average into Phix, mirror to the lower triangle
//   bias_comp      b += W (mu_new - mu_old), carried by extra CTAs of the moments_mat launch
//   accumulate     a call that leaves its block open: its split sums are added to the block's accumulators
#include <cstring>

#include "fw_internal.h"

namespace fw {
namespace {

constexpr int kPilotRows = 512;     // rows sampled for the pilot mean
constexpr int kPilotTY = 16;        // row lanes per block

__global__ void pilot_mean_kernel(const __grid_constant__ GroupDev g, const __grid_constant__ PtrTable X,
                                  const __grid_constant__ Rows64 rows, const __grid_constant__ Rows64 ldx,
                                  int in_bf16, int to_pmean) {
  const LayerDev* L = g.layer[blockIdx.y];
  const int M = L->M;
  const int col = blockIdx.x * 32 + threadIdx.x;
  if (blockIdx.x * 32 >= M) return;
  int64_t R = rows.v[blockIdx.y];
  if (R > kPilotRows) R = kPilotRows;
  const int64_t ld = ldx.v[blockIdx.y];
  float acc = 0.f;
  if (col < M) {
    if (in_bf16) {
      const __nv_bfloat16* x = reinterpret_cast<const __nv_bfloat16*>(X.p[blockIdx.y]);
      for (int64_t r = threadIdx.y; r < R; r += kPilotTY) acc += __bfloat162float(x[r * ld + col]);
    } else {
      const float* x = reinterpret_cast<const float*>(X.p[blockIdx.y]);
      for (int64_t r = threadIdx.y; r < R; r += kPilotTY) acc += x[r * ld + col];
    }
  }
  __shared__ float sm[kPilotTY][33];
  sm[threadIdx.y][threadIdx.x] = acc;
  __syncthreads();
  if (threadIdx.y == 0 && col < M) {
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < kPilotTY; ++i) s += sm[i][threadIdx.x];
    (to_pmean ? L->pmean : L->shift)[col] = s / (float)R;
  }
}

struct MomentArgs {
  int32_t splits[FW_MAX_GROUP];
  int32_t first[FW_MAX_GROUP];
  int32_t use_acc[FW_MAX_GROUP];     // add the sums accumulated by the block's earlier calls (accumulate kernel:
                                     // 0 = overwrite the accumulators, 1 = add to them)
  float corr[FW_MAX_GROUP];          // > 0: corr c c^T was taken out of this call's Gram sums (c = rounded pmean)
  TileTable tt;                      // flat grid over the upper-triangle 32x32 tiles of all layers
  int32_t bias_blocks;               // CTAs per layer placed before the tiles for b += W (mu_new - mu_old); 0: none
};

// One CTA per layer, 1024 threads (one column each for M <= 1024).
__global__ void __launch_bounds__(1024) moments_vec_kernel(const __grid_constant__ GroupDev g,
                                                          const __grid_constant__ Rows64 rows,
                                                          const __grid_constant__ MomentArgs a) {
  const LayerDev* L = g.layer[blockIdx.x];
  const int M = L->M;
  const int S = a.splits[blockIdx.x];
  const bool first = a.first[blockIdx.x] != 0;
  const float inv_rows = 1.0f / (float)rows.v[blockIdx.x];
  const float alpha = L->alpha;
  float phisum = 0.f;
  bool bad = false;
  // A narrow layer leaves most of the block idle while every column walks all S split partials, eight loads at a
  // time: the splits are dealt to KG groups of threads (group kg takes a contiguous range of splits), whose sums
  // are then added in group order -- a fixed order for given (M, S), and a chain of S / (8 KG) load latencies.
  __shared__ float part_s[1024], part_d[1024];
  const int KG = M <= 512 ? min(8, 1024 / M) : 1;
  const int per = (S + KG - 1) / KG;
  const int64_t MM = (int64_t)M * M;
  if (KG > 1) {
    const int kg = threadIdx.x / M, m = threadIdx.x - kg * M;
    if (kg < KG) {
      float s = 0.f, d = 0.f;
      const float* cp = L->colsum_part + m;
      const float* gp = L->gram_part + (int64_t)m * M + m;
      const int k1 = min(S, (kg + 1) * per);
      int k = kg * per;
      for (; k + 8 <= k1; k += 8) {
        float sv[8], dv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) { sv[u] = cp[(int64_t)(k + u) * M]; dv[u] = gp[(int64_t)(k + u) * MM]; }
#pragma unroll
        for (int u = 0; u < 8; ++u) { s += sv[u]; d += dv[u]; }
      }
      for (; k < k1; ++k) { s += cp[(int64_t)k * M]; d += gp[(int64_t)k * MM]; }
      part_s[threadIdx.x] = s; part_d[threadIdx.x] = d;
    }
    __syncthreads();
  }
  for (int m = threadIdx.x; m < M; m += blockDim.x) {
    // partial sums in split order; the loads of eight splits are issued together (the chain of additions is
    // short, the chain of load latencies is what a plain loop would pay)
    float s = 0.f, d = 0.f;
    if (KG > 1) {
      for (int kg = 0; kg < KG; ++kg) { s += part_s[kg * M + m]; d += part_d[kg * M + m]; }
    } else {
      const float* cp = L->colsum_part + m;
      const float* gp = L->gram_part + (int64_t)m * M + m;
      int k = 0;
      for (; k + 8 <= S; k += 8) {
        float sv[8], dv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) { sv[u] = cp[(int64_t)(k + u) * M]; dv[u] = gp[(int64_t)(k + u) * MM]; }
#pragma unroll
        for (int u = 0; u < 8; ++u) { s += sv[u]; d += dv[u]; }
      }
      for (; k < S; ++k) { s += cp[(int64_t)k * M]; d += gp[(int64_t)k * MM]; }
    }
    if (a.corr[blockIdx.x] > 0.f) {
      const float cm = corr_round(L->pmean[m], L->x_dtype == FW_BF16);
      d = fmaf(a.corr[blockIdx.x], cm * cm, d);
    }
    if (a.use_acc[blockIdx.x]) { s += L->colsum_acc[m]; d += L->gram_acc[(int64_t)m * M + m]; }
    const float c = L->shift[m];
    const float mh_rel = s * inv_rows;          // batch mean relative to the shift
    const float mhat = c + mh_rel;
    const float mu_old = L->mu[m];
    const float mu_new = first ? mhat : fmaf(alpha, mu_old, (1.f - alpha) * mhat);
    L->mu_prev[m] = mu_old;
    L->mu[m] = mu_new;
    // uncentred power (Eq. 37): mean x^2 = mean (x-c)^2 + 2 c mean(x-c) + c^2
    const float ph = fmaf(d, inv_rows, fmaf(2.f * c, mh_rel, c * c));
    const float ph_new = first ? ph : fmaf(alpha, L->phi[m], (1.f - alpha) * ph);
    L->phi[m] = ph_new;
    phisum += ph_new;
    // per-call scratch in the power-iteration vectors (dead outside a reduction call): batch mean and new
    // mean relative to the shift
    L->pv[0][m] = mh_rel;
    L->pv[1][m] = mu_new - c;
    if (!isfinite(s) || !isfinite(d)) bad = true;
  }
  // deterministic block reduction of phisum
  __shared__ float red[1024];
  red[threadIdx.x] = phisum;
  __syncthreads();
  for (int o = 512; o > 0; o >>= 1) {
    if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) L->scal[SC_LAMBDA_BAR] = red[0] / (float)M;   // Eq. 38
  if (bad) L->iscal[IS_STATUS_NONFINITE] = 1;
}

// One CTA (32x8 threads) per 32x32 tile of the upper triangle of one layer; the grid is the flat list of these
// tiles over all layers of the group (a grid sized for the largest layer would be mostly empty CTAs when the
// layers differ in size, and handing those out costs more than the work).
__device__ __forceinline__ void bias_comp_rows(const LayerDev* L, const float* Wp, float* bp, int blk, int tid);

__global__ void __launch_bounds__(256) moments_mat_kernel(const __grid_constant__ GroupDev g,
                                                          const __grid_constant__ Rows64 rows,
                                                          const __grid_constant__ MomentArgs a,
                                                          const __grid_constant__ PtrTable W,
                                                          const __grid_constant__ PtrTable b) {
  const int nbias = a.bias_blocks * g.n;
  if ((int)blockIdx.x < nbias) {
    // the first CTAs carry the bias compensation (Eq. 31), which needs the means only: long rows of W start early
    // and the tiles fill in behind them
    const int layer = (int)blockIdx.x / a.bias_blocks, blk = (int)blockIdx.x - layer * a.bias_blocks;
    bias_comp_rows(g.layer[layer], reinterpret_cast<const float*>(W.p[layer]),
                   const_cast<float*>(reinterpret_cast<const float*>(b.p[layer])), blk, threadIdx.y * 32 + threadIdx.x);
    return;
  }
  const int tile_id = (int)blockIdx.x - nbias;
  int li = 0;
#pragma unroll 1
  for (int i = 1; i < g.n; ++i)
    if (tile_id >= a.tt.tile0[i]) li = i;
  const LayerDev* L = g.layer[li];
  const int M = L->M;
  int bi, bj;
  tri_decode(tile_id - a.tt.tile0[li], (M + 31) / 32, bi, bj);
  const int S = a.splits[li];
  const bool first = a.first[li] != 0;
  const float inv_rows = 1.0f / (float)rows.v[li];
  const float alpha = L->alpha;
  __shared__ float tile[32][33];
  const int j = bj * 32 + threadIdx.x;
  const float* mh = L->pv[0];  // batch mean - shift
  const float* nu = L->pv[1];  // new running mean - shift
  const bool use_acc = a.use_acc[li] != 0;
  const float corr = a.corr[li];
  const int xbf = L->x_dtype == FW_BF16;
  float mh_j = 0.f, nu_j = 0.f, ct_j = 0.f;
  if (j < M) { mh_j = mh[j]; nu_j = nu[j]; if (corr > 0.f) ct_j = corr_round(L->pmean[j], xbf); }
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int ii = threadIdx.y + 8 * r;
    const int i = bi * 32 + ii;
    float out = 0.f;
    if (i < M && j < M) {
      float s2 = 0.f;
      const int64_t off = (int64_t)i * M + j;
      // split partials added in split order, eight loads in flight at a time
      const float* gp = L->gram_part + off;
      const int64_t MM = (int64_t)M * M;
      int k = 0;
      for (; k + 8 <= S; k += 8) {
        float v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = gp[(int64_t)(k + u) * MM];
#pragma unroll
        for (int u = 0; u < 8; ++u) s2 += v[u];
      }
      for (; k < S; ++k) s2 += gp[(int64_t)k * MM];
      if (corr > 0.f) s2 = fmaf(corr, __fmul_rn(corr_round(L->pmean[i], xbf), ct_j), s2);   // symmetric in (i, j)
      if (use_acc) s2 += L->gram_acc[off];
      const float mh_i = mh[i], nu_i = nu[i];
      // (1/rows) sum (x-mu)(x-mu)^T with x - mu = (x - c) - nu
      // written symmetrically in i, j so that the result mirrors exactly
      float corr = __fadd_rn(__fmul_rn(mh_i, nu_j), __fmul_rn(nu_i, mh_j));
      float chat = __fadd_rn(__fsub_rn(__fmul_rn(s2, inv_rows), corr), __fmul_rn(nu_i, nu_j));
      out = first ? chat : __fadd_rn(__fmul_rn(alpha, L->Phix[off]), __fmul_rn(1.f - alpha, chat));
      if (bi != bj || j >= i) L->Phix[off] = out;
    }
    tile[ii][threadIdx.x] = out;
  }
  __syncthreads();
  // mirror: element (i, j) of the tile goes to (j, i)
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int jj = threadIdx.y + 8 * r;           // column index inside the tile
    const int jg = bj * 32 + jj;
    const int ig = bi * 32 + threadIdx.x;
    if (jg < M && ig < M) {
      if (bi != bj || ig < jg) L->Phix[(int64_t)jg * M + ig] = tile[threadIdx.x][jj];
    }
  }
}

// A call that leaves its block open (FW_COV_ACCUMULATE): the split sums of this call are added, in split order,
// to the block's accumulators (or overwrite them on the block's first call).  Same flat grid over the
// upper-triangle 32x32 tiles as moments_mat_kernel; the CTAs of a layer's first tile row also carry the column sums.
__global__ void __launch_bounds__(256) accumulate_kernel(const __grid_constant__ GroupDev g,
                                                         const __grid_constant__ MomentArgs a) {
  const int tile_id = (int)blockIdx.x;
  int li = 0;
#pragma unroll 1
  for (int i = 1; i < g.n; ++i)
    if (tile_id >= a.tt.tile0[i]) li = i;
  const LayerDev* L = g.layer[li];
  const int M = L->M;
  int bi, bj;
  tri_decode(tile_id - a.tt.tile0[li], (M + 31) / 32, bi, bj);
  const int S = a.splits[li];
  const bool add = a.use_acc[li] != 0;
  const float corr = a.corr[li];
  const int xbf = L->x_dtype == FW_BF16;
  const int j = bj * 32 + threadIdx.x;
  const float ct_j = (corr > 0.f && j < M) ? corr_round(L->pmean[j], xbf) : 0.f;
  const int64_t MM = (int64_t)M * M;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int i = bi * 32 + threadIdx.y + 8 * r;
    if (i < M && j < M) {
      const int64_t off = (int64_t)i * M + j;
      float s2 = 0.f;
      for (int k = 0; k < S; ++k) s2 += L->gram_part[off + (int64_t)k * MM];
      if (corr > 0.f) s2 = fmaf(corr, __fmul_rn(corr_round(L->pmean[i], xbf), ct_j), s2);
      L->gram_acc[off] = add ? L->gram_acc[off] + s2 : s2;
    }
  }
  if (bi == 0 && threadIdx.y == 0 && j < M) {
    float s = 0.f;
    for (int k = 0; k < S; ++k) s += L->colsum_part[(int64_t)k * M + j];
    L->colsum_acc[j] = add ? L->colsum_acc[j] + s : s;
  }
}

// b += W (mu_new - mu_old); one warp per output row, 8 rows per CTA
__device__ __forceinline__ void bias_comp_rows(const LayerDev* L, const float* Wp, float* bp, int blk, int tid) {
  if (!Wp || !bp) return;
  const int M = L->M, N = L->N;
  const int row = blk * 8 + (tid >> 5);
  if (row >= N) return;
  const int lane = tid & 31;
  float acc = 0.f;
  for (int m = lane; m < M; m += 32) acc = fmaf(Wp[(int64_t)row * M + m], L->mu[m] - L->mu_prev[m], acc);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) bp[row] += acc;
}

// Zero-padded copies of NHWC activations: dst[b][y + 1][x + 1][:] = src[b][y][x][:], one pixel of zeros all round,
// for every layer of a group in one launch.  One thread per 16 bytes of the destinations (flat over the layers).
struct PadGroup {
  const float4* src[FW_MAX_GROUP];
  float4* dst[FW_MAX_GROUP];
  int64_t first4[FW_MAX_GROUP + 1];   // first 16-byte unit of each layer in the flat index space
  int32_t B[FW_MAX_GROUP], H[FW_MAX_GROUP], W[FW_MAX_GROUP], C4[FW_MAX_GROUP];
  int32_t n;
};
__global__ void __launch_bounds__(256) pad_nhwc_kernel(const __grid_constant__ PadGroup g) {
  const int64_t total4 = g.first4[g.n];
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total4; e += (int64_t)gridDim.x * blockDim.x) {
    int li = 0;
#pragma unroll 1
    for (int i = 1; i < g.n; ++i)
      if (e >= g.first4[i]) li = i;
    const int64_t l = e - g.first4[li];
    const int C4 = g.C4[li], W = g.W[li], H = g.H[li];
    const int c = (int)(l % C4);
    int64_t p = l / C4;
    const int xp = (int)(p % (W + 2)); p /= (W + 2);
    const int yp = (int)(p % (H + 2));
    const int64_t b = p / (H + 2);
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (xp >= 1 && xp <= W && yp >= 1 && yp <= H && b < g.B[li])
      v = g.src[li][((b * H + (yp - 1)) * W + (xp - 1)) * C4 + c];
    g.dst[li][l] = v;
  }
}

__global__ void init_identity_kernel(const LayerDev* L) {
  const int M = L->M;
  const int64_t n = (int64_t)M * M;
  const bool alias = (L->Qs == L->Q);
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x) {
    const int i = (int)(e / M), j = (int)(e - (int64_t)i * M);
    const float d = (i == j) ? 1.f : 0.f;
    L->Tt[e] = d;
    L->Q[e] = d;
    if (!alias) L->Qs[e] = d;
    L->Phix[e] = 0.f;
    L->Phiy[e] = 0.f;
  }
  if (blockIdx.x == 0) {
    for (int m = threadIdx.x; m < M; m += blockDim.x) {
      L->mu[m] = 0.f; L->mu_prev[m] = 0.f; L->phi[m] = 0.f; L->shift[m] = 0.f;
    }
    if (threadIdx.x < SC_COUNT) L->scal[threadIdx.x] = 0.f;
    if (threadIdx.x < IS_COUNT) L->iscal[threadIdx.x] = 0;
  }
}

__global__ void transpose_kernel(const float* __restrict__ src, float* __restrict__ dst, int M) {
  __shared__ float tile[32][33];
  const int bi = blockIdx.y * 32, bj = blockIdx.x * 32;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int i = bi + threadIdx.y + 8 * r, j = bj + threadIdx.x;
    if (i < M && j < M) tile[threadIdx.y + 8 * r][threadIdx.x] = src[(int64_t)i * M + j];
  }
  __syncthreads();
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int j = bj + threadIdx.y + 8 * r, i = bi + threadIdx.x;
    if (i < M && j < M) dst[(int64_t)j * M + i] = tile[threadIdx.x][threadIdx.y + 8 * r];
  }
}

// out = A^T x: one thread per column, rows in order (coalesced across the columns)
__global__ void __launch_bounds__(256) matT_vec_kernel(const float* __restrict__ A, const float* __restrict__ x,
                                                       float* __restrict__ out, int M) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= M) return;
  float acc = 0.f;
  for (int k = 0; k < M; ++k) acc = fmaf(A[(int64_t)k * M + j], x[k], acc);
  out[j] = acc;
}

// lam_bar = trace(Phix) / M after a covariance has been injected
__global__ void __launch_bounds__(256) trace_lambda_kernel(const LayerDev* L) {
  const int M = L->M;
  float s = 0.f;
  for (int m = threadIdx.x; m < M; m += blockDim.x) s += L->Phix[(int64_t)m * M + m];
  __shared__ float red[256];
  red[threadIdx.x] = s;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) L->scal[SC_LAMBDA_BAR] = red[0] / (float)M;
}

__global__ void sgd_bias_kernel(float* b, const float* gb, float lr, int N) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < N) b[i] = fmaf(-lr, gb[i], b[i]);
}

// b <- b - lr g_b for every layer of a group; grid (ceil(max N / 256), layers)
__global__ void sgd_bias_group_kernel(const __grid_constant__ GroupDev g, const __grid_constant__ PtrTable b,
                                      const __grid_constant__ PtrTable gb, float lr) {
  const LayerDev* L = g.layer[blockIdx.y];
  float* bp = const_cast<float*>(reinterpret_cast<const float*>(b.p[blockIdx.y]));
  const float* gp = reinterpret_cast<const float*>(gb.p[blockIdx.y]);
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (bp && gp && i < L->N) bp[i] = fmaf(-lr, gp[i], bp[i]);
}

__global__ void axpy_step_kernel(float* __restrict__ W, const float* __restrict__ G, float lr, int64_t n) {
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x)
    W[e] = fmaf(-lr, G[e], W[e]);
}

__global__ void momentum_step_kernel(float* __restrict__ W, const float* __restrict__ G, float* __restrict__ v,
                                     float lr, float momentum, float wd, int64_t n) {
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x) {
    const float w = W[e];
    const float vn = fmaf(momentum, v[e], fmaf(wd, w, G[e]));
    v[e] = vn;
    W[e] = fmaf(-lr, vn, w);
  }
}

// Eq. 51 over all index pairs.  One CTA; every thread sums its rows in fp64, fixed-order tree over the block.
__global__ void __launch_bounds__(1024) whiteness_kernel(const float* __restrict__ A, int M, float* __restrict__ out) {
  double acc = 0.0;
  for (int i = threadIdx.x >> 5; i < M; i += 32) {          // a warp per row
    const double dii = A[(int64_t)i * M + i];
    double r = 0.0;
    for (int j = threadIdx.x & 31; j < M; j += 32) {
      const double a = A[(int64_t)i * M + j];
      r += a * a / (dii * (double)A[(int64_t)j * M + j]);
    }
    acc += r;
  }
  __shared__ double red[1024];
  red[threadIdx.x] = acc;
  __syncthreads();
  for (int o = 512; o > 0; o >>= 1) {
    if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) out[0] = (float)((double)M / red[0]);
}

}  // namespace

cudaError_t launch_momentum_step(float* W, const float* G, float* v, float lr, float momentum, float wd, int64_t n,
                                 cudaStream_t s) {
  int blocks = (int)((n + 1023) / 1024);
  if (blocks > 2368) blocks = 2368;
  if (blocks < 1) blocks = 1;
  ProfScope ps(FW_PROF_MISC, s);
  momentum_step_kernel<<<blocks, 256, 0, s>>>(W, G, v, lr, momentum, wd, n);
  return cudaGetLastError();
}

cudaError_t launch_whiteness(const float* A, int M, float* out, cudaStream_t s) {
  ProfScope ps(FW_PROF_MISC, s);
  whiteness_kernel<<<1, 1024, 0, s>>>(A, M, out);
  return cudaGetLastError();
}

cudaError_t launch_pilot_mean(const GroupDev& g, const PtrTable& X, const Rows64& rows, const Rows64& ldx,
                              int in_bf16, int max_M, int to_pmean, cudaStream_t s) {
  dim3 grid((max_M + 31) / 32, g.n), block(32, kPilotTY);
  ProfScope ps(FW_PROF_PILOT, s);
  pilot_mean_kernel<<<grid, block, 0, s>>>(g, X, rows, ldx, in_bf16, to_pmean);
  return cudaGetLastError();
}

cudaError_t launch_accumulate(const GroupDev& g, const int32_t* splits, const int32_t* fresh, const float* corr,
                              const int32_t* layer_M, cudaStream_t s) {
  MomentArgs a;
  memset(&a, 0, sizeof(a));
  for (int i = 0; i < g.n; ++i) { a.splits[i] = splits[i]; a.use_acc[i] = fresh[i] ? 0 : 1; a.corr[i] = corr[i]; }
  const int total = fill_tile_table(a.tt, layer_M, g.n);
  ProfScope ps(FW_PROF_MOMENTS, s);
  accumulate_kernel<<<total, dim3(32, 8), 0, s>>>(g, a);
  return cudaGetLastError();
}

cudaError_t launch_moments(const GroupDev& g, const Rows64& rows, const int32_t* splits, const int32_t* first,
                           const int32_t* use_acc, const float* corr, const int32_t* layer_M, const PtrTable& W,
                           const PtrTable& b, int max_M, int max_N, bool any_params, cudaStream_t s) {
  (void)max_M;
  MomentArgs a;
  memset(&a, 0, sizeof(a));
  for (int i = 0; i < g.n; ++i) {
    a.splits[i] = splits[i]; a.first[i] = first[i]; a.use_acc[i] = use_acc[i]; a.corr[i] = corr[i];
  }
  { ProfScope ps(FW_PROF_MOMENTS, s); moments_vec_kernel<<<g.n, 1024, 0, s>>>(g, rows, a); }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const int total = fill_tile_table(a.tt, layer_M, g.n);
  a.bias_blocks = any_params ? (max_N + 7) / 8 : 0;
  {
    ProfScope ps(FW_PROF_MOMENTS, s);
    moments_mat_kernel<<<total + a.bias_blocks * g.n, dim3(32, 8), 0, s>>>(g, rows, a, W, b);
  }
  return cudaGetLastError();
}

cudaError_t launch_pad_nhwc(int n, const float* const* src, float* const* dst, const int* B, const int* H, const int* W,
                            const int* C, const int64_t* dst_floats, cudaStream_t s) {
  // dst_floats covers the padded tensor plus the slack the last window may read past it: all of it is written
  PadGroup g;
  memset(&g, 0, sizeof(g));
  int64_t total4 = 0;
  for (int i = 0; i < n; ++i) {
    g.src[i] = reinterpret_cast<const float4*>(src[i]); g.dst[i] = reinterpret_cast<float4*>(dst[i]);
    g.B[i] = B[i]; g.H[i] = H[i]; g.W[i] = W[i]; g.C4[i] = C[i] / 4;
    g.first4[i] = total4;
    total4 += dst_floats[i] / 4;
  }
  g.first4[n] = total4;
  g.n = n;
  int64_t blocks = (total4 + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  ProfScope ps(FW_PROF_PILOT, s);
  pad_nhwc_kernel<<<(int)blocks, 256, 0, s>>>(g);
  return cudaGetLastError();
}

cudaError_t launch_init_identity(const LayerDev* dev, int M, cudaStream_t s) {
  int64_t n = (int64_t)M * M;
  int blocks = (int)((n + 255) / 256);
  if (blocks > 1184) blocks = 1184;
  ProfScope ps(FW_PROF_MISC, s);
  init_identity_kernel<<<blocks, 256, 0, s>>>(dev);
  return cudaGetLastError();
}

cudaError_t launch_transpose(const float* src, float* dst, int M, cudaStream_t s) {
  const int t = (M + 31) / 32;
  ProfScope ps(FW_PROF_MISC, s);
  transpose_kernel<<<dim3(t, t), dim3(32, 8), 0, s>>>(src, dst, M);
  return cudaGetLastError();
}

cudaError_t launch_matT_vec(const float* A, const float* x, float* out, int M, cudaStream_t s) {
  ProfScope ps(FW_PROF_MISC, s);
  matT_vec_kernel<<<(M + 255) / 256, 256, 0, s>>>(A, x, out, M);
  return cudaGetLastError();
}

cudaError_t launch_trace_lambda(const LayerDev* dev, int M, cudaStream_t s) {
  (void)M;
  ProfScope ps(FW_PROF_MISC, s);
  trace_lambda_kernel<<<1, 256, 0, s>>>(dev);
  return cudaGetLastError();
}

cudaError_t launch_sgd_bias(float* b, const float* gb, float lr, int N, cudaStream_t s) {
  ProfScope ps(FW_PROF_MISC, s);
  sgd_bias_kernel<<<(N + 255) / 256, 256, 0, s>>>(b, gb, lr, N);
  return cudaGetLastError();
}

cudaError_t launch_sgd_bias_group(const GroupDev& g, const PtrTable& b, const PtrTable& gb, float lr, int max_N,
                                  cudaStream_t s) {
  ProfScope ps(FW_PROF_MISC, s);
  sgd_bias_group_kernel<<<dim3((max_N + 255) / 256, g.n), 256, 0, s>>>(g, b, gb, lr);
  return cudaGetLastError();
}

cudaError_t launch_axpy_step(float* W, const float* G, float lr, int64_t n, cudaStream_t s) {
  int blocks = (int)((n + 1023) / 1024);
  if (blocks > 2368) blocks = 2368;
  if (blocks < 1) blocks = 1;
  ProfScope ps(FW_PROF_MISC, s);
  axpy_step_kernel<<<blocks, 256, 0, s>>>(W, G, lr, n);
  return cudaGetLastError();
}

}  // namespace fw
