// Whitening from the eigenvalue decomposition (Sec. 2, Eqs. 7-10; practical gains Eqs. 32 and 34): the method the
// recursion of Sec. 4 is measured against.  Phi = V Lambda V^T is computed by one-sided Jacobi rotations in fp64:
// with W = Phi V (starting from W = Phi, V = I), the rotation of a pair of columns (p, q) that makes w_p, w_q
// orthogonal is applied to W and V alike; when all columns of W are orthogonal, V holds the eigenvectors and
// lambda_m = v_m . w_m.  A pair touches nothing but its own two columns, so the M / 2 disjoint pairs of a round
// (round-robin tournament: M - 1 rounds cover every pair once) run on different warps with one grid barrier per
// round, all layers of a group in the same launch.  Columns are stored as rows (Phi is symmetric), fp64 throughout:
// T = Phi^(-1/2) carries the rounding of the decomposition times cond(Phi) / 2, which fp32 cannot afford.
//
// Then T = V diag(sqrt g) V^T (Eq. 9), Q = T^T T = V diag(g) V^T and Phi_y = T Phi T^T = V diag(g lambda) V^T come
// out of one pass over V.
#include <cstring>

#include "fw_internal.h"

namespace fw {
namespace {

constexpr int ET = 512;               // threads per CTA of the rotation kernel: a warp per pair
constexpr int kRegCols = 20;          // columns per lane held in registers: rows of up to 640 entries are read once
constexpr int EW = ET / 32;
constexpr int kMaxSweeps = 30;
constexpr uint32_t kEvdSpin = 1u << 22;
constexpr double kOrthTol = 1e-14;    // |w_p . w_q| <= tol |w_p| |w_q|: the pair is left alone

struct EvdLayer {
  const float* A;    // M x M symmetric input (fp32, row-major)
  double* W;         // M x M: row m is column m of Phi V
  double* V;         // M x M: row m is eigenvector m (null: eigenvalues only)
  int32_t* status;   // time-out word of the layer
  int32_t M;
  int32_t n;         // players of the tournament: M rounded up to even (an odd M plays against a dummy)
};

struct EvdArgs {
  EvdLayer l[FW_MAX_GROUP];
  int32_t pair0[FW_MAX_GROUP + 1];   // first pair of each layer in the flat list of a round (n / 2 pairs per layer)
  int32_t nl;
  int32_t rounds_max;                // n_max - 1
  int32_t nctas;
  int32_t* bar;                      // [0] arrivals, [1] abort, [2 + s] rotations of sweep s (zeroed before the launch)
};

__device__ __forceinline__ double warp_sum_d(double x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// Grid barrier number idx (from 1) of this launch; false once the launch is aborted.  The wait is bounded.
__device__ bool evd_grid_barrier(const EvdArgs& a, uint32_t idx, int* s_abort) {
  __syncthreads();
  if (threadIdx.x == 0) {
    volatile int* ctr = a.bar;
    volatile int* ab = a.bar + 1;
    if (*s_abort == 0) {
      __threadfence();
      atomicAdd(a.bar, 1);
      const uint32_t target = idx * (uint32_t)a.nctas;
      bool ok = false;
      for (uint32_t i = 0; i < kEvdSpin; ++i) {
        if ((int32_t)((uint32_t)*ctr - target) >= 0) { ok = true; break; }
        if ((i & 63u) == 63u && *ab != 0) break;
      }
      if (!ok) {
        *ab = 1;
        for (int i = 0; i < a.nl; ++i) atomicExch(a.l[i].status, 601);
        *s_abort = 1;
      }
      __threadfence();
    }
  }
  __syncthreads();
  return *s_abort == 0;
}

__global__ void __launch_bounds__(ET, 1) jacobi_kernel(const __grid_constant__ EvdArgs a) {
  __shared__ int s_abort;
  __shared__ int s_rot;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gw = (int)blockIdx.x * EW + warp, nw = (int)gridDim.x * EW;
  if (threadIdx.x == 0) { s_abort = 0; s_rot = 0; }
  __syncthreads();
  // W = Phi, V = I
  for (int li = 0; li < a.nl; ++li) {
    const EvdLayer L = a.l[li];
    const int64_t mm = (int64_t)L.M * L.M;
    for (int64_t i = (int64_t)blockIdx.x * ET + threadIdx.x; i < mm; i += (int64_t)gridDim.x * ET) {
      L.W[i] = (double)L.A[i];
      if (L.V) L.V[i] = (i / L.M == i % L.M) ? 1.0 : 0.0;
    }
  }
  uint32_t bidx = 0;
  if (!evd_grid_barrier(a, ++bidx, &s_abort)) return;
  const int npairs = a.pair0[a.nl];
  for (int sweep = 0; sweep < kMaxSweeps; ++sweep) {
    for (int r = 0; r < a.rounds_max; ++r) {
      bool rotated = false;
      for (int t = gw; t < npairs; t += nw) {
        int li = 0;
#pragma unroll 1
        for (int i = 1; i < a.nl; ++i)
          if (t >= a.pair0[i]) li = i;
        const EvdLayer L = a.l[li];
        const int n1 = L.n - 1;
        if (r >= n1) continue;                      // this layer's sweep has fewer rounds
        const int k = t - a.pair0[li];
        int p, q;
        if (k == 0) { p = n1; q = r; }
        else { p = (r + k) % n1; q = (r - k + n1) % n1; }
        if (p > q) { const int x = p; p = q; q = x; }
        if (q >= L.M) continue;                     // the dummy player of an odd M
        const int M = L.M;
        double* wp = L.W + (int64_t)p * M;
        double* wq = L.W + (int64_t)q * M;
        double al = 0.0, be = 0.0, ga = 0.0;
        const bool in_regs = M <= 32 * kRegCols;
        double xr[kRegCols], yr[kRegCols];
        if (in_regs) {
          // every load of the two rows is in flight at once, and the rotation needs no second read
#pragma unroll
          for (int j = 0; j < kRegCols; ++j) {
            const int i = lane + 32 * j;
            xr[j] = i < M ? __ldcg(wp + i) : 0.0;
            yr[j] = i < M ? __ldcg(wq + i) : 0.0;
          }
#pragma unroll
          for (int j = 0; j < kRegCols; ++j) {
            al = fma(xr[j], xr[j], al); be = fma(yr[j], yr[j], be); ga = fma(xr[j], yr[j], ga);
          }
        } else {
          for (int i = lane; i < M; i += 32) {
            const double x = __ldcg(wp + i), y = __ldcg(wq + i);
            al = fma(x, x, al); be = fma(y, y, be); ga = fma(x, y, ga);
          }
        }
        al = warp_sum_d(al); be = warp_sum_d(be); ga = warp_sum_d(ga);
        if (!(fabs(ga) > kOrthTol * sqrt(al * be))) continue;
        rotated = true;
        // the rotation that makes the two columns orthogonal (the smaller of the two angles)
        const double zeta = (be - al) / (2.0 * ga);
        const double tt = (zeta >= 0.0 ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
        const double c = 1.0 / sqrt(1.0 + tt * tt), s = c * tt;
        if (in_regs) {
#pragma unroll
          for (int j = 0; j < kRegCols; ++j) {
            const int i = lane + 32 * j;
            if (i < M) {
              __stcg(wp + i, c * xr[j] - s * yr[j]);
              __stcg(wq + i, s * xr[j] + c * yr[j]);
            }
          }
        } else {
          for (int i = lane; i < M; i += 32) {
            const double x = __ldcg(wp + i), y = __ldcg(wq + i);
            __stcg(wp + i, c * x - s * y);
            __stcg(wq + i, s * x + c * y);
          }
        }
        if (L.V) {
          double* vp = L.V + (int64_t)p * M;
          double* vq = L.V + (int64_t)q * M;
          if (in_regs) {
#pragma unroll
            for (int j = 0; j < kRegCols; ++j) {
              const int i = lane + 32 * j;
              xr[j] = i < M ? __ldcg(vp + i) : 0.0;
              yr[j] = i < M ? __ldcg(vq + i) : 0.0;
            }
#pragma unroll
            for (int j = 0; j < kRegCols; ++j) {
              const int i = lane + 32 * j;
              if (i < M) {
                __stcg(vp + i, c * xr[j] - s * yr[j]);
                __stcg(vq + i, s * xr[j] + c * yr[j]);
              }
            }
          } else {
            for (int i = lane; i < M; i += 32) {
              const double x = __ldcg(vp + i), y = __ldcg(vq + i);
              __stcg(vp + i, c * x - s * y);
              __stcg(vq + i, s * x + c * y);
            }
          }
        }
      }
      if (rotated && lane == 0) s_rot = 1;
      // the sweep's count of rotations is complete before its last barrier
      if (r == a.rounds_max - 1) {
        __syncthreads();
        if (threadIdx.x == 0 && s_rot) { atomicAdd(a.bar + 2 + sweep, 1); s_rot = 0; }
      }
      if (!evd_grid_barrier(a, ++bidx, &s_abort)) return;
    }
    if (__ldcg(a.bar + 2 + sweep) == 0) break;      // every pair of every layer was already orthogonal
  }
}

struct FinishArgs {
  EvdLayer l[FW_MAX_GROUP];
  double* lam[FW_MAX_GROUP];       // M eigenvalues, in the order of the rows of V
  double* dvec[FW_MAX_GROUP];      // 3 M: sqrt(g), g, g lambda
  float* lam_sorted[FW_MAX_GROUP]; // optional output: eigenvalues in decreasing order
  float* kappa[FW_MAX_GROUP];      // optional output: rank estimate / M
  float eps[FW_MAX_GROUP];
  float g_max;                     // <= 0: g = 1 / max(lambda, eps) (Eq. 10); > 0: the gains of Eq. 34
};

// One CTA per layer: eigenvalues, their ranks, the rank estimate (Eq. 32 read as exp(-sum lbar log lbar)) and the gains.
__global__ void __launch_bounds__(1024) evd_finish_kernel(const __grid_constant__ FinishArgs a) {
  const EvdLayer L = a.l[blockIdx.x];
  const int M = L.M;
  double* lam = a.lam[blockIdx.x];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int m = warp; m < M; m += 32) {
    const double* w = L.W + (int64_t)m * M;
    double acc = 0.0;
    if (L.V) {
      const double* v = L.V + (int64_t)m * M;
      for (int i = lane; i < M; i += 32) acc = fma(v[i], w[i], acc);      // Rayleigh quotient v^T Phi v
      acc = warp_sum_d(acc);
    } else {
      for (int i = lane; i < M; i += 32) acc = fma(w[i], w[i], acc);      // |Phi v| (Phi positive semi-definite)
      acc = sqrt(warp_sum_d(acc));
    }
    if (lane == 0) lam[m] = acc;
  }
  __syncthreads();
  __shared__ double s_sum;
  __shared__ int s_ms;
  if (threadIdx.x == 0) {
    // fixed order: the sums decide an integer (the rank) and must not depend on the launch
    double S = 0.0;
    for (int m = 0; m < M; ++m) S += fmax(lam[m], 0.0);
    double H = 0.0;
    for (int m = 0; m < M; ++m) {
      const double lb = S > 0.0 ? fmax(lam[m], 0.0) / S : 0.0;
      if (lb > 0.0) H -= lb * log(lb);
    }
    const double ms_hat = exp(H);
    s_sum = S;
    int ms = (int)rint(ms_hat);
    if (ms < 1) ms = 1;
    if (ms > M) ms = M;
    s_ms = ms;
    if (a.kappa[blockIdx.x]) *a.kappa[blockIdx.x] = (float)(ms_hat / (double)M);
  }
  __syncthreads();
  const double S = s_sum;
  const int Ms = s_ms;
  double* dv = a.dvec[blockIdx.x];
  for (int m = threadIdx.x; m < M; m += blockDim.x) {
    const double lm = lam[m];
    int rank = 0;                                   // position of lambda_m in decreasing order
    for (int j = 0; j < M; ++j) {
      const double lj = lam[j];
      rank += (lj > lm || (lj == lm && j < m)) ? 1 : 0;
    }
    if (a.lam_sorted[blockIdx.x]) a.lam_sorted[blockIdx.x][rank] = (float)lm;
    if (dv) {
      double g;
      if (a.g_max <= 0.f) {
        g = 1.0 / fmax(lm, (double)a.eps[blockIdx.x]);                                  // Eq. 10
      } else {
        const double lb = S > 0.0 ? fmax(lm, 0.0) / S : 0.0;
        g = rank < Ms ? fmin(1.0 / fmax((double)M * lb, 1e-300), (double)a.g_max) : 1.0;   // Eq. 34
      }
      dv[m] = sqrt(g);
      dv[M + m] = g;
      dv[2 * M + m] = g * lm;
    }
  }
}

struct VdvArgs {
  EvdLayer l[FW_MAX_GROUP];
  const double* dvec[FW_MAX_GROUP];
  float* T[FW_MAX_GROUP];
  float* Q[FW_MAX_GROUP];
  float* Y[FW_MAX_GROUP];
  int32_t tile0[FW_MAX_GROUP + 1];   // flat grid over the 32 x 32 tiles of all layers
  int32_t nl;
};

// out_ij = sum_m d_m V_mi V_mj for the three weight vectors at once; the product V_mi V_mj is formed first, so
// entry (i, j) and entry (j, i) see the same operations in the same order: the outputs are exactly symmetric.
__global__ void __launch_bounds__(256) vdv_kernel(const __grid_constant__ VdvArgs a) {
  int li = 0;
#pragma unroll 1
  for (int i = 1; i < a.nl; ++i)
    if ((int)blockIdx.x >= a.tile0[i]) li = i;
  const EvdLayer L = a.l[li];
  const int M = L.M;
  const int nt = (M + 31) / 32;
  const int tile = (int)blockIdx.x - a.tile0[li];
  const int bi = tile / nt, bj = tile - bi * nt;
  __shared__ double sa[32][33], sb[32][33], sd[3][32];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;      // 32 x 8
  double acc[3][4];
#pragma unroll
  for (int o = 0; o < 3; ++o)
#pragma unroll
    for (int r = 0; r < 4; ++r) acc[o][r] = 0.0;
  const double* dv = a.dvec[li];
  for (int m0 = 0; m0 < M; m0 += 32) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int mm = m0 + ty + 8 * r;
      const int ci = bi * 32 + tx, cj = bj * 32 + tx;
      sa[ty + 8 * r][tx] = (mm < M && ci < M) ? L.V[(int64_t)mm * M + ci] : 0.0;
      sb[ty + 8 * r][tx] = (mm < M && cj < M) ? L.V[(int64_t)mm * M + cj] : 0.0;
    }
    if (threadIdx.x < 96) {
      const int o = threadIdx.x >> 5, mm = m0 + (threadIdx.x & 31);
      sd[o][threadIdx.x & 31] = mm < M ? dv[o * M + mm] : 0.0;
    }
    __syncthreads();
#pragma unroll 4
    for (int k = 0; k < 32; ++k) {
      const double bj_ = sb[k][tx];
      const double d0 = sd[0][k], d1 = sd[1][k], d2 = sd[2][k];
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const double pr = sa[k][ty + 8 * r] * bj_;
        acc[0][r] = fma(d0, pr, acc[0][r]);
        acc[1][r] = fma(d1, pr, acc[1][r]);
        acc[2][r] = fma(d2, pr, acc[2][r]);
      }
    }
    __syncthreads();
  }
  const int j = bj * 32 + tx;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int i = bi * 32 + ty + 8 * r;
    if (i < M && j < M) {
      const int64_t off = (int64_t)i * M + j;
      a.T[li][off] = (float)acc[0][r];
      a.Q[li][off] = (float)acc[1][r];
      a.Y[li][off] = (float)acc[2][r];
    }
  }
}

}  // namespace

// Scratch of one layer: W and V (fp64), eigenvalues and the three weight vectors, and the barrier words
size_t evd_scratch_bytes(int M) {
  return 2 * (size_t)M * M * sizeof(double) + 4 * (size_t)M * sizeof(double) + 1024;
}

// Decomposes src[i] (M x M fp32 symmetric) of every layer.  with_v: eigenvectors too, then T, Q, Phi_y are written to
// the three outputs (T is symmetric: it is its own transpose).  lam_out / kappa_out: optional per-layer outputs.
cudaError_t launch_evd(int n, const float* const* src, const int* layer_M, void* const* scratch,
                       int32_t* const* status, const float* eps, bool with_v, float g_max, float* const* T_out,
                       float* const* Q_out, float* const* Y_out, float* const* lam_out, float* const* kappa_out,
                       cudaStream_t s) {
  static int n_sm[64] = {0};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) dev = 0;
  if (n_sm[dev] == 0) {
    e = cudaDeviceGetAttribute(&n_sm[dev], cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
  }
  EvdArgs a;
  FinishArgs f;
  VdvArgs v;
  memset(&a, 0, sizeof(a)); memset(&f, 0, sizeof(f)); memset(&v, 0, sizeof(v));
  int pairs = 0, tiles = 0, n_max = 0;
  for (int i = 0; i < n; ++i) {
    const int M = layer_M[i];
    char* base = reinterpret_cast<char*>(scratch[i]);
    EvdLayer& l = a.l[i];
    l.A = src[i];
    l.W = reinterpret_cast<double*>(base + 1024);
    l.V = with_v ? l.W + (size_t)M * M : nullptr;
    l.status = status[i];
    l.M = M;
    l.n = M + (M & 1);
    a.pair0[i] = pairs;
    pairs += l.n / 2;
    if (l.n > n_max) n_max = l.n;
    f.l[i] = l; v.l[i] = l;
    f.lam[i] = l.W + 2 * (size_t)M * M;
    f.dvec[i] = with_v ? f.lam[i] + M : nullptr;
    f.lam_sorted[i] = lam_out ? lam_out[i] : nullptr;
    f.kappa[i] = kappa_out ? kappa_out[i] : nullptr;
    f.eps[i] = eps[i];
    v.dvec[i] = f.dvec[i];
    if (with_v) { v.T[i] = T_out[i]; v.Q[i] = Q_out[i]; v.Y[i] = Y_out[i]; }
    v.tile0[i] = tiles;
    tiles += ((M + 31) / 32) * ((M + 31) / 32);
  }
  a.pair0[n] = pairs; v.tile0[n] = tiles;
  a.nl = n; v.nl = n;
  a.rounds_max = n_max - 1;
  int nctas = n_sm[dev];
  if (nctas * EW > pairs) nctas = (pairs + EW - 1) / EW;
  if (nctas < 1) nctas = 1;
  a.nctas = nctas;
  a.bar = reinterpret_cast<int32_t*>(scratch[0]);
  f.g_max = g_max;
  e = cudaMemsetAsync(a.bar, 0, 1024, s);
  if (e != cudaSuccess) return e;
  {
    // n >= 2 players per layer, so every launch has at least one round
    void* args[] = {&a};
    ProfScope ps(FW_PROF_MISC, s);
    e = cudaLaunchCooperativeKernel((void*)jacobi_kernel, dim3(nctas), dim3(ET), args, 0, s);
    if (e != cudaSuccess) return e;
  }
  {
    ProfScope ps(FW_PROF_MISC, s);
    evd_finish_kernel<<<n, 1024, 0, s>>>(f);
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (with_v) {
    ProfScope ps(FW_PROF_MISC, s);
    vdv_kernel<<<tiles, 256, 0, s>>>(v);
    e = cudaGetLastError();
  }
  return e;
}

}  // namespace fw
