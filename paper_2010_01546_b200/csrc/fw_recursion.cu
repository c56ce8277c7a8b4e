// Recursive condition-number reduction (Sec. 4): one step is a fixed sequence
// of passes over the layer's M x M state, each pass one launch batched over all
// layers of the group (grid.y = layer).  Every pass is a row-wise product
// y = A x with A row-major: a warp owns rows, lanes stride the columns with
// 128-bit loads, partial sums are reduced by warp shuffles.  Scalars (m',
// |set|, norms, lambda_e, a_e) never leave the device; a pass recomputes what
// it needs from per-block partial sums written by the previous pass, always in
// the same order, so results are reproducible run to run.
//
//   pass ROWNORM  xi_m^2 = ||Phiy e_m||^2                         (Eq. 45; Phiy is kept exactly symmetric)
//   pass CORR     m' = argmax xi (lowest index on ties), c = Phiy (Phiy e_m')   (Eqs. 46-47)
//   pass ALIGN    set M = {|c_m| >= max(c_rel xi_m' xi_m, c_abs)}, v~ = (1/|M|) sum Phiy e_m / c_m  (Eqs. 48-49)
//   pass POWER    u = Phiy (prev / ||prev||), P times
//   pass FINAL    v = prev/||prev|| (Eq. 50), u = Phiy v, lambda_e = v.u (Eq. 36); t = T^T v
//   pass UPDATE   g_e, a_e (Eqs. 40-41); Q (Eq. 44), T (Eq. 42), Phiy rank updates
#include <cstdlib>
#include "fw_internal.h"

namespace fw {
namespace {

constexpr int RB = kGemvRowsPerBlock;      // rows per CTA of the update kernel and of the default pass shape
constexpr int WARPS = kGemvThreads / 32;   // 8
// Pass shapes (rows per warp R, column positions per trip C); a CTA covers 8 R rows.  Measured:
//   (4, 1)  many CTAs per SM (64 layers of the stress sweep): the lightest loop at four CTAs per SM
//   (4, 2)  a handful of layers: all 8 row loads of a trip issued before any is used (the bytes a warp keeps in
//           flight set the bandwidth it reaches when few CTAs share an SM)
//   (2, 4)  fewer 32-row blocks than SMs: twice as many CTAs.  Fewer rows per warp than that lose more to the
//           shared-memory reads of x, which every row of a warp shares, than the extra CTAs gain.

enum { PASS_ROWNORM = 0, PASS_CORR = 1, PASS_ALIGN = 2, PASS_POWER = 3, PASS_FINAL = 4 };

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// Sum of n per-block partials in a fixed order, computed redundantly by every CTA.
__device__ float block_sum_partials(const float* p, int n, float* red) {
  float s = 0.f;
  for (int i = threadIdx.x; i < n; i += blockDim.x) s += p[i];
  s = warp_sum(s);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < WARPS; ++w) tot += red[w];
  __syncthreads();
  return tot;
}

// Row-block product: for the RB rows of this CTA compute dot(A[r,:], x) where x
// sits in shared memory (or, for ROWNORM, x = the row itself).  Products and sums
// are carried in fp64: the passes are bound by memory traffic, and the alignment
// weights 1/c_m of Eq. 49 amplify any rounding of c_m by up to 1/c_rel.
template <bool SELF, int R, int C>
__device__ __forceinline__ void rows_dot(const float* __restrict__ A, const float* xs, int M, int row0,
                                         float out[R]) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r0 = row0 + warp * R;
  double acc[R];
#pragma unroll
  for (int r = 0; r < R; ++r) acc[r] = 0.0;
  if ((M & 3) == 0) {
    const int M4 = M >> 2;
    const float4* x4 = reinterpret_cast<const float4*>(xs);
    const float4 z4 = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int c = lane; c < M4; c += 32 * C) {
      float4 a[C][R];
#pragma unroll
      for (int h = 0; h < C; ++h) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const int row = r0 + r;
          a[h][r] = (row < M && c + 32 * h < M4)
                        ? __ldg(reinterpret_cast<const float4*>(A + (int64_t)row * M) + c + 32 * h) : z4;
        }
      }
#pragma unroll
      for (int h = 0; h < C; ++h) {
        double x0 = 0, x1 = 0, x2 = 0, x3 = 0;
        if (!SELF && c + 32 * h < M4) { const float4 xv = x4[c + 32 * h]; x0 = xv.x; x1 = xv.y; x2 = xv.z; x3 = xv.w; }
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const double ax = a[h][r].x, ay = a[h][r].y, az = a[h][r].z, aw = a[h][r].w;
          if (SELF) {
            acc[r] = fma(ax, ax, acc[r]); acc[r] = fma(ay, ay, acc[r]);
            acc[r] = fma(az, az, acc[r]); acc[r] = fma(aw, aw, acc[r]);
          } else {
            acc[r] = fma(ax, x0, acc[r]); acc[r] = fma(ay, x1, acc[r]);
            acc[r] = fma(az, x2, acc[r]); acc[r] = fma(aw, x3, acc[r]);
          }
        }
      }
    }
  } else {
    for (int c = lane; c < M; c += 32) {
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const int row = r0 + r;
        if (row < M) {
          const double a = A[(int64_t)row * M + c];
          acc[r] = fma(a, SELF ? a : (double)xs[c], acc[r]);
        }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < R; ++r) {
    double x = acc[r];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    out[r] = (float)x;
  }
}

// dynamic shared memory: x vector (M floats, 16-byte aligned)
extern __shared__ __align__(16) float smem_x[];

template <int PASS, int R, int C>
__global__ void __launch_bounds__(kGemvThreads, (C == 1) ? 4 : 2) recursion_pass_kernel(const __grid_constant__ GroupDev g,
                                                                      int src_slot, int dst_slot) {
  const LayerDev* L = g.layer[blockIdx.y];
  const int M = L->M;
  constexpr int RBk = WARPS * R;                // rows per CTA of this shape
  const int row0 = blockIdx.x * RBk;
  if (row0 >= M) return;
  // FINAL only: blockIdx.z == 1 is the product t = T^T v, blockIdx.z == 2 (leaky layers) q = P^T v
  const int zi = (PASS == PASS_FINAL) ? (int)blockIdx.z : 0;
  const bool second = zi != 0;
  if (zi == 2 && L->gamma == 1.f) return;
  const int nblk = (M + RBk - 1) / RBk;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __shared__ float red[WARPS];
  __shared__ float sred[kGemvThreads];
  __shared__ int ired[kGemvThreads];
  float* xs = smem_x;

  float res[R];
  if (PASS == PASS_ROWNORM) {
    rows_dot<true, R, C>(L->Phiy, nullptr, M, row0, res);
    if (lane == 0) {
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const int row = row0 + warp * R + r;
        if (row < M) L->xi2[row] = res[r];
      }
    }
    return;
  }

  if (PASS == PASS_CORR) {
    // argmax of xi^2 (monotone in xi), lowest index on ties
    float best = -1.f;
    int bi = 0x7fffffff;
    for (int m = threadIdx.x; m < M; m += blockDim.x) {
      const float x = L->xi2[m];
      if (x > best) { best = x; bi = m; }
    }
    sred[threadIdx.x] = best;
    ired[threadIdx.x] = bi;
    __syncthreads();
    for (int o = kGemvThreads / 2; o > 0; o >>= 1) {
      if (threadIdx.x < o) {
        const float xo = sred[threadIdx.x + o];
        const int io = ired[threadIdx.x + o];
        if (xo > sred[threadIdx.x] || (xo == sred[threadIdx.x] && io < ired[threadIdx.x])) {
          sred[threadIdx.x] = xo;
          ired[threadIdx.x] = io;
        }
      }
      __syncthreads();
    }
    int mp = ired[0];
    if (mp < 0 || mp >= M) mp = 0;   // all-NaN guard
    if (blockIdx.x == 0 && threadIdx.x == 0) L->iscal[IS_MPRIME] = mp;
    for (int m = threadIdx.x; m < M; m += blockDim.x) xs[m] = L->Phiy[(int64_t)mp * M + m];
    __syncthreads();
    rows_dot<false, R, C>(L->Phiy, xs, M, row0, res);
    if (lane == 0) {
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const int row = row0 + warp * R + r;
        if (row < M) L->cvec[row] = res[r];
      }
    }
    return;
  }

  if (PASS == PASS_ALIGN) {
    const int mp = L->iscal[IS_MPRIME];
    int cnt = 0;
    if (L->init == FW_INIT_MAXCOL) {
      for (int m = threadIdx.x; m < M; m += blockDim.x) xs[m] = (m == mp) ? 1.f : 0.f;
      cnt = 1;
    } else {
      const float xi_mp = sqrtf(L->xi2[mp]);
      const float c_rel = L->c_rel, c_abs = L->c_abs;
      int local = 0;
      for (int m = threadIdx.x; m < M; m += blockDim.x) {
        const float c = L->cvec[m];
        const float thr = fmaxf(c_rel * xi_mp * sqrtf(L->xi2[m]), c_abs);
        const bool in = fabsf(c) >= thr;       // false for NaN
        xs[m] = in ? (1.f / c) : 0.f;
        local += in ? 1 : 0;
      }
      ired[threadIdx.x] = local;
      __syncthreads();
      for (int o = kGemvThreads / 2; o > 0; o >>= 1) {
        if (threadIdx.x < o) ired[threadIdx.x] += ired[threadIdx.x + o];
        __syncthreads();
      }
      cnt = ired[0];
      if (blockIdx.x == 0) {
        for (int m = threadIdx.x; m < M; m += blockDim.x) L->wvec[m] = xs[m];
      }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) L->iscal[IS_SETSIZE] = cnt;
    __syncthreads();
    rows_dot<false, R, C>(L->Phiy, xs, M, row0, res);
    const float inv_cnt = cnt > 0 ? 1.f / (float)cnt : 0.f;
    float sq = 0.f;
    if (lane == 0) {
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const int row = row0 + warp * R + r;
        if (row < M) {
          const float y = res[r] * inv_cnt;
          L->pv[dst_slot][row] = y;
          sq = fmaf(y, y, sq);
        }
      }
      red[warp] = sq;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < WARPS; ++w) s += red[w];
      L->part[dst_slot * L->part_stride + blockIdx.x] = s;
    }
    return;
  }

  // POWER / FINAL: x = prev / ||prev||
  {
    const float n2 = block_sum_partials(L->part + src_slot * L->part_stride, nblk, red);
    const float inv = (n2 > 0.f && isfinite(n2)) ? rsqrtf(n2) : 0.f;
    // one Newton step so that inv is accurate to fp32 rounding
    const float invr = inv > 0.f ? inv * (1.5f - 0.5f * n2 * inv * inv) : 0.f;
    const float* prev = L->pv[src_slot];
    for (int m = threadIdx.x; m < M; m += blockDim.x) xs[m] = prev[m] * invr;
    __syncthreads();
    const float* A = zi == 0 ? L->Phiy : (zi == 1 ? L->Tt : L->tmp);
    rows_dot<false, R, C>(A, xs, M, row0, res);
    if (PASS == PASS_POWER) {
      float sq = 0.f;
      if (lane == 0) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const int row = row0 + warp * R + r;
          if (row < M) {
            L->pv[dst_slot][row] = res[r];
            sq = fmaf(res[r], res[r], sq);
          }
        }
        red[warp] = sq;
      }
      __syncthreads();
      if (threadIdx.x == 0) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < WARPS; ++w) s += red[w];
        L->part[dst_slot * L->part_stride + blockIdx.x] = s;
      }
    } else {  // FINAL
      if (second) {
        if (lane == 0) {
#pragma unroll
          for (int r = 0; r < R; ++r) {
            const int row = row0 + warp * R + r;
            if (row < M) (zi == 1 ? L->t : L->cvec)[row] = res[r];
          }
        }
      } else {
        float dt = 0.f;
        if (lane == 0) {
#pragma unroll
          for (int r = 0; r < R; ++r) {
            const int row = row0 + warp * R + r;
            if (row < M) {
              L->u[row] = res[r];
              L->v[row] = xs[row];
              dt = fmaf(xs[row], res[r], dt);
            }
          }
          red[warp] = dt;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
          float s = 0.f;
#pragma unroll
          for (int w = 0; w < WARPS; ++w) s += red[w];
          L->part[2 * L->part_stride + blockIdx.x] = s;       // slot 2: lambda_e partials
          if (blockIdx.x == 0) L->scal[SC_LAST_NORM2] = n2;    // norm^2 of the last iterate (validity check)
        }
      }
    }
  }
}

// Rank updates at gamma == 1 for a block of rows.  Element-wise, 128-bit accesses.
//   Q   += a (a + 2) t t^T                               (Eq. 44)
//   T^T += a t v^T            i.e. T += a v t^T          (Eq. 42)
//   Phiy += a (v u^T + u v^T) + a^2 lambda_e v v^T        (from Phiy = T Phix T^T)
// The Phiy and Q terms are evaluated symmetrically in (i, j) so both stay exactly symmetric.
__global__ void __launch_bounds__(kGemvThreads) recursion_update_kernel(const __grid_constant__ GroupDev g,
                                                                        const __grid_constant__ PtrTable traces,
                                                                        int step, int pass_rows) {
  const LayerDev* L = g.layer[blockIdx.y];
  const int M = L->M;
  const int row0 = blockIdx.x * RB;
  if (row0 >= M) return;
  const int nblk = (M + pass_rows - 1) / pass_rows;   // partials of lambda_e: one per CTA of the FINAL pass
  __shared__ float red[WARPS];
  const float lam_e = block_sum_partials(L->part + 2 * L->part_stride, nblk, red);
  const float n2 = L->scal[SC_LAST_NORM2];
  const int cnt = L->iscal[IS_SETSIZE];
  const bool ok = cnt > 0 && n2 > 0.f && isfinite(n2) && isfinite(lam_e);
  float g_e = 1.f, a = 0.f;
  if (ok) {
    g_e = L->delta * L->scal[SC_LAMBDA_BAR] / fmaxf(lam_e, L->eps);   // Eq. 40
    a = sqrtf(g_e) - 1.f;                                             // Eq. 41
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    L->scal[SC_LAMBDA_E] = lam_e; L->scal[SC_G_E] = g_e; L->scal[SC_A_E] = a;
    if (!ok) L->iscal[IS_STATUS_NOSUB] = 1;
    if (!isfinite(n2) || !isfinite(lam_e)) L->iscal[IS_STATUS_NONFINITE] = 1;   // NaN / Inf in the state
    float* tr = const_cast<float*>(reinterpret_cast<const float*>(traces.p[blockIdx.y]));
    if (tr) {
      tr[4 * step + 0] = lam_e; tr[4 * step + 1] = g_e;
      tr[4 * step + 2] = (float)cnt; tr[4 * step + 3] = (float)L->iscal[IS_MPRIME];
    }
  }
  if (L->gamma != 1.f) return;   // leaky layers are updated by recursion_update_leaky_kernel
  if (a == 0.f) return;          // gamma == 1 and a == 0: nothing changes
  const float aq = a * (a + 2.f);
  const float a2l = a * a * lam_e;
  const float* v = L->v; const float* u = L->u; const float* t = L->t;
  const int rows = min(RB, M - row0);
  if ((M & 3) == 0) {
    const int M4 = M >> 2;
    const int total = rows * M4;
    // two elements per trip, all six matrix loads issued before any is used: with few CTAs per SM (a handful of
    // layers) the bytes a thread keeps in flight set the bandwidth the kernel reaches
    for (int e0 = threadIdx.x; e0 < total; e0 += 2 * blockDim.x) {
      float4 q[2], tt[2], p[2];
      int64_t off[2];
      int ri[2], cj[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int e = e0 + h * blockDim.x;
        const bool in = e < total;
        const int r = in ? e / M4 : 0, c4 = in ? e - r * M4 : 0;
        ri[h] = in ? row0 + r : -1; cj[h] = c4;
        off[h] = (int64_t)(row0 + r) * M4 + c4;
        if (in) {
          q[h] = reinterpret_cast<const float4*>(L->Q)[off[h]];
          tt[h] = reinterpret_cast<const float4*>(L->Tt)[off[h]];
          p[h] = reinterpret_cast<const float4*>(L->Phiy)[off[h]];
        }
      }
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if (ri[h] < 0) continue;
        const int i = ri[h];
        const float vi = v[i], ui = u[i], ti = t[i];
        const float4 vj = reinterpret_cast<const float4*>(v)[cj[h]];
        const float4 uj = reinterpret_cast<const float4*>(u)[cj[h]];
        const float4 tj = reinterpret_cast<const float4*>(t)[cj[h]];
#define FW_UPD(X)                                                                              \
        q[h].X = __fadd_rn(q[h].X, __fmul_rn(aq, __fmul_rn(ti, tj.X)));                          \
        tt[h].X = fmaf(a * ti, vj.X, tt[h].X);                                                   \
        p[h].X = __fadd_rn(p[h].X, __fadd_rn(__fmul_rn(a, __fadd_rn(__fmul_rn(vi, uj.X), __fmul_rn(ui, vj.X))), \
                                             __fmul_rn(a2l, __fmul_rn(vi, vj.X))));
        FW_UPD(x) FW_UPD(y) FW_UPD(z) FW_UPD(w)
#undef FW_UPD
        reinterpret_cast<float4*>(L->Q)[off[h]] = q[h];
        reinterpret_cast<float4*>(L->Tt)[off[h]] = tt[h];
        reinterpret_cast<float4*>(L->Phiy)[off[h]] = p[h];
      }
    }
  } else {
    const int total = rows * M;
    for (int e = threadIdx.x; e < total; e += blockDim.x) {
      const int r = e / M, j = e - r * M;
      const int i = row0 + r;
      const float vi = v[i], ui = u[i], ti = t[i];
      const int64_t off = (int64_t)i * M + j;
      L->Q[off] = __fadd_rn(L->Q[off], __fmul_rn(aq, __fmul_rn(ti, t[j])));
      L->Tt[off] = fmaf(a * ti, v[j], L->Tt[off]);
      L->Phiy[off] = __fadd_rn(L->Phiy[off],
                               __fadd_rn(__fmul_rn(a, __fadd_rn(__fmul_rn(vi, u[j]), __fmul_rn(ui, v[j]))),
                                         __fmul_rn(a2l, __fmul_rn(vi, v[j]))));
    }
  }
}


// Rank updates with leakage gamma < 1 (Eqs. 42, 44).  With P = T Phix kept as Pt = P^T and q = P^T v:
//   Q    <- g^2 (Q + a(a+2) t t^T) + (1-g)^2 I + g(1-g) (a (v t^T + t v^T) + T + T^T)
//   T^T  <- g (T^T + a t v^T) + (1-g) I
//   Phiy <- g^2 (Phiy + a (v u^T + u v^T) + a^2 lambda_e v v^T) + g(1-g) (P + P^T + a (v q^T + q v^T)) + (1-g)^2 Phix
//   P^T  <- g (P^T + a q v^T) + (1-g) Phix
// T + T^T and P + P^T need the transposed element, so a CTA owns the pair of 32x32 tiles (bi, bj), (bj, bi).
// Q and Phiy are computed for the upper tile and mirrored, which keeps them exactly symmetric.
__global__ void __launch_bounds__(256) recursion_update_leaky_kernel(const __grid_constant__ GroupDev g) {
  const LayerDev* L = g.layer[blockIdx.z];
  const float gm = L->gamma;
  if (gm == 1.f) return;
  const int M = L->M;
  const int bi = blockIdx.y, bj = blockIdx.x;
  if (bj < bi || bi * 32 >= M || bj * 32 >= M) return;
  const float a = L->scal[SC_A_E], lam_e = L->scal[SC_LAMBDA_E];
  const float g2 = gm * gm, og = 1.f - gm, og2 = og * og, gog = gm * og;
  const float aq = a * (a + 2.f), a2l = a * a * lam_e;
  const float* v = L->v; const float* u = L->u; const float* t = L->t; const float* q = L->cvec;
  __shared__ float TtA[32][33], TtB[32][33], PtA[32][33], PtB[32][33], Qm[32][33], Ym[32][33];
  const int tx = threadIdx.x, ty = threadIdx.y;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int rr = ty + 8 * r;
    const int iA = bi * 32 + rr, jA = bj * 32 + tx;      // element of block (bi, bj)
    const int iB = bj * 32 + rr, jB = bi * 32 + tx;      // element of block (bj, bi)
    const bool inA = iA < M && jA < M, inB = iB < M && jB < M;
    TtA[rr][tx] = inA ? L->Tt[(int64_t)iA * M + jA] : 0.f;
    PtA[rr][tx] = inA ? L->tmp[(int64_t)iA * M + jA] : 0.f;
    TtB[rr][tx] = inB ? L->Tt[(int64_t)iB * M + jB] : 0.f;
    PtB[rr][tx] = inB ? L->tmp[(int64_t)iB * M + jB] : 0.f;
  }
  __syncthreads();
  // block (bi, bj): rows i (local rr), columns j (local tx)
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int rr = ty + 8 * r;
    const int i = bi * 32 + rr, j = bj * 32 + tx;
    float qn = 0.f, yn = 0.f;
    if (i < M && j < M) {
      const int64_t off = (int64_t)i * M + j;
      const float vi = v[i], vj = v[j], ti = t[i], tj = t[j], ui = u[i], uj = u[j], qi = q[i], qj = q[j];
      const float dij = (i == j) ? 1.f : 0.f;
      const float sumT = __fadd_rn(TtA[rr][tx], TtB[tx][rr]);
      const float sumP = __fadd_rn(PtA[rr][tx], PtB[tx][rr]);
      qn = __fadd_rn(__fadd_rn(__fmul_rn(g2, __fadd_rn(L->Q[off], __fmul_rn(aq, __fmul_rn(ti, tj)))), __fmul_rn(og2, dij)),
                     __fmul_rn(gog, __fadd_rn(__fmul_rn(a, __fadd_rn(__fmul_rn(vi, tj), __fmul_rn(ti, vj))), sumT)));
      const float inner = __fadd_rn(L->Phiy[off], __fadd_rn(__fmul_rn(a, __fadd_rn(__fmul_rn(vi, uj), __fmul_rn(ui, vj))),
                                                            __fmul_rn(a2l, __fmul_rn(vi, vj))));
      yn = __fadd_rn(__fadd_rn(__fmul_rn(g2, inner),
                               __fmul_rn(gog, __fadd_rn(sumP, __fmul_rn(a, __fadd_rn(__fmul_rn(vi, qj), __fmul_rn(qi, vj)))))),
                     __fmul_rn(og2, L->Phix[off]));
      // diagonal tiles: every (i, j) of the tile is computed here; the expressions are symmetric in (i, j)
      if (bi != bj || j >= i) { L->Q[off] = qn; L->Phiy[off] = yn; }
      L->Tt[off] = fmaf(gm, fmaf(a * ti, vj, TtA[rr][tx]), og * dij);
      L->tmp[off] = fmaf(gm, fmaf(a * qi, vj, PtA[rr][tx]), og * L->Phix[off]);
    }
    Qm[rr][tx] = qn; Ym[rr][tx] = yn;
  }
  __syncthreads();
  // mirror block (bj, bi): rows j' = bj*32 + rr, columns i' = bi*32 + tx
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int rr = ty + 8 * r;
    const int i = bj * 32 + rr, j = bi * 32 + tx;
    if (i < M && j < M) {
      const int64_t off = (int64_t)i * M + j;
      if (bi != bj) {
        L->Q[off] = Qm[tx][rr]; L->Phiy[off] = Ym[tx][rr];
        const float ti = t[i], qi = q[i], vj = v[j];
        L->Tt[off] = gm * fmaf(a * ti, vj, TtB[rr][tx]);                       // off-diagonal tile: no identity term
        L->tmp[off] = fmaf(gm, fmaf(a * qi, vj, PtB[rr][tx]), og * L->Phix[off]);
      } else if (j < i) {
        L->Q[off] = Qm[tx][rr]; L->Phiy[off] = Ym[tx][rr];
      }
    }
  }
}

// Qs <- beta Qs + (1 - beta) Q   (Eq. 35)
__global__ void __launch_bounds__(256) smooth_kernel(const __grid_constant__ GroupDev g) {
  const LayerDev* L = g.layer[blockIdx.y];
  if (L->Qs == L->Q) return;
  const int64_t n = (int64_t)L->M * L->M;
  const float beta = L->beta;
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x)
    L->Qs[e] = fmaf(beta, L->Qs[e], (1.f - beta) * L->Q[e]);
}

}  // namespace

template <int R, int C>
static cudaError_t recursion_step_launches(const GroupDev& g, int P, int step, const PtrTable& traces, int max_M,
                                           bool any_leaky, cudaStream_t s) {
  constexpr int RBk = WARPS * R;
  const int nblk = (max_M + RBk - 1) / RBk;
  const size_t shm = (size_t)((max_M + 3) & ~3) * sizeof(float);
  dim3 grid(nblk, g.n), block(kGemvThreads);
  { ProfScope ps(FW_PROF_RECUR_MV, s); recursion_pass_kernel<PASS_ROWNORM, R, C><<<grid, block, shm, s>>>(g, 0, 0); }
  { ProfScope ps(FW_PROF_RECUR_MV, s); recursion_pass_kernel<PASS_CORR, R, C><<<grid, block, shm, s>>>(g, 0, 0); }
  { ProfScope ps(FW_PROF_RECUR_MV, s); recursion_pass_kernel<PASS_ALIGN, R, C><<<grid, block, shm, s>>>(g, 0, 0); }
  int cur = 0;
  for (int p = 0; p < P; ++p) {
    ProfScope ps(FW_PROF_RECUR_MV, s);
    recursion_pass_kernel<PASS_POWER, R, C><<<grid, block, shm, s>>>(g, cur, cur ^ 1);
    cur ^= 1;
  }
  dim3 grid2(nblk, g.n, any_leaky ? 3 : 2);
  { ProfScope ps(FW_PROF_RECUR_MV, s); recursion_pass_kernel<PASS_FINAL, R, C><<<grid2, block, shm, s>>>(g, cur, 0); }
  dim3 gridu((max_M + RB - 1) / RB, g.n);
  { ProfScope ps(FW_PROF_RECUR_UPD, s); recursion_update_kernel<<<gridu, block, 0, s>>>(g, traces, step, RBk); }
  if (any_leaky) {
    const int t32 = (max_M + 31) / 32;
    ProfScope ps(FW_PROF_RECUR_UPD, s);
    recursion_update_leaky_kernel<<<dim3(t32, t32, g.n), dim3(32, 8), 0, s>>>(g);
  }
  return cudaGetLastError();
}

// row_blocks: 32-row blocks that have rows to work on, summed over the group's layers
cudaError_t launch_recursion_step(const GroupDev& g, int P, int step, const PtrTable& traces, int max_M,
                                  bool any_leaky, int row_blocks, cudaStream_t s) {
  const int forced = tuning().pass_shape;   // tuning aid
  if (forced == 42) return recursion_step_launches<4, 2>(g, P, step, traces, max_M, any_leaky, s);
  if (forced == 24) return recursion_step_launches<2, 4>(g, P, step, traces, max_M, any_leaky, s);
  if (forced == 18) return recursion_step_launches<1, 8>(g, P, step, traces, max_M, any_leaky, s);
  if (forced == 41) return recursion_step_launches<4, 1>(g, P, step, traces, max_M, any_leaky, s);
  if (row_blocks < 148) return recursion_step_launches<2, 4>(g, P, step, traces, max_M, any_leaky, s);
  if (row_blocks < 8 * 148) return recursion_step_launches<4, 2>(g, P, step, traces, max_M, any_leaky, s);
  return recursion_step_launches<4, 1>(g, P, step, traces, max_M, any_leaky, s);
}

cudaError_t launch_smooth(const GroupDev& g, int max_M, cudaStream_t s) {
  int64_t n = (int64_t)max_M * max_M;
  int bx = (int)((n + 1023) / 1024);
  if (bx > 1184) bx = 1184;
  if (bx < 1) bx = 1;
  ProfScope ps(FW_PROF_SMOOTH, s);
  smooth_kernel<<<dim3(bx, g.n), 256, 0, s>>>(g);
  return cudaGetLastError();
}

}  // namespace fw
