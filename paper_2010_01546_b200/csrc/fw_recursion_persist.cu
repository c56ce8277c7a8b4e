// Recursive condition-number reduction (Sec. 4) for layers too large for one
// cluster's shared memory, as ONE persistent cooperative launch for all K steps
// of a call: the passes of fw_recursion.cu (same arithmetic, same order of
// operations per row) separated by grid-wide barriers instead of kernel
// boundaries.
//
// Work split.  The rows of all layers of the group form one list, a row of a
// layer of size M weighing M; CTA c (one per SM) owns the c-th of nctas equal
// shares of it, in groups of four rows: one to a few contiguous row ranges
// ("segments"), each inside one layer.  A CTA owns its rows for the whole
// launch, so
//   - the leading rows of its segments stay in shared memory for all K steps
//     (as many as fit: all of Phi_y for a single layer up to M = 2304, about a
//     fifth of a ResNet-50-sized set), read from there by every pass and
//     written through on update;
//   - the rank update of a row (Q, T^T, Phi_y) also yields the squared norm of
//     the new row, which is the first pass of the next step.
// Vectors travel through global memory (they are small and L2-resident) and
// are read with L1 bypassed; every CTA recomputes the scalars it needs (norms,
// lambda_e, the argmax, the coherent set) from the full vectors in a fixed
// order, so all CTAs take bit-identical decisions and nothing depends on the
// number of CTAs.
//
// The grid barrier is a monotonic counter in the leading layer's workspace,
// compared wrap-safe against a target the host supplies; every wait is bounded
// and a wait that gives up raises a grid-wide abort flag, after which every CTA
// leaves at its next barrier and the host reports FW_ERR_TIMEOUT.
#include <climits>
#include <cstring>

#include "fw_internal.h"

namespace fw {
namespace {

constexpr int PT = 1024;             // threads per CTA: the streaming passes need every warp the SM can hold
constexpr int PW = PT / 32;          // warps
constexpr int PR = 4;                // rows per group of the work split (and per warp in the streaming shape)
constexpr int PC = 1;                // update pass: column positions per trip
constexpr int kMaxSegs = 16;
constexpr uint32_t kBarSpin = 1u << 22;

struct PersistArgs {
  GroupDev g;
  PtrTable traces;
  int64_t prefix[FW_MAX_GROUP + 1];   // cost (row groups x M) before each layer
  int32_t K, P;
  int32_t nctas;
  uint32_t bar_base;                  // value of the barrier counter when the launch starts
  int32_t* bar;                       // counter, abort flag (2 ints) in the leading layer's workspace
  int32_t* status;                    // time-out word of the leading layer
  int32_t vec_floats;                 // shared memory: 3 vectors of this many floats, then the row cache
  int32_t cache_floats;
};

struct Seg {
  const LayerDev* L;
  int layer;        // index in the group
  int M;
  int row0, nrows;  // rows owned
  int ncached;      // leading rows kept in shared memory
  int cache_off;    // float offset of their copy
  float n2;         // squared norm of the last iterate (set by the FINAL pass)
  int cnt;          // size of the coherent set
};

__device__ __forceinline__ float ldcg(const float* p) { return __ldcg(p); }

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// sum over the block of one value per thread, in a fixed order; the result is uniform over the block
__device__ float block_sum(float x, float* red) {
  x = warp_sum(x);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = x;
  __syncthreads();
  float t = 0.f;
#pragma unroll
  for (int w = 0; w < PW; ++w) t += red[w];
  return t;
}

__device__ __forceinline__ float inv_norm(float n2) {
  float inv = (n2 > 0.f && isfinite(n2)) ? rsqrtf(n2) : 0.f;
  return inv > 0.f ? inv * (1.5f - 0.5f * n2 * inv * inv) : 0.f;
}

// Grid barrier number `idx` of this launch (counting from 1).  Returns false once the launch is aborted.
__device__ bool grid_barrier(const PersistArgs& a, uint32_t idx, int* s_abort) {
  __syncthreads();
  if (threadIdx.x == 0) {
    volatile int* ctr = a.bar;
    volatile int* ab = a.bar + 1;
    if (*s_abort == 0) {
      __threadfence();
      atomicAdd(a.bar, 1);
      const uint32_t target = a.bar_base + idx * (uint32_t)a.nctas;
      bool ok = false;
      for (uint32_t i = 0; i < kBarSpin; ++i) {
        if ((int32_t)((uint32_t)*ctr - target) >= 0) { ok = true; break; }
        if ((i & 63u) == 63u && *ab != 0) break;
      }
      if (!ok) {
        *ab = 1;
        atomicExch(a.status, 501);
        *s_abort = 1;
      }
      __threadfence();
    }
  }
  __syncthreads();
  return *s_abort == 0;
}

// dot(A[row, :], x) for the rows of a segment; a row comes from the shared-memory cache or from global memory.
// SELF: x is the row itself (squared norm).  fp64 accumulation, columns in ascending order per lane -- the order
// the fused update below reproduces, whatever the shape.  Shape: a warp takes R rows at a time and C column
// positions per trip (R C loads of 16 bytes in flight per lane).  out(row, value) is called by lane 0.
template <bool SELF, int R, int C, class Out>
__device__ __forceinline__ void seg_rows_dot_shape(const float* __restrict__ A, const Seg& s, const float* cache,
                                                   const float* xs, Out out) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int M = s.M, M4 = M >> 2;
  const float4* x4 = reinterpret_cast<const float4*>(xs);
  const float4 z4 = make_float4(0.f, 0.f, 0.f, 0.f);
  const int ngroups = (s.nrows + R - 1) / R;
  for (int gidx = warp; gidx < ngroups; gidx += PW) {
    const bool from_global = gidx * R >= s.ncached;          // no row of this group is cached
    const float4* rp[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const int lr = gidx * R + r;
      if (lr >= s.nrows) rp[r] = nullptr;
      else if (lr < s.ncached) rp[r] = reinterpret_cast<const float4*>(cache + s.cache_off + (size_t)lr * M);
      else rp[r] = reinterpret_cast<const float4*>(A + (size_t)(s.row0 + lr) * M);
    }
    double acc[R];
#pragma unroll
    for (int r = 0; r < R; ++r) acc[r] = 0.0;
    for (int c = lane; c < M4; c += 32 * C) {
      float4 av[C][R];
      if (from_global) {
#pragma unroll
        for (int h = 0; h < C; ++h)
#pragma unroll
          for (int r = 0; r < R; ++r) av[h][r] = (rp[r] && c + 32 * h < M4) ? __ldg(rp[r] + c + 32 * h) : z4;
      } else {
#pragma unroll
        for (int h = 0; h < C; ++h)
#pragma unroll
          for (int r = 0; r < R; ++r) av[h][r] = (rp[r] && c + 32 * h < M4) ? rp[r][c + 32 * h] : z4;
      }
#pragma unroll
      for (int h = 0; h < C; ++h) {
        double x0 = 0, x1 = 0, x2 = 0, x3 = 0;
        if (!SELF && c + 32 * h < M4) { const float4 xv = x4[c + 32 * h]; x0 = xv.x; x1 = xv.y; x2 = xv.z; x3 = xv.w; }
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const double ax = av[h][r].x, ay = av[h][r].y, az = av[h][r].z, aw = av[h][r].w;
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
#pragma unroll
    for (int r = 0; r < R; ++r) {
      double x = acc[r];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
      if (lane == 0 && rp[r]) out(s.row0 + gidx * R + r, (float)x);
    }
  }
}

// Many rows: four rows per warp, one column position per trip (the lightest loop with every warp streaming).
// Few rows (a layer spread thin over the SMs, its rows in shared memory): one row per warp so that all warps work.
template <bool SELF, class Out>
__device__ __forceinline__ void seg_rows_dot(const float* __restrict__ A, const Seg& s, const float* cache,
                                             const float* xs, Out out) {
  if (s.nrows >= 2 * PW) seg_rows_dot_shape<SELF, 4, 1>(A, s, cache, xs, out);
  else seg_rows_dot_shape<SELF, 1, 4>(A, s, cache, xs, out);
}

extern __shared__ __align__(16) float psm[];

__global__ void __launch_bounds__(PT, 1) recursion_persistent_kernel(const __grid_constant__ PersistArgs a) {
  __shared__ Seg segs[kMaxSegs];
  __shared__ int s_nsegs, s_abort;
  __shared__ float red[PW];
  __shared__ float sredf[PW];
  __shared__ int sredi[PW + 1];
  float* xs = psm;                          // input vector of the current pass (later: v)
  float* us = psm + a.vec_floats;           // u, for the update
  float* ts = psm + 2 * a.vec_floats;       // t, for the update
  float* cache = psm + 3 * a.vec_floats;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int K = a.K, P = a.P;

  // ---- my share of the rows ----
  if (threadIdx.x == 0) {
    s_abort = 0;
    const int64_t W = a.prefix[a.g.n];
    const int64_t lo = W * (int64_t)blockIdx.x / a.nctas, hi = W * (int64_t)(blockIdx.x + 1) / a.nctas;
    int ns = 0, coff = 0;
    for (int l = 0; l < a.g.n && ns < kMaxSegs; ++l) {
      const LayerDev* L = a.g.layer[l];
      const int M = L->M;
      const int64_t G = (M + PR - 1) / PR;
      // row group g of this layer sits at cost prefix[l] + g M and belongs to the CTA whose share holds that point
      int64_t g_lo = (lo - a.prefix[l] + M - 1) / M, g_hi = (hi - a.prefix[l] + M - 1) / M;
      if (lo <= a.prefix[l]) g_lo = 0;
      if (g_lo < 0) g_lo = 0;
      if (g_hi > G) g_hi = G;
      if (hi <= a.prefix[l]) g_hi = 0;
      if (g_lo >= g_hi) continue;
      Seg& s = segs[ns++];
      s.L = L; s.layer = l; s.M = M;
      s.row0 = (int)(g_lo * PR);
      s.nrows = (int)min((int64_t)M, g_hi * PR) - s.row0;
      int fit = (a.cache_floats - coff) / M;
      if (fit < 0) fit = 0;
      s.ncached = min(fit, s.nrows);
      s.cache_off = coff;
      coff += s.ncached * M;
      s.n2 = 0.f; s.cnt = 0;
    }
    s_nsegs = ns;
  }
  __syncthreads();
  const int nsegs = s_nsegs;
  // ---- cached rows of Phi_y ----
  for (int si = 0; si < nsegs; ++si) {
    const Seg s = segs[si];
    const float4* src = reinterpret_cast<const float4*>(s.L->Phiy + (size_t)s.row0 * s.M);
    float4* dst = reinterpret_cast<float4*>(cache + s.cache_off);
    const int n4 = s.ncached * (s.M >> 2);
    for (int i = threadIdx.x; i < n4; i += PT) dst[i] = src[i];
  }
  __syncthreads();

  uint32_t bidx = 0;
  // ---- squared row norms of the state as it is (later steps get them from the update pass) ----   (Eq. 45)
  for (int si = 0; si < nsegs; ++si) {
    const Seg s = segs[si];
    float* xi2 = s.L->xi2;
    seg_rows_dot<true>(s.L->Phiy, s, cache, nullptr, [&](int row, float v) { xi2[row] = v; });
  }
  if (!grid_barrier(a, ++bidx, &s_abort)) return;

  for (int step = 0; step < K; ++step) {
    // ---- CORR: m' = argmax xi (lowest index on ties), c = Phi_y (Phi_y e_m')          (Eqs. 46-47) ----
    for (int si = 0; si < nsegs; ++si) {
      const Seg s = segs[si];
      const LayerDev* L = s.L;
      const int M = s.M;
      float best = -1.f;
      int bi = 0x7fffffff;
      for (int m = threadIdx.x; m < M; m += PT) {
        const float x = ldcg(L->xi2 + m);
        if (x > best) { best = x; bi = m; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float xo = __shfl_xor_sync(0xffffffffu, best, o);
        const int io = __shfl_xor_sync(0xffffffffu, bi, o);
        if (xo > best || (xo == best && io < bi)) { best = xo; bi = io; }
      }
      __syncthreads();
      if (lane == 0) { sredf[warp] = best; sredi[warp] = bi; }
      __syncthreads();
      if (threadIdx.x < 32) {
        best = threadIdx.x < PW ? sredf[threadIdx.x] : -1.f;
        bi = threadIdx.x < PW ? sredi[threadIdx.x] : 0x7fffffff;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const float xo = __shfl_xor_sync(0xffffffffu, best, o);
          const int io = __shfl_xor_sync(0xffffffffu, bi, o);
          if (xo > best || (xo == best && io < bi)) { best = xo; bi = io; }
        }
        if (threadIdx.x == 0) sredi[PW] = bi;
      }
      __syncthreads();
      int mp = sredi[PW];
      if (mp < 0 || mp >= M) mp = 0;   // all-NaN guard
      if (s.row0 == 0 && threadIdx.x == 0) L->iscal[IS_MPRIME] = mp;
      for (int m = threadIdx.x; m < M; m += PT) xs[m] = ldcg(L->Phiy + (size_t)mp * M + m);
      __syncthreads();
      float* cvec = L->cvec;
      seg_rows_dot<false>(L->Phiy, s, cache, xs, [&](int row, float v) { cvec[row] = v; });
      __syncthreads();
    }
    if (!grid_barrier(a, ++bidx, &s_abort)) return;

    // ---- ALIGN: coherent set, aligned average                                          (Eqs. 48-49) ----
    for (int si = 0; si < nsegs; ++si) {
      const Seg s = segs[si];
      const LayerDev* L = s.L;
      const int M = s.M;
      const int mp = __ldcg(L->iscal + IS_MPRIME);
      int cnt;
      if (L->init == FW_INIT_MAXCOL) {
        for (int m = threadIdx.x; m < M; m += PT) xs[m] = (m == mp) ? 1.f : 0.f;
        cnt = 1;
        __syncthreads();
      } else {
        const float xi_mp = sqrtf(ldcg(L->xi2 + mp));
        const float c_rel = L->c_rel, c_abs = L->c_abs;
        int local = 0;
        for (int m = threadIdx.x; m < M; m += PT) {
          const float c = ldcg(L->cvec + m);
          const float thr = fmaxf(c_rel * xi_mp * sqrtf(ldcg(L->xi2 + m)), c_abs);
          const bool in = fabsf(c) >= thr;       // false for NaN
          xs[m] = in ? (1.f / c) : 0.f;
          local += in ? 1 : 0;
        }
        cnt = (int)(block_sum((float)local, red) + 0.5f);
        if (s.row0 == 0)
          for (int m = threadIdx.x; m < M; m += PT) L->wvec[m] = xs[m];
      }
      if (threadIdx.x == 0) {
        segs[si].cnt = cnt;
        if (s.row0 == 0) L->iscal[IS_SETSIZE] = cnt;
      }
      __syncthreads();
      const float inv_cnt = cnt > 0 ? 1.f / (float)cnt : 0.f;
      float* dst = L->pv[0];
      seg_rows_dot<false>(L->Phiy, s, cache, xs, [&](int row, float v) { dst[row] = v * inv_cnt; });
      __syncthreads();
    }
    if (!grid_barrier(a, ++bidx, &s_abort)) return;

    // ---- POWER x P, then FINAL: x = prev / ||prev||, y = Phi_y x (and t = T^T x in the final pass) ----
    int cur = 0;
    for (int p = 0; p <= P; ++p) {
      const bool final_pass = (p == P);
      for (int si = 0; si < nsegs; ++si) {
        const Seg s = segs[si];
        const LayerDev* L = s.L;
        const int M = s.M;
        const float* prev = L->pv[cur];
        float sq = 0.f;
        for (int m = threadIdx.x; m < M; m += PT) { const float x = ldcg(prev + m); xs[m] = x; sq = fmaf(x, x, sq); }
        const float n2 = block_sum(sq, red);
        const float invr = inv_norm(n2);
        for (int m = threadIdx.x; m < M; m += PT) xs[m] *= invr;
        __syncthreads();
        if (!final_pass) {
          float* dst = L->pv[cur ^ 1];
          seg_rows_dot<false>(L->Phiy, s, cache, xs, [&](int row, float v) { dst[row] = v; });
        } else {
          if (threadIdx.x == 0) segs[si].n2 = n2;
          float* u = L->u; float* t = L->t; float* v = L->v;
          seg_rows_dot<false>(L->Phiy, s, cache, xs, [&](int row, float val) { u[row] = val; v[row] = xs[row]; });
          Seg st = s;
          st.ncached = 0;                      // T^T is not cached
          seg_rows_dot<false>(L->Tt, st, cache, xs, [&](int row, float val) { t[row] = val; });
        }
        __syncthreads();
      }
      if (!grid_barrier(a, ++bidx, &s_abort)) return;
      cur ^= 1;
    }

    // ---- UPDATE: lambda_e, g_e, a_e (Eqs. 36, 40-41); rank updates of Q, T^T, Phi_y (Eqs. 42, 44);
    //      squared norms of the new rows of Phi_y for the next step ----
    for (int si = 0; si < nsegs; ++si) {
      const Seg s = segs[si];
      const LayerDev* L = s.L;
      const int M = s.M, M4 = M >> 2;
      float dt = 0.f;
      for (int m = threadIdx.x; m < M; m += PT) {
        const float v = ldcg(L->v + m), u = ldcg(L->u + m);
        xs[m] = v; us[m] = u; ts[m] = ldcg(L->t + m);
        dt = fmaf(v, u, dt);
      }
      const float lam_e = block_sum(dt, red);
      const float n2 = s.n2;
      const int cnt = s.cnt;
      const bool ok = cnt > 0 && n2 > 0.f && isfinite(n2) && isfinite(lam_e);
      float g_e = 1.f, aa = 0.f;
      if (ok) {
        g_e = L->delta * L->scal[SC_LAMBDA_BAR] / fmaxf(lam_e, L->eps);   // Eq. 40
        aa = sqrtf(g_e) - 1.f;                                            // Eq. 41
      }
      if (s.row0 == 0 && threadIdx.x == 0) {
        L->scal[SC_LAMBDA_E] = lam_e; L->scal[SC_G_E] = g_e; L->scal[SC_A_E] = aa; L->scal[SC_LAST_NORM2] = n2;
        if (!ok) L->iscal[IS_STATUS_NOSUB] = 1;
        if (!isfinite(n2) || !isfinite(lam_e)) L->iscal[IS_STATUS_NONFINITE] = 1;
        float* tr = const_cast<float*>(reinterpret_cast<const float*>(a.traces.p[s.layer]));
        if (tr) {
          tr[4 * step + 0] = lam_e; tr[4 * step + 1] = g_e;
          tr[4 * step + 2] = (float)cnt; tr[4 * step + 3] = (float)__ldcg(L->iscal + IS_MPRIME);
        }
      }
      if (aa != 0.f) {
        const float aq = aa * (aa + 2.f), a2l = aa * aa * lam_e;
        const float4* v4 = reinterpret_cast<const float4*>(xs);
        const float4* u4 = reinterpret_cast<const float4*>(us);
        const float4* t4 = reinterpret_cast<const float4*>(ts);
        for (int lr = warp; lr < s.nrows; lr += PW) {
          const int i = s.row0 + lr;
          const float vi = xs[i], ui = us[i], ti = ts[i];
          const float ati = aa * ti;
          float4* Q4 = reinterpret_cast<float4*>(L->Q + (size_t)i * M);
          float4* T4 = reinterpret_cast<float4*>(L->Tt + (size_t)i * M);
          float4* P4 = reinterpret_cast<float4*>(L->Phiy + (size_t)i * M);
          float4* C4 = (lr < s.ncached) ? reinterpret_cast<float4*>(cache + s.cache_off + (size_t)lr * M) : nullptr;
          double acc = 0.0;
          for (int c0 = lane; c0 < M4; c0 += 32 * PC) {
            float4 q[PC], tt[PC], pp[PC];
#pragma unroll
            for (int h = 0; h < PC; ++h) {
              const int c = c0 + 32 * h;
              if (c < M4) { q[h] = Q4[c]; tt[h] = T4[c]; pp[h] = C4 ? C4[c] : P4[c]; }
            }
#pragma unroll
            for (int h = 0; h < PC; ++h) {
              const int c = c0 + 32 * h;
              if (c < M4) {
                const float4 vj = v4[c], uj = u4[c], tj = t4[c];
#define FW_UPD(X)                                                                                              \
                q[h].X = __fadd_rn(q[h].X, __fmul_rn(aq, __fmul_rn(ti, tj.X)));                                \
                tt[h].X = fmaf(ati, vj.X, tt[h].X);                                                            \
                pp[h].X = __fadd_rn(pp[h].X, __fadd_rn(__fmul_rn(aa, __fadd_rn(__fmul_rn(vi, uj.X), __fmul_rn(ui, vj.X))), \
                                                       __fmul_rn(a2l, __fmul_rn(vi, vj.X))));                  \
                acc = fma((double)pp[h].X, (double)pp[h].X, acc);
                FW_UPD(x) FW_UPD(y) FW_UPD(z) FW_UPD(w)
#undef FW_UPD
                Q4[c] = q[h]; T4[c] = tt[h]; P4[c] = pp[h];
                if (C4) C4[c] = pp[h];
              }
            }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
          if (lane == 0) L->xi2[i] = (float)acc;
        }
      }
      __syncthreads();
    }
    if (step + 1 < K)
      if (!grid_barrier(a, ++bidx, &s_abort)) return;
  }
}

}  // namespace

// Whether the persistent kernel can take this group: every M a multiple of 4 (16-byte rows), no leakage, and no
// CTA with more row ranges than its table holds.
bool recursion_persist_supported(const int* layer_M, const float* layer_gamma, int n) {
  if (n < 1 || n > FW_MAX_GROUP) return false;
  for (int i = 0; i < n; ++i)
    if ((layer_M[i] & 3) != 0 || layer_gamma[i] != 1.0f || layer_M[i] < 64) return false;
  return true;
}

// barriers a launch of K steps of P power iterations goes through
static uint32_t persist_barriers(int K, int P) { return 1u + (uint32_t)K * (uint32_t)(P + 4) - 1u; }

cudaError_t launch_recursion_persist(const GroupDev& g, const PtrTable& traces, const int* layer_M, int K, int P,
                                     int32_t* bar_words, int32_t* status, uint32_t* bar_base_host, cudaStream_t s) {
  static int n_sm[64] = {0};
  static SmemAttrCache attr;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) dev = 0;
  if (n_sm[dev] == 0) {
    e = cudaDeviceGetAttribute(&n_sm[dev], cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
  }
  int max_M = 0;
  for (int i = 0; i < g.n; ++i) max_M = layer_M[i] > max_M ? layer_M[i] : max_M;
  const int vec_floats = (max_M + 3) & ~3;
  const size_t smem_total = 220 * 1024;
  const size_t vec_bytes = 3 * (size_t)vec_floats * sizeof(float);
  if (vec_bytes + 4096 > smem_total) return cudaErrorInvalidValue;
  e = ensure_dyn_smem(recursion_persistent_kernel, smem_total, attr);
  if (e != cudaSuccess) return e;
  PersistArgs a;
  memset(&a, 0, sizeof(a));
  a.g = g; a.traces = traces; a.K = K; a.P = P;
  int64_t W = 0;
  int64_t min_cost = LLONG_MAX;
  for (int i = 0; i < g.n; ++i) {
    a.prefix[i] = W;
    const int64_t c = (int64_t)((layer_M[i] + PR - 1) / PR) * layer_M[i];
    W += c;
    if (c < min_cost) min_cost = c;
  }
  a.prefix[g.n] = W;
  // one CTA per SM, but no more CTAs than row groups, and few enough that no CTA's share spans more layers than
  // its segment table holds
  int nctas = n_sm[dev];
  int64_t groups = 0;
  for (int i = 0; i < g.n; ++i) groups += (layer_M[i] + PR - 1) / PR;
  if (nctas > groups) nctas = (int)groups;
  while (nctas > 1 && (W / nctas) / (min_cost > 0 ? min_cost : 1) + 2 > kMaxSegs) --nctas;   // never taken for M >= 64
  a.nctas = nctas;
  a.bar = bar_words; a.status = status;
  a.bar_base = *bar_base_host;
  a.vec_floats = vec_floats;
  a.cache_floats = (int)((smem_total - vec_bytes) / sizeof(float));
  *bar_base_host += persist_barriers(K, P) * (uint32_t)nctas;
  void* args[] = {&a};
  ProfScope ps(FW_PROF_RECUR_MV, s);
  return cudaLaunchCooperativeKernel((void*)recursion_persistent_kernel, dim3(nctas), dim3(PT), args, smem_total, s);
}

}  // namespace fw
