// On-chip recursion for small layers (Sec. 4): one thread-block cluster of 8
// CTAs per layer keeps the whitened covariance Phi_y resident in distributed
// shared memory for all K steps of a call.  CTA `rank` owns a slab of rows of
// Phi_y; every pass of a step is a slab-times-vector product out of shared
// memory whose results are scattered into all 8 CTAs' copies of the output
// vector through distributed shared memory, followed by one hardware cluster
// barrier.  Nothing but T^T and Q (touched once per step) goes to global memory,
// so a step costs (P + 4) cluster barriers instead of (P + 6) kernel launches.
//
// The arithmetic is that of the multi-launch path in fw_recursion.cu (same
// passes, symmetric evaluation of the rank updates); dot products are accumulated
// in fp32 here (rows are at most ~600 long and split over 64 partial sums).
#include <cooperative_groups.h>

#include "fw_internal.h"

namespace cg = cooperative_groups;

namespace fw {
namespace {

constexpr int CL = 8;              // CTAs per cluster = per layer
constexpr int CT = 512;            // threads per CTA: many warps hide the latency of the small dependent passes
constexpr int CW = CT / 32;        // warps per CTA

__device__ __forceinline__ float warp_sum_f(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// block-wide sum of a per-thread value (all threads get the result)
__device__ float block_sum(float x, float* red) {
  x = warp_sum_f(x);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = x;
  __syncthreads();
  float t = 0.f;
#pragma unroll
  for (int w = 0; w < CW; ++w) t += red[w];
  __syncthreads();
  return t;
}

struct Slab {
  float* phi;     // my rows of Phi_y in shared memory, leading dimension Mp
  int M, Mp, R;   // matrix size, padded row length, rows per CTA
  int row0, nrows;
};

constexpr int MAXRPW = 5;          // rows per warp: ceil(R / 16) with R <= 80
constexpr int MAXC4 = 5;           // float4 per lane per row: ceil(Mp / 128) with Mp <= 608

// y[row0 + r] = scale * dot(A[r,:], x) for my rows; A rows live in shared or global memory.
// The result for each row is stored into `dst` (a shared-memory vector of length Mp) of every
// CTA of the cluster.  A warp owns rows warp, warp + 8, ... and works on all of them at once:
// every lane keeps one fp32 accumulator pair per row, so all loads of a column step are in
// flight together (the slab is small: the pass is latency-, not bandwidth-bound).
template <bool SELF>
__device__ __noinline__ void slab_gemv_scatter(cg::cluster_group& cluster, const float* A, int lda,
                                                  const float* x, const Slab s, float scale, float* dst) {
  (void)cluster;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int M4 = s.Mp >> 2;
  const float4* x4 = reinterpret_cast<const float4*>(x);
  float acc[MAXRPW][2];
#pragma unroll
  for (int q = 0; q < MAXRPW; ++q) acc[q][0] = acc[q][1] = 0.f;
#pragma unroll
  for (int ci = 0; ci < MAXC4; ++ci) {
    const int c = lane + 32 * ci;
    if (c < M4) {
      float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
      if (!SELF) b = x4[c];
      float4 a[MAXRPW];
#pragma unroll
      for (int q = 0; q < MAXRPW; ++q) {
        const int r = warp + CW * q;
        if (r < s.nrows) a[q] = reinterpret_cast<const float4*>(A + (size_t)r * lda)[c];
      }
#pragma unroll
      for (int q = 0; q < MAXRPW; ++q) {
        const int r = warp + CW * q;
        if (r < s.nrows) {
          const float4 bb = SELF ? a[q] : b;
          acc[q][0] = fmaf(a[q].x, bb.x, acc[q][0]); acc[q][1] = fmaf(a[q].y, bb.y, acc[q][1]);
          acc[q][0] = fmaf(a[q].z, bb.z, acc[q][0]); acc[q][1] = fmaf(a[q].w, bb.w, acc[q][1]);
        }
      }
    }
  }
  float y[MAXRPW];
#pragma unroll
  for (int q = 0; q < MAXRPW; ++q) y[q] = acc[q][0] + acc[q][1];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
    for (int q = 0; q < MAXRPW; ++q) y[q] += __shfl_xor_sync(0xffffffffu, y[q], o);
  }
  // my slice of the result goes to my own copy of the vector; the peers fetch it after the cluster barrier
#pragma unroll
  for (int q = 0; q < MAXRPW; ++q) {
    const int r = warp + CW * q;
    if (r < s.nrows && lane == 0) dst[s.row0 + r] = y[q] * scale;
  }
}

// After a cluster barrier: complete my copy of a vector with the slices the peers computed (one remote
// 4-byte load per element, all in flight at once), then a block barrier.
// Same, and returns the squared norm of the completed vector (the block reduction doubles as the barrier).
__device__ __forceinline__ float gather_slices_norm2(cg::cluster_group& cluster, float* vec, const Slab& s, int rank,
                                                    float* red) {
  float part = 0.f;
  for (int m = threadIdx.x; m < s.M; m += CT) {
    const int owner = m / s.R;
    float x;
    if (owner != rank) { x = cluster.map_shared_rank(vec, owner)[m]; vec[m] = x; }
    else x = vec[m];
    part = fmaf(x, x, part);
  }
  return block_sum(part, red);
}

__device__ __forceinline__ void gather_slices(cg::cluster_group& cluster, float* vec, const Slab& s, int rank) {
  for (int m = threadIdx.x; m < s.M; m += CT) {
    const int owner = m / s.R;
    if (owner != rank) vec[m] = cluster.map_shared_rank(vec, owner)[m];
  }
  __syncthreads();
}

// dynamic shared memory: [phi slab R x Mp][xi2][cvec][wvec][bufA][bufB][vvec][uvec][tvec]
extern __shared__ __align__(16) float csm[];

__global__ void __cluster_dims__(CL, 1, 1) __launch_bounds__(CT, 1)
recursion_cluster_kernel(const __grid_constant__ GroupDev g, const __grid_constant__ PtrTable traces, int K, int P) {
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int layer = blockIdx.x / CL;
  const LayerDev* L = g.layer[layer];
  const int M = L->M;
  const int Mp = (M + 3) & ~3;
  const int R = (M + CL - 1) / CL;
  Slab s;
  s.M = M; s.Mp = Mp; s.R = R;
  s.row0 = rank * R;
  s.nrows = max(0, min(R, M - s.row0));
  s.phi = csm;
  float* xi2 = csm + (size_t)R * Mp;
  float* cvec = xi2 + Mp;
  float* wvec = cvec + Mp;
  float* buf[2] = {wvec + Mp, wvec + 2 * Mp};
  float* vvec = wvec + 3 * Mp;
  float* uvec = vvec + Mp;
  float* tvec = uvec + Mp;
  __shared__ float red[CW];
  __shared__ float sredf[CW];
  __shared__ int sredi[CW + 1];

  // ---- load my rows of Phi_y; clear the padding and the vectors ----
  for (int i = threadIdx.x; i < s.nrows * Mp; i += CT) {
    const int r = i / Mp, c = i - r * Mp;
    s.phi[i] = (c < M) ? L->Phiy[(size_t)(s.row0 + r) * M + c] : 0.f;
  }
  for (int i = threadIdx.x; i < 8 * Mp; i += CT) xi2[i] = 0.f;
  cluster.sync();

  float* tr = const_cast<float*>(reinterpret_cast<const float*>(traces.p[layer]));
  const float c_rel = L->c_rel, c_abs = L->c_abs, delta = L->delta, eps = L->eps;
  const float lam_bar = L->scal[SC_LAMBDA_BAR];
  const bool maxcol = (L->init == FW_INIT_MAXCOL);
  bool any_nosub = false;

  for (int step = 0; step < K; ++step) {
    // S1: squared column norms (= row norms, Phi_y is exactly symmetric)             (Eq. 45)
    slab_gemv_scatter<true>(cluster, s.phi, Mp, nullptr, s, 1.f, xi2);
    cluster.sync();
    gather_slices(cluster, xi2, s, rank);
    // S2: m' = argmax xi (lowest index on ties), x = row m' of Phi_y, c = Phi_y x    (Eqs. 46-47)
    {
      float best = -1.f;
      int bi = 0x7fffffff;
      for (int m = threadIdx.x; m < M; m += CT) {
        const float x = xi2[m];
        if (x > best) { best = x; bi = m; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float xo = __shfl_xor_sync(0xffffffffu, best, o);
        const int io = __shfl_xor_sync(0xffffffffu, bi, o);
        if (xo > best || (xo == best && io < bi)) { best = xo; bi = io; }
      }
      if ((threadIdx.x & 31) == 0) { sredf[threadIdx.x >> 5] = best; sredi[threadIdx.x >> 5] = bi; }
      __syncthreads();
      if (threadIdx.x < 32) {
        best = threadIdx.x < CW ? sredf[threadIdx.x] : -1.f;
        bi = threadIdx.x < CW ? sredi[threadIdx.x] : 0x7fffffff;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const float xo = __shfl_xor_sync(0xffffffffu, best, o);
          const int io = __shfl_xor_sync(0xffffffffu, bi, o);
          if (xo > best || (xo == best && io < bi)) { best = xo; bi = io; }
        }
        if (threadIdx.x == 0) sredi[CW] = bi;
      }
      __syncthreads();
    }
    int mp = sredi[CW];
    if (mp < 0 || mp >= M) mp = 0;
    __syncthreads();
    {
      const int owner = mp / R;
      const float* rphi = cluster.map_shared_rank(s.phi, owner) + (size_t)(mp - owner * R) * Mp;
      for (int m = threadIdx.x; m < Mp; m += CT) wvec[m] = rphi[m];
    }
    __syncthreads();
    slab_gemv_scatter<false>(cluster, s.phi, Mp, wvec, s, 1.f, cvec);
    cluster.sync();
    gather_slices(cluster, cvec, s, rank);
    // S3: coherent set and aligned average                                          (Eqs. 48-49)
    int cnt;
    {
      int local = 0;
      if (maxcol) {
        for (int m = threadIdx.x; m < Mp; m += CT) wvec[m] = (m == mp) ? 1.f : 0.f;
        local = (threadIdx.x == 0) ? 1 : 0;
      } else {
        const float xi_mp = sqrtf(xi2[mp]);
        for (int m = threadIdx.x; m < Mp; m += CT) {
          float wv = 0.f;
          if (m < M) {
            const float c = cvec[m];
            const float thr = fmaxf(c_rel * xi_mp * sqrtf(xi2[m]), c_abs);
            const bool in = fabsf(c) >= thr;
            wv = in ? (1.f / c) : 0.f;
            local += in ? 1 : 0;
          }
          wvec[m] = wv;
        }
      }
      cnt = (int)(block_sum((float)local, red) + 0.5f);
    }
    if (rank == 0 && !maxcol)
      for (int m = threadIdx.x; m < M; m += CT) L->wvec[m] = wvec[m];
    const float inv_cnt = cnt > 0 ? 1.f / (float)cnt : 0.f;
    slab_gemv_scatter<false>(cluster, s.phi, Mp, wvec, s, inv_cnt, buf[0]);
    cluster.sync();
    float n2 = gather_slices_norm2(cluster, buf[0], s, rank, red);
    // S4: P power iterations u = Phi_y (prev / ||prev||); the norm comes with the gather of each result
    int cur = 0;
    float inv = (n2 > 0.f && isfinite(n2)) ? rsqrtf(n2) : 0.f;
    inv = inv > 0.f ? inv * (1.5f - 0.5f * n2 * inv * inv) : 0.f;
    for (int p = 0; p < P; ++p) {
      slab_gemv_scatter<false>(cluster, s.phi, Mp, buf[cur], s, inv, buf[cur ^ 1]);
      cluster.sync();
      n2 = gather_slices_norm2(cluster, buf[cur ^ 1], s, rank, red);
      inv = (n2 > 0.f && isfinite(n2)) ? rsqrtf(n2) : 0.f;
      inv = inv > 0.f ? inv * (1.5f - 0.5f * n2 * inv * inv) : 0.f;
      cur ^= 1;
    }
    // S5: v = prev/||prev|| (Eq. 50), u = Phi_y v, t = T^T v
    for (int m = threadIdx.x; m < Mp; m += CT) vvec[m] = (m < M) ? buf[cur][m] * inv : 0.f;
    __syncthreads();
    slab_gemv_scatter<false>(cluster, s.phi, Mp, vvec, s, 1.f, uvec);
    if ((M & 3) == 0) {
      slab_gemv_scatter<false>(cluster, L->Tt + (size_t)s.row0 * M, M, vvec, s, 1.f, tvec);
    } else {
      // unaligned rows in global memory: scalar loads
      const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
      for (int r = warp; r < s.nrows; r += CW) {
        const float* a = L->Tt + (size_t)(s.row0 + r) * M;
        float acc = 0.f;
        for (int c = lane; c < M; c += 32) acc = fmaf(a[c], vvec[c], acc);
        acc = warp_sum_f(acc);
        if (lane == 0) tvec[s.row0 + r] = acc;
      }
    }
    cluster.sync();
    for (int m = threadIdx.x; m < M; m += CT) {
      const int owner = m / R;
      if (owner != rank) {
        uvec[m] = cluster.map_shared_rank(uvec, owner)[m];
        tvec[m] = cluster.map_shared_rank(tvec, owner)[m];
      }
    }
    __syncthreads();
    // S6: lambda_e = v.u (Eq. 36), g_e, a_e (Eqs. 40-41), rank updates (Eqs. 42, 44)
    float part = 0.f;
    for (int m = threadIdx.x; m < M; m += CT) part = fmaf(vvec[m], uvec[m], part);
    const float lam_e = block_sum(part, red);
    const bool ok = cnt > 0 && n2 > 0.f && isfinite(n2) && isfinite(lam_e);
    float g_e = 1.f, a = 0.f;
    if (ok) {
      g_e = delta * lam_bar / fmaxf(lam_e, eps);
      a = sqrtf(g_e) - 1.f;
    }
    any_nosub |= !ok;
    if (rank == 0 && threadIdx.x == 0) {
      L->scal[SC_LAMBDA_E] = lam_e; L->scal[SC_G_E] = g_e; L->scal[SC_A_E] = a;
      L->iscal[IS_MPRIME] = mp; L->iscal[IS_SETSIZE] = cnt;
      if (tr) {
        tr[4 * step + 0] = lam_e; tr[4 * step + 1] = g_e;
        tr[4 * step + 2] = (float)cnt; tr[4 * step + 3] = (float)mp;
      }
    }
    if (a != 0.f) {
      const float aq = a * (a + 2.f), a2l = a * a * lam_e;
      if ((M & 3) == 0) {
        // one float4 of one row per thread and iteration; independent iterations keep several L2 loads in flight
        const int M4 = M >> 2;
        const int total = s.nrows * M4;
        float4* Q4 = reinterpret_cast<float4*>(L->Q + (size_t)s.row0 * M);
        float4* T4 = reinterpret_cast<float4*>(L->Tt + (size_t)s.row0 * M);
        float4* P4 = reinterpret_cast<float4*>(s.phi);
#pragma unroll 4
        for (int e = threadIdx.x; e < total; e += CT) {
          const int r = e / M4, c = e - r * M4;
          const int i = s.row0 + r;
          const float vi = vvec[i], ui = uvec[i], ti = tvec[i];
          const float4 vj = reinterpret_cast<const float4*>(vvec)[c];
          const float4 uj = reinterpret_cast<const float4*>(uvec)[c];
          const float4 tj = reinterpret_cast<const float4*>(tvec)[c];
          float4 q = Q4[e], tt = T4[e], p = P4[e];
#define FW_UPD(X)                                                                                          \
          q.X = __fadd_rn(q.X, __fmul_rn(aq, __fmul_rn(ti, tj.X)));                                        \
          tt.X = fmaf(a * ti, vj.X, tt.X);                                                                 \
          p.X = __fadd_rn(p.X, __fadd_rn(__fmul_rn(a, __fadd_rn(__fmul_rn(vi, uj.X), __fmul_rn(ui, vj.X))), \
                                         __fmul_rn(a2l, __fmul_rn(vi, vj.X))));
          FW_UPD(x) FW_UPD(y) FW_UPD(z) FW_UPD(w)
#undef FW_UPD
          Q4[e] = q; T4[e] = tt; P4[e] = p;
        }
      } else {
        for (int e = threadIdx.x; e < s.nrows * Mp; e += CT) {
          const int r = e / Mp, j = e - r * Mp;
          if (j < M) {
            const int i = s.row0 + r;
            const float vi = vvec[i], ui = uvec[i], ti = tvec[i];
            const float vj = vvec[j], uj = uvec[j], tj = tvec[j];
            s.phi[e] = __fadd_rn(s.phi[e], __fadd_rn(__fmul_rn(a, __fadd_rn(__fmul_rn(vi, uj), __fmul_rn(ui, vj))),
                                                     __fmul_rn(a2l, __fmul_rn(vi, vj))));
            const size_t off = (size_t)i * M + j;
            L->Q[off] = __fadd_rn(L->Q[off], __fmul_rn(aq, __fmul_rn(ti, tj)));
            L->Tt[off] = fmaf(a * ti, vj, L->Tt[off]);
          }
        }
      }
    }
    __syncthreads();
    // the next step's first cluster barrier (after S1) orders these updates before any remote read
  }
  // ---- write my rows of Phi_y back ----
  for (int i = threadIdx.x; i < s.nrows * Mp; i += CT) {
    const int r = i / Mp, c = i - r * Mp;
    if (c < M) L->Phiy[(size_t)(s.row0 + r) * M + c] = s.phi[i];
  }
  if (any_nosub && rank == 0 && threadIdx.x == 0) L->iscal[IS_STATUS_NOSUB] = 1;
  cluster.sync();   // no CTA leaves while its shared memory may still be read by a peer
}

}  // namespace

size_t recursion_cluster_smem(int M) {
  const int Mp = (M + 3) & ~3;
  const int R = (M + CL - 1) / CL;
  return ((size_t)R * Mp + 8 * (size_t)Mp) * sizeof(float);
}

bool recursion_cluster_supported(int M) {
  const int Mp = (M + 3) & ~3;
  return recursion_cluster_smem(M) <= 200 * 1024 && (M + CL - 1) / CL <= MAXRPW * CW && Mp <= MAXC4 * 128;
}

cudaError_t launch_recursion_cluster(const GroupDev& g, const PtrTable& traces, int K, int P, int max_M,
                                     cudaStream_t s) {
  static size_t attr = 0;
  const size_t smem = recursion_cluster_smem(max_M);
  if (smem > attr) {
    cudaError_t e = cudaFuncSetAttribute(recursion_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return e;
    attr = smem;
  }
  ProfScope ps(FW_PROF_RECUR_MV, s);
  recursion_cluster_kernel<<<g.n * CL, CT, smem, s>>>(g, traces, K, P);
  return cudaGetLastError();
}

}  // namespace fw
