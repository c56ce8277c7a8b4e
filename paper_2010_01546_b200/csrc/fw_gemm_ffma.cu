// Grouped fp32 (FFMA) GEMM used by the FP32 engine:
//   - the Gram pass X^T X with fused column sums (Eqs. 3, 5: the covariance sum),
//   - G * Qs with the optional fused SGD epilogue (Eqs. 27, 29),
//   - the re-sync products T Phix and (T Phix) T^T.
// One launch covers every problem of a group; a CTA finds its problem, tile and
// K-split from its block index.  64x64 output tile, 16-deep K slab, 256 threads,
// 4x4 accumulators per thread, register-staged double buffering.
#include "fw_internal.h"

namespace fw {

namespace {

constexpr int BM = 64, BN = 64, BK = 16, NT = 256;

__device__ __forceinline__ float ld_elem(const void* base, int64_t idx, int bf16) {
  if (bf16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(base)[idx]);
  return reinterpret_cast<const float*>(base)[idx];
}

__global__ void __launch_bounds__(NT) gemm_ffma_kernel(const __grid_constant__ GemmGroup g) {
  // locate the problem this CTA works on
  int cta = blockIdx.x;
  int pi = 0;
#pragma unroll 1
  for (int i = 1; i < g.n; ++i)
    if (cta >= g.p[i].first_cta) pi = i;
  const GemmProblem& pr = g.p[pi];
  int local = cta - pr.first_cta;
  int split = local / pr.ntiles;
  int tile = local - split * pr.ntiles;
  int tm, tn;
  if (pr.sym) {
    // enumerate upper-triangular tiles row by row
    tm = 0;
    int rem = tile;
    int rowlen = pr.tiles_n;
    while (rem >= rowlen) { rem -= rowlen; ++tm; --rowlen; }
    tn = tm + rem;
  } else {
    tm = tile / pr.tiles_n;
    tn = tile - tm * pr.tiles_n;
  }
  const int m0 = tm * BM, n0 = tn * BN;
  // K range of this split, in multiples of BK
  int64_t kslabs = (pr.k + BK - 1) / BK;
  int64_t per = (kslabs + pr.splits - 1) / pr.splits;
  int64_t kb = (int64_t)split * per * BK;
  int64_t ke = kb + per * BK;
  if (ke > pr.k) ke = pr.k;

  __shared__ float As[2][BK][BM + 4];
  __shared__ float Bs[2][BK][BN + 4];

  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;   // 16 x 16 threads, 4x4 each
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  const bool want_colsum = (pr.colsum != nullptr) && (tm == tn);
  float colacc = 0.f;  // thread tid < BM accumulates column m0 + tid

  // staging registers: each thread moves 4 elements of A and 4 of B per slab
  float ra[4], rb[4];
  const int bf = pr.in_bf16;

  auto load_slab = [&](int64_t k0) {
    if (pr.a_kmajor) {
      // A stored k x m: element (k, m) at A[k*lda + m]; thread -> (kk = e/64, mm = e%64)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        int idx = tid + e * NT;
        int kk = idx >> 6, mm = idx & 63;
        int64_t kg = k0 + kk;
        int mg = m0 + mm;
        float val = 0.f;
        if (kg < ke && mg < pr.m) {
          val = ld_elem(pr.A, kg * pr.lda + mg, bf);
          if (pr.shift) val -= pr.shift[mg];
        }
        ra[e] = val;
      }
    } else {
      // A stored m x k: element (m, k) at A[m*lda + k]; thread -> (mm = e/16, kk = e%16)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        int idx = tid + e * NT;
        int mm = idx >> 4, kk = idx & 15;
        int64_t kg = k0 + kk;
        int mg = m0 + mm;
        float val = 0.f;
        if (kg < ke && mg < pr.m) val = ld_elem(pr.A, (int64_t)mg * pr.lda + kg, 0);
        ra[e] = val;
      }
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      int idx = tid + e * NT;
      int kk = idx >> 6, nn = idx & 63;
      int64_t kg = k0 + kk;
      int ng = n0 + nn;
      float val = 0.f;
      if (kg < ke && ng < pr.n) {
        val = ld_elem(pr.B, kg * pr.ldb + ng, bf);
        if (pr.shift) val -= pr.shift[ng];
      }
      rb[e] = val;
    }
  };
  auto store_slab = [&](int buf) {
    if (pr.a_kmajor) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        int idx = tid + e * NT;
        As[buf][idx >> 6][idx & 63] = ra[e];
      }
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        int idx = tid + e * NT;
        As[buf][idx & 15][idx >> 4] = ra[e];
      }
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      int idx = tid + e * NT;
      Bs[buf][idx >> 6][idx & 63] = rb[e];
    }
  };

  int buf = 0;
  if (kb < ke) {
    load_slab(kb);
    store_slab(0);
  }
  __syncthreads();
  for (int64_t k0 = kb; k0 < ke; k0 += BK) {
    const bool more = (k0 + BK) < ke;
    if (more) load_slab(k0 + BK);
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float4 a4 = *reinterpret_cast<const float4*>(&As[buf][kk][ty * 4]);
      float4 b4 = *reinterpret_cast<const float4*>(&Bs[buf][kk][tx * 4]);
      float a[4] = {a4.x, a4.y, a4.z, a4.w};
      float b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    if (want_colsum && tid < BM) {
#pragma unroll
      for (int kk = 0; kk < BK; ++kk) colacc += As[buf][kk][tid];
    }
    if (more) store_slab(buf ^ 1);
    __syncthreads();
    buf ^= 1;
  }

  // epilogue
  float* C = pr.C + (int64_t)split * pr.c_split_stride;
  bool bad = false;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int mg = m0 + ty * 4 + i;
    if (mg >= pr.m) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int ng = n0 + tx * 4 + j;
      if (ng >= pr.n) continue;
      int64_t off = (int64_t)mg * pr.ldc + ng;
      bad |= !isfinite(acc[i][j]);
      if (pr.epi == EPI_SGD) {
        C[off] = fmaf(-pr.lr, acc[i][j], C[off]);
      } else if (pr.epi == EPI_SYMM) {
        // make the result exactly symmetric from the upper tiles
        if (tm == tn) {
          if (ng >= mg) { C[off] = acc[i][j]; C[(int64_t)ng * pr.ldc + mg] = acc[i][j]; }
        } else {
          C[off] = acc[i][j];
          C[(int64_t)ng * pr.ldc + mg] = acc[i][j];
        }
      } else {
        C[off] = pr.colbias ? acc[i][j] - pr.colbias[ng] : acc[i][j];
      }
    }
  }
  if (want_colsum && tid < BM) {
    int mg = m0 + tid;
    if (mg < pr.m) pr.colsum[(int64_t)split * pr.m + mg] = colacc;
  }
  if (bad && pr.nonfinite) *pr.nonfinite = 1;
}

}  // namespace

cudaError_t launch_gemm_ffma(GemmGroup& g, cudaStream_t s, int prof_class) {
  int total = 0;
  for (int i = 0; i < g.n; ++i) {
    GemmProblem& p = g.p[i];
    p.tiles_m = (p.m + BM - 1) / BM;
    p.tiles_n = (p.n + BN - 1) / BN;
    p.ntiles = p.sym ? p.tiles_n * (p.tiles_n + 1) / 2 : p.tiles_m * p.tiles_n;
    if (p.splits < 1) p.splits = 1;
    p.first_cta = total;
    total += p.ntiles * p.splits;
  }
  g.total_ctas = total;
  if (total == 0) return cudaSuccess;
  ProfScope ps(prof_class, s);
  gemm_ffma_kernel<<<total, NT, 0, s>>>(g);
  return cudaGetLastError();
}

}  // namespace fw
