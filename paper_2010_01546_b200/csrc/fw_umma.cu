// Tensor-core engine for sm_100a: tcgen05.mma with TMEM accumulators, operands
// staged in shared memory by TMA, warp-specialised (one TMA producer warp, one
// MMA issuer warp, four epilogue warps), mbarrier pipeline with bounded waits.
//
//   gq_umma_kernel    G~ = G Qs (Eq. 29) computed as D = Qs G^T so that the small
//                     output dimension N is the MMA's N; optional fused SGD
//                     epilogue W <- W - lr G~ (Eq. 27).  TF32 inputs, fp32 accumulate.
#include <cstdio>
#include <cstring>
#include <vector>

#include "fw_sm100.cuh"
#include "fw_umma.h"

namespace fw {

using namespace sm100;

// ---------------------------------------------------------------------------
// host: tensor-map encoding through the driver entry point (no link-time libcuda)
// ---------------------------------------------------------------------------
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
    else
      cudaGetLastError();
  }
  return fn;
}

// 2-D row-major tensor [outer][inner] with leading dimension ld (elements); box = box_inner x box_outer.
bool encode_2d(CUtensorMap* m, CUtensorMapDataType dt, int elem_bytes, const void* base, uint64_t inner,
               uint64_t outer, uint64_t ld, uint32_t box_inner, uint32_t box_outer, CUtensorMapSwizzle sw) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {ld * (uint64_t)elem_bytes};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(m, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Set by a kernel whose bounded wait ran out (value = where); read and cleared by the host.
__device__ int g_umma_status = 0;

constexpr int kMaxUmmaGroup = 16;

// ---------------------------------------------------------------------------
// G~ = G Qs
// ---------------------------------------------------------------------------
struct GqProblem {
  float* out;          // N x M: G~ (EPI_STORE) or W (EPI_SGD)
  int32_t M, N;
  int32_t n_box;       // rows of the G tile = MMA N (multiple of 16, <= 256)
  int32_t mblocks, npanels, first_cta;
  int32_t epi;
  float lr;
};
struct GqGroup {
  CUtensorMap mapA[kMaxUmmaGroup];   // Qs: [M rows][M cols], box 32 x 128, 128-byte swizzle
  CUtensorMap mapB[kMaxUmmaGroup];   // G : [N rows][M cols], box 32 x n_box
  GqProblem p[kMaxUmmaGroup];
  int32_t n;
};

constexpr int GQ_STAGES = 4;
constexpr int GQ_BK = 32;                       // fp32 elements per stage along K = one 128-byte swizzle row
constexpr int GQ_A_BYTES = 128 * GQ_BK * 4;     // 16 KB
constexpr int GQ_THREADS = 192;

__global__ void __launch_bounds__(GQ_THREADS) gq_umma_kernel(const __grid_constant__ GqGroup g) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[GQ_STAGES], bar_empty[GQ_STAGES], bar_accum;
  __shared__ uint32_t tmem_base_sh;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int pi = 0;
#pragma unroll 1
  for (int i = 1; i < g.n; ++i)
    if ((int)blockIdx.x >= g.p[i].first_cta) pi = i;
  const GqProblem& pr = g.p[pi];
  const int local = blockIdx.x - pr.first_cta;
  const int mb = local / pr.npanels, np = local - mb * pr.npanels;
  const int m0 = mb * 128, n0 = np * pr.n_box;
  const int K = pr.M;
  const int nk = (K + GQ_BK - 1) / GQ_BK;
  const uint32_t b_bytes = (uint32_t)pr.n_box * GQ_BK * 4;
  const uint32_t stage_bytes = GQ_A_BYTES + ((b_bytes + 1023u) & ~1023u);

  // 1024-byte aligned stage buffers (128-byte swizzle atoms are 1024 bytes)
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint32_t ncols = 32;
  while ((int)ncols < pr.n_box) ncols <<= 1;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < GQ_STAGES; ++s) { mbar_init(smem_u32(&bar_full[s]), 1); mbar_init(smem_u32(&bar_empty[s]), 1); }
    mbar_init(smem_u32(&bar_accum), 1);
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_sh), ncols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_sh;
  const volatile int* abortp = &abort_flag;

  if (warp == 0) {
    // ---- TMA producer ----
    if (elect_one()) {
      tma_prefetch_desc(&g.mapA[pi]);
      tma_prefetch_desc(&g.mapB[pi]);
      for (int kb = 0; kb < nk; ++kb) {
        const int s = kb % GQ_STAGES;
        const uint32_t ph = (kb / GQ_STAGES) & 1;
        if (!mbar_wait(smem_u32(&bar_empty[s]), ph ^ 1, abortp)) { abort_flag = 1; atomicExch(&g_umma_status, 101); break; }
        const uint32_t sa = smem_base + s * stage_bytes, sb = sa + GQ_A_BYTES;
        mbar_expect_tx(smem_u32(&bar_full[s]), GQ_A_BYTES + b_bytes);
        tma_load_2d(sa, &g.mapA[pi], kb * GQ_BK, m0, smem_u32(&bar_full[s]));
        tma_load_2d(sb, &g.mapB[pi], kb * GQ_BK, n0, smem_u32(&bar_full[s]));
      }
    }
  } else if (warp == 1) {
    // ---- MMA issuer ----
    if (elect_one()) {
      const uint32_t idesc = make_idesc(2, (uint32_t)pr.n_box, 0, 0);
      bool ok = true;
      for (int kb = 0; kb < nk && ok; ++kb) {
        const int s = kb % GQ_STAGES;
        const uint32_t ph = (kb / GQ_STAGES) & 1;
        if (!mbar_wait(smem_u32(&bar_full[s]), ph, abortp)) { abort_flag = 1; atomicExch(&g_umma_status, 102); ok = false; break; }
        tc_fence_after();
        const uint32_t sa = smem_base + s * stage_bytes, sb = sa + GQ_A_BYTES;
#pragma unroll
        for (int k = 0; k < GQ_BK / 8; ++k) {
          const uint64_t ad = make_smem_desc(sa + k * 32, 16, 1024, kSwizzle128B);
          const uint64_t bd = make_smem_desc(sb + k * 32, 16, 1024, kSwizzle128B);
          mma_tf32(tmem_base, ad, bd, idesc, (kb | k) != 0 ? 1u : 0u);
        }
        mma_commit(smem_u32(&bar_empty[s]));   // frees the stage when these MMAs have read it
      }
      mma_commit(smem_u32(&bar_accum));        // accumulator complete
    }
  } else {
    // ---- epilogue: TMEM -> registers -> global (transposed: lanes are m, columns are n) ----
    const int q = warp & 3;                    // TMEM lane quarter this warp may access
    const int m = m0 + q * 32 + lane;
    if (mbar_wait(smem_u32(&bar_accum), 0, abortp)) {
      tc_fence_after();
      for (int c0 = 0; c0 < pr.n_box; c0 += 16) {
        uint32_t r[16];
        tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, r);
        tmem_ld_wait();
        if (m < pr.M) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int n = n0 + c0 + j;
            if (n < pr.N) {
              float* dst = pr.out + (int64_t)n * pr.M + m;
              const float v = __uint_as_float(r[j]);
              if (pr.epi == EPI_SGD) *dst = fmaf(-pr.lr, v, *dst);
              else *dst = v;
            }
          }
        }
      }
    } else {
      abort_flag = 1;
      atomicExch(&g_umma_status, 103);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, ncols);
  }
}

}  // namespace

// ---------------------------------------------------------------------------
// host entry points
// ---------------------------------------------------------------------------
bool umma_available() { return encode_fn() != nullptr; }

int umma_take_status() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_umma_status, sizeof(int)) != cudaSuccess) { cudaGetLastError(); return -1; }
  if (v != 0) {
    int z = 0;
    cudaMemcpyToSymbol(g_umma_status, &z, sizeof(int));
  }
  return v;
}

bool umma_gram_supported(const fw_layer_desc&, const void*, int64_t) { return false; }
fw_status umma_gram_launch(UmmaGramItem*, int, cudaStream_t) { return FW_ERR_UNSUPPORTED; }

bool umma_gq_supported(const fw_layer_desc& d) {
  return umma_available() && (d.M % 4 == 0) && d.M >= 8;
}

fw_status umma_gq_launch(const UmmaGqItem* items, int n, int epi, float lr, cudaStream_t s) {
  static bool attr_set = false;
  const size_t max_smem = 1024 + GQ_STAGES * (GQ_A_BYTES + 256 * GQ_BK * 4);
  if (!attr_set) {
    if (cudaFuncSetAttribute(gq_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem) != cudaSuccess) {
      cudaGetLastError();
      return FW_ERR_CUDA;
    }
    attr_set = true;
  }
  for (int base = 0; base < n; base += kMaxUmmaGroup) {
    GqGroup g;
    memset(&g, 0, sizeof(g));
    const int cnt = (n - base) < kMaxUmmaGroup ? (n - base) : kMaxUmmaGroup;
    int total = 0;
    size_t smem = 0;
    for (int i = 0; i < cnt; ++i) {
      const UmmaGqItem& it = items[base + i];
      GqProblem& p = g.p[i];
      p.out = it.out; p.M = it.M; p.N = it.N; p.epi = epi; p.lr = lr;
      int nb = (it.N + 15) / 16 * 16;
      if (nb > 256) nb = 256;
      p.n_box = nb;
      p.mblocks = (it.M + 127) / 128;
      p.npanels = (it.N + nb - 1) / nb;
      p.first_cta = total;
      total += p.mblocks * p.npanels;
      if (!encode_2d(&g.mapA[i], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, it.Qs, it.M, it.M, it.M, GQ_BK, 128,
                     CU_TENSOR_MAP_SWIZZLE_128B) ||
          !encode_2d(&g.mapB[i], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, it.G, it.M, it.N, it.M, GQ_BK, (uint32_t)nb,
                     CU_TENSOR_MAP_SWIZZLE_128B)) {
        fprintf(stderr, "[fw] tensor-map encoding failed (G Qs)\n");
        return FW_ERR_CUDA;
      }
      const size_t need = 1024 + GQ_STAGES * (size_t)(GQ_A_BYTES + (((size_t)nb * GQ_BK * 4 + 1023) & ~(size_t)1023));
      if (need > smem) smem = need;
    }
    g.n = cnt;
    ProfScope ps(FW_PROF_GQ, s);
    gq_umma_kernel<<<total, GQ_THREADS, smem, s>>>(g);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
      fprintf(stderr, "[fw] gq_umma_kernel launch: %s\n", cudaGetErrorString(e));
      return FW_ERR_CUDA;
    }
  }
  return FW_OK;
}

}  // namespace fw
