// Tensor-core engine, CTA-pair kernels (tcgen05 cta_group::2): the Gram pass X^T X
// with column sums (Eqs. 3, 5) and the re-sync products A^T B for matrices whose
// accumulators do not fit one CTA's TMEM.
//
// Why pairs.  With one CTA per tile (128 x 256 outputs) every MMA reads 12 KB of
// operands from shared memory per 128 tensor-core cycles while TMA writes the same
// amount into it, and the tile needs 96 bytes per cycle from L2: shared-memory
// bandwidth and bytes in flight bound the kernel well below the tensor peak.  A
// pair of CTAs on the two SMs of a TPC computes a 256 x 512 tile: each CTA stages
// its own 128 rows of A and only its half of each B panel, so a CTA loads 384
// columns for 128 x 512 outputs (48 bytes per tensor cycle) and the tensor core of
// each SM reads half of B from its own shared memory.
//
// Tile (I, t): Gram rows [256 I, 256 I + 256) x columns [c, c + 512), as two
// accumulators of <= 256 columns (all 512 TMEM columns of both CTAs).  For the
// symmetric Gram only tiles on or right of the diagonal exist, and on the diagonal
// tile the first B panel is the A block itself, so it is staged once.
// Both operands are MN-major chunks of 32 columns laid down by TMA (see the
// single-CTA kernel for the layouts); a column group is 4 chunks = 128 columns.
//
// Centred accumulators.  The tensor core adds into its fp32 accumulators with truncation, so a chain of n MMAs
// loses about n 2^-24 of the sum, and for data with a mean the sum is mostly rows mu mu^T: the loss, small against
// X^T X, is not small against the covariance that is left once the mean product is taken off.  A Gram problem
// therefore carries a pilot mean c (rounded to the operand type), and every eighth stage one extra MMA per
// accumulator adds (-s c)^T c from constant operand chunks, s = the rows of eight stages / the rows of one MMA: the
// accumulators hold X^T X - n c c^T, of the covariance's own size, and the moment kernels add n c c^T back in
// fp32 (n is known to the host).
//
// Roles per CTA: warp 0 TMA producer, warp 1 MMA issuer (even CTA only) and TMEM
// owner, warps 2..9 fix-up/column sums and epilogue.  Two stage protocols:
//   direct  both CTAs' loads complete on the even CTA's "full" barrier (armed with
//           the bytes of both); the MMA thread waits on it.
//   pass    (diagonal tiles: column sums; re-sync: rounding to TF32) each CTA's
//           loads complete on its own barrier, its 8 warps pass over the stage and
//           then arrive on the even CTA's "ready" barrier (16 arrivals).
// tcgen05.commit multicasts the "stage free" and "accumulator complete" arrivals
// to both CTAs.  Every wait is bounded; a time-out raises the abort flag of both
// CTAs, is recorded in the owning layer's status word, and all threads still meet
// at the final cluster barrier before TMEM is freed.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <vector>

#include "fw_sm100.cuh"
#include "fw_umma.h"

namespace fw {

using namespace sm100;

namespace {

constexpr int GP_SR_F32 = 32;              // rows of X per stage, fp32 (48 KB stages, 4 in flight)
constexpr int GP_SR_BF16 = 64;             // bf16: the same 48 KB and 1024 tensor cycles per stage as fp32; with 32 rows
                                           // (512 cycles) the per-stage hand-offs left the tensor pipe idle a third of the time
__host__ __device__ constexpr int pair_sr(bool bf16) { return bf16 ? GP_SR_BF16 : GP_SR_F32; }
constexpr int GP_GCOLS = 128;              // columns per column group (chunks of 32 fp32 or 64 bf16 columns)
constexpr int GP_MAX_GROUPS = 3;           // A block, first and second B panel halves
constexpr int GP_MAX_STAGES = 8;
constexpr int GP_FIX_WARPS = 8;
constexpr int GP_THREADS = 64 + GP_FIX_WARPS * 32;
constexpr int GP_SMEM = 192 * 1024;
constexpr int GP_CONST = 12 * 1024;        // constant operand chunks of the mean-product correction: 3 column groups x
                                           // one MMA's rows (16 bf16 / 8 fp32) x 128 columns
constexpr int GP_MAX_PROBLEMS = 16;
constexpr int GP_MAX_ITEMS = 2048;
constexpr int GP_CLUSTER_SLOTS = 74;       // CTA pairs resident at once if every TPC takes one (148 SMs, one CTA per SM)

struct PairProblem {
  float* out;            // split s writes its partial to out + s * M * M
  float* colsum_part;    // split s writes column sums to colsum_part + s * M (null: none owed)
  int64_t rows;
  int32_t M;
  int32_t full;          // 1: D = A^T B from two sources, every tile; 0: symmetric Gram of one source;
                         // 2: A^T B with a symmetric result: tiles below the diagonal skipped, entries mirrored
  int32_t fixup;         // 1 (fp32 only): round every staged value to TF32 (nearest) before the product
  int32_t rows_per_split;  // multiple of the stage's rows
  int32_t use3d;         // chunked 3-D tensor maps usable (M a multiple of 64)
  int32_t pad;
  int32_t* status;       // time-out word of the owning layer
  const float* pmean;    // pilot mean for the mean-product correction (Gram problems), or null
};
struct PairGroup {
  CUtensorMap mapA[GP_MAX_PROBLEMS];     // one-chunk boxes, A-side source (the only source of a Gram)
  CUtensorMap mapB[GP_MAX_PROBLEMS];     // one-chunk boxes, B-side source (full = 1)
  CUtensorMap map3A[GP_MAX_PROBLEMS];    // chunked 3-D views, boxes of one column group
  CUtensorMap map3B[GP_MAX_PROBLEMS];
  PairProblem p[GP_MAX_PROBLEMS];
  int32_t n, nitems;
  uint32_t item[GP_MAX_ITEMS];           // problem << 28 | tile << 14 | split, longest first
};

__host__ __device__ inline int pair_tiles_sym(int M16) {
  int t = 0;
  for (int c = 0; c < M16; c += 256) t += (M16 - c + 511) / 512;
  return t;
}
__host__ __device__ inline int pair_tiles_full(int M16) { return ((M16 + 255) / 256) * ((M16 + 511) / 512); }

__device__ __forceinline__ float4 lds128(uint32_t a) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ void sts128(uint32_t a, float4 v) {
  asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(a), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ float tf32_rna(float x) {
  return __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xffffe000u);
}

template <bool BF>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GP_THREADS, 1)
gram_pair_kernel(const __grid_constant__ PairGroup g) {
  // Chunk rows are 128 bytes for both element types (TMA fetches whole 128-byte lines):
  //   fp32: 32 columns, 128-byte swizzle with 32-byte atoms, K-atoms of 4 rows;
  //   bf16: 64 columns, 128-byte swizzle (16-byte units), K-atoms of 8 rows.
  constexpr int CW = BF ? 64 : 32;                // columns per chunk
  constexpr int GC = GP_GCOLS / CW;               // chunks per column group
  constexpr int SR = pair_sr(BF);                 // rows per stage
  constexpr int KSTEPS = SR / (BF ? 16 : 8);      // MMAs along K per stage (16 / 8 rows each)
  constexpr int CHUNK = SR * 128;                 // bytes per chunk
  constexpr int GROUP_BYTES = GC * CHUNK;         // bytes per column group per stage
  constexpr uint32_t SBO = BF ? 1024u : 512u;     // next K-atom
  constexpr uint32_t KSTEP16 = BF ? 128u : 64u;   // next MMA k-step, in 16-byte units (16 / 8 rows of 128 bytes)
  constexpr uint64_t LAYOUT = BF ? kSwizzle128B : kSwizzle128B32;
  constexpr uint32_t FMT = BF ? 1u : 2u;
  constexpr int KR = BF ? 16 : 8;                 // rows one MMA contracts over
  constexpr int CCHUNK = KR * 128;                // bytes per chunk of the constant operands
  constexpr int CGROUP = GC * CCHUNK;             // bytes per column group of them (4 KB)
  static_assert(3 * CGROUP <= GP_CONST, "constant operand region");

  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[GP_MAX_STAGES], bar_ready[GP_MAX_STAGES], bar_empty[GP_MAX_STAGES], bar_accum;
  __shared__ uint32_t tmem_base_sh;
  __shared__ int abort_flag;
  __shared__ int s_I, s_cbase, s_n0, s_n1, s_ngroups, s_bgroup, s_pass, s_cs, s_tmem_cols, s_skip;
  __shared__ int s_gcol[GP_MAX_GROUPS], s_gsrc[GP_MAX_GROUPS];
  __shared__ float s_csred[GP_FIX_WARPS][GP_GCOLS];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const uint32_t it = g.item[blockIdx.x >> 1];
  const int pi = (int)(it >> 28), tile = (int)((it >> 14) & 0x3fffu), split = (int)(it & 0x3fffu);
  const PairProblem& pr = g.p[pi];
  const int M = pr.M;
  const int M16 = (M + 15) / 16 * 16;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    int I = 0, t = tile;
    if (pr.full) {
      const int np = (M16 + 511) / 512;
      I = tile / np; t = tile - I * np;
    } else {
      for (;; ++I) {
        const int np = (M16 - 256 * I + 511) / 512;
        if (t < np) break;
        t -= np;
      }
    }
    const int cbase = (pr.full ? 0 : 256 * I) + 512 * t;
    const int n0 = min(256, M16 - cbase);
    const int n1 = max(0, min(256, M16 - cbase - 256));
    const bool diag = !pr.full && t == 0;
    const bool shared_b0 = diag && n0 == 256;      // first panel == the A block: staged once
    int ng = 0;
    s_gcol[ng] = 256 * I + 128 * (int)rank; s_gsrc[ng] = 0; ++ng;
    s_bgroup = shared_b0 ? 0 : ng;
    if (!shared_b0) { s_gcol[ng] = cbase + (int)rank * (n0 / 2); s_gsrc[ng] = pr.full ? 1 : 0; ++ng; }
    if (n1 > 0) { s_gcol[ng] = cbase + 256 + (int)rank * (n1 / 2); s_gsrc[ng] = pr.full ? 1 : 0; ++ng; }
    s_I = I; s_cbase = cbase; s_n0 = n0; s_n1 = n1; s_ngroups = ng;
    s_skip = (pr.full == 2 && cbase + n0 + n1 <= 256 * I) ? 1 : 0;
    s_cs = (diag && pr.colsum_part != nullptr) ? 1 : 0;
    s_pass = (s_cs || pr.fixup) ? 1 : 0;
    int nc = 32;
    while (nc < n0 + n1) nc <<= 1;
    s_tmem_cols = nc;
    for (int s = 0; s < GP_MAX_STAGES; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 1);
      mbar_init(smem_u32(&bar_ready[s]), 2 * GP_FIX_WARPS);
      mbar_init(smem_u32(&bar_empty[s]), 1);
    }
    mbar_init(smem_u32(&bar_accum), 1);
    mbar_fence_init();
  }
  __syncthreads();
  if (s_skip) return;       // both CTAs of the pair hold the same tile: both leave before any barrier or allocation
  const int ngroups = s_ngroups;
  const bool pass = s_pass != 0;
  const bool want_cs = s_cs != 0;
  const uint32_t ncols = (uint32_t)s_tmem_cols;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t stage_bytes = (uint32_t)ngroups * GROUP_BYTES;
  int nstages = GP_SMEM / (int)stage_bytes;
  if (nstages > GP_MAX_STAGES) nstages = GP_MAX_STAGES;
  const bool corr = (pr.pmean != nullptr) && !pr.full;
  const uint32_t const_base = smem_base + GP_SMEM;
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(&tmem_base_sh), ncols);
    tmem_relinquish_pair();
  } else if (warp >= 2 && corr) {
    // constant operands of the correction: every K row of a chunk holds the same values, -s c for the A block
    // (group 0), c for this CTA's halves of the two B panels (groups 1, 2), laid out as the TMA lays a stage down
    const int w = warp - 2;
    const float sA = -(float)(kCorrEveryStages * KSTEPS);
    for (int idx = w * 32 + lane; idx < 3 * GC * KR * 8; idx += GP_FIX_WARPS * 32) {
      const int u = idx & 7, r = (idx >> 3) % KR, j = (idx / (8 * KR)) % GC, cg = idx / (8 * KR * GC);
      int gcol;
      if (cg == 0) gcol = s_gcol[0];
      else if (cg == 1) gcol = s_gcol[s_bgroup];           // the A block itself when the first panel is shared
      else gcol = (s_n1 > 0) ? s_gcol[s_bgroup + 1] : -1;
      const float sc = (cg == 0) ? sA : 1.0f;
      const int col0 = gcol + j * CW + u * (BF ? 8 : 4);
      float v[8];
#pragma unroll
      for (int e = 0; e < (BF ? 8 : 4); ++e) {
        const int col = col0 + e;
        v[e] = (gcol >= 0 && col < M) ? sc * corr_round(pr.pmean[col], BF ? 1 : 0) : 0.f;
      }
      const uint32_t off = BF ? ((uint32_t)r * 128u + (((uint32_t)u ^ (uint32_t)(r & 7)) << 4))
                              : ((uint32_t)r * 128u + ((((uint32_t)(u >> 1) ^ (uint32_t)(r & 3)) << 5) | ((uint32_t)(u & 1) << 4)));
      float4 q;
      if (BF) {
        // exact: the values are on the bf16 grid (a power-of-two multiple of a rounded value)
        q.x = __uint_as_float((__float_as_uint(v[0]) >> 16) | (__float_as_uint(v[1]) & 0xffff0000u));
        q.y = __uint_as_float((__float_as_uint(v[2]) >> 16) | (__float_as_uint(v[3]) & 0xffff0000u));
        q.z = __uint_as_float((__float_as_uint(v[4]) >> 16) | (__float_as_uint(v[5]) & 0xffff0000u));
        q.w = __uint_as_float((__float_as_uint(v[6]) >> 16) | (__float_as_uint(v[7]) & 0xffff0000u));
      } else {
        q = make_float4(v[0], v[1], v[2], v[3]);
      }
      sts128(const_base + (uint32_t)cg * CGROUP + (uint32_t)j * CCHUNK + off, q);
    }
    fence_proxy_async_smem();
  }
  // barrier initialisation, TMEM allocation and the constant operands of both CTAs are complete past this point
  tc_fence_before();
  cluster_arrive();
  cluster_wait();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_sh;
  const volatile int* abortp = &abort_flag;
  const uint32_t peer_abort = mapa_shared(smem_u32(&abort_flag), rank ^ 1u);
#define GP_ABORT(code)                      \
  do {                                      \
    abort_flag = 1;                         \
    st_cluster_u32(peer_abort, 1u);         \
    atomicExch(pr.status, (code));     \
  } while (0)

  // row slab of this split
  const int64_t r_begin = (int64_t)split * pr.rows_per_split;
  int64_t r_end64 = r_begin + pr.rows_per_split;
  if (r_end64 > pr.rows) r_end64 = pr.rows;
  const int slab_rows = r_end64 > r_begin ? (int)(r_end64 - r_begin) : 0;
  const int nk = (slab_rows + SR - 1) / SR;

  if (warp == 0) {
    // ---- TMA producer (both CTAs): one instruction per column group, or one per chunk.  The loads of a stage
    // are issued by different lanes of the warp in one go: a lane that issued them one after the other spent
    // most of a bf16 stage's tensor time doing so.  Lane -> (group lane / GC, chunk lane % GC). ----
    {
      const CUtensorMap* m2[2] = {&g.mapA[pi], &g.mapB[pi]};
      const CUtensorMap* m3[2] = {&g.map3A[pi], &g.map3B[pi]};
      if (lane == 0) {
        tma_prefetch_desc(pr.use3d ? m3[0] : m2[0]);
        if (pr.full) tma_prefetch_desc(pr.use3d ? m3[1] : m2[1]);
      }
      const int q = lane / GC, c = lane - q * GC;
      const bool mine = q < ngroups;
      const int gcol = mine ? s_gcol[q] : 0;
      const int gsrc = mine ? s_gsrc[q] : 0;
      const bool box3 = pr.use3d && (gcol % CW) == 0;            // this group comes with one instruction
      const bool issue = mine && (!box3 || c == 0);
      const CUtensorMap* map = box3 ? m3[gsrc] : m2[gsrc];
      const int x = box3 ? 0 : gcol + c * CW;
      const int z = gcol / CW;
      const uint32_t doff = (uint32_t)q * GROUP_BYTES + (box3 ? 0u : (uint32_t)c * CHUNK);
      const uint32_t tx_bytes = stage_bytes;
      int s = 0;
      uint32_t ph = 0, sb = smem_base;
      int y = (int)r_begin;
      for (int kb = 0; kb < nk; ++kb) {
        const bool got = mbar_wait(smem_u32(&bar_empty[s]), ph ^ 1, abortp);
        if (!__all_sync(0xffffffffu, got)) { if (lane == 0) GP_ABORT(301); break; }
        const uint32_t own_full = smem_u32(&bar_full[s]);
        // pass protocol: this CTA's own barrier; direct: both CTAs' bytes are counted on the even CTA's barrier.
        // Bytes may be counted before the expectation is posted: the phase cannot end before that arrival.
        const uint32_t bar = pass ? own_full : mapa_shared(own_full, 0u);
        if (lane == 0) {
          if (pass) mbar_expect_tx(own_full, tx_bytes);
          else if (rank == 0) mbar_expect_tx(own_full, 2u * tx_bytes);
        }
        if (issue) {
          if (pass) {
            if (box3) tma_load_3d(sb + doff, map, 0, y, z, bar);
            else tma_load_2d(sb + doff, map, x, y, bar);
          } else {
            if (box3) tma_load_3d_pair(sb + doff, map, 0, y, z, bar);
            else tma_load_2d_pair(sb + doff, map, x, y, bar);
          }
        }
        y += SR;
        sb += stage_bytes;
        if (++s == nstages) { s = 0; ph ^= 1; sb = smem_base; }
      }
    }
  } else if (warp == 1) {
    // ---- MMA issuer: one thread of the even CTA drives the tensor cores of both SMs ----
    if (rank == 0 && elect_one()) {
      const int n0 = s_n0, n1 = s_n1;
      const uint64_t ad = make_smem_desc(smem_base, CHUNK, SBO, LAYOUT);
      const uint64_t bd0 = make_smem_desc(smem_base + s_bgroup * GROUP_BYTES, CHUNK, SBO, LAYOUT);
      const uint64_t bd1 = make_smem_desc(smem_base + (s_bgroup + 1) * GROUP_BYTES, CHUNK, SBO, LAYOUT);
      const uint32_t id0 = make_idesc(FMT, (uint32_t)n0, 1, 1, 256u);
      const uint32_t id1 = make_idesc(FMT, (uint32_t)(n1 > 0 ? n1 : 16), 1, 1, 256u);
      const uint64_t adc = make_smem_desc(const_base, CCHUNK, SBO, LAYOUT);
      const uint64_t bdc0 = make_smem_desc(const_base + CGROUP, CCHUNK, SBO, LAYOUT);
      const uint64_t bdc1 = make_smem_desc(const_base + 2 * CGROUP, CCHUNK, SBO, LAYOUT);
      int since_corr = 0;
      int s = 0;
      uint32_t ph = 0, soff16 = 0;
      const uint32_t stage16 = stage_bytes >> 4;
      uint32_t accum = 0;
      for (int kb = 0; kb < nk; ++kb) {
        if (!mbar_wait(smem_u32(pass ? &bar_ready[s] : &bar_full[s]), ph, abortp)) { GP_ABORT(302); break; }
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
          const uint64_t koff = (uint64_t)(soff16 + ks * KSTEP16);
          if (BF) mma_bf16_pair(tmem_base, ad + koff, bd0 + koff, id0, accum);
          else mma_tf32_pair(tmem_base, ad + koff, bd0 + koff, id0, accum);
          if (n1 > 0) {
            if (BF) mma_bf16_pair(tmem_base + 256u, ad + koff, bd1 + koff, id1, accum);
            else mma_tf32_pair(tmem_base + 256u, ad + koff, bd1 + koff, id1, accum);
          }
          accum = 1;
        }
        if (corr && ++since_corr == kCorrEveryStages) {
          // the mean product of the rows of the last stages leaves the accumulators
          since_corr = 0;
          if (BF) mma_bf16_pair(tmem_base, adc, bdc0, id0, 1u);
          else mma_tf32_pair(tmem_base, adc, bdc0, id0, 1u);
          if (n1 > 0) {
            if (BF) mma_bf16_pair(tmem_base + 256u, adc, bdc1, id1, 1u);
            else mma_tf32_pair(tmem_base + 256u, adc, bdc1, id1, 1u);
          }
        }
        mma_commit_pair(smem_u32(&bar_empty[s]), (uint16_t)3);    // frees the stage in both CTAs
        soff16 += stage16;
        if (++s == nstages) { s = 0; ph ^= 1; soff16 = 0; }
      }
      mma_commit_pair(smem_u32(&bar_accum), (uint16_t)3);
    }
  } else {
    // ---- fix-up / column sums over the stages (pass protocol only), then the epilogue ----
    const int w = warp - 2;
    // A warp pass covers 4 rows x 128 bytes of a chunk: lane -> (row lane >> 3, 16-byte unit lane & 7); warp w owns
    // rows 4w..4w+3 of every chunk of the stage.  The unit's position in its row is swizzled as the TMA wrote it.
    const int r_in = lane >> 3;
    const int u = lane & 7;
    const int r = w * 4 + r_in;
    const uint32_t off = BF ? ((uint32_t)r * 128u + (((uint32_t)u ^ (uint32_t)(r & 7)) << 4))
                            : ((uint32_t)r * 128u + ((((uint32_t)(u >> 1) ^ (uint32_t)(r & 3)) << 5) | ((uint32_t)(u & 1) << 4)));
    float acc[16];                                 // this lane's columns of the A group: 4 chunks x 4 or 2 chunks x 8
#pragma unroll
    for (int k = 0; k < 16; ++k) acc[k] = 0.f;
    bool ok = true;
    if (pass) {
      const uint32_t lead_ready0 = mapa_shared(smem_u32(&bar_ready[0]), 0u);
      const bool fix = !BF && pr.fixup != 0;
      const int nchunks = ngroups * GC;
      int s = 0;
      uint32_t ph = 0, sa = smem_base + off;
      for (int kb = 0; kb < nk; ++kb) {
        if (!mbar_wait(smem_u32(&bar_full[s]), ph, abortp)) { GP_ABORT(303); ok = false; break; }
        if (fix) {
          // every staged value rounded to the TF32 grid (nearest) in place: the tensor core would truncate
#pragma unroll
          for (int h = 0; h < GP_MAX_GROUPS; ++h) {
            if (h * GC < nchunks) {
              float4 v[GC];
#pragma unroll
              for (int jj = 0; jj < GC; ++jj) v[jj] = lds128(sa + (h * GC + jj) * CHUNK);
#pragma unroll
              for (int jj = 0; jj < GC; ++jj) {
                float4 x = v[jj];
                x.x = tf32_rna(x.x); x.y = tf32_rna(x.y); x.z = tf32_rna(x.z); x.w = tf32_rna(x.w);
                sts128(sa + (h * GC + jj) * CHUNK, x);
              }
            }
          }
          fence_proxy_async_smem();
        }
        if (want_cs) {
#pragma unroll
          for (int jh = 0; jh < GC * (SR / 32); ++jh) {
            const int j = jh % GC;                    // chunk; the 8 warps cover 32 rows of it per trip
            const float4 x = lds128(sa + j * CHUNK + (jh / GC) * 4096);
            const uint32_t qx = __float_as_uint(x.x), qy = __float_as_uint(x.y), qz = __float_as_uint(x.z), qw = __float_as_uint(x.w);
            if (!BF) {
              // column sums of the values as the tensor core reads them (fp32 operands are truncated to TF32)
              acc[4 * j + 0] += __uint_as_float(qx & 0xffffe000u);
              acc[4 * j + 1] += __uint_as_float(qy & 0xffffe000u);
              acc[4 * j + 2] += __uint_as_float(qz & 0xffffe000u);
              acc[4 * j + 3] += __uint_as_float(qw & 0xffffe000u);
            } else {
              acc[8 * j + 0] += __uint_as_float(qx << 16); acc[8 * j + 1] += __uint_as_float(qx & 0xffff0000u);
              acc[8 * j + 2] += __uint_as_float(qy << 16); acc[8 * j + 3] += __uint_as_float(qy & 0xffff0000u);
              acc[8 * j + 4] += __uint_as_float(qz << 16); acc[8 * j + 5] += __uint_as_float(qz & 0xffff0000u);
              acc[8 * j + 6] += __uint_as_float(qw << 16); acc[8 * j + 7] += __uint_as_float(qw & 0xffff0000u);
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(lead_ready0 + (uint32_t)s * 8u);
        sa += stage_bytes;
        if (++s == nstages) { s = 0; ph ^= 1; sa = smem_base + off; }
      }
    }
    if (want_cs) {
      // reduce over the row positions inside the warp, then over the warps through shared memory
#pragma unroll
      for (int k = 0; k < 16; ++k) {
        float x = acc[k];
        x += __shfl_xor_sync(0xffffffffu, x, 8);
        x += __shfl_xor_sync(0xffffffffu, x, 16);
        if (r_in == 0) {
          const int ci = BF ? ((k >> 3) * 64 + u * 8 + (k & 7)) : ((k >> 2) * 32 + u * 4 + (k & 3));
          s_csred[w][ci] = x;
        }
      }
    }
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (want_cs) {
      float* cs_out = pr.colsum_part + (int64_t)split * M;
      const int col0 = 256 * s_I + 128 * (int)rank;
      for (int i = threadIdx.x - 64; i < GP_GCOLS; i += GP_FIX_WARPS * 32) {
        float t = 0.f;
#pragma unroll
        for (int ww = 0; ww < GP_FIX_WARPS; ++ww) t += s_csred[ww][i];
        if (col0 + i < M) cs_out[col0 + i] = t;
      }
    }
    // ---- epilogue: this CTA's 128 rows of both accumulators -> partial output ----
    if (ok) {
      float* P = pr.out + (int64_t)split * M * M;
      const bool have = nk > 0;
      if (!have || mbar_wait(smem_u32(&bar_accum), 0, abortp)) {
        tc_fence_after();
        const int q = warp & 3, half = w >> 2;
        const int row = 256 * s_I + 128 * (int)rank + q * 32 + lane;
        for (int o = 0; o < 2; ++o) {
          const int n = o ? s_n1 : s_n0;
          const int cb = s_cbase + 256 * o;
          for (int c0 = 16 * half; c0 < n; c0 += 32) {
            uint32_t rr[16];
            if (have) {
              tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(256 * o + c0), rr);
              tmem_ld_wait();
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j) rr[j] = 0u;
            }
            const int col = cb + c0;
            if (pr.full == 2) {
              // symmetric output: (row, c) for c >= row and its mirror image (c, row) for c > row
              if (row < M && col + 15 >= row) {
                if (col > row && col + 15 < M) {
                  // wholly above the diagonal: the direct stores go out as 16-byte vectors
#pragma unroll
                  for (int j = 0; j < 16; j += 4)
                    *reinterpret_cast<float4*>(P + (int64_t)row * M + col + j) =
                        make_float4(__uint_as_float(rr[j]), __uint_as_float(rr[j + 1]), __uint_as_float(rr[j + 2]),
                                    __uint_as_float(rr[j + 3]));
#pragma unroll
                  for (int j = 0; j < 16; ++j) P[(int64_t)(col + j) * M + row] = __uint_as_float(rr[j]);
                } else {
#pragma unroll
                  for (int j = 0; j < 16; ++j) {
                    const int c = col + j;
                    if (c < M && c >= row) {
                      P[(int64_t)row * M + c] = __uint_as_float(rr[j]);
                      if (c > row) P[(int64_t)c * M + row] = __uint_as_float(rr[j]);
                    }
                  }
                }
              }
            } else if (row < M) {
#pragma unroll
              for (int j = 0; j < 16; j += 4) {
                if (col + j + 3 < M) {
                  *reinterpret_cast<float4*>(P + (int64_t)row * M + col + j) =
                      make_float4(__uint_as_float(rr[j]), __uint_as_float(rr[j + 1]), __uint_as_float(rr[j + 2]),
                                  __uint_as_float(rr[j + 3]));
                } else {
                  for (int jj = j; jj < j + 4; ++jj)
                    if (col + jj < M) P[(int64_t)row * M + col + jj] = __uint_as_float(rr[jj]);
                }
              }
            }
          }
        }
      } else {
        GP_ABORT(304);
      }
    }
  }
#undef GP_ABORT
  // no CTA leaves (or frees TMEM) while its peer may still signal it or the pair's MMAs may still run
  tc_fence_before();
  cluster_arrive();
  cluster_wait();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, ncols);
  }
}

// ---------------------------------------------------------------------------
// host: work list
// ---------------------------------------------------------------------------
struct PairTile { int n0, n1, ngroups; bool pass; bool skip; };   // skip: wholly below the diagonal of a symmetric product

void pair_tiles(int M, bool full, bool colsums, bool fixup, bool sym_out, std::vector<PairTile>& out) {
  const int M16 = (M + 15) / 16 * 16;
  out.clear();
  for (int I = 0; 256 * I < M16; ++I) {
    const int c_first = full ? 0 : 256 * I;
    for (int c = c_first, t = 0; c < M16; c += 512, ++t) {
      PairTile pt;
      pt.n0 = std::min(256, M16 - c);
      pt.n1 = std::max(0, std::min(256, M16 - c - 256));
      const bool diag = !full && t == 0;
      pt.ngroups = 1 + ((diag && pt.n0 == 256) ? 0 : 1) + (pt.n1 > 0 ? 1 : 0);
      pt.pass = fixup || (diag && colsums);
      pt.skip = full && sym_out && c + pt.n0 + pt.n1 <= 256 * I;
      out.push_back(pt);
    }
  }
}

// Estimated time of one tile over `rows` rows, microseconds: tensor time against staging time.  Staging rates
// are what a CTA sustains with every SM busy (measured: about 40 bytes per clock for bf16 tiles and 48 for fp32
// tiles, which then run at the TF32 tensor rate).
double pair_tile_us(const PairTile& t, bool bf16, bool fixup, double rows) {
  const double clk_us = 1800.0;                                   // SM clocks per microsecond under load
  const double tensor = (t.n0 + t.n1) / 512.0 * (bf16 ? 16.0 : 32.0);
  double load = t.ngroups * 128.0 * (bf16 ? 2.0 / 40.0 : 4.0 / 48.0);
  if (fixup) load *= 1.6;
  const double fixed = 4.0 + 128.0 * (t.n0 + t.n1) * 4.0 / 80e3;  // prologue, pipeline fill, epilogue stores
  return fixed + rows * std::max(tensor, load) / clk_us;
}

struct PairSpec {
  int M; int64_t rows; bool bf16, full, fixup, colsums, sym_out = false; int split_cap;
  std::vector<PairTile> tiles;
  int splits; int64_t per;     // chosen: splits, stages per split
};

// Chooses the split count of every problem so that the longest-first list schedule of all (tile, split) items
// over the resident CTA pairs ends earliest, counting what each further split costs the reduction that follows.
void pair_choose_splits(std::vector<PairSpec>& P, int slots) {
  double best = 1e300;
  std::vector<int> best_s(P.size(), 1);
  std::vector<double> items;
  // the search costs the host a fraction of a millisecond: its result is kept per list of problems
  static std::map<std::vector<int64_t>, std::pair<std::vector<int>, double>> memo;
  std::vector<int64_t> key;
  key.push_back(slots);
  for (const PairSpec& p : P) {
    key.push_back(p.M); key.push_back(p.rows); key.push_back(p.split_cap);
    key.push_back((p.bf16 ? 1 : 0) | (p.full ? 2 : 0) | (p.fixup ? 4 : 0) | (p.sym_out ? 8 : 0) | (p.colsums ? 16 : 0));
  }
  auto hit = memo.find(key);
  if (hit != memo.end()) { best_s = hit->second.first; best = hit->second.second; }
  for (int step = 0; hit == memo.end() && step < 64; ++step) {
    const double tau = 6.0 * std::pow(1.12, step);                // target item time, 6 us .. 7.5 ms
    double extra = 0;
    size_t count = 0;
    items.clear();
    std::vector<int> sp(P.size());
    for (size_t l = 0; l < P.size(); ++l) {
      PairSpec& p = P[l];
      double longest = 0;
      for (const PairTile& t : p.tiles)
        if (!t.skip) longest = std::max(longest, pair_tile_us(t, p.bf16, p.fixup, (double)p.rows));
      const int SRh = pair_sr(p.bf16);
      const int64_t nsr = (p.rows + SRh - 1) / SRh;
      int64_t s = (int64_t)(longest / tau + 0.5);
      s = std::max<int64_t>(1, std::min<int64_t>(s, std::min<int64_t>(p.split_cap, nsr)));
      const int64_t per = (nsr + s - 1) / s;
      s = (nsr + per - 1) / per;
      sp[l] = (int)s;
      for (const PairTile& t : p.tiles) {
        if (t.skip) continue;
        for (int64_t k = 0; k < s; ++k) {
          const double r = (double)std::min<int64_t>(per * SRh, p.rows - k * per * SRh);
          items.push_back(pair_tile_us(t, p.bf16, p.fixup, r));
        }
        count += (size_t)s;
      }
      // the reduction reads every partial once (upper triangle), at about 4 TB/s
      if (!p.full) extra += (double)(s - 1) * 0.55 * 4.0 * p.M * (double)p.M / 4e6;
    }
    if (count > (size_t)GP_MAX_ITEMS) continue;
    std::sort(items.begin(), items.end(), [](double a, double b) { return a > b; });
    std::vector<double> slot(slots, 0.0);
    for (double c : items) {
      auto m = std::min_element(slot.begin(), slot.end());
      *m += c;
    }
    const double span = *std::max_element(slot.begin(), slot.end()) + extra;
    if (span < best) { best = span; best_s = sp; }
  }
  if (hit == memo.end()) {
    if (memo.size() > 256) memo.clear();
    memo[key] = std::make_pair(best_s, best);
  }
  const int forced = tuning().pair_splits;   // tuning aid
  for (size_t l = 0; l < P.size(); ++l) {
    PairSpec& p = P[l];
    const int64_t nsr = (p.rows + pair_sr(p.bf16) - 1) / pair_sr(p.bf16);
    int64_t s = best_s[l];
    if (forced > 0) s = std::max<int64_t>(1, std::min<int64_t>(forced, std::min<int64_t>(p.split_cap, nsr)));
    if (tuning().pair_debug) fprintf(stderr, "[fw] pair: M=%d rows=%lld tiles=%zu splits=%lld (cap %d) est %.1f us\n", p.M, (long long)p.rows, p.tiles.size(), (long long)s, p.split_cap, best);
    const int64_t per = (nsr + s - 1) / s;
    p.splits = (int)((nsr + per - 1) / per);
    p.per = per;
  }
}

struct PairSource { const void* A; const void* B; int64_t lda, ldb; float* out; float* colsum; int32_t* status; const float* pmean; };

fw_status pair_launch(std::vector<PairSpec>& specs, const std::vector<PairSource>& src, int prof_class, cudaStream_t s) {
  static bool attr_set = false;
  static int slots = GP_CLUSTER_SLOTS;
  static SmemAttrCache attr_f32, attr_bf16;
  const int smem = GP_SMEM + GP_CONST + 1024;
  if (ensure_dyn_smem(gram_pair_kernel<false>, smem, attr_f32) != cudaSuccess ||
      ensure_dyn_smem(gram_pair_kernel<true>, smem, attr_bf16) != cudaSuccess) {
    cudaGetLastError();
    return FW_ERR_CUDA;
  }
  if (!attr_set) {
    // how many pairs the device really keeps resident (fewer than SMs / 2 when a GPC has an odd SM out)
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(2 * GP_MAX_ITEMS); cfg.blockDim = dim3(GP_THREADS); cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    int nc = 0;
    if (cudaOccupancyMaxActiveClusters(&nc, gram_pair_kernel<false>, &cfg) == cudaSuccess && nc > 0) slots = nc;
    else cudaGetLastError();
    if (tuning().pair_debug) fprintf(stderr, "[fw] pair: %d resident CTA pairs\n", slots);
    attr_set = true;
  }
  const int n = (int)specs.size();
  for (int base = 0; base < n;) {
    // one element type per launch, at most GP_MAX_PROBLEMS problems
    int cnt = 0;
    while (base + cnt < n && cnt < GP_MAX_PROBLEMS && specs[base + cnt].bf16 == specs[base].bf16) ++cnt;
    std::vector<PairSpec> grp(specs.begin() + base, specs.begin() + base + cnt);
    pair_choose_splits(grp, slots);
    std::vector<PairGroup> gbuf(1);           // 17 KB: kept off the stack; the launch copies it
    PairGroup& g = gbuf[0];
    memset(&g, 0, sizeof(g));
    struct Item { uint32_t code; double cost, pos; };
    std::vector<Item> items;
    for (int i = 0; i < cnt; ++i) {
      PairSpec& sp = grp[i];
      const PairSource& so = src[base + i];
      PairProblem& p = g.p[i];
      p.out = so.out; p.colsum_part = so.colsum; p.rows = sp.rows; p.M = sp.M;
      p.status = so.status; p.pmean = so.pmean; p.full = sp.full ? (sp.sym_out ? 2 : 1) : 0; p.fixup = sp.fixup; p.rows_per_split = (int)(sp.per * pair_sr(sp.bf16));
      const bool bf = sp.bf16;
      const uint32_t cw = bf ? 64 : 32;       // chunk rows of 128 bytes
      if (!tmap_encode_2d(&g.mapA[i], bf, so.A, (uint64_t)sp.M, (uint64_t)sp.rows, (uint64_t)so.lda, cw, (uint32_t)pair_sr(bf)) ||
          !tmap_encode_2d(&g.mapB[i], bf, so.B, (uint64_t)sp.M, (uint64_t)sp.rows, (uint64_t)so.ldb, cw, (uint32_t)pair_sr(bf))) {
        fprintf(stderr, "[fw] tensor-map encoding failed (pair kernel)\n");
        return FW_ERR_CUDA;
      }
      p.use3d = (sp.M % 64) == 0 &&
                tmap_encode_chunked_3d(&g.map3A[i], bf, so.A, (uint64_t)sp.M, (uint64_t)sp.rows, (uint64_t)so.lda, (uint32_t)pair_sr(bf), GP_GCOLS / cw, cw) &&
                tmap_encode_chunked_3d(&g.map3B[i], bf, so.B, (uint64_t)sp.M, (uint64_t)sp.rows, (uint64_t)so.ldb, (uint32_t)pair_sr(bf), GP_GCOLS / cw, cw);
      for (size_t t = 0; t < sp.tiles.size(); ++t) {
        if (sp.tiles[t].skip) continue;             // never launched: the mirrored entries of other tiles fill it
        for (int k = 0; k < sp.splits; ++k) {
          const double r = (double)std::min<int64_t>(sp.per * pair_sr(sp.bf16), sp.rows - (int64_t)k * sp.per * pair_sr(sp.bf16));
          Item itm;
          itm.code = ((uint32_t)i << 28) | ((uint32_t)t << 14) | (uint32_t)k;
          itm.cost = pair_tile_us(sp.tiles[t], sp.bf16, sp.fixup, r);
          itm.pos = (double)k / sp.splits;
          items.push_back(itm);
        }
      }
      specs[base + i].splits = sp.splits;
      specs[base + i].per = sp.per;
    }
    if (items.empty() || items.size() > (size_t)GP_MAX_ITEMS) return FW_ERR_SHAPE;
    // CTAs are handed to SMs in index order as SMs free up.  All tiles of a row slab run together (the slab comes
    // from DRAM once and the other tiles find it in L2), every problem advancing through its rows at the same
    // relative pace; within a slab the longest tiles go first so that short ones fill the end of the launch.
    std::stable_sort(items.begin(), items.end(), [](const Item& a, const Item& b) {
      if (a.pos != b.pos) return a.pos < b.pos;
      return a.cost > b.cost;
    });
    for (size_t i = 0; i < items.size(); ++i) g.item[i] = items[i].code;
    g.n = cnt; g.nitems = (int)items.size();
    ProfScope ps(prof_class, s);
    if (specs[base].bf16) gram_pair_kernel<true><<<2 * g.nitems, GP_THREADS, smem, s>>>(g);
    else gram_pair_kernel<false><<<2 * g.nitems, GP_THREADS, smem, s>>>(g);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
      fprintf(stderr, "[fw] gram_pair_kernel launch: %s\n", cudaGetErrorString(e));
      return FW_ERR_CUDA;
    }
    base += cnt;
  }
  return FW_OK;
}

// smallest matrix dimension the pair kernels take (below it one CTA's TMEM holds the whole triangle)
int pair_min_m() { return tuning().pair_min_m; }

}  // namespace

// Unshifted blocks only (bf16 X, or long fp32 blocks): centring by a pilot mean stays with the single-CTA kernel.
// Small products stay there too: they share its one launch with the other small layers of a group, which costs
// less than a second launch gains.
bool umma_pair_gram_eligible(const UmmaGramItem& it) {
  const int M16 = (it.M + 15) / 16 * 16;
  if (it.shift != nullptr) return false;
  if ((double)it.rows * M16 * M16 < 1e10) return false;
  return M16 >= pair_min_m() && pair_tiles_sym(M16) <= GP_MAX_ITEMS;
}

bool umma_pair_atb_eligible(int M) {
  const int M16 = (M + 15) / 16 * 16;
  return M16 >= std::max(pair_min_m(), 1024) && pair_tiles_full(M16) <= GP_MAX_ITEMS;
}

// Partial buffers a layer of dimension M should have for the pair kernel to balance its launch:
// eight rounds of resident pairs, within a quarter of a gigabyte.
int umma_pair_split_cap(int M) {
  const int M16 = (M + 15) / 16 * 16;
  if (M16 < pair_min_m()) return 1;
  const int tiles = pair_tiles_sym(M16);
  int64_t cap = (8 * GP_CLUSTER_SLOTS + tiles - 1) / tiles;
  const int64_t mem = ((int64_t)256 << 20) / ((int64_t)M * M * 4);
  if (cap > mem) cap = mem;
  if (cap < 2) cap = 2;
  if (cap > 296) cap = 296;
  return (int)cap;
}

fw_status umma_pair_gram_launch(UmmaGramItem* items, int n, cudaStream_t s) {
  if (n <= 0) return FW_OK;
  std::stable_sort(items, items + n, [](const UmmaGramItem& a, const UmmaGramItem& b) { return a.x_bf16 < b.x_bf16; });
  std::vector<PairSpec> specs(n);
  std::vector<PairSource> src(n);
  for (int i = 0; i < n; ++i) {
    const UmmaGramItem& it = items[i];
    PairSpec& p = specs[i];
    p.M = it.M; p.rows = it.rows; p.bf16 = it.x_bf16 != 0; p.full = false; p.fixup = false; p.colsums = true;
    p.split_cap = std::max(1, std::min(it.split_cap, 0x3fff));
    pair_tiles(p.M, false, true, false, false, p.tiles);
    src[i] = PairSource{it.X, it.X, it.ldx, it.ldx, it.gram_part, it.colsum_part, it.status, it.pmean};
  }
  fw_status st = pair_launch(specs, src, FW_PROF_GRAM, s);
  if (st != FW_OK) return st;
  for (int i = 0; i < n; ++i) {
    items[i].splits_out = specs[i].splits;
    // rows' worth of c c^T the kernel took out: per split, the stages covered by whole correction periods
    double taken = 0;
    if (items[i].pmean) {
      const int sr = pair_sr(specs[i].bf16);
      const int64_t per_rows = specs[i].per * sr;
      for (int k = 0; k < specs[i].splits; ++k) {
        const int64_t slab = std::min<int64_t>(per_rows, specs[i].rows - (int64_t)k * per_rows);
        const int64_t nk = slab > 0 ? (slab + sr - 1) / sr : 0;
        taken += (double)((nk / kCorrEveryStages) * kCorrEveryStages * sr);
      }
    }
    items[i].corr_out = (float)taken;
  }
  return FW_OK;
}

// D = A^T B, square fp32 matrices, operands rounded to TF32 (nearest) in shared memory
fw_status umma_pair_atb_launch(const UmmaAtbItem* items, int n, cudaStream_t s) {
  if (n <= 0) return FW_OK;
  std::vector<PairSpec> specs(n);
  std::vector<PairSource> src(n);
  for (int i = 0; i < n; ++i) {
    const UmmaAtbItem& it = items[i];
    PairSpec& p = specs[i];
    p.M = it.M; p.rows = it.M; p.bf16 = false; p.full = true; p.fixup = true; p.colsums = false; p.sym_out = it.sym != 0;
    p.split_cap = 1;
    pair_tiles(p.M, true, false, true, it.sym != 0, p.tiles);
    src[i] = PairSource{it.A, it.B, it.M, it.M, it.C, nullptr, it.status, nullptr};
  }
  return pair_launch(specs, src, FW_PROF_RESYNC, s);
}

}  // namespace fw
