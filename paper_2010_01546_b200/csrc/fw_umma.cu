// Tensor-core engine for sm_100a: tcgen05.mma with TMEM accumulators, operands
// staged in shared memory by TMA, warp-specialised (one TMA producer warp, one
// MMA issuer warp, four epilogue warps), mbarrier pipeline with bounded waits.
//
//   gram_umma_kernel  X^T X with column sums (Eqs. 3, 5), and the re-sync products A^T B,
//                     one CTA per tile.  (G Qs runs on CTA pairs: fw_umma_gq.cu.)
#include <algorithm>
#include <cstdio>
#include <cstdlib>
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

// 4-D view of a zero-padded NHWC fp32 activation [B][H + 2][W + 2][C] for implicit im2col: (i, x, yy, b) with i
// over the 3 C contiguous floats of three horizontally adjacent pixels and x advancing by one pixel (C floats), so
// the windows of neighbouring pixels overlap.  Box (32, bw, bh, 1); floats past 3 C read as zero.
bool encode_im2col_4d(CUtensorMap* m, const void* base, int B, int H, int W, int C, uint32_t bw, uint32_t bh) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[4] = {(cuuint64_t)(3 * C), (cuuint64_t)W, (cuuint64_t)(H + 2), (cuuint64_t)B};
  cuuint64_t strides[3] = {(cuuint64_t)C * 4, (cuuint64_t)(W + 2) * C * 4, (cuuint64_t)(H + 2) * (W + 2) * C * 4};
  cuuint32_t box[4] = {32, bw, bh, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// The same activation as (i, x, yy, q, b): q steps through the 32-float chunks of a window (stride 128 bytes), so a
// box (32, bw, bh, cpr, 1) lays all chunks of one patch row down chunk-major with one instruction.  The last chunk
// of a window whose 3 C floats do not fill it runs on into the next pixel; those columns are dropped downstream.
bool encode_im2col_5d(CUtensorMap* m, const void* base, int B, int H, int W, int C, uint32_t bw, uint32_t bh,
                      uint32_t cpr) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[5] = {32, (cuuint64_t)W, (cuuint64_t)(H + 2), (cuuint64_t)cpr, (cuuint64_t)B};
  cuuint64_t strides[4] = {(cuuint64_t)C * 4, (cuuint64_t)(W + 2) * C * 4, 128, (cuuint64_t)(H + 2) * (W + 2) * C * 4};
  cuuint32_t box[5] = {32, bw, bh, cpr, 1};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 5, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Chunked view of a row-major [rows][cols] matrix whose column count is a multiple of the chunk width cw:
// dims (cw columns, rows, cols / cw chunks), box (cw, box_rows, box_chunks).  One TMA instruction then lays
// box_chunks chunks down chunk-major in shared memory, the layout the MMA descriptors expect.
bool encode_chunked_3d(CUtensorMap* m, CUtensorMapDataType dt, int elem_bytes, const void* base, uint64_t cols,
                       uint64_t rows, uint64_t ld, uint32_t box_rows, uint32_t box_chunks, CUtensorMapSwizzle sw,
                       uint32_t cw = 32) {
  EncodeTiledFn fn = encode_fn();
  if (!fn || (cols % cw) != 0) return false;
  cuuint64_t dims[3] = {cw, rows, cols / cw};
  cuuint64_t strides[2] = {ld * (uint64_t)elem_bytes, cw * (uint64_t)elem_bytes};
  cuuint32_t box[3] = {cw, box_rows, box_chunks};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(m, dt, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

constexpr int kMaxUmmaGroup = 16;

// ---------------------------------------------------------------------------
// Gram pass: partial S2 = sum over a slab of rows of (x - c)(x - c)^T and the
// partial column sums of (x - c), for one output tile of one layer  (Eqs. 3, 5).
//
// X is row-major rows x M and the contraction runs over rows, so both MMA
// operands are "MN-major".  A stage holds SR rows of X as chunks of 32 columns,
// each laid down by one TMA box in the canonical MN-major operand layout:
//   fp32 (kind::tf32): rows of 128 bytes, 32-byte units swizzled by (row & 3)
//        -- the only MN-major layout the tensor cores accept for 32-bit operands
//        (TMA swizzle 128B with 32-byte atoms; 4-row x 128-byte atoms);
//   bf16 (kind::f16):  rows of 64 bytes, 16-byte units swizzled by (row >> 1) & 3
//        (TMA swizzle 64B; 8-row x 64-byte atoms).
// Next chunk = leading offset, next K-atom = 512 bytes, next MMA k-step = 1024 bytes
// in both cases.  The same chunk serves as A operand (its columns become Gram
// rows) and as B operand (its columns become Gram columns): X is fetched once per tile.
//
// Modes
//   STREAM (small M, all needed accumulators fit the 512 TMEM columns): the CTA
//     owns a slab of rows and the whole upper block-triangle of the Gram matrix:
//     block-row i (128 Gram rows) x columns [128 i, M).  X is read exactly once.
//   TILED: the CTA owns block-row i x a panel of <= 256 columns, and a row slab.
// A-operand chunks beyond the loaded range (last block-row) address whatever
// follows in shared memory; the Gram rows they produce are never read.
//
// Warp roles: 0 = TMA producer, 1 = MMA issuer, 2..9 = fix-up + epilogue.  The
// fix-up warps pass over every landed stage once: subtract the pilot mean and
// round to TF32 (fp32 X only), accumulate column sums, then hand the stage to
// the MMA warp.  Centring before the product keeps the one-pass covariance free
// of cancellation and makes the TF32 input conversion unbiased.
// ---------------------------------------------------------------------------
constexpr int GR_SR = 32;                 // rows of X per stage (ones mode: 32 << k, chosen per layer by the host)
constexpr int GR_CW = 32;                 // columns per chunk
constexpr int GR_ABL = 128 / GR_CW;       // chunks per 128-column block
constexpr int GR_MAX_STAGES = 8;
constexpr int GR_FIX_WARPS = 8;
constexpr int GR_THREADS = 64 + GR_FIX_WARPS * 32;   // producer + MMA issuer + fix-up/epilogue warps
constexpr int GR_MAX_OPS = 4;             // STREAM mode at M <= 288 needs four, TILED one
constexpr int GR_MAX_SLOTS = 12;          // chunks per stage: 4 (A block) + 8 (256-column panel)
constexpr int GR_SMEM_BUDGET = 184 * 1024;
constexpr int GR_SLACK = GR_ABL * GR_SR * 128;   // room for out-of-range A chunks after the last stage

struct GramProblem {
  const float* shift;      // may be null
  float* gram_part;
  float* colsum_part;
  int64_t rows;
  int32_t M, bf16;
  int32_t stream;          // 1: STREAM mode, 0: TILED
  int32_t splits;
  int32_t ntiles;          // tiles per split (1 in STREAM mode)
  int32_t first_cta;
  int32_t rows_per_split;  // multiple of GR_SR
  int32_t full;            // 1: D = A^T B with A from mapX, B from mapB, every tile of the full output;
                           // 2: the same for a symmetric D: tiles wholly below the diagonal are skipped, the others
                           //    write their entries on and above the diagonal and mirror those above it
  int32_t fixup;           // fp32 only. 1: subtract shift, round to TF32, write back; 0: read-only column sums
  int32_t use3d;           // 1: chunked 3-D tensor maps (map3a / map3b): one TMA instruction per column range
  int32_t box_a;           // chunks per map3a box (STREAM: all chunks; TILED: 4)
  int32_t sr;              // rows of X per stage: GR_SR, or a larger power of two for ones-mode layers
  int32_t* status;         // time-out word of the owning layer
  // Implicit im2col (3 x 3 patches, stride 1, zero padding 1): the rows of X are never materialised.  mapX is a 4-D
  // map of the zero-padded activation [b][y + 2][x + 2][C] seen as (i, x, yy, b): i runs over the 3 C contiguous
  // floats of the three horizontally adjacent pixels that start at padded pixel x, x has stride C (overlapping
  // windows), so a box (32, bw, bh, 1) at (32 q, x0, y0 + t, b) is chunk q of patch-row t for bw x bh pixels.
  // A stage is bw x bh pixels (sr of them, slots past W read as zeros); `rows` counts stage slots.
  int32_t im2col;
  int32_t i2c_bw, i2c_bh;  // pixels per stage along x and y
  int32_t i2c_nx, i2c_ny;  // stages per image along x and y
  int32_t i2c_cpr;         // chunks per patch row = ceil(3 C / 32)
  int32_t i2c_c3;          // 3 C: real columns per patch row
  int32_t Mp;              // columns as staged = 3 * cpr * 32 (= M when 3 C is a multiple of 32)
};

// column as staged -> column of the patch matrix (k = 3: patch row t, then the 3 C floats of its window); -1: padding
__device__ __forceinline__ int i2c_col(int mp, int cpr, int c3) {
  const int w = 32 * cpr;
  const int t = mp / w, r = mp - t * w;
  return r < c3 ? t * c3 + r : -1;
}
struct GramGroup {
  CUtensorMap mapX[kMaxUmmaGroup];
  CUtensorMap mapB[kMaxUmmaGroup];   // second source, used only by problems with full = 1
  CUtensorMap map3a[kMaxUmmaGroup];  // chunked 3-D views (use3d = 1): A-side box, and
  CUtensorMap map3b[kMaxUmmaGroup];  // B-side box of 8 chunks (on the second source when full = 1)
  GramProblem p[kMaxUmmaGroup];
  int32_t n;
};

// n: columns the MMA covers (N); n_out: leading columns that are Gram entries; cs_off: offset of the column-sum
// columns inside the accumulator (ones mode), -1 without
struct GramOp { int32_t a_slot, b_slot, n, tmem_col, row0, col0, n_out, cs_off; };

// number of (block-row, panel) tiles of the TILED mode; panels are 256 columns wide
__host__ __device__ inline int gram_tiled_count(int M16) {
  int nb = (M16 + 127) / 128, t = 0;
  for (int i = 0; i < nb; ++i) t += (M16 - 128 * i + 255) / 256;
  return t;
}

// Whether a STREAM-mode layer can take its column sums out of the tensor core (ones mode): the last MMA of every
// block row, widened by the chunk of ones, must stay within N <= 256 and all accumulators within 512 columns.
__host__ __device__ inline bool gram_ones_fits(int M16) {
  const int nb = (M16 + 127) / 128;
  const int ns = (M16 + GR_CW - 1) / GR_CW;
  int cols = 0;
  for (int i = 0; i < nb; ++i) {
    for (int c = 128 * i; c < M16; c += 256) {
      const int n = (256 < M16 - c) ? 256 : (M16 - c);
      if (c + n == M16) {
        const int wide = (ns - c / GR_CW) * GR_CW + 16;
        if (wide > 256) return false;
        cols += wide;
      } else {
        cols += n;
      }
    }
  }
  return cols <= 512;
}

// Rows per stage of a ones-mode layer.  Nothing but the TMA and the MMA warp touches its stages, and a 32-row
// stage of a narrow layer is a few hundred tensor cycles and a few KB: the hand-offs of a stage then cost more than
// its work.  Stages grow (powers of two, at most a 256-row TMA box) up to about 48 KB.
__host__ inline int gram_ones_stage_rows(int M16, bool bf16, int64_t rows, int budget = 48 * 1024) {
  const int ns = (M16 + GR_CW - 1) / GR_CW;
  const int row_bytes = (ns + 1) * (bf16 ? 64 : 128);
  int sr = GR_SR;
  while (sr * 2 <= 256 && sr * 2 * row_bytes <= budget && (int64_t)sr * 2 * 64 <= rows) sr *= 2;
  return sr;
}

__device__ __forceinline__ float4 lds128(uint32_t a) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ void sts128(uint32_t a, float4 v) {
  asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(a), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
// round-to-nearest (ties away) of an fp32 value to the TF32 grid, on the integer pipe
__device__ __forceinline__ float tf32_rna(float x) {
  return __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xffffe000u);
}

// BF = true: bf16 X (kind::f16), BF = false: fp32 X (kind::tf32).  All per-stage
// loops are free of divisions and descriptor rebuilding: the single issuing
// threads of the producer and MMA warps run serial code, so every instruction in
// their loops is on the critical path of the pipeline.
template <bool BF>
__global__ void __launch_bounds__(GR_THREADS, 1) gram_umma_kernel(const __grid_constant__ GramGroup g) {
  constexpr int RB = BF ? 64 : 128;               // bytes per chunk row
  constexpr int KROWS = BF ? 16 : 8;              // rows of X one MMA contracts over
  constexpr uint64_t LAYOUT = BF ? kSwizzle64B : kSwizzle128B32;
  constexpr uint32_t FMT = BF ? 1u : 2u;

  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[GR_MAX_STAGES], bar_ready[GR_MAX_STAGES], bar_empty[GR_MAX_STAGES], bar_accum;
  __shared__ uint32_t tmem_base_sh;
  __shared__ int abort_flag;
  __shared__ GramOp ops[GR_MAX_OPS];
  __shared__ int s_nops, s_nslots, s_r0_col, s_r0_slots, s_r1_col, s_r1_slots, s_tmem_cols, s_cs_slots, s_ones;
  __shared__ int s_slack_chunks, s_skip;
  __shared__ float s_csred[GR_FIX_WARPS][GR_MAX_SLOTS * GR_CW];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int pi = 0;
#pragma unroll 1
  for (int i = 1; i < g.n; ++i)
    if ((int)blockIdx.x >= g.p[i].first_cta) pi = i;
  const GramProblem& pr = g.p[pi];
  const int local = blockIdx.x - pr.first_cta;
  const int split = local / pr.ntiles, tile = local - split * pr.ntiles;
  const int M = pr.M;
  const int M16 = pr.im2col ? pr.Mp : (M + 15) / 16 * 16;   // MMA extents are multiples of 16
  const int SR = pr.sr;                           // rows per stage
  const int KSTEPS = SR / KROWS;                  // MMAs along K per stage
  const uint32_t CHUNK = (uint32_t)SR * RB;       // bytes per chunk

  if (threadIdx.x == 0) {
    abort_flag = 0;
    s_skip = 0;
    int nops = 0, tcol = 0;
    int ones = 0;
    if (pr.stream) {
      const int nb = (M16 + 127) / 128;
      const int ns = (M16 + GR_CW - 1) / GR_CW;
      // Ones mode: a chunk of ones follows the data chunks of every stage, and the last MMA of each block row
      // runs on into it, so the column sums of the values as the tensor core reads them come out as 16 extra
      // accumulator columns and no thread has to read the stage.  Taken when no fix-up pass is owed and the
      // widened MMAs fit (N <= 256, 512 accumulator columns in all).
      if (!pr.fixup && !pr.full) ones = gram_ones_fits(M16) ? 1 : 0;
      for (int i = 0; i < nb; ++i) {
        for (int c = 128 * i; c < M16; c += 256) {
          const int n = min(256, M16 - c);
          const bool last = ones && (c + n == M16);
          const int wide = last ? (ns - c / GR_CW) * GR_CW + 16 : n;
          ops[nops++] = GramOp{i * GR_ABL, c / GR_CW, wide, tcol, 128 * i, c, n, last ? wide - 16 : -1};
          tcol += wide;
        }
      }
      s_r0_col = 0; s_r0_slots = ns; s_r1_col = 0; s_r1_slots = 0;
      s_cs_slots = ones ? 0 : s_r0_slots;
    } else if (pr.full) {
      const int np = (M16 + 255) / 256;
      const int i = tile / np, t = tile - i * np;
      const int pc0 = 256 * t;
      const int pw = min(256, M16 - pc0);
      s_r0_col = 128 * i; s_r0_slots = GR_ABL; s_r1_col = pc0; s_r1_slots = (pw + GR_CW - 1) / GR_CW;
      ops[nops++] = GramOp{0, GR_ABL, pw, 0, 128 * i, pc0, pw, -1};
      s_cs_slots = 0;
      tcol = pw;
      s_skip = (pr.full == 2 && pc0 + pw <= 128 * i) ? 1 : 0;
    } else {
      int i = 0, t = tile;
      for (;; ++i) {
        const int np = (M16 - 128 * i + 255) / 256;
        if (t < np) break;
        t -= np;
      }
      const int pc0 = 128 * i + 256 * t;
      const int pw = min(256, M16 - pc0);
      const int pslots = (pw + GR_CW - 1) / GR_CW;
      if (t == 0) {
        s_r0_col = pc0; s_r0_slots = pslots; s_r1_col = 0; s_r1_slots = 0;
        ops[nops++] = GramOp{0, 0, pw, 0, 128 * i, pc0, pw, -1};
        s_cs_slots = min(GR_ABL, pslots);
      } else {
        s_r0_col = 128 * i; s_r0_slots = GR_ABL; s_r1_col = pc0; s_r1_slots = pslots;
        ops[nops++] = GramOp{0, GR_ABL, pw, 0, 128 * i, pc0, pw, -1};
        s_cs_slots = 0;
      }
      tcol = pw;
    }
    if (pr.use3d && !pr.stream && !pr.im2col) {
      // a 3-D box always delivers its full chunk count (chunks past the matrix are zero-filled)
      if (s_r1_slots == 0) s_r0_slots = 2 * GR_ABL;
      else { s_r0_slots = GR_ABL; s_r1_slots = 2 * GR_ABL; }
    }
    s_nops = nops;
    s_ones = ones;
    s_nslots = s_r0_slots + s_r1_slots;
    // A blocks are read as 4 chunks from their first slot: chunks past the end of a stage belong to the next one,
    // past the last stage to the slack that follows the ring
    int over = 0;
    for (int o = 0; o < nops; ++o) over = max(over, ops[o].a_slot + GR_ABL - (s_nslots + ones));
    s_slack_chunks = over;
    int nc = 32;
    while (nc < tcol) nc <<= 1;
    s_tmem_cols = nc;
    for (int s = 0; s < GR_MAX_STAGES; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 1);
      mbar_init(smem_u32(&bar_ready[s]), GR_FIX_WARPS);
      mbar_init(smem_u32(&bar_empty[s]), 1);
    }
    mbar_init(smem_u32(&bar_accum), 1);
    mbar_fence_init();
  }
  __syncthreads();
  if (s_skip) return;                             // nothing allocated yet; every thread of the CTA leaves
  const int nslots = s_nslots, nops = s_nops;
  const bool ones = s_ones != 0;
  // no pass of the fix-up warps over the stages: nothing to centre and no column sums owed to them
  const bool direct = ones || (!pr.fixup && s_cs_slots == 0);
  const uint32_t ncols = (uint32_t)s_tmem_cols;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t tx_bytes = (uint32_t)nslots * CHUNK;                    // what the TMA delivers per stage
  const uint32_t stage_bytes = tx_bytes + (ones ? (uint32_t)CHUNK : 0u);  // + the chunk of ones
  int nstages = (GR_SMEM_BUDGET - (SR == GR_SR ? GR_SLACK : s_slack_chunks * (int)CHUNK)) / (int)stage_bytes;
  if (nstages > GR_MAX_STAGES) nstages = GR_MAX_STAGES;
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_sh), ncols);
    tmem_relinquish();
  } else if (warp >= 2 && ones) {
    // the value 1 in every element of the extra chunk of each stage (uniform, so the swizzle does not matter)
    const float one = BF ? __uint_as_float(0x3f803f80u) : 1.0f;
    const float4 v1 = make_float4(one, one, one, one);
    for (int st = 0; st < nstages; ++st)
      for (int i = (int)threadIdx.x - 64; i < CHUNK / 16; i += GR_FIX_WARPS * 32)
        sts128(smem_base + st * stage_bytes + tx_bytes + i * 16, v1);
    fence_proxy_async_smem();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_sh;
  const volatile int* abortp = &abort_flag;

  // row slab of this split
  const int64_t r_begin = (int64_t)split * pr.rows_per_split;
  int64_t r_end64 = r_begin + pr.rows_per_split;
  if (r_end64 > pr.rows) r_end64 = pr.rows;
  const int slab_rows = r_end64 > r_begin ? (int)(r_end64 - r_begin) : 0;
  const int nk = (slab_rows + SR - 1) / SR;
  const int r0c = s_r0_col, r0n = s_r0_slots, r1c = s_r1_col;

  if (warp == 0 && pr.im2col) {
    // ---- TMA producer, implicit im2col: lane j fetches chunk j of the stage (one 4-D box each), all lanes of the
    //      warp issuing together ----
    const bool win = pr.use3d != 0;          // one instruction per patch row (all chunks of the stage are loaded)
    if (lane == 0) tma_prefetch_desc(win ? &g.map3a[pi] : &g.mapX[pi]);
    const int cpr = pr.i2c_cpr;
    const bool mine = win ? (lane < 3) : (lane < nslots);
    const int ch = mine ? ((lane < r0n) ? r0c / GR_CW + lane : r1c / GR_CW + (lane - r0n)) : 0;
    const int tap = ch / cpr, q = ch - tap * cpr;
    // first stage of the slab -> (image, y, x)
    const int per_img = pr.i2c_nx * pr.i2c_ny;
    const int64_t st0 = r_begin / SR;
    int b = (int)(st0 / per_img);
    const int rem0 = (int)(st0 - (int64_t)b * per_img);
    int yb = rem0 / pr.i2c_nx, xb = rem0 - yb * pr.i2c_nx;
    int s = 0;
    uint32_t ph = 0, sb = smem_base;
    for (int kb = 0; kb < nk; ++kb) {
      const bool got = mbar_wait(smem_u32(&bar_empty[s]), ph ^ 1, abortp);
      if (!__all_sync(0xffffffffu, got)) { if (lane == 0) { abort_flag = 1; atomicExch(pr.status, 205); } break; }
      const uint32_t fb = smem_u32(&bar_full[s]);
      if (lane == 0) mbar_expect_tx(fb, tx_bytes);
      __syncwarp();
      if (mine && win) {
        asm volatile(
            "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
            ::"r"(sb + (uint32_t)(lane * cpr) * CHUNK), "l"(reinterpret_cast<uint64_t>(&g.map3a[pi])), "r"(0),
              "r"(xb * pr.i2c_bw), "r"(yb * pr.i2c_bh + lane), "r"(0), "r"(b), "r"(fb)
            : "memory");
      } else if (mine) {
        asm volatile(
            "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
            ::"r"(sb + (uint32_t)lane * CHUNK), "l"(reinterpret_cast<uint64_t>(&g.mapX[pi])), "r"(q * GR_CW),
              "r"(xb * pr.i2c_bw), "r"(yb * pr.i2c_bh + tap), "r"(b), "r"(fb)
            : "memory");
      }
      if (++xb == pr.i2c_nx) { xb = 0; if (++yb == pr.i2c_ny) { yb = 0; ++b; } }
      sb += stage_bytes;
      if (++s == nstages) { s = 0; ph ^= 1; sb = smem_base; }
    }
  } else if (warp == 0) {
    // ---- TMA producer: one 32-column box per chunk ----
    if (elect_one()) {
      tma_prefetch_desc(&g.mapX[pi]);
      if (pr.full) tma_prefetch_desc(&g.mapB[pi]);
      if (pr.use3d) { tma_prefetch_desc(&g.map3a[pi]); tma_prefetch_desc(&g.map3b[pi]); }
      int s = 0;
      uint32_t ph = 0, sb = smem_base;
      int y = (int)r_begin;
      for (int kb = 0; kb < nk; ++kb) {
        if (!mbar_wait(smem_u32(&bar_empty[s]), ph ^ 1, abortp)) { abort_flag = 1; atomicExch(pr.status, 201); break; }
        const uint32_t fb = smem_u32(&bar_full[s]);
        mbar_expect_tx(fb, tx_bytes);
        if (pr.use3d) {
          // one instruction per column range
          if (nslots == r0n) {
            tma_load_3d(sb, pr.stream ? &g.map3a[pi] : &g.map3b[pi], 0, y, r0c / GR_CW, fb);
          } else {
            tma_load_3d(sb, &g.map3a[pi], 0, y, r0c / GR_CW, fb);
            tma_load_3d(sb + r0n * CHUNK, &g.map3b[pi], 0, y, r1c / GR_CW, fb);
          }
        } else {
          uint32_t dst = sb;
          int col = r0c;
          for (int c = 0; c < r0n; ++c, dst += CHUNK, col += GR_CW) tma_load_2d(dst, &g.mapX[pi], col, y, fb);
          col = r1c;
          const CUtensorMap* m1 = pr.full ? &g.mapB[pi] : &g.mapX[pi];
          for (int c = r0n; c < nslots; ++c, dst += CHUNK, col += GR_CW) tma_load_2d(dst, m1, col, y, fb);
        }
        y += SR;
        sb += stage_bytes;
        if (++s == nstages) { s = 0; ph ^= 1; sb = smem_base; }
      }
    }
  } else if (warp == 1) {
    // ---- MMA issuer: descriptors prebuilt, one 64-bit add per operand per MMA ----
    if (elect_one()) {
      uint64_t ad0[4], bd0[4];
      uint32_t idesc[4], tm[4];
#pragma unroll
      for (int o = 0; o < 4; ++o) {
        const int oo = o < nops ? o : 0;
        ad0[o] = make_smem_desc(smem_base + ops[oo].a_slot * CHUNK, CHUNK, 512, LAYOUT);
        bd0[o] = make_smem_desc(smem_base + ops[oo].b_slot * CHUNK, CHUNK, 512, LAYOUT);
        idesc[o] = make_idesc(FMT, (uint32_t)ops[oo].n, 1, 1);
        tm[o] = tmem_base + (uint32_t)ops[oo].tmem_col;
      }
      int s = 0;
      uint32_t ph = 0, soff16 = 0;                  // stage offset in 16-byte units
      const uint32_t stage16 = stage_bytes >> 4;
      uint32_t accum = 0;
      for (int kb = 0; kb < nk; ++kb) {
        // without a pass of the fix-up warps over the stage the TMA's completion is the go-ahead
        if (!mbar_wait(smem_u32(direct ? &bar_full[s] : &bar_ready[s]), ph, abortp)) { abort_flag = 1; atomicExch(pr.status, 202); break; }
        tc_fence_after();
#pragma unroll 2
        for (int ks = 0; ks < KSTEPS; ++ks) {
          const uint64_t koff = (uint64_t)(soff16 + ks * 64);      // 1024 bytes per k-step
#pragma unroll
          for (int o = 0; o < 4; ++o) {
            if (o < nops) {
              if (BF) mma_bf16(tm[o], ad0[o] + koff, bd0[o] + koff, idesc[o], accum);
              else mma_tf32(tm[o], ad0[o] + koff, bd0[o] + koff, idesc[o], accum);
            }
          }
          accum = 1;
        }
        mma_commit(smem_u32(&bar_empty[s]));
        soff16 += stage16;
        if (++s == nstages) { s = 0; ph ^= 1; soff16 = 0; }
      }
      mma_commit(smem_u32(&bar_accum));
    }
  } else {
    // ---- fix-up + column sums, then epilogue (8 warps) ----
    const int w = warp - 2;                       // 0..7
    // fp32: a warp pass covers one 4-row x 128-byte atom: lane -> (row lane>>3, 16-byte unit lane&7);
    //       warp w owns rows 4w..4w+3 of every chunk of the stage.
    // bf16: a warp pass covers one 8-row x 64-byte atom: lane -> (row lane>>2, 16-byte unit lane&3);
    //       warp w owns rows 8(w&3).. of the chunks with parity w>>2.
    const int r_in = BF ? (lane >> 2) : (lane >> 3);
    const int u = BF ? (lane & 3) : (lane & 7);
    const int r = BF ? ((w & 3) * 8 + r_in) : (w * 4 + r_in);
    // byte offset of this lane's 16-byte unit inside a chunk (swizzled position)
    const uint32_t off = BF ? ((uint32_t)r * 64u + (((uint32_t)u ^ (uint32_t)((r >> 1) & 3)) << 4))
                            : ((uint32_t)r * 128u + ((((uint32_t)(u >> 1) ^ (uint32_t)(r & 3)) << 5) | ((uint32_t)(u & 1) << 4)));
    float acc[GR_MAX_SLOTS][4];
    float4 sh[BF ? 1 : GR_MAX_SLOTS];
#pragma unroll
    for (int j = 0; j < GR_MAX_SLOTS; ++j) {
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[j][e] = 0.f;
      if (!BF) {
        float c4[4] = {0.f, 0.f, 0.f, 0.f};
        if (pr.shift && j < nslots) {
          const int col = ((j < r0n) ? (r0c + j * GR_CW) : (r1c + (j - r0n) * GR_CW)) + u * 4;
#pragma unroll
          for (int e = 0; e < 4; ++e)
            if (col + e < M) c4[e] = pr.shift[col + e];
        }
        sh[BF ? 0 : j] = make_float4(c4[0], c4[1], c4[2], c4[3]);
      }
    }
    const bool fixup = pr.fixup != 0;
    const int cs_slots = s_cs_slots;
    bool ok = true;
    int s = 0;
    uint32_t ph = 0, sa = smem_base + off;
    int rem = slab_rows;                           // rows of the slab not yet consumed
    for (int kb = 0; kb < (direct ? 0 : nk); ++kb) {
      if (!mbar_wait(smem_u32(&bar_full[s]), ph, abortp)) { abort_flag = 1; atomicExch(pr.status, 203); ok = false; break; }
      // rows at or past the end of the tensor were zero-filled by the TMA and are left alone
      if (r < rem) {
        if (!BF && !fixup) {
          // read-only: the tensor core truncates fp32 operands to TF32, so the column sums are taken of the
          // truncated values; the covariance assembled from them is then exactly that of the data as multiplied
#pragma unroll
          for (int j = 0; j < GR_MAX_SLOTS; ++j) {
            if (j < cs_slots) {                       // column sums are owed for the first cs_slots chunks only
              const float4 x = lds128(sa + j * CHUNK);
              acc[j][0] += __uint_as_float(__float_as_uint(x.x) & 0xffffe000u);
              acc[j][1] += __uint_as_float(__float_as_uint(x.y) & 0xffffe000u);
              acc[j][2] += __uint_as_float(__float_as_uint(x.z) & 0xffffe000u);
              acc[j][3] += __uint_as_float(__float_as_uint(x.w) & 0xffffe000u);
            }
          }
        } else if (!BF) {
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            float4 v[GR_MAX_SLOTS / 2];
#pragma unroll
            for (int jj = 0; jj < GR_MAX_SLOTS / 2; ++jj) {
              const int j = h * (GR_MAX_SLOTS / 2) + jj;
              if (j < nslots) v[jj] = lds128(sa + j * CHUNK);
            }
#pragma unroll
            for (int jj = 0; jj < GR_MAX_SLOTS / 2; ++jj) {
              const int j = h * (GR_MAX_SLOTS / 2) + jj;
              if (j < nslots) {
                float4 x = v[jj];
                const float4 c = sh[BF ? 0 : j];
                x.x = tf32_rna(x.x - c.x); x.y = tf32_rna(x.y - c.y); x.z = tf32_rna(x.z - c.z); x.w = tf32_rna(x.w - c.w);
                sts128(sa + j * CHUNK, x);
                acc[j][0] += x.x; acc[j][1] += x.y; acc[j][2] += x.z; acc[j][3] += x.w;
              }
            }
          }
        } else {
#pragma unroll
          for (int jj = 0; jj < GR_MAX_SLOTS / 2; ++jj) {
            const int slot = 2 * jj + (w >> 2);
            if (slot < cs_slots) {
              const float4 qf = lds128(sa + slot * CHUNK);
              const uint32_t qx = __float_as_uint(qf.x), qy = __float_as_uint(qf.y), qz = __float_as_uint(qf.z), qw = __float_as_uint(qf.w);
              acc[2 * jj][0] += __uint_as_float(qx << 16); acc[2 * jj][1] += __uint_as_float(qx & 0xffff0000u);
              acc[2 * jj][2] += __uint_as_float(qy << 16); acc[2 * jj][3] += __uint_as_float(qy & 0xffff0000u);
              acc[2 * jj + 1][0] += __uint_as_float(qz << 16); acc[2 * jj + 1][1] += __uint_as_float(qz & 0xffff0000u);
              acc[2 * jj + 1][2] += __uint_as_float(qw << 16); acc[2 * jj + 1][3] += __uint_as_float(qw & 0xffff0000u);
            }
          }
        }
      }
      if (!BF && fixup) fence_proxy_async_smem();   // generic-proxy writes -> visible to the tensor core's reads
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bar_ready[s]));
      rem -= SR;
      sa += stage_bytes;
      if (++s == nstages) { s = 0; ph ^= 1; sa = smem_base + off; }
    }
    // column sums: reduce over the row positions inside the warp, then over the 8 warps through shared memory
#pragma unroll
    for (int j = 0; j < GR_MAX_SLOTS; ++j) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float x = acc[j][e];
        if (BF) x += __shfl_xor_sync(0xffffffffu, x, 4);
        x += __shfl_xor_sync(0xffffffffu, x, 8);
        x += __shfl_xor_sync(0xffffffffu, x, 16);
        acc[j][e] = x;
      }
      if (r_in == 0) {
        int ci;                                     // column inside the stage (chunk-major)
        if (!BF) ci = j * GR_CW + u * 4;
        else ci = (2 * (j >> 1) + (w >> 2)) * GR_CW + u * 8 + (j & 1) * 4;
#pragma unroll
        for (int e = 0; e < 4; ++e) s_csred[w][ci + e] = acc[j][e];
      }
    }
    asm volatile("bar.sync 1, 256;" ::: "memory");
    {
      float* cs_out = pr.colsum_part + (int64_t)split * M;
      const int cs_cols = cs_slots * GR_CW;
      for (int i = threadIdx.x - 64; i < cs_cols; i += GR_FIX_WARPS * 32) {
        float t = 0.f;
        if (!BF) {
#pragma unroll
          for (int ww = 0; ww < GR_FIX_WARPS; ++ww) t += s_csred[ww][i];
        } else {
          const int par = (i / GR_CW) & 1;        // the chunk's parity selects which four warps hold it
#pragma unroll
          for (int ww = 0; ww < 4; ++ww) t += s_csred[4 * par + ww][i];
        }
        int col = r0c + i;
        if (pr.im2col) col = (col < M16) ? i2c_col(col, pr.i2c_cpr, pr.i2c_c3) : -1;
        if (col >= 0 && col < M) cs_out[col] = t;
      }
    }
    // ---- epilogue: accumulators -> partial Gram; two warps per TMEM lane quarter ----
    const bool have = nk > 0;
    bool good = ok;
    if (good && have && !mbar_wait(smem_u32(&bar_accum), 0, abortp)) {
      good = false;
      abort_flag = 1;
      atomicExch(pr.status, 204);
    }
    float* P = pr.gram_part + (int64_t)split * M * M;
    const int q = warp & 3, half = w >> 2;
    if (pr.im2col) {
      if (good) {
        tc_fence_after();
        for (int o = 0; o < nops; ++o) {
          int row = ops[o].row0 + q * 32 + lane;
          {
            // rows and columns as staged -> rows and columns of the patch matrix; padding columns are dropped
            // (a group of four staged columns is all real or all padding, and real ones stay adjacent)
            const int rr_ = (row < M16) ? i2c_col(row, pr.i2c_cpr, pr.i2c_c3) : -1;
            for (int c0 = 16 * half; c0 < ops[o].n_out; c0 += 32) {
              uint32_t rv[16];
              if (have) {
                tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(ops[o].tmem_col + c0), rv);
                tmem_ld_wait();
              } else {
#pragma unroll
                for (int j = 0; j < 16; ++j) rv[j] = 0u;
              }
              if (rr_ >= 0) {
#pragma unroll
                for (int j = 0; j < 16; j += 4) {
                  const int cs = ops[o].col0 + c0 + j;
                  const int cc = (cs < M16) ? i2c_col(cs, pr.i2c_cpr, pr.i2c_c3) : -1;
                  if (cc >= 0)
                    *reinterpret_cast<float4*>(P + (int64_t)rr_ * M + cc) =
                        make_float4(__uint_as_float(rv[j]), __uint_as_float(rv[j + 1]), __uint_as_float(rv[j + 2]),
                                    __uint_as_float(rv[j + 3]));
                }
              }
            }
            if (ops[o].cs_off >= 0 && half == 0) {
              uint32_t rv[16];
              if (have) {
                tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(ops[o].tmem_col + ops[o].cs_off), rv);
                tmem_ld_wait();
              } else {
                rv[0] = 0u;
              }
              if (rr_ >= 0) pr.colsum_part[(int64_t)split * M + rr_] = __uint_as_float(rv[0]);
            }
          }
        }
      }
    } else {
      // A TMEM lane is a row of the tile, so stores straight from the registers put the 32 lanes of a warp on 32
      // different rows of the output: half-filled sectors, and an SM stores one sector per clock (7 us for a
      // 128 x 256 tile).  The tile goes through shared memory instead (the stages are free: every MMA has completed)
      // and leaves as whole rows, 512 bytes per warp instruction (2 us).  The mirror image of a symmetric product
      // leaves from the registers: there the lanes' rows are consecutive entries of one output row.
      // The verdict of the waits is made common to the eight warps first: the barriers below are taken by all of
      // them or by none.
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (*abortp == 0) {
        tc_fence_after();
        constexpr int TS = 308;      // row pitch in floats: >= 288 + 16 columns, and 8 consecutive rows on distinct banks
        float* tile = reinterpret_cast<float*>(smem_raw) + ((smem_base - smem_u32(smem_raw)) >> 2);
        for (int o = 0; o < nops; ++o) {
          const int n_out = ops[o].n_out, row0 = ops[o].row0, col0 = ops[o].col0;
          {
            const int row = row0 + q * 32 + lane;
            float* trow = tile + (q * 32 + lane) * TS;
            for (int c0 = 16 * half; c0 < n_out; c0 += 32) {
              uint32_t rr[16];
              if (have) {
                tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(ops[o].tmem_col + c0), rr);
                tmem_ld_wait();
              } else {
#pragma unroll
                for (int j = 0; j < 16; ++j) rr[j] = 0u;
              }
#pragma unroll
              for (int j = 0; j < 16; j += 4)
                *reinterpret_cast<float4*>(trow + c0 + j) =
                    make_float4(__uint_as_float(rr[j]), __uint_as_float(rr[j + 1]), __uint_as_float(rr[j + 2]),
                                __uint_as_float(rr[j + 3]));
              if (pr.full == 2 && row < M) {
                // symmetric product: entry (row, c) with c > row also goes to (c, row)
                const int col = col0 + c0;
#pragma unroll
                for (int j = 0; j < 16; ++j)
                  if (col + j > row && col + j < M) P[(int64_t)(col + j) * M + row] = __uint_as_float(rr[j]);
              }
            }
            if (ops[o].cs_off >= 0 && half == 0) {
              // ones mode: every one of the 16 extra columns holds the column sum of this lane's feature
              uint32_t rr[16];
              if (have) {
                tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(ops[o].tmem_col + ops[o].cs_off), rr);
                tmem_ld_wait();
              } else {
                rr[0] = 0u;
              }
              if (row < M) pr.colsum_part[(int64_t)split * M + row] = __uint_as_float(rr[0]);
            }
          }
          asm volatile("bar.sync 1, 256;" ::: "memory");
          // rows of the tile, four at a time per warp: every load of a batch precedes its stores
          const int n4 = n_out >> 2;
          const bool sym = pr.full == 2;
          for (int t0 = w; t0 < 128; t0 += 4 * GR_FIX_WARPS) {
            if (row0 + t0 >= M) break;
            float4 v[4][3];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float* trow = tile + (t0 + i * GR_FIX_WARPS) * TS;
#pragma unroll
              for (int k = 0; k < 3; ++k) {
                const int c4 = lane + 32 * k;
                if (c4 < n4) v[i][k] = *reinterpret_cast<const float4*>(trow + 4 * c4);
              }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int row = row0 + t0 + i * GR_FIX_WARPS;
              float* prow = P + (int64_t)row * M;
#pragma unroll
              for (int k = 0; k < 3; ++k) {
                const int c4 = lane + 32 * k;
                const int col = col0 + 4 * c4;
                // symmetric product: the entries on and above the diagonal only
                if (c4 >= n4 || row >= M || col >= M || (sym && col + 3 < row)) continue;
                if (col + 3 < M && (!sym || col >= row)) {
                  *reinterpret_cast<float4*>(prow + col) = v[i][k];
                } else {
                  const float ve[4] = {v[i][k].x, v[i][k].y, v[i][k].z, v[i][k].w};
#pragma unroll
                  for (int e = 0; e < 4; ++e)
                    if (col + e < M && (!sym || col + e >= row)) prow[col + e] = ve[e];
                }
              }
            }
          }
          if (o + 1 < nops) asm volatile("bar.sync 1, 256;" ::: "memory");
        }
      }
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

bool tmap_encode_2d(CUtensorMap* m, bool bf16, const void* base, uint64_t inner, uint64_t outer, uint64_t ld,
                    uint32_t box_inner, uint32_t box_outer) {
  // bf16 chunks of 32 columns: 64-byte swizzle; of 64 columns: 128-byte swizzle
  const CUtensorMapSwizzle sw = !bf16 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B
                                      : (box_inner == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B);
  return encode_2d(m, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, bf16 ? 2 : 4, base,
                   inner, outer, ld, box_inner, box_outer, sw);
}
bool tmap_encode_chunked_3d(CUtensorMap* m, bool bf16, const void* base, uint64_t cols, uint64_t rows, uint64_t ld,
                            uint32_t box_rows, uint32_t box_chunks, uint32_t chunk_cols) {
  const CUtensorMapSwizzle sw = !bf16 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B
                                      : (chunk_cols == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B);
  return encode_chunked_3d(m, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                           bf16 ? 2 : 4, base, cols, rows, ld, box_rows, box_chunks, sw, chunk_cols);
}

bool umma_gram_supported(const fw_layer_desc& d, const void* X, int64_t ldx) {
  const int es = (d.x_dtype == FW_BF16) ? 2 : 4;
  if (!umma_available()) return false;
  if (((uintptr_t)X & 15) != 0 || ((ldx * es) & 15) != 0) return false;
  if (d.M < 16 || (d.M % (16 / es)) != 0) return false;
  return true;
}

// Whether this layer's Gram pass is fed unshifted (no pilot mean, no in-place centring): bf16 X always; fp32 X
// when the block is long: the shared-memory read-modify-write of the centred values is what limits the kernel,
// and with >= 4096 rows the TF32 truncation noise averages out well below the engine's tolerance.
bool umma_gram_unshifted(const fw_layer_desc& d, int64_t rows) {
  if (d.x_dtype == FW_BF16) return true;
  return rows >= 4096;
}

static bool gram_smem_attr(int smem) {
  static SmemAttrCache attr_f32, attr_bf16;
  if (ensure_dyn_smem(gram_umma_kernel<false>, smem, attr_f32) != cudaSuccess ||
      ensure_dyn_smem(gram_umma_kernel<true>, smem, attr_bf16) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  return true;
}

// Pixels per stage of an implicit-im2col layer: bw along x (a power of two covering W, at most 32; slots past W
// read as zeros), bh rows of the image (a power of two that divides H), bw * bh = the stage's rows >= 32.
bool umma_gram_im2col_geometry(int H, int W, int C, int want_rows, int* bw_out, int* bh_out) {
  if (H < 1 || W < 1 || C < 4 || (C % 4) != 0) return false;
  int bw = 8;
  while (bw < 32 && bw < W) bw *= 2;
  int bh = std::max(1, want_rows / bw);
  while (bh > 1 && (H % bh) != 0) bh /= 2;
  if (bw * bh < GR_SR || bh > 256) return false;
  *bw_out = bw; *bh_out = bh;
  return true;
}
static inline int i2c_cpr(int C) { return (3 * C + GR_CW - 1) / GR_CW; }
static inline int gram_item_mpad(const UmmaGramItem& it) {
  return it.im2col ? 3 * i2c_cpr(it.i2c_C) * GR_CW : (it.M + 15) / 16 * 16;
}

fw_status umma_gram_launch(UmmaGramItem* items, int n, cudaStream_t s) {
  const int smem = GR_SMEM_BUDGET + 1024;
  if (!gram_smem_attr(smem)) return FW_ERR_CUDA;
  // one element type per launch: order the items so that each group of a launch is homogeneous
  std::stable_sort(items, items + n, [](const UmmaGramItem& a, const UmmaGramItem& b) { return a.x_bf16 < b.x_bf16; });
  // cost model: bytes a tile streams through shared memory; aim at two waves of equal items
  std::vector<double> tile_cost(n);
  std::vector<int> ntiles(n), stream(n);
  double total = 0;
  for (int i = 0; i < n; ++i) {
    const UmmaGramItem& it = items[i];
    const int es = it.x_bf16 ? 2 : 4;
    const int Mpad = gram_item_mpad(it);
    const int nb = (Mpad + 127) / 128;
    int tri = 0;
    for (int b = 0; b < nb; ++b) tri += Mpad - 128 * b;
    stream[i] = tri <= 512;
    double loaded_cols;
    if (stream[i]) { ntiles[i] = 1; loaded_cols = Mpad; }
    else {
      ntiles[i] = gram_tiled_count(Mpad);
      loaded_cols = 0;
      for (int b = 0; b < nb; ++b)
        for (int c = 128 * b, t = 0; c < Mpad; c += 256, ++t) loaded_cols += (t ? 128 : 0) + std::min(256, Mpad - c);
      loaded_cols /= ntiles[i];
    }
    // bytes through shared memory, weighted by how fast each mode moves them (measured): tiles of the TILED
    // mode re-read X out of L2, blocks whose column sums are taken by the fix-up warps are bound by those reads
    double w = 1.0;
    if (!stream[i]) w = 0.8;
    else if (Mpad + 16 > 256 || tri + 16 * nb > 512 || it.shift) w = 1.2;
    tile_cost[i] = (double)it.rows * loaded_cols * es * w;
    total += tile_cost[i] * ntiles[i];
  }
  // rows per stage: larger stages for the layers whose stages nothing but the TMA and the MMA warp touches
  auto stage_rows = [&](int i) -> int {
    const int Mpad = gram_item_mpad(items[i]);
    int sr = GR_SR;
    if (stream[i] && items[i].shift == nullptr && gram_ones_fits(Mpad))
      sr = gram_ones_stage_rows(Mpad, items[i].x_bf16 != 0, items[i].rows, items[i].im2col ? 60 * 1024 : 48 * 1024);
    if (items[i].im2col) {
      int bw = 0, bh = 0;
      if (!umma_gram_im2col_geometry(items[i].i2c_H, items[i].i2c_W, items[i].i2c_C, sr, &bw, &bh)) return 0;
      sr = bw * bh;
    }
    return sr;
  };
  // implicit im2col: the kernel walks stage slots (bw x bh pixels, slots past W are zeros), not rows
  auto virtual_rows = [&](int i) -> int64_t {
    if (!items[i].im2col) return items[i].rows;
    int bw = 0, bh = 0;
    const int sr = stage_rows(i);
    if (sr == 0) return 0;
    umma_gram_im2col_geometry(items[i].i2c_H, items[i].i2c_W, items[i].i2c_C, sr, &bw, &bh);
    return (int64_t)items[i].i2c_B * (items[i].i2c_H / bh) * ((items[i].i2c_W + bw - 1) / bw) * sr;
  };
  for (int i = 0; i < n; ++i)
    if (items[i].im2col && (stage_rows(i) == 0 || items[i].x_bf16 || items[i].shift)) return FW_ERR_UNSUPPORTED;
  // Split counts: about two waves of CTAs (one CTA per SM) of near-equal cost.  Rounding to nearest keeps every
  // item within ~1.4x of the target; rounding down would leave layers whose share is just under 2 with one
  // item of twice the cost, which then is the tail of the launch.
  const double target = total / (148.0 * tuning().gram_waves_pct / 100.0);
  std::vector<int64_t> split_of(n);
  std::vector<double> cta_cost(n);
  for (int i = 0; i < n; ++i) {
    const int64_t nsr = (virtual_rows(i) + stage_rows(i) - 1) / stage_rows(i);
    const int64_t cap = std::min<int64_t>(items[i].split_cap, nsr);
    int64_t sp = (int64_t)(tile_cost[i] / target + 0.5);
    split_of[i] = std::max<int64_t>(1, std::min(sp, cap));
    cta_cost[i] = tile_cost[i] / (double)split_of[i];
  }
  // longest items first: the hardware hands CTAs to SMs in index order as they free up, so the short items
  // fill the end of the launch
  {
    std::vector<int> order(n);
    for (int i = 0; i < n; ++i) order[i] = i;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
      if (items[a].x_bf16 != items[b].x_bf16) return items[a].x_bf16 < items[b].x_bf16;
      return cta_cost[a] > cta_cost[b];
    });
    std::vector<UmmaGramItem> it2(n);
    std::vector<int64_t> sp2(n);
    std::vector<int> nt2(n), st2(n);
    for (int i = 0; i < n; ++i) { it2[i] = items[order[i]]; sp2[i] = split_of[order[i]]; nt2[i] = ntiles[order[i]]; st2[i] = stream[order[i]]; }
    for (int i = 0; i < n; ++i) { items[i] = it2[i]; split_of[i] = sp2[i]; ntiles[i] = nt2[i]; stream[i] = st2[i]; }
  }
  for (int base = 0; base < n;) {
    GramGroup g;
    memset(&g, 0, sizeof(g));
    int cnt = 0;
    while (base + cnt < n && cnt < kMaxUmmaGroup && items[base + cnt].x_bf16 == items[base].x_bf16) ++cnt;
    const bool group_bf16 = items[base].x_bf16 != 0;
    int total_ctas = 0;
    for (int i = 0; i < cnt; ++i) {
      UmmaGramItem& it = items[base + i];
      GramProblem& p = g.p[i];
      const int sr = stage_rows(base + i);
      const int64_t vrows = virtual_rows(base + i);
      const int64_t nsr = (vrows + sr - 1) / sr;
      int64_t sp = split_of[base + i];
      const int64_t per = (nsr + sp - 1) / sp;
      sp = (nsr + per - 1) / per;
      p.shift = it.shift; p.gram_part = it.gram_part; p.colsum_part = it.colsum_part;
      p.fixup = it.shift != nullptr;
      p.rows = vrows; p.M = it.M; p.bf16 = it.x_bf16; p.stream = stream[base + i];
      p.splits = (int)sp; p.ntiles = ntiles[base + i]; p.first_cta = total_ctas;
      p.rows_per_split = (int)(per * sr);
      p.sr = sr;
      p.status = it.status;
      it.splits_out = (int)sp;
      total_ctas += p.splits * p.ntiles;
      if (it.im2col) {
        int bw = 0, bh = 0;
        umma_gram_im2col_geometry(it.i2c_H, it.i2c_W, it.i2c_C, sr, &bw, &bh);
        p.im2col = 1; p.i2c_bw = bw; p.i2c_bh = bh;
        p.i2c_nx = (it.i2c_W + bw - 1) / bw; p.i2c_ny = it.i2c_H / bh;
        p.i2c_cpr = i2c_cpr(it.i2c_C); p.i2c_c3 = 3 * it.i2c_C; p.Mp = gram_item_mpad(it);
        p.box_a = GR_ABL;
        // STREAM mode loads every chunk of the stage: one instruction per patch row through the 5-D view
        p.use3d = p.stream && encode_im2col_5d(&g.map3a[i], it.X, it.i2c_B, it.i2c_H, it.i2c_W, it.i2c_C, (uint32_t)bw,
                                               (uint32_t)bh, (uint32_t)p.i2c_cpr);
        if (!encode_im2col_4d(&g.mapX[i], it.X, it.i2c_B, it.i2c_H, it.i2c_W, it.i2c_C, (uint32_t)bw, (uint32_t)bh)) {
          fprintf(stderr, "[fw] tensor-map encoding failed (Gram, implicit im2col)\n");
          return FW_ERR_CUDA;
        }
        continue;
      }
      const int es = it.x_bf16 ? 2 : 4;
      if (!encode_2d(&g.mapX[i], it.x_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, es,
                     it.X, (uint64_t)it.M, (uint64_t)it.rows, (uint64_t)it.ldx, GR_CW, (uint32_t)sr,
                     it.x_bf16 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B)) {
        fprintf(stderr, "[fw] tensor-map encoding failed (Gram)\n");
        return FW_ERR_CUDA;
      }
      {
        const CUtensorMapDataType dt = it.x_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
        const CUtensorMapSwizzle sw = it.x_bf16 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B;
        p.box_a = p.stream ? it.M / GR_CW : GR_ABL;
        p.use3d = (it.M % GR_CW) == 0 &&
                  encode_chunked_3d(&g.map3a[i], dt, es, it.X, (uint64_t)it.M, (uint64_t)it.rows, (uint64_t)it.ldx,
                                    (uint32_t)sr, (uint32_t)p.box_a, sw) &&
                  encode_chunked_3d(&g.map3b[i], dt, es, it.X, (uint64_t)it.M, (uint64_t)it.rows, (uint64_t)it.ldx,
                                    (uint32_t)sr, 2 * GR_ABL, sw);
      }
    }
    g.n = cnt;
    ProfScope ps(FW_PROF_GRAM, s);
    if (group_bf16) gram_umma_kernel<true><<<total_ctas, GR_THREADS, smem, s>>>(g);
    else gram_umma_kernel<false><<<total_ctas, GR_THREADS, smem, s>>>(g);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
      fprintf(stderr, "[fw] gram_umma_kernel launch: %s\n", cudaGetErrorString(e));
      return FW_ERR_CUDA;
    }
    base += cnt;
  }
  return FW_OK;
}

bool tmap_encode_kmajor_f32(CUtensorMap* m, const void* base, uint64_t inner, uint64_t outer, uint64_t ld,
                            uint32_t box_inner, uint32_t box_outer) {
  return encode_2d(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, base, inner, outer, ld, box_inner, box_outer,
                   CU_TENSOR_MAP_SWIZZLE_128B);
}

// A wait that nothing ever satisfies, with a short poll limit: the bounded wait of every pipeline in this engine
// gives up, the kernel records the code in the layer's status word and returns normally.
namespace {
__global__ void wait_probe_kernel(int32_t* status, uint32_t polls) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    mbar_fence_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    if (!mbar_wait(smem_u32(&bar), 0, &abort_flag, polls)) atomicExch(status, 901);
  }
}
}  // namespace

cudaError_t launch_wait_probe(int32_t* status, uint32_t polls, cudaStream_t s) {
  ProfScope ps(FW_PROF_MISC, s);
  wait_probe_kernel<<<1, 32, 0, s>>>(status, polls);
  return cudaGetLastError();
}

// D = A^T B for square fp32 matrices (TF32 inputs rounded to nearest, fp32 accumulation):
// the re-sync products Phi_x T^T and T (Phi_x T^T) when T is kept transposed.
fw_status umma_atb_launch(const UmmaAtbItem* items, int n, cudaStream_t s) {
  const int smem = GR_SMEM_BUDGET + 1024;
  if (!gram_smem_attr(smem)) return FW_ERR_CUDA;
  for (int base = 0; base < n; base += kMaxUmmaGroup) {
    GramGroup g;
    memset(&g, 0, sizeof(g));
    const int cnt = (n - base) < kMaxUmmaGroup ? (n - base) : kMaxUmmaGroup;
    int total_ctas = 0;
    for (int i = 0; i < cnt; ++i) {
      const UmmaAtbItem& it = items[base + i];
      GramProblem& p = g.p[i];
      const int M16 = (it.M + 15) / 16 * 16;
      p.shift = nullptr; p.gram_part = it.C; p.colsum_part = nullptr;
      p.rows = it.M; p.M = it.M; p.bf16 = 0; p.stream = 0; p.full = it.sym ? 2 : 1; p.fixup = 1;
      p.splits = 1; p.ntiles = ((M16 + 127) / 128) * ((M16 + 255) / 256); p.first_cta = total_ctas;
      p.rows_per_split = (it.M + GR_SR - 1) / GR_SR * GR_SR;
      p.sr = GR_SR;
      p.status = it.status;
      total_ctas += p.ntiles;
      if (!encode_2d(&g.mapX[i], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, it.A, (uint64_t)it.M, (uint64_t)it.M,
                     (uint64_t)it.M, GR_CW, GR_SR, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B) ||
          !encode_2d(&g.mapB[i], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, it.B, (uint64_t)it.M, (uint64_t)it.M,
                     (uint64_t)it.M, GR_CW, GR_SR, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B)) {
        fprintf(stderr, "[fw] tensor-map encoding failed (A^T B)\n");
        return FW_ERR_CUDA;
      }
      p.box_a = GR_ABL;
      p.use3d = (it.M % GR_CW) == 0 &&
                encode_chunked_3d(&g.map3a[i], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, it.A, (uint64_t)it.M, (uint64_t)it.M,
                                  (uint64_t)it.M, GR_SR, GR_ABL, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B) &&
                encode_chunked_3d(&g.map3b[i], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, it.B, (uint64_t)it.M, (uint64_t)it.M,
                                  (uint64_t)it.M, GR_SR, 2 * GR_ABL, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B);
    }
    g.n = cnt;
    ProfScope ps(FW_PROF_RESYNC, s);
    gram_umma_kernel<false><<<total_ctas, GR_THREADS, smem, s>>>(g);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
      fprintf(stderr, "[fw] gram_umma_kernel (A^T B) launch: %s\n", cudaGetErrorString(e));
      return FW_ERR_CUDA;
    }
  }
  return FW_OK;
}

}  // namespace fw
