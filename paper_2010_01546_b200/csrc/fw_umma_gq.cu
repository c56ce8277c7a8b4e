// Tensor-core engine, G~ = G Qs on CTA pairs (tcgen05 cta_group::2): Eq. 29, with the optional fused SGD step
// W <- W - lr G~ (Eq. 27).  Also the general product out = G B for a row-major fp32 B (M x M): the explicit
// whitening products Y = X T^T (Eq. 11) and dX = dY T (Eq. 14) of the comparison path.
//
// Shape of the problem.  out[n][m] = sum_k G[n][k] B[k][m]; N (rows of G) runs from 16 to hundreds of thousands,
// M from 64 to 4608.  The tile is computed as D = B^T G^T: the MMA's 256 rows (128 per CTA of the pair) are 256
// values of m, its columns are up to 512 values of n in two accumulators of up to 256 (all 512 TMEM columns of
// both CTAs), the contraction runs over k.
//   A operand: B[k][m], m contiguous: MN-major chunks of 32 columns laid down by TMA (as in the Gram kernels);
//              each CTA stages its own 128 values of m: 16 KB per 32-row stage.
//   B operand: G[n][k], k contiguous: K-major, 128-byte swizzle, rows of 32 floats; each CTA stages its half of
//              each panel (up to 128 rows of G): 16 KB per accumulator per stage.
// A CTA therefore stages 48 KB for 128 x 512 x 32 multiply-adds -- the 48 bytes per tensor clock that the TMA
// sustains -- where one CTA per 128 x 256 tile staged twice that per multiply-add.
//
// K is split over `ksplit` items per tile when the tiles alone would not fill the machine; split s writes its
// partial tile to a scratch buffer and a second kernel adds the partials in split order (the same order in every
// run) and applies the epilogue.  Items are numbered problem-major, the problems in order of decreasing item
// length, and a CTA pair finds its (problem, tile, split) from its index.
//
// Roles per CTA: warp 0 TMA producer, warp 1 MMA issuer (even CTA only) and TMEM owner, warps 2..9 epilogue.
// Both CTAs' loads complete on the even CTA's "full" barrier; tcgen05.commit multicasts the "stage free" and
// "accumulator complete" arrivals to both CTAs.  Every wait is bounded; a time-out raises both CTAs' abort flags,
// is recorded in the owning layer's status word, and all threads still meet at the final cluster barrier before
// TMEM is freed.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <map>
#include <vector>

#include "fw_sm100.cuh"
#include "fw_umma.h"

namespace fw {

using namespace sm100;

namespace {

constexpr int QP_SR = 32;                 // k rows per stage
constexpr int QP_KSTEPS = QP_SR / 8;      // TF32 MMAs contract over 8
constexpr int QP_A_BYTES = 4 * QP_SR * 128;       // 4 chunks of 32 columns: 16 KB
constexpr int QP_B_BYTES = 128 * QP_SR * 4;       // 128 rows of G x 32 floats: 16 KB per accumulator
constexpr int QP_STAGE = QP_A_BYTES + 2 * QP_B_BYTES;   // 48 KB
constexpr int QP_STAGES = 4;
constexpr int QP_THREADS = 64 + 8 * 32;
constexpr int QP_SMEM = QP_STAGES * QP_STAGE;
constexpr int QP_MAX_PROBLEMS = 16;
constexpr int QP_MAX_ITEMS = 1 << 20;    // items of one launch (the grid is twice that)
constexpr int QP_MAX_KSPLIT = 8;

struct QpProblem {
  float* out;              // N x M (ld = M): result, or W for the SGD epilogue
  float* part;             // ksplit > 1: partial tiles, split s at part + s * N * M
  const float* colbias;    // optional, length M: subtracted from every row of the result (Eq. 11's T mu)
  int32_t* status;         // time-out word of the owning layer
  int32_t* nonfinite;      // non-finite word of the owning layer (may be null)
  int64_t N;               // rows of G
  int32_t M;
  int32_t ksplit, kb_per;  // splits, k blocks (of 32) per split
  int32_t ntiles_n;        // tiles along n (512 rows of G each)
  int32_t epi;             // EPI_STORE / EPI_SGD
  int32_t use3d;           // mapA is the chunked 3-D view (M a multiple of 32), else one-chunk 2-D boxes
  float lr;
  int32_t first_item;      // items are problem-major: problem, then tile, then split (no list: the kernel's
                           // parameter block is kept small, its size is paid on every launch)
};
struct QpGroup {
  CUtensorMap mapA[QP_MAX_PROBLEMS];    // right-hand matrix as MN-major A operand: chunked 3-D view with 4 chunks of
                                        // 32 columns x 32 rows per box, or a 2-D map with one chunk per box
  CUtensorMap mapB[QP_MAX_PROBLEMS];    // G, 32 floats x 128 rows, 128-byte swizzle (K-major B operand)
  QpProblem p[QP_MAX_PROBLEMS];
  int32_t n, nitems;
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(QP_THREADS, 1)
gq_pair_kernel(const __grid_constant__ QpGroup g) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[QP_STAGES], bar_empty[QP_STAGES], bar_accum;
  __shared__ uint32_t tmem_base_sh;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int item = (int)(blockIdx.x >> 1);
  int pi = 0;
#pragma unroll 1
  for (int i = 1; i < g.n; ++i)
    if (item >= g.p[i].first_item) pi = i;
  const QpProblem& pr = g.p[pi];
  const int local = item - pr.first_item;
  const int tile = local / pr.ksplit, split = local - tile * pr.ksplit;
  const int M = pr.M;
  const int I = tile / pr.ntiles_n, t = tile - I * pr.ntiles_n;
  const int64_t n_base = (int64_t)t * 512;
  int64_t nrem = pr.N - n_base;
  if (nrem > 512) nrem = 512;
  const int nall = ((int)nrem + 15) & ~15;          // columns of this tile, a multiple of 16
  const int n0 = nall < 256 ? nall : 256;
  const int n1 = nall - n0;
  const int m_cta = 256 * I + 128 * (int)rank;       // first value of m this CTA holds
  uint32_t ncols = 32;
  while ((int)ncols < nall) ncols <<= 1;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < QP_STAGES; ++s) { mbar_init(smem_u32(&bar_full[s]), 1); mbar_init(smem_u32(&bar_empty[s]), 1); }
    mbar_init(smem_u32(&bar_accum), 1);
    mbar_fence_init();
  }
  __syncthreads();
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(&tmem_base_sh), ncols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  cluster_arrive();
  cluster_wait();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_sh;
  const volatile int* abortp = &abort_flag;
  const uint32_t peer_abort = mapa_shared(smem_u32(&abort_flag), rank ^ 1u);
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
#define QP_ABORT(code)                      \
  do {                                      \
    abort_flag = 1;                         \
    st_cluster_u32(peer_abort, 1u);         \
    atomicExch(pr.status, (code));          \
  } while (0)

  // k blocks of this split
  const int nkb_all = (M + QP_SR - 1) / QP_SR;
  const int kb0 = min(nkb_all, split * pr.kb_per), kb1 = min(nkb_all, kb0 + pr.kb_per);
  const int nk = kb1 - kb0;
  // bytes both CTAs deliver per stage: A always, one or two B panels
  const uint32_t tx_cta = (uint32_t)QP_A_BYTES + (uint32_t)QP_B_BYTES * (n1 > 0 ? 2u : 1u);

  if (warp == 0) {
    // ---- TMA producer (both CTAs).  Lane 0..3: the A chunks (or lane 0 alone with the 3-D map), lanes 4, 5: the
    //      two B panels; all loads of a stage are issued together ----
    if (lane == 0) {
      tma_prefetch_desc(&g.mapA[pi]);
      tma_prefetch_desc(&g.mapB[pi]);
    }
    const bool issue_a = pr.use3d ? (lane == 0) : (lane < 4);
    const bool issue_b = (lane == 4) || (lane == 5 && n1 > 0);
    // rows of G this CTA stages for the panel: its half of the panel's n0 (n1) rows
    const int64_t brow = n_base + (lane == 4 ? (int64_t)rank * (n0 / 2) : 256 + (int64_t)rank * (n1 / 2));
    int s = 0;
    uint32_t ph = 0, sb = smem_base;
    for (int kb = 0; kb < nk; ++kb) {
      const bool got = mbar_wait(smem_u32(&bar_empty[s]), ph ^ 1, abortp);
      if (!__all_sync(0xffffffffu, got)) { if (lane == 0) QP_ABORT(401); break; }
      const uint32_t bar = mapa_shared(smem_u32(&bar_full[s]), 0u);       // counted on the even CTA's barrier
      if (lane == 0 && rank == 0) mbar_expect_tx(smem_u32(&bar_full[s]), 2u * tx_cta);
      const int k = (kb0 + kb) * QP_SR;
      if (issue_a) {
        if (pr.use3d) tma_load_3d_pair(sb, &g.mapA[pi], 0, k, m_cta / 32, bar);
        else tma_load_2d_pair(sb + (uint32_t)lane * (QP_SR * 128), &g.mapA[pi], m_cta + lane * 32, k, bar);
      }
      if (issue_b) tma_load_2d_pair(sb + QP_A_BYTES + (lane == 5 ? QP_B_BYTES : 0), &g.mapB[pi], k, (int)brow, bar);
      sb += QP_STAGE;
      if (++s == QP_STAGES) { s = 0; ph ^= 1; sb = smem_base; }
    }
  } else if (warp == 1) {
    // ---- MMA issuer: one thread of the even CTA drives the tensor cores of both SMs ----
    if (rank == 0 && elect_one()) {
      const uint64_t ad = make_smem_desc(smem_base, QP_SR * 128, 512, kSwizzle128B32);           // MN-major chunks
      const uint64_t bd0 = make_smem_desc(smem_base + QP_A_BYTES, 16, 1024, kSwizzle128B);        // K-major rows
      const uint64_t bd1 = make_smem_desc(smem_base + QP_A_BYTES + QP_B_BYTES, 16, 1024, kSwizzle128B);
      const uint32_t id0 = make_idesc(2, (uint32_t)n0, 1, 0, 256u);
      const uint32_t id1 = make_idesc(2, (uint32_t)(n1 > 0 ? n1 : 16), 1, 0, 256u);
      int s = 0;
      uint32_t ph = 0, soff16 = 0;
      uint32_t accum = 0;
      for (int kb = 0; kb < nk; ++kb) {
        if (!mbar_wait(smem_u32(&bar_full[s]), ph, abortp)) { QP_ABORT(402); break; }
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < QP_KSTEPS; ++ks) {
          const uint64_t aoff = (uint64_t)(soff16 + ks * 64);     // 8 rows of 128 bytes
          const uint64_t boff = (uint64_t)(soff16 + ks * 2);      // 8 floats inside the swizzled 128-byte rows
          mma_tf32_pair(tmem_base, ad + aoff, bd0 + boff, id0, accum);
          if (n1 > 0) mma_tf32_pair(tmem_base + 256u, ad + aoff, bd1 + boff, id1, accum);
          accum = 1;
        }
        mma_commit_pair(smem_u32(&bar_empty[s]), (uint16_t)3);
        soff16 += QP_STAGE >> 4;
        if (++s == QP_STAGES) { s = 0; ph ^= 1; soff16 = 0; }
      }
      mma_commit_pair(smem_u32(&bar_accum), (uint16_t)3);
    }
  } else {
    // ---- epilogue: this CTA's 128 values of m (TMEM lanes) x the tile's columns n ----
    const int w = warp - 2;
    const int q = warp & 3, half = w >> 2;
    const int m = m_cta + q * 32 + lane;
    const bool have = nk > 0;
    bool bad = false;
    if (!have || mbar_wait(smem_u32(&bar_accum), 0, abortp)) {
      tc_fence_after();
      const bool direct = pr.ksplit == 1;
      float* dst = direct ? pr.out : pr.part + (int64_t)split * pr.N * M;
      const float cb = (direct && pr.colbias && m < M) ? pr.colbias[m] : 0.f;
      // 32 columns per trip: both TMEM loads, then (SGD) all 32 loads of W, are in flight before anything is
      // used -- a read-modify-write one element at a time is a chain of global-memory round trips
      const bool sgd = direct && pr.epi == EPI_SGD;
      for (int c0 = 32 * half; c0 < nall; c0 += 64) {
        uint32_t ra[16], rb[16];
        const bool second = c0 + 16 < nall;
        if (have) {
          tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, ra);
          if (second) tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(c0 + 16), rb);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) { ra[j] = 0u; rb[j] = 0u; }
        }
        if (m < M) {
          float* d0 = dst + (n_base + c0) * M + m;
          const int64_t nleft = pr.N - (n_base + c0);          // rows of the result from this column on
          const int ncol = second ? 32 : 16;
          float w[32];
          if (sgd) {
#pragma unroll
            for (int j = 0; j < 32; ++j) w[j] = (j < ncol && j < nleft) ? d0[(int64_t)j * M] : 0.f;
          }
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            if (j < ncol && j < nleft) {
              const float v = __uint_as_float(j < 16 ? ra[j & 15] : rb[j & 15]) - cb;
              if (direct) bad |= !isfinite(v);
              d0[(int64_t)j * M] = sgd ? fmaf(-pr.lr, v, w[j]) : v;
            }
          }
        }
      }
    } else {
      QP_ABORT(403);
    }
    if (bad && pr.nonfinite) *pr.nonfinite = 1;
  }
#undef QP_ABORT
  tc_fence_before();
  cluster_arrive();
  cluster_wait();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, ncols);
  }
}

// out (+)= sum over the splits, in split order, of the partial tiles; flat grid over the float4s of all problems
struct QrProblem {
  float* out; const float* part; const float* colbias; int32_t* nonfinite;
  int64_t elems4;          // N * M / 4
  int64_t first4;          // first float4 of this problem in the flat index space
  int32_t M4, ksplit, epi; float lr;
};
struct QrGroup { QrProblem p[QP_MAX_PROBLEMS]; int32_t n; int32_t pad; int64_t total4; };

__global__ void __launch_bounds__(256) gq_reduce_kernel(const __grid_constant__ QrGroup g) {
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < g.total4; e += (int64_t)gridDim.x * blockDim.x) {
    int pi = 0;
#pragma unroll 1
    for (int i = 1; i < g.n; ++i)
      if (e >= g.p[i].first4) pi = i;
    const QrProblem& pr = g.p[pi];
    const int64_t l = e - pr.first4;
    const float4* src = reinterpret_cast<const float4*>(pr.part) + l;
    float4 a = src[0];
    for (int s = 1; s < pr.ksplit; ++s) {
      const float4 b = src[(int64_t)s * pr.elems4];
      a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
    }
    if (pr.colbias) {
      const float4 c = reinterpret_cast<const float4*>(pr.colbias)[l % pr.M4];
      a.x -= c.x; a.y -= c.y; a.z -= c.z; a.w -= c.w;
    }
    if (pr.nonfinite && !(isfinite(a.x) && isfinite(a.y) && isfinite(a.z) && isfinite(a.w))) *pr.nonfinite = 1;
    float4* d = reinterpret_cast<float4*>(pr.out) + l;
    if (pr.epi == EPI_SGD) {
      float4 w = *d;
      w.x = fmaf(-pr.lr, a.x, w.x); w.y = fmaf(-pr.lr, a.y, w.y); w.z = fmaf(-pr.lr, a.z, w.z); w.w = fmaf(-pr.lr, a.w, w.w);
      *d = w;
    } else {
      *d = a;
    }
  }
}

}  // namespace

bool umma_gq_pair_supported(int M) { return umma_available() && (M % 4) == 0 && M >= 16; }

fw_status umma_gq_pair_launch(const UmmaGqItem* items_in, int n, int epi, float lr, int prof_class, cudaStream_t s) {
  if (n <= 0) return FW_OK;
  static SmemAttrCache attr;
  const int smem = QP_SMEM + 1024;
  if (ensure_dyn_smem(gq_pair_kernel, smem, attr) != cudaSuccess) { cudaGetLastError(); return FW_ERR_CUDA; }
  for (int base = 0; base < n;) {
    std::vector<QpGroup> gbuf(1);
    QpGroup& g = gbuf[0];
    memset(&g, 0, sizeof(g));
    QrGroup gr;
    memset(&gr, 0, sizeof(gr));
    // problems of this launch: as many as fit the problem table and the item list (ksplit = 1 counts)
    int cnt = 0;
    size_t tiles_total = 0;
    while (base + cnt < n && cnt < QP_MAX_PROBLEMS) {
      const UmmaGqItem& itx = items_in[base + cnt];
      const size_t tiles = (size_t)((itx.M + 255) / 256) * (size_t)((itx.N + 511) / 512);
      if (cnt > 0 && (tiles_total + tiles) * QP_MAX_KSPLIT > (size_t)QP_MAX_ITEMS) break;
      if (tiles * QP_MAX_KSPLIT > (size_t)QP_MAX_ITEMS) return FW_ERR_SHAPE;
      tiles_total += tiles;
      ++cnt;
    }
    // K split per problem: the choice whose longest-first list schedule over the resident pairs ends earliest,
    // counting what the reduction of the partial tiles costs.  Estimates in microseconds: a stage of 32 k rows
    // takes about 0.55 us (48 KB staged against 1024 tensor clocks), two thirds of that for tiles of one panel;
    // an item costs about 8 us besides (set-up, pipeline fill, epilogue); the reduction streams at about 4 TB/s.
    std::vector<int> ks_best(cnt, 1);
    // the search costs the host a fraction of a millisecond: its result is kept per list of shapes
    static std::map<std::vector<int64_t>, std::vector<int>> memo;
    std::vector<int64_t> key;
    for (int i = 0; i < cnt; ++i) {
      const UmmaGqItem& itx = items_in[base + i];
      key.push_back(itx.M); key.push_back(itx.N); key.push_back(itx.part ? itx.part_floats : 0);
    }
    bool can_split = false;
    for (int i = 0; i < cnt; ++i) can_split |= items_in[base + i].part != nullptr;
    auto hit = memo.find(key);
    if (!can_split) {
      // no scratch for partial tiles anywhere: nothing to choose
    } else if (hit != memo.end()) {
      ks_best = hit->second;
    } else {
      double best = 1e300;
      std::vector<int> ks_try(cnt);
      std::vector<double> costs;
      for (int step = 0; step < 40; ++step) {
        const double tau = 4.0 * std::pow(1.15, step);           // stages per item, 4 .. 900
        costs.clear();
        double extra = 0;
        for (int i = 0; i < cnt; ++i) {
          const UmmaGqItem& itx = items_in[base + i];
          const int nkb = (itx.M + QP_SR - 1) / QP_SR;
          const int64_t tiles = (int64_t)((itx.M + 255) / 256) * ((itx.N + 511) / 512);
          int ks = (int)((double)nkb / tau + 0.5);
          ks = std::max(1, std::min(ks, std::min(QP_MAX_KSPLIT, std::max(1, nkb / 4))));
          if (ks > 1 && (itx.part == nullptr || (double)ks * (double)itx.N * itx.M > (double)itx.part_floats))
            ks = itx.part ? (int)std::max<double>(1.0, std::min<double>(ks, (double)itx.part_floats / ((double)itx.N * itx.M))) : 1;
          const int per = (nkb + ks - 1) / ks;
          ks = (nkb + per - 1) / per;
          ks_try[i] = ks;
          const double st_us = 0.55 * (itx.N > 256 ? 1.0 : 2.0 / 3.0);
          for (int64_t t = 0; t < tiles; ++t)
            for (int k = 0; k < ks; ++k) costs.push_back(8.0 + st_us * std::min(per, nkb - k * per));
          if (ks > 1) extra += 3.0 + (double)(ks + 1) * (double)itx.N * itx.M * 4.0 / 4e6;
        }
        std::sort(costs.begin(), costs.end(), [](double a, double b) { return a > b; });
        std::vector<double> slot(74, 0.0);
        for (double c : costs) *std::min_element(slot.begin(), slot.end()) += c;
        const double span = *std::max_element(slot.begin(), slot.end()) + extra;
        if (span < best) { best = span; ks_best = ks_try; }
      }
      if (memo.size() > 256) memo.clear();
      memo[key] = ks_best;
    }
    // problems in order of decreasing item length: items start in index order, so the long ones start first
    std::vector<int> order(cnt);
    for (int i = 0; i < cnt; ++i) order[i] = i;
    auto item_len = [&](int i) {
      const UmmaGqItem& itx = items_in[base + i];
      const int nkb = (itx.M + QP_SR - 1) / QP_SR;
      return (double)((nkb + ks_best[i] - 1) / ks_best[i]) * (itx.N > 256 ? 1.0 : 2.0 / 3.0);
    };
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return item_len(a) > item_len(b); });
    int64_t nitems = 0;
    for (int oi = 0; oi < cnt; ++oi) {
      const int i = order[oi];
      const UmmaGqItem& itx = items_in[base + i];
      QpProblem& p = g.p[oi];
      const int nkb = (itx.M + QP_SR - 1) / QP_SR;
      const int tiles_m = (itx.M + 255) / 256;
      const int64_t tiles_n = (itx.N + 511) / 512;
      int ks = ks_best[i];
      const int per = (nkb + ks - 1) / ks;
      ks = (nkb + per - 1) / per;
      p.out = itx.out; p.part = itx.part; p.colbias = itx.colbias; p.status = itx.status; p.nonfinite = itx.nonfinite;
      p.N = itx.N; p.M = itx.M; p.ksplit = ks; p.kb_per = per; p.ntiles_n = (int)tiles_n; p.epi = epi; p.lr = lr;
      p.first_item = (int)nitems;
      nitems += (int64_t)tiles_m * tiles_n * ks;
      p.use3d = (itx.M % 32) == 0 &&
                tmap_encode_chunked_3d(&g.mapA[oi], false, itx.Qs, (uint64_t)itx.M, (uint64_t)itx.M, (uint64_t)itx.M, QP_SR, 4, 32);
      if ((!p.use3d && !tmap_encode_2d(&g.mapA[oi], false, itx.Qs, (uint64_t)itx.M, (uint64_t)itx.M, (uint64_t)itx.M, 32, QP_SR)) ||
          !tmap_encode_kmajor_f32(&g.mapB[oi], itx.G, (uint64_t)itx.M, (uint64_t)itx.N, (uint64_t)itx.M, 32, 128)) {
        fprintf(stderr, "[fw] tensor-map encoding failed (G Qs, CTA pairs)\n");
        return FW_ERR_CUDA;
      }
      if (ks > 1) {
        QrProblem& q = gr.p[gr.n++];
        q.out = itx.out; q.part = itx.part; q.colbias = itx.colbias; q.nonfinite = itx.nonfinite;
        q.elems4 = (int64_t)itx.N * itx.M / 4; q.first4 = gr.total4; q.M4 = itx.M / 4; q.ksplit = ks; q.epi = epi; q.lr = lr;
        gr.total4 += q.elems4;
      }
    }
    if (nitems < 1 || nitems > (int64_t)QP_MAX_ITEMS) return FW_ERR_SHAPE;
    g.n = cnt; g.nitems = (int)nitems;
    {
      ProfScope ps(prof_class, s);
      gq_pair_kernel<<<2 * g.nitems, QP_THREADS, smem, s>>>(g);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
      fprintf(stderr, "[fw] gq_pair_kernel launch: %s\n", cudaGetErrorString(e));
      return FW_ERR_CUDA;
    }
    if (gr.n > 0) {
      int64_t blocks = (gr.total4 + 255) / 256;
      if (blocks > 148 * 8) blocks = 148 * 8;
      ProfScope ps(prof_class, s);
      gq_reduce_kernel<<<(int)blocks, 256, 0, s>>>(gr);
      e = cudaGetLastError();
      if (e != cudaSuccess) {
        fprintf(stderr, "[fw] gq_reduce_kernel launch: %s\n", cudaGetErrorString(e));
        return FW_ERR_CUDA;
      }
    }
    base += cnt;
  }
  return FW_OK;
}

}  // namespace fw
