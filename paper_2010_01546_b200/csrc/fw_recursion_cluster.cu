// On-chip recursion for small layers (Sec. 4): one thread-block cluster of 8
// CTAs per layer keeps the whitened covariance Phi_y resident in distributed
// shared memory for all K steps of a call.  CTA `rank` owns a slab of rows of
// Phi_y; every pass of a step is a slab-times-vector product out of shared
// memory.  The passes are chained as a dataflow: each CTA pushes its slice of a
// result straight into all peers' copies of the vector with asynchronous
// remote stores that count bytes on the receiver's mbarrier, and every CTA
// waits only on its own barrier.  No cluster-wide barrier is taken inside a
// step, and the partial sums a pass needs next (squared norm, v.u) travel with
// the slices.  Nothing but T^T and Q (touched once per step) goes to global
// memory.
//
// Buffer reuse is safe without further synchronisation: a peer can send
// exchange e + 1 only after it received this CTA's slice of exchange e, so
// while this CTA works between its sends e and e + 1 only the target of
// exchange e + 1 can change under it, and that buffer is never read in that
// window (vectors alternate, partial-sum slots and barriers are double-buffered).
//
// The arithmetic is that of the multi-launch path in fw_recursion.cu (same
// passes, symmetric evaluation of the rank updates); dot products are accumulated
// in fp32 here (rows are at most ~600 long and split over 64 partial sums).
#include <cooperative_groups.h>

#include "fw_internal.h"
#include "fw_sm100.cuh"

namespace cg = cooperative_groups;

namespace fw {
namespace {

using sm100::smem_u32;

constexpr int CL = 8;              // CTAs per cluster = per layer
#ifndef FW_CLUSTER_THREADS
#define FW_CLUSTER_THREADS 512
#endif
constexpr int CT = FW_CLUSTER_THREADS;   // threads per CTA
constexpr int CW = CT / 32;        // warps per CTA
constexpr int NSLOT = CL * CW;     // one partial sum per warp of the cluster
constexpr int MAXR = 80;           // rows per CTA
constexpr int MAXRPW = (MAXR + CW - 1) / CW;   // rows per warp

__device__ __forceinline__ float warp_sum_f(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// shared-memory address of the same variable in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_cluster(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
// asynchronous 4-byte store into a peer's shared memory; the peer's mbarrier counts the bytes
__device__ __forceinline__ void st_async_f32(uint32_t raddr, float v, uint32_t rbar) {
  asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];"
               ::"r"(raddr), "r"(__float_as_uint(v)), "r"(rbar) : "memory");
}
__device__ __forceinline__ bool try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}\n"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait of the whole CTA for an exchange to land; the verdict is uniform over the CTA.
// The block barrier inside also publishes the slice this CTA stored into its own copy.
// Only the first warp polls (the others sleep at the block barrier and leave the issue slots to the warps
// still at work); its acquire together with the barrier makes the received data visible to every thread.
__device__ __forceinline__ bool exchange_wait(uint32_t bar, uint32_t parity) {
  bool ok = true;
#ifdef FW_X_POLLALL
  if (true) {
#else
  if (threadIdx.x < 32) {
#endif
    ok = false;
    for (uint32_t i = 0; i < sm100::kSpinLimit; ++i)
      if (try_wait_cluster(bar, parity)) { ok = true; break; }
  }
  return __syncthreads_and(ok) != 0;
}

struct Slab {
  float* phi;     // my rows of Phi_y in shared memory, leading dimension Mp
  int M, Mp, R;   // matrix size, padded row length, rows per CTA
  int row0, nrows;
  int rank;
  uint32_t rdelta;  // per lane: cluster address of peer (lane & 7)'s shared memory minus this CTA's own
};

// 1/sqrt(n2) refined by one Newton step, 0 when n2 is not a positive finite number
__device__ __forceinline__ float inv_norm(float n2) {
  float inv = (n2 > 0.f && isfinite(n2)) ? rsqrtf(n2) : 0.f;
  return inv > 0.f ? inv * (1.5f - 0.5f * n2 * inv * inv) : 0.f;
}

// this lane's share of the NSLOT partial sums of an exchange (sum it over the warp)
__device__ __forceinline__ float slot_part(const float* slots) {
  static_assert(NSLOT % 64 == 0, "float2 per lane and round");
  const float2* s2 = reinterpret_cast<const float2*>(slots);
  const int lane = threadIdx.x & 31;
  float t = 0.f;
#pragma unroll
  for (int i = 0; i < NSLOT / 64; ++i) {
    const float2 a = s2[lane + 32 * i];
    t += a.x + a.y;
  }
  return t;
}
// sum of the partial sums: every warp of every CTA adds them in the same order
__device__ __forceinline__ float slot_sum(const float* slots) { return warp_sum_f(slot_part(slots)); }

__device__ __forceinline__ void send_one(float* tgt, float v, int peer, const Slab& s, uint32_t bar) {
  if (peer == s.rank) *tgt = v;
  else st_async_f32(smem_u32(tgt) + s.rdelta, v, bar + s.rdelta);
}

// y[row0 + r] = scale * dot(A[r,:], x) for my rows; A rows live in shared or global memory.
// With `nrm_in` the scale is 1 / sqrt(sum of the partial sums at nrm_in), i.e. x is normalised; that sum is
// reduced in the same shuffle rounds as the row sums, so it adds no latency of its own.
// Each result is sent into `dst` (a shared-memory vector of length Mp) of every CTA of the cluster.
// When `slots` is given, the warp also sends its partial sum of y*y (wgt == nullptr) or y*wgt[row]
// into slot rank*CW + warp of every CTA.  A warp owns rows warp, warp + CW, ... (NQ of them) and works
// on all of them at once.  The code is specialised on NQ and loops over the columns at run time: the
// passes of small layers are bound by instruction issue and latency, so no instruction is spent on rows or
// columns a layer does not have, and up to three rows plus the partial sum leave in one store instruction
// (lane 8q + p carries item q to peer p).  POWER: the pass of a power iteration, where nrm_in and slots are
// known to be given and wgt not (no tests on the dependent chain).
template <bool SELF, int NQ, bool POWER = false>
__device__ __forceinline__ void gemv_send_rows(const float* A, int lda, const float* x, const Slab& s,
                                               const float* nrm_in, float scale, float* dst, const float* wgt,
                                               float* slots, uint32_t bar) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int M4 = s.Mp >> 2;
  const float4* x4 = reinterpret_cast<const float4*>(x);
  const float4* A4 = reinterpret_cast<const float4*>(A + (size_t)warp * lda);
  const int ld4 = (CW * lda) >> 2;                 // float4 stride between two rows of this warp
  float acc[NQ > 0 ? NQ : 1][2];
#pragma unroll
  for (int q = 0; q < NQ; ++q) acc[q][0] = acc[q][1] = 0.f;
  if (NQ > 0) {
#pragma unroll 2
    for (int c = lane; c < M4; c += 32) {
      float4 a[NQ > 0 ? NQ : 1];
#pragma unroll
      for (int q = 0; q < NQ; ++q) a[q] = A4[q * ld4 + c];
      float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
      if (!SELF) b = x4[c];
#pragma unroll
      for (int q = 0; q < NQ; ++q) {
        const float4 bb = SELF ? a[q] : b;
        acc[q][0] = fmaf(a[q].x, bb.x, acc[q][0]); acc[q][1] = fmaf(a[q].y, bb.y, acc[q][1]);
        acc[q][0] = fmaf(a[q].z, bb.z, acc[q][0]); acc[q][1] = fmaf(a[q].w, bb.w, acc[q][1]);
      }
    }
  }
  float y[NQ > 0 ? NQ : 1];
  y[0] = 0.f;
#pragma unroll
  for (int q = 0; q < NQ; ++q) y[q] = acc[q][0] + acc[q][1];
  float nin = (POWER || nrm_in) ? slot_part(nrm_in) : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
    for (int q = 0; q < NQ; ++q) y[q] += __shfl_xor_sync(0xffffffffu, y[q], o);
    nin += __shfl_xor_sync(0xffffffffu, nin, o);
  }
  if (POWER || nrm_in) scale = inv_norm(nin);
  float part = 0.f;
#pragma unroll
  for (int q = 0; q < NQ; ++q) {
    y[q] *= scale;
    part = fmaf(y[q], (!POWER && wgt) ? wgt[s.row0 + warp + CW * q] : y[q], part);
  }
  // items 0..NQ-1 are the rows, item NQ the partial sum; a store instruction carries four items
  const int peer = lane & 7, grp = lane >> 3;
#pragma unroll
  for (int i0 = 0; i0 < NQ + 1; i0 += 4) {
    const int item = i0 + grp;
    float* tgt = nullptr;
    float v = part;
    if (item < NQ) {
      tgt = dst + s.row0 + warp + CW * item;
#pragma unroll
      for (int q = 0; q < NQ; ++q)
        if (q >= i0 && q < i0 + 4 && q == item) v = y[q];
    } else if (item == NQ && (POWER || slots)) {
      tgt = slots + s.rank * CW + warp;
    }
    if (tgt) send_one(tgt, v, peer, s, bar);
  }
}

template <bool SELF>
__device__ __noinline__ void slab_gemv_send(const float* A, int lda, const float* x, const Slab s,
                                               const float* nrm_in, float scale, float* dst, const float* wgt,
                                               float* slots, uint32_t bar) {
  static_assert(MAXRPW <= 10, "specialisations below");
  const int warp = threadIdx.x >> 5;
  const int nq = s.nrows > warp ? (s.nrows - warp + CW - 1) / CW : 0;   // rows of this warp
#define FW_CASE(n) case n: if (n <= MAXRPW) gemv_send_rows<SELF, (n <= MAXRPW ? n : 0)>(A, lda, x, s, nrm_in, scale, dst, wgt, slots, bar); break;
  switch (nq) {
    FW_CASE(0) FW_CASE(1) FW_CASE(2) FW_CASE(3) FW_CASE(4) FW_CASE(5)
    FW_CASE(6) FW_CASE(7) FW_CASE(8) FW_CASE(9) FW_CASE(10)
    default: break;
  }
#undef FW_CASE
}

// The P power iterations of a step (S4) as one specialised loop: the pass, its exchange and the next pass
// follow each other without a call or a dispatch in between, and everything that does not change from pass to
// pass stays in registers.  Returns false when a wait gave up.
template <int NQ>
__device__ __forceinline__ bool power_loop_rows(const Slab& s, float* buf0, float* slots, uint32_t bar0, uint32_t& e,
                                                int P, int& cur, uint32_t tx_bytes) {
  for (int p = 0; p < P; ++p) {
    const uint32_t bar = bar0 + ((e & 1) << 3);
    if (threadIdx.x == 0) sm100::mbar_expect_tx(bar, tx_bytes);     // armed ahead of the pass, off the chain
    gemv_send_rows<false, NQ, true>(s.phi, s.Mp, buf0 + cur * s.Mp, s, slots + ((e - 1) & 1) * NSLOT, 0.f,
                              buf0 + (cur ^ 1) * s.Mp, nullptr, slots + (e & 1) * NSLOT, bar);
    if (!exchange_wait(bar, (e >> 1) & 1)) return false;
    ++e;
    cur ^= 1;
  }
  return true;
}

__device__ __noinline__ bool power_loop(const Slab s, float* buf0, float* slots, uint32_t bar0, uint32_t& e, int P,
                                        int& cur, uint32_t tx_bytes) {
  const int warp = threadIdx.x >> 5;
  const int nq = s.nrows > warp ? (s.nrows - warp + CW - 1) / CW : 0;
#define FW_CASE(n) case n: return power_loop_rows<(n <= MAXRPW ? n : 0)>(s, buf0, slots, bar0, e, P, cur, tx_bytes);
  switch (nq) {
    FW_CASE(0) FW_CASE(1) FW_CASE(2) FW_CASE(3) FW_CASE(4) FW_CASE(5)
    FW_CASE(6) FW_CASE(7) FW_CASE(8) FW_CASE(9) FW_CASE(10)
    default: return true;
  }
#undef FW_CASE
}

// dynamic shared memory:
// [phi slab R x Mp][xi2][cvec][wvec][bufA][bufB][vvec][uvec][tvec][slots 2 x NSLOT]
extern __shared__ __align__(16) float csm[];

__global__ void __cluster_dims__(CL, 1, 1) __launch_bounds__(CT, 1)
recursion_cluster_kernel(const __grid_constant__ GroupDev g, const __grid_constant__ PtrTable traces, int K, int P) {
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int layer = blockIdx.x / CL;
  const LayerDev* L = g.layer[layer];
  const int M = L->M;
  const int Mp = (M + 3) & ~3;
  const int R = (M + CL - 1) / CL;
  Slab s;
  s.M = M; s.Mp = Mp; s.R = R; s.rank = rank;
  s.row0 = rank * R;
  s.nrows = max(0, min(R, M - s.row0));
  s.phi = csm;
  float* xi2 = csm + (size_t)R * Mp;
  float* cvec = xi2 + Mp;
  float* wvec = cvec + Mp;
  float* buf0 = wvec + Mp;           // two alternating power-iteration vectors, Mp apart
  float* vvec = wvec + 3 * Mp;
  float* uvec = vvec + Mp;
  float* tvec = uvec + Mp;
  float* slots = tvec + Mp;          // 2 x NSLOT
  __shared__ __align__(8) uint64_t xbar[2];
  __shared__ float sredf[32 * 4];
  __shared__ int sredi[CW + 1];

  // ---- load my rows of Phi_y; clear the padding and the vectors ----
  if ((M & 3) == 0) {
    // a warp per row, 16 bytes per lane, all loads of a row in flight together
    for (int r = warp; r < s.nrows; r += CW) {
      const float4* src = reinterpret_cast<const float4*>(L->Phiy + (size_t)(s.row0 + r) * M);
      float4* dstp = reinterpret_cast<float4*>(s.phi + (size_t)r * Mp);
#pragma unroll 5
      for (int c = lane; c < (M >> 2); c += 32) dstp[c] = src[c];
    }
  } else {
    for (int i = threadIdx.x; i < s.nrows * Mp; i += CT) {
      const int r = i / Mp, c = i - r * Mp;
      s.phi[i] = (c < M) ? L->Phiy[(size_t)(s.row0 + r) * M + c] : 0.f;
    }
  }
  for (int i = threadIdx.x; i < 8 * Mp + 2 * NSLOT; i += CT) xi2[i] = 0.f;
  if (threadIdx.x == 0) {
    sm100::mbar_init(smem_u32(&xbar[0]), 1);
    sm100::mbar_init(smem_u32(&xbar[1]), 1);
    sm100::mbar_fence_init();
  }
  const uint32_t bar0 = smem_u32(&xbar[0]);                       // the two barriers are 8 bytes apart
  // A peer's window of the cluster address space is this CTA's window shifted by a constant; the stores
  // below rely on it, so it is checked on two addresses far apart before anything is sent.
  s.rdelta = map_cluster(bar0, (uint32_t)(lane & 7)) - bar0;
  const bool linear = (map_cluster(smem_u32(slots), (uint32_t)(lane & 7)) - smem_u32(slots)) == s.rdelta;
  bool failed = __syncthreads_or(!linear) != 0;
  cluster.sync();   // every barrier is initialised before the first remote store can arrive

  const uint32_t vec_bytes = (uint32_t)(M - s.nrows) * 4u;        // one vector's slices from the 7 peers
  const uint32_t slot_bytes = (uint32_t)(CL - 1) * CW * 4u;
  uint32_t e = 0;                                                 // exchanges completed so far
  // arm the barrier of the current exchange for `nvec` vectors (+ slots), wait for it, advance
#define FW_BAR (bar0 + ((e & 1) << 3))
#define FW_SLOTS_OUT (slots + (e & 1) * NSLOT)
#define FW_SLOTS_IN (slots + ((e - 1) & 1) * NSLOT)
#define FW_EXCHANGE(nvec)                                                                 \
  {                                                                                       \
    if (threadIdx.x == 0) sm100::mbar_expect_tx(FW_BAR, (nvec) * vec_bytes + slot_bytes); \
    if (!exchange_wait(FW_BAR, (e >> 1) & 1)) { failed = true; goto done; }               \
    ++e;                                                                                  \
  }
  if (failed) goto done;

  {
  float* tr = const_cast<float*>(reinterpret_cast<const float*>(traces.p[layer]));
  const float c_rel = L->c_rel, c_abs = L->c_abs, delta = L->delta, eps = L->eps;
  const float lam_bar = L->scal[SC_LAMBDA_BAR];
  const bool maxcol = (L->init == FW_INIT_MAXCOL);
  bool any_nosub = false, any_nonfinite = false;

  for (int step = 0; step < K; ++step) {
    // S1: squared column norms (= row norms, Phi_y is exactly symmetric)             (Eq. 45)
    slab_gemv_send<true>(s.phi, Mp, nullptr, s, nullptr, 1.f, xi2, nullptr, FW_SLOTS_OUT, FW_BAR);
    FW_EXCHANGE(1u)
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
      if (lane == 0) { sredf[warp] = best; sredi[warp] = bi; }
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
    {
      // the owner's slab is current: its updates of the previous step precede its S1 sends, which this
      // CTA has received
      const int owner = mp / R;
      const float* rphi = cluster.map_shared_rank(s.phi, owner) + (size_t)(mp - owner * R) * Mp;
      for (int m = threadIdx.x; m < Mp; m += CT) wvec[m] = rphi[m];
    }
    __syncthreads();
    slab_gemv_send<false>(s.phi, Mp, wvec, s, nullptr, 1.f, cvec, nullptr, FW_SLOTS_OUT, FW_BAR);
    FW_EXCHANGE(1u)
    // S3: coherent set and aligned average                                          (Eqs. 48-49)
    int cnt = 0;
    if (maxcol) {
      for (int m = threadIdx.x; m < Mp; m += CT) wvec[m] = (m == mp) ? 1.f : 0.f;
      cnt = 1;
      __syncthreads();
    } else {
      const float xi_mp = sqrtf(xi2[mp]);
      for (int base = 0; base < Mp; base += CT) {
        const int m = base + threadIdx.x;
        bool in = false;
        if (m < Mp) {
          float wv = 0.f;
          if (m < M) {
            const float c = cvec[m];
            const float thr = fmaxf(c_rel * xi_mp * sqrtf(xi2[m]), c_abs);
            in = fabsf(c) >= thr;
            wv = in ? (1.f / c) : 0.f;
          }
          wvec[m] = wv;
        }
        cnt += __syncthreads_count(in);
      }
      if (rank == 0)
        for (int m = threadIdx.x; m < M; m += CT) L->wvec[m] = wvec[m];
    }
    const float inv_cnt = cnt > 0 ? 1.f / (float)cnt : 0.f;
    slab_gemv_send<false>(s.phi, Mp, wvec, s, nullptr, inv_cnt, buf0, nullptr, FW_SLOTS_OUT, FW_BAR);
    FW_EXCHANGE(1u)
    // S4: P power iterations u = Phi_y (prev / ||prev||); the squared norm of each result arrives with it
    // and is turned into the scale inside the next pass
    int cur = 0;
    if (!power_loop(s, buf0, slots, bar0, e, P, cur, vec_bytes + slot_bytes)) { failed = true; goto done; }
    // S5: v = prev/||prev|| (Eq. 50), u = Phi_y v, t = T^T v; lambda_e = v.u (Eq. 36) comes with u
    const float n2 = slot_sum(FW_SLOTS_IN);
    const float inv = inv_norm(n2);
    for (int m = threadIdx.x; m < Mp; m += CT) vvec[m] = (m < M) ? buf0[cur * Mp + m] * inv : 0.f;
    __syncthreads();
    slab_gemv_send<false>(s.phi, Mp, vvec, s, nullptr, 1.f, uvec, vvec, FW_SLOTS_OUT, FW_BAR);
    if ((M & 3) == 0) {
      slab_gemv_send<false>(L->Tt + (size_t)s.row0 * M, M, vvec, s, nullptr, 1.f, tvec, nullptr, nullptr, FW_BAR);
    } else {
      // unaligned rows in global memory: scalar loads
      for (int r = warp; r < s.nrows; r += CW) {
        const float* a = L->Tt + (size_t)(s.row0 + r) * M;
        float acc = 0.f;
        for (int c = lane; c < M; c += 32) acc = fmaf(a[c], vvec[c], acc);
        acc = warp_sum_f(acc);
        if (lane < CL) send_one(tvec + s.row0 + r, acc, lane, s, FW_BAR);
      }
    }
    FW_EXCHANGE(2u)
    const float lam_e = slot_sum(FW_SLOTS_IN);
    // S6: g_e, a_e (Eqs. 40-41), rank updates (Eqs. 42, 44)
    const bool ok = cnt > 0 && n2 > 0.f && isfinite(n2) && isfinite(lam_e);
    float g_e = 1.f, a = 0.f;
    if (ok) {
      g_e = delta * lam_bar / fmaxf(lam_e, eps);
      a = sqrtf(g_e) - 1.f;
    }
    any_nosub |= !ok;
    any_nonfinite |= !isfinite(n2) || !isfinite(lam_e);
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
        // a warp walks its rows, a lane its float4 columns: no index arithmetic beyond additions, the row's
        // scalars are loaded once, and the independent iterations keep several L2 loads in flight
        const int M4 = M >> 2;
        for (int r = warp; r < s.nrows; r += CW) {
          const int i = s.row0 + r;
          const float vi = vvec[i], ui = uvec[i], ti = tvec[i];
          const float ati = a * ti;
          float4* Q4 = reinterpret_cast<float4*>(L->Q + (size_t)i * M);
          float4* T4 = reinterpret_cast<float4*>(L->Tt + (size_t)i * M);
          float4* P4 = reinterpret_cast<float4*>(s.phi + (size_t)r * Mp);
#pragma unroll 5
          for (int c = lane; c < M4; c += 32) {
            const float4 vj = reinterpret_cast<const float4*>(vvec)[c];
            const float4 uj = reinterpret_cast<const float4*>(uvec)[c];
            const float4 tj = reinterpret_cast<const float4*>(tvec)[c];
            float4 q = Q4[c], tt = T4[c], p = P4[c];
#define FW_UPD(X)                                                                                          \
            q.X = __fadd_rn(q.X, __fmul_rn(aq, __fmul_rn(ti, tj.X)));                                      \
            tt.X = fmaf(ati, vj.X, tt.X);                                                                  \
            p.X = __fadd_rn(p.X, __fadd_rn(__fmul_rn(a, __fadd_rn(__fmul_rn(vi, uj.X), __fmul_rn(ui, vj.X))), \
                                           __fmul_rn(a2l, __fmul_rn(vi, vj.X))));
            FW_UPD(x) FW_UPD(y) FW_UPD(z) FW_UPD(w)
#undef FW_UPD
            Q4[c] = q; T4[c] = tt; P4[c] = p;
          }
        }
      } else {
        for (int e1 = threadIdx.x; e1 < s.nrows * Mp; e1 += CT) {
          const int r = e1 / Mp, j = e1 - r * Mp;
          if (j < M) {
            const int i = s.row0 + r;
            const float vi = vvec[i], ui = uvec[i], ti = tvec[i];
            const float vj = vvec[j], uj = uvec[j], tj = tvec[j];
            s.phi[e1] = __fadd_rn(s.phi[e1], __fadd_rn(__fmul_rn(a, __fadd_rn(__fmul_rn(vi, uj), __fmul_rn(ui, vj))),
                                                       __fmul_rn(a2l, __fmul_rn(vi, vj))));
            const size_t off = (size_t)i * M + j;
            L->Q[off] = __fadd_rn(L->Q[off], __fmul_rn(aq, __fmul_rn(ti, tj)));
            L->Tt[off] = fmaf(a * ti, vj, L->Tt[off]);
          }
        }
      }
    }
    // the slab updates are ordered before this CTA's next sends, whose receipt lets a peer read the slab
    asm volatile("fence.acq_rel.cluster;" ::: "memory");
    __syncthreads();
  }
  if (any_nosub && rank == 0 && threadIdx.x == 0) L->iscal[IS_STATUS_NOSUB] = 1;
  if (any_nonfinite && rank == 0 && threadIdx.x == 0) L->iscal[IS_STATUS_NONFINITE] = 1;
  }
done:
#undef FW_EXCHANGE
#undef FW_BAR
#undef FW_SLOTS_OUT
#undef FW_SLOTS_IN
  if (failed) {
    // a wait gave up: the state of this layer is not to be trusted; report and leave in step with the peers
    if (threadIdx.x == 0) L->iscal[IS_STATUS_TIMEOUT] = 1;
  } else {
    // ---- write my rows of Phi_y back ----
    if ((M & 3) == 0) {
      for (int r = warp; r < s.nrows; r += CW) {
        float4* dstp = reinterpret_cast<float4*>(L->Phiy + (size_t)(s.row0 + r) * M);
        const float4* src = reinterpret_cast<const float4*>(s.phi + (size_t)r * Mp);
        for (int c = lane; c < (M >> 2); c += 32) dstp[c] = src[c];
      }
    } else {
      for (int i = threadIdx.x; i < s.nrows * Mp; i += CT) {
        const int r = i / Mp, c = i - r * Mp;
        if (c < M) L->Phiy[(size_t)(s.row0 + r) * M + c] = s.phi[i];
      }
    }
  }
  cluster.sync();   // no CTA leaves while a peer may still read or write its shared memory
}

}  // namespace

size_t recursion_cluster_smem(int M) {
  const int Mp = (M + 3) & ~3;
  const int R = (M + CL - 1) / CL;
  return ((size_t)R * Mp + 8 * (size_t)Mp + 2 * NSLOT) * sizeof(float);
}

bool recursion_cluster_supported(int M) {
  const int Mp = (M + 3) & ~3;
  (void)Mp;
  return recursion_cluster_smem(M) <= 226 * 1024 && (M + CL - 1) / CL <= MAXR;
}

cudaError_t launch_recursion_cluster(const GroupDev& g, const PtrTable& traces, int K, int P, int max_M,
                                     cudaStream_t s) {
  static SmemAttrCache attr;
  const size_t smem = recursion_cluster_smem(max_M);
  {
    cudaError_t e = ensure_dyn_smem(recursion_cluster_kernel, smem, attr);
    if (e != cudaSuccess) return e;
  }
  ProfScope ps(FW_PROF_RECUR_CHIP, s);
  recursion_cluster_kernel<<<g.n * CL, CT, smem, s>>>(g, traces, K, P);
  return cudaGetLastError();
}

}  // namespace fw
