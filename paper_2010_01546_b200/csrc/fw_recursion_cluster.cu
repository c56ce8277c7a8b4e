// On-chip recursion for small layers (Sec. 4): a layer's whitened covariance
// Phi_y AND its transform T^T stay resident in distributed shared memory for
// all K steps of a call.  The launch uses thread-block clusters of 16 CTAs; a
// layer takes n = 1 ... 16 consecutive CTAs of one cluster (at least as many
// as its slabs need; more while the clusters of one wave allow and the layer
// is the launch's slowest), so a cluster carries one large layer or several
// small ones and every SM does a similar amount of work per pass.  CTA `sub`
// of a layer owns a slab of rows of both matrices; every pass of a step is a
// slab-times-vector product out of shared memory.  The passes are chained as a
// dataflow: each CTA pushes its slice of a result straight into all peers'
// copies of the vector with asynchronous remote stores that count bytes on the
// receiver's mbarrier, and every CTA waits only on its own barrier.  No
// cluster-wide barrier is taken inside a step, and the partial sums a pass
// needs next (squared norm, v.u) travel with the slices.  Global memory is
// touched three times per call: the slabs come in, the slabs go out, and Q
// takes the rank-one terms of the steps (Eq. 44) a few steps at a time -- the
// recursion itself never reads Q.
//
// Buffer reuse is safe without further synchronisation: a peer can send
// exchange e + 1 only after it received this CTA's slice of exchange e, so
// while this CTA works between its sends e and e + 1 only the target of
// exchange e + 1 can change under it, and that buffer is never read in that
// window (vectors alternate, partial-sum slots and barriers are double-buffered).
//
// The arithmetic is that of the multi-launch path in fw_recursion.cu (same
// passes, symmetric evaluation of the rank updates); dot products are accumulated
// in fp32 here (rows are at most ~600 long and split over two accumulators).
#include <cooperative_groups.h>
#include <cstring>

#include "fw_internal.h"
#include "fw_sm100.cuh"

namespace cg = cooperative_groups;

namespace fw {
namespace {

using sm100::smem_u32;

constexpr int CL = 16;             // CTAs per cluster of the launch
constexpr int CT = 512;            // threads per CTA
constexpr int CW = CT / 32;        // warps per CTA
constexpr int MAXGPW = 2;          // groups of four rows per warp, at most (rows per CTA <= 128); three were
                                   // measured: twelve rows per warp cost 1.8 us per pass (13 values through five
                                   // shuffle rounds) against 1.1 us for eight
constexpr int kMaxIt = 5;          // float4 columns per lane, at most (rows of at most 640 entries)
constexpr int KQ = 4;              // steps whose rank-one terms of Q are applied together
constexpr size_t kSmemLimit = 226 * 1024;   // plus the static variables below: within the 227 KB of a CTA

struct ClusterArgs {
  GroupDev g;
  PtrTable traces;
  int32_t first_cta[FW_MAX_GROUP];   // first CTA of each layer (a layer never straddles a cluster)
  int32_t ncta[FW_MAX_GROUP];        // CTAs of each layer: 1 ... 16
  int32_t K, P;
};

// shared-memory address of the same variable in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_cluster(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
// asynchronous 16-byte store into a peer's shared memory; the peer's mbarrier counts the bytes.  One message
// carries four results: the receiver's barrier takes a few clocks per message, so the count of messages, not
// their size, is what an exchange costs.
__device__ __forceinline__ void st_async_v4(uint32_t raddr, float4 v, uint32_t rbar) {
  asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
               ::"r"(raddr), "r"(__float_as_uint(v.x)), "r"(__float_as_uint(v.y)), "r"(__float_as_uint(v.z)),
                 "r"(__float_as_uint(v.w)), "r"(rbar) : "memory");
}
__device__ __forceinline__ void cp_async16(uint32_t saddr, const float* g) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(saddr), "l"(g) : "memory");
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
  if (threadIdx.x < 32) {
    ok = false;
    for (uint32_t i = 0; i < sm100::kSpinLimit; ++i)
      if (try_wait_cluster(bar, parity)) { ok = true; break; }
  }
  return __syncthreads_and(ok) != 0;
}

struct Slab {
  float* phi;     // my rows of Phi_y in shared memory, leading dimension Mp
  float* tt;      // my rows of T^T, same shape
  int M, Mp;      // matrix size, padded row length
  int R;          // rows per CTA, a multiple of four (rows past the matrix are zero rows)
  int row0, nrows;  // my first row; how many of my rows are rows of the matrix
  int n;          // CTAs of this layer
  int sub;        // my index among them
  uint32_t rdelta;  // lane p < n: cluster address of peer p's shared memory minus this CTA's own
};

// 1/sqrt(n2) refined by one Newton step, 0 when n2 is not a positive finite number
__device__ __forceinline__ float inv_norm(float n2) {
  float inv = (n2 > 0.f && isfinite(n2)) ? rsqrtf(n2) : 0.f;
  return inv > 0.f ? inv * (1.5f - 0.5f * n2 * inv * inv) : 0.f;
}

// x . y over the first Mp entries, by one warp; every warp of every CTA of a layer adds in the same order, so all
// of them hold the same bits
__device__ __forceinline__ float warp_dot(const float* x, const float* y, int Mp) {
  const int lane = threadIdx.x & 31;
  const float4* x4 = reinterpret_cast<const float4*>(x);
  const float4* y4 = reinterpret_cast<const float4*>(y);
  float a0 = 0.f, a1 = 0.f;
  for (int c = lane; c < (Mp >> 2); c += 32) {
    const float4 a = x4[c], b = y4[c];
    a0 = fmaf(a.x, b.x, a0); a1 = fmaf(a.y, b.y, a1);
    a0 = fmaf(a.z, b.z, a0); a1 = fmaf(a.w, b.w, a1);
  }
  float t = a0 + a1;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
  return t;
}

// y[row0 + r] = scale * dot(A[r,:], x) for my rows; A rows live in shared memory.  POWER: the pass of a power
// iteration, where the scale is 1 / ||x||: the squared norm is summed from the values of x the pass loads anyway
// and reduced in the same shuffle rounds as the row sums, so normalising adds no latency of its own.
// Each result is sent into `dst` (a shared-memory vector) of every CTA of the layer.  A warp owns groups of four
// consecutive rows (groups warp, warp + CW, ...: NG of them) and works on all of them at once; lane p < n sends
// each group's four results to peer p as one 16-byte message.  The code is specialised on NG and loops over the
// columns at run time: the passes of small layers are bound by instruction issue and latency, so no instruction is
// spent on rows or columns a layer does not have.
template <bool SELF, int NG, bool POWER = false>
__device__ __forceinline__ void gemv_send_rows(const float* A, int lda, const float* x, const Slab& s, float scale,
                                               float* dst, uint32_t bar) {
  constexpr int NQ = 4 * NG;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (NG == 0) return;
  const int M4 = s.Mp >> 2;
  const int ld4 = lda >> 2;
  const float4* x4 = reinterpret_cast<const float4*>(x);
  const float4* A4 = reinterpret_cast<const float4*>(A) + (size_t)(4 * warp) * ld4;
  float acc[NQ > 0 ? NQ : 1][2];
#pragma unroll
  for (int q = 0; q < NQ; ++q) acc[q][0] = acc[q][1] = 0.f;
  float n0 = 0.f, n1 = 0.f;
#pragma unroll 2
  for (int c = lane; c < M4; c += 32) {
    float4 a[NQ > 0 ? NQ : 1];
#pragma unroll
    for (int q = 0; q < NQ; ++q) a[q] = A4[((q >> 2) * 4 * CW + (q & 3)) * ld4 + c];
    float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
    if (!SELF) b = x4[c];
    if (POWER) {
      n0 = fmaf(b.x, b.x, n0); n1 = fmaf(b.y, b.y, n1);
      n0 = fmaf(b.z, b.z, n0); n1 = fmaf(b.w, b.w, n1);
    }
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
      const float4 bb = SELF ? a[q] : b;
      acc[q][0] = fmaf(a[q].x, bb.x, acc[q][0]); acc[q][1] = fmaf(a[q].y, bb.y, acc[q][1]);
      acc[q][0] = fmaf(a[q].z, bb.z, acc[q][0]); acc[q][1] = fmaf(a[q].w, bb.w, acc[q][1]);
    }
  }
  float y[NQ > 0 ? NQ : 1];
#pragma unroll
  for (int q = 0; q < NQ; ++q) y[q] = acc[q][0] + acc[q][1];
  float nin = n0 + n1;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
    for (int q = 0; q < NQ; ++q) y[q] += __shfl_xor_sync(0xffffffffu, y[q], o);
    if (POWER) nin += __shfl_xor_sync(0xffffffffu, nin, o);
  }
  if (POWER) scale = inv_norm(nin);
  if (lane < s.n) {
#pragma unroll
    for (int k = 0; k < NG; ++k) {
      const float4 v = make_float4(y[4 * k] * scale, y[4 * k + 1] * scale, y[4 * k + 2] * scale, y[4 * k + 3] * scale);
      float* tgt = dst + s.row0 + 4 * (warp + CW * k);
      if (lane == s.sub) *reinterpret_cast<float4*>(tgt) = v;
      else st_async_v4(smem_u32(tgt) + s.rdelta, v, bar + s.rdelta);
    }
  }
}

// groups of four rows this warp owns in a slab of R rows
__device__ __forceinline__ int warp_groups(int R) {
  const int warp = threadIdx.x >> 5, ng = R >> 2;
  return ng > warp ? (ng - warp + CW - 1) / CW : 0;
}

template <bool SELF>
__device__ __noinline__ void slab_gemv_send(const float* A, int lda, const float* x, const Slab s, float scale,
                                            float* dst, uint32_t bar) {
  static_assert(MAXGPW == 2, "specialisations below");
  switch (warp_groups(s.R)) {
    case 1: gemv_send_rows<SELF, 1>(A, lda, x, s, scale, dst, bar); break;
    case 2: gemv_send_rows<SELF, 2>(A, lda, x, s, scale, dst, bar); break;
    default: break;
  }
}

// The P power iterations of a step (S4) as one specialised loop: the pass, its exchange and the next pass
// follow each other without a call or a dispatch in between, and everything that does not change from pass to
// pass stays in registers.  Returns false when a wait gave up.
template <int NG>
__device__ __forceinline__ bool power_loop_rows(const Slab& s, float* buf0, int Mv, uint32_t bar0, uint32_t& e, int P,
                                                int& cur, uint32_t tx_bytes) {
  for (int p = 0; p < P; ++p) {
    const uint32_t bar = bar0 + ((e & 1) << 3);
    if (threadIdx.x == 0) sm100::mbar_expect_tx(bar, tx_bytes);     // armed ahead of the pass, off the chain
    gemv_send_rows<false, NG, true>(s.phi, s.Mp, buf0 + cur * Mv, s, 0.f, buf0 + (cur ^ 1) * Mv, bar);
    if (!exchange_wait(bar, (e >> 1) & 1)) return false;
    ++e;
    cur ^= 1;
  }
  return true;
}

__device__ __noinline__ bool power_loop(const Slab s, float* buf0, int Mv, uint32_t bar0, uint32_t& e, int P,
                                        int& cur, uint32_t tx_bytes) {
  switch (warp_groups(s.R)) {
    case 0: return power_loop_rows<0>(s, buf0, Mv, bar0, e, P, cur, tx_bytes);
    case 1: return power_loop_rows<1>(s, buf0, Mv, bar0, e, P, cur, tx_bytes);
    case 2: return power_loop_rows<2>(s, buf0, Mv, bar0, e, P, cur, tx_bytes);
    default: return true;
  }
}

// Q <- Q + aq t t^T on my rows for the pending steps (Eq. 44), in step order, each with the roundings of a step
// applied alone.  A thread has all its loads of a round in flight before it uses the first.
__device__ __noinline__ void flush_q(float* Q, const Slab s, const float* tk, int Mv, const float* aq, int pending) {
  const int M = s.M;
  if ((M & 3) == 0) {
    constexpr int U = 6;
    const int M4 = M >> 2, total = s.nrows * M4;
    float4* Q4 = reinterpret_cast<float4*>(Q + (size_t)s.row0 * M);
    for (int base = threadIdx.x; base < total; base += CT * U) {
      float4 q[U];
#pragma unroll
      for (int u = 0; u < U; ++u)
        if (base + u * CT < total) q[u] = Q4[base + u * CT];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int i = base + u * CT;
        if (i < total) {
          const int r = i / M4, c = i - r * M4;
          for (int k = 0; k < pending; ++k) {
            const float ti = tk[k * Mv + s.row0 + r], ak = aq[k];
            const float4 tj = reinterpret_cast<const float4*>(tk + k * Mv)[c];
            q[u].x = __fadd_rn(q[u].x, __fmul_rn(ak, __fmul_rn(ti, tj.x)));
            q[u].y = __fadd_rn(q[u].y, __fmul_rn(ak, __fmul_rn(ti, tj.y)));
            q[u].z = __fadd_rn(q[u].z, __fmul_rn(ak, __fmul_rn(ti, tj.z)));
            q[u].w = __fadd_rn(q[u].w, __fmul_rn(ak, __fmul_rn(ti, tj.w)));
          }
          Q4[i] = q[u];
        }
      }
    }
  } else {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int r = warp; r < s.nrows; r += CW) {
      const int i = s.row0 + r;
      float* Qr = Q + (size_t)i * M;
      for (int c = lane; c < M; c += 32) {
        float q = Qr[c];
        for (int k = 0; k < pending; ++k)
          q = __fadd_rn(q, __fmul_rn(aq[k], __fmul_rn(tk[k * Mv + i], tk[k * Mv + c])));
        Qr[c] = q;
      }
    }
  }
}

// dynamic shared memory (Mv = n R >= Mp: the length of a vector that n slices of R results fill):
// [phi slab R x Mp][tt slab R x Mp][xi2][cvec][wvec][bufA][bufB][vvec][uvec][tvec][tk: KQ x Mv]
extern __shared__ __align__(16) float csm[];

__host__ __device__ inline int slab_rows(int M, int n) { return (((M + n - 1) / n) + 3) & ~3; }

__global__ void __cluster_dims__(CL, 1, 1) __launch_bounds__(CT, 1)
recursion_cluster_kernel(const __grid_constant__ ClusterArgs a) {
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // my layer: the one whose CTA range holds this CTA (none: a filler CTA of the last cluster)
  int layer = -1;
#pragma unroll 1
  for (int l = 0; l < a.g.n; ++l)
    if ((int)blockIdx.x >= a.first_cta[l] && (int)blockIdx.x < a.first_cta[l] + a.ncta[l]) layer = l;
  if (layer < 0) {
    cluster.sync();     // the two cluster-wide meetings of the kernel
    cluster.sync();
    return;
  }
  const LayerDev* L = a.g.layer[layer];
  const int K = a.K, P = a.P;
  const int n = a.ncta[layer];
  const int sub = (int)blockIdx.x - a.first_cta[layer];
  const int rank0 = rank - sub;                 // cluster rank of the layer's first CTA
  const int M = L->M;
  const int Mp = (M + 3) & ~3;
  const int R = slab_rows(M, n);
  const int Mv = n * R;
  Slab s;
  s.M = M; s.Mp = Mp; s.R = R; s.n = n; s.sub = sub;
  s.row0 = sub * R;
  s.nrows = max(0, min(R, M - s.row0));
  s.phi = csm;
  s.tt = csm + (size_t)R * Mp;
  float* xi2 = csm + 2 * (size_t)R * Mp;
  float* cvec = xi2 + Mv;
  float* wvec = cvec + Mv;
  float* buf0 = wvec + Mv;           // two alternating power-iteration vectors, Mv apart
  float* vvec = wvec + 3 * Mv;
  float* uvec = vvec + Mv;
  float* tvec = uvec + Mv;
  float* tk = tvec + Mv;             // the vectors t of the steps whose Q terms are pending
  __shared__ __align__(8) uint64_t xbar[2];
  __shared__ float sredf[CW];
  __shared__ int sredi[CW + 1];
  __shared__ float s_aq[KQ];

  // ---- load my rows of Phi_y and T^T (padded with zeros to R rows of Mp); clear the vectors ----
  for (int which = 0; which < 2; ++which) {
    const float* G = which ? L->Tt : L->Phiy;
    float* S = which ? s.tt : s.phi;
    if ((M & 3) == 0) {
      // 16-byte asynchronous copies, every one of a thread in flight at once: the load costs one trip to
      // memory, not one per row
      const int M4 = M >> 2;
      for (int i = threadIdx.x; i < R * M4; i += CT) {
        const int r = i / M4, c = i - r * M4;
        float* d = S + (size_t)r * Mp + 4 * c;
        if (r < s.nrows) cp_async16(smem_u32(d), G + (size_t)(s.row0 + r) * M + 4 * c);
        else *reinterpret_cast<float4*>(d) = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    } else {
      for (int i = threadIdx.x; i < R * Mp; i += CT) {
        const int r = i / Mp, c = i - r * Mp;
        S[i] = (c < M && r < s.nrows) ? G[(size_t)(s.row0 + r) * M + c] : 0.f;
      }
    }
  }
  for (int i = threadIdx.x; i < (8 + KQ) * Mv; i += CT) xi2[i] = 0.f;
  asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
  if (threadIdx.x == 0) {
    sm100::mbar_init(smem_u32(&xbar[0]), 1);
    sm100::mbar_init(smem_u32(&xbar[1]), 1);
    sm100::mbar_fence_init();
  }
  const uint32_t bar0 = smem_u32(&xbar[0]);                       // the two barriers are 8 bytes apart
  // A peer's window of the cluster address space is this CTA's window shifted by a constant; the stores
  // below rely on it, so it is checked on two addresses far apart before anything is sent.
  const uint32_t peer_rank = (uint32_t)(rank0 + min(lane, n - 1));
  s.rdelta = map_cluster(bar0, peer_rank) - bar0;
  const bool linear = (map_cluster(smem_u32(tk), peer_rank) - smem_u32(tk)) == s.rdelta;
  bool failed = __syncthreads_or(!linear) != 0;
  cluster.sync();   // every barrier is initialised before the first remote store can arrive

  const uint32_t vec_bytes = (uint32_t)(n - 1) * (uint32_t)R * 4u;   // one vector's slices from the n - 1 peers
  uint32_t e = 0;                                                 // exchanges completed so far
  int pending = 0;                                                // steps whose Q terms wait in tk
  // arm the barrier of the current exchange for `nvec` vectors, wait for it, advance
#define FW_BAR (bar0 + ((e & 1) << 3))
#define FW_EXCHANGE(nvec)                                                    \
  {                                                                          \
    if (threadIdx.x == 0) sm100::mbar_expect_tx(FW_BAR, (nvec) * vec_bytes); \
    if (!exchange_wait(FW_BAR, (e >> 1) & 1)) { failed = true; goto done; }  \
    ++e;                                                                     \
  }
#define FW_FLUSH_Q()                                   \
  {                                                    \
    if (pending > 0) {                                 \
      flush_q(L->Q, s, tk, Mv, s_aq, pending);         \
      __syncthreads();                                 \
      pending = 0;                                     \
    }                                                  \
  }
  if (failed) goto done;

  {
  float* tr = const_cast<float*>(reinterpret_cast<const float*>(a.traces.p[layer]));
  const float c_rel = L->c_rel, c_abs = L->c_abs, delta = L->delta, eps = L->eps;
  const float lam_bar = L->scal[SC_LAMBDA_BAR];
  const bool maxcol = (L->init == FW_INIT_MAXCOL);
  bool any_nosub = false, any_nonfinite = false;

  for (int step = 0; step < K; ++step) {
    // S1: squared column norms (= row norms, Phi_y is exactly symmetric)             (Eq. 45)
    slab_gemv_send<true>(s.phi, Mp, nullptr, s, 1.f, xi2, FW_BAR);
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
      const float* rphi = cluster.map_shared_rank(s.phi, rank0 + owner) + (size_t)(mp - owner * R) * Mp;
      for (int m = threadIdx.x; m < Mp; m += CT) wvec[m] = rphi[m];
    }
    __syncthreads();
    slab_gemv_send<false>(s.phi, Mp, wvec, s, 1.f, cvec, FW_BAR);
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
      if (sub == 0)
        for (int m = threadIdx.x; m < M; m += CT) L->wvec[m] = wvec[m];
    }
    const float inv_cnt = cnt > 0 ? 1.f / (float)cnt : 0.f;
    slab_gemv_send<false>(s.phi, Mp, wvec, s, inv_cnt, buf0, FW_BAR);
    FW_EXCHANGE(1u)
    // S4: P power iterations u = Phi_y (prev / ||prev||)
    int cur = 0;
    if (!power_loop(s, buf0, Mv, bar0, e, P, cur, vec_bytes)) { failed = true; goto done; }
    // S5: v = prev/||prev|| (Eq. 50), u = Phi_y v, t = T^T v; lambda_e = v.u (Eq. 36)
    const float n2 = warp_dot(buf0 + cur * Mv, buf0 + cur * Mv, Mp);
    const float inv = inv_norm(n2);
    for (int m = threadIdx.x; m < Mp; m += CT) vvec[m] = buf0[cur * Mv + m] * inv;
    __syncthreads();
    slab_gemv_send<false>(s.phi, Mp, vvec, s, 1.f, uvec, FW_BAR);
    slab_gemv_send<false>(s.tt, Mp, vvec, s, 1.f, tvec, FW_BAR);
    FW_EXCHANGE(2u)
    const float lam_e = warp_dot(vvec, uvec, Mp);
    // S6: g_e, a_e (Eqs. 40-41), rank updates (Eqs. 42, 44)
    const bool ok = cnt > 0 && n2 > 0.f && isfinite(n2) && isfinite(lam_e);
    float g_e = 1.f, aa = 0.f;
    if (ok) {
      g_e = delta * lam_bar / fmaxf(lam_e, eps);
      aa = sqrtf(g_e) - 1.f;
    }
    any_nosub |= !ok;
    any_nonfinite |= !isfinite(n2) || !isfinite(lam_e);
    if (sub == 0 && threadIdx.x == 0) {
      L->scal[SC_LAMBDA_E] = lam_e; L->scal[SC_G_E] = g_e; L->scal[SC_A_E] = aa;
      L->iscal[IS_MPRIME] = mp; L->iscal[IS_SETSIZE] = cnt;
      if (tr) {
        tr[4 * step + 0] = lam_e; tr[4 * step + 1] = g_e;
        tr[4 * step + 2] = (float)cnt; tr[4 * step + 3] = (float)mp;
      }
    }
    if (aa != 0.f) {
      const float a2l = aa * aa * lam_e;
      // both slabs in shared memory: a warp walks its rows, a lane its float4 columns (the padding columns
      // hold zeros in every vector, so they stay zero in the slabs)
      // a lane's entries of v and u are the same for every row: they stay in registers
      const int M4 = Mp >> 2;
      float4 vj[kMaxIt], uj[kMaxIt];
#pragma unroll
      for (int k = 0; k < kMaxIt; ++k) {
        const int c = lane + 32 * k;
        vj[k] = uj[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < M4) { vj[k] = reinterpret_cast<const float4*>(vvec)[c]; uj[k] = reinterpret_cast<const float4*>(uvec)[c]; }
      }
      for (int r = warp; r < s.nrows; r += CW) {
        const int i = s.row0 + r;
        const float vi = vvec[i], ui = uvec[i], ti = tvec[i];
        const float ati = aa * ti;
        float4* T4 = reinterpret_cast<float4*>(s.tt + (size_t)r * Mp);
        float4* P4 = reinterpret_cast<float4*>(s.phi + (size_t)r * Mp);
#pragma unroll
        for (int k = 0; k < kMaxIt; ++k) {
          const int c = lane + 32 * k;
          if (c < M4) {
            float4 tt = T4[c], p = P4[c];
#define FW_UPD(X)                                                                                                  \
            tt.X = fmaf(ati, vj[k].X, tt.X);                                                                       \
            p.X = __fadd_rn(p.X, __fadd_rn(__fmul_rn(aa, __fadd_rn(__fmul_rn(vi, uj[k].X), __fmul_rn(ui, vj[k].X))), \
                                           __fmul_rn(a2l, __fmul_rn(vi, vj[k].X))));
            FW_UPD(x) FW_UPD(y) FW_UPD(z) FW_UPD(w)
#undef FW_UPD
            T4[c] = tt; P4[c] = p;
          }
        }
      }
      // the step's term of Q (Eq. 44) waits: the recursion does not read Q
      for (int m = threadIdx.x; m < Mp; m += CT) tk[pending * Mv + m] = tvec[m];
      if (threadIdx.x == 0) s_aq[pending] = aa * (aa + 2.f);
      __syncthreads();
      ++pending;
      if (pending == KQ) FW_FLUSH_Q()
    }
    // the slab updates are ordered before this CTA's next sends, whose receipt lets a peer read the slab
    asm volatile("fence.acq_rel.cluster;" ::: "memory");
    __syncthreads();
  }
  FW_FLUSH_Q()
  if (any_nosub && sub == 0 && threadIdx.x == 0) L->iscal[IS_STATUS_NOSUB] = 1;
  if (any_nonfinite && sub == 0 && threadIdx.x == 0) L->iscal[IS_STATUS_NONFINITE] = 1;
  }
done:
#undef FW_EXCHANGE
#undef FW_FLUSH_Q
#undef FW_BAR
  if (failed) {
    // a wait gave up: the state of this layer is not to be trusted; report and leave in step with the peers
    if (threadIdx.x == 0) L->iscal[IS_STATUS_TIMEOUT] = 1;
  } else {
    // ---- write my rows of Phi_y and T^T back ----
    for (int which = 0; which < 2; ++which) {
      float* G = which ? L->Tt : L->Phiy;
      const float* S = which ? s.tt : s.phi;
      if ((M & 3) == 0) {
        for (int r = warp; r < s.nrows; r += CW) {
          float4* dstp = reinterpret_cast<float4*>(G + (size_t)(s.row0 + r) * M);
          const float4* src = reinterpret_cast<const float4*>(S + (size_t)r * Mp);
          for (int c = lane; c < (M >> 2); c += 32) dstp[c] = src[c];
        }
      } else {
        for (int i = threadIdx.x; i < s.nrows * Mp; i += CT) {
          const int r = i / Mp, c = i - r * Mp;
          if (c < M) G[(size_t)(s.row0 + r) * M + c] = S[i];
        }
      }
    }
  }
  cluster.sync();   // no CTA leaves while a peer may still read or write its shared memory
}

size_t cluster_smem(int M, int n) {
  const int Mp = (M + 3) & ~3;
  const int R = slab_rows(M, n);
  return (2 * (size_t)R * Mp + (8 + KQ) * (size_t)n * R) * sizeof(float);
}


bool cluster_fits(int M, int n) {
  return cluster_smem(M, n) <= kSmemLimit && slab_rows(M, n) <= 4 * MAXGPW * CW && M <= 128 * kMaxIt;
}

// what a pass costs the busiest warp of a layer on n CTAs: its groups of four rows times the trips over the columns
int cluster_cost(int M, int n) {
  const int groups = slab_rows(M, n) / 4;
  return ((groups + CW - 1) / CW) * ((((M + 3) >> 2) + 31) / 32);
}

// first-fit of the layers' CTA counts (largest first) into clusters of CL: the clusters needed; first[i] (optional)
// receives the first CTA of layer i.  A layer never straddles a cluster.
int cluster_pack(const int* cnt, int n, int32_t* first) {
  int order[FW_MAX_GROUP], used[FW_MAX_GROUP];
  for (int i = 0; i < n; ++i) { order[i] = i; used[i] = 0; }
  for (int i = 1; i < n; ++i)                       // insertion sort, stable
    for (int j = i; j > 0 && cnt[order[j]] > cnt[order[j - 1]]; --j) {
      const int t = order[j]; order[j] = order[j - 1]; order[j - 1] = t;
    }
  int bins = 0;
  for (int oi = 0; oi < n; ++oi) {
    const int i = order[oi];
    int b = 0;
    while (b < bins && used[b] + cnt[i] > CL) ++b;
    if (b == bins) ++bins;
    if (first) first[i] = b * CL + used[b];
    used[b] += cnt[i];
  }
  return bins;
}

}  // namespace

// CTAs a layer of size M needs at least: the smallest count whose slabs of Phi_y and T^T fit a CTA's shared memory
// with at most MAXGPW groups of four rows per warp; 0: the layer does not fit on chip
int recursion_cluster_ctas(int M) {
  for (int n = 1; n <= CL; ++n)
    if (cluster_fits(M, n)) return n;
  return 0;
}

bool recursion_cluster_supported(int M) { return recursion_cluster_ctas(M) > 0; }

cudaError_t launch_recursion_cluster(const GroupDev& g, const PtrTable& traces, const int* layer_M, int K, int P,
                                     cudaStream_t s) {
  static SmemAttrCache attr;
  static bool nonportable_set[64] = {false};
  static int max_clusters[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); dev = 0; }
  if (!nonportable_set[dev]) {
    // clusters of 16 CTAs are beyond the portable size of 8
    cudaError_t e = cudaFuncSetAttribute(recursion_cluster_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
    nonportable_set[dev] = true;
  }
  cudaError_t e = ensure_dyn_smem(recursion_cluster_kernel, kSmemLimit, attr);
  if (e != cudaSuccess) return e;
  if (max_clusters[dev] == 0) {
    // clusters of 16 that can be resident together (7 on a B200): the plan below stays within one wave of them
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(CL * 64); cfg.blockDim = dim3(CT); cfg.dynamicSmemBytes = kSmemLimit;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = CL; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    int nc = 0;
    if (cudaOccupancyMaxActiveClusters(&nc, recursion_cluster_kernel, &cfg) != cudaSuccess || nc < 1) {
      cudaGetLastError();
      nc = 1;
    }
    max_clusters[dev] = nc;
  }
  ClusterArgs a;
  memset(&a, 0, sizeof(a));
  a.g = g; a.traces = traces; a.K = K; a.P = P;
  // Every layer starts on the fewest CTAs that hold it; then, while the clusters of one wave allow, the layer whose
  // busiest warp has the most work per pass is spread over more CTAs (the launch ends with its slowest layer).
  int cnt[FW_MAX_GROUP];
  for (int i = 0; i < g.n; ++i) {
    cnt[i] = recursion_cluster_ctas(layer_M[i]);
    if (cnt[i] == 0) return cudaErrorInvalidValue;
  }
  for (int round = 0; round < 16 * FW_MAX_GROUP; ++round) {
    int worst = -1, worst_cost = 0;
    for (int i = 0; i < g.n; ++i) {
      const int c = cluster_cost(layer_M[i], cnt[i]);
      if (c > worst_cost) { worst_cost = c; worst = i; }
    }
    if (worst < 0) break;
    // all layers at the worst cost have to improve for the launch to gain: try them in turn
    bool improved = false;
    for (int i = 0; i < g.n && !improved; ++i) {
      if (cluster_cost(layer_M[i], cnt[i]) != worst_cost) continue;
      int n2 = cnt[i] + 1;
      while (n2 <= CL && !(cluster_fits(layer_M[i], n2) && cluster_cost(layer_M[i], n2) < worst_cost)) ++n2;
      if (n2 > CL) { improved = false; break; }       // this layer cannot get cheaper: the maximum stays
      const int keep = cnt[i];
      cnt[i] = n2;
      if (cluster_pack(cnt, g.n, nullptr) > max_clusters[dev]) { cnt[i] = keep; break; }
      improved = true;
    }
    if (!improved) break;
  }
  const int bins = cluster_pack(cnt, g.n, a.first_cta);
  for (int i = 0; i < g.n; ++i) a.ncta[i] = cnt[i];
  size_t smem = 0;
  for (int i = 0; i < g.n; ++i) {
    const size_t need = cluster_smem(layer_M[i], cnt[i]);
    if (need > smem) smem = need;
  }
  ProfScope ps(FW_PROF_RECUR_CHIP, s);
  recursion_cluster_kernel<<<bins * CL, CT, smem, s>>>(a);
  return cudaGetLastError();
}

}  // namespace fw
