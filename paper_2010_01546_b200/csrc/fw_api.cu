// Host side of the C ABI: argument checks, workspace carving, launch sequencing.
// Every step of the path runs in the library's own kernels; there is no CPU
// fallback and no call into another GEMM library.
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "fw_internal.h"
#include "fw_umma.h"

using namespace fw;

struct fw_layer {
  fw_layer_desc d;
  LayerDev h;          // host mirror of the device descriptor
  LayerDev* dev;       // device copy at the start of the workspace
  cudaStream_t stream;
  void* ws;
  size_t ws_bytes;
  bool have_cov;       // a covariance exists (a block was seen or Phix was injected)
  bool first_block;    // the next fw_cov_update is the first block (Eqs. 4-5)
  bool phiy_stale;     // Phiy != T Phix T^T
  bool t_identity;     // T == I exactly (no step taken, T not injected)
  bool shift_zero;     // the pilot-mean vector on the device is all zero (nothing wrote it since it was cleared)
  bool block_open;     // earlier calls of the current block left their sums in the accumulators (FW_COV_ACCUMULATE)
  bool block_shifted;  // the current block is centred on the pilot mean taken from its first call
  int64_t acc_rows;    // rows accumulated by those calls
  uint32_t bar_base;   // arrivals so far at this layer's grid-barrier counter (persistent recursion launches it led)
  float* W;
  float* b;
};

namespace {

constexpr int kMaxDim = 8192;
constexpr size_t kAlign = 256;

size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

int split_cap_for(int M) {
  const int t = (M + 63) / 64;
  const int tiles = t * (t + 1) / 2;
  int s = (1184 + tiles - 1) / tiles;
  if (s < 1) s = 1;
  if (s > 296) s = 296;
  return s;
}

bool desc_valid(const fw_layer_desc* d) {
  if (!d) return false;
  if (d->M < 1 || d->M > kMaxDim || d->N < 1 || d->N > kMaxDim) return false;
  if (d->x_dtype != FW_F32 && d->x_dtype != FW_BF16) return false;
  if (d->prec != FW_PREC_FP32 && d->prec != FW_PREC_TF32 && d->prec != FW_PREC_BF16) return false;
  if (d->init != FW_INIT_ALIGN && d->init != FW_INIT_MAXCOL) return false;
  if (!(d->alpha >= 0.f && d->alpha < 1.f)) return false;
  if (!(d->beta >= 0.f && d->beta < 1.f)) return false;
  if (!(d->gamma > 0.f && d->gamma <= 1.f)) return false;
  if (!(d->delta > 0.f) || !(d->eps > 0.f)) return false;
  if (!(d->c_rel >= 0.f) || !(d->c_abs >= 0.f)) return false;
  return true;
}

// Lays the layer's arrays out in the workspace.  With base == nullptr only the
// total size is computed.
size_t carve(const fw_layer_desc& d, char* base, LayerDev* h) {
  size_t off = 0;
  auto take = [&](size_t bytes) -> char* {
    char* p = base ? base + off : nullptr;
    off += align_up(bytes);
    return p;
  };
  const size_t M = (size_t)d.M;
  const size_t vec = M * sizeof(float), mat = M * M * sizeof(float);
  LayerDev tmp;
  LayerDev& L = h ? *h : tmp;
  memset(&L, 0, sizeof(L));
  L.M = d.M; L.N = d.N; L.init = d.init; L.x_dtype = d.x_dtype;
  L.alpha = d.alpha; L.beta = d.beta; L.gamma = d.gamma; L.delta = d.delta;
  L.eps = d.eps; L.c_rel = d.c_rel; L.c_abs = d.c_abs;
  take(align_up(sizeof(LayerDev)));   // the descriptor itself
  L.mu = (float*)take(vec); L.mu_prev = (float*)take(vec); L.phi = (float*)take(vec);
  L.shift = (float*)take(vec);
  L.xi2 = (float*)take(vec); L.cvec = (float*)take(vec); L.wvec = (float*)take(vec);
  L.pv[0] = (float*)take(vec); L.pv[1] = (float*)take(vec);
  L.v = (float*)take(vec); L.u = (float*)take(vec); L.t = (float*)take(vec);
  L.part_stride = (d.M + kGemvMinRowsPerBlock - 1) / kGemvMinRowsPerBlock;
  L.part = (float*)take(3 * (size_t)L.part_stride * sizeof(float));
  L.scal = (float*)take(SC_COUNT * sizeof(float));
  L.iscal = (int32_t*)take(IS_COUNT * sizeof(int32_t));
  L.Phix = (float*)take(mat); L.Phiy = (float*)take(mat); L.Tt = (float*)take(mat);
  L.Q = (float*)take(mat);
  L.Qs = (d.beta > 0.f) ? (float*)take(mat) : L.Q;
  L.tmp = (float*)take(mat);
  L.split_cap = std::max(split_cap_for(d.M), d.prec != FW_PREC_FP32 ? umma_pair_split_cap(d.M) : 1);
  L.gram_part = (float*)take((size_t)L.split_cap * mat);
  L.colsum_part = (float*)take((size_t)L.split_cap * vec);
  L.gram_acc = (float*)take(mat);
  L.colsum_acc = (float*)take(vec);
  L.gq_tmp = (float*)take((size_t)d.N * vec);
  L.pmean = (float*)take(vec);
  return off;
}

fw_status cuda_fail(cudaError_t e, const char* where) {
  if (e == cudaSuccess) return FW_OK;
  fprintf(stderr, "[fw] CUDA error in %s: %s\n", where, cudaGetErrorString(e));
  return FW_ERR_CUDA;
}

#define FW_CUDA(call, where)                              \
  do {                                                    \
    cudaError_t _e = (call);                              \
    if (_e != cudaSuccess) return cuda_fail(_e, where);   \
  } while (0)

fw_status check_group(fw_layer* const* L, int32_t n) {
  if (!L || n < 1 || n > FW_MAX_GROUP) return FW_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) {
    if (!L[i]) return FW_ERR_INVALID_ARG;
    if (L[i]->stream != L[0]->stream) return FW_ERR_INVALID_ARG;
    for (int j = 0; j < i; ++j)
      if (L[j] == L[i]) return FW_ERR_INVALID_ARG;
  }
  return FW_OK;
}

void fill_group(fw_layer* const* L, int n, GroupDev& g, int& max_M, int& max_N) {
  g.n = n; g.pad = 0;
  max_M = 0; max_N = 0;
  for (int i = 0; i < n; ++i) {
    g.layer[i] = L[i]->dev;
    if (L[i]->d.M > max_M) max_M = L[i]->d.M;
    if (L[i]->d.N > max_N) max_N = L[i]->d.N;
  }
}

// Phiy <- T Phix T^T for the layers whose Phiy is stale (a5).  With T kept transposed
// (Tt = T^T) both products have the form A^T B:  tmp = Phix^T Tt (= Phix T^T, Phix is
// symmetric) and Phiy = Tt^T tmp.  Tensor-core engines run them as TF32 MMAs, the FP32
// engine as FFMA GEMMs; the result is mirrored from its upper triangle.
fw_status resync_phiy(fw_layer* const* L, int n) {
  GemmGroup g1, g2;
  g1.n = g2.n = 0;
  std::vector<UmmaAtbItem> t1, t2, p1, p2;   // single-CTA kernel / CTA-pair kernel, first and second product
  for (int i = 0; i < n; ++i) {
    fw_layer* l = L[i];
    if (!l->phiy_stale) continue;
    const int M = l->d.M;
    const size_t mat = (size_t)M * M * sizeof(float);
    if (l->t_identity) {
      FW_CUDA(cudaMemcpyAsync(l->h.Phiy, l->h.Phix, mat, cudaMemcpyDeviceToDevice, l->stream), "resync copy");
      if (l->d.gamma != 1.0f)   // Pt = (T Phix)^T = Phix at T = I
        FW_CUDA(cudaMemcpyAsync(l->h.tmp, l->h.Phix, mat, cudaMemcpyDeviceToDevice, l->stream), "resync copy Pt");
    } else if (l->d.prec != FW_PREC_FP32 && umma_available() && M >= 16 && (M % 4) == 0) {
      const bool pair = umma_pair_atb_eligible(M);
      UmmaAtbItem it;
      it.status = l->h.iscal + IS_STATUS_TIMEOUT;
      it.A = l->h.Phix; it.B = l->h.Tt; it.C = l->h.tmp; it.M = M; it.sym = 0;
      (pair ? p1 : t1).push_back(it);
      // T (Phix T^T) is symmetric: its upper triangle is computed and mirrored by the kernel
      it.A = l->h.Tt; it.B = l->h.tmp; it.C = l->h.Phiy; it.M = M; it.sym = 1;
      (pair ? p2 : t2).push_back(it);
    } else {
      GemmProblem p;
      memset(&p, 0, sizeof(p));
      // tmp = Pt = Phix^T Tt: A = Phix stored (k x m), B = Tt
      p.A = l->h.Phix; p.B = l->h.Tt; p.C = l->h.tmp;
      p.lda = p.ldb = p.ldc = M; p.m = p.n = M; p.k = M;
      p.a_kmajor = 1; p.sym = 0; p.splits = 1; p.epi = EPI_STORE;
      g1.p[g1.n++] = p;
      // Phiy = Tt^T Pt: A = Tt stored (k x m), B = Pt; symmetric result
      memset(&p, 0, sizeof(p));
      p.A = l->h.Tt; p.B = l->h.tmp; p.C = l->h.Phiy;
      p.lda = p.ldb = p.ldc = M; p.m = p.n = M; p.k = M;
      p.a_kmajor = 1; p.sym = 1; p.splits = 1; p.epi = EPI_SYMM;
      g2.p[g2.n++] = p;
    }
    l->phiy_stale = false;
  }
  if (g1.n) {
    FW_CUDA(launch_gemm_ffma(g1, L[0]->stream, FW_PROF_RESYNC), "resync gemm 1");
    FW_CUDA(launch_gemm_ffma(g2, L[0]->stream, FW_PROF_RESYNC), "resync gemm 2");
  }
  if (!t1.empty() || !p1.empty()) {
    // first products of every layer, then the second products (which read the first)
    fw_status st = FW_OK;
    if (!t1.empty()) st = umma_atb_launch(t1.data(), (int)t1.size(), L[0]->stream);
    if (st == FW_OK && !p1.empty()) st = umma_pair_atb_launch(p1.data(), (int)p1.size(), L[0]->stream);
    if (st == FW_OK && !t2.empty()) st = umma_atb_launch(t2.data(), (int)t2.size(), L[0]->stream);
    if (st == FW_OK && !p2.empty()) st = umma_pair_atb_launch(p2.data(), (int)p2.size(), L[0]->stream);
    if (st != FW_OK) return st;
  }
  return FW_OK;
}

// ---- launch accounting and optional event timing ----
struct ProfRec { int cls; cudaEvent_t a, b; };
bool g_prof_on = false;
std::vector<ProfRec> g_prof;
std::vector<cudaEvent_t> g_event_pool;
int64_t g_launches = 0;

cudaEvent_t prof_event() {
  if (!g_event_pool.empty()) { cudaEvent_t e = g_event_pool.back(); g_event_pool.pop_back(); return e; }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}

}  // namespace

namespace fw {
const Tuning& tuning() {
  static const Tuning t = [] {
    auto geti = [](const char* name, int dflt) { const char* e = getenv(name); return e ? atoi(e) : dflt; };
    Tuning v;
    v.pair_min_m = geti("FW_PAIR_MIN_M", 289);
    if (v.pair_min_m < 16) v.pair_min_m = 289;
    v.pair_splits = geti("FW_PAIR_SPLITS", 0);
    v.pair_debug = getenv("FW_PAIR_DEBUG") ? 1 : 0;
    v.pass_shape = geti("FW_PASS_SHAPE", 0);
    v.persist_max_mb = geti("FW_PERSIST_MAX_MB", 512);
    v.gram_waves_pct = geti("FW_GRAM_WAVES_PCT", 200);
    if (v.gram_waves_pct < 50 || v.gram_waves_pct > 1600) v.gram_waves_pct = 200;
    return v;
  }();
  return t;
}
void prof_open(int cls, cudaStream_t s) {
  ++g_launches;
  if (!g_prof_on) return;
  ProfRec r; r.cls = cls; r.a = prof_event(); r.b = nullptr;
  cudaEventRecord(r.a, s);
  g_prof.push_back(r);
}
void prof_close(int cls, cudaStream_t s) {
  (void)cls;
  if (!g_prof_on || g_prof.empty()) return;
  ProfRec& r = g_prof.back();
  r.b = prof_event();
  cudaEventRecord(r.b, s);
}
}  // namespace fw

extern "C" {

fw_status fw_profile_begin(void) {
  g_prof.clear();
  g_prof_on = true;
  return FW_OK;
}

fw_status fw_profile_end(float* ms_per_class, int64_t* launches_per_class) {
  g_prof_on = false;
  float ms[FW_PROF_CLASSES] = {0};
  int64_t cnt[FW_PROF_CLASSES] = {0};
  fw_status st = FW_OK;
  for (ProfRec& r : g_prof) {
    if (r.a && r.b) {
      float t = 0.f;
      if (cudaEventSynchronize(r.b) != cudaSuccess || cudaEventElapsedTime(&t, r.a, r.b) != cudaSuccess) {
        cudaGetLastError();
        st = FW_ERR_CUDA;
      }
      if (r.cls >= 0 && r.cls < FW_PROF_CLASSES) { ms[r.cls] += t; cnt[r.cls] += 1; }
    }
    if (r.a) g_event_pool.push_back(r.a);
    if (r.b) g_event_pool.push_back(r.b);
  }
  g_prof.clear();
  for (int i = 0; i < FW_PROF_CLASSES; ++i) {
    if (ms_per_class) ms_per_class[i] = ms[i];
    if (launches_per_class) launches_per_class[i] = cnt[i];
  }
  return st;
}

int64_t fw_launch_count(void) { return g_launches; }

int32_t fw_recursion_on_chip(const fw_layer_desc* d) {
  if (!desc_valid(d)) return 0;
  return (d->gamma == 1.0f && recursion_cluster_supported(d->M)) ? 1 : 0;
}

void fw_layer_desc_default(fw_layer_desc* d, int32_t M, int32_t N) {
  if (!d) return;
  d->M = M; d->N = N;
  d->x_dtype = FW_F32; d->prec = FW_PREC_FP32; d->init = FW_INIT_ALIGN;
  d->alpha = 0.1f; d->beta = 0.1f; d->gamma = 0.99f; d->delta = 0.25f;
  d->eps = 1e-5f; d->c_rel = 0.025f; d->c_abs = 1e-6f;
}

size_t fw_layer_workspace_bytes(const fw_layer_desc* d) {
  if (!desc_valid(d)) return 0;
  return carve(*d, nullptr, nullptr);
}

fw_status fw_layer_create(const fw_layer_desc* d, void* dev_workspace, size_t bytes, void* cuda_stream,
                          fw_layer** out) {
  if (!out) return FW_ERR_INVALID_ARG;
  *out = nullptr;
  if (!d || !dev_workspace) return FW_ERR_INVALID_ARG;
  if (!desc_valid(d)) return (d->M < 1 || d->M > kMaxDim || d->N < 1 || d->N > kMaxDim) ? FW_ERR_SHAPE
                                                                                         : FW_ERR_INVALID_ARG;
  if (d->prec == FW_PREC_BF16 && d->x_dtype != FW_BF16) return FW_ERR_INVALID_ARG;
  if (d->prec == FW_PREC_TF32 && d->x_dtype != FW_F32) return FW_ERR_INVALID_ARG;
  if (((uintptr_t)dev_workspace % kAlign) != 0) return FW_ERR_WORKSPACE;
  const size_t need = carve(*d, nullptr, nullptr);
  if (bytes < need) return FW_ERR_WORKSPACE;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) {
    cudaGetLastError();
    fprintf(stderr, "[fw] no CUDA device: this library has no CPU path\n");
    return FW_ERR_CUDA;
  }
  fw_layer* L = new (std::nothrow) fw_layer;
  if (!L) return FW_ERR_INVALID_ARG;
  memset(L, 0, sizeof(*L));
  L->d = *d;
  L->stream = (cudaStream_t)cuda_stream;
  L->ws = dev_workspace;
  L->ws_bytes = bytes;
  carve(*d, (char*)dev_workspace, &L->h);
  L->dev = (LayerDev*)dev_workspace;
  L->have_cov = false; L->first_block = true; L->phiy_stale = true; L->t_identity = true;
  L->shift_zero = false;               // cleared by init_identity, but the first block settles it either way
  L->block_open = false; L->block_shifted = false; L->acc_rows = 0; L->bar_base = 0;
  cudaError_t e = cudaMemcpyAsync(L->dev, &L->h, sizeof(LayerDev), cudaMemcpyHostToDevice, L->stream);
  if (e == cudaSuccess) e = launch_init_identity(L->dev, d->M, L->stream);
  if (e != cudaSuccess) { delete L; return cuda_fail(e, "fw_layer_create"); }
  *out = L;
  return FW_OK;
}

fw_status fw_layer_destroy(fw_layer* L) {
  if (!L) return FW_ERR_INVALID_ARG;
  delete L;
  return FW_OK;
}

fw_status fw_layer_reset(fw_layer* L) {
  if (!L) return FW_ERR_INVALID_ARG;
  FW_CUDA(launch_init_identity(L->dev, L->d.M, L->stream), "fw_layer_reset");
  L->have_cov = false; L->first_block = true; L->phiy_stale = true; L->t_identity = true;
  L->shift_zero = true;                // init_identity clears the shift vector
  L->block_open = false; L->block_shifted = false; L->acc_rows = 0; L->bar_base = 0;
  return FW_OK;
}

fw_status fw_layer_attach_params(fw_layer* L, float* W, float* b) {
  if (!L) return FW_ERR_INVALID_ARG;
  if ((W == nullptr) != (b == nullptr)) return FW_ERR_INVALID_ARG;
  L->W = W; L->b = b;
  return FW_OK;
}

// Geometry of a layer whose rows are 3 x 3 patches of a zero-padded NHWC activation (implicit im2col); C == 0: the
// layer's X is an ordinary row-major matrix.
struct NhwcSpec { int32_t B, H, W, C; };

static fw_status cov_update_impl(fw_layer* const* L, int32_t n, const void* const* X, const int64_t* rows,
                                 const int64_t* ldx, uint32_t flags, const NhwcSpec* nh) {
  fw_status st = check_group(L, n);
  if (st != FW_OK) return st;
  if (!X || !rows || !ldx) return FW_ERR_INVALID_ARG;
  if (flags != FW_COV_COMMIT && flags != FW_COV_ACCUMULATE) return FW_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) {
    if (!X[i]) return FW_ERR_INVALID_ARG;
    if (rows[i] < 1 || ldx[i] < L[i]->d.M) return FW_ERR_SHAPE;
    if (rows[i] > ((int64_t)1 << 40) || L[i]->acc_rows + rows[i] > ((int64_t)1 << 40)) return FW_ERR_SHAPE;
  }
  const bool commit = (flags == FW_COV_COMMIT);
  cudaStream_t s = L[0]->stream;
  GroupDev g; int max_M, max_N;
  fill_group(L, n, g, max_M, max_N);
  PtrTable xt, wt, bt; Rows64 rt;
  memset(&xt, 0, sizeof(xt)); memset(&wt, 0, sizeof(wt)); memset(&bt, 0, sizeof(bt));
  bool any_params = false;
  for (int i = 0; i < n; ++i) {
    xt.p[i] = X[i]; rt.v[i] = L[i]->acc_rows + rows[i];   // the moments see the whole block
    wt.p[i] = L[i]->W; bt.p[i] = L[i]->b;
    any_params |= (L[i]->W != nullptr);
  }
  // The tensor-core engine handles the layers it supports; the rest run on FFMA.
  int32_t splits[FW_MAX_GROUP], first[FW_MAX_GROUP];
  float corr[FW_MAX_GROUP];
  for (int i = 0; i < n; ++i) corr[i] = 0.f;
  bool on_tc[FW_MAX_GROUP], unshifted[FW_MAX_GROUP];
  std::vector<int> ffma_idx, umma_idx;
  for (int i = 0; i < n; ++i) {
    on_tc[i] = L[i]->d.prec != FW_PREC_FP32 && umma_gram_supported(L[i]->d, X[i], ldx[i]);
    if (nh && nh[i].C > 0) {
      // implicit im2col exists on the tensor-core engine with fp32 activations only, and not inside a block that
      // an ordinary call opened with a pilot shift
      int bw = 0, bh = 0;
      if (!on_tc[i] || L[i]->d.x_dtype != FW_F32 ||
          !umma_gram_im2col_geometry(nh[i].H, nh[i].W, nh[i].C, 32, &bw, &bh))
        return FW_ERR_UNSUPPORTED;
      if (L[i]->block_open && L[i]->block_shifted) return FW_ERR_STATE;
    }
    (on_tc[i] ? umma_idx : ffma_idx).push_back(i);
  }
  // Centring inside the Gram pass.  A block's first call decides: tensor-core layers with bf16 X or a long fp32
  // block are fed unshifted (zero shift vector), every other block is centred on the pilot mean of that call's
  // first rows.  Later calls of an open block keep the block's shift: the sums they add must be relative to it.
  // Unshifted blocks that go to the CTA-pair kernel get a pilot mean of their own (pmean): the kernel takes its
  // outer product out of the accumulators as the rows go by and the moment kernels put it back.
  bool pilot[FW_MAX_GROUP], to_pair[FW_MAX_GROUP];
  {
    for (int i = 0; i < n; ++i) {
      const bool i2c = nh && nh[i].C > 0;
      const bool can_unshift = on_tc[i] && (i2c || umma_gram_unshifted(L[i]->d, rows[i]));
      pilot[i] = false;
      if (L[i]->block_open) {
        unshifted[i] = can_unshift && !L[i]->block_shifted;
      } else {
        unshifted[i] = can_unshift;
        L[i]->block_shifted = !can_unshift;
        if (can_unshift) {
          // the moments expect a zero shift; cleared once, not on every block
          if (!L[i]->shift_zero) {
            FW_CUDA(cudaMemsetAsync(L[i]->h.shift, 0, (size_t)L[i]->d.M * sizeof(float), s), "shift memset");
            L[i]->shift_zero = true;
          }
        } else {
          pilot[i] = true;
          L[i]->shift_zero = false;            // the pilot-mean kernel writes it
        }
      }
      UmmaGramItem probe;
      memset(&probe, 0, sizeof(probe));
      probe.rows = rows[i]; probe.M = L[i]->d.M; probe.shift = unshifted[i] ? nullptr : L[i]->h.shift;
      to_pair[i] = on_tc[i] && !i2c && umma_pair_gram_eligible(probe);
    }
    // up to four pilot launches: (fp32, bf16) x (into the shift, into pmean)
    for (int pass = 0; pass < 4; ++pass) {
      const bool want_bf16 = (pass & 1) != 0, want_pmean = (pass & 2) != 0;
      GroupDev gp; PtrTable xp; Rows64 rp, lp; gp.n = 0; gp.pad = 0; int mm = 0;
      for (int i = 0; i < n; ++i) {
        if (want_pmean ? !to_pair[i] : !pilot[i]) continue;
        if ((L[i]->d.x_dtype == FW_BF16) != want_bf16) continue;
        gp.layer[gp.n] = L[i]->dev; xp.p[gp.n] = X[i]; rp.v[gp.n] = rows[i]; lp.v[gp.n] = ldx[i];
        if (L[i]->d.M > mm) mm = L[i]->d.M;
        ++gp.n;
      }
      if (gp.n) FW_CUDA(launch_pilot_mean(gp, xp, rp, lp, want_bf16 ? 1 : 0, mm, want_pmean ? 1 : 0, s), "pilot mean");
    }
  }
  if (!ffma_idx.empty()) {
    // choose K-splits so that the launch fills the machine a few times over
    double work = 0;
    for (int i : ffma_idx) {
      const int t = (L[i]->d.M + 63) / 64;
      work += (double)(t * (t + 1) / 2) * (double)rows[i];
    }
    double klen = work / 1184.0;
    if (klen < 256) klen = 256;
    GemmGroup gg; gg.n = 0;
    for (int i : ffma_idx) {
      const int M = L[i]->d.M;
      int sp = (int)((double)rows[i] / klen + 0.999);
      if (sp < 1) sp = 1;
      if (sp > L[i]->h.split_cap) sp = L[i]->h.split_cap;
      int64_t kslabs = (rows[i] + 15) / 16;
      if (sp > kslabs) sp = (int)kslabs;
      splits[i] = sp;
      GemmProblem p;
      memset(&p, 0, sizeof(p));
      p.A = X[i]; p.B = X[i]; p.C = L[i]->h.gram_part;
      p.shift = L[i]->h.shift; p.colsum = L[i]->h.colsum_part;
      p.lda = p.ldb = ldx[i]; p.ldc = M; p.c_split_stride = (int64_t)M * M;
      p.m = p.n = M; p.k = rows[i];
      p.a_kmajor = 1; p.sym = 1; p.splits = sp; p.epi = EPI_STORE;
      p.in_bf16 = (L[i]->d.x_dtype == FW_BF16);
      gg.p[gg.n++] = p;
    }
    FW_CUDA(launch_gemm_ffma(gg, s, FW_PROF_GRAM), "gram ffma");
  }
  if (!umma_idx.empty()) {
    // large layers run on CTA pairs, the rest on the single-CTA kernel
    std::vector<UmmaGramItem> items, pair_items;
    for (int i : umma_idx) {
      UmmaGramItem it;
      memset(&it, 0, sizeof(it));
      it.X = X[i]; it.rows = rows[i]; it.ldx = ldx[i]; it.M = L[i]->d.M;
      it.x_bf16 = (L[i]->d.x_dtype == FW_BF16);
      it.shift = unshifted[i] ? nullptr : L[i]->h.shift;
      it.gram_part = L[i]->h.gram_part; it.colsum_part = L[i]->h.colsum_part;
      it.split_cap = L[i]->h.split_cap;
      it.tag = i;
      it.status = L[i]->h.iscal + IS_STATUS_TIMEOUT;
      it.pmean = to_pair[i] ? L[i]->h.pmean : nullptr;
      if (nh && nh[i].C > 0) {
        it.im2col = 1; it.i2c_B = nh[i].B; it.i2c_H = nh[i].H; it.i2c_W = nh[i].W; it.i2c_C = nh[i].C;
      }
      (to_pair[i] ? pair_items : items).push_back(it);
    }
    if (!pair_items.empty()) {
      st = umma_pair_gram_launch(pair_items.data(), (int)pair_items.size(), s);
      if (st != FW_OK) return st;
      for (const UmmaGramItem& it : pair_items) { splits[it.tag] = it.splits_out; corr[it.tag] = it.corr_out; }
    }
    if (!items.empty()) {
      st = umma_gram_launch(items.data(), (int)items.size(), s);
      if (st != FW_OK) return st;
      for (const UmmaGramItem& it : items) splits[it.tag] = it.splits_out;
    }
  }
  int32_t dims[FW_MAX_GROUP], cont[FW_MAX_GROUP];
  for (int i = 0; i < n; ++i) {
    first[i] = L[i]->first_block ? 1 : 0; dims[i] = L[i]->d.M; cont[i] = L[i]->block_open ? 1 : 0;
  }
  if (!commit) {
    // the block stays open: this call's sums join the accumulators, no moment changes
    int32_t fresh[FW_MAX_GROUP];
    for (int i = 0; i < n; ++i) fresh[i] = cont[i] ? 0 : 1;
    FW_CUDA(launch_accumulate(g, splits, fresh, corr, dims, s), "accumulate");
    for (int i = 0; i < n; ++i) { L[i]->block_open = true; L[i]->acc_rows += rows[i]; }
    return FW_OK;
  }
  FW_CUDA(launch_moments(g, rt, splits, first, cont, corr, dims, wt, bt, max_M, max_N, any_params, s), "moments");
  for (int i = 0; i < n; ++i) {
    L[i]->first_block = false; L[i]->have_cov = true; L[i]->phiy_stale = true;
    L[i]->block_open = false; L[i]->acc_rows = 0;
  }
  return FW_OK;
}

fw_status fw_group_cov_update(fw_layer* const* L, int32_t n, const void* const* X, const int64_t* rows,
                              const int64_t* ldx, uint32_t flags) {
  return cov_update_impl(L, n, X, rows, ldx, flags, nullptr);
}

fw_status fw_cov_update(fw_layer* L, const void* X, int64_t rows, int64_t ldx, uint32_t flags) {
  if (!L) return FW_ERR_INVALID_ARG;
  return cov_update_impl(&L, 1, &X, &rows, &ldx, flags, nullptr);
}

// floats of the padded copy [B][H + 2][W + 2][C], plus the floats a chunk of the last window may reach past it
static int64_t nhwc_scratch_floats(int64_t B, int64_t H, int64_t W, int64_t C) {
  return (B * (H + 2) * (W + 2) * C + 64 + 3) / 4 * 4;
}

size_t fw_nhwc_scratch_bytes(int32_t B, int32_t H, int32_t W, int32_t C, int32_t k) {
  if (B < 1 || H < 1 || W < 1 || C < 1 || k != 3) return 0;
  return (size_t)nhwc_scratch_floats(B, H, W, C) * sizeof(float);
}

fw_status fw_group_cov_update_nhwc(fw_layer* const* L, int32_t n, const float* const* A, const int32_t* B,
                                   const int32_t* H, const int32_t* W, const int32_t* C, const int32_t* k,
                                   void* const* scratch, const size_t* scratch_bytes, uint32_t flags) {
  fw_status st = check_group(L, n);
  if (st != FW_OK) return st;
  if (!A || !B || !H || !W || !C || !k) return FW_ERR_INVALID_ARG;
  const void* X[FW_MAX_GROUP];
  int64_t rows[FW_MAX_GROUP], ldx[FW_MAX_GROUP];
  NhwcSpec nh[FW_MAX_GROUP];
  for (int i = 0; i < n; ++i) {
    if (!A[i]) return FW_ERR_INVALID_ARG;
    if (B[i] < 1 || H[i] < 1 || W[i] < 1 || C[i] < 1) return FW_ERR_SHAPE;
    if (k[i] != 1 && k[i] != 3) return FW_ERR_UNSUPPORTED;
    if ((int64_t)C[i] * k[i] * k[i] != L[i]->d.M) return FW_ERR_SHAPE;
    rows[i] = (int64_t)B[i] * H[i] * W[i];
    ldx[i] = L[i]->d.M;
    nh[i] = NhwcSpec{0, 0, 0, 0};
    if (k[i] == 1) { X[i] = A[i]; continue; }
    if (L[i]->d.x_dtype != FW_F32 || L[i]->d.prec == FW_PREC_FP32 || (C[i] % 4) != 0) return FW_ERR_UNSUPPORTED;
    if (!scratch || !scratch_bytes || !scratch[i]) return FW_ERR_INVALID_ARG;
    const int64_t need = nhwc_scratch_floats(B[i], H[i], W[i], C[i]);
    if (scratch_bytes[i] < (size_t)need * sizeof(float) || ((uintptr_t)scratch[i] % kAlign) != 0) return FW_ERR_WORKSPACE;
    X[i] = scratch[i];
    nh[i] = NhwcSpec{B[i], H[i], W[i], C[i]};
  }
  // zero-padded copies first (they are what the Gram kernel's windows read), all layers in one launch
  {
    const float* src[FW_MAX_GROUP]; float* dst[FW_MAX_GROUP];
    int pb[FW_MAX_GROUP], ph[FW_MAX_GROUP], pw[FW_MAX_GROUP], pc[FW_MAX_GROUP];
    int64_t pf[FW_MAX_GROUP];
    int np = 0;
    for (int i = 0; i < n; ++i) {
      if (nh[i].C == 0) continue;
      src[np] = A[i]; dst[np] = (float*)scratch[i]; pb[np] = B[i]; ph[np] = H[i]; pw[np] = W[i]; pc[np] = C[i];
      pf[np] = nhwc_scratch_floats(B[i], H[i], W[i], C[i]);
      ++np;
    }
    if (np) FW_CUDA(launch_pad_nhwc(np, src, dst, pb, ph, pw, pc, pf, L[0]->stream), "pad activations");
  }
  return cov_update_impl(L, n, X, rows, ldx, flags, nh);
}

fw_status fw_cov_update_nhwc(fw_layer* L, const float* A, int32_t B, int32_t H, int32_t W, int32_t C, int32_t k,
                             void* scratch, size_t scratch_bytes, uint32_t flags) {
  if (!L) return FW_ERR_INVALID_ARG;
  return fw_group_cov_update_nhwc(&L, 1, &A, &B, &H, &W, &C, &k, &scratch, &scratch_bytes, flags);
}

fw_status fw_group_cond_reduce(fw_layer* const* L, int32_t n, int32_t K, int32_t P,
                               float* const* traces_or_null) {
  fw_status st = check_group(L, n);
  if (st != FW_OK) return st;
  if (K < 0 || P < 0 || K > 100000 || P > 100000) return FW_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) {
    if (!L[i]->have_cov) return FW_ERR_STATE;
  }
  cudaStream_t s = L[0]->stream;
  st = resync_phiy(L, n);
  if (st != FW_OK) return st;
  if (K == 0) return FW_OK;      // no step: Phi_y has been brought up to date, nothing else changes
  GroupDev g; int max_M, max_N;
  fill_group(L, n, g, max_M, max_N);
  // small layers: the whole K-step recursion runs on chip, a layer on 1 to 16 CTAs of a cluster;
  // the rest takes the multi-launch path (one launch per pass, batched over layers)
  GroupDev gc, gl; PtrTable tc, tl;
  memset(&tc, 0, sizeof(tc)); memset(&tl, 0, sizeof(tl));
  gc.n = gl.n = 0; gc.pad = gl.pad = 0;
  int ml = 0;
  int dims_c[FW_MAX_GROUP];
  // largest layers first: CTAs are handed out in launch order, so the long row blocks start early and the
  // short ones fill the end of every pass
  std::vector<int> order(n);
  for (int i = 0; i < n; ++i) order[i] = i;
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return L[a]->d.M > L[b]->d.M; });
  for (int oi = 0; oi < n; ++oi) {
    const int i = order[oi];
    float* t = traces_or_null ? traces_or_null[i] : nullptr;
    if (L[i]->d.gamma == 1.0f && recursion_cluster_supported(L[i]->d.M)) {
      gc.layer[gc.n] = L[i]->dev; tc.p[gc.n] = t; dims_c[gc.n] = L[i]->d.M; ++gc.n;
    } else {
      gl.layer[gl.n] = L[i]->dev; tl.p[gl.n] = t; ++gl.n;
      if (L[i]->d.M > ml) ml = L[i]->d.M;
    }
  }
  if (gc.n) FW_CUDA(launch_recursion_cluster(gc, tc, dims_c, K, P, s), "recursion (cluster)");
  if (gl.n) {
    // large layers: gamma = 1 layers with 16-byte rows take all K steps in one persistent cooperative launch;
    // leaky layers (their update needs transposed tiles) and odd sizes take one launch per pass
    GroupDev gp, go; PtrTable tp, to;
    memset(&tp, 0, sizeof(tp)); memset(&to, 0, sizeof(to));
    gp.n = go.n = 0; gp.pad = go.pad = 0;
    int dims_p[FW_MAX_GROUP];
    fw_layer* leader = nullptr;
    int mo = 0, row_blocks = 0;
    bool any_leaky = false;
    // The persistent launch wins where a pass is short against a kernel boundary (a handful of layers, up to a few
    // hundred MB of state in all); past that the statically split rows stream a few percent below the many small
    // CTAs of the per-pass launches, which the hardware balances as it goes.
    double state_mb = 0;
    for (int i = 0; i < n; ++i)
      if (!(L[i]->d.gamma == 1.0f && recursion_cluster_supported(L[i]->d.M)))
        state_mb += 4.0 * L[i]->d.M * (double)L[i]->d.M / 1e6;
    const bool persist_ok = state_mb <= (double)tuning().persist_max_mb;
    for (int oi = 0; oi < n; ++oi) {
      const int i = order[oi];
      if (L[i]->d.gamma == 1.0f && recursion_cluster_supported(L[i]->d.M)) continue;
      float* t = traces_or_null ? traces_or_null[i] : nullptr;
      const int Mi = L[i]->d.M;
      const float gi = L[i]->d.gamma;
      if (persist_ok && recursion_persist_supported(&Mi, &gi, 1)) {
        if (!leader) leader = L[i];
        dims_p[gp.n] = Mi;
        gp.layer[gp.n] = L[i]->dev; tp.p[gp.n] = t; ++gp.n;
      } else {
        go.layer[go.n] = L[i]->dev; to.p[go.n] = t; ++go.n;
        if (Mi > mo) mo = Mi;
        row_blocks += (Mi + kGemvRowsPerBlock - 1) / kGemvRowsPerBlock;
        any_leaky |= (gi != 1.0f);
      }
    }
    if (gp.n)
      FW_CUDA(launch_recursion_persist(gp, tp, dims_p, K, P, leader->h.iscal + IS_GRID_BAR,
                                       leader->h.iscal + IS_STATUS_TIMEOUT, &leader->bar_base, s),
              "recursion (persistent)");
    for (int k = 0; k < K && go.n; ++k)
      FW_CUDA(launch_recursion_step(go, P, k, to, mo, any_leaky, row_blocks, s), "recursion step");
  }
  bool any_beta = false;
  for (int i = 0; i < n; ++i) any_beta |= (L[i]->d.beta > 0.f);
  if (any_beta) FW_CUDA(launch_smooth(g, max_M, s), "smooth");
  for (int i = 0; i < n; ++i) L[i]->t_identity = false;
  return FW_OK;
}

fw_status fw_cond_reduce(fw_layer* L, int32_t K, int32_t P, float* trace_or_null) {
  if (!L) return FW_ERR_INVALID_ARG;
  float* tr = trace_or_null;
  return fw_group_cond_reduce(&L, 1, K, P, trace_or_null ? &tr : nullptr);
}

static fw_status grad_transform_impl(fw_layer* const* L, int32_t n, const float* const* G, float* const* out,
                                     int epi, float lr) {
  cudaStream_t s = L[0]->stream;
  std::vector<int> ffma_idx, umma_idx;
  for (int i = 0; i < n; ++i) {
    if (L[i]->d.prec != FW_PREC_FP32 && umma_gq_pair_supported(L[i]->d.M)) umma_idx.push_back(i);
    else ffma_idx.push_back(i);
  }
  if (!ffma_idx.empty()) {
    GemmGroup gg; gg.n = 0;
    for (int i : ffma_idx) {
      const int M = L[i]->d.M, N = L[i]->d.N;
      GemmProblem p;
      memset(&p, 0, sizeof(p));
      p.A = G[i]; p.B = L[i]->h.Qs; p.C = out[i];
      p.lda = M; p.ldb = M; p.ldc = M; p.m = N; p.n = M; p.k = M;
      p.a_kmajor = 0; p.sym = 0; p.splits = 1; p.epi = epi; p.lr = lr;
      p.nonfinite = L[i]->h.iscal + IS_STATUS_NONFINITE;
      gg.p[gg.n++] = p;
    }
    FW_CUDA(launch_gemm_ffma(gg, s, FW_PROF_GQ), "grad transform ffma");
  }
  if (!umma_idx.empty()) {
    std::vector<UmmaGqItem> items;
    for (int i : umma_idx) {
      UmmaGqItem it;
      memset(&it, 0, sizeof(it));
      it.Qs = L[i]->h.Qs; it.G = G[i]; it.out = out[i]; it.M = L[i]->d.M; it.N = L[i]->d.N;
      it.status = L[i]->h.iscal + IS_STATUS_TIMEOUT; it.nonfinite = L[i]->h.iscal + IS_STATUS_NONFINITE;
      // the Gram pass's split partials are free between covariance updates: scratch for the K split
      it.part = L[i]->h.gram_part; it.part_floats = (int64_t)L[i]->h.split_cap * L[i]->d.M * L[i]->d.M;
      items.push_back(it);
    }
    // longest K first: items start in list order
    std::stable_sort(items.begin(), items.end(), [](const UmmaGqItem& a, const UmmaGqItem& b) { return a.M > b.M; });
    fw_status st = umma_gq_pair_launch(items.data(), (int)items.size(), epi, lr, FW_PROF_GQ, s);
    if (st != FW_OK) return st;
  }
  return FW_OK;
}

fw_status fw_grad_transform(fw_layer* L, const float* G, float* G_out) {
  if (!L || !G || !G_out) return FW_ERR_INVALID_ARG;
  const size_t bytes = (size_t)L->d.N * L->d.M * sizeof(float);
  if (G == G_out) {
    // in place: every tile of the product reads whole rows of G, so the product is formed in the workspace
    float* tmp = L->h.gq_tmp;
    fw_status st = grad_transform_impl(&L, 1, &G, &tmp, EPI_STORE, 0.f);
    if (st != FW_OK) return st;
    FW_CUDA(cudaMemcpyAsync(G_out, tmp, bytes, cudaMemcpyDeviceToDevice, L->stream), "grad transform in place");
    return FW_OK;
  }
  const uintptr_t a = (uintptr_t)G, b = (uintptr_t)G_out;
  if (a < b + bytes && b < a + bytes) return FW_ERR_INVALID_ARG;   // partial overlap
  return grad_transform_impl(&L, 1, &G, &G_out, EPI_STORE, 0.f);
}

// out (rows x M) = In (rows x M) * Bmat (M x M, row-major) - 1 colbias^T on the layer's engine
static fw_status rows_times_matrix(fw_layer* L, const float* In, int64_t rows, const float* Bmat, const float* colbias,
                                   float* out) {
  const int M = L->d.M;
  if (L->d.prec != FW_PREC_FP32 && umma_gq_pair_supported(M)) {
    UmmaGqItem it;
    memset(&it, 0, sizeof(it));
    it.Qs = Bmat; it.G = In; it.out = out; it.M = M; it.N = rows;
    it.status = L->h.iscal + IS_STATUS_TIMEOUT; it.nonfinite = L->h.iscal + IS_STATUS_NONFINITE;
    it.colbias = colbias;            // no K split: these products have tiles in plenty
    return umma_gq_pair_launch(&it, 1, EPI_STORE, 0.f, FW_PROF_GQ, L->stream);
  }
  if (rows > 0x7fffffff) return FW_ERR_SHAPE;
  GemmGroup gg; gg.n = 1;
  GemmProblem& p = gg.p[0];
  memset(&p, 0, sizeof(p));
  p.A = In; p.B = Bmat; p.C = out; p.lda = M; p.ldb = M; p.ldc = M; p.m = (int32_t)rows; p.n = M; p.k = M;
  p.a_kmajor = 0; p.sym = 0; p.splits = 1; p.epi = EPI_STORE; p.colbias = colbias;
  p.nonfinite = L->h.iscal + IS_STATUS_NONFINITE;
  FW_CUDA(launch_gemm_ffma(gg, L->stream, FW_PROF_GQ), "rows x matrix (ffma)");
  return FW_OK;
}

static bool ranges_overlap(const void* a, const void* b, size_t bytes) {
  const uintptr_t x = (uintptr_t)a, y = (uintptr_t)b;
  return x < y + bytes && y < x + bytes;
}

fw_status fw_whiten_forward(fw_layer* L, const float* X, int64_t rows, float* Y) {
  if (!L || !X || !Y) return FW_ERR_INVALID_ARG;
  if (rows < 1) return FW_ERR_SHAPE;
  const int M = L->d.M;
  if (ranges_overlap(X, Y, (size_t)rows * M * sizeof(float))) return FW_ERR_INVALID_ARG;
  // Y = X T^T - 1 (T mu)^T: the product takes the stored T^T as it is (Y[r][j] = sum_k X[r][k] T^T[k][j]);
  // T mu = (T^T)^T mu goes into a recursion vector that is free outside fw_cond_reduce
  FW_CUDA(launch_matT_vec(L->h.Tt, L->h.mu, L->h.u, M, L->stream), "T mu");
  return rows_times_matrix(L, X, rows, L->h.Tt, L->h.u, Y);
}

fw_status fw_whiten_backward(fw_layer* L, const float* dY, int64_t rows, float* dX) {
  if (!L || !dY || !dX) return FW_ERR_INVALID_ARG;
  if (rows < 1) return FW_ERR_SHAPE;
  if (L->block_open) return FW_ERR_STATE;       // the Gram scratch holds nothing between calls, but keep it simple
  const int M = L->d.M;
  if (ranges_overlap(dY, dX, (size_t)rows * M * sizeof(float))) return FW_ERR_INVALID_ARG;
  // dX[r][k] = sum_j dY[r][j] T[j][k]: needs T row-major, built from T^T in the Gram scratch
  float* T = L->h.gram_part;
  FW_CUDA(launch_transpose(L->h.Tt, T, M, L->stream), "T from T^T");
  return rows_times_matrix(L, dY, rows, T, nullptr, dX);
}

fw_status fw_step(fw_layer* L, float* W, float* b, const float* G_t, const float* g_b, float lr) {
  if (!L || !W || !G_t) return FW_ERR_INVALID_ARG;
  if ((b == nullptr) != (g_b == nullptr)) return FW_ERR_INVALID_ARG;
  FW_CUDA(launch_axpy_step(W, G_t, lr, (int64_t)L->d.N * L->d.M, L->stream), "step W");
  if (b) FW_CUDA(launch_sgd_bias(b, g_b, lr, L->d.N, L->stream), "step b");
  return FW_OK;
}

fw_status fw_step_momentum(fw_layer* L, float* W, float* b, const float* G_t, const float* g_b, float* vW,
                           float* vb, float lr, float momentum, float weight_decay) {
  if (!L || !W || !G_t || !vW) return FW_ERR_INVALID_ARG;
  if (!((b == nullptr) == (g_b == nullptr) && (b == nullptr) == (vb == nullptr))) return FW_ERR_INVALID_ARG;
  if (!(momentum >= 0.f && momentum < 1.f) || !(weight_decay >= 0.f)) return FW_ERR_INVALID_ARG;
  FW_CUDA(launch_momentum_step(W, G_t, vW, lr, momentum, weight_decay, (int64_t)L->d.N * L->d.M, L->stream),
          "momentum step W");
  if (b) FW_CUDA(launch_momentum_step(b, g_b, vb, lr, momentum, 0.f, L->d.N, L->stream), "momentum step b");
  return FW_OK;
}

fw_status fw_whiteness(fw_layer* L, float* rho_out) {
  if (!L || !rho_out) return FW_ERR_INVALID_ARG;
  if (!L->have_cov) return FW_ERR_STATE;
  if (L->phiy_stale) {
    fw_status st = resync_phiy(&L, 1);
    if (st != FW_OK) return st;
  }
  FW_CUDA(launch_whiteness(L->h.Phiy, L->d.M, rho_out, L->stream), "whiteness");
  return FW_OK;
}

size_t fw_evd_scratch_bytes(int32_t M) { return (M >= 1 && M <= kMaxDim) ? evd_scratch_bytes(M) : 0; }

fw_status fw_group_evd_whiten(fw_layer* const* L, int32_t n, void* const* scratch, const size_t* scratch_bytes,
                              float g_max) {
  fw_status st = check_group(L, n);
  if (st != FW_OK) return st;
  if (!scratch || !scratch_bytes || !(g_max == g_max)) return FW_ERR_INVALID_ARG;
  const float* src[FW_MAX_GROUP];
  float* t_out[FW_MAX_GROUP]; float* q_out[FW_MAX_GROUP]; float* y_out[FW_MAX_GROUP];
  int32_t* status[FW_MAX_GROUP];
  int dims[FW_MAX_GROUP];
  float eps[FW_MAX_GROUP];
  for (int i = 0; i < n; ++i) {
    if (!L[i]->have_cov || L[i]->block_open) return FW_ERR_STATE;
    if (!scratch[i] || (reinterpret_cast<uintptr_t>(scratch[i]) & 255u)) return FW_ERR_INVALID_ARG;
    if (scratch_bytes[i] < evd_scratch_bytes(L[i]->d.M)) return FW_ERR_WORKSPACE;
    src[i] = L[i]->h.Phix; t_out[i] = L[i]->h.Tt; q_out[i] = L[i]->h.Q; y_out[i] = L[i]->h.Phiy;
    status[i] = L[i]->h.iscal + IS_STATUS_TIMEOUT;
    dims[i] = L[i]->d.M; eps[i] = L[i]->d.eps;
  }
  cudaStream_t s = L[0]->stream;
  FW_CUDA(launch_evd(n, src, dims, scratch, status, eps, true, g_max, t_out, q_out, y_out, nullptr, nullptr, s),
          "evd whitening");
  GroupDev g; int max_M, max_N;
  fill_group(L, n, g, max_M, max_N);
  bool any_beta = false;
  for (int i = 0; i < n; ++i) any_beta |= (L[i]->d.beta > 0.f);
  if (any_beta) FW_CUDA(launch_smooth(g, max_M, s), "smooth");          // Eq. 35
  for (int i = 0; i < n; ++i) {
    L[i]->t_identity = false;
    // a leaky layer also tracks P = T Phi_x: the next reduction rebuilds it (and Phi_y) from T
    L[i]->phiy_stale = (L[i]->d.gamma != 1.0f);
  }
  return FW_OK;
}

fw_status fw_evd_whiten(fw_layer* L, void* scratch, size_t scratch_bytes, float g_max) {
  if (!L) return FW_ERR_INVALID_ARG;
  return fw_group_evd_whiten(&L, 1, &scratch, &scratch_bytes, g_max);
}

fw_status fw_spectrum(fw_layer* L, int32_t which, void* scratch, size_t scratch_bytes, float* lam_out,
                      float* kappa_out) {
  if (!L || (which != 0 && which != 1) || !scratch || (reinterpret_cast<uintptr_t>(scratch) & 255u))
    return FW_ERR_INVALID_ARG;
  if (!lam_out && !kappa_out) return FW_ERR_INVALID_ARG;
  if (!L->have_cov || L->block_open) return FW_ERR_STATE;
  if (scratch_bytes < evd_scratch_bytes(L->d.M)) return FW_ERR_WORKSPACE;
  if (which == 1 && L->phiy_stale) {
    fw_status st = resync_phiy(&L, 1);
    if (st != FW_OK) return st;
  }
  const float* src = which ? L->h.Phiy : L->h.Phix;
  int32_t* status = L->h.iscal + IS_STATUS_TIMEOUT;
  const int M = L->d.M;
  const float eps = L->d.eps;
  float* const* lo = lam_out ? &lam_out : nullptr;
  float* const* ko = kappa_out ? &kappa_out : nullptr;
  FW_CUDA(launch_evd(1, &src, &M, &scratch, &status, &eps, false, 0.f, nullptr, nullptr, nullptr, lo, ko, L->stream),
          "spectrum");
  return FW_OK;
}

fw_status fw_group_grad_transform_step(fw_layer* const* L, int32_t n, const float* const* G, float* const* W,
                                       float* const* b, const float* const* g_b, float lr) {
  fw_status st = check_group(L, n);
  if (st != FW_OK) return st;
  if (!G || !W) return FW_ERR_INVALID_ARG;
  if ((b == nullptr) != (g_b == nullptr)) return FW_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) {
    if (!G[i] || !W[i] || (const float*)W[i] == G[i]) return FW_ERR_INVALID_ARG;
    if (b && ((b[i] == nullptr) != (g_b[i] == nullptr))) return FW_ERR_INVALID_ARG;
  }
  st = grad_transform_impl(L, n, G, W, EPI_SGD, lr);
  if (st != FW_OK) return st;
  if (b) {
    GroupDev g; int max_M, max_N;
    fill_group(L, n, g, max_M, max_N);
    PtrTable bt, gt;
    memset(&bt, 0, sizeof(bt)); memset(&gt, 0, sizeof(gt));
    for (int i = 0; i < n; ++i) { bt.p[i] = b[i]; gt.p[i] = g_b[i]; }
    FW_CUDA(launch_sgd_bias_group(g, bt, gt, lr, max_N, L[0]->stream), "step b");
  }
  return FW_OK;
}

static float* field_ptr(fw_layer* L, fw_field f, size_t* bytes) {
  const size_t M = (size_t)L->d.M;
  const size_t vec = M * sizeof(float), mat = M * M * sizeof(float);
  switch (f) {
    case FW_F_MU: *bytes = vec; return L->h.mu;
    case FW_F_PHIX: *bytes = mat; return L->h.Phix;
    case FW_F_PHI_DIAG: *bytes = vec; return L->h.phi;
    case FW_F_LAMBDA_BAR: *bytes = sizeof(float); return L->h.scal + SC_LAMBDA_BAR;
    case FW_F_T: *bytes = mat; return L->h.Tt;
    case FW_F_Q: *bytes = mat; return L->h.Q;
    case FW_F_QS: *bytes = mat; return L->h.Qs;
    case FW_F_PHIY: *bytes = mat; return L->h.Phiy;
    case FW_F_ALIGN_W: *bytes = vec; return L->h.wvec;
  }
  *bytes = 0;
  return nullptr;
}

fw_status fw_layer_get(fw_layer* L, fw_field f, void* dev_dst, size_t bytes) {
  if (!L || !dev_dst) return FW_ERR_INVALID_ARG;
  size_t need = 0;
  float* src = field_ptr(L, f, &need);
  if (!src) return FW_ERR_INVALID_ARG;
  if (bytes < need) return FW_ERR_SHAPE;
  if (f == FW_F_PHIY && L->phiy_stale) {
    if (!L->have_cov) return FW_ERR_STATE;
    fw_status st = resync_phiy(&L, 1);
    if (st != FW_OK) return st;
  }
  if (f == FW_F_T) {
    FW_CUDA(launch_transpose(L->h.Tt, (float*)dev_dst, L->d.M, L->stream), "get T");
    return FW_OK;
  }
  FW_CUDA(cudaMemcpyAsync(dev_dst, src, need, cudaMemcpyDeviceToDevice, L->stream), "fw_layer_get");
  return FW_OK;
}

fw_status fw_layer_set(fw_layer* L, fw_field f, const void* dev_src, size_t bytes) {
  if (!L || !dev_src) return FW_ERR_INVALID_ARG;
  size_t need = 0;
  float* dst = field_ptr(L, f, &need);
  if (!dst) return FW_ERR_INVALID_ARG;
  if (bytes < need) return FW_ERR_SHAPE;
  if (f == FW_F_ALIGN_W) return FW_ERR_INVALID_ARG;
  const int M = L->d.M;
  if (f == FW_F_T) {
    FW_CUDA(launch_transpose((const float*)dev_src, L->h.Tt, M, L->stream), "set T");
    // Q = T^T T = Tt Tt^T: A = Tt (m x k), B[k][j] = Tt[j][k] = T[k][j]
    GemmGroup g; g.n = 1;
    GemmProblem& p = g.p[0];
    memset(&p, 0, sizeof(p));
    p.A = L->h.Tt; p.B = dev_src; p.C = L->h.Q;
    p.lda = p.ldb = p.ldc = M; p.m = p.n = M; p.k = M;
    p.a_kmajor = 0; p.sym = 1; p.splits = 1; p.epi = EPI_SYMM;
    FW_CUDA(launch_gemm_ffma(g, L->stream, FW_PROF_MISC), "set T: Q");
    L->t_identity = false;
    L->phiy_stale = true;
    return FW_OK;
  }
  FW_CUDA(cudaMemcpyAsync(dst, dev_src, need, cudaMemcpyDeviceToDevice, L->stream), "fw_layer_set");
  if (f == FW_F_PHIX) {
    FW_CUDA(launch_trace_lambda(L->dev, M, L->stream), "set Phix: lam_bar");
    L->have_cov = true; L->first_block = false; L->phiy_stale = true;
  } else if (f == FW_F_PHIY) {
    // a leaky layer also tracks (T Phix)^T, which an injected Phiy does not provide: it stays stale
    L->phiy_stale = (L->d.gamma != 1.0f);
  }
  return FW_OK;
}

fw_status fw_layer_sync_status(fw_layer* L) {
  if (!L) return FW_ERR_INVALID_ARG;
  int32_t is[IS_COUNT];
  FW_CUDA(cudaMemcpyAsync(is, L->h.iscal, sizeof(is), cudaMemcpyDeviceToHost, L->stream), "status read");
  FW_CUDA(cudaStreamSynchronize(L->stream), "status sync");
  if (is[IS_STATUS_NONFINITE] || is[IS_STATUS_NOSUB] || is[IS_STATUS_TIMEOUT]) {
    FW_CUDA(cudaMemsetAsync(L->h.iscal + IS_STATUS_NOSUB, 0, 3 * sizeof(int32_t), L->stream), "status clear");
  }
  if (is[IS_STATUS_TIMEOUT]) {
    // a persistent launch this layer led may have left its barrier counter short: start it afresh
    FW_CUDA(cudaMemsetAsync(L->h.iscal + IS_GRID_BAR, 0, 2 * sizeof(int32_t), L->stream), "barrier clear");
    L->bar_base = 0;
  }
  if (is[IS_STATUS_TIMEOUT]) return FW_ERR_TIMEOUT;
  if (is[IS_STATUS_NONFINITE]) return FW_WARN_NONFINITE;
  if (is[IS_STATUS_NOSUB]) return FW_WARN_NO_SUBSPACE;
  return FW_OK;
}

fw_status fw_debug_wait_probe(fw_layer* L, uint32_t polls) {
  if (!L) return FW_ERR_INVALID_ARG;
  if (polls < 1 || polls > (1u << 16)) return FW_ERR_INVALID_ARG;
  FW_CUDA(launch_wait_probe(L->h.iscal + IS_STATUS_TIMEOUT, polls, L->stream), "wait probe");
  return FW_OK;
}

const char* fw_status_string(fw_status s) {
  switch (s) {
    case FW_OK: return "ok";
    case FW_ERR_INVALID_ARG: return "invalid argument";
    case FW_ERR_SHAPE: return "unsupported shape";
    case FW_ERR_STATE: return "call order: no covariance yet";
    case FW_ERR_WORKSPACE: return "workspace too small or misaligned";
    case FW_ERR_CUDA: return "CUDA error (or no CUDA device)";
    case FW_ERR_TIMEOUT: return "device-side wait timed out";
    case FW_ERR_UNSUPPORTED: return "not supported by this build";
    case FW_WARN_NO_SUBSPACE: return "a step found no usable subspace";
    case FW_WARN_NONFINITE: return "non-finite values seen";
  }
  return "unknown status";
}

int32_t fw_version(void) { return 100; }

}  // extern "C"
