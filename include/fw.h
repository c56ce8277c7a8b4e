/*
 * fw.h -- C ABI of the feature-whitening-by-gradient-transformation hot path
 * for NVIDIA B200 (sm_100a).
 *
 * Method: "Feature Whitening via Gradient Transformation for Improved
 * Convergence" (arXiv 2010.01546).  Per layer and per batch the library
 *   (a) folds a block of layer inputs into the running mean, covariance and
 *       feature power                                   (Sec. 2, Eqs. 2-5; Eqs. 37-38),
 *   (b) runs the recursive condition-number reduction that builds the
 *       whitening transform T and Q = T^T T             (Sec. 4, Eqs. 36-50),
 *   (c) multiplies the weight gradient by the smoothed Q and applies the SGD
 *       step                                            (Sec. 3.1, Eqs. 27-30; Eq. 35).
 *
 * Notation (im2col form): a layer input is a patch vector of length M, the
 * layer is z = W (x - mu) + b with W of shape N x M (the paper's S is N here).
 * X holds one patch per row: rows = B*H*W, leading dimension ldx >= M.
 *
 * Conventions
 *  - Every pointer except fw_layer*, fw_layer_desc* and the arrays of a
 *    grouped call (layer handles, pointer tables, row counts: HOST arrays of
 *    DEVICE pointers) is a DEVICE pointer owned by the caller.  Matrices are
 *    dense row-major fp32 unless stated; X may be bf16.
 *  - The library never allocates or frees device memory.  All per-layer state
 *    and scratch live in the caller-supplied workspace, which must outlive the
 *    layer and be 256-byte aligned.
 *  - Compute calls validate their arguments on the host, return an error code
 *    synchronously and launch nothing on error; otherwise they enqueue work on
 *    the layer's CUDA stream and return without waiting.  Conditions found on
 *    the device (non-finite input, a step with no usable subspace, a bounded
 *    wait that gave up) are kept in a per-layer status word in the layer's own
 *    workspace, read by fw_layer_sync_status; no kernel reports through
 *    process-wide state.
 *  - A layer is not thread-safe.  Calls on different layers are independent;
 *    a grouped call requires all its layers to share one stream.
 *  - There is no CPU fallback: without a CUDA device every compute call
 *    returns FW_ERR_CUDA.
 */
#ifndef FW_H_
#define FW_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fw_layer fw_layer; /* opaque host object owned by the library */

typedef enum {
  FW_OK = 0,
  FW_ERR_INVALID_ARG = 1, /* null pointer, negative count, bad enum            */
  FW_ERR_SHAPE = 2,       /* M, N, rows, ld outside the supported range        */
  FW_ERR_STATE = 3,       /* call order: e.g. reduction before any covariance  */
  FW_ERR_WORKSPACE = 4,   /* workspace too small or misaligned                 */
  FW_ERR_CUDA = 5,        /* a CUDA runtime call failed                        */
  FW_ERR_TIMEOUT = 6,     /* a bounded device-side wait gave up                */
  FW_ERR_UNSUPPORTED = 7, /* valid request this build has no kernel for        */
  FW_WARN_NO_SUBSPACE = 64, /* some step found no coherent column set: a_e = 0 */
  FW_WARN_NONFINITE = 65    /* NaN/Inf seen in X, G or the state               */
} fw_status;

typedef enum { FW_F32 = 0, FW_BF16 = 1 } fw_dtype; /* element type of X */

/* Engine of the two dense contractions (X^T X and G Q) and of the re-sync
 * products.  FP32: FFMA, matches an fp64 reference to ~1e-6.  TF32 / BF16:
 * tcgen05 tensor cores with fp32 accumulation (TF32 for fp32 X, BF16 for bf16
 * X), matches to ~1e-3.  The recursion itself is always fp32. */
typedef enum { FW_PREC_FP32 = 0, FW_PREC_TF32 = 1, FW_PREC_BF16 = 2 } fw_prec;

/* Start vector of the power iterations: the column-alignment estimate of
 * Sec. 4.2 (Eqs. 45-50), or simply the largest-norm column normalised. */
typedef enum { FW_INIT_ALIGN = 0, FW_INIT_MAXCOL = 1 } fw_init;

typedef struct {
  int32_t M, N;      /* input features (patch length), output features          */
  int32_t x_dtype;   /* fw_dtype                                                 */
  int32_t prec;      /* fw_prec                                                  */
  int32_t init;      /* fw_init                                                  */
  float alpha;       /* inter-block averaging of the moments, Eqs. 2-3, 37      */
  float beta;        /* smoothing of Q, Eq. 35                                   */
  float gamma;       /* leakage of the transform, Eq. 42 (0 < gamma <= 1)       */
  float delta;       /* power-reduction target, Eq. 40                           */
  float eps;         /* floor of the denominator in Eq. 40                       */
  float c_rel;       /* relative coherence threshold, Eq. 48                     */
  float c_abs;       /* absolute coherence threshold, Eq. 48                     */
} fw_layer_desc;

/* Fills *d with the recursive method's hyper-parameters of Sec. 6
 * (alpha 0.1, beta 0.1, gamma 0.99, delta 0.25, c_rel 0.025, c_abs 1e-6,
 * eps 1e-5), fp32 X, FP32 engine, alignment start vector. */
void fw_layer_desc_default(fw_layer_desc* d, int32_t M, int32_t N);

/* Device bytes a layer of this description needs (state + scratch); 0 if the
 * description is invalid.  Supported: 1 <= M <= 8192, 1 <= N <= 8192. */
size_t fw_layer_workspace_bytes(const fw_layer_desc* d);

/* Creates a layer in the given workspace and enqueues its initialisation on
 * `cuda_stream` (a cudaStream_t, may be 0): T = Q = Qs = I, mu = 0, no block
 * seen yet (Eqs. 12-13; Qs(-1) = I of Sec. 3.2).  The handle is host memory
 * owned by the library until fw_layer_destroy. */
fw_status fw_layer_create(const fw_layer_desc* d, void* dev_workspace, size_t bytes,
                          void* cuda_stream, fw_layer** out);

/* Frees the host object only; the workspace stays the caller's. */
fw_status fw_layer_destroy(fw_layer* L);

/* Puts the layer back into the state fw_layer_create leaves it in (T = Q = Qs
 * = I, mu = 0, no block seen, no open block, status cleared), in the same
 * workspace, on the layer's stream.  Attached parameters stay attached. */
fw_status fw_layer_reset(fw_layer* L);

/* Optional.  Attaches the layer's parameters (W: N x M, b: N, device fp32) so
 * that fw_cov_update can compensate the bias for the change of the running
 * mean (Eq. 31: b += W (mu_new - mu_old), the sign that leaves
 * z = W (x - mu) + b unchanged).  Pass NULLs to detach. */
fw_status fw_layer_attach_params(fw_layer* L, float* W, float* b);

/* (a) Moments of one block of patch rows (Eqs. 2-5, 37-38).
 * X: rows x M, row-major, leading dimension ldx (elements), fp32 or bf16 per
 * the description.  Computes X^T X and the column sums in one pass over X,
 * then mu, Phi_x (centred on the updated running mean, normalised by the
 * block's rows), phi and lam_bar; the first block sets them, later blocks
 * average with alpha.  Marks the whitened covariance Phi_y = T Phi_x T^T stale.
 *
 * flags: a block may span several calls (Sec. 2: the moments are computed "in
 * blocks of L batches").  FW_COV_ACCUMULATE adds this call's X^T X, column
 * sums and row count to the open block and changes no moment; FW_COV_COMMIT
 * (the default, 0) adds this call's rows and closes the block: mu, Phi_x, phi
 * and the bias compensation then see all rows accumulated since the last
 * commit, exactly as if they had been passed in one call.  The pilot shift
 * that centres short fp32 blocks inside the Gram pass is fixed by the block's
 * first call.
 * rows must be >= 1; ldx >= M; for the tensor-core engines X must be 16-byte
 * aligned and ldx * sizeof(element) a multiple of 16. */
#define FW_COV_COMMIT 0u
#define FW_COV_ACCUMULATE 1u
fw_status fw_cov_update(fw_layer* L, const void* X, int64_t rows, int64_t ldx, uint32_t flags);

/* (a) from the activation itself.  The layer input of a convolution is "any
 * spatial dimension vectorised" (Sec. 2): patch rows of length M = C k k cut
 * from an NHWC activation A[B][H][W][C] (stride 1, zero padding (k - 1) / 2,
 * columns ordered (ky, kx, c)).  These calls take A and never materialise the
 * patch matrix, which for k = 3 is nine times the activation: the Gram kernel
 * reads shifted windows of a zero-padded copy of A.  Semantics, flags and
 * results are those of fw_cov_update on the patch matrix of rows = B H W.
 *   k = 1: A is the patch matrix; no scratch is needed.
 *   k = 3: scratch (device, caller-owned, 256-byte aligned, at least
 *          fw_nhwc_scratch_bytes bytes, free again when the call's work on the
 *          stream is done) holds the padded copy.  Needs a tensor-core layer
 *          with fp32 X (FW_PREC_TF32), C a multiple of 4, and H divisible by
 *          the image rows a pipeline stage covers (any power-of-two H; 14 and
 *          28 also); otherwise FW_ERR_UNSUPPORTED and the caller falls back to
 *          fw_cov_update on a patch matrix of its own. */
size_t fw_nhwc_scratch_bytes(int32_t B, int32_t H, int32_t W, int32_t C, int32_t k);
fw_status fw_cov_update_nhwc(fw_layer* L, const float* A, int32_t B, int32_t H, int32_t W, int32_t C, int32_t k,
                             void* scratch, size_t scratch_bytes, uint32_t flags);
/* HOST arrays of length n, as in the other grouped calls. */
fw_status fw_group_cov_update_nhwc(fw_layer* const* L, int32_t n, const float* const* A, const int32_t* B,
                                   const int32_t* H, const int32_t* W, const int32_t* C, const int32_t* k,
                                   void* const* scratch, const size_t* scratch_bytes, uint32_t flags);

/* (b) K steps of the recursion of Sec. 4 on the current moments, each with P
 * power iterations refining the subspace estimate (P = 0: the estimate of
 * Sec. 4.2 as it is), then one smoothing update of Qs (Eq. 35).  Per step:
 * xi, m' (Eqs. 45-46); c (Eq. 47); coherent set and aligned average
 * (Eqs. 48-50); v <- Phi_y v / ||Phi_y v||, P times; lambda_e = v^T Phi_y v
 * (Eq. 36); g_e, a_e (Eqs. 40-41); t = T^T v; rank-one updates of Q (Eq. 44),
 * T (Eq. 42) and Phi_y, with the leakage gamma of the description (gamma < 1
 * additionally tracks T Phi_x so that Phi_y stays T Phi_x T^T at O(M^2) per
 * step).  Runs entirely on the device.
 * trace_or_null: K x 4 device floats (lambda_e, g_e, |set|, m') per step.
 * K = 0 takes no step and leaves T, Q, Qs alone; it only brings Phi_y =
 * T Phi_x T^T up to date when the moments changed since the last call.
 * Requires a covariance (FW_ERR_STATE otherwise). */
fw_status fw_cond_reduce(fw_layer* L, int32_t K, int32_t P, float* trace_or_null);

/* (c) G_out = G Qs (Eq. 29 with the smoothed Q of Eq. 35).  G, G_out: N x M.
 * G_out may be G itself (in place: the product is formed in the layer's
 * workspace and copied over G); any other overlap of the two arrays is
 * rejected with FW_ERR_INVALID_ARG. */
fw_status fw_grad_transform(fw_layer* L, const float* G, float* G_out);

/* The direct method the gradient transformation replaces (Sec. 2), for
 * comparison: every sample is whitened on the way forward and its gradient is
 * sent back through the transform, two rows x M x M products per batch where
 * fw_grad_transform does one N x M x M product.  Same engine as fw_grad_transform.
 *   fw_whiten_forward   Y  = (X - 1 mu^T) T^T      (Eq. 11), X, Y: rows x M fp32
 *   fw_whiten_backward  dX = dY T                   (Eq. 14), dY, dX: rows x M fp32
 * with the layer's current mu and T.  Outputs may not overlap inputs.
 * fw_whiten_backward builds T (the library keeps T^T) in the Gram scratch of
 * the layer's workspace. */
fw_status fw_whiten_forward(fw_layer* L, const float* X, int64_t rows, float* Y);
fw_status fw_whiten_backward(fw_layer* L, const float* dY, int64_t rows, float* dX);

/* SGD step W <- W - lr G_t, b <- b - lr g_b (Eqs. 27-28; the bias gradient is
 * not transformed).  g_b and b may both be NULL to skip the bias. */
fw_status fw_step(fw_layer* L, float* W, float* b, const float* G_t, const float* g_b, float lr);

/* SGD with momentum and weight decay, the optimiser of the paper's experiments
 * (Sec. 6: momentum 0.9, weight decay 5e-4 / 1e-4), applied to the transformed
 * gradient:  v <- momentum v + (G_t + weight_decay W),  W <- W - lr v, and the
 * same for the bias with its untransformed gradient (no decay on the bias).
 * vW (N x M) and vb (N) are the caller's velocity buffers, zero before the
 * first step; b, g_b, vb may all be NULL.  momentum = weight_decay = 0 is fw_step. */
fw_status fw_step_momentum(fw_layer* L, float* W, float* b, const float* G_t, const float* g_b, float* vW,
                           float* vb, float lr, float momentum, float weight_decay);

/* Whitening from the eigenvalue decomposition (Sec. 2, Eqs. 7-10; Sec. 3.2,
 * Eqs. 32, 34, 35): the direct construction the recursion of Sec. 4 replaces.
 * Phi_x = V Lambda V^T is computed on the device (one-sided Jacobi rotations in
 * fp64, all layers of a group in one cooperative launch) and the layer's state is
 * set to  T = V diag(sqrt g) V^T (the symmetric, "ZCA" whitening matrix, Eq. 9),
 * Q = T^T T, Phi_y = T Phi_x T^T, Qs <- beta Qs + (1 - beta) Q (Eq. 35), with gains
 *   g_max <= 0:  g_m = 1 / max(lambda_m, eps)                            (Eq. 10)
 *   g_max  > 0:  g_m = min(1 / (M lbar_m), g_max) for the Ms_hat largest
 *                eigenvalues, 1 for the others, lbar = lambda / sum lambda,
 *                Ms_hat = round(exp(-sum lbar log lbar)) in [1, M]      (Eqs. 32, 34;
 *                Eq. 32 in the reading that gives M for equal eigenvalues and 1
 *                for a single dominant one, as the text states).
 * The gradient transform, the step and a later fw_cond_reduce continue from this
 * state.  scratch: caller-owned device memory, 256-byte aligned, at least
 * fw_evd_scratch_bytes(M) bytes per layer, used only during the call's kernels.
 * Cost: about 12 M^3 fp64 operations per sweep and 6-10 sweeps; M - 1 grid
 * barriers per sweep (bounded waits; a time-out is reported by
 * fw_layer_sync_status as FW_ERR_TIMEOUT).  Errors: FW_ERR_STATE without a
 * covariance or inside an open block, FW_ERR_WORKSPACE for a short scratch. */
size_t fw_evd_scratch_bytes(int32_t M);
fw_status fw_evd_whiten(fw_layer* L, void* scratch, size_t scratch_bytes, float g_max);
fw_status fw_group_evd_whiten(fw_layer* const* L, int32_t n, void* const* scratch, const size_t* scratch_bytes,
                              float g_max);

/* Eigenvalues of Phi_x (which = 0) or Phi_y (which = 1) in decreasing order to
 * lam_out (M device floats, may be NULL) and the normalised rank of Sec. 6,
 * kappa = exp(-sum lbar log lbar) / M, to kappa_out (one device float, may be
 * NULL).  Same decomposition and scratch as fw_evd_whiten; the layer's state is
 * not changed (Phi_y is brought up to date first when it is stale). */
fw_status fw_spectrum(fw_layer* L, int32_t which, void* scratch, size_t scratch_bytes, float* lam_out,
                      float* kappa_out);

/* Whiteness of the transformed input (Sec. 6, Eq. 51):
 * rho = M / sum_{m,m'} Phi_y[m][m']^2 / (Phi_y[m][m] Phi_y[m'][m']), the sum over
 * all pairs (1 for a diagonal Phi_y, 1/M for fully correlated features).
 * Writes one float to rho_out (device).  Requires a covariance. */
fw_status fw_whiteness(fw_layer* L, float* rho_out);

/* Grouped forms: the same operations over n layers in one launch sequence.
 * All arrays are HOST arrays of length n; the pointers inside are device
 * pointers.  n <= FW_MAX_GROUP; all layers must share a stream. */
#define FW_MAX_GROUP 64
fw_status fw_group_cov_update(fw_layer* const* L, int32_t n, const void* const* X,
                              const int64_t* rows, const int64_t* ldx, uint32_t flags);
fw_status fw_group_cond_reduce(fw_layer* const* L, int32_t n, int32_t K, int32_t P,
                               float* const* traces_or_null);
/* Fused (c): W <- W - lr (G Qs), b <- b - lr g_b for every layer.  b / g_b
 * tables may be NULL. */
fw_status fw_group_grad_transform_step(fw_layer* const* L, int32_t n, const float* const* G,
                                       float* const* W, float* const* b,
                                       const float* const* g_b, float lr);

/* First-block mean and covariance of `rows` patch rows without any workspace:
 * mu_out[M] = column means, phix_out[M x M] = (1/rows) sum (x - mu)(x - mu)^T,
 * i.e. what fw_cov_update leaves in FW_F_MU / FW_F_PHIX on a fresh layer.
 * (The paper has no counterpart for this entry point; it exists for callers
 * that cannot allocate.)  X: rows x M fp32, row-major, leading dimension ldx;
 * mu_out, phix_out: device fp32; cuda_stream: a cudaStream_t, may be 0.
 *
 * For callers that may not allocate device memory and therefore cannot give a
 * layer its workspace -- e.g. a hook running inside a framework whose caching
 * allocator owns the whole device, where a raw cudaMalloc would synchronise the
 * device and may fail.  The call allocates nothing, neither on the device nor
 * through any library: its split partial sums go to a fixed 8 MiB array inside
 * the library image, which every GPU that loads the library holds until the
 * process exits.
 *  - M <= FW_STATIC_MAX_M; a larger M returns FW_ERR_SHAPE with a message.
 *  - The first call on each device resolves the array's device address (with
 *    that device current); make that first call before any stream capture.
 *  - All calls share the one array, and it keeps the previous call's contents.
 *    Every slot a call reads it has written first, so nothing needs clearing,
 *    but two calls that overlap on the GPU (different streams, or different
 *    host threads) race on it: serialise them. */
#define FW_STATIC_MAX_M 256
fw_status fw_cov_block_static(const float* X, int64_t rows, int64_t ldx, int32_t M, float* mu_out,
                              float* phix_out, void* cuda_stream);

/* State access (checkpointing, injecting a covariance, parity checks).
 * Matrices are M x M fp32 row-major, vectors M fp32, FW_F_LAMBDA_BAR one fp32.
 * Copies run on the layer's stream.  Setting FW_F_PHIX marks Phi_y stale, sets
 * lam_bar = trace(Phi_x)/M and counts as a first block having been seen;
 * setting FW_F_T also recomputes Q = T^T T and marks Phi_y stale. */
typedef enum {
  FW_F_MU = 0, FW_F_PHIX = 1, FW_F_PHI_DIAG = 2, FW_F_LAMBDA_BAR = 3,
  FW_F_T = 4, FW_F_Q = 5, FW_F_QS = 6, FW_F_PHIY = 7,
  FW_F_ALIGN_W = 8 /* get only: alignment weights of the last step, 1/c_m on the coherent set, else 0 */
} fw_field;
fw_status fw_layer_get(fw_layer* L, fw_field f, void* dev_dst, size_t bytes);
fw_status fw_layer_set(fw_layer* L, fw_field f, const void* dev_src, size_t bytes);

/* Waits for the layer's stream, then returns (and clears) the first
 * device-side condition recorded since the last call, or FW_OK. */
fw_status fw_layer_sync_status(fw_layer* L);

const char* fw_status_string(fw_status s);

/* Test aid for the time-out path (the paper has no counterpart).  Enqueues on
 * the layer's stream a one-warp kernel that waits on a barrier nothing arrives
 * on, with the same bounded wait the tensor-core pipelines use but a limit of
 * `polls` polls (1 .. 65536, microseconds in all).  The wait gives up, the
 * kernel records it in the layer's status word and returns normally, so the
 * next fw_layer_sync_status returns FW_ERR_TIMEOUT and the layer stays usable.
 * Nothing traps and nothing hangs. */
fw_status fw_debug_wait_probe(fw_layer* L, uint32_t polls);

/* Per-kernel-class device timing (a tracing aid; the paper has no counterpart).
 * Between fw_profile_begin and fw_profile_end every kernel launch of the
 * library is bracketed by CUDA events on its stream.  fw_profile_end waits for
 * them and writes, per class, the summed device time in milliseconds and the
 * number of launches into HOST arrays of length FW_PROF_CLASSES (either may be
 * NULL).  Off by default; event recording perturbs back-to-back launches a
 * little, so whole-step timings are taken with profiling off. */
typedef enum {
  FW_PROF_PILOT = 0,    /* pilot column means                         */
  FW_PROF_GRAM = 1,     /* X^T X + column sums                        */
  FW_PROF_MOMENTS = 2,  /* split reduction, centring, running average */
  FW_PROF_RESYNC = 3,   /* T Phi_x T^T products                       */
  FW_PROF_RECUR_MV = 4, /* matrix-vector passes of the recursion      */
  FW_PROF_RECUR_UPD = 5,/* rank-update pass over Q, T, Phi_y          */
  FW_PROF_SMOOTH = 6,   /* Qs update                                  */
  FW_PROF_GQ = 7,       /* G Qs (+ SGD epilogue)                      */
  FW_PROF_MISC = 8,
  FW_PROF_RECUR_CHIP = 9, /* whole K-step recursion of small layers, on chip */
  FW_PROF_CLASSES = 10
} fw_prof_class;
fw_status fw_profile_begin(void);
fw_status fw_profile_end(float* ms_per_class, int64_t* launches_per_class);

/* Tuning aids: environment variables read once, when the first call needs them.
 * None changes results; they exist for measurements.
 *   FW_PAIR_MIN_M   smallest M the CTA-pair Gram / re-sync kernels take (default 289)
 *   FW_PAIR_SPLITS  row slabs per problem of the CTA-pair kernels (default: chosen by the scheduler)
 *   FW_PAIR_DEBUG   print the chosen slabs to stderr
 *   FW_PASS_SHAPE   42 / 24 / 18 / 41: shape of the streaming recursion passes (default: by row-block count)
 *   FW_PERSIST_MAX_MB  largest total state (MB, 4 M^2 over the large layers of a call) whose recursion runs as one
 *                   persistent launch (default 512; 0: one launch per pass always)
 *   FW_GRAM_WAVES_PCT  CTAs of a single-CTA Gram launch in percent of the SM count (default 200: two waves) */

/* 1 when fw_cond_reduce keeps this layer's Phi_y in distributed shared memory
 * for all K steps of a call (small M, gamma = 1), 0 when it streams the state
 * from HBM pass by pass.  Reporting aid: the two paths are bound by different
 * things (latency of dependent passes vs HBM bandwidth). */
int32_t fw_recursion_on_chip(const fw_layer_desc* d);

/* Number of kernels this library has launched since it was loaded. */
int64_t fw_launch_count(void);

/* Library version (major * 100 + minor). */
int32_t fw_version(void);

#ifdef __cplusplus
}
#endif
#endif /* FW_H_ */
