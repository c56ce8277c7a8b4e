"""fp64 CPU oracle for feature whitening by gradient transformation.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, obviously-correct
statement of what the hot path computes, written from the paper
("Feature Whitening via Gradient Transformation for Improved Convergence",
arXiv 2010.01546).  Only the test-suite, the smoke check and the benchmark's
CPU-baseline leg may import it; the CUDA library never does, shares no code
with it, and must fail loudly when its extension is missing rather than fall
back to anything in here.

Everything is numpy float64.  Each routine follows the paper's definition step
by step with no blocking, fusion, incremental shortcut or reordering: the
whitened covariance is recomputed densely as T Phi_x T^T at every recursion
step, covariances are two-pass, and a library matmul / eigensolver is used only
as a single step where the paper writes a product or an EVD.

Notation (im2col form): a layer input is a patch vector x of length M, the
layer is z = W (x - mu) + b with W of shape N x M; X holds one patch per row
(rows = B*H*W).  The paper's S (output features) is N here, and the paper's
sums over spatial positions n, r are folded into the patch rows.

Parity pins: every routine below is pinned by tests/test_oracle_pins.py against
closed forms, invariants the paper states, brute force on tiny sizes or an
independent library routine.  The paper prints no worked numerical example, so
there is no golden vector taken from it; the pins are the mathematical ones
listed in that test file.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

INIT_ALIGN = 0   # start vector = the paper's column-alignment estimate (Sec. 4.2)
INIT_MAXCOL = 1  # start vector = the largest-norm column, normalised


# =============================================================================
# state
# =============================================================================
@dataclass
class Hyper:
    """Hyper-parameters; defaults are the recursive method's of Sec. 6."""
    alpha: float = 0.1     # inter-block averaging of the moments, Eqs. 2-3, 37
    beta: float = 0.1      # smoothing of Q, Eq. 35
    gamma: float = 0.99    # leakage, Eq. 42
    delta: float = 0.25    # power-reduction target, Eq. 40
    eps: float = 1e-5      # floor of the denominator, Eqs. 10, 40
    c_rel: float = 0.025   # relative coherence threshold, Sec. 4.2
    c_abs: float = 1e-6    # absolute coherence threshold, Sec. 4.2
    init: int = INIT_ALIGN


@dataclass
class Layer:
    M: int
    N: int
    hp: Hyper = field(default_factory=Hyper)
    mu: np.ndarray = None
    Phix: np.ndarray = None
    phi: np.ndarray = None
    lam_bar: float = 0.0
    T: np.ndarray = None
    Q: np.ndarray = None
    Qs: np.ndarray = None
    first: bool = True
    W: np.ndarray = None
    b: np.ndarray = None

    def __post_init__(self):
        M = self.M
        # Initialisation: T(-1) = I, mu(-1) = 0 (Eqs. 12-13), Qs(-1) = I (Sec. 3.2).
        self.mu = np.zeros(M)
        self.Phix = np.zeros((M, M))
        self.phi = np.zeros(M)
        self.T = np.eye(M)
        self.Q = np.eye(M)
        self.Qs = np.eye(M)

    def attach_params(self, W, b):
        self.W = np.array(W, dtype=np.float64)
        self.b = np.array(b, dtype=np.float64)

    def set_phix(self, Phix, lam_bar=None):
        """Inject a covariance directly (no samples).  The mean feature power
        is then taken as trace(Phix)/M, which is what Eqs. 37-38 give for
        zero-mean inputs, unless it is supplied."""
        self.Phix = np.array(Phix, dtype=np.float64)
        self.lam_bar = float(np.trace(self.Phix) / self.M) if lam_bar is None else float(lam_bar)
        self.first = False

    def phiy(self):
        """Covariance of the whitened input y = T (x - mu): T Phi_x T^T."""
        return self.T @ self.Phix @ self.T.T


# =============================================================================
# (a) moments: Eqs. 2-5 (mean, covariance), Eqs. 37-38 (feature power)
# =============================================================================
def cov_update(L: Layer, X: np.ndarray) -> None:
    """One block of samples.  Running mean (Eq. 2; first block Eq. 4), running
    covariance centred on the *updated* running mean (Eq. 3; first block
    Eq. 5), running uncentred per-feature power and its average (Eqs. 37-38),
    and the bias compensation for the change of the mean (Eq. 31, with the sign
    that keeps the layer's function unchanged) when the layer's parameters are
    attached.  Normaliser is the number of rows."""
    X = np.asarray(X, dtype=np.float64)
    rows, M = X.shape
    assert M == L.M and rows >= 1
    a = L.hp.alpha
    m_hat = X.sum(axis=0) / rows
    mu_old = L.mu.copy()
    L.mu = m_hat.copy() if L.first else a * L.mu + (1.0 - a) * m_hat
    Xc = X - L.mu[None, :]                       # second pass, centred on mu(i)
    C_hat = (Xc.T @ Xc) / rows
    C_hat = 0.5 * (C_hat + C_hat.T)
    L.Phix = C_hat if L.first else a * L.Phix + (1.0 - a) * C_hat
    phi_hat = (X * X).sum(axis=0) / rows          # uncentred, Eq. 37
    L.phi = phi_hat if L.first else a * L.phi + (1.0 - a) * phi_hat
    L.lam_bar = float(L.phi.sum() / M)            # Eq. 38
    if L.W is not None:
        # Eq. 31 in im2col form.  The paper derives the rule from the requirement
        # W (x - mu(i)) + b|i = W (x - mu(i-1)) + b|i-, i.e. the layer's function
        # must not change; solving it gives b|i = b|i- + W (mu(i) - mu(i-1)).
        # The printed equation has the two means in the opposite order, which
        # would double the change instead of cancelling it; the stated
        # requirement is taken as the definition.
        L.b = L.b + L.W @ (L.mu - mu_old)
    L.first = False


# =============================================================================
# EVD / ZCA whitening (oracle only): Eqs. 6-10, 32-34
# =============================================================================
def jacobi_evd(A: np.ndarray, sweeps: int = 60, tol: float = 1e-30):
    """Cyclic Jacobi eigen-decomposition of a symmetric matrix.
    Returns (lam, V) with lam sorted in decreasing order (Eq. 8) and
    A = V diag(lam) V^T (Eq. 7).  Plain loops: meant for small M."""
    A = np.array(A, dtype=np.float64)
    M = A.shape[0]
    V = np.eye(M)
    for _ in range(sweeps):
        off = 0.0
        for p in range(M):
            for q in range(p + 1, M):
                off += A[p, q] * A[p, q]
        if off <= tol * max(1.0, float(np.sum(np.diag(A) ** 2))):
            break
        for p in range(M - 1):
            for q in range(p + 1, M):
                apq = A[p, q]
                if apq == 0.0:
                    continue
                theta = (A[q, q] - A[p, p]) / (2.0 * apq)
                t = (1.0 if theta >= 0 else -1.0) / (abs(theta) + math.sqrt(theta * theta + 1.0))
                c = 1.0 / math.sqrt(t * t + 1.0)
                s = t * c
                # A <- J^T A J, J the rotation in the (p, q) plane
                Ap = A[:, p].copy(); Aq = A[:, q].copy()
                A[:, p] = c * Ap - s * Aq
                A[:, q] = s * Ap + c * Aq
                Ap = A[p, :].copy(); Aq = A[q, :].copy()
                A[p, :] = c * Ap - s * Aq
                A[q, :] = s * Ap + c * Aq
                Vp = V[:, p].copy(); Vq = V[:, q].copy()
                V[:, p] = c * Vp - s * Vq
                V[:, q] = s * Vp + c * Vq
    lam = np.diag(A).copy()
    order = np.argsort(-lam, kind="stable")
    return lam[order], V[:, order]


def eigenvalues_desc(A: np.ndarray) -> np.ndarray:
    """Eigenvalues in decreasing order; Jacobi for small M, the library's
    symmetric solver (one library step) above that."""
    A = np.asarray(A, dtype=np.float64)
    if A.shape[0] <= 24:
        return jacobi_evd(A)[0]
    return np.linalg.eigvalsh(0.5 * (A + A.T))[::-1].copy()


def condition_number(A: np.ndarray) -> float:
    """lambda_max / lambda_min of a symmetric PSD matrix (Sec. 4)."""
    lam = eigenvalues_desc(A)
    return float(lam[0] / lam[-1]) if lam[-1] > 0 else float("inf")


def aic_rank(lam: np.ndarray) -> float:
    """Signal-subspace rank estimate, Eq. 32, read as exp(-sum lbar log lbar)
    with 0 log 0 = 0: the form that yields M for equal eigenvalues and 1 for a
    single dominant one, the two limits the paper states for it."""
    lam = np.maximum(np.asarray(lam, dtype=np.float64), 0.0)
    lb = lam / lam.sum()
    nz = lb > 0
    return float(math.exp(-np.sum(lb[nz] * np.log(lb[nz]))))


def zca_transform(Phix: np.ndarray, eps: float = 1e-5, g_max: float | None = None,
                  use_jacobi: bool | None = None):
    """ZCA whitening matrix T = V diag(g)^(1/2) V^T (Eq. 9).
    g_max None: g_m = 1/max(lam_m, eps) (Eq. 10), giving T Phi_x T^T = I (Eq. 6)
    when every lam_m > eps.  g_max given: the practical gains of Eq. 34,
    g_m = min(1/(M lbar_m), g_max) for m below the rounded AIC rank, else 1."""
    Phix = np.asarray(Phix, dtype=np.float64)
    M = Phix.shape[0]
    if use_jacobi is None:
        use_jacobi = M <= 24
    if use_jacobi:
        lam, V = jacobi_evd(Phix)
    else:
        w, Vv = np.linalg.eigh(0.5 * (Phix + Phix.T))
        lam, V = w[::-1].copy(), Vv[:, ::-1].copy()
    if g_max is None:
        g = 1.0 / np.maximum(lam, eps)
    else:
        lb = np.maximum(lam, 0.0) / np.maximum(lam, 0.0).sum()
        Ms = int(min(M, max(1, round(aic_rank(lam)))))
        g = np.ones(M)
        g[:Ms] = np.minimum(1.0 / np.maximum(M * lb[:Ms], 1e-300), g_max)
    T = (V * np.sqrt(g)[None, :]) @ V.T
    return T, lam, V


def normalised_rank(Phiy: np.ndarray) -> float:
    """kappa = Ms_hat / M (Sec. 6)."""
    return aic_rank(eigenvalues_desc(Phiy)) / Phiy.shape[0]


def whiteness(Phiy: np.ndarray) -> float:
    """rho of Eq. 51 with the sum taken over all index pairs (m, m'),
    the reading under which a diagonal matrix gives 1 and a fully correlated
    one gives 1/M, as the paper states."""
    d = np.diag(Phiy)
    R2 = (Phiy * Phiy) / np.outer(d, d)
    return float(Phiy.shape[0] / R2.sum())


# =============================================================================
# (b) recursive condition-number reduction: Sec. 4
# =============================================================================
def principal_subspace(Phiy: np.ndarray, c_rel: float, c_abs: float, init: int = INIT_ALIGN,
                       forced=None):
    """High-power subspace estimate of Sec. 4.2.

    xi_m = ||Phi_y e_m|| (Eq. 45); m' = argmax, lowest index on ties (Eq. 46);
    c^T = e_m'^T Phi_y^T Phi_y (Eq. 47); the coherent set holds every m with
    |c_m| >= max(c_rel xi_m' xi_m, c_abs) (Eq. 48); the estimate is the
    normalised mean of the columns in the set, each divided by its c_m
    (Eqs. 49-50).  `forced` = (m', boolean mask) overrides the two discrete
    decisions (used to replay another implementation's decisions on near-ties).

    Returns dict(v, m_prime, mask, xi, c, ok, margin_argmax, margin_set);
    ok is False when the set is empty or the average vanishes."""
    M = Phiy.shape[0]
    xi = np.sqrt((Phiy * Phiy).sum(axis=0))
    m_prime = int(np.argmax(xi))                   # numpy returns the first maximum
    if forced is not None:
        m_prime = int(forced[0])
    col = Phiy[:, m_prime]
    c = Phiy.T @ col
    thr = np.maximum(c_rel * xi[m_prime] * xi, c_abs)
    mask = np.abs(c) >= thr
    if forced is not None and forced[1] is not None:
        mask = np.asarray(forced[1], dtype=bool)
    # distance of the two decisions from flipping (relative)
    others = np.delete(xi, m_prime)
    margin_argmax = float((xi[m_prime] - others.max()) / xi[m_prime]) if M > 1 and xi[m_prime] > 0 else 1.0
    margin_each = np.abs(np.abs(c) - thr) / thr
    margin_set = float(margin_each.min())
    out = dict(m_prime=m_prime, mask=mask, xi=xi, c=c, margin_argmax=margin_argmax,
               margin_set=margin_set, margin_each=margin_each)
    if init == INIT_MAXCOL:
        if xi[m_prime] > 0:
            out.update(v=col / xi[m_prime], ok=True)
        else:
            e = np.zeros(M); e[m_prime] = 1.0
            out.update(v=e, ok=False)
        return out
    idx = np.nonzero(mask)[0]
    if idx.size == 0:
        e = np.zeros(M); e[m_prime] = 1.0
        out.update(v=e, ok=False)
        return out
    v_t = np.zeros(M)
    for m in idx:                                   # Eq. 49, term by term
        v_t += Phiy[:, m] / c[m]
    v_t /= idx.size
    nrm = float(np.linalg.norm(v_t))
    if nrm == 0.0 or not np.isfinite(nrm):
        e = np.zeros(M); e[m_prime] = 1.0
        out.update(v=e, ok=False)
        return out
    out.update(v=v_t / nrm, ok=True)                # Eq. 50
    return out


def power_iterations(Phiy: np.ndarray, v: np.ndarray, P: int) -> np.ndarray:
    """P plain power iterations v <- Phi_y v / ||Phi_y v|| refining the start
    vector (P = 0 leaves the paper's estimate as it is)."""
    for _ in range(P):
        u = Phiy @ v
        n = float(np.linalg.norm(u))
        if n == 0.0:
            break
        v = u / n
    return v


def transformation_step(L: Layer, v: np.ndarray, a: float) -> None:
    """Append the step I + a v v^T to the transform with leakage gamma.

    T(i) = gamma (I + a v v^T) T(i-1) + (1 - gamma) I            (Eq. 42, definition)
    Q(i) by the O(M^2) recursion of Eq. 44 with t = T(i-1)^T v.

    Reading of Eq. 43: expanding the definition gives
    (I + a v v^T) T = T + a v (T^T v)^T, so the vector paired with v in the
    rank-one term is T^T v (it equals T v only while T is symmetric, i.e. for
    the first step); with it Eq. 44 reproduces T(i)^T T(i) exactly."""
    g = L.hp.gamma
    M = L.M
    I = np.eye(M)
    T_old = L.T
    t = T_old.T @ v
    Q_new = (g * g * (L.Q + a * (a + 2.0) * np.outer(t, t)) + (1.0 - g) ** 2 * I
             + g * (1.0 - g) * (a * (np.outer(v, t) + np.outer(t, v)) + T_old + T_old.T))
    T_new = g * ((I + a * np.outer(v, v)) @ T_old) + (1.0 - g) * I
    L.T = T_new
    L.Q = Q_new


def cond_reduce(L: Layer, K: int, P: int, forced=None, record_cond: bool = False):
    """K steps of the recursion of Sec. 4.1 on frozen moments, then one
    smoothing update of Qs (Eq. 35).

    Per step: Phi_y = T Phi_x T^T; the subspace estimate of Sec. 4.2 refined by
    P power iterations; lambda_e = v^T Phi_y v (Eq. 36);
    g_e = delta lam_bar / max(lambda_e, eps) (Eq. 40); a_e = sqrt(g_e) - 1
    (Eq. 41); the transformation step.  A step with no usable subspace uses
    a_e = 0 (only the leakage acts).  `forced` is a list of K (m', mask)
    decisions or None.  Returns the per-step trace."""
    hp = L.hp
    trace = []
    for k in range(K):
        Phiy = L.phiy()
        Phiy = 0.5 * (Phiy + Phiy.T)
        f = None if forced is None else forced[k]
        est = principal_subspace(Phiy, hp.c_rel, hp.c_abs, hp.init, f)
        rec = dict(m_prime=est["m_prime"], set_size=int(est["mask"].sum()), mask=est["mask"].copy(),
                   margin_argmax=est["margin_argmax"], margin_set=est["margin_set"], ok=est["ok"])
        if record_cond:
            rec["cond_before"] = condition_number(Phiy)
        if est["ok"]:
            v = power_iterations(Phiy, est["v"], P)
            u = Phiy @ v
            lam_e = float(v @ u)
            g_e = hp.delta * L.lam_bar / max(lam_e, hp.eps)
            a_e = math.sqrt(g_e) - 1.0
        else:
            v = est["v"]
            lam_e = float(v @ (Phiy @ v))
            g_e = 1.0
            a_e = 0.0
        rec.update(lam_e=lam_e, g_e=g_e, a_e=a_e, v=v.copy())
        transformation_step(L, v, a_e)
        trace.append(rec)
    if K > 0:
        L.Qs = hp.beta * L.Qs + (1.0 - hp.beta) * L.Q     # Eq. 35, once per call
    return trace


# =============================================================================
# (c) gradient transformation and SGD step: Eqs. 27-30
# =============================================================================
def grad_transform(L: Layer, G: np.ndarray) -> np.ndarray:
    """dL/dW_bar = dL/dW_tilde Q (Eq. 29) with the smoothed Q of Eq. 35."""
    return np.asarray(G, dtype=np.float64) @ L.Qs


def sgd_step(W, b, G_t, g_b, lr):
    """W <- W - eta G_t (Eq. 27);  b <- b - eta g_b (Eq. 28; bias gradient untransformed)."""
    return W - lr * G_t, b - lr * g_b


def sgd_momentum_step(W, b, G_t, g_b, vW, vb, lr, momentum, weight_decay):
    """SGD with momentum and weight decay as used in the experiments (Sec. 6), on the transformed gradient:
    v <- momentum v + (G_t + weight_decay W), W <- W - eta v; the bias likewise with its untransformed gradient
    and no decay.  Returns (W, b, vW, vb)."""
    vW = momentum * vW + (G_t + weight_decay * W)
    vb = momentum * vb + g_b
    return W - lr * vW, b - lr * vb, vW, vb


# =============================================================================
# direct (per-sample) whitening of a tiny layer: Eqs. 11, 14-20
# used only to pin the equivalence the gradient transformation rests on
# =============================================================================
def whiten_forward(L: Layer, X: np.ndarray) -> np.ndarray:
    """Direct whitening of the samples, y = T (x - mu), one sample per row (Eq. 11)."""
    return (np.asarray(X, dtype=np.float64) - L.mu[None, :]) @ L.T.T


def whiten_backward(L: Layer, dY: np.ndarray) -> np.ndarray:
    """Gradient through the whitening, dL/dx = T^T dL/dy, one sample per row (Eq. 14)."""
    return np.asarray(dY, dtype=np.float64) @ L.T


def direct_layer_update(W, b, T, mu, X, target, lr):
    """One SGD step of the *direct* method on the split layer
    z = W y + b, y = T (x - mu), with loss 0.5 sum ||z - target||^2.
    Returns (W_new, b_new, dL/dx) -- dL/dx through the whitening (Eq. 14)."""
    Y = (X - mu[None, :]) @ T.T                    # Eq. 11
    Z = Y @ W.T + b[None, :]                       # Eq. 15
    D = Z - target                                 # dL/dz
    dW = D.T @ Y                                   # Eq. 17
    db = D.sum(axis=0)                             # Eq. 18
    dY = D @ W
    dX = dY @ T                                    # Eq. 14: T^T dL/dy, row form
    return W - lr * dW, b - lr * db, dX


def gradient_layer_update(Wt, bt, Q, mu, X, target, lr):
    """One SGD step of the gradient-based method on the unsplit layer
    z = W_tilde (x - mu) + b_tilde (Eq. 21) with the same loss: the ordinary
    weight gradient is multiplied by Q = T^T T before the step (Eqs. 27-30)."""
    Xc = X - mu[None, :]
    Z = Xc @ Wt.T + bt[None, :]
    D = Z - target
    dWt = D.T @ Xc
    dbt = D.sum(axis=0)
    dX = D @ Wt
    return Wt - lr * (dWt @ Q), bt - lr * dbt, dX


def rel_fro(a, b) -> float:
    """|| a - b ||_F / || b ||_F (b is the reference)."""
    a = np.asarray(a, dtype=np.float64); b = np.asarray(b, dtype=np.float64)
    n = float(np.linalg.norm(b))
    d = float(np.linalg.norm(a - b))
    return d / n if n > 0 else d
