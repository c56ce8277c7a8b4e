"""Pins of the fp64 oracle against what the paper and the mathematics fix.

None of these compare the oracle with itself: each is a closed form, a hand
computation (tests/golden), an invariant stated in the paper, brute force on a
tiny case, or an independent library routine.  A test that "plants" a mistake
does so on the CPU, in a modified copy of the oracle's step.
"""
import math
import os

import numpy as np
import pytest

from oracle import fw_oracle as O
from paper_2010_01546_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _load(name):
    rows = []
    with open(os.path.join(GOLD, name)) as f:
        for ln in f:
            if ln.strip() and not ln.startswith("#"):
                rows.append([float(t) for t in ln.split()])
    return rows


def _spd(M, cond, seed):
    Phi, U, lam = synth.spd_with_spectrum(M, cond, seed)
    return Phi, U, lam


# ----------------------------------------------------------------------------
# moments (Eqs. 2-5, 37-38)
# ----------------------------------------------------------------------------
def test_moments_hand_computed_fixture():
    g = _load("moments_tiny.txt")
    L = O.Layer(1, 1, O.Hyper(alpha=0.5))
    O.cov_update(L, np.array([[1.0], [3.0]]))
    assert [L.mu[0], L.Phix[0, 0], L.phi[0], L.lam_bar] == pytest.approx(g[0][1:], abs=1e-15)
    O.cov_update(L, np.array([[5.0]]))
    assert [L.mu[0], L.Phix[0, 0], L.phi[0], L.lam_bar] == pytest.approx(g[1][1:], abs=1e-15)


def test_first_block_is_biased_sample_covariance():
    rng = np.random.default_rng(1)
    X = rng.standard_normal((57, 9)) + 3.0
    L = O.Layer(9, 2, O.Hyper(alpha=0.7))
    O.cov_update(L, X)
    assert np.allclose(L.mu, X.mean(axis=0), atol=1e-14)
    assert np.allclose(L.Phix, np.cov(X.T, bias=True), atol=1e-13)       # divide by rows, never rows-1
    assert np.allclose(L.phi, (X ** 2).mean(axis=0), atol=1e-13)          # uncentred power
    assert L.lam_bar == pytest.approx((X ** 2).mean(), rel=1e-14)


def test_block_of_several_batches_is_the_block_of_their_rows():
    # Sec. 2: moments are computed in blocks of L batches; Eqs. 2-3 sum over every sample of the block.  The
    # block's statistics follow from the batches' own by the law of total covariance, written out here from
    # per-batch means and biased covariances.
    rng = np.random.default_rng(21)
    M = 6
    batches = [rng.standard_normal((r, M)) * (1 + k) + k for k, r in enumerate((11, 30, 7))]
    L = O.Layer(M, 1, O.Hyper(alpha=0.3))
    O.cov_update(L, rng.standard_normal((15, M)))               # an earlier block, so that alpha acts
    mu0, Phi0 = L.mu.copy(), L.Phix.copy()
    O.cov_update(L, np.concatenate(batches, axis=0))
    n = np.array([b.shape[0] for b in batches], dtype=np.float64)
    w = n / n.sum()
    m_k = [b.mean(axis=0) for b in batches]
    m_blk = sum(wk * mk for wk, mk in zip(w, m_k))
    mu1 = 0.3 * mu0 + 0.7 * m_blk
    # covariance about the updated running mean mu1 (Eq. 3), not about the block mean
    C = sum(wk * (np.cov(b.T, bias=True) + np.outer(mk - mu1, mk - mu1)) for wk, b, mk in zip(w, batches, m_k))
    assert np.allclose(L.mu, mu1, atol=1e-13)
    assert np.allclose(L.Phix, 0.3 * Phi0 + 0.7 * C, atol=1e-12)


def test_alpha_zero_reduces_to_block_statistics_and_constant_rows_give_zero():
    rng = np.random.default_rng(2)
    L = O.Layer(5, 1, O.Hyper(alpha=0.0))
    O.cov_update(L, rng.standard_normal((20, 5)))
    X2 = rng.standard_normal((31, 5)) * 2 + 1
    O.cov_update(L, X2)
    assert np.allclose(L.Phix, np.cov(X2.T, bias=True), atol=1e-13)
    Lc = O.Layer(5, 1)
    O.cov_update(Lc, np.tile(np.arange(5.0), (7, 1)))
    assert np.abs(Lc.Phix).max() == 0.0


def test_running_covariance_is_centred_on_the_updated_running_mean():
    # second block: C_hat must use mu(i) = alpha mu(i-1) + (1-alpha) m_hat, not the batch mean
    rng = np.random.default_rng(3)
    a = 0.6
    X1 = rng.standard_normal((40, 4)); X2 = rng.standard_normal((25, 4)) + 2.0
    L = O.Layer(4, 1, O.Hyper(alpha=a))
    O.cov_update(L, X1); P1 = L.Phix.copy(); m1 = L.mu.copy()
    O.cov_update(L, X2)
    mu2 = a * m1 + (1 - a) * X2.mean(axis=0)
    # E[(x-mu)(x-mu)^T] = Cov_batch + (m_hat-mu)(m_hat-mu)^T : textbook shift identity
    d = X2.mean(axis=0) - mu2
    C = np.cov(X2.T, bias=True) + np.outer(d, d)
    assert np.allclose(L.mu, mu2, atol=1e-14)
    assert np.allclose(L.Phix, a * P1 + (1 - a) * C, atol=1e-13)


def test_zero_mean_inputs_give_lam_bar_equal_trace_over_M():
    rng = np.random.default_rng(4)
    X = rng.standard_normal((64, 6)); X -= X.mean(axis=0)
    L = O.Layer(6, 1, O.Hyper(alpha=0.0))
    O.cov_update(L, X)
    assert L.lam_bar == pytest.approx(np.trace(L.Phix) / 6, rel=1e-13)


def test_bias_compensation_keeps_the_network_function(  ):
    # Eq. 31: z = W (x - mu) + b must be the same function before and after a mean update
    rng = np.random.default_rng(5)
    M, N = 7, 3
    L = O.Layer(M, N, O.Hyper(alpha=0.3))
    W = rng.standard_normal((N, M)); b = rng.standard_normal(N)
    L.attach_params(W, b)
    xs = rng.standard_normal((11, M))
    O.cov_update(L, rng.standard_normal((30, M)) + 1.0)
    for _ in range(2):
        z_before = (xs - L.mu) @ L.W.T + L.b
        O.cov_update(L, rng.standard_normal((30, M)) * 2 - 0.5)
        z_after = (xs - L.mu) @ L.W.T + L.b
        assert np.allclose(z_before, z_after, atol=1e-12)


def test_initial_state():
    L = O.Layer(4, 2)
    assert np.array_equal(L.T, np.eye(4)) and np.array_equal(L.Qs, np.eye(4)) and np.array_equal(L.Q, np.eye(4))
    assert not L.mu.any() and L.first


# ----------------------------------------------------------------------------
# EVD / ZCA (Eqs. 6-10), AIC rank (Eq. 32), whiteness (Eq. 51)
# ----------------------------------------------------------------------------
def test_jacobi_two_by_two_closed_form():
    A = np.array([[2.0, 1.0], [1.0, 3.0]])
    lam, V = O.jacobi_evd(A)
    assert lam == pytest.approx([(5 + math.sqrt(5)) / 2, (5 - math.sqrt(5)) / 2], abs=1e-14)
    assert np.allclose(V @ np.diag(lam) @ V.T, A, atol=1e-14)


@pytest.mark.parametrize("M", [3, 8, 16])
def test_jacobi_matches_library_eigensolver_and_deflated_power_iteration(M):
    rng = np.random.default_rng(M)
    A = rng.standard_normal((M, M)); A = A @ A.T + 0.1 * np.eye(M)
    lam, V = O.jacobi_evd(A)
    w = np.linalg.eigvalsh(A)[::-1]
    assert np.allclose(lam, w, rtol=1e-12, atol=1e-12)
    assert np.all(np.diff(lam) <= 0)                                    # decreasing order, Eq. 8
    assert np.allclose(V.T @ V, np.eye(M), atol=1e-12)
    # brute force: long power iteration with deflation for the top three pairs
    B = A.copy()
    for k in range(min(3, M)):
        v = np.ones(M) / math.sqrt(M)
        v = O.power_iterations(B, v, 20000)
        l = v @ B @ v
        assert l == pytest.approx(lam[k], rel=1e-8)
        assert abs(v @ V[:, k]) == pytest.approx(1.0, abs=1e-6)
        B = B - l * np.outer(v, v)


@pytest.mark.parametrize("M,cond,use_jacobi", [(8, 1e2, True), (16, 1e3, True), (64, 1e3, False)])
def test_zca_whitens(M, cond, use_jacobi):
    Phi, U, lam = _spd(M, cond, 11 + M)
    T, lam_hat, V = O.zca_transform(Phi, eps=1e-9, use_jacobi=use_jacobi)
    assert np.allclose(T @ Phi @ T.T, np.eye(M), atol=1e-9)             # Eq. 6
    assert np.allclose(T, T.T, atol=1e-12)                               # ZCA is symmetric
    assert np.allclose(lam_hat, lam, rtol=1e-9)
    # closed form in the known basis: T = U diag(lam^-1/2) U^T
    assert np.allclose(T, (U / np.sqrt(lam)[None, :]) @ U.T, atol=1e-8 * math.sqrt(cond))


def test_zca_eps_floor_and_capped_gains():
    lam = np.array([4.0, 1.0, 1e-8])
    T, _, _ = O.zca_transform(np.diag(lam), eps=1e-4)
    assert np.allclose(np.diag(T), [0.5, 1.0, 100.0], rtol=1e-12)        # 1/sqrt(max(lam, eps)), Eq. 10
    # Eq. 34: equal eigenvalues -> rank M, lbar = 1/M, gain min(1, gmax) = 1 -> T = I
    T2, _, _ = O.zca_transform(3.0 * np.eye(5), g_max=10.0)
    assert np.allclose(T2, np.eye(5), atol=1e-12)
    # one dominant eigenvalue -> rank 1; its gain is 1/(M lbar_0) ~ 1/M, the others 1
    T3, _, _ = O.zca_transform(np.diag([1.0, 1e-9, 1e-9, 1e-9]), g_max=10.0)
    assert np.allclose(np.diag(T3) ** 2, [0.25, 1, 1, 1], rtol=1e-6)


def test_aic_rank_extremes():
    assert O.aic_rank(np.full(12, 0.37)) == pytest.approx(12.0, rel=1e-12)
    assert O.aic_rank(np.array([5.0] + [1e-14] * 9)) == pytest.approx(1.0, abs=1e-10)
    assert O.aic_rank(np.array([1.0, 0.0, 0.0])) == 1.0


def test_normalised_rank_extremes_and_a_hand_value():
    # kappa = Ms_hat / M (Sec. 6) of a matrix given by its eigenvalues in some orthogonal basis
    U = synth.orthogonal_qr(6, 3)
    assert O.normalised_rank(2.5 * np.eye(6)) == pytest.approx(1.0, rel=1e-12)              # white: full rank
    A = (U * np.array([4.0] + [1e-13] * 5)[None, :]) @ U.T
    assert O.normalised_rank(A) == pytest.approx(1.0 / 6, abs=1e-9)                        # one dominant direction
    # eigenvalues (2, 1, 1): normalised (1/2, 1/4, 1/4), entropy (1/2) ln 2 + (1/2) ln 4 = (3/2) ln 2,
    # so Ms_hat = 2^(3/2) and kappa = 2^(3/2) / 3
    V = synth.orthogonal_qr(3, 4)
    A3 = (V * np.array([2.0, 1.0, 1.0])[None, :]) @ V.T
    assert O.normalised_rank(A3) == pytest.approx(2.0 ** 1.5 / 3.0, rel=1e-12)
    # the basis does not matter, only the spectrum
    assert O.normalised_rank(np.diag([1.0, 2.0, 1.0])) == pytest.approx(2.0 ** 1.5 / 3.0, rel=1e-12)


def test_whiteness_extremes():
    assert O.whiteness(np.diag([3.0, 0.2, 7.0])) == pytest.approx(1.0)
    u = np.array([1.0, -2.0, 0.5, 3.0])
    assert O.whiteness(np.outer(u, u)) == pytest.approx(1.0 / 4)


# ----------------------------------------------------------------------------
# equivalence of direct whitening and gradient transformation (Sec. 3.1)
# ----------------------------------------------------------------------------
def _loss(Wt, bt, mu, X, tgt):
    Z = (X - mu) @ Wt.T + bt
    return 0.5 * np.sum((Z - tgt) ** 2)


def test_layer_gradients_by_finite_differences():
    rng = np.random.default_rng(7)
    M, N, rows = 5, 3, 9
    X = rng.standard_normal((rows, M)); tgt = rng.standard_normal((rows, N))
    Wt = rng.standard_normal((N, M)); bt = rng.standard_normal(N); mu = rng.standard_normal(M)
    W1, b1, dX = O.gradient_layer_update(Wt, bt, np.eye(M), mu, X, tgt, 1.0)
    dW = Wt - W1; db = bt - b1
    h = 1e-6
    for (i, j) in [(0, 0), (2, 3), (1, 4)]:
        E = np.zeros_like(Wt); E[i, j] = h
        fd = (_loss(Wt + E, bt, mu, X, tgt) - _loss(Wt - E, bt, mu, X, tgt)) / (2 * h)
        assert dW[i, j] == pytest.approx(fd, rel=1e-6, abs=1e-7)
    e = np.zeros(N); e[1] = h
    assert db[1] == pytest.approx((_loss(Wt, bt + e, mu, X, tgt) - _loss(Wt, bt - e, mu, X, tgt)) / (2 * h), rel=1e-6)
    E = np.zeros_like(X); E[4, 2] = h
    assert dX[4, 2] == pytest.approx((_loss(Wt, bt, mu, X + E, tgt) - _loss(Wt, bt, mu, X - E, tgt)) / (2 * h), rel=1e-6)
    # direct method, Eq. 14: gradient w.r.t. x passes through T^T
    T = rng.standard_normal((M, M))
    W = rng.standard_normal((N, M))
    _, _, dXd = O.direct_layer_update(W, bt, T, mu, X, tgt, 1.0)
    fd = (_loss(W @ T, bt, mu, X + E, tgt) - _loss(W @ T, bt, mu, X - E, tgt)) / (2 * h)
    assert dXd[4, 2] == pytest.approx(fd, rel=1e-6)


@pytest.mark.parametrize("kind", ["zca", "recursive"])
@pytest.mark.parametrize("M,N,rows", [(4, 2, 16), (8, 4, 32)])
def test_explicit_whitening_equals_gradient_transformation(kind, M, N, rows):
    rng = np.random.default_rng(100 + M)
    Phi, U, lam = _spd(M, 50.0, 5 + M)
    Xs = [synth.gaussian_rows(rows, U, lam, 77 + i, mean=np.linspace(-1, 1, M)) for i in range(4)]
    L = O.Layer(M, N, O.Hyper(alpha=0.0, beta=0.0, gamma=0.9, delta=0.25))
    O.cov_update(L, Xs[0])
    if kind == "zca":
        T, _, _ = O.zca_transform(L.Phix)
        Q = T.T @ T
    else:
        O.cond_reduce(L, 5, 8)
        T, Q = L.T, L.Q                      # Q from the O(M^2) recursion of Eq. 44
    W = rng.standard_normal((N, M)); b = rng.standard_normal(N)
    Wt = W @ T; bt = b.copy()                # Eqs. 23-24
    lr = 0.01
    for X in Xs[1:]:
        tgt = rng.standard_normal((rows, N))
        W, b, dX_d = O.direct_layer_update(W, b, T, L.mu, X, tgt, lr)
        Wt, bt, dX_g = O.gradient_layer_update(Wt, bt, Q, L.mu, X, tgt, lr)
        assert O.rel_fro(Wt, W @ T) < 1e-12
        assert O.rel_fro(bt, b) < 1e-12
        assert O.rel_fro(dX_g, dX_d) < 1e-12     # the propagated gradients agree too


def test_sample_whitening_forward_and_backward():
    # Eq. 11 / Eq. 14 per sample, against explicit loops; with the ZCA transform the whitened samples have identity
    # covariance (Eq. 6); the backward product is the transpose map, so <T(x - mu), g> = <x - mu, T^T g>
    rng = np.random.default_rng(31)
    M, rows = 7, 40
    Phi, U, lam = _spd(M, 30.0, 5)
    X = synth.gaussian_rows(rows, U, lam, 6) + 2.0
    L = O.Layer(M, 2, O.Hyper(alpha=0.0))
    O.cov_update(L, X)
    L.T, _, _ = O.zca_transform(L.Phix, eps=1e-12)
    Y = O.whiten_forward(L, X)
    for r in (0, 17, rows - 1):
        assert np.allclose(Y[r], L.T @ (X[r] - L.mu), atol=1e-12)
    assert np.allclose(Y.T @ Y / rows, np.eye(M), atol=1e-9)
    G = rng.standard_normal((rows, M))
    dX = O.whiten_backward(L, G)
    for r in (3, 21):
        assert np.allclose(dX[r], L.T.T @ G[r], atol=1e-12)
    assert np.sum(Y * G) == pytest.approx(np.sum((X - L.mu) * dX), rel=1e-12)
    # and it is the map direct_layer_update sends dL/dy through
    W = rng.standard_normal((2, M)); b = rng.standard_normal(2); tgt = rng.standard_normal((rows, 2))
    _, _, dX2 = O.direct_layer_update(W, b, L.T, L.mu, X, tgt, 0.1)
    D = (Y @ W.T + b) - tgt
    assert np.allclose(dX2, O.whiten_backward(L, D @ W), atol=1e-12)


def test_momentum_step_hand_values_and_reduction_to_plain_sgd():
    W = np.array([[1.0, -2.0]]); b = np.array([0.5]); G = np.array([[0.5, 0.25]]); gb = np.array([2.0])
    vW = np.zeros((1, 2)); vb = np.zeros(1)
    # step 1: v = G + 0.1 W = (0.6, 0.05); W = W - 0.5 v = (0.7, -2.025); vb = 2, b = -0.5
    W, b, vW, vb = O.sgd_momentum_step(W, b, G, gb, vW, vb, 0.5, 0.9, 0.1)
    assert np.allclose(vW, [[0.6, 0.05]]) and np.allclose(W, [[0.7, -2.025]]) and np.allclose(b, [-0.5])
    # step 2: v = 0.9 (0.6, 0.05) + (0.5 + 0.07, 0.25 - 0.2025) = (1.11, 0.0925); W = (0.145, -2.07125)
    W, b, vW, vb = O.sgd_momentum_step(W, b, G, gb, vW, vb, 0.5, 0.9, 0.1)
    assert np.allclose(vW, [[1.11, 0.0925]]) and np.allclose(W, [[0.145, -2.07125]])
    assert np.allclose(vb, [3.8]) and np.allclose(b, [-2.4])
    # no momentum, no decay: Eqs. 27-28
    W0 = np.array([[1.0, 2.0]]); b0 = np.array([1.0])
    W1, b1, _, _ = O.sgd_momentum_step(W0, b0, G, gb, np.zeros((1, 2)), np.zeros(1), 0.1, 0.0, 0.0)
    W2, b2 = O.sgd_step(W0, b0, G, gb, 0.1)
    assert np.array_equal(W1, W2) and np.array_equal(b1, b2)


def test_transform_and_step_are_plain_products():
    rng = np.random.default_rng(8)
    L = O.Layer(3, 2)
    L.Qs = np.array([[2.0, 0, 0], [0, 1, 1], [0, 1, 3.0]])
    G = np.array([[1.0, 2, 3], [0, -1, 1]])
    Gt = O.grad_transform(L, G)
    assert np.array_equal(Gt, np.array([[2.0, 5, 11], [0, 0, 2]]))       # G Qs by hand (Eq. 29)
    W, b = O.sgd_step(np.ones((2, 3)), np.ones(2), Gt, np.array([1.0, -1.0]), 0.5)
    assert np.array_equal(W, 1 - 0.5 * Gt) and np.array_equal(b, [0.5, 1.5])


# ----------------------------------------------------------------------------
# transformation step (Eqs. 36, 39-44)
# ----------------------------------------------------------------------------
def test_step_hand_computed_fixture():
    g_e, a_e, T00, T11, Q00, Q11 = _load("step_tiny.txt")[0]
    L = O.Layer(2, 1, O.Hyper(gamma=0.5, delta=0.25, eps=1e-5, beta=0.0, init=O.INIT_MAXCOL))
    L.set_phix(np.diag([0.25, 0.01]), lam_bar=4.0)
    tr = O.cond_reduce(L, 1, 0)
    assert tr[0]["g_e"] == pytest.approx(g_e) and tr[0]["a_e"] == pytest.approx(a_e)
    assert np.allclose(L.T, np.diag([T00, T11]), atol=1e-15)
    assert np.allclose(L.Q, np.diag([Q00, Q11]), atol=1e-15)


@pytest.mark.parametrize("gamma", [1.0, 0.99, 0.6])
def test_Q_recursion_equals_TtT_every_step_and_literal_Tv_does_not(gamma):
    M = 12
    Phi, _, _ = _spd(M, 1e3, 21)
    L = O.Layer(M, 1, O.Hyper(gamma=gamma, beta=0.0))
    L.set_phix(Phi)
    for k in range(6):
        O.cond_reduce(L, 1, 4)
        assert O.rel_fro(L.Q, L.T.T @ L.T) < 1e-13                        # Eqs. 30, 44
        assert np.allclose(L.Qs, L.Q)                                     # beta = 0
    assert not np.allclose(L.T, L.T.T, atol=1e-6)                         # T is no longer symmetric
    # planted mistake: t = T v (Eq. 43 as printed) breaks the identity from the second step on
    L2 = O.Layer(M, 1, O.Hyper(gamma=gamma, beta=0.0)); L2.set_phix(Phi)
    bad = 0.0
    for k in range(6):
        Phiy = L2.phiy()
        est = O.principal_subspace(Phiy, 0.025, 1e-6)
        v = O.power_iterations(Phiy, est["v"], 4)
        lam_e = v @ Phiy @ v
        a = math.sqrt(0.25 * L2.lam_bar / max(lam_e, 1e-5)) - 1
        t = L2.T @ v
        g = gamma
        Qn = (g * g * (L2.Q + a * (a + 2) * np.outer(t, t)) + (1 - g) ** 2 * np.eye(M)
              + g * (1 - g) * (a * (np.outer(v, t) + np.outer(t, v)) + L2.T + L2.T.T))
        L2.T = g * (np.eye(M) + a * np.outer(v, v)) @ L2.T + (1 - g) * np.eye(M)
        L2.Q = Qn
        bad = O.rel_fro(L2.Q, L2.T.T @ L2.T)
        if k == 0:
            assert bad < 1e-13                                            # symmetric T: both readings agree
    assert bad > 1e-6


def test_step_sets_subspace_power_and_leaves_orthogonal_directions():
    # v^T Tt^T Phi_y Tt v = delta lam_bar for any unit v with lambda_e > eps (text after Eq. 41)
    M = 10
    Phi, U, lam = _spd(M, 1e2, 31)
    L = O.Layer(M, 1, O.Hyper(gamma=1.0, delta=0.25, beta=0.0))
    L.set_phix(Phi)
    tr = O.cond_reduce(L, 1, 3)
    v = tr[0]["v"]
    Phiy2 = L.phiy()
    assert v @ Phiy2 @ v == pytest.approx(0.25 * L.lam_bar, rel=1e-12)
    w = np.random.default_rng(0).standard_normal(M); w -= (w @ v) * v
    assert np.allclose(L.T @ w, w, atol=1e-13)                            # orthogonal subspace untouched
    assert tr[0]["lam_e"] == pytest.approx(v @ Phi @ v, rel=1e-13)       # Eq. 36 at T = I


def test_leak_only_step_when_no_subspace():
    L = O.Layer(4, 1, O.Hyper(gamma=0.9, beta=0.0))
    L.set_phix(np.zeros((4, 4)))
    tr = O.cond_reduce(L, 2, 5)
    assert not tr[0]["ok"] and tr[0]["a_e"] == 0.0
    assert np.allclose(L.T, np.eye(4)) and np.allclose(L.Q, np.eye(4))
    L2 = O.Layer(4, 1); L2.set_phix(1e-9 * np.eye(4))                     # xi^2 < c_abs
    assert not O.cond_reduce(L2, 1, 0)[0]["ok"]


def test_smoothing_of_Q():
    L = O.Layer(3, 1, O.Hyper(beta=0.25, gamma=1.0))
    L.set_phix(np.diag([4.0, 1.0, 0.5]))
    O.cond_reduce(L, 2, 2)
    assert np.allclose(L.Qs, 0.25 * np.eye(3) + 0.75 * L.Q)               # Eq. 35 from Qs(-1) = I
    Q1 = L.Q.copy(); Qs1 = L.Qs.copy()
    O.cond_reduce(L, 1, 2)
    assert np.allclose(L.Qs, 0.25 * Qs1 + 0.75 * L.Q) and not np.allclose(L.Q, Q1)


# ----------------------------------------------------------------------------
# subspace estimate (Eqs. 45-50) and power iterations
# ----------------------------------------------------------------------------
def test_rank_one_covariance_returns_its_vector_exactly():
    rng = np.random.default_rng(9)
    u = rng.standard_normal(9); u /= np.linalg.norm(u)
    Phi = 2.5 * np.outer(u, u)
    for P in (0, 3):
        est = O.principal_subspace(Phi, 0.025, 1e-6)
        v = O.power_iterations(Phi, est["v"], P)
        assert abs(v @ u) == pytest.approx(1.0, abs=1e-14)
    assert est["m_prime"] == int(np.argmax(np.abs(u)))                    # largest column of u u^T
    assert est["mask"][est["m_prime"]]


def test_high_snr_estimate_is_close_to_principal_eigenvector():
    # dominant rank-one signal plus weak white noise: error of the estimate is O(sigma^2 / lambda_1)
    rng = np.random.default_rng(10)
    M = 16
    u = rng.standard_normal(M); u /= np.linalg.norm(u)
    for s2 in (1e-3, 1e-5):
        Phi = 4.0 * np.outer(u, u) + s2 * np.eye(M)
        est = O.principal_subspace(Phi, 0.025, 1e-6)
        assert 1.0 - abs(est["v"] @ u) < 10 * (s2 / 4.0) ** 2 + 1e-15 or math.acos(min(1, abs(est["v"] @ u))) < 10 * s2 / 4.0


def test_estimator_pieces_by_brute_force_loops():
    rng = np.random.default_rng(12)
    M = 6
    A = rng.standard_normal((M, M)); Phi = A @ A.T
    est = O.principal_subspace(Phi, 0.3, 1e-6)
    xi = [math.sqrt(sum(Phi[j][m] ** 2 for j in range(M))) for m in range(M)]
    mp = max(range(M), key=lambda m: (xi[m], -m))
    c = [sum(Phi[j][mp] * Phi[j][m] for j in range(M)) for m in range(M)]
    S = [m for m in range(M) if abs(c[m]) >= max(0.3 * xi[mp] * xi[m], 1e-6)]
    vt = [sum(Phi[j][m] / c[m] for m in S) / len(S) for j in range(M)]
    n = math.sqrt(sum(x * x for x in vt))
    assert est["m_prime"] == mp and list(np.nonzero(est["mask"])[0]) == S
    assert 0 < len(S) < M                                                  # the threshold really selects
    assert np.allclose(est["v"], np.array(vt) / n, atol=1e-14)
    assert c[mp] == pytest.approx(xi[mp] ** 2)                            # so m' is in the set when xi^2 >= c_abs


def test_argmax_tie_takes_lowest_index_and_forced_decisions_are_used():
    Phi = np.diag([2.0, 2.0, 1.0])
    est = O.principal_subspace(Phi, 0.025, 1e-6)
    assert est["m_prime"] == 0 and est["margin_argmax"] == 0.0
    est2 = O.principal_subspace(Phi, 0.025, 1e-6, forced=(1, np.array([False, True, False])))
    assert est2["m_prime"] == 1 and abs(est2["v"][1]) == 1.0


def test_power_iteration_angle_bound():
    M = 12
    Phi, U, lam = _spd(M, 1e2, 41)
    rng = np.random.default_rng(13)
    v0 = rng.standard_normal(M); v0 /= np.linalg.norm(v0)
    def tan_angle(v):
        cth = abs(v @ U[:, 0]); return math.sqrt(max(0.0, 1 - cth * cth)) / cth
    t0 = tan_angle(v0)
    for P in (1, 5, 20):
        v = O.power_iterations(Phi, v0, P)
        assert tan_angle(v) <= (lam[1] / lam[0]) ** P * t0 * (1 + 1e-9) + 1e-15
        assert np.linalg.norm(v) == pytest.approx(1.0, abs=1e-14)
    assert np.array_equal(O.power_iterations(Phi, v0, 0), v0)


# ----------------------------------------------------------------------------
# condition number along the recursion (Sec. 4)
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("M,cond", [(8, 1e2), (16, 1e3), (48, 1e3)])
def test_condition_number_non_increasing_with_exact_eigenvector(M, cond):
    # gamma = 1, converged eigenvector, lam_min <= delta lam_bar <= lam_max:
    # each step replaces the largest eigenvalue by delta lam_bar and keeps the rest.
    Phi, U, lam = _spd(M, cond, 51)
    L = O.Layer(M, 1, O.Hyper(gamma=1.0, delta=0.25, beta=0.0, eps=1e-12))
    L.set_phix(Phi)
    spec = np.sort(lam)[::-1].copy()
    prev = O.condition_number(L.phiy())
    assert prev == pytest.approx(cond, rel=1e-8)
    for k in range(6):
        target = 0.25 * L.lam_bar
        if not (spec.min() <= target <= spec.max()):
            break
        O.cond_reduce(L, 1, 4000)
        spec[np.argmax(spec)] = target
        got = O.eigenvalues_desc(L.phiy())
        assert np.allclose(got, np.sort(spec)[::-1], rtol=1e-7, atol=1e-12)
        cur = O.condition_number(L.phiy())
        assert cur <= prev * (1 + 1e-9)
        prev = cur
    assert k >= 2


def test_condition_number_library_path_matches_jacobi():
    Phi, _, lam = _spd(24, 1e4, 61)
    assert O.condition_number(Phi) == pytest.approx(1e4, rel=1e-8)
    Phi2, _, _ = _spd(40, 1e4, 62)
    assert O.condition_number(Phi2) == pytest.approx(O.jacobi_evd(Phi2)[0][0] / O.jacobi_evd(Phi2)[0][-1], rel=1e-8)


def test_recursion_reduces_condition_number_on_the_small_workload():
    # the small single-layer workload: 8 steps of 16 power iterations
    d = synth.single_linear_layer()
    L = O.Layer(64, 32, O.Hyper(alpha=0.9, beta=0.0, gamma=1.0, delta=0.25))
    O.cov_update(L, d["X"])
    c0 = O.condition_number(L.phiy())
    tr = O.cond_reduce(L, 8, 16, record_cond=True)
    c1 = O.condition_number(L.phiy())
    assert c1 < c0
    assert all(t["ok"] for t in tr)
    assert O.rel_fro(L.Q, L.T.T @ L.T) < 1e-12


def test_cost_sweep_generator_has_the_stated_spectrum():
    # input recipe of the large-batch layer: rows ~ N(0, U diag(logspace(0, -4)) U^T); on a reduced size the
    # sample covariance must have that trace and a largest eigenvalue near 1
    d = synth.cost_sweep_layer(B=16, M=96, N=8, HW=14, cond=1e4, chunk_rows=1000)
    X = d["X"].astype(np.float64)
    assert X.shape == (16 * 196, 96) and d["G"].shape == (8, 96)
    C = X.T @ X / X.shape[0]
    lam = np.logspace(0.0, -4.0, 96)
    assert abs(np.trace(C) - lam.sum()) <= 0.05 * lam.sum()
    w = np.linalg.eigvalsh(C)
    assert 0.8 <= w[-1] <= 1.25
    d2 = synth.cost_sweep_layer(B=16, M=96, N=8, HW=14, cond=1e4, chunk_rows=1000)
    assert np.array_equal(d["X"], d2["X"])            # seeded: the same bits every time
