"""Whitening from the eigenvalue decomposition on the device (Sec. 2, Eqs. 7-10; Sec. 3.2, Eqs. 32, 34, 35) and the
spectrum diagnostics (normalised rank kappa of Sec. 6) against the fp64 oracle on the same fp32 covariance."""
import numpy as np
import pytest

from oracle import fw_oracle as O
from paper_2010_01546_b200 import synth

from fwtest_util import TOL_FP32, oracle_hyper, rel_fro, t2n

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2010_01546_b200 import binding as B, build
    build.build_library()
    return torch, B


def spd32(M, cond, seed):
    Phi, _, _ = synth.spd_with_spectrum(M, cond, seed, basis="qr" if M <= 300 else "householder")
    P = Phi.astype(np.float32)
    return np.triu(P) + np.triu(P, 1).T


def scratch_for(torch, B, M):
    nb = B.fw_evd_scratch_bytes(M)
    assert nb >= 2 * M * M * 8
    return torch.empty(nb, dtype=torch.uint8, device="cuda"), nb


def oracle_state(Phi32, eps, g_max):
    T, lam, V = O.zca_transform(Phi32.astype(np.float64), eps=eps, g_max=g_max, use_jacobi=False)
    return T, T.T @ T, T @ Phi32.astype(np.float64) @ T.T, lam


@pytest.mark.parametrize("M,cond", [(1, 1.0), (2, 10.0), (8, 1e2), (33, 1e3), (64, 1e3), (144, 1e3), (300, 1e4),
                                    (576, 1e3),
                                    (700, 1e3)])     # rows longer than the register-resident limit: two passes per pair
@pytest.mark.parametrize("g_max", [0.0, 4.0])
def test_evd_whitening_matches_oracle(env, M, cond, g_max):
    torch, B = env
    Phi32 = spd32(M, cond, 900 + M)
    L = B.Layer(M, 4, beta=0.0, gamma=1.0)
    L.set(B.FW_F_PHIX, torch.from_numpy(Phi32).cuda())
    scratch, nb = scratch_for(torch, B, M)
    B.fw_evd_whiten(L.handle, scratch, nb, g_max)
    assert L.sync_status() == B.FW_OK
    To, Qo, Yo, lam = oracle_state(Phi32, L.desc.eps, g_max if g_max > 0 else None)
    T, Q, Y = t2n(L.get(B.FW_F_T)), t2n(L.get(B.FW_F_Q)), t2n(L.get(B.FW_F_PHIY))
    assert rel_fro(T, To) <= TOL_FP32
    assert rel_fro(Q, Qo) <= TOL_FP32
    assert rel_fro(Y, Yo) <= TOL_FP32
    for A in (T, Q, Y):
        assert np.array_equal(A, A.T)                     # exactly symmetric
    if g_max == 0.0 and lam[-1] > L.desc.eps:
        # Eq. 6: T Phi_x T^T = I (every eigenvalue above eps); T is stored in fp32, so to a few ulp of cond^(1/2)
        assert np.linalg.norm(Y - np.eye(M)) / np.sqrt(M) <= 1e-4
    # the gradient transform uses it: Qs = Q at beta = 0
    G = np.random.default_rng(M).standard_normal((4, M)).astype(np.float32)
    Gt = t2n(L.grad_transform(torch.from_numpy(G).cuda()))
    assert rel_fro(Gt, G.astype(np.float64) @ Qo) <= TOL_FP32


def test_evd_whitening_group_mixed_sizes_and_smoothing(env):
    torch, B = env
    Ms = [17, 64, 96, 145, 288]
    beta = 0.3
    Ls, Phis, scr = [], [], []
    for i, M in enumerate(Ms):
        Ls.append(B.Layer(M, 4, beta=beta, gamma=1.0))
        Phis.append(spd32(M, 1e3, 950 + i))
        Ls[-1].set(B.FW_F_PHIX, torch.from_numpy(Phis[-1]).cuda())
        scr.append(scratch_for(torch, B, M))
    B.fw_group_evd_whiten([L.handle for L in Ls], [s[0] for s in scr], [s[1] for s in scr], 3.0)
    for L, Phi32, M in zip(Ls, Phis, Ms):
        assert L.sync_status() == B.FW_OK
        To, Qo, Yo, _ = oracle_state(Phi32, L.desc.eps, 3.0)
        assert rel_fro(t2n(L.get(B.FW_F_T)), To) <= TOL_FP32
        assert rel_fro(t2n(L.get(B.FW_F_PHIY)), Yo) <= TOL_FP32
        # Eq. 35 from Qs(-1) = I
        assert rel_fro(t2n(L.get(B.FW_F_QS)), beta * np.eye(M) + (1 - beta) * Qo) <= TOL_FP32
    # a second block: the single-layer call on the same state gives the same T, and Qs is smoothed once more
    L, Phi32, M = Ls[2], Phis[2], Ms[2]
    B.fw_evd_whiten(L.handle, scr[2][0], scr[2][1], 3.0)
    _, Qo, _, _ = oracle_state(Phi32, L.desc.eps, 3.0)
    Qs1 = beta * np.eye(M) + (1 - beta) * Qo
    assert rel_fro(t2n(L.get(B.FW_F_QS)), beta * Qs1 + (1 - beta) * Qo) <= TOL_FP32


@pytest.mark.parametrize("M,cond", [(7, 1e2), (64, 1e4), (145, 1e3), (300, 1e2)])
def test_spectrum_and_normalised_rank(env, M, cond):
    torch, B = env
    Phi32 = spd32(M, cond, 970 + M)
    L = B.Layer(M, 4, beta=0.0, gamma=1.0)
    L.set(B.FW_F_PHIX, torch.from_numpy(Phi32).cuda())
    scratch, nb = scratch_for(torch, B, M)
    lam = torch.zeros(M, device="cuda"); kap = torch.zeros(1, device="cuda")
    B.fw_spectrum(L.handle, 0, scratch, nb, lam, kap)
    lam_o = O.eigenvalues_desc(Phi32.astype(np.float64))
    assert np.max(np.abs(t2n(lam) - lam_o)) <= 1e-6 * lam_o[0]
    assert abs(float(kap[0]) - O.normalised_rank(Phi32.astype(np.float64))) <= 1e-5
    # of Phi_y, after two reduction steps: the state is untouched by the query
    L.cond_reduce(2, 8)
    before = [L.get(f).clone() for f in (B.FW_F_T, B.FW_F_Q, B.FW_F_PHIY)]
    B.fw_spectrum(L.handle, 1, scratch, nb, lam, kap)
    Py = t2n(L.get(B.FW_F_PHIY))
    lam_y = O.eigenvalues_desc(Py)
    assert np.max(np.abs(t2n(lam) - lam_y)) <= 1e-6 * lam_y[0]
    assert abs(float(kap[0]) - O.normalised_rank(Py)) <= 1e-5
    for f, b in zip((B.FW_F_T, B.FW_F_Q, B.FW_F_PHIY), before):
        assert torch.equal(L.get(f), b)
    # kappa alone; the two extremes of Sec. 3.2: equal eigenvalues -> 1, one dominant -> 1 / M
    L.set(B.FW_F_PHIX, 2.0 * torch.eye(M, device="cuda"))
    B.fw_spectrum(L.handle, 0, scratch, nb, None, kap)
    assert abs(float(kap[0]) - 1.0) <= 1e-6
    u = np.random.default_rng(5).standard_normal(M); u /= np.linalg.norm(u)
    R1 = np.outer(u, u).astype(np.float32); R1 = np.triu(R1) + np.triu(R1, 1).T
    L.set(B.FW_F_PHIX, torch.from_numpy(R1).cuda())
    B.fw_spectrum(L.handle, 0, scratch, nb, None, kap)
    assert abs(float(kap[0]) - 1.0 / M) <= 1e-4


def test_evd_from_samples_then_recursion_continues(env):
    """Covariance from samples (FP32 engine), EVD whitening with capped gains, then the recursion goes on from that
    state: Q = T^T T and Phi_y = T Phi_x T^T hold on the device state before and after."""
    torch, B = env
    M, rows = 96, 4000
    rng = np.random.default_rng(990)
    A = rng.standard_normal((M, M)) / np.sqrt(M)
    X = np.abs(rng.standard_normal((rows, M)) @ A).astype(np.float32)
    L = B.Layer(M, 4, beta=0.0, gamma=1.0)
    Lo = O.Layer(M, 4, oracle_hyper(L.desc))
    L.cov_update(torch.from_numpy(X).cuda()); O.cov_update(Lo, X)
    scratch, nb = scratch_for(torch, B, M)
    B.fw_evd_whiten(L.handle, scratch, nb, 2.0)
    Px = t2n(L.get(B.FW_F_PHIX))
    To, Qo, Yo, _ = oracle_state(Px.astype(np.float32), L.desc.eps, 2.0)
    assert rel_fro(t2n(L.get(B.FW_F_T)), To) <= TOL_FP32
    # against the oracle's own covariance the decomposition of a 1e-5-close matrix: gains are continuous in Phi_x
    # except at the rank boundary, so only the looser bound holds in general
    To2, _, _ = O.zca_transform(Lo.Phix, eps=L.desc.eps, g_max=2.0, use_jacobi=False)
    assert rel_fro(t2n(L.get(B.FW_F_T)), To2) <= 1e-3
    L.cond_reduce(3, 8)
    assert L.sync_status() in (B.FW_OK, B.FW_WARN_NO_SUBSPACE)
    T, Q, Y = t2n(L.get(B.FW_F_T)), t2n(L.get(B.FW_F_Q)), t2n(L.get(B.FW_F_PHIY))
    assert rel_fro(Q, T.T @ T) <= TOL_FP32
    assert rel_fro(Y, T @ Px @ T.T) <= TOL_FP32


def test_evd_then_leaky_recursion(env):
    """A leaky layer (gamma < 1) also tracks P = T Phi_x: after the decomposition the next reduction rebuilds it from
    the new T, and the invariants of the leaky update hold on the device state."""
    torch, B = env
    M = 80
    Phi32 = spd32(M, 1e3, 995)
    L = B.Layer(M, 4, beta=0.0, gamma=0.99)
    L.set(B.FW_F_PHIX, torch.from_numpy(Phi32).cuda())
    scratch, nb = scratch_for(torch, B, M)
    B.fw_evd_whiten(L.handle, scratch, nb, 2.0)
    To, _, _, _ = oracle_state(Phi32, L.desc.eps, 2.0)
    assert rel_fro(t2n(L.get(B.FW_F_T)), To) <= TOL_FP32
    L.cond_reduce(3, 8)
    assert L.sync_status() in (B.FW_OK, B.FW_WARN_NO_SUBSPACE)
    T, Q, Y = t2n(L.get(B.FW_F_T)), t2n(L.get(B.FW_F_Q)), t2n(L.get(B.FW_F_PHIY))
    assert rel_fro(Q, T.T @ T) <= TOL_FP32
    assert rel_fro(Y, T @ Phi32.astype(np.float64) @ T.T) <= TOL_FP32


def test_evd_argument_errors(env):
    torch, B = env
    M = 32
    L = B.Layer(M, 4)
    scratch, nb = scratch_for(torch, B, M)
    with pytest.raises(B.FwError) as e:
        B.fw_evd_whiten(L.handle, scratch, nb, 0.0)                   # no covariance yet
    assert e.value.status == B.FW_ERR_STATE
    L.set(B.FW_F_PHIX, torch.eye(M, device="cuda"))
    with pytest.raises(B.FwError) as e:
        B.fw_evd_whiten(L.handle, scratch, nb - 1024, 0.0)
    assert e.value.status == B.FW_ERR_WORKSPACE
    with pytest.raises(B.FwError) as e:
        B.fw_spectrum(L.handle, 2, scratch, nb, None, torch.zeros(1, device="cuda"))
    assert e.value.status == B.FW_ERR_INVALID_ARG
    assert B.fw_evd_scratch_bytes(0) == 0
