"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (grouped calls,
tensor-core engine), on sampled outputs the oracle's definition can give one by one, and on
properties that hold at any size."""
import numpy as np
import pytest

from oracle import fw_oracle as O
from paper_2010_01546_b200 import synth

from fwtest_util import TOL_FP32, TOL_TC, oracle_hyper, reduce_with_replay, rel_fro, t2n

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2010_01546_b200 import binding as B, build
    build.build_library()
    return torch, B


def sampled_cov(X, mu, pairs):
    """(1/rows) sum (x_i - mu_i)(x_j - mu_j) for the sampled (i, j), in fp64 (Eq. 5 entry by entry)."""
    out = []
    for i, j in pairs:
        out.append(float(np.mean((X[:, i].astype(np.float64) - mu[i]) * (X[:, j].astype(np.float64) - mu[j]))))
    return np.array(out)


@pytest.mark.parametrize("engine", ["tc", "fp32"])
def test_resnet20_full_batch_grouped_cov_update_sampled(env, engine):
    torch, B = env
    shapes = synth.resnet20_shapes(128)
    ids = [0, 5, 10]                                  # one layer of each of the three shapes, full B = 128
    ins = [synth.conv_layer_inputs(shapes[i]["B"], shapes[i]["HW"], shapes[i]["C_in"], shapes[i]["C_out"], 3,
                                   synth.layer_seed(2, i)) for i in ids]
    prec = B.FW_PREC_TF32 if engine == "tc" else B.FW_PREC_FP32
    tol = TOL_TC if engine == "tc" else TOL_FP32
    Ls = [B.Layer(d["M"], d["N"], alpha=0.9, beta=0.0, gamma=1.0, prec=prec) for d in ins]
    Xd = [torch.from_numpy(d["X"]).cuda() for d in ins]
    B.fw_group_cov_update([L.handle for L in Ls], Xd, [d["rows"] for d in ins], [d["M"] for d in ins])
    rng = np.random.default_rng(0)
    for L, d in zip(Ls, ins):
        M, X = d["M"], d["X"]
        mu = X.astype(np.float64).mean(axis=0)
        assert rel_fro(t2n(L.get(B.FW_F_MU)), mu) <= tol
        Px = t2n(L.get(B.FW_F_PHIX))
        assert np.array_equal(Px, Px.T)
        pairs = [(int(rng.integers(M)), int(rng.integers(M))) for _ in range(60)] + [(k, k) for k in (0, M // 2, M - 1)]
        ref = sampled_cov(X, mu, pairs)
        got = np.array([Px[i, j] for i, j in pairs])
        scale = np.sqrt(np.array([Px[i, i] * Px[j, j] for i, j in pairs]))      # entry tolerance relative to the
        assert np.all(np.abs(got - ref) <= tol * scale + 1e-12)                    # geometric mean of the variances
        phi = t2n(L.get(B.FW_F_PHI_DIAG))
        k = M // 3
        assert phi[k] == pytest.approx(float(np.mean(X[:, k].astype(np.float64) ** 2)), rel=tol)
        assert L.sync_status() == B.FW_OK


def test_resnet50_shaped_bf16_layers_sampled(env):
    torch, B = env
    # the widest and the longest layer of the ResNet-50-shaped set at B = 256, bf16 inputs
    for (rows, M, seed) in ((12544, 4608, 31), (802816, 64, 32)):
        rng = np.random.default_rng(seed)
        C = M if M < 512 else 512
        S = synth.wishart_corr(C, seed, decades=1.0)
        Lc = np.linalg.cholesky(S + 1e-9 * np.eye(C))
        X = np.empty((rows, M), dtype=np.float32)
        for r0 in range(0, rows, 65536):
            r1 = min(rows, r0 + 65536)
            z = np.abs(rng.standard_normal((r1 - r0, C)) @ Lc.T).astype(np.float32)
            X[r0:r1] = np.tile(z, (1, M // C))[:, :M] * (1.0 + 0.1 * rng.standard_normal(M)).astype(np.float32)
        X = synth.to_bf16_grid(X)
        L = B.Layer(M, 64, alpha=0.9, beta=0.0, gamma=1.0, x_dtype=B.FW_BF16, prec=B.FW_PREC_BF16)
        Xd = torch.from_numpy(synth.bf16_bits(X).view(np.int16)).cuda().view(torch.bfloat16)
        L.cov_update(Xd)
        mu = X.astype(np.float64).mean(axis=0)
        assert rel_fro(t2n(L.get(B.FW_F_MU)), mu) <= TOL_TC
        Px = t2n(L.get(B.FW_F_PHIX))
        pairs = [(int(rng.integers(M)), int(rng.integers(M))) for _ in range(40)] + [(0, 0), (M - 1, M - 1)]
        ref = sampled_cov(X, mu, pairs)
        got = np.array([Px[i, j] for i, j in pairs])
        scale = np.sqrt(np.array([Px[i, i] * Px[j, j] for i, j in pairs]))
        assert np.all(np.abs(got - ref) <= TOL_TC * scale + 1e-12)
        assert np.array_equal(Px, Px.T)
        assert L.sync_status() == B.FW_OK
        del L, Xd


def test_recursion_stress_size_against_oracle(env):
    # M = 1152 (streaming multi-launch path), cond 1e4, K = 3, P = 32: the oracle still finishes in seconds
    torch, B = env
    M = 1152
    Phi, _, _ = synth.spd_with_spectrum(M, 1e4, synth.layer_seed(5, 0), basis="householder")
    Phi32 = Phi.astype(np.float32); Phi32 = np.triu(Phi32) + np.triu(Phi32, 1).T
    L = B.Layer(M, 4, beta=0.0, gamma=1.0)
    Lo = O.Layer(M, 4, oracle_hyper(L.desc))
    L.set(B.FW_F_PHIX, torch.from_numpy(Phi32).cuda()); Lo.set_phix(Phi32)
    tr = torch.zeros(3 * 4, device="cuda")
    L.cond_reduce(3, 32, tr)
    rec = O.cond_reduce(Lo, 3, 32, record_cond=True)
    t = t2n(tr).reshape(3, 4)
    assert all(int(t[k, 3]) == rec[k]["m_prime"] and int(t[k, 2]) == rec[k]["set_size"] for k in range(3)) or \
        min(min(r["margin_argmax"], r["margin_set"]) for r in rec) < 1e-4
    if all(int(t[k, 3]) == rec[k]["m_prime"] and int(t[k, 2]) == rec[k]["set_size"] for k in range(3)):
        assert rel_fro(t2n(L.get(B.FW_F_T)), Lo.T) <= TOL_FP32
        assert rel_fro(t2n(L.get(B.FW_F_Q)), Lo.Q) <= TOL_FP32
        assert rel_fro(t2n(L.get(B.FW_F_PHIY)), Lo.phiy()) <= TOL_FP32
        assert np.allclose(t[:, 0], [r["lam_e"] for r in rec], rtol=1e-4)
    # condition number after the steps, against the oracle's (log10 within 0.1)
    c_gpu = O.condition_number(t2n(L.get(B.FW_F_PHIY)))
    c_ora = O.condition_number(Lo.phiy())
    assert abs(np.log10(c_gpu) - np.log10(c_ora)) <= 0.1
    assert c_ora <= rec[0]["cond_before"] * (1 + 1e-6)


@pytest.mark.parametrize("M,K", [(2304, 8), (4608, 2)])
def test_recursion_large_M_properties(env, M, K):
    # sizes beyond what the oracle does in seconds: invariants of the device state, checked in fp64
    torch, B = env
    Phi, _, _ = synth.spd_with_spectrum(M, 1e4, synth.layer_seed(5, 1), basis="householder")
    Phi32 = torch.from_numpy(Phi.astype(np.float32)).cuda()
    Phi32 = torch.triu(Phi32) + torch.triu(Phi32, 1).T
    L = B.Layer(M, 4, beta=0.0, gamma=1.0)
    L.set(B.FW_F_PHIX, Phi32)
    tr = torch.zeros(K * 4, device="cuda")
    L.cond_reduce(K, 32, tr)
    T = L.get(B.FW_F_T).double(); Q = L.get(B.FW_F_Q).double(); Py = L.get(B.FW_F_PHIY).double()
    assert float((Q - T.T @ T).norm() / Q.norm()) <= TOL_FP32                   # Eq. 44 == T^T T
    ref = T @ Phi32.double() @ T.T
    assert float((Py - ref).norm() / ref.norm()) <= TOL_FP32                     # Phi_y == T Phi_x T^T
    assert torch.equal(Py, Py.T) and torch.equal(Q, Q.T)
    t = t2n(tr).reshape(K, 4)
    lam_bar = float(L.get(B.FW_F_LAMBDA_BAR)[0])
    assert np.allclose(t[:, 1], 0.25 * lam_bar / np.maximum(t[:, 0], 1e-5), rtol=1e-5)   # Eq. 40 on the trace
    # a Rayleigh quotient of Phi_y: between the floor the steps impose and the largest eigenvalue of Phi_x (= 1)
    assert np.all(t[:, 0] > 0.25 * lam_bar) and np.all(t[:, 0] <= 1.0 + 1e-4)
    assert L.sync_status() == B.FW_OK


def test_cost_sweep_layer_full_size_sampled(env):
    # the large-batch layer of the cost sweep at B = 256 (M = 2304, N = 256, rows = 50176, fp32 inputs, TF32
    # engine), as bench.py runs it: Gram on CTA pairs, K = 8 recursion steps (with the tensor-core re-sync of
    # Phi_y), G Qs with K split over a cluster
    torch, B = env
    d = synth.cost_sweep_layer(256)
    M, N, X = d["M"], d["N"], d["X"]
    L = B.Layer(M, N, alpha=0.9, beta=0.0, gamma=1.0, delta=0.25, prec=B.FW_PREC_TF32)
    Xd = torch.from_numpy(X).cuda()
    rng = np.random.default_rng(4)
    mu = X.astype(np.float64).mean(axis=0)
    sd = X.astype(np.float64).std(axis=0)
    for blk in range(2):                              # second block: running average with the same data
        L.cov_update(Xd)
    assert np.all(np.abs(t2n(L.get(B.FW_F_MU)) - mu) <= TOL_TC * sd)      # zero-mean data: error relative to the spread
    Px = t2n(L.get(B.FW_F_PHIX))
    assert np.array_equal(Px, Px.T)
    pairs = [(int(rng.integers(M)), int(rng.integers(M))) for _ in range(60)] + [(0, 0), (M // 2, M // 2), (M - 1, M - 1)]
    ref = sampled_cov(X, mu, pairs)                   # both blocks have the same covariance
    got = np.array([Px[i, j] for i, j in pairs])
    scale = np.sqrt(np.array([Px[i, i] * Px[j, j] for i, j in pairs]))
    assert np.all(np.abs(got - ref) <= TOL_TC * scale + 1e-12)
    tr = torch.zeros(8 * 4, dtype=torch.float32, device="cuda")
    L.cond_reduce(8, 16, trace=tr)
    assert L.sync_status() == B.FW_OK
    tr = t2n(tr).reshape(8, 4).astype(np.float64)    # per step: lambda_e, g_e, |set|, m'
    T = t2n(L.get(B.FW_F_T)).astype(np.float64)
    Q = t2n(L.get(B.FW_F_Q)).astype(np.float64)
    assert rel_fro(Q, T.T @ T) <= 1e-4               # Eq. 44 tracks T^T T
    Py = t2n(L.get(B.FW_F_PHIY)).astype(np.float64)
    assert rel_fro(Py, T @ Px.astype(np.float64) @ T.T) <= TOL_TC
    # every step scales one unit direction v by sqrt(g_e): (I + a v v^T) Phi_y (I + a v v^T) has the trace of Phi_y
    # plus (g_e - 1) lambda_e, exactly (Eqs. 36, 40-42); the spectrum's top is nearly flat, so the directions found
    # carry about the largest eigenvalue and are scaled down
    lam_max = np.linalg.eigvalsh(Px.astype(np.float64))[-1]
    assert np.all(tr[:, 0] > 0.5 * lam_max) and np.all(tr[:, 1] < 0.5) and np.all(tr[:, 2] >= 1)
    drop = float(np.sum((1.0 - tr[:, 1]) * tr[:, 0]))
    assert abs(np.trace(Px.astype(np.float64)) - drop - np.trace(Py)) <= TOL_TC * drop
    G = torch.from_numpy(d["G"]).cuda()
    Gt = t2n(L.grad_transform(G))
    Qs = t2n(L.get(B.FW_F_QS)).astype(np.float64)
    e = rel_fro(Gt, d["G"].astype(np.float64) @ Qs)
    assert e <= TOL_TC, e
    assert L.sync_status() == B.FW_OK


@pytest.mark.parametrize("M,cond,K", [(256, 1e6, 32), (256, 1e2, 8), (640, 1e6, 8)])
def test_recursion_stress_condition_number_after_every_step(env, M, cond, K):
    # the recursion stress sweep's corner: condition number 1e6, up to 32 steps of 32 power iterations, the
    # condition number of Phi_y after every step against the oracle's (both evaluated by the oracle's eigenvalue
    # routine in fp64; at 1e6 an fp32 Phi_y carries errors of a tenth of its smallest eigenvalue, hence log10
    # within 0.1), on chip (M = 256) and through the persistent launch (M = 640)
    torch, B = env
    Phi, _, _ = synth.spd_with_spectrum(M, cond, synth.layer_seed(5, 7), basis="qr" if M <= 512 else "householder")
    Phi32 = Phi.astype(np.float32); Phi32 = np.triu(Phi32) + np.triu(Phi32, 1).T
    L = B.Layer(M, 4, beta=0.0, gamma=1.0)
    Lo = O.Layer(M, 4, oracle_hyper(L.desc))
    L.set(B.FW_F_PHIX, torch.from_numpy(Phi32).cuda()); Lo.set_phix(Phi32)
    c_prev = O.condition_number(Lo.Phix)
    for k in range(K):
        reduce_with_replay(L, Lo, 1, 32, B, torch)
        c_dev = O.condition_number(t2n(L.get(B.FW_F_PHIY)))
        c_ora = O.condition_number(Lo.phiy())
        assert abs(np.log10(c_dev) - np.log10(c_ora)) <= 0.1, (k, c_dev, c_ora)
        assert c_ora <= c_prev * (1 + 1e-6), (k, c_ora, c_prev)      # the steps never raise it (Sec. 4)
        c_prev = c_ora
    assert rel_fro(t2n(L.get(B.FW_F_T)), Lo.T) <= 10 * TOL_FP32     # 32 steps of fp32 rounding compound
    assert rel_fro(t2n(L.get(B.FW_F_Q)), Lo.Q) <= 10 * TOL_FP32
    assert L.sync_status() == B.FW_OK
