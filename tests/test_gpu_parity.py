"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle
on identical seeded inputs.  Bar: relative Frobenius error <= 1e-5 for the fp32
engine (<= 5e-3 for tensor-core engines, tested in test_gpu_tensorcore.py);
discrete decisions (argmax, coherent set) must agree except on near-ties, which
are replayed into the oracle."""
import numpy as np
import pytest

from oracle import fw_oracle as O
from paper_2010_01546_b200 import synth

from fwtest_util import TOL_FP32, group_reduce_with_replay, oracle_hyper, reduce_with_replay, rel_fro, t2n

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2010_01546_b200 import binding as B, build
    build.build_library()
    assert torch.cuda.is_available()
    return torch, B


def dev(torch, a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def check_moments(L, Lo, B, tol=TOL_FP32):
    assert rel_fro(t2n(L.get(B.FW_F_MU)), Lo.mu) <= tol
    assert rel_fro(t2n(L.get(B.FW_F_PHIX)), Lo.Phix) <= tol
    assert rel_fro(t2n(L.get(B.FW_F_PHI_DIAG)), Lo.phi) <= tol
    assert abs(float(L.get(B.FW_F_LAMBDA_BAR)[0]) - Lo.lam_bar) <= tol * abs(Lo.lam_bar)
    Px = t2n(L.get(B.FW_F_PHIX))
    assert np.array_equal(Px, Px.T)                      # exactly symmetric by construction


def check_transform(L, Lo, B, tol=TOL_FP32, phiy_scale="strict"):
    """T, Q, Qs: relative Frobenius error <= tol.  Phi_y = T Phi_x T^T: the same
    bound when phiy_scale == "strict".  With "product" the error is measured
    against || |T| |Phi_x| |T|^T ||_F, the scale of the standard forward error
    bound of the product: when the recursion has removed most of the power of a
    (nearly) rank-deficient covariance, Phi_y is the small remainder of a
    cancellation and fp32 storage of T and Phi_x alone perturbs it by
    eps * || |T| |Phi_x| |T|^T ||, which can exceed tol * ||Phi_y||."""
    T, Q, Py = t2n(L.get(B.FW_F_T)), t2n(L.get(B.FW_F_Q)), t2n(L.get(B.FW_F_PHIY))
    assert rel_fro(T, Lo.T) <= tol
    assert rel_fro(Q, Lo.Q) <= tol
    if phiy_scale == "strict":
        assert rel_fro(Py, Lo.phiy()) <= tol
    else:
        scale = np.linalg.norm(np.abs(Lo.T) @ np.abs(Lo.Phix) @ np.abs(Lo.T).T)
        assert np.linalg.norm(Py - Lo.phiy()) <= tol * scale
    assert rel_fro(t2n(L.get(B.FW_F_QS)), Lo.Qs) <= tol
    assert np.array_equal(Py, Py.T) and np.array_equal(Q, Q.T)


# ----------------------------------------------------------------------------
# the small single-layer workload, whole path
# ----------------------------------------------------------------------------
def test_single_linear_layer_whole_path(env):
    torch, B = env
    d = synth.single_linear_layer()            # M=64, N=32, B=128
    M, N = d["M"], d["N"]
    Xf = d["X"].astype(np.float32); Gf = d["G"].astype(np.float32)
    Wf = d["W"].astype(np.float32); bf = d["b"].astype(np.float32); gbf = d["gb"].astype(np.float32)
    L = B.Layer(M, N, alpha=0.9, beta=0.0, gamma=1.0, delta=0.25)
    Lo = O.Layer(M, N, oracle_hyper(L.desc))
    L.cov_update(dev(torch, Xf)); O.cov_update(Lo, Xf)
    check_moments(L, Lo, B)
    recs, replayed = reduce_with_replay(L, Lo, 8, 16, B, torch)
    check_transform(L, Lo, B)
    for r in recs:                                  # per-step scalars
        assert r["gpu_trace"][0] == pytest.approx(r["lam_e"], rel=1e-4)
        assert r["gpu_trace"][1] == pytest.approx(r["g_e"], rel=1e-4)
        assert int(r["gpu_trace"][2]) == r["set_size"]
    G = dev(torch, Gf)
    Gt = L.grad_transform(G)
    Gt_o = O.grad_transform(Lo, Gf)
    assert rel_fro(t2n(Gt), Gt_o) <= TOL_FP32
    W, b = dev(torch, Wf), dev(torch, bf)
    L.step(W, b, Gt, dev(torch, gbf), 0.1)
    W_o, b_o = O.sgd_step(Wf.astype(np.float64), bf.astype(np.float64), Gt_o, gbf, 0.1)
    assert rel_fro(t2n(W), W_o) <= TOL_FP32
    assert rel_fro(t2n(b), b_o) <= TOL_FP32
    assert L.sync_status() == B.FW_OK
    # the recursion did its job: condition number went down
    assert O.condition_number(t2n(L.get(B.FW_F_PHIY))) < O.condition_number(Lo.Phix)


# ----------------------------------------------------------------------------
# moments: ragged shapes, strides, two blocks, non-zero mean
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("M", [1, 7, 16, 17, 64, 144, 145])
@pytest.mark.parametrize("rows", [1, 127, 129, 3000])
def test_cov_update_shapes(env, M, rows):
    torch, B = env
    rng = np.random.default_rng(1000 * M + rows)
    L = B.Layer(M, 3, alpha=0.7, beta=0.0, gamma=1.0)
    Lo = O.Layer(M, 3, oracle_hyper(L.desc))
    ld = M + 5
    for blk in range(2):
        X = (np.abs(rng.standard_normal((rows, ld))) * rng.uniform(0.5, 2.0, ld) + 0.3 * blk).astype(np.float32)
        Xd = dev(torch, X)
        B.fw_cov_update(L.handle, Xd, rows, ld)
        O.cov_update(Lo, X[:, :M])
        if rows == 1 and blk == 0:
            # one row: covariance is exactly zero, mean is the row
            assert np.abs(t2n(L.get(B.FW_F_PHIX))).max() <= 1e-6 * (np.abs(X).max() ** 2)
            assert rel_fro(t2n(L.get(B.FW_F_MU)), Lo.mu) <= TOL_FP32
        else:
            check_moments(L, Lo, B)


def test_cov_update_large_mean_and_many_rows(env):
    # mean^2 / variance = 400: the one-pass covariance must not lose it to cancellation
    torch, B = env
    rng = np.random.default_rng(5)
    M, rows = 96, 40000
    Phi, U, lam = synth.spd_with_spectrum(M, 1e2, 9)
    X = (synth.gaussian_rows(rows, U, lam, 10) * 0.05 + 1.0).astype(np.float32)
    L = B.Layer(M, 4, alpha=0.5, beta=0.0, gamma=1.0)
    Lo = O.Layer(M, 4, oracle_hyper(L.desc))
    for blk in range(2):
        Xb = X[blk * 20000:(blk + 1) * 20000]
        L.cov_update(dev(torch, Xb)); O.cov_update(Lo, Xb)
    check_moments(L, Lo, B)


def test_cov_update_bf16_input_fp32_engine(env):
    torch, B = env
    rng = np.random.default_rng(6)
    M, rows = 80, 1000
    X = synth.to_bf16_grid(np.abs(rng.standard_normal((rows, M))).astype(np.float32))
    L = B.Layer(M, 4, x_dtype=B.FW_BF16, prec=B.FW_PREC_FP32, alpha=0.0, beta=0.0, gamma=1.0)
    Lo = O.Layer(M, 4, oracle_hyper(L.desc))
    Xd = torch.from_numpy(synth.bf16_bits(X).view(np.int16)).cuda().view(torch.bfloat16)
    L.cov_update(Xd); O.cov_update(Lo, X)
    check_moments(L, Lo, B)


def test_bias_compensation(env):
    torch, B = env
    rng = np.random.default_rng(7)
    M, N = 40, 9
    W = rng.standard_normal((N, M)).astype(np.float32); b = rng.standard_normal(N).astype(np.float32)
    L = B.Layer(M, N, alpha=0.5, beta=0.0, gamma=1.0)
    Lo = O.Layer(M, N, oracle_hyper(L.desc)); Lo.attach_params(W, b)
    Wd, bd = dev(torch, W), dev(torch, b)
    L.attach_params(Wd, bd)
    for blk in range(3):
        X = (rng.standard_normal((200, M)) + blk).astype(np.float32)
        L.cov_update(dev(torch, X)); O.cov_update(Lo, X)
    assert rel_fro(t2n(bd), Lo.b) <= TOL_FP32
    assert np.array_equal(t2n(Wd), W.astype(np.float64))


# ----------------------------------------------------------------------------
# recursion on an injected covariance
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("M,cond,K,P", [(7, 1e2, 3, 4), (64, 1e3, 8, 16), (145, 1e2, 4, 8), (256, 1e4, 8, 32),
                                        (256, 1e2, 1, 32), (300, 1e3, 3, 0),
                                        (400, 1e3, 4, 8),      # on chip, 8 CTAs of a cluster
                                        (577, 1e3, 3, 8),      # on chip, 16 CTAs, rows not 16-byte multiples
                                        (620, 1e3, 3, 8),      # on chip, close to the largest resident size
                                        (642, 1e3, 3, 8),      # rows not 16-byte multiples: one launch per pass
                                        (700, 1e3, 4, 8)])     # persistent launch, rows resident in shared memory
def test_recursion_injected_covariance(env, M, cond, K, P):
    torch, B = env
    Phi, _, _ = synth.spd_with_spectrum(M, cond, 500 + M, basis="qr" if M <= 300 else "householder")
    Phi32 = Phi.astype(np.float32); Phi32 = np.triu(Phi32) + np.triu(Phi32, 1).T
    L = B.Layer(M, 4, beta=0.0, gamma=1.0)
    Lo = O.Layer(M, 4, oracle_hyper(L.desc))
    L.set(B.FW_F_PHIX, dev(torch, Phi32)); Lo.set_phix(Phi32)
    assert abs(float(L.get(B.FW_F_LAMBDA_BAR)[0]) - Lo.lam_bar) <= 1e-5 * Lo.lam_bar
    recs, replayed = reduce_with_replay(L, Lo, K, P, B, torch)
    check_transform(L, Lo, B)
    # Q = T^T T on the device state itself
    T, Q = t2n(L.get(B.FW_F_T)), t2n(L.get(B.FW_F_Q))
    assert rel_fro(Q, T.T @ T) <= TOL_FP32
    # Phiy is T Phix T^T of the device's own state
    assert rel_fro(t2n(L.get(B.FW_F_PHIY)), T @ Phi32.astype(np.float64) @ T.T) <= TOL_FP32


def test_recursion_K_steps_in_one_call_match_single_steps(env):
    torch, B = env
    M = 128
    Phi, _, _ = synth.spd_with_spectrum(M, 1e3, 77)
    Phi32 = Phi.astype(np.float32); Phi32 = np.triu(Phi32) + np.triu(Phi32, 1).T
    La = B.Layer(M, 4, beta=0.0, gamma=1.0); Lb = B.Layer(M, 4, beta=0.0, gamma=1.0)
    for L in (La, Lb):
        L.set(B.FW_F_PHIX, dev(torch, Phi32))
    tr = torch.zeros(6 * 4, device="cuda")
    La.cond_reduce(6, 8, tr)
    for _ in range(6):
        Lb.cond_reduce(1, 8)
    for f in (B.FW_F_T, B.FW_F_Q, B.FW_F_PHIY):
        assert torch.equal(La.get(f), Lb.get(f))       # deterministic and identical
    t = t2n(tr).reshape(6, 4)
    assert np.all(t[:, 0] > 0) and np.all(t[:, 2] >= 1)


def test_recursion_maxcol_init_and_smoothing(env):
    torch, B = env
    M = 96
    Phi, _, _ = synth.spd_with_spectrum(M, 1e3, 78)
    Phi32 = Phi.astype(np.float32); Phi32 = np.triu(Phi32) + np.triu(Phi32, 1).T
    L = B.Layer(M, 4, beta=0.3, gamma=1.0, init=B.FW_INIT_MAXCOL)
    Lo = O.Layer(M, 4, oracle_hyper(L.desc))
    L.set(B.FW_F_PHIX, dev(torch, Phi32)); Lo.set_phix(Phi32)
    for _ in range(3):
        L.cond_reduce(2, 8); O.cond_reduce(Lo, 2, 8)
    check_transform(L, Lo, B)
    assert not np.allclose(t2n(L.get(B.FW_F_QS)), t2n(L.get(B.FW_F_Q)))


def test_recursion_degenerate_covariances(env):
    torch, B = env
    M = 32
    L = B.Layer(M, 4, beta=0.0, gamma=1.0)
    L.set(B.FW_F_PHIX, torch.zeros(M, M, device="cuda"))
    L.cond_reduce(2, 4)
    assert L.sync_status() == B.FW_WARN_NO_SUBSPACE
    assert torch.equal(L.get(B.FW_F_T), torch.eye(M, device="cuda"))
    assert torch.equal(L.get(B.FW_F_Q), torch.eye(M, device="cuda"))
    L2 = B.Layer(M, 4, beta=0.0, gamma=1.0)
    L2.set(B.FW_F_PHIX, 1e-9 * torch.eye(M, device="cuda"))      # xi^2 below c_abs
    L2.cond_reduce(1, 4)
    assert L2.sync_status() == B.FW_WARN_NO_SUBSPACE
    assert L2.sync_status() == B.FW_OK                             # cleared by the read
    # rank one: the estimate is the vector itself, the step sets its power to delta*lam_bar
    rng = np.random.default_rng(3)
    u = rng.standard_normal(M); u /= np.linalg.norm(u)
    Phi = (2.0 * np.outer(u, u)).astype(np.float32); Phi = np.triu(Phi) + np.triu(Phi, 1).T
    L3 = B.Layer(M, 4, beta=0.0, gamma=1.0)
    Lo = O.Layer(M, 4, oracle_hyper(L3.desc))
    L3.set(B.FW_F_PHIX, dev(torch, Phi)); Lo.set_phix(Phi)
    L3.cond_reduce(1, 2); O.cond_reduce(Lo, 1, 2)
    assert rel_fro(t2n(L3.get(B.FW_F_T)), Lo.T) <= TOL_FP32
    assert rel_fro(t2n(L3.get(B.FW_F_Q)), Lo.Q) <= TOL_FP32
    # The step removes (1 - g_e) of the only eigenvalue (2 -> delta*lam_bar = 1/64): the fp32 state
    # carries rounding errors relative to the matrix before the step, so that is the scale of the bound.
    err = np.linalg.norm(t2n(L3.get(B.FW_F_PHIY)) - Lo.phiy())
    assert err <= TOL_FP32 * np.linalg.norm(Phi.astype(np.float64))
    v = u / np.linalg.norm(u)
    assert float(v @ t2n(L3.get(B.FW_F_PHIY)) @ v) == pytest.approx(0.25 * Lo.lam_bar, rel=1e-3)


def test_state_errors_and_call_order(env):
    torch, B = env
    L = B.Layer(16, 4, beta=0.0, gamma=1.0)
    with pytest.raises(B.FwError) as e:
        L.cond_reduce(1, 1)                      # no covariance yet
    assert e.value.status == B.FW_ERR_STATE
    X = torch.randn(10, 16, device="cuda")
    with pytest.raises(B.FwError) as e:
        B.fw_cov_update(L.handle, X, 0, 16)
    assert e.value.status == B.FW_ERR_SHAPE
    with pytest.raises(B.FwError) as e:
        B.fw_cov_update(L.handle, X, 10, 8)      # ldx < M
    assert e.value.status == B.FW_ERR_SHAPE
    G = torch.randn(4, 16, device="cuda")
    G2 = torch.randn(2 * 4 * 16, device="cuda")
    with pytest.raises(B.FwError) as e:
        B.fw_grad_transform(L.handle, G2[:64], G2[16:80])      # partial overlap
    assert e.value.status == B.FW_ERR_INVALID_ARG
    with pytest.raises(B.FwError) as e:
        B.fw_cov_update(L.handle, X, 10, 16, 7)  # unknown flag
    assert e.value.status == B.FW_ERR_INVALID_ARG
    Lg = B.Layer(16, 4)                          # gamma = 0.99 (paper default) is supported
    Lg.cov_update(X)
    Lg.cond_reduce(1, 1)
    assert Lg.sync_status() in (B.FW_OK, B.FW_WARN_NO_SUBSPACE)
    # before any step Qs = I: the transform is the identity
    out = L.grad_transform(G)
    assert torch.equal(out, G)


# ----------------------------------------------------------------------------
# gradient transform + step
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("M,N", [(64, 32), (144, 16), (145, 3), (300, 70), (576, 64)])
def test_grad_transform_and_fused_step(env, M, N):
    torch, B = env
    rng = np.random.default_rng(M + N)
    Phi, _, _ = synth.spd_with_spectrum(M, 1e2, 900 + M)
    Phi32 = Phi.astype(np.float32); Phi32 = np.triu(Phi32) + np.triu(Phi32, 1).T
    L = B.Layer(M, N, beta=0.0, gamma=1.0)
    L.set(B.FW_F_PHIX, dev(torch, Phi32))
    L.cond_reduce(3, 4)
    Qs = t2n(L.get(B.FW_F_QS))
    G = rng.standard_normal((N, M)).astype(np.float32)
    W = rng.standard_normal((N, M)).astype(np.float32)
    b = rng.standard_normal(N).astype(np.float32); gb = rng.standard_normal(N).astype(np.float32)
    Gt = L.grad_transform(dev(torch, G))
    ref = G.astype(np.float64) @ Qs
    assert rel_fro(t2n(Gt), ref) <= TOL_FP32
    Wd, bd = dev(torch, W), dev(torch, b)
    B.fw_group_grad_transform_step([L.handle], [dev(torch, G)], [Wd], [bd], [dev(torch, gb)], 0.05)
    assert rel_fro(t2n(Wd), W - 0.05 * ref) <= TOL_FP32
    assert rel_fro(t2n(bd), b.astype(np.float64) - 0.05 * gb) <= TOL_FP32


# ----------------------------------------------------------------------------
# grouped calls over a mixed layer set (ResNet-20-shaped, reduced batch)
# ----------------------------------------------------------------------------
def test_grouped_layer_set_three_batches(env):
    # Twin layer sets on the same inputs.  Set A takes the K steps of a batch in ONE grouped call, the launch
    # shape the benchmark times; set B takes them one grouped call per step, each step's discrete decisions read
    # back and replayed into the oracle where they flipped on a near-tie.  B is compared with the oracle, and A
    # must equal B bit for bit.  Every layer has rows >= M, so Phi_y is held to the strict bound.
    torch, B = env
    shapes = synth.resnet20_shapes(B=4)
    shapes = [shapes[0], shapes[1], shapes[5], shapes[6], dict(shapes[10], B=16), dict(shapes[14], B=16)]
    setA, setB, oras = [], [], []
    for i, s in enumerate(shapes):
        rows, M, N = synth.shape_dims(s)
        assert rows >= M
        LA = B.Layer(M, N, alpha=0.9, beta=0.0, gamma=1.0, delta=0.25)
        LB = B.Layer(M, N, alpha=0.9, beta=0.0, gamma=1.0, delta=0.25)
        setA.append(LA); setB.append(LB); oras.append(O.Layer(M, N, oracle_hyper(LA.desc)))
    K, P, lr = 4, 16, 0.1
    hA, hB = [L.handle for L in setA], [L.handle for L in setB]
    for batch in range(3):
        ins = [synth.conv_layer_inputs(s["B"], s["HW"], s["C_in"], s["C_out"], s["k"], synth.layer_seed(2, i),
                                       batch_index=batch) for i, s in enumerate(shapes)]
        if batch == 0:
            Ws = [dev(torch, d["W"]) for d in ins]; bs = [dev(torch, d["b"]) for d in ins]
            Wo = [d["W"].astype(np.float64) for d in ins]; bo = [d["b"].astype(np.float64) for d in ins]
        Xd = [dev(torch, d["X"]) for d in ins]
        Gd = [dev(torch, d["G"]) for d in ins]
        gbd = [dev(torch, d["gb"]) for d in ins]
        for hs in (hA, hB):
            B.fw_group_cov_update(hs, Xd, [d["rows"] for d in ins], [d["M"] for d in ins])
        for Lo, d in zip(oras, ins):
            O.cov_update(Lo, d["X"])
        for L, Lo in zip(setA, oras):
            check_moments(L, Lo, B)
        traces = [torch.zeros(K * 4, device="cuda") for _ in setA]
        B.fw_group_cond_reduce(hA, K, P, traces)
        recs, _ = group_reduce_with_replay(setB, oras, K, P, B, torch)
        for LA, LB, Lo, tr, rec in zip(setA, setB, oras, traces, recs):
            check_transform(LB, Lo, B)                     # strict bound on Phi_y too
            for f in (B.FW_F_T, B.FW_F_Q, B.FW_F_QS, B.FW_F_PHIY):
                assert torch.equal(LA.get(f), LB.get(f))   # K steps in one call == K calls of one step
            t = t2n(tr).reshape(K, 4)
            for k in range(K):
                assert t[k, 0] == pytest.approx(rec[k]["lam_e"], rel=1e-4)
                assert int(t[k, 2]) == rec[k]["set_size"] and int(t[k, 3]) == rec[k]["m_prime"]
        B.fw_group_grad_transform_step(hA, Gd, Ws, bs, gbd, lr)
        for j, (Lo, d) in enumerate(zip(oras, ins)):
            Gt = O.grad_transform(Lo, d["G"])
            Wo[j], bo[j] = O.sgd_step(Wo[j], bo[j], Gt, d["gb"].astype(np.float64), lr)
            assert rel_fro(t2n(Ws[j]), Wo[j]) <= TOL_FP32
            assert rel_fro(t2n(bs[j]), bo[j]) <= TOL_FP32
    for L in setA + setB:
        assert L.sync_status() == B.FW_OK


def test_grouped_streamed_layers_K_steps_in_one_call_match_single_steps(env):
    # layers too large for the on-chip kernel (streaming passes, one launch per pass batched over layers)
    torch, B = env
    Ms = [640, 1000, 1024]
    setA, setB = [], []
    for i, M in enumerate(Ms):
        Phi, _, _ = synth.spd_with_spectrum(M, 1e3, 1200 + i, basis="householder")
        Phi32 = Phi.astype(np.float32); Phi32 = np.triu(Phi32) + np.triu(Phi32, 1).T
        for st in (setA, setB):
            L = B.Layer(M, 4, beta=0.0, gamma=1.0)
            L.set(B.FW_F_PHIX, dev(torch, Phi32))
            st.append(L)
    B.fw_group_cond_reduce([L.handle for L in setA], 3, 8)
    for _ in range(3):
        B.fw_group_cond_reduce([L.handle for L in setB], 1, 8)
    for LA, LB in zip(setA, setB):
        for f in (B.FW_F_T, B.FW_F_Q, B.FW_F_PHIY):
            assert torch.equal(LA.get(f), LB.get(f))


def test_get_set_roundtrip_and_set_T(env):
    torch, B = env
    M = 50
    rng = np.random.default_rng(11)
    L = B.Layer(M, 4, beta=0.0, gamma=1.0)
    T = (np.eye(M) + 0.1 * rng.standard_normal((M, M))).astype(np.float32)
    L.set(B.FW_F_T, dev(torch, T))
    assert np.array_equal(t2n(L.get(B.FW_F_T)), T.astype(np.float64))
    assert rel_fro(t2n(L.get(B.FW_F_Q)), T.astype(np.float64).T @ T.astype(np.float64)) <= TOL_FP32
    Phi, _, _ = synth.spd_with_spectrum(M, 10.0, 12)
    Phi32 = Phi.astype(np.float32); Phi32 = np.triu(Phi32) + np.triu(Phi32, 1).T
    L.set(B.FW_F_PHIX, dev(torch, Phi32))
    Py = t2n(L.get(B.FW_F_PHIY))                       # re-sync through the dense products
    T64 = T.astype(np.float64)
    assert rel_fro(Py, T64 @ Phi32.astype(np.float64) @ T64.T) <= TOL_FP32
    assert np.array_equal(Py, Py.T)
    mu = rng.standard_normal(M).astype(np.float32)
    L.set(B.FW_F_MU, dev(torch, mu))
    assert np.array_equal(t2n(L.get(B.FW_F_MU)), mu.astype(np.float64))


# ----------------------------------------------------------------------------
# leaky transform (gamma < 1, Eqs. 42 and 44 in full)
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("M,gamma,K,P", [(7, 0.9, 4, 4), (64, 0.99, 8, 16), (145, 0.9, 5, 8), (256, 0.99, 6, 16),
                                         (700, 0.95, 3, 8)])
def test_recursion_leaky_injected_covariance(env, M, gamma, K, P):
    torch, B = env
    Phi, _, _ = synth.spd_with_spectrum(M, 1e3, 600 + M, basis="qr" if M <= 300 else "householder")
    Phi32 = Phi.astype(np.float32); Phi32 = np.triu(Phi32) + np.triu(Phi32, 1).T
    L = B.Layer(M, 4, beta=0.2, gamma=gamma)
    Lo = O.Layer(M, 4, oracle_hyper(L.desc))
    L.set(B.FW_F_PHIX, dev(torch, Phi32)); Lo.set_phix(Phi32)
    recs, replayed = reduce_with_replay(L, Lo, K, P, B, torch)
    check_transform(L, Lo, B)
    T, Q = t2n(L.get(B.FW_F_T)), t2n(L.get(B.FW_F_Q))
    assert rel_fro(Q, T.T @ T) <= TOL_FP32                      # Eq. 44 tracks T^T T with leakage too
    assert rel_fro(t2n(L.get(B.FW_F_PHIY)), T @ Phi32.astype(np.float64) @ T.T) <= TOL_FP32
    assert not np.allclose(T, T.T, atol=1e-4) or K < 2


def test_leaky_step_without_subspace_only_leaks(env):
    # Phi_x = 0: a_e = 0, the step is T <- gamma T + (1 - gamma) I, i.e. T stays I; with an injected T != I it moves
    torch, B = env
    M = 24
    rng = np.random.default_rng(4)
    T0 = (np.eye(M) + 0.2 * rng.standard_normal((M, M))).astype(np.float32)
    L = B.Layer(M, 4, beta=0.0, gamma=0.8)
    Lo = O.Layer(M, 4, oracle_hyper(L.desc))
    L.set(B.FW_F_T, dev(torch, T0)); Lo.T = T0.astype(np.float64); Lo.Q = Lo.T.T @ Lo.T; Lo.Qs = Lo.Q.copy()
    L.set(B.FW_F_PHIX, torch.zeros(M, M, device="cuda")); Lo.set_phix(np.zeros((M, M)))
    L.cond_reduce(3, 2); O.cond_reduce(Lo, 3, 2)
    assert L.sync_status() == B.FW_WARN_NO_SUBSPACE
    assert rel_fro(t2n(L.get(B.FW_F_T)), Lo.T) <= TOL_FP32
    assert rel_fro(t2n(L.get(B.FW_F_Q)), Lo.Q) <= TOL_FP32


def test_whole_path_paper_hyperparameters_two_batches(env):
    # the recursive method's own hyper-parameters: alpha 0.1, beta 0.1, gamma 0.99, delta 0.25
    torch, B = env
    d = synth.single_linear_layer(M=96, N=24, B=512, seed=synth.layer_seed(1, 7))
    M, N = d["M"], d["N"]
    L = B.Layer(M, N)
    Lo = O.Layer(M, N, oracle_hyper(L.desc))
    W = d["W"].astype(np.float32); b = d["b"].astype(np.float32)
    Wd, bd = dev(torch, W), dev(torch, b)
    L.attach_params(Wd, bd); Lo.attach_params(W, b)
    Wo, bo = W.astype(np.float64), b.astype(np.float64)
    for blk in range(2):
        X = d["X"][blk * 256:(blk + 1) * 256].astype(np.float32) + 0.1 * blk
        L.cov_update(dev(torch, X)); O.cov_update(Lo, X)
        check_moments(L, Lo, B)
        recs, _ = reduce_with_replay(L, Lo, 2, 8, B, torch)
        check_transform(L, Lo, B)
        G = d["G"].astype(np.float32)
        Gt = L.grad_transform(dev(torch, G))
        Gt_o = O.grad_transform(Lo, G)
        assert rel_fro(t2n(Gt), Gt_o) <= TOL_FP32
    assert rel_fro(t2n(bd), Lo.b) <= TOL_FP32
