"""GPU tests of the boundary's finer points, through the C ABI: blocks spread over
several calls (FW_COV_ACCUMULATE), the in-place gradient transform, per-layer
device-side status (time-out, non-finite values), against the fp64 oracle."""
import numpy as np
import pytest

from oracle import fw_oracle as O
from paper_2010_01546_b200 import synth

from fwtest_util import TOL_FP32, TOL_TC, oracle_hyper, rel_fro, t2n

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2010_01546_b200 import binding as B, build
    build.build_library()
    return torch, B


def to_dev(torch, X, bf16):
    if bf16:
        return torch.from_numpy(synth.bf16_bits(X).view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(X)).cuda()


def check(L, Lo, B, tol):
    assert rel_fro(t2n(L.get(B.FW_F_MU)), Lo.mu) <= tol
    e = rel_fro(t2n(L.get(B.FW_F_PHIX)), Lo.Phix)
    assert e <= tol, e
    assert rel_fro(t2n(L.get(B.FW_F_PHI_DIAG)), Lo.phi) <= tol
    assert abs(float(L.get(B.FW_F_LAMBDA_BAR)[0]) - Lo.lam_bar) <= tol * abs(Lo.lam_bar)
    Px = t2n(L.get(B.FW_F_PHIX))
    assert np.array_equal(Px, Px.T)


# A block of L batches (Sec. 2): calls with FW_COV_ACCUMULATE, closed by one with FW_COV_COMMIT, give what one
# call on the concatenated rows gives -- which is how the oracle takes the block.
@pytest.mark.parametrize("engine,M,chunks", [
    ("fp32", 17, (40, 1, 129)), ("fp32", 144, (300, 700, 200)),
    ("tf32", 144, (300, 700, 200)),          # short calls: centred on the pilot mean of the block's first call
    ("tf32", 144, (5000, 4100, 6000)),       # long calls: unshifted, column sums out of the tensor core
    ("tf32", 160, (5000, 300, 4500)),        # a short call inside an unshifted block
    ("tf32", 288, (500, 5000, 100)),         # a long call inside a pilot-centred block
    ("tf32", 576, (30157, 31000)),           # CTA-pair kernel
    ("bf16", 64, (40000, 33000, 100)), ("bf16", 576, (30157, 1000, 31000)),
])
def test_block_accumulated_over_several_calls(env, engine, M, chunks):
    torch, B = env
    rng = np.random.default_rng(M * 41 + len(chunks) + sum(chunks))
    bf16 = engine == "bf16"
    kw = dict(alpha=0.6, beta=0.0, gamma=1.0)
    if engine == "tf32":
        kw.update(prec=B.FW_PREC_TF32)
    elif bf16:
        kw.update(prec=B.FW_PREC_BF16, x_dtype=B.FW_BF16)
    tol = TOL_FP32 if engine == "fp32" else TOL_TC
    N = 5
    L = B.Layer(M, N, **kw)
    Lo = O.Layer(M, N, oracle_hyper(L.desc))
    W = rng.standard_normal((N, M)).astype(np.float32); b = rng.standard_normal(N).astype(np.float32)
    Wd, bd = to_dev(torch, W, False), to_dev(torch, b, False)
    L.attach_params(Wd, bd); Lo.attach_params(W, b)
    scale = rng.uniform(0.5, 2.0, M)
    mix = np.abs(rng.standard_normal((4, M))) * 0.3
    for blk in range(2):                      # second block: running average; the accumulators start afresh
        parts = []
        for c, rows in enumerate(chunks):
            F = np.abs(rng.standard_normal((rows, 4)))
            X = (np.abs(rng.standard_normal((rows, M))) * scale + F @ mix + 0.2 * blk + 0.05 * c).astype(np.float32)
            if bf16:
                X = synth.to_bf16_grid(X)
            parts.append(X)
            flag = B.FW_COV_COMMIT if c == len(chunks) - 1 else B.FW_COV_ACCUMULATE
            mu_before = L.get(B.FW_F_MU).clone()
            L.cov_update(to_dev(torch, X, bf16), flag)
            if flag == B.FW_COV_ACCUMULATE:
                assert torch.equal(L.get(B.FW_F_MU), mu_before)       # an open block changes no moment
        O.cov_update(Lo, np.concatenate(parts, axis=0))
        check(L, Lo, B, tol)
        assert rel_fro(t2n(bd), Lo.b) <= tol                            # Eq. 31 once per block
    assert L.sync_status() == B.FW_OK


def test_grouped_accumulate_with_layers_in_different_block_states(env):
    torch, B = env
    rng = np.random.default_rng(77)
    Ms = [48, 144, 320]
    Ls = [B.Layer(M, 4, alpha=0.5, beta=0.0, gamma=1.0, prec=B.FW_PREC_TF32) for M in Ms]
    Los = [O.Layer(M, 4, oracle_hyper(L.desc)) for M, L in zip(Ms, Ls)]
    X1 = [np.abs(rng.standard_normal((700, M))).astype(np.float32) for M in Ms]
    X2 = [np.abs(rng.standard_normal((900, M))).astype(np.float32) + 0.3 for M in Ms]
    # layer 0 opened its block on its own before the grouped calls
    X0 = np.abs(rng.standard_normal((333, Ms[0]))).astype(np.float32)
    Ls[0].cov_update(to_dev(torch, X0, False), B.FW_COV_ACCUMULATE)
    hs = [L.handle for L in Ls]
    B.fw_group_cov_update(hs, [to_dev(torch, x, False) for x in X1], [700] * 3, Ms, B.FW_COV_ACCUMULATE)
    B.fw_group_cov_update(hs, [to_dev(torch, x, False) for x in X2], [900] * 3, Ms, B.FW_COV_COMMIT)
    for i, (L, Lo) in enumerate(zip(Ls, Los)):
        parts = ([X0] if i == 0 else []) + [X1[i], X2[i]]
        O.cov_update(Lo, np.concatenate(parts, axis=0))
        check(L, Lo, B, TOL_TC)


@pytest.mark.parametrize("prec", ["fp32", "tf32"])
def test_grad_transform_in_place(env, prec):
    torch, B = env
    rng = np.random.default_rng(5)
    for M, N in ((64, 32), (300, 70), (1024, 260)):
        Phi, _, _ = synth.spd_with_spectrum(M, 1e2, 900 + M, basis="householder")
        Phi32 = Phi.astype(np.float32); Phi32 = np.triu(Phi32) + np.triu(Phi32, 1).T
        L = B.Layer(M, N, beta=0.0, gamma=1.0, prec=B.FW_PREC_TF32 if prec == "tf32" else B.FW_PREC_FP32)
        L.set(B.FW_F_PHIX, torch.from_numpy(Phi32).cuda())
        L.cond_reduce(2, 4)
        G = rng.standard_normal((N, M)).astype(np.float32)
        Gd = torch.from_numpy(G).cuda()
        out = L.grad_transform(Gd)                   # separate output
        B.fw_grad_transform(L.handle, Gd, Gd)        # in place
        assert torch.equal(Gd, out)
        ref = G.astype(np.float64) @ t2n(L.get(B.FW_F_QS))
        assert rel_fro(t2n(Gd), ref) <= (TOL_TC if prec == "tf32" else TOL_FP32)


def test_bounded_wait_gives_up_and_the_layer_stays_usable(env):
    # A wait nothing satisfies runs into its poll limit: the kernel records it and returns, the host reads
    # FW_ERR_TIMEOUT for THIS layer only, the flag clears, and the next calls work.
    torch, B = env
    rng = np.random.default_rng(8)
    M = 64
    La = B.Layer(M, 4, alpha=0.5, beta=0.0, gamma=1.0, prec=B.FW_PREC_TF32)
    Lb = B.Layer(M, 4, alpha=0.5, beta=0.0, gamma=1.0, prec=B.FW_PREC_TF32)
    X = np.abs(rng.standard_normal((500, M))).astype(np.float32)
    Xd = torch.from_numpy(X).cuda()
    La.cov_update(Xd); Lb.cov_update(Xd)
    B.fw_debug_wait_probe(La.handle, 2048)
    assert Lb.sync_status() == B.FW_OK               # the other layer is not blamed
    with pytest.raises(B.FwError) as e:
        La.sync_status()
    assert e.value.status == B.FW_ERR_TIMEOUT
    assert La.sync_status() == B.FW_OK               # cleared by the read
    Lo = O.Layer(M, 4, oracle_hyper(La.desc))
    O.cov_update(Lo, X)
    La.cov_update(Xd); O.cov_update(Lo, X)
    La.cond_reduce(2, 4); O.cond_reduce(Lo, 2, 4)
    assert La.sync_status() == B.FW_OK
    check(La, Lo, B, TOL_TC)
    assert rel_fro(t2n(La.get(B.FW_F_Q)), Lo.Q) <= TOL_TC
    with pytest.raises(B.FwError) as e:
        B.fw_debug_wait_probe(La.handle, 0)
    assert e.value.status == B.FW_ERR_INVALID_ARG


@pytest.mark.parametrize("prec", ["fp32", "tf32"])
def test_nonfinite_values_are_reported_not_trapped(env, prec):
    torch, B = env
    rng = np.random.default_rng(9)
    M, N = 96, 8
    p = B.FW_PREC_TF32 if prec == "tf32" else B.FW_PREC_FP32
    # NaN in X -> moments
    L = B.Layer(M, N, alpha=0.5, beta=0.0, gamma=1.0, prec=p)
    X = np.abs(rng.standard_normal((5000, M))).astype(np.float32)
    X[1234, 17] = np.nan
    L.cov_update(torch.from_numpy(X).cuda())
    assert L.sync_status() == B.FW_WARN_NONFINITE
    assert L.sync_status() == B.FW_OK
    # Inf in G -> gradient transform
    L2 = B.Layer(M, N, beta=0.0, gamma=1.0, prec=p)
    G = rng.standard_normal((N, M)).astype(np.float32)
    G[3, 5] = np.inf
    L2.grad_transform(torch.from_numpy(G).cuda())
    assert L2.sync_status() == B.FW_WARN_NONFINITE
    # NaN in an injected covariance -> recursion scalars (on chip, and streamed for a larger layer)
    for Mr in (96, 700):
        L3 = B.Layer(Mr, N, beta=0.0, gamma=1.0, prec=p)
        Phi = np.eye(Mr, dtype=np.float32)
        Phi[2, 2] = np.nan
        L3.set(B.FW_F_PHIX, torch.from_numpy(Phi).cuda())
        L3.cond_reduce(1, 2)
        assert L3.sync_status() == B.FW_WARN_NONFINITE


def test_alignment_weights_survive_a_covariance_update(env):
    # FW_F_ALIGN_W is the last reduction's 1/c_m on the coherent set; the moment kernels keep their scratch elsewhere
    torch, B = env
    rng = np.random.default_rng(10)
    M = 80
    L = B.Layer(M, 4, alpha=0.5, beta=0.0, gamma=1.0)
    X = torch.from_numpy(np.abs(rng.standard_normal((400, M))).astype(np.float32)).cuda()
    L.cov_update(X)
    L.cond_reduce(1, 4)
    w = L.get(B.FW_F_ALIGN_W).clone()
    assert float(w.abs().sum()) > 0
    L.cov_update(X)
    assert torch.equal(L.get(B.FW_F_ALIGN_W), w)


def test_on_chip_query_matches_the_dispatch(env):
    torch, B = env
    assert B.fw_recursion_on_chip(B.fw_layer_desc_default(576, 64, gamma=1.0))
    assert not B.fw_recursion_on_chip(B.fw_layer_desc_default(576, 64, gamma=0.99))
    assert not B.fw_recursion_on_chip(B.fw_layer_desc_default(2304, 64, gamma=1.0))


def test_momentum_step_and_whiteness(env):
    torch, B = env
    rng = np.random.default_rng(12)
    M, N = 72, 9
    L = B.Layer(M, N, alpha=0.5, beta=0.0, gamma=1.0)
    Lo = O.Layer(M, N, oracle_hyper(L.desc))
    Phi, U, lam = synth.spd_with_spectrum(M, 1e2, 321)
    X = synth.gaussian_rows(600, U, lam, 322).astype(np.float32) + 0.3
    L.cov_update(torch.from_numpy(X).cuda()); O.cov_update(Lo, X)
    rho = torch.zeros(1, device="cuda")
    B.fw_whiteness(L.handle, rho)
    assert float(rho[0]) == pytest.approx(O.whiteness(Lo.phiy()), rel=1e-4)
    L.cond_reduce(4, 8); O.cond_reduce(Lo, 4, 8)
    B.fw_whiteness(L.handle, rho)
    assert float(rho[0]) == pytest.approx(O.whiteness(Lo.phiy()), rel=1e-4)
    W = rng.standard_normal((N, M)).astype(np.float32); b = rng.standard_normal(N).astype(np.float32)
    Wd, bd = torch.from_numpy(W).cuda(), torch.from_numpy(b).cuda()
    vW, vb = torch.zeros(N, M, device="cuda"), torch.zeros(N, device="cuda")
    Wo, bo, vWo, vbo = W.astype(np.float64), b.astype(np.float64), np.zeros((N, M)), np.zeros(N)
    for it in range(3):
        G = rng.standard_normal((N, M)).astype(np.float32); gb = rng.standard_normal(N).astype(np.float32)
        Gt = L.grad_transform(torch.from_numpy(G).cuda())
        B.fw_step_momentum(L.handle, Wd, bd, Gt, torch.from_numpy(gb).cuda(), vW, vb, 0.05, 0.9, 5e-4)
        Wo, bo, vWo, vbo = O.sgd_momentum_step(Wo, bo, O.grad_transform(Lo, G), gb.astype(np.float64), vWo, vbo,
                                                0.05, 0.9, 5e-4)
    assert rel_fro(t2n(Wd), Wo) <= TOL_FP32 and rel_fro(t2n(bd), bo) <= TOL_FP32
    assert rel_fro(t2n(vW), vWo) <= TOL_FP32
    with pytest.raises(B.FwError) as e:
        B.fw_step_momentum(L.handle, Wd, bd, Gt, None, vW, vb, 0.05, 0.9, 0.0)     # bias given without its gradient
    assert e.value.status == B.FW_ERR_INVALID_ARG
