"""GPU parity of the tensor-core engine (tcgen05 / TMEM / TMA kernels, TF32 or
BF16 inputs with fp32 accumulation) against the fp64 oracle.  Bar: relative
Frobenius error <= 5e-3."""
import numpy as np
import pytest

from oracle import fw_oracle as O
from paper_2010_01546_b200 import synth

from fwtest_util import NEAR_TIE_TC, TOL_TC, group_reduce_with_replay, oracle_hyper, phiy_error_tc, rel_fro, t2n

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2010_01546_b200 import binding as B, build
    build.build_library()
    return torch, B


def dev(torch, a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def spd32(M, cond, seed):
    Phi, _, _ = synth.spd_with_spectrum(M, cond, seed, basis="qr" if M <= 600 else "householder")
    P = Phi.astype(np.float32)
    return np.triu(P) + np.triu(P, 1).T


@pytest.mark.parametrize("M,N", [(64, 32), (144, 16), (288, 32), (576, 64), (64, 256), (1152, 300), (2048, 1000),
                                 (100, 7), (36, 20)])
def test_grad_transform_tf32(env, M, N):
    torch, B = env
    rng = np.random.default_rng(M * 7 + N)
    L = B.Layer(M, N, beta=0.0, gamma=1.0, prec=B.FW_PREC_TF32)
    Q = spd32(M, 50.0, 300 + M) + np.eye(M, dtype=np.float32)
    L.set(B.FW_F_Q, dev(torch, Q))
    G = rng.standard_normal((N, M)).astype(np.float32)
    W = rng.standard_normal((N, M)).astype(np.float32)
    ref = G.astype(np.float64) @ Q.astype(np.float64)
    out = L.grad_transform(dev(torch, G))
    e = rel_fro(t2n(out), ref)
    assert e <= TOL_TC, e
    assert e > 1e-7                       # TF32 inputs: not bit-for-bit the fp32 result (the tensor cores ran)
    Wd = dev(torch, W)
    B.fw_group_grad_transform_step([L.handle], [dev(torch, G)], [Wd], None, None, 0.05)
    assert rel_fro(t2n(Wd), W - 0.05 * ref) <= TOL_TC
    assert L.sync_status() == B.FW_OK


def test_grad_transform_tf32_grouped_mixed_shapes(env):
    torch, B = env
    rng = np.random.default_rng(99)
    shapes = [(144, 16), (288, 32), (576, 64), (144, 16), (64, 32)]
    Ls, Gs, Ws, refs = [], [], [], []
    for i, (M, N) in enumerate(shapes):
        L = B.Layer(M, N, beta=0.0, gamma=1.0, prec=B.FW_PREC_TF32)
        Q = spd32(M, 20.0, 700 + i) + np.eye(M, dtype=np.float32)
        L.set(B.FW_F_Q, dev(torch, Q))
        G = rng.standard_normal((N, M)).astype(np.float32); W = rng.standard_normal((N, M)).astype(np.float32)
        Ls.append(L); Gs.append(dev(torch, G)); Ws.append(dev(torch, W))
        refs.append(W - 0.1 * (G.astype(np.float64) @ Q.astype(np.float64)))
    B.fw_group_grad_transform_step([L.handle for L in Ls], Gs, Ws, None, None, 0.1)
    for W, r in zip(Ws, refs):
        assert rel_fro(t2n(W), r) <= TOL_TC


def check_moments_tc(L, Lo, B, tol=TOL_TC):
    assert rel_fro(t2n(L.get(B.FW_F_MU)), Lo.mu) <= tol
    e = rel_fro(t2n(L.get(B.FW_F_PHIX)), Lo.Phix)
    assert e <= tol, e
    assert rel_fro(t2n(L.get(B.FW_F_PHI_DIAG)), Lo.phi) <= tol
    assert abs(float(L.get(B.FW_F_LAMBDA_BAR)[0]) - Lo.lam_bar) <= tol * abs(Lo.lam_bar)
    return e


@pytest.mark.parametrize("M", [16, 64, 144, 160, 288, 320, 576, 1152])
@pytest.mark.parametrize("rows", [1, 33, 1000, 8197])
def test_cov_update_tf32(env, M, rows):
    torch, B = env
    if M >= 576 and rows == 8197:
        rows = 4101
    rng = np.random.default_rng(M * 13 + rows)
    L = B.Layer(M, 4, alpha=0.7, beta=0.0, gamma=1.0, prec=B.FW_PREC_TF32)
    Lo = O.Layer(M, 4, oracle_hyper(L.desc))
    ld = M + 4
    scale = rng.uniform(0.5, 2.0, ld)
    for blk in range(2):
        # half-normal (mean^2/var ~ 1.75), correlated through a random mixing of a few shared factors
        F = np.abs(rng.standard_normal((rows, 8)))
        X = (np.abs(rng.standard_normal((rows, ld))) * scale + F @ np.abs(rng.standard_normal((8, ld))) * 0.3
             + 0.2 * blk).astype(np.float32)
        Xd = dev(torch, X)
        B.fw_cov_update(L.handle, Xd, rows, ld)
        O.cov_update(Lo, X[:, :M])
        if rows == 1 and blk == 0:
            assert np.abs(t2n(L.get(B.FW_F_PHIX))).max() <= 1e-5 * (np.abs(X).max() ** 2)
        else:
            e = check_moments_tc(L, Lo, B)
            assert e > 1e-8 or rows < 8      # tensor cores (TF32 inputs), not the FFMA path
    assert L.sync_status() == B.FW_OK
    Px = t2n(L.get(B.FW_F_PHIX))
    assert np.array_equal(Px, Px.T)


@pytest.mark.parametrize("M", [64, 256, 288, 576, 1024])
@pytest.mark.parametrize("rows", [40, 1000, 5003])
def test_cov_update_bf16(env, M, rows):
    torch, B = env
    rng = np.random.default_rng(M * 17 + rows)
    L = B.Layer(M, 4, alpha=0.5, beta=0.0, gamma=1.0, x_dtype=B.FW_BF16, prec=B.FW_PREC_BF16)
    Lo = O.Layer(M, 4, oracle_hyper(L.desc))
    scale = rng.uniform(0.5, 2.0, M)
    for blk in range(2):
        F = np.abs(rng.standard_normal((rows, 8)))
        X = synth.to_bf16_grid((np.abs(rng.standard_normal((rows, M))) * scale
                                + F @ np.abs(rng.standard_normal((8, M))) * 0.3).astype(np.float32))
        Xd = torch.from_numpy(synth.bf16_bits(X).view(np.int16)).cuda().view(torch.bfloat16)
        L.cov_update(Xd)
        O.cov_update(Lo, X)
        check_moments_tc(L, Lo, B)
    assert L.sync_status() == B.FW_OK


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("M", [32, 128, 176, 192, 224, 240, 256])
def test_cov_update_long_blocks_column_sums(env, M, bf16):
    # long read-only blocks: up to M = 224 the column sums come out of the tensor core with the Gram (the widened
    # last MMA of each block row), above that from the fix-up warps; both sides of the switch, dense ld and padded
    torch, B = env
    rows = 4133
    rng = np.random.default_rng(M * 29 + int(bf16))
    for ld in (M, M + 8):
        if bf16:
            L = B.Layer(M, 4, alpha=0.6, beta=0.0, gamma=1.0, x_dtype=B.FW_BF16, prec=B.FW_PREC_BF16)
        else:
            L = B.Layer(M, 4, alpha=0.6, beta=0.0, gamma=1.0, prec=B.FW_PREC_TF32)
        Lo = O.Layer(M, 4, oracle_hyper(L.desc))
        scale = rng.uniform(0.5, 2.0, ld)
        for blk in range(2):
            X = (np.abs(rng.standard_normal((rows, ld))) * scale + 0.1 * blk).astype(np.float32)
            if bf16:
                X = synth.to_bf16_grid(X)
                Xd = torch.from_numpy(synth.bf16_bits(X).view(np.int16)).cuda().view(torch.bfloat16)
            else:
                Xd = dev(torch, X)
            B.fw_cov_update(L.handle, Xd, rows, ld)
            O.cov_update(Lo, X[:, :M])
            check_moments_tc(L, Lo, B)
        assert L.sync_status() == B.FW_OK


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("M,rows", [(32, 40007), (64, 33003), (128, 20011), (144, 16397), (208, 8200)])
def test_cov_update_large_stages_of_narrow_layers(env, M, rows, bf16):
    # narrow layers whose column sums come out of the tensor core take stages of 64 to 256 rows once the block is
    # long enough (64 stages at least): ragged last stage and last slab, dense and padded leading dimension
    torch, B = env
    rng = np.random.default_rng(M * 37 + int(bf16))
    for ld in (M, M + 8):
        if bf16:
            L = B.Layer(M, 4, alpha=0.6, beta=0.0, gamma=1.0, x_dtype=B.FW_BF16, prec=B.FW_PREC_BF16)
        else:
            L = B.Layer(M, 4, alpha=0.6, beta=0.0, gamma=1.0, prec=B.FW_PREC_TF32)
        Lo = O.Layer(M, 4, oracle_hyper(L.desc))
        scale = rng.uniform(0.5, 2.0, ld)
        for blk in range(2):
            X = (np.abs(rng.standard_normal((rows, ld))) * scale + 0.1 * blk).astype(np.float32)
            if bf16:
                X = synth.to_bf16_grid(X)
                Xd = torch.from_numpy(synth.bf16_bits(X).view(np.int16)).cuda().view(torch.bfloat16)
            else:
                Xd = dev(torch, X)
            B.fw_cov_update(L.handle, Xd, rows, ld)
            O.cov_update(Lo, X[:, :M])
            check_moments_tc(L, Lo, B)
        assert L.sync_status() == B.FW_OK


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("M,rows", [(576, 30157), (520, 36001), (1152, 7541), (328, 93011)])
def test_cov_update_large_products_cta_pairs(env, M, rows, bf16):
    # products of 1e10 multiply-adds and more run on CTA pairs (256 x 512 tiles): column counts that are and are
    # not multiples of 64 (one TMA instruction per column group / one per chunk), ragged last block rows, narrow
    # last panels, a ragged last row slab, dense and padded leading dimension; two blocks (running average)
    torch, B = env
    rng = np.random.default_rng(M * 31 + int(bf16))
    ld = M + (8 if M == 520 else 0)
    if bf16:
        L = B.Layer(M, 4, alpha=0.6, beta=0.0, gamma=1.0, x_dtype=B.FW_BF16, prec=B.FW_PREC_BF16)
    else:
        L = B.Layer(M, 4, alpha=0.6, beta=0.0, gamma=1.0, prec=B.FW_PREC_TF32)
    Lo = O.Layer(M, 4, oracle_hyper(L.desc))
    scale = rng.uniform(0.5, 2.0, ld)
    mix = np.abs(rng.standard_normal((8, ld))) * 0.3
    for blk in range(2):
        F = np.abs(rng.standard_normal((rows, 8)))
        X = (np.abs(rng.standard_normal((rows, ld))) * scale + F @ mix + 0.1 * blk).astype(np.float32)
        if bf16:
            X = synth.to_bf16_grid(X)
            Xd = torch.from_numpy(synth.bf16_bits(X).view(np.int16)).cuda().view(torch.bfloat16)
        else:
            Xd = dev(torch, X)
        B.fw_cov_update(L.handle, Xd, rows, ld)
        O.cov_update(Lo, X[:, :M])
        e = check_moments_tc(L, Lo, B)
        assert e > 1e-8
    assert L.sync_status() == B.FW_OK
    Px = t2n(L.get(B.FW_F_PHIX))
    assert np.array_equal(Px, Px.T)


@pytest.mark.parametrize("M", [64, 144, 288, 576, 1040, 1152])
def test_resync_products_tf32(env, M):
    # Phi_y = T Phi_x T^T through the tensor-core A^T B kernel (T injected, so T != I)
    torch, B = env
    rng = np.random.default_rng(M)
    L = B.Layer(M, 4, beta=0.0, gamma=1.0, prec=B.FW_PREC_TF32)
    T = (np.eye(M) + 0.3 * rng.standard_normal((M, M)) / np.sqrt(M)).astype(np.float32)
    Phi = spd32(M, 1e2, 40 + M)
    L.set(B.FW_F_T, dev(torch, T))
    L.set(B.FW_F_PHIX, dev(torch, Phi))
    Py = t2n(L.get(B.FW_F_PHIY))
    T64 = T.astype(np.float64)
    ref = T64 @ Phi.astype(np.float64) @ T64.T
    e = rel_fro(Py, ref)
    assert e <= TOL_TC, e
    assert e > 1e-7
    assert np.array_equal(Py, Py.T)
    assert L.sync_status() == B.FW_OK


def test_whole_path_tensorcore_engine_three_batches(env):
    # ResNet-20-shaped layers (reduced batch), TF32 engine for Gram, re-sync and G Qs; fp32 recursion.  Twin sets
    # as in the FP32-engine test: A takes K steps per grouped call, B one step per call with its decisions
    # replayed into the oracle where they flipped on a near-tie of the engine's tolerance; A must equal B.
    torch, B = env
    shapes = synth.resnet20_shapes(B=8)
    shapes = [shapes[0], shapes[5], dict(shapes[10], B=16)]
    setA, setB, oras = [], [], []
    for s in shapes:
        rows, M, N = synth.shape_dims(s)
        for st in (setA, setB):
            st.append(B.Layer(M, N, alpha=0.9, beta=0.0, gamma=1.0, delta=0.25, prec=B.FW_PREC_TF32))
        oras.append(O.Layer(M, N, oracle_hyper(setA[-1].desc)))
    K, P, lr = 4, 16, 0.1
    hA, hB = [L.handle for L in setA], [L.handle for L in setB]
    for batch in range(3):
        ins = [synth.conv_layer_inputs(s["B"], s["HW"], s["C_in"], s["C_out"], s["k"], synth.layer_seed(2, i),
                                       batch_index=batch) for i, s in enumerate(shapes)]
        if batch == 0:
            Ws = [dev(torch, d["W"]) for d in ins]; bs = [dev(torch, d["b"]) for d in ins]
            Wo = [d["W"].astype(np.float64) for d in ins]; bo = [d["b"].astype(np.float64) for d in ins]
        Xd = [dev(torch, d["X"]) for d in ins]
        for hs in (hA, hB):
            B.fw_group_cov_update(hs, Xd, [d["rows"] for d in ins], [d["M"] for d in ins])
        for Lo, d in zip(oras, ins):
            O.cov_update(Lo, d["X"])
        for L, Lo in zip(setA, oras):
            check_moments_tc(L, Lo, B)
        B.fw_group_cond_reduce(hA, K, P, None)
        group_reduce_with_replay(setB, oras, K, P, B, torch, near_tie=NEAR_TIE_TC, on_device_state=True)
        for LA, LB, Lo in zip(setA, setB, oras):
            assert rel_fro(t2n(LB.get(B.FW_F_T)), Lo.T) <= TOL_TC
            assert rel_fro(t2n(LB.get(B.FW_F_Q)), Lo.Q) <= TOL_TC
            assert phiy_error_tc(t2n(LB.get(B.FW_F_PHIY)), Lo) <= TOL_TC
            for f in (B.FW_F_T, B.FW_F_Q, B.FW_F_PHIY):
                assert torch.equal(LA.get(f), LB.get(f))
        B.fw_group_grad_transform_step(hA, [dev(torch, d["G"]) for d in ins], Ws, bs,
                                       [dev(torch, d["gb"]) for d in ins], lr)
        for j, (Lo, d) in enumerate(zip(oras, ins)):
            Gt = O.grad_transform(Lo, d["G"])
            Wo[j], bo[j] = O.sgd_step(Wo[j], bo[j], Gt, d["gb"].astype(np.float64), lr)
            assert rel_fro(t2n(Ws[j]), Wo[j]) <= TOL_TC
            assert rel_fro(t2n(bs[j]), bo[j]) <= TOL_TC
    for L in setA + setB:
        assert L.sync_status() == B.FW_OK
