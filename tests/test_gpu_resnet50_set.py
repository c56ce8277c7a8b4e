"""Parity of the launch shapes the ImageNet-ResNet-50-shaped workload runs: bf16
inputs, BF16 engine, all fourteen layers (M = 64 ... 4608, N = 64 ... 2048) in
ONE grouped call per stage of the path, so that several problems share one
launch of the CTA-pair Gram kernel and one of the single-CTA Gram kernel, the
re-sync runs on both tensor-core kernels, the recursion on chip for the small
layers and streamed for the large ones, and G Qs as one grouped launch.  The
batch is reduced to 64 (the oracle has to finish in about a minute) but keeps
the same seven layers on the CTA-pair kernel as the full batch of 256 does.
Every output is compared with the fp64 oracle at the tensor-core tolerance."""
import numpy as np
import pytest

from oracle import fw_oracle as O
from paper_2010_01546_b200 import synth

from fwtest_util import (NEAR_TIE_TC, TOL_TC, group_reduce_with_replay, oracle_hyper, phiy_error_tc,
                         reduce_with_replay, rel_fro, t2n)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2010_01546_b200 import binding as B, build
    build.build_library()
    return torch, B


def bf16_dev(torch, X):
    return torch.from_numpy(synth.bf16_bits(X).view(np.int16)).cuda().view(torch.bfloat16)


def test_resnet50_shaped_set_grouped_bf16_two_batches(env):
    torch, B = env
    shapes = synth.resnet50_shapes(64)
    K, P, lr = 2, 16, 0.05
    layers, oras = [], []
    for s in shapes:
        rows, M, N = synth.shape_dims(s)
        L = B.Layer(M, N, alpha=0.9, beta=0.0, gamma=1.0, delta=0.25, x_dtype=B.FW_BF16, prec=B.FW_PREC_BF16)
        layers.append(L); oras.append(O.Layer(M, N, oracle_hyper(L.desc)))
    hs = [L.handle for L in layers]
    n_pair = sum(1 for s in shapes if synth.shape_dims(s)[0] * float(synth.shape_dims(s)[1]) ** 2 >= 1e10
                 and synth.shape_dims(s)[1] >= 289)
    assert n_pair == 7                                  # as at the full batch
    Ws = bs = Wo = bo = None
    for batch in range(2):
        ins = []
        for i, s in enumerate(shapes):
            d = synth.conv_layer_inputs(s["B"], s["HW"], s["C_in"], s["C_out"], s["k"], synth.layer_seed(3, i),
                                        decades=1.0, batch_index=batch)
            d["X"] = synth.to_bf16_grid(d["X"])
            ins.append(d)
        if batch == 0:
            Ws = [torch.from_numpy(d["W"]).cuda() for d in ins]; bs = [torch.from_numpy(d["b"]).cuda() for d in ins]
            Wo = [d["W"].astype(np.float64) for d in ins]; bo = [d["b"].astype(np.float64) for d in ins]
            for L, Lo, W, b, d in zip(layers, oras, Ws, bs, ins):
                L.attach_params(W, b); Lo.attach_params(d["W"], d["b"])
        Xd = [bf16_dev(torch, d["X"]) for d in ins]
        B.fw_group_cov_update(hs, Xd, [d["rows"] for d in ins], [d["M"] for d in ins])
        del Xd
        for i, (L, Lo, d) in enumerate(zip(layers, oras, ins)):
            O.cov_update(Lo, d["X"])
            assert rel_fro(t2n(L.get(B.FW_F_MU)), Lo.mu) <= TOL_TC, i
            e = rel_fro(t2n(L.get(B.FW_F_PHIX)), Lo.Phix)
            assert e <= TOL_TC, (i, e)
            assert rel_fro(t2n(L.get(B.FW_F_PHI_DIAG)), Lo.phi) <= TOL_TC, i
            assert rel_fro(t2n(bs[i]), Lo.b) <= TOL_TC, i                 # bias compensation (Eq. 31)
            bo[i] = Lo.b.copy()
        group_reduce_with_replay(layers, oras, K, P, B, torch, near_tie=NEAR_TIE_TC, on_device_state=True)
        for i, (L, Lo, d) in enumerate(zip(layers, oras, ins)):
            T, Q, Py = t2n(L.get(B.FW_F_T)), t2n(L.get(B.FW_F_Q)), t2n(L.get(B.FW_F_PHIY))
            assert rel_fro(T, Lo.T) <= TOL_TC, i
            assert rel_fro(Q, Lo.Q) <= TOL_TC, i
            # Phi_y = T Phi_x T^T inherits the engine's error of Phi_x (and, from the second batch on, that of the
            # TF32 re-sync products) on the forward-error scale of the product: see phiy_error_tc
            e = phiy_error_tc(Py, Lo)
            assert e <= TOL_TC, (i, e, rel_fro(Py, Lo.phiy()))
            assert np.array_equal(Py, Py.T) and np.array_equal(Q, Q.T)
        Gd = [torch.from_numpy(d["G"]).cuda() for d in ins]
        gbd = [torch.from_numpy(d["gb"]).cuda() for d in ins]
        B.fw_group_grad_transform_step(hs, Gd, Ws, bs, gbd, lr)
        for i, (Lo, d) in enumerate(zip(oras, ins)):
            Gt = O.grad_transform(Lo, d["G"])
            Wo[i], bo[i] = O.sgd_step(Wo[i], bo[i], Gt, d["gb"].astype(np.float64), lr)
            Lo.W, Lo.b = Wo[i].copy(), bo[i].copy()
            assert rel_fro(t2n(Ws[i]), Wo[i]) <= TOL_TC, i
            assert rel_fro(t2n(bs[i]), bo[i]) <= TOL_TC, i
    for L in layers:
        assert L.sync_status() == B.FW_OK


def test_bf16_layer_single_calls_transform_and_reduce(env):
    # a BF16-engine layer through the single-layer entry points: fw_cond_reduce (tensor-core re-sync on the second
    # batch) and fw_grad_transform (TF32 G Qs of a BF16-precision layer)
    torch, B = env
    rng = np.random.default_rng(12)
    M, N, rows = 640, 130, 3000
    L = B.Layer(M, N, alpha=0.8, beta=0.2, gamma=1.0, x_dtype=B.FW_BF16, prec=B.FW_PREC_BF16)
    Lo = O.Layer(M, N, oracle_hyper(L.desc))
    scale = rng.uniform(0.5, 2.0, M)
    mix = np.abs(rng.standard_normal((6, M))) * 0.4
    for batch in range(2):
        X = synth.to_bf16_grid((np.abs(rng.standard_normal((rows, M))) * scale
                                + np.abs(rng.standard_normal((rows, 6))) @ mix).astype(np.float32))
        L.cov_update(bf16_dev(torch, X)); O.cov_update(Lo, X)
        reduce_with_replay(L, Lo, 3, 8, B, torch, near_tie=NEAR_TIE_TC, on_device_state=True)
        assert rel_fro(t2n(L.get(B.FW_F_T)), Lo.T) <= TOL_TC
        assert rel_fro(t2n(L.get(B.FW_F_QS)), Lo.Qs) <= TOL_TC
        assert phiy_error_tc(t2n(L.get(B.FW_F_PHIY)), Lo) <= TOL_TC
        G = rng.standard_normal((N, M)).astype(np.float32)
        Gt = L.grad_transform(torch.from_numpy(G).cuda())
        assert rel_fro(t2n(Gt), O.grad_transform(Lo, G)) <= TOL_TC
    assert L.sync_status() == B.FW_OK


@pytest.mark.parametrize("M,rows", [(1024, 2500), (1152, 9000)])
def test_leaky_transform_with_tensorcore_resync(env, M, rows):
    # gamma < 1 with the TF32 engine at a size whose re-sync runs on the CTA-pair kernel: from the second batch
    # on, P = T Phi_x (the leaky update's extra state) and Phi_y come out of the tensor-core products
    torch, B = env
    rng = np.random.default_rng(M)
    L = B.Layer(M, 8, alpha=0.7, beta=0.1, gamma=0.99, delta=0.25, prec=B.FW_PREC_TF32)
    Lo = O.Layer(M, 8, oracle_hyper(L.desc))
    Phi, U, lam = synth.spd_with_spectrum(M, 1e3, 4000 + M, basis="householder")
    for batch in range(3):
        X = synth.gaussian_rows(rows, U, lam, 4100 + 10 * M + batch).astype(np.float32) + 0.1
        L.cov_update(torch.from_numpy(X).cuda()); O.cov_update(Lo, X)
        reduce_with_replay(L, Lo, 2, 8, B, torch, near_tie=NEAR_TIE_TC, on_device_state=True)
        T, Q = t2n(L.get(B.FW_F_T)), t2n(L.get(B.FW_F_Q))
        assert rel_fro(T, Lo.T) <= TOL_TC
        assert rel_fro(Q, Lo.Q) <= TOL_TC
        assert rel_fro(t2n(L.get(B.FW_F_QS)), Lo.Qs) <= TOL_TC
        e = phiy_error_tc(t2n(L.get(B.FW_F_PHIY)), Lo)
        assert e <= TOL_TC, e
        assert rel_fro(Q, T.T @ T) <= 1e-4                              # Eq. 44 tracks T^T T with leakage
    assert L.sync_status() == B.FW_OK
