"""GPU parity of the tensor-core engine (tcgen05 / TMEM / TMA kernels, TF32 or
BF16 inputs with fp32 accumulation) against the fp64 oracle.  Bar: relative
Frobenius error <= 5e-3."""
import numpy as np
import pytest

from oracle import fw_oracle as O
from paper_2010_01546_b200 import synth

from fwtest_util import TOL_TC, oracle_hyper, rel_fro, t2n

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
