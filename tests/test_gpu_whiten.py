"""The direct method's per-sample products (Sec. 2, Eqs. 11 and 14), which the
gradient transformation replaces and the cost comparison times: fw_whiten_forward
and fw_whiten_backward against the fp64 oracle."""
import numpy as np
import pytest

from oracle import fw_oracle as O
from paper_2010_01546_b200 import synth

from fwtest_util import TOL_FP32, TOL_TC, rel_fro, t2n

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2010_01546_b200 import binding as B, build
    build.build_library()
    return torch, B


@pytest.mark.parametrize("engine,M,rows", [("fp32", 96, 1000), ("fp32", 145, 77), ("tf32", 64, 130), ("tf32", 320, 5003),
                                           ("tf32", 1152, 3000), ("tf32", 100, 515)])
def test_whiten_forward_and_backward(env, engine, M, rows):
    torch, B = env
    rng = np.random.default_rng(M + rows)
    L = B.Layer(M, 4, beta=0.0, gamma=1.0, prec=B.FW_PREC_TF32 if engine == "tf32" else B.FW_PREC_FP32)
    tol = TOL_TC if engine == "tf32" else TOL_FP32
    T = (np.eye(M) + 0.5 * rng.standard_normal((M, M)) / np.sqrt(M)).astype(np.float32)
    mu = rng.standard_normal(M).astype(np.float32)
    L.set(B.FW_F_T, torch.from_numpy(T).cuda())
    L.set(B.FW_F_MU, torch.from_numpy(mu).cuda())
    Lo = O.Layer(M, 4)
    Lo.T = T.astype(np.float64); Lo.mu = mu.astype(np.float64)
    X = (rng.standard_normal((rows, M)) + 1.5).astype(np.float32)
    dY = rng.standard_normal((rows, M)).astype(np.float32)
    Y = torch.full((rows, M), float("nan"), device="cuda")
    dX = torch.full((rows, M), float("nan"), device="cuda")
    B.fw_whiten_forward(L.handle, torch.from_numpy(X).cuda(), rows, Y)
    B.fw_whiten_backward(L.handle, torch.from_numpy(dY).cuda(), rows, dX)
    # error of Y relative to the product before the mean is taken off: the subtraction T mu cancels part of X T^T
    Yref = O.whiten_forward(Lo, X)
    scale = np.linalg.norm(X.astype(np.float64) @ Lo.T.T)
    assert np.linalg.norm(t2n(Y) - Yref) <= tol * scale
    assert rel_fro(t2n(dX), O.whiten_backward(Lo, dY)) <= tol
    assert L.sync_status() == B.FW_OK


def test_whiten_argument_errors(env):
    torch, B = env
    L = B.Layer(32, 4)
    X = torch.zeros(10, 32, device="cuda")
    with pytest.raises(B.FwError) as e:
        B.fw_whiten_forward(L.handle, X, 10, X)
    assert e.value.status == B.FW_ERR_INVALID_ARG
    with pytest.raises(B.FwError) as e:
        B.fw_whiten_backward(L.handle, X, 0, torch.zeros(10, 32, device="cuda"))
    assert e.value.status == B.FW_ERR_SHAPE
