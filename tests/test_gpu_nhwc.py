"""Moments straight from the NHWC activation (implicit im2col, Sec. 2: "any
spatial dimension can be vectorized"): fw_cov_update_nhwc against the fp64
oracle run on the materialised patch matrix (synth.im2col is the definition of
the patch rows: 3 x 3, stride 1, zero padding 1, columns ordered (ky, kx, c))."""
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


def check(L, Lo, B, tol=TOL_TC):
    assert rel_fro(t2n(L.get(B.FW_F_MU)), Lo.mu) <= tol
    e = rel_fro(t2n(L.get(B.FW_F_PHIX)), Lo.Phix)
    assert e <= tol, e
    assert rel_fro(t2n(L.get(B.FW_F_PHI_DIAG)), Lo.phi) <= tol
    assert abs(float(L.get(B.FW_F_LAMBDA_BAR)[0]) - Lo.lam_bar) <= tol * abs(Lo.lam_bar)
    Px = t2n(L.get(B.FW_F_PHIX))
    assert np.array_equal(Px, Px.T)
    return e


def scratch_for(torch, B, Bn, H, W, C):
    nb = B.fw_nhwc_scratch_bytes(Bn, H, W, C, 3)
    assert nb >= Bn * (H + 2) * (W + 2) * C * 4
    return torch.empty(nb, dtype=torch.uint8, device="cuda"), nb


# the three ResNet-20 stages (reduced batch), shapes whose width is not a power of two, a channel count whose
# three-pixel window does not fill whole 32-column chunks (C = 16, 48), a layer of the tiled Gram mode (C = 64, 96)
@pytest.mark.parametrize("Bn,HW,C", [(8, 32, 16), (8, 16, 32), (16, 8, 64), (6, 14, 32), (3, 28, 16), (5, 12, 48),
                                     (2, 64, 16), (4, 8, 96)])
def test_cov_update_nhwc_matches_oracle_on_patch_matrix(env, Bn, HW, C):
    torch, B = env
    M = 9 * C
    L = B.Layer(M, 4, alpha=0.8, beta=0.0, gamma=1.0, prec=B.FW_PREC_TF32)
    Lo = O.Layer(M, 4, oracle_hyper(L.desc))
    scratch, nb = scratch_for(torch, B, Bn, HW, HW, C)
    for batch in range(2):
        fm = synth.halfnormal_feature_map(Bn, HW, HW, C, 7000 + C + HW, batch_index=batch)
        X = synth.im2col(fm, 3, 1)
        B.fw_cov_update_nhwc(L.handle, torch.from_numpy(fm).cuda(), Bn, HW, HW, C, 3, scratch, nb)
        O.cov_update(Lo, X)
        e = check(L, Lo, B)
        assert e > 1e-8                      # the tensor cores ran (TF32 inputs)
    assert L.sync_status() == B.FW_OK


def test_nhwc_grouped_resnet20_stages_and_agreement_with_materialised_rows(env):
    torch, B = env
    shapes = [(8, 32, 16), (8, 16, 32), (8, 8, 64)]
    Ls, Lm, Los, fms, scr = [], [], [], [], []
    for (Bn, HW, C) in shapes:
        Ls.append(B.Layer(9 * C, 4, alpha=0.9, beta=0.0, gamma=1.0, prec=B.FW_PREC_TF32))
        Lm.append(B.Layer(9 * C, 4, alpha=0.9, beta=0.0, gamma=1.0, prec=B.FW_PREC_TF32))
        Los.append(O.Layer(9 * C, 4, oracle_hyper(Ls[-1].desc)))
        fms.append(synth.halfnormal_feature_map(Bn, HW, HW, C, 7100 + C))
        scr.append(scratch_for(torch, B, Bn, HW, HW, C))
    A = [torch.from_numpy(f).cuda() for f in fms]
    B.fw_group_cov_update_nhwc([L.handle for L in Ls], A, [s[0] for s in shapes], [s[1] for s in shapes],
                               [s[1] for s in shapes], [s[2] for s in shapes], [3, 3, 3],
                               [s[0] for s in scr], [s[1] for s in scr])
    for L, L2, Lo, f in zip(Ls, Lm, Los, fms):
        X = synth.im2col(f, 3, 1)
        O.cov_update(Lo, X)
        check(L, Lo, B)
        L2.cov_update(torch.from_numpy(X).cuda())            # the same moments from the materialised patch rows
        assert rel_fro(t2n(L.get(B.FW_F_PHIX)), t2n(L2.get(B.FW_F_PHIX))) <= 2e-3
        assert rel_fro(t2n(L.get(B.FW_F_MU)), t2n(L2.get(B.FW_F_MU))) <= 1e-3   # both sum TF32-truncated values


def test_nhwc_block_over_two_calls_and_kernel_size_one(env):
    torch, B = env
    Bn, HW, C = 4, 16, 32
    L = B.Layer(9 * C, 4, alpha=0.5, beta=0.0, gamma=1.0, prec=B.FW_PREC_TF32)
    Lo = O.Layer(9 * C, 4, oracle_hyper(L.desc))
    scratch, nb = scratch_for(torch, B, Bn, HW, HW, C)
    parts = []
    for c in range(2):
        fm = synth.halfnormal_feature_map(Bn, HW, HW, C, 7200, batch_index=c)
        parts.append(synth.im2col(fm, 3, 1))
        B.fw_cov_update_nhwc(L.handle, torch.from_numpy(fm).cuda(), Bn, HW, HW, C, 3, scratch, nb,
                             B.FW_COV_ACCUMULATE if c == 0 else B.FW_COV_COMMIT)
    O.cov_update(Lo, np.concatenate(parts, axis=0))
    check(L, Lo, B)
    # k = 1: the activation is the patch matrix
    L1 = B.Layer(C, 4, alpha=0.5, beta=0.0, gamma=1.0, prec=B.FW_PREC_TF32)
    Lo1 = O.Layer(C, 4, oracle_hyper(L1.desc))
    fm = synth.halfnormal_feature_map(Bn, HW, HW, C, 7300)
    B.fw_cov_update_nhwc(L1.handle, torch.from_numpy(fm).cuda(), Bn, HW, HW, C, 1)
    O.cov_update(Lo1, fm.reshape(-1, C))
    check(L1, Lo1, B)


def test_nhwc_argument_errors(env):
    torch, B = env
    C, HW, Bn = 16, 8, 2
    A = torch.zeros(Bn, HW, HW, C, device="cuda")
    scratch, nb = scratch_for(torch, B, Bn, HW, HW, C)
    L = B.Layer(9 * C, 4, prec=B.FW_PREC_TF32)
    with pytest.raises(B.FwError) as e:
        B.fw_cov_update_nhwc(L.handle, A, Bn, HW, HW, C, 3, scratch, nb - 256)       # scratch too small
    assert e.value.status == B.FW_ERR_WORKSPACE
    with pytest.raises(B.FwError) as e:
        B.fw_cov_update_nhwc(L.handle, A, Bn, HW, HW, 2 * C, 3, scratch, nb)         # C k k != M
    assert e.value.status == B.FW_ERR_SHAPE
    with pytest.raises(B.FwError) as e:
        B.fw_cov_update_nhwc(L.handle, A, Bn, HW, HW, C, 5, scratch, nb)
    assert e.value.status == B.FW_ERR_UNSUPPORTED
    Lf = B.Layer(9 * C, 4)                                                           # FP32 engine: no implicit path
    with pytest.raises(B.FwError) as e:
        B.fw_cov_update_nhwc(Lf.handle, A, Bn, HW, HW, C, 3, scratch, nb)
    assert e.value.status == B.FW_ERR_UNSUPPORTED
    A7 = torch.zeros(Bn, 7, 7, C, device="cuda")                                     # 7 rows: no stage shape divides them
    s7, n7 = scratch_for(torch, B, Bn, 7, 7, C)
    with pytest.raises(B.FwError) as e:
        B.fw_cov_update_nhwc(L.handle, A7, Bn, 7, 7, C, 3, s7, n7)
    assert e.value.status == B.FW_ERR_UNSUPPORTED
