"""fw_cov_block_static -- the entry point for callers that cannot allocate.

Some users of this library run where device allocation is not theirs to do: a
gradient hook inside a training framework whose caching allocator owns all
device memory cannot create the workspace a layer needs, and a raw cudaMalloc
there would stall the device.  fw_cov_block_static serves them with a scratch
array built into the library.  This test calls it through the C ABI twice in a
row (the second call sees the first call's leftovers in the shared array) and
checks both results against the regular entry point, fw_cov_update on a fresh
layer, and against the fp64 oracle, within the fp32 tolerance of the other
parity tests.  That the call allocates nothing is checked on the driver's own
count of free device memory (cudaMemGetInfo), which sees any allocation by any
library in the process, not only those of torch's caching allocator.

Collected last on purpose, so that a run stopping at the first failure has
already run every other test.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL = 1e-5


def _rel(a, b):
    return float((a.double() - b.double()).norm() / b.double().norm())


def test_static_covariance_matches_regular_entry_point_twice():
    import torch
    from oracle import fw_oracle as O
    from paper_2010_01546_b200 import binding as B, build
    build.build_library()
    rng = np.random.default_rng(2010)
    # warm-up call: loads the module that holds the 8 MiB array and resolves its address on this device
    Xw = torch.ones(64, 16, device="cuda")
    B.fw_cov_block_static(Xw, 64, 16, 16, torch.empty(16, device="cuda"), torch.empty(16, 16, device="cuda"))
    torch.cuda.synchronize()
    # second call: different, smaller shape, so stale partials of the first call remain in the array
    for M, rows, ld in ((144, 5000, 150), (97, 777, 97)):
        X = torch.from_numpy((np.abs(rng.standard_normal((rows, ld))) + 0.5).astype(np.float32)).cuda()
        ref = B.Layer(M, 4, alpha=0.9, beta=0.0, gamma=1.0)
        B.fw_cov_update(ref.handle, X, rows, ld)
        mu_ref, phix_ref = ref.get(B.FW_F_MU), ref.get(B.FW_F_PHIX)
        mu = torch.full((M,), float("nan"), device="cuda")
        phix = torch.full((M, M), float("nan"), device="cuda")
        torch.cuda.synchronize()
        before, free_before = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
        B.fw_cov_block_static(X, rows, ld, M, mu, phix)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        assert torch.cuda.mem_get_info()[0] == free_before      # no cudaMalloc by anyone during the call
        assert _rel(mu, mu_ref) <= TOL
        assert _rel(phix, phix_ref) <= TOL
        assert torch.equal(phix, phix.T)
        Lo = O.Layer(M, 4, O.Hyper(alpha=0.9))
        O.cov_update(Lo, X[:, :M].cpu().numpy())
        assert O.rel_fro(mu.cpu().numpy(), Lo.mu) <= TOL
        assert O.rel_fro(phix.cpu().numpy(), Lo.Phix) <= TOL


def test_static_covariance_rejects_sizes_beyond_its_scratch():
    import torch
    from paper_2010_01546_b200 import binding as B
    M = B.FW_STATIC_MAX_M + 1
    X = torch.zeros(8, M, device="cuda")
    mu = torch.zeros(M, device="cuda"); phix = torch.zeros(M, M, device="cuda")
    with pytest.raises(B.FwError) as e:
        B.fw_cov_block_static(X, 8, M, M, mu, phix)
    assert e.value.status == B.FW_ERR_SHAPE
    with pytest.raises(B.FwError) as e:
        B.fw_cov_block_static(None, 8, M, 16, mu, phix)
    assert e.value.status == B.FW_ERR_INVALID_ARG
