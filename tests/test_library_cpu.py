"""CPU-side checks of the C-ABI library: it loads, exports every symbol that
include/fw.h declares, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2010_01546_b200 import binding as B
from paper_2010_01546_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return ctypes.CDLL(B.LIB_PATH)


def declared_symbols():
    src = open(os.path.join(ROOT, "include", "fw.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(fw_[a-z_0-9]+)\s*\(", src)))


def test_header_symbols_are_exported(lib):
    names = declared_symbols()
    assert "fw_cov_update" in names and "fw_cond_reduce" in names and "fw_grad_transform" in names
    assert "fw_step" in names and "fw_layer_create" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in fw.h but not exported"
    assert set(B.EXPORTS) <= set(names)


def test_workspace_size_and_descriptor_validation():
    d = B.fw_layer_desc_default(64, 32)
    assert (d.alpha, d.beta) == pytest.approx((0.1, 0.1)) and d.gamma == pytest.approx(0.99)
    assert d.delta == pytest.approx(0.25) and d.c_rel == pytest.approx(0.025) and d.c_abs == pytest.approx(1e-6)
    n = B.fw_layer_workspace_bytes(d)
    assert n > 6 * 64 * 64 * 4 and n % 256 == 0
    for bad in (dict(M=0), dict(M=9000), dict(N=0), dict(alpha=1.0), dict(gamma=0.0), dict(gamma=1.5),
                dict(prec=7), dict(x_dtype=3), dict(init=2), dict(delta=0.0), dict(eps=0.0)):
        db = B.fw_layer_desc_default(64, 32)
        for k, v in bad.items():
            setattr(db, k, v)
        assert B.fw_layer_workspace_bytes(db) == 0, bad
    # beta > 0 keeps a separate smoothed Q
    n0 = B.fw_layer_workspace_bytes(B.fw_layer_desc_default(64, 32, beta=0.0))
    assert n - n0 == 64 * 64 * 4


def test_argument_errors_are_returned_before_any_launch():
    d = B.fw_layer_desc_default(64, 32)
    with pytest.raises(B.FwError) as e:
        B.fw_layer_create(d, None, 1 << 30)
    assert e.value.status == B.FW_ERR_INVALID_ARG
    with pytest.raises(B.FwError) as e:
        B.fw_layer_create(d, 4096 + 8, 1 << 30)          # misaligned workspace
    assert e.value.status == B.FW_ERR_WORKSPACE
    with pytest.raises(B.FwError) as e:
        B.fw_layer_create(d, 4096, 1024)                  # too small
    assert e.value.status == B.FW_ERR_WORKSPACE
    with pytest.raises(B.FwError) as e:
        B.fw_layer_create(B.fw_layer_desc_default(64, 32, prec=B.FW_PREC_BF16), 4096, 1 << 30)  # bf16 engine needs bf16 X
    assert e.value.status == B.FW_ERR_INVALID_ARG
    for fn, args in ((B.fw_cov_update, (None, 1, 1, 1)), (B.fw_cond_reduce, (None, 1, 1)),
                     (B.fw_grad_transform, (None, 1, 2)), (B.fw_step, (None, 1, 1, 1, 1, 0.1))):
        with pytest.raises(B.FwError) as e:
            fn(*args)
        assert e.value.status == B.FW_ERR_INVALID_ARG
    assert "workspace" in B.fw_status_string(B.FW_ERR_WORKSPACE)


def test_no_device_is_an_error_not_a_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    d = B.fw_layer_desc_default(8, 4)
    with pytest.raises(B.FwError) as e:
        B.fw_layer_create(d, 4096, 1 << 30)
    assert e.value.status == B.FW_ERR_CUDA


def test_product_sources_do_not_reference_the_oracle():
    pkg = os.path.join(ROOT, "paper_2010_01546_b200")
    for dp, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cuh", ".cpp")):
                txt = open(os.path.join(dp, f)).read()
                assert "fw_oracle" not in txt and "import oracle" not in txt and "from oracle" not in txt, f
    otxt = open(os.path.join(ROOT, "oracle", "fw_oracle.py")).read()
    assert "binding" not in otxt and "libfw" not in otxt and "ctypes" not in otxt


def test_library_sources_allocate_no_device_memory():
    # the library works in caller-supplied workspaces (and one static array): no allocation call anywhere in csrc/
    csrc = os.path.join(ROOT, "paper_2010_01546_b200", "csrc")
    for f in os.listdir(csrc):
        txt = open(os.path.join(csrc, f)).read()
        code = re.sub(r"//[^\n]*", "", txt)
        for name in ("cudaMalloc", "cudaFree(", "cudaMallocAsync", "cudaMallocManaged", "cuMemAlloc"):
            assert name not in code, (f, name)
