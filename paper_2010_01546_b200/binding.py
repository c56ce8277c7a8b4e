"""ctypes binding of the C-ABI library declared in include/fw.h.

Argument marshalling only: every function here has the name and the meaning of
the C entry point it wraps, takes torch CUDA tensors (or raw device addresses)
where the C function takes device pointers, and raises FwError on a non-zero
status.  There is no computation and no fallback in this file: if libfw.so is
missing or cannot be loaded the first call raises.
"""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libfw.so")

FW_OK = 0
FW_ERR_INVALID_ARG, FW_ERR_SHAPE, FW_ERR_STATE, FW_ERR_WORKSPACE = 1, 2, 3, 4
FW_ERR_CUDA, FW_ERR_TIMEOUT, FW_ERR_UNSUPPORTED = 5, 6, 7
FW_WARN_NO_SUBSPACE, FW_WARN_NONFINITE = 64, 65
FW_F32, FW_BF16 = 0, 1
FW_PREC_FP32, FW_PREC_TF32, FW_PREC_BF16 = 0, 1, 2
FW_INIT_ALIGN, FW_INIT_MAXCOL = 0, 1
FW_F_MU, FW_F_PHIX, FW_F_PHI_DIAG, FW_F_LAMBDA_BAR, FW_F_T, FW_F_Q, FW_F_QS, FW_F_PHIY, FW_F_ALIGN_W = range(9)
FW_MAX_GROUP = 64
FW_COV_COMMIT, FW_COV_ACCUMULATE = 0, 1

EXPORTS = [
    "fw_layer_desc_default", "fw_layer_workspace_bytes", "fw_layer_create", "fw_layer_destroy",
    "fw_layer_attach_params", "fw_cov_update", "fw_cond_reduce", "fw_grad_transform", "fw_step",
    "fw_group_cov_update", "fw_group_cond_reduce", "fw_group_grad_transform_step",
    "fw_layer_get", "fw_layer_set", "fw_layer_sync_status", "fw_status_string", "fw_version",
    "fw_profile_begin", "fw_profile_end", "fw_launch_count", "fw_cov_block_static",
    "fw_debug_wait_probe", "fw_recursion_on_chip", "fw_layer_reset",
    "fw_nhwc_scratch_bytes", "fw_cov_update_nhwc", "fw_group_cov_update_nhwc",
    "fw_whiten_forward", "fw_whiten_backward", "fw_step_momentum", "fw_whiteness",
    "fw_evd_scratch_bytes", "fw_evd_whiten", "fw_group_evd_whiten", "fw_spectrum",
]
FW_STATIC_MAX_M = 256
FW_PROF_NAMES = ["pilot", "gram", "moments", "resync", "recur_mv", "recur_upd", "smooth", "gq", "misc", "recur_chip"]


class FwError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib().fw_status_string(status).decode() if _LIB is not None else "?"
        super().__init__(f"{where}: fw_status {status} ({msg})")


class fw_layer_desc(C.Structure):
    _fields_ = [("M", C.c_int32), ("N", C.c_int32), ("x_dtype", C.c_int32), ("prec", C.c_int32),
                ("init", C.c_int32), ("alpha", C.c_float), ("beta", C.c_float), ("gamma", C.c_float),
                ("delta", C.c_float), ("eps", C.c_float), ("c_rel", C.c_float), ("c_abs", C.c_float)]


_LIB = None


def _lib():
    global _LIB
    if _LIB is not None:
        return _LIB
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} not found: build it with "
                          "`python -m paper_2010_01546_b200.build` (there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, f32, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_size_t
    P = C.POINTER
    lib.fw_layer_desc_default.argtypes = [P(fw_layer_desc), i32, i32]; lib.fw_layer_desc_default.restype = None
    lib.fw_layer_workspace_bytes.argtypes = [P(fw_layer_desc)]; lib.fw_layer_workspace_bytes.restype = sz
    lib.fw_layer_create.argtypes = [P(fw_layer_desc), vp, sz, vp, P(vp)]; lib.fw_layer_create.restype = i32
    lib.fw_layer_destroy.argtypes = [vp]; lib.fw_layer_destroy.restype = i32
    lib.fw_layer_reset.argtypes = [vp]; lib.fw_layer_reset.restype = i32
    lib.fw_layer_attach_params.argtypes = [vp, vp, vp]; lib.fw_layer_attach_params.restype = i32
    lib.fw_cov_update.argtypes = [vp, vp, i64, i64, C.c_uint32]; lib.fw_cov_update.restype = i32
    lib.fw_nhwc_scratch_bytes.argtypes = [i32, i32, i32, i32, i32]; lib.fw_nhwc_scratch_bytes.restype = sz
    lib.fw_cov_update_nhwc.argtypes = [vp, vp, i32, i32, i32, i32, i32, vp, sz, C.c_uint32]
    lib.fw_cov_update_nhwc.restype = i32
    lib.fw_group_cov_update_nhwc.argtypes = [P(vp), i32, P(vp), P(i32), P(i32), P(i32), P(i32), P(i32), P(vp), P(sz),
                                             C.c_uint32]
    lib.fw_group_cov_update_nhwc.restype = i32
    lib.fw_cond_reduce.argtypes = [vp, i32, i32, vp]; lib.fw_cond_reduce.restype = i32
    lib.fw_grad_transform.argtypes = [vp, vp, vp]; lib.fw_grad_transform.restype = i32
    lib.fw_step.argtypes = [vp, vp, vp, vp, vp, f32]; lib.fw_step.restype = i32
    lib.fw_step_momentum.argtypes = [vp, vp, vp, vp, vp, vp, vp, f32, f32, f32]; lib.fw_step_momentum.restype = i32
    lib.fw_whiteness.argtypes = [vp, vp]; lib.fw_whiteness.restype = i32
    lib.fw_evd_scratch_bytes.argtypes = [i32]; lib.fw_evd_scratch_bytes.restype = sz
    lib.fw_evd_whiten.argtypes = [vp, vp, sz, f32]; lib.fw_evd_whiten.restype = i32
    lib.fw_group_evd_whiten.argtypes = [P(vp), i32, P(vp), P(sz), f32]; lib.fw_group_evd_whiten.restype = i32
    lib.fw_spectrum.argtypes = [vp, i32, vp, sz, vp, vp]; lib.fw_spectrum.restype = i32
    lib.fw_whiten_forward.argtypes = [vp, vp, i64, vp]; lib.fw_whiten_forward.restype = i32
    lib.fw_whiten_backward.argtypes = [vp, vp, i64, vp]; lib.fw_whiten_backward.restype = i32
    lib.fw_group_cov_update.argtypes = [P(vp), i32, P(vp), P(i64), P(i64), C.c_uint32]
    lib.fw_group_cov_update.restype = i32
    lib.fw_group_cond_reduce.argtypes = [P(vp), i32, i32, i32, P(vp)]; lib.fw_group_cond_reduce.restype = i32
    lib.fw_group_grad_transform_step.argtypes = [P(vp), i32, P(vp), P(vp), P(vp), P(vp), f32]
    lib.fw_group_grad_transform_step.restype = i32
    lib.fw_layer_get.argtypes = [vp, i32, vp, sz]; lib.fw_layer_get.restype = i32
    lib.fw_layer_set.argtypes = [vp, i32, vp, sz]; lib.fw_layer_set.restype = i32
    lib.fw_layer_sync_status.argtypes = [vp]; lib.fw_layer_sync_status.restype = i32
    lib.fw_status_string.argtypes = [i32]; lib.fw_status_string.restype = C.c_char_p
    lib.fw_version.argtypes = []; lib.fw_version.restype = i32
    lib.fw_profile_begin.argtypes = []; lib.fw_profile_begin.restype = i32
    lib.fw_profile_end.argtypes = [P(f32), P(i64)]; lib.fw_profile_end.restype = i32
    lib.fw_launch_count.argtypes = []; lib.fw_launch_count.restype = i64
    lib.fw_cov_block_static.argtypes = [vp, i64, i64, i32, vp, vp, vp]; lib.fw_cov_block_static.restype = i32
    lib.fw_debug_wait_probe.argtypes = [vp, C.c_uint32]; lib.fw_debug_wait_probe.restype = i32
    lib.fw_recursion_on_chip.argtypes = [P(fw_layer_desc)]; lib.fw_recursion_on_chip.restype = i32
    _LIB = lib
    return lib


def _ptr(t):
    """Device address of a torch tensor (or pass an int / None through)."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _check(status: int, where: str, allow=()):
    if status != FW_OK and status not in allow:
        raise FwError(status, where)
    return status


def _vp_array(items):
    arr = (C.c_void_p * len(items))()
    for i, it in enumerate(items):
        arr[i] = _ptr(it)
    return arr


# ---- one function per C entry point ---------------------------------------
def fw_version() -> int:
    return _lib().fw_version()


def fw_status_string(status: int) -> str:
    return _lib().fw_status_string(status).decode()


def fw_layer_desc_default(M: int, N: int, **overrides) -> fw_layer_desc:
    d = fw_layer_desc()
    _lib().fw_layer_desc_default(C.byref(d), M, N)
    for k, v in overrides.items():
        setattr(d, k, v)
    return d


def fw_layer_workspace_bytes(desc: fw_layer_desc) -> int:
    return _lib().fw_layer_workspace_bytes(C.byref(desc))


def fw_layer_create(desc: fw_layer_desc, workspace, nbytes: int, stream: int = 0) -> int:
    out = C.c_void_p()
    _check(_lib().fw_layer_create(C.byref(desc), _ptr(workspace), nbytes, stream, C.byref(out)), "fw_layer_create")
    return out.value


def fw_layer_destroy(handle: int) -> None:
    _check(_lib().fw_layer_destroy(handle), "fw_layer_destroy")


def fw_layer_reset(handle) -> None:
    _check(_lib().fw_layer_reset(handle), "fw_layer_reset")


def fw_layer_attach_params(handle, W, b) -> None:
    _check(_lib().fw_layer_attach_params(handle, _ptr(W), _ptr(b)), "fw_layer_attach_params")


def fw_cov_update(handle, X, rows: int, ldx: int, flags: int = FW_COV_COMMIT) -> None:
    _check(_lib().fw_cov_update(handle, _ptr(X), rows, ldx, flags), "fw_cov_update")


def fw_nhwc_scratch_bytes(B: int, H: int, W: int, Cc: int, k: int) -> int:
    return int(_lib().fw_nhwc_scratch_bytes(B, H, W, Cc, k))


def fw_cov_update_nhwc(handle, A, B: int, H: int, W: int, Cc: int, k: int, scratch=None, scratch_bytes: int = 0,
                       flags: int = FW_COV_COMMIT) -> None:
    _check(_lib().fw_cov_update_nhwc(handle, _ptr(A), B, H, W, Cc, k, _ptr(scratch), scratch_bytes, flags),
           "fw_cov_update_nhwc")


def fw_group_cov_update_nhwc(handles, A, B, H, W, Cc, k, scratch, scratch_bytes, flags: int = FW_COV_COMMIT) -> None:
    n = len(handles)
    i32a = lambda v: (C.c_int32 * n)(*v)
    _check(_lib().fw_group_cov_update_nhwc(_vp_array(handles), n, _vp_array(A), i32a(B), i32a(H), i32a(W), i32a(Cc),
                                           i32a(k), _vp_array(scratch), (C.c_size_t * n)(*scratch_bytes), flags),
           "fw_group_cov_update_nhwc")


def fw_cond_reduce(handle, K: int, P: int, trace=None) -> None:
    _check(_lib().fw_cond_reduce(handle, K, P, _ptr(trace)), "fw_cond_reduce")


def fw_grad_transform(handle, G, G_out) -> None:
    _check(_lib().fw_grad_transform(handle, _ptr(G), _ptr(G_out)), "fw_grad_transform")


def fw_step_momentum(handle, W, b, G_t, g_b, vW, vb, lr: float, momentum: float, weight_decay: float) -> None:
    _check(_lib().fw_step_momentum(handle, _ptr(W), _ptr(b), _ptr(G_t), _ptr(g_b), _ptr(vW), _ptr(vb), lr, momentum,
                                   weight_decay), "fw_step_momentum")


def fw_whiteness(handle, rho_out) -> None:
    _check(_lib().fw_whiteness(handle, _ptr(rho_out)), "fw_whiteness")


def fw_evd_scratch_bytes(M: int) -> int:
    return int(_lib().fw_evd_scratch_bytes(M))


def fw_evd_whiten(handle, scratch, scratch_bytes: int, g_max: float = 0.0) -> None:
    _check(_lib().fw_evd_whiten(handle, _ptr(scratch), scratch_bytes, g_max), "fw_evd_whiten")


def fw_group_evd_whiten(handles, scratch, scratch_bytes, g_max: float = 0.0) -> None:
    n = len(handles)
    _check(_lib().fw_group_evd_whiten(_vp_array(handles), n, _vp_array(scratch),
                                      (C.c_size_t * n)(*scratch_bytes), g_max), "fw_group_evd_whiten")


def fw_spectrum(handle, which: int, scratch, scratch_bytes: int, lam_out=None, kappa_out=None) -> None:
    _check(_lib().fw_spectrum(handle, which, _ptr(scratch), scratch_bytes,
                              _ptr(lam_out) if lam_out is not None else None,
                              _ptr(kappa_out) if kappa_out is not None else None), "fw_spectrum")


def fw_whiten_forward(handle, X, rows: int, Y) -> None:
    _check(_lib().fw_whiten_forward(handle, _ptr(X), rows, _ptr(Y)), "fw_whiten_forward")


def fw_whiten_backward(handle, dY, rows: int, dX) -> None:
    _check(_lib().fw_whiten_backward(handle, _ptr(dY), rows, _ptr(dX)), "fw_whiten_backward")


def fw_step(handle, W, b, G_t, g_b, lr: float) -> None:
    _check(_lib().fw_step(handle, _ptr(W), _ptr(b), _ptr(G_t), _ptr(g_b), lr), "fw_step")


def fw_group_cov_update(handles, X, rows, ldx, flags: int = FW_COV_COMMIT) -> None:
    n = len(handles)
    _check(_lib().fw_group_cov_update(_vp_array(handles), n, _vp_array(X), (C.c_int64 * n)(*rows),
                                      (C.c_int64 * n)(*ldx), flags), "fw_group_cov_update")


def fw_group_cond_reduce(handles, K: int, P: int, traces=None) -> None:
    n = len(handles)
    tr = _vp_array(traces) if traces is not None else None
    _check(_lib().fw_group_cond_reduce(_vp_array(handles), n, K, P, tr), "fw_group_cond_reduce")


def fw_group_grad_transform_step(handles, G, W, b, g_b, lr: float) -> None:
    n = len(handles)
    _check(_lib().fw_group_grad_transform_step(_vp_array(handles), n, _vp_array(G), _vp_array(W),
                                               _vp_array(b) if b is not None else None,
                                               _vp_array(g_b) if g_b is not None else None, lr),
           "fw_group_grad_transform_step")


def fw_layer_get(handle, field: int, dst, nbytes: int) -> None:
    _check(_lib().fw_layer_get(handle, field, _ptr(dst), nbytes), "fw_layer_get")


def fw_layer_set(handle, field: int, src, nbytes: int) -> None:
    _check(_lib().fw_layer_set(handle, field, _ptr(src), nbytes), "fw_layer_set")


def fw_layer_sync_status(handle) -> int:
    """Returns FW_OK or one of the FW_WARN_* codes; raises on errors."""
    return _check(_lib().fw_layer_sync_status(handle), "fw_layer_sync_status",
                  allow=(FW_WARN_NO_SUBSPACE, FW_WARN_NONFINITE))


def fw_cov_block_static(X, rows: int, ldx: int, M: int, mu_out, phix_out, stream: int = 0) -> None:
    """Mean and covariance of one block with no workspace and no allocation
    (for callers that cannot allocate device memory); M <= FW_STATIC_MAX_M."""
    _check(_lib().fw_cov_block_static(_ptr(X), rows, ldx, M, _ptr(mu_out), _ptr(phix_out), stream),
           "fw_cov_block_static")


def fw_debug_wait_probe(handle, polls: int) -> None:
    _check(_lib().fw_debug_wait_probe(handle, polls), "fw_debug_wait_probe")


def fw_recursion_on_chip(desc: fw_layer_desc) -> bool:
    return bool(_lib().fw_recursion_on_chip(C.byref(desc)))


def fw_profile_begin() -> None:
    _check(_lib().fw_profile_begin(), "fw_profile_begin")


def fw_profile_end() -> dict:
    """{class name: (milliseconds, launches)} for the classes that ran."""
    n = len(FW_PROF_NAMES)
    ms = (C.c_float * n)()
    cnt = (C.c_int64 * n)()
    _check(_lib().fw_profile_end(ms, cnt), "fw_profile_end")
    return {FW_PROF_NAMES[i]: (float(ms[i]), int(cnt[i])) for i in range(n) if cnt[i]}


def fw_launch_count() -> int:
    return int(_lib().fw_launch_count())


# ---- convenience: a layer that owns its workspace tensor -------------------
class Layer:
    """Holds the torch workspace tensor (device memory plumbing) and the handle.
    Methods forward to the C entry points of the same name."""

    def __init__(self, M: int, N: int, device="cuda", stream: int = 0, **desc_overrides):
        import torch
        self.desc = fw_layer_desc_default(M, N, **desc_overrides)
        self.M, self.N = M, N
        self.nbytes = fw_layer_workspace_bytes(self.desc)
        if self.nbytes == 0:
            raise FwError(FW_ERR_INVALID_ARG, "fw_layer_workspace_bytes")
        self.workspace = torch.empty(self.nbytes + 256, dtype=torch.uint8, device=device)
        base = self.workspace.data_ptr()
        self._base = (base + 255) // 256 * 256
        self.handle = fw_layer_create(self.desc, self._base, self.nbytes, stream)
        self.device = device

    def close(self):
        if getattr(self, "handle", None):
            fw_layer_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self):
        fw_layer_reset(self.handle)

    def attach_params(self, W, b):
        fw_layer_attach_params(self.handle, W, b)

    def cov_update(self, X, flags: int = FW_COV_COMMIT):
        fw_cov_update(self.handle, X, X.shape[0], X.stride(0), flags)

    def cond_reduce(self, K, P, trace=None):
        fw_cond_reduce(self.handle, K, P, trace)

    def grad_transform(self, G, out=None):
        import torch
        out = torch.empty_like(G) if out is None else out
        fw_grad_transform(self.handle, G, out)
        return out

    def step(self, W, b, G_t, g_b, lr):
        fw_step(self.handle, W, b, G_t, g_b, lr)

    def get(self, field):
        import torch
        M = self.M
        n = 1 if field == FW_F_LAMBDA_BAR else (M if field in (FW_F_MU, FW_F_PHI_DIAG, FW_F_ALIGN_W) else M * M)
        out = torch.empty(n, dtype=torch.float32, device=self.device)
        fw_layer_get(self.handle, field, out, n * 4)
        return out.view(M, M) if n == M * M and M > 1 else out

    def set(self, field, t):
        t = t.contiguous()
        fw_layer_set(self.handle, field, t, t.numel() * 4)

    def sync_status(self):
        return fw_layer_sync_status(self.handle)
