"""Seeded synthetic inputs shaped like the workloads the method is run on.

This module only draws random numbers and lays them out (orthogonal bases,
prescribed spectra, Wishart channel correlation, half-normal feature maps,
im2col patch extraction).  It contains none of the whitening method's
arithmetic: no moment tracking, no recursion, no gradient transform.  It is the
single piece shared by the fp64 CPU checker and the CUDA tests / benchmark so
both see bit-identical inputs.

Every generator takes an explicit integer seed and uses numpy's PCG64, so the
same call returns the same bits on every machine.
"""
from __future__ import annotations

import numpy as np

SEED_BASE = 20100154


def layer_seed(config: int, layer: int = 0) -> int:
    """Seed convention: one stream per (workload, layer)."""
    return SEED_BASE + 1000 * int(config) + int(layer)


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(int(seed)))


# ----------------------------------------------------------------------------
# orthogonal bases and matrices with a prescribed spectrum
# ----------------------------------------------------------------------------
def orthogonal_qr(M: int, seed: int) -> np.ndarray:
    """Haar-distributed orthogonal matrix: Q factor of a Gaussian matrix with
    the sign ambiguity removed by making diag(R) positive."""
    g = _rng(seed).standard_normal((M, M))
    q, r = np.linalg.qr(g)
    d = np.sign(np.diag(r))
    d[d == 0] = 1.0
    return q * d[None, :]


def orthogonal_householder(M: int, seed: int, reflectors: int = 8) -> np.ndarray:
    """Orthogonal matrix built as a product of a few random Householder
    reflectors; O(M^2) per reflector, used where a QR of a large matrix per
    layer would dominate set-up time.  Exactly orthogonal up to rounding."""
    rng = _rng(seed)
    U = np.eye(M)
    for _ in range(reflectors):
        w = rng.standard_normal(M)
        w /= np.linalg.norm(w)
        U -= 2.0 * np.outer(U @ w, w)
    return U


def spd_with_spectrum(M: int, cond: float, seed: int, basis: str = "qr"):
    """Symmetric positive definite matrix U diag(logspace(0,-log10 cond)) U^T.

    Returns (Phi, U, lam) in fp64; Phi is symmetrised exactly."""
    lam = np.logspace(0.0, -np.log10(cond), M)
    U = orthogonal_qr(M, seed) if basis == "qr" else orthogonal_householder(M, seed)
    Phi = (U * lam[None, :]) @ U.T
    Phi = 0.5 * (Phi + Phi.T)
    return Phi, U, lam


def gaussian_rows(rows: int, U: np.ndarray, lam: np.ndarray, seed: int,
                  mean: np.ndarray | None = None) -> np.ndarray:
    """rows samples of N(mean, U diag(lam) U^T), one per row, fp64."""
    M = U.shape[0]
    z = _rng(seed).standard_normal((rows, M))
    x = (z * np.sqrt(lam)[None, :]) @ U.T
    if mean is not None:
        x += mean[None, :]
    return x


def cost_sweep_layer(B: int, M: int = 2304, N: int = 256, HW: int = 14, cond: float = 1e4,
                     chunk_rows: int = 25088) -> dict:
    """Large-batch single layer of the cost sweep: a 3x3 convolution with 256 input channels on 14x14 maps
    (M = 2304, N = 256, rows = 196 B).  Rows are Gaussian with covariance U diag(logspace(0, -log10 cond)) U^T,
    drawn chunk by chunk (each chunk its own seed) in fp32; Householder-product basis."""
    rows = B * HW * HW
    lam = np.logspace(0.0, -np.log10(cond), M)
    U = orthogonal_householder(M, layer_seed(4, 0))
    Ut = np.ascontiguousarray((U * np.sqrt(lam)[None, :]).T).astype(np.float32)   # diag(sqrt(lam)) U^T
    X = np.empty((rows, M), dtype=np.float32)
    for c, r0 in enumerate(range(0, rows, chunk_rows)):
        r1 = min(rows, r0 + chunk_rows)
        z = _rng(layer_seed(4, 1 + c)).standard_normal((r1 - r0, M), dtype=np.float32)
        np.matmul(z, Ut, out=X[r0:r1])
    g = _rng(layer_seed(4, 900))
    G = g.standard_normal((N, M)).astype(np.float32)
    W = (g.standard_normal((N, M)) / np.sqrt(M)).astype(np.float32)
    b = np.zeros(N, dtype=np.float32)
    gb = g.standard_normal(N).astype(np.float32)
    return dict(M=M, N=N, rows=rows, X=X, G=G, W=W, b=b, gb=gb)


# ----------------------------------------------------------------------------
# single linear layer (the small fp32 case)
# ----------------------------------------------------------------------------
def single_linear_layer(M: int = 64, N: int = 32, B: int = 128, decades: float = 3.0,
                        seed: int | None = None) -> dict:
    """Rows of X ~ N(0, Phi), Phi = U diag(logspace(0,-decades,M)) U^T with a
    seeded orthogonal U; G is N x M i.i.d. N(0,1); W ~ N(0, 1/M); b = 0."""
    seed = layer_seed(1) if seed is None else seed
    Phi, U, lam = spd_with_spectrum(M, 10.0 ** decades, seed)
    X = gaussian_rows(B, U, lam, seed + 1)
    r = _rng(seed + 2)
    G = r.standard_normal((N, M))
    W = r.standard_normal((N, M)) / np.sqrt(M)
    b = np.zeros(N)
    gb = r.standard_normal(N)
    return dict(M=M, N=N, rows=B, X=X, G=G, W=W, b=b, gb=gb, Phi=Phi)


# ----------------------------------------------------------------------------
# convolution-shaped layers: Wishart channel correlation, half-normal pixels,
# im2col patch rows
# ----------------------------------------------------------------------------
def wishart_corr(C: int, seed: int, decades: float = 0.0) -> np.ndarray:
    """Channel covariance A A^T / nu with A a C x nu Gaussian, nu = 2C.
    With decades > 0 the spectrum is additionally shaped by
    S^{1/2} diag(logspace(0,-decades,C)) S^{1/2} to widen the eigenvalue spread."""
    nu = 2 * C
    A = _rng(seed).standard_normal((C, nu))
    S = A @ A.T / nu
    if decades > 0.0:
        w, V = np.linalg.eigh(S)
        Sh = (V * np.sqrt(np.maximum(w, 0.0))[None, :]) @ V.T
        d = np.logspace(0.0, -decades, C)
        S = (Sh * d[None, :]) @ Sh
        S = 0.5 * (S + S.T)
    return S


def halfnormal_feature_map(B: int, H: int, W: int, C: int, seed: int,
                           decades: float = 0.0, dtype=np.float32, batch_index: int = 0) -> np.ndarray:
    """B x H x W x C map with pixels |z|, z ~ N(0, Sigma) i.i.d. over pixels,
    Sigma from wishart_corr (post-ReLU-like, non-negative, correlated channels).
    Sigma depends on the seed only (a property of the layer); batch_index picks
    an independent draw of the pixels."""
    S = wishart_corr(C, seed, decades)
    L = np.linalg.cholesky(S + 1e-12 * np.eye(C))
    rng = _rng(seed + 7 + 101 * batch_index)
    out = np.empty((B, H, W, C), dtype=dtype)
    # generate a few images at a time so the peak fp64 footprint stays small
    step = max(1, (1 << 22) // (H * W * C))
    for b0 in range(0, B, step):
        b1 = min(B, b0 + step)
        z = rng.standard_normal((b1 - b0, H, W, C))
        out[b0:b1] = np.abs(z @ L.T).astype(dtype)
    return out


def im2col(fm: np.ndarray, k: int = 3, pad: int = 1) -> np.ndarray:
    """B x H x W x C  ->  (B*H*W) x (k*k*C) patch rows, stride 1, zero padding.
    Column order is (ky, kx, c)."""
    B, H, W, C = fm.shape
    if k == 1:
        return fm.reshape(B * H * W, C)
    p = np.zeros((B, H + 2 * pad, W + 2 * pad, C), dtype=fm.dtype)
    p[:, pad:pad + H, pad:pad + W, :] = fm
    X = np.empty((B, H, W, k * k * C), dtype=fm.dtype)
    for ky in range(k):
        for kx in range(k):
            j = (ky * k + kx) * C
            X[..., j:j + C] = p[:, ky:ky + H, kx:kx + W, :]
    return X.reshape(B * H * W, k * k * C)


def conv_layer_inputs(B: int, HW: int, C_in: int, C_out: int, k: int, seed: int,
                      decades: float = 0.0, dtype=np.float32, batch_index: int = 0) -> dict:
    """Patch matrix X (rows = B*HW*HW, M = C_in*k*k), gradient G (N x M),
    weights W, bias b, bias gradient gb for one convolution-shaped layer."""
    fm = halfnormal_feature_map(B, HW, HW, C_in, seed, decades, dtype, batch_index)
    X = im2col(fm, k, (k - 1) // 2)
    M = C_in * k * k
    r = _rng(seed + 3 + 101 * batch_index)
    G = r.standard_normal((C_out, M)).astype(np.float32)
    r2 = _rng(seed + 5)
    W = (r2.standard_normal((C_out, M)) / np.sqrt(M)).astype(np.float32)
    b = np.zeros(C_out, dtype=np.float32)
    gb = r.standard_normal(C_out).astype(np.float32)
    return dict(M=M, N=C_out, rows=X.shape[0], X=X, G=G, W=W, b=b, gb=gb, fm=fm)


# layer shape tables (rows = B*HW*HW, M = C_in*k*k, N = C_out)
def resnet20_shapes(B: int = 128):
    """Fifteen 3x3 convolutions in three stages of five."""
    out = []
    for (C, HW) in ((16, 32), (32, 16), (64, 8)):
        for _ in range(5):
            out.append(dict(B=B, HW=HW, C_in=C, C_out=C, k=3))
    return out


def resnet50_shapes(B: int = 256):
    """Bottleneck 1x1 / 3x3 shapes per stage plus the final fully connected layer."""
    s = []
    s += [dict(B=B, HW=56, C_in=64, C_out=64, k=1), dict(B=B, HW=56, C_in=256, C_out=64, k=1),
          dict(B=B, HW=56, C_in=64, C_out=64, k=3), dict(B=B, HW=56, C_in=64, C_out=256, k=1)]
    s += [dict(B=B, HW=28, C_in=512, C_out=128, k=1), dict(B=B, HW=28, C_in=128, C_out=128, k=3),
          dict(B=B, HW=28, C_in=128, C_out=512, k=1)]
    s += [dict(B=B, HW=14, C_in=1024, C_out=256, k=1), dict(B=B, HW=14, C_in=256, C_out=256, k=3),
          dict(B=B, HW=14, C_in=256, C_out=1024, k=1)]
    s += [dict(B=B, HW=7, C_in=2048, C_out=512, k=1), dict(B=B, HW=7, C_in=512, C_out=512, k=3),
          dict(B=B, HW=7, C_in=512, C_out=2048, k=1)]
    s += [dict(B=B, HW=1, C_in=2048, C_out=1000, k=1)]
    return s


def shape_dims(s: dict):
    return s["B"] * s["HW"] * s["HW"], s["C_in"] * s["k"] * s["k"], s["C_out"]


def to_bf16_grid(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bfloat16 (ties to even) and return them
    as fp32, so that a bf16 device copy and the fp64 checker see equal values."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> 16) & 1) + np.uint32(0x7FFF)
    u2 = ((u + r) & np.uint32(0xFFFF0000)).astype(np.uint32)
    return u2.view(np.float32).reshape(x.shape)


def bf16_bits(x_on_grid: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of values already on the bf16 grid."""
    u = np.ascontiguousarray(x_on_grid, dtype=np.float32).view(np.uint32)
    return (u >> 16).astype(np.uint16).reshape(x_on_grid.shape)


# ----------------------------------------------------------------------------
# device-side twins of the generators above, for timing-only workloads whose
# inputs (gigabytes of patch rows) would take the host cores minutes to draw.
# Same recipe and layout; the random stream is torch's, seeded per layer.
# ----------------------------------------------------------------------------
def conv_layer_inputs_device(torch, device, B: int, HW: int, C_in: int, C_out: int, k: int, seed: int,
                             decades: float = 0.0, bf16: bool = False, batch_index: int = 0) -> dict:
    """As conv_layer_inputs, drawn on the device: X (rows x M, fp32 or bf16), G, W, b, gb as device tensors."""
    S = wishart_corr(C_in, seed, decades)
    Lc = torch.from_numpy(np.linalg.cholesky(S + 1e-12 * np.eye(C_in)).astype(np.float32)).to(device)
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) + 7 + 101 * int(batch_index))
    M = C_in * k * k
    rows = B * HW * HW
    X = torch.empty((B, HW, HW, M), dtype=torch.bfloat16 if bf16 else torch.float32, device=device)
    step = max(1, (1 << 25) // (HW * HW * C_in))
    pad = (k - 1) // 2
    for b0 in range(0, B, step):
        b1 = min(B, b0 + step)
        fm = (torch.randn((b1 - b0, HW, HW, C_in), generator=g, device=device) @ Lc.T).abs_()
        if k == 1:
            X[b0:b1] = fm
        else:
            p = torch.zeros((b1 - b0, HW + 2 * pad, HW + 2 * pad, C_in), device=device)
            p[:, pad:pad + HW, pad:pad + HW, :] = fm
            for ky in range(k):
                for kx in range(k):
                    j = (ky * k + kx) * C_in
                    X[b0:b1, :, :, j:j + C_in] = p[:, ky:ky + HW, kx:kx + HW, :]
    X = X.view(rows, M)
    G = torch.randn((C_out, M), generator=g, device=device)
    W = torch.randn((C_out, M), generator=g, device=device) / float(np.sqrt(M))
    b = torch.zeros(C_out, device=device)
    gb = torch.randn(C_out, generator=g, device=device)
    return dict(M=M, N=C_out, rows=rows, X=X, G=G, W=W, b=b, gb=gb)


def cost_sweep_layer_device(torch, device, B: int, M: int = 2304, N: int = 256, HW: int = 14, cond: float = 1e4,
                            batch_index: int = 0) -> dict:
    """As cost_sweep_layer, drawn on the device (fp32 rows with covariance U diag(logspace) U^T)."""
    rows = B * HW * HW
    lam = np.logspace(0.0, -np.log10(cond), M)
    U = orthogonal_householder(M, layer_seed(4, 0))
    Ut = torch.from_numpy(np.ascontiguousarray((U * np.sqrt(lam)[None, :]).T).astype(np.float32)).to(device)
    g = torch.Generator(device=device)
    g.manual_seed(layer_seed(4, 1) + 101 * int(batch_index))
    X = torch.empty((rows, M), dtype=torch.float32, device=device)
    chunk = 25088
    allow = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = False
    for r0 in range(0, rows, chunk):
        r1 = min(rows, r0 + chunk)
        torch.matmul(torch.randn((r1 - r0, M), generator=g, device=device), Ut, out=X[r0:r1])
    torch.backends.cuda.matmul.allow_tf32 = allow
    G = torch.randn((N, M), generator=g, device=device)
    W = torch.randn((N, M), generator=g, device=device) / float(np.sqrt(M))
    return dict(M=M, N=N, rows=rows, X=X, G=G, W=W, b=torch.zeros(N, device=device),
                gb=torch.randn(N, generator=g, device=device))
