"""Seeded synthetic layer inputs (W, X) shaped like the workloads of the Optimal Brain Compression paper.

This module only draws random numbers and arranges them (im2col, LayerNorm, GELU of the *inputs*); it
holds none of the method's arithmetic (no Hessian, no inverse, no OBS step, no quantiser).  It is the one
module that both the CPU oracle's tests and the CUDA path's tests / benchmark import, so that both sides
consume bit-identical FP32 arrays.

Layer convention (Section 2 of the paper, Eq. 2): W is d_row x d_col, X is d_col x N, conv layers are
unfolded so that d_col = c_in * kh * kw and every output position contributes one column of X.

The paper's own layers (ResNet / YOLOv5 / BERT weights, ImageNet / COCO / SQuAD activations) are not
available; these generators stand in for them with the same shapes and comparable value distributions.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np

DAMP_REL = 0.01  # relative dampening lambda = DAMP_REL * mean(diag(2 X X^T)), used by every config


@dataclasses.dataclass(frozen=True)
class LayerSpec:
    name: str
    seed: int
    d_row: int
    d_col: int
    n: int
    task: str          # "prune+quant", "prune", "quant", "compound"
    bits: int          # quantisation bits (0 = none)
    symmetric: bool
    sparsities: tuple  # global-mask sparsity targets (fractions of d_row*d_col)
    note: str


SPECS = {
    "C1": LayerSpec("C1", 0, 32, 64, 1024, "prune+quant", 4, True, (0.5,),
                    "tiny linear layer, correlated Gaussian inputs"),
    "C2": LayerSpec("C2", 1, 64, 576, 16384, "prune", 0, False, (0.6,),
                    "ResNet-18-style 3x3 conv 64->64, im2col of ReLU'd N(0,1), 56x56 stride 2"),
    "C3": LayerSpec("C3", 2, 256, 2304, 32768, "quant", 4, False, (),
                    "ResNet-50-bottleneck-style 3x3 conv 256->256, im2col of half-normal, 14x14 stride 1"),
    "C4": LayerSpec("C4", 3, 3072, 768, 65536, "compound", 8, True, (0.5,),
                    "BERT-base FFN up-projection, LayerNorm'd Gaussian with heavy-tailed channels"),
    "C5": LayerSpec("C5", 4, 768, 3072, 65536, "prune", 0, False, (0.4, 0.6, 0.8),
                    "BERT-base FFN down-projection, post-GELU activations"),
}


def pruned_count(d_row: int, d_col: int, sparsity: float) -> int:
    """k = round(sparsity * d_row * d_col): the integer number of weights the global mask removes."""
    return int(round(float(sparsity) * int(d_row) * int(d_col)))


def _im2col_3x3(act: np.ndarray, stride: int, pad: int, n_cols: int) -> np.ndarray:
    """act: (images, C, Hs, Ws) float32 -> X of shape (C*9, n_cols); row index = c*9 + ky*3 + kx;
    columns are ordered image-major, then output row, then output column; only the first n_cols are kept."""
    imgs, c, hs, ws = act.shape
    ho = (hs + 2 * pad - 3) // stride + 1
    wo = (ws + 2 * pad - 3) // stride + 1
    per_img = ho * wo
    need_imgs = (n_cols + per_img - 1) // per_img
    assert need_imgs <= imgs
    x = np.empty((c * 9, need_imgs * per_img), dtype=np.float32)
    padded = np.zeros((need_imgs, c, hs + 2 * pad, ws + 2 * pad), dtype=np.float32)
    padded[:, :, pad:pad + hs, pad:pad + ws] = act[:need_imgs]
    xv = x.reshape(c, 3, 3, need_imgs, ho, wo)
    for ky in range(3):
        for kx in range(3):
            patch = padded[:, :, ky:ky + stride * ho:stride, kx:kx + stride * wo:stride]  # (img, c, ho, wo)
            xv[:, ky, kx] = patch.transpose(1, 0, 2, 3)
    return np.ascontiguousarray(x[:, :n_cols])


def _gelu_erf(x: np.ndarray) -> np.ndarray:
    from scipy.special import erf
    return (0.5 * x * (1.0 + erf(x / np.float32(math.sqrt(2.0))))).astype(np.float32)


def make_layer(name: str, n_override: int | None = None):
    """Return (W, X, spec) for config `name` in SPECS.  W: float32 (d_row, d_col); X: float32 (d_col, N).

    n_override (tests only) shortens the calibration axis; the draw order is unchanged, the first
    n_override columns of the full X are NOT reproduced in general (C4/C5 draw N-dependent blocks).
    """
    spec = SPECS[name]
    rng = np.random.default_rng(spec.seed)
    r, d = spec.d_row, spec.d_col
    n = spec.n if n_override is None else int(n_override)
    if name == "C1":
        w = rng.normal(0.0, math.sqrt(1.0 / 64.0), size=(r, d))
        a = rng.normal(size=(d, d))
        cov = a @ a.T + 0.1 * np.eye(d)
        z = rng.normal(size=(d, n))
        x = np.linalg.cholesky(cov) @ z
    elif name == "C2":
        w = rng.normal(0.0, math.sqrt(2.0 / d), size=(r, d))
        per_img = 28 * 28
        imgs = (n + per_img - 1) // per_img
        act = np.maximum(rng.normal(size=(imgs, 64, 56, 56)), 0.0).astype(np.float32)
        x = _im2col_3x3(act, stride=2, pad=1, n_cols=n)
    elif name == "C3":
        w = rng.normal(0.0, math.sqrt(2.0 / d), size=(r, d))
        per_img = 14 * 14
        imgs = (n + per_img - 1) // per_img
        act = np.abs(rng.normal(size=(imgs, 256, 14, 14))).astype(np.float32)
        x = _im2col_3x3(act, stride=1, pad=1, n_cols=n)
    elif name == "C4":
        w = rng.normal(0.0, 0.02, size=(r, d))
        g = rng.standard_normal(size=(d, n), dtype=np.float32)
        heavy = rng.choice(d, size=6, replace=False)
        g[heavy, :] = rng.standard_t(3.0, size=(6, n)).astype(np.float32)
        mu = g.mean(axis=0, keepdims=True, dtype=np.float64)
        var = g.var(axis=0, keepdims=True, dtype=np.float64)
        x = ((g - mu) / np.sqrt(var + 1e-12))
    elif name == "C5":
        w = rng.normal(0.0, 0.02, size=(r, d))
        b = rng.normal(0.0, math.sqrt(1.0 / 768.0), size=(d, 768)).astype(np.float32)
        g = rng.standard_normal(size=(768, n), dtype=np.float32)
        x = np.empty((d, n), dtype=np.float32)
        step = 8192
        for c0 in range(0, n, step):
            x[:, c0:c0 + step] = _gelu_erf(b @ g[:, c0:c0 + step])
    else:
        raise KeyError(name)
    return (np.ascontiguousarray(w, dtype=np.float32), np.ascontiguousarray(x, dtype=np.float32), spec)


def make_small(d_row: int, d_col: int, n: int, seed: int, kind: str = "correlated"):
    """Small seeded problems for tests: 'correlated' (dense covariance), 'orthogonal' (X X^T diagonal),
    'relu' (non-negative skewed inputs)."""
    rng = np.random.default_rng(seed)
    w = rng.normal(0.0, 1.0 / math.sqrt(d_col), size=(d_row, d_col))
    if kind == "correlated":
        a = rng.normal(size=(d_col, d_col))
        z = rng.normal(size=(d_col, n))
        x = np.linalg.cholesky(a @ a.T + 0.1 * np.eye(d_col)) @ z
    elif kind == "relu":
        a = rng.normal(size=(d_col, d_col)) / math.sqrt(d_col)
        x = np.maximum(a @ rng.normal(size=(d_col, n)), 0.0)
    elif kind == "orthogonal":
        assert n >= d_col
        q, _ = np.linalg.qr(rng.normal(size=(n, d_col)))
        x = (q * rng.uniform(0.5, 2.0, size=(1, d_col))).T
    else:
        raise KeyError(kind)
    return np.ascontiguousarray(w, dtype=np.float32), np.ascontiguousarray(x, dtype=np.float32)
