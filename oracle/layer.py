"""The element-wise pre- and post-operations of the GSA layer (Sec. 3.3 of arXiv 2409.07146) in
plain numpy fp64 -- TEST INFRASTRUCTURE ONLY, like the rest of this package.

    q, k, v = Swish(W_q x), Swish(W_k x), Swish(W_v x)          (feature map, per head)
    y       = W_o RMSNorm(Swish(concat_h o^h))                   (output path)

Only the element-wise parts live here (the projections are the caller's GEMMs): the Swish
feature map with its derivative, and Swish followed by RMSNorm over all heads of a token,
forward and backward.  RMSNorm is taken as  y = w * x / sqrt(mean(x^2) + eps)  (root mean
square over the H d_v values of a token, optional per-channel weight w, eps inside the root).
"""
from __future__ import annotations

import numpy as np


def swish(x):
    x = np.asarray(x, dtype=np.float64)
    return x / (1.0 + np.exp(-x))


def swish_grad(x):
    """d Swish(x) / dx = s (1 + x (1 - s)), s = sigmoid(x)."""
    x = np.asarray(x, dtype=np.float64)
    s = 1.0 / (1.0 + np.exp(-x))
    return s * (1.0 + x * (1.0 - s))


def out_norm_fwd(o, weight=None, eps=1e-6):
    """o [B,T,H,d_v] -> y [B,T,H,d_v] = RMSNorm(Swish(o)) over the H d_v values of every token."""
    o = np.asarray(o, dtype=np.float64)
    B, T, H, D = o.shape
    x = swish(o).reshape(B, T, H * D)
    r = np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps)
    y = x / r
    if weight is not None:
        y = y * np.asarray(weight, dtype=np.float64).reshape(1, 1, H * D)
    return y.reshape(B, T, H, D)


def out_norm_bwd(o, dy, weight=None, eps=1e-6):
    """Gradients of out_norm_fwd: returns (do [B,T,H,d_v], dweight [H d_v])."""
    o = np.asarray(o, dtype=np.float64)
    dy = np.asarray(dy, dtype=np.float64)
    B, T, H, D = o.shape
    N = H * D
    x = swish(o).reshape(B, T, N)
    g = dy.reshape(B, T, N)
    w = np.ones(N) if weight is None else np.asarray(weight, dtype=np.float64).reshape(N)
    r = np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps)
    xhat = x / r
    dweight = (g * xhat).sum(axis=(0, 1))
    gx = g * w                                     # gradient w.r.t. xhat
    dx = (gx - xhat * np.mean(gx * xhat, axis=-1, keepdims=True)) / r
    do = dx.reshape(B, T, H, D) * swish_grad(o)
    return do, dweight
