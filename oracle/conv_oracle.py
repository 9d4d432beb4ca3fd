"""fp64 CPU oracle of the short causal depthwise convolution that precedes the selective scan in the block
(Section 3.4 / Figure 3: "Conv" followed by the SiLU activation on the SSM branch).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only tests/, the smoke check and the benchmark's CPU-baseline leg may import
this module; it shares nothing with the CUDA path.

Definition, per batch b and channel d independently (depthwise), with a kernel of W taps w[d, 0..W-1] whose last tap
multiplies the current step (causal):
    pre[b, t, d] = bias[d] + sum_{k=0}^{W-1} w[d, k] * x[b, t - (W - 1) + k, d],      x[b, s, d] = x_prev or 0 for s < 0
    y[b, t, d]   = silu(pre) = pre / (1 + exp(-pre))     (or y = pre without the activation)
`x_prev` (batch, W-1, D) holds the W-1 inputs before the first step when a sequence is processed in pieces.
The backward functions are the adjoint for loss = sum(dy * y):
    dpre = dy * silu'(pre),  silu'(v) = sig(v) (1 + v (1 - sig(v)))
    dx[b, s, d]  = sum_k w[d, k] * dpre[b, s + (W - 1) - k, d]         (terms past the end of the sequence vanish)
    dw[d, k]     = sum_{b, t} dpre[b, t, d] * x[b, t - (W - 1) + k, d]
    dbias[d]     = sum_{b, t} dpre[b, t, d]
The loops below run over taps and use whole-array slices for (b, t, d): that is the definition written out, not a
reorganisation of it.
"""
from __future__ import annotations

import numpy as np


def _padded(x, W, x_prev):
    batch, L, D = x.shape
    xp = np.zeros((batch, L + W - 1, D), dtype=np.float64)
    if x_prev is not None and W > 1:
        xp[:, :W - 1] = np.asarray(x_prev, dtype=np.float64)
    xp[:, W - 1:] = x
    return xp


def conv1d_fwd(x, w, bias=None, silu=True, x_prev=None, return_pre=False):
    """x: (batch, L, D); w: (D, W); bias: (D) or None; returns y (batch, L, D) in float64."""
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    batch, L, D = x.shape
    W = w.shape[1]
    assert w.shape == (D, W)
    xp = _padded(x, W, x_prev)
    pre = np.zeros((batch, L, D))
    if bias is not None:
        pre += np.asarray(bias, dtype=np.float64)[None, None, :]
    for k in range(W):
        pre += w[:, k][None, None, :] * xp[:, k:k + L]          # xp[t + k] = x[t - (W - 1) + k]
    y = pre / (1.0 + np.exp(-pre)) if silu else pre
    return (y, pre) if return_pre else y


def conv1d_bwd(x, w, bias, dy, silu=True, x_prev=None):
    """Returns dict dx (batch, L, D), dw (D, W), dbias (D), dx_prev (batch, W-1, D), all float64."""
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    dy = np.asarray(dy, dtype=np.float64)
    batch, L, D = x.shape
    W = w.shape[1]
    _, pre = conv1d_fwd(x, w, bias, silu, x_prev, return_pre=True)
    if silu:
        sg = 1.0 / (1.0 + np.exp(-pre))
        dpre = dy * sg * (1.0 + pre * (1.0 - sg))
    else:
        dpre = dy
    xp = _padded(x, W, x_prev)
    dxp = np.zeros_like(xp)
    dw = np.zeros((D, W))
    for k in range(W):
        dxp[:, k:k + L] += w[:, k][None, None, :] * dpre
        dw[:, k] = (dpre * xp[:, k:k + L]).sum(axis=(0, 1))
    return {"dx": dxp[:, W - 1:], "dx_prev": dxp[:, :W - 1], "dw": dw, "dbias": dpre.sum(axis=(0, 1))}
