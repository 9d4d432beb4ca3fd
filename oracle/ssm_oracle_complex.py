"""fp64 CPU oracle of the selective scan with a complex-valued state (Section 3.6, "Real vs. Complex").

TEST INFRASTRUCTURE, NOT THE PRODUCT: only tests/ may import this module.  It shares no code with the CUDA path.

What it computes, per batch entry b and channel d independently, with A (D, N), B and C (batch, L, N) complex and
x, delta, z, D_skip real:

    a[t,n]  = exp(delta[t] * A[d,n])                              Eq. 4's A-bar, complex exponential
    h[t,n]  = a[t,n] * h[t-1,n] + delta[t] * B[t,n] * x[t]        Eq. 2a; h[0] = h0 or 0; h complex
    s[t]    = 2 * Re(sum_n C[t,n] * h[t,n]) + D_skip[d] * x[t]    Eq. 2b for a real output, plus the skip term
    out[t]  = s[t] * silu(z[t])                                   gate (Section 3.4)

Reading taken where the paper is silent: the paper says only that the state may be complex (and that S4D-Lin,
A_n = -1/2 + n i, is its initialisation); it does not say how a complex state yields a real output.  The N complex
states are taken to stand for N conjugate pairs of a real system (the convention of the S4D parameterisation the paper
cites for its initialisations), so the real output is twice the real part of the readout.  B-bar is delta * B (the
default rule of the real path).

The forward is the definition written out one step after another (numpy complex128 arithmetic over the (batch, D, N)
axes of a step is a library primitive; there is no blocking or reordering in time).  The backward is the analytic
adjoint for the real loss sum(dout * out).  The gradient of a complex quantity q = q_re + i q_im is returned as
dL/dq_re + i dL/dq_im.  With lam[t] the gradient of h[t] in that convention (lam[L+1] = 0 or dh_last):

    ds[t]   = dout[t] * silu(z[t]);   dz[t] = dout[t] * s[t] * silu'(z[t])
    lam[t]  = 2 ds[t] conj(C[t]) + conj(a[t+1]) lam[t+1]
    dC[t,n] = sum_d 2 ds[t] conj(h[t,n]);   dB[t,n] = sum_d delta[t] x[t] lam[t,n];   dD = sum ds x
    dx[t]   = ds[t] D_skip + delta[t] sum_n Re(conj(B[t,n]) lam[t,n])
    w[t,n]  = conj(a[t,n] h[t-1,n]) lam[t,n]          (gradient reaching the exponent delta A)
    ddelta[t] = sum_n Re(conj(A[n]) w[t,n]) + x[t] sum_n Re(conj(B[t,n]) lam[t,n]);   dA[n] = sum_t delta[t] w[t,n]
    dh0[n]  = conj(a[1,n]) lam[1,n]

(the rule used throughout: for a product p = u v of complex numbers, the gradient of u is conj(v) times the gradient
of p; for a real u, its real part).  Pins: tests/test_oracle_complex_pins.py.
"""
from __future__ import annotations

import numpy as np


def _silu(z):
    return z / (1.0 + np.exp(-z))


def _f64(a):
    return None if a is None else np.asarray(a, dtype=np.float64)


def _c128(a):
    return None if a is None else np.asarray(a, dtype=np.complex128)


def scan_fwd(x, delta, A, B, C, D_skip=None, z=None, h0=None, return_pregate=False, return_h_last=False,
             return_states=False):
    """x, delta, z: (batch, L, D) real; A: (D, N) complex; B, C: (batch, L, N) complex; D_skip: (D); h0: (batch, D, N)
    complex or None.  Returns float64 out (batch, L, D) and, if asked, the pre-gate readout s, the final state
    (batch, D, N) and all states (batch, L + 1, D, N)."""
    x, delta, z, D_skip = _f64(x), _f64(delta), _f64(z), _f64(D_skip)
    A, B, C, h0 = _c128(A), _c128(B), _c128(C), _c128(h0)
    batch, L, D = x.shape
    N = A.shape[1]
    assert A.shape == (D, N) and B.shape == (batch, L, N) and C.shape == (batch, L, N) and delta.shape == x.shape
    h = np.zeros((batch, D, N), dtype=np.complex128) if h0 is None else h0.copy()
    s = np.empty((batch, L, D))
    states = np.empty((batch, L + 1, D, N), dtype=np.complex128) if return_states else None
    if return_states:
        states[:, 0] = h
    for t in range(L):
        a = np.exp(delta[:, t, :, None] * A[None])
        h = a * h + (delta[:, t] * x[:, t])[:, :, None] * B[:, t, None, :]
        s[:, t] = 2.0 * np.real((C[:, t, None, :] * h).sum(-1))
        if D_skip is not None:
            s[:, t] += D_skip[None] * x[:, t]
        if return_states:
            states[:, t + 1] = h
    out = s * _silu(z) if z is not None else s.copy()
    res = (out,)
    if return_pregate:
        res += (s,)
    if return_h_last:
        res += (h,)
    if return_states:
        res += (states,)
    return res[0] if len(res) == 1 else res


def scan_bwd(x, delta, A, B, C, D_skip, z, dout, h0=None, dh_last=None):
    """Adjoint of scan_fwd for loss = sum(dout * out).  Returns a dict: dx, ddelta, dz (batch, L, D) float64; dB, dC
    (batch, L, N), dA (D, N), dh0 (batch, D, N) complex128 (real-part and imaginary-part gradients); dD (D)."""
    x, delta, z, D_skip, dout = _f64(x), _f64(delta), _f64(z), _f64(D_skip), _f64(dout)
    A, B, C = _c128(A), _c128(B), _c128(C)
    batch, L, D = x.shape
    N = A.shape[1]
    _, s, _, hs = scan_fwd(x, delta, A, B, C, D_skip, z, h0, return_pregate=True, return_h_last=True, return_states=True)
    if z is not None:
        sg = 1.0 / (1.0 + np.exp(-z))
        ds = dout * z * sg
        dz = dout * s * sg * (1.0 + z * (1.0 - sg))
    else:
        ds = dout.copy()
        dz = np.zeros_like(dout)
    g = dict(dx=np.empty((batch, L, D)), ddelta=np.empty((batch, L, D)), dz=dz,
             dB=np.empty((batch, L, N), dtype=np.complex128), dC=np.empty((batch, L, N), dtype=np.complex128),
             dA=np.zeros((D, N), dtype=np.complex128), dD=np.zeros(D))
    mu = np.zeros((batch, D, N), dtype=np.complex128) if dh_last is None else _c128(dh_last).copy()   # conj(a[t+1]) lam[t+1]
    for t in range(L - 1, -1, -1):
        a = np.exp(delta[:, t, :, None] * A[None])
        lam = 2.0 * ds[:, t, :, None] * np.conj(C[:, t, None, :]) + mu
        g["dC"][:, t] = (2.0 * ds[:, t, :, None] * np.conj(hs[:, t + 1])).sum(1)
        g["dB"][:, t] = ((delta[:, t] * x[:, t])[:, :, None] * lam).sum(1)
        lamB = np.real(np.conj(B[:, t, None, :]) * lam).sum(-1)
        w = np.conj(a * hs[:, t]) * lam
        g["dx"][:, t] = delta[:, t] * lamB + (ds[:, t] * D_skip[None] if D_skip is not None else 0.0)
        g["ddelta"][:, t] = np.real(np.conj(A[None]) * w).sum(-1) + x[:, t] * lamB
        g["dA"] += (delta[:, t, :, None] * w).sum(0)
        mu = np.conj(a) * lam
    if D_skip is not None:
        g["dD"] = (ds * x).sum((0, 1))
    g["dh0"] = mu
    return g
