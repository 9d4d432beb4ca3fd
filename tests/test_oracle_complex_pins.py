"""Pins of the complex-state oracle (oracle/ssm_oracle_complex.py) against routes other than its own time loop: the
already pinned real oracle, a closed-form convolution kernel, a library matrix exponential of the equivalent real 2x2
system, a closed-form oscillation, finite differences and invariants.  CPU only."""
import numpy as np
import pytest

from oracle import ssm_oracle as O
from oracle import ssm_oracle_complex as OC

RNG = np.random.default_rng(20231203)


def _problem(batch, L, D, N, rng=RNG, dt_scale=0.3):
    cplx = lambda *s: rng.standard_normal(s) + 1j * rng.standard_normal(s)
    return dict(x=rng.standard_normal((batch, L, D)), z=rng.standard_normal((batch, L, D)),
                delta=dt_scale * rng.uniform(0.05, 1.0, (batch, L, D)), B=cplx(batch, L, N), C=cplx(batch, L, N),
                A=-rng.uniform(0.2, 2.0, (D, N)) + 1j * rng.uniform(-3.0, 3.0, (D, N)), D_skip=rng.standard_normal(D))


def _fwd(p, **kw):
    return OC.scan_fwd(p["x"], p["delta"], p["A"], p["B"], p["C"], D_skip=p["D_skip"], z=p["z"], **kw)


# A complex system whose A, B, C all have zero imaginary part is the real system with the readout doubled: the
# complex oracle must reproduce the real oracle (pinned in test_oracle_pins.py) on it, forward and backward.
def test_zero_imaginary_parts_reduce_to_the_real_oracle():
    p = _problem(2, 40, 5, 4)
    for k in ("A", "B", "C"):
        p[k] = p[k].real + 0j
    dout = RNG.standard_normal(p["x"].shape)
    out = _fwd(p)
    ref = O.scan_fwd(p["x"], p["delta"], p["A"].real, p["B"].real, 2.0 * p["C"].real, D_skip=p["D_skip"], z=p["z"])
    np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-13)
    g = OC.scan_bwd(p["x"], p["delta"], p["A"], p["B"], p["C"], p["D_skip"], p["z"], dout)
    r = O.scan_bwd(p["x"], p["delta"], p["A"].real, p["B"].real, 2.0 * p["C"].real, p["D_skip"], p["z"], dout)
    for k in ("dx", "ddelta", "dz", "dD"):
        np.testing.assert_allclose(g[k], r[k], rtol=1e-11, atol=1e-12, err_msg=k)
    # gradients with respect to the real parts: dB as is, dC through C' = 2 C, dA as is
    np.testing.assert_allclose(g["dB"].real, r["dB"], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(g["dC"].real, 2.0 * r["dC"], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(g["dA"].real, r["dA"], rtol=1e-11, atol=1e-12)


# LTI closed form (Eq. 3 with a complex diagonal A): constant delta, B, C give the causal convolution with the real
# kernel K_k = 2 Re(sum_n C_n Abar_n^k Bbar_n), computed with numpy's own complex power and numpy.convolve.
def test_lti_equals_convolution_with_complex_kernel():
    batch, L, D, N = 2, 80, 4, 5
    p = _problem(batch, L, D, N)
    dt_d = RNG.uniform(0.01, 0.4, D)
    Bn = RNG.standard_normal(N) + 1j * RNG.standard_normal(N)
    Cn = RNG.standard_normal(N) + 1j * RNG.standard_normal(N)
    p["delta"] = np.broadcast_to(dt_d, (batch, L, D)).copy()
    p["B"] = np.broadcast_to(Bn, (batch, L, N)).copy()
    p["C"] = np.broadcast_to(Cn, (batch, L, N)).copy()
    s = OC.scan_fwd(p["x"], p["delta"], p["A"], p["B"], p["C"], D_skip=p["D_skip"], z=None)
    k = np.arange(L)
    for b in range(batch):
        for d in range(D):
            Abar = np.exp(dt_d[d] * p["A"][d])
            K = 2.0 * np.real(((Cn * dt_d[d] * Bn)[None, :] * Abar[None, :] ** k[:, None]).sum(-1))
            ref = np.convolve(p["x"][b, :, d], K)[:L] + p["D_skip"][d] * p["x"][b, :, d]
            np.testing.assert_allclose(s[b, :, d], ref, rtol=1e-11, atol=1e-12)


# One complex state alpha + i omega is the real 2-d system v' = [[alpha, -omega], [omega, alpha]] v: the transition over
# a step comes from scipy's matrix exponential, the input enters as (Re, Im) of delta B x, and the output is
# 2 (Re C, -Im C) . v.  This fixes the sign conventions of the complex multiply independently of numpy's complex type.
def test_single_state_equals_real_rotation_system():
    from scipy.linalg import expm
    batch, L, D = 1, 30, 3
    p = _problem(batch, L, D, 1)
    s = OC.scan_fwd(p["x"], p["delta"], p["A"], p["B"], p["C"], D_skip=None, z=None)
    for d in range(D):
        al, om = p["A"][d, 0].real, p["A"][d, 0].imag
        M = np.array([[al, -om], [om, al]])
        v = np.zeros(2)
        for t in range(L):
            dt, u = p["delta"][0, t, d], p["x"][0, t, d]
            Bt, Ct = p["B"][0, t, 0], p["C"][0, t, 0]
            v = expm(dt * M) @ v + dt * u * np.array([Bt.real, Bt.imag])
            np.testing.assert_allclose(s[0, t, d], 2.0 * (Ct.real * v[0] - Ct.imag * v[1]), rtol=1e-11, atol=1e-12)


# A purely imaginary A (no decay), constant step, B = C = 1 and a unit impulse: the output is 2 cos(omega delta k)
# delta, the impulse response of an undamped oscillator.
def test_undamped_oscillation_closed_form():
    L, om, dt = 64, 1.7, 0.05
    x = np.zeros((1, L, 1)); x[0, 0, 0] = 1.0
    ones = np.ones((1, L, 1), dtype=np.complex128)
    s = OC.scan_fwd(x, np.full((1, L, 1), dt), np.array([[1j * om]]), ones, ones)
    np.testing.assert_allclose(s[0, :, 0], 2.0 * dt * np.cos(om * dt * np.arange(L)), rtol=1e-12, atol=1e-13)


def test_causality_and_channel_independence():
    p = _problem(2, 24, 4, 3)
    out = _fwd(p)
    q = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in p.items()}
    q["x"][:, 15:] += 1.0
    q["B"][:, 15:] *= 2.0
    np.testing.assert_array_equal(_fwd(q)[:, :15], out[:, :15])      # the past does not see the future
    q = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in p.items()}
    q["x"][:, :, 2] = 0.0
    q["A"][2] *= 1.5
    got = _fwd(q)
    np.testing.assert_array_equal(np.delete(got, 2, axis=2), np.delete(out, 2, axis=2))


def test_split_in_two_pieces_with_carried_state():
    p = _problem(2, 50, 3, 4)
    cut = 21
    out, hL = _fwd(p, return_h_last=True)
    sl = lambda a, b: dict(x=p["x"][:, a:b], delta=p["delta"][:, a:b], z=p["z"][:, a:b], B=p["B"][:, a:b],
                           C=p["C"][:, a:b], A=p["A"], D_skip=p["D_skip"])
    o1, h1 = _fwd(sl(0, cut), return_h_last=True)
    o2, h2 = _fwd(sl(cut, 50), h0=h1, return_h_last=True)
    np.testing.assert_array_equal(np.concatenate([o1, o2], axis=1), out)
    np.testing.assert_array_equal(h2, hL)
    # backward in two pieces: the adjoint leaving the second piece enters the first
    dout = RNG.standard_normal(out.shape)
    ref = OC.scan_bwd(p["x"], p["delta"], p["A"], p["B"], p["C"], p["D_skip"], p["z"], dout)
    q1, q2 = sl(0, cut), sl(cut, 50)
    g2 = OC.scan_bwd(q2["x"], q2["delta"], q2["A"], q2["B"], q2["C"], q2["D_skip"], q2["z"], dout[:, cut:], h0=h1)
    g1 = OC.scan_bwd(q1["x"], q1["delta"], q1["A"], q1["B"], q1["C"], q1["D_skip"], q1["z"], dout[:, :cut],
                     dh_last=g2["dh0"])
    for k in ("dx", "ddelta", "dz", "dB", "dC"):
        np.testing.assert_allclose(np.concatenate([g1[k], g2[k]], axis=1), ref[k], rtol=1e-11, atol=1e-12, err_msg=k)
    for k in ("dA", "dD"):
        np.testing.assert_allclose(g1[k] + g2[k], ref[k], rtol=1e-11, atol=1e-12, err_msg=k)


# Gradients against central finite differences of loss = sum(dout * out) in fp64; for a complex input the real and the
# imaginary part are perturbed separately and compared with the real and imaginary part of the returned gradient.
@pytest.mark.parametrize("gate,skip", [(True, True), (False, False)])
def test_gradients_match_finite_differences(gate, skip):
    batch, L, D, N = 2, 10, 3, 3
    p = _problem(batch, L, D, N)
    if not gate:
        p["z"] = None
    if not skip:
        p["D_skip"] = None
    h0 = RNG.standard_normal((batch, D, N)) + 1j * RNG.standard_normal((batch, D, N))
    dhl = RNG.standard_normal((batch, D, N)) + 1j * RNG.standard_normal((batch, D, N))
    dout = RNG.standard_normal((batch, L, D))

    def loss(q, h0q):
        out, hL = OC.scan_fwd(q["x"], q["delta"], q["A"], q["B"], q["C"], D_skip=q["D_skip"], z=q["z"], h0=h0q,
                              return_h_last=True)
        # dh_last is the gradient of a term Re(sum conj(dhl) h_L) = sum (dhl_re h_re + dhl_im h_im) added to the loss
        return float((dout * out).sum() + np.real(np.conj(dhl) * hL).sum())

    g = OC.scan_bwd(p["x"], p["delta"], p["A"], p["B"], p["C"], p["D_skip"], p["z"], dout, h0=h0, dh_last=dhl)
    names = {"x": "dx", "delta": "ddelta", "z": "dz", "A": "dA", "B": "dB", "C": "dC", "D_skip": "dD"}
    eps = 1e-6
    rng = np.random.default_rng(5)
    for key, gname in names.items():
        if p[key] is None:
            continue
        for _ in range(6):
            idx = tuple(int(rng.integers(0, n)) for n in p[key].shape)
            for part in ((1.0, 1j) if np.iscomplexobj(p[key]) else (1.0,)):
                hi = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in p.items()}
                lo = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in p.items()}
                hi[key][idx] += eps * part
                lo[key][idx] -= eps * part
                fd = (loss(hi, h0) - loss(lo, h0)) / (2 * eps)
                an = g[gname][idx]
                an = an.real if part == 1.0 else an.imag
                assert abs(fd - an) <= 2e-6 * max(1.0, abs(an)), (key, idx, part, fd, an)
    for _ in range(6):
        idx = tuple(int(rng.integers(0, n)) for n in h0.shape)
        for part in (1.0, 1j):
            hi, lo = h0.copy(), h0.copy()
            hi[idx] += eps * part
            lo[idx] -= eps * part
            fd = (loss(p, hi) - loss(p, lo)) / (2 * eps)
            an = g["dh0"][idx].real if part == 1.0 else g["dh0"][idx].imag
            assert abs(fd - an) <= 2e-6 * max(1.0, abs(an)), ("h0", idx, part, fd, an)
