"""Pins of the fp64 CPU oracle against what the paper and the mathematics fix (no GPU, no CUDA code).

Each pin is a result obtained by a route other than the oracle's own time loop: a closed form, a library routine,
a brute-force matrix, a finite difference, or an invariant.  A dropped term, a wrong sign or index, or a transposed
operand in the oracle fails at least one of them.
"""
import numpy as np
import pytest

from oracle import ssm_oracle as O

RNG = np.random.default_rng(20231201)


def _rand_problem(batch, L, D, N, rng=RNG, dt_scale=0.3):
    x = rng.standard_normal((batch, L, D))
    z = rng.standard_normal((batch, L, D))
    delta = dt_scale * rng.uniform(0.05, 1.0, (batch, L, D))
    B = rng.standard_normal((batch, L, N))
    C = rng.standard_normal((batch, L, N))
    A = -rng.uniform(0.2, 3.0, (D, N))
    Dk = rng.standard_normal(D)
    return dict(x=x, delta=delta, A=A, B=B, C=C, D_skip=Dk, z=z)


def _silu(z):
    return z / (1.0 + np.exp(-z))


# --------------------------------------------------------------------------------------------------------------
# P1  LTI closed form: with delta, B, C constant in time the recurrence equals a causal convolution with
#     kernel K_k = sum_n C_n * Abar_n^k * Bbar_n  (Eq. 3a / 3b).
def test_lti_equals_convolution():
    batch, L, D, N = 2, 96, 5, 4
    p = _rand_problem(batch, L, D, N)
    dt_d = RNG.uniform(0.01, 0.5, D)
    Bn, Cn = RNG.standard_normal(N), RNG.standard_normal(N)
    p["delta"] = np.broadcast_to(dt_d, (batch, L, D)).copy()
    p["B"] = np.broadcast_to(Bn, (batch, L, N)).copy()
    p["C"] = np.broadcast_to(Cn, (batch, L, N)).copy()
    s = O.scan_fwd(p["x"], p["delta"], p["A"], p["B"], p["C"], D_skip=p["D_skip"], z=None)
    k = np.arange(L)
    for b in range(batch):
        for d in range(D):
            Abar = np.exp(dt_d[d] * p["A"][d])                       # (N,)
            K = ((Cn * dt_d[d] * Bn)[None, :] * Abar[None, :] ** k[:, None]).sum(-1)
            ref = np.convolve(p["x"][b, :, d], K)[:L] + p["D_skip"][d] * p["x"][b, :, d]
            np.testing.assert_allclose(s[b, :, d], ref, rtol=1e-12, atol=1e-13)


# --------------------------------------------------------------------------------------------------------------
# P2  Brute-force lower-triangular matrix form on tiny inputs:
#     M[t,s] = sum_n C[t,n] * exp(A_n * sum_{r=s+1..t} delta_r) * delta_s * B[s,n],  s <= t.
@pytest.mark.parametrize("L,N", [(1, 1), (7, 3), (16, 4)])
def test_matrix_form(L, N):
    batch, D = 2, 3
    p = _rand_problem(batch, L, D, N)
    s = O.scan_fwd(p["x"], p["delta"], p["A"], p["B"], p["C"], D_skip=p["D_skip"], z=None)
    out = O.scan_fwd(p["x"], p["delta"], p["A"], p["B"], p["C"], D_skip=p["D_skip"], z=p["z"])
    for b in range(batch):
        for d in range(D):
            M = np.zeros((L, L))
            for t in range(L):
                for si in range(t + 1):
                    dsum = p["delta"][b, si + 1:t + 1, d].sum()
                    M[t, si] = (p["C"][b, t] * np.exp(p["A"][d] * dsum) * p["delta"][b, si, d] * p["B"][b, si]).sum()
            ref = M @ p["x"][b, :, d] + p["D_skip"][d] * p["x"][b, :, d]
            np.testing.assert_allclose(s[b, :, d], ref, rtol=1e-12, atol=1e-13)
            np.testing.assert_allclose(out[b, :, d], ref * _silu(p["z"][b, :, d]), rtol=1e-12, atol=1e-13)


# --------------------------------------------------------------------------------------------------------------
# Gate (Section 3.4, Figure 3: the SiLU branch multiplies the SSM output): the gated output equals the pre-gate readout
# times z * sigmoid(z), with the sigmoid taken from a library (scipy's expit) rather than retyped; and, for the
# backward pass, dz equals dout * s * d/dz [z expit(z)], the derivative written with the library function alone
# (expit'(z) = expit(z) expit(-z)).
def test_gate_is_library_silu():
    from scipy.special import expit
    p = _rand_problem(2, 40, 6, 4)
    p["z"] = p["z"] * 4.0     # reach both saturated ends of the sigmoid
    out, s_pre = O.scan_fwd(p["x"], p["delta"], p["A"], p["B"], p["C"], D_skip=p["D_skip"], z=p["z"], return_pregate=True)
    ungated = O.scan_fwd(p["x"], p["delta"], p["A"], p["B"], p["C"], D_skip=p["D_skip"], z=None)
    np.testing.assert_allclose(s_pre, ungated, rtol=0, atol=0)
    np.testing.assert_allclose(out, s_pre * p["z"] * expit(p["z"]), rtol=1e-14, atol=1e-15)
    dout = RNG.standard_normal(out.shape)
    g = O.scan_bwd(p["x"], p["delta"], p["A"], p["B"], p["C"], p["D_skip"], p["z"], dout)
    sig = expit(p["z"])
    dsilu = sig + p["z"] * sig * expit(-p["z"])     # d/dz [z expit(z)], expit'(z) = expit(z) expit(-z)
    np.testing.assert_allclose(g["dz"], dout * s_pre * dsilu, rtol=1e-12, atol=1e-13)


# --------------------------------------------------------------------------------------------------------------
# P3  A = 0 makes Abar = 1, so the state is a plain running sum: h_t = cumsum(delta * B * x).
def test_zero_A_is_cumsum():
    batch, L, D, N = 2, 50, 4, 3
    p = _rand_problem(batch, L, D, N)
    p["A"] = np.zeros((D, N))
    s = O.scan_fwd(p["x"], p["delta"], p["A"], p["B"], p["C"], z=None)
    h = np.cumsum((p["delta"] * p["x"])[..., None] * p["B"][:, :, None, :], axis=1)     # (b, L, D, N)
    ref = (h * p["C"][:, :, None, :]).sum(-1)
    np.testing.assert_allclose(s, ref, rtol=1e-13, atol=1e-14)


# --------------------------------------------------------------------------------------------------------------
# P4  Theorem 1: N = 1, A = -1, B = 1, delta = softplus(v)  =>  Abar = 1 - sigmoid(v) and, under zero-order hold,
#     Bbar = sigmoid(v), i.e. the gated recurrence h_t = (1 - g_t) h_{t-1} + g_t x_t with g = sigmoid(v).
def test_gating_theorem():
    batch, L, D = 2, 40, 3
    v = RNG.standard_normal((batch, L, D)) * 2.0
    x = RNG.standard_normal((batch, L, D))
    delta = np.log1p(np.exp(v))
    A = -np.ones((D, 1))
    ones = np.ones((batch, L, 1))
    g = 1.0 / (1.0 + np.exp(-v))
    # zero-order hold: the gated RNN itself
    h = np.zeros((batch, D))
    ref = np.empty((batch, L, D))
    for t in range(L):
        h = (1.0 - g[:, t]) * h + g[:, t] * x[:, t]
        ref[:, t] = h
    got = O.scan_fwd(x, delta, A, ones, ones, zoh=True)
    np.testing.assert_allclose(got, ref, rtol=1e-13, atol=1e-14)
    # default rule Bbar = delta * B: same decay 1 - g, input weight delta
    h = np.zeros((batch, D))
    for t in range(L):
        h = (1.0 - g[:, t]) * h + delta[:, t] * x[:, t]
        ref[:, t] = h
    got = O.scan_fwd(x, delta, A, ones, ones)
    np.testing.assert_allclose(got, ref, rtol=1e-13, atol=1e-14)


def test_zoh_tends_to_default_rule_for_small_steps():
    # Bbar_zoh = delta*B*(1 + delta*A/2 + ...): the two rules agree to first order in delta*A.
    p = _rand_problem(1, 30, 2, 3, dt_scale=1e-6)
    a = O.scan_fwd(p["x"], p["delta"], p["A"], p["B"], p["C"], zoh=True)
    b = O.scan_fwd(p["x"], p["delta"], p["A"], p["B"], p["C"], zoh=False)
    assert 0 < np.abs(a - b).max() <= 1e-5 * np.abs(b).max()


# --------------------------------------------------------------------------------------------------------------
# P5  Gradients against central finite differences of loss = sum(dout * out), in fp64.
def _loss(p, dout):
    return float((dout * O.scan_fwd(p["x"], p["delta"], p["A"], p["B"], p["C"], D_skip=p["D_skip"], z=p["z"])).sum())


@pytest.mark.parametrize("gate,skip", [(True, True), (False, True), (True, False)])
def test_gradients_match_finite_differences(gate, skip):
    batch, L, D, N = 2, 12, 3, 4
    p = _rand_problem(batch, L, D, N)
    if not gate:
        p["z"] = None
    if not skip:
        p["D_skip"] = None
    dout = RNG.standard_normal((batch, L, D))
    g = O.scan_bwd(p["x"], p["delta"], p["A"], p["B"], p["C"], p["D_skip"], p["z"], dout)
    names = {"x": "dx", "delta": "ddelta", "A": "dA", "B": "dB", "C": "dC", "D_skip": "dD", "z": "dz"}
    eps = 1e-6
    for key, gname in names.items():
        if p[key] is None:
            assert np.all(g[gname] == 0.0)
            continue
        # a random direction: checks the whole gradient tensor at once
        for trial in range(3):
            v = RNG.standard_normal(p[key].shape)
            pp, pm = dict(p), dict(p)
            pp[key] = p[key] + eps * v
            pm[key] = p[key] - eps * v
            fd = (_loss(pp, dout) - _loss(pm, dout)) / (2 * eps)
            an = float((g[gname] * v).sum())
            assert abs(fd - an) <= 1e-6 * max(1.0, abs(an)), (key, fd, an)
        # and single entries, which a direction check could average away
        flat = p[key].reshape(-1)
        for idx in RNG.choice(flat.size, size=min(6, flat.size), replace=False):
            e = np.zeros(flat.size)
            e[idx] = eps
            pp, pm = dict(p), dict(p)
            pp[key] = p[key] + e.reshape(p[key].shape)
            pm[key] = p[key] - e.reshape(p[key].shape)
            fd = (_loss(pp, dout) - _loss(pm, dout)) / (2 * eps)
            an = float(g[gname].reshape(-1)[idx])
            assert abs(fd - an) <= 2e-6 * max(1.0, abs(an)), (key, idx, fd, an)


# --------------------------------------------------------------------------------------------------------------
# P6  Invariants.
def test_causality_bitwise():
    p = _rand_problem(1, 32, 3, 4)
    a = O.scan_fwd(**p)
    q = {k: (v.copy() if v is not None else None) for k, v in p.items()}
    t0 = 20
    for k in ("x", "delta", "B", "C", "z"):
        q[k][:, t0:] = RNG.standard_normal(q[k][:, t0:].shape) if k != "delta" else RNG.uniform(0.01, 0.3, q[k][:, t0:].shape)
    b = O.scan_fwd(**q)
    assert np.array_equal(a[:, :t0], b[:, :t0])
    assert not np.array_equal(a[:, t0:], b[:, t0:])


def test_linearity_in_x_and_zero_cases():
    p = _rand_problem(2, 24, 3, 4)
    p["z"] = None
    x2 = RNG.standard_normal(p["x"].shape)
    f = lambda xx: O.scan_fwd(xx, p["delta"], p["A"], p["B"], p["C"], D_skip=p["D_skip"])
    np.testing.assert_allclose(f(2.5 * p["x"] - 0.75 * x2), 2.5 * f(p["x"]) - 0.75 * f(x2), rtol=1e-12, atol=1e-12)
    assert np.all(f(np.zeros_like(x2)) == 0.0)
    zg = np.zeros_like(x2)
    assert np.all(O.scan_fwd(p["x"], p["delta"], p["A"], p["B"], p["C"], D_skip=p["D_skip"], z=zg) == 0.0)


def test_channel_and_batch_independence():
    p = _rand_problem(3, 20, 5, 4)
    full = O.scan_fwd(**p)
    perm = RNG.permutation(5)
    q = dict(p)
    for k in ("x", "delta", "z"):
        q[k] = p[k][:, :, perm]
    q["A"], q["D_skip"] = p["A"][perm], p["D_skip"][perm]
    assert np.array_equal(O.scan_fwd(**q), full[:, :, perm])
    one = O.scan_fwd(p["x"][1:2], p["delta"][1:2], p["A"], p["B"][1:2], p["C"][1:2], D_skip=p["D_skip"], z=p["z"][1:2])
    assert np.array_equal(one[0], full[1])


def test_step_size_limits():
    # Section 3.5.2: a large step resets the state and keeps only the current input; a zero step ignores the
    # input and carries the state over unchanged.
    p = _rand_problem(1, 10, 2, 3)
    p["z"] = None
    big = dict(p)
    big["delta"] = np.full_like(p["delta"], 60.0)
    s = O.scan_fwd(**big)
    ref = (big["delta"] * p["x"]) * (p["C"] * p["B"]).sum(-1)[:, :, None] + p["D_skip"] * p["x"]
    np.testing.assert_allclose(s, ref, rtol=1e-13)
    # zero step at t >= 5: state frozen, readout moves only through C_t and the skip term
    q = dict(p)
    q["delta"] = p["delta"].copy()
    q["delta"][:, 5:] = 0.0
    s, hl = O.scan_fwd(**q, return_h_last=True)
    _, h5 = O.scan_fwd(q["x"][:, :5], q["delta"][:, :5], q["A"], q["B"][:, :5], q["C"][:, :5], D_skip=q["D_skip"],
                       return_h_last=True)
    assert np.array_equal(hl, h5)
    ref = np.einsum("btn,bdn->btd", q["C"][:, 5:], h5) + q["D_skip"] * q["x"][:, 5:]
    np.testing.assert_allclose(s[:, 5:], ref, rtol=1e-13, atol=1e-14)


# --------------------------------------------------------------------------------------------------------------
# P7  Chunk split: scanning [1..m] and then [m+1..L] from the carried state equals scanning [1..L] (bitwise).
@pytest.mark.parametrize("m", [1, 13, 31])
def test_chunk_split_bitwise(m):
    p = _rand_problem(2, 32, 3, 4)
    full, hL = O.scan_fwd(**p, return_h_last=True)
    sl = lambda k, a, b: None if p[k] is None else p[k][:, a:b]
    o1, h1 = O.scan_fwd(sl("x", 0, m), sl("delta", 0, m), p["A"], sl("B", 0, m), sl("C", 0, m), D_skip=p["D_skip"],
                        z=sl("z", 0, m), return_h_last=True)
    o2, h2 = O.scan_fwd(sl("x", m, 32), sl("delta", m, 32), p["A"], sl("B", m, 32), sl("C", m, 32),
                        D_skip=p["D_skip"], z=sl("z", m, 32), h0=h1, return_h_last=True)
    assert np.array_equal(np.concatenate([o1, o2], axis=1), full)
    assert np.array_equal(h2, hL)


# --------------------------------------------------------------------------------------------------------------
# P8  The associative operator (a, b) o (a', b') = (a a', a' b + b'): folding the per-step pairs in any
#     bracketing reproduces the state.  The state is read through one-hot C rows, which also pins the n index
#     of the readout.
def _combine(p, q):
    return (p[0] * q[0], q[0] * p[1] + q[1])


def _fold_tree(pairs):
    if len(pairs) == 1:
        return pairs[0]
    cut = int(RNG.integers(1, len(pairs)))
    return _combine(_fold_tree(pairs[:cut]), _fold_tree(pairs[cut:]))


def test_operator_fold_reproduces_state():
    L, D, N = 23, 2, 3
    p = _rand_problem(1, L, D, N)
    for n in range(N):
        C1 = np.zeros((1, L, N))
        C1[:, :, n] = 1.0
        h_n = O.scan_fwd(p["x"], p["delta"], p["A"], p["B"], C1)         # (1, L, D): h[t, d, n]
        for d in range(D):
            pairs = [(np.exp(p["delta"][0, t, d] * p["A"][d, n]), p["delta"][0, t, d] * p["B"][0, t, n] * p["x"][0, t, d])
                     for t in range(L)]
            for t in (0, 5, L - 1):
                _, b = _fold_tree(pairs[:t + 1])
                np.testing.assert_allclose(h_n[0, t, d], b, rtol=1e-12, atol=1e-14)


# --------------------------------------------------------------------------------------------------------------
# storage variants and threading
def test_f32_storage_matches_f64_and_threads_do_not_matter():
    p = _rand_problem(2, 40, 70, 4)        # 70 channels: two channel blocks in the backward reduction
    p32 = {k: v.astype(np.float32) for k, v in p.items()}
    p64 = {k: v.astype(np.float64) for k, v in p32.items()}
    dout = RNG.standard_normal(p["x"].shape).astype(np.float32)
    assert np.array_equal(O.scan_fwd(**p32), O.scan_fwd(**p64))
    g1 = O.scan_bwd(p32["x"], p32["delta"], p32["A"], p32["B"], p32["C"], p32["D_skip"], p32["z"], dout, nthreads=1)
    g8 = O.scan_bwd(p64["x"], p64["delta"], p64["A"], p64["B"], p64["C"], p64["D_skip"], p64["z"],
                    dout.astype(np.float64), nthreads=8)
    for k in g1:
        assert np.array_equal(g1[k], g8[k]), k


# --------------------------------------------------------------------------------------------------------------
# Step size through the softplus (Algorithm 2 step 4: Delta = softplus(Parameter + s_Delta(x))).
def test_softplus_switch_equals_precomputed_step_and_gating_theorem():
    batch, L, D, N = 2, 30, 4, 3
    p = _rand_problem(batch, L, D, N)
    v = RNG.standard_normal((batch, L, D)) * 3.0 - 2.0
    bias = RNG.standard_normal(D)
    step = np.logaddexp(0.0, v + bias)                          # library softplus, another route than the oracle's
    a = O.scan_fwd(p["x"], v, p["A"], p["B"], p["C"], D_skip=p["D_skip"], z=p["z"], delta_softplus=True, delta_bias=bias)
    b = O.scan_fwd(p["x"], step, p["A"], p["B"], p["C"], D_skip=p["D_skip"], z=p["z"])
    np.testing.assert_allclose(a, b, rtol=1e-13, atol=1e-14)
    # Theorem 1 stated on the pre-activation: N = 1, A = -1, B = C = 1, zero-order hold  =>  gate g = sigmoid(v)
    x = RNG.standard_normal((batch, L, D))
    ones = np.ones((batch, L, 1))
    g = 1.0 / (1.0 + np.exp(-v))
    h = np.zeros((batch, D))
    ref = np.empty((batch, L, D))
    for t in range(L):
        h = (1.0 - g[:, t]) * h + g[:, t] * x[:, t]
        ref[:, t] = h
    got = O.scan_fwd(x, v, -np.ones((D, 1)), ones, ones, zoh=True, delta_softplus=True)
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-13)


def test_softplus_gradients_match_finite_differences():
    batch, L, D, N = 2, 10, 3, 4
    p = _rand_problem(batch, L, D, N)
    v = RNG.standard_normal((batch, L, D)) * 2.0 - 1.0
    bias = RNG.standard_normal(D)
    dout = RNG.standard_normal((batch, L, D))
    g = O.scan_bwd(p["x"], v, p["A"], p["B"], p["C"], p["D_skip"], p["z"], dout, delta_softplus=True, delta_bias=bias)

    def loss(vv, bb):
        return float((dout * O.scan_fwd(p["x"], vv, p["A"], p["B"], p["C"], D_skip=p["D_skip"], z=p["z"],
                                        delta_softplus=True, delta_bias=bb)).sum())
    eps = 1e-6
    for trial in range(3):
        dv, db = RNG.standard_normal(v.shape), RNG.standard_normal(D)
        fd_v = (loss(v + eps * dv, bias) - loss(v - eps * dv, bias)) / (2 * eps)
        fd_b = (loss(v, bias + eps * db) - loss(v, bias - eps * db)) / (2 * eps)
        assert abs(fd_v - (g["ddelta"] * dv).sum()) <= 1e-6 * max(1.0, abs(fd_v))
        assert abs(fd_b - (g["ddelta_bias"] * db).sum()) <= 1e-6 * max(1.0, abs(fd_b))
    # the other gradients equal those of the unfused problem with the precomputed step size
    step = np.logaddexp(0.0, v + bias)
    g0 = O.scan_bwd(p["x"], step, p["A"], p["B"], p["C"], p["D_skip"], p["z"], dout)
    for k in ("dx", "dz", "dA", "dB", "dC", "dD"):
        np.testing.assert_allclose(g[k], g0[k], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(g["ddelta"], g0["ddelta"] / (1.0 + np.exp(-(v + bias))), rtol=1e-11, atol=1e-12)


# --------------------------------------------------------------------------------------------------------------
# Zero-order-hold B-bar (Eq. 4) -- forward against a library matrix exponential, backward against finite differences.
def test_zoh_is_the_exact_solution_for_held_inputs():
    # Eq. 1a with the input held constant over a step of length delta: [h; 1](t + delta) = expm(delta * M) [h; 1](t),
    # M = [[diag(A), B x], [0, 0]].  The library matrix exponential knows nothing of the closed form (e^{dA} - 1) / A.
    from scipy.linalg import expm
    L, N = 9, 3
    p = _rand_problem(1, L, 1, N)
    p["A"][0, 1] = 0.0                      # the removable singularity of (e^{dA} - 1) / A
    got, s_pre = O.scan_fwd(p["x"], p["delta"], p["A"], p["B"], p["C"], zoh=True, return_pregate=True)
    h = np.zeros(N)
    for t in range(L):
        M = np.zeros((N + 1, N + 1))
        M[:N, :N] = np.diag(p["A"][0])
        M[:N, N] = p["B"][0, t] * p["x"][0, t, 0]
        h = (expm(p["delta"][0, t, 0] * M) @ np.append(h, 1.0))[:N]
        assert abs(s_pre[0, t, 0] - p["C"][0, t] @ h) <= 1e-12 * max(1.0, abs(s_pre[0, t, 0]))


@pytest.mark.parametrize("small_steps", [False, True])
def test_zoh_gradients_match_finite_differences(small_steps):
    batch, L, D, N = 2, 10, 3, 4
    p = _rand_problem(batch, L, D, N, dt_scale=2e-3 if small_steps else 0.5)   # both branches of dE/dA
    p["A"][1, 2] = 0.0
    dout = RNG.standard_normal((batch, L, D))
    g = O.scan_bwd(p["x"], p["delta"], p["A"], p["B"], p["C"], p["D_skip"], p["z"], dout, zoh=True)

    def loss(q):
        return float((dout * O.scan_fwd(q["x"], q["delta"], q["A"], q["B"], q["C"], D_skip=q["D_skip"], z=q["z"],
                                        zoh=True)).sum())
    names = {"x": "dx", "delta": "ddelta", "A": "dA", "B": "dB", "C": "dC", "D_skip": "dD", "z": "dz"}
    for key, gname in names.items():
        eps = 1e-6 * max(1.0, float(np.abs(p[key]).max())) if key != "delta" else 1e-6 * float(p["delta"].mean())
        for trial in range(3):
            v = RNG.standard_normal(p[key].shape)
            pp, pm = dict(p), dict(p)
            pp[key] = p[key] + eps * v
            pm[key] = p[key] - eps * v
            fd = (loss(pp) - loss(pm)) / (2 * eps)
            an = float((g[gname] * v).sum())
            assert abs(fd - an) <= 2e-6 * max(1.0, abs(an)), (key, fd, an)
    # the entry with A = 0 on its own (the limit delta^2 / 2 of dE/dA)
    e = np.zeros_like(p["A"])
    e[1, 2] = 1e-6
    pp, pm = dict(p), dict(p)
    pp["A"], pm["A"] = p["A"] + e, p["A"] - e
    fd = (loss(pp) - loss(pm)) / 2e-6
    assert abs(fd - g["dA"][1, 2]) <= 2e-6 * max(1.0, abs(fd))


# --------------------------------------------------------------------------------------------------------------
# Backward with a carried-in state and an adjoint arriving at the last state.
def test_backward_in_two_pieces_equals_one_backward():
    # The gradient of a sequence equals the gradients of its two pieces when the second piece starts from the first
    # piece's last state and hands the first piece the gradient of that state (chain rule across the cut).
    batch, L, D, N, m = 2, 23, 3, 4, 9
    p = _rand_problem(batch, L, D, N)
    dout = RNG.standard_normal((batch, L, D))
    whole = O.scan_bwd(p["x"], p["delta"], p["A"], p["B"], p["C"], p["D_skip"], p["z"], dout)
    cut = lambda a, lo, hi: a[:, lo:hi]
    first = {k: cut(p[k], 0, m) for k in ("x", "delta", "B", "C", "z")}
    second = {k: cut(p[k], m, L) for k in ("x", "delta", "B", "C", "z")}
    _, h_m = O.scan_fwd(first["x"], first["delta"], p["A"], first["B"], first["C"], D_skip=p["D_skip"], z=first["z"],
                        return_h_last=True)
    g2 = O.scan_bwd(second["x"], second["delta"], p["A"], second["B"], second["C"], p["D_skip"], second["z"],
                    dout[:, m:], h0=h_m)
    g1 = O.scan_bwd(first["x"], first["delta"], p["A"], first["B"], first["C"], p["D_skip"], first["z"],
                    dout[:, :m], dh_last=g2["dh0"])
    for k in ("dx", "ddelta", "dz", "dB", "dC"):
        np.testing.assert_allclose(np.concatenate([g1[k], g2[k]], axis=1), whole[k], rtol=1e-11, atol=1e-12)
    for k in ("dA", "dD"):
        np.testing.assert_allclose(g1[k] + g2[k], whole[k], rtol=1e-11, atol=1e-12)
    assert np.all(whole["dh0"] == g1["dh0"]) or np.allclose(whole["dh0"], g1["dh0"], rtol=1e-11, atol=1e-13)


def test_initial_state_gradient_matches_finite_differences():
    batch, L, D, N = 2, 8, 3, 4
    p = _rand_problem(batch, L, D, N)
    h0 = RNG.standard_normal((batch, D, N))
    dhl = RNG.standard_normal((batch, D, N))
    dout = RNG.standard_normal((batch, L, D))

    def loss(hh, xx=None):
        out, hl = O.scan_fwd(p["x"] if xx is None else xx, p["delta"], p["A"], p["B"], p["C"], D_skip=p["D_skip"],
                             z=p["z"], h0=hh, return_h_last=True)
        return float((dout * out).sum() + (dhl * hl).sum())
    g = O.scan_bwd(p["x"], p["delta"], p["A"], p["B"], p["C"], p["D_skip"], p["z"], dout, h0=h0, dh_last=dhl)
    eps = 1e-6
    for trial in range(3):
        v = RNG.standard_normal(h0.shape)
        fd = (loss(h0 + eps * v) - loss(h0 - eps * v)) / (2 * eps)
        assert abs(fd - (g["dh0"] * v).sum()) <= 1e-6 * max(1.0, abs(fd))
        vx = RNG.standard_normal(p["x"].shape)       # dh_last must reach the other gradients too
        fd = (loss(h0, p["x"] + eps * vx) - loss(h0, p["x"] - eps * vx)) / (2 * eps)
        assert abs(fd - (g["dx"] * vx).sum()) <= 1e-6 * max(1.0, abs(fd))


# --------------------------------------------------------------------------------------------------------------
# Regression anchor: the stored outputs of the oracle on a tiny seeded problem (tests/golden/, written by a committed
# script that calls only the oracle; the paper prints no worked example to store instead).
def test_oracle_reproduces_its_stored_tiny_problem():
    import importlib.util
    import os
    here = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(here, "make_golden.py"))
    mg = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mg)
    now = mg.compute()
    seen = set()
    for line in open(os.path.join(here, "scan_tiny.txt")):
        if line.startswith("#"):
            continue
        name, shape, *vals = line.split()
        ref = np.array([float(v) for v in vals]).reshape([int(s) for s in shape.split("x")])
        np.testing.assert_allclose(now[name], ref, rtol=1e-13, atol=1e-15, err_msg=name)
        seen.add(name)
    assert seen == set(now)
