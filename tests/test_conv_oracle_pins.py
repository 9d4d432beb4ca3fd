"""Pins of the fp64 oracle of the short causal depthwise convolution (no GPU): a library convolution per channel,
special cases, causality, piecewise processing and finite differences."""
import numpy as np
import pytest

from oracle import conv_oracle as CO

RNG = np.random.default_rng(7)


def _case(batch=2, L=19, D=5, W=4):
    return (RNG.standard_normal((batch, L, D)), RNG.standard_normal((D, W)), RNG.standard_normal(D),
            RNG.standard_normal((batch, L, D)))


@pytest.mark.parametrize("W", [1, 2, 3, 4])
def test_equals_library_convolution_per_channel(W):
    x, w, bias, _ = _case(W=W)
    got = CO.conv1d_fwd(x, w, bias, silu=False)
    for b in range(x.shape[0]):
        for d in range(x.shape[2]):
            # numpy.convolve flips its second argument: tap k multiplies x[t - (W-1) + k]  <=>  kernel w[::-1]
            ref = np.convolve(x[b, :, d], w[d, ::-1])[: x.shape[1]] + bias[d]
            np.testing.assert_allclose(got[b, :, d], ref, rtol=1e-13, atol=1e-13)


def test_special_cases_and_activation():
    x, w, bias, _ = _case(W=4)
    # a kernel with only its last tap is a per-channel scale of the current step
    w1 = np.zeros_like(w)
    w1[:, -1] = w[:, -1]
    np.testing.assert_allclose(CO.conv1d_fwd(x, w1, None, silu=False), x * w[:, -1], rtol=1e-15)
    # only the first tap: a delay by W-1 steps
    w0 = np.zeros_like(w)
    w0[:, 0] = 1.0
    got = CO.conv1d_fwd(x, w0, None, silu=False)
    assert np.all(got[:, :3] == 0) and np.array_equal(got[:, 3:], x[:, :-3])
    # activation
    pre = CO.conv1d_fwd(x, w, bias, silu=False)
    np.testing.assert_allclose(CO.conv1d_fwd(x, w, bias), pre / (1 + np.exp(-pre)), rtol=1e-15)


def test_causality_and_piecewise_processing():
    x, w, bias, _ = _case(L=30)
    y = CO.conv1d_fwd(x, w, bias)
    x2 = x.copy()
    x2[:, 17:] += 1.0
    assert np.array_equal(CO.conv1d_fwd(x2, w, bias)[:, :17], y[:, :17])
    # two pieces with the last W-1 inputs of the first piece carried over equal the whole sequence
    m = 11
    y1 = CO.conv1d_fwd(x[:, :m], w, bias)
    y2 = CO.conv1d_fwd(x[:, m:], w, bias, x_prev=x[:, m - 3:m])
    assert np.array_equal(np.concatenate([y1, y2], axis=1), y)


@pytest.mark.parametrize("silu,W", [(True, 4), (False, 3), (True, 2)])
def test_gradients_match_finite_differences(silu, W):
    x, w, bias, dy = _case(W=W)
    xprev = RNG.standard_normal((x.shape[0], W - 1, x.shape[2]))
    g = CO.conv1d_bwd(x, w, bias, dy, silu=silu, x_prev=xprev)
    loss = lambda xx, ww, bb, pp: float((dy * CO.conv1d_fwd(xx, ww, bb, silu=silu, x_prev=pp)).sum())
    eps = 1e-6
    for trial in range(3):
        vx, vw, vb, vp = (RNG.standard_normal(a.shape) for a in (x, w, bias, xprev))
        for args_p, args_m, an in [
            ((x + eps * vx, w, bias, xprev), (x - eps * vx, w, bias, xprev), (g["dx"] * vx).sum()),
            ((x, w + eps * vw, bias, xprev), (x, w - eps * vw, bias, xprev), (g["dw"] * vw).sum()),
            ((x, w, bias + eps * vb, xprev), (x, w, bias - eps * vb, xprev), (g["dbias"] * vb).sum()),
            ((x, w, bias, xprev + eps * vp), (x, w, bias, xprev - eps * vp), (g["dx_prev"] * vp).sum()),
        ]:
            fd = (loss(*args_p) - loss(*args_m)) / (2 * eps)
            assert abs(fd - an) <= 1e-6 * max(1.0, abs(an))
    # single entries of dw (a direction check could average an index error away)
    for d, k in [(0, 0), (2, W - 1), (4, W // 2)]:
        e = np.zeros_like(w)
        e[d, k] = eps
        fd = (loss(x, w + e, bias, xprev) - loss(x, w - e, bias, xprev)) / (2 * eps)
        assert abs(fd - g["dw"][d, k]) <= 1e-6 * max(1.0, abs(fd))
