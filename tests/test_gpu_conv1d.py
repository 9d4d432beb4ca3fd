"""Short causal depthwise convolution + SiLU on the GPU against its oracle, forward and backward."""
import numpy as np
import pytest

from paper_2312_00752_b200 import synth
from tests import _gpu_util as U

pytestmark = pytest.mark.gpu


def _case(batch, L, D, W, io, seed=0, prev=False):
    rng = np.random.default_rng(1000 + seed)
    r = lambda *s: synth.round_to_io(rng.standard_normal(s), io)
    x, dy = r(batch, L, D), r(batch, L, D)
    w = (rng.standard_normal((D, W)) / np.sqrt(W)).astype(np.float32)
    bias = (0.1 * rng.standard_normal(D)).astype(np.float32)
    xp = r(batch, W - 1, D) if prev and W > 1 else None
    return x, w, bias, dy, xp


@pytest.mark.parametrize("batch,L,D,W,io,silu,bias,prev", [
    (2, 200, 64, 4, "bf16", True, True, False),      # vector path, several chunks and a ragged one
    (2, 131, 40, 4, "bf16", True, True, True),       # carried context, D not a multiple of the thread block
    (1, 70, 24, 3, "f32", True, False, True),
    (3, 65, 20, 2, "f32", False, True, False),
    (2, 50, 7, 4, "bf16", True, True, True),         # scalar path (D % 4 != 0)
    (1, 3, 16, 4, "f32", True, True, False),         # sequence shorter than the kernel
    (2, 64, 32, 1, "bf16", True, True, False),       # one tap: per-channel scale, bias, activation
])
def test_conv1d_forward_backward(batch, L, D, W, io, silu, bias, prev):
    import torch
    from oracle import conv_oracle as CO
    from paper_2312_00752_b200 import binding as K
    x, w, b, dy, xp = _case(batch, L, D, W, io, prev=prev)
    if not bias:
        b = None
    dt = torch.bfloat16 if io == "bf16" else torch.float32
    tx, tdy = torch.from_numpy(x).cuda().to(dt), torch.from_numpy(dy).cuda().to(dt)
    txp = None if xp is None else torch.from_numpy(xp).cuda().to(dt)
    tw = torch.from_numpy(w).cuda()
    tb = None if b is None else torch.from_numpy(b).cuda()
    y = K.ssm_conv1d_fwd(tx, tw, tb, silu=silu, x_prev=txp)
    g = K.ssm_conv1d_bwd(tx, tw, tb, tdy, silu=silu, x_prev=txp, want_dx_prev=True)
    ref_y = CO.conv1d_fwd(x, w, b, silu=silu, x_prev=xp)
    ref = CO.conv1d_bwd(x, w, b, dy, silu=silu, x_prev=xp)
    tol = U.TOL[io]
    assert U.rel_err(U.to_host(y), ref_y) <= tol["out"]
    assert U.rel_err(U.to_host(g["dx"]), ref["dx"]) <= tol["grad"]
    assert U.rel_err(U.to_host(g["dw"]), ref["dw"]) <= tol["grad"]
    if b is not None:
        assert U.rel_err(U.to_host(g["dbias"]), ref["dbias"]) <= tol["grad"]
    if W > 1:
        assert U.rel_err(U.to_host(g["dx_prev"]), ref["dx_prev"]) <= tol["grad"]


def test_conv1d_layer_shape_sampled_and_deterministic():
    # the 2.8B layer shape: every output of a sample of channels against the oracle; two runs bit-identical
    import torch
    from oracle import conv_oracle as CO
    from paper_2312_00752_b200 import binding as K
    batch, L, D, W = 4, 2048, 5120, 4
    g = torch.Generator(device="cuda").manual_seed(3)
    x = torch.randn((batch, L, D), device="cuda", generator=g).to(torch.bfloat16)
    dy = torch.randn((batch, L, D), device="cuda", generator=g).to(torch.bfloat16)
    w = torch.randn((D, W), device="cuda", generator=g) * 0.5
    b = torch.randn((D,), device="cuda", generator=g) * 0.1
    y = K.ssm_conv1d_fwd(x, w, b)
    r1 = K.ssm_conv1d_bwd(x, w, b, dy)
    r2 = K.ssm_conv1d_bwd(x, w, b, dy)
    assert torch.equal(r1["dw"], r2["dw"]) and torch.equal(r1["dx"], r2["dx"]) and torch.equal(r1["dbias"], r2["dbias"])
    ch = np.array([0, 1, 7, 8, 511, 512, 2047, 4096, 5119])
    xs, dys = U.to_host(x[:, :, ch]), U.to_host(dy[:, :, ch])
    ws, bs = U.to_host(w[ch]), U.to_host(b[ch])
    ref_y = CO.conv1d_fwd(xs, ws, bs)
    ref = CO.conv1d_bwd(xs, ws, bs, dys)
    assert U.rel_err(U.to_host(y[:, :, ch]), ref_y) <= 1e-2
    assert U.rel_err(U.to_host(r1["dx"][:, :, ch]), ref["dx"]) <= 3e-2
    assert U.rel_err(U.to_host(r1["dw"][ch]), ref["dw"]) <= 3e-2
    assert U.rel_err(U.to_host(r1["dbias"][ch]), ref["dbias"]) <= 3e-2


def _draw_conv(rng):
    return dict(io=str(rng.choice(["bf16", "f32"])), W=int(rng.integers(1, 5)), D=int(rng.choice([4, 8, 20, 64, 260, 7, 33])),
                L=int(rng.choice([1, 2, 3, 5, 31, 32, 33, 64, 127, 129, 300])), batch=int(rng.integers(1, 4)),
                silu=bool(rng.integers(0, 2)), bias=bool(rng.integers(0, 2)), prev=bool(rng.integers(0, 2)))


CONV_CASES = [_draw_conv(np.random.default_rng([2312, 754, i])) for i in range(48)]


@pytest.mark.parametrize("c", CONV_CASES, ids=[f"{i}" for i in range(len(CONV_CASES))])
def test_conv1d_random_problem(c):
    import torch
    from oracle import conv_oracle as CO
    from paper_2312_00752_b200 import binding as K
    x, w, b, dy, xp = _case(c["batch"], c["L"], c["D"], c["W"], c["io"], seed=3, prev=c["prev"])
    if not c["bias"]:
        b = None
    dt = torch.bfloat16 if c["io"] == "bf16" else torch.float32
    tx, tdy = torch.from_numpy(x).cuda().to(dt), torch.from_numpy(dy).cuda().to(dt)
    txp = None if xp is None else torch.from_numpy(xp).cuda().to(dt)
    tw = torch.from_numpy(w).cuda()
    tb = None if b is None else torch.from_numpy(b).cuda()
    y = K.ssm_conv1d_fwd(tx, tw, tb, silu=c["silu"], x_prev=txp)
    g = K.ssm_conv1d_bwd(tx, tw, tb, tdy, silu=c["silu"], x_prev=txp, want_dx_prev=True)
    ref_y = CO.conv1d_fwd(x, w, b, silu=c["silu"], x_prev=xp)
    ref = CO.conv1d_bwd(x, w, b, dy, silu=c["silu"], x_prev=xp)
    tol = U.TOL[c["io"]]
    assert U.rel_err(U.to_host(y), ref_y) <= tol["out"], c
    assert U.rel_err(U.to_host(g["dx"]), ref["dx"]) <= tol["grad"], c
    assert U.rel_err(U.to_host(g["dw"]), ref["dw"]) <= tol["grad"], c
    if b is not None:
        assert U.rel_err(U.to_host(g["dbias"]), ref["dbias"]) <= tol["grad"], c
    if c["W"] > 1 and xp is not None:
        assert U.rel_err(U.to_host(g["dx_prev"]), ref["dx_prev"]) <= tol["grad"], c
