"""Seeded sweep over WIDE, short problems (thousands of channels, tens to hundreds of steps) and option combinations
against the oracle.  At these widths the tuned kernels have more chains than resident warps, so neighbouring warps
share chains and the carried values (state, adjoint, dA, dD, bias gradient) cross the hand-off; the forward may take
its two-stage ring, the backward may or may not split time.  The sequences are short enough for the fp64 oracle to
run on every element."""
import numpy as np
import pytest

from paper_2312_00752_b200 import synth
from tests import _gpu_util as U

pytestmark = pytest.mark.gpu


def _draw(rng):
    return dict(batch=int(rng.choice([3, 4, 8])), L=int(rng.choice([17, 40, 72, 130, 300, 520])),
                D=int(rng.choice([5120, 5000, 4104, 2560])), gate=bool(rng.integers(0, 2)), skip=bool(rng.integers(0, 2)),
                zoh=bool(rng.integers(0, 2)), general_A=bool(rng.integers(0, 2)), saved=bool(rng.integers(0, 2)),
                carry=bool(rng.integers(0, 2)), fused=bool(rng.integers(0, 2)), softplus=bool(rng.integers(0, 2)))


CASES = [_draw(np.random.default_rng([2312, 754, i])) for i in range(24)]


@pytest.mark.parametrize("case", CASES, ids=[f"{i}" for i in range(len(CASES))])
def test_random_wide_problem(case):
    import torch
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    c = case
    io, N = "bf16", 16
    cfg = synth.ScanConfig("random_wide", 20, c["batch"], c["L"], c["D"], N, io, 1e-3, 1e-1)
    inp = synth.make_inputs(cfg, seed=3, perturb_A=0.01 if c["general_A"] else 0.0)
    rng = np.random.default_rng(17)
    bias = None
    if c["fused"]:
        tau = synth.channel_tau(cfg, 3)
        if c["softplus"]:
            bias = (tau + np.log(-np.expm1(-tau))).astype(np.float32)
            inp["delta"] = synth.round_to_io(0.1 * rng.standard_normal(inp["delta"].shape), io)
        else:
            bias = (0.5 * tau).astype(np.float32)
            inp["delta"] = synth.round_to_io(0.5 * np.abs(inp["delta"]), io)
    if not c["gate"]:
        inp["z"] = None
    if not c["skip"]:
        inp["D_skip"] = None
    shape = (c["batch"], c["D"], N)
    h0 = rng.standard_normal(shape).astype(np.float32) if c["carry"] else None
    dhl = rng.standard_normal(shape).astype(np.float32) if c["carry"] else None
    dev = U.to_device(inp, io)
    t = lambda a: None if a is None else torch.from_numpy(a).cuda()
    if c["fused"]:
        args = (dev["x"], dev["delta"], t(bias), dev["A"], dev["B"], dev["C"], dev["D_skip"], dev["z"])
        out, saved = K.ssm_scan_fwd_fused_dt(*args, softplus=c["softplus"], save_states=True, zoh=c["zoh"], h0=t(h0))
        g = K.ssm_scan_bwd_fused_dt(*args, dev["dout"], saved if c["saved"] else None, softplus=c["softplus"],
                                    zoh=c["zoh"], h0=t(h0), dh_last=t(dhl), want_dh0=True)
        kw = dict(delta_softplus=c["softplus"], delta_bias=bias)
    else:
        args = (dev["x"], dev["delta"], dev["A"], dev["B"], dev["C"], dev["D_skip"], dev["z"])
        out, saved = K.ssm_scan_fwd(*args, save_states=True, zoh=c["zoh"], general_A=c["general_A"], h0=t(h0))
        g = K.ssm_scan_bwd(*args, dev["dout"], saved if c["saved"] else None, zoh=c["zoh"], general_A=c["general_A"],
                           h0=t(h0), dh_last=t(dhl), want_dh0=True)
        kw = {}
    ref_out = O.scan_fwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], D_skip=inp["D_skip"], z=inp["z"],
                         h0=h0, zoh=c["zoh"], **kw)
    ref = O.scan_bwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], inp["D_skip"], inp["z"], inp["dout"],
                     zoh=c["zoh"], h0=h0, dh_last=dhl, **kw)
    tol = U.TOL[io]
    assert U.rel_err(U.to_host(out), ref_out) <= tol["out"], c
    for k in U.GRADS + ("dh0",) + (("ddelta_bias",) if c["fused"] else ()):
        if g.get(k) is None:
            continue
        state_tol = 1e-4 if k == "dh0" else tol["grad"]      # dh0 is float32 on both paths
        assert U.rel_err(U.to_host(g[k]), ref[k]) <= state_tol, (k, c)
