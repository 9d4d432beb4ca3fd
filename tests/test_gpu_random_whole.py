"""Seeded sweep over problems whose tiles and channel groups are all whole (L a multiple of 32, D a multiple of 32): these
take the instantiations of the tuned kernels that carry no range tests.  Same options as the other sweeps (gate / skip,
both B-bar rules, arithmetic-progression or general A, saved or rebuilt checkpoints, carried state and adjoint, every
state size up to 16, both io dtypes), several time-split lengths among them."""
import numpy as np
import pytest

from paper_2312_00752_b200 import synth
from tests import _gpu_util as U

pytestmark = pytest.mark.gpu


def _draw(rng):
    return dict(io=str(rng.choice(["bf16", "bf16", "f32"])), N=int(rng.choice([16, 16, 16, 8, 4, 2, 1])),
                D=int(rng.choice([32, 64, 96, 128, 160])), L=int(rng.choice([32, 64, 96, 128, 256, 512, 1024, 2048])),
                batch=int(rng.integers(1, 4)), gate=bool(rng.integers(0, 2)), skip=bool(rng.integers(0, 2)),
                zoh=bool(rng.integers(0, 2)), general_A=bool(rng.integers(0, 2)), saved=bool(rng.integers(0, 2)),
                carry=bool(rng.integers(0, 2)), big_steps=bool(rng.integers(0, 2)))


CASES = [_draw(np.random.default_rng([2312, 755, i])) for i in range(48)]


@pytest.mark.parametrize("case", CASES, ids=[f"{i}" for i in range(len(CASES))])
def test_random_whole_problem(case):
    import torch
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    c = case
    cfg = synth.ScanConfig("random_whole", 22, c["batch"], c["L"], c["D"], c["N"], c["io"],
                           *((5e-2, 1.0) if c["big_steps"] else (1e-3, 1e-1)))
    inp = synth.make_inputs(cfg, seed=4, perturb_A=0.01 if c["general_A"] else 0.0)
    if not c["gate"]:
        inp["z"] = None
    if not c["skip"]:
        inp["D_skip"] = None
    rng = np.random.default_rng(41)
    shape = (c["batch"], c["D"], c["N"])
    h0 = rng.standard_normal(shape).astype(np.float32) if c["carry"] else None
    dhl = rng.standard_normal(shape).astype(np.float32) if c["carry"] else None
    dev = U.to_device(inp, c["io"])
    args = (dev["x"], dev["delta"], dev["A"], dev["B"], dev["C"], dev["D_skip"], dev["z"])
    t = lambda a: None if a is None else torch.from_numpy(a).cuda()
    h_last = torch.empty(shape, dtype=torch.float32, device="cuda")
    out, saved = K.ssm_scan_fwd(*args, save_states=True, zoh=c["zoh"], general_A=c["general_A"], h0=t(h0), h_last=h_last)
    g = K.ssm_scan_bwd(*args, dev["dout"], saved if c["saved"] else None, zoh=c["zoh"], general_A=c["general_A"],
                       h0=t(h0), dh_last=t(dhl), want_dh0=True)
    ref_out, ref_h = O.scan_fwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], D_skip=inp["D_skip"], z=inp["z"],
                                h0=h0, zoh=c["zoh"], return_h_last=True)
    ref = O.scan_bwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], inp["D_skip"], inp["z"], inp["dout"],
                     zoh=c["zoh"], h0=h0, dh_last=dhl)
    tol = U.TOL[c["io"]]
    assert U.rel_err(U.to_host(out), ref_out) <= tol["out"], c
    assert U.rel_err(U.to_host(h_last), ref_h) <= (1e-5 if c["io"] == "f32" else 1e-4), c
    for k in U.GRADS + ("dh0",):
        if g.get(k) is None:
            continue
        state_tol = 1e-4 if k == "dh0" and c["io"] == "bf16" else tol["grad"]   # dh0 is float32 on both paths
        assert U.rel_err(U.to_host(g[k]), ref[k]) <= state_tol, (k, c)
    if c["io"] == "bf16":
        got = {k: U.to_host(v) for k, v in g.items() if v is not None}
        got["out"] = U.to_host(out)
        U.assert_elementwise(got, dict(ref, out=ref_out), "bf16", f"whole case {c}")


FUSED_CASES = [_draw(np.random.default_rng([2312, 756, i])) for i in range(24)]


@pytest.mark.parametrize("case", FUSED_CASES, ids=[f"{i}" for i in range(len(FUSED_CASES))])
def test_random_whole_fused_step_size_problem(case):
    # the same shapes through the fused step-size entry points (pre-activation + bias, softplus on or off)
    import torch
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    c = case
    softplus = c["general_A"]          # reuse the drawn bits: this entry point has no general-A switch
    cfg = synth.ScanConfig("random_whole_fused", 23, c["batch"], c["L"], c["D"], c["N"], c["io"], 1e-3, 1e-1)
    inp = synth.make_inputs(cfg, seed=5)
    rng = np.random.default_rng(43)
    tau = synth.channel_tau(cfg, 5)
    if softplus:
        bias = (tau + np.log(-np.expm1(-tau))).astype(np.float32)
        inp["delta"] = synth.round_to_io(0.1 * rng.standard_normal(inp["delta"].shape), c["io"])
    else:
        bias = (0.5 * tau).astype(np.float32)          # delta = pre-activation + bias stays positive
        inp["delta"] = synth.round_to_io(0.5 * np.abs(inp["delta"]), c["io"])
    if not c["gate"]:
        inp["z"] = None
    if not c["skip"]:
        inp["D_skip"] = None
    shape = (c["batch"], c["D"], c["N"])
    h0 = rng.standard_normal(shape).astype(np.float32) if c["carry"] else None
    dhl = rng.standard_normal(shape).astype(np.float32) if c["carry"] else None
    dev = U.to_device(inp, c["io"])
    t = lambda a: None if a is None else torch.from_numpy(a).cuda()
    args = (dev["x"], dev["delta"], t(bias), dev["A"], dev["B"], dev["C"], dev["D_skip"], dev["z"])
    out, saved = K.ssm_scan_fwd_fused_dt(*args, softplus=softplus, save_states=True, zoh=c["zoh"], h0=t(h0))
    g = K.ssm_scan_bwd_fused_dt(*args, dev["dout"], saved if c["saved"] else None, softplus=softplus, zoh=c["zoh"],
                                h0=t(h0), dh_last=t(dhl), want_dh0=True)
    kw = dict(delta_softplus=softplus, delta_bias=bias, zoh=c["zoh"], h0=h0)
    ref_out = O.scan_fwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], D_skip=inp["D_skip"], z=inp["z"], **kw)
    ref = O.scan_bwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], inp["D_skip"], inp["z"], inp["dout"],
                     dh_last=dhl, **kw)
    tol = U.TOL[c["io"]]
    assert U.rel_err(U.to_host(out), ref_out) <= tol["out"], c
    for k in U.GRADS + ("ddelta_bias", "dh0"):
        if g.get(k) is None:
            continue
        state_tol = 1e-4 if k == "dh0" and c["io"] == "bf16" else tol["grad"]
        assert U.rel_err(U.to_host(g[k]), ref[k]) <= state_tol, (k, c)
