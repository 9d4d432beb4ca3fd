"""bf16 problems with fewer than 16 states per channel (the state sizes of Table 10) run on the tuned 16-state kernels
with A, B, C and the state arrays widened by columns that stay zero.  Checked here against the oracle at the problem's
own N: every N below 16, the options that touch a widened array (carried state and adjoint, non-selective B / C, both
B-bar rules, the fused step size), A rows that are and are not arithmetic progressions (the widening of A continues a
progression only while it stays non-positive), and a wide shape where neighbouring warps share chains."""
import numpy as np
import pytest

from paper_2312_00752_b200 import synth
from tests import _gpu_util as U

pytestmark = pytest.mark.gpu


def _problem(batch, L, D, N, seed=0, dt=(1e-3, 1e-1)):
    cfg = synth.ScanConfig("small_state", 19, batch, L, D, N, "bf16", dt[0], dt[1])
    return cfg, synth.make_inputs(cfg, seed=seed)


@pytest.mark.parametrize("N", [1, 2, 4, 8])
def test_the_widened_route_is_taken_and_matches_the_oracle(N):
    import torch
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    batch, L, D = 2, 150, 72
    cfg, inp = _problem(batch, L, D, N)
    rng = np.random.default_rng(3)
    shape = (batch, D, N)
    h0 = rng.standard_normal(shape).astype(np.float32)
    dhl = rng.standard_normal(shape).astype(np.float32)
    dev = U.to_device(inp, "bf16")
    prob = K.make_problem(dev["x"], dev["B"], True, True)
    assert prob.N == N and K.plan(prob)["states_per_thread"] == 16          # the plan of the 16-state problem
    args = (dev["x"], dev["delta"], dev["A"], dev["B"], dev["C"], dev["D_skip"], dev["z"])
    t = lambda a: torch.from_numpy(a).cuda()
    h_last = torch.empty(shape, dtype=torch.float32, device="cuda")
    out, saved = K.ssm_scan_fwd(*args, save_states=True, h0=t(h0), h_last=h_last)
    ref_out, ref_h = O.scan_fwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], D_skip=inp["D_skip"], z=inp["z"],
                                h0=h0, return_h_last=True)
    ref = O.scan_bwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], inp["D_skip"], inp["z"], inp["dout"], h0=h0,
                     dh_last=dhl)
    tol = U.TOL["bf16"]
    assert U.rel_err(U.to_host(out), ref_out) <= tol["out"]
    assert U.rel_err(U.to_host(h_last), ref_h) <= 1e-4
    for sv in (saved, None):
        g = K.ssm_scan_bwd(*args, dev["dout"], sv, h0=t(h0), dh_last=t(dhl), want_dh0=True)
        for k in U.GRADS + ("dh0",):
            assert g[k].shape == tuple(ref[k].shape), k
            assert U.rel_err(U.to_host(g[k]), ref[k]) <= (1e-4 if k == "dh0" else tol["grad"]), (k, sv is None)
        got = {k: U.to_host(v) for k, v in g.items() if v is not None}
        got["out"] = U.to_host(out)
        U.assert_elementwise(got, dict(ref, out=ref_out), "bf16", f"N={N}")


@pytest.mark.parametrize("kind", ["rising", "irregular", "positive_step_far", "constant"])
def test_rows_of_A_that_cannot_be_continued_as_a_progression(kind):
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    batch, L, D, N = 2, 90, 40, 4
    cfg, inp = _problem(batch, L, D, N, seed=4)
    rng = np.random.default_rng(11)
    if kind == "rising":            # a progression whose continuation would turn positive: -4, -3, -2, -1 | 0, 1, ...
        A = np.tile(np.array([-4.0, -3.0, -2.0, -1.0]), (D, 1))
    elif kind == "irregular":       # no progression at all
        A = -np.exp(rng.uniform(-2.0, 1.5, (D, N)))
    elif kind == "positive_step_far":   # stays negative over the real states and just over the added ones
        A = np.tile(np.array([-16.0, -15.0, -14.0, -13.0]), (D, 1))
    else:                           # equal values: a progression with step 0
        A = np.tile(np.array([-0.7]), (D, N))
    inp["A"] = A.astype(np.float32)
    dev = U.to_device(inp, "bf16")
    args = (dev["x"], dev["delta"], dev["A"], dev["B"], dev["C"], dev["D_skip"], dev["z"])
    out, saved = K.ssm_scan_fwd(*args, save_states=True)
    g = K.ssm_scan_bwd(*args, dev["dout"], saved)
    ref_out = O.scan_fwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], D_skip=inp["D_skip"], z=inp["z"])
    ref = O.scan_bwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], inp["D_skip"], inp["z"], inp["dout"])
    assert np.isfinite(U.to_host(out)).all()
    assert U.rel_err(U.to_host(out), ref_out) <= U.TOL["bf16"]["out"]
    for k in U.GRADS:
        assert np.isfinite(U.to_host(g[k])).all(), k
        assert U.rel_err(U.to_host(g[k]), ref[k]) <= U.TOL["bf16"]["grad"], k


@pytest.mark.parametrize("N,sB,sC", [(8, True, True), (4, True, False), (2, False, True)])
def test_non_selective_b_and_c_with_a_small_state(N, sB, sC):
    import torch
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    batch, L, D = 2, 80, 24
    cfg, inp = _problem(batch, L, D, N, seed=5)
    rng = np.random.default_rng(6)
    Bs = rng.standard_normal((D, N)).astype(np.float32) if sB else None
    Cs = rng.standard_normal((D, N)).astype(np.float32) if sC else None
    dev = U.to_device(inp, "bf16")
    Bd = torch.from_numpy(Bs).cuda() if sB else dev["B"]
    Cd = torch.from_numpy(Cs).cuda() if sC else dev["C"]
    args = (dev["x"], dev["delta"], dev["A"], Bd, Cd, dev["D_skip"], dev["z"])
    out, saved = K.ssm_scan_fwd(*args, save_states=True, static_B=sB, static_C=sC)
    g = K.ssm_scan_bwd(*args, dev["dout"], saved, static_B=sB, static_C=sC)
    # the oracle one channel at a time with that channel's parameter rows broadcast over (batch, L)
    ref_out = np.empty((batch, L, D))
    ref = {k: np.zeros((batch, L, D)) for k in ("dx", "ddelta", "dz")}
    ref.update(dA=np.zeros((D, N)), dD=np.zeros(D), dB=np.zeros((D, N) if sB else (batch, L, N)),
               dC=np.zeros((D, N) if sC else (batch, L, N)))
    for d in range(D):
        sl = lambda a: a[:, :, d:d + 1]
        Bq = np.broadcast_to(Bs[d].astype(np.float64), (batch, L, N)) if sB else inp["B"]
        Cq = np.broadcast_to(Cs[d].astype(np.float64), (batch, L, N)) if sC else inp["C"]
        a = (sl(inp["x"]), sl(inp["delta"]), inp["A"][d:d + 1], Bq, Cq)
        ref_out[:, :, d:d + 1] = O.scan_fwd(*a, D_skip=inp["D_skip"][d:d + 1], z=sl(inp["z"]))
        r = O.scan_bwd(*a, inp["D_skip"][d:d + 1], sl(inp["z"]), sl(inp["dout"]))
        for k in ("dx", "ddelta", "dz"):
            ref[k][:, :, d:d + 1] = r[k]
        ref["dA"][d], ref["dD"][d] = r["dA"][0], r["dD"][0]
        if sB:
            ref["dB"][d] = r["dB"].sum(axis=(0, 1))
        else:
            ref["dB"] += r["dB"]
        if sC:
            ref["dC"][d] = r["dC"].sum(axis=(0, 1))
        else:
            ref["dC"] += r["dC"]
    assert U.rel_err(U.to_host(out), ref_out) <= U.TOL["bf16"]["out"]
    for k in U.GRADS:
        assert g[k].shape == tuple(ref[k].shape), k
        assert U.rel_err(U.to_host(g[k]), ref[k]) <= U.TOL["bf16"]["grad"], k


@pytest.mark.parametrize("N,zoh,softplus", [(8, True, False), (4, False, True), (1, True, True)])
def test_zoh_and_fused_step_size_with_a_small_state(N, zoh, softplus):
    import torch
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    batch, L, D = 2, 200, 48
    cfg, inp = _problem(batch, L, D, N, seed=7)
    rng = np.random.default_rng(8)
    tau = synth.channel_tau(cfg, 7)
    if softplus:
        bias = (tau + np.log(-np.expm1(-tau))).astype(np.float32)
        inp["delta"] = synth.round_to_io(0.1 * rng.standard_normal(inp["delta"].shape), "bf16")
    else:
        bias = (0.5 * tau).astype(np.float32)
        inp["delta"] = synth.round_to_io(0.5 * np.abs(inp["delta"]), "bf16")
    dev = U.to_device(inp, "bf16")
    args = (dev["x"], dev["delta"], torch.from_numpy(bias).cuda(), dev["A"], dev["B"], dev["C"], dev["D_skip"], dev["z"])
    out, saved = K.ssm_scan_fwd_fused_dt(*args, softplus=softplus, save_states=True, zoh=zoh)
    g = K.ssm_scan_bwd_fused_dt(*args, dev["dout"], saved, softplus=softplus, zoh=zoh)
    kw = dict(delta_softplus=softplus, delta_bias=bias, zoh=zoh)
    ref_out = O.scan_fwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], D_skip=inp["D_skip"], z=inp["z"], **kw)
    ref = O.scan_bwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], inp["D_skip"], inp["z"], inp["dout"], **kw)
    assert U.rel_err(U.to_host(out), ref_out) <= U.TOL["bf16"]["out"]
    for k in U.GRADS + ("ddelta_bias",):
        assert U.rel_err(U.to_host(g[k]), ref[k]) <= U.TOL["bf16"]["grad"], k


def test_wide_problem_with_shared_chains_and_a_small_state():
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    batch, L, D, N = 4, 130, 5000, 4        # 628 chains of 32 channels (the last one ragged) for 592 sub-partitions
    cfg, inp = _problem(batch, L, D, N, seed=9)
    dev = U.to_device(inp, "bf16")
    args = (dev["x"], dev["delta"], dev["A"], dev["B"], dev["C"], dev["D_skip"], dev["z"])
    out, saved = K.ssm_scan_fwd(*args, save_states=True)
    g = K.ssm_scan_bwd(*args, dev["dout"], saved)
    ref_out = O.scan_fwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], D_skip=inp["D_skip"], z=inp["z"])
    ref = O.scan_bwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], inp["D_skip"], inp["z"], inp["dout"])
    assert U.rel_err(U.to_host(out), ref_out) <= U.TOL["bf16"]["out"]
    for k in U.GRADS:
        assert U.rel_err(U.to_host(g[k]), ref[k]) <= U.TOL["bf16"]["grad"], k
    # run-to-run bit equality through the widening and narrowing copies
    g2 = K.ssm_scan_bwd(*args, dev["dout"], saved)
    for k in ("dx", "dB", "dC", "dA"):
        assert np.array_equal(U.to_host(g[k]), U.to_host(g2[k])), k
