"""Step size through the fused softplus (Algorithm 2 step 4) on the GPU against the oracle, forward and backward."""
import numpy as np
import pytest

from paper_2312_00752_b200 import synth
from tests import _gpu_util as U

pytestmark = pytest.mark.gpu


def _pre_activation_case(batch, L, D, N, io, seed=0):
    """Inputs of a workload with `delta` replaced by a pre-activation and a per-channel bias: the pre-activation is
    the small noise term of the recipe (rounded to the io dtype), the bias is softplus^-1 of the per-channel target
    step (float32), so that softplus(pre + bias) has the recipe's distribution."""
    cfg = synth.ScanConfig("fused_dt", 13, batch, L, D, N, io, 1e-3, 1e-1)
    inp = synth.make_inputs(cfg, seed=seed)
    rng = np.random.default_rng(100 + seed)
    tau = synth.channel_tau(cfg, seed)
    bias = (tau + np.log(-np.expm1(-tau))).astype(np.float32)
    pre = synth.round_to_io(0.1 * rng.standard_normal((batch, L, D)), io)
    inp["delta"] = pre
    return inp, bias


@pytest.mark.parametrize("batch,L,D,N,io", [(2, 130, 40, 16, "bf16"), (1, 200, 24, 8, "f32"), (1, 4200, 32, 16, "f32"), (1, 4200, 48, 16, "bf16"),
                                           (3, 1000, 328, 16, "bf16")])
@pytest.mark.parametrize("softplus", [True, False])
def test_fused_step_size_forward_backward(batch, L, D, N, io, softplus):
    import torch
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    inp, bias = _pre_activation_case(batch, L, D, N, io)
    if not softplus:
        bias = np.abs(bias) * 0.01 + 0.05          # keeps delta_pre + bias positive
        inp["delta"] = synth.round_to_io(np.abs(inp["delta"]) * 0.1, io)
    dev = U.to_device(inp, io)
    dbias = torch.from_numpy(bias).cuda()
    args = (dev["x"], dev["delta"], dbias, dev["A"], dev["B"], dev["C"], dev["D_skip"], dev["z"])
    out, saved = K.ssm_scan_fwd_fused_dt(*args, softplus=softplus, save_states=True)
    g = K.ssm_scan_bwd_fused_dt(*args, dev["dout"], saved, softplus=softplus)
    ref_out = O.scan_fwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], D_skip=inp["D_skip"], z=inp["z"],
                         delta_softplus=softplus, delta_bias=bias)
    ref = O.scan_bwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], inp["D_skip"], inp["z"], inp["dout"],
                     delta_softplus=softplus, delta_bias=bias)
    tol = U.TOL[io]
    assert U.rel_err(U.to_host(out), ref_out) <= tol["out"]
    for k in ("dx", "ddelta", "ddelta_bias", "dz", "dB", "dC", "dA", "dD"):
        assert U.rel_err(U.to_host(g[k]), ref[k]) <= tol["grad"], k
    # without saved states the backward rebuilds the checkpoints with the same fused step size
    g2 = K.ssm_scan_bwd_fused_dt(*args, dev["dout"], None, softplus=softplus)
    for k in ("dx", "ddelta", "ddelta_bias", "dA"):
        assert U.rel_err(U.to_host(g2[k]), ref[k]) <= tol["grad"], k


@pytest.mark.parametrize("batch,L,D,N,io", [(2, 130, 40, 16, "bf16"), (1, 100, 24, 8, "f32")])
def test_fused_step_size_with_the_zoh_rule(batch, L, D, N, io):
    # both options at once: delta = softplus(v + bias) and B-bar = (exp(delta A) - 1) / A * B
    import torch
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    inp, bias = _pre_activation_case(batch, L, D, N, io)
    dev = U.to_device(inp, io)
    dbias = torch.from_numpy(bias).cuda()
    args = (dev["x"], dev["delta"], dbias, dev["A"], dev["B"], dev["C"], dev["D_skip"], dev["z"])
    out, saved = K.ssm_scan_fwd_fused_dt(*args, save_states=True, zoh=True)
    g = K.ssm_scan_bwd_fused_dt(*args, dev["dout"], saved, zoh=True)
    ref_out = O.scan_fwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], D_skip=inp["D_skip"], z=inp["z"],
                         delta_softplus=True, delta_bias=bias, zoh=True)
    ref = O.scan_bwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], inp["D_skip"], inp["z"], inp["dout"],
                     delta_softplus=True, delta_bias=bias, zoh=True)
    tol = U.TOL[io]
    assert U.rel_err(U.to_host(out), ref_out) <= tol["out"]
    for k in ("dx", "ddelta", "ddelta_bias", "dz", "dB", "dC", "dA", "dD"):
        assert U.rel_err(U.to_host(g[k]), ref[k]) <= tol["grad"], k


@pytest.mark.parametrize("batch,L,D,N,io,cut", [(2, 300, 40, 16, "bf16", 130), (1, 6000, 64, 16, "bf16", 2048)])
def test_fused_step_size_backward_in_two_pieces(batch, L, D, N, io, cut):
    # the chunked use (carried state, adjoint handed back across the cut) together with the fused step size
    import torch
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    inp, bias = _pre_activation_case(batch, L, D, N, io)
    dev = U.to_device(inp, io)
    dbias = torch.from_numpy(bias).cuda()
    ref = O.scan_bwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], inp["D_skip"], inp["z"], inp["dout"],
                     delta_softplus=True, delta_bias=bias)
    sl = lambda k, a, b: dev[k][:, a:b].contiguous()
    piece = lambda a, b: (sl("x", a, b), sl("delta", a, b), dbias, dev["A"], sl("B", a, b), sl("C", a, b), dev["D_skip"],
                          sl("z", a, b))
    h_mid = torch.empty((batch, D, N), dtype=torch.float32, device="cuda")
    _, sv1 = K.ssm_scan_fwd_fused_dt(*piece(0, cut), save_states=True, h_last=h_mid)
    _, sv2 = K.ssm_scan_fwd_fused_dt(*piece(cut, L), save_states=True, h0=h_mid)
    g2 = K.ssm_scan_bwd_fused_dt(*piece(cut, L), sl("dout", cut, L), sv2, h0=h_mid, want_dh0=True)
    g1 = K.ssm_scan_bwd_fused_dt(*piece(0, cut), sl("dout", 0, cut), sv1, dh_last=g2["dh0"])
    tol = U.TOL[io]["grad"]
    for k in ("dx", "ddelta", "dz", "dB", "dC"):
        got = np.concatenate([U.to_host(g1[k]), U.to_host(g2[k])], axis=1)
        assert U.rel_err(got, ref[k]) <= tol, k
    for k in ("dA", "dD", "ddelta_bias"):
        assert U.rel_err(U.to_host(g1[k]) + U.to_host(g2[k]), ref[k]) <= tol, k


def test_fused_step_size_on_a_wide_short_problem():
    """Batch 8 of the 2.8B layer width on a short, ragged sequence: 1280 chains, which the forward runs with the two-stage
    ring at two warps per sub-partition and shared chains, the backward without a time split.  The oracle runs on
    sampled channels (B and C are shared by all channels, so dB / dC are not checked here)."""
    import torch
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    batch, L, D, N, io = 8, 72, 5120, 16, "bf16"
    inp, bias = _pre_activation_case(batch, L, D, N, io)
    dev = U.to_device(inp, io)
    dbias = torch.from_numpy(bias).cuda()
    args = (dev["x"], dev["delta"], dbias, dev["A"], dev["B"], dev["C"], dev["D_skip"], dev["z"])
    out, saved = K.ssm_scan_fwd_fused_dt(*args, save_states=True)
    g = K.ssm_scan_bwd_fused_dt(*args, dev["dout"], saved)
    rng = np.random.default_rng(3)
    ch = np.array(sorted(set([0, 31, 32, 2559, 2560, 5119] + [int(c) for c in rng.integers(0, D, 42)])))
    sub = lambda k: np.ascontiguousarray(inp[k][:, :, ch])
    ref_out = O.scan_fwd(sub("x"), sub("delta"), inp["A"][ch], inp["B"], inp["C"], D_skip=inp["D_skip"][ch], z=sub("z"),
                         delta_softplus=True, delta_bias=bias[ch])
    ref = O.scan_bwd(sub("x"), sub("delta"), inp["A"][ch], inp["B"], inp["C"], inp["D_skip"][ch], sub("z"), sub("dout"),
                     delta_softplus=True, delta_bias=bias[ch])
    tol = U.TOL[io]
    assert U.rel_err(U.to_host(out)[:, :, ch], ref_out) <= tol["out"]
    for k in ("dx", "ddelta", "dz"):
        assert U.rel_err(U.to_host(g[k])[:, :, ch], ref[k]) <= tol["grad"], k
    for k in ("dA", "dD", "ddelta_bias"):
        assert U.rel_err(U.to_host(g[k])[ch], ref[k]) <= tol["grad"], k
    # the plain calls on the same shape (step sizes given): forward with and without checkpoints agree bit for bit
    delta = torch.nn.functional.softplus(dev["delta"].float() + dbias).to(torch.bfloat16)
    plain = (dev["x"], delta, dev["A"], dev["B"], dev["C"], dev["D_skip"], dev["z"])
    o1, _ = K.ssm_scan_fwd(*plain, save_states=True)
    o2 = K.ssm_scan_fwd(*plain)
    assert torch.equal(o1, o2)
    ref_plain = O.scan_fwd(sub("x"), U.to_host(delta)[:, :, ch], inp["A"][ch], inp["B"], inp["C"], D_skip=inp["D_skip"][ch],
                           z=sub("z"))
    assert U.rel_err(U.to_host(o1)[:, :, ch], ref_plain) <= tol["out"]
