"""Carried-in / carried-out state of the forward and the single recurrent step (the recurrent mode of Eq. 2), on the
GPU against the oracle: chunked processing of a sequence, prompt -> token-by-token hand-off, and the step on its own."""
import numpy as np
import pytest

from paper_2312_00752_b200 import synth
from tests import _gpu_util as U

pytestmark = pytest.mark.gpu


def _case(batch, L, D, N, io, dt=(1e-3, 1e-1), seed=0):
    cfg = synth.ScanConfig("state", 12, batch, L, D, N, io, dt[0], dt[1])
    return synth.make_inputs(cfg, seed=seed, with_dout=False)


def _oracle(inp, h0=None):
    from oracle import ssm_oracle as O
    return O.scan_fwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], D_skip=inp["D_skip"], z=inp["z"], h0=h0,
                      return_h_last=True)


@pytest.mark.parametrize("batch,L,D,N,io,cut", [
    (2, 300, 40, 16, "bf16", 130),      # tuned kernels
    (1, 200, 24, 8, "f32", 77),         # generic kernels
    (1, 6000, 64, 16, "bf16", 2048),    # both pieces split time into segments
])
def test_two_pieces_equal_one_sequence(batch, L, D, N, io, cut):
    import torch
    from paper_2312_00752_b200 import binding as K
    inp = _case(batch, L, D, N, io, dt=(1e-4, 1e-2) if L > 1000 else (1e-3, 1e-1))
    dev = U.to_device(inp, io)
    ref_out, ref_h = _oracle(inp)
    h_mid = torch.empty((batch, D, N), dtype=torch.float32, device="cuda")
    h_end = torch.empty_like(h_mid)
    sl = lambda k, a, b: dev[k][:, a:b].contiguous()
    o1 = K.ssm_scan_fwd(sl("x", 0, cut), sl("delta", 0, cut), dev["A"], sl("B", 0, cut), sl("C", 0, cut), dev["D_skip"],
                        sl("z", 0, cut), h_last=h_mid)
    o2 = K.ssm_scan_fwd(sl("x", cut, L), sl("delta", cut, L), dev["A"], sl("B", cut, L), sl("C", cut, L), dev["D_skip"],
                        sl("z", cut, L), h0=h_mid, h_last=h_end)
    got = np.concatenate([U.to_host(o1), U.to_host(o2)], axis=1)
    assert U.rel_err(got, ref_out) <= U.TOL[io]["out"]
    assert U.rel_err(U.to_host(h_end), ref_h) <= (1e-5 if io == "f32" else 1e-4)     # states are float32 in both
    # and the state in the middle is the oracle's state after `cut` steps
    mid = {k: (v[:, :cut] if v.ndim == 3 and v.shape[1] == L else v) for k, v in inp.items()}
    assert U.rel_err(U.to_host(h_mid), _oracle(mid)[1]) <= (1e-5 if io == "f32" else 1e-4)


@pytest.mark.parametrize("batch,D,N,io", [(3, 40, 16, "bf16"), (2, 33, 8, "f32"), (1, 70, 1, "bf16")])
def test_step_by_step_equals_scan(batch, D, N, io):
    import torch
    from paper_2312_00752_b200 import binding as K
    T = 24
    inp = _case(batch, T, D, N, io)
    dev = U.to_device(inp, io)
    ref_out, ref_h = _oracle(inp)
    h = torch.zeros((batch, D, N), dtype=torch.float32, device="cuda")
    outs = []
    for t in range(T):
        outs.append(K.ssm_step(dev["x"][:, t].contiguous(), dev["delta"][:, t].contiguous(), dev["A"],
                               dev["B"][:, t].contiguous(), dev["C"][:, t].contiguous(), dev["D_skip"],
                               dev["z"][:, t].contiguous(), h))
    got = np.stack([U.to_host(o) for o in outs], axis=1)
    assert U.rel_err(got, ref_out) <= U.TOL[io]["out"]
    assert U.rel_err(U.to_host(h), ref_h) <= 1e-5


def test_prompt_then_generation_hand_off():
    import torch
    from paper_2312_00752_b200 import binding as K
    batch, Lp, Lg, D, N, io = 2, 96, 8, 64, 16, "bf16"
    inp = _case(batch, Lp + Lg, D, N, io)
    dev = U.to_device(inp, io)
    ref_out, ref_h = _oracle(inp)
    h = torch.empty((batch, D, N), dtype=torch.float32, device="cuda")
    sl = lambda k: dev[k][:, :Lp].contiguous()
    o_prompt = K.ssm_scan_fwd(sl("x"), sl("delta"), dev["A"], sl("B"), sl("C"), dev["D_skip"], sl("z"), h_last=h)
    outs = [U.to_host(o_prompt)]
    for t in range(Lp, Lp + Lg):
        o = K.ssm_step(dev["x"][:, t].contiguous(), dev["delta"][:, t].contiguous(), dev["A"],
                       dev["B"][:, t].contiguous(), dev["C"][:, t].contiguous(), dev["D_skip"],
                       dev["z"][:, t].contiguous(), h)
        outs.append(U.to_host(o)[:, None, :])
    got = np.concatenate(outs, axis=1)
    assert U.rel_err(got, ref_out) <= U.TOL[io]["out"]
    assert U.rel_err(U.to_host(h), ref_h) <= 1e-4


def test_saved_states_carry_h0_into_backward():
    """Backward given the checkpoint states of a forward that started from h0 differentiates that forward."""
    import torch
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    batch, L, D, N, io, cut = 1, 160, 16, 16, "f32", 64
    cfg = synth.ScanConfig("state", 12, batch, L, D, N, io, 1e-3, 1e-1)
    inp = synth.make_inputs(cfg, seed=3)
    dev = U.to_device(inp, io)
    # oracle: gradients of the second piece alone are the tail of the full-sequence gradients for dx, ddelta, dz, dB, dC
    ref = U.oracle_fwd_bwd(inp)
    sl = lambda k, a, b: dev[k][:, a:b].contiguous()
    h_mid = torch.empty((batch, D, N), dtype=torch.float32, device="cuda")
    K.ssm_scan_fwd(sl("x", 0, cut), sl("delta", 0, cut), dev["A"], sl("B", 0, cut), sl("C", 0, cut), dev["D_skip"],
                   sl("z", 0, cut), h_last=h_mid)
    args2 = (sl("x", cut, L), sl("delta", cut, L), dev["A"], sl("B", cut, L), sl("C", cut, L), dev["D_skip"], sl("z", cut, L))
    _, saved = K.ssm_scan_fwd(*args2, save_states=True, h0=h_mid)
    g = K.ssm_scan_bwd(*args2, sl("dout", cut, L), saved)
    for k in ("dx", "ddelta", "dz", "dB", "dC"):
        assert U.rel_err(U.to_host(g[k]), ref[k][:, cut:]) <= U.TOL[io]["grad"], k


@pytest.mark.parametrize("batch,L,D,N,io,cut,saved", [
    (2, 300, 40, 16, "bf16", 130, True),       # tuned kernels
    (2, 300, 40, 16, "bf16", 130, False),      # ... with the checkpoints rebuilt from h0
    (1, 200, 24, 8, "f32", 77, True),          # generic kernels
    (1, 200, 24, 8, "f32", 77, False),
    (1, 6000, 64, 16, "bf16", 2048, True),     # both pieces split time: dh_last enters the reverse carry
])
def test_backward_in_two_pieces(batch, L, D, N, io, cut, saved):
    import torch
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    cfg = synth.ScanConfig("state", 12, batch, L, D, N, io, *((1e-4, 1e-2) if L > 1000 else (1e-3, 1e-1)))
    inp = synth.make_inputs(cfg, seed=3)
    dev = U.to_device(inp, io)
    ref = O.scan_bwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], inp["D_skip"], inp["z"], inp["dout"])
    sl = lambda k, a, b: dev[k][:, a:b].contiguous()
    piece = lambda a, b: (sl("x", a, b), sl("delta", a, b), dev["A"], sl("B", a, b), sl("C", a, b), dev["D_skip"],
                          sl("z", a, b))
    h_mid = torch.empty((batch, D, N), dtype=torch.float32, device="cuda")
    _, sv1 = K.ssm_scan_fwd(*piece(0, cut), save_states=True, h_last=h_mid)
    _, sv2 = K.ssm_scan_fwd(*piece(cut, L), save_states=True, h0=h_mid)
    g2 = K.ssm_scan_bwd(*piece(cut, L), sl("dout", cut, L), sv2 if saved else None, h0=h_mid, want_dh0=True)
    g1 = K.ssm_scan_bwd(*piece(0, cut), sl("dout", 0, cut), sv1 if saved else None, dh_last=g2["dh0"], want_dh0=True)
    tol = U.TOL[io]["grad"]
    for k in ("dx", "ddelta", "dz", "dB", "dC"):
        got = np.concatenate([U.to_host(g1[k]), U.to_host(g2[k])], axis=1)
        assert U.rel_err(got, ref[k]) <= tol, k
    for k in ("dA", "dD"):
        assert U.rel_err(U.to_host(g1[k]) + U.to_host(g2[k]), ref[k]) <= tol, k
    # the gradient of the state at the cut, against the oracle's for the second piece alone
    mid = {k: (v[:, cut:] if v.ndim == 3 and v.shape[1] == L else v) for k, v in inp.items()}
    _, h_m = O.scan_fwd(inp["x"][:, :cut], inp["delta"][:, :cut], inp["A"], inp["B"][:, :cut], inp["C"][:, :cut],
                        D_skip=inp["D_skip"], z=inp["z"][:, :cut], return_h_last=True)
    r2 = O.scan_bwd(mid["x"], mid["delta"], mid["A"], mid["B"], mid["C"], mid["D_skip"], mid["z"], mid["dout"], h0=h_m)
    assert U.rel_err(U.to_host(g2["dh0"]), r2["dh0"]) <= (1e-4 if io == "f32" else 3e-2)
    assert U.rel_err(U.to_host(g1["dh0"]), ref["dh0"]) <= (1e-4 if io == "f32" else 3e-2)
