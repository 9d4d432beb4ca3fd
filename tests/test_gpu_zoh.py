"""Zero-order-hold B-bar (Eq. 4: B-bar = (exp(delta A) - 1) / A * B) on the GPU against the oracle: forward, backward,
the single recurrent step, and the gated-recurrence special case of Theorem 1."""
import numpy as np
import pytest

from paper_2312_00752_b200 import synth
from tests import _gpu_util as U

pytestmark = pytest.mark.gpu


def _case(batch, L, D, N, io, dt=(1e-3, 1e-1), seed=0):
    cfg = synth.ScanConfig("zoh", 14, batch, L, D, N, io, dt[0], dt[1])
    inp = synth.make_inputs(cfg, seed=seed)
    inp["A"] = inp["A"].copy()
    inp["A"][0, 0] = 0.0            # the removable singularity: B-bar = delta * B there
    return inp


@pytest.mark.parametrize("batch,L,D,N,io,dt", [
    (2, 130, 40, 16, "bf16", (1e-3, 1e-1)),
    (1, 200, 24, 8, "f32", (1e-3, 1e-1)),
    (2, 97, 33, 4, "f32", (5e-2, 2.0)),        # large steps: the two rules differ by O(1)
    (1, 4200, 32, 16, "f32", (1e-4, 1e-2)),    # time split: segment summaries and both carries under ZOH
    (1, 64, 16, 1, "bf16", (1e-2, 1.0)),
    (2, 200, 64, 16, "bf16", (5e-2, 2.0)),     # tuned kernels, large steps
    (1, 4200, 48, 16, "bf16", (1e-4, 1e-2)),   # tuned kernels with a time split
])
def test_zoh_forward_backward(batch, L, D, N, io, dt):
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    inp = _case(batch, L, D, N, io, dt)
    dev = U.to_device(inp, io)
    args = (dev["x"], dev["delta"], dev["A"], dev["B"], dev["C"], dev["D_skip"], dev["z"])
    out, saved = K.ssm_scan_fwd(*args, save_states=True, zoh=True)
    g = K.ssm_scan_bwd(*args, dev["dout"], saved, zoh=True)
    ref_out = O.scan_fwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], D_skip=inp["D_skip"], z=inp["z"], zoh=True)
    ref = O.scan_bwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], inp["D_skip"], inp["z"], inp["dout"], zoh=True)
    tol = U.TOL[io]
    assert U.rel_err(U.to_host(out), ref_out) <= tol["out"]
    for k in U.GRADS:
        assert U.rel_err(U.to_host(g[k]), ref[k]) <= tol["grad"], k
    # the flag is not a no-op: the default rule gives a different answer where delta * A is not small
    if dt[1] >= 1.0:
        plain = O.scan_fwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], D_skip=inp["D_skip"], z=inp["z"])
        assert U.rel_err(U.to_host(out), plain) > 0.03
    # backward without saved states rebuilds the checkpoints under the same rule
    g2 = K.ssm_scan_bwd(*args, dev["dout"], None, zoh=True)
    for k in ("dx", "ddelta", "dA", "dB"):
        assert U.rel_err(U.to_host(g2[k]), ref[k]) <= tol["grad"], k


@pytest.mark.parametrize("batch,L,D,N,io,dt", [
    (2, 200, 64, 16, "bf16", (1e-6, 1e-5)),    # tuned kernels: delta |A| down to 1e-6, where (exp(delta A) - 1) / A
    (2, 200, 64, 16, "bf16", (1e-6, 1.0)),     # cancels in float32; the second range crosses over to the closed form
    (1, 4200, 32, 16, "bf16", (1e-6, 1e-4)),   # the same through a time split
    (1, 150, 24, 16, "f32", (1e-6, 1e-5)),     # generic kernels
])
def test_zoh_tiny_steps(batch, L, D, N, io, dt):
    # Without the skip term the output is C h alone, so a relative error of the input gain E shows in full.
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    inp = _case(batch, L, D, N, io, dt)
    dev = U.to_device(inp, io)
    args = (dev["x"], dev["delta"], dev["A"], dev["B"], dev["C"], None, dev["z"])
    out, saved = K.ssm_scan_fwd(*args, save_states=True, zoh=True)
    g = K.ssm_scan_bwd(*args, dev["dout"], saved, zoh=True)
    ref_out = O.scan_fwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], z=inp["z"], zoh=True)
    ref = O.scan_bwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], None, inp["z"], inp["dout"], zoh=True)
    tol = U.TOL[io]
    assert U.rel_err(U.to_host(out), ref_out) <= tol["out"]
    for k in ("dx", "ddelta", "dz", "dB", "dC", "dA"):
        assert U.rel_err(U.to_host(g[k]), ref[k]) <= tol["grad"], k
    if io == "bf16":
        # float32 output of the tuned kernels: far inside the io tolerance when the series is in use
        assert U.rel_err(U.to_host(g["dA"]), ref["dA"]) <= 1e-3


def test_zoh_gated_recurrence_of_theorem_1():
    # N = 1, A = -1, B = C = 1, delta = softplus(v): h_t = (1 - g_t) h_{t-1} + g_t x_t with g = sigmoid(v)
    import torch
    from paper_2312_00752_b200 import binding as K
    rng = np.random.default_rng(5)
    batch, L, D = 2, 150, 24
    v = rng.standard_normal((batch, L, D)) * 2.0
    x = rng.standard_normal((batch, L, D)).astype(np.float32)
    delta = np.log1p(np.exp(v)).astype(np.float32)
    g = -np.expm1(-delta.astype(np.float64))          # 1 - exp(-delta), the gate the rounded step size stands for
    h = np.zeros((batch, D))
    ref = np.empty((batch, L, D))
    for t in range(L):
        h = (1.0 - g[:, t]) * h + g[:, t] * x[:, t]
        ref[:, t] = h
    ones = torch.ones((batch, L, 1), dtype=torch.float32, device="cuda")
    A = -torch.ones((D, 1), dtype=torch.float32, device="cuda")
    out = K.ssm_scan_fwd(torch.from_numpy(x).cuda(), torch.from_numpy(delta).cuda(), A, ones, ones, zoh=True)
    assert U.rel_err(U.to_host(out), ref) <= 1e-5


@pytest.mark.parametrize("batch,D,N,io", [(3, 40, 16, "bf16"), (2, 33, 8, "f32")])
def test_zoh_step_by_step_equals_scan(batch, D, N, io):
    import torch
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    T = 20
    inp = _case(batch, T, D, N, io, (5e-2, 1.0))
    dev = U.to_device(inp, io)
    ref_out, ref_h = O.scan_fwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], D_skip=inp["D_skip"], z=inp["z"],
                                zoh=True, return_h_last=True)
    h = torch.zeros((batch, D, N), dtype=torch.float32, device="cuda")
    outs = []
    for t in range(T):
        outs.append(K.ssm_step(dev["x"][:, t].contiguous(), dev["delta"][:, t].contiguous(), dev["A"],
                               dev["B"][:, t].contiguous(), dev["C"][:, t].contiguous(), dev["D_skip"],
                               dev["z"][:, t].contiguous(), h, zoh=True))
    got = np.stack([U.to_host(o) for o in outs], axis=1)
    assert U.rel_err(got, ref_out) <= U.TOL[io]["out"]
    assert U.rel_err(U.to_host(h), ref_h) <= 1e-5


@pytest.mark.parametrize("batch,L,D,N,io,cut", [(2, 300, 40, 16, "bf16", 130), (1, 150, 24, 8, "f32", 70),
                                               (1, 6000, 64, 16, "bf16", 2048)])    # the last: both pieces split time
def test_zoh_backward_in_two_pieces(batch, L, D, N, io, cut):
    # carried state and adjoint across a cut under the ZOH rule (ragged last tiles with an adjoint flowing through)
    import torch
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    inp = _case(batch, L, D, N, io, (5e-3, 0.5) if L < 1000 else (1e-4, 1e-2))
    dev = U.to_device(inp, io)
    ref = O.scan_bwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], inp["D_skip"], inp["z"], inp["dout"], zoh=True)
    sl = lambda k, a, b: dev[k][:, a:b].contiguous()
    piece = lambda a, b: (sl("x", a, b), sl("delta", a, b), dev["A"], sl("B", a, b), sl("C", a, b), dev["D_skip"],
                          sl("z", a, b))
    h_mid = torch.empty((batch, D, N), dtype=torch.float32, device="cuda")
    _, sv1 = K.ssm_scan_fwd(*piece(0, cut), save_states=True, h_last=h_mid, zoh=True)
    _, sv2 = K.ssm_scan_fwd(*piece(cut, L), save_states=True, h0=h_mid, zoh=True)
    g2 = K.ssm_scan_bwd(*piece(cut, L), sl("dout", cut, L), sv2, h0=h_mid, want_dh0=True, zoh=True)
    g1 = K.ssm_scan_bwd(*piece(0, cut), sl("dout", 0, cut), sv1, dh_last=g2["dh0"], want_dh0=True, zoh=True)
    tol = U.TOL[io]["grad"]
    for k in ("dx", "ddelta", "dz", "dB", "dC"):
        assert U.rel_err(np.concatenate([U.to_host(g1[k]), U.to_host(g2[k])], axis=1), ref[k]) <= tol, k
    for k in ("dA", "dD"):
        assert U.rel_err(U.to_host(g1[k]) + U.to_host(g2[k]), ref[k]) <= tol, k
    assert U.rel_err(U.to_host(g1["dh0"]), ref["dh0"]) <= (1e-4 if io == "f32" else 3e-2)
