"""State sizes above the ones the paper ablates (N = 32, 64) on the generic kernels against the oracle: forward and
backward, both io dtypes, both B-bar rules, saved or rebuilt checkpoints, a time split, the carried state with the
single recurrent step, and the backward in two pieces."""
import numpy as np
import pytest

from paper_2312_00752_b200 import synth
from tests import _gpu_util as U

pytestmark = pytest.mark.gpu


def _case(batch, L, D, N, io, dt=(1e-3, 5e-2), seed=0):
    cfg = synth.ScanConfig("large_state", 15, batch, L, D, N, io, dt[0], dt[1])
    return synth.make_inputs(cfg, seed=seed)


@pytest.mark.parametrize("batch,L,D,N,io", [
    (2, 100, 24, 32, "f32"),      # ragged time tail, channels 16 + 8 of a 16-channel block
    (1, 257, 40, 32, "bf16"),
    (2, 70, 20, 64, "f32"),       # 8-channel blocks: 8 + 8 + 4
    (1, 130, 9, 64, "bf16"),      # odd channel count
    (1, 1, 8, 64, "f32"),         # a single step
])
def test_forward_backward(batch, L, D, N, io):
    inp = _case(batch, L, D, N, io)
    dev = U.to_device(inp, io)
    ref = U.oracle_fwd_bwd(inp)
    for use_saved in (True, False):
        U.assert_parity(U.gpu_fwd_bwd(dev, use_saved=use_saved), ref, io, f"{(batch, L, D, N, io)} saved={use_saved}")
    U.assert_parity(U.gpu_fwd_bwd(dev, general_A=True), ref, io, "general-A flag")


@pytest.mark.parametrize("N,io", [(32, "f32"), (64, "bf16")])
def test_time_split(N, io):
    from paper_2312_00752_b200 import binding as K
    inp = _case(1, 4200, 16, N, io, dt=(1e-4, 5e-3))
    dev = U.to_device(inp, io)
    assert K.plan(K.make_problem(dev["x"], dev["B"], True, True))["n_segments"] > 1
    ref = U.oracle_fwd_bwd(inp)
    for use_saved in (True, False):
        U.assert_parity(U.gpu_fwd_bwd(dev, use_saved=use_saved), ref, io, f"time split N={N} saved={use_saved}")


@pytest.mark.parametrize("N,io", [(32, "bf16"), (64, "f32")])
def test_zoh(N, io):
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    inp = _case(2, 90, 24, N, io, dt=(1e-2, 0.5))
    dev = U.to_device(inp, io)
    args = (dev["x"], dev["delta"], dev["A"], dev["B"], dev["C"], dev["D_skip"], dev["z"])
    out, saved = K.ssm_scan_fwd(*args, save_states=True, zoh=True)
    g = K.ssm_scan_bwd(*args, dev["dout"], saved, zoh=True)
    ref_out = O.scan_fwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], D_skip=inp["D_skip"], z=inp["z"], zoh=True)
    ref = O.scan_bwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], inp["D_skip"], inp["z"], inp["dout"], zoh=True)
    assert U.rel_err(U.to_host(out), ref_out) <= U.TOL[io]["out"]
    for k in U.GRADS:
        assert U.rel_err(U.to_host(g[k]), ref[k]) <= U.TOL[io]["grad"], k


@pytest.mark.parametrize("N,io", [(32, "f32"), (64, "bf16")])
def test_step_by_step_equals_scan(N, io):
    import torch
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    batch, T, D = 2, 20, 24
    inp = _case(batch, T, D, N, io)
    dev = U.to_device(inp, io)
    ref_out, ref_h = O.scan_fwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], D_skip=inp["D_skip"], z=inp["z"],
                                return_h_last=True)
    h = torch.zeros((batch, D, N), dtype=torch.float32, device="cuda")
    outs = []
    for t in range(T):
        outs.append(K.ssm_step(dev["x"][:, t].contiguous(), dev["delta"][:, t].contiguous(), dev["A"],
                               dev["B"][:, t].contiguous(), dev["C"][:, t].contiguous(), dev["D_skip"],
                               dev["z"][:, t].contiguous(), h))
    got = np.stack([U.to_host(o) for o in outs], axis=1)
    assert U.rel_err(got, ref_out) <= U.TOL[io]["out"]
    assert U.rel_err(U.to_host(h), ref_h) <= 1e-5


@pytest.mark.parametrize("N,io,L,cut", [(32, "f32", 150, 70), (64, "bf16", 5000, 2048)])
def test_backward_in_two_pieces(N, io, L, cut):
    import torch
    from paper_2312_00752_b200 import binding as K
    batch, D = 1, 16
    inp = _case(batch, L, D, N, io, dt=(1e-3, 5e-2) if L < 1000 else (1e-4, 5e-3))
    dev = U.to_device(inp, io)
    ref = U.oracle_fwd_bwd(inp)
    sl = lambda k, a, b: dev[k][:, a:b].contiguous()
    piece = lambda a, b: (sl("x", a, b), sl("delta", a, b), dev["A"], sl("B", a, b), sl("C", a, b), dev["D_skip"],
                          sl("z", a, b))
    h_mid = torch.empty((batch, D, N), dtype=torch.float32, device="cuda")
    _, sv1 = K.ssm_scan_fwd(*piece(0, cut), save_states=True, h_last=h_mid)
    _, sv2 = K.ssm_scan_fwd(*piece(cut, L), save_states=True, h0=h_mid)
    g2 = K.ssm_scan_bwd(*piece(cut, L), sl("dout", cut, L), sv2, h0=h_mid, want_dh0=True)
    g1 = K.ssm_scan_bwd(*piece(0, cut), sl("dout", 0, cut), sv1, dh_last=g2["dh0"])
    tol = U.TOL[io]["grad"]
    for k in ("dx", "ddelta", "dz", "dB", "dC"):
        assert U.rel_err(np.concatenate([U.to_host(g1[k]), U.to_host(g2[k])], axis=1), ref[k]) <= tol, k
    for k in ("dA", "dD"):
        assert U.rel_err(U.to_host(g1[k]) + U.to_host(g2[k]), ref[k]) <= tol, k


@pytest.mark.parametrize("N", [32, 64])
def test_non_selective_B_and_C(N):
    # B and C as parameters [D][N]: the oracle is driven one channel at a time with that channel's rows broadcast
    import torch
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    batch, L, D, io = 2, 60, 12, "f32"
    inp = _case(batch, L, D, N, io)
    rng = np.random.default_rng(7)
    Bs = rng.standard_normal((D, N)).astype(np.float32)
    Cs = rng.standard_normal((D, N)).astype(np.float32)
    dev = U.to_device(inp, io)
    dBs, dCs = torch.from_numpy(Bs).cuda(), torch.from_numpy(Cs).cuda()
    args = (dev["x"], dev["delta"], dev["A"], dBs, dCs, dev["D_skip"], dev["z"])
    out, saved = K.ssm_scan_fwd(*args, save_states=True, static_B=True, static_C=True)
    g = K.ssm_scan_bwd(*args, dev["dout"], saved, static_B=True, static_C=True)
    ref_out = np.empty((batch, L, D))
    ref_dB, ref_dC = np.empty((D, N)), np.empty((D, N))
    for d in range(D):
        one = lambda k: inp[k][:, :, d:d + 1]
        Bd = np.broadcast_to(Bs[d], (batch, L, N)).copy()
        Cd = np.broadcast_to(Cs[d], (batch, L, N)).copy()
        ref_out[:, :, d] = O.scan_fwd(one("x"), one("delta"), inp["A"][d:d + 1], Bd, Cd, D_skip=inp["D_skip"][d:d + 1],
                                      z=one("z"))[:, :, 0]
        r = O.scan_bwd(one("x"), one("delta"), inp["A"][d:d + 1], Bd, Cd, inp["D_skip"][d:d + 1], one("z"), one("dout"))
        ref_dB[d], ref_dC[d] = r["dB"].sum((0, 1)), r["dC"].sum((0, 1))
    assert U.rel_err(U.to_host(out), ref_out) <= 1e-5
    assert U.rel_err(U.to_host(g["dB"]), ref_dB) <= 1e-4
    assert U.rel_err(U.to_host(g["dC"]), ref_dC) <= 1e-4
