"""B and / or C that are not input-dependent (Algorithm 1; the selective-parameter ablation, Table 7): float32
parameters [D][N] instead of [batch][L][N] inputs, with gradients summed over batch and time.  The oracle has no such
mode of its own; here it is driven one channel at a time with that channel's B / C rows broadcast over (batch, L), and
its dB / dC are summed over (batch, L) -- the definition of a shared parameter's gradient."""
import numpy as np
import pytest

from paper_2312_00752_b200 import synth
from tests import _gpu_util as U

pytestmark = pytest.mark.gpu


def _oracle_static(inp, Bs, Cs, zoh=False):
    """Bs / Cs: (D, N) or None (then inp['B'] / inp['C'] are used as they are)."""
    from oracle import ssm_oracle as O
    batch, L, D = inp["x"].shape
    N = inp["A"].shape[1]
    out = np.empty((batch, L, D))
    g = {k: np.zeros((batch, L, D)) for k in ("dx", "ddelta", "dz")}
    g.update(dA=np.zeros((D, N)), dD=np.zeros(D),
             dB=np.zeros((D, N)) if Bs is not None else np.zeros((batch, L, N)),
             dC=np.zeros((D, N)) if Cs is not None else np.zeros((batch, L, N)))
    for d in range(D):
        sl = lambda a: a[:, :, d:d + 1]
        Bd = np.broadcast_to(Bs[d], (batch, L, N)) if Bs is not None else inp["B"]
        Cd = np.broadcast_to(Cs[d], (batch, L, N)) if Cs is not None else inp["C"]
        args = (sl(inp["x"]), sl(inp["delta"]), inp["A"][d:d + 1], Bd, Cd)
        out[:, :, d:d + 1] = O.scan_fwd(*args, D_skip=inp["D_skip"][d:d + 1], z=sl(inp["z"]), zoh=zoh)
        r = O.scan_bwd(*args, inp["D_skip"][d:d + 1], sl(inp["z"]), sl(inp["dout"]), zoh=zoh)
        for k in ("dx", "ddelta", "dz"):
            g[k][:, :, d:d + 1] = r[k]
        g["dA"][d], g["dD"][d] = r["dA"][0], r["dD"][0]
        if Bs is not None:
            g["dB"][d] = r["dB"].sum(axis=(0, 1))
        else:
            g["dB"] += r["dB"]
        if Cs is not None:
            g["dC"][d] = r["dC"].sum(axis=(0, 1))
        else:
            g["dC"] += r["dC"]
    g["out"] = out
    return g


@pytest.mark.parametrize("batch,L,D,N,io,sB,sC,zoh", [
    (2, 100, 24, 16, "bf16", True, True, False),     # fully time-invariant B and C (the S4 layer of Algorithm 1)
    (2, 70, 12, 8, "f32", True, False, False),       # selective C only
    (1, 90, 16, 4, "f32", False, True, True),        # selective B only, ZOH rule
    (1, 1200, 16, 16, "f32", True, True, False),     # time split: the adjoint pre-pass with static C
    (2, 130, 40, 16, "bf16", True, False, False),    # tuned kernels (bf16, N = 16, default B-bar rule): selective C only
    (1, 97, 72, 16, "bf16", False, True, False),     # tuned kernels: selective B only, channel blocks 32 + 32 + 8
    (1, 4200, 48, 16, "bf16", True, True, False),    # tuned kernels with a time split in both directions
    (2, 64, 32, 16, "bf16", True, True, True),       # ZOH with non-selective B / C stays on the generic kernels
])
def test_static_b_and_c(batch, L, D, N, io, sB, sC, zoh):
    import torch
    from paper_2312_00752_b200 import binding as K
    cfg = synth.ScanConfig("static_bc", 16, batch, L, D, N, io, 1e-3, 1e-1)
    inp = synth.make_inputs(cfg, seed=0)
    rng = np.random.default_rng(5)
    Bs = rng.standard_normal((D, N)).astype(np.float32) if sB else None
    Cs = rng.standard_normal((D, N)).astype(np.float32) if sC else None
    dev = U.to_device(inp, io)
    B = torch.from_numpy(Bs).cuda() if sB else dev["B"]
    C = torch.from_numpy(Cs).cuda() if sC else dev["C"]
    args = (dev["x"], dev["delta"], dev["A"], B, C, dev["D_skip"], dev["z"])
    out, saved = K.ssm_scan_fwd(*args, save_states=True, zoh=zoh, static_B=sB, static_C=sC)
    g = K.ssm_scan_bwd(*args, dev["dout"], saved, zoh=zoh, static_B=sB, static_C=sC)
    assert g["dB"].shape == B.shape and g["dC"].shape == C.shape
    ref = _oracle_static(inp, Bs, Cs, zoh)
    tol = U.TOL[io]
    assert U.rel_err(U.to_host(out), ref["out"]) <= tol["out"]
    for k in U.GRADS:
        assert U.rel_err(U.to_host(g[k]), ref[k]) <= tol["grad"], k
    # the recurrent step with the same parameters reproduces the first outputs of the scan
    h = torch.zeros((batch, D, N), dtype=torch.float32, device="cuda")
    outs = []
    for t in range(3):
        Bt = B if sB else dev["B"][:, t].contiguous()
        Ct = C if sC else dev["C"][:, t].contiguous()
        outs.append(K.ssm_step(dev["x"][:, t].contiguous(), dev["delta"][:, t].contiguous(), dev["A"], Bt, Ct,
                               dev["D_skip"], dev["z"][:, t].contiguous(), h, zoh=zoh, static_B=sB, static_C=sC))
    got = np.stack([U.to_host(o) for o in outs], axis=1)
    assert U.rel_err(got, ref["out"][:, :3]) <= tol["out"] * max(1.0, np.abs(ref["out"]).max() / np.abs(ref["out"][:, :3]).max())
