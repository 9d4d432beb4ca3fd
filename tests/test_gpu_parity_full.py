"""GPU parity at the full benchmark sizes, in the launch configuration bench.py times.

Configs 1-3 (Mamba layer shapes) are compared with the oracle on every element.  Config 4 (524288 steps) is compared
on sampled channels for everything that is per channel (out, dx, ddelta, dz, dA, dD) and through two identities that
hold at any size for the channel-summed dB and dC; a shortened copy of config 4 is compared on every element.
"""
import numpy as np
import pytest

from paper_2312_00752_b200 import synth
from tests import _gpu_util as U

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("idx", [1, 2, 3])
def test_layer_shapes_every_element(idx):
    cfg = synth.CONFIGS[idx]
    inp = synth.make_inputs(cfg, seed=0)
    got = U.gpu_fwd_bwd(U.to_device(inp, cfg.io))
    ref = U.oracle_fwd_bwd(inp)
    errs = U.assert_parity(got, ref, cfg.io, cfg.name)
    U.assert_elementwise(got, ref, cfg.io, cfg.name)
    print(cfg.name, {k: f"{v:.2e}" for k, v in errs.items()})


def test_general_A_layer_shape():
    """A perturbed so that no row is an arithmetic progression: the general discretization path at full width."""
    cfg = synth.CONFIGS[1].scaled(batch=2)
    inp = synth.make_inputs(cfg, seed=0, perturb_A=0.05)
    got = U.gpu_fwd_bwd(U.to_device(inp, cfg.io))
    U.assert_parity(got, U.oracle_fwd_bwd(inp), cfg.io, "perturbed A")


def test_long_sequence_shortened_every_element():
    cfg = synth.CONFIGS[4].scaled(L=65536, D=128)
    inp = synth.make_inputs(cfg, seed=0)
    got = U.gpu_fwd_bwd(U.to_device(inp, cfg.io))
    errs = U.assert_parity(got, U.oracle_fwd_bwd(inp), cfg.io, "config 4 shortened")
    print({k: f"{v:.2e}" for k, v in errs.items()})


def test_long_sequence_full_length_every_element():
    """The long-sequence workload at its full length (524288 steps) on 128 channels: still split in time in both
    directions, and cheap enough for the oracle that every element of all eight outputs is compared, the channel-summed
    dB and dC included."""
    from paper_2312_00752_b200 import binding as K
    cfg = synth.CONFIGS[4].scaled(D=128)
    inp = synth.make_inputs(cfg, seed=0)
    dev = U.to_device(inp, cfg.io)
    prob = K.make_problem(dev["x"], dev["B"], True, True)
    assert K.plan(prob)["n_segments"] > 1
    got = U.gpu_fwd_bwd(dev)
    ref = U.oracle_fwd_bwd(inp)
    errs = U.assert_parity(got, ref, cfg.io, "config 4 at full length, 128 channels")
    assert set(errs) == {"out", "dx", "ddelta", "dz", "dB", "dC", "dA", "dD"}
    U.assert_elementwise(got, ref, cfg.io, "config 4 at full length, 128 channels")
    print({k: f"{v:.2e}" for k, v in errs.items()})


@pytest.mark.parametrize("N", [16, 1])
def test_fp32_long_memory(N):
    """fp32 io where the state remembers thousands of steps (step sizes log-uniform in [1e-4, 1e-2], 65536 steps): a
    relative error eps in the decay costs about eps / (delta |A|) in the state, so this is where an inexact
    exponential would show against the fp32 tolerances (1e-5 on out, 1e-4 on the gradients)."""
    cfg = synth.ScanConfig("fp32 long memory", 12, 1, 65536, 64, N, "f32", 1e-4, 1e-2)
    inp = synth.make_inputs(cfg, seed=3)
    got = U.gpu_fwd_bwd(U.to_device(inp, "f32"))
    ref = U.oracle_fwd_bwd(inp)
    errs = U.assert_parity(got, ref, "f32", cfg.name)
    print(N, {k: f"{v:.2e}" for k, v in errs.items()})


def test_long_sequence_full_size():
    import torch
    from paper_2312_00752_b200 import binding as K
    cfg = synth.CONFIGS[4]
    inp = synth.make_inputs(cfg, seed=0)
    dev = U.to_device(inp, cfg.io)
    plan = K.plan(K.make_problem(dev["x"], dev["B"], True, True))
    assert plan["n_segments"] > 1
    got = U.gpu_fwd_bwd(dev)

    # (1) sampled channels, every time step
    ch = np.array(sorted(set(np.linspace(0, cfg.D - 1, 40).astype(int)) | {0, 31, 32, 63, 64, cfg.D - 1}))
    sub = {k: (np.ascontiguousarray(v[:, :, ch]) if k in ("x", "delta", "z", "dout") else v) for k, v in inp.items()}
    sub["A"], sub["D_skip"] = inp["A"][ch], inp["D_skip"][ch]
    ref = U.oracle_fwd_bwd(sub)
    tol = U.TOL[cfg.io]
    # the denominators are taken over the sampled channels, a subset of the tensor: slightly stricter than the rule
    for k in ("out", "dx", "ddelta", "dz"):
        e = U.rel_err(got[k][:, :, ch], ref[k])
        assert e <= tol["out" if k == "out" else "grad"], (k, e)
    assert U.rel_err(got["dA"][ch], ref["dA"]) <= tol["grad"]
    assert U.rel_err(got["dD"][ch], ref["dD"]) <= tol["grad"]

    # (2) identities for the channel-summed gradients (double precision on the host, all channels, all steps):
    #     sum_n dB[t,n] B[t,n] = sum_d x[t,d] (dx[t,d] - ds[t,d] D_skip[d]),   ds = dout * silu(z)
    #     sum_n dC[t,n] C[t,n] = sum_d ds[t,d] (s[t,d] - D_skip[d] x[t,d]),    s = ungated forward output
    s_ungated = U.to_host(K.ssm_scan_fwd(dev["x"], dev["delta"], dev["A"], dev["B"], dev["C"], dev["D_skip"], None))
    x64, z64, g64 = (inp[k].astype(np.float64) for k in ("x", "z", "dout"))
    ds = g64 * z64 / (1.0 + np.exp(-z64))
    Dk = inp["D_skip"].astype(np.float64)
    lhs_B = (got["dB"].astype(np.float64) * inp["B"]).sum(-1)
    rhs_B = (x64 * (got["dx"].astype(np.float64) - ds * Dk)).sum(-1)
    lhs_C = (got["dC"].astype(np.float64) * inp["C"]).sum(-1)
    rhs_C = (ds * (s_ungated.astype(np.float64) - Dk * x64)).sum(-1)
    # both sides carry bf16 rounding of D-term sums; compare on the scale of the row sums
    assert np.abs(lhs_B - rhs_B).max() <= 3e-2 * np.abs(rhs_B).max()
    assert np.abs(lhs_C - rhs_C).max() <= 3e-2 * np.abs(rhs_C).max()
    del dev
    torch.cuda.empty_cache()


@pytest.mark.parametrize("general_A", [False, True])
def test_wide_ragged_shape_on_sampled_channels(general_A):
    """Batch 8, 70 steps (two tiles and a ragged one), 5000 channels (156 full groups of 32 and one of 8): 1256 chains,
    so the forward takes the two-stage ring with two warps per sub-partition and neighbouring warps share chains in
    both directions.  The oracle runs on sampled channels, the partial group included (dB / dC are sums over all
    channels and are checked by the other tests of this file)."""
    from oracle import ssm_oracle as O
    from paper_2312_00752_b200 import binding as K
    cfg = synth.ScanConfig("wide_ragged", 19, 8, 70, 5000, 16, "bf16", 1e-3, 1e-1)
    inp = synth.make_inputs(cfg, seed=0)
    if general_A:
        rng = np.random.default_rng(5)
        inp["A"] = (inp["A"] * (1 + 0.05 * rng.standard_normal(inp["A"].shape))).astype(np.float32)
    dev = U.to_device(inp, "bf16")
    got = U.gpu_fwd_bwd(dev, general_A=general_A)
    rng = np.random.default_rng(9)
    ch = np.array(sorted(set([0, 31, 32, 4991, 4992, 4995, 4999] + [int(c) for c in rng.integers(0, 5000, 40)])))
    sub = lambda k: np.ascontiguousarray(inp[k][:, :, ch])
    ref_out = O.scan_fwd(sub("x"), sub("delta"), inp["A"][ch], inp["B"], inp["C"], D_skip=inp["D_skip"][ch], z=sub("z"))
    ref = O.scan_bwd(sub("x"), sub("delta"), inp["A"][ch], inp["B"], inp["C"], inp["D_skip"][ch], sub("z"), sub("dout"))
    tol = U.TOL["bf16"]
    assert U.rel_err(got["out"][:, :, ch], ref_out) <= tol["out"]
    for k in ("dx", "ddelta", "dz"):
        assert U.rel_err(got[k][:, :, ch], ref[k]) <= tol["grad"], k
    for k in ("dA", "dD"):
        assert U.rel_err(got[k][ch], ref[k]) <= tol["grad"], k
    # run-to-run bit equality with shared chains
    again = U.gpu_fwd_bwd(dev, general_A=general_A)
    for k in ("out", "dx", "ddelta", "dz", "dB", "dC", "dA", "dD"):
        assert np.array_equal(got[k], again[k]), k
