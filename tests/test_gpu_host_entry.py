"""ssm_scan_fwd_bwd_host: the forward + backward call that takes HOST buffers and pipelines copies with compute.
Its results must equal those of the device calls (bit for bit where no cross-batch sum is involved) and match the
oracle within the tolerances."""
import numpy as np
import pytest

from paper_2312_00752_b200 import synth
from tests import _gpu_util as U

pytestmark = pytest.mark.gpu


def _host_tensors(inp, io, pin=True):
    import torch
    dt = torch.float32 if io == "f32" else torch.bfloat16
    out = {}
    for k, v in inp.items():
        t = torch.from_numpy(np.ascontiguousarray(v))
        t = t if k in ("A", "D_skip") else t.to(dt)
        out[k] = t.pin_memory() if pin else t
    return out


@pytest.mark.parametrize("batch,L,D,N,io,pin", [
    (5, 300, 40, 16, "bf16", True),      # five pieces of one batch entry, tuned kernels
    (11, 64, 24, 8, "f32", True),        # six pieces, the last one smaller
    (1, 200, 16, 16, "bf16", True),      # a single piece
    (3, 130, 32, 16, "bf16", False),     # pageable host memory: same results, no overlap
    (3, 90, 24, 4, "bf16", True),        # fewer than 16 states: the widened problem inside every piece
])
def test_host_call_equals_device_calls_and_oracle(batch, L, D, N, io, pin):
    import torch
    from paper_2312_00752_b200 import binding as K
    cfg = synth.ScanConfig("host", 15, batch, L, D, N, io, 1e-3, 1e-1)
    inp = synth.make_inputs(cfg, seed=0)
    h = _host_tensors(inp, io, pin)
    res = K.ssm_scan_fwd_bwd_host(h["x"], h["delta"], h["A"], h["B"], h["C"], h["D_skip"], h["z"], h["dout"],
                                  device="cuda:0")
    torch.cuda.synchronize()
    got = {k: v.to(torch.float32).numpy() for k, v in res.items()}
    dev = U.to_device(inp, io)
    ref_dev = U.gpu_fwd_bwd(dev)
    for k in ("out", "dx", "ddelta", "dz", "dB", "dC"):
        assert np.array_equal(got[k], ref_dev[k]), k
    for k in ("dA", "dD"):      # summed over pieces instead of over batch entries: equal up to float32 rounding
        assert U.rel_err(got[k], ref_dev[k]) <= 2e-6, k
    U.assert_parity(got, U.oracle_fwd_bwd(inp), io, "host entry vs oracle")


def test_host_call_twice_on_one_arena_and_argument_errors():
    import torch
    from paper_2312_00752_b200 import binding as K
    cfg = synth.ScanConfig("host", 15, 4, 96, 32, 16, "bf16", 1e-3, 1e-1)
    h1 = _host_tensors(synth.make_inputs(cfg, seed=1), "bf16")
    h2 = _host_tensors(synth.make_inputs(cfg, seed=2), "bf16")
    prob = K.make_problem(h1["x"], h1["B"], True, True)
    arena = torch.empty(K.host_arena_bytes(prob), dtype=torch.uint8, device="cuda:0")
    call = lambda h, **kw: K.ssm_scan_fwd_bwd_host(h["x"], h["delta"], h["A"], h["B"], h["C"], h["D_skip"], h["z"],
                                                   h["dout"], device="cuda:0", **kw)
    # two calls back to back on the same arena and stream: the second must not disturb the first one's results
    r1 = call(h1, arena=arena)
    r2 = call(h2, arena=arena)
    torch.cuda.synchronize()
    s1 = call(h1)
    torch.cuda.synchronize()
    for k in r1:
        assert torch.equal(r1[k], s1[k]), k
    assert not torch.equal(r1["out"], r2["out"])
    # a short arena is refused before anything is enqueued
    with pytest.raises(K.SsmScanError):
        call(h1, arena=arena[: arena.numel() // 2])
    # device tensors are not host buffers
    with pytest.raises(K.SsmScanError):
        K.ssm_scan_fwd_bwd_host(h1["x"].cuda(), h1["delta"], h1["A"], h1["B"], h1["C"], h1["D_skip"], h1["z"],
                                h1["dout"], device="cuda:0")


def test_host_call_honours_the_zoh_flag():
    import torch
    from paper_2312_00752_b200 import binding as K
    cfg = synth.ScanConfig("host", 15, 3, 100, 32, 16, "bf16", 5e-2, 1.0)
    inp = synth.make_inputs(cfg, seed=4)
    h = _host_tensors(inp, "bf16")
    res = K.ssm_scan_fwd_bwd_host(h["x"], h["delta"], h["A"], h["B"], h["C"], h["D_skip"], h["z"], h["dout"],
                                  device="cuda:0", zoh=True)
    torch.cuda.synchronize()
    dev = U.to_device(inp, "bf16")
    args = (dev["x"], dev["delta"], dev["A"], dev["B"], dev["C"], dev["D_skip"], dev["z"])
    out, saved = K.ssm_scan_fwd(*args, save_states=True, zoh=True)
    g = K.ssm_scan_bwd(*args, dev["dout"], saved, zoh=True)
    assert torch.equal(res["out"], out.cpu()) and torch.equal(res["dx"], g["dx"].cpu())
    plain = K.ssm_scan_fwd(*args)
    assert not torch.equal(out, plain)
