"""Helpers shared by the GPU parity tests: host arrays -> device tensors, oracle calls, the error metric."""
import numpy as np

TOL = {  # max|v - ref| / max|ref| per tensor
    "f32": {"out": 1e-5, "grad": 1e-4},
    "bf16": {"out": 1e-2, "grad": 3e-2},
}
GRADS = ("dx", "ddelta", "dz", "dB", "dC", "dA", "dD")


def rel_err(got, ref) -> float:
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    denom = np.abs(ref).max()
    if denom == 0.0:
        return float(np.abs(got).max())
    return float(np.abs(got - ref).max() / denom)


def to_device(inp: dict, io: str, device="cuda:0") -> dict:
    """float32 host arrays holding io-representable values -> device tensors of the io dtype (exact)."""
    import torch
    dt = torch.float32 if io == "f32" else torch.bfloat16
    out = {}
    for k, v in inp.items():
        if v is None:
            out[k] = None
            continue
        t = torch.from_numpy(np.ascontiguousarray(v)).to(device)
        out[k] = t if k in ("A", "D_skip") else t.to(dt)
    return out


def to_host(t) -> np.ndarray:
    import torch
    return t.detach().to(torch.float32).cpu().numpy()


def gpu_fwd_bwd(dev: dict, use_saved=True, general_A=False):
    """Runs the CUDA forward (+ saved states) and backward through the binding; returns host float arrays."""
    from paper_2312_00752_b200 import binding as K
    args = (dev["x"], dev["delta"], dev["A"], dev["B"], dev["C"], dev.get("D_skip"), dev.get("z"))
    if use_saved:
        out, saved = K.ssm_scan_fwd(*args, save_states=True, general_A=general_A)
    else:
        out, saved = K.ssm_scan_fwd(*args, general_A=general_A), None
    res = {"out": to_host(out)}
    if dev.get("dout") is not None:
        g = K.ssm_scan_bwd(*args, dev["dout"], saved, general_A=general_A)
        ws = K.last_bwd_workspace(dev["x"].device)
        if ws is not None:
            K.check_status(K.make_problem(dev["x"], dev["B"], dev.get("z") is not None, dev.get("D_skip") is not None,
                                          False, general_A), ws)
        for k, v in g.items():
            res[k] = None if v is None else to_host(v)
    return res


def oracle_fwd_bwd(inp: dict, nthreads=0):
    from oracle import ssm_oracle as O
    res = {"out": O.scan_fwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], D_skip=inp.get("D_skip"),
                             z=inp.get("z"), nthreads=nthreads)}
    if inp.get("dout") is not None:
        res.update(O.scan_bwd(inp["x"], inp["delta"], inp["A"], inp["B"], inp["C"], inp.get("D_skip"), inp.get("z"),
                              inp["dout"], nthreads=nthreads))
    return res


def elementwise_excess(got, ref, io: str) -> float:
    """Largest |got - ref| in units of what a correctly rounded result of this size may be off by: a few units in the last
    place of the element itself (bf16: 2^-8 relative, f32: 2^-22) plus a floor tied to the rms of the tensor (sums of many
    terms cancel, so an element far below the rms carries the rounding of its larger terms).  The tolerances of the benchmark spec
    statement are relative to the largest element of a tensor, so a wrong value on a few small elements would pass them;
    this measure is per element.  A value of 1 means "at the bound"."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    ulp = 2.0 ** -8 if io == "bf16" else 2.0 ** -22
    rms = float(np.sqrt(np.mean(ref * ref)))
    bound = 4.0 * ulp * np.abs(ref) + 8.0 * ulp * rms
    if rms == 0.0:
        return float(np.abs(got).max())
    return float((np.abs(got - ref) / bound).max())


def assert_elementwise(got: dict, ref: dict, io: str, what="", keys=("out", "dx", "ddelta", "dz", "dB", "dC")):
    bad = {}
    for k in keys:
        if got.get(k) is None or k not in ref:
            continue
        e = elementwise_excess(got[k], ref[k], io)
        if not e <= 1.0:
            bad[k] = e
    assert not bad, f"{what}: elements beyond their own rounding bound (in units of the bound): {bad}"


def assert_parity(got: dict, ref: dict, io: str, what=""):
    errs = {}
    for k, r in ref.items():
        if got.get(k) is None:
            continue
        errs[k] = rel_err(got[k], r)
    bad = {k: e for k, e in errs.items() if not (e <= TOL[io]["out" if k == "out" else "grad"])}
    assert not bad, f"{what}: over tolerance {bad}; all errors {errs}"
    return errs
