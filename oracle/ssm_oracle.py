"""ctypes front end of the fp64 CPU oracle (oracle/ssm_oracle.c).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only tests/, the smoke check and the benchmark's CPU-baseline / reference arm
may import this module.  It imports nothing from the CUDA package and the CUDA package imports nothing from here.

`build()` compiles the C file with gcc into oracle/libssm_oracle.so (done on first use if the library is missing
or older than its source).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ssm_oracle.c")
_LIB = os.path.join(_HERE, "libssm_oracle.so")
_lock = threading.Lock()
_lib = None


class _Dims(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("L", ctypes.c_int32), ("D", ctypes.c_int32), ("N", ctypes.c_int32),
                ("has_z", ctypes.c_int32), ("has_dskip", ctypes.c_int32), ("zoh_bbar", ctypes.c_int32),
                ("softplus", ctypes.c_int32), ("nthreads", ctypes.c_int32)]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP, no fast-math: IEEE semantics are part of the definition)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-std=gnu11", "-fopenmp", "-fPIC", "-shared", "-fno-fast-math", "-ffp-contract=off",
               _SRC, "-o", tmp, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            _lib = ctypes.CDLL(build())
            _lib.ssm_oracle_threads_available.restype = ctypes.c_int
        return _lib


def threads_available() -> int:
    return int(_load().ssm_oracle_threads_available())


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _prep(arrs: dict, names, dtype):
    out = {}
    for k in names:
        v = arrs.get(k)
        out[k] = None if v is None else np.ascontiguousarray(v, dtype=dtype)
    return out


def _storage_dtype(x):
    return np.float32 if np.asarray(x).dtype == np.float32 else np.float64


def scan_fwd(x, delta, A, B, C, D_skip=None, z=None, h0=None, zoh=False, nthreads=0,
             return_pregate=False, return_h_last=False, delta_softplus=False, delta_bias=None):
    """Sequential fp64 selective scan (Algorithm 2 steps 5-6, Eq. 2, Eq. 4) + skip term + SiLU gate.

    x, delta, z: (batch, L, D); B, C: (batch, L, N); A: (D, N); D_skip: (D); h0: (batch, D, N) or None.
    Inputs stored as float32 are upcast exactly; anything else is taken as float64.  Returns float64 `out`
    (and, if asked, the pre-gate readout s and the final state h_L).  With delta_softplus the argument `delta` is
    the pre-activation and the step size is softplus(delta + delta_bias[d]) (Algorithm 2 step 4).
    """
    lib = _load()
    st = _storage_dtype(x)
    io = _prep(dict(x=x, delta=delta, B=B, C=C, z=z), ["x", "delta", "B", "C", "z"], st)
    batch, L, D = io["x"].shape
    N = io["B"].shape[-1]
    assert io["delta"].shape == (batch, L, D) and io["B"].shape == (batch, L, N) and io["C"].shape == (batch, L, N)
    A64 = np.ascontiguousarray(A, dtype=np.float64)
    assert A64.shape == (D, N)
    Dk = None if D_skip is None else np.ascontiguousarray(D_skip, dtype=np.float64)
    H0 = None if h0 is None else np.ascontiguousarray(h0, dtype=np.float64)
    out = np.empty((batch, L, D), dtype=np.float64)
    s_pre = np.empty((batch, L, D), dtype=np.float64) if return_pregate else None
    h_last = np.empty((batch, D, N), dtype=np.float64) if return_h_last else None
    bias = None if delta_bias is None else np.ascontiguousarray(delta_bias, dtype=np.float64)
    dims = _Dims(batch, L, D, N, int(z is not None), int(D_skip is not None), int(bool(zoh)), int(bool(delta_softplus)),
                 int(nthreads))
    fn = lib.ssm_oracle_fwd_f32 if st == np.float32 else lib.ssm_oracle_fwd_f64
    rc = fn(ctypes.byref(dims), _ptr(io["x"]), _ptr(io["delta"]), _ptr(A64), _ptr(io["B"]), _ptr(io["C"]),
            _ptr(Dk), _ptr(io["z"]), _ptr(H0), _ptr(bias), _ptr(out), _ptr(s_pre), _ptr(h_last))
    if rc != 0:
        raise RuntimeError(f"ssm_oracle_fwd failed with code {rc}")
    res = (out,)
    if return_pregate:
        res += (s_pre,)
    if return_h_last:
        res += (h_last,)
    return res[0] if len(res) == 1 else res


def scan_bwd(x, delta, A, B, C, D_skip, z, dout, nthreads=0, delta_softplus=False, delta_bias=None, zoh=False,
             h0=None, dh_last=None):
    """Analytic adjoint of scan_fwd for loss = sum(dout * out), sequential, fp64.

    Returns a dict with dx, ddelta, dz (batch, L, D); dB, dC (batch, L, N); dA (D, N); dD (D) -- all float64.
    dz is zero when z is None, dD is zero when D_skip is None.  With delta_softplus, `delta` is the pre-activation,
    ddelta its gradient, and the dict also holds ddelta_bias (D) = ddelta summed over batch and time.  `zoh` selects
    the zero-order-hold B-bar of Eq. 4 as in scan_fwd.  `h0` (batch, D, N) is the state before the first step and
    `dh_last` (batch, D, N) a gradient that reaches the last state from outside; the dict holds dh0 (batch, D, N).
    """
    lib = _load()
    st = _storage_dtype(x)
    io = _prep(dict(x=x, delta=delta, B=B, C=C, z=z, dout=dout), ["x", "delta", "B", "C", "z", "dout"], st)
    batch, L, D = io["x"].shape
    N = io["B"].shape[-1]
    A64 = np.ascontiguousarray(A, dtype=np.float64)
    Dk = None if D_skip is None else np.ascontiguousarray(D_skip, dtype=np.float64)
    g = {k: np.empty((batch, L, D), dtype=np.float64) for k in ("dx", "ddelta", "dz")}
    g["dB"] = np.empty((batch, L, N), dtype=np.float64)
    g["dC"] = np.empty((batch, L, N), dtype=np.float64)
    g["dA"] = np.empty((D, N), dtype=np.float64)
    g["dD"] = np.empty((D,), dtype=np.float64)
    g["ddelta_bias"] = np.empty((D,), dtype=np.float64)
    g["dh0"] = np.empty((batch, D, N), dtype=np.float64)
    H0 = None if h0 is None else np.ascontiguousarray(h0, dtype=np.float64)
    dHL = None if dh_last is None else np.ascontiguousarray(dh_last, dtype=np.float64)
    assert H0 is None or H0.shape == (batch, D, N)
    assert dHL is None or dHL.shape == (batch, D, N)
    bias = None if delta_bias is None else np.ascontiguousarray(delta_bias, dtype=np.float64)
    dims = _Dims(batch, L, D, N, int(z is not None), int(D_skip is not None), int(bool(zoh)), int(bool(delta_softplus)),
                 int(nthreads))
    fn = lib.ssm_oracle_bwd_f32 if st == np.float32 else lib.ssm_oracle_bwd_f64
    rc = fn(ctypes.byref(dims), _ptr(io["x"]), _ptr(io["delta"]), _ptr(A64), _ptr(io["B"]), _ptr(io["C"]), _ptr(Dk),
            _ptr(io["z"]), _ptr(io["dout"]), _ptr(bias), _ptr(H0), _ptr(dHL), _ptr(g["dx"]), _ptr(g["ddelta"]),
            _ptr(g["dA"]), _ptr(g["dB"]), _ptr(g["dC"]), _ptr(g["dD"]), _ptr(g["dz"]), _ptr(g["ddelta_bias"]),
            _ptr(g["dh0"]))
    if rc != 0:
        raise RuntimeError(f"ssm_oracle_bwd failed with code {rc}")
    return g
