"""Thin Python binding of the C ABI in include/ssm_scan.h (same names, argument marshalling only).

Every step of the selective scan runs in the CUDA kernels of libssm_scan.so; torch is used for device memory and
streams.  There is no CPU or eager fallback: if the library is missing or fails to load, importing a symbol raises.
"""
from __future__ import annotations

import ctypes
import os
import shutil

import torch

from . import build as _build

SSM_OK = 0
SSM_F32, SSM_BF16 = 0, 1
SSM_FLAG_HAS_Z, SSM_FLAG_HAS_DSKIP, SSM_FLAG_SAVE_STATES, SSM_FLAG_GENERAL_A, SSM_FLAG_TEST_WITHHOLD = 1, 2, 4, 8, 16
SSM_FLAG_DELTA_SOFTPLUS = 32
SSM_FLAG_ZOH_BBAR = 64
SSM_FLAG_STATIC_B, SSM_FLAG_STATIC_C = 256, 512
SSM_FLAG_COMPLEX = 1024

EXPORTED_SYMBOLS = (
    "ssm_scan_fwd_workspace_bytes", "ssm_scan_bwd_workspace_bytes", "ssm_scan_saved_state_bytes",
    "ssm_scan_checkpoint_steps", "ssm_scan_fwd", "ssm_scan_bwd", "ssm_status_string", "ssm_scan_plan", "ssm_scan_bwd_plan",
    "ssm_scan_fwd_static", "ssm_scan_check_status", "ssm_scan_fwd_state", "ssm_step",
    "ssm_scan_fwd_fused_dt", "ssm_scan_bwd_fused_dt", "ssm_scan_host_arena_bytes", "ssm_scan_fwd_bwd_host",
    "ssm_scan_bwd_state", "ssm_scan_bwd_fused_dt_state", "ssm_conv1d_fwd", "ssm_conv1d_bwd_workspace_bytes", "ssm_conv1d_bwd",
)
SSM_STATIC_SCRATCH_BYTES = 4 << 20


SSM_CONV_FLAG_SILU, SSM_CONV_FLAG_HAS_BIAS = 1, 2


class ssm_conv_problem_t(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("L", ctypes.c_int32), ("D", ctypes.c_int32), ("width", ctypes.c_int32),
                ("io_dtype", ctypes.c_int32), ("flags", ctypes.c_uint32)]


class ssm_problem_t(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("L", ctypes.c_int32), ("D", ctypes.c_int32), ("N", ctypes.c_int32),
                ("io_dtype", ctypes.c_int32), ("flags", ctypes.c_uint32)]


class SsmScanError(RuntimeError):
    pass


_lib = None


def library_path() -> str:
    return _build.LIB_PATH


def load_library() -> ctypes.CDLL:
    """dlopen libssm_scan.so (building it first if nvcc is present and the sources are newer)."""
    global _lib
    if _lib is not None:
        return _lib
    path = os.environ.get("SSM_SCAN_LIBRARY")    # e.g. the bounds-checking build (build.DEBUG_LIB_PATH)
    if path is None:
        if _build.is_stale() and shutil.which(os.environ.get("NVCC", "nvcc")):
            _build.build_library()
        path = _build.LIB_PATH
    if not os.path.exists(path):
        raise SsmScanError(f"{path} is missing and nvcc is not available to build it; there is no fallback path")
    lib = ctypes.CDLL(path)
    P = ctypes.POINTER(ssm_problem_t)
    vp, sz = ctypes.c_void_p, ctypes.c_size_t
    for name in ("ssm_scan_fwd_workspace_bytes", "ssm_scan_bwd_workspace_bytes", "ssm_scan_saved_state_bytes",
                 "ssm_scan_host_arena_bytes"):
        getattr(lib, name).restype = sz
        getattr(lib, name).argtypes = [P]
    lib.ssm_scan_checkpoint_steps.restype = ctypes.c_int32
    lib.ssm_scan_checkpoint_steps.argtypes = []
    lib.ssm_status_string.restype = ctypes.c_char_p
    lib.ssm_status_string.argtypes = [ctypes.c_int]
    lib.ssm_scan_plan.restype = ctypes.c_int
    lib.ssm_scan_plan.argtypes = [P] + [ctypes.POINTER(ctypes.c_int32)] * 4
    lib.ssm_scan_bwd_plan.restype = ctypes.c_int
    lib.ssm_scan_bwd_plan.argtypes = [P] + [ctypes.POINTER(ctypes.c_int32)] * 3
    lib.ssm_scan_fwd.restype = ctypes.c_int
    lib.ssm_scan_fwd.argtypes = [P] + [vp] * 9 + [vp, sz, vp]
    lib.ssm_scan_bwd.restype = ctypes.c_int
    lib.ssm_scan_bwd.argtypes = [P] + [vp] * 16 + [vp, sz, vp]
    CP = ctypes.POINTER(ssm_conv_problem_t)
    lib.ssm_conv1d_fwd.restype = ctypes.c_int
    lib.ssm_conv1d_fwd.argtypes = [CP] + [vp] * 5 + [vp]
    lib.ssm_conv1d_bwd_workspace_bytes.restype = sz
    lib.ssm_conv1d_bwd_workspace_bytes.argtypes = [CP]
    lib.ssm_conv1d_bwd.restype = ctypes.c_int
    lib.ssm_conv1d_bwd.argtypes = [CP] + [vp] * 9 + [vp, sz, vp]
    lib.ssm_scan_bwd_fused_dt_state.restype = ctypes.c_int
    lib.ssm_scan_bwd_fused_dt_state.argtypes = [P] + [vp] * 21 + [vp, sz, vp]
    lib.ssm_scan_bwd_state.restype = ctypes.c_int
    lib.ssm_scan_bwd_state.argtypes = [P] + [vp] * 19 + [vp, sz, vp]
    lib.ssm_scan_fwd_state.restype = ctypes.c_int
    lib.ssm_scan_fwd_state.argtypes = [P] + [vp] * 11 + [vp, sz, vp]
    lib.ssm_scan_fwd_fused_dt.restype = ctypes.c_int
    lib.ssm_scan_fwd_fused_dt.argtypes = [P] + [vp] * 12 + [vp, sz, vp]
    lib.ssm_scan_bwd_fused_dt.restype = ctypes.c_int
    lib.ssm_scan_bwd_fused_dt.argtypes = [P] + [vp] * 18 + [vp, sz, vp]
    lib.ssm_step.restype = ctypes.c_int
    lib.ssm_step.argtypes = [P] + [vp] * 10
    lib.ssm_scan_check_status.restype = ctypes.c_int
    lib.ssm_scan_check_status.argtypes = [P, vp, vp]
    lib.ssm_scan_fwd_bwd_host.restype = ctypes.c_int
    lib.ssm_scan_fwd_bwd_host.argtypes = [P] + [vp] * 16 + [vp, sz, vp]
    lib.ssm_scan_fwd_static.restype = ctypes.c_int
    lib.ssm_scan_fwd_static.argtypes = [P] + [vp] * 9 + [vp]
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().ssm_status_string(int(code)).decode()


def _check(code: int, what: str) -> None:
    if code != SSM_OK:
        raise SsmScanError(f"{what}: {status_string(code)}")


def _io_dtype(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return SSM_F32
    if t.dtype == torch.bfloat16:
        return SSM_BF16
    raise SsmScanError(f"io dtype must be float32 or bfloat16, got {t.dtype}")


def make_problem(x: torch.Tensor, B: torch.Tensor, has_z: bool, has_dskip: bool, save_states: bool = False,
                 general_A: bool = False, zoh: bool = False, static_B: bool = False,
                 static_C: bool = False, complex_state: bool = False) -> ssm_problem_t:
    """complex_state: B is (batch, L, N, 2), interleaved (re, im) pairs (SSM_FLAG_COMPLEX)."""
    batch, L, D = x.shape
    flags = (SSM_FLAG_HAS_Z if has_z else 0) | (SSM_FLAG_HAS_DSKIP if has_dskip else 0) \
        | (SSM_FLAG_SAVE_STATES if save_states else 0) | (SSM_FLAG_GENERAL_A if general_A else 0) \
        | (SSM_FLAG_ZOH_BBAR if zoh else 0) | (SSM_FLAG_STATIC_B if static_B else 0) \
        | (SSM_FLAG_STATIC_C if static_C else 0) | (SSM_FLAG_COMPLEX if complex_state else 0)
    return ssm_problem_t(batch, L, D, B.shape[-2] if complex_state else B.shape[-1], _io_dtype(x), flags)


def _dev_ptr(t, name, shape=None, dtype=None):
    if t is None:
        return None
    if not t.is_cuda:
        raise SsmScanError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise SsmScanError(f"{name} must be contiguous")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise SsmScanError(f"{name} has shape {tuple(t.shape)}, expected {tuple(shape)}")
    if dtype is not None and t.dtype != dtype:
        raise SsmScanError(f"{name} has dtype {t.dtype}, expected {dtype}")
    return ctypes.c_void_p(t.data_ptr())


_workspaces: dict = {}


def _workspace(nbytes: int, device, stream_ptr: int) -> torch.Tensor | None:
    """Grow-only scratch buffer per (device, stream): calls on different streams never share scratch memory."""
    if nbytes == 0:
        return None
    key = (str(device), int(stream_ptr))
    ws = _workspaces.get(key)
    if ws is None or ws.numel() < nbytes:
        if ws is not None:
            # kernels already enqueued on that stream may still use the old buffer: the caching allocator must not hand
            # its memory to other work before they are done
            ws.record_stream(torch.cuda.ExternalStream(int(stream_ptr), device=device))
        ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
        _workspaces[key] = ws
    return ws


def plan(problem: ssm_problem_t) -> dict:
    lib = load_library()
    v = [ctypes.c_int32() for _ in range(4)]
    _check(lib.ssm_scan_plan(ctypes.byref(problem), *[ctypes.byref(c) for c in v]), "ssm_scan_plan")
    return dict(zip(("n_segments", "segment_steps", "channels_per_block", "states_per_thread"), [c.value for c in v]))


def bwd_plan(problem: ssm_problem_t) -> dict:
    lib = load_library()
    v = [ctypes.c_int32() for _ in range(3)]
    _check(lib.ssm_scan_bwd_plan(ctypes.byref(problem), *[ctypes.byref(c) for c in v]), "ssm_scan_bwd_plan")
    return dict(zip(("n_segments", "segment_steps", "channels_per_group"), [c.value for c in v]))


def checkpoint_steps() -> int:
    return int(load_library().ssm_scan_checkpoint_steps())


def fwd_workspace_bytes(problem: ssm_problem_t) -> int:
    return int(load_library().ssm_scan_fwd_workspace_bytes(ctypes.byref(problem)))


def bwd_workspace_bytes(problem: ssm_problem_t) -> int:
    return int(load_library().ssm_scan_bwd_workspace_bytes(ctypes.byref(problem)))


def saved_state_bytes(problem: ssm_problem_t) -> int:
    return int(load_library().ssm_scan_saved_state_bytes(ctypes.byref(problem)))


def ssm_scan_fwd(x, delta, A, B, C, D_skip=None, z=None, *, save_states=False, general_A=False, zoh=False, out=None,
                 saved_states=None, workspace=None, stream=None, h0=None, h_last=None, static_B=False, static_C=False,
                 complex_state=False):
    """out = selective_scan(x, delta, A, B, C) (+ D_skip * x) (* silu(z)); see include/ssm_scan.h.

    complex_state=True (SSM_FLAG_COMPLEX): A is float32 (D, N, 2), B and C are io dtype (batch, L, N, 2), h0 / h_last
    float32 (batch, D, N, 2), all interleaved (re, im) pairs (torch.view_as_real of a complex tensor).

    x, delta, z: (batch, L, D) io dtype; B, C: (batch, L, N) io dtype; A: (D, N) float32; D_skip: (D) float32.
    Returns `out`, or `(out, saved_states)` with save_states=True.  Enqueues on `stream` (default: torch's current
    stream) and does not synchronise.  zoh=True selects the zero-order-hold B-bar of Eq. 4.  `h0` (batch, D, N) float32 is the state before the first step (default zero);
    if a float32 tensor `h_last` (batch, D, N) is passed it receives the state after the last step
    (ssm_scan_fwd_state).
    """
    lib = load_library()
    prob = make_problem(x, B, z is not None, D_skip is not None, save_states, general_A, zoh, static_B, static_C,
                        complex_state)
    batch, L, D, N = prob.batch, prob.L, prob.D, prob.N
    io = x.dtype
    c2 = (2,) if complex_state else ()
    bshape, bdt = ((D, N), torch.float32) if static_B else ((batch, L, N) + c2, io)   # static: a parameter like A
    cshape, cdt = ((D, N), torch.float32) if static_C else ((batch, L, N) + c2, io)
    if out is None:
        out = torch.empty_like(x)
    if save_states and saved_states is None:
        saved_states = torch.empty(saved_state_bytes(prob) // 4, dtype=torch.float32, device=x.device)
    stream_ptr = (stream if stream is not None else torch.cuda.current_stream(x.device)).cuda_stream
    need = fwd_workspace_bytes(prob)
    ws = workspace if workspace is not None else _workspace(need, x.device, stream_ptr)
    code = lib.ssm_scan_fwd_state(
        ctypes.byref(prob), _dev_ptr(x, "x", (batch, L, D), io), _dev_ptr(delta, "delta", (batch, L, D), io),
        _dev_ptr(A, "A", (D, N) + c2, torch.float32), _dev_ptr(B, "B", bshape, bdt),
        _dev_ptr(C, "C", cshape, cdt), _dev_ptr(D_skip, "D_skip", (D,), torch.float32),
        _dev_ptr(z, "z", (batch, L, D), io), _dev_ptr(h0, "h0", (batch, D, N) + c2, torch.float32),
        _dev_ptr(out, "out", (batch, L, D), io), _dev_ptr(h_last, "h_last", (batch, D, N) + c2, torch.float32),
        _dev_ptr(saved_states if save_states else None, "saved_states"),
        _dev_ptr(ws, "workspace"), ctypes.c_size_t(0 if ws is None else ws.numel() * ws.element_size()),
        ctypes.c_void_p(stream_ptr))
    _check(code, "ssm_scan_fwd_state")
    return (out, saved_states) if save_states else out


def ssm_scan_fwd_fused_dt(x, delta_pre, delta_bias, A, B, C, D_skip=None, z=None, *, softplus=True, save_states=False,
                          out=None, saved_states=None, stream=None, h0=None, h_last=None, zoh=False, static_B=False,
                          static_C=False):
    """Forward with the step-size activation fused: delta = softplus(delta_pre + delta_bias) (or the plain sum with
    softplus=False), in float32.  Otherwise as ssm_scan_fwd (static_B / static_C: B / C float32 (D, N))."""
    lib = load_library()
    prob = make_problem(x, B, z is not None, D_skip is not None, save_states, False, zoh, static_B, static_C)
    if softplus:
        prob.flags |= SSM_FLAG_DELTA_SOFTPLUS
    batch, L, D, N = prob.batch, prob.L, prob.D, prob.N
    io = x.dtype
    bshape, bdt = ((D, N), torch.float32) if static_B else ((batch, L, N), io)
    cshape, cdt = ((D, N), torch.float32) if static_C else ((batch, L, N), io)
    if out is None:
        out = torch.empty_like(x)
    if save_states and saved_states is None:
        saved_states = torch.empty(saved_state_bytes(prob) // 4, dtype=torch.float32, device=x.device)
    stream_ptr = (stream if stream is not None else torch.cuda.current_stream(x.device)).cuda_stream
    ws = _workspace(fwd_workspace_bytes(prob), x.device, stream_ptr)
    code = lib.ssm_scan_fwd_fused_dt(
        ctypes.byref(prob), _dev_ptr(x, "x", (batch, L, D), io), _dev_ptr(delta_pre, "delta_pre", (batch, L, D), io),
        _dev_ptr(delta_bias, "delta_bias", (D,), torch.float32), _dev_ptr(A, "A", (D, N), torch.float32),
        _dev_ptr(B, "B", bshape, bdt), _dev_ptr(C, "C", cshape, cdt),
        _dev_ptr(D_skip, "D_skip", (D,), torch.float32), _dev_ptr(z, "z", (batch, L, D), io),
        _dev_ptr(h0, "h0", (batch, D, N), torch.float32), _dev_ptr(out, "out", (batch, L, D), io),
        _dev_ptr(h_last, "h_last", (batch, D, N), torch.float32),
        _dev_ptr(saved_states if save_states else None, "saved_states"),
        _dev_ptr(ws, "workspace"), ctypes.c_size_t(0 if ws is None else ws.numel() * ws.element_size()),
        ctypes.c_void_p(stream_ptr))
    _check(code, "ssm_scan_fwd_fused_dt")
    return (out, saved_states) if save_states else out


def ssm_scan_bwd_fused_dt(x, delta_pre, delta_bias, A, B, C, D_skip, z, dout, saved_states=None, *, softplus=True,
                          stream=None, zoh=False, h0=None, dh_last=None, want_dh0=False, static_B=False,
                          static_C=False):
    """Backward of ssm_scan_fwd_fused_dt.  Returns the dict of ssm_scan_bwd with `ddelta` the gradient of delta_pre
    and an extra `ddelta_bias` (D,) float32.  h0, dh_last, want_dh0 as in ssm_scan_bwd (ssm_scan_bwd_fused_dt_state)."""
    lib = load_library()
    prob = make_problem(x, B, z is not None, D_skip is not None, False, False, zoh, static_B, static_C)
    if softplus:
        prob.flags |= SSM_FLAG_DELTA_SOFTPLUS
    batch, L, D, N = prob.batch, prob.L, prob.D, prob.N
    io = x.dtype
    bshape, bdt = ((D, N), torch.float32) if static_B else ((batch, L, N), io)
    cshape, cdt = ((D, N), torch.float32) if static_C else ((batch, L, N), io)
    o = {"dx": torch.empty_like(x), "ddelta": torch.empty_like(x),
         "ddelta_bias": torch.empty((D,), dtype=torch.float32, device=x.device),
         "dA": torch.empty((D, N), dtype=torch.float32, device=x.device), "dB": torch.empty_like(B),
         "dC": torch.empty_like(C),
         "dD": torch.empty((D,), dtype=torch.float32, device=x.device) if D_skip is not None else None,
         "dz": torch.empty_like(x) if z is not None else None}
    stream_ptr = (stream if stream is not None else torch.cuda.current_stream(x.device)).cuda_stream
    ws = _workspace(bwd_workspace_bytes(prob), x.device, stream_ptr)
    if h0 is not None or dh_last is not None or want_dh0:
        f32 = torch.float32
        if want_dh0:
            o["dh0"] = torch.empty((batch, D, N), dtype=f32, device=x.device)
        code = lib.ssm_scan_bwd_fused_dt_state(
            ctypes.byref(prob), _dev_ptr(x, "x", (batch, L, D), io), _dev_ptr(delta_pre, "delta_pre", (batch, L, D), io),
            _dev_ptr(delta_bias, "delta_bias", (D,), f32), _dev_ptr(A, "A", (D, N), f32),
            _dev_ptr(B, "B", bshape, bdt), _dev_ptr(C, "C", cshape, cdt), _dev_ptr(D_skip, "D_skip", (D,), f32),
            _dev_ptr(z, "z", (batch, L, D), io), _dev_ptr(dout, "dout", (batch, L, D), io),
            _dev_ptr(h0, "h0", (batch, D, N), f32), _dev_ptr(dh_last, "dh_last", (batch, D, N), f32),
            _dev_ptr(saved_states, "saved_states"), _dev_ptr(o["dx"], "dx"), _dev_ptr(o["ddelta"], "ddelta"),
            _dev_ptr(o["ddelta_bias"], "ddelta_bias"), _dev_ptr(o["dA"], "dA"), _dev_ptr(o["dB"], "dB"),
            _dev_ptr(o["dC"], "dC"), _dev_ptr(o["dD"], "dD"), _dev_ptr(o["dz"], "dz"), _dev_ptr(o.get("dh0"), "dh0"),
            _dev_ptr(ws, "workspace"), ctypes.c_size_t(0 if ws is None else ws.numel() * ws.element_size()),
            ctypes.c_void_p(stream_ptr))
        _check(code, "ssm_scan_bwd_fused_dt_state")
        return o
    code = lib.ssm_scan_bwd_fused_dt(
        ctypes.byref(prob), _dev_ptr(x, "x", (batch, L, D), io), _dev_ptr(delta_pre, "delta_pre", (batch, L, D), io),
        _dev_ptr(delta_bias, "delta_bias", (D,), torch.float32), _dev_ptr(A, "A", (D, N), torch.float32),
        _dev_ptr(B, "B", bshape, bdt), _dev_ptr(C, "C", cshape, cdt),
        _dev_ptr(D_skip, "D_skip", (D,), torch.float32), _dev_ptr(z, "z", (batch, L, D), io),
        _dev_ptr(dout, "dout", (batch, L, D), io), _dev_ptr(saved_states, "saved_states"),
        _dev_ptr(o["dx"], "dx"), _dev_ptr(o["ddelta"], "ddelta"), _dev_ptr(o["ddelta_bias"], "ddelta_bias"),
        _dev_ptr(o["dA"], "dA"), _dev_ptr(o["dB"], "dB"), _dev_ptr(o["dC"], "dC"), _dev_ptr(o["dD"], "dD"),
        _dev_ptr(o["dz"], "dz"),
        _dev_ptr(ws, "workspace"), ctypes.c_size_t(0 if ws is None else ws.numel() * ws.element_size()),
        ctypes.c_void_p(stream_ptr))
    _check(code, "ssm_scan_bwd_fused_dt")
    return o


def ssm_step(x, delta, A, B, C, D_skip, z, h, *, zoh=False, out=None, stream=None, static_B=False, static_C=False,
             complex_state=False):
    """One recurrent step: x, delta, z (batch, D), B, C (batch, N) io dtype; h (batch, D, N) float32 is updated in
    place.  Returns out (batch, D).  complex_state: A (D, N, 2), B, C (batch, N, 2), h (batch, D, N, 2)."""
    lib = load_library()
    batch, D = x.shape
    N = B.shape[-2] if complex_state else B.shape[-1]
    c2 = (2,) if complex_state else ()
    prob = ssm_problem_t(batch, 1, D, N, _io_dtype(x),
                         (SSM_FLAG_HAS_Z if z is not None else 0) | (SSM_FLAG_HAS_DSKIP if D_skip is not None else 0)
                         | (SSM_FLAG_ZOH_BBAR if zoh else 0) | (SSM_FLAG_STATIC_B if static_B else 0)
                         | (SSM_FLAG_STATIC_C if static_C else 0) | (SSM_FLAG_COMPLEX if complex_state else 0))
    io = x.dtype
    if out is None:
        out = torch.empty_like(x)
    stream_ptr = (stream if stream is not None else torch.cuda.current_stream(x.device)).cuda_stream
    code = lib.ssm_step(
        ctypes.byref(prob), _dev_ptr(x, "x", (batch, D), io), _dev_ptr(delta, "delta", (batch, D), io),
        _dev_ptr(A, "A", (D, N) + c2, torch.float32),
        _dev_ptr(B, "B", (D, N) if static_B else (batch, N) + c2, torch.float32 if static_B else io),
        _dev_ptr(C, "C", (D, N) if static_C else (batch, N) + c2, torch.float32 if static_C else io),
        _dev_ptr(D_skip, "D_skip", (D,), torch.float32), _dev_ptr(z, "z", (batch, D), io),
        _dev_ptr(h, "h", (batch, D, N) + c2, torch.float32), _dev_ptr(out, "out", (batch, D), io),
        ctypes.c_void_p(stream_ptr))
    _check(code, "ssm_step")
    return out


def check_status(problem: ssm_problem_t, workspace: torch.Tensor, stream=None) -> None:
    """Synchronises the stream and raises SsmScanError if the last backward call on `workspace` gave up a wait."""
    stream_ptr = (stream if stream is not None else torch.cuda.current_stream(workspace.device)).cuda_stream
    _check(load_library().ssm_scan_check_status(ctypes.byref(problem), ctypes.c_void_p(workspace.data_ptr()),
                                                ctypes.c_void_p(stream_ptr)), "ssm_scan_check_status")


def last_bwd_workspace(device, stream=None):
    """The cached workspace tensor the binding used for calls on (device, stream), or None."""
    stream_ptr = (stream if stream is not None else torch.cuda.current_stream(device)).cuda_stream
    return _workspaces.get((str(device), int(stream_ptr)))


def ssm_scan_fwd_static(x, delta, A, B, C, D_skip=None, z=None, *, save_states=False, general_A=False, out=None,
                        saved_states=None, stream=None):
    """ssm_scan_fwd for callers that may not allocate: no workspace argument, and this wrapper allocates none either
    when `out` (and `saved_states`, if asked for) are passed in.  The scratch memory is the fixed array inside the
    library (SSM_STATIC_SCRATCH_BYTES); a problem that needs more raises SsmScanError (SSM_ERR_WORKSPACE).  Calls that
    may overlap on the GPU must be ordered by the caller, because they share that array."""
    lib = load_library()
    prob = make_problem(x, B, z is not None, D_skip is not None, save_states, general_A)
    batch, L, D, N = prob.batch, prob.L, prob.D, prob.N
    io = x.dtype
    if out is None:
        out = torch.empty_like(x)
    if save_states and saved_states is None:
        saved_states = torch.empty(saved_state_bytes(prob) // 4, dtype=torch.float32, device=x.device)
    stream_ptr = (stream if stream is not None else torch.cuda.current_stream(x.device)).cuda_stream
    code = lib.ssm_scan_fwd_static(
        ctypes.byref(prob), _dev_ptr(x, "x", (batch, L, D), io), _dev_ptr(delta, "delta", (batch, L, D), io),
        _dev_ptr(A, "A", (D, N), torch.float32), _dev_ptr(B, "B", (batch, L, N), io),
        _dev_ptr(C, "C", (batch, L, N), io), _dev_ptr(D_skip, "D_skip", (D,), torch.float32),
        _dev_ptr(z, "z", (batch, L, D), io), _dev_ptr(out, "out", (batch, L, D), io),
        _dev_ptr(saved_states if save_states else None, "saved_states"), ctypes.c_void_p(stream_ptr))
    _check(code, "ssm_scan_fwd_static")
    return (out, saved_states) if save_states else out


def ssm_scan_bwd(x, delta, A, B, C, D_skip, z, dout, saved_states=None, *, general_A=False, zoh=False, workspace=None,
                 stream=None, outputs=None, extra_flags=0, h0=None, dh_last=None, want_dh0=False, static_B=False,
                 static_C=False, complex_state=False):
    """Gradients of sum(dout * out) w.r.t. x, delta, A, B, C, D_skip, z; see include/ssm_scan.h.

    Returns a dict with dx, ddelta, dz (io dtype, (batch, L, D)); dB, dC (io dtype, (batch, L, N)); dA (float32, (D, N));
    dD (float32, (D)).  dz / dD are None when z / D_skip is None.  `outputs` may pass preallocated tensors.
    With h0, dh_last or want_dh0 the call goes through ssm_scan_bwd_state: h0 / dh_last (batch, D, N) float32 are the
    state before the first step and the gradient arriving at the state after the last step, and the dict also holds
    dh0 (batch, D, N) float32.  With static_B / static_C, B / C is a float32 (D, N) parameter and dB / dC is its
    float32 (D, N) gradient.  With complex_state every complex array (A, B, C, their gradients, h0, dh_last, dh0) has a
    trailing dimension 2 of (re, im) pairs, and a gradient pair is (dL/dRe, dL/dIm).
    """
    lib = load_library()
    prob = make_problem(x, B, z is not None, D_skip is not None, False, general_A, zoh, static_B, static_C, complex_state)
    prob.flags |= int(extra_flags)
    batch, L, D, N = prob.batch, prob.L, prob.D, prob.N
    io = x.dtype
    c2 = (2,) if complex_state else ()
    bshape, bdt = ((D, N), torch.float32) if static_B else ((batch, L, N) + c2, io)
    cshape, cdt = ((D, N), torch.float32) if static_C else ((batch, L, N) + c2, io)
    o = dict(outputs or {})
    o.setdefault("dx", torch.empty_like(x))
    o.setdefault("ddelta", torch.empty_like(x))
    o.setdefault("dA", torch.empty((D, N) + c2, dtype=torch.float32, device=x.device))
    o.setdefault("dB", torch.empty_like(B))
    o.setdefault("dC", torch.empty_like(C))
    if D_skip is not None:
        o.setdefault("dD", torch.empty((D,), dtype=torch.float32, device=x.device))
    else:
        o["dD"] = None
    if z is not None:
        o.setdefault("dz", torch.empty_like(x))
    else:
        o["dz"] = None
    stream_ptr = (stream if stream is not None else torch.cuda.current_stream(x.device)).cuda_stream
    need = bwd_workspace_bytes(prob)
    ws = workspace if workspace is not None else _workspace(need, x.device, stream_ptr)
    if h0 is not None or dh_last is not None or want_dh0:
        f32 = torch.float32
        if want_dh0:
            o.setdefault("dh0", torch.empty((batch, D, N) + c2, dtype=f32, device=x.device))
        code = lib.ssm_scan_bwd_state(
            ctypes.byref(prob), _dev_ptr(x, "x", (batch, L, D), io), _dev_ptr(delta, "delta", (batch, L, D), io),
            _dev_ptr(A, "A", (D, N) + c2, f32), _dev_ptr(B, "B", bshape, bdt), _dev_ptr(C, "C", cshape, cdt),
            _dev_ptr(D_skip, "D_skip", (D,), f32), _dev_ptr(z, "z", (batch, L, D), io),
            _dev_ptr(dout, "dout", (batch, L, D), io), _dev_ptr(h0, "h0", (batch, D, N) + c2, f32),
            _dev_ptr(dh_last, "dh_last", (batch, D, N) + c2, f32), _dev_ptr(saved_states, "saved_states"),
            _dev_ptr(o["dx"], "dx", (batch, L, D), io), _dev_ptr(o["ddelta"], "ddelta", (batch, L, D), io),
            _dev_ptr(o["dA"], "dA", (D, N) + c2, f32), _dev_ptr(o["dB"], "dB", bshape, bdt),
            _dev_ptr(o["dC"], "dC", cshape, cdt), _dev_ptr(o["dD"], "dD", (D,), f32),
            _dev_ptr(o["dz"], "dz", (batch, L, D), io), _dev_ptr(o.get("dh0"), "dh0", (batch, D, N) + c2, f32),
            _dev_ptr(ws, "workspace"), ctypes.c_size_t(0 if ws is None else ws.numel() * ws.element_size()),
            ctypes.c_void_p(stream_ptr))
        _check(code, "ssm_scan_bwd_state")
        return o
    code = lib.ssm_scan_bwd(
        ctypes.byref(prob), _dev_ptr(x, "x", (batch, L, D), io), _dev_ptr(delta, "delta", (batch, L, D), io),
        _dev_ptr(A, "A", (D, N) + c2, torch.float32), _dev_ptr(B, "B", bshape, bdt),
        _dev_ptr(C, "C", cshape, cdt), _dev_ptr(D_skip, "D_skip", (D,), torch.float32),
        _dev_ptr(z, "z", (batch, L, D), io), _dev_ptr(dout, "dout", (batch, L, D), io),
        _dev_ptr(saved_states, "saved_states"),
        _dev_ptr(o["dx"], "dx", (batch, L, D), io), _dev_ptr(o["ddelta"], "ddelta", (batch, L, D), io),
        _dev_ptr(o["dA"], "dA", (D, N) + c2, torch.float32), _dev_ptr(o["dB"], "dB", bshape, bdt),
        _dev_ptr(o["dC"], "dC", cshape, cdt), _dev_ptr(o["dD"], "dD", (D,), torch.float32),
        _dev_ptr(o["dz"], "dz", (batch, L, D), io),
        _dev_ptr(ws, "workspace"), ctypes.c_size_t(0 if ws is None else ws.numel() * ws.element_size()),
        ctypes.c_void_p(stream_ptr))
    _check(code, "ssm_scan_bwd")
    return o


def _host_ptr(t, name, shape, dtype):
    if t is None:
        return None
    if t.is_cuda:
        raise SsmScanError(f"{name} must be a host tensor")
    if not t.is_contiguous() or tuple(t.shape) != tuple(shape) or t.dtype != dtype:
        raise SsmScanError(f"{name}: expected a contiguous host tensor of shape {tuple(shape)} and dtype {dtype}")
    return ctypes.c_void_p(t.data_ptr())


def host_arena_bytes(problem: ssm_problem_t) -> int:
    return int(load_library().ssm_scan_host_arena_bytes(ctypes.byref(problem)))


def ssm_scan_fwd_bwd_host(x, delta, A, B, C, D_skip, z, dout, *, device, arena=None, outputs=None, stream=None,
                          general_A=False, zoh=False):
    """Forward + backward of host tensors (page-locked for the copies to overlap), copies included
    (ssm_scan_fwd_bwd_host).  Returns a dict of host tensors out, dx, ddelta, dz, dB, dC, dA, dD; pass `outputs` to
    reuse page-locked result tensors and `arena` (a uint8 CUDA tensor of host_arena_bytes) to reuse the device scratch.
    Enqueues on `stream` (default: torch's current stream of `device`) and does not synchronise."""
    lib = load_library()
    device = torch.device(device)
    batch, L, D = x.shape
    N = B.shape[-1]
    prob = make_problem(x, B, z is not None, D_skip is not None, False, general_A, zoh)
    io = x.dtype
    need = host_arena_bytes(prob)
    if arena is None:
        arena = torch.empty(need, dtype=torch.uint8, device=device)
    if outputs is None:
        mk = lambda shape, dt: torch.empty(shape, dtype=dt).pin_memory()
        outputs = {"out": mk((batch, L, D), io), "dx": mk((batch, L, D), io), "ddelta": mk((batch, L, D), io),
                   "dz": mk((batch, L, D), io) if z is not None else None, "dB": mk((batch, L, N), io),
                   "dC": mk((batch, L, N), io), "dA": mk((D, N), torch.float32),
                   "dD": mk((D,), torch.float32) if D_skip is not None else None}
    stream_ptr = (stream if stream is not None else torch.cuda.current_stream(device)).cuda_stream
    f32 = torch.float32
    with torch.cuda.device(device):
        code = lib.ssm_scan_fwd_bwd_host(
            ctypes.byref(prob), _host_ptr(x, "x", (batch, L, D), io), _host_ptr(delta, "delta", (batch, L, D), io),
            _host_ptr(A, "A", (D, N), f32), _host_ptr(B, "B", (batch, L, N), io), _host_ptr(C, "C", (batch, L, N), io),
            _host_ptr(D_skip, "D_skip", (D,), f32), _host_ptr(z, "z", (batch, L, D), io),
            _host_ptr(dout, "dout", (batch, L, D), io),
            _host_ptr(outputs["out"], "out", (batch, L, D), io), _host_ptr(outputs["dx"], "dx", (batch, L, D), io),
            _host_ptr(outputs["ddelta"], "ddelta", (batch, L, D), io), _host_ptr(outputs["dA"], "dA", (D, N), f32),
            _host_ptr(outputs["dB"], "dB", (batch, L, N), io), _host_ptr(outputs["dC"], "dC", (batch, L, N), io),
            _host_ptr(outputs.get("dD"), "dD", (D,), f32), _host_ptr(outputs.get("dz"), "dz", (batch, L, D), io),
            _dev_ptr(arena, "device_arena"), ctypes.c_size_t(arena.numel()), ctypes.c_void_p(stream_ptr))
    _check(code, "ssm_scan_fwd_bwd_host")
    return outputs


def make_conv_problem(x: torch.Tensor, w: torch.Tensor, silu: bool, has_bias: bool) -> ssm_conv_problem_t:
    batch, L, D = x.shape
    return ssm_conv_problem_t(batch, L, D, w.shape[1], _io_dtype(x),
                              (SSM_CONV_FLAG_SILU if silu else 0) | (SSM_CONV_FLAG_HAS_BIAS if has_bias else 0))


def ssm_conv1d_fwd(x, w, bias=None, *, silu=True, x_prev=None, out=None, stream=None):
    """y = silu(causal depthwise conv1d(x; w) + bias), see include/ssm_conv1d.h.  x (batch, L, D) io dtype; w (D, W)
    float32 with the last tap on the current step; bias (D) float32 or None; x_prev (batch, W-1, D) io dtype or None."""
    lib = load_library()
    prob = make_conv_problem(x, w, silu, bias is not None)
    batch, L, D, W = prob.batch, prob.L, prob.D, prob.width
    io = x.dtype
    if out is None:
        out = torch.empty_like(x)
    stream_ptr = (stream if stream is not None else torch.cuda.current_stream(x.device)).cuda_stream
    code = lib.ssm_conv1d_fwd(ctypes.byref(prob), _dev_ptr(x, "x", (batch, L, D), io),
                              _dev_ptr(w, "w", (D, W), torch.float32), _dev_ptr(bias, "bias", (D,), torch.float32),
                              _dev_ptr(x_prev, "x_prev", (batch, W - 1, D), io), _dev_ptr(out, "y", (batch, L, D), io),
                              ctypes.c_void_p(stream_ptr))
    _check(code, "ssm_conv1d_fwd")
    return out


def ssm_conv1d_bwd(x, w, bias, dy, *, silu=True, x_prev=None, want_dx_prev=False, outputs=None, stream=None):
    """Gradients of sum(dy * y) of ssm_conv1d_fwd: dict with dx (io dtype), dw (D, W) and dbias (D) float32 (dbias None
    without bias), and dx_prev (batch, W-1, D) if asked for."""
    lib = load_library()
    prob = make_conv_problem(x, w, silu, bias is not None)
    batch, L, D, W = prob.batch, prob.L, prob.D, prob.width
    io = x.dtype
    o = dict(outputs or {})
    o.setdefault("dx", torch.empty_like(x))
    o.setdefault("dw", torch.empty((D, W), dtype=torch.float32, device=x.device))
    if bias is not None:
        o.setdefault("dbias", torch.empty((D,), dtype=torch.float32, device=x.device))
    else:
        o["dbias"] = None
    if want_dx_prev and W > 1:
        o.setdefault("dx_prev", torch.empty((batch, W - 1, D), dtype=io, device=x.device))
    stream_ptr = (stream if stream is not None else torch.cuda.current_stream(x.device)).cuda_stream
    ws = _workspace(int(lib.ssm_conv1d_bwd_workspace_bytes(ctypes.byref(prob))), x.device, stream_ptr)
    code = lib.ssm_conv1d_bwd(ctypes.byref(prob), _dev_ptr(x, "x", (batch, L, D), io),
                              _dev_ptr(w, "w", (D, W), torch.float32), _dev_ptr(bias, "bias", (D,), torch.float32),
                              _dev_ptr(x_prev, "x_prev", (batch, W - 1, D), io), _dev_ptr(dy, "dy", (batch, L, D), io),
                              _dev_ptr(o["dx"], "dx", (batch, L, D), io), _dev_ptr(o["dw"], "dw", (D, W), torch.float32),
                              _dev_ptr(o["dbias"], "dbias", (D,), torch.float32),
                              _dev_ptr(o.get("dx_prev"), "dx_prev", (batch, W - 1, D), io),
                              _dev_ptr(ws, "workspace"), ctypes.c_size_t(0 if ws is None else ws.numel() * ws.element_size()),
                              ctypes.c_void_p(stream_ptr))
    _check(code, "ssm_conv1d_bwd")
    return o
