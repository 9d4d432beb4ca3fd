"""The forward entry point that needs no scratch memory from the caller (ssm_scan_fwd_static).

It serves callers that cannot allocate device memory where they call the scan (a plug-in that is handed only input and
output buffers and must not allocate while enqueueing, an application with a memory budget fixed at start-up), so its
scratch is a fixed array inside the library.  The checks here: through the C ABI it returns what ssm_scan_fwd returns
for the same inputs, on two calls in a row that share the array (the second with different inputs and a different
shape, so stale contents of the first would show), and it refuses a problem whose scratch would not fit.

Collected last on purpose: a run that stops at the first failure has then already run every other test.
"""
import ctypes

import numpy as np
import pytest

from paper_2312_00752_b200 import synth
from tests import _gpu_util as U

pytestmark = pytest.mark.gpu


def _inputs(batch, L, D, io, seed):
    cfg = synth.ScanConfig("static", 11, batch, L, D, 16, io, 1e-4, 1e-2)
    return U.to_device(synth.make_inputs(cfg, seed=seed, with_dout=False), io)


def test_static_scratch_matches_workspace_entry_point_twice():
    import torch
    from paper_2312_00752_b200 import binding as K
    calls = [(1, 8192, 64, "bf16", 0), (2, 5000, 40, "f32", 1)]      # both split the sequence in time
    for batch, L, D, io, seed in calls:
        dev = _inputs(batch, L, D, io, seed)
        prob = K.make_problem(dev["x"], dev["B"], True, True)
        assert K.plan(prob)["n_segments"] > 1, "the case must use the scratch memory"
        assert 0 < K.fwd_workspace_bytes(prob) <= K.SSM_STATIC_SCRATCH_BYTES
        args = (dev["x"], dev["delta"], dev["A"], dev["B"], dev["C"], dev["D_skip"], dev["z"])
        ref, ref_saved = K.ssm_scan_fwd(*args, save_states=True)
        out = torch.full_like(dev["x"], float("nan"))
        saved = torch.full_like(ref_saved, float("nan"))
        got, got_saved = K.ssm_scan_fwd_static(*args, save_states=True, out=out, saved_states=saved)
        torch.cuda.synchronize()
        # same kernels, same inputs, same order of operations: the tolerance of the parity tests is met with zero error
        assert U.rel_err(U.to_host(got), U.to_host(ref)) <= U.TOL[io]["out"]
        assert torch.equal(got, ref) and torch.equal(got_saved, ref_saved)


def test_static_scratch_refuses_what_does_not_fit():
    from paper_2312_00752_b200 import binding as K
    lib = K.load_library()
    big = K.ssm_problem_t(1, 524288, 1536, 16, K.SSM_BF16, 3)
    assert K.fwd_workspace_bytes(big) > K.SSM_STATIC_SCRATCH_BYTES
    a = ctypes.c_void_p(4096)
    code = lib.ssm_scan_fwd_static(ctypes.byref(big), a, a, a, a, a, a, a, a, None, None)
    assert code == 3 and "WORKSPACE" in K.status_string(code)
