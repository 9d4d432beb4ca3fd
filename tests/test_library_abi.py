"""Host-only checks of the C-ABI library: it loads, exports every declared symbol, and validates arguments before
launching anything (no GPU needed: every call here returns before a CUDA call is made)."""
import ctypes
import os
import re

import pytest

from paper_2312_00752_b200 import binding as K

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    import glob
    text = "".join(open(h).read() for h in sorted(glob.glob(os.path.join(ROOT, "include", "*.h"))))
    return sorted(set(re.findall(r"SSM_API[^;(]*?\b(ssm_\w+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = K.load_library()
    names = _declared_symbols()
    assert set(names) == set(K.EXPORTED_SYMBOLS) and len(names) >= 8
    for n in names:
        assert getattr(lib, n) is not None


def _prob(batch=2, L=100, D=64, N=16, io=K.SSM_BF16, flags=3):
    return K.ssm_problem_t(batch, L, D, N, io, flags)


def test_queries_and_plan():
    ck = K.checkpoint_steps()
    assert ck in (8, 16, 32, 64)
    p = _prob(4, 2048, 5120)
    assert K.saved_state_bytes(p) == 4 * (2048 // ck) * 5120 * 16 * 4
    pl = K.plan(p)
    assert pl["n_segments"] == 1 and pl["segment_steps"] == 2048 and pl["states_per_thread"] in (4, 8, 16)
    # 640 groups of 32 channels for 592 resident warps: some groups are shared by two warps, which needs hand-off slots
    assert 0 < K.fwd_workspace_bytes(p) < 4 << 20
    assert K.fwd_workspace_bytes(_prob(64, 256, 64)) == 0 and K.fwd_workspace_bytes(_prob(2, 100, 64, io=K.SSM_F32)) == 0
    assert K.bwd_workspace_bytes(p) > 0
    long = _prob(1, 524288, 1536)
    pl = K.plan(long)
    assert pl["n_segments"] > 1 and pl["segment_steps"] % ck == 0
    assert pl["n_segments"] * pl["segment_steps"] >= 524288 > (pl["n_segments"] - 1) * pl["segment_steps"]
    assert K.fwd_workspace_bytes(long) >= 2 * pl["n_segments"] * 1536 * 16 * 4


@pytest.mark.parametrize("bad,code", [
    (dict(N=3), 2), (dict(N=128), 2), (dict(io=5), 2), (dict(L=0), 1), (dict(batch=-1), 1), (dict(flags=1 << 12), 1),
])
def test_invalid_problems_are_rejected(bad, code):
    lib = K.load_library()
    p = _prob(**bad)
    assert lib.ssm_scan_plan(ctypes.byref(p), None, None, None, None) == code
    assert K.fwd_workspace_bytes(p) == 0 and K.bwd_workspace_bytes(p) == 0
    one = ctypes.c_void_p(256)
    assert lib.ssm_scan_fwd(ctypes.byref(p), one, one, one, one, one, one, one, one, None, None, 0, None) == code


def test_complex_state_queries_and_refused_combinations():
    lib = K.load_library()
    real = _prob(2, 100, 64, N=8, io=K.SSM_F32, flags=3)
    cplx = _prob(2, 100, 64, N=8, io=K.SSM_F32, flags=3 | K.SSM_FLAG_COMPLEX)
    assert K.saved_state_bytes(cplx) == 2 * K.saved_state_bytes(real)        # (re, im) pairs
    assert K.fwd_workspace_bytes(cplx) == 0 and K.bwd_workspace_bytes(cplx) > 0
    assert K.plan(_prob(1, 524288, 64, N=8, flags=3 | K.SSM_FLAG_COMPLEX))["n_segments"] == 1   # no time split
    for extra in (K.SSM_FLAG_ZOH_BBAR, K.SSM_FLAG_STATIC_B, K.SSM_FLAG_STATIC_C, K.SSM_FLAG_DELTA_SOFTPLUS):
        bad = _prob(2, 100, 64, N=8, flags=3 | K.SSM_FLAG_COMPLEX | extra)
        assert lib.ssm_scan_plan(ctypes.byref(bad), None, None, None, None) == 2
    assert lib.ssm_scan_plan(ctypes.byref(_prob(2, 100, 64, N=64, flags=3 | K.SSM_FLAG_COMPLEX)), None, None, None, None) == 2


def test_null_misaligned_and_workspace_errors_before_launch():
    lib = K.load_library()
    p = _prob()
    a = ctypes.c_void_p(4096)
    args = [a] * 8
    assert lib.ssm_scan_fwd(ctypes.byref(p), None, *args[1:], None, None, 0, None) == 1          # x missing
    assert lib.ssm_scan_fwd(ctypes.byref(p), *args[:6], None, a, None, None, 0, None) == 1       # z flagged, missing
    assert lib.ssm_scan_fwd(ctypes.byref(p), ctypes.c_void_p(4097), *args[1:], None, None, 0, None) == 1  # misaligned
    ps = _prob(flags=7)
    assert lib.ssm_scan_fwd(ctypes.byref(ps), *args, None, None, 0, None) == 1                   # saved_states missing
    long = _prob(1, 524288, 1536)
    assert lib.ssm_scan_fwd(ctypes.byref(long), *args, None, None, 0, None) == 3                 # workspace missing
    assert lib.ssm_scan_fwd(ctypes.byref(long), *args, None, a, 16, None) == 3                   # workspace too small
    b16 = [a] * 16
    assert lib.ssm_scan_bwd(ctypes.byref(p), *b16, None, 0, None) == 3
    assert lib.ssm_scan_bwd(ctypes.byref(p), *b16[:7], None, *b16[8:], None, 0, None) == 1       # dout missing
    assert "WORKSPACE" in K.status_string(3) and K.status_string(0) == "SSM_OK"


def test_conv1d_argument_errors_before_launch():
    lib = K.load_library()
    a = ctypes.c_void_p(4096)
    ok = K.ssm_conv_problem_t(2, 100, 64, 4, K.SSM_BF16, 3)
    assert lib.ssm_conv1d_fwd(ctypes.byref(ok), None, a, a, None, a, None) == 1                  # x missing
    assert lib.ssm_conv1d_fwd(ctypes.byref(ok), a, a, None, None, a, None) == 1                  # bias flagged, missing
    for bad, code in [(dict(width=5), 2), (dict(width=0), 2), (dict(io=7), 2), (dict(L=0), 1), (dict(flags=8), 1)]:
        f = dict(batch=2, L=100, D=64, width=4, io=K.SSM_BF16, flags=3)
        f.update(bad)
        p = K.ssm_conv_problem_t(f["batch"], f["L"], f["D"], f["width"], f["io"], f["flags"])
        assert lib.ssm_conv1d_fwd(ctypes.byref(p), a, a, a, None, a, None) == code
        assert lib.ssm_conv1d_bwd_workspace_bytes(ctypes.byref(p)) == 0
    need = lib.ssm_conv1d_bwd_workspace_bytes(ctypes.byref(ok))
    assert need == 2 * 4 * 64 * 5 * 4                                                            # room for 4 chunks of 32 steps
    assert lib.ssm_conv1d_bwd(ctypes.byref(ok), a, a, a, None, a, a, a, a, None, None, 0, None) == 3
    assert lib.ssm_conv1d_bwd(ctypes.byref(ok), a, a, a, None, a, a, a, a, None, a, need - 1, None) == 3
