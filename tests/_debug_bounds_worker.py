"""Runs small tuned-path problems through whatever library SSM_SCAN_LIBRARY names (the bounds-checking build), compares
with the oracle and asserts that no index check fired.  Executed as a child process by test_gpu_debug_bounds.py, because a
process loads only one build of the library."""
import sys

import numpy as np


def main() -> int:
    import torch
    from paper_2312_00752_b200 import binding as K, synth
    from tests import _gpu_util as U

    shapes = [  # (batch, L, D): ragged tiles, partial channel groups, one step, time splits in both directions
        (2, 300, 192), (1, 1, 64), (3, 33, 72), (1, 31, 8), (2, 257, 40), (1, 4096, 64), (2, 1000, 1600), (5, 515, 104),
    ]
    for i, (batch, L, D) in enumerate(shapes):
        cfg = synth.CONFIGS[1].scaled(batch=batch, L=L, D=D)
        inp = synth.make_inputs(cfg, seed=20 + i, perturb_A=0.05 if i % 2 else 0.0)
        dev = U.to_device(inp, "bf16")
        args = (dev["x"], dev["delta"], dev["A"], dev["B"], dev["C"], dev["D_skip"], dev["z"])
        prob = K.make_problem(dev["x"], dev["B"], True, True, save_states=True)
        out, saved = K.ssm_scan_fwd(*args, save_states=True)
        ws = K.last_bwd_workspace(dev["x"].device)
        if ws is not None and K.fwd_workspace_bytes(prob) > 0:
            K.check_status(prob, ws)                      # raises SsmScanError on SSM_ERR_BOUNDS / SSM_ERR_TIMEOUT
        g = K.ssm_scan_bwd(*args, dev["dout"], saved)
        K.check_status(prob, K.last_bwd_workspace(dev["x"].device))
        got = {"out": U.to_host(out), **{k: U.to_host(v) for k, v in g.items() if v is not None}}
        U.assert_parity(got, U.oracle_fwd_bwd(inp), "bf16", f"bounds-checking build, shape {batch, L, D}")
        # the fused step size and a carried state take other template instances of the same kernels
        bias = torch.from_numpy(np.linspace(-3.0, -1.0, D, dtype=np.float32)).to(dev["x"].device)
        K.ssm_scan_fwd_fused_dt(dev["x"], dev["delta"], bias, dev["A"], dev["B"], dev["C"], dev["D_skip"], dev["z"])
        torch.cuda.synchronize()
    print("bounds-checking build: no index left its range on", len(shapes), "shapes")
    return 0


if __name__ == "__main__":
    sys.exit(main())
