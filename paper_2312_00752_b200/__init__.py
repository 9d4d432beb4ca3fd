"""B200 (sm_100a) selective scan (S6): C-ABI CUDA library plus a thin ctypes binding.

`ssm_scan_fwd` / `ssm_scan_bwd` are resolved lazily so that importing the package (for example to reach the
seeded input generator in `synth`) does not need torch or the compiled library.
"""

__all__ = ["ssm_scan_fwd", "ssm_scan_bwd", "ssm_scan_fwd_static", "ssm_step", "binding", "synth", "build"]


def __getattr__(name):
    if name in ("ssm_scan_fwd", "ssm_scan_bwd", "ssm_scan_fwd_static", "ssm_step"):
        from . import binding
        return getattr(binding, name)
    if name in ("binding", "synth", "build"):
        import importlib
        return importlib.import_module(f".{name}", __name__)
    raise AttributeError(name)
