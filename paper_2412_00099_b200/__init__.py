"""Cache-conditional MoE decode step for many independent token streams on B200 (sm_100a).

`synth` holds the seeded workload generators; `binding` is the thin ctypes layer over the C-ABI
library `libmcce.so` (built from `csrc/`), which does all of the work on the GPU.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
