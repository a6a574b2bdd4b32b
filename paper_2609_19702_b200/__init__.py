"""Diagonal-aware sparse decode attention for B200 (sm_100a).

The package holds the CUDA kernels with their C-ABI library (``csrc/``), a thin ctypes binding
with the same entry-point names (``binding``), and seeded synthetic workloads (``synth``).
``binding`` is imported on first use so that host-only tools can import ``synth`` without the
compiled library; any compute call without the library raises.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(__name__ + ".binding")
    raise AttributeError(name)
