"""W4A16 matrix multiplication for B200 (sm_100a): hand-written CUDA behind a C ABI.

``binding`` is the thin ctypes layer over ``libw4a16.so`` (argument marshalling
only); ``workloads`` draws the seeded synthetic inputs.  There is no CPU
fallback: using ``binding`` without the compiled library raises.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(__name__ + ".binding")
    raise AttributeError(name)
