"""Fused tile-partitioned CNN training step for B200 (sm_100a).

`synth` describes the seeded synthetic workloads; every other name is loaded on
first use from the Python binding of the C-ABI library (`libftp.so`), which
must have been built: nothing here computes on the CPU.
"""
from . import synth  # noqa: F401

_BINDING_NAMES = None


def __getattr__(name):
    import importlib
    if name in ("build", "binding", "dp"):          # plain submodules: no library needed to import `build`
        return importlib.import_module("." + name, __name__)
    binding = importlib.import_module(".binding", __name__)
    if hasattr(binding, name):
        return getattr(binding, name)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
