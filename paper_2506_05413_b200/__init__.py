"""SmoothRot W4A4 linear layer for NVIDIA B200: a C-ABI CUDA library
(libsmoothrot.so, see include/smoothrot.h) and this thin binding.

`synth` (seeded inputs) is importable without the library; the binding loads
the library on first use and fails loudly if it is absent.
"""
from . import synth  # noqa: F401


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
