"""B200-native N:M sparse linear layers for vision transformers (ELSA, arXiv 2409.09708).

``synth`` holds seeded inputs and workload tables; ``binding`` is the thin
ctypes layer over the C-ABI CUDA library ``libelsa.so`` (it raises at import if
the library has not been built: there is no CPU fallback).
"""
from . import synth  # noqa: F401


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
