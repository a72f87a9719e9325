"""ReHyAt recurrent hybrid attention operator for B200 (sm_100a).

The operator itself lives in a C-ABI shared library (csrc/, declared in include/rehyat.h);
`binding` is a thin ctypes layer over it.  Importing this package does not load the library;
the first use of `binding` does, and fails loudly if it has not been built.
"""
from . import geometry, synth  # noqa: F401

__all__ = ["geometry", "synth", "binding", "build"]


def __getattr__(name):
    if name in ("binding", "build"):
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
