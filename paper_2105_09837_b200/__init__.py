"""pdADMM-G / pdADMM-G-Q on B200: one ADMM iteration over every layer of a GA-MLP.

The package holds the CUDA sources (``csrc/``), the build step (``build``),
the ctypes binding of the C-ABI library (``binding``) and the seeded synthetic
input generators (``synth``).  Sub-modules are imported on demand so that
``synth`` (no CUDA, no arithmetic of the method) can be used on its own.
"""

import importlib

__all__ = ["synth", "binding", "build", "replicas"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
