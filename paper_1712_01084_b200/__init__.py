"""Inference through fully-connected layers pruned by matrix pivoting (PBP form),
as hand-written sm_100a CUDA behind a small C library.

``synth`` draws seeded inputs; ``binding`` (imported on first attribute access)
marshals arguments into the C library ``libpp_b200.so``.  There is no CPU or
PyTorch fallback: without the compiled library every call raises.
"""
import importlib

__all__ = ["synth", "binding"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
