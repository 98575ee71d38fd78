"""ThinK hot path for B200: C-ABI library + thin Python binding.

``workloads`` (seeded synthetic inputs) imports on its own; the binding is
loaded on first use and raises if the compiled library is missing.
"""
import importlib

__all__ = ["workloads", "binding"]


def __getattr__(name):
    if name in ("binding", "workloads", "build", "replicas"):
        return importlib.import_module("." + name, __name__)
    raise AttributeError(name)
