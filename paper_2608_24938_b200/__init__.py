"""B200 (sm_100a) folded Mixture-of-Experts layer (ExFold hot path).

    paper_2608_24938_b200.build     builds libexfold.so in-tree with nvcc
    paper_2608_24938_b200.binding   ctypes binding of the C ABI declared in include/exfold.h

The binding is imported lazily so that the build module can be used before the
shared library exists; using the binding without the library raises ImportError
(there is no CPU or PyTorch fallback).
"""
import importlib

__all__ = ["binding", "build"]


def __getattr__(name):
    if name in ("binding", "build"):
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
