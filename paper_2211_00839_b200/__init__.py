"""Resource-constrained submodular data partition (RCD-SGD, Algorithm 1) on B200.

The compute lives in the C-ABI CUDA library under ``csrc/`` (see ``include/rcd.h``);
``binding`` marshals arguments to it.  ``workloads`` draws seeded synthetic inputs.
The binding is loaded on first use and raises if the compiled library is missing:
there is no CPU fallback.
"""

__all__ = ["workloads", "binding"]


def __getattr__(name):
    if name in ("binding", "workloads", "distributed"):
        import importlib
        return importlib.import_module("." + name, __name__)
    raise AttributeError(name)
