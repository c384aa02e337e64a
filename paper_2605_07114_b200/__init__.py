"""HORA rollout-allocation hot path for B200: Python binding over the C-ABI CUDA library.

``hora`` (the binding) marshals torch tensors into the four C calls declared in ``include/hora.h``;
every step of the path runs in the library's kernels.  ``workloads`` draws seeded synthetic inputs.
Importing this package does not load the shared library; the first call does, and fails loudly if
``libhora.so`` has not been built (see ``build.py``).
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "hora"]


def __getattr__(name):
    if name == "hora":
        import importlib
        return importlib.import_module(".hora", __name__)
    raise AttributeError(name)
