"""AsyncLM serving-step attention for B200: mixed decode + interrupt-append over a paged KV cache.

The product is the C ABI library (include/asynclm.h); `binding` marshals arguments to it and
`workload` draws seeded synthetic steps.  Importing the package loads nothing; the first call into
`binding` loads (and if needed builds) the CUDA library and raises if that is impossible.
"""
from . import workload  # noqa: F401

__all__ = ["workload", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
