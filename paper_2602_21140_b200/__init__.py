"""Failure-aware MoE token routing with dispatch (A2E) and combine (E2A) for B200.

``workloads`` draws the seeded synthetic inputs and imports nothing else.  The
CUDA library binding (``binding``) is loaded on first use of any ``moe_*`` /
``MoeRouter`` name and raises if the compiled library is missing: there is no
CPU fallback.
"""
import importlib

from . import workloads  # noqa: F401

_SUBMODULES = ("binding", "build", "workloads")


def __getattr__(name):
    if name.startswith("_"):
        raise AttributeError(name)
    if name in _SUBMODULES:
        return importlib.import_module(f"{__name__}.{name}")
    binding = importlib.import_module(f"{__name__}.binding")
    if hasattr(binding, name):
        return getattr(binding, name)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
