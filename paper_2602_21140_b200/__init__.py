"""Failure-aware MoE token routing with dispatch (A2E) and combine (E2A) for B200.

``workloads`` draws the seeded synthetic inputs and imports nothing else.  The
CUDA library binding is loaded on first use of any ``moe_*`` name, and raises
if the compiled library is missing: there is no CPU fallback.
"""
from . import workloads  # noqa: F401

_BINDING_NAMES = None


def __getattr__(name):
    if name.startswith("_"):
        raise AttributeError(name)
    from . import binding
    if hasattr(binding, name):
        return getattr(binding, name)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
