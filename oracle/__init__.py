"""CPU oracle (test infrastructure only; see ``moe_oracle.c``).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It has no dependency on, and is never imported by, the CUDA
library or its Python binding.
"""
from .ep_reference import ep_combine, ep_dispatch  # noqa: F401
from .reference import (  # noqa: F401
    OracleConfig,
    build,
    combine,
    compact_ranks,
    dispatch,
    double_to_bf16,
    exp_spec,
    failure_set_ok,
    permutation,
    route,
    scatter,
    sigmoid_spec,
)
