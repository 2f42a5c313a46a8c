"""Seeded synthetic workloads for the H-Spec draft step.

This package holds the workload shapes and the seeded random generators that
feed BOTH the CPU oracle and the CUDA library.  It contains none of the
method's arithmetic: only shapes, random draws and the page-table layout.
"""
from .configs import CONFIGS, get_config, derived, sweep_config  # noqa: F401
from .generate import (  # noqa: F401
    BASE_SEED, make_weights, make_ctx_lens, make_request_batch, tensor_seed,
    weight_shapes,
)
