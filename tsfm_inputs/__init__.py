"""Seeded synthetic inputs (weights and series) for the speculative patch decoder.

This package only *generates inputs*: model shapes, random weight tensors and
random time series.  It contains none of the method's arithmetic (no forward
pass, no acceptance rule, no uniform generator for the acceptance draws), so
both the CPU oracle and the CUDA library can be fed from it without sharing
any code of the method itself.
"""
from .configs import Arch, Workload, WORKLOADS, workload  # noqa: F401
from .weights import (  # noqa: F401
    make_model, layer_skip_draft, perturbed_draft, round_to_bf16, tensor_names,
    build_models,
)
from .series import make_series  # noqa: F401
